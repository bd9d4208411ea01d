"""Unit parity of the dense kernels (linear layers, attention) against the oracle's definitions."""
import numpy as np
import pytest

from oracle import bsr_oracle as O
from paper_2405_10951_b200 import synth

pytestmark = pytest.mark.gpu


def rel(a, b):
    return float(np.linalg.norm(a - b) / np.linalg.norm(b))


def linear_case(m, n, k, dtype, gelu, use_tc, with_res=True):
    import torch
    from paper_2405_10951_b200 import binding as Bd
    rng = np.random.default_rng(m + 3 * n + 7 * k)
    x, w = rng.standard_normal((m, k)), rng.standard_normal((n, k)) / np.sqrt(k)
    bias, res = rng.standard_normal(n), rng.standard_normal((m, n))
    if dtype == "bf16":
        x, w, res = synth.round_to_bf16(x), synth.round_to_bf16(w), synth.round_to_bf16(res)
    y = O.linear(x, w, bias)
    if gelu:
        y = O.gelu(y)
    if with_res:
        y = y + res
    tdt = torch.float32 if dtype == "fp32" else torch.bfloat16
    g = lambda a: torch.as_tensor(a.astype(np.float32)).cuda().to(tdt)
    out = Bd.bsr_linear_forward(g(x), g(w), torch.as_tensor(bias.astype(np.float32)).cuda(), g(res) if with_res else None,
                                act_gelu=gelu, use_tensor_cores=use_tc)
    torch.cuda.synchronize()
    return rel(out.float().cpu().numpy().astype(np.float64), y)


@pytest.mark.parametrize("m,n,k", [(65, 192, 192), (130, 100, 72), (520, 768, 192), (8, 10, 192), (333, 72, 40)])
@pytest.mark.parametrize("gelu", [False, True])
def test_linear_fp32(m, n, k, gelu):
    assert linear_case(m, n, k, "fp32", gelu, False) < 2e-6


@pytest.mark.parametrize("m,n,k", [(65, 192, 192), (520, 768, 192), (197, 384, 1536)])
def test_linear_bf16_simt(m, n, k):
    assert linear_case(m, n, k, "bf16", True, False) < 4e-3


@pytest.mark.parametrize("dtype,tol,tc", [("fp32", 2e-6, False), ("bf16", 4e-3, False), ("bf16", 6e-3, True)])
@pytest.mark.parametrize("B,T,H,d", [(2, 65, 3, 64), (3, 47, 2, 32), (2, 197, 6, 64), (1, 5, 1, 16), (1, 290, 2, 64),
                                     (3, 140, 12, 64), (2, 100, 2, 64), (5, 72, 3, 64), (1, 256, 1, 64), (2, 129, 2, 64),
                                     (1, 16, 1, 64), (4, 1, 2, 64), (2, 577, 3, 64), (1, 257, 2, 64), (1, 512, 1, 64),
                                     # more (image, head) pairs than SMs: every persistent CTA walks several tiles
                                     (40, 197, 12, 64), (31, 140, 12, 64), (64, 100, 12, 64), (50, 72, 7, 64), (13, 256, 12, 64)])
def test_attention_forward(dtype, tol, tc, B, T, H, d):
    import torch
    from paper_2405_10951_b200 import binding as Bd
    if dtype == "fp32" and T > 200:
        pytest.skip("fp32 rows of this length exceed the kernel's shared memory by design")
    if tc and d != 64:
        pytest.skip("the tcgen05 attention kernels take head dimension 64")
    rng = np.random.default_rng(T * 31 + d)
    qkv = rng.standard_normal((B, T, 3, H, d))
    if dtype == "bf16":
        qkv = synth.round_to_bf16(qkv)
    q, k, v = (qkv[:, :, i].transpose(0, 2, 1, 3) for i in range(3))

    class Cfg:
        heads = H
        dim = H * d
    o, A = O.attention_fwd(Cfg, q, k, v)
    want = O.merge_heads(o)
    tdt = torch.float32 if dtype == "fp32" else torch.bfloat16
    out, cp = Bd.bsr_attention_forward(torch.as_tensor(qkv.astype(np.float32)).cuda().to(tdt), H, use_tensor_cores=tc)
    torch.cuda.synchronize()
    assert rel(out.float().cpu().numpy().astype(np.float64), want) < tol
    if T > 1:
        assert rel(cp.cpu().numpy().astype(np.float64), A[:, :, 0, 1:]) < (2e-6 if dtype == "fp32" else 2e-5)


@pytest.mark.parametrize("B,T,H", [(2, 577, 3), (1, 290, 2), (1, 512, 1), (3, 1000, 2)])
@pytest.mark.parametrize("pattern", ["rising", "steps", "falling"])
def test_long_attention_when_the_row_maximum_jumps_between_key_blocks(B, T, H, pattern):
    """The kernel for more than 256 tokens walks the keys once and rescales its accumulator when a block's row maximum
    exceeds the reference by more than eight binary orders.  Standard normal inputs never do that after the first
    block, so here the key rows grow (or shrink) from one 64-key block to the next: 'rising' makes every block jump,
    'steps' makes some rows jump late and leaves others alone, 'falling' must never rescale."""
    import torch
    from paper_2405_10951_b200 import binding as Bd
    d = 64
    rng = np.random.default_rng(T + len(pattern))
    qkv = rng.standard_normal((B, T, 3, H, d))
    blk = np.arange(T) // 64
    if pattern == "rising":
        f = 1.0 + 1.5 * blk
    elif pattern == "falling":
        f = 1.0 + 1.5 * (blk.max() - blk)
    else:
        f = np.where(blk % 3 == 2, 6.0, 1.0)
    qkv[:, :, 1] *= f[None, :, None, None]
    if pattern == "steps":                                     # half of the queries barely see the large keys
        qkv[:, ::2, 0] *= 0.05
    qkv = synth.round_to_bf16(qkv)
    q, k, v = (qkv[:, :, i].transpose(0, 2, 1, 3) for i in range(3))

    class Cfg:
        heads = H
        dim = H * d
    o, A = O.attention_fwd(Cfg, q, k, v)
    out, cp = Bd.bsr_attention_forward(torch.as_tensor(qkv.astype(np.float32)).cuda().bfloat16(), H, use_tensor_cores=True)
    torch.cuda.synchronize()
    assert rel(out.float().cpu().numpy().astype(np.float64), O.merge_heads(o)) < 6e-3
    assert rel(cp.cpu().numpy().astype(np.float64), A[:, :, 0, 1:]) < 2e-5


@pytest.mark.parametrize("tc", [False, True])
@pytest.mark.parametrize("with_score_grad", [False, True])
@pytest.mark.parametrize("B,T,H", [(2, 100, 3), (1, 128, 2), (2, 129, 2), (3, 140, 4), (2, 197, 6), (1, 256, 2), (2, 145, 1),
                                   (30, 197, 12), (1, 17, 1)])
def test_attention_backward(B, T, H, with_score_grad, tc):
    """dQ, dK, dV of Eq. 1 from the gradient at the attention output, on identical bf16 inputs, against the oracle;
    with and without a gradient that reaches the classification row through the scores of Eq. 6.  T <= 128 takes the
    one-tile tcgen05 kernel, 128 < T <= 256 the two-tile one; tc = False the kernels without tensor cores."""
    import torch
    from paper_2405_10951_b200 import binding as Bd
    d = 64
    rng = np.random.default_rng(T * 7 + B)
    qkv = synth.round_to_bf16(rng.standard_normal((B, T, 3, H, d)))
    do = synth.round_to_bf16(rng.standard_normal((B, T, H * d)))
    sg = rng.standard_normal((B, T - 1)) * 3.0 if with_score_grad else None
    q, k, v = (qkv[:, :, i].transpose(0, 2, 1, 3) for i in range(3))

    class Cfg:
        heads = H
        dim = H * d
    _, A = O.attention_fwd(Cfg, q, k, v)
    dA_cls = None
    if sg is not None:
        dA_cls = np.zeros((B, T))
        dA_cls[:, 1:] = sg / H
    dq, dk, dv = O.attention_bwd(Cfg, A, q, k, v, do.reshape(B, T, H, d).transpose(0, 2, 1, 3), dA_cls)
    want = np.stack([dq, dk, dv], axis=0).transpose(1, 3, 0, 2, 4)            # [B, T, 3, H, d]
    dev = torch.as_tensor(qkv.astype(np.float32)).cuda().bfloat16()
    _, _, lse = Bd.bsr_attention_forward(dev, H, use_tensor_cores=True, want_lse=True)
    got = Bd.bsr_attention_backward(dev, torch.as_tensor(do.astype(np.float32)).cuda().bfloat16(), lse,
                                    None if sg is None else torch.as_tensor(sg.astype(np.float32)).cuda(), use_tensor_cores=tc)
    torch.cuda.synchronize()
    got = got.float().cpu().numpy().astype(np.float64)
    for i, name in enumerate(("dq", "dk", "dv")):
        assert rel(got[:, :, i], want[:, :, i]) < 8e-3, name


TC_SHAPES = [(128, 256, 64), (197, 384, 192), (1000, 3072, 768), (2600, 768, 3072), (100, 72, 40), (9216, 2304, 768)]


@pytest.mark.parametrize("m,n,k", TC_SHAPES)
@pytest.mark.parametrize("gelu", [False, True])
def test_linear_bf16_tensor_cores(m, n, k, gelu):
    """tcgen05 kernel, operands contiguous along k; tiles spanning several CTAs and ragged edges in m, n and k."""
    assert linear_case(m, n, k, "bf16", gelu, True) < 4e-3
    assert linear_case(m, n, k, "bf16", gelu, True, with_res=False) < 4e-3


@pytest.mark.parametrize("m,n,k,ws", [(128, 256, 64, False), (200, 384, 192, False), (1024, 768, 384, True),
                                      (12800, 768, 768, True), (9216, 3072, 768, True), (72, 40, 104, False)])
@pytest.mark.parametrize("tc", [False, True])
def test_linear_backward_bf16(m, n, k, ws, tc):
    """Input and weight gradients of a linear layer (Eq. 2 and Eq. 4), operands read in place (no transposes)."""
    import torch
    from paper_2405_10951_b200 import binding as Bd
    rng = np.random.default_rng(m + n + k)
    x = synth.round_to_bf16(rng.standard_normal((m, k)))
    w = synth.round_to_bf16(rng.standard_normal((n, k)) / np.sqrt(k))
    dy = synth.round_to_bf16(rng.standard_normal((m, n)))
    dx_ref, dw_ref, _ = O.linear_bwd(dy, x, w)
    g = lambda a: torch.as_tensor(a.astype(np.float32)).cuda().to(torch.bfloat16)
    wsb = torch.empty(160 * 128 * 256, dtype=torch.float32, device="cuda") if ws else None
    dx, dw = Bd.bsr_linear_backward(g(x), g(w), g(dy), use_tensor_cores=tc, workspace=wsb)
    torch.cuda.synchronize()
    assert rel(dx.float().cpu().numpy().astype(np.float64), dx_ref) < 4e-3
    assert rel(dw.cpu().numpy().astype(np.float64), dw_ref) < 1e-4


def test_linear_backward_fp32():
    import torch
    from paper_2405_10951_b200 import binding as Bd
    rng = np.random.default_rng(3)
    m, n, k = 130, 72, 100
    x, w, dy = rng.standard_normal((m, k)), rng.standard_normal((n, k)), rng.standard_normal((m, n))
    dx_ref, dw_ref, _ = O.linear_bwd(dy, x, w)
    g = lambda a: torch.as_tensor(a.astype(np.float32)).cuda()
    dx, dw = Bd.bsr_linear_backward(g(x), g(w), g(dy))
    torch.cuda.synchronize()
    assert rel(dx.cpu().numpy().astype(np.float64), dx_ref) < 2e-6
    assert rel(dw.cpu().numpy().astype(np.float64), dw_ref) < 2e-6


@pytest.mark.parametrize("m,n,k", [(128, 256, 128), (197, 384, 192), (1000, 3072, 768), (2600, 2304, 768), (100, 72, 48), (9216, 3072, 768)])
@pytest.mark.parametrize("gelu", [False, True])
def test_linear_e4m3_tensor_cores(m, n, k, gelu):
    """tcgen05 kind::f8f6f4 on row-quantised E4M3 operands against the oracle's statement of the same product: the
    inputs are bf16 on both sides, so the 8-bit codes agree exactly and what is left is fp32 accumulation order and the
    bf16 rounding of the output."""
    import torch
    from paper_2405_10951_b200 import binding as Bd
    rng = np.random.default_rng(m + 3 * n + 7 * k)
    x = synth.round_to_bf16(rng.standard_normal((m, k)) * np.exp(rng.standard_normal((m, 1))))      # rows of different scale
    w = synth.round_to_bf16(rng.standard_normal((n, k)) / np.sqrt(k))
    bias = rng.standard_normal(n)
    want = O.linear_e4m3(x, w, bias)
    if gelu:
        want = O.gelu(want)
    g = lambda a: torch.as_tensor(a.astype(np.float32)).cuda().to(torch.bfloat16)
    y = Bd.bsr_linear_forward_e4m3(g(x), g(w), torch.as_tensor(bias.astype(np.float32)).cuda(), act_gelu=gelu)
    torch.cuda.synchronize()
    got = y.float().cpu().numpy().astype(np.float64)
    assert rel(got, want) < 4e-3
    # and it is the quantised product, not the bf16 one: the two differ by a few percent
    plain = O.linear(x, w, bias)
    if gelu:
        plain = O.gelu(plain)
    assert rel(got, plain) > 5 * rel(got, want)
