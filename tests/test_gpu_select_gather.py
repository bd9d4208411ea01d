"""A4/A5: token selection is bit-exact against the oracle (same float32 head mean on both sides);
the compaction matches it to rounding."""
import numpy as np
import pytest

from oracle import bsr_oracle as O
from paper_2405_10951_b200 import synth

pytestmark = pytest.mark.gpu

SHAPES = [(8, 3, 64, 45), (128, 12, 196, 138), (32, 12, 576, 288), (5, 6, 99, 70), (3, 2, 33, 33), (4, 1, 1, 1),
          (2, 3, 4096, 1000), (7, 12, 139, 98), (1, 1, 50, 1)]


@pytest.mark.parametrize("ties", [False, True])
@pytest.mark.parametrize("B,H,M,k", SHAPES)
def test_select_bit_exact(B, H, M, k, ties):
    import torch
    from paper_2405_10951_b200 import binding as Bd
    rng = np.random.default_rng(B * 1000 + M)
    p = synth.make_scores(rng, B, H, M, ties=ties)
    s_gpu, kept, dropped = Bd.bsr_token_select(torch.as_tensor(p).cuda(), k)
    torch.cuda.synchronize()
    s_ref = O.head_mean_scores(p, np.float32)
    assert np.array_equal(s_gpu.cpu().numpy(), s_ref)          # same precision, same order: identical bits
    kept, dropped = kept.cpu().numpy(), dropped.cpu().numpy()
    for b in range(B):
        kr, dr = O.select_tokens(s_ref[b], k)
        assert np.array_equal(kept[b], kr), (b,)
        assert np.array_equal(dropped[b], dr), (b,)


@pytest.mark.parametrize("dtype", ["fp32", "bf16"])
@pytest.mark.parametrize("B,M,D,k,fuse", [(8, 64, 192, 45, 1), (16, 196, 768, 138, 1), (3, 139, 384, 98, 0), (2, 9, 8, 9, 1),
                                           (4, 576, 768, 288, 1), (5, 33, 64, 1, 1),
                                           # weighted mean of the dropped tokens (fuse mode 2)
                                           (8, 64, 192, 45, 2), (16, 196, 768, 138, 2), (3, 33, 64, 32, 2)])
def test_gather_fuse_matches_oracle(dtype, B, M, D, k, fuse):
    import torch
    from paper_2405_10951_b200 import binding as Bd
    if dtype == "fp32" and D % 4:
        pytest.skip("row not a multiple of 16 bytes")
    rng = np.random.default_rng(M * 7 + D)
    x = rng.standard_normal((B, M + 1, D))
    x = synth.round_to_bf16(x) if dtype == "bf16" else x.astype(np.float32).astype(np.float64)
    p = synth.make_scores(rng, B, 2, M)
    s = O.head_mean_scores(p, np.float32)
    kept = np.stack([O.select_tokens(s[b], k)[0] for b in range(B)])
    dropped = np.stack([O.select_tokens(s[b], k)[1] for b in range(B)]).reshape(B, M - k)
    want = O.gather_fuse(x, kept, dropped, s.astype(np.float64), fuse)
    tdt = torch.float32 if dtype == "fp32" else torch.bfloat16
    xg = torch.as_tensor(x.astype(np.float32)).cuda().to(tdt)
    out = Bd.bsr_gather_fuse(xg, torch.as_tensor(kept.astype(np.int32)).cuda(), torch.as_tensor(dropped.astype(np.int32)).cuda(),
                             torch.as_tensor(s).cuda(), fuse)
    torch.cuda.synchronize()
    got = out.float().cpu().numpy().astype(np.float64)
    assert got.shape == want.shape
    assert np.array_equal(got[:, : 1 + k], want[:, : 1 + k])    # copied rows are bit-exact
    if fuse and k < M:
        tol = 2e-6 if dtype == "fp32" else 2.0 ** -8
        err = np.linalg.norm(got[:, -1] - want[:, -1]) / np.linalg.norm(want[:, -1])
        assert err < tol, err


def test_select_gather_at_benchmark_size_sampled():
    """ViT-B block 3 at batch 128 (the launch shape the benchmark times): a sample of images checked one by one."""
    import torch
    from paper_2405_10951_b200 import binding as Bd
    B, H, M, D, k = 128, 12, 196, 768, 138
    rng = np.random.default_rng(42)
    p = synth.make_scores(rng, B, H, M)
    x = synth.round_to_bf16(rng.standard_normal((B, M + 1, D)))
    pg = torch.as_tensor(p).cuda()
    xg = torch.as_tensor(x.astype(np.float32)).cuda().to(torch.bfloat16)
    s, kept, dropped = Bd.bsr_token_select(pg, k)
    out = Bd.bsr_gather_fuse(xg, kept, dropped, s, 1)
    torch.cuda.synchronize()
    s_ref = O.head_mean_scores(p, np.float32)
    got = out.float().cpu().numpy().astype(np.float64)
    for b in (0, 17, 63, 64, 127):
        kr, dr = O.select_tokens(s_ref[b], k)
        assert np.array_equal(kept[b].cpu().numpy(), kr)
        want = O.gather_fuse(x[b:b + 1], kr[None], dr[None], s_ref[b:b + 1].astype(np.float64))
        assert np.array_equal(got[b, : 1 + k], want[0, : 1 + k])
        assert np.linalg.norm(got[b, -1] - want[0, -1]) / np.linalg.norm(want[0, -1]) < 2.0 ** -8
