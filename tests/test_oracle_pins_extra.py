"""Pins of the oracle parts that the comparison rules themselves lean on: the boundary margin (it decides where kept
sets must be identical), the forced-expert branch of the MoE layer (Section 5.2; it is what a GPU run with a
different choice between near-equal gate logits is compared against) and the MoE term of the MAC counter."""
import math

import numpy as np

from oracle import bsr_oracle as O
from oracle import counters as C
from paper_2405_10951_b200 import synth

MOE = synth.Config("pin_moe", 16, 4, 32, 2, 2, 48, (5, 3), 4, (0, 1), (), 1, 1, dtype="fp32", seed=11,
                   moe_experts=4, moe_top_k=2, moe_blocks=(1,))


def test_boundary_margin_hand_computed_cases():
    # (s_(K) - s_(K+1)) / s_(K): the gap below the weakest kept score, relative to that score (not to the largest
    # score, not to the strongest dropped one)
    s = np.array([0.10, 0.40, 0.25, 0.05, 0.20])
    kept, dropped = O.select_tokens(s, 3)                       # keeps 0.40, 0.25, 0.20; drops 0.10, 0.05
    assert list(kept) == [1, 2, 4] and list(dropped) == [0, 3]
    assert abs(O.boundary_margin(s, kept, dropped) - (0.20 - 0.10) / 0.20) < 1e-15
    kept, dropped = O.select_tokens(s, 1)                       # keeps 0.40; strongest dropped 0.25
    assert abs(O.boundary_margin(s, kept, dropped) - (0.40 - 0.25) / 0.40) < 1e-15
    t = np.array([0.3, 0.2, 0.2, 0.1])
    kept, dropped = O.select_tokens(t, 2)                       # a tie across the boundary: margin exactly zero
    assert list(kept) == [0, 1] and O.boundary_margin(t, kept, dropped) == 0.0
    kept, dropped = O.select_tokens(t, 4)                       # nothing dropped: no boundary
    assert O.boundary_margin(t, kept, dropped) == np.inf
    # normalising by the largest score or by the dropped score would give other numbers on the first case
    assert abs((0.20 - 0.10) / 0.40 - 0.5) > 0.1 and abs((0.20 - 0.10) / 0.10 - 0.5) > 0.1


def _moe_inputs():
    rng = np.random.default_rng(5)
    images, labels, task_ids, params = synth.make_workload(MOE)
    for n in params:                                              # larger weights: well separated gate logits
        if ".moe." in n and n.endswith("weight"):
            params[n] = rng.standard_normal(params[n].shape) * 0.3
    y = rng.standard_normal((MOE.batch, 6, MOE.dim))
    return params, y, task_ids


def test_forcing_the_routers_own_choice_changes_nothing():
    params, y, task_ids = _moe_inputs()
    free, c0 = O.moe_fwd(MOE, params, 1, y, task_ids)
    forced, c1 = O.moe_fwd(MOE, params, 1, y, task_ids, forced_experts=c0["experts"])
    assert np.array_equal(free, forced)                           # bit for bit
    assert np.array_equal(c0["w"], c1["w"])
    partial = np.full_like(c0["experts"], -1)                     # -1 leaves the choice to the router
    partial[:, ::2] = c0["experts"][:, ::2]
    assert np.array_equal(O.moe_fwd(MOE, params, 1, y, task_ids, forced_experts=partial)[0], free)


def test_forced_experts_equal_a_hand_built_two_expert_sum():
    """Forcing experts (a, b) for every token: out = w_a MLP_a(y) + w_b MLP_b(y) with (w_a, w_b) the softmax over the
    two gate logits of those experts -- written out here with plain matrix products."""
    params, y, task_ids = _moe_inputs()
    p = "blocks.1.moe."
    B, T, D = y.shape
    for a, b in ((3, 0), (1, 2)):
        forced = np.empty((B, T, 2), dtype=np.int64)
        forced[..., 0], forced[..., 1] = a, b
        got, cache = O.moe_fwd(MOE, params, 1, y, task_ids, forced_experts=forced)
        want = np.zeros_like(y)
        for i in range(B):
            wg = params[p + "gate.weight"][task_ids[i]]
            gl = y[i] @ wg.T                                      # [T, E]
            za, zb = gl[:, a], gl[:, b]
            wa = 1.0 / (1.0 + np.exp(zb - za))                    # two-way softmax
            for e, w in ((a, wa), (b, 1.0 - wa)):
                h = y[i] @ params[p + "fc1.weight"][e].T + params[p + "fc1.bias"][e]
                h = 0.5 * h * (1.0 + np.vectorize(math.erf)(h / np.sqrt(2.0)))
                want[i] += w[:, None] * (h @ params[p + "fc2.weight"][e].T + params[p + "fc2.bias"][e])
        assert np.abs(got - want).max() < 1e-12
        assert not np.array_equal(cache["experts"], cache["own_experts"])
    # the backward pass of a forced choice is the derivative of that forced forward (finite differences on y)
    forced = np.empty((B, T, 2), dtype=np.int64)
    forced[..., 0], forced[..., 1] = 2, 1
    rng = np.random.default_rng(1)
    dout = rng.standard_normal(y.shape)
    _, cache = O.moe_fwd(MOE, params, 1, y, task_ids, forced_experts=forced)
    dy = O.moe_bwd(MOE, params, 1, dout, cache, task_ids, {}, False)
    h = 1e-6
    for idx in ((0, 0, 0), (1, 3, 7), (3, 5, 31)):
        yp, ym = y.copy(), y.copy()
        yp[idx] += h
        ym[idx] -= h
        fd = ((O.moe_fwd(MOE, params, 1, yp, task_ids, forced_experts=forced)[0] -
               O.moe_fwd(MOE, params, 1, ym, task_ids, forced_experts=forced)[0]) * dout).sum() / (2 * h)
        assert abs(fd - dy[idx]) < 1e-6 * max(1.0, abs(fd))


def test_moe_mac_term_counts_the_rows_each_expert_processes():
    """Brute force on a tiny model: every (token, slot) pair sends one row through one expert's two layers
    (2 D F multiply-accumulates), and every token meets the gate once (D E)."""
    images, labels, task_ids, params = synth.make_workload(MOE)
    fw = O.forward(MOE, params, images, task_ids)
    dense = MOE.with_(moe_experts=0, moe_top_k=0, moe_blocks=())
    D, F = MOE.dim, MOE.mlp_hidden
    rows = sum(int((fw["routing"][1]["experts"][b] == e).sum()) for b in range(MOE.batch) for e in range(MOE.moe_experts))
    tokens = fw["routing"][1]["experts"].shape[1]
    per_image = rows // MOE.batch * 2 * D * F + tokens * D * MOE.moe_experts
    assert rows == MOE.batch * tokens * MOE.moe_top_k
    assert C.forward_macs(MOE) - C.forward_macs(dense) == per_image - 2 * tokens * D * F


def test_e4m3_rounding_matches_the_library_type_and_the_format_definition():
    import torch
    rng = np.random.default_rng(8)
    x = np.concatenate([rng.standard_normal(20000) * s for s in (1e-3, 0.05, 1.0, 30.0, 150.0)])
    x = np.clip(x, -448.0, 448.0).astype(np.float32)
    want = torch.tensor(x).to(torch.float8_e4m3fn).float().numpy().astype(np.float64)
    assert np.array_equal(O.e4m3_round(x), want)
    # format facts: 3 mantissa bits, ties to the even mantissa, subnormal steps of 2^-9, top value 448, saturation
    assert list(O.e4m3_round(np.array([17.0, 19.0, 21.0, 1.0625, 1.1875]))) == [16.0, 20.0, 20.0, 1.0, 1.25]
    assert list(O.e4m3_round(np.array([2.0 ** -9, 2.0 ** -10, 1.5 * 2.0 ** -10, 3 * 2.0 ** -10]))) == [2.0 ** -9, 0.0, 2.0 ** -9, 2.0 ** -8]
    assert list(O.e4m3_round(np.array([448.0, 449.0, 1e6, -1e6, 0.0]))) == [448.0, 448.0, 448.0, -448.0, 0.0]
    grid = O.e4m3_round(np.linspace(-448, 448, 200001))
    assert len(np.unique(np.abs(grid))) <= 127                   # 7 bits of magnitude, one code short of 128 (no NaN / inf here)


def test_row_quantisation_scales_each_row_to_the_top_of_the_format():
    rng = np.random.default_rng(9)
    a = rng.standard_normal((7, 96)) * rng.random((7, 1)) * 10
    a[3] = 0.0
    deq, scale = O.quantize_rows_e4m3(a)
    assert scale.shape == (7, 1) and scale[3, 0] == 1.0 and not deq[3].any()
    for r in (0, 1, 2, 4, 5, 6):
        assert abs(np.abs(deq[r]).max() - np.abs(a[r]).max()) <= 1e-6 * np.abs(a[r]).max()     # the largest entry maps to 448 exactly
        assert np.abs(deq[r] - a[r]).max() <= np.abs(a[r]).max() / 448 * 16 + 1e-12             # half a step of the top binade
        rel = np.abs(deq[r] - a[r]) / np.maximum(np.abs(a[r]), np.abs(a[r]).max() * 2.0 ** -6)
        assert rel.max() <= 2.0 ** -4 + 1e-6                                                    # 3 mantissa bits: half an ulp
    x, w, b = rng.standard_normal((5, 64)), rng.standard_normal((9, 64)), rng.standard_normal(9)
    y = O.linear_e4m3(x, w, b)
    assert np.linalg.norm(y - O.linear(x, w, b)) / np.linalg.norm(O.linear(x, w, b)) < 0.06    # a few percent, not exact
    assert np.array_equal(y, O.quantize_rows_e4m3(x)[0] @ O.quantize_rows_e4m3(w)[0].T + b)


def test_fp8_prefix_touches_only_the_blocks_before_the_first_trainable_one():
    cfg = synth.CONFIGS["tiny_fp32"]
    images, labels, task_ids, params = synth.make_workload(cfg, peaked=True)
    plain = O.train_step(cfg, params, images, labels, task_ids)
    q = O.train_step(cfg.with_(frozen_fp8=1), params, images, labels, task_ids, forced_keep=plain["kept"])
    assert q["loss"] != plain["loss"] and abs(q["loss"] - plain["loss"]) < 0.05 * plain["loss"]
    allb = cfg.with_(trainable=tuple(range(cfg.depth)), frozen_fp8=1)                # no frozen prefix: nothing to quantise
    a = O.train_step(allb, params, images, labels, task_ids)
    b = O.train_step(allb.with_(frozen_fp8=0), params, images, labels, task_ids)
    assert a["loss"] == b["loss"]


def test_attention_backward_equals_autograd_through_softmax():
    """dq, dk, dv of the oracle against torch autograd through softmax(q k^T / sqrt(d)) v, with a second loss term that
    reaches the classification row of the map directly (what the fused token's score gradient does)."""
    import torch
    rng = np.random.default_rng(21)
    B, H, T, d = 2, 3, 7, 8
    q, k, v, do = (rng.standard_normal((B, H, T, d)) for _ in range(4))
    dA_cls = rng.standard_normal((B, T))

    class Cfg:
        heads = H
        dim = H * d
    _, A = O.attention_fwd(Cfg, q, k, v)
    got = O.attention_bwd(Cfg, A, q, k, v, do, dA_cls)
    tq, tk, tv = (torch.tensor(a, requires_grad=True) for a in (q, k, v))
    att = torch.softmax(tq @ tk.transpose(-1, -2) / math.sqrt(d), dim=-1)
    loss = ((att @ tv) * torch.tensor(do)).sum() + (att[:, :, 0, :] * torch.tensor(dA_cls)[:, None, :]).sum()
    loss.backward()
    for g, t in zip(got, (tq, tk, tv)):
        assert np.abs(g - t.grad.numpy()).max() < 1e-12
    plain = O.attention_bwd(Cfg, A, q, k, v, do)                 # without the extra term the answer differs
    assert np.abs(plain[0] - got[0]).max() > 1e-3
