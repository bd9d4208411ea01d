"""Finite-difference pin of the oracle's backward pass and brute-force pin of its top-k."""
import numpy as np
import pytest

from oracle import bsr_oracle as O
from paper_2405_10951_b200 import synth

from test_oracle_vit import CASES, workload


def loss_of(cfg, params, images, labels, task_ids, forced):
    fw = O.forward(cfg, params, images, task_ids, forced_keep=forced)
    return O.cross_entropy(fw["logits"], labels)[0]


@pytest.mark.parametrize("case", ["drop_with_fusion", "drop_with_mean_fusion", "suffix_trainable", "moe_multitask"])
def test_gradients_match_central_differences(case):
    """Directional derivatives along random directions, every trainable tensor, rel. error < 1e-6.

    The kept sets are frozen to those of the unperturbed point (they are constants of the
    backward pass), and the case has a trainable block that is a token drop location, so the
    gradient through the fusion weights is exercised.
    """
    cfg = CASES[case]
    images, labels, task_ids, params = workload(cfg)
    out = O.train_step(cfg, params, images, labels, task_ids)
    assert min(m.min() for m in out["margins"]) > 1e-4
    forced = out["kept"]
    rng = np.random.default_rng(5)
    h = 2e-4
    for name in O.trainable_names(cfg, params):
        g = out["grads"][name]
        for _ in range(2):
            u = rng.standard_normal(g.shape)
            u /= np.linalg.norm(u)
            def central(step):
                pp = dict(params); pp[name] = params[name] + step * u
                pm = dict(params); pm[name] = params[name] - step * u
                return (loss_of(cfg, pp, images, labels, task_ids, forced) -
                        loss_of(cfg, pm, images, labels, task_ids, forced)) / (2 * step)
            fd = (4.0 * central(h / 2) - central(h)) / 3.0          # Richardson: O(h^4) truncation
            an = float((g * u).sum())
            assert abs(fd - an) <= 1e-6 * max(abs(an), np.linalg.norm(g) * 1e-2) + 1e-11, (name, fd, an)


def brute_force_topk(s, k):
    """Pick the largest remaining score k times; on equal scores the lower index wins."""
    s = list(s)
    chosen = []
    for _ in range(k):
        best = None
        for j, v in enumerate(s):
            if j in chosen:
                continue
            if best is None or v > s[best]:
                best = j
        chosen.append(best)
    return sorted(chosen)


@pytest.mark.parametrize("ties", [False, True])
def test_select_matches_brute_force(ties):
    rng = np.random.default_rng(11)
    for m, k in [(1, 1), (7, 3), (64, 45), (196, 138), (99, 70), (33, 33), (50, 1)]:
        p = synth.make_scores(rng, 4, 3, m, ties=ties)
        s = O.head_mean_scores(p, np.float32)
        assert s.dtype == np.float32
        for b in range(4):
            kept, dropped = O.select_tokens(s[b], k)
            assert list(kept) == brute_force_topk(s[b], k)
            assert len(kept) == k and len(dropped) == m - k
            assert sorted(list(kept) + list(dropped)) == list(range(m))
            assert np.all(np.diff(kept) > 0) and np.all(np.diff(dropped) > 0)
    if ties:
        assert len(np.unique(s[0])) < len(s[0])


def test_head_mean_is_fixed_order_sum_then_divide():
    p = np.array([[1e8, 1.0], [1.0, 2.0], [-1e8, 3.0]], dtype=np.float32)   # [H=3, M=2]
    s = O.head_mean_scores(p, np.float32)
    assert s[0] == np.float32((np.float32(1e8) + np.float32(1.0)) + np.float32(-1e8)) / np.float32(3)
    assert s[1] == np.float32(6.0) / np.float32(3)


def test_gather_fuse_definition():
    rng = np.random.default_rng(2)
    B, M, D, k = 2, 9, 5, 4
    xp = rng.standard_normal((B, M + 1, D))
    s = rng.random((B, M))
    kept = np.stack([np.sort(rng.permutation(M)[:k]) for _ in range(B)])
    dropped = np.stack([np.setdiff1d(np.arange(M), kept[b]) for b in range(B)])
    out = O.gather_fuse(xp, kept, dropped, s)
    assert out.shape == (B, k + 2, D)
    for b in range(B):
        assert np.array_equal(out[b, 0], xp[b, 0])
        for i, j in enumerate(kept[b]):
            assert np.array_equal(out[b, 1 + i], xp[b, 1 + j])
        fused = sum(s[b, j] * xp[b, 1 + j] for j in dropped[b])
        assert np.allclose(out[b, -1], fused, rtol=1e-13)
    assert O.gather_fuse(xp, kept, dropped, s, fuse_mode=0).shape == (B, k + 1, D)
    # weighted mean (fuse_mode 2): the weighted sum over the sum of the weights; equal weights give the plain mean of
    # the dropped tokens, a single dropped token comes back unchanged
    mean = O.gather_fuse(xp, kept, dropped, s, fuse_mode=2)
    for b in range(B):
        assert np.allclose(mean[b, -1], out[b, -1] / s[b, dropped[b]].sum(), rtol=1e-13)
    flat = O.gather_fuse(xp, kept, dropped, np.full_like(s, 0.125), fuse_mode=2)
    for b in range(B):
        assert np.allclose(flat[b, -1], xp[b, 1 + dropped[b]].mean(axis=0), rtol=1e-13)
    one = O.gather_fuse(xp, np.stack([np.arange(M - 1)] * B), np.full((B, 1), M - 1), s, fuse_mode=2)
    assert np.allclose(one[:, -1], xp[:, M], rtol=1e-15)
