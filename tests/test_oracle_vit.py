"""Pins of the oracle's forward, backward and optimiser against library routines and invariants."""
import math

import numpy as np
import pytest
import torch

from oracle import bsr_oracle as O
from paper_2405_10951_b200 import synth
from paper_2405_10951_b200.synth import Config

import torch_vit

TINY = Config("t", 16, 4, 32, 2, 4, 64, (5,), 3, (0, 1, 2, 3), (1, 2), 7, 10, dtype="fp32", seed=3)


def workload(cfg, peaked=True, scale=6.0):
    images, labels, task_ids, params = synth.make_workload(cfg, peaked=peaked)
    rng = np.random.default_rng(99)
    for k in params:                                     # non-degenerate biases and norms, larger weights
        if k.endswith("bias"):
            params[k] = rng.standard_normal(params[k].shape) * 0.1
        elif "norm" in k:
            params[k] = 1.0 + 0.2 * rng.standard_normal(params[k].shape)
        else:
            params[k] = params[k] * scale
    return images, labels, task_ids, params


def close(a, b, tol=1e-9):
    a, b = np.asarray(a), np.asarray(b)
    return np.linalg.norm(a - b) <= tol * max(np.linalg.norm(b), 1e-30)


CASES = {
    "plain_vit_all_trainable": TINY.with_(drop_blocks=(), keep_num=1, keep_den=1),
    "keep_one_at_locations": TINY.with_(keep_num=1, keep_den=1),
    "drop_with_fusion": TINY,
    "drop_without_fusion": TINY.with_(fuse_mode=0),
    "drop_with_mean_fusion": TINY.with_(fuse_mode=2),
    "suffix_trainable": TINY.with_(trainable=(2, 3), drop_blocks=(1, 3)),
    "interleaved_trainable": TINY.with_(trainable=(1, 3), drop_blocks=(1, 2)),
    "moe_multitask": TINY.with_(num_classes=(5, 3), batch=4, moe_experts=4, moe_top_k=2, moe_blocks=(1, 3)),
}


@pytest.mark.parametrize("case", list(CASES))
def test_step_matches_autograd_vit(case):
    """Loss, logits, kept sets and every gradient equal a float64 autograd ViT built from library ops."""
    cfg = CASES[case]
    images, labels, task_ids, params = workload(cfg)
    out = O.train_step(cfg, params, images, labels, task_ids)
    loss, logits, grads, kept = torch_vit.run(cfg, params, images, labels, task_ids,
                                              lambda m: O.keep_count(m, cfg.keep_num, cfg.keep_den))
    assert abs(out["loss"] - loss) < 1e-12 * max(1.0, abs(loss))
    for b in range(cfg.batch):
        n = cfg.num_classes[task_ids[b]]
        assert close(out["logits"][b, :n], logits[b])
    assert len(kept) == len(out["kept"])
    for a, b in zip(out["kept"], kept):
        assert np.array_equal(a, b)
    t0 = min(cfg.trainable)
    for name in O.trainable_names(cfg, params):
        assert close(out["grads"][name], grads[name], 1e-8), name
    # gradient propagation stops at the earliest trainable block: nothing is formed before it,
    # nor for patch embedding, positional embedding or the classification token.
    for name in params:
        if name not in O.trainable_names(cfg, params):
            assert name not in out["grads"], name
    if t0 == 0 and case == "plain_vit_all_trainable":
        assert all(ta == tf == cfg.num_patches + 1 for ta, tf in out["tokens"])


def test_frozen_params_unchanged_and_token_counts():
    cfg = CASES["suffix_trainable"]
    images, labels, task_ids, params = workload(cfg)
    out = O.train_step(cfg, params, images, labels, task_ids)
    names = set(O.trainable_names(cfg, params))
    for k in params:
        if k in names:
            assert not np.array_equal(out["params"][k], params[k]), k
        else:
            assert out["params"][k] is params[k]
    m0 = cfg.num_patches
    k1 = math.ceil(0.7 * m0)
    assert out["tokens"][1] == (m0 + 1, k1 + 2)
    k2 = math.ceil(0.7 * (k1 + 1))
    assert out["tokens"][3] == (k1 + 2, k2 + 2)
    assert [k.shape for k in out["kept"]] == [(cfg.batch, k1), (cfg.batch, k2)]


def test_adamw_matches_library_optimiser():
    """Three steps of the oracle's update equal torch.optim.AdamW (decay on matrices only)."""
    cfg = CASES["drop_with_fusion"].with_(lr=1e-2, weight_decay=0.1)
    images, labels, task_ids, params = workload(cfg)
    names = O.trainable_names(cfg, params)
    tp = {n: torch.tensor(params[n], dtype=torch.float64, requires_grad=True) for n in names}
    opt = torch.optim.AdamW([
        {"params": [tp[n] for n in names if O.is_decayed(n)], "weight_decay": cfg.weight_decay},
        {"params": [tp[n] for n in names if not O.is_decayed(n)], "weight_decay": 0.0}],
        lr=cfg.lr, betas=(cfg.beta1, cfg.beta2), eps=cfg.eps)
    state, cur = None, params
    for step in (1, 2, 3):
        out = O.train_step(cfg, cur, images, labels, task_ids, opt_state=state, step=step)
        for n in names:
            tp[n].grad = torch.tensor(out["grads"][n])
        opt.step()
        cur, state = out["params"], out["opt_state"]
        for n in names:
            assert close(cur[n], tp[n].detach().numpy(), 1e-12), (step, n)
    assert {n for n in names if O.is_decayed(n)} >= {"head.0.weight", "blocks.0.attn.qkv.weight"}
    assert not O.is_decayed("norm.weight") and not O.is_decayed("blocks.0.mlp.fc1.bias")


def test_adamw_first_step_closed_form():
    cfg = TINY.with_(lr=1e-3, weight_decay=0.05)
    g = np.array([0.3, -2.0, 1e-3])
    p = np.array([1.0, -1.0, 0.5])
    new, m, v = O.adamw(cfg, p, g, np.zeros(3), np.zeros(3), 1, True)
    assert np.allclose(new, p - cfg.lr * g / (np.abs(g) + cfg.eps) - cfg.lr * cfg.weight_decay * p, rtol=1e-12)


def test_sgd_matches_library_optimiser():
    """Three steps of the oracle's SGD-with-momentum update (Section 5: the ViT-B recipe) equal torch.optim.SGD, decay on
    matrices only."""
    cfg = CASES["drop_with_fusion"].with_(optimizer="sgd", momentum=0.9, lr=5e-2, weight_decay=0.01)
    images, labels, task_ids, params = workload(cfg)
    names = O.trainable_names(cfg, params)
    tp = {n: torch.tensor(params[n], dtype=torch.float64, requires_grad=True) for n in names}
    opt = torch.optim.SGD([
        {"params": [tp[n] for n in names if O.is_decayed(n)], "weight_decay": cfg.weight_decay},
        {"params": [tp[n] for n in names if not O.is_decayed(n)], "weight_decay": 0.0}],
        lr=cfg.lr, momentum=cfg.momentum)
    state, cur = None, params
    for step in (1, 2, 3):
        out = O.train_step(cfg, cur, images, labels, task_ids, opt_state=state, step=step)
        for n in names:
            tp[n].grad = torch.tensor(out["grads"][n])
        opt.step()
        cur, state = out["params"], out["opt_state"]
        for n in names:
            assert close(cur[n], tp[n].detach().numpy(), 1e-12), (step, n)


def test_sgd_closed_forms():
    """First step: p - lr (g + wd p).  Constant gradient without decay: after n steps the parameter has moved by
    lr g sum_{k=1..n} (1 - mu^k) / (1 - mu)."""
    cfg = TINY.with_(optimizer="sgd", momentum=0.8, lr=1e-2, weight_decay=0.05)
    g = np.array([0.3, -2.0, 1e-3])
    p = np.array([1.0, -1.0, 0.5])
    new, buf = O.sgd_momentum(cfg, p, g, np.zeros(3), True)
    assert np.allclose(new, p - cfg.lr * (g + cfg.weight_decay * p), rtol=1e-13)
    assert np.allclose(buf, g + cfg.weight_decay * p, rtol=1e-13)
    q, buf = p.copy(), np.zeros(3)
    for _ in range(5):
        q, buf = O.sgd_momentum(cfg, q, g, buf, False)
    mu = cfg.momentum
    assert np.allclose(p - q, cfg.lr * g * sum((1 - mu ** k) / (1 - mu) for k in range(1, 6)), rtol=1e-12)


def test_order_of_kept_rows_is_immaterial():
    """No positional term is added after the embedding, so permuting the compacted rows leaves the CLS output alone."""
    cfg = TINY.with_(drop_blocks=(1,), depth=3, trainable=(2,))
    images, labels, task_ids, params = workload(cfg)
    rng = np.random.default_rng(0)
    x = O.embed(cfg, params, images)
    x, _, _ = O.block_fwd(cfg, params, 0, x, task_ids, None, None)
    k = O.token_schedule(cfg)[1][2]
    x1, _, _ = O.block_fwd(cfg, params, 1, x, task_ids, k, None)
    perm = np.concatenate([[0], 1 + rng.permutation(x1.shape[1] - 1)])
    ya, _, _ = O.block_fwd(cfg, params, 2, x1, task_ids, None, None)
    yb, _, _ = O.block_fwd(cfg, params, 2, x1[:, perm], task_ids, None, None)
    assert np.abs(ya[:, 0] - yb[:, 0]).max() < 1e-12
    assert np.abs(ya[:, perm] - yb).max() < 1e-12


def test_score_invariants():
    cfg = CASES["drop_with_fusion"]
    images, labels, task_ids, params = workload(cfg)
    fw = O.forward(cfg, params, images, task_ids, keep_cache=True)
    A = fw["caches"][1]["A"]
    assert np.abs(A.sum(axis=-1) - 1.0).max() < 1e-13
    s = fw["scores"][0]
    assert np.abs(s.sum(axis=1) - (1.0 - A[:, :, 0, 0].mean(axis=1))).max() < 1e-13
    for kept, sc in zip(fw["kept"], fw["scores"]):
        for b in range(cfg.batch):
            m = sc.shape[1]
            rest = np.setdiff1d(np.arange(m), kept[b])
            assert np.all(np.diff(kept[b]) > 0)
            assert sc[b][kept[b]].min() >= sc[b][rest].max()


def test_single_head_pre_and_post_softmax_rank_alike():
    """Eq. 6 is written before the softmax; with one head the softmax is monotone, so the sets agree."""
    cfg = TINY.with_(heads=1, drop_blocks=(1,))
    images, labels, task_ids, params = workload(cfg)
    fw = O.forward(cfg, params, images, task_ids, keep_cache=True)
    c = fw["caches"][1]
    raw = (c["q"][:, 0, 0:1] @ c["k"][:, 0].transpose(0, 2, 1))[:, 0, 1:] / math.sqrt(cfg.dim)
    k = fw["kept"][0].shape[1]
    for b in range(cfg.batch):
        assert np.array_equal(O.select_tokens(raw[b], k)[0], fw["kept"][0][b])


def test_loss_at_initialisation_is_log_classes():
    for name, ncls in (("tiny_fp32", 10),):
        cfg = synth.CONFIGS[name]
        images, labels, task_ids, params = synth.make_workload(cfg)
        fw = O.forward(cfg, params, images, task_ids)
        loss, _ = O.cross_entropy(fw["logits"], labels)
        assert abs(loss - math.log(ncls)) < 0.15


def test_moe_with_identical_experts_is_the_dense_ffn():
    cfg = CASES["moe_multitask"]
    images, labels, task_ids, params = workload(cfg)
    dense = cfg.with_(moe_experts=0, moe_top_k=0, moe_blocks=())
    dparams = {k: v for k, v in params.items() if ".moe." not in k}
    for l in cfg.moe_blocks:
        p = f"blocks.{l}."
        for nm in ("fc1.weight", "fc1.bias", "fc2.weight", "fc2.bias"):
            params[p + "moe." + nm][:] = params[p + "moe." + nm][0]
            dparams[p + "mlp." + nm] = params[p + "moe." + nm][0].copy()
    a = O.forward(cfg, params, images, task_ids)
    b = O.forward(dense, dparams, images, task_ids)
    fin = np.isfinite(a["logits"])
    assert np.array_equal(fin, np.isfinite(b["logits"]))
    assert np.abs(a["logits"][fin] - b["logits"][fin]).max() < 1e-12


def test_forced_keep_replaces_the_selection():
    cfg = CASES["drop_with_fusion"]
    images, labels, task_ids, params = workload(cfg)
    base = O.train_step(cfg, params, images, labels, task_ids)
    same = O.train_step(cfg, params, images, labels, task_ids, forced_keep=[k for k in base["kept"]])
    assert same["loss"] == base["loss"]
    forced = [k.copy() for k in base["kept"]]
    m = cfg.num_patches
    missing = np.setdiff1d(np.arange(m), forced[0][0])
    forced[0][0][0] = missing[0]
    other = O.train_step(cfg, params, images, labels, task_ids, forced_keep=forced)
    assert other["loss"] != base["loss"]
    assert sorted(other["kept"][0][0]) == sorted(forced[0][0])


def test_cosine_schedule_matches_library_scheduler_and_closed_forms():
    import torch
    lr_max, lr_min, total = 3e-3, 2e-5, 37
    assert O.cosine_lr(lr_max, lr_min, 0, total) == lr_max
    assert abs(O.cosine_lr(lr_max, lr_min, total, total) - lr_min) < 1e-18
    assert O.cosine_lr(lr_max, lr_min, total + 5, total) == O.cosine_lr(lr_max, lr_min, total, total)       # held at the floor
    assert abs(O.cosine_lr(1.0, 0.0, 1, 2) - 0.5) < 1e-15 and abs(O.cosine_lr(1.0, 0.0, 1, 3) - 0.75) < 1e-15   # cos(pi/2), cos(pi/3)
    rates = [O.cosine_lr(lr_max, lr_min, t, total) for t in range(total + 1)]
    assert all(a > b for a, b in zip(rates, rates[1:]))                                                      # strictly decaying
    p = torch.nn.Parameter(torch.zeros(1))
    opt = torch.optim.SGD([p], lr=lr_max)
    sch = torch.optim.lr_scheduler.CosineAnnealingLR(opt, T_max=total, eta_min=lr_min)
    for t in range(total + 1):
        assert abs(opt.param_groups[0]["lr"] - rates[t]) < 1e-12 * lr_max, t
        opt.step()
        sch.step()


def test_run_of_steps_uses_the_schedule_per_step():
    cfg = CASES["drop_with_fusion"].with_(optimizer="sgd", momentum=0.0, weight_decay=0.0)
    images, labels, task_ids, params = workload(cfg)
    batches = [(images, labels, task_ids)] * 3
    runs = O.train_steps(cfg, params, batches, 1e-2, 1e-3, 4)
    # plain SGD: every step moves a parameter by exactly -lr(t) * gradient of that step
    prev = params
    for t, r in enumerate(runs):
        lr = O.cosine_lr(1e-2, 1e-3, t, 4)
        n = "head.0.weight"
        assert np.allclose(r["params"][n] - prev[n], -lr * r["grads"][n], rtol=1e-9, atol=1e-15)
        prev = r["params"]
    assert runs[1]["loss"] < runs[0]["loss"]
