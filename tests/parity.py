"""Shared machinery of the GPU-vs-oracle parity tests (GPU side always through the C ABI)."""
import numpy as np

from oracle import bsr_oracle as O
from paper_2405_10951_b200 import synth

FP32_TOL = 1e-4          # relative, ||gpu - ref||_2 / ||ref||_2 per tensor
BF16_TOL = 2e-2
EXACT_MARGIN = 1e-3      # kept sets must be identical where the oracle's boundary margin exceeds this (fp32)
# bf16 storage perturbs every score by up to ~1e-2 relative (8 mantissa bits on q, k and on the block input),
# so a bf16 run may legitimately swap tokens whose scores are closer than that.
BF16_SCORE_TOL = 1e-1


def rel_err(a, b):
    a = np.asarray(a, dtype=np.float64).ravel()
    b = np.asarray(b, dtype=np.float64).ravel()
    return float(np.linalg.norm(a - b) / max(np.linalg.norm(b), 1e-300))


def param_shape(cfg, name):
    return synth.param_shapes(cfg)[name]


def run_gpu_step(cfg, images, labels, task_ids, params, batch=None, steps=1):
    """One (or more) bsr_train_step calls; returns everything the comparison needs as numpy."""
    import torch
    from paper_2405_10951_b200 import binding as Bd
    eng = Bd.Engine(cfg, max_batch=images.shape[0])
    eng.set_params(params)
    img = eng.images_to_device(images)
    lab = torch.as_tensor(labels.astype(np.int32)).cuda()
    tid = torch.as_tensor(task_ids.astype(np.int32)).cuda() if cfg.num_tasks > 1 else None
    out = {}
    for _ in range(steps):
        loss, kept = eng.train_step(img, lab, tid)
    eng.sync_status()
    out["loss"] = float(loss.cpu()[0])
    out["kept"] = [k.cpu().numpy().astype(np.int64) for k in kept] if kept else []
    B = images.shape[0]
    out["logits"] = eng.get_tensor("logits", (B, eng.cmax)).cpu().numpy().astype(np.float64)
    names = O.trainable_names(cfg, params)
    shapes = synth.param_shapes(cfg)
    out["grads"] = {n: eng.get_tensor("grad/" + n, shapes[n]).cpu().numpy().astype(np.float64) for n in names}
    out["m"] = {n: eng.get_tensor("adam_m/" + n, shapes[n]).cpu().numpy().astype(np.float64) for n in names}
    out["v"] = {n: eng.get_tensor("adam_v/" + n, shapes[n]).cpu().numpy().astype(np.float64) for n in names}
    out["params"] = {n: eng.get_tensor(n, shapes[n]).cpu().numpy().astype(np.float64) for n in shapes}
    out["experts"] = {}
    for l in cfg.moe_blocks:
        tokens = 1 if (l == cfg.depth - 1 and l not in cfg.drop_blocks) else eng.tf[l]     # last block: classification rows only
        e = eng.get_tensor(f"moe_experts/{l}", (B * tokens * cfg.moe_top_k,)).cpu().numpy()
        out["experts"][l] = e.astype(np.int64).reshape(B, tokens, cfg.moe_top_k)
    out["footprint"] = eng.footprint()
    out["engine"] = eng
    return out


def check_selection(cfg, gpu_kept, forced_run, exact_margin, score_tol):
    """The rule for kept-index sets.

    `forced_run` is the oracle run with the GPU's kept sets forced, so its scores at every location are
    the oracle's scores for exactly the token sequence the GPU saw.  Per image and location:
      * the GPU's set must be a valid top-K of those scores within score_tol
        (weakest kept score >= strongest dropped score - score_tol * s_(K));
      * where the oracle's own boundary margin exceeds exact_margin the set must be identical to the
        oracle's own choice.
    Returns (number of sets compared, number identical to the oracle's own choice).
    """
    total = same = 0
    for loc, (kept, scores) in enumerate(zip(gpu_kept, forced_run["scores"])):
        B, k = kept.shape
        m = scores.shape[1]
        for b in range(B):
            own, own_dropped = O.select_tokens(scores[b], k)
            mine = np.sort(kept[b])
            assert len(np.unique(mine)) == k and mine.min() >= 0 and mine.max() < m, (loc, b)
            assert np.array_equal(mine, kept[b]), "kept indices must be ascending"
            rest = np.setdiff1d(np.arange(m), mine)
            identical = np.array_equal(own, mine)
            total += 1
            same += int(identical)
            if len(rest):
                sk = scores[b][own].min()
                assert scores[b][mine].min() >= scores[b][rest].max() - score_tol * sk, (loc, b)
                margin = O.boundary_margin(scores[b], own, own_dropped)
                if margin > exact_margin:
                    assert identical, f"location {loc} image {b}: margin {margin:.3e} but sets differ"
    return total, same


def forced_experts_of(cfg, gpu, token_counts):
    """The GPU's routing as the oracle's forced_experts input; tokens the GPU never routed (rows of the last
    block other than the classification row) are left to the oracle (-1)."""
    out = {}
    for l, e in gpu.get("experts", {}).items():
        B, t, k = e.shape
        full = np.full((B, token_counts[l], k), -1, dtype=np.int64)
        full[:, :t] = e
        out[l] = full
    return out


def check_routing(cfg, ref, gpu, logit_tol):
    """Every expert the GPU chose must be a valid top-k choice of the oracle's gate logits within logit_tol."""
    flips = total = 0
    for l, e in gpu.get("experts", {}).items():
        gl = ref["routing"][l]["glogits"]
        own = ref["routing"][l]["own_experts"]
        B, t, k = e.shape
        for b in range(B):
            for i in range(t):
                kth = np.sort(gl[b, i])[-k]
                assert len(set(e[b, i])) == k
                assert gl[b, i][e[b, i]].min() >= kth - logit_tol, (l, b, i)
                total += 1
                flips += int(set(e[b, i]) != set(own[b, i]))
    return total, flips


def compare_step(cfg, images, labels, task_ids, params, gpu, tol, exact_margin, score_tol):
    forced = gpu["kept"] if gpu["kept"] else None
    fe = None
    if gpu.get("experts"):
        sched = O.token_schedule(cfg)
        fe = forced_experts_of(cfg, gpu, {l: sched[l][1] for l in cfg.moe_blocks})
    ref = O.train_step(cfg, params, images, labels, task_ids, forced_keep=forced, forced_experts=fe)
    if fe:
        check_routing(cfg, ref, gpu, 2e-2)
    total, same = check_selection(cfg, gpu["kept"], ref, exact_margin, score_tol) if forced else (0, 0)
    report = {"sets": total, "sets_identical": same}
    assert abs(gpu["loss"] - ref["loss"]) <= tol * abs(ref["loss"]), (gpu["loss"], ref["loss"])
    B = images.shape[0]
    fin = np.isfinite(ref["logits"])
    assert np.array_equal(fin, np.isfinite(gpu["logits"][:B]))
    e = rel_err(gpu["logits"][:B][fin], ref["logits"][fin])
    report["logits"] = e
    assert e <= tol, ("logits", e)
    worst = 0.0
    for n, g in ref["grads"].items():
        e = rel_err(gpu["grads"][n], g)
        worst = max(worst, e)
        assert e <= tol, (n, e)
        assert rel_err(gpu["m"][n], (1 - cfg.beta1) * g) <= tol, n
    report["worst_grad"] = worst
    # the update itself, from the GPU's own gradient (AdamW's first step is a sign function of g: comparing
    # updated weights across implementations would amplify rounding of near-zero gradients without bound)
    for n in ref["grads"]:
        if np.abs(gpu["grads"][n]).max() < 1e-6:         # an identically-zero gradient (e.g. the gate of a top-1 router):
            continue                                     # g / (|g| + eps) is then dominated by float rounding of g itself
        want, _, _ = O.adamw(cfg, params[n], gpu["grads"][n], np.zeros_like(params[n]), np.zeros_like(params[n]), 1, O.is_decayed(n))
        d_gpu = gpu["params"][n] - params[n]
        d_ref = want - params[n]
        assert rel_err(d_gpu, d_ref) <= 2e-3, (n, rel_err(d_gpu, d_ref))
    for n in params:                       # frozen parameters are untouched (bit-exact round trip)
        if n not in ref["grads"]:
            assert np.array_equal(gpu["params"][n], params[n].astype(np.float32).astype(np.float64)), n
    return report
