"""Float64 CPU oracle for one Block Selective Reprogramming (BSR) fine-tuning step.

TEST INFRASTRUCTURE ONLY.  This file is the slow, plain statement of what the step
computes, written from the paper (arXiv 2405.10951).  Only the tests, the smoke check
and the benchmark's CPU-baseline leg may import it; the CUDA library shares no code,
table or helper with it and never calls it.

What it follows, passage by passage:

* ViT forward, N patches + classification token, positional embedding, encoder blocks of
  multi-head self-attention (Eq. 1) followed by a 2-layer GELU feed-forward network
  (Section 3.1 "Preliminaries").
* Token importance from the classification token's attention row (Eq. 6), top-K kept,
  the rest fused and passed on to the FFN of the same block; tokens are discarded
  incrementally at the "token drop locations" (Section 4.1; Section 4.3 Discussion 3:
  MHSA sees all incoming tokens, the FFN the reduced set).
* Only chosen blocks and the classification head train; gradient propagation stops at the
  earliest trainable block and never reaches patch embedding, positional embedding or the
  classification token (Fig. 2 caption; Eq. 8; Section 4.1 last paragraph).
* Backward by the chain rule for linear and non-linear layers (Eq. 2-5).
* AdamW (Section 5 "Training Hyperparameters").
* MoE layer in place of the FFN: a task-dependent router picks the top experts per token
  and their outputs are added (Section 5.2).

Readings where the paper is silent:
  score = post-softmax CLS row averaged over heads; CLS itself is not a candidate;
  K = ceil(keep * M) in integer arithmetic; kept tokens stay in ascending position and the
  fused token goes last; fused token = sum_j s_j x'_j over the dropped tokens (fuse_mode 1), or that
  sum divided by sum_j s_j (fuse_mode 2, the weighted mean: the other natural reading of "fused"); keep = 1
  appends nothing; ties go to the lower index; the index sets are constants for the
  backward pass while the fusion weights s_j are differentiated; final LayerNorm and head
  train with the chosen blocks; weight decay on matrices only.

Parity pins (tests/test_oracle_*.py): an autograd float64 ViT written with library ops
(forward, all gradients, with and without dropping), torch.optim.AdamW, central finite
differences, the paper's MAC tables and memory closed forms, brute-force top-k, permutation
invariance.  Unpinned by the paper itself (fixed by reading only): the fusion formula, the
MoE gate details (softmax over the selected logits, one gate per task).  "parity unpinned"
applies to those two readings, not to their arithmetic, which the autograd and
finite-difference pins cover.
"""

from __future__ import annotations

import math

import numpy as np
from scipy.special import erf

SQRT2 = np.sqrt(2.0)
SQRT2PI = np.sqrt(2.0 * np.pi)


# ----------------------------------------------------------------------------------------------
# token schedule (Section 4.1 "K being determined by the token drop rate"; Section 4.3 Discussion 3)
# ----------------------------------------------------------------------------------------------
def keep_count(m: int, keep_num: int, keep_den: int) -> int:
    """K = ceil(keep * M) with keep = keep_num / keep_den, clamped to [1, M]."""
    k = (keep_num * m + keep_den - 1) // keep_den
    return max(1, min(m, k))


def token_schedule(cfg):
    """Per block: (tokens seen by MHSA, tokens seen by the FFN, K or None)."""
    t = cfg.num_patches + 1
    out = []
    for l in range(cfg.depth):
        ta = t
        k = None
        if l in cfg.drop_blocks:
            m = t - 1
            k = keep_count(m, cfg.keep_num, cfg.keep_den)
            if k < m:
                t = 1 + k + (1 if cfg.fuse_mode in (1, 2) else 0)
        out.append((ta, t, k))
    return out


# ----------------------------------------------------------------------------------------------
# elementary layers
# ----------------------------------------------------------------------------------------------
def layer_norm(x, g, b, eps):
    mu = x.mean(axis=-1, keepdims=True)
    var = ((x - mu) ** 2).mean(axis=-1, keepdims=True)
    rstd = 1.0 / np.sqrt(var + eps)
    xhat = (x - mu) * rstd
    return xhat * g + b, (xhat, rstd)


def layer_norm_bwd(dy, cache, g):
    xhat, rstd = cache
    dg = (dy * xhat).reshape(-1, xhat.shape[-1]).sum(axis=0)
    db = dy.reshape(-1, xhat.shape[-1]).sum(axis=0)
    dxhat = dy * g
    dx = rstd * (dxhat - dxhat.mean(axis=-1, keepdims=True) - xhat * (dxhat * xhat).mean(axis=-1, keepdims=True))
    return dx, dg, db


def gelu(z):
    """Exact GELU: z * Phi(z)."""
    return 0.5 * z * (1.0 + erf(z / SQRT2))


def gelu_grad(z):
    return 0.5 * (1.0 + erf(z / SQRT2)) + z * np.exp(-0.5 * z * z) / SQRT2PI


def linear(x, w, b):
    """y = x W^T + b with W stored [out, in]."""
    return x @ w.T + b


def linear_bwd(dy, x, w):
    """Eq. 2 (input gradient needs only W) and Eq. 4 (weight gradient needs the input)."""
    dx = dy @ w
    dw = dy.reshape(-1, dy.shape[-1]).T @ x.reshape(-1, x.shape[-1])
    db = dy.reshape(-1, dy.shape[-1]).sum(axis=0)
    return dx, dw, db


# ----------------------------------------------------------------------------------------------
# 8-bit floating point for the frozen prefix (Conclusions: activation / weight quantisation is orthogonal to BSR and
# can be added on top; the paper fixes no format).  Reading taken: the frozen blocks before the earliest trainable
# one carry no gradient, so their two LayerNorm-fed linear layers (QKV and the first FFN layer) may run on operands
# rounded to E4M3 -- each LayerNorm output row and each weight row scaled so that its largest magnitude maps to 448,
# the products accumulated exactly and rescaled.  Everything else stays as it is.
# ----------------------------------------------------------------------------------------------
E4M3_MAX = 448.0


def e4m3_round(x):
    """Nearest value of the 8-bit floating-point format E4M3 (1 sign bit, 4 exponent bits with bias 7, 3 mantissa bits,
    no infinities: largest magnitude 448, normal numbers down to 2^-6, subnormals in steps of 2^-9), ties to the even
    mantissa; magnitudes beyond 448 saturate to 448."""
    x = np.asarray(x, dtype=np.float64)
    a = np.minimum(np.abs(x), E4M3_MAX)
    e = np.floor(np.log2(np.where(a > 0, a, 1.0)))
    e = np.maximum(e, -6.0)                        # below the smallest normal binade the spacing stays 2^-9
    step = 2.0 ** (e - 3.0)                        # 3 mantissa bits: 8 steps per binade
    q = np.minimum(np.round(a / step) * step, E4M3_MAX)      # a / step is exact (power of two); np.round ties to even
    return np.sign(x) * q


def quantize_rows_e4m3(a):
    """Each row of a [..., K] rounded to E4M3 after scaling by scale = max|row| / 448 (1 for an all-zero row); scale and
    quotient are formed in float32, as a kernel forms them.  Returns the dequantised values and the scales."""
    a32 = np.asarray(a, dtype=np.float32)
    amax = np.abs(a32).max(axis=-1, keepdims=True)
    scale = np.where(amax > 0, amax / np.float32(E4M3_MAX), np.float32(1.0)).astype(np.float32)
    q = e4m3_round((a32 / scale).astype(np.float32))
    return q * scale.astype(np.float64), scale


def linear_e4m3(x, w, b):
    """y = x W^T + b with the rows of x and of W rounded to E4M3 (quantize_rows_e4m3), exact accumulation."""
    return quantize_rows_e4m3(x)[0] @ quantize_rows_e4m3(w)[0].T + b


# ----------------------------------------------------------------------------------------------
# token selection (Eq. 6; Section 4.1)
# ----------------------------------------------------------------------------------------------
def head_mean_scores(p, dtype=np.float64):
    """s_j = (1/H) sum_h p[h, j], summed in the order h = 0..H-1 in ``dtype`` then divided by H."""
    p = np.asarray(p, dtype=dtype)
    acc = p[..., 0, :].copy()
    for h in range(1, p.shape[-2]):
        acc = acc + p[..., h, :]
    return acc / dtype(p.shape[-2])


def select_tokens(s, k):
    """Indices (ascending) of the k largest scores of one image; ties go to the lower index.

    Returns (kept, dropped), both ascending; together they partition range(len(s)).
    """
    order = np.argsort(-np.asarray(s), kind="stable")      # descending, equal scores keep index order
    kept = np.sort(order[:k])
    dropped = np.sort(order[k:])
    return kept.astype(np.int64), dropped.astype(np.int64)


def boundary_margin(s, kept, dropped):
    """(s_(k) - s_(k+1)) / s_(k): relative gap between the weakest kept and strongest dropped score."""
    if len(dropped) == 0:
        return np.inf
    lo = s[kept].min()
    hi = s[dropped].max()
    return float((lo - hi) / lo) if lo > 0 else 0.0


# ----------------------------------------------------------------------------------------------
# forward
# ----------------------------------------------------------------------------------------------
def patchify(images, patch):
    """[B, C, S, S] -> [B, N, C*P*P]; each patch flattened as (channel, row, column)."""
    B, C, S, _ = images.shape
    g = S // patch
    x = images.reshape(B, C, g, patch, g, patch)
    x = x.transpose(0, 2, 4, 1, 3, 5)
    return x.reshape(B, g * g, C * patch * patch)


def embed(cfg, params, images):
    x = linear(patchify(images, cfg.patch_size), params["patch_embed.weight"], params["patch_embed.bias"])
    B = x.shape[0]
    cls = np.broadcast_to(params["cls_token"], (B, 1, cfg.dim))
    return np.concatenate([cls, x], axis=1) + params["pos_embed"]


def attention_fwd(cfg, q, k, v):
    """Eq. 1 per head.  q, k, v: [B, H, T, d]."""
    d = q.shape[-1]
    S = (q @ k.transpose(0, 1, 3, 2)) / np.sqrt(d)
    S = S - S.max(axis=-1, keepdims=True)
    A = np.exp(S)
    A = A / A.sum(axis=-1, keepdims=True)
    return A @ v, A


def attention_bwd(cfg, A, q, k, v, do, dA_cls=None):
    """Chain rule through Eq. 1 for one block.  A [B, H, T, T] the attention map, q, k, v, do [B, H, T, d];
    dA_cls [B, T] (optional): a gradient that reaches the classification row of every head's map directly (through
    the scores of Eq. 6), added to that row of dA.  Returns dq, dk, dv."""
    d = q.shape[-1]
    dA = do @ v.transpose(0, 1, 3, 2)
    if dA_cls is not None:
        dA[:, :, 0, :] += dA_cls[:, None, :]
    dv = A.transpose(0, 1, 3, 2) @ do
    dS = A * (dA - (dA * A).sum(axis=-1, keepdims=True))
    dq = dS @ k / np.sqrt(d)
    dk = dS.transpose(0, 1, 3, 2) @ q / np.sqrt(d)
    return dq, dk, dv


def split_heads(cfg, qkv):
    B, T, _ = qkv.shape
    H, d = cfg.heads, cfg.dim // cfg.heads
    qkv = qkv.reshape(B, T, 3, H, d).transpose(2, 0, 3, 1, 4)
    return qkv[0], qkv[1], qkv[2]


def merge_heads(x):
    B, H, T, d = x.shape
    return x.transpose(0, 2, 1, 3).reshape(B, T, H * d)


def moe_route(cfg, glogits):
    """Top experts per token by gate logit (ties -> lower expert id); weights = softmax over the chosen logits."""
    order = np.argsort(-glogits, axis=-1, kind="stable")[..., : cfg.moe_top_k]
    sel = np.take_along_axis(glogits, order, axis=-1)
    e = np.exp(sel - sel.max(axis=-1, keepdims=True))
    return order, e / e.sum(axis=-1, keepdims=True)


def moe_fwd(cfg, params, l, y, task_ids, forced_experts=None):
    """y: [B, T, D] (LayerNorm output).  Returns output and cache.

    forced_experts [B, T, k] replaces the router's top-k choice (the weights are still the softmax of this
    oracle's own gate logits at those experts): used when a lower-precision run made a different choice
    between near-equal logits, exactly as forced_keep does for the kept tokens."""
    p = f"blocks.{l}.moe."
    B, T, D = y.shape
    wg = params[p + "gate.weight"][task_ids]                 # [B, E, D]: task-dependent router
    glogits = np.einsum("btd,bed->bte", y, wg)
    experts, w = moe_route(cfg, glogits)                     # [B, T, k]
    own_experts = experts
    if forced_experts is not None:
        forced = np.asarray(forced_experts, dtype=np.int64).reshape(B, T, cfg.moe_top_k)
        experts = np.where(forced < 0, own_experts, forced)          # negative entries: keep this oracle's choice
        sel = np.take_along_axis(glogits, experts, axis=-1)
        ee = np.exp(sel - sel.max(axis=-1, keepdims=True))
        w = ee / ee.sum(axis=-1, keepdims=True)
    out = np.zeros_like(y)
    cache = {"y": y, "experts": experts, "w": w, "z": {}, "h": {}, "yo": {}, "own_experts": own_experts, "glogits": glogits}
    for e in range(cfg.moe_experts):
        for slot in range(cfg.moe_top_k):
            mask = experts[..., slot] == e                   # [B, T]
            if not mask.any():
                continue
            ye = y[mask]
            z = linear(ye, params[p + "fc1.weight"][e], params[p + "fc1.bias"][e])
            h = gelu(z)
            yo = linear(h, params[p + "fc2.weight"][e], params[p + "fc2.bias"][e])
            out[mask] += w[..., slot][mask][:, None] * yo
            cache["z"][(e, slot)] = z
            cache["h"][(e, slot)] = h
            cache["yo"][(e, slot)] = yo
    return out, cache


def moe_bwd(cfg, params, l, dout, cache, task_ids, grads, want_param_grads):
    p = f"blocks.{l}.moe."
    y, experts, w = cache["y"], cache["experts"], cache["w"]
    B, T, D = y.shape
    dy = np.zeros_like(y)
    dw_sel = np.zeros_like(w)
    g_fc1w = np.zeros_like(params[p + "fc1.weight"])
    g_fc1b = np.zeros_like(params[p + "fc1.bias"])
    g_fc2w = np.zeros_like(params[p + "fc2.weight"])
    g_fc2b = np.zeros_like(params[p + "fc2.bias"])
    for (e, slot), z in cache["z"].items():
        mask = experts[..., slot] == e
        h, yo = cache["h"][(e, slot)], cache["yo"][(e, slot)]
        d_o = dout[mask]
        dw_sel[..., slot][mask] = (d_o * yo).sum(axis=-1)
        dyo = d_o * w[..., slot][mask][:, None]
        dh, dw2, db2 = linear_bwd(dyo, h, params[p + "fc2.weight"][e])
        dz = dh * gelu_grad(z)
        dye, dw1, db1 = linear_bwd(dz, y[mask], params[p + "fc1.weight"][e])
        dy[mask] += dye
        g_fc1w[e] += dw1
        g_fc1b[e] += db1
        g_fc2w[e] += dw2
        g_fc2b[e] += db2
    # softmax over the selected logits
    dsel = w * (dw_sel - (w * dw_sel).sum(axis=-1, keepdims=True))        # [B, T, k]
    wg_all = params[p + "gate.weight"]
    g_gate = np.zeros_like(wg_all)
    for b in range(B):
        t = task_ids[b]
        for slot in range(cfg.moe_top_k):
            e_idx = experts[b, :, slot]
            dy[b] += dsel[b, :, slot][:, None] * wg_all[t][e_idx]
            np.add.at(g_gate[t], e_idx, dsel[b, :, slot][:, None] * y[b])
    if want_param_grads:
        grads[p + "gate.weight"] = g_gate
        grads[p + "fc1.weight"] = g_fc1w
        grads[p + "fc1.bias"] = g_fc1b
        grads[p + "fc2.weight"] = g_fc2w
        grads[p + "fc2.bias"] = g_fc2b
    return dy


def block_fwd(cfg, params, l, x, task_ids, k, forced_keep, forced_experts=None, fp8=False):
    """One encoder block; at a token drop location the compaction sits between MHSA and FFN.  fp8: the two
    LayerNorm-fed linear layers of this (frozen, gradient-free) block run on E4M3 operands."""
    p = f"blocks.{l}."
    c = {"x": x}
    lin = linear_e4m3 if fp8 else linear
    y1, c["ln1"] = layer_norm(x, params[p + "norm1.weight"], params[p + "norm1.bias"], cfg.ln_eps)
    c["y1"] = y1
    q, kk, v = split_heads(cfg, lin(y1, params[p + "attn.qkv.weight"], params[p + "attn.qkv.bias"]))
    o, A = attention_fwd(cfg, q, kk, v)
    c.update(q=q, k=kk, v=v, A=A)
    oc = merge_heads(o)
    c["oc"] = oc
    xp = x + linear(oc, params[p + "attn.proj.weight"], params[p + "attn.proj.bias"])
    info = None
    if k is not None:
        B, T, D = xp.shape
        m = T - 1
        s = head_mean_scores(A[:, :, 0, 1:])                 # [B, M]: CLS row, CLS column excluded
        kept = np.zeros((B, k), dtype=np.int64)
        dropped = np.zeros((B, m - k), dtype=np.int64)
        margins = np.zeros(B)
        for b in range(B):
            kb, db_ = select_tokens(s[b], k)
            margins[b] = boundary_margin(s[b], kb, db_)
            if forced_keep is not None:
                kb = np.sort(np.asarray(forced_keep[b], dtype=np.int64))
                db_ = np.setdiff1d(np.arange(m), kb)
            kept[b], dropped[b] = kb, db_
        info = {"kept": kept, "dropped": dropped, "scores": s, "margins": margins}
        if k < m:
            rows = [xp[:, :1], np.take_along_axis(xp[:, 1:], kept[:, :, None], axis=1)]
            if cfg.fuse_mode in (1, 2):
                xd = np.take_along_axis(xp[:, 1:], dropped[:, :, None], axis=1)
                sd = np.take_along_axis(s, dropped, axis=1)
                fused = (sd[:, :, None] * xd).sum(axis=1, keepdims=True)
                if cfg.fuse_mode == 2:                          # weighted mean: the weights are normalised to sum to one
                    c["ssum"] = sd.sum(axis=1)
                    fused = fused / c["ssum"][:, None, None]
                    c["fused"] = fused[:, 0]
                rows.append(fused)
                c["xd"], c["sd"] = xd, sd
            c["xp_full_shape"] = xp.shape
            xp = np.concatenate(rows, axis=1)
            c["drop"] = info
    c["xp"] = xp
    y2, c["ln2"] = layer_norm(xp, params[p + "norm2.weight"], params[p + "norm2.bias"], cfg.ln_eps)
    c["y2"] = y2
    if l in cfg.moe_blocks:
        f, c["moe"] = moe_fwd(cfg, params, l, y2, task_ids, forced_experts)
    else:
        z = lin(y2, params[p + "mlp.fc1.weight"], params[p + "mlp.fc1.bias"])
        h = gelu(z)
        c.update(z=z, h=h)
        f = linear(h, params[p + "mlp.fc2.weight"], params[p + "mlp.fc2.bias"])
    return xp + f, c, info


def block_bwd(cfg, params, l, dout, c, task_ids, grads, want_param_grads, need_dx):
    p = f"blocks.{l}."
    g = {}
    if l in cfg.moe_blocks:
        dy2 = moe_bwd(cfg, params, l, dout, c["moe"], task_ids, grads, want_param_grads)
    else:
        dh, g["mlp.fc2.weight"], g["mlp.fc2.bias"] = linear_bwd(dout, c["h"], params[p + "mlp.fc2.weight"])
        dz = dh * gelu_grad(c["z"])
        dy2, g["mlp.fc1.weight"], g["mlp.fc1.bias"] = linear_bwd(dz, c["y2"], params[p + "mlp.fc1.weight"])
    dln, g["norm2.weight"], g["norm2.bias"] = layer_norm_bwd(dy2, c["ln2"], params[p + "norm2.weight"])
    dxp = dout + dln
    dA_cls = None
    if "drop" in c:
        info = c["drop"]
        B, T, D = c["xp_full_shape"]
        kept, dropped = info["kept"], info["dropped"]
        kk = kept.shape[1]
        full = np.zeros((B, T, D))
        full[:, 0] = dxp[:, 0]
        bidx = np.arange(B)[:, None]
        full[bidx, 1 + kept] = dxp[:, 1 : 1 + kk]
        if cfg.fuse_mode in (1, 2):
            gf = dxp[:, 1 + kk]                                        # gradient of the fused token
            ds = (c["xd"] * gf[:, None, :]).sum(axis=-1)               # dL/ds_j for dropped j (weighted sum)
            wj = c["sd"]
            if cfg.fuse_mode == 2:                                     # f = u / S, u = sum_j s_j x_j, S = sum_j s_j:
                S = c["ssum"][:, None]                                 # df/dx_j = s_j / S, df/ds_j = (x_j - f) / S
                ds = (ds - (c["fused"] * gf).sum(axis=-1)[:, None]) / S
                wj = wj / S
            full[bidx, 1 + dropped] = wj[:, :, None] * gf[:, None, :]
            dA_cls = np.zeros((B, T))
            dA_cls[bidx, 1 + dropped] = ds / cfg.heads                 # every head gets 1/H of it
        dxp = full
    doc, g["attn.proj.weight"], g["attn.proj.bias"] = linear_bwd(dxp, c["oc"], params[p + "attn.proj.weight"])
    B, T, D = doc.shape
    H, d = cfg.heads, D // cfg.heads
    do = doc.reshape(B, T, H, d).transpose(0, 2, 1, 3)
    dq, dk, dv = attention_bwd(cfg, c["A"], c["q"], c["k"], c["v"], do, dA_cls)
    dqkv = np.stack([dq, dk, dv], axis=0).transpose(1, 3, 0, 2, 4).reshape(B, T, 3 * D)
    dy1, g["attn.qkv.weight"], g["attn.qkv.bias"] = linear_bwd(dqkv, c["y1"], params[p + "attn.qkv.weight"])
    dln1, g["norm1.weight"], g["norm1.bias"] = layer_norm_bwd(dy1, c["ln1"], params[p + "norm1.weight"])
    if want_param_grads:
        for name, val in g.items():
            grads[p + name] = val
    return (dxp + dln1) if need_dx else None


def forward(cfg, params, images, task_ids=None, forced_keep=None, keep_cache=False, forced_experts=None):
    """Forward with token dropping.  Returns a dict with logits (list per image), kept sets, caches."""
    B = images.shape[0]
    if task_ids is None:
        task_ids = np.zeros(B, dtype=np.int64)
    sched = token_schedule(cfg)
    x = embed(cfg, params, np.asarray(images, dtype=np.float64))
    t0 = min(cfg.trainable) if len(cfg.trainable) else cfg.depth
    fp8_upto = t0 if getattr(cfg, "frozen_fp8", 0) else 0          # dense blocks before the earliest trainable one
    caches, kept, margins, scores, tokens = [], [], [], [], []
    routing = {}
    di = 0
    for l in range(cfg.depth):
        ta, tf, k = sched[l]
        fk = None
        if k is not None and forced_keep is not None and forced_keep[di] is not None:
            fk = forced_keep[di]
        fe = forced_experts.get(l) if forced_experts else None
        x, c, info = block_fwd(cfg, params, l, x, task_ids, k, fk, fe, fp8=(l < fp8_upto and l not in cfg.moe_blocks))
        if l in cfg.moe_blocks:
            routing[l] = {"experts": c["moe"]["experts"], "own_experts": c["moe"]["own_experts"], "glogits": c["moe"]["glogits"]}
        if k is not None:
            kept.append(info["kept"])
            margins.append(info["margins"])
            scores.append(info["scores"])
            di += 1
        tokens.append((ta, x.shape[1]))
        caches.append(c if keep_cache else None)
    xn, lnf = layer_norm(x[:, 0], params["norm.weight"], params["norm.bias"], cfg.ln_eps)
    cmax = max(cfg.num_classes)
    logits = np.full((B, cmax), -np.inf)
    for t, ncls in enumerate(cfg.num_classes):
        sel = task_ids == t
        if sel.any():
            logits[sel, :ncls] = linear(xn[sel], params[f"head.{t}.weight"], params[f"head.{t}.bias"])
    return {"logits": logits, "kept": kept, "margins": margins, "scores": scores, "tokens": tokens,
            "caches": caches, "xn": xn, "lnf": lnf, "x_last": x, "task_ids": task_ids, "routing": routing}


def cross_entropy(logits, labels):
    """Mean over the batch of -log softmax(logits)[label]; padded classes hold -inf."""
    mx = logits.max(axis=-1, keepdims=True)
    e = np.exp(logits - mx)
    prob = e / e.sum(axis=-1, keepdims=True)
    B = logits.shape[0]
    loss = -np.mean(np.log(prob[np.arange(B), labels]))
    dlogits = prob.copy()
    dlogits[np.arange(B), labels] -= 1.0
    return loss, dlogits / B


def is_decayed(name):
    """Weight decay applies to matrices (and the CLS-free embeddings never train): not biases, not LayerNorm."""
    return name.endswith("weight") and "norm" not in name


def trainable_names(cfg, params):
    names = []
    for n in params:
        if n.startswith("blocks."):
            if int(n.split(".")[1]) in cfg.trainable:
                names.append(n)
        elif n.startswith("norm.") or n.startswith("head."):
            names.append(n)
    return names


def adamw(cfg, p, g, m, v, step, decay):
    m = cfg.beta1 * m + (1.0 - cfg.beta1) * g
    v = cfg.beta2 * v + (1.0 - cfg.beta2) * g * g
    mhat = m / (1.0 - cfg.beta1 ** step)
    vhat = v / (1.0 - cfg.beta2 ** step)
    new = p - cfg.lr * mhat / (np.sqrt(vhat) + cfg.eps)
    if decay:
        new = new - cfg.lr * cfg.weight_decay * p
    return new, m, v


def sgd_momentum(cfg, p, g, buf, decay):
    """SGD with momentum (Section 5, training hyper-parameters: the ViT-B runs use SGD with cosine decay; the paper
    gives neither momentum nor weight decay, so both are configuration values).  The weight decay is added to the
    gradient, the buffer accumulates it with factor momentum and starts at zero: d = g + wd p; buf <- mu buf + d;
    p <- p - lr buf."""
    d = g + (cfg.weight_decay * p if decay else 0.0)
    buf = cfg.momentum * buf + d
    return p - cfg.lr * buf, buf


def cosine_lr(lr_max, lr_min, t, total_steps):
    """Cosine learning-rate decay (Section 5, training hyper-parameters: "cosine learning rate decay"; the paper
    gives neither end value nor warm-up, so both ends are arguments and there is no warm-up): step t (from 0) of
    total_steps uses lr_min + (lr_max - lr_min) (1 + cos(pi t / total_steps)) / 2; from t = total_steps on the rate
    stays at lr_min."""
    tt = min(int(t), int(total_steps))
    return lr_min + 0.5 * (lr_max - lr_min) * (1.0 + math.cos(math.pi * tt / total_steps))


def train_steps(cfg, params, batches, lr_max, lr_min, total_steps, first_step=1, opt_state=None, forced_keeps=None):
    """A run of steps, one batch (images, labels, task_ids) each, under the cosine schedule: the step numbered
    `first_step + i` (optimiser steps count from 1) uses cosine_lr(.., t = first_step - 1 + i, ..).  Returns the list of
    per-step results of train_step."""
    out = []
    for i, (images, labels, task_ids) in enumerate(batches):
        step = first_step + i
        c = cfg.with_(lr=cosine_lr(lr_max, lr_min, step - 1, total_steps))
        r = train_step(c, params, images, labels, task_ids, forced_keep=forced_keeps[i] if forced_keeps else None,
                       opt_state=opt_state, step=step)
        params, opt_state = r["params"], r["opt_state"]
        out.append(r)
    return out


def train_step(cfg, params, images, labels, task_ids=None, forced_keep=None, opt_state=None, step=1, forced_experts=None):
    """One BSR fine-tuning step.  Returns loss, logits, gradients, updated parameters and moments."""
    fw = forward(cfg, params, images, task_ids, forced_keep, keep_cache=True, forced_experts=forced_experts)
    task_ids = fw["task_ids"]
    loss, dlogits = cross_entropy(fw["logits"], np.asarray(labels))
    grads = {}
    dxn = np.zeros_like(fw["xn"])
    for t, ncls in enumerate(cfg.num_classes):                # each image uses its task's head
        sel = task_ids == t
        dl = dlogits[sel, :ncls]
        dxn[sel], grads[f"head.{t}.weight"], grads[f"head.{t}.bias"] = linear_bwd(
            dl, fw["xn"][sel], params[f"head.{t}.weight"])
    dcls, grads["norm.weight"], grads["norm.bias"] = layer_norm_bwd(dxn, fw["lnf"], params["norm.weight"])
    t0 = min(cfg.trainable) if len(cfg.trainable) else cfg.depth
    dx = np.zeros_like(fw["x_last"])
    dx[:, 0] = dcls
    for l in range(cfg.depth - 1, t0 - 1, -1):               # nothing earlier than the first trainable block
        dx = block_bwd(cfg, params, l, dx, fw["caches"][l], task_ids, grads,
                       want_param_grads=(l in cfg.trainable), need_dx=(l > t0))
    names = trainable_names(cfg, params)
    if opt_state is None:
        opt_state = {"m": {n: np.zeros_like(params[n]) for n in names},
                     "v": {n: np.zeros_like(params[n]) for n in names}}
    new_params = dict(params)
    new_m, new_v = {}, {}
    for n in names:
        if getattr(cfg, "optimizer", "adamw") == "sgd":      # the momentum buffer takes the place of m, v stays zero
            new_params[n], new_m[n] = sgd_momentum(cfg, params[n], grads[n], opt_state["m"][n], is_decayed(n))
            new_v[n] = opt_state["v"][n]
        else:
            new_params[n], new_m[n], new_v[n] = adamw(cfg, params[n], grads[n], opt_state["m"][n],
                                                      opt_state["v"][n], step, is_decayed(n))
    fw.pop("caches")
    return {"loss": loss, "logits": fw["logits"], "grads": grads, "params": new_params,
            "opt_state": {"m": new_m, "v": new_v}, "kept": fw["kept"], "margins": fw["margins"],
            "scores": fw["scores"], "tokens": fw["tokens"], "routing": fw["routing"]}


def gather_fuse(xp, kept, dropped, s, fuse_mode=1):
    """Stand-alone compaction of one batch: xp [B, 1+M, D], index lists per image, scores s [B, M]."""
    rows = [xp[:, :1], np.take_along_axis(xp[:, 1:], kept[:, :, None], axis=1)]
    if fuse_mode in (1, 2) and dropped.shape[1] > 0:
        xd = np.take_along_axis(xp[:, 1:], dropped[:, :, None], axis=1)
        sd = np.take_along_axis(s, dropped, axis=1)
        fused = (sd[:, :, None] * xd).sum(axis=1, keepdims=True)
        rows.append(fused / sd.sum(axis=1)[:, None, None] if fuse_mode == 2 else fused)
    return np.concatenate(rows, axis=1)
