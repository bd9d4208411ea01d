"""A ViT with BSR token dropping written with stock torch ops in float64 (test-only).

It is an independent statement of the same forward function: library layer_norm, linear,
gelu, softmax, cross_entropy and topk, with gradients from autograd.  The oracle's
hand-written forward, selection and backward are pinned against it.
"""
import math

import torch
import torch.nn.functional as F


def run(cfg, params, images, labels, task_ids, keep_count_fn):
    P = {k: torch.tensor(v, dtype=torch.float64, requires_grad=True) for k, v in params.items()}
    x = torch.tensor(images, dtype=torch.float64)
    labels = torch.tensor(labels, dtype=torch.long)
    task = torch.tensor(task_ids, dtype=torch.long)
    B = x.shape[0]
    D, H = cfg.dim, cfg.heads
    d = D // H
    ps = cfg.patch_size
    x = F.unfold(x, kernel_size=ps, stride=ps).transpose(1, 2)      # [B, N, C*P*P], (c, row, col) order
    x = F.linear(x, P["patch_embed.weight"], P["patch_embed.bias"])
    x = torch.cat([P["cls_token"].expand(B, 1, D), x], dim=1) + P["pos_embed"]
    kept_all = []
    for l in range(cfg.depth):
        p = f"blocks.{l}."
        T = x.shape[1]
        y = F.layer_norm(x, (D,), P[p + "norm1.weight"], P[p + "norm1.bias"], cfg.ln_eps)
        qkv = F.linear(y, P[p + "attn.qkv.weight"], P[p + "attn.qkv.bias"]).view(B, T, 3, H, d).permute(2, 0, 3, 1, 4)
        att = torch.softmax(qkv[0] @ qkv[1].transpose(-1, -2) / math.sqrt(d), dim=-1)
        o = (att @ qkv[2]).transpose(1, 2).reshape(B, T, D)
        x = x + F.linear(o, P[p + "attn.proj.weight"], P[p + "attn.proj.bias"])
        if l in cfg.drop_blocks:
            M = T - 1
            k = keep_count_fn(M)
            s = att[:, :, 0, 1:].mean(dim=1)                         # [B, M]
            idx = torch.topk(s.detach(), k, dim=1).indices.sort(dim=1).values
            kept_all.append(idx.numpy())
            if k < M:
                body = x[:, 1:]
                rows = [x[:, :1], torch.gather(body, 1, idx[:, :, None].expand(B, k, D))]
                if cfg.fuse_mode in (1, 2):
                    mask = torch.ones(B, M, dtype=torch.float64)
                    mask.scatter_(1, idx, 0.0)
                    w = s * mask
                    if cfg.fuse_mode == 2:                           # weighted mean of the dropped tokens
                        w = w / w.sum(dim=1, keepdim=True)
                    rows.append((w[:, :, None] * body).sum(dim=1, keepdim=True))
                x = torch.cat(rows, dim=1)
        y = F.layer_norm(x, (D,), P[p + "norm2.weight"], P[p + "norm2.bias"], cfg.ln_eps)
        if l in cfg.moe_blocks:
            wg = P[p + "moe.gate.weight"][task]                      # [B, E, D]
            gl = torch.einsum("btd,bed->bte", y, wg)
            top = torch.topk(gl, cfg.moe_top_k, dim=-1)
            w = torch.softmax(top.values, dim=-1)
            out = torch.zeros_like(y)
            for e in range(cfg.moe_experts):
                he = F.gelu(F.linear(y, P[p + "moe.fc1.weight"][e], P[p + "moe.fc1.bias"][e]))
                ye = F.linear(he, P[p + "moe.fc2.weight"][e], P[p + "moe.fc2.bias"][e])
                we = (w * (top.indices == e)).sum(dim=-1, keepdim=True)
                out = out + we * ye
            x = x + out
        else:
            h = F.gelu(F.linear(y, P[p + "mlp.fc1.weight"], P[p + "mlp.fc1.bias"]))
            x = x + F.linear(h, P[p + "mlp.fc2.weight"], P[p + "mlp.fc2.bias"])
    xn = F.layer_norm(x[:, 0], (D,), P["norm.weight"], P["norm.bias"], cfg.ln_eps)
    losses = []
    logits = []
    for b in range(B):
        t = int(task[b])
        lg = F.linear(xn[b], P[f"head.{t}.weight"], P[f"head.{t}.bias"])
        logits.append(lg.detach().numpy())
        losses.append(F.cross_entropy(lg[None], labels[b:b + 1]))
    loss = torch.stack(losses).mean()
    loss.backward()
    grads = {k: (v.grad.numpy() if v.grad is not None else None) for k, v in P.items()}
    return float(loss.detach()), logits, grads, kept_all
