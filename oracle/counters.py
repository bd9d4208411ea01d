"""Analytic counters of the BSR paper: forward MACs and the fp32 activation-memory accounting.

TEST INFRASTRUCTURE ONLY (same rules as bsr_oracle.py).  These closed forms are what the
paper's tables print, so the tests can pin the token schedule (K = ceil(keep * M), one fused
token, MHSA on the incoming tokens and FFN on the reduced set) against printed numbers:

* forward MACs per image: Tables 3, 4 and 8 ("FLOPS (GMacs)", batch 128);
* stored activations per block in fp32: Table 1 (Q, K, V; softmax input; GELU input),
  Section 3.2 (a frozen block in the gradient path stores ~2.9 MB, a trainable one ~5.5 MB).
"""

from __future__ import annotations

from .bsr_oracle import token_schedule


def forward_macs(cfg) -> int:
    """Multiply-accumulates of one image's forward pass (patch embedding, blocks, head)."""
    D, F = cfg.dim, cfg.mlp_hidden
    n = cfg.num_patches
    macs = n * (cfg.in_chans * cfg.patch_size ** 2) * D
    for l, (ta, tf, _k) in enumerate(token_schedule(cfg)):
        macs += ta * D * 3 * D            # Q, K, V projections
        macs += 2 * ta * ta * D           # Q K^T and A V over all heads (Eq. 1)
        macs += ta * D * D                # output projection
        ffn = 2 * tf * D * F              # the two FFN layers, on the tokens that remain
        if l in cfg.moe_blocks:
            ffn = ffn * cfg.moe_top_k + tf * D * cfg.moe_experts
        macs += ffn
    macs += D * max(cfg.num_classes)
    return macs


def block_activation_bytes(cfg, ta: int, tf: int, trainable: bool, bytes_per_el: int = 4) -> int:
    """Activations one block keeps for the backward pass, in the paper's accounting (Table 1).

    Every block in the gradient path keeps the inputs of its non-linear layers: Q, K, V
    [H, T, L/H] x 3, the softmax input [H, T, T] and the GELU input [T, D_ffn * L].  A
    trainable block also keeps the input of each linear layer (Eq. 4): LayerNorm 1, QKV and
    projection at the MHSA token count; LayerNorm 2, FC1 (width L) and FC2 (width D_ffn * L)
    at the FFN token count.
    """
    D, F, H = cfg.dim, cfg.mlp_hidden, cfg.heads
    el = 3 * ta * D + H * ta * ta + tf * F
    if trainable:
        el += 3 * ta * D + 2 * tf * D + tf * F
    return el * bytes_per_el


def trainable_param_count(cfg) -> int:
    D, F = cfg.dim, cfg.mlp_hidden
    per_block = 2 * D + (3 * D * D + 3 * D) + (D * D + D) + 2 * D + (F * D + F) + (D * F + D)
    head = sum(c * D + c for c in cfg.num_classes)
    return len(cfg.trainable) * per_block + 2 * D + head


def train_memory_bytes(cfg, batch: int) -> int:
    """Estimated training memory: stored activations from the earliest trainable block on, plus trainable weights."""
    if not cfg.trainable:
        return 0
    t0 = min(cfg.trainable)
    total = 0
    for l, (ta, tf, _k) in enumerate(token_schedule(cfg)):
        if l >= t0:
            total += batch * block_activation_bytes(cfg, ta, tf, l in cfg.trainable)
    return total + 4 * trainable_param_count(cfg)
