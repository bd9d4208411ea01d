"""Seeded synthetic workloads for the BSR fine-tuning step.

This module only *draws numbers and names shapes*.  It holds none of the method's
arithmetic (no token schedule, no attention, no selection), so that the CPU oracle
and the CUDA path can both be fed from it without sharing any computation.

Recipe (stands in for the paper's CIFAR/Flowers/Pets/Food images and ImageNet
pre-trained weights, Section 5 "Models and Datasets", which are not available):

* pixels: i.i.d. N(0, 1), NCHW;
* labels: i.i.d. uniform integers in [0, classes of the image's task);
* task ids: the first half of the batch is task 0, the second half task 1 (multitask only);
* matrices, CLS token, positional embedding, heads, gates: N(0, 0.02^2) re-drawn
  outside +-2 sigma; biases 0; LayerNorm weight 1, bias 0;
* draw order: images, labels, then parameters in the order of ``param_shapes``;
* for a bf16 configuration every pixel and parameter is rounded to the nearest
  bf16-representable value (ties to even), so both sides start from identical numbers.

The "peaked" variant multiplies the query and key rows of every QKV matrix by
gamma = sqrt(2.5 / (0.0004 * dim)), which gives attention logits a standard
deviation of about 2.5 (as in trained ViTs) and therefore wide top-k margins.
"""

from __future__ import annotations

from dataclasses import dataclass, replace, field
from typing import Dict, Tuple

import numpy as np


@dataclass(frozen=True)
class Config:
    name: str
    image_size: int
    patch_size: int
    dim: int
    heads: int
    depth: int
    mlp_hidden: int
    num_classes: Tuple[int, ...]
    batch: int
    trainable: Tuple[int, ...]            # 0-based block indices; head and final norm always train
    drop_blocks: Tuple[int, ...]          # 0-based token drop locations
    keep_num: int                         # keep rate = keep_num / keep_den at every location
    keep_den: int
    dtype: str = "bf16"                   # "fp32" or "bf16"
    in_chans: int = 3
    fuse_mode: int = 1                    # 0: dropped tokens vanish, 1: fused into one weighted token
    moe_experts: int = 0
    moe_top_k: int = 0
    moe_blocks: Tuple[int, ...] = ()
    ln_eps: float = 1e-6
    lr: float = 1e-4
    beta1: float = 0.9
    beta2: float = 0.999
    eps: float = 1e-8
    weight_decay: float = 0.05
    optimizer: str = "adamw"              # "adamw" or "sgd" (with momentum)
    momentum: float = 0.9
    frozen_fp8: int = 0                   # 1: the LayerNorm-fed linear layers of the blocks before the first trainable one run in E4M3
    seed: int = 0

    @property
    def num_patches(self) -> int:
        return (self.image_size // self.patch_size) ** 2

    @property
    def num_tasks(self) -> int:
        return len(self.num_classes)

    def with_(self, **kw) -> "Config":
        return replace(self, **kw)


# The five benchmark configurations (shapes of DeiT-S / ViT-B at 224 and 384, Section 5).
CONFIGS: Dict[str, Config] = {
    "tiny_fp32": Config("tiny_fp32", 32, 4, 192, 3, 6, 768, (10,), 8, (4, 5), (2,), 7, 10, dtype="fp32"),
    "deit_s": Config("deit_s", 224, 16, 384, 6, 12, 1536, (10,), 64, (8, 9, 10, 11), (3, 6, 9), 7, 10),
    "vit_b": Config("vit_b", 224, 16, 768, 12, 12, 3072, (100,), 128, (8, 9, 10, 11), (3, 6, 9), 7, 10),
    "vit_b_384": Config("vit_b_384", 384, 16, 768, 12, 12, 3072, (100,), 32, (10, 11), (3, 6, 9), 1, 2),
    "moe_vit_s": Config("moe_vit_s", 224, 16, 384, 6, 12, 1536, (10, 40), 64, (8, 9, 10, 11), (3, 6, 9), 7, 10,
                        moe_experts=16, moe_top_k=2, moe_blocks=(1, 3, 5, 7, 9, 11)),
}


def param_shapes(cfg: Config) -> Dict[str, Tuple[int, ...]]:
    """Parameter names and shapes, in draw order.  Linear weights are [out, in]."""
    D, F = cfg.dim, cfg.mlp_hidden
    pin = cfg.in_chans * cfg.patch_size * cfg.patch_size
    shapes: Dict[str, Tuple[int, ...]] = {}
    shapes["patch_embed.weight"] = (D, pin)      # input flattened as (channel, row in patch, column in patch)
    shapes["patch_embed.bias"] = (D,)
    shapes["cls_token"] = (D,)
    shapes["pos_embed"] = (cfg.num_patches + 1, D)
    for l in range(cfg.depth):
        p = f"blocks.{l}."
        shapes[p + "norm1.weight"] = (D,)
        shapes[p + "norm1.bias"] = (D,)
        shapes[p + "attn.qkv.weight"] = (3 * D, D)   # rows: all Q heads, all K heads, all V heads
        shapes[p + "attn.qkv.bias"] = (3 * D,)
        shapes[p + "attn.proj.weight"] = (D, D)
        shapes[p + "attn.proj.bias"] = (D,)
        shapes[p + "norm2.weight"] = (D,)
        shapes[p + "norm2.bias"] = (D,)
        if l in cfg.moe_blocks:
            E = cfg.moe_experts
            shapes[p + "moe.gate.weight"] = (cfg.num_tasks, E, D)
            shapes[p + "moe.fc1.weight"] = (E, F, D)
            shapes[p + "moe.fc1.bias"] = (E, F)
            shapes[p + "moe.fc2.weight"] = (E, D, F)
            shapes[p + "moe.fc2.bias"] = (E, D)
        else:
            shapes[p + "mlp.fc1.weight"] = (F, D)
            shapes[p + "mlp.fc1.bias"] = (F,)
            shapes[p + "mlp.fc2.weight"] = (D, F)
            shapes[p + "mlp.fc2.bias"] = (D,)
    shapes["norm.weight"] = (D,)
    shapes["norm.bias"] = (D,)
    for t, c in enumerate(cfg.num_classes):
        shapes[f"head.{t}.weight"] = (c, D)
        shapes[f"head.{t}.bias"] = (c,)
    return shapes


def round_to_bf16(a: np.ndarray) -> np.ndarray:
    """Nearest bf16-representable value (ties to even), returned as float64."""
    f = np.ascontiguousarray(a, dtype=np.float32)
    u = f.view(np.uint32).astype(np.uint64)
    u = (u + 0x7FFF + ((u >> 16) & 1)) & 0xFFFF0000
    return u.astype(np.uint32).view(np.float32).astype(np.float64).reshape(a.shape)


def to_bf16_bits(a: np.ndarray) -> np.ndarray:
    """uint16 bit patterns of values that are already bf16-representable."""
    f = np.ascontiguousarray(a, dtype=np.float32)
    return (f.view(np.uint32) >> 16).astype(np.uint16).reshape(a.shape)


def from_bf16_bits(b: np.ndarray) -> np.ndarray:
    u = np.ascontiguousarray(b, dtype=np.uint16).astype(np.uint32) << 16
    return u.view(np.float32).reshape(b.shape)


def _trunc_normal(rng: np.random.Generator, shape, std: float) -> np.ndarray:
    x = rng.standard_normal(shape)
    bad = np.abs(x) > 2.0
    while bad.any():
        x[bad] = rng.standard_normal(int(bad.sum()))
        bad = np.abs(x) > 2.0
    return x * std


def make_params(cfg: Config, rng: np.random.Generator, peaked: bool = False) -> Dict[str, np.ndarray]:
    params: Dict[str, np.ndarray] = {}
    for name, shape in param_shapes(cfg).items():
        if name.endswith("bias"):
            p = np.zeros(shape)
        elif ("norm" in name) and name.endswith("weight"):
            p = np.ones(shape)
        else:
            p = _trunc_normal(rng, shape, 0.02)
        params[name] = p
    if peaked:
        gamma = float(np.sqrt(2.5 / (0.0004 * cfg.dim)))
        for l in range(cfg.depth):
            params[f"blocks.{l}.attn.qkv.weight"][: 2 * cfg.dim] *= gamma
    if cfg.dtype == "bf16":
        params = {k: round_to_bf16(v) for k, v in params.items()}
    return params


def make_batch(cfg: Config, rng: np.random.Generator, batch: int | None = None):
    """images [B, C, S, S] float64, labels [B] int32, task_ids [B] int32."""
    B = cfg.batch if batch is None else batch
    images = rng.standard_normal((B, cfg.in_chans, cfg.image_size, cfg.image_size))
    if cfg.dtype == "bf16":
        images = round_to_bf16(images)
    task_ids = np.zeros(B, dtype=np.int32)
    if cfg.num_tasks > 1:
        per = -(-B // cfg.num_tasks)
        task_ids = np.minimum(np.arange(B) // per, cfg.num_tasks - 1).astype(np.int32)
    u = rng.random(B)
    ncls = np.asarray(cfg.num_classes)[task_ids]
    labels = np.minimum((u * ncls).astype(np.int32), ncls - 1).astype(np.int32)
    return images, labels, task_ids


def make_workload(cfg: Config, batch: int | None = None, peaked: bool = False, seed: int | None = None):
    """One seeded workload: (images, labels, task_ids, params)."""
    rng = np.random.default_rng(cfg.seed if seed is None else seed)
    images, labels, task_ids = make_batch(cfg, rng, batch)
    params = make_params(cfg, rng, peaked)
    return images, labels, task_ids, params


def make_scores(rng: np.random.Generator, batch: int, heads: int, m: int, ties: bool = False) -> np.ndarray:
    """CLS-row attention probabilities [B, H, M] (float32) for the stand-alone select tests.

    Rows are positive and sum to less than one (the CLS column holds the rest).  With
    ``ties`` the values are drawn from a handful of levels so that equal scores abound.
    """
    if ties:
        levels = rng.integers(1, 5, size=(batch, heads, m)).astype(np.float32)
        p = levels / np.float32(8 * m)
    else:
        z = rng.standard_normal((batch, heads, m + 1)) * 2.5
        e = np.exp(z - z.max(axis=-1, keepdims=True))
        p = (e / e.sum(axis=-1, keepdims=True))[..., 1:].astype(np.float32)
    return np.ascontiguousarray(p, dtype=np.float32)
