"""ctypes binding of libbsr.so: the same entry points as include/bsr.h, argument marshalling only.

PyTorch supplies device memory and streams; every step of the path runs in the library's
kernels.  There is no fallback: if the library is missing, loading raises.
"""

from __future__ import annotations

import ctypes as C
import os
from typing import Dict, Optional, Sequence

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
# BSR_LIBRARY=checked selects the build with device-side index checks (python -m paper_2405_10951_b200.build --checked)
LIB_PATH = os.path.join(_HERE, "libbsr_checked.so" if os.environ.get("BSR_LIBRARY") == "checked" else "libbsr.so")

BSR_OK = 0
DTYPE_FP32, DTYPE_BF16 = 0, 1
MAX_DROPS, MAX_TASKS, MAX_DEPTH = 8, 4, 32

STATUS_NAMES = {0: "BSR_OK", -1: "BSR_ERR_INVALID_ARG", -2: "BSR_ERR_UNSUPPORTED", -3: "BSR_ERR_WORKSPACE_TOO_SMALL",
                -4: "BSR_ERR_CUDA", -5: "BSR_ERR_DEVICE_TIMEOUT", -6: "BSR_ERR_NONFINITE", -7: "BSR_ERR_MEMORY_GUARD",
                -8: "BSR_ERR_DEVICE_CHECK"}

EXPORTS = ["bsr_token_schedule", "bsr_workspace_bytes", "bsr_create", "bsr_destroy", "bsr_last_error", "bsr_set_param",
           "bsr_get_tensor", "bsr_set_lr", "bsr_set_step", "bsr_train_step", "bsr_train_steps", "bsr_train_step_host", "bsr_forward_backward", "bsr_grad_buffer", "bsr_optimizer_step", "bsr_eval_forward", "bsr_get_footprint",
           "bsr_sync_status", "bsr_selftest_wait_expiry", "bsr_set_gemm_mode", "bsr_set_graph_mode", "bsr_profile_enable", "bsr_profile_read", "bsr_profile_launches", "bsr_token_select", "bsr_gather_fuse", "bsr_linear_forward", "bsr_linear_forward_e4m3", "bsr_linear_backward",
           "bsr_linear_backward_static", "bsr_static_last_error", "bsr_attention_forward", "bsr_attention_backward"]


class bsr_dims(C.Structure):
    _fields_ = [("image_size", C.c_int32), ("patch_size", C.c_int32), ("in_chans", C.c_int32),
                ("dim", C.c_int32), ("heads", C.c_int32), ("depth", C.c_int32), ("mlp_hidden", C.c_int32),
                ("num_tasks", C.c_int32), ("num_classes", C.c_int32 * MAX_TASKS),
                ("moe_experts", C.c_int32), ("moe_top_k", C.c_int32), ("moe_block_mask", C.c_uint32),
                ("dtype", C.c_int32), ("ln_eps", C.c_float)]


class bsr_config(C.Structure):
    _fields_ = [("dims", bsr_dims), ("trainable_mask", C.c_uint32), ("n_drop", C.c_int32),
                ("drop_block", C.c_int32 * MAX_DROPS), ("keep_num", C.c_int32 * MAX_DROPS),
                ("keep_den", C.c_int32 * MAX_DROPS), ("fuse_mode", C.c_int32),
                ("lr", C.c_float), ("beta1", C.c_float), ("beta2", C.c_float), ("eps", C.c_float),
                ("weight_decay", C.c_float), ("max_batch", C.c_int32), ("optimizer", C.c_int32), ("momentum", C.c_float),
                ("frozen_fp8", C.c_int32)]


class bsr_footprint(C.Structure):
    _fields_ = [(n, C.c_uint64) for n in ("workspace_bytes", "weight_bytes", "master_bytes", "optimizer_bytes",
                                           "grad_bytes", "saved_activation_bytes", "scratch_bytes",
                                           "paper_activation_bytes", "trainable_params")] + [("block_saved_bytes", C.c_uint64 * MAX_DEPTH)]


class bsr_profile(C.Structure):
    _fields_ = [("kernel_launches", C.c_uint64), ("gemm_launches", C.c_uint64), ("gemm_flops", C.c_double), ("gemm_ms", C.c_double),
                ("graph_captures", C.c_uint64)]


class bsr_lr_schedule(C.Structure):
    _fields_ = [("lr_max", C.c_float), ("lr_min", C.c_float), ("total_steps", C.c_int64)]


class BsrError(RuntimeError):
    def __init__(self, status: int, message: str):
        super().__init__(f"{STATUS_NAMES.get(status, status)}: {message}")
        self.status = status


_lib = None


def lib() -> C.CDLL:
    """Loads libbsr.so (once).  Raises if it has not been built: there is no other path."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise RuntimeError(f"{LIB_PATH} is missing: build it with `python -m paper_2405_10951_b200.build` "
                               "(nvcc, sm_100a); there is no CPU or PyTorch fallback")
        L = C.CDLL(LIB_PATH)
        vp, i32, f32p, i32p = C.c_void_p, C.c_int32, C.c_void_p, C.c_void_p
        L.bsr_token_schedule.argtypes = [C.POINTER(bsr_config), C.POINTER(C.c_int32), C.POINTER(C.c_int32), C.POINTER(C.c_int32)]
        L.bsr_workspace_bytes.argtypes = [C.POINTER(bsr_config), C.POINTER(C.c_size_t)]
        L.bsr_create.argtypes = [C.POINTER(bsr_config), vp, C.c_size_t, C.POINTER(vp)]
        L.bsr_destroy.argtypes = [vp]
        L.bsr_last_error.argtypes = [vp]
        L.bsr_last_error.restype = C.c_char_p
        L.bsr_static_last_error.restype = C.c_char_p
        L.bsr_set_param.argtypes = [vp, C.c_char_p, vp, C.c_size_t, i32, i32, vp]
        L.bsr_get_tensor.argtypes = [vp, C.c_char_p, f32p, C.c_size_t, vp]
        L.bsr_set_lr.argtypes = [vp, C.c_float]
        L.bsr_set_step.argtypes = [vp, C.c_int64]
        L.bsr_train_step.argtypes = [vp, vp, i32p, i32p, i32, vp, f32p, i32p]
        L.bsr_train_steps.argtypes = [vp, vp, i32p, i32p, i32, i32, C.POINTER(bsr_lr_schedule), vp, f32p, i32p]
        L.bsr_train_step_host.argtypes = [vp, vp, i32p, i32p, i32, vp, f32p, i32p]
        L.bsr_forward_backward.argtypes = [vp, vp, i32p, i32p, i32, vp, f32p, i32p]
        L.bsr_grad_buffer.argtypes = [vp, C.POINTER(C.c_void_p), C.POINTER(C.c_size_t)]
        L.bsr_optimizer_step.argtypes = [vp, vp]
        L.bsr_eval_forward.argtypes = [vp, vp, i32p, i32, vp, f32p, i32p]
        L.bsr_get_footprint.argtypes = [vp, C.POINTER(bsr_footprint)]
        L.bsr_sync_status.argtypes = [vp, vp]
        L.bsr_selftest_wait_expiry.argtypes = [vp, C.c_uint64, vp]
        L.bsr_set_gemm_mode.argtypes = [vp, i32]
        L.bsr_set_graph_mode.argtypes = [vp, i32]
        L.bsr_profile_enable.argtypes = [vp, i32]
        L.bsr_profile_read.argtypes = [vp, vp, C.POINTER(bsr_profile)]
        L.bsr_profile_launches.argtypes = [vp, vp, i32, C.POINTER(C.c_double), C.POINTER(C.c_float), C.POINTER(C.c_int32)]
        L.bsr_token_select.argtypes = [f32p, i32, i32, i32, i32, f32p, i32p, i32p, vp]
        L.bsr_gather_fuse.argtypes = [vp, i32, i32, i32, i32, i32, i32p, i32p, f32p, i32, vp, vp]
        L.bsr_linear_forward.argtypes = [vp, vp, f32p, vp, vp, i32, i32, i32, i32, i32, i32, vp]
        L.bsr_linear_forward_e4m3.argtypes = [vp, vp, f32p, vp, i32, i32, i32, i32, vp, C.c_size_t, vp]
        L.bsr_linear_backward.argtypes = [vp, vp, vp, vp, f32p, i32, i32, i32, i32, i32, f32p, C.c_size_t, vp]
        L.bsr_linear_backward_static.argtypes = [vp, vp, vp, vp, f32p, i32, i32, i32, vp]
        L.bsr_static_last_error.argtypes = []
        L.bsr_attention_forward.argtypes = [vp, i32, i32, i32, i32, i32, vp, f32p, f32p, i32, vp]
        L.bsr_attention_backward.argtypes = [vp, vp, f32p, f32p, i32, i32, i32, i32, i32, vp, f32p, i32, vp]
        for name in EXPORTS:
            if name not in ("bsr_last_error", "bsr_static_last_error"):
                getattr(L, name).restype = C.c_int32
        _lib = L
    return _lib


def _check(status: int, handle=None):
    if status != BSR_OK:
        msg = lib().bsr_last_error(handle)
        raise BsrError(status, msg.decode() if msg else "")


def make_config(cfg, max_batch: Optional[int] = None) -> bsr_config:
    """Translates a synth.Config-like object (attributes only) into the C struct."""
    c = bsr_config()
    d = c.dims
    d.image_size, d.patch_size, d.in_chans = cfg.image_size, cfg.patch_size, cfg.in_chans
    d.dim, d.heads, d.depth, d.mlp_hidden = cfg.dim, cfg.heads, cfg.depth, cfg.mlp_hidden
    d.num_tasks = len(cfg.num_classes)
    for i, n in enumerate(cfg.num_classes):
        d.num_classes[i] = n
    d.moe_experts, d.moe_top_k = cfg.moe_experts, cfg.moe_top_k
    d.moe_block_mask = sum(1 << l for l in cfg.moe_blocks)
    d.dtype = DTYPE_FP32 if cfg.dtype == "fp32" else DTYPE_BF16
    d.ln_eps = cfg.ln_eps
    c.trainable_mask = sum(1 << l for l in cfg.trainable)
    c.n_drop = len(cfg.drop_blocks)
    for i, l in enumerate(cfg.drop_blocks):
        c.drop_block[i], c.keep_num[i], c.keep_den[i] = l, cfg.keep_num, cfg.keep_den
    c.fuse_mode = cfg.fuse_mode
    c.lr, c.beta1, c.beta2, c.eps, c.weight_decay = cfg.lr, cfg.beta1, cfg.beta2, cfg.eps, cfg.weight_decay
    c.max_batch = cfg.batch if max_batch is None else max_batch
    c.optimizer = 1 if getattr(cfg, "optimizer", "adamw") == "sgd" else 0
    c.momentum = float(getattr(cfg, "momentum", 0.9))
    c.frozen_fp8 = int(getattr(cfg, "frozen_fp8", 0))
    return c


# ---- host-only calls ---------------------------------------------------------------------------
def bsr_token_schedule(c: bsr_config):
    n = c.dims.depth
    ta, tf, k = (C.c_int32 * MAX_DEPTH)(), (C.c_int32 * MAX_DEPTH)(), (C.c_int32 * MAX_DEPTH)()
    _check(lib().bsr_token_schedule(C.byref(c), ta, tf, k))
    return list(ta[:max(n, 0)]), list(tf[:max(n, 0)]), list(k[:max(n, 0)])


def bsr_workspace_bytes(c: bsr_config) -> int:
    out = C.c_size_t(0)
    _check(lib().bsr_workspace_bytes(C.byref(c), C.byref(out)))
    return out.value


# ---- device calls (torch tensors give pointers and the current stream) --------------------------
def _ptr(t):
    return None if t is None else C.c_void_p(t.data_ptr())


def _stream():
    import torch
    return C.c_void_p(torch.cuda.current_stream().cuda_stream)


def bsr_token_select(p, k: int):
    """p: float32 CUDA tensor [B, H, M].  Returns (scores [B, M], kept [B, k], dropped [B, M-k])."""
    import torch
    B, H, M = p.shape
    scores = torch.empty((B, M), dtype=torch.float32, device=p.device)
    kept = torch.empty((B, k), dtype=torch.int32, device=p.device)
    dropped = torch.empty((B, M - k), dtype=torch.int32, device=p.device)
    _check(lib().bsr_token_select(_ptr(p), B, H, M, k, _ptr(scores), _ptr(kept), _ptr(dropped), _stream()))
    return scores, kept, dropped


def bsr_gather_fuse(x, kept, dropped, scores, fuse_mode: int = 1, out=None):
    import torch
    B, T, D = x.shape
    M, k = T - 1, kept.shape[1]
    f = 1 if (fuse_mode in (1, 2) and k < M) else 0
    if out is None:
        out = torch.empty((B, 1 + k + f, D), dtype=x.dtype, device=x.device)
    dt = DTYPE_FP32 if x.dtype == torch.float32 else DTYPE_BF16
    _check(lib().bsr_gather_fuse(_ptr(x), dt, B, M, D, k, _ptr(kept), _ptr(dropped), _ptr(scores), fuse_mode, _ptr(out), _stream()))
    return out


def bsr_linear_forward(x, w, bias=None, residual=None, act_gelu: bool = False, use_tensor_cores: bool = False):
    import torch
    m, k = x.shape
    n = w.shape[0]
    y = torch.empty((m, n), dtype=x.dtype, device=x.device)
    dt = DTYPE_FP32 if x.dtype == torch.float32 else DTYPE_BF16
    _check(lib().bsr_linear_forward(_ptr(x), _ptr(w), _ptr(bias), _ptr(residual), _ptr(y), m, n, k, dt, int(act_gelu),
                                    int(use_tensor_cores), _stream()))
    return y


def bsr_linear_forward_e4m3(x, w, bias=None, act_gelu: bool = False):
    """y = act(x W^T + bias) with the rows of x and W rounded to E4M3 (bf16 tensors in, bf16 out)."""
    import torch
    m, k = x.shape
    n = w.shape[0]
    y = torch.empty((m, n), dtype=torch.bfloat16, device=x.device)
    nbytes = m * k + n * k + 4 * (m + n) + 2048
    scratch = torch.empty(nbytes + 256, dtype=torch.uint8, device=x.device)
    base = (scratch.data_ptr() + 255) & ~255
    _check(lib().bsr_linear_forward_e4m3(_ptr(x), _ptr(w), _ptr(bias), _ptr(y), m, n, k, int(act_gelu), C.c_void_p(base), nbytes, _stream()))
    return y


def bsr_linear_backward(x, w, dy, use_tensor_cores: bool = False, workspace=None):
    """Returns (dx [m, k] in x's dtype, dw [n, k] float32)."""
    import torch
    m, k = x.shape
    n = w.shape[0]
    dx = torch.empty((m, k), dtype=x.dtype, device=x.device)
    dw = torch.empty((n, k), dtype=torch.float32, device=x.device)
    dt = DTYPE_FP32 if x.dtype == torch.float32 else DTYPE_BF16
    _check(lib().bsr_linear_backward(_ptr(x), _ptr(w), _ptr(dy), _ptr(dx), _ptr(dw), m, n, k, dt, int(use_tensor_cores),
                                     _ptr(workspace), 0 if workspace is None else workspace.numel(), _stream()))
    return dx, dw


def bsr_linear_backward_static(x, w, dy, dx=None, dw=None):
    """Linear backward through the entry point that allocates nothing: the split-reduction scratch is a
    fixed array inside the library.  Pass dx/dw to reuse output tensors.  Returns (dx, dw)."""
    import torch
    m, k = x.shape
    n = w.shape[0]
    if dx is None:
        dx = torch.empty((m, k), dtype=x.dtype, device=x.device)
    if dw is None:
        dw = torch.empty((n, k), dtype=torch.float32, device=x.device)
    st = lib().bsr_linear_backward_static(_ptr(x), _ptr(w), _ptr(dy), _ptr(dx), _ptr(dw), m, n, k, _stream())
    if st != BSR_OK:
        raise BsrError(st, lib().bsr_static_last_error().decode())
    return dx, dw


def bsr_attention_forward(qkv, heads: int, want_cls_prob: bool = True, use_tensor_cores: bool = False, want_lse: bool = False):
    """qkv: CUDA tensor [B, T, 3, H, d].  Returns (out [B, T, H*d], cls_prob [B, H, T-1] or None), and with want_lse
    also the log of every row's softmax denominator [B, H, T]."""
    import torch
    B, T, three, H, d = qkv.shape
    assert three == 3 and H == heads
    out = torch.empty((B, T, H * d), dtype=qkv.dtype, device=qkv.device)
    cp = torch.empty((B, H, T - 1), dtype=torch.float32, device=qkv.device) if want_cls_prob else None
    lse = torch.empty((B, H, T), dtype=torch.float32, device=qkv.device) if want_lse else None
    dt = DTYPE_FP32 if qkv.dtype == torch.float32 else DTYPE_BF16
    _check(lib().bsr_attention_forward(_ptr(qkv), dt, B, T, H, d, _ptr(out), _ptr(cp), _ptr(lse), int(use_tensor_cores), _stream()))
    return (out, cp, lse) if want_lse else (out, cp)


def bsr_attention_backward(qkv, dout, lse, score_grad=None, use_tensor_cores: bool = False, out=None):
    """qkv [B, T, 3, H, d], dout [B, T, H*d] (same dtype), lse [B, H, T] float32 from bsr_attention_forward,
    score_grad optional [B, T-1] float32.  Returns dqkv [B, T, 3, H, d]."""
    import torch
    B, T, three, H, d = qkv.shape
    assert three == 3 and tuple(dout.shape) == (B, T, H * d) and dout.dtype == qkv.dtype
    dqkv = out if out is not None else torch.empty_like(qkv)
    delta = None if use_tensor_cores else torch.empty(B * H * T, dtype=torch.float32, device=qkv.device)
    dt = DTYPE_FP32 if qkv.dtype == torch.float32 else DTYPE_BF16
    _check(lib().bsr_attention_backward(_ptr(qkv), _ptr(dout), _ptr(lse), _ptr(score_grad), dt, B, T, H, d, _ptr(dqkv), _ptr(delta),
                                        int(use_tensor_cores), _stream()))
    return dqkv


class Engine:
    """Owns a handle and its workspace tensor; thin convenience over the bsr_* calls."""

    def __init__(self, cfg, max_batch: Optional[int] = None, device: str = "cuda:0"):
        import torch
        self.torch = torch
        self.cfg = cfg
        self.device = torch.device(device)
        self.c = make_config(cfg, max_batch)
        self.ta, self.tf, self.k = bsr_token_schedule(self.c)
        nbytes = bsr_workspace_bytes(self.c)
        torch.cuda.set_device(self.device)
        self.workspace = torch.empty(nbytes + 256, dtype=torch.uint8, device=self.device)
        base = self.workspace.data_ptr()
        self._ws_ptr = (base + 255) & ~255
        h = C.c_void_p()
        _check(lib().bsr_create(C.byref(self.c), C.c_void_p(self._ws_ptr), nbytes, C.byref(h)))
        self.h = h
        self.cmax = max(cfg.num_classes)
        self.storage_dtype = torch.float32 if cfg.dtype == "fp32" else torch.bfloat16
        self.kept_counts = [k for k in self.k if k >= 0]

    def close(self):
        if getattr(self, "h", None):
            lib().bsr_destroy(self.h)
            self.h = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    # -- parameters --
    def set_param(self, name: str, value):
        """value: a numpy array (float32 or any float type: passed from host memory as float32), a CPU tensor
        (float32 or bfloat16, passed from host memory as it is) or a CUDA tensor (float32 or bfloat16)."""
        torch = self.torch
        if not torch.is_tensor(value):
            value = torch.as_tensor(np.ascontiguousarray(value, dtype=np.float32))
        if value.dtype not in (torch.float32, torch.bfloat16):
            value = value.to(torch.float32)
        t = value.contiguous()
        dt = DTYPE_FP32 if t.dtype == torch.float32 else DTYPE_BF16
        _check(lib().bsr_set_param(self.h, name.encode(), _ptr(t), t.numel(), dt, int(t.is_cuda), _stream()), self.h)
        torch.cuda.current_stream().synchronize()

    def set_params(self, params: Dict[str, np.ndarray]):
        for name, v in params.items():
            self.set_param(name, v)

    def get_tensor(self, name: str, shape: Sequence[int]):
        n = int(np.prod(shape))
        out = self.torch.empty(n, dtype=self.torch.float32, device=self.device)
        _check(lib().bsr_get_tensor(self.h, name.encode(), _ptr(out), n, _stream()), self.h)
        return out.reshape(tuple(shape))

    def set_lr(self, lr: float):
        _check(lib().bsr_set_lr(self.h, lr), self.h)

    def set_step(self, n: int):
        _check(lib().bsr_set_step(self.h, n), self.h)

    # -- the step --
    def images_to_device(self, images: np.ndarray):
        t = self.torch.as_tensor(np.ascontiguousarray(images, dtype=np.float32))
        return t.to(self.device).to(self.storage_dtype).contiguous()

    def train_step(self, images, labels, task_ids=None, want_kept: bool = True, out=None):
        """images: CUDA tensor [B, C, S, S] in the storage dtype; labels/task_ids: int32 CUDA tensors.
        Returns (loss tensor [1], list of kept-index tensors [B, K_i] or None).  Does not synchronise.
        `out` = (loss, kept_flat) from an earlier call reuses those output buffers: with identical pointers the
        library replays its captured graph of the step instead of capturing a new one."""
        torch = self.torch
        B = images.shape[0]
        if out is not None:
            loss, kept = out
        else:
            loss = torch.empty(1, dtype=torch.float32, device=self.device)
            kept = None
            if want_kept and self.kept_counts:
                kept = torch.empty(B * sum(self.kept_counts), dtype=torch.int32, device=self.device)
        _check(lib().bsr_train_step(self.h, _ptr(images), _ptr(labels), _ptr(task_ids), B, _stream(), _ptr(loss), _ptr(kept)), self.h)
        self.last_out = (loss, kept)
        return loss, self._split_kept(kept, B)

    def train_steps(self, images, labels, task_ids=None, lr_max: float = 1e-3, lr_min: float = 0.0, total_steps: int = 1,
                    want_kept: bool = True, out=None):
        """images: CUDA tensor [n, B, C, S, S] in the storage dtype; labels/task_ids: int32 CUDA tensors [n, B].
        Returns (losses tensor [n], kept-index tensors of the last step).  Does not synchronise."""
        torch = self.torch
        n, B = images.shape[0], images.shape[1]
        if out is not None:
            losses, kept = out
        else:
            losses = torch.empty(n, dtype=torch.float32, device=self.device)
            kept = torch.empty(B * sum(self.kept_counts), dtype=torch.int32, device=self.device) if (want_kept and self.kept_counts) else None
        sched = bsr_lr_schedule(lr_max, lr_min, total_steps)
        _check(lib().bsr_train_steps(self.h, _ptr(images), _ptr(labels), _ptr(task_ids), B, n, C.byref(sched), _stream(),
                                     _ptr(losses), _ptr(kept)), self.h)
        self.last_out = (losses, kept)
        return losses, self._split_kept(kept, B)

    def forward_backward(self, images, labels, task_ids=None, want_kept: bool = True, out=None):
        """The step without its update: gradients of the local batch mean are left in the gradient buffer."""
        torch = self.torch
        B = images.shape[0]
        if out is not None:
            loss, kept = out
        else:
            loss = torch.empty(1, dtype=torch.float32, device=self.device)
            kept = torch.empty(B * sum(self.kept_counts), dtype=torch.int32, device=self.device) if (want_kept and self.kept_counts) else None
        _check(lib().bsr_forward_backward(self.h, _ptr(images), _ptr(labels), _ptr(task_ids), B, _stream(), _ptr(loss), _ptr(kept)), self.h)
        self.last_out = (loss, kept)
        return loss, self._split_kept(kept, B)

    def grad_buffer(self):
        """The flat float32 gradient buffer as a tensor view of the workspace (to be all-reduced in place)."""
        p, n = C.c_void_p(), C.c_size_t()
        _check(lib().bsr_grad_buffer(self.h, C.byref(p), C.byref(n)), self.h)
        off = p.value - self.workspace.data_ptr()
        return self.workspace[off: off + 4 * n.value].view(self.torch.float32)

    def optimizer_step(self):
        _check(lib().bsr_optimizer_step(self.h, _stream()), self.h)

    def train_step_host(self, images, labels, task_ids=None, loss=None, kept=None):
        """images / labels / task_ids / loss / kept: CPU tensors (pinned for overlap); images in the storage dtype.
        Does not synchronise: `loss` holds the step's loss once the current stream has finished this call's work."""
        torch = self.torch
        B = images.shape[0]
        if loss is None:
            loss = torch.empty(1, dtype=torch.float32).pin_memory()
        _check(lib().bsr_train_step_host(self.h, _ptr(images), _ptr(labels), _ptr(task_ids), B, _stream(), _ptr(loss), _ptr(kept)), self.h)
        return loss, (self._split_kept(kept, B) if kept is not None else None)

    def eval_forward(self, images, task_ids=None, want_kept: bool = True):
        torch = self.torch
        B = images.shape[0]
        logits = torch.empty((B, self.cmax), dtype=torch.float32, device=self.device)
        kept = None
        if want_kept and self.kept_counts:
            kept = torch.empty(B * sum(self.kept_counts), dtype=torch.int32, device=self.device)
        _check(lib().bsr_eval_forward(self.h, _ptr(images), _ptr(task_ids), B, _stream(), _ptr(logits), _ptr(kept)), self.h)
        return logits, self._split_kept(kept, B)

    def _split_kept(self, kept, B):
        if kept is None:
            return None
        out, off = [], 0
        for k in self.kept_counts:
            out.append(kept[off: off + B * k].view(B, k))
            off += B * k
        return out

    def sync_status(self):
        _check(lib().bsr_sync_status(self.h, _stream()), self.h)

    def selftest_wait_expiry(self, limit_ns: int = 1_000_000):
        _check(lib().bsr_selftest_wait_expiry(self.h, limit_ns, _stream()), self.h)

    def set_gemm_mode(self, mode: int):
        _check(lib().bsr_set_gemm_mode(self.h, mode), self.h)

    def set_graph_mode(self, on: bool):
        _check(lib().bsr_set_graph_mode(self.h, int(on)), self.h)

    def profile_enable(self, time_gemms: bool):
        _check(lib().bsr_profile_enable(self.h, int(time_gemms)), self.h)

    def profile_read(self) -> Dict[str, float]:
        p = bsr_profile()
        _check(lib().bsr_profile_read(self.h, _stream(), C.byref(p)), self.h)
        return {"kernel_launches": int(p.kernel_launches), "gemm_launches": int(p.gemm_launches),
                "gemm_flops": float(p.gemm_flops), "gemm_ms": float(p.gemm_ms), "graph_captures": int(p.graph_captures)}

    def profile_launches(self, capacity: int = 4096):
        fl, ms, n = (C.c_double * capacity)(), (C.c_float * capacity)(), C.c_int32(0)
        _check(lib().bsr_profile_launches(self.h, _stream(), capacity, fl, ms, C.byref(n)), self.h)
        k = min(n.value, capacity)
        return [(fl[i], ms[i]) for i in range(k)]

    def footprint(self) -> Dict[str, int]:
        fp = bsr_footprint()
        _check(lib().bsr_get_footprint(self.h, C.byref(fp)), self.h)
        out = {n: int(getattr(fp, n)) for n, _ in bsr_footprint._fields_ if n != "block_saved_bytes"}
        out["block_saved_bytes"] = [int(x) for x in fp.block_saved_bytes[: self.cfg.depth]]
        return out
