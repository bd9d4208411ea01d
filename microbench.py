"""Stand-alone timing of single kernels of the BSR step through the C ABI.

    python microbench.py gemm --m 25216 --n 2304 --k 768 [--gelu] [--e4m3] [--mode 1|2] [--iters 20]
    python microbench.py backward --m 12800 --n 2304 --k 768
    python microbench.py select_gather --batch 4096 --heads 12 --tokens 197 --dim 768 --keep 0.7
    python microbench.py attention --batch 128 --heads 12 --tokens 197
    python microbench.py step --workload vit_b --batch 32 --iters 4

Each prints one JSON line with the time per launch (CUDA events on the current stream, after warm-up) and the
achieved TFLOP/s or GB/s on the kernel's algorithmic work.  Inputs are seeded and synthetic.
"""
from __future__ import annotations

import argparse
import json
import math

import os
import sys

import torch

sys.path.insert(0, os.path.dirname(os.path.abspath(__file__)))
from paper_2405_10951_b200 import binding as Bd  # noqa: E402


def timed(fn, iters, flush=None, reps=1):
    """Mean time of one call in ms.  reps > 1: that many calls back to back inside each event pair (a kernel shorter
    than the host's launch path is otherwise timed together with the launch gap); not combined with an L2 flush."""
    for _ in range(3):
        fn()
    torch.cuda.synchronize()
    if flush is not None:
        reps = 1
    total = 0.0
    for _ in range(iters):
        if flush is not None:
            flush.zero_()                       # evict the previous iteration's data from L2
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for _ in range(reps):
            fn()
        e1.record()
        torch.cuda.synchronize()
        total += e0.elapsed_time(e1) / reps
    return total / iters


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("what", choices=["gemm", "backward", "select_gather", "attention", "step"])
    ap.add_argument("--workload", default="vit_b")
    ap.add_argument("--m", type=int, default=25216)
    ap.add_argument("--n", type=int, default=2304)
    ap.add_argument("--k", type=int, default=768)
    ap.add_argument("--gelu", action="store_true")
    ap.add_argument("--residual", action="store_true")
    ap.add_argument("--e4m3", action="store_true", help="gemm: operands rounded to E4M3 row by row (the 8-bit prefix's product)")
    ap.add_argument("--mode", type=int, default=1)
    ap.add_argument("--iters", type=int, default=20)
    ap.add_argument("--batch", type=int, default=4096)
    ap.add_argument("--heads", type=int, default=12)
    ap.add_argument("--tokens", type=int, default=197)
    ap.add_argument("--dim", type=int, default=768)
    ap.add_argument("--keep", type=float, default=0.7)
    ap.add_argument("--dtype", default="bf16", choices=["bf16", "fp32"])
    ap.add_argument("--flush-l2", action="store_true")
    ap.add_argument("--backward", action="store_true", help="attention: also time the backward pass (--mode 0: without tensor cores)")
    a = ap.parse_args()
    torch.manual_seed(0)
    dev = "cuda"
    flush = torch.empty(256 * 1024 * 1024, dtype=torch.uint8, device=dev) if a.flush_l2 else None
    out = {"kernel": a.what}
    if a.what == "step":
        # whole fine-tuning steps of a named workload at a chosen batch: the launch sequence a profiler is pointed at
        from paper_2405_10951_b200 import synth
        cfg = synth.CONFIGS[a.workload]
        cfg = cfg.with_(batch=min(a.batch, cfg.batch))
        images, labels, task_ids, params = synth.make_workload(cfg)
        eng = Bd.Engine(cfg)
        eng.set_params(params)
        img, lab = eng.images_to_device(images), torch.as_tensor(labels).cuda()
        tid = torch.as_tensor(task_ids).cuda() if cfg.num_tasks > 1 else None
        eng.set_graph_mode(False)
        ms = timed(lambda: eng.train_step(img, lab, tid, want_kept=False), a.iters)
        eng.sync_status()
        out.update(workload=cfg.name, batch=cfg.batch, ms_per_step=ms, images_per_s=cfg.batch / ms * 1e3)
    elif a.what == "gemm":
        x = torch.randn(a.m, a.k, device=dev).bfloat16()
        w = (torch.randn(a.n, a.k, device=dev) / math.sqrt(a.k)).bfloat16()
        b = torch.randn(a.n, device=dev)
        r = torch.randn(a.m, a.n, device=dev).bfloat16() if a.residual else None
        if a.e4m3:
            ms = timed(lambda: Bd.bsr_linear_forward_e4m3(x, w, b, act_gelu=a.gelu), a.iters, flush)     # includes the two row-quantisation passes
        else:
            import ctypes as C
            y = torch.empty(a.m, a.n, dtype=torch.bfloat16, device=dev)      # output allocated once: the timed region holds launches only
            L, st = Bd.lib(), C.c_void_p(torch.cuda.current_stream().cuda_stream)
            ptr = lambda t: C.c_void_p(t.data_ptr()) if t is not None else None
            ms = timed(lambda: L.bsr_linear_forward(ptr(x), ptr(w), ptr(b), ptr(r), ptr(y), a.m, a.n, a.k, Bd.DTYPE_BF16, int(a.gelu), a.mode, st),
                       a.iters, flush, reps=10)
        out.update(m=a.m, n=a.n, k=a.k, gelu=a.gelu, mode=a.mode, e4m3=a.e4m3, us=ms * 1e3, tflops=2.0 * a.m * a.n * a.k / ms / 1e9)
    elif a.what == "backward":
        x = torch.randn(a.m, a.k, device=dev).bfloat16()
        w = (torch.randn(a.n, a.k, device=dev) / math.sqrt(a.k)).bfloat16()
        dy = torch.randn(a.m, a.n, device=dev).bfloat16()
        ws = torch.empty(160 * 128 * 256, dtype=torch.float32, device=dev)
        ms = timed(lambda: Bd.bsr_linear_backward(x, w, dy, use_tensor_cores=a.mode, workspace=ws), a.iters, flush)
        out.update(m=a.m, n=a.n, k=a.k, mode=a.mode, us=ms * 1e3, tflops=4.0 * a.m * a.n * a.k / ms / 1e9)
    elif a.what == "select_gather":
        B, H, T, D = a.batch, a.heads, a.tokens, a.dim
        M = T - 1
        k = max(1, min(M, math.ceil(a.keep * M - 1e-9)))
        tdt = torch.bfloat16 if a.dtype == "bf16" else torch.float32
        z = torch.randn(B, H, M + 1, device=dev) * 2.5
        p = torch.softmax(z, dim=-1)[..., 1:].contiguous()
        x = torch.randn(B, T, D, device=dev).to(tdt)
        s, kept, dropped = Bd.bsr_token_select(p, k)
        o = Bd.bsr_gather_fuse(x, kept, dropped, s, 1)
        import ctypes as C
        L, st = Bd.lib(), C.c_void_p(torch.cuda.current_stream().cuda_stream)
        ptr = lambda t: C.c_void_p(t.data_ptr())
        # outputs pre-allocated so that the timed region holds the launch only
        ms_sel = timed(lambda: L.bsr_token_select(ptr(p), B, H, M, k, ptr(s), ptr(kept), ptr(dropped), st), a.iters, flush)
        ms_gat = timed(lambda: Bd.bsr_gather_fuse(x, kept, dropped, s, 1, out=o), a.iters, flush)
        es = x.element_size()
        sel_bytes = B * (H * M * 4 + M * 4 + M * 4)
        gat_bytes = B * ((1 + M) * D * es + (1 + k + 1) * D * es + M * 8)
        out.update(batch=B, heads=H, tokens=T, dim=D, k=k, dtype=a.dtype, select_us=ms_sel * 1e3, select_gbs=sel_bytes / ms_sel / 1e6,
                   gather_us=ms_gat * 1e3, gather_gbs=gat_bytes / ms_gat / 1e6, select_bytes=sel_bytes, gather_bytes=gat_bytes)
    else:
        B, H, T = a.batch, a.heads, a.tokens
        qkv = torch.randn(B, T, 3, H, 64, device=dev).bfloat16()
        import ctypes as C
        o = torch.empty(B, T, H * 64, device=dev, dtype=torch.bfloat16)
        cp = torch.empty(B, H, T - 1, device=dev, dtype=torch.float32)
        L, st = Bd.lib(), C.c_void_p(torch.cuda.current_stream().cuda_stream)
        ptr = lambda t: C.c_void_p(t.data_ptr())
        reps = 10                                  # back-to-back launches per timing: the kernel is shorter than a host call

        def run():
            for _ in range(reps):
                L.bsr_attention_forward(ptr(qkv), 1, B, T, H, 64, ptr(o), ptr(cp), None, 1, st)
        ms = timed(run, a.iters, flush) / reps
        out.update(batch=B, heads=H, tokens=T, us=ms * 1e3, tflops=4.0 * B * H * T * T * 64 / ms / 1e9)
        if a.backward:
            lse = torch.empty(B, H, T, device=dev, dtype=torch.float32)
            L.bsr_attention_forward(ptr(qkv), 1, B, T, H, 64, ptr(o), ptr(cp), ptr(lse), 1, st)
            do = torch.randn(B, T, H * 64, device=dev).bfloat16()
            dq = torch.empty_like(qkv)
            delta = torch.empty(B * H * T, device=dev, dtype=torch.float32)

            def run_b():
                for _ in range(reps):
                    L.bsr_attention_backward(ptr(qkv), ptr(do), ptr(lse), None, 1, B, T, H, 64, ptr(dq), ptr(delta), a.mode, st)
            msb = timed(run_b, a.iters, flush) / reps
            out.update(backward_us=msb * 1e3, backward_tflops=10.0 * B * H * T * T * 64 / msb / 1e9, backward_tensor_cores=a.mode)
    print(json.dumps(out), flush=True)


if __name__ == "__main__":
    main()
