"""Throughput of one BSR fine-tuning step (ViT-B/16, bf16, batch 128) on B200, with the CPU oracle beside it.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference] [--workload vit_b]

Prints ONE JSON line (rank 0).  A step is one pass of the whole path (frozen-prefix forward, token
selection and fusion, forward + backward of the trainable blocks and head, AdamW) over one synthetic
batch.  `value` is images/s with inputs resident in HBM; `e2e` includes the pinned-host -> device copy of
the images and the device -> host read of the loss in every step, through bsr_train_step_host.  With N > 1 every rank runs an
its share of the global batch (data parallel: images are independent up to the batch-mean loss, so the one exchange
is an all-reduce of the trainable gradients between backward pass and update); the time is the maximum over ranks.
"""
from __future__ import annotations

import argparse
import json
import os
import subprocess
import sys
import tempfile
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

from paper_2405_10951_b200 import synth  # noqa: E402

METRIC = "BSR fine-tune images/s"
UNIT = "images/s"


def step_flops(cfg, batch, executed=False):
    """Algorithmic FLOPs of one step: forward of every block at its token counts, plus twice the forward
    FLOPs of the trainable blocks for their backward pass, head x3.  Token counts from the library.
    executed=True counts what the engine runs: in the last block only the classification row goes through the
    projection and the FFN (forward and backward), because nothing else of that block's output is ever read."""
    from paper_2405_10951_b200 import binding as Bd
    ta, tf, keep = Bd.bsr_token_schedule(Bd.make_config(cfg))
    D, F = cfg.dim, cfg.mlp_hidden
    ffn_mult = lambda l: (cfg.moe_top_k if l in cfg.moe_blocks else 1)
    fwd = 2 * cfg.num_patches * (cfg.in_chans * cfg.patch_size ** 2) * D
    bwd = 0
    for l in range(cfg.depth):
        t_proj, t_ffn = ta[l], tf[l]
        if executed and l == cfg.depth - 1 and keep[l] < 0:
            t_proj = t_ffn = 1
        blk = 2 * (ta[l] * 3 * D * D + t_proj * D * D + 2 * ta[l] * ta[l] * D + 2 * t_ffn * D * F * ffn_mult(l))
        fwd += blk
        if l in cfg.trainable:
            bwd += 2 * blk
    head = 2 * D * max(cfg.num_classes)
    return float(batch) * (fwd + bwd + 3 * head)


def step_bytes(cfg, batch, fp):
    """HBM bytes a step must move even with perfect fusion: the images, every stored weight once, the saved
    activations written and read back, and per trainable parameter its gradient, master copy, both moments (read and
    written) and the bf16 shadow: about 30 bytes."""
    es = 2 if cfg.dtype == "bf16" else 4
    images = batch * cfg.in_chans * cfg.image_size ** 2 * es
    return float(images + fp["weight_bytes"] + 2 * fp["saved_activation_bytes"] + 30 * fp["trainable_params"])


# DRAM traffic of the dominant kernel (tcgen05 GEMM), bytes per launch averaged over the GEMM launches of one step
# (dram__bytes_read.sum + dram__bytes_write.sum of every gemm_tc_kernel launch of the step, divided by their number),
# from the one-pass ncu launch lists summarised in profiles/launch_list_<workload>_step.txt, taken at the batch sizes
# bench.py runs.  Absent (null in the output) for a workload whose list has not been taken on the kernel as it stands.
GEMM_DRAM_BYTES_PER_LAUNCH = {"vit_b": 82660169, "deit_s": 15886456, "vit_b_384": 39582905}


def peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            p = json.load(f)
        return {"tflops": float(p["bf16_tflops_sustained"]), "tflops_burst": float(p["bf16_tflops"]),
                "hbm_gbs": float(p["hbm_gbs"]), "source": "measured"}
    return {"tflops": 1400.0, "tflops_burst": 1590.0, "hbm_gbs": 6650.0, "source": "fallback"}


class ClockSampler:
    """nvidia-smi clocks and throttle reasons while the timed regions run."""
    Q = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
         "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, index):
        self.index, self.proc, self.path = index, None, None

    def start(self):
        try:
            fd, self.path = tempfile.mkstemp(suffix=".csv")
            os.close(fd)
            self.proc = subprocess.Popen(["nvidia-smi", f"--query-gpu={self.Q}", "--format=csv,noheader,nounits", "-lms", "100",
                                          "-i", str(self.index)], stdout=open(self.path, "w"), stderr=subprocess.DEVNULL)
        except Exception:
            self.proc = None

    def stop(self):
        out = {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "samples": 0}
        if self.proc is None:
            return out
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        try:
            for line in open(self.path):
                f = [x.strip() for x in line.split(",")]
                if len(f) < 8:
                    continue
                try:
                    sm.append(float(f[1])); mx.append(float(f[2]))
                except ValueError:
                    continue
                for n, v in zip(names, f[4:8]):
                    if v == "Active":
                        reasons.add(n)
            os.unlink(self.path)
        except Exception:
            pass
        if sm:
            out.update(sm_mhz=float(np.median(sm)), sm_max_mhz=float(max(mx)), reasons=sorted(reasons), samples=len(sm))
        return out


def aggregate(dist, world, batch, steps, ms_local):
    """Whole-job throughput from per-rank timings: max over ranks of each elapsed time (a list of milliseconds),
    then images of all ranks over that time.  `dist` is torch.distributed (any backend) or None."""
    import torch
    t = torch.tensor(list(ms_local), dtype=torch.float64)
    if dist is not None and world > 1:
        if dist.get_backend() == "nccl":
            t = t.cuda()
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
    ms = [float(x) for x in t.cpu()]
    return ms, [world * batch * steps / (m / 1e3) for m in ms]


def dp_average(dist, world, grads):
    """Data-parallel gradient exchange: in-place mean over the ranks of the flat gradient buffer (one all-reduce).
    Every rank holds the gradient of its local batch mean; with equal shares their mean is the gradient of the
    global batch mean."""
    if dist is None:
        return
    if dist.get_backend() == "nccl":
        dist.all_reduce(grads, op=dist.ReduceOp.AVG)
    else:                                             # gloo has no AVG
        dist.all_reduce(grads, op=dist.ReduceOp.SUM)
        grads /= world


def oracle_sample_step(cfg, images, labels, task_ids, params):
    from oracle import bsr_oracle as O
    t0 = time.perf_counter()
    O.train_step(cfg, params, images, labels, task_ids)
    return time.perf_counter() - t0


def blas_threads():
    try:
        from threadpoolctl import threadpool_info
        n = [p.get("num_threads", 0) for p in threadpool_info() if p.get("user_api") == "blas"]
        return max(n) if n else os.cpu_count()
    except Exception:
        return os.cpu_count()


def run_reference(args, cfg):
    """The CPU oracle, as it stands, on the host cores: each step is a bounded sample of the workload."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    n_ref = max(1, min(cfg.batch, args.ref_batch))
    images, labels, task_ids, params = synth.make_workload(cfg, batch=n_ref)
    t1 = oracle_sample_step(cfg, images[:1], labels[:1], task_ids[:1], params)       # calibration, untimed
    budget = 150.0 / max(1, args.steps + args.warmup)
    n_ref = int(max(1, min(n_ref, budget / max(t1, 1e-3))))
    for _ in range(args.warmup):
        oracle_sample_step(cfg, images[:n_ref], labels[:n_ref], task_ids[:n_ref], params)
    t = [oracle_sample_step(cfg, images[:n_ref], labels[:n_ref], task_ids[:n_ref], params) for _ in range(args.steps)]
    ms = 1e3 * sum(t) / len(t)
    v = n_ref / (ms / 1e3)
    cores = blas_threads()
    line = {"impl": "reference", "metric": METRIC, "value": v, "unit": UNIT, "n_gpus": args.gpus, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": ms, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
            "dtype": "f64", "data": "synthetic",
            "config": {"workload": cfg.name, "sample": f"{n_ref} of {cfg.batch} images per step, full model dimensions"},
            "cpu_baseline": {"value": v, "unit": UNIT, "cores": cores, "kind": "oracle",
                             "sample": f"{n_ref} images per step, {args.steps} steps"},
            "e2e": {"value": v, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}}
    print(json.dumps(line), flush=True)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=200, help="timed steps (the default keeps the timed region above one second)")
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="vit_b", choices=list(synth.CONFIGS))
    ap.add_argument("--ref-batch", type=int, default=48)
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--gemm-mode", type=int, default=None, help="1: one CTA per tile, 2: CTA pairs (library default if omitted)")
    ap.add_argument("--frozen-fp8", action="store_true",
                    help="NOT the headline: the gradient-free prefix's LayerNorm-fed layers on E4M3 operands (reduced precision)")
    ap.add_argument("--parallel", default="auto", choices=["auto", "dp", "replicas"],
                    help="several GPUs: dp = data parallel, one all-reduce of the trainable gradients per step (the default); "
                         "replicas = independent copies with no exchange")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 0)
    cfg = synth.CONFIGS[args.workload]
    if args.frozen_fp8:
        cfg = cfg.with_(frozen_fp8=1)
    if args.impl == "reference":
        run_reference(args, cfg)
        return

    import torch
    from paper_2405_10951_b200 import binding as Bd
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the BSR step has no CPU path")
    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    torch.cuda.set_device(local)
    dist = None
    dp = args.parallel == "dp" or (args.parallel == "auto" and world > 1)
    if world > 1 or dp:
        import torch.distributed as dist
        os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
        os.environ.setdefault("MASTER_PORT", "29577")
        dist.init_process_group("nccl", rank=rank, world_size=world, device_id=torch.device("cuda", local))
    warm = max(args.warmup, 3)

    images, labels, task_ids, params = synth.make_workload(cfg, seed=cfg.seed + rank)      # every rank its own batch ...
    if rank > 0:
        params = synth.make_workload(cfg, seed=cfg.seed)[3]                                # ... and the same parameters
    eng = Bd.Engine(cfg, device=f"cuda:{local}")
    eng.set_params(params)
    if args.gemm_mode is not None:
        eng.set_gemm_mode(args.gemm_mode)
    del params
    storage = eng.storage_dtype
    host_img = torch.as_tensor(np.ascontiguousarray(images, dtype=np.float32)).to(storage).pin_memory()
    dev_img = host_img.cuda(non_blocking=True)
    lab = torch.as_tensor(labels).cuda()
    tid = torch.as_tensor(task_ids).cuda() if cfg.num_tasks > 1 else None
    host_loss = torch.empty(1, dtype=torch.float32).pin_memory()
    torch.cuda.synchronize()
    side = torch.cuda.Stream()          # a capturable stream: the library replays the step as a CUDA graph on it
    torch.cuda.set_stream(side)
    stream = torch.cuda.current_stream()

    def barrier():
        torch.cuda.synchronize()
        if dist is not None:
            dist.barrier()
        torch.cuda.synchronize()

    grads = eng.grad_buffer() if dp else None

    def step(img, out):
        """One step on device-resident inputs: the whole step in one call, or, data parallel, its two halves with the
        gradient all-reduce between them."""
        if not dp:
            return eng.train_step(img, lab, tid, want_kept=False, out=out)
        r = eng.forward_backward(img, lab, tid, want_kept=False, out=out)
        dp_average(dist, world, grads)
        eng.optimizer_step()
        return r

    out = None
    for _ in range(warm):
        step(dev_img, out)
        out = eng.last_out
    eng.sync_status()

    sampler = ClockSampler(local)
    if rank == 0:
        sampler.start()
        time.sleep(0.3)

    # ---- device-resident throughput -------------------------------------------------------------
    eng.profile_enable(False)
    barrier()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record(stream)
    for _ in range(args.steps):
        loss, _ = step(dev_img, out)
    e1.record(stream)
    barrier()
    ms_total = e0.elapsed_time(e1)
    launches = eng.profile_read()["kernel_launches"]

    # ---- end to end: pinned host images in, loss out, every step ----------------------------------
    # bsr_train_step_host takes HOST buffers: it copies the images and labels into one of two staging slots of the
    # workspace on its own copy stream (the copy of step i overlaps the kernels of step i-1, as an input pipeline
    # would), runs the step and copies the loss back to pinned host memory; the host reads every loss, one step behind
    # the launches.
    host_lab = torch.as_tensor(labels.astype(np.int32)).pin_memory()
    host_tid = torch.as_tensor(task_ids.astype(np.int32)).pin_memory() if cfg.num_tasks > 1 else None
    host_losses = [torch.empty(1, dtype=torch.float32).pin_memory(), torch.empty(1, dtype=torch.float32).pin_memory()]
    done = [torch.cuda.Event(), torch.cuda.Event()]
    e2e_losses = []
    stage_img = torch.empty_like(dev_img) if dp else None

    def host_step(slot):
        """One step from host memory.  Data parallel, the two halves of the step have no host-buffer form: the images
        are copied by torch into a device staging tensor on the step's stream (no overlap with the previous step)."""
        if not dp:
            eng.train_step_host(host_img, host_lab, host_tid, host_losses[slot])
            return
        stage_img.copy_(host_img, non_blocking=True)
        loss_dev, _ = step(stage_img, out)
        host_losses[slot].copy_(loss_dev, non_blocking=True)

    for i in range(2):                                    # untimed: lets the library capture its graph for each slot
        host_step(i)
    eng.sync_status()
    barrier()
    f0, f1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    f0.record(stream)
    for i in range(args.steps):
        cur = i & 1
        host_step(cur)
        done[cur].record(stream)
        if i > 0:
            done[cur ^ 1].synchronize()
            e2e_losses.append(float(host_losses[cur ^ 1][0]))
    done[(args.steps - 1) & 1].synchronize()
    e2e_losses.append(float(host_losses[(args.steps - 1) & 1][0]))
    f1.record(stream)
    barrier()
    ms_e2e = f0.elapsed_time(f1)
    h2d_bytes = int(host_img.numel() * host_img.element_size() + host_lab.numel() * 4 + (host_tid.numel() * 4 if host_tid is not None else 0))

    # ---- dominant kernel (tcgen05 GEMM): every launch bracketed by CUDA events ---------------------
    eng.profile_enable(True)
    for _ in range(min(args.steps, 5)):
        step(dev_img, out)
    prof = eng.profile_read()
    eng.profile_enable(False)
    eng.sync_status()
    clocks = sampler.stop() if rank == 0 else {}

    (ms_total, ms_e2e), (value, e2e_value) = aggregate(dist, world, cfg.batch, args.steps, [ms_total, ms_e2e])
    ms_step = ms_total / args.steps

    if rank == 0:
        pk = peaks()
        fp = eng.footprint()
        flops = step_flops(cfg, cfg.batch)
        flops_exec = step_flops(cfg, cfg.batch, executed=True)
        nbytes = step_bytes(cfg, cfg.batch, fp)
        n_prof = max(1, min(args.steps, 5))
        gemm_tflops = prof["gemm_flops"] / (prof["gemm_ms"] * 1e-3) / 1e12 if prof["gemm_ms"] > 0 else 0.0
        # The denominator is the measured burst peak (a cuBLAS GEMM timed alone), the stricter of the two measured
        # figures, whatever the clocks did: under the 1 kW cap a long run of steps settles nearer the sustained figure,
        # which is given beside it.
        t_flops_ms = flops / (pk["tflops_burst"] * 1e12) * 1e3
        t_bytes_ms = nbytes / (pk["hbm_gbs"] * 1e9) * 1e3
        t_roof_ms = max(t_flops_ms, t_bytes_ms)
        traffic = GEMM_DRAM_BYTES_PER_LAUNCH.get(cfg.name)
        line = {
            "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps, "warmup": warm,
            "ms_per_step": ms_step, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
            "dtype": ("bf16 (gradient-free prefix: E4M3 operands in the LayerNorm-fed layers)" if cfg.frozen_fp8 else "bf16") if cfg.dtype == "bf16" else "f32",
            "data": "synthetic",
            "config": {"workload": cfg.name, "global_batch": world * cfg.batch, "tokens": cfg.num_patches + 1,
                       "trainable_blocks": list(cfg.trainable), "drop_blocks": list(cfg.drop_blocks),
                       "keep_rate": cfg.keep_num / cfg.keep_den,
                       "parallelism": (f"data parallel x{world}: one NCCL all-reduce (mean) of the {fp['trainable_params']} trainable gradients per step"
                                       if dp else (f"replicas x{world}" if world > 1 else "single GPU")),
                       "l2": "no flush: weights (172 MB) plus per-step activations (> 1 GB) exceed the 126 MB L2"},
            "clocks": {k: clocks.get(k) for k in ("sm_mhz", "sm_max_mhz", "reasons", "samples")},
            "e2e": {"value": e2e_value, "unit": UNIT, "h2d_bytes_per_step": h2d_bytes, "d2h_bytes_per_step": 4,
                    "api": ("bsr_forward_backward + all-reduce + bsr_optimizer_step around torch host copies" if dp
                            else "bsr_train_step_host (host buffers in, loss to host memory)")},
            "gpu_launches": int(launches),
            # the dominant kernel: all tcgen05 GEMM launches of a step, each bracketed by CUDA events on the launching stream
            "roofline": {"bound": "tensor", "kernel": "gemm_tc_kernel (tcgen05 bf16 GEMM, all launches of a step)",
                         "achieved": gemm_tflops, "peak": pk["tflops_burst"], "unit": "TFLOP/s",
                         "frac": gemm_tflops / pk["tflops_burst"], "traffic": traffic,
                         "peak_source": pk["source"] + " burst (cuBLAS bf16 GEMM timed alone); sustained " + f"{pk['tflops']:.0f}",
                         "frac_of_sustained": gemm_tflops / pk["tflops"],
                         "gemm_ms_per_step": prof["gemm_ms"] / n_prof, "gemm_launches_per_step": prof["gemm_launches"] / n_prof,
                         "gemm_flops_per_step": prof["gemm_flops"] / n_prof},
            # the whole step against the slower of its FLOPs at the tensor peak and its bytes at the HBM peak
            "step_roofline": {"bound": "tensor" if t_flops_ms >= t_bytes_ms else "hbm", "step_flops": flops, "executed_flops": flops_exec,
                              "step_bytes": nbytes, "t_flops_ms": t_flops_ms, "t_bytes_ms": t_bytes_ms, "peak_tflops": pk["tflops_burst"],
                              "peak_hbm_gbs": pk["hbm_gbs"], "frac": t_roof_ms / ms_step,
                              "frac_of_sustained": max(flops / (pk["tflops"] * 1e12) * 1e3, t_bytes_ms) / ms_step,
                              "frac_executed": flops_exec / (pk["tflops_burst"] * 1e12) * 1e3 / ms_step},
            "footprint_bytes": {k: fp[k] for k in ("workspace_bytes", "weight_bytes", "master_bytes", "optimizer_bytes", "grad_bytes",
                                                   "saved_activation_bytes", "scratch_bytes", "paper_activation_bytes")},
            "step_flops": flops,
            "executed_flops": flops_exec,
            "step_tflops": flops / (ms_step * 1e-3) / 1e12,
            "step_roofline_frac": t_roof_ms / ms_step,
        }
        if world == 1 and not args.no_cpu_baseline:
            n_ref = min(cfg.batch, args.ref_batch)
            im, lb, tk, pr = synth.make_workload(cfg, batch=n_ref)
            sec = oracle_sample_step(cfg, im, lb, tk, pr)
            line["cpu_baseline"] = {"value": n_ref / sec, "unit": UNIT, "cores": blas_threads(), "kind": "oracle",
                                    "sample": f"one step on {n_ref} of {cfg.batch} images, full model dimensions, {sec:.1f} s"}
        else:
            line["cpu_baseline"] = None
        print(json.dumps(line), flush=True)
    if dist is not None:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
