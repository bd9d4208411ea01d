"""Entry points around the single step: a run of steps under the on-device cosine schedule (Section 5), the step fed
from host memory, and parameter loading from host / device memory in float32 / bfloat16."""
import numpy as np
import pytest

from oracle import bsr_oracle as O
from paper_2405_10951_b200 import synth
from paper_2405_10951_b200.synth import CONFIGS, Config

import parity as P

pytestmark = pytest.mark.gpu

TINY = CONFIGS["tiny_fp32"]
MINI_BF16 = Config("mini_bf16", 64, 8, 128, 2, 6, 256, (10,), 6, (3, 4, 5), (1, 3, 4), 7, 10, dtype="bf16", seed=1)


def batches_of(cfg, n, peaked=True):
    """n different seeded batches for one set of parameters."""
    images, labels, task_ids, params = synth.make_workload(cfg, peaked=peaked)
    out = [(images, labels, task_ids)]
    for i in range(1, n):
        out.append(synth.make_batch(cfg, np.random.default_rng(1000 + i)))
    return out, params


def stack_to_device(eng, batches):
    import torch
    imgs = torch.stack([eng.images_to_device(b[0]) for b in batches]).contiguous()
    labs = torch.stack([torch.as_tensor(b[1].astype(np.int32)) for b in batches]).cuda().contiguous()
    tids = torch.stack([torch.as_tensor(b[2].astype(np.int32)) for b in batches]).cuda().contiguous()
    return imgs, labs, tids


@pytest.mark.parametrize("dtype", ["fp32", "bf16"])
def test_run_of_steps_with_cosine_schedule_follows_the_oracle(dtype):
    """SGD with momentum makes the schedule visible: every step moves the parameters by lr(t) times the buffer, so the
    parameter change after the run is compared with the oracle stepped with math.cos learning rates, per tensor."""
    import torch
    from paper_2405_10951_b200 import binding as Bd
    base = TINY.with_(trainable=(2, 3, 4, 5)) if dtype == "fp32" else MINI_BF16
    cfg = base.with_(optimizer="sgd", momentum=0.9, weight_decay=0.01)
    n, total, lr_max, lr_min = 4, 4, 2e-2, 1e-3
    batches, params = batches_of(cfg, n)
    eng = Bd.Engine(cfg)
    eng.set_params(params)
    imgs, labs, tids = stack_to_device(eng, batches)
    stream = torch.cuda.Stream()
    with torch.cuda.stream(stream):                               # a capturable stream: one graph, replayed n times
        losses, kept = eng.train_steps(imgs, labs, None, lr_max=lr_max, lr_min=lr_min, total_steps=total)
        eng.sync_status()
        prof = eng.profile_read()
    assert prof["graph_captures"] == 1
    losses = losses.cpu().numpy().astype(np.float64)
    # the oracle, given the kept sets of a step-by-step GPU run of the same sequence (needed for every step)
    eng2 = Bd.Engine(cfg)
    eng2.set_params(params)
    forced = []
    for t, (im, lb, tk) in enumerate(batches):
        eng2.set_lr(O.cosine_lr(lr_max, lr_min, t, total))
        _, k = eng2.train_step(eng2.images_to_device(im), torch.as_tensor(lb).cuda())
        forced.append([x.cpu().numpy().astype(np.int64) for x in k])
    eng2.sync_status()
    assert all(np.array_equal(a.cpu().numpy(), b) for a, b in zip(kept, forced[-1]))
    runs = O.train_steps(cfg, params, batches, lr_max, lr_min, total, forced_keeps=forced)
    tol = P.FP32_TOL if dtype == "fp32" else P.BF16_TOL * 1.5
    for t in range(n):
        assert abs(losses[t] - runs[t]["loss"]) < max(tol, 2e-3) * abs(runs[t]["loss"]), t
    shapes = synth.param_shapes(cfg)
    final = runs[-1]
    for name in O.trainable_names(cfg, params):
        got = eng.get_tensor(name, shapes[name]).cpu().numpy().astype(np.float64) - params[name]
        same = eng2.get_tensor(name, shapes[name]).cpu().numpy().astype(np.float64) - params[name]
        want = final["params"][name] - params[name]
        bound = 2 * tol * np.linalg.norm(want) + 2.4e-7 * n * np.linalg.norm(params[name])
        assert np.linalg.norm(got - want) < bound, (name, np.linalg.norm(got - want), bound)
        # the loop and the step-by-step run with host-side math.cos rates agree to float rounding of the rate; in bf16
        # one ulp of the rate flips the rounding of a few bf16 shadow weights, which the later steps then see
        close = 1e-5 if dtype == "fp32" else 1e-3
        assert np.linalg.norm(got - same) <= close * np.linalg.norm(want) + 2.4e-7 * n * np.linalg.norm(params[name]), name
    # a wrong schedule would show: with a constant rate the change of the head would be off by far more than the bound
    const = O.train_steps(cfg, params, batches, lr_max, lr_max, total, forced_keeps=forced)[-1]
    d_const = const["params"]["head.0.weight"] - params["head.0.weight"]
    d_want = final["params"]["head.0.weight"] - params["head.0.weight"]
    assert np.linalg.norm(d_const - d_want) > 4 * 2 * tol * np.linalg.norm(d_want)
    eng.close()
    eng2.close()


def test_run_of_steps_continues_the_step_count_and_matches_single_steps_adamw():
    """AdamW: two calls of two steps equal four single steps with host-side rates (bias corrections continue from the
    handle's step counter); compared through losses and parameters to float rounding of the scalars."""
    import torch
    from paper_2405_10951_b200 import binding as Bd
    cfg = MINI_BF16
    n, total, lr_max, lr_min = 4, 10, 1e-3, 1e-5
    batches, params = batches_of(cfg, n)
    a = Bd.Engine(cfg)
    a.set_params(params)
    imgs, labs, tids = stack_to_device(a, batches)
    l1, _ = a.train_steps(imgs[:2], labs[:2], None, lr_max=lr_max, lr_min=lr_min, total_steps=total)
    l2, _ = a.train_steps(imgs[2:], labs[2:], None, lr_max=lr_max, lr_min=lr_min, total_steps=total)
    a.sync_status()
    b = Bd.Engine(cfg)
    b.set_params(params)
    single = []
    for t in range(n):
        b.set_lr(O.cosine_lr(lr_max, lr_min, t, total))
        loss, _ = b.train_step(imgs[t], labs[t])
        single.append(float(loss.cpu()[0]))
    b.sync_status()
    got = np.concatenate([l1.cpu().numpy(), l2.cpu().numpy()]).astype(np.float64)
    assert np.allclose(got, single, rtol=1e-4), (got, single)
    shapes = synth.param_shapes(cfg)
    for name in ("head.0.weight", "blocks.5.mlp.fc1.weight", "blocks.3.attn.qkv.weight", "norm.bias"):
        pa = a.get_tensor(name, shapes[name]).cpu().numpy().astype(np.float64)
        pb = b.get_tensor(name, shapes[name]).cpu().numpy().astype(np.float64)
        assert np.linalg.norm(pa - pb) <= 1e-3 * np.linalg.norm(pb - params[name]) + 1e-9, name
    a.close()
    b.close()


def test_step_from_host_memory_equals_step_from_device_memory():
    """bsr_train_step_host: pinned host inputs, loss and kept positions back in host memory, three steps through both
    staging slots; bit-identical to bsr_train_step on device-resident copies of the same inputs."""
    import torch
    from paper_2405_10951_b200 import binding as Bd
    cfg = MINI_BF16
    batches, params = batches_of(cfg, 3)
    dev = Bd.Engine(cfg)
    dev.set_params(params)
    host = Bd.Engine(cfg)
    host.set_params(params)
    want_loss, want_kept = [], []
    for im, lb, tk in batches:
        loss, kept = dev.train_step(dev.images_to_device(im), torch.as_tensor(lb).cuda())
        want_loss.append(float(loss.cpu()[0]))
        want_kept.append(torch.cat([k.flatten() for k in kept]).cpu().numpy())
    dev.sync_status()
    stream = torch.cuda.Stream()
    got_loss, got_kept = [], []
    with torch.cuda.stream(stream):
        outs = []
        for im, lb, tk in batches:
            himg = torch.as_tensor(np.ascontiguousarray(im, dtype=np.float32)).to(host.storage_dtype).pin_memory()
            hlab = torch.as_tensor(lb.astype(np.int32)).pin_memory()
            hloss = torch.empty(1, dtype=torch.float32).pin_memory()
            hkept = torch.empty(cfg.batch * sum(host.kept_counts), dtype=torch.int32).pin_memory()
            host.train_step_host(himg, hlab, None, hloss, hkept)
            outs.append((himg, hlab, hloss, hkept))               # the buffers stay alive until the stream is done
        host.sync_status()
    for _, _, hloss, hkept in outs:
        got_loss.append(float(hloss[0]))
        got_kept.append(hkept.numpy().copy())
    assert got_loss == want_loss
    assert all(np.array_equal(a, b) for a, b in zip(got_kept, want_kept))
    shapes = synth.param_shapes(cfg)
    for name in ("head.0.weight", "blocks.4.mlp.fc2.weight", "blocks.3.norm1.bias"):
        assert torch.equal(host.get_tensor(name, shapes[name]), dev.get_tensor(name, shapes[name])), name
    dev.close()
    host.close()


@pytest.mark.parametrize("dtype", ["fp32", "bf16"])
def test_parameters_load_from_host_or_device_in_float_or_bf16(dtype):
    """bsr_set_param with the four (source type, source place) combinations: the stored values read back identically
    (the synthetic values are exact in bf16 for a bf16 model; for the fp32 model the bf16 sources carry rounded values,
    which must read back as exactly those rounded values) and a training step gives the same loss."""
    import torch
    from paper_2405_10951_b200 import binding as Bd
    cfg = MINI_BF16 if dtype == "bf16" else TINY
    images, labels, task_ids, params = synth.make_workload(cfg, peaked=True)
    rounded = {n: synth.round_to_bf16(v) for n, v in params.items()}
    shapes = synth.param_shapes(cfg)
    losses = {}
    for src in ("host_f32", "dev_f32", "host_bf16", "dev_bf16"):
        eng = Bd.Engine(cfg)
        for n, v in params.items():
            t = torch.as_tensor(np.ascontiguousarray(v, dtype=np.float32))
            if src.endswith("bf16"):
                t = t.to(torch.bfloat16)
            if src.startswith("dev"):
                t = t.cuda()
            eng.set_param(n, t)
        expect = rounded if src.endswith("bf16") else params
        for n in ("patch_embed.weight", "pos_embed", "blocks.0.attn.qkv.weight", f"blocks.{max(cfg.trainable)}.mlp.fc1.weight",
                  f"blocks.{max(cfg.trainable)}.norm2.weight", "head.0.weight", "head.0.bias"):
            got = eng.get_tensor(n, shapes[n]).cpu().numpy()
            assert np.array_equal(got, expect[n].astype(np.float32)), (src, n)
        loss, _ = eng.train_step(eng.images_to_device(images), torch.as_tensor(labels).cuda())
        eng.sync_status()
        losses[src] = float(loss.cpu()[0])
        eng.close()
    assert losses["host_f32"] == losses["dev_f32"] and losses["host_bf16"] == losses["dev_bf16"]
    if dtype == "bf16":
        assert losses["host_f32"] == losses["host_bf16"]


def test_graph_cache_keeps_eight_buffer_sets():
    """An input pipeline rotating through eight sets of buffers captures eight graphs and then only replays."""
    import torch
    from paper_2405_10951_b200 import binding as Bd
    cfg = MINI_BF16
    images, labels, task_ids, params = synth.make_workload(cfg)
    eng = Bd.Engine(cfg)
    eng.set_params(params)
    stream = torch.cuda.Stream()
    with torch.cuda.stream(stream):
        bufs = [eng.images_to_device(images).clone() for _ in range(8)]
        lab = torch.as_tensor(labels).cuda()
        stream.synchronize()
        out = None
        for rounds in range(3):
            for b in bufs:
                eng.train_step(b, lab, out=out)
                out = eng.last_out
        eng.sync_status()
        assert eng.profile_read()["graph_captures"] == 8
    eng.close()


def test_split_step_equals_whole_step_and_exposes_the_gradient_buffer():
    """bsr_forward_backward + bsr_optimizer_step (the data-parallel halves) equal bsr_train_step bit for bit on one
    GPU; the gradient buffer handed out for the all-reduce holds exactly the gradients bsr_get_tensor reports, and
    scaling it before the update scales the SGD update (what an average over ranks does)."""
    import torch
    from paper_2405_10951_b200 import binding as Bd
    cfg = MINI_BF16
    images, labels, task_ids, params = synth.make_workload(cfg, peaked=True)
    shapes = synth.param_shapes(cfg)
    names = ("head.0.weight", "blocks.5.mlp.fc1.weight", "blocks.3.attn.qkv.weight", "norm.bias", "blocks.4.mlp.fc2.bias")
    whole = Bd.Engine(cfg)
    whole.set_params(params)
    split = Bd.Engine(cfg)
    split.set_params(params)
    stream = torch.cuda.Stream()
    with torch.cuda.stream(stream):
        img = whole.images_to_device(images)
        lab = torch.as_tensor(labels).cuda()
        for _ in range(2):
            l1, k1 = whole.train_step(img, lab)
            l2, k2 = split.forward_backward(img, lab)
            g = split.grad_buffer()
            assert g.numel() >= sum(int(np.prod(shapes[n])) for n in O.trainable_names(cfg, params))
            split.optimizer_step()
            stream.synchronize()
            assert float(l1.cpu()[0]) == float(l2.cpu()[0])
            assert all(torch.equal(a, b) for a, b in zip(k1, k2))
        whole.sync_status()
        split.sync_status()
        for n in names:
            assert torch.equal(whole.get_tensor(n, shapes[n]), split.get_tensor(n, shapes[n])), n
            assert torch.equal(whole.get_tensor("grad/" + n, shapes[n]), split.get_tensor("grad/" + n, shapes[n])), n
        # the buffer is what the optimiser reads: the head's gradient sits in it verbatim
        gh = split.get_tensor("grad/head.0.weight", shapes["head.0.weight"]).flatten()
        flat = split.grad_buffer()
        windows = flat.unfold(0, gh.numel(), 64)                     # tensors start at multiples of 64 values
        assert bool((windows == gh).all(dim=1).any())
    whole.close()
    split.close()


def test_bench_data_parallel_path_runs_on_one_rank():
    """bench.py --parallel dp with a one-rank NCCL group: the split step, the all-reduce of the gradient buffer view and
    the update run end to end and give the single-GPU throughput line."""
    import json
    import os
    import subprocess
    import sys
    root = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
    env = dict(os.environ, MASTER_ADDR="127.0.0.1", MASTER_PORT="29631", RANK="0", WORLD_SIZE="1", LOCAL_RANK="0")
    r = subprocess.run([sys.executable, os.path.join(root, "bench.py"), "--workload", "deit_s", "--steps", "5", "--warmup", "3",
                        "--parallel", "dp", "--no-cpu-baseline"], capture_output=True, text=True, env=env, timeout=600)
    assert r.returncode == 0, r.stderr[-2000:]
    line = json.loads(r.stdout.strip().splitlines()[-1])
    assert line["value"] > 0 and "data parallel" in line["config"]["parallelism"] and line["gpu_launches"] > 0
