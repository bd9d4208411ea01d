"""The benchmark workloads at full size, in the launch configurations bench.py times.

Images are independent until the batch-mean loss, so the oracle runs the full batch in chunks (with the GPU's kept
sets and expert choices forced) and its chunk gradients, weighted by chunk size, are the full-batch gradient: every
gradient tensor, the loss, all logits and all kept sets of the full-batch GPU step are compared with it.  The
headline workload additionally checks properties that hold at any size (bit-for-bit reproducibility, the gradient
of the batch mean being the mean over its halves)."""
import numpy as np
import pytest

from oracle import bsr_oracle as O
from paper_2405_10951_b200 import synth
from paper_2405_10951_b200.synth import CONFIGS

import parity as P

pytestmark = pytest.mark.gpu


def test_vit_b_full_batch_sampled_outputs_and_properties():
    import torch
    from paper_2405_10951_b200 import binding as Bd
    cfg = CONFIGS["vit_b"]
    images, labels, task_ids, params = synth.make_workload(cfg)
    eng = Bd.Engine(cfg)
    eng.set_params(params)
    img = eng.images_to_device(images)
    lab = torch.as_tensor(labels).cuda()
    loss, kept = eng.train_step(img, lab)
    eng.sync_status()
    B = cfg.batch
    logits = eng.get_tensor("logits", (B, eng.cmax)).cpu().numpy().astype(np.float64)
    kept = [k.cpu().numpy().astype(np.int64) for k in kept]
    # 1. the loss is the mean cross-entropy of the logits the step produced
    want_loss, _ = O.cross_entropy(logits, labels)
    assert abs(float(loss.cpu()[0]) - want_loss) < 1e-5 * want_loss
    assert abs(want_loss - np.log(100)) < 0.2                     # near ln(classes) at initialisation
    # 2. sampled images, one by one, through the oracle with the GPU's kept sets
    for b in (0, 41, 127):
        forced = [k[b:b + 1] for k in kept]
        ref = O.forward(cfg, params, images[b:b + 1], forced_keep=forced)
        assert P.rel_err(logits[b], ref["logits"][0]) < P.BF16_TOL
        P.check_selection(cfg, forced, ref, P.BF16_EXACT_MARGIN, P.BF16_SCORE_TOL)
    # 3. kept sets are valid index sets for every image
    ks = [138, 98, 70]
    for loc, k in enumerate(kept):
        assert k.shape == (B, ks[loc])
        assert np.all(np.diff(k, axis=1) > 0) and k.min() >= 0
    # 4. gradient of the batch mean = mean of the gradients of the two halves (same parameters, two fresh handles)
    names = ["head.0.weight", "blocks.11.attn.qkv.weight", "blocks.8.mlp.fc1.weight", "blocks.9.norm1.weight", "blocks.8.attn.proj.bias",
             "blocks.9.mlp.fc2.bias", "blocks.10.mlp.fc1.bias", "blocks.9.attn.qkv.bias", "blocks.11.mlp.fc2.weight"]
    shapes = synth.param_shapes(cfg)
    full = {n: eng.get_tensor("grad/" + n, shapes[n]).cpu().numpy().astype(np.float64) for n in names}
    eng.close()
    # 5. a second handle on the same inputs reproduces the step bit for bit (no atomics, fixed reduction orders)
    e1 = Bd.Engine(cfg)
    e1.set_params(params)
    loss1, kept1 = e1.train_step(e1.images_to_device(images), torch.as_tensor(labels).cuda())
    e1.sync_status()
    assert float(loss1.cpu()[0]) == float(loss.cpu()[0])
    assert all(np.array_equal(a.cpu().numpy(), b) for a, b in zip(kept1, kept))
    for n in names:
        assert np.array_equal(e1.get_tensor("grad/" + n, shapes[n]).cpu().numpy().astype(np.float64), full[n]), n
    e1.close()
    halves = []
    for sl in (slice(0, 64), slice(64, 128)):
        e2 = Bd.Engine(cfg, max_batch=64)
        e2.set_params(params)
        e2.train_step(e2.images_to_device(images[sl]), torch.as_tensor(labels[sl]).cuda())
        e2.sync_status()
        halves.append({n: e2.get_tensor("grad/" + n, shapes[n]).cpu().numpy().astype(np.float64) for n in names})
        e2.close()
    for n in names:
        assert P.rel_err(full[n], 0.5 * (halves[0][n] + halves[1][n])) < 5e-3, n


# workload -> images per oracle chunk (bounded by the oracle's memory: it keeps every attention map of a chunk)
FULL_BATCH = {"vit_b": 32, "deit_s": 32, "vit_b_384": 8, "moe_vit_s": 32}


@pytest.mark.parametrize("name", list(FULL_BATCH))
def test_full_batch_step_every_gradient_against_the_oracle(name):
    """Full BASELINE batch (128 / 64 / 32 / 64 images): loss, logits, kept sets, scores and every gradient tensor."""
    cfg = CONFIGS[name]
    images, labels, task_ids, params = synth.make_workload(cfg)
    gpu = P.run_gpu_step(cfg, images, labels, task_ids, params)
    gpu.pop("engine").close()
    rep = P.compare_step(cfg, images, labels, task_ids, params, gpu, P.BF16_TOL, P.BF16_EXACT_MARGIN, P.BF16_SCORE_TOL,
                         chunk=FULL_BATCH[name])
    print(name, rep)
