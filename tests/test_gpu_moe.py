"""MoE FFN (paper Section 5.2) on the GPU against the oracle: routing, grouped expert GEMMs, gate gradients."""
import numpy as np
import pytest

from paper_2405_10951_b200 import synth
from paper_2405_10951_b200.synth import CONFIGS, Config

import parity as P

pytestmark = pytest.mark.gpu

MINI_MOE = Config("mini_moe", 64, 8, 128, 2, 5, 256, (10, 6), 6, (2, 3, 4), (1,), 7, 10, dtype="bf16", seed=2,
                  moe_experts=4, moe_top_k=2, moe_blocks=(1, 3))
CASES = {
    "trainable_moe_mid_block": MINI_MOE,
    "moe_is_last_block": MINI_MOE.with_(depth=4, trainable=(2, 3)),
    "top1_single_task": MINI_MOE.with_(num_classes=(10,), moe_top_k=1, moe_experts=8),
    "moe_drop_block_trainable": MINI_MOE.with_(drop_blocks=(3,), trainable=(3, 4)),
    "frozen_moe_in_gradient_path": MINI_MOE.with_(trainable=(2, 4)),
    "moe_vit_s_batch16": CONFIGS["moe_vit_s"].with_(batch=16),
    # the paper's own arrangement (Section 5.2): MoE layers only in the trainable blocks, 16 experts, the top four per
    # token, a router per task, drops at frozen and trainable locations
    "paper_style_top4_of_16": Config("mini_moe_paper", 64, 8, 128, 2, 6, 256, (10, 6), 6, (1, 3, 5), (1, 2, 4), 1, 2,
                                     dtype="bf16", seed=3, moe_experts=16, moe_top_k=4, moe_blocks=(1, 3, 5)),
    "paper_style_vit_b_batch4": CONFIGS["vit_b"].with_(name="vit_b_moe", batch=4, num_classes=(100, 10), trainable=(3, 7, 11),
                                                       moe_experts=16, moe_top_k=4, moe_blocks=(3, 7, 11), mlp_hidden=768,
                                                       keep_num=1, keep_den=2),
}


@pytest.mark.parametrize("case", list(CASES))
def test_moe_step_matches_oracle(case):
    cfg = CASES[case]
    images, labels, task_ids, params = synth.make_workload(cfg, peaked=False)
    gpu = P.run_gpu_step(cfg, images, labels, task_ids, params)
    rep = P.compare_step(cfg, images, labels, task_ids, params, gpu, P.BF16_TOL, P.BF16_EXACT_MARGIN, P.BF16_SCORE_TOL)
    print(case, rep)
    assert rep["worst_grad"] <= P.BF16_TOL
