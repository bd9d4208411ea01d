"""Host-side checks that need no GPU: the C-ABI library loads, exports what include/bsr.h declares,
validates configurations, and its token schedule equals the oracle's."""
import os
import re

import pytest

from oracle import bsr_oracle as O
from paper_2405_10951_b200 import binding as Bd
from paper_2405_10951_b200 import synth

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def declared_symbols():
    text = open(os.path.join(ROOT, "include", "bsr.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(bsr_[a-z_0-9]+)\s*\(", text)))


def test_library_exports_every_declared_symbol():
    names = declared_symbols()
    assert len(names) >= 15
    L = Bd.lib()
    for n in names:
        assert hasattr(L, n), n
    assert sorted(Bd.EXPORTS) == names


@pytest.mark.parametrize("name", list(synth.CONFIGS))
def test_token_schedule_matches_oracle(name):
    cfg = synth.CONFIGS[name]
    ta, tf, k = Bd.bsr_token_schedule(Bd.make_config(cfg))
    want = O.token_schedule(cfg)
    assert ta == [w[0] for w in want]
    assert tf == [w[1] for w in want]
    assert k == [(-1 if w[2] is None else w[2]) for w in want]


def test_schedule_other_rates():
    base = synth.CONFIGS["deit_s"]
    for num, den, drops in [(1, 2, (3, 6, 9)), (3, 10, (5, 7, 9)), (7, 10, (1, 3, 5, 7, 9)), (1, 1, (3, 6, 9)), (1, 197, (0,))]:
        for fuse in (0, 1):
            cfg = base.with_(keep_num=num, keep_den=den, drop_blocks=drops, fuse_mode=fuse)
            ta, tf, k = Bd.bsr_token_schedule(Bd.make_config(cfg))
            want = O.token_schedule(cfg)
            assert list(zip(ta, tf)) == [w[:2] for w in want]


def test_workspace_size_and_validation():
    for name in ("tiny_fp32", "deit_s", "vit_b", "vit_b_384"):
        cfg = synth.CONFIGS[name]
        n = Bd.bsr_workspace_bytes(Bd.make_config(cfg))
        assert n > 0 and n % 256 == 0
    small = Bd.bsr_workspace_bytes(Bd.make_config(synth.CONFIGS["vit_b"], max_batch=8))
    assert small < Bd.bsr_workspace_bytes(Bd.make_config(synth.CONFIGS["vit_b"]))
    assert Bd.bsr_workspace_bytes(Bd.make_config(synth.CONFIGS["vit_b"])) < 20 * 2 ** 30

    def status_of(cfg):
        with pytest.raises(Bd.BsrError) as e:
            Bd.bsr_workspace_bytes(Bd.make_config(cfg))
        return e.value.status

    tiny = synth.CONFIGS["tiny_fp32"]
    assert status_of(tiny.with_(heads=5)) == -1                      # dim not a multiple of heads
    assert status_of(tiny.with_(image_size=30)) == -1                # not a multiple of the patch size
    assert status_of(tiny.with_(drop_blocks=(3, 2))) == -1           # not ascending
    assert status_of(tiny.with_(keep_num=11)) == -1                  # keep rate above one
    assert status_of(tiny.with_(trainable=(7,))) == -1               # beyond depth
    assert Bd.bsr_workspace_bytes(Bd.make_config(tiny.with_(trainable=(1, 5)))) > 0   # frozen blocks inside the gradient path
    assert Bd.bsr_workspace_bytes(Bd.make_config(synth.CONFIGS["moe_vit_s"])) > 0
    assert status_of(synth.CONFIGS["moe_vit_s"].with_(dtype="fp32")) == -2          # MoE runs on the bf16 kernels only
    assert status_of(synth.CONFIGS["moe_vit_s"].with_(moe_top_k=5)) == -1
    c = Bd.make_config(tiny)
    c.max_batch = 0
    with pytest.raises(Bd.BsrError):
        Bd.bsr_workspace_bytes(c)
