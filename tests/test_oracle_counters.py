"""Pins of the oracle's token schedule and counters against numbers printed in the paper."""
import os

import pytest

from oracle import bsr_oracle as O
from oracle import counters as C
from paper_2405_10951_b200.synth import CONFIGS

MB = 2 ** 20
HERE = os.path.dirname(os.path.abspath(__file__))


def golden():
    vals = {}
    with open(os.path.join(HERE, "golden", "paper_tables.txt")) as f:
        for line in f:
            line = line.split("#")[0].split()
            if len(line) == 2:
                vals[line[0]] = float(line[1])
    return vals


G = golden()
DEIT, VITB = CONFIGS["deit_s"], CONFIGS["vit_b"]


def cfg_of(base, keep, drops, train=(3, 7, 11)):
    return base.with_(keep_num=keep[0], keep_den=keep[1], drop_blocks=tuple(drops), trainable=tuple(train))


MAC_ROWS = [
    ("deit_s_full_gmacs", DEIT, (1, 1), (), 0.55),
    ("deit_s_bsr_gmacs", DEIT, (1, 2), (3, 6, 9), 0.55),
    ("vit_b_full_gmacs", VITB, (1, 1), (), 1.0),
    ("vit_b_bsr_gmacs", VITB, (1, 2), (3, 6, 9), 0.55),
    ("deit_s_drop03_gmacs", DEIT, (7, 10), (1, 3, 5, 7, 9), 0.55),   # paper's "drop rate 0.3" = keep 0.7
    ("deit_s_drop07_gmacs", DEIT, (3, 10), (5, 7, 9), 0.55),
]


@pytest.mark.parametrize("key,base,keep,drops,tol", MAC_ROWS)
def test_forward_macs_match_paper_tables(key, base, keep, drops, tol):
    gm = C.forward_macs(cfg_of(base, keep, drops)) * 128 / 1e9
    assert abs(gm - G[key]) <= tol, (key, gm, G[key])


def test_macs_batch1_table5():
    gm = C.forward_macs(cfg_of(DEIT, (1, 1), ())) / 1e9
    assert abs(gm - G["deit_s_b1_gmacs"]) < 0.05


def test_token_counts_halving_schedule():
    # Section 4.3: tokens N -> N/2 -> N/4 -> N/8 at blocks 3, 6, 9 with drop rate 0.5
    sched = O.token_schedule(cfg_of(DEIT, (1, 2), (3, 6, 9)))
    assert [s[:2] for s in sched] == [(197, 197)] * 3 + [(197, 100)] + [(100, 100)] * 2 + [(100, 52)] + \
        [(52, 52)] * 2 + [(52, 28)] + [(28, 28)] * 2
    # K = ceil(keep * M)
    assert [s[2] for s in sched if s[2] is not None] == [98, 50, 26]
    sched = O.token_schedule(CONFIGS["vit_b"])
    assert [s[2] for s in sched if s[2] is not None] == [138, 98, 70]
    assert sched[-1][:2] == (72, 72)
    assert O.token_schedule(CONFIGS["tiny_fp32"])[2] == (65, 47, 45)
    assert [s[2] for s in O.token_schedule(CONFIGS["vit_b_384"]) if s[2] is not None] == [288, 145, 73]


def test_keep_one_drops_nothing():
    cfg = cfg_of(DEIT, (1, 1), (3, 6, 9))
    assert all(s[:2] == (197, 197) for s in O.token_schedule(cfg))


@pytest.mark.parametrize("mistake", ["floor", "no_fused_token", "keep_is_drop"])
def test_wrong_readings_miss_the_tables(monkeypatch, mistake):
    """A floor instead of a ceiling, a missing fused token, or keep/drop swapped each miss a printed value."""
    cfg = cfg_of(VITB, (1, 2), (3, 6, 9))
    cfg8 = cfg_of(DEIT, (7, 10), (1, 3, 5, 7, 9))
    if mistake == "floor":
        monkeypatch.setattr(O, "keep_count", lambda m, a, b: max(1, min(m, (a * m) // b)))
    elif mistake == "no_fused_token":
        cfg = cfg.with_(fuse_mode=0)
        cfg8 = cfg8.with_(fuse_mode=0)
    else:
        cfg8 = cfg8.with_(keep_num=3)
    off = abs(C.forward_macs(cfg) * 128 / 1e9 - G["vit_b_bsr_gmacs"])
    off8 = abs(C.forward_macs(cfg8) * 128 / 1e9 - G["deit_s_drop03_gmacs"])
    assert max(off, off8) > 2.0


def test_table1_closed_forms():
    full = cfg_of(DEIT, (1, 1), (), range(12))
    t, d, f, h = 197, 384, 1536, 6
    assert round(3 * t * d * 4 / MB, 2) == G["qkv_mb"]
    assert round(h * t * t * 4 / MB, 2) == G["softmax_mb"]
    assert round(t * f * 4 / MB, 2) == G["gelu_mb"]
    frozen = C.block_activation_bytes(full, t, t, False) / MB
    train = C.block_activation_bytes(full, t, t, True) / MB
    assert round(frozen, 1) == G["frozen_block_mb"]
    assert round(train, 1) == G["trainable_block_mb"]
    assert abs(12 * train - G["full_ft_activation_mb"]) / G["full_ft_activation_mb"] < 0.015


MEM_ROWS = [("mem_3_7_11", (3, 7, 11)), ("mem_10_11", (10, 11)), ("mem_9_10_11", (9, 10, 11)),
            ("mem_8_9_10_11", (8, 9, 10, 11)), ("mem_4_7_11", (4, 7, 11)), ("mem_4_11", (4, 11)),
            ("mem_7_11", (7, 11)), ("mem_3_6_9_11", (3, 6, 9, 11)), ("mem_4_7_10_11", (4, 7, 10, 11))]


@pytest.mark.parametrize("key,train", MEM_ROWS)
def test_train_memory_with_dropping_tracks_table7(key, train):
    """The accounting reproduces the 'Train Mem' column up to a near-constant residue (15-30 MB)."""
    est = C.train_memory_bytes(cfg_of(DEIT, (1, 2), (3, 6, 9), train), 128) / MB
    assert 15.0 <= G[key] - est <= 30.0, (key, est, G[key])


@pytest.mark.parametrize("key,train,hi", [("mem_nodrop_10_11", (10, 11), 60), ("mem_nodrop_9_10_11", (9, 10, 11), 60),
                                          ("mem_nodrop_8_9_10_11", (8, 9, 10, 11), 60),
                                          ("mem_nodrop_full", tuple(range(12)), 115)])
def test_train_memory_without_dropping_tracks_table2(key, train, hi):
    est = C.train_memory_bytes(cfg_of(DEIT, (1, 1), (), train), 128) / MB
    assert 45.0 <= G[key] - est <= hi, (key, est, G[key])
