"""Host-side logic of bench.py that needs no GPU: how the event stream is cut into update windows
and backlogs, the algorithmic byte counts of a launch, and the bookkeeping of recorded ncu traffic."""
import os
import sys

import numpy as np
import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
sys.path.insert(0, ROOT)
import bench  # noqa: E402
from paper_1509_04210_b200 import synth  # noqa: E402


@pytest.mark.parametrize("name", ["tiny", "cifar10", "mid", "imagenet", "stress"])
def test_windows_hold_one_update_each_and_agree_with_the_oracle_stream(name):
    w = synth.WORKLOADS[name]
    a = bench.make_windows(w, 40)
    b = bench.make_windows(w, 40, from_oracle=True)
    assert len(a) == len(b) == 40
    for x, y in zip(a, b):
        assert x.tobytes() == y.tobytes()
        assert int((x["kind"] == bench.EV_STEP).sum()) == 1 and int((x["kind"] == bench.EV_PUSH).sum()) == w.c
        assert x["kind"][0] == bench.EV_PUSH                      # a window opens with the group's first push
    pulls = sum(int((x["kind"] == bench.EV_PULL).sum()) for x in a)
    casts = sum(int((x["kind"] == bench.EV_BROADCAST).sum()) for x in a)
    assert (casts == 40) == (w.downcast or w.mode == synth.HARDSYNC)
    assert pulls <= 40 * w.c


def test_tree_windows_carry_the_relays():
    w = synth.WORKLOADS["imagenet"]
    wins = bench.make_windows(w, 36, fanin=3)
    for x in wins:
        assert int((x["kind"] == 6).sum()) == 1 and int((x["kind"] == bench.EV_STEP).sum()) == 1   # c = 3 = one leaf's relay


def test_default_backlog_fits_the_launch_tables():
    for name, want in [("tiny", 1), ("cifar10", 30), ("mid", 4), ("imagenet", 18), ("stress", 1)]:
        w = synth.WORKLOADS[name]
        W = bench.default_window(w)
        assert W == want
        pulls = w.lam if (w.downcast or w.mode == synth.HARDSYNC) else w.c
        assert W <= 32 and W * w.c <= 128 and W * pulls <= 128
    assert bench.default_window(synth.WORKLOADS["stress"], views=True) == 4


def test_launch_bytes_follow_the_stated_formula():
    w = synth.WORKLOADS["imagenet"]
    wins = bench.make_windows(w, 36)
    chunk = np.concatenate(wins[:18])
    updates, vectors, copies = bench.batch_shape(w, chunk)
    assert (updates, vectors) == (18, 54) and copies <= 54
    region = {"launches": 2, "batches": 2, "shapes": [bench.batch_shape(w, np.concatenate(wins[i:i + 18])) for i in (0, 18)],
              "launch_ms": [4.0, 4.0], "copies": 0}
    shapes = bench.launch_shapes(w, w.nparams, 18, region)
    assert sum(rec["launches"] for rec in shapes.values()) == 2
    for (updates, vectors, copies), rec in shapes.items():       # the first round has fewer pulls: a shape of its own
        assert (updates, vectors) == (18, 54)
        assert rec["bytes_per_launch"] == w.nparams * (54 * 4 + 16 + 4 * copies)
        assert rec["gbs"] == pytest.approx(rec["bytes_per_launch"] / 4.0e-3 / 1e9)
    assert bench.update_bytes_per_param(w) == 28 and bench.update_bytes_per_param(synth.WORKLOADS["stress"]) == 80


def test_recorded_traffic_is_dropped_when_sources_or_shape_differ(monkeypatch):
    key = ("update", "imagenet", 18, 54, 54)
    rec = bench.NCU_TRAFFIC[key]
    if rec["sha"] == bench.sources_sha(rec["sources"]):
        assert bench.ncu_traffic(key, 1000) == pytest.approx(rec["bytes_per_weight"] * 1000)
    assert bench.ncu_traffic(("update", "imagenet", 18, 54, 53), 1000) is None          # another launch shape
    monkeypatch.setitem(bench.NCU_TRAFFIC, key, dict(rec, sha="0" * 16))
    assert bench.ncu_traffic(key, 1000) is None                                         # the kernel has changed since
    snap = bench.NCU_TRAFFIC[("snapshot", 1)]
    if snap["sha"] == bench.sources_sha(snap["sources"]):
        assert bench.ncu_traffic(("snapshot", 1), snap["bytes_per_launch_at"][0]) == snap["bytes_per_launch_at"][1]
        assert bench.ncu_traffic(("snapshot", 1), 12345) is None                        # captured at full size only
