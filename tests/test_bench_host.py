"""Host arithmetic of bench.py's roofline objects (no GPU): the fraction is the time at the roofline,
max(FLOPs / dense bf16 peak, bytes / HBM bandwidth), over the measured time, for the dominant kernel and
for the whole forward."""
import os
import sys

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
sys.path.insert(0, ROOT)

import bench  # noqa: E402
from paper_2306_15799_b200 import configs  # noqa: E402

PEAKS = {"hbm_gbs": 6500.0, "bf16_tflops": 1600.0, "bf16_tflops_sustained": 1400.0, "source": "measured"}


def _res(stage_ms, step_ms):
    return {"stage_ms": stage_ms, "total_ms": sum(step_ms), "step_ms": step_ms}


def test_stage_work_adds_up_to_the_counted_flops():
    for w in (configs.C2, configs.C3, configs.C4, configs.c5(512, 64)):
        names, flops, byts, exps = bench.stage_work(w)
        assert names == ["down_projection", "key_side", "query_side"]
        assert sum(flops) == w.flops()
        assert exps[0] == 0 and exps[2] == w.B * w.H * w.N * (w.m if w.variant == configs.PERFORMER else w.d)
        # every stage's bytes include its share of the compulsory traffic: Q, K, V in and O out
        s = w.elem_bytes
        assert byts[0] >= 2 * w.tokens * w.d * s + 2 * w.k * w.N * s
        assert byts[2] >= 2 * w.tokens * w.d * s


def test_roofline_fraction_can_be_recomputed_from_the_line():
    w = configs.C3
    res = _res([0.075, 0.025, 0.120], [0.22, 0.24])
    roof, path = bench.rooflines(w, res, PEAKS, steps=2, world=1, exp_rate=4000.0)
    names, flops, byts, exps = bench.stage_work(w)
    assert roof["kernel"] == "query_side"
    t_tensor = flops[2] / (PEAKS["bf16_tflops"] * 1e12)
    t_hbm = byts[2] / (PEAKS["hbm_gbs"] * 1e9)
    assert abs(roof["frac"] - max(t_tensor, t_hbm) / 0.120e-3) < 1e-12
    assert roof["bound"] == ("hbm" if t_hbm >= t_tensor else "tensor")
    assert abs(roof["achieved"] / roof["peak"] - (t_hbm if roof["bound"] == "hbm" else t_tensor) / 0.120e-3) < 1e-9
    assert roof["frac_sustained"] >= roof["frac"]
    assert abs(roof["exp"]["frac"] - exps[2] / 0.120e-3 / 1e9 / 4000.0) < 1e-12
    assert roof["traffic"] is None or roof["traffic"] > 0
    ms = 0.23e-3
    want = max(w.flops() / (PEAKS["bf16_tflops"] * 1e12), w.compulsory_bytes() / (PEAKS["hbm_gbs"] * 1e9)) / ms
    assert abs(path["frac"] - want) < 1e-12


def test_dominant_kernel_follows_the_stage_times():
    w = configs.C4
    roof, _ = bench.rooflines(w, _res([0.21, 0.03, 0.15], [0.4]), PEAKS, steps=1, world=1, exp_rate=None)
    assert roof["kernel"] == "down_projection" and roof["bound"] == "tensor" and "exp" not in roof


def test_backward_block_counts_the_backward_work():
    """The backward's FLOPs: stage 1 again, the four products with E, F, K, V and, for PERFORMER, the
    four N x m x d products of the query side and the four k x m x d ones of the key side."""
    w = configs.C3
    flops, byts = bench.backward_work(w)
    BH = w.B * w.H
    assert flops == BH * (12 * w.N * w.k * w.d + 8 * w.N * w.m * w.d + 12 * w.k * w.m * w.d)
    assert byts == 7 * w.tokens * w.d * w.elem_bytes + 4 * w.k * w.N * w.elem_bytes
    rb = {"total_ms": 2.2, "step_ms": [1.0, 1.2], "path": "tensor", "launches": 20, "status": 0, "flushed": False}
    blk = bench.backward_block(w, rb, PEAKS, steps=2, world=1)
    assert abs(blk["ms_per_step"] - 1.1) < 1e-12
    assert abs(blk["value"] - w.tokens / 1.1e-3) < 1e-3
    want = max(flops / (PEAKS["bf16_tflops"] * 1e12), byts / (PEAKS["hbm_gbs"] * 1e9)) / 1.1e-3
    assert abs(blk["path_roofline"]["frac"] - want) < 1e-12
    # RNN: no feature products on either side beyond the d x d ones the forward counts
    f2, _ = bench.backward_work(configs.C2)
    assert f2 == configs.C2.B * configs.C2.H * 12 * configs.C2.N * configs.C2.k * configs.C2.d
