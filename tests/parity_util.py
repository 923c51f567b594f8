"""Shared helpers for the CUDA-vs-oracle parity tests (no method arithmetic here)."""
import numpy as np
import torch

import oracle
from paper_2306_15799_b200 import binding, configs, synth

# Tolerances of the parity gate: GPU (up-cast to fp64) against the un-rounded fp64 oracle.
BF16_REL_FRO = 1e-2
BF16_MAX_ABS = 5e-2
FP32_REL = 1e-4


def to_device(inputs):
    return {n: (t.cuda() if t is not None else None) for n, t in inputs.items()}


def oracle_head(inputs, w, b, h, rows=None, intermediates=False):
    f64 = lambda t: t.double().numpy()
    W = f64(inputs["W"]) if inputs["W"] is not None else None
    return oracle.head(f64(inputs["Q"][b, h]), f64(inputs["K"][b, h]), f64(inputs["V"][b, h]),
                       f64(inputs["E"]), f64(inputs["F"]), W, w.variant, rows=rows,
                       intermediates=intermediates)


def bf16_floor(ref):
    """max-abs error of merely rounding the oracle's own output to bfloat16."""
    r = torch.from_numpy(np.ascontiguousarray(ref))
    return float((r.to(torch.bfloat16).double() - r).abs().max())


def compare(got, ref, io):
    got = np.asarray(got, dtype=np.float64)
    diff = got - ref
    rel = float(np.linalg.norm(diff) / max(np.linalg.norm(ref), 1e-300))
    mx = float(np.abs(diff).max()) if diff.size else 0.0
    return rel, mx


def assert_close(got, ref, io, what=""):
    rel, mx = compare(got, ref, io)
    if io == "fp32":
        assert rel <= FP32_REL, "%s: rel-Fro %.3e > %.1e (max-abs %.3e)" % (what, rel, FP32_REL, mx)
    else:
        floor = bf16_floor(ref)
        assert rel <= BF16_REL_FRO, "%s: rel-Fro %.3e > %.1e" % (what, rel, BF16_REL_FRO)
        # The output's own bf16 rounding (half an ulp: 0.031 for |O| in [8,16), 0.0625 in [16,32)) is
        # part of any bf16 result; the bound applies on top of what exceeds 5e-2 by rounding alone.
        bound = max(BF16_MAX_ABS, floor + 0.5 * BF16_MAX_ABS)
        assert mx <= bound, "%s: max-abs %.3e > %.3e (bf16 rounding floor %.3e)" % (what, mx, bound, floor)
    return rel, mx


def run_gpu(w, inputs, path=binding.PATH_AUTO):
    dev = to_device(inputs)
    prev = binding.flurka_set_path(path)
    try:
        out = binding.flurka_forward(dev["Q"], dev["K"], dev["V"], dev["E"], dev["F"], dev["W"], w.variant)
        torch.cuda.synchronize()
        assert binding.flurka_last_status() == 0, "device status word is not clean"
    finally:
        binding.flurka_set_path(prev)
    return out


def check_all_heads(w, path=binding.PATH_AUTO, what=None):
    inputs = synth.make_inputs(w)
    out = run_gpu(w, inputs, path).cpu().double().numpy()
    for b in range(w.B):
        for h in range(w.H):
            ref = oracle_head(inputs, w, b, h)
            assert_close(out[b, h], ref, w.io, "%s head (%d,%d)" % (what or w.name, b, h))
    return out
