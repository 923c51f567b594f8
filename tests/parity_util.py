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


def bf16_half_ulp(ref):
    """Half a unit in the last place of bfloat16 at each |ref| (8 significand bits): what rounding the
    exact value to bfloat16 can cost by itself."""
    a = np.maximum(np.abs(np.asarray(ref, dtype=np.float64)), 2.0 ** -126)
    return 2.0 ** (np.floor(np.log2(a)) - 8)


def assert_close(got, ref, io, what=""):
    """The parity gate.  bf16: rel-Frobenius <= 1e-2 and max-abs <= 5e-2, element by element.  Only an
    element whose own bfloat16 rounding can already cost more than 5e-2 (|ref| >= 16: half an ulp is
    0.0625) gets half an ulp + 2.5e-2 instead; such elements are counted and printed."""
    rel, mx = compare(got, ref, io)
    if io == "fp32":
        assert rel <= FP32_REL, "%s: rel-Fro %.3e > %.1e (max-abs %.3e)" % (what, rel, FP32_REL, mx)
    else:
        assert rel <= BF16_REL_FRO, "%s: rel-Fro %.3e > %.1e" % (what, rel, BF16_REL_FRO)
        diff = np.abs(np.asarray(got, dtype=np.float64) - ref)
        half_ulp = bf16_half_ulp(ref)
        wide = half_ulp >= BF16_MAX_ABS
        bound = np.where(wide, half_ulp + 0.5 * BF16_MAX_ABS, BF16_MAX_ABS)
        bad = diff > bound
        assert not bad.any(), "%s: max-abs %.3e > %.1e at %d elements (worst excess %.3e; %d elements on the widened bound)" % (
            what, mx, BF16_MAX_ABS, int(bad.sum()), float((diff - bound).max()), int(wide.sum()))
        if wide.any():
            print("%s: %d of %d elements have |ref| >= 16 (bf16 half-ulp 0.0625 > 5e-2) and use half-ulp + 2.5e-2; "
                  "max-abs over the others %.3e" % (what, int(wide.sum()), wide.size,
                                                    float(diff[~wide].max()) if (~wide).any() else 0.0))
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
