"""The entry point with un-projected inputs (Eq. (2) with W^Q, W^K, W^V inside the call) against the fp64
oracle, element by element, through the C ABI."""
import numpy as np
import pytest
import torch

import oracle
from paper_2306_15799_b200 import binding, build, configs, synth
from paper_2306_15799_b200.configs import PERFORMER, RNN, FusedWorkload

import parity_util as pu

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module", autouse=True)
def _lib():
    build.build()
    binding.load()


def _fw(name, variant, io, B, H, N, dm, d, k, m, seed, shared_x=True):
    return FusedWorkload(name, variant, io, B, H, N, d, k, m if variant == PERFORMER else 0, seed, dm=dm, shared_x=shared_x)


def _oracle_head(x, w, b, h, rows=None, intermediates=False):
    f64 = lambda t: t.double().numpy()
    cols = slice(h * w.d, (h + 1) * w.d)
    W = f64(x["W"]) if x["W"] is not None else None
    return oracle.fused_head(f64(x["Xq"][b]), f64(x["Xk"][b]), f64(x["Xv"][b]), f64(x["E"]), f64(x["F"]),
                             f64(x["Wq"][:, cols]), f64(x["Wk"][:, cols]), f64(x["Wv"][:, cols]), W, w.variant,
                             rows=rows, intermediates=intermediates)


def _run(w, x, path):
    dev = {n: (t.cuda() if t is not None else None) for n, t in x.items()}
    prev = binding.flurka_set_path(path)
    try:
        out = binding.flurka_forward_fused(dev["Xq"], dev["Xk"], dev["Xv"], dev["E"], dev["F"], dev["Wq"], dev["Wk"],
                                           dev["Wv"], dev["W"], w.variant, w.H)
        torch.cuda.synchronize()
        assert binding.flurka_last_status() == 0
        assert binding.flurka_last_path() == (binding.PATH_SIMT if path == binding.PATH_SIMT else binding.PATH_TENSOR)
    finally:
        binding.flurka_set_path(prev)
    return out


def _check(w, path):
    x = synth.make_fused_inputs(w)
    out = _run(w, x, path).cpu().double().numpy()             # [B,N,H,d]
    Kp = binding.flurka_debug_copy(0, (w.B, w.H, w.k, w.d)).cpu().double().numpy()
    Vp = binding.flurka_debug_copy(1, (w.B, w.H, w.k, w.d)).cpu().double().numpy()
    torch.cuda.synchronize()
    for b in range(w.B):
        for h in range(w.H):
            ref, mid = _oracle_head(x, w, b, h, intermediates=True)
            # K', V' after the maps carry fp32 accumulation error only (the exponent needs that: an
            # absolute error in k' is a relative error in a feature)
            for got, want, nm in ((Kp[b, h], mid["Kp"], "K'"), (Vp[b, h], mid["Vp"], "V'")):
                err = np.abs(got - want).max()
                assert err <= 3e-5 * max(np.abs(want).max(), 1.0), "%s %s (%d,%d): %.3e" % (w.name, nm, b, h, err)
            pu.assert_close(out[b, :, h, :], ref, w.io, "%s head (%d,%d)" % (w.name, b, h))


TENSOR_CASES = [
    _fw("fused_perf_small", PERFORMER, "bf16", 1, 2, 1024, 128, 64, 128, 128, 61),
    _fw("fused_perf_m256_distinct_x", PERFORMER, "bf16", 2, 4, 1536, 256, 64, 256, 256, 62, shared_x=False),
    _fw("fused_perf_d128", PERFORMER, "bf16", 1, 2, 768, 320, 128, 192, 256, 63),
    _fw("fused_rnn", RNN, "bf16", 2, 2, 1024, 192, 64, 128, 0, 64),
    _fw("fused_perf_ragged_n", PERFORMER, "bf16", 1, 3, 1000, 192, 64, 64, 64, 65, shared_x=False),
    _fw("fused_perf_k512", PERFORMER, "bf16", 1, 6, 640, 384, 64, 512, 128, 66),
    # smallest sizes of every dimension of the map kernels: one 64-wide chunk of d_m, one head of 64 columns,
    # 64 projected rows (half an MMA tile), a batch whose B*N is not a multiple of the 256-row block
    _fw("fused_perf_dm64_one_head", PERFORMER, "bf16", 3, 1, 200, 64, 64, 64, 64, 74),
    _fw("fused_rnn_d128_k64", RNN, "bf16", 1, 1, 136, 128, 128, 64, 0, 75),
    _fw("fused_perf_wide_dm", PERFORMER, "bf16", 1, 2, 256, 1024, 64, 128, 192, 76, shared_x=False),
    # H d a multiple of 256 (the query map runs as pairs of CTAs): one 512-column group with a ragged last row
    # block, and a 512-column group followed by a 256-column one
    _fw("fused_perf_hd512_ragged_rows", PERFORMER, "bf16", 1, 8, 1000, 192, 64, 128, 128, 77),
    _fw("fused_perf_hd768", PERFORMER, "bf16", 2, 12, 640, 128, 64, 256, 64, 78, shared_x=False),
]


@pytest.mark.parametrize("w", TENSOR_CASES, ids=lambda w: w.name)
def test_fused_tensor_path_matches_oracle(w):
    _check(w, binding.PATH_TENSOR)


@pytest.mark.parametrize("limit", [1, 3])
def test_fused_tensor_path_with_few_ctas(limit):
    """Several sequence splits and tiles per CTA in every kernel of the chain."""
    prev = binding.flurka_set_cta_limit(limit)
    try:
        _check(_fw("fused_perf_few_ctas", PERFORMER, "bf16", 1, 2, 896, 128, 64, 128, 128, 67), binding.PATH_TENSOR)
    finally:
        binding.flurka_set_cta_limit(prev)


def test_fused_tensor_path_without_cta_pairs():
    """The one-CTA kernels of the query map and of stage 1 on a shape that otherwise runs as pairs."""
    prev = binding.flurka_set_stage1_pairs(0)
    try:
        _check(_fw("fused_perf_hd512_single_ctas", PERFORMER, "bf16", 1, 8, 1000, 192, 64, 256, 128, 79), binding.PATH_TENSOR)
    finally:
        binding.flurka_set_stage1_pairs(prev)


SIMT_CASES = [
    _fw("fused_simt_perf_fp32", PERFORMER, "fp32", 2, 2, 200, 40, 24, 20, 36, 71, shared_x=False),
    _fw("fused_simt_rnn_fp32", RNN, "fp32", 1, 3, 150, 33, 16, 9, 0, 72),
    _fw("fused_simt_perf_bf16_odd", PERFORMER, "bf16", 1, 2, 264, 72, 40, 24, 48, 73),
]


@pytest.mark.parametrize("w", SIMT_CASES, ids=lambda w: w.name)
def test_fused_simt_path_matches_oracle(w):
    _check(w, binding.PATH_SIMT)


def test_fused_equals_plain_forward_on_projected_inputs():
    """(E K) W^K = E (K W^K): the fused call agrees with flurka_forward fed with inputs projected in torch
    (fp32 matmul, rounded to bf16), up to the roundings of those intermediates."""
    w = _fw("fused_vs_plain", PERFORMER, "bf16", 1, 2, 1024, 128, 64, 128, 128, 68)
    x = synth.make_fused_inputs(w)
    fused = _run(w, x, binding.PATH_TENSOR).float()
    dev = {n: (t.cuda() if t is not None else None) for n, t in x.items()}
    proj = lambda X, Wm: (X.float() @ Wm.float()).to(torch.bfloat16).view(w.B, w.N, w.H, w.d).contiguous()
    plain = binding.flurka_forward(proj(dev["Xq"], dev["Wq"]), proj(dev["Xk"], dev["Wk"]), proj(dev["Xv"], dev["Wv"]),
                                   dev["E"], dev["F"], dev["W"], w.variant, layout="bnhd").float()
    torch.cuda.synchronize()
    rel = float((fused - plain).norm() / plain.norm())
    assert rel < 2e-2, rel


def test_fused_argument_errors():
    w = _fw("fused_args", RNN, "bf16", 1, 1, 256, 64, 64, 64, 0, 69)
    x = {n: (t.cuda() if t is not None else None) for n, t in synth.make_fused_inputs(w).items()}
    lib = binding.load()
    out = torch.empty((1, 256, 1, 64), dtype=torch.bfloat16, device="cuda")
    args = [x["Xq"].data_ptr(), x["Xk"].data_ptr(), x["Xv"].data_ptr(), x["E"].data_ptr(), x["F"].data_ptr(),
            x["Wq"].data_ptr(), x["Wk"].data_ptr(), x["Wv"].data_ptr(), None]
    assert lib.flurka_forward_fused(*args, RNN | 0x200, 1, 1, 256, 64, 64, 64, 0, out.data_ptr(), None) == -2
    assert lib.flurka_forward_fused(*args, RNN, 1, 1, 256, 0, 64, 64, 0, out.data_ptr(), None) == -3
    assert lib.flurka_forward_fused(*args, RNN, 1, 1, 256, 64, 64, 64, 0, x["Xq"].data_ptr(), None) == -8
    bad = list(args)
    bad[5] = None
    assert lib.flurka_forward_fused(*bad, RNN, 1, 1, 256, 64, 64, 64, 0, out.data_ptr(), None) == -1
    assert binding.flurka_fused_workspace_bytes(RNN, torch.bfloat16, 1, 1, 256, 64, 64, 64, 0) > \
        binding.flurka_workspace_bytes(RNN, torch.bfloat16, 1, 1, 256, 64, 64, 0)
