"""flurka_backward against the fp64 oracle's backward pass (itself pinned by finite differences of the
forward oracle), element-wise through relative Frobenius norms per gradient."""
import numpy as np
import pytest
import torch

import oracle
from paper_2306_15799_b200 import binding, build, synth
from paper_2306_15799_b200.configs import PERFORMER, RNN, Workload

import parity_util as pu

pytestmark = pytest.mark.gpu

# fp32 I/O: every step is fp32 with sums of up to N (or k, m) terms and one cancelling difference
# (a_i.dO_n - O_n.dO_n), so gradients carry about 1e-5 relative error; bf16 I/O adds the rounding of the
# stored gradients (2^-9 each): the gates are 1e-3 and 1e-2 of the gradient's Frobenius norm.
TOL = {"fp32": 1e-3, "bf16": 1e-2}


@pytest.fixture(scope="module", autouse=True)
def _lib():
    build.build()
    binding.load()


def _oracle_grads(w, x, dO, per_head):
    f64 = lambda t: t.double().numpy()
    W = f64(x["W"]) if x["W"] is not None else None
    g = {n: np.zeros(tuple(x[n[1:]].shape)) for n in ("dQ", "dK", "dV", "dE", "dF")}
    for b in range(w.B):
        for h in range(w.H):
            E, F = (f64(x["E"][h]), f64(x["F"][h])) if per_head else (f64(x["E"]), f64(x["F"]))
            r = oracle.head_backward(f64(x["Q"][b, h]), f64(x["K"][b, h]), f64(x["V"][b, h]), E, F, W, f64(dO[b, h]), w.variant)
            for n in ("dQ", "dK", "dV"):
                g[n][b, h] = r[n]
            for n in ("dE", "dF"):
                if per_head:
                    g[n][h] += r[n]
                else:
                    g[n] += r[n]
    return g


def _check(w, layout="bhnd", per_head=False):
    x = synth.make_inputs(w)
    gen = torch.Generator().manual_seed(w.seed + 5)
    if per_head:
        for name in ("E", "F"):
            x[name] = (torch.randn(w.H, w.k, w.N, generator=gen, dtype=torch.float64) * float(w.k) ** -0.5).to(x["Q"].dtype)
    dO = torch.randn(w.B, w.H, w.N, w.d, generator=gen, dtype=torch.float64).to(x["Q"].dtype)
    dev = pu.to_device(x)
    t = (lambda a: a.transpose(1, 2).contiguous()) if layout == "bnhd" else (lambda a: a)
    got = binding.flurka_backward(t(dev["Q"]), t(dev["K"]), t(dev["V"]), dev["E"], dev["F"], dev["W"], t(dO.cuda()),
                                  w.variant, layout=layout)
    torch.cuda.synchronize()
    assert binding.flurka_last_status() == 0
    ref = _oracle_grads(w, x, dO, per_head)
    for name, tensor in zip(("dQ", "dK", "dV", "dE", "dF"), got):
        arr = tensor.transpose(1, 2) if (layout == "bnhd" and tensor.dim() == 4) else tensor
        arr = arr.cpu().double().numpy()
        assert np.isfinite(arr).all(), name
        rel = np.linalg.norm(arr - ref[name]) / max(np.linalg.norm(ref[name]), 1e-300)
        assert rel <= TOL[w.io], "%s %s: rel-Fro %.3e > %.0e" % (w.name, name, rel, TOL[w.io])


CASES = [
    Workload("bwd_perf_fp32", PERFORMER, "fp32", 2, 2, 100, 24, 12, 40, 301),
    Workload("bwd_rnn_fp32", RNN, "fp32", 1, 3, 77, 20, 9, 0, 302),
    Workload("bwd_perf_bf16_d64", PERFORMER, "bf16", 1, 2, 300, 64, 40, 96, 303),
    Workload("bwd_rnn_bf16_d128", RNN, "bf16", 1, 2, 160, 128, 33, 0, 304),
    Workload("bwd_perf_fp32_ragged", PERFORMER, "fp32", 1, 1, 45, 33, 5, 37, 305),
]


@pytest.mark.parametrize("w", CASES, ids=lambda w: w.name)
def test_backward_matches_oracle(w):
    _check(w)


TENSOR_CASES = [
    # bf16 PERFORMER with d = 64 and 128 or 256 features: stage 1 and the query side on the tensor-core kernels
    Workload("bwd_tc_m256", PERFORMER, "bf16", 1, 3, 520, 64, 64, 256, 311),
    Workload("bwd_tc_m128", PERFORMER, "bf16", 2, 2, 384, 64, 128, 128, 312),
    Workload("bwd_tc_m256_k256", PERFORMER, "bf16", 1, 2, 1000, 64, 256, 256, 313),
    # a last feature tile of 64: padded to 128 inside the kernel with weights that are exactly zero
    Workload("bwd_tc_m64", PERFORMER, "bf16", 1, 3, 392, 64, 128, 64, 320),
    Workload("bwd_tc_m192", PERFORMER, "bf16", 2, 2, 264, 64, 64, 192, 321),
    # RNN with d = 64: its 64 features are the head dimension, the weights need no product and no exponent
    Workload("bwd_tc_rnn", RNN, "bf16", 2, 2, 392, 64, 192, 0, 322),
    Workload("bwd_tc_rnn_k256", RNN, "bf16", 1, 3, 1000, 64, 256, 0, 323),
    # d = 128 (PERFORMER): W and a arrive per step of 128 features, every tile is visited once per 64-column half
    Workload("bwd_tc_d128_m128", PERFORMER, "bf16", 1, 2, 520, 128, 320, 128, 319),
    Workload("bwd_tc_d128_m256", PERFORMER, "bf16", 2, 2, 392, 128, 64, 256, 325),
    Workload("bwd_tc_d128_m64", PERFORMER, "bf16", 1, 3, 264, 128, 128, 64, 326),
    # key side on its tensor-core kernel with a last chunk of 64 keys (k = 320) and with four chunks (k = 512)
    Workload("bwd_tc_k320", PERFORMER, "bf16", 1, 2, 264, 64, 320, 128, 329),
    Workload("bwd_tc_k512_m64", PERFORMER, "bf16", 2, 1, 392, 64, 512, 64, 330),
]


@pytest.mark.parametrize("w", TENSOR_CASES, ids=lambda w: w.name)
def test_backward_tensor_path_matches_oracle(w):
    _check(w)
    assert binding.flurka_last_path() == binding.PATH_TENSOR


def test_backward_tensor_stage1_and_projection_gradients_only():
    """Shapes whose query side has no tensor-core backward still take stage 1 and dK, dV, dE, dF from the
    tensor-core kernels: RNN with d = 128 (two 64-column blocks per head), ragged N, k = 64 and 320."""
    for w, layout in ((Workload("bwd_tc1_rnn_d128", RNN, "bf16", 1, 3, 200, 128, 64, 0, 317), "bhnd"),
                      (Workload("bwd_tc1_rnn_d128_bnhd", RNN, "bf16", 2, 2, 328, 128, 192, 0, 318), "bnhd"),
                      (Workload("bwd_tc1_rnn_d128_k320", RNN, "bf16", 1, 2, 520, 128, 320, 0, 327), "bhnd")):
        _check(w, layout=layout)
        assert binding.flurka_last_path() == binding.PATH_TENSOR_STAGE1


@pytest.mark.parametrize("limit", [1, 2])
def test_backward_tensor_path_with_few_ctas(limit):
    """A CTA's tiles cross from one head to the next: its accumulators of da, db leave and start again."""
    prev = binding.flurka_set_cta_limit(limit)
    try:
        _check(Workload("bwd_tc_few_ctas", PERFORMER, "bf16", 1, 3, 520, 64, 64, 256, 314))
        _check(Workload("bwd_tc_few_ctas_bnhd", PERFORMER, "bf16", 2, 2, 264, 64, 64, 128, 315), layout="bnhd")
        _check(Workload("bwd_tc_few_ctas_rnn", RNN, "bf16", 1, 3, 392, 64, 64, 0, 324), layout="bnhd")
        _check(Workload("bwd_tc_few_ctas_d128", PERFORMER, "bf16", 2, 2, 264, 128, 64, 256, 328), layout="bnhd")
        assert binding.flurka_last_path() == binding.PATH_TENSOR
    finally:
        binding.flurka_set_cta_limit(prev)


def test_backward_full_length_sequences():
    """c3's and c2's sequence lengths and projection sizes with two heads: every gradient against the oracle;
    with few CTAs each one accumulates da, db over 64 tiles of a head before they leave TMEM."""
    from paper_2306_15799_b200 import configs
    w3 = configs.shrink(configs.C3, name="bwd_c3_two_heads", B=1, H=2)
    w2 = configs.shrink(configs.C2, name="bwd_c2_two_heads", B=1, H=2)
    _check(w3)
    assert binding.flurka_last_path() == binding.PATH_TENSOR
    prev = binding.flurka_set_cta_limit(4)
    try:
        _check(w3)
        _check(w2)
        assert binding.flurka_last_path() == binding.PATH_TENSOR
    finally:
        binding.flurka_set_cta_limit(prev)


def test_backward_tensor_path_with_per_head_projections():
    """One pair E_i, F_i per head on a tensor-core shape: stage 1, the key side and the query side on their
    tcgen05 kernels, the products with E, F, K, V on CUDA cores (the tensor-core ones need shared E, F)."""
    _check(Workload("bwd_tc_per_head", PERFORMER, "bf16", 2, 3, 392, 64, 128, 128, 331), per_head=True)
    assert binding.flurka_last_path() == binding.PATH_TENSOR
    _check(Workload("bwd_tc_per_head_rnn_bnhd", RNN, "bf16", 2, 2, 264, 64, 64, 0, 332), layout="bnhd", per_head=True)
    assert binding.flurka_last_path() == binding.PATH_TENSOR


@pytest.mark.parametrize("d,m", [(64, 256), (128, 256)])
def test_backward_in_a_caller_workspace_of_exactly_the_stated_size(d, m):
    """flurka_backward_workspace_bytes covers every scratch area of the tensor-core kernels (the bf16 terms of a
    and of dK', dV', the per-row statistics at d = 128): a caller's block of exactly that size works, a smaller
    one is refused."""
    w = Workload("bwd_ws_d%d" % d, PERFORMER, "bf16", 1, 2, 392, d, 128, m, 340 + d)
    need = binding.flurka_backward_workspace_bytes(w.variant, torch.bfloat16, w.B, w.H, w.N, w.d, w.k, w.m)
    assert need > binding.flurka_workspace_bytes(w.variant, torch.bfloat16, w.B, w.H, w.N, w.d, w.k, w.m)
    x = pu.to_device(synth.make_inputs(w))
    dO = torch.randn_like(x["Q"])
    small = torch.empty(need - 256, dtype=torch.uint8, device="cuda")
    binding.flurka_set_workspace(small)
    try:
        with pytest.raises(binding.FlurkaError) as ei:
            binding.flurka_backward(x["Q"], x["K"], x["V"], x["E"], x["F"], x["W"], dO, w.variant)
        assert ei.value.code == -5
        # poisoned, so that anything the kernels read without having written it shows
        buf = torch.full((need,), 0xFF, dtype=torch.uint8, device="cuda")
        binding.flurka_set_workspace(buf)
        _check(w)
        assert binding.flurka_last_path() == binding.PATH_TENSOR
    finally:
        binding.flurka_set_workspace(None)


def test_backward_cuda_core_path_on_a_tensor_shape():
    prev = binding.flurka_set_path(binding.PATH_SIMT)
    try:
        _check(Workload("bwd_simt_on_tc_shape", PERFORMER, "bf16", 1, 2, 264, 64, 64, 128, 316))
        assert binding.flurka_last_path() == binding.PATH_SIMT
    finally:
        binding.flurka_set_path(prev)


def test_backward_seq_major_layout_and_per_head_projections():
    _check(Workload("bwd_bnhd", PERFORMER, "fp32", 2, 3, 64, 16, 8, 24, 306), layout="bnhd")
    _check(Workload("bwd_per_head", RNN, "fp32", 2, 2, 64, 16, 8, 0, 307), per_head=True)
    _check(Workload("bwd_per_head_perf", PERFORMER, "fp32", 2, 2, 72, 16, 8, 24, 308), per_head=True)


def test_backward_is_the_derivative_of_the_forward():
    """Directional derivative of sum(out * dO) through flurka_forward (fp32) against <gradient, direction>."""
    w = Workload("bwd_fd", PERFORMER, "fp32", 1, 1, 64, 16, 8, 24, 309)
    x = pu.to_device(synth.make_inputs(w))
    gen = torch.Generator().manual_seed(7)
    dO = torch.randn(1, 1, 64, 16, generator=gen).cuda()
    u = torch.randn(1, 1, 64, 16, generator=gen).cuda()
    dQ = binding.flurka_backward(x["Q"], x["K"], x["V"], x["E"], x["F"], x["W"], dO, w.variant)[0]
    h = 1e-2
    f = lambda q: float((binding.flurka_forward(q.contiguous(), x["K"], x["V"], x["E"], x["F"], x["W"], w.variant).double()
                         * dO.double()).sum())
    fd = (f(x["Q"] + h * u) - f(x["Q"] - h * u)) / (2 * h)
    an = float((dQ.double() * u.double()).sum())
    assert abs(fd - an) <= 2e-2 * max(abs(fd), 1e-3), (fd, an)


def test_backward_argument_errors():
    w = Workload("bwd_args", RNN, "fp32", 1, 1, 32, 8, 4, 0, 310)
    x = pu.to_device(synth.make_inputs(w))
    lib = binding.load()
    g = [torch.empty_like(x[n]) for n in ("Q", "K", "V", "E", "F")]
    ptr = lambda t: t.data_ptr()
    base = [ptr(x["Q"]), ptr(x["K"]), ptr(x["V"]), ptr(x["E"]), ptr(x["F"]), None, ptr(g[0])]
    dims = [RNN | 0x100, 1, 1, 32, 8, 4, 0]
    outs = [ptr(t) for t in g]
    assert lib.flurka_backward(*base, *dims, *outs, None) == -8                 # dO is also dQ
    dO = torch.zeros_like(x["Q"])
    base[6] = ptr(dO)
    assert lib.flurka_backward(*base, *dims, outs[0], outs[0], *outs[2:], None) == -8
    assert lib.flurka_backward(*base, *dims, None, *outs[1:], None) == -1
    assert lib.flurka_backward(*base, *dims, *outs, None) == 0
    assert binding.flurka_backward_workspace_bytes(RNN, torch.float32, 1, 1, 32, 8, 4, 0) > 0
