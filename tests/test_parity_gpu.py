"""CUDA path against the fp64 oracle, element by element, through the C ABI."""
import numpy as np
import pytest
import torch

from paper_2306_15799_b200 import binding, build, configs, synth
from paper_2306_15799_b200.configs import PERFORMER, RNN, Workload

import oracle
import parity_util as pu

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module", autouse=True)
def _lib():
    build.build()
    binding.load()


def _wl(name, variant, io, B, H, N, d, k, m, seed):
    return Workload(name, variant, io, B, H, N, d, k, m if variant == PERFORMER else 0, seed)


def test_c1_fp32_exact_config():
    pu.check_all_heads(configs.C1)
    assert binding.flurka_last_path() == binding.PATH_SIMT


SIMT_CASES = [
    # several tiles in every dimension plus ragged tails
    _wl("simt_perf_fp32_ragged", PERFORMER, "fp32", 2, 3, 333, 48, 40, 72, 11),
    _wl("simt_rnn_fp32_ragged", RNN, "fp32", 2, 2, 301, 40, 37, 0, 12),
    _wl("simt_perf_bf16_ragged", PERFORMER, "bf16", 1, 3, 520, 64, 72, 100, 13),
    _wl("simt_rnn_bf16", RNN, "bf16", 2, 2, 512, 64, 64, 0, 14),
    _wl("simt_perf_bf16_d128", PERFORMER, "bf16", 1, 2, 384, 128, 128, 256, 15),
    # degenerate sizes
    _wl("simt_perf_n1", PERFORMER, "fp32", 1, 2, 1, 8, 1, 1, 16),
    _wl("simt_rnn_k1", RNN, "fp32", 1, 1, 65, 1, 1, 0, 17),
    _wl("simt_perf_d1", PERFORMER, "fp32", 1, 1, 40, 1, 3, 5, 18),
]


@pytest.mark.parametrize("w", SIMT_CASES, ids=lambda w: w.name)
def test_simt_path_matches_oracle(w):
    pu.check_all_heads(w, path=binding.PATH_SIMT)
    assert binding.flurka_last_path() == binding.PATH_SIMT
    assert binding.flurka_last_launches() == 3


def test_intermediates_match_oracle():
    """K' = E K and V' = F V (Eq. (2)) and the per-feature log-weights, stage by stage."""
    w = _wl("stage_perf_bf16", PERFORMER, "bf16", 1, 2, 640, 64, 64, 128, 21)
    inputs = synth.make_inputs(w)
    pu.run_gpu(w, inputs, binding.PATH_SIMT)
    Kp = binding.flurka_debug_copy(0, (w.B, w.H, w.k, w.d)).cpu().double().numpy()
    Vp = binding.flurka_debug_copy(1, (w.B, w.H, w.k, w.d)).cpu().double().numpy()
    a = binding.flurka_debug_copy(2, (w.B, w.H, w.m, w.d)).cpu().double().numpy()
    bw = binding.flurka_debug_copy(3, (w.B, w.H, w.m)).cpu().double().numpy()
    torch.cuda.synchronize()
    for h in range(w.H):
        _, inter = pu.oracle_head(inputs, w, 0, h, rows=[0], intermediates=True)
        assert np.abs(Kp[0, h] - inter["Kp"]).max() < 2e-5 * max(1.0, np.abs(inter["Kp"]).max())
        assert np.abs(Vp[0, h] - inter["Vp"]).max() < 2e-5 * max(1.0, np.abs(inter["Vp"]).max())
        # oracle: KV_i = sum_j Phi_ji v'_j, z_i = sum_j Phi_ji  =>  a_i = KV_i / z_i and
        # b_i - b_i' = log z_i - log z_i' (the global stabiliser drops out of differences)
        a_ref = inter["KV"] / inter["z"][:, None]
        big = inter["z"] > 1e-30 * inter["z"].max()
        assert np.abs(a[0, h][big] - a_ref[big]).max() < 5e-3 * max(1.0, np.abs(a_ref[big]).max())
        lz = np.log(inter["z"][big])
        assert np.abs((bw[0, h][big] - bw[0, h][big][0]) - (lz - lz[0])).max() < 5e-3


def test_v_ones_gives_equal_columns_within_projection_range():
    """Convexity invariant (rows of the normalised weights sum to one) on a GPU output."""
    w = _wl("ones_perf_bf16", PERFORMER, "bf16", 1, 2, 512, 64, 64, 64, 31)
    inputs = synth.make_inputs(w)
    inputs["V"] = torch.ones_like(inputs["V"])
    out = pu.run_gpu(w, inputs).float().cpu()
    s = inputs["F"].double().sum(dim=1)
    assert float((out - out[..., :1]).abs().max()) <= 2e-2 * float(s.abs().max())
    assert out.min() >= s.min() - 2e-2 * s.abs().max() and out.max() <= s.max() + 2e-2 * s.abs().max()


def test_host_entry_point_matches_device_entry_point():
    w = _wl("host_perf_bf16", PERFORMER, "bf16", 1, 2, 512, 64, 64, 64, 41)
    inputs = synth.make_inputs(w)
    dev_out = pu.run_gpu(w, inputs).cpu()
    pinned = {n: (t.pin_memory() if t is not None else None) for n, t in inputs.items()}
    host_out = binding.flurka_forward_host(pinned["Q"], pinned["K"], pinned["V"], pinned["E"], pinned["F"],
                                           pinned["W"], w.variant)
    assert torch.equal(host_out, dev_out) or float((host_out.float() - dev_out.float()).abs().max()) < 2e-2


@pytest.mark.parametrize("variant,H", [(PERFORMER, 4), (RNN, 3)])
def test_host_entry_point_in_head_groups(variant, H):
    """Large enough (4 MiB / 3 MiB of Q) for the host entry point to work through the heads in groups,
    copying finished groups back while the next ones are copied in; twice, to re-use its staging."""
    w = _wl("host_groups", variant, "bf16", 2, H, 4096, 64, 64, 64, 42)
    inputs = synth.make_inputs(w)
    dev_out = pu.run_gpu(w, inputs).cpu()
    pinned = {n: (t.pin_memory() if t is not None else None) for n, t in inputs.items()}
    for _ in range(2):
        host_out = binding.flurka_forward_host(pinned["Q"], pinned["K"], pinned["V"], pinned["E"], pinned["F"],
                                               pinned["W"], w.variant)
        assert binding.flurka_last_status() == 0
        # a group of heads is split over CTAs differently from the whole batch, so sums are taken in
        # another order and intermediate roundings differ: outputs agree to a few bf16 ulps (2^-7 each)
        diff = (host_out.float() - dev_out.float()).abs()
        assert bool((diff <= 4 * 2.0 ** -7 * dev_out.float().abs() + 2e-3).all())
    got = host_out.double().numpy()
    for b in range(w.B):
        for h in range(w.H):
            pu.assert_close(got[b, h], pu.oracle_head(inputs, w, b, h), "bf16", "host entry point, head (%d,%d)" % (b, h))


@pytest.mark.parametrize("variant,heads", [(PERFORMER, 12), (PERFORMER, 10), (RNN, 12)])
def test_host_entry_point_with_unequal_head_groups(variant, heads):
    """1 MiB of Q per head, so the host entry point takes 12 (10) heads in eight groups of 1 and 2 heads:
    the workspace layout differs from group to group.  PERFORMER with k = 256 and so few heads per group
    also splits the keys of stage 2 over two CTAs, whose arrival counters live next to the status words."""
    w = _wl("host_uneven_groups", variant, "bf16", 1, heads, 8192, 64, 256, 256, 43 + heads)
    inputs = synth.make_inputs(w)
    pinned = {n: (t.pin_memory() if t is not None else None) for n, t in inputs.items()}
    # a small problem first, so that the library-owned workspace has to grow inside the big call
    small = _wl("host_uneven_small", variant, "bf16", 1, 1, 256, 64, 64, 64, 44)
    pu.run_gpu(small, synth.make_inputs(small))
    for _ in range(2):
        host_out = binding.flurka_forward_host(pinned["Q"], pinned["K"], pinned["V"], pinned["E"], pinned["F"],
                                               pinned["W"], w.variant)
        assert binding.flurka_last_status() == 0
        assert binding.flurka_last_path() == binding.PATH_TENSOR
    got = host_out.double().numpy()
    assert np.isfinite(got).all()
    for h in range(w.H):
        pu.assert_close(got[0, h], pu.oracle_head(inputs, w, 0, h), "bf16", "host entry point, head %d of %d" % (h, heads))


def test_caller_workspace_and_too_small_workspace():
    w = _wl("ws_rnn_bf16", RNN, "bf16", 1, 2, 256, 64, 64, 0, 51)
    inputs = synth.make_inputs(w)
    need = binding.flurka_workspace_bytes(w.variant, torch.bfloat16, w.B, w.H, w.N, w.d, w.k, w.m)
    assert need > 0
    dev = pu.to_device(inputs)
    small = torch.empty(need - 256, dtype=torch.uint8, device="cuda")
    binding.flurka_set_workspace(small)
    try:
        with pytest.raises(binding.FlurkaError) as ei:
            binding.flurka_forward(dev["Q"], dev["K"], dev["V"], dev["E"], dev["F"], None, w.variant)
        assert ei.value.code == -5
        buf = torch.full((need,), 0xFF, dtype=torch.uint8, device="cuda")     # poisoned: nothing may be read unwritten
        binding.flurka_set_workspace(buf)
        out = binding.flurka_forward(dev["Q"], dev["K"], dev["V"], dev["E"], dev["F"], None, w.variant)
        torch.cuda.synchronize()
    finally:
        binding.flurka_set_workspace(None)
    ref = pu.oracle_head(inputs, w, 0, 1)
    pu.assert_close(out[0, 1].cpu().double().numpy(), ref, "bf16", "caller workspace")


def test_performer_tensor_path_in_a_poisoned_caller_workspace():
    """The PERFORMER tensor path (key split included: k = 256, two heads) in a caller's block of exactly the
    stated size that was filled with 0xFF: every scratch area is written before it is read."""
    w = _wl("ws_perf_bf16", PERFORMER, "bf16", 1, 2, 520, 64, 256, 256, 52)
    inputs = synth.make_inputs(w)
    need = binding.flurka_workspace_bytes(w.variant, torch.bfloat16, w.B, w.H, w.N, w.d, w.k, w.m)
    dev = pu.to_device(inputs)
    buf = torch.full((need,), 0xFF, dtype=torch.uint8, device="cuda")
    binding.flurka_set_workspace(buf)
    try:
        out = binding.flurka_forward(dev["Q"], dev["K"], dev["V"], dev["E"], dev["F"], dev["W"], w.variant)
        torch.cuda.synchronize()
        assert binding.flurka_last_status() == 0 and binding.flurka_last_path() == binding.PATH_TENSOR
    finally:
        binding.flurka_set_workspace(None)
    for h in range(2):
        pu.assert_close(out[0, h].cpu().double().numpy(), pu.oracle_head(inputs, w, 0, h), "bf16", "poisoned workspace head %d" % h)


def test_repeated_calls_are_independent():
    """The workspace is re-zeroed every call: a second call on other data is not polluted."""
    w1 = _wl("rep_a", PERFORMER, "bf16", 1, 2, 256, 64, 64, 64, 61)
    w2 = _wl("rep_b", PERFORMER, "bf16", 1, 2, 256, 64, 64, 64, 62)
    i1, i2 = synth.make_inputs(w1), synth.make_inputs(w2)
    pu.run_gpu(w1, i1)
    o2 = pu.run_gpu(w2, i2).cpu().double().numpy()
    o2b = pu.run_gpu(w2, i2).cpu().double().numpy()
    pu.assert_close(o2[0, 0], pu.oracle_head(i2, w2, 0, 0), "bf16", "second call")
    assert np.abs(o2 - o2b).max() <= 2e-2


# ------------------------------------------------------------------------------- tensor-core path
TENSOR_CASES = [
    _wl("tc_perf_d64_k256_m256", PERFORMER, "bf16", 1, 3, 1024, 64, 256, 256, 101),
    _wl("tc_perf_d64_k64_m64", PERFORMER, "bf16", 2, 2, 512, 64, 64, 64, 102),
    _wl("tc_perf_d64_k128_m128", PERFORMER, "bf16", 1, 5, 768, 64, 128, 128, 103),
    _wl("tc_perf_d128_k512_m256", PERFORMER, "bf16", 1, 2, 1024, 128, 512, 256, 104),
    _wl("tc_perf_d128_k192_m192", PERFORMER, "bf16", 1, 3, 640, 128, 192, 192, 105),
    _wl("tc_rnn_d64_k256", RNN, "bf16", 2, 3, 1024, 64, 256, 0, 106),
    _wl("tc_rnn_d128_k64", RNN, "bf16", 1, 2, 512, 128, 64, 0, 107),
    # one 128-row tile per head, and key counts whose last 128-key chunk holds 64 keys
    _wl("tc_perf_d64_k320_m256_n128", PERFORMER, "bf16", 1, 2, 128, 64, 320, 256, 109),
    _wl("tc_perf_d128_k448_m128", PERFORMER, "bf16", 2, 1, 256, 128, 448, 128, 110),
    _wl("tc_rnn_d128_k512_n128", RNN, "bf16", 1, 1, 128, 128, 512, 0, 111),
    # sequence lengths that are not multiples of the 64-wide chunks of stage 1 or the 128-row tiles of stage 3
    _wl("tc_perf_d64_n1000", PERFORMER, "bf16", 1, 3, 1000, 64, 128, 256, 115),
    _wl("tc_rnn_d128_n200", RNN, "bf16", 2, 1, 200, 128, 64, 0, 116),
    _wl("tc_perf_d128_n72", PERFORMER, "bf16", 1, 2, 72, 128, 64, 64, 117),
    # two and four 256-column groups with 256-row tiles in stage 1
    _wl("tc_perf_d64_k256_pairs", PERFORMER, "bf16", 2, 4, 1024, 64, 256, 128, 113),
    _wl("tc_rnn_d128_k512_pairs", RNN, "bf16", 2, 4, 512, 128, 512, 0, 114),
]


@pytest.mark.parametrize("w", TENSOR_CASES, ids=lambda w: w.name)
def test_tensor_stage1_projections_match_oracle(w):
    """K' = E K, V' = F V from the tcgen05 down-projection, element by element."""
    inputs = synth.make_inputs(w)
    pu.run_gpu(w, inputs, binding.PATH_TENSOR_STAGE1)
    assert binding.flurka_last_path() == binding.PATH_TENSOR_STAGE1
    Kp = binding.flurka_debug_copy(0, (w.B, w.H, w.k, w.d)).cpu().double().numpy()
    Vp = binding.flurka_debug_copy(1, (w.B, w.H, w.k, w.d)).cpu().double().numpy()
    torch.cuda.synchronize()
    for b in range(w.B):
        for h in range(w.H):
            _, inter = pu.oracle_head(inputs, w, b, h, rows=[0], intermediates=True)
            for got, ref, nm in ((Kp[b, h], inter["Kp"], "K'"), (Vp[b, h], inter["Vp"], "V'")):
                err = np.abs(got - ref).max()
                assert err < 3e-5 * max(1.0, np.abs(ref).max()), "%s %s head (%d,%d): %.3e" % (w.name, nm, b, h, err)


@pytest.mark.parametrize("limit", [0, 3])
@pytest.mark.parametrize("w", TENSOR_CASES, ids=lambda w: w.name)
def test_tensor_stage3_matches_oracle(w, limit):
    """tcgen05 query side (several tiles per CTA and head changes when the CTA count is limited)."""
    prev = binding.flurka_set_cta_limit(limit)
    try:
        pu.check_all_heads(w, path=binding.PATH_TENSOR_STAGE3)
    finally:
        binding.flurka_set_cta_limit(prev)


@pytest.mark.parametrize("w", TENSOR_CASES, ids=lambda w: w.name)
def test_tensor_stage2_matches_oracle(w):
    """tcgen05 key side (with the tcgen05 query side behind it) on CUDA-core projections; also the
    per-feature log-weights against the oracle's z (differences, the global stabiliser drops out)."""
    inputs = synth.make_inputs(w)
    out = pu.run_gpu(w, inputs, binding.PATH_TENSOR_STAGE23).cpu().double().numpy()
    p = w.m if w.variant == PERFORMER else w.d
    bw = binding.flurka_debug_copy(3, (w.B, w.H, p)).cpu().double().numpy()
    torch.cuda.synchronize()
    for b in range(w.B):
        for h in range(w.H):
            ref, inter = pu.oracle_head(inputs, w, b, h, intermediates=True)
            pu.assert_close(out[b, h], ref, w.io, "%s head (%d,%d)" % (w.name, b, h))
            z = inter["z"]
            big = z > 1e-30 * z.max()
            if w.variant == PERFORMER:
                lz = np.log(z[big])
                got = bw[b, h][big]
                assert np.abs((got - got[0]) - (lz - lz[0])).max() < 5e-3
            else:
                assert np.abs(bw[b, h] / z - 1.0).max() < 2e-3


@pytest.mark.parametrize("limit", [0, 5])
@pytest.mark.parametrize("w", TENSOR_CASES, ids=lambda w: w.name)
def test_tensor_path_matches_oracle(w, limit):
    prev = binding.flurka_set_cta_limit(limit)
    try:
        pu.check_all_heads(w, path=binding.PATH_TENSOR)
        assert binding.flurka_last_path() == binding.PATH_TENSOR
        assert binding.flurka_last_launches() == 3
    finally:
        binding.flurka_set_cta_limit(prev)


@pytest.mark.parametrize("limit,tiles", [(1, 1), (2, 3), (3, 1)])
def test_rnn_head_change_at_a_ctas_second_tile(limit, tiles):
    """RNN query side: a row-owner group whose first tile already belongs to the CTA's second head must still
    get that head's scale vector (tiles of one head per CTA: 1 or 3, so the odd group starts in a later head).
    Repeated, because a stale vector shows only when the group runs ahead of the operand builder."""
    from paper_2306_15799_b200.configs import Workload
    w = Workload("rnn_head_change_t%d" % tiles, RNN, "bf16", 2, 5, 128 * tiles, 64, 64, 0, 417 + tiles)
    prev = binding.flurka_set_cta_limit(limit)
    try:
        for _ in range(6):
            pu.check_all_heads(w, path=binding.PATH_TENSOR)
    finally:
        binding.flurka_set_cta_limit(prev)


def test_rnn_forward_is_repeatable_with_every_sm_busy():
    """Twelve runs of an RNN forward with 148 CTAs whose tile ranges cross heads at every position: apart from the
    order of stage 1's fp32 partial sums (which RNN features do not amplify) nothing may differ from run to run.
    A stale per-head operand shows here as a difference of many units in the last place."""
    w = Workload("rnn_repeatable", RNN, "bf16", 2, 12, 4096, 64, 256, 0, 431)
    dev = pu.to_device(synth.make_inputs(w))
    first = None
    for _ in range(12):
        out = binding.flurka_forward(dev["Q"], dev["K"], dev["V"], dev["E"], dev["F"], dev["W"], w.variant).float()
        torch.cuda.synchronize()
        assert binding.flurka_last_status() == 0 and binding.flurka_last_path() == binding.PATH_TENSOR
        if first is None:
            first = out.clone()
            continue
        spacing = torch.clamp(first.abs(), min=1e-2) * 2.0 ** -7          # bf16 spacing of the first run's values
        assert float(((out - first).abs() / spacing).max()) <= 2.0


def test_auto_picks_tensor_path_when_the_shape_allows():
    w = TENSOR_CASES[0]
    pu.check_all_heads(w)
    assert binding.flurka_last_path() == binding.PATH_TENSOR
    odd = _wl("auto_simt", PERFORMER, "bf16", 1, 1, 204, 64, 64, 64, 108)      # N % 8 != 0
    pu.check_all_heads(odd)
    assert binding.flurka_last_path() == binding.PATH_SIMT


@pytest.mark.parametrize("scale", [2.0, 0.05])
def test_tensor_path_with_large_and_small_logits(scale):
    """Q and K scaled away from the benchmark recipe: logits of several tens (sharply peaked
    weights, every stabiliser at work) and logits near zero (almost uniform weights)."""
    w = _wl("tc_perf_scaled", PERFORMER, "bf16", 1, 2, 512, 64, 128, 256, 112)
    inputs = synth.make_inputs(w)
    for name in ("Q", "K"):
        inputs[name] = (inputs[name].double() * scale).to(inputs[name].dtype)
    out = pu.run_gpu(w, inputs, binding.PATH_TENSOR).cpu().double().numpy()
    assert binding.flurka_last_path() == binding.PATH_TENSOR
    assert np.isfinite(out).all()
    for h in range(w.H):
        pu.assert_close(out[0, h], pu.oracle_head(inputs, w, 0, h), "bf16", "scaled x%g head %d" % (scale, h))


# ------------------------------------------------------------------------------- [B,N,H,d] tensors
BNHD_CASES = [
    (_wl("bnhd_tc_perf", PERFORMER, "bf16", 2, 3, 640, 64, 128, 256, 121), binding.PATH_TENSOR),
    (_wl("bnhd_tc_rnn_d128", RNN, "bf16", 1, 4, 384, 128, 256, 0, 122), binding.PATH_TENSOR),
    (_wl("bnhd_tc_perf_8groups", PERFORMER, "bf16", 2, 8, 512, 64, 256, 64, 123), binding.PATH_TENSOR),
    (_wl("bnhd_simt_perf_fp32", PERFORMER, "fp32", 2, 3, 200, 24, 20, 40, 124), binding.PATH_SIMT),
    (_wl("bnhd_simt_rnn_bf16", RNN, "bf16", 1, 2, 300, 64, 48, 0, 125), binding.PATH_SIMT),
]


@pytest.mark.parametrize("w,path", BNHD_CASES, ids=lambda v: v.name if hasattr(v, "name") else str(v))
def test_heads_merged_into_the_row(w, path):
    """Q, K, V, out as [B,N,H,d]: the same inputs, transposed, must give the transposed output of the
    oracle (which works head by head)."""
    inputs = synth.make_inputs(w)
    dev = pu.to_device(inputs)
    t = {n: dev[n].transpose(1, 2).contiguous() for n in ("Q", "K", "V")}
    prev = binding.flurka_set_path(path)
    try:
        out = binding.flurka_forward(t["Q"], t["K"], t["V"], dev["E"], dev["F"], dev["W"], w.variant, layout="bnhd")
        torch.cuda.synchronize()
        assert binding.flurka_last_status() == 0
        assert binding.flurka_last_path() == path
    finally:
        binding.flurka_set_path(prev)
    assert out.shape == (w.B, w.N, w.H, w.d)
    got = out.transpose(1, 2).cpu().double().numpy()
    for b in range(w.B):
        for h in range(w.H):
            pu.assert_close(got[b, h], pu.oracle_head(inputs, w, b, h), w.io, "%s head (%d,%d)" % (w.name, b, h))


def test_heads_merged_into_the_row_host_entry():
    w = _wl("bnhd_host", PERFORMER, "bf16", 4, 2, 4096, 64, 64, 64, 126)      # 4 MiB of Q: four groups of one batch
    inputs = synth.make_inputs(w)
    pinned = {n: (inputs[n].transpose(1, 2).contiguous().pin_memory() if n in ("Q", "K", "V") else
                  (inputs[n].pin_memory() if inputs[n] is not None else None)) for n in inputs}
    out = binding.flurka_forward_host(pinned["Q"], pinned["K"], pinned["V"], pinned["E"], pinned["F"], pinned["W"],
                                      w.variant, layout="bnhd")
    assert binding.flurka_last_status() == 0
    got = out.transpose(1, 2).double().numpy()
    for b in range(w.B):
        for h in range(w.H):
            pu.assert_close(got[b, h], pu.oracle_head(inputs, w, b, h), "bf16", "host, head (%d,%d)" % (b, h))


# ----------------------------------------------------------------------------- one E_i, F_i per head
def _per_head_inputs(w):
    """The workload's inputs with E, F redrawn as [H,k,N]: one projection pair per head (Theorem 1)."""
    x = synth.make_inputs(w)
    gen = torch.Generator().manual_seed(w.seed + 17)
    for name in ("E", "F"):
        x[name] = (torch.randn(w.H, w.k, w.N, generator=gen, dtype=torch.float64) * float(w.k) ** -0.5).to(x["Q"].dtype)
    return x


def _check_per_head(w, x, out):
    f64 = lambda t: t.double().numpy()
    W = f64(x["W"]) if x["W"] is not None else None
    got = out.cpu().double().numpy()
    for b in range(w.B):
        for h in range(w.H):
            ref = oracle.head(f64(x["Q"][b, h]), f64(x["K"][b, h]), f64(x["V"][b, h]), f64(x["E"][h]), f64(x["F"][h]),
                              W, w.variant)
            pu.assert_close(got[b, h], ref, w.io, "%s per-head E, F, head (%d,%d)" % (w.name, b, h))


PER_HEAD_CASES = [
    (_wl("ph_simt_perf_fp32", PERFORMER, "fp32", 2, 3, 200, 24, 20, 40, 81), binding.PATH_SIMT),
    (_wl("ph_simt_rnn_bf16", RNN, "bf16", 1, 2, 264, 64, 40, 0, 82), binding.PATH_SIMT),
    (_wl("ph_tensor_perf_d64", PERFORMER, "bf16", 2, 3, 1024, 64, 128, 128, 83), binding.PATH_TENSOR),
    (_wl("ph_tensor_perf_d128_k512", PERFORMER, "bf16", 1, 2, 768, 128, 512, 256, 84), binding.PATH_TENSOR),
    (_wl("ph_tensor_rnn", RNN, "bf16", 2, 2, 1000, 64, 64, 0, 85), binding.PATH_TENSOR),
]


@pytest.mark.parametrize("w,path", PER_HEAD_CASES, ids=lambda v: v.name if hasattr(v, "name") else str(v))
def test_per_head_projections(w, path):
    import oracle  # noqa: F401
    x = _per_head_inputs(w)
    out = pu.run_gpu(w, x, path)
    assert binding.flurka_last_path() == path
    _check_per_head(w, x, out)


def test_per_head_projections_seq_major_and_host_entry():
    """[B,N,H,d] tensors with one E_i, F_i per head, and the host entry point, whose head groups must be
    whole batches so that every head keeps its own pair."""
    w = _wl("ph_host", PERFORMER, "bf16", 3, 4, 2048, 64, 128, 128, 86)
    x = _per_head_inputs(w)
    dev = pu.to_device(x)
    t = lambda a: a.transpose(1, 2).contiguous()
    out = binding.flurka_forward(t(dev["Q"]), t(dev["K"]), t(dev["V"]), dev["E"], dev["F"], dev["W"], w.variant, layout="bnhd")
    torch.cuda.synchronize()
    assert binding.flurka_last_status() == 0
    _check_per_head(w, x, out.transpose(1, 2))
    pinned = {n: (a.pin_memory() if a is not None else None) for n, a in x.items()}
    host_out = binding.flurka_forward_host(pinned["Q"], pinned["K"], pinned["V"], pinned["E"], pinned["F"], pinned["W"], w.variant)
    assert binding.flurka_last_status() == 0
    _check_per_head(w, x, host_out)


# ----------------------------------------------------------------------------- stage 1 as CTA pairs
@pytest.mark.parametrize("shape", [(1, 4, 1024, 64, 256), (2, 2, 1536, 128, 512), (1, 12, 1000, 64, 256), (3, 4, 640, 64, 512)],
                         ids=lambda s: "B%d_H%d_N%d_d%d_k%d" % s)
def test_stage1_pairs_and_single_ctas_match_oracle(shape):
    """The down-projection as pairs of CTAs (two-CTA MMAs; k a multiple of 256 and B*H*d a multiple of 256)
    and as single CTAs: K' = E K and V' = F V of every head against the oracle, both ways, with the ragged
    last chunk, one and two 256-column halves per pair, and both halves of k = 512."""
    B, H, N, d, k = shape
    w = _wl("stage1_pairs", PERFORMER, "bf16", B, H, N, d, k, 64, 97 + N)
    x = synth.make_inputs(w)
    f64 = lambda t: t.double().numpy()
    for on in (True, False):
        prev = binding.flurka_set_stage1_pairs(on)
        try:
            out = pu.run_gpu(w, x, binding.PATH_TENSOR)
            Kp = binding.flurka_debug_copy(0, (w.B, w.H, w.k, w.d)).cpu().double().numpy()
            Vp = binding.flurka_debug_copy(1, (w.B, w.H, w.k, w.d)).cpu().double().numpy()
            torch.cuda.synchronize()
        finally:
            binding.flurka_set_stage1_pairs(prev)
        for b in range(B):
            for h in range(H):
                for got, want in ((Kp[b, h], f64(x["E"]) @ f64(x["K"][b, h])), (Vp[b, h], f64(x["F"]) @ f64(x["V"][b, h]))):
                    assert np.abs(got - want).max() <= 3e-5 * max(1.0, np.abs(want).max())
        got = out.cpu().double().numpy()
        pu.assert_close(got[B - 1, H - 1], pu.oracle_head(x, w, B - 1, H - 1), "bf16", "stage 1 %s" % ("pairs" if on else "single"))
