"""Pins for the fp64 oracle: closed forms, invariants, brute force and the softmax limit.

Each ``pin_*`` function takes an ``oracle.OracleLib`` and raises AssertionError when the
library under test disagrees with what the paper (arxiv 2306.15799) and the mathematics
fix.  ``test_planted_mistakes_are_caught`` rebuilds the oracle source with one planted
mistake at a time and requires at least one pin to fail for each.
"""
import math
import os

import numpy as np
import pytest

import oracle
from oracle import PERFORMER, RNN

GOLDEN = os.path.join(os.path.dirname(os.path.abspath(__file__)), "golden")


# ----------------------------------------------------------------------------- helpers
def _rng(seed):
    return np.random.default_rng(seed)


def _tiny(seed, N=24, d=6, k=5, m=12, scale=0.5):
    r = _rng(seed)
    Q = r.normal(size=(N, d)) * scale
    K = r.normal(size=(N, d)) * scale
    V = r.normal(size=(N, d))
    E = r.normal(size=(k, N)) / math.sqrt(k)
    F = r.normal(size=(k, N)) / math.sqrt(k)
    W = r.normal(size=(m, d))
    return Q, K, V, E, F, W


def _softmax_rows(S):
    S = S - S.max(axis=1, keepdims=True)
    P = np.exp(S)
    return P / P.sum(axis=1, keepdims=True)


def _rel(a, b):
    return np.linalg.norm(a - b) / max(np.linalg.norm(b), 1e-300)


# ----------------------------------------------------------------------------- pins
def pin_quadratic_equals_associative(orc):
    """Section 2.1: the linear-cost ordering is the same product as the N x k form (App. D weights)."""
    for variant in (PERFORMER, RNN):
        for seed in (1, 2, 3):
            Q, K, V, E, F, W = _tiny(seed, N=40, d=7, k=9, m=20)
            Wv = W if variant == PERFORMER else None
            for stab in (False, True):
                a = orc.head(Q, K, V, E, F, Wv, variant, stabilise=stab)
                q, Ahat = orc.head_quadratic(Q, K, V, E, F, Wv, variant, stabilise=stab, weights=True)
                assert _rel(a, q) < 1e-11, ("assoc vs quadratic", variant, stab, _rel(a, q))
                assert np.all(Ahat >= 0) and np.allclose(Ahat.sum(axis=1), 1.0, atol=1e-12)
                # the quadratic form really is Ahat @ V'
                Vp = F @ V
                assert _rel(q, Ahat @ Vp) < 1e-12


def pin_identity_projection(orc):
    """k = N, E = F = I reduces Eq. (2) to plain kernel attention (Section 2.1), written here in numpy."""
    Q, K, V, _, _, W = _tiny(11, N=16, d=5, k=16, m=10)
    I = np.eye(16)
    # Performer
    def phi_perf(X):
        return np.exp(X @ W.T - 0.5 * (X * X).sum(axis=1, keepdims=True)) / math.sqrt(W.shape[0])
    fq, fk = phi_perf(Q), phi_perf(K)
    ref = (fq @ (fk.T @ V)) / (fq @ fk.sum(axis=0))[:, None]
    got = orc.head(Q, K, V, I, I, W, PERFORMER, stabilise=True)
    assert _rel(got, ref) < 1e-11, _rel(got, ref)
    # RNN
    def phi_elu(X):
        return np.where(X > 0, X + 1.0, np.exp(X))
    fq, fk = phi_elu(Q), phi_elu(K)
    ref = (fq @ (fk.T @ V)) / (fq @ fk.sum(axis=0))[:, None]
    got = orc.head(Q, K, V, I, I, None, RNN)
    assert _rel(got, ref) < 1e-12, _rel(got, ref)


def pin_projection_is_E_times_K(orc):
    """Eq. (2): K' = E K and V' = F V with E, F of shape k x N (Section 2.1); numpy matmul is the routine."""
    Q, K, V, E, F, W = _tiny(21, N=33, d=4, k=6, m=8)
    _, inter = orc.head(Q, K, V, E, F, W, PERFORMER, intermediates=True)
    assert _rel(inter["Kp"], E @ K) < 1e-13
    assert _rel(inter["Vp"], F @ V) < 1e-13


def pin_convexity(orc):
    """App. D: weights are non-negative and sum to one, so O lies in the column-wise hull of V'."""
    for variant in (PERFORMER, RNN):
        Q, K, V, E, F, W = _tiny(31, N=50, d=6, k=7, m=16)
        Wv = W if variant == PERFORMER else None
        O = orc.head(Q, K, V, E, F, Wv, variant)
        Vp = F @ V
        assert np.all(O <= Vp.max(axis=0) + 1e-12) and np.all(O >= Vp.min(axis=0) - 1e-12)
        # V = 1 and F 1_N = 1_k  =>  V' = 1  =>  O = 1
        Fn = np.abs(F)
        Fn /= Fn.sum(axis=1, keepdims=True)
        O1 = orc.head(Q, K, np.ones_like(V), E, Fn, Wv, variant)
        assert np.allclose(O1, 1.0, atol=1e-12)
        # V = 1 with a general F: all columns equal and inside [min_j s_j, max_j s_j], s = F 1
        O2 = orc.head(Q, K, np.ones_like(V), E, F, Wv, variant)
        s = F.sum(axis=1)
        assert np.allclose(O2, O2[:, :1], atol=1e-12)
        assert O2.min() >= s.min() - 1e-12 and O2.max() <= s.max() + 1e-12


def pin_single_projected_key(orc):
    """k = 1: the one weight is 1 for every query, so every output row equals F V."""
    for variant in (PERFORMER, RNN):
        Q, K, V, E, F, W = _tiny(41, N=20, d=5, k=1, m=6)
        Wv = W if variant == PERFORMER else None
        O = orc.head(Q, K, V, E, F, Wv, variant)
        assert np.allclose(O, np.broadcast_to(F @ V, O.shape), atol=1e-12)


def pin_single_feature_is_softmax_over_keys(orc):
    """m = 1: phi(q) cancels and O_n = sum_j softmax_j(w.k'_j - |k'_j|^2/2) V'_j for every n."""
    Q, K, V, E, F, W = _tiny(51, N=18, d=5, k=7, m=1)
    Kp, Vp = E @ K, F @ V
    logits = (Kp @ W.T)[:, 0] - 0.5 * (Kp * Kp).sum(axis=1)
    p = _softmax_rows(logits[None, :])[0]
    ref = np.broadcast_to(p @ Vp, (Q.shape[0], V.shape[1]))
    for stab in (False, True):
        O = orc.head(Q, K, V, E, F, W, PERFORMER, stabilise=stab)
        assert _rel(O, ref) < 1e-12, _rel(O, ref)


def pin_scale_invariance(orc):
    """The stabilisers are scalars that cancel in the ratio: stabilised == literal evaluation."""
    Q, K, V, E, F, W = _tiny(61, N=30, d=6, k=8, m=24)
    a = orc.head(Q, K, V, E, F, W, PERFORMER, stabilise=False)
    b = orc.head(Q, K, V, E, F, W, PERFORMER, stabilise=True)
    assert _rel(a, b) < 1e-12
    # and the stabilised path survives exponents that underflow fp64 when taken literally
    big = 12.0
    c = orc.head(Q, K * big, V, E * 4, F, W, PERFORMER, stabilise=True)
    assert np.all(np.isfinite(c))
    Vp = F @ V
    assert np.all(c <= Vp.max(axis=0) + 1e-9) and np.all(c >= Vp.min(axis=0) - 1e-9)
    cq = orc.head_quadratic(Q, K * big, V, E * 4, F, W, PERFORMER, stabilise=True)
    assert _rel(c, cq) < 1e-9


def pin_symmetries(orc):
    """Linearity in V; permutations of queries, of the sequence axis, of projected keys and of features."""
    r = _rng(71)
    for variant in (PERFORMER, RNN):
        Q, K, V, E, F, W = _tiny(72, N=26, d=5, k=6, m=10)
        Wv = W if variant == PERFORMER else None
        O = orc.head(Q, K, V, E, F, Wv, variant)
        V2 = r.normal(size=V.shape)
        O2 = orc.head(Q, K, V2, E, F, Wv, variant)
        O12 = orc.head(Q, K, 2.0 * V - 3.0 * V2, E, F, Wv, variant)
        assert _rel(O12, 2.0 * O - 3.0 * O2) < 1e-11
        pq = r.permutation(Q.shape[0])
        assert _rel(orc.head(Q[pq], K, V, E, F, Wv, variant), O[pq]) < 1e-12
        ps = r.permutation(Q.shape[0])
        assert _rel(orc.head(Q, K[ps], V[ps], E[:, ps], F[:, ps], Wv, variant), O) < 1e-11
        pk = r.permutation(E.shape[0])
        assert _rel(orc.head(Q, K, V, E[pk], F[pk], Wv, variant), O) < 1e-11
        if variant == PERFORMER:
            pf = r.permutation(W.shape[0])
            assert _rel(orc.head(Q, K, V, E, F, W[pf], variant), O) < 1e-11
        # row subset selection returns the same rows
        rows = np.array([3, 0, 25, 7])
        assert _rel(orc.head(Q, K, V, E, F, Wv, variant, rows=rows), O[rows]) < 1e-13
        assert _rel(orc.head_quadratic(Q, K, V, E, F, Wv, variant, rows=rows), O[rows]) < 1e-11


def pin_rnn_worked_example(orc):
    """The hand-worked N=1, d=1, k=2 example in tests/golden/rnn_worked_example.txt."""
    vals = {}
    with open(os.path.join(GOLDEN, "rnn_worked_example.txt")) as fh:
        for line in fh:
            if line.startswith("#") or not line.strip():
                continue
            key, *nums = line.split()
            vals[key] = np.array([float(x) for x in nums])
    Q = vals["Q"].reshape(1, 1); K = vals["K"].reshape(1, 1); V = vals["V"].reshape(1, 1)
    E = vals["E"].reshape(2, 1); F = vals["F"].reshape(2, 1)
    for fn in (orc.head, orc.head_quadratic):
        O = fn(Q, K, V, E, F, None, RNN)
        assert abs(O[0, 0] - vals["O"][0]) < 1e-14, O
    # elu + 1 at a few points, including 0 where both branches meet
    x = np.array([[-2.0, -0.5, 0.0, 0.5, 3.0]])
    phi = orc.features(x, None, RNN)
    assert np.allclose(phi, [[math.exp(-2.0), math.exp(-0.5), 1.0, 1.5, 4.0]], atol=1e-15)


def pin_feature_expectation(orc):
    """Section 2.1: E[psi_i(x) psi_i(y)] = exp(x.y) for w_i ~ N(0, I); phi(x).phi(y) is the sample mean.

    With m i.i.d. features the mean is within 5 sample standard errors of exp(x.y) (CLT; for the
    fixed seed below the check is deterministic).
    """
    r = _rng(81)
    d, m = 6, 200000
    W = r.normal(size=(m, d))
    X = r.normal(size=(4, d)) * 0.35
    Y = r.normal(size=(4, d)) * 0.35
    fx = orc.features(X, W, PERFORMER, stabilise=False)
    fy = orc.features(Y, W, PERFORMER, stabilise=False)
    for a in range(4):
        for b in range(4):
            prod = fx[a] * fy[b] * m          # psi_i(x) psi_i(y)
            est = fx[a] @ fy[b]               # phi(x).phi(y)
            target = math.exp(X[a] @ Y[b])
            se = prod.std(ddof=1) / math.sqrt(m)
            assert abs(est - target) <= 5.0 * se, (a, b, est, target, se)
            assert abs(est - prod.mean()) < 1e-12 * max(1.0, abs(est))
    # the stabiliser is a pure rescaling of each row (query side) or of the whole matrix (key side)
    Wm = W[:64]
    raw = orc.features(X, Wm, PERFORMER, stabilise=False)
    per_row = orc.features(X, Wm, PERFORMER, stabilise=True, scope_global=False)
    glob = orc.features(X, Wm, PERFORMER, stabilise=True, scope_global=True)
    ratio_row = per_row / raw
    assert np.allclose(ratio_row, ratio_row[:, :1], rtol=1e-12)
    ratio_glob = glob / raw
    assert np.allclose(ratio_glob, ratio_glob[0, 0], rtol=1e-12)
    assert np.isclose(per_row.max(axis=1), 1.0 / math.sqrt(64)).all()
    assert np.isclose(glob.max(), 1.0 / math.sqrt(64))


def pin_softmax_limit(orc):
    """Theorem 1's proof sketch: phi(x).phi(y) -> exp(x.y) as m grows, so the output tends to
    softmax(Q K'^T) V' (the Linformer form of Section 2.1); Monte-Carlo error decays like m^-1/2."""
    from paper_2306_15799_b200.synth import block_orthogonal_features
    import torch

    r = _rng(91)
    N, d, k = 32, 16, 8
    Q = r.normal(size=(N, d)) * d ** -0.25 * 0.5
    K = r.normal(size=(N, d)) * d ** -0.25 * 0.5
    V = r.normal(size=(N, d))
    E = r.normal(size=(k, N)) / math.sqrt(k) * 0.5
    F = r.normal(size=(k, N)) / math.sqrt(k)
    Kp, Vp = E @ K, F @ V
    target = _softmax_rows(Q @ Kp.T) @ Vp
    ms = [64, 256, 1024, 4096, 16384]
    errs = []
    for m in ms:
        e = []
        for seed in range(8):
            g = torch.Generator().manual_seed(1000 * m + seed)
            W = block_orthogonal_features(m, d, g).numpy()
            O = orc.head(Q, K, V, E, F, W, PERFORMER)
            e.append(_rel(O, target))
        errs.append(float(np.mean(e)))
    slope = np.polyfit(np.log(ms), np.log(errs), 1)[0]
    assert -0.62 <= slope <= -0.33, (slope, errs)
    assert errs[-1] < 0.05 and errs[-1] < 0.2 * errs[0], errs


def pin_forward_layout(orc):
    """[B,H,N,d] batching: every (b,h) slice is the single-head result with the shared E, F, W."""
    r = _rng(101)
    B, H, N, d, k, m = 2, 3, 12, 4, 5, 8
    Q = r.normal(size=(B, H, N, d)) * 0.5
    K = r.normal(size=(B, H, N, d)) * 0.5
    V = r.normal(size=(B, H, N, d))
    E = r.normal(size=(k, N)) / math.sqrt(k)
    F = r.normal(size=(k, N)) / math.sqrt(k)
    W = r.normal(size=(m, d))
    for variant, Wv in ((PERFORMER, W), (RNN, None)):
        O = orc.forward(Q, K, V, E, F, Wv, variant)
        for b in range(B):
            for h in range(H):
                ref = orc.head_quadratic(Q[b, h], K[b, h], V[b, h], E, F, Wv, variant)
                assert _rel(O[b, h], ref) < 1e-11


def _tiny_fused(seed, N=24, dm=10, d=6, k=5, m=12, scale=0.5):
    r = _rng(seed)
    Xq, Xk, Xv = (r.normal(size=(N, dm)) for _ in range(3))
    Wq = r.normal(size=(dm, d)) * scale / math.sqrt(dm)
    Wk = r.normal(size=(dm, d)) * scale / math.sqrt(dm)
    Wv = r.normal(size=(dm, d)) / math.sqrt(dm)
    E = r.normal(size=(k, N)) / math.sqrt(k)
    F = r.normal(size=(k, N)) / math.sqrt(k)
    W = r.normal(size=(m, d))
    return Xq, Xk, Xv, E, F, Wq, Wk, Wv, W


def pin_fused_maps_commute_with_the_contraction(orc):
    """Eq. (2): (E1 K) W^K = E1 (K W^K).  The head with its linear maps written out, which contracts the
    un-projected keys and values first, equals the plain head on inputs projected beforehand (numpy)."""
    for variant in (PERFORMER, RNN):
        for seed in (11, 12):
            Xq, Xk, Xv, E, F, Wq, Wk, Wv, W = _tiny_fused(seed)
            Wf = W if variant == PERFORMER else None
            got, mid = orc.fused_head(Xq, Xk, Xv, E, F, Wq, Wk, Wv, Wf, variant, intermediates=True)
            ref = orc.head_quadratic(Xq @ Wq, Xk @ Wk, Xv @ Wv, E, F, Wf, variant)
            assert _rel(got, ref) < 1e-10, ("fused vs projected inputs", variant, _rel(got, ref))
            assert _rel(mid["Kp"], E @ (Xk @ Wk)) < 1e-12 and _rel(mid["Vp"], F @ (Xv @ Wv)) < 1e-12
            assert _rel(mid["Q"], Xq @ Wq) < 1e-12
            rows = [3, 0, 17]
            sub = orc.fused_head(Xq, Xk, Xv, E, F, Wq, Wk, Wv, Wf, variant, rows=rows)
            assert _rel(sub, got[rows]) < 1e-12


def pin_fused_special_cases(orc):
    """Identity maps give back the plain head; one projected key gives O_n = (F Xv) W^V for every row;
    the output is linear in Xv and does not change when Xq's rows the call does not select change."""
    Q, K, V, E, F, W = _tiny(21, N=20, d=6, k=4, m=10)
    eye = np.eye(6)
    for variant, Wf in ((PERFORMER, W), (RNN, None)):
        a = orc.fused_head(Q, K, V, E, F, eye, eye, eye, Wf, variant)
        assert _rel(a, orc.head(Q, K, V, E, F, Wf, variant)) < 1e-11
        Xq, Xk, Xv, E2, F2, Wq, Wk, Wv, W2 = _tiny_fused(22, k=1)
        Wf2 = W2 if variant == PERFORMER else None
        o = orc.fused_head(Xq, Xk, Xv, E2, F2, Wq, Wk, Wv, Wf2, variant)
        assert np.allclose(o, np.broadcast_to((F2 @ Xv) @ Wv, o.shape), atol=1e-12)
        Xq, Xk, Xv, E3, F3, Wq, Wk, Wv, W3 = _tiny_fused(23)
        Wf3 = W3 if variant == PERFORMER else None
        Xv2 = _rng(24).normal(size=Xv.shape)
        lin = orc.fused_head(Xq, Xk, 2.0 * Xv - 3.0 * Xv2, E3, F3, Wq, Wk, Wv, Wf3, variant)
        sep = 2.0 * orc.fused_head(Xq, Xk, Xv, E3, F3, Wq, Wk, Wv, Wf3, variant) \
            - 3.0 * orc.fused_head(Xq, Xk, Xv2, E3, F3, Wq, Wk, Wv, Wf3, variant)
        assert _rel(lin, sep) < 1e-11


def pin_backward_matches_finite_differences(orc):
    """The backward pass is the derivative of the (pinned) forward pass: for a random dO, the directional
    derivative of sum(O * dO) along random directions in Q, K, V, E, F equals <gradient, direction>."""
    for variant in (PERFORMER, RNN):
        for seed in (31, 32):
            Q, K, V, E, F, W = _tiny(seed, N=14, d=5, k=4, m=9)
            Wv = W if variant == PERFORMER else None
            r = _rng(seed + 100)
            dO = r.normal(size=Q.shape)
            g = orc.head_backward(Q, K, V, E, F, Wv, dO, variant)
            x = {"Q": Q, "K": K, "V": V, "E": E, "F": F}
            loss = lambda y: float((orc.head(y["Q"], y["K"], y["V"], y["E"], y["F"], Wv, variant) * dO).sum())
            for name in ("Q", "K", "V", "E", "F"):
                u = r.normal(size=x[name].shape)
                h = 1e-5
                plus, minus = dict(x), dict(x)
                plus[name] = x[name] + h * u
                minus[name] = x[name] - h * u
                fd = (loss(plus) - loss(minus)) / (2 * h)
                an = float((g["d" + name] * u).sum())
                assert abs(fd - an) <= 2e-6 * max(1.0, abs(fd)), ("backward vs finite differences", variant, name, fd, an)


def pin_backward_special_cases(orc):
    """One projected key: O_n = F V for every row, so nothing flows to Q, K, E, and dV = F^T (sum_n dO_n),
    dF = (sum_n dO_n) V^T.  The gradients are linear in dO.  V = const * 1 with F 1 = 1 gives O = const:
    the gradients with respect to Q, K, E vanish again."""
    for variant in (PERFORMER, RNN):
        Q, K, V, E, F, W = _tiny(41, N=12, d=4, k=1, m=6)
        Wv = W if variant == PERFORMER else None
        dO = _rng(42).normal(size=Q.shape)
        g = orc.head_backward(Q, K, V, E, F, Wv, dO, variant)
        s = dO.sum(axis=0)
        assert max(np.abs(g["dQ"]).max(), np.abs(g["dK"]).max(), np.abs(g["dE"]).max()) < 1e-12
        assert np.allclose(g["dV"], np.outer(F[0], s), atol=1e-12) and np.allclose(g["dF"], (V @ s)[None, :], atol=1e-12)
        Q, K, V, E, F, W = _tiny(43, N=16, d=4, k=5, m=8)
        Wv = W if variant == PERFORMER else None
        d1, d2 = _rng(44).normal(size=Q.shape), _rng(45).normal(size=Q.shape)
        ga, gb = orc.head_backward(Q, K, V, E, F, Wv, d1, variant), orc.head_backward(Q, K, V, E, F, Wv, d2, variant)
        gc = orc.head_backward(Q, K, V, E, F, Wv, 2.0 * d1 - 0.5 * d2, variant)
        for name in gc:
            assert _rel(gc[name], 2.0 * ga[name] - 0.5 * gb[name]) < 1e-11
        Fm = np.abs(F) / np.abs(F).sum(axis=1, keepdims=True)          # rows sum to one
        gconst = orc.head_backward(Q, K, np.full_like(V, 0.7), E, Fm, Wv, d1, variant)
        assert max(np.abs(gconst["dQ"]).max(), np.abs(gconst["dK"]).max(), np.abs(gconst["dE"]).max()) < 1e-10


ALL_PINS = [
    pin_quadratic_equals_associative,
    pin_identity_projection,
    pin_projection_is_E_times_K,
    pin_convexity,
    pin_single_projected_key,
    pin_single_feature_is_softmax_over_keys,
    pin_scale_invariance,
    pin_symmetries,
    pin_rnn_worked_example,
    pin_feature_expectation,
    pin_softmax_limit,
    pin_forward_layout,
    pin_fused_maps_commute_with_the_contraction,
    pin_fused_special_cases,
    pin_backward_matches_finite_differences,
    pin_backward_special_cases,
]


@pytest.mark.parametrize("pin", ALL_PINS, ids=lambda f: f.__name__)
def test_pin(pin):
    pin(oracle.default())


# ----------------------------------------------------------------------------- planted mistakes
MUTANTS = {
    "norm_term_sign": ("return dot - 0.5 * sq;", "return dot + 0.5 * sq;"),
    "norm_term_dropped": ("return dot - 0.5 * sq;", "return dot;"),
    "norm_term_not_halved": ("return dot - 0.5 * sq;", "return dot - sq;"),
    "projection_transposed": ("P[(size_t)j * N + n]", "P[(size_t)n * k + j]"),
    "values_projected_with_E": ("down_project(F, V, N, d, k, Vp);", "down_project(E, V, N, d, k, Vp);"),
    "elu_without_plus_one": ("x > 0.0 ? x + 1.0 : exp(x)", "x > 0.0 ? x : exp(x) - 1.0"),
    "elu_branch_swapped": ("x > 0.0 ? x + 1.0 : exp(x)", "x < 0.0 ? x + 1.0 : exp(x)"),
    "normaliser_ignores_z": ("den += f * z[i];", "den += f;"),
    "normaliser_missing": ("for (int c = 0; c < d; ++c) o[c] /= den;", ""),
    "epsilon_in_denominator": ("o[c] /= den;", "o[c] /= (den + 1e-3);"),
    "per_key_stabiliser": (
        "feature_map(Kp, k, d, W, m, variant, stabilise, /*scope_global=*/1, Phik);",
        "feature_map(Kp, k, d, W, m, variant, stabilise, /*scope_global=*/0, Phik);"),
    "sqrt_m_dropped": ("* inv_sqrt_m;", ";"),
    "kv_uses_keys_as_values": ("+= f * Vp[(size_t)j * d + c];", "+= f * Kp[(size_t)j * d + c];"),
    "quadratic_unnormalised": ("a[j] /= rowsum;", ""),
    "features_from_unprojected_keys": (
        "feature_map(Kp, k, d, W, m, variant, stabilise, /*scope_global=*/1, Phik);",
        "feature_map(K, k, d, W, m, variant, stabilise, /*scope_global=*/1, Phik);"),
    "fused_value_map_is_key_map": ("linear_map(Vt, k, dm, Wv, d, Vp);", "linear_map(Vt, k, dm, Wk, d, Vp);"),
    "fused_keys_from_value_input": ("down_project(E, Xk, N, dm, k, Kt);", "down_project(E, Xv, N, dm, k, Kt);"),
    "fused_query_map_is_key_map": ("linear_map(Xs, (int)n_rows, dm, Wq, d, Qs);", "linear_map(Xs, (int)n_rows, dm, Wk, d, Qs);"),
    "linear_map_transposed": ("y[c] += x * w[c];", "y[c] += x * Wm[(size_t)c * dm + e];"),
    "fused_queries_contracted_too": ("double *Xs = gather_rows(Xq, dm, rows, nq);", "double *Xs = gather_rows(Xk, dm, rows, nq);"),
    "backward_denominator_sign": ("const double dden = -odo / den;", "const double dden = odo / den;"),
    "backward_feature_shift_dropped": ("dx[c] += g * (w[c] - x[c]);", "dx[c] += g * w[c];"),
    "backward_elu_slope": ("(x[c] > 0.0 ? 1.0 : exp(x[c]))", "(x[c] > 0.0 ? 1.0 : exp(x[c]) - 1.0)"),
    "backward_normaliser_gradient_dropped": ("double acc = dz[i];", "double acc = 0.0;"),
    "backward_dE_uses_values": ("ge += dKp[(size_t)j * d + c] * K[(size_t)n * d + c];", "ge += dKp[(size_t)j * d + c] * V[(size_t)n * d + c];"),
    "backward_dK_through_F": ("gk += E[(size_t)j * N + n] * dKp[(size_t)j * d + c];", "gk += F[(size_t)j * N + n] * dKp[(size_t)j * d + c];"),
    "head_stride_wrong": ("const size_t head = (size_t)N * d;", "const size_t head = (size_t)N * d / 2 * 2 - d;"),
}


@pytest.mark.parametrize("name", sorted(MUTANTS), ids=str)
def test_planted_mistakes_are_caught(name, tmp_path):
    old, new = MUTANTS[name]
    src = open(oracle.SOURCE).read()
    assert old in src, "mutation site vanished: %r" % old
    mutated = tmp_path / ("mutant_%s.c" % name)
    mutated.write_text(src.replace(old, new))
    lib = oracle.OracleLib(oracle.compile_source(str(mutated), str(tmp_path / ("mutant_%s.so" % name))))
    caught = []
    for pin in ALL_PINS:
        try:
            pin(lib)
        except AssertionError:
            caught.append(pin.__name__)
    assert caught, "no pin notices the planted mistake %s" % name


# ----------------------------------------------------------------------------- harness pins
def test_block_orthogonal_generator():
    """Each block of d rows is orthogonal with chi_d distributed norms; E has variance 1/k."""
    import torch
    from paper_2306_15799_b200.synth import block_orthogonal_features, make_inputs
    from paper_2306_15799_b200 import configs

    g = torch.Generator().manual_seed(5)
    d, m = 16, 16 * 40 + 5
    W = block_orthogonal_features(m, d, g).numpy()
    assert W.shape == (m, d)
    sq = []
    for b in range(40):
        blk = W[b * d:(b + 1) * d]
        G = blk @ blk.T
        off = G - np.diag(np.diag(G))
        assert np.abs(off).max() < 1e-10
        sq.extend(np.diag(G))
    assert abs(np.mean(sq) - d) < 4.0 * math.sqrt(2.0 * d / len(sq)) * 1.5     # E|g|^2 = d, Var = 2d
    w = configs.shrink(configs.C3, B=1, H=2, N=512, k=64, m=96)
    x = make_inputs(w)
    assert x["Q"].shape == (1, 2, 512, 64) and x["E"].shape == (64, 512) and x["W"].shape == (96, 64)
    assert str(x["Q"].dtype) == "torch.bfloat16"
    assert abs(x["E"].double().var().item() * 64 - 1.0) < 0.05
    assert abs(x["Q"].double().var().item() * 8.0 - 1.0) < 0.05          # d^-1/2 = 1/8
    y = make_inputs(w)
    assert all(torch.equal(x[n], y[n]) for n in ("Q", "K", "V", "E", "F", "W"))
    assert make_inputs(configs.shrink(configs.C2, B=1, H=1, N=64, k=16))["W"] is None


def test_flop_and_byte_counters():
    """The counted work: 4Nkd + 2(N+k)dm + 2kmd + 2Nmd per head; App. B's terms with 2 FLOP per MAC."""
    from paper_2306_15799_b200 import configs

    w = configs.C3
    N, d, k, m, BH = w.N, w.d, w.k, w.m, w.B * w.H
    assert w.flops() == BH * (4 * N * k * d + 2 * (N + k) * d * m + 2 * k * m * d + 2 * N * m * d)
    assert abs(w.flops() / 1e9 - 138.5) < 0.1
    assert abs(w.compulsory_bytes() / 1e6 - 553.7) < 0.1
    assert abs(configs.C4.flops() / 1e9 - 412.9) < 0.1
    assert abs(configs.C4.compulsory_bytes() / 1e6 - 1342.2) < 0.1
    assert abs(configs.C2.flops() / 1e9 - 29.2) < 0.1
    assert abs(configs.C2.compulsory_bytes() / 1e6 - 205.5) < 0.1
    # Appendix B, per layer with d_m = H d_h and one count per MAC: down-sampling 2 N d_k d_m and the
    # product d_k d_m d_h + N d_h d_m  <->  per head 4Nkd and 2kmd + 2Nmd when the feature dim is d_h.
    H, dh, dk, Nn = 4, 64, 256, 4096
    dm = H * dh
    assert 2 * (2 * Nn * dk * dm) == H * 4 * Nn * dk * dh
    assert 2 * (dk * dm * dh + Nn * dh * dm) == H * (2 * dk * dh * dh + 2 * Nn * dh * dh)
    assert len(configs.C5_GRID) == 12 and len({configs.c5(k, m).seed for k, m in configs.C5_GRID}) == 12
