"""Pins for the fp64 CPU oracle: every check here compares the oracle against something that is NOT
its own arithmetic -- values the paper prints, closed forms the paper derives, brute force, an
independent scalar root finder, invariances, and finite differences."""
import itertools
import math
import os

import numpy as np
import pytest
from scipy.optimize import brentq, minimize

import oracle

ALPHAS = [1.25, 1.5, 2.0, 1.1, 1.75, 3.0, 4.0, 16.0]


def _rows(rng, n, kind):
    if kind == "gauss":
        return rng.normal(size=n) * rng.choice([0.3, 1.0, 4.0])
    if kind == "uniform":
        return rng.uniform(-5, 5, size=n)
    if kind == "flat":
        return np.full(n, rng.normal())
    if kind == "ties":
        return rng.integers(-2, 3, size=n).astype(np.float64) * 0.5
    if kind == "centroid":
        # the centroid-simulation logits of the paper's appendix: U(-5,5) + 0.2*10*(1-0.5|j-i|/i) + N(0,0.5^2)
        i = n - 1 if n > 1 else 1
        j = np.arange(n)
        return rng.uniform(-5, 5, size=n) + 2.0 * (1 - 0.5 * np.abs(j - i) / i) + rng.normal(size=n) * 0.5
    raise AssertionError(kind)


# ---------------------------------------------------------------- definition-level invariants (Eq. 1)
@pytest.mark.parametrize("alpha", ALPHAS)
@pytest.mark.parametrize("kind", ["gauss", "uniform", "flat", "ties", "centroid"])
def test_row_sums_to_one_bracket_and_exact_zeros(alpha, kind):
    rng = np.random.default_rng(hash((alpha, kind)) % 2**32)
    for n in [1, 2, 3, 7, 64, 1000]:
        z = _rows(rng, n, kind)
        p, tau, supp = oracle.entmax_row(z, alpha)
        # tau is bisected to 1e-12; for alpha > 2, p = y^(1/(alpha-1)) is not Lipschitz at y = 0 and tau (of the
        # row shifted to max 0, so in [-1, 0)) cannot be told apart below the spacing of doubles there, 2^-53:
        # an entry at the edge of the support moves by up to that spacing to the power 1/(alpha-1)
        # (1e-8 at alpha = 3, 5e-6 at alpha = 4, 0.09 at alpha = 16 -- the map itself is that ill-conditioned)
        assert abs(p.sum() - 1.0) < (1e-9 if alpha <= 2 else 4 * (2.0 ** -53) ** (1.0 / (alpha - 1)))
        x = (alpha - 1) * z
        # bracket of App. A, un-normalised: p_max in [1/n, 1]
        assert x.max() - 1.0 - 1e-12 <= tau <= x.max() - n ** (1.0 - alpha) + 1e-9
        supp_ref = int((p > 0).sum())
        assert supp == supp_ref
        if alpha <= 2:
            below = x <= tau
            assert np.all(p[below] == 0.0)
            assert np.all(p[~below] > 0.0)
            # Eq. 1 itself, evaluated here with numpy's power
            np.testing.assert_allclose(p, np.maximum(x - tau, 0.0) ** (1.0 / (alpha - 1)), rtol=1e-9, atol=1e-15)
        else:
            # the returned tau carries the rounding of "+ max": compare on the shifted row, where the oracle works
            xs = x - x.max()
            ts = tau - x.max()
            y = np.maximum(xs - ts, 0.0)
            far = np.abs(xs - ts) > 1e-9 * max(1.0, abs(x.max()))
            assert np.all(p[far & (xs < ts)] == 0.0) and np.all(p[far & (xs > ts)] > 0.0)
            np.testing.assert_allclose(p[far], y[far] ** (1.0 / (alpha - 1)), rtol=1e-5, atol=1e-15)


@pytest.mark.parametrize("alpha", [1.5, 2.0])
def test_sort_and_bisection_agree(alpha):
    rng = np.random.default_rng(5)
    for n in [1, 2, 5, 33, 500]:
        for kind in ["gauss", "uniform", "centroid"]:
            z = _rows(rng, n, kind)
            _, t_sort, _ = oracle.entmax_row(z, alpha, oracle.METHOD_SORT)
            _, t_bis, _ = oracle.entmax_row(z, alpha, oracle.METHOD_BISECT)
            assert abs(t_sort - t_bis) < 1e-10


# ---------------------------------------------------------------- values the paper prints
def _read_cases(path):
    out = []
    with open(path) as f:
        for line in f:
            line = line.strip()
            if not line or line.startswith("#"):
                continue
            out.append([part.split() for part in line.split(";")])
    return out


def test_paper_worked_sparsemax_example(golden_dir):
    for (alpha,), z, want in _read_cases(os.path.join(golden_dir, "sparsemax_worked_example.txt")):
        z = np.array([float(t) for t in z])
        want = np.array([float(t) for t in want])
        p, tau, supp = oracle.entmax_row(z, float(alpha))
        # boundary tie: the zeros sit exactly AT the threshold and must come out exactly zero
        np.testing.assert_array_equal(p, want)
        assert tau == 0.0 and supp == 2


def test_paper_dense_example_and_limit(golden_dir):
    for (alpha,), (b,), (phi,), (pstar,) in _read_cases(os.path.join(golden_dir, "collapse_limit.txt")):
        alpha, b, phi, pstar = float(alpha), float(b), float(phi), float(pstar)
        prev_gap = None
        for n in [8, 64, 512, 4096, 32768]:
            z = np.full(n, b)
            z[-1] = phi
            p, tau, supp = oracle.entmax_row(z, alpha)
            assert supp == n                      # the paper's "dense" regime
            assert 0 < p[0] < p[-1] < 1
            # finite-n scalar equation of the paper, solved by an independent root finder
            g = lambda x: x ** (alpha - 1) - ((1 - x) / (n - 1)) ** (alpha - 1) - (alpha - 1) * (phi - b)
            pn = brentq(g, 1e-15, 1 - 1e-15, xtol=1e-15, rtol=1e-14)
            assert abs(p[-1] - pn) < 1e-9
            np.testing.assert_allclose(p[:-1], (1 - pn) / (n - 1), rtol=1e-7)
            gap = abs(p[-1] - pstar)
            if prev_gap is not None:
                assert gap < prev_gap               # p_n -> p*
            prev_gap = gap
        assert prev_gap < 5e-3


def test_sparsemax_dense_closed_form():
    # alpha = 2, z = [0,...,0,0.5]: sum (z - tau) = 0.5 - n tau = 1
    for n in [2, 5, 100]:
        z = np.zeros(n)
        z[-1] = 0.5
        p, tau, _ = oracle.entmax_row(z, 2.0)
        assert abs(tau + 0.5 / n) < 1e-14
        np.testing.assert_allclose(p[:-1], 0.5 / n, rtol=1e-12)
        assert abs(p[-1] - (0.5 + 0.5 / n)) < 1e-14


# ---------------------------------------------------------------- Lemma 2 (two-level logits)
@pytest.mark.parametrize("alpha", ALPHAS)
@pytest.mark.parametrize("k", [1, 2, 4, 8])
def test_two_level_closed_form(alpha, k):
    rng = np.random.default_rng(k)
    for n in [k, k + 1, 40]:
        M = rng.normal() * 3
        gap_min = k ** (-(alpha - 1)) / (alpha - 1)
        for gap in [gap_min * 1.0001, gap_min * 3, 50.0]:
            z = np.full(n, M - gap)
            idx = rng.choice(n, size=k, replace=False)
            z[idx] = M
            p, tau, supp = oracle.entmax_row(z, alpha)
            assert supp == k
            assert abs(tau - ((alpha - 1) * M - k ** (-(alpha - 1)))) < 1e-9
            np.testing.assert_allclose(p[idx], 1.0 / k, rtol=1e-8)
            assert np.all(np.delete(p, idx) == 0.0)
        if n > k and k ** (-(alpha - 1)) > 1e-12:
            # just inside the gap the low level is attended too (skipped where the gap itself is below the
            # spacing of the doubles that hold the logits: k = 8 at alpha = 16 has a gap of 2e-15)
            z = np.full(n, M - gap_min * 0.9)
            z[:k] = M
            _, _, supp = oracle.entmax_row(z, alpha)
            assert supp == n


# ---------------------------------------------------------------- brute force over supports
def _brute_force(z, alpha):
    """Try every non-empty support S: solve sum_{j in S} (x_j - tau)^(1/(alpha-1)) = 1 with brentq, keep
    the S whose tau is consistent (all of S above tau, everything else at or below)."""
    n = len(z)
    x = (alpha - 1) * np.asarray(z)
    e = 1.0 / (alpha - 1)
    found = []
    for r in range(1, n + 1):
        for S in itertools.combinations(range(n), r):
            xs = x[list(S)]
            lo, hi = xs.min() - 1.0 - 1e-9, xs.min()
            f = lambda t: np.sum(np.maximum(xs - t, 0.0) ** e) - 1.0
            if f(hi) > 0:        # even with the smallest member at zero the mass exceeds 1: S too big
                continue
            if f(hi) == 0.0:     # smallest member sits exactly at tau: not a strict support
                continue
            tau = brentq(f, lo, hi, xtol=1e-15, rtol=1e-15, maxiter=500)
            rest = np.delete(x, list(S))
            if np.all(xs > tau) and np.all(rest <= tau + 1e-13):
                found.append((S, tau))
    return found


@pytest.mark.parametrize("alpha", [1.25, 1.5, 2.0, 1.7, 3.0, 4.0])
def test_brute_force_support_enumeration(alpha):
    rng = np.random.default_rng(int(alpha * 100))
    for trial in range(12):
        n = int(rng.integers(1, 9))
        z = rng.normal(size=n) * rng.choice([0.2, 1.0, 3.0])
        found = _brute_force(z, alpha)
        assert len(found) == 1, (z, found)
        S, tau_bf = found[0]
        p, tau, supp = oracle.entmax_row(z, alpha)
        assert set(np.flatnonzero(p > 0)) == set(S)
        assert abs(tau - tau_bf) < 1e-9


# ---------------------------------------------------------------- special cases and limits
def test_sparsemax_is_euclidean_projection():
    rng = np.random.default_rng(11)
    for n in [2, 3, 6]:
        z = rng.normal(size=n) * 2
        p, _, _ = oracle.entmax_row(z, 2.0)
        res = minimize(lambda x: np.sum((x - z) ** 2), np.full(n, 1.0 / n), jac=lambda x: 2 * (x - z),
                       bounds=[(0, 1)] * n, constraints=[{"type": "eq", "fun": lambda x: x.sum() - 1}],
                       method="SLSQP", options={"ftol": 1e-14, "maxiter": 500})
        np.testing.assert_allclose(p, res.x, atol=1e-6)


def test_alpha_to_one_is_softmax():
    rng = np.random.default_rng(3)
    z = rng.normal(size=12)
    sm = np.exp(z - z.max())
    sm /= sm.sum()
    errs = []
    for alpha in [1.5, 1.1, 1.01, 1.001]:
        p, _, _ = oracle.entmax_row(z, alpha)
        errs.append(np.abs(p - sm).max())
    assert all(a > b for a, b in zip(errs, errs[1:]))
    assert errs[-1] < 2e-3


@pytest.mark.parametrize("alpha", [1.25, 1.5, 2.0, 1.6])
def test_shift_append_and_monotone(alpha):
    rng = np.random.default_rng(21)
    z = rng.normal(size=50) * 2
    p, tau, _ = oracle.entmax_row(z, alpha)
    # shift: same p, tau moves by (alpha-1) t
    p2, tau2, _ = oracle.entmax_row(z + 3.7, alpha)
    np.testing.assert_allclose(p2, p, atol=1e-10)
    assert abs(tau2 - tau - (alpha - 1) * 3.7) < 1e-10
    # appending logits at or below tau/(alpha-1) changes nothing (non-vanishing attention lemma)
    # (the entry nearest the threshold sits 1e-9 below it: an exact tie is only resolved by the sort path)
    extra = np.array([tau / (alpha - 1) - 1e-9, tau / (alpha - 1) - 1.0, -100.0])
    p3, tau3, _ = oracle.entmax_row(np.concatenate([z, extra]), alpha)
    np.testing.assert_allclose(p3[:50], p, atol=1e-10)
    assert np.all(p3[50:] == 0.0) and abs(tau3 - tau) < 1e-10
    # appending anything never lowers tau
    for val in [-3.0, 0.0, z.max(), z.max() + 2]:
        _, tau4, _ = oracle.entmax_row(np.append(z, val), alpha)
        assert tau4 >= tau - 1e-12


@pytest.mark.parametrize("alpha", [1.25, 1.5, 2.0])
def test_variational_objective(alpha):
    # alpha-entmax maximises p.z + H_alpha(p), H_alpha = sum (p - p^alpha) / (alpha (alpha-1))
    rng = np.random.default_rng(8)
    z = rng.normal(size=9) * 1.5
    obj = lambda p: p @ z + np.sum(p - p ** alpha) / (alpha * (alpha - 1))
    p, _, _ = oracle.entmax_row(z, alpha)
    best = obj(p)
    sm = np.exp(z - z.max())
    sm /= sm.sum()
    assert best >= obj(sm) - 1e-12
    for _ in range(1000):
        r = rng.dirichlet(np.full(9, rng.choice([0.1, 1.0, 5.0])))
        assert best >= obj(r) - 1e-12
    for eps in [1e-3, 1e-5]:
        for _ in range(50):
            dvec = rng.normal(size=9)
            cand = np.maximum(p + eps * dvec, 0)
            cand /= cand.sum()
            assert best >= obj(cand) - 1e-12


# ---------------------------------------------------------------- ASEntmax scale (Eq. asentmax)
def test_asentmax_scale_arithmetic():
    # beta = 0 recovers the unscaled map
    assert oracle.asentmax_scale(0.0, 0.7, 1.0, 5000) == 1.0
    # gamma = -1/2, delta = 0: scale * 2 sigma sqrt(2 log n) = 2 sqrt(2) sigma beta for every n
    sigma, beta = 0.8, 1.3
    for n in [2, 10, 1000, 65536]:
        c = oracle.asentmax_scale(beta, -0.5, 0.0, n)
        assert abs(c * 2 * sigma * math.sqrt(2 * math.log(n)) - 2 * math.sqrt(2) * sigma * beta) < 1e-12
    # natural log, hand value: delta + beta (ln n)^gamma at n = e^2 rounded
    assert abs(oracle.asentmax_scale(2.0, 1.0, 0.25, 100) - (0.25 + 2.0 * math.log(100))) < 1e-12
    assert abs(oracle.asentmax_scale(1.0, 2.0, 0.0, 8) - math.log(8) ** 2) < 1e-12
    # a single visible key: c = delta
    assert oracle.asentmax_scale(1.5, -0.5, 0.75, 1) == 0.75


# ---------------------------------------------------------------- attention level
def _attn_case(rng, N, d):
    q = rng.normal(size=(N, d)).astype(np.float32)
    k = rng.normal(size=(N, d)).astype(np.float32)
    v = rng.normal(size=(N, d)).astype(np.float32)
    return q, k, v


@pytest.mark.parametrize("alpha", [1.25, 1.5, 2.0])
@pytest.mark.parametrize("causal", [True, False])
def test_attention_rows_reduce_to_row_entmax_with_one_hot_keys(alpha, causal):
    """With K_j = e_j the logit of (i, j) is c_i * q_ij * scale, so each attention row must equal the
    (separately pinned) row-level map applied to a hand-built logit vector; with V_j = e_j the output
    reads the probabilities back.  A transposed operand or a wrong mask breaks this."""
    rng = np.random.default_rng(17)
    N = d = 10
    q = (rng.normal(size=(N, d)) * 3).astype(np.float32)
    k = np.eye(N, dtype=np.float32)
    v = np.eye(N, dtype=np.float32)
    scale = (0.9, 0.6, 0.4)
    sm_scale = 0.37
    rows = np.arange(N)
    out = oracle.attn_fwd_rows(q, k, v, rows, alpha, sm_scale, causal, scale=scale, want_p=True)
    for i in range(N):
        nv = i + 1 if causal else N
        c = 0.4 + 0.9 * math.log(nv) ** 0.6 if nv > 1 else 0.4
        z = c * (q[i, :nv].astype(np.float64) * sm_scale)
        p, tau, supp = oracle.entmax_row(z, alpha)
        np.testing.assert_allclose(out["p"][i, :nv], p, atol=1e-12)
        assert np.all(out["p"][i, nv:] == 0.0)
        assert abs(out["tau"][i] - tau) < 1e-12
        np.testing.assert_allclose(out["o"][i, :nv], p, atol=1e-12)
        assert out["supp"][i] == supp
    # n_mode = 1 uses the total length for every row
    out1 = oracle.attn_fwd_rows(q, k, v, rows, alpha, sm_scale, causal, scale=scale, n_mode=1, want_p=True)
    c = 0.4 + 0.9 * math.log(N) ** 0.6
    p, tau, _ = oracle.entmax_row(c * (q[2, : (3 if causal else N)].astype(np.float64) * sm_scale), alpha)
    assert abs(out1["tau"][2] - tau) < 1e-12


def test_attention_matches_dense_numpy_formula():
    rng = np.random.default_rng(4)
    N, d = 37, 16
    q, k, v = _attn_case(rng, N, d)
    alpha, sm_scale = 1.5, 1 / math.sqrt(d)
    out = oracle.attn_fwd_rows(q, k, v, np.arange(N), alpha, sm_scale, True, want_p=True)
    s = (q.astype(np.float64) @ k.astype(np.float64).T) * sm_scale
    for i in range(N):
        p, tau, _ = oracle.entmax_row(s[i, : i + 1], alpha)
        np.testing.assert_allclose(out["o"][i], p @ v[: i + 1].astype(np.float64), atol=1e-12)
    np.testing.assert_allclose(out["p"].sum(axis=1), 1.0, atol=1e-9)
    # V = 1 gives O = 1
    out = oracle.attn_fwd_rows(q, k, np.ones_like(v), np.arange(N), alpha, sm_scale, False)
    np.testing.assert_allclose(out["o"], 1.0, atol=1e-9)


# ---------------------------------------------------------------- backward
@pytest.mark.parametrize("alpha", [1.25, 1.5, 2.0, 1.7, 3.0, 4.0])
@pytest.mark.parametrize("causal", [True, False])
def test_backward_matches_finite_differences(alpha, causal):
    rng = np.random.default_rng(int(alpha * 1000) + causal)
    N, d = 7, 4
    q, k, v = _attn_case(rng, N, d)
    d_o = rng.normal(size=(N, d)).astype(np.float32)
    scale = (0.8, 0.5, 0.6)
    sm_scale = 0.5
    rows = np.arange(N)

    def loss(q_, k_, v_):
        o = oracle.attn_fwd_rows(q_, k_, v_, rows, alpha, sm_scale, causal, scale=scale)["o"]
        return float(np.sum(o * d_o.astype(np.float64)))

    dq, dk, dv = oracle.attn_bwd_head(q, k, v, d_o, alpha, sm_scale, causal, scale=scale)
    # float32 storage limits the step: use a step that is exactly representable around each value
    h = 2.0 ** -9
    for name, grad, which in [("q", dq, 0), ("k", dk, 1), ("v", dv, 2)]:
        for _ in range(10):
            i, t = int(rng.integers(N)), int(rng.integers(d))
            args_p = [q.copy(), k.copy(), v.copy()]
            args_m = [q.copy(), k.copy(), v.copy()]
            base = np.float32(np.round(args_p[which][i, t] * 512) / 512)
            args_p[which][i, t] = base + np.float32(h)
            args_m[which][i, t] = base - np.float32(h)
            fd = (loss(*args_p) - loss(*args_m)) / (2 * h)
            # gradient at the rounded base point
            args_0 = [q.copy(), k.copy(), v.copy()]
            args_0[which][i, t] = base
            g0 = oracle.attn_bwd_head(*args_0, d_o, alpha, sm_scale, causal, scale=scale)[which][i, t]
            assert abs(fd - g0) < 5e-4 * max(1.0, abs(g0)), (name, i, t, fd, g0)
    # row-local variant agrees with the full one and dS rows sum to zero
    dq_r, ds = oracle.attn_bwd_rows(q, k, v, d_o, rows, alpha, sm_scale, causal, scale=scale, want_ds=True)
    np.testing.assert_allclose(dq_r, dq, atol=1e-12)
    np.testing.assert_allclose(ds.sum(axis=1), 0.0, atol=1e-12)


def test_backward_sparsemax_form_and_single_key_rows():
    rng = np.random.default_rng(2)
    N, d = 9, 5
    q, k, v = _attn_case(rng, N, d)
    d_o = rng.normal(size=(N, d)).astype(np.float32)
    rows = np.arange(N)
    fwd = oracle.attn_fwd_rows(q, k, v, rows, 2.0, 0.8, True, want_p=True)
    _, ds = oracle.attn_bwd_rows(q, k, v, d_o, rows, 2.0, 0.8, True, want_ds=True)
    dP = d_o.astype(np.float64) @ v.astype(np.float64).T
    for i in range(N):
        on = fwd["p"][i] > 0
        want = np.where(on, dP[i] - dP[i][on].mean(), 0.0)
        np.testing.assert_allclose(ds[i], want, atol=1e-12)
    assert np.all(ds[0] == 0.0)          # row 0 sees one key: one-hot, zero Jacobian


@pytest.mark.parametrize("alpha", [1.25, 1.5, 2.0])
@pytest.mark.parametrize("causal", [True, False])
def test_scale_parameter_gradients_match_finite_differences(alpha, causal):
    # L(beta, gamma, delta) = sum_i <O_i, dO_i>; central differences of the fp64 forward in each parameter
    rng = np.random.default_rng(77)
    N, d = 24, 8
    q, k, v, g = (rng.normal(size=(N, d)).astype(np.float32) for _ in range(4))
    sm = 1.0 / np.sqrt(d)
    params = np.array([0.9, 0.7, 1.1])          # beta, gamma, delta
    rows = np.arange(N)

    def loss(par):
        out = oracle.attn_fwd_rows(q, k, v, rows, alpha, sm, causal, scale=tuple(par))
        return float((out["o"] * g.astype(np.float64)).sum())

    dc, grads = oracle.attn_bwd_scale_head(q, k, v, g, alpha, sm, causal, scale=tuple(params))
    for idx in range(3):
        h = 1e-6
        up, dn = params.copy(), params.copy()
        up[idx] += h
        dn[idx] -= h
        fd = (loss(up) - loss(dn)) / (2 * h)
        assert abs(fd - grads[idx]) <= 1e-5 * max(1.0, abs(fd)), (idx, fd, grads[idx])
    # delta's gradient is the plain sum of the per-row scale gradients
    assert abs(dc.sum() - grads[2]) <= 1e-12 * max(1.0, abs(grads[2]))


# ------------------------------------------------------------------ ALiBi term (App. B, positional encodings)
@pytest.mark.parametrize("alpha", [1.25, 1.5, 2.0])
def test_alibi_equals_plain_attention_on_augmented_vectors(alpha):
    # m (j - i) = m j - m i: the first part is one more feature (q' = [q, 1], k'_j = [k_j, m j / sm_scale]),
    # the second a per-row shift, which leaves p unchanged and moves tau by (alpha-1) c_i (-m i)
    rng = np.random.default_rng(5)
    N, d, m, sm = 40, 4, 0.25, 0.5
    q, k, v = (rng.normal(size=(N, d)).astype(np.float32) for _ in range(3))
    scale = (0.7, 0.9, 1.2)
    rows = np.arange(N)
    with_bias = oracle.attn_fwd_rows(q, k, v, rows, alpha, sm, True, scale=scale, want_p=True, alibi=m)
    q2 = np.concatenate([q, np.ones((N, 1), np.float32)], axis=1)
    k2 = np.concatenate([k, (m * np.arange(N) / sm).astype(np.float32)[:, None]], axis=1)
    v2 = np.concatenate([v, np.zeros((N, 1), np.float32)], axis=1)
    plain = oracle.attn_fwd_rows(q2, k2, v2, rows, alpha, sm, True, scale=scale, want_p=True)
    np.testing.assert_allclose(with_bias["p"], plain["p"], atol=1e-12)
    np.testing.assert_allclose(with_bias["o"], plain["o"][:, :d], atol=1e-12)
    c = np.array([oracle.asentmax_scale(*scale, i + 1) for i in range(N)])
    np.testing.assert_allclose(with_bias["tau"], plain["tau"] - (alpha - 1) * c * m * np.arange(N), atol=1e-10)


@pytest.mark.parametrize("alpha", [1.5, 2.0])
def test_alibi_hard_cutoff_distance(alpha):
    # the paper's ALiBi proposition: a key farther than d_max = floor((z_max - z_min + 1/(alpha-1)) / m + 1)
    # from the query gets exactly zero weight (z: content logits of the row)
    rng = np.random.default_rng(9)
    N, d, m, sm = 300, 8, 0.05, 1.0 / np.sqrt(8)
    q, k, v = (rng.normal(size=(N, d)).astype(np.float32) for _ in range(3))
    out = oracle.attn_fwd_rows(q, k, v, np.arange(N), alpha, sm, True, want_p=True, alibi=m)
    z = (q.astype(np.float64) @ k.astype(np.float64).T) * sm
    checked = 0
    for i in range(N):
        zi = z[i, : i + 1]
        d_max = int(np.floor((zi.max() - zi.min() + 1.0 / (alpha - 1)) / m + 1))
        far = np.arange(i + 1) < i - d_max
        checked += int(far.sum())
        assert np.all(out["p"][i, : i + 1][far] == 0.0)
    assert checked > 1000       # the bound actually bites on this input


def test_alibi_backward_matches_finite_differences():
    rng = np.random.default_rng(31)
    N, d, m, sm, alpha = 9, 4, 0.3, 0.5, 1.5
    q, k, v = _attn_case(rng, N, d)
    d_o = rng.normal(size=(N, d)).astype(np.float32)
    scale = (0.8, 0.5, 0.6)
    rows = np.arange(N)

    def loss(q_, k_, v_, sc=scale):
        o = oracle.attn_fwd_rows(q_, k_, v_, rows, alpha, sm, True, scale=sc, alibi=m)["o"]
        return float(np.sum(o * d_o.astype(np.float64)))

    h = 2.0 ** -9
    for which in range(3):
        for _ in range(8):
            i, t = int(rng.integers(N)), int(rng.integers(d))
            args = [q.copy(), k.copy(), v.copy()]
            base = np.float32(np.round(args[which][i, t] * 512) / 512)
            args[which][i, t] = base
            g0 = oracle.attn_bwd_head(*args, d_o, alpha, sm, True, scale=scale, alibi=m)[which][i, t]
            up = [a.copy() for a in args]
            dn = [a.copy() for a in args]
            up[which][i, t] = base + np.float32(h)
            dn[which][i, t] = base - np.float32(h)
            fd = (loss(*up) - loss(*dn)) / (2 * h)
            assert abs(fd - g0) < 5e-4 * max(1.0, abs(g0)), (which, i, t, fd, g0)
    # scale parameters: the ASEntmax scale multiplies the whole logit, bias included
    _, grads = oracle.attn_bwd_scale_head(q, k, v, d_o, alpha, sm, True, scale=scale, alibi=m)
    for idx in range(3):
        e = 1e-6
        up, dn = list(scale), list(scale)
        up[idx] += e
        dn[idx] -= e
        fd = (loss(q, k, v, tuple(up)) - loss(q, k, v, tuple(dn))) / (2 * e)
        assert abs(fd - grads[idx]) <= 1e-5 * max(1.0, abs(fd)), (idx, fd, grads[idx])


def test_alibi_noncausal_hand_built_rows():
    # q = 0: the content logits vanish and row i's logits are -m |j - i| alone, keys on both sides of the query.
    # Sparsemax (alpha = 2) of three such logits, m = 1/4, worked by hand from Eq. 1 with sum p = 1:
    #   row 1: z = [-1/4, 0, -1/4]: all three in the support, tau = (-1/2 - 1)/3 = -1/2, p = [1/4, 1/2, 1/4]
    #   row 0: z = [0, -1/4, -1/2]: tau = (-3/4 - 1)/3 = -7/12, p = [7/12, 1/3, 1/12]
    #   row 2: the mirror image of row 0
    N, d, m = 3, 2, 0.25
    q = np.zeros((N, d), np.float32)
    k = np.ones((N, d), np.float32)
    v = np.eye(N, d, dtype=np.float32)
    out = oracle.attn_fwd_rows(q, k, v, np.arange(N), 2.0, 1.0, False, want_p=True, alibi=m)
    np.testing.assert_allclose(out["p"][1], [0.25, 0.5, 0.25], atol=1e-15)
    np.testing.assert_allclose(out["p"][0], [7 / 12, 1 / 3, 1 / 12], atol=1e-15)
    np.testing.assert_allclose(out["p"][2], [1 / 12, 1 / 3, 7 / 12], atol=1e-15)
    np.testing.assert_allclose(out["tau"], [-7 / 12, -0.5, -7 / 12], atol=1e-15)
    # a steeper slope pushes the far key out of the support: m = 1 on row 0 gives z = [0, -1, -2],
    # tau = -1 exactly at the second key (a tie: p = 0 there), p = [1, 0, 0]
    out = oracle.attn_fwd_rows(q, k, v, np.arange(N), 2.0, 1.0, False, want_p=True, alibi=1.0)
    np.testing.assert_allclose(out["p"][0], [1.0, 0.0, 0.0], atol=1e-15)
    np.testing.assert_allclose(out["p"][1], [0.0, 1.0, 0.0], atol=1e-15)


@pytest.mark.parametrize("alpha", [1.5, 2.0, 1.25])
def test_alibi_noncausal_mirror_and_two_sided_decomposition(alpha):
    # (1) the penalty depends on the distance only: reversing the sequence (queries, keys and values alike)
    #     reverses the result.  A bias with the wrong sign on one side of the query breaks this.
    # (2) for one query row i the non-causal logits are those of two causal problems glued together: keys
    #     j <= i carry m (j - i) as they stand; keys j >= i, read backwards, are the causal keys of the reversed
    #     sequence for query N - 1 - i.  Entmax of the concatenation, computed by the row function, must agree.
    rng = np.random.default_rng(77)
    N, d, m, sm = 23, 4, 0.3, 0.5
    q, k, v = (rng.normal(size=(N, d)).astype(np.float32) for _ in range(3))
    scale = (0.6, 0.8, 1.1)
    rows = np.arange(N)
    fwd = oracle.attn_fwd_rows(q, k, v, rows, alpha, sm, False, scale=scale, want_p=True, alibi=m)
    rev = oracle.attn_fwd_rows(q[::-1].copy(), k[::-1].copy(), v[::-1].copy(), rows, alpha, sm, False, scale=scale,
                               want_p=True, alibi=m)
    np.testing.assert_allclose(fwd["p"], rev["p"][::-1, ::-1], atol=1e-13)
    np.testing.assert_allclose(fwd["o"], rev["o"][::-1], atol=1e-13)
    np.testing.assert_allclose(fwd["tau"], rev["tau"][::-1], atol=1e-13)
    c = oracle.asentmax_scale(*scale, N)
    z = (q.astype(np.float64) @ k.astype(np.float64).T) * sm
    for i in (0, 5, 11, 22):
        bias = np.array([m * (j - i) if j <= i else -m * (j - i) for j in range(N)])
        p, tau, _ = oracle.entmax_row(c * (z[i] + bias), alpha)
        np.testing.assert_allclose(fwd["p"][i], p, atol=1e-13)
        assert abs(fwd["tau"][i] - tau) < 1e-12
    # the bias is not symmetric content: a row far from the middle puts more mass on its own side
    assert not np.allclose(fwd["p"], fwd["p"][:, ::-1])


def test_alibi_noncausal_backward_matches_finite_differences():
    rng = np.random.default_rng(33)
    N, d, m, sm, alpha = 8, 4, 0.3, 0.5, 1.5
    q, k, v = _attn_case(rng, N, d)
    d_o = rng.normal(size=(N, d)).astype(np.float32)
    scale = (0.8, 0.5, 0.6)
    rows = np.arange(N)

    def loss(q_, k_, v_):
        o = oracle.attn_fwd_rows(q_, k_, v_, rows, alpha, sm, False, scale=scale, alibi=m)["o"]
        return float(np.sum(o * d_o.astype(np.float64)))

    h = 2.0 ** -9
    for which in range(3):
        for _ in range(8):
            i, t = int(rng.integers(N)), int(rng.integers(d))
            args = [q.copy(), k.copy(), v.copy()]
            base = np.float32(np.round(args[which][i, t] * 512) / 512)
            args[which][i, t] = base
            g0 = oracle.attn_bwd_head(*args, d_o, alpha, sm, False, scale=scale, alibi=m)[which][i, t]
            up = [a.copy() for a in args]
            dn = [a.copy() for a in args]
            up[which][i, t] = base + np.float32(h)
            dn[which][i, t] = base - np.float32(h)
            fd = (loss(*up) - loss(*dn)) / (2 * h)
            assert abs(fd - g0) < 5e-4 * max(1.0, abs(g0)), (which, i, t, fd, g0)


# ---------------------------------------------------------------- content-dependent scale (Sec. 4.1)
def test_scale_projection_values_and_limits():
    rng = np.random.default_rng(41)
    B, H, N, dm, s = 2, 3, 9, 5, 2.0
    x = rng.normal(size=(B, N, dm))
    wb, wg = rng.normal(size=(H, dm)) * 0.5, rng.normal(size=(H, dm)) * 0.5
    delta = np.array([1.0, 0.5, 1.5])
    c, beta, gamma = oracle.scale_projection(x, wb, wg, delta, s, True)
    # written out with numpy: softplus and tanh of the projections, then Eq. "asentmax" through its own function
    pb = np.einsum("bnd,hd->bhn", x, wb)
    pg = np.einsum("bnd,hd->bhn", x, wg)
    np.testing.assert_allclose(beta, np.logaddexp(0.0, pb), rtol=1e-13)
    np.testing.assert_allclose(gamma, s * np.tanh(pg), rtol=1e-13)
    assert np.all(beta > 0) and np.all(np.abs(gamma) < s)          # beta > 0, gamma in (-s, s) as the paper states
    for b, h, i in [(0, 0, 0), (1, 2, 4), (0, 1, 8)]:
        assert abs(c[b, h, i] - oracle.asentmax_scale(beta[b, h, i], gamma[b, h, i], delta[h], i + 1)) < 1e-14
    assert np.all(c[:, :, 0] == delta[None, :])                    # one visible key: c = delta
    # zero weights: beta = log 2, gamma = 0, so c = delta + log 2 for every row that sees more than one key
    c0, _, _ = oracle.scale_projection(x, np.zeros_like(wb), np.zeros_like(wg), delta, s, True)
    np.testing.assert_allclose(c0[:, :, 1:], (delta + math.log(2.0))[None, :, None] * np.ones((B, H, N - 1)), rtol=1e-14)
    # the non-causal problem and n_mode = 1 use the total length for every row
    cn, bn, gn = oracle.scale_projection(x, wb, wg, delta, s, False)
    cm, _, _ = oracle.scale_projection(x, wb, wg, delta, s, True, n_mode=1)
    np.testing.assert_allclose(cn, cm, rtol=0, atol=0)
    np.testing.assert_allclose(cn, delta[None, :, None] + bn * math.log(N) ** gn, rtol=1e-13)
    # very negative / positive projections: softplus stays finite and positive
    big = np.full((1, 3, dm), 40.0)
    cb, bb, _ = oracle.scale_projection(big, np.ones((1, dm)), np.zeros((1, dm)), np.array([0.0]), s, False)
    assert np.all(np.isfinite(bb)) and abs(bb[0, 0, 0] - 200.0) < 1e-9
    _, bs, _ = oracle.scale_projection(-big, np.ones((1, dm)), np.zeros((1, dm)), np.array([0.0]), s, False)
    assert np.all(bs > 0) and bs[0, 0, 0] < 1e-80


def test_scale_projection_backward_matches_finite_differences():
    rng = np.random.default_rng(43)
    B, H, N, dm, s = 2, 2, 6, 4, 1.5
    x = rng.normal(size=(B, N, dm))
    wb, wg = rng.normal(size=(H, dm)) * 0.7, rng.normal(size=(H, dm)) * 0.7
    delta = np.array([1.0, 0.6])
    dc = rng.normal(size=(B, H, N))
    for causal in (True, False):
        loss = lambda x_, wb_, wg_, dl_: float(np.sum(oracle.scale_projection(x_, wb_, wg_, dl_, s, causal)[0] * dc))
        dwb, dwg, dd, dx = oracle.scale_projection_bwd(x, wb, wg, dc, s, causal)
        e = 1e-6
        for arr, grad, which in ((wb, dwb, 1), (wg, dwg, 2), (delta, dd, 3), (x, dx, 0)):
            for _ in range(6):
                idx = tuple(int(rng.integers(n)) for n in arr.shape)
                args = [x.copy(), wb.copy(), wg.copy(), delta.copy()]
                up = [a.copy() for a in args]
                dn = [a.copy() for a in args]
                up[which][idx] += e
                dn[which][idx] -= e
                fd = (loss(*up) - loss(*dn)) / (2 * e)
                assert abs(fd - grad[idx]) <= 1e-6 * max(1.0, abs(fd)), (which, idx, fd, grad[idx])


def test_threads_reported():
    assert oracle.num_threads() >= 1
