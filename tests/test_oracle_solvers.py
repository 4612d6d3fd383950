"""Pins of the oracle's further estimators and sensor (CPU only): orthogonal matching pursuit, the
normalised-step iteration, the temporal regulariser, the normalised drift, the subsampled randomized
Hadamard sketch.  Each is checked against something other than itself: textbook special cases, the
paper's incoherence proposition (Sec. 9), closed forms, exhaustive search, library routines."""
import json
import os

import numpy as np
import pytest
import scipy.linalg

import oracle

GOLDEN = os.path.join(os.path.dirname(__file__), "golden", "solver_cases.json")


def _gauss(rs, m, G):
    return (rs.standard_normal((m, G)) / np.sqrt(m)).astype(np.float32)


def _orthonormal_columns(rs, m, G):
    q, _ = np.linalg.qr(rs.standard_normal((m, G)))
    return q.astype(np.float32)


# --------------------------------------------------------------------------- orthogonal matching pursuit
def test_omp_hand_worked_case():
    """A 2 x 3 example worked by hand (tests/golden/solver_cases.json)."""
    case = json.load(open(GOLDEN))["omp_2x3"]
    Phi = np.array(case["Phi"], dtype=np.float32)
    r = oracle.omp(Phi, np.array(case["y"]), case["k"])
    assert r.order.tolist() == case["order"]
    assert r.support.tolist() == case["support"]
    np.testing.assert_allclose(r.z, case["z"], atol=1e-12)
    assert abs(r.resid - case["resid"]) <= 1e-12


def test_omp_orthonormal_columns_is_best_k_term():
    rs = np.random.default_rng(1)
    Phi = _orthonormal_columns(rs, 40, 24)
    y = rs.standard_normal(40)
    c = Phi.astype(np.float64).T @ y
    for k in (1, 5, 24):
        r = oracle.omp(Phi, y, k)
        want = np.sort(np.argsort(-np.abs(c), kind="stable")[:k])
        assert r.support.tolist() == want.tolist()
        # float32 storage of Q leaves the columns orthonormal to ~1e-7 only
        np.testing.assert_allclose(r.z[r.support], c[want], atol=1e-5)
        assert r.order.tolist() == np.argsort(-np.abs(c), kind="stable")[:k].tolist()


def test_omp_recovers_under_the_incoherence_condition():
    """Sec. 9 proposition: k < (1 + 1/mu_t) / 2 makes the k-sparse representation identifiable and OMP
    recovers it in the noiseless case.  Phi = [I | H/8] (m = 64, G = 128) has coherence exactly 1/8, so
    every support of up to 4 columns must come back exactly, with its coefficients."""
    H = scipy.linalg.hadamard(64).astype(np.float64) / 8.0
    Phi = np.concatenate([np.eye(64), H], axis=1).astype(np.float32)
    Pn = Phi.astype(np.float64)
    gram = np.abs(Pn.T @ Pn - np.eye(128))
    assert abs(gram.max() - 0.125) < 1e-12
    rs = np.random.default_rng(2)
    for trial in range(200):
        k = int(rs.integers(1, 5))
        sup = np.sort(rs.choice(128, k, replace=False))
        c = rs.standard_normal(k)
        c = np.where(np.abs(c) < 0.2, 0.2 * np.sign(c) + (c == 0), c)
        y = Pn[:, sup] @ c
        r = oracle.omp(Phi, y, k)
        assert r.support.tolist() == sup.tolist(), trial
        np.testing.assert_allclose(r.z[sup], c, atol=1e-10)
        assert r.resid <= 1e-10


def test_omp_refit_is_the_least_squares_solution():
    rs = np.random.default_rng(3)
    Phi = _gauss(rs, 32, 86)
    Pn = Phi.astype(np.float64)
    y = rs.standard_normal(32)
    r = oracle.omp(Phi, y, 22)
    cols = Pn[:, r.support]
    z_ls, *_ = np.linalg.lstsq(cols, y, rcond=None)
    np.testing.assert_allclose(r.z[r.support], z_ls, rtol=1e-8, atol=1e-10)
    res = y - cols @ r.z[r.support]
    assert np.abs(cols.T @ res).max() <= 1e-10          # the residual is orthogonal to every chosen column
    assert abs(np.linalg.norm(res) - r.resid) <= 1e-12
    # each pick was the largest normalised correlation with the residual of the picks before it
    picked = []
    for j in r.order:
        if picked:
            zz, *_ = np.linalg.lstsq(Pn[:, picked], y, rcond=None)
            rr = y - Pn[:, picked] @ zz
        else:
            rr = y
        corr = np.abs(Pn.T @ rr) / np.linalg.norm(Pn, axis=0)
        corr[picked] = -1
        assert int(np.argmax(corr)) == j
        picked.append(int(j))


def test_omp_agrees_with_exhaustive_search_where_it_must():
    rs = np.random.default_rng(4)
    Phi = _gauss(rs, 8, 16)
    for trial in range(20):                      # k = 1: the first pick IS the best single column
        y = rs.standard_normal(8)
        sup, c, res = oracle.brute_force_support(Phi, y, 1)
        r = oracle.omp(Phi, y, 1)
        assert r.support.tolist() == sup.tolist() and abs(r.resid - res) <= 1e-12
    Phi = _gauss(rs, 48, 64)                     # planted pair on the easy shape
    for trial in range(10):
        sup = np.sort(rs.choice(64, 2, replace=False))
        y = Phi.astype(np.float64)[:, sup] @ np.array([1.0, -0.7])
        r = oracle.omp(Phi, y, 2)
        bf, _, res = oracle.brute_force_support(Phi, y, 2)
        assert r.support.tolist() == bf.tolist() == sup.tolist()
    Phi = _gauss(rs, 8, 16)                      # never better than the exhaustive optimum
    for trial in range(10):
        y = rs.standard_normal(8)
        assert oracle.omp(Phi, y, 4).resid >= oracle.brute_force_support(Phi, y, 4)[2] - 1e-12


def test_omp_degenerate_inputs_still_return_k_indices():
    rs = np.random.default_rng(5)
    Phi = _gauss(rs, 6, 10)
    r = oracle.omp(Phi, np.zeros(6), 3)          # nothing correlates: the lowest indices, zero coefficients
    assert r.support.tolist() == [0, 1, 2] and not r.z.any() and r.order.tolist() == [-1, -1, -1]
    Phi[:, 7] = Phi[:, 2]                        # a duplicated column adds nothing once its twin is in
    y = 2.0 * Phi[:, 2].astype(np.float64)
    r = oracle.omp(Phi, y, 2)
    assert r.order[0] == 2 and r.resid <= 1e-12 and abs(r.z[2] - 2.0) <= 1e-12
    assert len(set(r.support.tolist())) == 2
    r = oracle.omp(Phi, rs.standard_normal(6), 10)   # k = G > m: exactly G indices, exact fit
    assert r.support.tolist() == list(range(10)) and r.resid <= 1e-10


# --------------------------------------------------------------------------- normalised step
def test_niht_orthonormal_columns_is_unit_step_iht():
    rs = np.random.default_rng(6)
    Phi = _orthonormal_columns(rs, 40, 24)
    y = rs.standard_normal(40)
    n = oracle.niht(Phi, y, 5, 6, 0.3)
    np.testing.assert_allclose(n.step_hist, 1.0, atol=1e-6)      # ||Phi g_S|| = ||g_S||
    i = oracle.iht(Phi, y, 5, 6, 1.0)
    assert n.support.tolist() == i.support.tolist()
    np.testing.assert_allclose(n.z, i.z, atol=1e-6)


def test_niht_first_step_formula_and_exact_line_search():
    rs = np.random.default_rng(7)
    Phi = _gauss(rs, 32, 86)
    Pn = Phi.astype(np.float64)
    y = rs.standard_normal(32)
    k = 22
    n = oracle.niht(Phi, y, k, 1, 0.1)
    g = Pn.T @ y
    S = np.argsort(-np.abs(g), kind="stable")[:k]
    mu0 = (g[S] @ g[S]) / np.linalg.norm(Pn[:, S] @ g[S]) ** 2
    assert abs(n.step_hist[0] - mu0) <= 1e-12 * mu0
    # along g restricted to S the step minimises the residual: no nearby step does better
    f = lambda mu: np.linalg.norm(y - Pn[:, S] @ (mu * g[S]))
    assert f(mu0) <= min(f(mu0 * 0.99), f(mu0 * 1.01))
    # k = G: every iteration is steepest descent with exact line search, so the residual never rises
    n = oracle.niht(Phi[:, :20], y, 20, 15, 0.1)
    assert (np.diff(n.resid_hist) <= 1e-12).all()


def test_niht_zero_gradient_uses_the_fallback_step():
    Phi = _gauss(np.random.default_rng(8), 8, 16)
    n = oracle.niht(Phi, np.zeros(8), 4, 3, 0.25)
    assert n.step_hist.tolist() == [0.25] * 3 and not n.z.any() and n.support.tolist() == [0, 1, 2, 3]


def test_normalised_step_recovers_planted_supports_more_often_than_the_fixed_step():
    """Noiseless planted supports at m = 32, G = 86: the recovery rate of the three estimators at a sparsity
    the fixed step already finds hard.  (Reported by the benchmark too; here only the ordering that the
    paper's solver list leads one to expect is asserted: the pursuit and the normalised step are not worse
    than the fixed step.)"""
    rs = np.random.default_rng(9)
    m, G, k, trials = 32, 86, 6, 60
    hit = {"iht": 0, "niht": 0, "omp": 0}
    for _ in range(trials):
        Phi = _gauss(rs, m, G)
        Pn = Phi.astype(np.float64)
        sup = np.sort(rs.choice(G, k, replace=False))
        c = rs.standard_normal(k)
        c = np.sign(c) * np.maximum(np.abs(c), 0.5)
        y = Pn[:, sup] @ c
        mu = 1.0 / np.linalg.norm(Pn, 2) ** 2
        hit["iht"] += oracle.iht(Phi, y, k, 40, mu).support.tolist() == sup.tolist()
        hit["niht"] += oracle.niht(Phi, y, k, 40, mu).support.tolist() == sup.tolist()
        hit["omp"] += oracle.omp(Phi, y, k).support.tolist() == sup.tolist()
    print(hit)
    assert hit["niht"] >= hit["iht"] and hit["omp"] >= hit["iht"] and hit["omp"] >= 0.8 * trials


# --------------------------------------------------------------------------- temporal regulariser
def test_temporal_term_zero_weight_is_plain_iht_bit_for_bit():
    rs = np.random.default_rng(10)
    Phi = _gauss(rs, 32, 86)
    y = rs.standard_normal(32)
    zp = np.zeros(86); zp[rs.choice(86, 22, replace=False)] = rs.standard_normal(22)
    a = oracle.iht_temporal(Phi, y, 22, 20, 0.15, 0.0, zp)
    b = oracle.iht(Phi, y, 22, 20, 0.15)
    assert np.array_equal(a.z, b.z) and a.support.tolist() == b.support.tolist()


def test_temporal_term_closed_form_without_thresholding():
    """Phi = I, k = G: the objective separates and the iteration converges to (y + 2 gamma z_prev) / (1 + 2 gamma)."""
    rs = np.random.default_rng(11)
    G = 12
    Phi = np.eye(G, dtype=np.float32)
    y, zp = rs.standard_normal(G), rs.standard_normal(G)
    for gamma in (0.0, 0.3, 2.0):
        r = oracle.iht_temporal(Phi, y, G, 400, 0.1, gamma, zp)
        np.testing.assert_allclose(r.z, (y + 2 * gamma * zp) / (1 + 2 * gamma), atol=1e-10)


def test_temporal_term_fixed_point_and_monotone_objective():
    rs = np.random.default_rng(12)
    Phi = _gauss(rs, 48, 64)
    Pn = Phi.astype(np.float64)
    zs = np.zeros(64); zs[[3, 30]] = [1.5, -1.0]
    y = Pn @ zs
    for gamma in (0.0, 0.5, 5.0):                 # y = Phi z*, z_prev = z*: z* stays where it is
        r = oracle.iht_temporal(Phi, y, 2, 10, 0.2, gamma, zs, z0=zs)
        np.testing.assert_allclose(r.z, zs, atol=1e-12)
    # the objective 1/2 ||y - Phi z||^2 + gamma ||z - z_prev||^2 never rises when mu (||Phi||^2 + 2 gamma) <= 1
    y = rs.standard_normal(48)
    zp = np.zeros(64); zp[rs.choice(64, 6, replace=False)] = rs.standard_normal(6)
    gamma = 0.4
    mu = 1.0 / (np.linalg.norm(Pn, 2) ** 2 + 2 * gamma)
    obj = []
    for T in range(0, 25):
        z = oracle.iht_temporal(Phi, y, 6, T, mu, gamma, zp).z
        obj.append(0.5 * np.linalg.norm(y - Pn @ z) ** 2 + gamma * np.linalg.norm(z - zp) ** 2)
    assert (np.diff(obj[1:]) <= 1e-12).all()
    # a heavy weight keeps the previous support where the plain iteration moves away from it
    plain = set(oracle.iht(Phi, y, 6, 30, mu).support.tolist())
    held = set(oracle.iht_temporal(Phi, y, 6, 30, 1.0 / (np.linalg.norm(Pn, 2) ** 2 + 40.0), 20.0, 3.0 * np.sign(zp) * (zp != 0)).support.tolist())
    prev = set(np.flatnonzero(zp).tolist())
    assert len(held & prev) >= len(plain & prev) and len(held & prev) >= 5


# --------------------------------------------------------------------------- normalised drift
def test_support_drift_ratio_worked_values():
    prev = np.array([[0, 1, 2, 3], [0, 1, 2, 3], [0, 1, 2, 3]])
    cur = np.array([[0, 1, 2, 3], [4, 5, 6, 7], [0, 1, 2, 9]])
    # identical: 0 / 4;  disjoint: 8 / 8;  one entry swapped: 2 / 5
    np.testing.assert_allclose(oracle.support_drift_ratio(prev, cur), [0.0, 1.0, 0.4])
    d = oracle.support_drift(prev, cur)
    np.testing.assert_allclose(oracle.support_drift_ratio(prev, cur), d / (4 + d / 2))   # |union| = k + Delta / 2


# --------------------------------------------------------------------------- subsampled randomized Hadamard sketch
def test_srht_against_a_library_hadamard_matrix():
    rs = np.random.default_rng(13)
    for d, m in ((8, 3), (64, 64), (256, 17), (4096, 32)):
        sign = rs.choice([-1, 1], d).astype(np.int8)
        rows = rs.choice(d, m, replace=False).astype(np.int32)
        h = rs.standard_normal((2, d))
        H = scipy.linalg.hadamard(d).astype(np.float64)       # Sylvester order: H[a, i] = (-1)^popcount(a & i)
        want = (h * sign) @ H[rows].T / np.sqrt(m)
        np.testing.assert_allclose(oracle.srht(sign, rows, h), want, rtol=1e-12, atol=1e-12)


def test_srht_unit_vectors_norm_and_linearity():
    rs = np.random.default_rng(14)
    d = 128
    sign = rs.choice([-1, 1], d).astype(np.int8)
    rows = np.arange(d, dtype=np.int32)
    h = rs.standard_normal(d)
    y = oracle.srht(sign, rows, h)
    assert abs(np.linalg.norm(y) - np.linalg.norm(h)) <= 1e-12 * np.linalg.norm(h)   # all d rows: an isometry
    e = np.zeros(d); e[37] = 1.0
    ye = oracle.srht(sign, rows, e)
    par = np.array([bin(a & 37).count("1") & 1 for a in range(d)])
    np.testing.assert_allclose(ye, sign[37] * (1 - 2 * par) / np.sqrt(d), atol=1e-15)
    g = rs.standard_normal(d)
    sub = rs.choice(d, 9, replace=False).astype(np.int32)
    np.testing.assert_allclose(oracle.srht(sign, sub, 2 * h - 3 * g),
                               2 * oracle.srht(sign, sub, h) - 3 * oracle.srht(sign, sub, g), atol=1e-12)
