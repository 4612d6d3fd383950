"""Pins for the fp64 CPU oracle: what the paper and the mathematics fix, independent of the oracle.

Each test names the fact it checks.  None of them calls the CUDA library.
"""
import itertools
import json
import math
import os

import numpy as np
import pytest
import torch

from gen import rng, workloads as W

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def _gauss(seed, stream, shape, scale=1.0):
    return rng.normal(seed, stream, shape, scale=scale).numpy()


def _phi(seed, m, G):
    return _gauss(seed, (100,), (m, G), 1.0 / math.sqrt(m)).astype(np.float32)


def _top_by_order(v, k):
    """Independent statement of the total order: sort by (-|v|, index)."""
    order = sorted(range(len(v)), key=lambda g: (-abs(v[g]), g))
    return sorted(order[:k])


# ------------------------------------------------------------------ sketch
def test_sketch_unit_rows_pick_coordinates(oracle):
    d = 40
    S = np.zeros((3, d), dtype=np.float32)
    S[0, 5] = 1; S[1, 0] = 1; S[2, 39] = 1
    h = _gauss(1, 0, d)
    assert np.array_equal(oracle.sketch(S, h), h[[5, 0, 39]])


def test_sketch_matches_library_matvec_and_is_not_transposed(oracle):
    S = _gauss(2, 0, (8, 256)).astype(np.float32)
    h = _gauss(2, 1, (5, 256))
    y = oracle.sketch(S, h)
    assert y.shape == (5, 8)
    np.testing.assert_allclose(y, h @ S.astype(np.float64).T, rtol=1e-13, atol=1e-13)


def test_sketch_linearity_mean_of_sketches_is_sketch_of_mean(oracle):
    S = _gauss(3, 0, (16, 128)).astype(np.float32)
    H = _gauss(3, 1, (37, 128))
    np.testing.assert_allclose(oracle.sketch(S, H).mean(0), oracle.sketch(S, H.mean(0)), rtol=0, atol=1e-12)


# ------------------------------------------------------------------ H_k
def test_hard_threshold_golden_tie_cases(oracle):
    """Hand-worked cases of the order (|v| descending, index ascending)."""
    cases = json.load(open(os.path.join(GOLDEN, "hard_threshold_cases.json")))["cases"]
    for c in cases:
        keep, gap = oracle.hard_threshold(np.array(c["v"], dtype=np.float64), c["k"])
        assert list(np.nonzero(keep)[0]) == c["keep"], c
        if c["gap"] == "inf":
            assert gap == math.inf
        else:
            assert gap == pytest.approx(c["gap"], abs=1e-15), c


def test_hard_threshold_exactly_k_idempotent_and_matches_sorted_order(oracle):
    for trial in range(50):
        G = 5 + trial % 40
        k = 1 + trial % G
        v = _gauss(7, (trial,), G)
        if trial % 3 == 0:  # plant ties and zeros
            v[: G // 2] = np.round(v[: G // 2])
        keep, gap = oracle.hard_threshold(v, k)
        assert keep.sum() == k
        assert list(np.nonzero(keep)[0]) == _top_by_order(v, k)
        z = np.where(keep, v, 0.0)
        keep2, _ = oracle.hard_threshold(z, k)
        if np.count_nonzero(z) == k:
            assert np.array_equal(keep, keep2)
        mags = np.sort(np.abs(v))[::-1]
        if k < G and mags[k - 1] > 0:
            assert gap == pytest.approx((mags[k - 1] - mags[k]) / mags[k - 1], abs=1e-15)


def test_hard_threshold_permutation_equivariance(oracle):
    v = _gauss(8, 0, 30)
    perm = torch.argsort(rng.bits(8, 1, 30)).numpy()
    keep, _ = oracle.hard_threshold(v, 7)
    keep_p, _ = oracle.hard_threshold(v[perm], 7)
    assert np.array_equal(keep[perm], keep_p)


# ------------------------------------------------------------------ IHT: textbook special cases
def test_iht_one_step_is_thresholded_backprojection(oracle):
    Phi = _phi(11, 12, 30); y = _gauss(11, 1, 12)
    r = oracle.iht(Phi, y, k=5, T=1, mu=0.37)
    b = Phi.astype(np.float64).T @ y
    sup = _top_by_order(b, 5)
    assert list(r.support) == sup
    expect = np.zeros(30); expect[sup] = 0.37 * b[sup]
    np.testing.assert_allclose(r.z, expect, rtol=1e-14, atol=1e-15)


def test_iht_zero_iterations(oracle):
    Phi = _phi(12, 6, 10); y = _gauss(12, 1, 6)
    r = oracle.iht(Phi, y, k=3, T=0, mu=1.0)
    assert list(r.support) == [0, 1, 2] and not r.z.any()
    assert r.resid == pytest.approx(np.linalg.norm(y))


def test_iht_orthonormal_columns_converges_in_one_step(oracle):
    """Phi^T Phi = I and mu = 1: z_1 = H_k(Phi^T y) and every later iterate equals it."""
    Q, _ = np.linalg.qr(_gauss(13, 0, (40, 24)))
    Phi = Q.astype(np.float32)           # float32 rounding: orthonormal to ~1e-7
    y = _gauss(13, 1, 40)
    b = Phi.astype(np.float64).T @ y
    sup = _top_by_order(b, 6)
    for T in (1, 2, 9):
        r = oracle.iht(Phi, y, k=6, T=T, mu=1.0)
        assert list(r.support) == sup
        np.testing.assert_allclose(r.z[sup], b[sup], rtol=1e-5)


def test_iht_identity_is_best_k_term_approximation(oracle):
    y = _gauss(14, 0, 20)
    r = oracle.iht(np.eye(20, dtype=np.float32), y, k=4, T=5, mu=1.0)
    sup = _top_by_order(y, 4)
    expect = np.zeros(20); expect[sup] = y[sup]
    assert list(r.support) == sup and np.array_equal(r.z, expect)
    rest = np.delete(y, sup)
    assert r.resid == pytest.approx(np.linalg.norm(rest), rel=1e-14)


# ------------------------------------------------------------------ IHT: invariants
def test_iht_fixed_point_for_any_step(oracle):
    """y = Phi z* with z* k-sparse: started at z*, the gradient vanishes, so z* stays."""
    Phi = _phi(21, 10, 32)
    zs = np.zeros(32); zs[[3, 17, 30]] = [1.5, -2.0, 0.75]
    y = Phi.astype(np.float64) @ zs
    for mu in (0.05, 0.3, 1.0, 2.5):
        r = oracle.iht(Phi, y, k=3, T=7, mu=mu, z0=zs)
        np.testing.assert_allclose(r.z, zs, rtol=0, atol=1e-13)
        assert list(r.support) == [3, 17, 30]


@pytest.mark.parametrize("name", ["tiny_f32", "l2_7b_b1", "l3_8b_stack", "l2_13b_prompt"])
def test_iht_monotone_residual_when_step_is_within_spectral_bound(oracle, name):
    """mu ||Phi||_2^2 <= 1  =>  ||y - Phi z_{t+1}|| <= ||y - Phi z_t|| (majorisation argument)."""
    cfg = W.CONFIGS[name]
    for trial in range(20):
        Phi = _phi(1000 + trial, cfg.m, cfg.G)
        mu = W.spectral_step(torch.from_numpy(Phi))
        y = _gauss(22, (trial,), cfg.m)
        r = oracle.iht(Phi, y, k=cfg.k, T=cfg.T, mu=mu)
        assert (np.diff(r.resid_hist) <= 1e-12).all()
        assert np.count_nonzero(r.z) <= cfg.k


def test_iht_literal_unit_step_is_not_monotone_on_gaussian_phi(oracle):
    """With Phi ~ N(0, 1/m) and mu = 1 the bound above is violated and the iteration blows up;
    this is why the gated runs take mu = 1/||Phi||_2^2 (unit step for Phi scaled to unit norm)."""
    cfg = W.CONFIGS["l2_7b_b1"]
    blown = 0
    for trial in range(10):
        Phi = _phi(2000 + trial, cfg.m, cfg.G)
        r = oracle.iht(Phi, _gauss(23, (trial,), cfg.m), k=cfg.k, T=cfg.T, mu=1.0)
        blown += r.resid_hist[-1] > r.resid_hist[0]
    assert blown >= 8


def test_iht_homogeneity_is_bit_exact_for_powers_of_two(oracle):
    Phi = _phi(24, 16, 48); y = _gauss(24, 1, 16)
    a = oracle.iht(Phi, y, k=6, T=12, mu=0.2)
    b = oracle.iht(Phi, 2.0 * y, k=6, T=12, mu=0.2)
    assert np.array_equal(b.z, 2.0 * a.z) and np.array_equal(a.support, b.support)
    assert np.array_equal(a.gap_hist, b.gap_hist)


def test_iht_column_permutation_permutes_the_support(oracle):
    Phi = _phi(25, 16, 40); y = _gauss(25, 1, 16)
    perm = torch.argsort(rng.bits(25, 2, 40)).numpy()
    a = oracle.iht(Phi, y, k=5, T=10, mu=0.2)
    b = oracle.iht(np.ascontiguousarray(Phi[:, perm]), y, k=5, T=10, mu=0.2)
    assert a.min_gap > 1e-9
    np.testing.assert_allclose(b.z, a.z[perm], rtol=1e-12, atol=1e-14)
    assert sorted(perm[b.support]) == list(a.support)


def test_iht_uses_phi_not_its_transpose(oracle):
    """A rectangular hand case: Phi = [I_2 | 0] picks coordinates of y for groups 0,1 only."""
    Phi = np.zeros((2, 5), dtype=np.float32); Phi[0, 0] = 1; Phi[1, 1] = 1
    r = oracle.iht(Phi, np.array([3.0, -4.0]), k=2, T=3, mu=1.0)
    assert list(r.support) == [0, 1]
    np.testing.assert_array_equal(r.z, [3.0, -4.0, 0, 0, 0])
    assert r.resid == 0.0


# ------------------------------------------------------------------ planted recovery + brute force
def _orthonormal_probe(seed, G, d):
    Q, _ = np.linalg.qr(_gauss(seed, (200,), (d, G)))
    return Q.T  # [G, d], orthonormal rows: A A^T = I


@pytest.mark.parametrize("G,m,k,T", [(64, 48, 2, 600), (24, 20, 1, 600)])
def test_iht_recovers_planted_support_in_the_easy_regime_and_agrees_with_brute_force(oracle, G, m, k, T):
    """Noiseless, exactly sparse, m well above k log(G/k): IHT finds the planted support and the
    planted coefficients (exact recovery when sigma = eta = 0, Theorem 1), and so does
    exhaustive least squares over all C(G,k) supports."""
    d = 96
    A = _orthonormal_probe(31, G, d)
    for trial in range(6):
        Phi = _phi(3000 + trial, m, G)
        S = (Phi.astype(np.float64) @ A).astype(np.float32)
        planted = rng.k_subset(31, (trial,), G, k)[0].numpy()
        c = _gauss(31, (trial, 1), k)
        c = np.where(np.abs(c) < 0.5, np.sign(c) * 0.5 + (c == 0) * 0.5, c)
        h = c @ A[planted]
        y = oracle.sketch(S, h)
        mu = W.spectral_step(torch.from_numpy(Phi))
        r = oracle.iht(Phi, y, k=k, T=T, mu=mu)
        assert list(r.support) == list(planted)
        assert (np.diff(r.resid_hist) <= 1e-12).all()
        # S was rounded to float32, so y = Phi c only to ~1e-7: recovery is exact to that level
        np.testing.assert_allclose(r.z[planted], c, rtol=0, atol=2e-6)
        bs, bc, bres = oracle.brute_force_support(Phi, y, k)
        assert list(bs) == list(planted)
        np.testing.assert_allclose(bc, c, atol=2e-6)
        assert r.resid >= bres - 1e-12


def test_brute_force_finds_planted_support_at_the_tiny_config_shape(oracle):
    """C(16,4) = 1820 supports; noiseless exactly-sparse y = Phi c.  IHT need not find it, but its
    residual can never beat the exhaustive optimum."""
    cfg = W.CONFIGS["tiny_f32"]
    for trial in range(3):
        Phi = _phi(4000 + trial, cfg.m, cfg.G)
        planted = rng.k_subset(41, (trial,), cfg.G, cfg.k)[0].numpy()
        c = _gauss(41, (trial, 1), cfg.k)
        c = np.where(np.abs(c) < 0.5, np.sign(c) * 0.5 + (c == 0) * 0.5, c)
        y = Phi.astype(np.float64)[:, planted] @ c
        bs, bc, bres = oracle.brute_force_support(Phi, y, cfg.k)
        assert list(bs) == list(planted) and bres < 1e-12
        np.testing.assert_allclose(bc, c, atol=1e-9)
        r = oracle.iht(Phi, y, k=cfg.k, T=cfg.T, mu=W.spectral_step(torch.from_numpy(Phi)))
        assert r.resid >= bres - 1e-12


def test_brute_force_on_a_hand_case(oracle):
    Phi = np.array([[1, 0, 1], [0, 1, 1]], dtype=np.float32)
    sup, c, res = oracle.brute_force_support(Phi, np.array([2.0, 2.0]), 1)
    assert list(sup) == [2] and c[0] == pytest.approx(2.0) and res == pytest.approx(0.0, abs=1e-15)
    sup, c, res = oracle.brute_force_support(Phi, np.array([2.0, -1.0]), 1)
    assert list(sup) == [0] and res == pytest.approx(1.0)


def test_coherence_condition_k1_is_identifiable(oracle):
    """k = 1 < (1 + 1/mu_t)/2 whenever no two columns are parallel (mutual-incoherence
    proposition): exhaustive search and long-run IHT pick the planted column."""
    Phi = _phi(51, 12, 20)
    Pn = Phi.astype(np.float64) / np.linalg.norm(Phi.astype(np.float64), axis=0)
    gram = np.abs(Pn.T @ Pn) - np.eye(20)
    mu_t = gram.max()
    assert mu_t < 1 and 1 < 0.5 * (1 + 1 / mu_t)
    for g in (0, 7, 19):
        y = 1.3 * Phi.astype(np.float64)[:, g]
        bs, _, bres = oracle.brute_force_support(Phi, y, 1)
        assert list(bs) == [g] and bres < 1e-12
        r = oracle.iht(Phi, y, k=1, T=200, mu=W.spectral_step(torch.from_numpy(Phi)))
        assert list(r.support) == [g]


# ------------------------------------------------------------------ FFN
def _dense_ffn_numpy(Wg, Wu, Wdt, h):
    """Dense SwiGLU FFN with library matmuls, W_down in its natural [d, d_ff] orientation."""
    Wg = Wg.double().numpy(); Wu = Wu.double().numpy(); Wd = Wdt.double().numpy().T.copy()
    g = Wg @ h; u = Wu @ h
    return Wd @ ((g / (1.0 + np.exp(-g))) * u)


@pytest.mark.parametrize("name", ["tiny_f32", "bf16_small"])
def test_ffn_all_groups_equals_dense_ffn(oracle, name):
    """k = G: the masked model is the dense model."""
    cfg = W.CONFIGS["tiny_f32"] if name == "tiny_f32" else \
        W.CONFIGS["l2_7b_b1"].with_(d=192, d_ff=640, k=5)
    L = W.make_layer(cfg)
    h = W.make_tokens(cfg, L.A, B=2).h.double().numpy()
    for t in range(2):
        out = oracle.ffn(L.W_gate, L.W_up, L.Wd_t, cfg.group, h[t], np.arange(cfg.G))
        ref = _dense_ffn_numpy(L.W_gate, L.W_up, L.Wd_t, h[t])
        assert np.linalg.norm(out - ref) <= 1e-13 * np.linalg.norm(ref)


def test_ffn_additive_over_disjoint_supports_and_masked_dense(oracle):
    cfg = W.CONFIGS["tiny_f32"]
    L = W.make_layer(cfg)
    h = W.make_tokens(cfg, L.A).h[0].double().numpy()
    s1, s2 = [1, 4, 9], [0, 5, 15]
    f = lambda s: oracle.ffn(L.W_gate, L.W_up, L.Wd_t, cfg.group, h, s)
    np.testing.assert_allclose(f(sorted(s1 + s2)), f(s1) + f(s2), rtol=1e-12, atol=1e-15)
    # masking the dense intermediate to the support gives the same thing
    Wg = L.W_gate.double().numpy(); Wu = L.W_up.double().numpy(); Wdt = L.Wd_t.double().numpy()
    g = Wg @ h; u = Wu @ h
    a = (g / (1 + np.exp(-g))) * u
    mask = np.zeros(cfg.d_ff);
    for gidx in s1:
        mask[gidx * cfg.group:(gidx + 1) * cfg.group] = 1
    np.testing.assert_allclose(f(s1), (a * mask) @ Wdt, rtol=1e-12, atol=1e-15)


def test_ffn_zero_input_zero_gate_and_single_channel_by_hand(oracle):
    d, b = 4, 2
    Wg = torch.tensor([[1., 0, 0, 0], [0, 1, 0, 0], [0, 0, 2, 0], [0, 0, 0, 1]])
    Wu = torch.tensor([[0., 1, 0, 0], [1, 0, 0, 0], [0, 0, 0, 3], [0, 0, 1, 0]])
    Wdt = torch.tensor([[1., 2, 3, 4], [0, 0, 0, 0], [0, 1, 0, 0], [5, 0, 0, 0]])
    h = np.array([1.0, 2.0, 0.5, -1.0])
    assert not oracle.ffn(Wg, Wu, Wdt, b, np.zeros(d), [0, 1]).any()
    assert not oracle.ffn(torch.zeros(4, 4), Wu, Wdt, b, h, [0, 1]).any()
    # group 0 = channels 0,1: a0 = silu(1)*2, a1 = silu(2)*1 ; Wd_t row 1 is zero
    silu = lambda x: x / (1 + math.exp(-x))
    out, act = oracle.ffn(Wg, Wu, Wdt, b, h, [0], return_act=True)
    np.testing.assert_allclose(act, [silu(1.0) * 2.0, silu(2.0) * 1.0], rtol=1e-15)
    np.testing.assert_allclose(out, silu(1.0) * 2.0 * np.array([1., 2, 3, 4]), rtol=1e-15)
    # group 1 = channels 2,3: a2 = silu(1)*(-3), a3 = silu(-1)*0.5
    out = oracle.ffn(Wg, Wu, Wdt, b, h, [1])
    expect = silu(1.0) * -3.0 * np.array([0., 1, 0, 0]) + silu(-1.0) * 0.5 * np.array([5., 0, 0, 0])
    np.testing.assert_allclose(out, expect, rtol=1e-15)


def test_bf16_weights_are_widened_exactly(oracle):
    w = torch.tensor([[1.0, 0.00390625, -3.140625, 65280.0]], dtype=torch.bfloat16)
    out, act = oracle.ffn(w, w, w, 1, np.array([1.0, 0, 0, 0]), [0], return_act=True)
    assert act[0] == (1 / (1 + math.exp(-1.0))) * 1.0
    np.testing.assert_array_equal(out, act[0] * np.array([1.0, 0.00390625, -3.140625, 65280.0]))


# ------------------------------------------------------------------ RMSNorm
def test_rmsnorm_identities(oracle):
    d, eps = 64, 1e-5
    x = _gauss(61, 0, d) * 3
    gamma = (1 + 0.1 * _gauss(61, 1, d)).astype(np.float32)
    n = oracle.rmsnorm(x, gamma, eps)
    ms = np.mean(x * x)
    assert np.sum((n / gamma) ** 2) == pytest.approx(d * (1 - eps / (ms + eps)), rel=1e-13)
    c = oracle.rmsnorm(np.full(d, 2.0), np.ones(d, dtype=np.float32), eps)
    np.testing.assert_allclose(c, 2.0 / math.sqrt(4.0 + eps), rtol=1e-15)


# ------------------------------------------------------------------ composition
def test_layer_step_is_the_composition_of_its_stages(oracle):
    cfg = W.CONFIGS["l3_8b_stack"].with_(d=128, d_ff=1024, group=64, m=12, k=4, B=3)
    L = W.make_layer(cfg)
    x = W.make_tokens(cfg, L.A).h.double().numpy()
    r = oracle.layer_step(L, x, group=cfg.group, k=cfg.k, T=cfg.T, rms_eps=cfg.rms_eps)
    for t in range(cfg.B):
        n = oracle.rmsnorm(x[t], L.gamma, cfg.rms_eps)
        y = oracle.sketch(L.S, n)
        it = oracle.iht(L.Phi, y, cfg.k, cfg.T, L.mu)
        f = oracle.ffn(L.W_gate, L.W_up, L.Wd_t, cfg.group, n, it.support)
        np.testing.assert_array_equal(r.y[t], y)
        np.testing.assert_array_equal(r.support[t], it.support)
        np.testing.assert_array_equal(r.z[t], it.z[it.support])
        np.testing.assert_array_equal(r.x_out[t], x[t] + f)
        assert r.resid[t] == it.resid and r.min_gap[t] == it.min_gap
    forced = np.tile(np.arange(cfg.k, dtype=np.int32), (cfg.B, 1))
    r2 = oracle.layer_step(L, x, group=cfg.group, k=cfg.k, T=cfg.T, forced_support=forced,
                           add_residual=False)
    n0 = oracle.rmsnorm(x[0], L.gamma, cfg.rms_eps)
    np.testing.assert_array_equal(r2.x_out[0], oracle.ffn(L.W_gate, L.W_up, L.Wd_t, cfg.group, n0, forced[0]))
    np.testing.assert_array_equal(r2.support, r.support)


def test_prompt_support_uses_the_mean_sketch(oracle):
    cfg = W.CONFIGS["l2_13b_prompt"].with_(d=256, d_ff=2048, m=24, k=4, B=50)
    L = W.make_layer(cfg)
    H = W.make_tokens(cfg, L.A).h.double().numpy()
    ybar, it = oracle.prompt_support(L.S, L.Phi, H, cfg.k, cfg.T, L.mu)
    np.testing.assert_allclose(ybar, oracle.sketch(L.S, H.mean(0)), rtol=0, atol=1e-12)
    ref = oracle.iht(L.Phi, ybar, cfg.k, cfg.T, L.mu)
    np.testing.assert_array_equal(it.support, ref.support)
    np.testing.assert_array_equal(it.z, ref.z)


# ------------------------------------------------------------------ uncertainty-driven budget
def test_uds_entropy_closed_forms(oracle):
    """Uniform over V: H = log V.  n1 entries at logit a and n2 at logit b: the two-level closed
    form.  A constant added to every logit changes nothing.  One dominant logit: H -> 0."""
    for V in (2, 17, 1000, 32000):
        r = oracle.uds_budget(np.full((1, V), 3.25), 1.0, 1.0, 0, 10 ** 9)
        assert r.H[0] == pytest.approx(math.log(V), rel=1e-13)
    n1, n2, a, b = 5, 11, 1.7, -0.4
    Z = n1 * math.exp(a) + n2 * math.exp(b)
    p1, p2 = math.exp(a) / Z, math.exp(b) / Z
    want = -(n1 * p1 * math.log(p1) + n2 * p2 * math.log(p2))
    row = np.array([a] * n1 + [b] * n2)
    perm = np.random.default_rng(0).permutation(n1 + n2)
    r = oracle.uds_budget(row[perm][None, :], 1.0, 1.0, 0, 10 ** 9)
    assert r.H[0] == pytest.approx(want, rel=1e-13)
    r2 = oracle.uds_budget(row[perm][None, :] + 123.0, 1.0, 1.0, 0, 10 ** 9)
    assert r2.H[0] == pytest.approx(want, rel=1e-12)
    spike = np.zeros((1, 500)); spike[0, 77] = 800.0   # exp underflows for the rest: 0 log 0 = 0
    assert oracle.uds_budget(spike, 1.0, 1.0, 0, 10 ** 9).H[0] == 0.0


def test_uds_entropy_matches_python_loop(oracle):
    rs = np.random.default_rng(5)
    L = rs.normal(0, 2.0, (3, 40))
    r = oracle.uds_budget(L, 8.0, 0.5, 4, 64)
    for t in range(3):
        Z = sum(math.exp(v) for v in L[t])
        H = -sum(math.exp(v) / Z * math.log(math.exp(v) / Z) for v in L[t])
        assert r.H[t] == pytest.approx(H, rel=1e-12)
        assert r.m[t] == min(max(math.floor(8.0 * (1 + 0.5 * H)), 4), 64)


def test_uds_budget_formula_and_clipping(oracle):
    """m = clip(floor(m_base (1 + gamma H))): worked values with H = log 4 (uniform over 4)."""
    L = np.zeros((1, 4))                       # H = log 4 = 1.386...
    assert oracle.uds_budget(L, 32, 0.5, 16, 64).m[0] == 54      # 32 * 1.6931 = 54.18
    assert oracle.uds_budget(L, 32, 0.5, 16, 48).m[0] == 48      # upper bound
    assert oracle.uds_budget(L, 4, 0.5, 16, 48).m[0] == 16       # lower bound: 6.77 -> 16
    assert oracle.uds_budget(L, 32, 0.0, 1, 64).m[0] == 32       # gamma = 0: the base budget
    sure = np.zeros((1, 9)); sure[0, 2] = 900.0
    assert oracle.uds_budget(sure, 32, 0.5, 1, 64).m[0] == 32    # H = 0: the base budget
    # entropy grows with temperature, so the budget is monotone in it
    rs = np.random.default_rng(1)
    base = rs.normal(size=(1, 300))
    ms = [oracle.uds_budget(base / T, 16, 1.0, 1, 10 ** 6).m[0] for T in (0.1, 0.5, 1.0, 2.0, 10.0)]
    assert ms == sorted(ms) and ms[0] < ms[-1]


def test_support_drift_worked_values(oracle):
    """Sec. 11: Delta_t = |S_t symmetric-difference S_{t-1}|.  Equal supports: 0; disjoint: 2k; one
    group replaced: 2; counted by hand for a small case."""
    prev = np.array([[0, 1, 2, 3], [0, 1, 2, 3], [0, 1, 2, 3], [1, 4, 6, 9]], dtype=np.int32)
    cur = np.array([[0, 1, 2, 3], [4, 5, 6, 7], [0, 1, 2, 9], [0, 4, 5, 9]], dtype=np.int32)
    assert oracle.support_drift(prev, cur).tolist() == [0, 8, 2, 4]
    assert oracle.support_drift(cur, prev).tolist() == [0, 8, 2, 4]      # symmetric
