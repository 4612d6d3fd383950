"""GPU parity of the further estimators, the temporal term, the drift, the structured sensor and the
confidence fallback (through the C boundary) against the CPU oracle.  A choice between groups that the
oracle made with a relative margin of at most 1e-4 may fall the other way in float32; such a token is
excused (counted, bounded) and must still be consistent with itself."""
import numpy as np
import pytest
import torch

import oracle
import paper_2604_14156_b200 as cs
from gen import rng, workloads as W
from parity_util import GAP_TOL, TIGHT_TOL, Z_TOL, device_layer, make_plan, rel

pytestmark = pytest.mark.gpu
DEV = "cuda"


def _problem(cfg, B, seed=0):
    Phi = rng.normal(cfg.seed + seed, (W.T_PHI, 0), (cfg.m, cfg.G), dtype=torch.float32, scale=cfg.m ** -0.5)
    mu = W.spectral_step(Phi)
    y = rng.normal(cfg.seed + seed, (77,), (B, cfg.m), dtype=torch.float32)
    return Phi, mu, y


def _dense(sup, z, G):
    out = np.zeros(G)
    out[np.asarray(sup)] = np.asarray(z, dtype=np.float64)
    return out


def _self_consistent(sup, z, resid, Phi, y, G):
    assert (np.diff(sup) > 0).all() and sup[0] >= 0 and sup[-1] < G
    own = np.linalg.norm(np.asarray(y, dtype=np.float64) - np.asarray(Phi, dtype=np.float64)[:, sup] @ z.astype(np.float64))
    assert abs(resid - own) <= 1e-4 * max(1.0, own)


@pytest.mark.parametrize("name", ["tiny_f32", "l2_7b_b64", "l3_8b_stack", "l2_13b_prompt"])
@pytest.mark.parametrize("solver", ["niht", "omp"])
def test_recover_ex_other_solvers_match_oracle(name, solver):
    cfg = W.CONFIGS[name]
    B = 24
    Phi, mu, y = _problem(cfg, B)
    plan = make_plan(cfg, max_tokens=B)
    opt = cs.StepOptions(plan, B, solver=solver)
    sup, z, resid = (t.cpu().numpy() for t in cs.cs_recover_ex(plan, Phi.to(DEV), mu, y.to(DEV), opt))
    assert plan.device_status() == 0
    excused = 0
    for t in range(B):
        ref = oracle.niht(Phi, y[t], cfg.k, cfg.T, mu) if solver == "niht" else oracle.omp(Phi, y[t], cfg.k)
        same = np.array_equal(sup[t], ref.support)
        zr = ref.z[ref.support]
        # the pursuit solves k x k least-squares problems in float32: its coefficients carry the conditioning of
        # the chosen columns, so they are held to the residual they leave rather than to 1e-4 each
        z_ok = same and (rel(z[t], zr) <= (Z_TOL if solver == "niht" else 5e-3))
        r_ok = abs(resid[t] - ref.resid) <= 1e-4 * max(1.0, ref.resid)
        if not (same and z_ok and r_ok):
            assert ref.min_gap <= GAP_TOL, (name, solver, t, same, ref.min_gap)
            excused += 1
        _self_consistent(sup[t], z[t], resid[t], Phi.numpy(), y[t].numpy(), cfg.G)
    assert excused <= 2
    plan.close()


def test_recover_ex_solvers_on_planted_supports_and_degenerate_inputs():
    """Noiseless planted supports (the pursuit must find them where the oracle does), an all-zero sketch
    (completion by the lowest indices) and a duplicated column (the twin enters with coefficient 0)."""
    cfg = W.CONFIGS["l2_7b_b64"].with_(k=6)
    B = 32
    rs = np.random.default_rng(3)
    Phi = rng.normal(cfg.seed, (W.T_PHI, 3), (cfg.m, cfg.G), dtype=torch.float32, scale=cfg.m ** -0.5)
    Pn = Phi.double().numpy()
    y = np.zeros((B, cfg.m))
    planted = []
    for t in range(B - 2):
        sup = np.sort(rs.choice(cfg.G, cfg.k, replace=False))
        c = rs.standard_normal(cfg.k); c = np.sign(c) * np.maximum(np.abs(c), 0.5)
        y[t] = Pn[:, sup] @ c
        planted.append(sup)
    y[B - 1] = 2.0 * Pn[:, 5]
    Phi2 = Phi.clone(); Phi2[:, 40] = Phi2[:, 5]          # row B-1 meets a duplicated column
    plan = make_plan(cfg, max_tokens=B)
    yt = torch.tensor(y, dtype=torch.float32)
    found = {"omp": 0, "niht": 0, "oracle_omp": 0}
    for solver in ("omp", "niht"):
        opt = cs.StepOptions(plan, B, solver=solver, T=40)
        sup, z, resid = (t.cpu().numpy() for t in cs.cs_recover_ex(plan, Phi2.to(DEV), W.spectral_step(Phi2), yt.to(DEV), opt))
        for t in range(B - 2):
            found[solver] += np.array_equal(sup[t], planted[t])
            if solver == "omp":
                found["oracle_omp"] += np.array_equal(oracle.omp(Phi2, yt[t], cfg.k).support, planted[t])
        assert sup[B - 2].tolist() == list(range(cfg.k)) and not z[B - 2].any()     # zero sketch
        if solver == "omp":
            assert 5 in sup[B - 1] and abs(resid[B - 1]) <= 1e-5
            zz = _dense(sup[B - 1], z[B - 1], cfg.G)
            assert abs(zz[5] - 2.0) <= 1e-4 and np.abs(np.delete(zz, 5)).max() <= 1e-4
    assert plan.device_status() == 0
    assert found["omp"] >= found["oracle_omp"] - 1 and found["omp"] >= 0.6 * (B - 2) and found["niht"] >= 0.4 * (B - 2)
    print(found)
    plan.close()


def test_recover_ex_temporal_term_and_warm_start_match_oracle():
    cfg = W.CONFIGS["l2_7b_b64"]
    B = 16
    Phi, mu, y = _problem(cfg, B, seed=5)
    plan = make_plan(cfg, max_tokens=B)
    s0, z0, _ = cs.cs_recover(plan, Phi.to(DEV), mu, y.to(DEV))
    y2 = (y * 1.03 + 0.05 * y.roll(1, 1))
    s0n, z0n = s0.cpu().numpy(), z0.cpu().numpy()
    excused = 0
    for gamma, warm, T in ((0.5, False, 20), (0.5, True, 6), (3.0, True, 20), (0.0, True, 4)):
        opt = cs.StepOptions(plan, B, T=T, support_prev=s0, z_prev=z0, warm_start=warm, gamma=gamma, want_drift=True)
        mu_g = float(np.float32(1.0 / (1.0 / mu + 2.0 * gamma)))      # keeps the regularised objective monotone
        sup, z, resid = (t.cpu().numpy() for t in cs.cs_recover_ex(plan, Phi.to(DEV), mu_g, y2.to(DEV), opt))
        assert plan.device_status() == 0
        for t in range(B):
            zp = _dense(s0n[t], z0n[t], cfg.G)
            ref = oracle.iht_temporal(Phi, y2[t], cfg.k, T, mu_g, gamma, zp if gamma > 0 else None, z0=zp if warm else None)
            ok = np.array_equal(sup[t], ref.support) and rel(z[t], ref.z[ref.support]) <= Z_TOL and \
                abs(resid[t] - ref.resid) <= 1e-4 * max(1.0, ref.resid)
            if not ok:
                assert ref.min_gap <= GAP_TOL, (gamma, warm, T, t, ref.min_gap)
                excused += 1
        # the drift against the previous supports, both forms
        assert opt.delta.cpu().numpy().tolist() == oracle.support_drift(s0n, sup).tolist()
        np.testing.assert_allclose(opt.drift.cpu().numpy(), oracle.support_drift_ratio(s0n, sup), rtol=1e-6)
    assert excused <= 3
    d, D = cs.cs_support_drift_ratio(plan, s0, torch.tensor(sup, device=DEV))
    assert d.cpu().numpy().tolist() == oracle.support_drift(s0n, sup).tolist()
    np.testing.assert_allclose(D.cpu().numpy(), oracle.support_drift_ratio(s0n, sup), rtol=1e-6)
    plan.close()


def _srht_operator(cfg, seed):
    rs = np.random.default_rng(seed)
    sign = rs.choice([-1, 1], cfg.d).astype(np.int8)
    rows = np.sort(rs.choice(cfg.d, cfg.m, replace=False)).astype(np.int32)
    bits = np.packbits((sign < 0).astype(np.uint8), bitorder="little").view(np.uint32).astype(np.int64)
    bits = torch.tensor(np.where(bits >= 2 ** 31, bits - 2 ** 32, bits), dtype=torch.int32)
    return sign, rows, bits


@pytest.mark.parametrize("d,m,B", [(256, 8, 4), (512, 20, 3), (4096, 32, 5), (8192, 64, 2), (1024, 1, 1)])
def test_sketch_srht_matches_oracle(d, m, B):
    cfg = W.CONFIGS["tiny_f32"].with_(d=d, m=m, d_ff=64 * 16)
    sign, rows, bits = _srht_operator(cfg, d + m)
    h = rng.normal(91, (d, m), (B, d), dtype=torch.float32)
    plan = make_plan(cfg, max_tokens=B)
    y = cs.cs_sketch_srht(plan, bits.to(DEV), torch.tensor(rows, device=DEV), h.to(DEV)).cpu().numpy()
    ref = oracle.srht(sign, rows, h)
    assert rel(y, ref) <= 1e-5 and np.abs(y - ref).max() <= 1e-5 * np.abs(ref).max()
    with pytest.raises(cs.CSError) as e:          # d not a power of two
        bad = make_plan(cfg.with_(d=192), max_tokens=1)
        cs.cs_sketch_srht(bad, bits[:6].to(DEV), torch.tensor(rows, device=DEV), torch.zeros(1, 192, device=DEV))
    assert e.value.code == 3
    plan.close()


def _ex_reference(cfg, L, x, solver, T, srht=None, prev=None, gamma=0.0, warm=False):
    """Oracle composition of one step with options: (support [B,k], z [B,k], resid [B], out [B,d])."""
    Lc = L.to("cpu")
    B = x.shape[0]
    xs = x.double().numpy()
    y = oracle.srht(srht[0], srht[1], xs) if srht is not None else oracle.sketch(Lc.S, xs)
    sups, zs, res, gaps, outs = [], [], [], [], []
    for t in range(B):
        if solver == "niht":
            r = oracle.niht(Lc.Phi, y[t], cfg.k, T, Lc.mu)
        elif solver == "omp":
            r = oracle.omp(Lc.Phi, y[t], cfg.k)
        else:
            zp = None if prev is None else _dense(prev[0][t], prev[1][t], cfg.G)
            r = oracle.iht_temporal(Lc.Phi, y[t], cfg.k, T, Lc.mu, gamma, zp if gamma > 0 else None, z0=zp if warm else None)
        sups.append(r.support); zs.append(r.z[r.support]); res.append(r.resid); gaps.append(r.min_gap)
        outs.append(oracle.ffn(Lc.W_gate, Lc.W_up, Lc.Wd_t, cfg.group, xs[t], r.support))
    return np.array(sups), np.array(zs), np.array(res), np.array(gaps), np.array(outs), y


@pytest.mark.parametrize("name,B", [("tiny_f32", 4), ("l2_7b_b1", 2), ("l2_7b_b64", 9)])
def test_layer_step_ex_options_match_oracle(name, B):
    """The whole step with another estimator, with the structured sensor, with the previous step's result
    (warm start + temporal term + drift), and on the previous supports without any estimation."""
    cfg = W.CONFIGS[name].with_(B=B)
    L = _dense_layer = W.make_layer(cfg, device=DEV)
    Lc = L.to("cpu")
    tk = W.make_tokens(cfg, L.A, B=B)
    plan = make_plan(cfg, max_tokens=B)
    lay = device_layer(plan, L)
    x = tk.h.to(DEV)
    tol = TIGHT_TOL[cfg.w_dtype]

    def check(got, want, what):
        out, sup, z, resid = (t.cpu().numpy() for t in got)
        rs_, rz, rr, gaps, ro, _ = want
        bad = 0
        for t in range(B):
            if np.array_equal(sup[t], rs_[t]):
                assert rel(out[t], ro[t]) <= tol, (what, t)
            else:
                assert gaps[t] <= GAP_TOL, (what, t, gaps[t])
                ref2 = oracle.ffn(Lc.W_gate, Lc.W_up, Lc.Wd_t, cfg.group, tk.h[t].double().numpy(), sup[t])
                assert rel(out[t], ref2) <= tol, (what, t)
                bad += 1
        assert bad <= 1, what
        return sup, z

    for solver in ("niht", "omp"):
        opt = cs.StepOptions(plan, B, solver=solver)
        check(cs.cs_layer_step_ex(plan, lay, x, opt), _ex_reference(cfg, L, tk.h, solver, cfg.T), solver)
    sup0, z0 = check(cs.cs_layer_step_ex(plan, lay, x, cs.StepOptions(plan, B)), _ex_reference(cfg, L, tk.h, "iht", cfg.T), "iht")
    # next decoding step: a drifted hidden state, warm start + temporal term from (sup0, z0), 5 iterations
    tk2 = W.make_tokens(cfg, L.A, batch=1, B=B)
    x2 = (0.9 * tk.h + 0.1 * tk2.h)
    s0d, z0d = torch.tensor(sup0, device=DEV), torch.tensor(z0, device=DEV)
    opt = cs.StepOptions(plan, B, T=5, support_prev=s0d, z_prev=z0d, warm_start=True, gamma=0.25, want_drift=True)
    want = _ex_reference(cfg, L, x2, "iht", 5, prev=(sup0, z0), gamma=0.25, warm=True)
    sup1, _ = check(cs.cs_layer_step_ex(plan, lay, x2.to(DEV), opt), want, "temporal")
    assert opt.delta.cpu().numpy().tolist() == oracle.support_drift(sup0, sup1).tolist()
    # a step that re-uses the previous supports: the FFN on them, nothing estimated
    opt = cs.StepOptions(plan, B, support_prev=s0d, reuse_support=True)
    out, sup, _, _ = cs.cs_layer_step_ex(plan, lay, x2.to(DEV), opt)
    assert torch.equal(sup, s0d)
    for t in range(B):
        ref = oracle.ffn(Lc.W_gate, Lc.W_up, Lc.Wd_t, cfg.group, x2[t].double().numpy(), sup0[t])
        assert rel(out[t].cpu().numpy(), ref) <= tol
    assert plan.device_status() == 0
    plan.close()


def test_layer_step_ex_with_the_structured_sensor():
    """SRHT in place of the dense sketch: Phi is the operator applied to the probe's transpose, as S = Phi A is
    for the dense one; d a power of two."""
    cfg = W.CONFIGS["l2_7b_b1"].with_(B=3)
    L = W.make_layer(cfg, device=DEV)
    sign, rows, bits = _srht_operator(cfg, 5)
    A = L.A.numpy()                                                    # [G, d], unit rows
    Phi = np.ascontiguousarray(oracle.srht(sign, rows, A).T.astype(np.float32))   # [m, G]: column g = operator applied to A_g
    Phi_t = torch.tensor(Phi)
    L2 = W.Layer(L.A, Phi_t.to(DEV), L.S, W.spectral_step(Phi_t), L.W_gate, L.W_up, L.Wd_t, None)
    tk = W.make_tokens(cfg, L.A, B=3)
    plan = make_plan(cfg, max_tokens=3)
    opt = cs.StepOptions(plan, 3, srht=(bits.to(DEV), torch.tensor(rows, device=DEV)))
    out, sup, z, resid = (t.cpu().numpy() for t in cs.cs_layer_step_ex(plan, device_layer(plan, L2), tk.h.to(DEV), opt))
    rs_, rz, rr, gaps, ro, y = _ex_reference(cfg, L2, tk.h, "iht", cfg.T, srht=(sign, rows))
    for t in range(3):
        if gaps[t] > GAP_TOL:
            assert np.array_equal(sup[t], rs_[t])
            assert rel(z[t], rz[t]) <= Z_TOL and rel(out[t], ro[t]) <= TIGHT_TOL["bf16"]
    plan.close()


def test_layer_step_fallback_reruns_low_confidence_tokens_on_the_denser_plan():
    for name, B, k2 in (("tiny_f32", 6, 16), ("l2_7b_b64", 7, 40)):
        cfg = W.CONFIGS[name].with_(B=B)
        L = W.make_layer(cfg, device=DEV)
        Lc = L.to("cpu")
        tk = W.make_tokens(cfg, L.A, B=B)
        plan = make_plan(cfg, max_tokens=B)
        dense = make_plan(cfg.with_(k=k2), max_tokens=B)
        lay = device_layer(plan, L)
        ref = oracle.layer_step(Lc, tk.h, group=cfg.group, k=cfg.k, T=cfg.T)
        ref2 = oracle.layer_step(Lc, tk.h, group=cfg.group, k=k2, T=cfg.T)
        conf = ref.resid / np.linalg.norm(ref.y, axis=1)
        tau = float(np.sort(conf)[B // 2 - 1] + np.sort(conf)[B // 2]) / 2     # half of the tokens fall back
        assert np.abs(conf - tau).min() > 1e-3 * tau
        out, sup, z, resid, flags, n = cs.cs_layer_step_fallback(plan, dense, lay, tk.h.to(DEV), tau)
        assert plan.device_status() == 0 and dense.device_status() == 0
        want_flags = (conf > tau).astype(np.int32)
        assert flags.cpu().numpy().tolist() == want_flags.tolist() and n == int(want_flags.sum()) == B - B // 2
        out = out.cpu().numpy()
        for t in range(B):
            r = ref2 if want_flags[t] else ref
            if r.min_gap[t] > GAP_TOL:
                assert rel(out[t], r.x_out[t]) <= TIGHT_TOL[cfg.w_dtype], (name, t, want_flags[t])
        # a threshold nobody exceeds: nothing falls back, the outputs are the plain step's
        out0, *_, n0 = cs.cs_layer_step_fallback(plan, dense, lay, tk.h.to(DEV), 10.0)
        plain, *_ = cs.cs_layer_step_ex(plan, lay, tk.h.to(DEV), cs.StepOptions(plan, B))
        assert n0 == 0 and torch.equal(out0, plain)
        plan.close(); dense.close()
