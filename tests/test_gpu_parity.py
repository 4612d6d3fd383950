"""GPU parity: the CUDA library (through the C boundary) against the fp64 CPU oracle on the same
seeded inputs.  Tolerances are those of tests/parity_util.py."""
import numpy as np
import pytest
import torch

import oracle
import paper_2604_14156_b200 as cs
from gen import rng, workloads as W
from parity_util import (GAP_TOL, OUT_TOL, PROMPT_TIGHT_TOL, TIGHT_TOL, Z_TOL, compare_layer_step, device_layer,
                         make_plan, recovery_matches, rel)

pytestmark = pytest.mark.gpu
DEV = "cuda"


def _layer(cfg, layer=0, **kw):
    return W.make_layer(cfg, layer, device=DEV, **kw)


# ------------------------------------------------------------------ single entry points
@pytest.mark.parametrize("name,B", [("tiny_f32", 4), ("l2_7b_b1", 1), ("l2_7b_b64", 64), ("l3_8b_stack", 5)])
def test_sketch_matches_oracle(name, B):
    cfg = W.CONFIGS[name]
    A = W.make_probe(cfg)
    Phi = rng.normal(cfg.seed, (W.T_PHI, 0), (cfg.m, cfg.G), dtype=torch.float32, scale=cfg.m ** -0.5)
    S = (Phi.double() @ A).float()
    h = W.make_tokens(cfg, A, B=B).h
    plan = make_plan(cfg, max_tokens=max(B, 1))
    y = cs.cs_sketch(plan, S.to(DEV), h.to(DEV)).cpu().numpy()
    ref = oracle.sketch(S, h)
    assert rel(y, ref) <= 1e-5
    assert np.abs(y - ref).max() <= 1e-5 * np.abs(ref).max()


@pytest.mark.parametrize("name", ["tiny_f32", "l2_7b_b64", "l3_8b_stack", "l2_13b_prompt"])
def test_recover_matches_oracle(name):
    cfg = W.CONFIGS[name]
    B = 48
    Phi = rng.normal(cfg.seed, (W.T_PHI, 0), (cfg.m, cfg.G), dtype=torch.float32, scale=cfg.m ** -0.5)
    mu = W.spectral_step(Phi)
    y = rng.normal(cfg.seed, (77,), (B, cfg.m), dtype=torch.float32)
    plan = make_plan(cfg, max_tokens=B)
    sup, z, resid = cs.cs_recover(plan, Phi.to(DEV), mu, y.to(DEV))
    sup = sup.cpu().numpy(); z = z.cpu().numpy(); resid = resid.cpu().numpy()
    excused = 0
    for t in range(B):
        ref = oracle.iht(Phi, y[t], cfg.k, cfg.T, mu)
        if not recovery_matches(sup[t], z[t], resid[t], ref, Phi.numpy(), y[t].numpy(), (name, t)):
            excused += 1
    assert excused <= 2


def test_recover_edge_cases():
    """T = 0, k = G, k = 1, all-zero sketch (every comparison a tie), exact ties between groups."""
    cfg = W.CONFIGS["tiny_f32"]
    Phi = rng.normal(5, (1,), (cfg.m, cfg.G), dtype=torch.float32, scale=cfg.m ** -0.5)
    mu = W.spectral_step(Phi)
    y = rng.normal(5, (2,), (3, cfg.m), dtype=torch.float32)
    for k, T in [(4, 0), (16, 10), (1, 10), (15, 3)]:
        c = cfg.with_(k=k, T=T)
        plan = make_plan(c, max_tokens=3)
        sup, z, resid = cs.cs_recover(plan, Phi.to(DEV), mu, y.to(DEV))
        for t in range(3):
            ref = oracle.iht(Phi, y[t], k, T, mu)
            assert np.array_equal(sup[t].cpu().numpy(), ref.support), (k, T)
            assert rel(z[t].cpu().numpy(), ref.z[ref.support]) <= Z_TOL or not ref.z.any()
            assert abs(resid[t].item() - ref.resid) <= 1e-4 * max(1.0, ref.resid)
    # y = 0: v is identically zero, the order falls back to the index -> 0..k-1
    plan = make_plan(cfg, max_tokens=2)
    sup, z, resid = cs.cs_recover(plan, Phi.to(DEV), mu, torch.zeros(2, cfg.m, device=DEV))
    assert sup.cpu().tolist() == [[0, 1, 2, 3]] * 2 and not z.any() and not resid.any()
    # duplicated columns give exact ties: the lower index must win on both sides
    Phi2 = Phi.clone(); Phi2[:, 9] = Phi2[:, 2]; Phi2[:, 12] = -Phi2[:, 5]
    sup, z, _ = cs.cs_recover(plan, Phi2.to(DEV), W.spectral_step(Phi2), y[:2].to(DEV))
    for t in range(2):
        ref = oracle.iht(Phi2, y[t], cfg.k, cfg.T, W.spectral_step(Phi2))
        if ref.min_gap > GAP_TOL or not ref.z.any():
            assert np.array_equal(sup[t].cpu().numpy(), ref.support)


@pytest.mark.parametrize("name,k", [("l2_7b_b64", 22), ("l3_8b_stack", 28), ("l3_8b_stack", 60)])
def test_recover_ties_across_warps(name, k):
    """Exact ties between groups owned by different warps and by the same warp (duplicated and
    negated columns of Phi), for the list form (k <= 56) and the dense form (k = 60) of the kernel."""
    cfg = W.CONFIGS[name].with_(k=k)
    Phi = rng.normal(cfg.seed, (W.T_PHI, 3), (cfg.m, cfg.G), dtype=torch.float32, scale=cfg.m ** -0.5)
    Phi[:, 70] = Phi[:, 3]; Phi[:, 40] = -Phi[:, 35]; Phi[:, 71] = Phi[:, 3]; Phi[:, 10] = Phi[:, 9]
    mu = W.spectral_step(Phi)
    B = 16
    y = rng.normal(cfg.seed, (78,), (B, cfg.m), dtype=torch.float32)
    y[0] = 0.0                                      # every comparison a tie
    plan = make_plan(cfg, max_tokens=B)
    sup, z, resid = cs.cs_recover(plan, Phi.to(DEV), mu, y.to(DEV))
    sup = sup.cpu().numpy(); z = z.cpu().numpy(); resid = resid.cpu().numpy()
    assert sup[0].tolist() == list(range(k)) and not z[0].any()
    checked = 0
    for t in range(1, B):
        ref = oracle.iht(Phi, y[t], cfg.k, cfg.T, mu)
        checked += recovery_matches(sup[t], z[t], resid[t], ref, Phi.numpy(), y[t].numpy(), (name, k, t))
    assert checked >= B - 3
    # one iteration only: v = mu Phi^T y has the exact ties, and they decide the support directly
    plan1 = make_plan(cfg.with_(T=1), max_tokens=B)
    sup1, _, _ = cs.cs_recover(plan1, Phi.to(DEV), mu, y.to(DEV))
    for t in range(1, B):
        one = oracle.iht(Phi, y[t], cfg.k, 1, mu)
        if one.min_gap > GAP_TOL or one.min_gap == 0.0:
            assert np.array_equal(sup1[t].cpu().numpy(), one.support), t


def test_recover_random_shapes():
    """Eighty random (G, m, k, T) shapes, all warp counts and both forms of the kernel (list for
    k <= 56, dense above), some with duplicated columns or an all-zero sketch."""
    rs = np.random.default_rng(7)
    excused = total = 0
    for trial in range(80):
        G = int(rs.integers(2, 129)); m = int(rs.integers(2, 65)); k = int(rs.integers(1, G + 1)); T = int(rs.integers(0, 31))
        if trial % 5 == 0 and G >= 57:
            k = int(rs.integers(57, G + 1))
        B = 4
        Phi = torch.tensor(rs.normal(0, m ** -0.5, (m, G)), dtype=torch.float32)
        if trial % 7 == 0 and G > 40:
            Phi[:, 33] = Phi[:, 1]; Phi[:, 7] = -Phi[:, 6]
        mu = W.spectral_step(Phi)
        y = torch.tensor(rs.normal(size=(B, m)), dtype=torch.float32)
        if trial % 11 == 0:
            y[0] = 0
        plan = cs.Plan(256, G * 64, 64, m, k, T, torch.float32, B, 1e-5)
        sup, z, resid = cs.cs_recover(plan, Phi.to(DEV), mu, y.to(DEV))
        sup = sup.cpu().numpy(); z = z.cpu().numpy(); resid = resid.cpu().numpy()
        for t in range(B):
            ref = oracle.iht(Phi, y[t], k, T, mu)
            total += 1
            if not recovery_matches(sup[t], z[t], resid[t], ref, Phi.numpy(), y[t].numpy(), (G, m, k, T, t)):
                excused += 1
        plan.close()
    assert excused <= total // 20


def test_recover_warm_matches_oracle():
    """Warm start (Sec. 5, Sec. 8): T iterations from the previous token's k-sparse iterate, against
    the oracle started from the same dense z_0.  Random shapes over both kernel forms, a drifted y,
    warm starts that hold zeros, outputs written over the warm-start buffers."""
    rs = np.random.default_rng(11)
    excused = total = 0
    for trial in range(40):
        G = int(rs.integers(2, 129)); m = int(rs.integers(2, 65)); k = int(rs.integers(1, G + 1))
        if trial % 4 == 0 and G >= 57:
            k = int(rs.integers(57, G + 1))
        T0 = int(rs.integers(0, 21)); T1 = int(rs.integers(1, 9))
        B = 4
        Phi = torch.tensor(rs.normal(0, m ** -0.5, (m, G)), dtype=torch.float32)
        mu = W.spectral_step(Phi)
        y0 = torch.tensor(rs.normal(size=(B, m)), dtype=torch.float32)
        y1 = y0 + 0.2 * torch.tensor(rs.normal(size=(B, m)), dtype=torch.float32)
        plan = cs.Plan(256, G * 64, 64, m, k, T0, torch.float32, B, 1e-5)
        Pd = Phi.to(DEV)
        sup0, z0, _ = cs.cs_recover(plan, Pd, mu, y0.to(DEV))
        if trial % 3 == 0:   # an arbitrary k-sparse start instead: random ascending support, some zero values
            sup0 = torch.tensor(np.stack([np.sort(rs.choice(G, k, replace=False)) for _ in range(B)]), dtype=torch.int32, device=DEV)
            z0 = torch.tensor(rs.normal(size=(B, k)) * (rs.random((B, k)) > 0.3), dtype=torch.float32, device=DEV)
        s0 = sup0.cpu().numpy().copy(); v0 = z0.cpu().numpy().copy()
        sup, z, resid = cs.cs_recover_warm(plan, Pd, mu, y1.to(DEV), T1, sup0, z0)
        assert plan.device_status() == 0
        if trial % 5 == 0:   # in place: the outputs are the warm-start buffers
            lib = plan.lib
            r2 = torch.empty(B, dtype=torch.float32, device=DEV)
            plan.check(lib.cs_recover_warm(plan.handle, Pd.data_ptr(), float(mu), y1.to(DEV).data_ptr(), B, T1, sup0.data_ptr(),
                                           z0.data_ptr(), sup0.data_ptr(), z0.data_ptr(), r2.data_ptr(), None), "cs_recover_warm")
            torch.cuda.synchronize()
            assert torch.equal(sup0, sup) and torch.equal(z0, z) and torch.equal(r2, resid)
        sup = sup.cpu().numpy(); z = z.cpu().numpy(); resid = resid.cpu().numpy()
        for t in range(B):
            dense = np.zeros(G); dense[s0[t]] = v0[t]
            ref = oracle.iht(Phi, y1[t], k, T1, mu, z0=dense)
            total += 1
            if not recovery_matches(sup[t], z[t], resid[t], ref, Phi.numpy(), y1[t].numpy(), (G, m, k, T1, t)):
                excused += 1
        plan.close()
    assert excused <= total // 20


def test_recover_warm_needs_fewer_iterations():
    """Sec. 11 (slow support drift): from the previous token's result, a few iterations reach the
    support that a cold start needs the plan's T for, on the benchmark's recovery shape."""
    cfg = W.CONFIGS["l2_7b_b64"]
    L = _layer(cfg)
    tk = W.make_tokens(cfg, L.A, B=8)
    plan = make_plan(cfg, max_tokens=8)
    y = cs.cs_sketch(plan, L.S, tk.h.to(DEV))
    sup_c, z_c, _ = cs.cs_recover(plan, L.Phi, L.mu, y)
    # the next token's sketch: a small drift of this one's
    g = torch.Generator().manual_seed(3)
    y2 = y + 0.02 * y.abs().mean() * torch.randn(y.shape, generator=g).to(DEV)
    sup_cold, _, _ = cs.cs_recover(plan, L.Phi, L.mu, y2)
    sup_w, z_w, res_w = cs.cs_recover_warm(plan, L.Phi, L.mu, y2, 4, sup_c, z_c)
    Phi = L.Phi.cpu(); yc = y2.cpu()
    s0 = sup_c.cpu().numpy(); v0 = z_c.cpu().numpy()
    agree = 0
    for t in range(8):
        dense = np.zeros(cfg.G); dense[s0[t]] = v0[t]
        ref = oracle.iht(Phi, yc[t], cfg.k, 4, L.mu, z0=dense)
        if ref.min_gap > GAP_TOL:
            assert np.array_equal(sup_w[t].cpu().numpy(), ref.support), t
            assert rel(z_w[t].cpu().numpy(), ref.z[ref.support]) <= Z_TOL
        agree += len(set(sup_w[t].tolist()) & set(sup_cold[t].tolist()))
    assert agree >= 0.95 * 8 * cfg.k   # 4 warm iterations land on (nearly) the cold start's T-iteration support
    plan.close()


@pytest.mark.parametrize("name,B", [("tiny_f32", 4), ("l2_7b_b1", 1), ("l2_7b_b64", 3)])
def test_ffn_exec_matches_oracle_on_given_supports(name, B):
    cfg = W.CONFIGS[name]
    L = _layer(cfg)
    Lc = L.to("cpu")
    tk = W.make_tokens(cfg, L.A, B=B)
    plan = make_plan(cfg, max_tokens=B)
    lay = device_layer(plan, L)
    res = rng.normal(cfg.seed, (78,), (B, cfg.d), dtype=torch.float32)
    out = cs.cs_ffn_exec(plan, lay, tk.h.to(DEV), tk.planted.to(DEV), residual=res.to(DEV)).cpu().numpy()
    out0 = cs.cs_ffn_exec(plan, lay, tk.h.to(DEV), tk.planted.to(DEV)).cpu().numpy()
    assert plan.device_status() == 0
    for t in range(B):
        ref = oracle.ffn(Lc.W_gate, Lc.W_up, Lc.Wd_t, cfg.group, tk.h[t], tk.planted[t])
        assert rel(out0[t], ref) <= TIGHT_TOL[cfg.w_dtype]
        assert rel(out[t], ref + res[t].double().numpy()) <= TIGHT_TOL[cfg.w_dtype]


def test_ffn_exec_all_groups_is_the_dense_ffn():
    cfg = W.CONFIGS["tiny_f32"].with_(k=16)
    L = _layer(cfg)
    tk = W.make_tokens(cfg, L.A, B=2)
    plan = make_plan(cfg, max_tokens=2)
    sup = torch.arange(16, dtype=torch.int32).repeat(2, 1)
    out = cs.cs_ffn_exec(plan, device_layer(plan, L), tk.h.to(DEV), sup.to(DEV)).cpu().double().numpy()
    Wg, Wu, Wdt = (w.cpu().double().numpy() for w in (L.W_gate, L.W_up, L.Wd_t))
    for t in range(2):
        h = tk.h[t].double().numpy()
        g = Wg @ h; u = Wu @ h
        dense = ((g / (1 + np.exp(-g))) * u) @ Wdt
        assert rel(out[t], dense) <= 1e-5


def test_ffn_exec_flags_invalid_supports():
    cfg = W.CONFIGS["tiny_f32"]
    L = _layer(cfg)
    plan = make_plan(cfg, max_tokens=2)
    lay = device_layer(plan, L)
    h = torch.zeros(2, cfg.d, device=DEV)
    good = torch.tensor([[0, 1, 2, 3], [4, 5, 6, 15]], dtype=torch.int32, device=DEV)
    cs.cs_ffn_exec(plan, lay, h, good)
    assert plan.device_status() == 0
    # unsorted but in range: flagged, and harmless to execute
    bad = torch.tensor([[0, 1, 2, 3], [4, 6, 5, 15]], dtype=torch.int32, device=DEV)
    cs.cs_ffn_exec(plan, lay, h, bad)
    assert plan.device_status() == 4
    assert plan.device_status() == 0  # reading clears it


def test_ffn_exec_out_of_range_groups_are_skipped_not_read():
    """A group index outside [0, G) never becomes an address: it is flagged, its channels contribute
    zero, and every other entry and token is computed as usual (gather path and tensor-core path)."""
    for name, B in (("tiny_f32", 3), ("l2_7b_b64", 3), ("l2_7b_b64", 7)):
        cfg = W.CONFIGS[name]
        L = _layer(cfg)
        Lc = L.to("cpu")
        tk = W.make_tokens(cfg, L.A, B=B)
        plan = make_plan(cfg, max_tokens=B)
        sup = tk.planted.clone()
        sup[1, 0] = -3
        sup[1, cfg.k - 1] = cfg.G + 5
        out = cs.cs_ffn_exec(plan, device_layer(plan, L), tk.h.to(DEV), sup.to(DEV)).cpu().numpy()
        assert plan.device_status() == 4
        for t in range(B):
            valid = sup[t][(sup[t] >= 0) & (sup[t] < cfg.G)]
            ref = oracle.ffn(Lc.W_gate, Lc.W_up, Lc.Wd_t, cfg.group, tk.h[t], valid)
            assert rel(out[t], ref) <= TIGHT_TOL[cfg.w_dtype], (name, B, t)
        plan.close()


def test_recover_non_finite_row_stays_in_its_row():
    """A NaN in one token's sketch: that token's outputs are k valid, ascending, distinct indices (its
    values are NaN) and the status word reports it; the neighbouring tokens are untouched."""
    for name in ("tiny_f32", "l2_7b_b64"):
        cfg = W.CONFIGS[name]
        Phi = rng.normal(cfg.seed, (W.T_PHI, 0), (cfg.m, cfg.G), dtype=torch.float32, scale=cfg.m ** -0.5)
        mu = W.spectral_step(Phi)
        y = rng.normal(cfg.seed, (81,), (3, cfg.m), dtype=torch.float32)
        y[1, cfg.m // 2] = float("nan")
        plan = make_plan(cfg, max_tokens=3)
        guard = torch.full((5, cfg.k), -7, dtype=torch.int32, device=DEV)   # rows 1..3 are the outputs
        zg = torch.full((5, cfg.k), 123.0, dtype=torch.float32, device=DEV)
        resid = torch.empty(3, dtype=torch.float32, device=DEV)
        Phi_d, y_d = Phi.to(DEV), y.to(DEV)   # named: a temporary would be freed (and reused) before the launch
        st = plan.lib.cs_recover(plan.handle, Phi_d.data_ptr(), float(mu), y_d.data_ptr(), 3,
                                 guard[1:4].data_ptr(), zg[1:4].data_ptr(), resid.data_ptr(),
                                 torch.cuda.current_stream().cuda_stream)
        assert st == 0
        assert plan.device_status() == 5
        g = guard.cpu().numpy(); zz = zg.cpu().numpy()
        assert (g[0] == -7).all() and (g[4] == -7).all() and (zz[0] == 123.0).all() and (zz[4] == 123.0).all()
        for row, t in ((1, 0), (3, 2)):
            ref = oracle.iht(Phi, y[t], cfg.k, cfg.T, mu)
            assert recovery_matches(g[row], zz[row], resid[t].item(), ref, Phi.numpy(), y[t].numpy(), (name, t))
        assert (np.diff(g[2]) > 0).all() and g[2][0] >= 0 and g[2][-1] < cfg.G
        plan.close()


def test_layer_step_non_finite_token_does_not_disturb_the_others():
    """The whole step with a NaN hidden state in the middle token (gather path)."""
    cfg = W.CONFIGS["tiny_f32"].with_(B=3)
    L = _layer(cfg)
    tk = W.make_tokens(cfg, L.A, B=3)
    x = tk.h.clone()
    x[1, 7] = float("nan")
    plan = make_plan(cfg, max_tokens=3)
    out, sup, z, resid = cs.cs_layer_step(plan, device_layer(plan, L), x.to(DEV))
    torch.cuda.synchronize()
    assert plan.device_status() == 5
    ref = oracle.layer_step(L.to("cpu"), tk.h, group=cfg.group, k=cfg.k, T=cfg.T)
    sup = sup.cpu().numpy(); out = out.cpu().numpy()
    for t in (0, 2):
        if ref.min_gap[t] > GAP_TOL:
            assert np.array_equal(sup[t], ref.support[t])
            assert rel(out[t], ref.x_out[t]) <= TIGHT_TOL["f32"]
    assert (np.diff(sup[1]) > 0).all() and sup[1][0] >= 0 and sup[1][-1] < cfg.G
    plan.close()


def test_call_errors_come_back_as_codes():
    cfg = W.CONFIGS["tiny_f32"]
    plan = make_plan(cfg, max_tokens=2)
    S = torch.zeros(cfg.m, cfg.d, device=DEV)
    with pytest.raises(cs.CSError) as e:
        cs.cs_sketch(plan, S, torch.zeros(3, cfg.d, device=DEV))  # B > max_tokens
    assert e.value.code == 2
    with pytest.raises(cs.CSError) as e:
        cs.cs_recover(plan, torch.zeros(cfg.m, cfg.G, device=DEV), float("nan"), torch.zeros(1, cfg.m, device=DEV))
    assert e.value.code == 5
    misaligned = torch.zeros(2 * cfg.d + 1, device=DEV)[1:1 + cfg.d].view(1, cfg.d)  # 4-byte offset
    with pytest.raises(cs.CSError) as e:
        cs.cs_sketch(plan, S, misaligned)
    assert e.value.code == 3


# ------------------------------------------------------------------ whole step, the five workloads
@pytest.mark.parametrize("seed_offset", [0, 1000, 2000])
@pytest.mark.parametrize("name", ["tiny_f32", "l2_7b_b1", "l2_7b_b64"])
def test_layer_step_parity(name, seed_offset):
    cfg = W.CONFIGS[name]
    cfg = cfg.with_(index=cfg.index + seed_offset)
    L = _layer(cfg)
    tk = W.make_tokens(cfg, L.A)
    plan = make_plan(cfg)
    rep, _, _ = compare_layer_step(cfg, L, plan, tk.h)
    assert rep.excused <= max(1, cfg.B // 16)
    print(f"{name}+{seed_offset}: {rep}")


@pytest.mark.parametrize("name,B", [("tiny_f32", 4), ("tiny_f32", 1), ("l2_7b_b1", 1), ("l2_7b_b1", 3), ("l2_7b_b64", 4)])
def test_layer_step_speculative_start(name, B):
    """The opt-in small-batch path (sketch + recovery in one launch, the weight stream started on the first
    iterate): parity with the oracle, and the plain chain's supports and (to rounding: the rows are dealt
    to one CTA fewer) outputs, also when the step is repeated on the same plan (the slot table and the
    tickets are reused) and with a NaN token."""
    cfg = W.CONFIGS[name].with_(B=B)
    L = _layer(cfg)
    spec, plain = make_plan(cfg, speculative=True), make_plan(cfg)
    for batch in range(3):
        tk = W.make_tokens(cfg, L.A, batch=batch, B=B)
        rep, _, out_spec = compare_layer_step(cfg, L, spec, tk.h)
        want, sup, z, resid = cs.cs_layer_step(plain, device_layer(plain, L), tk.h.to(DEV))
        got, sup2, z2, resid2 = cs.cs_layer_step(spec, device_layer(spec, L), tk.h.to(DEV))
        torch.cuda.synchronize()
        if rep.excused == 0:   # (a near-tie may be broken differently by the two forms of the iteration)
            assert torch.equal(sup, sup2)
            assert rel(got.cpu().numpy(), want.cpu().numpy()) <= 1e-6 and torch.equal(got, out_spec), batch
    if B >= 3:
        x = W.make_tokens(cfg, L.A, batch=7, B=B).h
        x[1, 5] = float("nan")
        got, sup2, _, _ = cs.cs_layer_step(spec, device_layer(spec, L), x.to(DEV))
        want, sup, _, _ = cs.cs_layer_step(plain, device_layer(plain, L), x.to(DEV))
        torch.cuda.synchronize()
        assert spec.device_status() == 5 and plain.device_status() == 5
        for t in (0, 2):
            assert torch.equal(sup[t], sup2[t]) and rel(got[t].cpu().numpy(), want[t].cpu().numpy()) <= 1e-6
        s1 = sup2[1].cpu().numpy()
        assert (np.diff(s1) > 0).all() and s1[0] >= 0 and s1[-1] < cfg.G
    spec.close(); plain.close()


@pytest.mark.parametrize("name,B", [("tiny_f32", 4), ("l2_7b_b1", 1), ("l2_7b_b1", 3), ("l2_7b_b64", 4)])
def test_layer_step_l2_warmup(name, B):
    """Mode 2 of the small-batch option (sketch + recovery in one launch, the plain gather kernel behind it
    asking L2 for the first iterate's weight blocks before it waits for the final supports): the hint changes
    no result, so parity with the oracle holds and, where no near-tie is excused, supports and outputs are
    those of the plain chain bit for bit; repeated on the same plan."""
    cfg = W.CONFIGS[name].with_(B=B)
    L = _layer(cfg)
    warm, plain = make_plan(cfg), make_plan(cfg)
    warm.set_speculative(2)
    for batch in range(3):
        tk = W.make_tokens(cfg, L.A, batch=batch, B=B)
        rep, _, _ = compare_layer_step(cfg, L, warm, tk.h)
        want, sup, _, _ = cs.cs_layer_step(plain, device_layer(plain, L), tk.h.to(DEV))
        got, sup2, _, _ = cs.cs_layer_step(warm, device_layer(warm, L), tk.h.to(DEV))
        torch.cuda.synchronize()
        assert warm.device_status() == 0
        if rep.excused == 0:
            assert torch.equal(sup, sup2) and torch.equal(got, want), batch
    warm.close(); plain.close()


def test_layer_step_speculative_random_shapes():
    """Random small-batch shapes through the opt-in path against the oracle and the plain chain."""
    rs = np.random.default_rng(11)
    done = 0
    for trial in range(40):
        group = int(rs.choice([64, 128]))
        G = int(rs.integers(2, 100)); k = int(rs.integers(1, min(G, 32) + 1))
        d = int(rs.choice([64, 192, 256, 1024, 4096])); m = int(rs.integers(1, 33))
        B = int(rs.integers(1, 5)); T = int(rs.choice([0, 1, 2, 7, 20]))
        w = str(rs.choice(["f32", "bf16"]))
        cfg = W.CONFIGS["tiny_f32"].with_(d=d, d_ff=group * G, group=group, m=m, k=k, T=T, B=B, w_dtype=w, index=300 + trial)
        L = _layer(cfg)
        spec, plain = make_plan(cfg, speculative=True), make_plan(cfg)
        tk = W.make_tokens(cfg, L.A, B=B)
        rep, _, got = compare_layer_step(cfg, L, spec, tk.h)
        want, sup, _, _ = cs.cs_layer_step(plain, device_layer(plain, L), tk.h.to(DEV))
        _, sup2, _, _ = cs.cs_layer_step(spec, device_layer(spec, L), tk.h.to(DEV))
        torch.cuda.synchronize()
        if rep.excused == 0:
            assert torch.equal(sup, sup2), (trial, group, G, k, d, m, B, T, w)
            assert rel(got.cpu().numpy(), want.cpu().numpy()) <= 1e-5, (trial, group, G, k, d, m, B, T, w)
            done += 1
        spec.close(); plain.close()
    assert done >= 30


def test_layer_step_literal_unit_step_tiny():
    """The tiny workload with the literal mu = 1 (diverging iterates): parity must still hold."""
    cfg = W.CONFIGS["tiny_f32"]
    L = _layer(cfg, literal_mu=1.0)
    tk = W.make_tokens(cfg, L.A)
    rep, _, _ = compare_layer_step(cfg, L, make_plan(cfg), tk.h)
    print(rep)


@pytest.mark.parametrize("shape", [
    dict(d=192, d_ff=64 * 5, group=64, m=5, k=2, B=3),         # nothing a multiple of 32
    dict(d=8192, d_ff=128 * 7, group=128, m=64, k=7, B=2),     # widest rows, k = G
    dict(d=1024, d_ff=128 * 128, group=128, m=33, k=1, B=17),  # most groups, ragged token tail
    dict(d=320, d_ff=64 * 33, group=64, m=17, k=9, B=37),
])
@pytest.mark.parametrize("w", ["f32", "bf16"])
def test_layer_step_ragged_shapes(shape, w):
    cfg = W.CONFIGS["l3_8b_stack"].with_(n_layers=1, w_dtype=w, T=6, **shape)
    L = _layer(cfg)
    tk = W.make_tokens(cfg, L.A)
    rep, _, _ = compare_layer_step(cfg, L, make_plan(cfg), tk.h)
    print(shape, w, rep)


def test_layer_step_random_shapes():
    """Forty random layer shapes through the fused step: both group sizes, d from 64 to 5120, any m, k,
    T, batches on both sides of the crossover and past 128 tokens, both weight types, with and
    without RMSNorm + residual."""
    rs = np.random.default_rng(3)
    for trial in range(40):
        group = int(rs.choice([64, 128]))
        G = int(rs.integers(2, 60))
        d = int(rs.choice([64, 128, 192, 256, 320, 512, 768, 1024, 2048, 4096, 5120]))
        m = int(rs.integers(2, 65)); k = int(rs.integers(1, G + 1)); T = int(rs.integers(0, 12))
        B = int(rs.choice([1, 2, 3, 4, 5, 7, 9, 17, 33, 70, 130]))
        w = str(rs.choice(["f32", "bf16"]))
        base = W.CONFIGS["l3_8b_stack"] if rs.integers(0, 2) else W.CONFIGS["l2_7b_b64"]
        cfg = base.with_(n_layers=1, w_dtype=w, T=T, d=d, d_ff=group * G, group=group, m=m, k=k, B=B,
                         index=100 + trial)
        L = _layer(cfg)
        tk = W.make_tokens(cfg, L.A)
        plan = make_plan(cfg)
        rep, _, _ = compare_layer_step(cfg, L, plan, tk.h)
        assert rep.excused <= max(1, B // 16), (trial, rep)
        plan.close()


def test_layer_step_in_place_and_without_aux_outputs():
    cfg = W.CONFIGS["l3_8b_stack"].with_(n_layers=1, d=512, d_ff=2048, m=16, k=4, B=6)
    L = _layer(cfg)
    tk = W.make_tokens(cfg, L.A)
    plan = make_plan(cfg)
    lay = device_layer(plan, L)
    x = tk.h.to(DEV)
    ref_out, *_ = cs.cs_layer_step(plan, lay, x)
    y = x.clone()
    cs.cs_layer_step(plan, lay, y, x_out=y, want_aux=False)
    assert torch.equal(y, ref_out)
    again, *_ = cs.cs_layer_step(plan, lay, x)
    assert torch.equal(again, ref_out)  # deterministic: no atomics on the path


def test_every_regime_is_deterministic():
    """No atomics and fixed summation orders everywhere: the same call twice (on a plan that has run other
    work in between) gives the same bits, in the gather regime, on the decode GEMMs, and in the prompt-level
    kernels (single tiles, paired tiles, CTA pairs)."""
    for name, B in (("l2_7b_b1", 1), ("l2_7b_b1", 3), ("l2_7b_b64", 64), ("l3_8b_stack", 32)):
        cfg = W.CONFIGS[name].with_(B=B, n_layers=1)
        L = _layer(cfg)
        plan = make_plan(cfg)
        lay = device_layer(plan, L)
        x = W.make_tokens(cfg, L.A, B=B).h.to(DEV)
        other = W.make_tokens(cfg, L.A, batch=3, B=B).h.to(DEV)
        first = [t.clone() for t in cs.cs_layer_step(plan, lay, x)]
        cs.cs_layer_step(plan, lay, other)
        second = cs.cs_layer_step(plan, lay, x)
        torch.cuda.synchronize()
        for a, b in zip(first, second):
            assert torch.equal(a, b), (name, B)
        plan.close()
    for k in W.PROMPT_K_SWEEP:
        cfg = W.CONFIGS["l2_13b_prompt"].with_(k=k)
        L = _layer(cfg)
        plan = make_plan(cfg)
        lay = device_layer(plan, L)
        H = W.make_tokens(cfg, L.A).h.to(DEV).to(torch.bfloat16)
        sup = torch.arange(0, 2 * k, 2, dtype=torch.int32, device=DEV)
        first = cs.cs_ffn_exec_shared(plan, lay, H, sup).clone()
        cs.cs_ffn_exec_shared(plan, lay, H.flip(0).contiguous(), sup)
        second = cs.cs_ffn_exec_shared(plan, lay, H, sup)
        torch.cuda.synchronize()
        assert plan.device_status() == 0 and torch.equal(first, second), k
        plan.close()


def test_stack_parity_teacher_forced_and_chained():
    """32 Llama-3-8B-shaped layers, batch 32.
    (i) Teacher forcing: every layer is fed the oracle's input for that layer; supports and outputs
        must match under the usual tolerances.
    (ii) Chained: the library runs on its own residual stream.  Rounding differences accumulate
        over the layers and can move a later sketch by more than the 1e-4 margin that pins a
        support, so the free-running chains may pick different supports; the library's chain is
        therefore compared with an oracle chain replayed on the library's supports, which checks
        every layer's arithmetic on the library's own inputs."""
    cfg = W.CONFIGS["l3_8b_stack"]
    plan = make_plan(cfg)
    L0 = _layer(cfg, 0)
    x_ref = W.make_tokens(cfg, L0.A).h.double().numpy()
    x_replay = x_ref.copy()
    x_gpu = torch.from_numpy(x_ref).float().to(DEV)
    excused = 0
    worst = 0.0
    same_support_rows = 0
    for layer in range(cfg.n_layers):
        L = L0 if layer == 0 else _layer(cfg, layer)
        x_in = torch.from_numpy(x_ref).float()      # teacher forcing: oracle's stream, as stored f32
        rep, ref_out, _ = compare_layer_step(cfg, L, plan, x_in)
        excused += rep.excused
        worst = max(worst, rep.max_out_err)
        # chained: the library's own residual stream, and the oracle replayed on its supports
        lay = device_layer(plan, L)
        _, sup, _, _ = cs.cs_layer_step(plan, lay, x_gpu, x_out=x_gpu)
        sup = sup.cpu().numpy()
        Lc = L.to("cpu")
        free = oracle.layer_step(Lc, x_replay, group=cfg.group, k=cfg.k, T=cfg.T, rms_eps=cfg.rms_eps,
                                 forced_support=sup)
        same_support_rows += int((free.support == sup).all(axis=1).sum())
        x_replay = free.x_out
        x_ref = ref_out
        del L, lay, Lc
    torch.cuda.synchronize()
    chain_err = rel(x_gpu.cpu().numpy(), x_replay)
    print(f"stack: excused {excused}/{cfg.B * cfg.n_layers}, worst layer err {worst:.2e}, "
          f"chained err vs support-forced replay {chain_err:.2e}, "
          f"chain rows whose support equals the replay's own recovery {same_support_rows}/{cfg.B * cfg.n_layers}")
    assert excused <= 8
    assert chain_err <= OUT_TOL["bf16"]


@pytest.mark.parametrize("k", W.PROMPT_K_SWEEP)
def test_prompt_support_parity(k):
    cfg = W.CONFIGS["l2_13b_prompt"].with_(k=k)
    A = W.make_probe(cfg)
    Phi = rng.normal(cfg.seed, (W.T_PHI, 0), (cfg.m, cfg.G), dtype=torch.float32, scale=cfg.m ** -0.5)
    S = (Phi.double() @ A).float()
    mu = W.spectral_step(Phi)
    H = W.make_tokens(cfg, A).h
    plan = make_plan(cfg)
    sup, z, resid = cs.cs_prompt_support(plan, S.to(DEV), Phi.to(DEV), mu, H.to(DEV))
    ybar, ref = oracle.prompt_support(S, Phi, H, k, cfg.T, mu)
    sup = sup.cpu().numpy()
    if ref.min_gap > GAP_TOL:
        assert np.array_equal(sup, ref.support)
    if np.array_equal(sup, ref.support):
        assert rel(z.cpu().numpy(), ref.z[ref.support]) <= Z_TOL
        assert abs(resid.item() - ref.resid) <= 1e-4 * max(1.0, ref.resid)


# ------------------------------------------------------------------ tensor-core regime
def test_bucket_inverts_supports():
    cfg = W.CONFIGS["l2_7b_b64"]
    sup = rng.k_subset(cfg.seed, (55,), cfg.G, cfg.k, rows=cfg.B)
    plan = make_plan(cfg)
    counts, offsets, token_ids = (t.cpu().numpy() for t in cs.cs_bucket(plan, sup.to(DEV)))
    assert plan.device_status() == 0
    s = sup.numpy()
    for g in range(cfg.G):
        members = [t for t in range(cfg.B) if g in s[t]]
        assert counts[g] == len(members)
        assert list(token_ids[offsets[g]:offsets[g + 1]]) == members
    assert offsets[0] == 0 and offsets[cfg.G] == cfg.B * cfg.k


@pytest.mark.parametrize("B", [5, 8, 11, 16, 64, 100, 128, 130])
def test_ffn_exec_tensor_path_matches_oracle(B):
    """Decode batches from the crossover batch (5 tokens at this shape) up run as grouped GEMMs over
    the union of the supports."""
    cfg = W.CONFIGS["l2_7b_b64"].with_(B=B)
    L = _layer(cfg)
    Lc = L.to("cpu")
    tk = W.make_tokens(cfg, L.A, B=B)
    plan = make_plan(cfg, max_tokens=B)
    lay = device_layer(plan, L)
    res = rng.normal(cfg.seed, (79,), (B, cfg.d), dtype=torch.float32)
    out = cs.cs_ffn_exec(plan, lay, tk.h.to(DEV), tk.planted.to(DEV), residual=res.to(DEV)).cpu().numpy()
    assert plan.device_status() == 0
    for t in range(B):   # every token
        ref = oracle.ffn(Lc.W_gate, Lc.W_up, Lc.Wd_t, cfg.group, tk.h[t], tk.planted[t])
        err = rel(out[t].astype(np.float64) - res[t].double().numpy(), ref)
        assert err <= OUT_TOL["bf16"] and err <= TIGHT_TOL["bf16"], (t, err)


@pytest.mark.parametrize("B", [4, 5, 9])
def test_layer_step_around_the_crossover_batch(B):
    """The fused step on both sides of the batch where the tensor-core path takes over."""
    cfg = W.CONFIGS["l2_7b_b64"].with_(B=B)
    L = _layer(cfg)
    tk = W.make_tokens(cfg, L.A, B=B)
    rep, _, _ = compare_layer_step(cfg, L, make_plan(cfg, max_tokens=B), tk.h)
    print(B, rep)


def test_plan_crossover_setting_moves_a_batch_between_the_paths():
    """cs_plan_set_crossover: the same 6-token batch through the gather path (crossover above it) and through
    the tensor cores (crossover below it) gives the oracle's result either way and the same supports; the
    default is max(2, min(16, ceil(1.15 G / k))) and values outside 1..129 are refused."""
    cfg = W.CONFIGS["l2_7b_b64"].with_(B=6)
    L = _layer(cfg)
    tk = W.make_tokens(cfg, L.A, B=6)
    lo, hi = make_plan(cfg, max_tokens=6), make_plan(cfg, max_tokens=6)
    assert lo.crossover == max(2, min(16, -(-115 * cfg.G // (100 * cfg.k))))
    lo.set_crossover(2); hi.set_crossover(129)
    assert lo.crossover == 2 and hi.crossover == 129
    for bad in (0, 130, -3):
        with pytest.raises(Exception):
            lo.set_crossover(bad)
    rep_lo, _, out_lo = compare_layer_step(cfg, L, lo, tk.h)
    rep_hi, _, out_hi = compare_layer_step(cfg, L, hi, tk.h)
    if rep_lo.excused == 0 and rep_hi.excused == 0:
        assert rel(out_lo.cpu().numpy(), out_hi.cpu().numpy()) <= 2e-5
    assert lo.launches != hi.launches     # different chains of kernels ran
    lo.close(); hi.close()


def test_ffn_exec_tensor_path_skips_unused_groups():
    """A batch whose supports leave most groups unused: the union list is short and ragged."""
    cfg = W.CONFIGS["l2_7b_b64"].with_(B=20, k=3)
    L = _layer(cfg)
    Lc = L.to("cpu")
    tk = W.make_tokens(cfg, L.A, B=20)
    sup = torch.tensor([[1, 40, 85], [1, 2, 85], [0, 40, 41]], dtype=torch.int32).repeat(7, 1)[:20].contiguous()
    plan = make_plan(cfg, max_tokens=20)
    out = cs.cs_ffn_exec(plan, device_layer(plan, L), tk.h.to(DEV), sup.to(DEV)).cpu().numpy()
    for t in range(20):
        ref = oracle.ffn(Lc.W_gate, Lc.W_up, Lc.Wd_t, cfg.group, tk.h[t], sup[t])
        assert rel(out[t], ref) <= TIGHT_TOL["bf16"], t


@pytest.mark.parametrize("k", W.PROMPT_K_SWEEP)
def test_ffn_exec_shared_parity(k):
    """Prompt-level variant at full size: 2048 tokens, one shared support; the first, a middle and the
    last token of each of the sixteen 128-token tiles against the oracle."""
    cfg = W.CONFIGS["l2_13b_prompt"].with_(k=k)
    L = _layer(cfg)
    Lc = L.to("cpu")
    tk = W.make_tokens(cfg, L.A)
    plan = make_plan(cfg)
    lay = device_layer(plan, L)
    H = tk.h.to(DEV)
    sup, _, _ = cs.cs_prompt_support(plan, L.S, L.Phi, L.mu, H)
    out = cs.cs_ffn_exec_shared(plan, lay, H, sup)
    torch.cuda.synchronize()
    assert plan.device_status() == 0
    out = out.float().cpu().numpy()
    s = sup.cpu().numpy()
    worst = 0.0
    for tile in range(cfg.B // 128):
        for t in (128 * tile, 128 * tile + 37 + tile, 128 * tile + 127):
            ref = oracle.ffn(Lc.W_gate, Lc.W_up, Lc.Wd_t, cfg.group, tk.h[t].double().numpy(), s)
            err = rel(out[t], ref)
            assert err <= OUT_TOL["bf16"] and err <= PROMPT_TIGHT_TOL, (t, err)
            worst = max(worst, err)
    print(f"k={k}: worst relative error over 48 tokens {worst:.2e}")


def test_ffn_exec_shared_ragged_prompt_length():
    cfg = W.CONFIGS["l2_13b_prompt"].with_(k=5, B=333, d=1024, d_ff=128 * 9, m=16)
    L = _layer(cfg)
    Lc = L.to("cpu")
    tk = W.make_tokens(cfg, L.A)
    plan = make_plan(cfg)
    sup = torch.tensor([0, 2, 3, 7, 8], dtype=torch.int32, device=DEV)
    out = cs.cs_ffn_exec_shared(plan, device_layer(plan, L), tk.h.to(DEV), sup).float().cpu().numpy()
    assert plan.device_status() == 0
    for t in (0, 127, 128, 255, 256, 332):
        ref = oracle.ffn(Lc.W_gate, Lc.W_up, Lc.Wd_t, cfg.group, tk.h[t].double().numpy(), sup.cpu().numpy())
        assert rel(out[t], ref) <= PROMPT_TIGHT_TOL, t


def test_ffn_exec_shared_random_shapes():
    """Twenty random prompt-level shapes: d with and without the 320-column tiling, prompt lengths
    around the 128-token tile, any k of G groups; sampled tokens against the oracle."""
    rs = np.random.default_rng(5)
    for trial in range(20):
        G = int(rs.integers(2, 40)); k = int(rs.integers(1, G + 1))
        d = int(rs.choice([256, 512, 768, 1024, 1280, 2560, 4096, 5120]))
        n = int(rs.choice([1, 5, 127, 128, 129, 300, 640, 1000]))
        cfg = W.CONFIGS["l2_13b_prompt"].with_(k=k, B=n, d=d, d_ff=128 * G, m=16, index=200 + trial)
        L = _layer(cfg)
        Lc = L.to("cpu")
        tk = W.make_tokens(cfg, L.A)
        plan = make_plan(cfg)
        sup = torch.tensor(np.sort(rs.choice(G, k, replace=False)), dtype=torch.int32, device=DEV)
        out = cs.cs_ffn_exec_shared(plan, device_layer(plan, L), tk.h.to(DEV), sup).float().cpu().numpy()
        assert plan.device_status() == 0
        for t in sorted({0, n // 2, n - 1, min(n - 1, 127), min(n - 1, 128)}):
            ref = oracle.ffn(Lc.W_gate, Lc.W_up, Lc.Wd_t, cfg.group, tk.h[t].double().numpy(), sup.cpu().numpy())
            assert rel(out[t], ref) <= PROMPT_TIGHT_TOL, (trial, G, k, d, n, t)
        plan.close()


# ------------------------------------------------------------------ uncertainty-driven budget
def _check_budget(m_gpu, H_gpu, ref, m_base, gamma):
    H_gpu = H_gpu.cpu().numpy().astype(np.float64); m_gpu = m_gpu.cpu().numpy()
    for t in range(len(ref.H)):
        assert abs(H_gpu[t] - ref.H[t]) <= 2e-5 * max(1.0, ref.H[t]), (t, H_gpu[t], ref.H[t])
        # the floor may differ only where f32 rounding of H can carry x across an integer
        slack = m_base * gamma * 2e-5 * max(1.0, ref.H[t])
        if abs(ref.x[t] - round(ref.x[t])) > slack:
            assert m_gpu[t] == ref.m[t], (t, m_gpu[t], ref.m[t], ref.x[t])
        else:
            assert abs(int(m_gpu[t]) - int(ref.m[t])) <= 1


@pytest.mark.parametrize("B,V", [(1, 128256), (5, 32000), (64, 32000), (3, 50257), (2, 7), (4, 4096), (1, 1)])
def test_uds_budget_matches_oracle(B, V):
    """Sec. 8.1: entropy of the previous step's distribution and the budget it sets, at vocabulary
    sizes of the benchmark's model families, ragged sizes, and temperatures from peaked to flat."""
    g = torch.Generator().manual_seed(100 + B + V)
    logits = torch.randn((B, V), generator=g) * torch.logspace(-1, 1.3, B)[:, None] + 3.0
    plan = cs.Plan(256, 1024, 64, 8, 4, 4, torch.float32, max(B, 1), 1e-5)
    m_base, gamma, m_min, m_max = 16.0, 0.75, 8, 64
    m_t, H = cs.cs_uds_budget(plan, logits.to(DEV), m_base, gamma, m_min, m_max)
    _check_budget(m_t, H, oracle.uds_budget(logits, m_base, gamma, m_min, m_max), m_base, gamma)
    plan.close()


def test_uds_budget_special_rows():
    """Uniform row (H = log V), one dominant logit (H = 0, m = m_base), masked entries (-inf),
    an entirely masked row, a NaN row (m_max), clipping at both ends, H not requested."""
    V = 10000
    L = torch.zeros((7, V))
    L[1, 123] = 500.0
    L[2] = torch.randn(V, generator=torch.Generator().manual_seed(1)); L[2, ::3] = float("-inf")
    L[3] = float("-inf")
    L[4, 5] = float("nan")
    L[5] = torch.randn(V, generator=torch.Generator().manual_seed(2)) * 0.01     # near uniform: clipped at m_max
    L[6, 0] = 40.0                                                               # near certain: H ~ 0
    plan = cs.Plan(256, 1024, 64, 8, 4, 4, torch.float32, 8, 1e-5)
    m_t, H = cs.cs_uds_budget(plan, L.to(DEV), 32.0, 0.5, 16, 100)
    m = m_t.cpu().numpy(); Hh = H.cpu().numpy()
    assert abs(Hh[0] - np.log(V)) < 1e-4 and m[0] == min(100, int(np.floor(32 * (1 + 0.5 * np.log(V)))))
    assert Hh[1] == 0.0 and m[1] == 32
    ref = oracle.uds_budget(L[2:3], 32.0, 0.5, 16, 100)
    assert abs(Hh[2] - ref.H[0]) < 1e-4 and m[2] == ref.m[0]
    assert Hh[3] == 0.0 and m[3] == 32
    assert np.isnan(Hh[4]) and m[4] == 100
    assert m[5] == 100 and m[6] == 32
    lib = plan.lib
    m2 = torch.empty(7, dtype=torch.int32, device=DEV)
    Ld = L.to(DEV)
    plan.check(lib.cs_uds_budget(plan.handle, Ld.data_ptr(), 7, V, 2.0, 0.5, 16, 100, None, m2.data_ptr(), None), "cs_uds_budget")
    torch.cuda.synchronize()
    assert (m2.cpu().numpy()[[0, 1, 6]] == 16).all()                             # lower bound
    for bad, code in [((0, V, 2.0, 0.5, 16, 100), 2), ((9, V, 2.0, 0.5, 16, 100), 2), ((7, V, 2.0, 0.5, 0, 100), 2),
                      ((7, V, 2.0, 0.5, 17, 16), 2), ((7, V, 0.0, 0.5, 16, 100), 5), ((7, V, 2.0, -1.0, 16, 100), 5),
                      ((7, V, float("nan"), 0.5, 16, 100), 5)]:
        assert lib.cs_uds_budget(plan.handle, Ld.data_ptr(), bad[0], bad[1], bad[2], bad[3], bad[4], bad[5], None,
                                 m2.data_ptr(), None) == code, bad
    plan.close()


def test_uds_budget_selects_a_row_prefix_of_the_measurement_bank():
    """Sec. 8.1 (the sensing matrix varies in its row dimension): the first m_t rows of a bank
    S [m_max, d], Phi [m_max, G] are the operands of a plan created with m = m_t."""
    cfg = W.CONFIGS["tiny_f32"]
    m_max = 24
    big = cfg.with_(m=m_max)
    L = _layer(big)
    tk = W.make_tokens(big, L.A, B=3)
    logits = torch.randn((3, 5000), generator=torch.Generator().manual_seed(9)) * torch.tensor([8.0, 2.0, 0.2])[:, None]
    ctl = make_plan(big, max_tokens=3)
    m_t, _ = cs.cs_uds_budget(ctl, logits.to(DEV), 6.0, 0.35, 4, m_max)
    m_t = m_t.cpu().numpy()
    assert list(m_t) == list(oracle.uds_budget(logits, 6.0, 0.35, 4, m_max).m) and len(set(m_t)) == 3
    for t in range(3):
        mt = int(m_t[t])
        plan = make_plan(big.with_(m=mt), max_tokens=1)
        S_t, Phi_t = L.S[:mt], L.Phi[:mt]                    # contiguous row prefixes of the bank
        assert S_t.is_contiguous() and Phi_t.is_contiguous()
        mu = W.spectral_step(Phi_t.cpu())
        x = tk.h[t:t + 1]
        y = cs.cs_sketch(plan, S_t, x.to(DEV))
        sup, z, _ = cs.cs_recover(plan, Phi_t, mu, y)
        yr = oracle.sketch(S_t.cpu(), x[0])
        ref = oracle.iht(Phi_t.cpu(), yr, big.k, big.T, mu)
        assert rel(y[0].cpu().numpy(), yr) <= 1e-5
        if ref.min_gap > GAP_TOL:
            assert np.array_equal(sup[0].cpu().numpy(), ref.support)
            assert rel(z[0].cpu().numpy(), ref.z[ref.support]) <= Z_TOL
        plan.close()
    ctl.close()


# ------------------------------------------------------------------ host-buffer entry point
@pytest.mark.parametrize("name,B,pinned", [("l2_7b_b1", 1, True), ("l2_7b_b1", 1, False), ("tiny_f32", 4, True),
                                           ("l2_7b_b64", 3, True), ("l2_7b_b64", 9, True), ("l2_7b_b64", 9, False),
                                           ("l3_8b_stack", 2, True)])   # RMSNorm + residual stream
def test_layer_step_host_matches_device_entry(name, B, pinned):
    """Host buffers in, host buffers out: page-locked small batches travel inside the step's own
    kernels, everything else through the copy engine; both give the device entry's bits, also when
    the host rewrites the input between calls and when the calls are replayed from a graph."""
    cfg = W.CONFIGS[name].with_(B=B)
    L = _layer(cfg)
    plan = make_plan(cfg, max_tokens=B)
    lay = device_layer(plan, L)
    hx = torch.empty((B, cfg.d), dtype=torch.float32)
    hout = torch.empty((B, cfg.d), dtype=torch.float32)
    hsup = torch.empty((B, cfg.k), dtype=torch.int32)
    if pinned:
        hx, hout, hsup = hx.pin_memory(), hout.pin_memory(), hsup.pin_memory()
    for batch in range(3):
        tk = W.make_tokens(cfg, L.A, batch=batch, B=B)
        hx.copy_(tk.h)
        hout.fill_(float("nan"))
        cs.cs_layer_step_host(plan, lay, hx, hout, hsup if batch != 1 else None)
        torch.cuda.synchronize()
        want, sup, _, _ = cs.cs_layer_step(plan, lay, tk.h.to(DEV))
        assert plan.device_status() == 0
        assert torch.equal(hout, want.cpu()), batch
        if batch != 1:
            assert torch.equal(hsup, sup.cpu())
    if pinned:
        stream = torch.cuda.Stream()
        g = torch.cuda.CUDAGraph()
        with torch.cuda.stream(stream):
            cs.cs_layer_step_host(plan, lay, hx, hout)
            stream.synchronize()
            with torch.cuda.graph(g, stream=stream):
                for _ in range(3):
                    cs.cs_layer_step_host(plan, lay, hx, hout)
        for batch in (4, 5):
            tk = W.make_tokens(cfg, L.A, batch=batch, B=B)
            hx.copy_(tk.h)                      # the replay must see what the host wrote
            hout.fill_(float("nan"))
            g.replay()
            torch.cuda.synchronize()
            want, _, _, _ = cs.cs_layer_step(plan, lay, tk.h.to(DEV))
            assert torch.equal(hout, want.cpu()), batch
    plan.close()


def test_layer_step_host_chained_through_one_buffer():
    """Three layers chained through ONE pinned buffer with no synchronisation in between: layer i stores
    its result into the buffer layer i + 1 reads, so the staging load must respect stream order."""
    cfg = W.CONFIGS["l3_8b_stack"].with_(B=2)
    plan = make_plan(cfg, max_tokens=2)
    Ls = [_layer(cfg, i) for i in range(3)]
    lays = [device_layer(plan, L) for L in Ls]
    x0 = W.make_tokens(cfg, Ls[0].A, B=2).h
    buf = torch.empty((2, cfg.d), dtype=torch.float32).pin_memory()
    for rep in range(3):
        buf.copy_(x0)
        for lay in lays:
            cs.cs_layer_step_host(plan, lay, buf, buf)
        torch.cuda.synchronize()
        x = x0.to(DEV)
        for lay in lays:
            x, _, _, _ = cs.cs_layer_step(plan, lay, x)
        assert torch.equal(buf, x.cpu()), rep
    plan.close()


def test_support_drift_matches_oracle():
    """Sec. 11: |S_t symmetric-difference S_{t-1}| for random supports (k from 1 to G), identical and
    disjoint rows, and for the supports of two consecutive recoveries."""
    rs = np.random.default_rng(21)
    for G, k in [(86, 22), (112, 28), (128, 128), (16, 1), (108, 54), (128, 64)]:
        B = 9
        plan = cs.Plan(256, G * 64, 64, 8, k, 4, torch.float32, B, 1e-5)
        prev = np.stack([np.sort(rs.choice(G, k, replace=False)) for _ in range(B)]).astype(np.int32)
        cur = np.stack([np.sort(rs.choice(G, k, replace=False)) for _ in range(B)]).astype(np.int32)
        cur[0] = prev[0]
        if 2 * k <= G:
            cur[1] = np.sort(np.setdiff1d(np.arange(G), prev[1])[:k])
        got = cs.cs_support_drift(plan, torch.tensor(prev, device=DEV), torch.tensor(cur, device=DEV)).cpu().numpy()
        assert plan.device_status() == 0
        assert got.tolist() == oracle.support_drift(prev, cur).tolist(), (G, k)
        assert got[0] == 0 and (2 * k > G or got[1] == 2 * k)
        plan.close()
    cfg = W.CONFIGS["l2_7b_b64"]
    L = _layer(cfg)
    tk = W.make_tokens(cfg, L.A, B=8)
    plan = make_plan(cfg, max_tokens=8)
    y = cs.cs_sketch(plan, L.S, tk.h.to(DEV))
    s0, z0, _ = cs.cs_recover(plan, L.Phi, L.mu, y)
    s1, _, _ = cs.cs_recover_warm(plan, L.Phi, L.mu, y * 1.02 + 0.05 * y.roll(1, 1), 4, s0, z0)
    got = cs.cs_support_drift(plan, s0, s1).cpu().numpy()
    assert got.tolist() == oracle.support_drift(s0.cpu().numpy(), s1.cpu().numpy()).tolist()
    bad = s1.clone(); bad[2, 0] = bad[2, 1]                    # not ascending: flagged, not a fault
    cs.cs_support_drift(plan, s0, bad)
    assert plan.device_status() == 4
    plan.close()
