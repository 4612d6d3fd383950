"""The seeded generators: counter-based words, distributions, workload shapes."""
import numpy as np
import torch

from gen import rng, workloads as W


def test_words_match_integer_reference():
    w = rng.bits(12345, (3, 7), 64)
    for i in (0, 1, 2, 31, 63):
        v = rng.word_int(12345, (3, 7), i)
        v = v - (1 << 64) if v >= (1 << 63) else v
        assert int(w[i]) == v


def test_offset_and_chunking_are_index_addressable():
    a = rng.bits(9, 1, 100)
    b = rng.bits(9, 1, 40, offset=60)
    assert torch.equal(a[60:], b)
    old = rng._CHUNK
    try:
        full = rng.normal(5, (2,), (1000,))
        rng._CHUNK = 64
        assert torch.equal(full, rng.normal(5, (2,), (1000,)))
    finally:
        rng._CHUNK = old


def test_streams_differ_and_moments():
    x = rng.normal(1, (1,), 200000)
    y = rng.normal(1, (2,), 200000)
    assert abs(x.mean()) < 0.01 and abs(x.std() - 1) < 0.01
    assert abs((x * y).mean()) < 0.01
    assert abs((x ** 4).mean() - 3.0) < 0.1
    u = rng.uniform(3, 0, 100000)
    assert 0 < u.min() and u.max() < 1 and abs(u.mean() - 0.5) < 0.01


def test_k_subset():
    s = rng.k_subset(4, 0, 16, 4, rows=2000)
    assert s.shape == (2000, 4)
    assert (s[:, 1:] > s[:, :-1]).all() and s.min() >= 0 and s.max() < 16
    counts = torch.bincount(s.flatten().long(), minlength=16).double() / 2000
    assert (counts - 0.25).abs().max() < 0.05


def test_tiny_workload_recipe():
    cfg = W.CONFIGS["tiny_f32"]
    L = W.make_layer(cfg)
    assert L.A.shape == (16, 256) and L.Phi.shape == (8, 16) and L.S.shape == (8, 256)
    assert torch.allclose(L.A.norm(dim=1), torch.ones(16, dtype=torch.float64))
    assert L.W_gate.dtype == torch.float32 and L.Wd_t.shape == (1024, 256)
    # S is the fp64 product of the stored Phi and A, rounded once
    assert torch.equal(L.S, (L.Phi.double() @ L.A).float())
    smax = np.linalg.svd(L.Phi.double().numpy(), compute_uv=False)[0]
    assert abs(L.mu * smax ** 2 - 1) < 1e-6
    tk = W.make_tokens(cfg, L.A)
    assert tk.h.shape == (4, 256) and tk.h.dtype == torch.float32 and tk.planted.shape == (4, 4)
    # the planted part dominates the noise: projecting on the planted rows explains almost all of h
    for t in range(4):
        rows = L.A[tk.planted[t].long()]
        c, *_ = np.linalg.lstsq(rows.numpy().T, tk.h[t].double().numpy(), rcond=None)
        res = tk.h[t].double().numpy() - rows.numpy().T @ c
        assert np.linalg.norm(res) < 0.01 * np.sqrt(256) * 1.5


def test_prompt_workload_shares_one_support():
    cfg = W.CONFIGS["l2_13b_prompt"].with_(B=32)
    tk = W.make_tokens(cfg, W.make_probe(cfg))
    assert tk.planted.shape == (1, 27) and tk.h.shape == (32, 5120) and tk.h.dtype == torch.bfloat16


def test_config_table_matches_the_stated_shapes():
    c = W.CONFIGS
    assert (c["l2_7b_b1"].G, c["l2_7b_b64"].G, c["l3_8b_stack"].G, c["l2_13b_prompt"].G) == (86, 86, 112, 108)
    assert [round(p * 108) for p in (0.10, 0.25, 0.50)] == list(W.PROMPT_K_SWEEP)
