"""Pins for the oracle's GATHER-ATT (Section 4 formula) and single-query SDPA (Section 3.1):
hand-derived closed forms, torch's float64 scaled_dot_product_attention, and invariants; plus
the composition of the whole decode step.  CPU only."""
import math
import os

import numpy as np
import torch

import oracle
from paper_2412_14468_b200 import workloads as wl

GOLD = os.path.join(os.path.dirname(__file__), "golden")
D = 128


def bf16(a):
    t = torch.as_tensor(np.asarray(a, dtype=np.float32)).to(torch.bfloat16)
    return t.view(torch.int16).numpy().view(np.uint16).copy()


def f64(bits):
    return oracle.bf16_bits_to_f64(bits)


def _rand(n, seed, scale=1.0):
    rng = np.random.default_rng(seed)
    return (bf16(rng.standard_normal(D)), bf16(scale * rng.standard_normal((n, D))), bf16(rng.standard_normal((n, D))))


def test_golden_attention_closed_forms():
    with open(os.path.join(GOLD, "attention_cases.txt")) as f:
        lines = [ln.strip() for ln in f if ln.strip() and not ln.startswith("#")]
    for ln in lines:
        kap, nus, idx, exp = [p.strip() for p in ln.split("|")]
        kap = [float(v) for v in kap.split()]
        nus = [float(v) for v in nus.split()]
        n = len(kap)
        q = np.zeros(D, np.float32); q[0] = 1.0
        K = np.zeros((n, D), np.float32); K[:, 0] = kap
        V = np.repeat(np.asarray(nus, np.float32)[:, None], D, axis=1)
        out, lse, out64 = oracle.gather_attn(bf16(q), bf16(K), bf16(V), [int(v) for v in idx.split()], sm_scale=1.0)
        assert np.allclose(out64, float(exp), rtol=0, atol=1e-14), ln
        assert np.allclose(f64(out), float(exp), rtol=2 ** -8, atol=0), ln


def test_dense_matches_torch_sdpa_float64():
    for seed, n in ((20, 1), (21, 17), (22, 300)):
        q, K, V = _rand(n, seed)
        out, lse, out64 = oracle.dense(q, K, V)
        tq = torch.tensor(f64(q)).view(1, 1, 1, D)
        tk = torch.tensor(f64(K)).view(1, 1, n, D)
        tv = torch.tensor(f64(V)).view(1, 1, n, D)
        ref = torch.nn.functional.scaled_dot_product_attention(tq, tk, tv).view(D).numpy()
        assert np.max(np.abs(out64 - ref)) < 1e-12
        logits = (tk.view(n, D) @ tq.view(D)) / math.sqrt(D)
        assert abs(lse - torch.logsumexp(logits, 0).item()) < 1e-12
        # the bf16 result is the float64 result rounded once
        assert np.array_equal(out, np.array([oracle.f64_to_bf16_bits(v) for v in out64], dtype=np.uint16))


def test_sm_scale_is_applied_to_logits():
    q, K, V = _rand(50, 23)
    _, _, a = oracle.dense(q, K, V, sm_scale=0.25)
    tq, tk, tv = (torch.tensor(f64(x)) for x in (q, K, V))
    p = torch.softmax(0.25 * (tk @ tq), 0)
    assert np.max(np.abs(a - (p[:, None] * tv).sum(0).numpy())) < 1e-12


def test_k_equals_n_is_dense_and_permutation_is_irrelevant():
    q, K, V = _rand(128, 24)
    d_out, d_lse, d64 = oracle.dense(q, K, V)
    g_out, g_lse, g64 = oracle.gather_attn(q, K, V, np.arange(128))
    assert np.array_equal(d_out, g_out) and d_lse == g_lse
    perm = np.random.default_rng(0).permutation(128)
    p_out, p_lse, p64 = oracle.gather_attn(q, K, V, perm)
    assert np.max(np.abs(p64 - d64)) < 1e-13 and abs(p_lse - d_lse) < 1e-13


def test_single_index_returns_that_value_row_exactly():
    q, K, V = _rand(40, 25)
    out, lse, _ = oracle.gather_attn(q, K, V, [17])
    assert np.array_equal(out, V[17])
    assert abs(lse - float(f64(q) @ f64(K[17])) / math.sqrt(D)) < 1e-12


def test_zero_query_gives_plain_mean_and_identical_values_give_that_row():
    _, K, V = _rand(64, 26)
    idx = [3, 9, 27, 40]
    _, lse, out64 = oracle.gather_attn(np.zeros(D, np.uint16), K, V, idx)
    assert np.max(np.abs(out64 - f64(V[idx]).mean(axis=0))) < 1e-14
    assert abs(lse - math.log(4)) < 1e-14
    q, K, _ = _rand(64, 27)
    Vsame = np.repeat(V[5:6], 64, axis=0)
    out, _, _ = oracle.gather_attn(q, K, Vsame, np.arange(0, 64, 3))
    assert np.array_equal(out, V[5])


def test_lse_merge_identity_across_a_split_of_the_index_set():
    q, K, V = _rand(90, 28, scale=3.0)
    idx = np.random.default_rng(1).permutation(90)[:60]
    _, lse, full = oracle.gather_attn(q, K, V, idx)
    _, l1, o1 = oracle.gather_attn(q, K, V, idx[:23])
    _, l2, o2 = oracle.gather_attn(q, K, V, idx[23:])
    m = max(l1, l2)
    w1, w2 = math.exp(l1 - m), math.exp(l2 - m)
    assert abs(lse - (m + math.log(w1 + w2))) < 1e-12
    assert np.max(np.abs(full - (w1 * o1 + w2 * o2) / (w1 + w2))) < 1e-12


def test_invalid_and_duplicate_indices_and_empty_list():
    q, K, V = _rand(30, 29)
    a = oracle.gather_attn(q, K, V, [2, 5, -1, 29, 30, 1000], n_valid=30)[2]
    b = oracle.gather_attn(q, K, V, [2, 5, 29])[2]
    assert np.array_equal(a, b)
    c = oracle.gather_attn(q, K, V, [2, 5, 10], n_valid=10)[2]       # tokens beyond the sequence are skipped
    assert np.array_equal(c, oracle.gather_attn(q, K, V, [2, 5])[2])
    out, lse, out64 = oracle.gather_attn(q, K, V, np.array([], dtype=np.int32))
    assert not out.any() and lse == -math.inf
    dup = oracle.gather_attn(q, K, V, [4, 4, 7])[2]                  # each occurrence counts
    tq, tk, tv = f64(q), f64(K), f64(V)
    l = np.array([tk[4] @ tq, tk[4] @ tq, tk[7] @ tq]) / math.sqrt(D)
    p = np.exp(l - l.max()); p /= p.sum()
    assert np.max(np.abs(dup - (p[0] * tv[4] + p[1] * tv[4] + p[2] * tv[7]))) < 1e-13


def test_f64_to_bf16_rounds_to_nearest_even_once():
    assert oracle.f64_to_bf16_bits(1.0) == 0x3F80
    assert oracle.f64_to_bf16_bits(1.0 + 2 ** -8) == 0x3F80          # tie -> even
    assert oracle.f64_to_bf16_bits(1.0 + 3 * 2 ** -8) == 0x3F82      # tie -> even (up)
    assert oracle.f64_to_bf16_bits(1.0 + 2 ** -8 + 2 ** -40) == 0x3F81
    assert oracle.f64_to_bf16_bits(-2.5) == 0xC020
    assert oracle.f64_to_bf16_bits(0.0) == 0
    rng = np.random.default_rng(30)
    x = rng.standard_normal(2000) * np.exp(rng.uniform(-20, 20, 2000))
    got = np.array([oracle.f64_to_bf16_bits(v) for v in x], dtype=np.uint16)
    # torch rounds float32 -> bf16 to nearest even; feed values that are exact in float32
    x32 = x.astype(np.float32)
    got32 = np.array([oracle.f64_to_bf16_bits(float(v)) for v in x32], dtype=np.uint16)
    assert np.array_equal(got32, bf16(x32))
    assert np.all(np.abs(f64(got) - x) <= np.abs(x) * 2 ** -8)


def test_decode_step_is_the_composition_and_k_equals_n_is_dense():
    cfg = wl.Config("t", 77, 2, [96, 61], None, 0.05, n_q_heads=8, n_kv_heads=2, sparsity=4)
    w = wl.make_workload(cfg)
    q, K, V, k_new = (wl.as_u16(w[x]) for x in ("q", "K", "V", "k_new"))
    mq, mk = wl.mapping_numpy(w["map_q"]), wl.mapping_numpy(w["map_k"])
    B, Hq, Hkv, G = 2, 8, 2, 4
    codes = np.zeros((B, Hkv, w["n_cap"]), np.uint32)
    for b in range(B):
        for g in range(Hkv):
            codes[b, g] = oracle.encode(K[b, g], mk["w1"][g], mk["w2"][g], mk["w3"][g], mk["b1"][g], mk["b2"][g], mk["b3"][g])
    stale = codes.copy()
    for b in range(B):
        stale[b, :, w["lens"][b] - 1] = 0xFFFFFFFF         # the step must rewrite the appended slot
    r = oracle.decode_step(q, k_new, K, V, stale, mq, mk, w["lens"], w["ks"])
    assert np.array_equal(stale, codes)
    for b in range(B):
        n, k = w["lens"][b], w["ks"][b]
        for g in range(Hkv):
            qc = oracle.encode(q[b, g * G:(g + 1) * G], mq["w1"][g], mq["w2"][g], mq["w3"][g], mq["b1"][g], mq["b2"][g], mq["b3"][g])
            assert np.array_equal(r["qcodes"][b, g * G:(g + 1) * G], qc)
            idx = oracle.topk(oracle.score(qc, codes[b, g, :n]), k)
            assert r["count"][b, g] == min(k, n) and np.array_equal(r["idx"][b, g, :len(idx)], idx)
            assert np.all(r["idx"][b, g, len(idx):] == -1)
            for j in range(G):
                out, lse, _ = oracle.gather_attn(q[b, g * G + j], K[b, g], V[b, g], idx, n_valid=n)
                assert np.array_equal(r["out"][b, g * G + j], out) and r["lse"][b, g * G + j] == lse
    # k = n: the sparse step equals dense SDPA
    full = oracle.decode_step(q, k_new, K, V, codes.copy(), mq, mk, w["lens"], w["lens"], n_threads=2)
    for b in range(B):
        for h in range(Hq):
            out, lse, _ = oracle.dense(q[b, h], K[b, h // G], V[b, h // G], n=w["lens"][b])
            assert np.array_equal(full["out"][b, h], out) and abs(full["lse"][b, h] - lse) < 1e-12


def test_unpaging_is_storage_only():
    """A paged cache read back through its block table gives the rows that were put in, whatever the page
    order and page size; attention over them equals attention over the contiguous rows."""
    rng = np.random.default_rng(5)
    n, Hkv = 70, 2
    K = rng.integers(0, 2 ** 16, size=(Hkv, n, 128), dtype=np.uint64).astype(np.uint16) & 0xBFFF   # finite bf16 patterns
    for ps in (1, 16, 64):
        n_pages = (n + ps - 1) // ps
        perm = rng.permutation(n_pages + 3)[:n_pages]                 # pages scattered over a larger pool
        pool = np.zeros((n_pages + 3, Hkv, ps, 128), np.uint16)
        for t in range(n):
            pool[perm[t // ps], :, t % ps] = K[:, t]
        for h in range(Hkv):
            assert np.array_equal(oracle.unpage_rows(pool, perm, ps, h, n), K[h])
