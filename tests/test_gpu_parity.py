"""GPU parity: every C-ABI entry point against the CPU oracle on the same seeded inputs.
Codes, scores (through the histogram), counts and index sets must match bit for bit; attention
outputs within 1e-2 max-abs (fp32 accumulate, bf16 I/O)."""
import math

import numpy as np
import pytest
import torch

import oracle
from paper_2412_14468_b200 import binding as ha
from paper_2412_14468_b200 import workloads as wl
from tests._util import OUT_AIM, OUT_TOL, assert_out_close, bf16_to_f64, codes_np, max_abs_diff_bf16, \
    oracle_key_codes, oracle_query_codes, u16

pytestmark = pytest.mark.gpu
DEV = "cuda"


def _mapping(hkv, seed):
    g = torch.Generator(device=DEV)
    g.manual_seed(seed)
    return wl.make_mapping(hkv, g, DEV)


# ---------------------------------------------------------------------------- ENCODE

@pytest.mark.parametrize("T", [1, 2, 63, 64, 65, 200])
def test_encode_bulk_and_single_bit_exact(T):
    B, H = 2, 4
    mp = _mapping(H, 100 + T)
    x = torch.randn(B, H, T, 128, device=DEV, generator=torch.Generator(DEV).manual_seed(T)).to(torch.bfloat16)
    codes = torch.zeros(B, H, T + 3, dtype=torch.int32, device=DEV)
    ha.ha_encode(ha.Mapping(mp), 1, x, codes)
    torch.cuda.synchronize()
    got = codes_np(codes)
    m = wl.mapping_numpy(mp)
    xu = u16(x)
    for b in range(B):
        for h in range(H):
            exp = oracle.encode(xu[b, h], m["w1"][h], m["w2"][h], m["w3"][h], m["b1"][h], m["b2"][h], m["b3"][h])
            assert np.array_equal(got[b, h, :T], exp)
            assert not got[b, h, T:].any()          # nothing written past the tokens


def test_encode_query_side_group_sharing_and_append_slot():
    B, Hq, Hkv = 3, 8, 2
    mp = _mapping(Hkv, 7)
    q = torch.randn(B, Hq, 128, device=DEV).to(torch.bfloat16)
    qc = torch.zeros(B, Hq, 1, dtype=torch.int32, device=DEV)
    ha.ha_encode(ha.Mapping(mp), Hq // Hkv, q, qc)
    assert np.array_equal(codes_np(qc)[:, :, 0], oracle_query_codes(q, mp, Hkv))
    # append: code of k_new lands in slot[b]; a negative slot skips the sequence
    k_new = torch.randn(B, Hkv, 128, device=DEV).to(torch.bfloat16)
    cache = torch.full((B, Hkv, 40), 0x55, dtype=torch.int32, device=DEV)
    slot = torch.tensor([0, 39, -1], dtype=torch.int32, device=DEV)
    ha.ha_encode(ha.Mapping(mp), 1, k_new, cache, slot=slot)
    got = codes_np(cache)
    exp = oracle_query_codes(k_new, mp, Hkv)        # heads_per_kv = 1 on the key side
    assert np.array_equal(got[0, :, 0], exp[0]) and np.array_equal(got[1, :, 39], exp[1])
    got[0, :, 0] = 0x55
    got[1, :, 39] = 0x55
    assert np.all(got == 0x55)


@pytest.mark.parametrize("B,Hq,Hkv", [(1, 8, 2), (19, 8, 2), (50, 8, 2), (101, 8, 2), (300, 32, 8), (37, 16, 2), (333, 3, 3),
                                      (1300, 1, 1), (1600, 1, 1), (2200, 1, 1), (2500, 1, 1)])   # item widths 5, 6, 8, 2 x 5
def test_encode_single_token_batches_cover_every_item_width(B, Hq, Hkv):
    """One vector per head and sequence: small batches run one vector per CTA, larger ones items of 2 to 8
    vectors (ragged last item), and the largest several items per CTA; all bit-exact."""
    mp = _mapping(Hkv, 1000 + B)
    g = torch.Generator(DEV).manual_seed(B)
    q = torch.randn(B, Hq, 128, device=DEV, generator=g).to(torch.bfloat16)
    qc = torch.full((B, Hq, 2), 0x33, dtype=torch.int32, device=DEV)
    slot = torch.ones(B, dtype=torch.int32, device=DEV)
    slot[B // 2] = -1                                    # this sequence is skipped
    ha.ha_encode(ha.Mapping(mp), Hq // Hkv, q, qc, slot=slot)
    got = codes_np(qc)
    exp = oracle_query_codes(q, mp, Hkv)
    keep = np.ones(B, bool)
    keep[B // 2] = False
    assert np.array_equal(got[keep, :, 1], exp[keep])
    assert np.all(got[:, :, 0] == 0x33) and np.all(got[~keep] == 0x33)


def test_encode_without_biases_and_strided_input():
    H, T = 2, 70
    mp = _mapping(H, 9)
    nb = {k: v for k, v in mp.items() if k.startswith("w")}
    big = torch.randn(1, T, H, 256, device=DEV).to(torch.bfloat16)
    x = big[..., :128].permute(0, 2, 1, 3)           # [1,H,T,128] view with token stride H*256
    codes = torch.zeros(1, H, T, dtype=torch.int32, device=DEV)
    ha.ha_encode(ha.Mapping(nb), 1, x, codes)
    m = wl.mapping_numpy(nb)
    xu = u16(x.contiguous())
    for h in range(H):
        assert np.array_equal(codes_np(codes)[0, h], oracle.encode(xu[0, h], m["w1"][h], m["w2"][h], m["w3"][h]))


@pytest.mark.parametrize("path", [ha.HA_PREFILL_TCGEN05, ha.HA_PREFILL_MMA_SYNC])
@pytest.mark.parametrize("T,strided", [(1, False), (77, False), (300, True), (4099, False)])
def test_encode_prefill_on_tensor_cores_matches_the_chain_up_to_its_margin(T, strided, path):
    """The tensor-core prompt encoder sums in another order and feeds 16-bit activations to the next layer:
    its signature bits must equal the chain-exact ones wherever the exact last-layer output is not within
    1e-3 of zero (the stated accuracy is ~1e-5), and at most one bit in 100000 may differ at all (a
    16-bit split that loses the sign of its remainder already fails this)."""
    B, H, heads_per_kv = 2, 4, 2
    mp = _mapping(H // heads_per_kv, 500 + T)
    g = torch.Generator(DEV).manual_seed(T)
    if strided:
        big = torch.randn(B, T, H, 256, device=DEV, generator=g).to(torch.bfloat16)
        x = big[..., :128].permute(0, 2, 1, 3)           # [B,H,T,128] view with token stride H*256
    else:
        x = torch.randn(B, H, T, 128, device=DEV, generator=g).to(torch.bfloat16)
    codes = torch.full((B, H, T + 5), 0x33, dtype=torch.int32, device=DEV)
    shape = ha.make_shape(B, H, H // heads_per_kv, 1.0)
    ws = ha.alloc_workspace(shape, 16, 16)
    ha.ha_encode_prefill(ha.Mapping(mp), heads_per_kv, x, codes, path=path, workspace=ws)
    assert ha.ha_read_device_status(ws) == 0          # no wait on the tensor cores ran out
    exact = torch.zeros(B, H, T, dtype=torch.int32, device=DEV)
    ha.ha_encode(ha.Mapping(mp), heads_per_kv, x, exact)
    torch.cuda.synchronize()
    got, ref = codes_np(codes), codes_np(exact)
    assert np.all(got[:, :, T:] == 0x33)                 # nothing written past the tokens
    m = wl.mapping_numpy(mp)
    xu = u16(x.contiguous())
    n_diff = 0
    for b in range(B):
        for h in range(H):
            net = h // heads_per_kv
            ora, z3 = oracle.encode(xu[b, h], m["w1"][net], m["w2"][net], m["w3"][net], m["b1"][net], m["b2"][net],
                                    m["b3"][net], return_z3=True)
            assert np.array_equal(ref[b, h], ora)        # ha_encode stays chain-exact
            diff = got[b, h, :T] ^ ora
            for t in np.nonzero(diff)[0]:
                for o in range(32):
                    if (int(diff[t]) >> o) & 1:
                        n_diff += 1
                        assert abs(float(z3[t, o])) < 1e-3, (b, h, t, o, float(z3[t, o]))
    assert n_diff <= max(2, B * H * T * 32 // 100000)


# ---------------------------------------------------------------------------- SCORE + TOPK

def _run_score_topk(qc_np, kc_np, lens, ks, Hq, Hkv, k_uniform=None, n_sink=0, n_local=0, reduce="max"):
    B = len(lens)
    n_cap = kc_np.shape[2]
    k_max = max(max(ks) + n_sink + n_local, 1)
    shape = ha.make_shape(B, Hq, Hkv, 1.0, n_sink=n_sink, n_local=n_local)
    ws = ha.alloc_workspace(shape, n_cap, k_max)
    qc = torch.from_numpy(qc_np.view(np.int32)).to(DEV)
    kc = torch.from_numpy(kc_np.view(np.int32)).to(DEV)
    sl = torch.tensor(lens, dtype=torch.int32, device=DEV)
    kp = None if k_uniform is not None else torch.tensor(ks, dtype=torch.int32, device=DEV)
    idx = torch.full((B, Hkv, k_max), -7, dtype=torch.int32, device=DEV)
    cnt = torch.full((B, Hkv), -7, dtype=torch.int32, device=DEV)
    hist = torch.full((B, Hkv, 33 if reduce == "max" else 32 * (Hq // Hkv) + 1), -7, dtype=torch.int32, device=DEV)
    if reduce == "max":
        ha.ha_score_topk(shape, qc, kc, sl, kp, k_uniform if k_uniform is not None else 0, n_cap, k_max, idx, cnt, ws,
                         hist_out=hist)
    else:   # the per-head scores added up: a stand-alone entry without workspace
        ha.ha_score_topk_sum(shape, qc, kc, sl, kp, k_uniform if k_uniform is not None else 0, k_max, idx, cnt,
                             hist_out=hist)
    torch.cuda.synchronize()
    return idx.cpu().numpy(), cnt.cpu().numpy(), hist.cpu().numpy()


def _check_score_topk(qc_np, kc_np, lens, ks, Hq, Hkv, n_sink=0, n_local=0, reduce="max", **kw):
    idx, cnt, hist = _run_score_topk(qc_np, kc_np, lens, ks, Hq, Hkv, n_sink=n_sink, n_local=n_local, reduce=reduce, **kw)
    G = Hq // Hkv
    score_of = oracle.score if reduce == "max" else oracle.score_sum
    for b, (n, k) in enumerate(zip(lens, ks)):
        for g in range(Hkv):
            s = score_of(qc_np[b, g * G:(g + 1) * G], kc_np[b, g, :n])
            if n_sink == 0 and n_local == 0:
                exp = oracle.topk(s, k)
                assert cnt[b, g] == len(exp) == min(k, n)
                others = s
            else:
                exp = oracle.topk_windows(s, k, n_sink, n_local)
                forced = np.zeros(n, bool)
                forced[:n_sink] = True
                forced[max(n - n_local, 0):] = True
                assert cnt[b, g] == len(exp) == forced.sum() + min(k, n - forced.sum())
                others = s[~forced]
            assert np.array_equal(idx[b, g, :len(exp)], exp), (b, g, n, k, n_sink, n_local)
            assert np.all(idx[b, g, len(exp):] == -1)
            assert np.array_equal(hist[b, g], np.bincount(others, minlength=hist.shape[2]))


@pytest.mark.parametrize("G", [1, 4])
def test_score_topk_sizes_ragged_tail_and_budgets(G):
    rng = np.random.default_rng(5 + G)
    Hkv, Hq = 2, 2 * G
    lens = [0, 1, 5, 1023, 2047, 2048, 2049, 5000, 70001]
    n_cap = 70004
    kc = rng.integers(0, 2 ** 32, size=(len(lens), Hkv, n_cap), dtype=np.uint64).astype(np.uint32)
    qc = rng.integers(0, 2 ** 32, size=(len(lens), Hq), dtype=np.uint64).astype(np.uint32)
    for ks in ([n // 16 for n in lens], [n for n in lens], [n + 5 for n in lens], [1] * len(lens), [0] * len(lens),
               [min(n, 777) for n in lens]):
        _check_score_topk(qc, kc, lens, ks, Hq, Hkv)


@pytest.mark.parametrize("lens,n_cap", [([140001, 131073, 9], 140004), ([600001, 524289, 9], 600004)])
def test_score_topk_long_sequences(lens, n_cap):
    """Sequences longer than 131072 tokens take the chunked scan + select kernels; shorter ones in the same
    batch ride along."""
    rng = np.random.default_rng(77)
    Hkv, Hq = 1, 4
    kc = rng.integers(0, 2 ** 32, size=(len(lens), Hkv, n_cap), dtype=np.uint64).astype(np.uint32)
    qc = rng.integers(0, 2 ** 32, size=(len(lens), Hq), dtype=np.uint64).astype(np.uint32)
    for ks in ([n // 32 for n in lens], [3, lens[1], 20]):
        _check_score_topk(qc, kc, lens, ks, Hq, Hkv)


@pytest.mark.parametrize("B,Hkv,G,n_hi", [(16, 8, 4, 2100), (30, 8, 2, 9000), (40, 4, 4, 2100), (14, 8, 1, 30000)])
def test_score_topk_grids_that_are_launched_with_a_cap_on_ctas_per_sm(B, Hkv, G, n_hi):
    """Batches whose cluster grid needs fewer than six CTAs per SM are launched with padded shared memory (at most
    ceil(CTAs / SMs) CTAs per SM): clusters of 4, 2, 4 and 8 here, ragged lengths, same lists as the oracle."""
    rng = np.random.default_rng(500 + B)
    Hq = Hkv * G
    lens = [int(v) for v in rng.integers(1, n_hi, size=B)]
    lens[0], lens[-1] = n_hi, 0
    n_cap = (n_hi + 3) // 4 * 4
    kc = rng.integers(0, 2 ** 32, size=(B, Hkv, n_cap), dtype=np.uint64).astype(np.uint32)
    qc = rng.integers(0, 2 ** 32, size=(B, Hq), dtype=np.uint64).astype(np.uint32)
    for ks in ([n // 16 for n in lens], [min(n, 300) for n in lens]):
        _check_score_topk(qc, kc, lens, ks, Hq, Hkv)
    _check_score_topk(qc, kc, lens, [n // 32 for n in lens], Hq, Hkv, n_sink=7, n_local=33)


@pytest.mark.parametrize("n_sink,n_local", [(128, 128), (1, 0), (0, 3), (5000, 7), (300, 70000)])
def test_score_topk_with_always_kept_windows(n_sink, n_local):
    """First n_sink and most recent n_local tokens always selected, the budget on top (Section 5, baselines):
    sequences shorter than a window, windows that overlap, the cluster kernel at every cluster size and the
    two-kernel path."""
    rng = np.random.default_rng(21 + n_sink)
    Hkv, Hq = 2, 8
    lens = [0, 1, 5, 100, 255, 256, 257, 2049, 5000, 70001, 140001]
    n_cap = 140004
    kc = rng.integers(0, 2 ** 32, size=(len(lens), Hkv, n_cap), dtype=np.uint64).astype(np.uint32)
    qc = rng.integers(0, 2 ** 32, size=(len(lens), Hq), dtype=np.uint64).astype(np.uint32)
    for ks in ([n // 16 for n in lens], [0] * len(lens), [n for n in lens]):
        _check_score_topk(qc, kc, lens, ks, Hq, Hkv, n_sink=n_sink, n_local=n_local)
    short = [n for n in lens if n <= 5000]          # shorter batch: the cluster kernel with clusters of 8 and 4
    _check_score_topk(qc[:len(short)], kc[:len(short), :, :5000].copy(), short, [n // 8 for n in short], Hq, Hkv,
                      n_sink=n_sink, n_local=n_local)


def test_score_topk_windows_with_heavy_ties_and_small_k_max():
    rng = np.random.default_rng(12)
    Hq, Hkv, n = 8, 2, 9000
    pool = rng.integers(0, 2 ** 32, size=4, dtype=np.uint64).astype(np.uint32)
    kc = pool[rng.integers(0, 4, size=(2, Hkv, n))]
    qc = rng.integers(0, 2 ** 32, size=(2, Hq), dtype=np.uint64).astype(np.uint32)
    for k in (1, 100, 4500):
        _check_score_topk(qc, kc, [n, n - 13], [k, k], Hq, Hkv, k_uniform=k, n_sink=128, n_local=128)
    # windows that do not fit the index rows are refused on the host
    shape = ha.make_shape(2, Hq, Hkv, 1.0, n_sink=128, n_local=128)
    ws = ha.alloc_workspace(shape, n, 256)
    t = lambda *s_: torch.zeros(*s_, dtype=torch.int32, device=DEV)
    with pytest.raises(RuntimeError):
        ha.ha_score_topk(shape, t(2, Hq), t(2, Hkv, n), t(2), None, 10, n, 200, t(2, Hkv, 200), t(2, Hkv), ws)


@pytest.mark.parametrize("seed", range(12))
def test_score_topk_random_shapes_budgets_and_windows(seed):
    """Seeded sweep: batch, heads, group size, ragged lengths, budgets (0 .. beyond n) and window sizes drawn at
    random; few distinct signatures in some cases (long tie blocks).  Index sets, counts and histograms exact."""
    rng = np.random.default_rng(9000 + seed)
    B = int(rng.integers(1, 7))
    Hkv = int(rng.choice([1, 2, 4]))
    G = int(rng.choice([1, 2, 4, 8]))
    lens = [int(v) for v in rng.integers(0, int(rng.choice([40, 3000, 20000])), size=B)]
    n_cap = (max(max(lens), 4) + 3) // 4 * 4
    if seed % 3 == 0:
        pool = rng.integers(0, 2 ** 32, size=5, dtype=np.uint64).astype(np.uint32)
        kc = pool[rng.integers(0, 5, size=(B, Hkv, n_cap))]
    else:
        kc = rng.integers(0, 2 ** 32, size=(B, Hkv, n_cap), dtype=np.uint64).astype(np.uint32)
    qc = rng.integers(0, 2 ** 32, size=(B, Hkv * G), dtype=np.uint64).astype(np.uint32)
    ks = [int(rng.integers(0, n + 10)) for n in lens]
    n_sink, n_local = (0, 0) if seed % 2 == 0 else (int(rng.integers(0, 200)), int(rng.integers(0, 200)))
    _check_score_topk(qc, kc, lens, ks, Hkv * G, Hkv, n_sink=n_sink, n_local=n_local)


def test_score_topk_heavy_ties():
    rng = np.random.default_rng(11)
    Hq, Hkv, n = 8, 2, 9000
    # few distinct codes -> huge tie blocks; all-equal codes -> lowest indices win
    pool = rng.integers(0, 2 ** 32, size=6, dtype=np.uint64).astype(np.uint32)
    kc = pool[rng.integers(0, 6, size=(3, Hkv, n))]
    kc[2] = 0xABCDEF01
    qc = rng.integers(0, 2 ** 32, size=(3, Hq), dtype=np.uint64).astype(np.uint32)
    qc[1, :4] = pool[0]                                # exact matches: score 32
    for k in (1, 100, 1500, 4500, 8999):
        _check_score_topk(qc, kc, [n, n - 13, n], [k, k, k], Hq, Hkv, k_uniform=k)


def test_score_topk_biased_bits_like_random_init_mappings():
    # narrow score distribution (many tokens on the threshold level), as random-init ReLU nets give
    rng = np.random.default_rng(12)
    Hq, Hkv, n = 32, 8, 32768
    p1 = rng.uniform(0.02, 0.98, size=32)
    bits = rng.random((1, Hkv, n, 32)) < p1
    kc = (bits * (1 << np.arange(32, dtype=np.uint64))).sum(-1).astype(np.uint32)
    qbits = rng.random((1, Hq, 32)) < p1
    qc = (qbits * (1 << np.arange(32, dtype=np.uint64))).sum(-1).astype(np.uint32)
    _check_score_topk(qc, kc, [n], [1024], Hq, Hkv)


# ---- the other group reduction: per-head scores added up (ha_score_topk_sum), 32 G + 1 levels

@pytest.mark.parametrize("G", [1, 2, 4, 8])
def test_score_topk_sum_sizes_ragged_tail_and_budgets(G):
    rng = np.random.default_rng(105 + G)
    Hkv, Hq = 2, 2 * G
    lens = [0, 1, 5, 31, 32, 33, 1023, 2047, 4096 * 8, 4096 * 8 + 1, 5000, 70001]   # 32768: one full tile per CTA
    n_cap = 70004
    kc = rng.integers(0, 2 ** 32, size=(len(lens), Hkv, n_cap), dtype=np.uint64).astype(np.uint32)
    qc = rng.integers(0, 2 ** 32, size=(len(lens), Hq), dtype=np.uint64).astype(np.uint32)
    for ks in ([n // 16 for n in lens], [n for n in lens], [n + 5 for n in lens], [1] * len(lens), [0] * len(lens),
               [min(n, 777) for n in lens]):
        _check_score_topk(qc, kc, lens, ks, Hq, Hkv, reduce="sum")


def test_score_topk_sum_equals_the_maximum_variant_for_single_head_groups():
    rng = np.random.default_rng(31)
    lens, n_cap = [9000, 1, 33000], 33000
    kc = rng.integers(0, 2 ** 32, size=(3, 4, n_cap), dtype=np.uint64).astype(np.uint32)
    qc = rng.integers(0, 2 ** 32, size=(3, 4), dtype=np.uint64).astype(np.uint32)
    ks = [500, 1, 2000]
    a = _run_score_topk(qc, kc, lens, ks, 4, 4, reduce="max")
    b = _run_score_topk(qc, kc, lens, ks, 4, 4, reduce="sum")
    for x, y in zip(a, b):
        assert np.array_equal(x, y)


def test_score_topk_sum_long_sequence_and_windows():
    rng = np.random.default_rng(78)
    Hkv, Hq = 1, 4
    lens, n_cap = [600001, 131073, 9], 600004
    kc = rng.integers(0, 2 ** 32, size=(len(lens), Hkv, n_cap), dtype=np.uint64).astype(np.uint32)
    qc = rng.integers(0, 2 ** 32, size=(len(lens), Hq), dtype=np.uint64).astype(np.uint32)
    _check_score_topk(qc, kc, lens, [n // 32 for n in lens], Hq, Hkv, reduce="sum")
    _check_score_topk(qc, kc, lens, [n // 32 for n in lens], Hq, Hkv, n_sink=128, n_local=128, reduce="sum")
    _check_score_topk(qc, kc, lens, [3, lens[1], 20], Hq, Hkv, n_sink=5000, n_local=70000, reduce="sum")


@pytest.mark.parametrize("B,Hkv", [(9, 2), (12, 2), (40, 2), (100, 2), (300, 2), (150, 4)])
def test_score_topk_sum_every_cluster_size(B, Hkv):
    """The cluster size follows the number of units: 16 CTAs up to 18 units, then 8, 4 (from 74), 2 (from 148) and
    single CTAs (from 592), whose slices span several tiles here."""
    rng = np.random.default_rng(600 + B)
    G = 4
    lens = [int(v) for v in rng.integers(0, 7000, size=B)]
    lens[0], lens[-1] = 6999, 0
    n_cap = 7000
    kc = rng.integers(0, 2 ** 32, size=(B, Hkv, n_cap), dtype=np.uint64).astype(np.uint32)
    kc[1] = kc[1] & np.uint32(0x3)                      # four distinct signatures: long tie blocks across tiles
    qc = rng.integers(0, 2 ** 32, size=(B, Hkv * G), dtype=np.uint64).astype(np.uint32)
    ks = [int(rng.integers(0, n + 3)) for n in lens]
    _check_score_topk(qc, kc, lens, ks, Hkv * G, Hkv, reduce="sum")
    _check_score_topk(qc, kc, lens, [min(k, 500) for k in ks], Hkv * G, Hkv, n_sink=100, n_local=2100, reduce="sum")


def test_score_topk_sum_slices_beyond_the_score_byte_cache():
    """Slices of up to 16384 tokens (65536 in the few-CTA variant) keep one score byte per token in shared memory
    between the passes; longer ones are scored twice.  Both kinds in one batch, and one sequence of over a million
    tokens for the few-CTA variant."""
    rng = np.random.default_rng(4242)
    B, Hkv, G = 80, 2, 4                                # 160 units: clusters of 2
    lens = [int(v) for v in rng.integers(0, 3000, size=B)]
    lens[3], lens[40], lens[79] = 40000, 30000, 32769   # slices of 20000 (scored twice), 15000 and 16388 tokens
    n_cap = 40000
    kc = rng.integers(0, 2 ** 32, size=(B, Hkv, n_cap), dtype=np.uint64).astype(np.uint32)
    kc[3, 1] &= np.uint32(0x7)                          # tie blocks
    qc = rng.integers(0, 2 ** 32, size=(B, Hkv * G), dtype=np.uint64).astype(np.uint32)
    ks = [n // 16 for n in lens]
    _check_score_topk(qc, kc, lens, ks, Hkv * G, Hkv, reduce="sum")
    _check_score_topk(qc, kc, lens, ks, Hkv * G, Hkv, n_sink=128, n_local=128, reduce="sum")
    n = 1100003                                         # 16 CTAs, slices of 68752 tokens
    kc1 = rng.integers(0, 2 ** 32, size=(1, 1, n + 1), dtype=np.uint64).astype(np.uint32)
    qc1 = rng.integers(0, 2 ** 32, size=(1, G), dtype=np.uint64).astype(np.uint32)
    _check_score_topk(qc1, kc1, [n], [n // 64], G, 1, reduce="sum")


def test_score_topk_sum_and_per_head_replay_from_a_cuda_graph():
    """Both stand-alone selections are plain launches on the caller's stream: captured once (after a first call that
    sets the kernel attributes), replayed on new signatures."""
    rng = np.random.default_rng(77)
    B, Hq, Hkv, n, k = 2, 8, 2, 9000, 300
    shape = ha.make_shape(B, Hq, Hkv, 1.0)
    kc = torch.zeros(B, Hkv, n, dtype=torch.int32, device=DEV)
    qc = torch.zeros(B, Hq, dtype=torch.int32, device=DEV)
    sl = torch.tensor([n, n - 77], dtype=torch.int32, device=DEV)
    idx = torch.zeros(B, Hkv, k, dtype=torch.int32, device=DEV)
    cnt = torch.zeros(B, Hkv, dtype=torch.int32, device=DEV)
    idx_h = torch.zeros(B, Hq, k, dtype=torch.int32, device=DEV)
    cnt_h = torch.zeros(B, Hq, dtype=torch.int32, device=DEV)
    st = torch.cuda.Stream()
    with torch.cuda.stream(st):
        ha.ha_score_topk_sum(shape, qc, kc, sl, None, k, k, idx, cnt, stream=st)
        ha.ha_score_topk_per_head(shape, qc, kc, sl, None, k, k, idx_h, cnt_h, stream=st)
        st.synchronize()
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph, stream=st):
            ha.ha_score_topk_sum(shape, qc, kc, sl, None, k, k, idx, cnt, stream=st)
            ha.ha_score_topk_per_head(shape, qc, kc, sl, None, k, k, idx_h, cnt_h, stream=st)
    for rep in range(2):
        kc_np = rng.integers(0, 2 ** 32, size=(B, Hkv, n), dtype=np.uint64).astype(np.uint32)
        qc_np = rng.integers(0, 2 ** 32, size=(B, Hq), dtype=np.uint64).astype(np.uint32)
        kc.copy_(torch.from_numpy(kc_np.view(np.int32)))
        qc.copy_(torch.from_numpy(qc_np.view(np.int32)))
        torch.cuda.synchronize()
        graph.replay()
        torch.cuda.synchronize()
        for b, nb in enumerate([n, n - 77]):
            for g in range(Hkv):
                exp = oracle.topk(oracle.score_sum(qc_np[b, 4 * g:4 * g + 4], kc_np[b, g, :nb]), k)
                assert np.array_equal(idx[b, g].cpu().numpy(), exp) and int(cnt[b, g]) == k
            for h in range(Hq):
                exp = oracle.topk(oracle.score(qc_np[b, h:h + 1], kc_np[b, h // 4, :nb]), k)
                assert np.array_equal(idx_h[b, h].cpu().numpy(), exp) and int(cnt_h[b, h]) == k


@pytest.mark.parametrize("seed", range(12))
def test_score_topk_sum_random_shapes_budgets_windows_and_ties(seed):
    rng = np.random.default_rng(9500 + seed)
    B = int(rng.integers(1, 7))
    Hkv = int(rng.choice([1, 2, 4]))
    G = int(rng.choice([1, 2, 4, 8]))
    lens = [int(v) for v in rng.integers(0, int(rng.choice([40, 3000, 40000])), size=B)]
    n_cap = (max(max(lens), 4) + 3) // 4 * 4
    if seed % 3 == 0:   # few distinct signatures: long tie blocks
        pool = rng.integers(0, 2 ** 32, size=5, dtype=np.uint64).astype(np.uint32)
        kc = pool[rng.integers(0, 5, size=(B, Hkv, n_cap))]
    else:
        kc = rng.integers(0, 2 ** 32, size=(B, Hkv, n_cap), dtype=np.uint64).astype(np.uint32)
    qc = rng.integers(0, 2 ** 32, size=(B, Hkv * G), dtype=np.uint64).astype(np.uint32)
    if seed % 4 == 1:
        qc[:, :] = kc[:, :, 0].repeat(G, axis=1)[:, :Hkv * G]   # exact matches: the top level 32 G is reached
    ks = [int(rng.integers(0, n + 10)) for n in lens]
    n_sink, n_local = (0, 0) if seed % 2 == 0 else (int(rng.integers(0, 200)), int(rng.integers(0, 200)))
    _check_score_topk(qc, kc, lens, ks, Hkv * G, Hkv, n_sink=n_sink, n_local=n_local, reduce="sum")


# ---------------------------------------------------------------------------- GATHER-ATT / dense

def _attn_inputs(B, Hq, Hkv, n_cap, seed, scale=1.0):
    g = torch.Generator(DEV).manual_seed(seed)
    q = torch.randn(B, Hq, 128, device=DEV, generator=g).to(torch.bfloat16)
    K = (scale * torch.randn(B, Hkv, n_cap, 128, device=DEV, generator=g)).to(torch.bfloat16)
    V = torch.randn(B, Hkv, n_cap, 128, device=DEV, generator=g).to(torch.bfloat16)
    return q, K, V


def _check_gather(q, K, V, lens, idx_np, cnt_np, sm_scale, expect_flag=0):
    B, Hq, _ = q.shape
    Hkv = K.shape[1]
    G = Hq // Hkv
    k_max = idx_np.shape[2]
    shape = ha.make_shape(B, Hq, Hkv, sm_scale)
    ws = ha.alloc_workspace(shape, K.shape[2], k_max)
    out = torch.full((B, Hq, 128), 7.0, dtype=torch.bfloat16, device=DEV)
    lse = torch.full((B, Hq), 7.0, dtype=torch.float32, device=DEV)
    ha.ha_gather_attn(shape, q, K, V, torch.tensor(lens, dtype=torch.int32, device=DEV),
                      torch.from_numpy(idx_np).to(DEV), torch.from_numpy(cnt_np).to(DEV), k_max, out, ws, lse=lse)
    assert ha.ha_read_device_status(ws) == expect_flag
    qu, Ku, Vu, ou = u16(q), u16(K), u16(V), u16(out)
    lse_np = lse.cpu().numpy()
    worst = 0.0
    for b in range(B):
        for h in range(Hq):
            g = h // G
            eo, el, _ = oracle.gather_attn(qu[b, h], Ku[b, g], Vu[b, g], idx_np[b, g, :cnt_np[b, g]],
                                           sm_scale=sm_scale, n_valid=lens[b])
            worst = max(worst, assert_out_close(ou[b, h], eo))
            if math.isinf(el):
                assert lse_np[b, h] == -math.inf and not ou[b, h].any()
            else:
                assert abs(lse_np[b, h] - el) < 1e-3 * max(1.0, abs(el))
    assert worst <= OUT_TOL
    return worst


@pytest.mark.parametrize("k_max", [700, 2100])   # index rows of up to 2048 entries: one cluster per unit; wider: split-K kernel
@pytest.mark.parametrize("G", [1, 4, 8])
def test_gather_attn_random_lists(G, k_max):
    Hkv, Hq, n_cap = 2, 2 * G, 3000
    B = 3
    lens = [3000, 1777, 64]
    q, K, V = _attn_inputs(B, Hq, Hkv, n_cap, 40 + G)
    rng = np.random.default_rng(41)
    idx = np.full((B, Hkv, k_max), -1, np.int32)
    cnt = np.zeros((B, Hkv), np.int32)
    for b in range(B):
        for g in range(Hkv):
            c = [700, 333, 17][b] if g == 0 else [1, 64, 0][b]
            c = min(c, lens[b])
            cnt[b, g] = c
            idx[b, g, :c] = np.sort(rng.choice(lens[b], size=c, replace=False))
    _check_gather(q, K, V, lens, idx, cnt, 1.0 / math.sqrt(128))


@pytest.mark.parametrize("B", [20, 50])
def test_gather_attn_with_smaller_clusters(B):
    """34 to 71 units with short lists: the stand-alone gather runs one cluster of 4 CTAs per unit, up to 148 units one
    of 2 (several blocks per warp, one after the other); random lists with padding inside, duplicates, and one index
    outside its sequence."""
    Hkv, G, n_cap, k_max = 2, 4, 2500, 900
    Hq = Hkv * G
    rng = np.random.default_rng(77)
    lens = [int(v) for v in rng.integers(1, n_cap + 1, size=B)]
    q, K, V = _attn_inputs(B, Hq, Hkv, n_cap, 78)
    idx = np.full((B, Hkv, k_max), -1, np.int32)
    cnt = np.zeros((B, Hkv), np.int32)
    for b in range(B):
        for g in range(Hkv):
            c = int(rng.integers(0, k_max + 1))
            cnt[b, g] = c
            idx[b, g, :c] = rng.integers(0, lens[b], size=c)
            idx[b, g, :c][rng.random(c) < 0.05] = -1
    before = ha.ha_kernel_launches()
    _check_gather(q, K, V, lens, idx, cnt, 1.0 / math.sqrt(128))
    assert ha.ha_kernel_launches() - before == 1
    idx[7, 1, 0] = lens[7]                       # one entry past the end of its sequence: skipped and flagged
    cnt[7, 1] = max(cnt[7, 1], 1)
    _check_gather(q, K, V, lens, idx, cnt, 1.0 / math.sqrt(128), expect_flag=ha.HA_DEV_BAD_INDEX)


@pytest.mark.parametrize("ragged", [False, True])
def test_gather_attn_equal_lists_on_most_of_the_ctas_are_taken_as_whole_units(ragged):
    """240 units (more than the cluster kernel takes, at least three quarters of the split-K kernel's CTAs): lists of
    equal length are attended to one whole unit per CTA, a batch with one shorter list by the balanced split; both
    against the oracle."""
    B, Hkv, G, n_cap, k_max = 60, 4, 2, 700, 200
    Hq = Hkv * G
    rng = np.random.default_rng(91)
    lens = [n_cap] * B
    q, K, V = _attn_inputs(B, Hq, Hkv, n_cap, 92)
    idx = np.full((B, Hkv, k_max), -1, np.int32)
    cnt = np.full((B, Hkv), k_max, np.int32)
    for b in range(B):
        for g in range(Hkv):
            idx[b, g] = np.sort(rng.choice(n_cap, size=k_max, replace=False))
    if ragged:
        cnt[17, 2] = 37
        idx[17, 2, 37:] = -1
    before = ha.ha_kernel_launches()
    _check_gather(q, K, V, lens, idx, cnt, 1.0 / math.sqrt(128))
    assert ha.ha_kernel_launches() - before == 1


@pytest.mark.parametrize("width", [64, 2100])   # both stand-alone gather kernels (see test_gather_attn_random_lists)
def test_gather_attn_padding_invalid_and_unsorted_indices(width):
    Hq, Hkv, n_cap = 8, 2, 500
    q, K, V = _attn_inputs(1, Hq, Hkv, n_cap, 50, scale=2.0)
    idx = np.full((1, Hkv, width), -1, np.int32)
    idx[0, 0, :10] = [499, 3, 3, -1, 250, 7, -1, 0, 42, 499]       # padding inside, duplicates, unsorted
    idx[0, 1, :6] = [5, 400, 450, 10, 399, 1]                       # 400, 450 are beyond seq_len = 400
    cnt = np.array([[10, 6]], np.int32)
    _check_gather(q, K, V, [400 + 100], idx[:, :, :], np.array([[10, 0]], np.int32), 0.2)
    _check_gather(q, K, V, [400], np.where(idx == 499, 399, idx), cnt, 0.2, expect_flag=ha.HA_DEV_BAD_INDEX)


def test_single_index_returns_value_row_exactly_and_k_equals_n_is_dense():
    Hq, Hkv, n = 8, 2, 1234
    q, K, V = _attn_inputs(1, Hq, Hkv, n, 60)
    shape = ha.make_shape(1, Hq, Hkv, 1.0 / math.sqrt(128))
    ws = ha.alloc_workspace(shape, n, n)
    sl = torch.tensor([n], dtype=torch.int32, device=DEV)
    one = torch.tensor([[[777], [5]]], dtype=torch.int32, device=DEV)
    out = torch.zeros(1, Hq, 128, dtype=torch.bfloat16, device=DEV)
    ha.ha_gather_attn(shape, q, K, V, sl, one, torch.ones(1, Hkv, dtype=torch.int32, device=DEV), 1, out, ws)
    assert torch.equal(out[0, :4], V[0, 0, 777].expand(4, 128)) and torch.equal(out[0, 4:], V[0, 1, 5].expand(4, 128))
    # k = n through the gather kernel equals the dense kernel equals the oracle
    full = torch.arange(n, dtype=torch.int32, device=DEV).expand(1, Hkv, n).contiguous()
    cnt = torch.full((1, Hkv), n, dtype=torch.int32, device=DEV)
    o_sparse = torch.zeros_like(out)
    o_dense = torch.zeros_like(out)
    l_s = torch.zeros(1, Hq, device=DEV)
    l_d = torch.zeros(1, Hq, device=DEV)
    ha.ha_gather_attn(shape, q, K, V, sl, full, cnt, n, o_sparse, ws, lse=l_s)
    ha.ha_dense_decode(shape, q, K, V, sl, n, o_dense, ws, lse=l_d)
    assert_out_close(u16(o_sparse), u16(o_dense))
    assert float((l_s - l_d).abs().max()) < 1e-4
    qu, Ku, Vu = u16(q), u16(K), u16(V)
    for h in range(Hq):
        eo, el, _ = oracle.dense(qu[0, h], Ku[0, h // 4], Vu[0, h // 4])
        assert_out_close(u16(o_dense)[0, h], eo)
        assert abs(float(l_d[0, h]) - el) < 1e-3


@pytest.mark.parametrize("lens,cap", [([1], None), ([33, 4097], None), ([20000, 1, 0], None),
                                      ([100, 1], 30000)])   # a cache far longer than its sequences: fewer blocks than CTAs
def test_dense_decode_matches_oracle(lens, cap):
    Hq, Hkv = 8, 2
    B, n_cap = len(lens), cap or max(max(lens), 1)
    q, K, V = _attn_inputs(B, Hq, Hkv, n_cap, 70 + len(lens))
    shape = ha.make_shape(B, Hq, Hkv, 1.0 / math.sqrt(128))
    ws = ha.alloc_workspace(shape, n_cap, n_cap)
    out = torch.full((B, Hq, 128), 3.0, dtype=torch.bfloat16, device=DEV)
    lse = torch.zeros(B, Hq, device=DEV)
    ha.ha_dense_decode(shape, q, K, V, torch.tensor(lens, dtype=torch.int32, device=DEV), n_cap, out, ws, lse=lse)
    qu, Ku, Vu, ou = u16(q), u16(K), u16(V), u16(out)
    for b in range(B):
        for h in range(Hq):
            eo, el, _ = oracle.dense(qu[b, h], Ku[b, h // 4], Vu[b, h // 4], n=lens[b])
            assert_out_close(ou[b, h], eo)
            if lens[b] == 0:
                assert float(lse[b, h]) == -math.inf
            else:
                assert abs(float(lse[b, h]) - el) < 1e-3


@pytest.mark.parametrize("page_size", [1, 16, 64])
def test_gather_attn_over_a_paged_cache(page_size):
    """K/V rows live in pages scattered over a pool and are found through a block table (page sizes 1 and 16
    of the vLLM integration, and a larger one); results equal the oracle over the un-paged rows."""
    rng = np.random.default_rng(40 + page_size)
    B, Hq, Hkv = 3, 8, 2
    lens = [300, 2049, 17]
    n_cap = max(lens)
    g = torch.Generator(DEV).manual_seed(page_size)
    q = torch.randn(B, Hq, 128, device=DEV, generator=g).to(torch.bfloat16)
    pages_per_seq = (n_cap + page_size - 1) // page_size
    n_pages = B * pages_per_seq + 5
    K_pool = torch.randn(n_pages, Hkv, page_size, 128, device=DEV, generator=g).to(torch.bfloat16)
    V_pool = torch.randn(n_pages, Hkv, page_size, 128, device=DEV, generator=g).to(torch.bfloat16)
    table = torch.from_numpy(rng.permutation(n_pages)[:B * pages_per_seq].reshape(B, pages_per_seq).astype(np.int32)).to(DEV)
    k_max = 256
    idx_np = np.full((B, Hkv, k_max), -1, np.int32)
    cnt_np = np.zeros((B, Hkv), np.int32)
    for b, n in enumerate(lens):
        for h in range(Hkv):
            c = min(n, int(rng.integers(1, k_max + 1)))
            idx_np[b, h, :c] = np.sort(rng.choice(n, size=c, replace=False))
            cnt_np[b, h] = c
    shape = ha.make_shape(B, Hq, Hkv, 1.0 / np.sqrt(128))
    ws = ha.alloc_workspace(shape, n_cap, k_max)
    out = torch.zeros(B, Hq, 128, dtype=torch.bfloat16, device=DEV)
    lse = torch.zeros(B, Hq, device=DEV)
    ha.ha_gather_attn_paged(shape, q, K_pool, V_pool, table, page_size, torch.tensor(lens, dtype=torch.int32, device=DEV),
                            torch.from_numpy(idx_np).to(DEV), torch.from_numpy(cnt_np).to(DEV), k_max, out, ws, lse=lse)
    torch.cuda.synchronize()
    assert ha.ha_read_device_status(ws) == 0
    G = Hq // Hkv
    qu, Kp, Vp, tb = u16(q), u16(K_pool), u16(V_pool), table.cpu().numpy()
    for b, n in enumerate(lens):
        for h in range(Hkv):
            Kr, Vr = oracle.unpage_rows(Kp, tb[b], page_size, h, n), oracle.unpage_rows(Vp, tb[b], page_size, h, n)
            for j in range(G):
                eo, el, _ = oracle.gather_attn(qu[b, h * G + j], Kr, Vr, idx_np[b, h, :cnt_np[b, h]], sm_scale=1.0 / np.sqrt(128))
                assert_out_close(u16(out[b, h * G + j]), eo)
                assert abs(float(lse[b, h * G + j]) - el) < 1e-3


# ---------------------------------------------------------------------------- whole step

def _run_step(w, host=False, pinned=True, n_sink=0, n_local=0, prepared=False, pipelined=False):
    cfg = w["cfg"]
    B, Hq, Hkv = cfg.batch, cfg.n_q_heads, cfg.n_kv_heads
    shape = ha.make_shape(B, Hq, Hkv, w["sm_scale"], n_sink=n_sink, n_local=n_local)
    if n_sink or n_local:
        w = dict(w, k_max=w["k_max"] + n_sink + n_local)             # the index rows hold the windows too
    ws = ha.alloc_workspace(shape, w["n_cap"], w["k_max"])
    mq, mk = ha.Mapping(w["map_q"]), ha.Mapping(w["map_k"])
    kc = torch.zeros(B, Hkv, (w["n_cap"] + 3) // 4 * 4, dtype=torch.int32, device=DEV)
    ha.ha_encode(mk, 1, w["K"], kc)                                  # signature cache of the prompt
    for b in range(B):
        if w["lens"][b] > 0:
            kc[b, :, w["lens"][b] - 1] = 0x7FFFFFFF                  # the step must rewrite the appended slot
    qc = torch.zeros(B, Hq, dtype=torch.int32, device=DEV)
    idx = torch.zeros(B, Hkv, w["k_max"], dtype=torch.int32, device=DEV)
    cnt = torch.zeros(B, Hkv, dtype=torch.int32, device=DEV)
    out = torch.zeros(B, Hq, 128, dtype=torch.bfloat16, device=DEV)
    lse = torch.zeros(B, Hq, device=DEV)
    if host:
        K2, V2 = w["K"].clone(), w["V"].clone()
        for b in range(B):
            if w["lens"][b] > 0:
                K2[b, :, w["lens"][b] - 1] = 0
                V2[b, :, w["lens"][b] - 1] = 0
        pin = (lambda t: t.pin_memory()) if pinned else (lambda t: t)     # pageable buffers take the staged-copy route
        hq, hk, hv = (pin(w[x].cpu()) for x in ("q", "k_new", "v_new"))
        ho = pin(torch.zeros(B, Hq, 128, dtype=torch.bfloat16))
        if prepared:
            step = ha.SparseDecodeHostStep(shape, mq, mk, hq, hk, hv, K2, V2, kc, w["seq_lens"], w["k_per_seq"], 0,
                                           w["n_cap"], w["k_max"], idx, cnt, ho, ws)
            step()
            ho.zero_()
            step()                                                   # the second call sees the same inputs
        else:
            ha.ha_sparse_decode_host(shape, mq, mk, hq, hk, hv, K2, V2, kc, w["seq_lens"], w["k_per_seq"], 0, w["n_cap"],
                                     w["k_max"], idx, cnt, ho, ws)
        assert torch.equal(K2, w["K"]) and torch.equal(V2, w["V"])   # the new rows were appended in place
        out = ho.to(DEV)
        lse = None
    else:
        step = ha.ha_sparse_decode_pipelined if pipelined else ha.ha_sparse_decode
        step(shape, mq, mk, w["q"], w["k_new"], w["K"], w["V"], kc, w["seq_lens"], w["k_per_seq"], 0,
             w["n_cap"], w["k_max"], qc, idx, cnt, out, ws, lse=lse)
    torch.cuda.synchronize()
    assert ha.ha_read_device_status(ws) == 0
    return dict(kc=kc, qc=qc, idx=idx, cnt=cnt, out=out, lse=lse)


@pytest.mark.parametrize("cfg", [
    wl.Config("tiny-ragged", 50, 3, [300, 2049, 1], None, 0.02, n_q_heads=8, n_kv_heads=2, sparsity=8),
    wl.Config("tiny-g1", 51, 2, [700, 64], 32, 0.05, n_q_heads=2, n_kv_heads=2, sparsity=8),
    wl.CONFIGS["c1"],
])
def test_sparse_decode_step_matches_oracle(cfg):
    w = wl.make_workload(cfg, DEV)
    r = _run_step(w)
    Kc = oracle_key_codes(w["K"], w["map_k"], w["lens"])
    B, Hkv = cfg.batch, cfg.n_kv_heads
    n_cap = w["n_cap"]
    assert np.array_equal(codes_np(r["kc"])[:, :, :n_cap] * (np.arange(n_cap)[None, None, :] < np.array(w["lens"])[:, None, None]),
                          Kc)
    ref = oracle.decode_step(u16(w["q"]), u16(w["k_new"]), u16(w["K"]), u16(w["V"]), Kc.copy(),
                             wl.mapping_numpy(w["map_q"]), wl.mapping_numpy(w["map_k"]), w["lens"], w["ks"],
                             sm_scale=w["sm_scale"], n_threads=4)
    assert np.array_equal(codes_np(r["qc"]), ref["qcodes"])
    assert np.array_equal(r["cnt"].cpu().numpy(), ref["count"])
    assert np.array_equal(r["idx"].cpu().numpy(), ref["idx"])
    assert_out_close(u16(r["out"]), ref["out"])
    got_lse = r["lse"].cpu().numpy().astype(np.float64)
    finite = np.isfinite(ref["lse"])
    assert np.array_equal(np.isneginf(got_lse), ~finite)            # empty selections: lse = -inf on both sides
    assert np.max(np.abs(got_lse[finite] - ref["lse"][finite]), initial=0.0) < 1e-3
    # the host-buffer entry point gives the same result
    for pinned in (True, False):
        rh = _run_step(w, host=True, pinned=pinned)
        assert torch.equal(rh["idx"], r["idx"]) and torch.equal(rh["out"], r["out"])
    # ... and so does the same call with its arguments marshalled once (SparseDecodeHostStep), run twice
    rp = _run_step(w, host=True, pinned=True, prepared=True)
    assert torch.equal(rp["idx"], r["idx"]) and torch.equal(rp["out"], r["out"])


@pytest.mark.parametrize("world", [2, 4])
@pytest.mark.parametrize("B", [2, 20])          # one fused launch per shard / the three-kernel path
def test_head_parallel_shards_reproduce_the_whole_step(B, world):
    """The (sequence, KV head) units are independent: the step run on each rank's KV heads alone (strided K/V views,
    sliced mappings) gives the slices of the unsharded result (signatures, lists and counts bit for bit, outputs to
    rounding); no exchange exists on the data path."""
    lens = ([700, 2049] + [500 + 61 * i for i in range(B)])[:B]
    cfg = wl.Config("head-shards", 62, B, lens, None, 0.02, n_q_heads=16, n_kv_heads=4, sparsity=8)
    w = wl.make_workload(cfg, DEV)
    whole = _run_step(w)
    hk, G = 4 // world, 4
    for rank in range(world):
        r = _run_step(wl.shard_heads(w, rank, world))
        kv, qh = slice(rank * hk, (rank + 1) * hk), slice(rank * hk * G, (rank + 1) * hk * G)
        assert torch.equal(r["idx"], whole["idx"][:, kv]) and torch.equal(r["cnt"], whole["cnt"][:, kv])
        assert torch.equal(r["qc"], whole["qc"][:, qh]) and torch.equal(r["kc"], whole["kc"][:, kv])
        # a shard may take another launch variant than the whole (fewer units): same index sets, while the fp32 sums
        # are taken in another order
        assert max_abs_diff_bf16(u16(r["out"]), u16(whole["out"][:, qh].contiguous())) <= OUT_AIM
        assert float((r["lse"] - whole["lse"][:, qh]).abs().max()) < 1e-3


def test_step_from_entry_points_with_summed_group_scores():
    """ENCODE, the summed-score SCORE + TOPK and GATHER-ATT chained through their entry points against the same chain
    of oracle functions: the lists of ha_score_topk_sum feed ha_gather_attn unchanged."""
    cfg = wl.Config("sum-chain", 58, 3, [300, 5000, 1], None, 0.02, n_q_heads=8, n_kv_heads=2, sparsity=8)
    w = wl.make_workload(cfg, DEV)
    B, Hq, Hkv, G = cfg.batch, cfg.n_q_heads, cfg.n_kv_heads, 4
    shape = ha.make_shape(B, Hq, Hkv, w["sm_scale"])
    ws = ha.alloc_workspace(shape, w["n_cap"], w["k_max"])
    kc = torch.zeros(B, Hkv, (w["n_cap"] + 3) // 4 * 4, dtype=torch.int32, device=DEV)
    qc = torch.zeros(B, Hq, dtype=torch.int32, device=DEV)
    ha.ha_encode(ha.Mapping(w["map_k"]), 1, w["K"], kc)
    ha.ha_encode(ha.Mapping(w["map_q"]), G, w["q"], qc.unsqueeze(2))
    idx = torch.zeros(B, Hkv, w["k_max"], dtype=torch.int32, device=DEV)
    cnt = torch.zeros(B, Hkv, dtype=torch.int32, device=DEV)
    out = torch.zeros(B, Hq, 128, dtype=torch.bfloat16, device=DEV)
    ha.ha_score_topk_sum(shape, qc, kc, w["seq_lens"], w["k_per_seq"], 0, w["k_max"], idx, cnt)
    ha.ha_gather_attn(shape, w["q"], w["K"], w["V"], w["seq_lens"], idx, cnt, w["k_max"], out, ws)
    torch.cuda.synchronize()
    assert ha.ha_read_device_status(ws) == 0
    Kc = oracle_key_codes(w["K"], w["map_k"], w["lens"])
    Qc = oracle_query_codes(w["q"], w["map_q"], Hkv)
    assert np.array_equal(codes_np(qc), Qc)
    qu, Ku, Vu = u16(w["q"]), u16(w["K"]), u16(w["V"])
    differs = 0
    for b, (n, k) in enumerate(zip(w["lens"], w["ks"])):
        for g in range(Hkv):
            s = oracle.score_sum(Qc[b, g * G:(g + 1) * G], Kc[b, g, :n])
            exp = oracle.topk(s, k)
            differs += int(not np.array_equal(exp, oracle.topk(oracle.score(Qc[b, g * G:(g + 1) * G], Kc[b, g, :n]), k)))
            assert int(cnt[b, g]) == len(exp)
            assert np.array_equal(idx[b, g, :len(exp)].cpu().numpy(), exp)
            for j in range(G):
                eo, _, _ = oracle.gather_attn(qu[b, g * G + j], Ku[b, g], Vu[b, g], exp, sm_scale=w["sm_scale"])
                assert_out_close(u16(out[b, g * G + j]), eo)
    assert differs > 0   # the two reductions pick different tokens on these inputs: the test would notice a mix-up


@pytest.mark.parametrize("n_sink,n_local", [(0, 0), (16, 40)])
@pytest.mark.parametrize("B,Hq,Hkv", [(3, 8, 2), (2, 16, 2), (30, 8, 4), (5, 4, 4)])
def test_step_from_entry_points_with_one_list_per_query_head(B, Hq, Hkv, n_sink, n_local):
    """No reduction over the group: every query head scores the signatures of its KV head by Eq. 1, keeps its own
    top-k and attends through its own list (ha_score_topk_per_head + ha_gather_attn_per_head), against the oracle's
    single-head score, top-k and GATHER-ATT."""
    G = Hq // Hkv
    lens = ([300, 5000, 1] + [int(v) for v in np.random.default_rng(B).integers(0, 2500, size=B)])[:B]
    cfg = wl.Config("per-head", 59, B, lens, None, 0.02, n_q_heads=Hq, n_kv_heads=Hkv, sparsity=8)
    w = wl.make_workload(cfg, DEV)
    k_max = w["k_max"] + n_sink + n_local
    shape = ha.make_shape(B, Hq, Hkv, w["sm_scale"], n_sink=n_sink, n_local=n_local)
    ws = ha.alloc_workspace(ha.make_shape(B, Hq, Hq, w["sm_scale"]), w["n_cap"], k_max)   # one unit per query head
    kc = torch.zeros(B, Hkv, (w["n_cap"] + 3) // 4 * 4, dtype=torch.int32, device=DEV)
    qc = torch.zeros(B, Hq, dtype=torch.int32, device=DEV)
    ha.ha_encode(ha.Mapping(w["map_k"]), 1, w["K"], kc)
    ha.ha_encode(ha.Mapping(w["map_q"]), G, w["q"], qc.unsqueeze(2))
    idx = torch.full((B, Hq, k_max), -7, dtype=torch.int32, device=DEV)
    cnt = torch.full((B, Hq), -7, dtype=torch.int32, device=DEV)
    hist = torch.full((B, Hq, 33), -7, dtype=torch.int32, device=DEV)
    out = torch.zeros(B, Hq, 128, dtype=torch.bfloat16, device=DEV)
    lse = torch.zeros(B, Hq, device=DEV)
    ha.ha_score_topk_per_head(shape, qc, kc, w["seq_lens"], w["k_per_seq"], 0, k_max, idx, cnt, hist_out=hist)
    ha.ha_gather_attn_per_head(shape, w["q"], w["K"], w["V"], w["seq_lens"], idx, cnt, k_max, out, ws, lse=lse)
    torch.cuda.synchronize()
    assert ha.ha_read_device_status(ws) == 0
    Kc = oracle_key_codes(w["K"], w["map_k"], w["lens"])
    Qc = oracle_query_codes(w["q"], w["map_q"], Hkv)
    qu, Ku, Vu = u16(w["q"]), u16(w["K"]), u16(w["V"])
    idx_np, cnt_np, hist_np = idx.cpu().numpy(), cnt.cpu().numpy(), hist.cpu().numpy()
    lists_differ = 0
    for b, (n, k) in enumerate(zip(w["lens"], w["ks"])):
        for h in range(Hq):
            s = oracle.score(Qc[b, h:h + 1], Kc[b, h // G, :n])
            exp = oracle.topk_windows(s, k, n_sink, n_local) if (n_sink or n_local) else oracle.topk(s, k)
            forced = np.zeros(n, bool)
            forced[:n_sink] = True
            forced[max(n - n_local, 0):] = bool(n_local)
            assert cnt_np[b, h] == len(exp)
            assert np.array_equal(idx_np[b, h, :len(exp)], exp), (b, h)
            assert np.all(idx_np[b, h, len(exp):] == -1)
            assert np.array_equal(hist_np[b, h], np.bincount(s[~forced], minlength=33))
            lists_differ += int(h % G != 0 and not np.array_equal(exp, idx_np[b, h - 1, :cnt_np[b, h - 1]]))
            eo, el, _ = oracle.gather_attn(qu[b, h], Ku[b, h // G], Vu[b, h // G], exp, sm_scale=w["sm_scale"])
            assert_out_close(u16(out[b, h]), eo)
            if len(exp):
                assert abs(float(lse[b, h]) - el) < 1e-3
    assert G == 1 or lists_differ > 0   # heads of one group really select on their own


@pytest.mark.parametrize("cfg", [
    wl.Config("win-ragged", 55, 3, [300, 2049, 1], None, 0.02, n_q_heads=8, n_kv_heads=2, sparsity=8),     # one fused launch
    wl.Config("win-batch", 56, 24, [900 + 37 * i for i in range(24)], None, 0.02, n_q_heads=8, n_kv_heads=2,
              sparsity=8),                                                             # one fused launch, clusters of 4
    wl.Config("win-large-batch", 59, 90, [500 + 11 * i for i in range(90)], None, 0.02, n_q_heads=8, n_kv_heads=2,
              sparsity=8),                                                                                  # three kernels
    wl.CONFIGS["c1"],
])
@pytest.mark.parametrize("n_sink,n_local", [(128, 128), (4, 500)])
def test_sparse_decode_step_with_always_kept_windows(cfg, n_sink, n_local):
    w = wl.make_workload(cfg, DEV)
    r = _run_step(w, n_sink=n_sink, n_local=n_local)
    Kc = oracle_key_codes(w["K"], w["map_k"], w["lens"])
    ref = oracle.decode_step(u16(w["q"]), u16(w["k_new"]), u16(w["K"]), u16(w["V"]), Kc.copy(),
                             wl.mapping_numpy(w["map_q"]), wl.mapping_numpy(w["map_k"]), w["lens"], w["ks"],
                             sm_scale=w["sm_scale"], n_threads=4, n_sink=n_sink, n_local=n_local)
    assert np.array_equal(r["cnt"].cpu().numpy(), ref["count"])
    assert np.array_equal(r["idx"].cpu().numpy(), ref["idx"])
    for b, n in enumerate(w["lens"]):                                # the windows really are in every list
        for g in range(cfg.n_kv_heads):
            got = set(r["idx"][b, g, :int(r["cnt"][b, g])].tolist())
            assert set(range(min(n_sink, n))) <= got and set(range(max(n - n_local, 0), n)) <= got
    assert_out_close(u16(r["out"]), ref["out"])
    rh = _run_step(w, host=True, n_sink=n_sink, n_local=n_local)
    assert torch.equal(rh["idx"], r["idx"]) and torch.equal(rh["out"], r["out"])


@pytest.mark.parametrize("cfg", [
    wl.Config("paged-small", 57, 2, [1500, 333], None, 0.02, n_q_heads=8, n_kv_heads=2, sparsity=8),        # one fused launch
    wl.Config("paged-batch", 58, 20, [700 + 53 * i for i in range(20)], None, 0.02, n_q_heads=8, n_kv_heads=2,
              sparsity=8),                                                              # one fused launch, clusters of 4
    wl.Config("paged-large-batch", 60, 85, [300 + 13 * i for i in range(85)], None, 0.02, n_q_heads=8, n_kv_heads=2,
              sparsity=8),                                                                                   # three kernels
])
@pytest.mark.parametrize("page_size", [1, 16])
def test_sparse_decode_step_over_a_paged_cache(cfg, page_size):
    """The whole step with K/V in pages scattered over a pool gives exactly what it gives on the contiguous
    cache (same lists, same outputs), with and without always-kept windows."""
    w = wl.make_workload(cfg, DEV)
    B, Hq, Hkv, N = cfg.batch, cfg.n_q_heads, cfg.n_kv_heads, w["n_cap"]
    pps = (N + page_size - 1) // page_size
    g = torch.Generator(DEV).manual_seed(page_size)
    perm = torch.randperm(B * pps + 7, device=DEV, generator=g)[:B * pps].to(torch.int32).reshape(B, pps)
    pools = []
    for X in (w["K"], w["V"]):
        Xp = torch.zeros(B * pps + 7, Hkv, page_size, 128, dtype=X.dtype, device=DEV)
        Xp[perm.reshape(-1).long()] = torch.nn.functional.pad(X, (0, 0, 0, pps * page_size - N)) \
            .reshape(B, Hkv, pps, page_size, 128).permute(0, 2, 1, 3, 4).reshape(B * pps, Hkv, page_size, 128)
        pools.append(Xp)
    for n_sink, n_local in ((0, 0), (16, 48)):
        ref = _run_step(w, n_sink=n_sink, n_local=n_local)            # contiguous cache (itself checked against the oracle)
        k_max = w["k_max"] + n_sink + n_local
        shape = ha.make_shape(B, Hq, Hkv, w["sm_scale"], n_sink=n_sink, n_local=n_local)
        ws = ha.alloc_workspace(shape, N, k_max)
        kc = ref["kc"].clone()
        qc = torch.zeros(B, Hq, dtype=torch.int32, device=DEV)
        idx = torch.zeros(B, Hkv, k_max, dtype=torch.int32, device=DEV)
        cnt = torch.zeros(B, Hkv, dtype=torch.int32, device=DEV)
        out = torch.zeros(B, Hq, 128, dtype=torch.bfloat16, device=DEV)
        ha.ha_sparse_decode_paged(shape, ha.Mapping(w["map_q"]), ha.Mapping(w["map_k"]), w["q"], w["k_new"], pools[0], pools[1],
                                  perm, page_size, kc, w["seq_lens"], w["k_per_seq"], 0, N, k_max, qc, idx, cnt, out, ws)
        torch.cuda.synchronize()
        assert ha.ha_read_device_status(ws) == 0
        assert torch.equal(idx, ref["idx"]) and torch.equal(cnt, ref["cnt"]) and torch.equal(qc, ref["qc"])
        assert torch.equal(out, ref["out"])
        # The host-buffer entry over the same pools: the rows of the appended token are wiped first, the call has to
        # put them back (into the right page and slot) and to give the same lists and outputs, from pinned and from
        # pageable host buffers.
        last = [(b, int(perm[b, (w["lens"][b] - 1) // page_size]), (w["lens"][b] - 1) % page_size) for b in range(B) if w["lens"][b] > 0]
        for pinned in (True, False):
            pk, pv = pools[0].clone(), pools[1].clone()
            for (b, page, slot) in last:
                pk[page, :, slot] = 0
                pv[page, :, slot] = 0
            pin = (lambda t: t.pin_memory()) if pinned else (lambda t: t)
            hq, hk, hv = (pin(w[x].cpu()) for x in ("q", "k_new", "v_new"))
            ho = pin(torch.zeros(B, Hq, 128, dtype=torch.bfloat16))
            kc2, idx2, cnt2 = ref["kc"].clone(), torch.zeros_like(idx), torch.zeros_like(cnt)
            ha.ha_sparse_decode_paged_host(shape, ha.Mapping(w["map_q"]), ha.Mapping(w["map_k"]), hq, hk, hv, pk, pv, perm,
                                           page_size, kc2, w["seq_lens"], w["k_per_seq"], 0, N, k_max, idx2, cnt2, ho, ws)
            assert torch.equal(pk, pools[0]) and torch.equal(pv, pools[1])
            assert torch.equal(idx2, ref["idx"]) and torch.equal(cnt2, ref["cnt"]) and torch.equal(ho.to(DEV), ref["out"])


@pytest.mark.parametrize("seed", range(14))
def test_sparse_decode_step_random_configs(seed):
    """Seeded sweep over batch (both the fused launch and the three-kernel path), KV heads, group size, ragged
    lengths, sparsity and window sizes; everything the step returns is checked against the oracle."""
    rng = np.random.default_rng(7000 + seed)
    B = int(rng.integers(1, 13)) if seed < 8 else int(rng.integers(13, 110))   # up to 24 units / up to 220 units
    Hkv = int(rng.choice([1, 2]))
    G = int(rng.choice([1, 2, 4, 8]))
    lens = [int(v) for v in rng.integers(1, 3000, size=B)]
    cfg = wl.Config(f"rand{seed}", 70 + seed, B, lens, None, 0.02, n_q_heads=Hkv * G, n_kv_heads=Hkv,
                    sparsity=int(rng.choice([2, 8, 16])))
    n_sink, n_local = (0, 0) if seed % 2 == 0 else (int(rng.integers(0, 100)), int(rng.integers(0, 100)))
    w = wl.make_workload(cfg, DEV)
    r = _run_step(w, n_sink=n_sink, n_local=n_local)
    Kc = oracle_key_codes(w["K"], w["map_k"], w["lens"])
    ref = oracle.decode_step(u16(w["q"]), u16(w["k_new"]), u16(w["K"]), u16(w["V"]), Kc.copy(),
                             wl.mapping_numpy(w["map_q"]), wl.mapping_numpy(w["map_k"]), w["lens"], w["ks"],
                             sm_scale=w["sm_scale"], n_threads=4, n_sink=n_sink, n_local=n_local)
    assert np.array_equal(codes_np(r["qc"]), ref["qcodes"])
    assert np.array_equal(r["cnt"].cpu().numpy(), ref["count"])
    assert np.array_equal(r["idx"].cpu().numpy(), ref["idx"])
    assert_out_close(u16(r["out"]), ref["out"])


@pytest.mark.parametrize("cfg,launches", [
    # 32 units, small budgets: one fused launch of the one-stage variant (two CTAs per SM), clusters of 8
    (wl.Config("fused-32-units", 80, 16, [1000 + 61 * i for i in range(16)], None, 0.02, n_q_heads=8, n_kv_heads=2,
               sparsity=8), 1),
    # 60 units: clusters of 4 (two query vectors per encoding CTA, 32 tokens per thread)
    (wl.Config("fused-60-units", 84, 30, [1500 + 97 * i for i in range(30)], None, 0.02, n_q_heads=8, n_kv_heads=2,
               sparsity=8), 1),
    # 100 units: more clusters of four than the device holds at once
    (wl.Config("split-100-units", 85, 50, [2500 + 301 * i for i in range(50)], None, 0.02, n_q_heads=16, n_kv_heads=2,
               sparsity=16), 3),
    # 6 units, budgets above 2048 rows: one fused launch of the two-stage variant, several blocks per warp
    (wl.Config("fused-large-k", 81, 3, [9000, 5000, 12001], None, 0.02, n_q_heads=8, n_kv_heads=2, sparsity=2), 1),
    # 20 units with budgets of 1500 rows: more clusters than the two-stage variant holds at once, so the
    # one-stage variant takes them, two blocks per warp one after the other
    (wl.Config("fused-20-units-1500", 86, 10, [6000 + 7 * i for i in range(10)], None, 0.02, n_q_heads=8, n_kv_heads=2,
               sparsity=4), 1),
    # 20 units with budgets above 2048 rows: three kernels
    (wl.Config("split-large-k", 82, 10, [6000 + 7 * i for i in range(10)], None, 0.02, n_q_heads=8, n_kv_heads=2,
               sparsity=2), 3),
    # 1200 units: more than the balanced work split of GATHER-ATT holds: one CTA per unit
    (wl.Config("three-kernels-1200-units", 87, 600, [150 + (37 * i) % 200 for i in range(600)], None, 0.02, n_q_heads=4,
               n_kv_heads=2, sparsity=8), 3),
])
def test_sparse_decode_step_every_launch_variant(cfg, launches):
    """The step picks the fused cluster kernel (one or two row stages per warp) or the three-kernel path from
    the number of units and the budget; each choice gives the oracle's result."""
    w = wl.make_workload(cfg, DEV)
    _run_step(w)                                   # first call: attributes, occupancy query
    before = ha.ha_kernel_launches()
    r = _run_step(w)
    # _run_step also builds the prompt's signature cache with one ha_encode launch
    assert ha.ha_kernel_launches() - before == launches + 1
    Kc = oracle_key_codes(w["K"], w["map_k"], w["lens"])
    ref = oracle.decode_step(u16(w["q"]), u16(w["k_new"]), u16(w["K"]), u16(w["V"]), Kc.copy(),
                             wl.mapping_numpy(w["map_q"]), wl.mapping_numpy(w["map_k"]), w["lens"], w["ks"],
                             sm_scale=w["sm_scale"], n_threads=4)
    assert np.array_equal(codes_np(r["qc"]), ref["qcodes"])
    assert np.array_equal(r["cnt"].cpu().numpy(), ref["count"])
    assert np.array_equal(r["idx"].cpu().numpy(), ref["idx"])
    assert_out_close(u16(r["out"]), ref["out"])
    # The host-buffer entry takes the same variant.  The one-stage fused kernel reads q / k_new / v_new from the
    # pinned buffers and appends the new rows itself (one launch); every other variant is preceded by the small
    # kernel that pulls the inputs across the bus and appends (one launch more).
    before = ha.ha_kernel_launches()
    rh = _run_step(w, host=True)                   # checks that the new K/V rows were appended in place
    one_stage_fused = launches == 1 and w["k_max"] <= 2048 and cfg.name != "fused-large-k"
    assert ha.ha_kernel_launches() - before == (1 if one_stage_fused else launches + 1) + 1
    assert torch.equal(rh["idx"], r["idx"]) and torch.equal(rh["out"], r["out"])


@pytest.mark.parametrize("name,B,Hq,Hkv,lens,sparsity,windows", [
    # 120 ragged units, a few blocks each: most CTAs of the persistent kernel share units with their neighbours
    ("ragged-120-units", 60, 8, 2, [1 + (997 * i) % 5000 for i in range(60)], 8, (0, 0)),
    # 200 short units: several whole units per CTA, empty sequences and one-token sequences among them
    ("short-200-units", 100, 4, 2, [(53 * i) % 300 for i in range(100)], 4, (0, 0)),
    # 6 long units: every unit is scored by many CTAs, chunk by chunk, through the workspace
    ("long-6-units", 3, 8, 2, [70001, 40000, 9], 16, (0, 0)),
    # 128 units of 9000 tokens with half of them selected: units of more than 32768 / fewer tokens side by side
    ("wide-budget-128-units", 64, 4, 2, [9000 - 13 * i for i in range(64)], 2, (0, 0)),
    # one unit longer than the score bytes a CTA keeps in shared memory, owned by ONE CTA (tiny budgets around it)
    ("owned-long-unit", 40, 4, 2, [40000] + [600] * 39, 1000, (0, 0)),
    # always-kept windows on shared units; groups of one and of eight query heads
    ("windows-150-units", 75, 16, 2, [300 + (211 * i) % 4000 for i in range(75)], 8, (16, 100)),
    ("one-head-groups", 80, 2, 2, [1 + (389 * i) % 3000 for i in range(80)], 8, (0, 0)),
    ("eight-head-groups", 40, 16, 2, [2000 + 77 * i for i in range(40)], 16, (3, 0)),
])
def test_pipelined_step_ragged_lengths_shared_and_owned_units(name, B, Hq, Hkv, lens, sparsity, windows):
    """ha_sparse_decode_pipelined (ENCODE, then the persistent SCORE + TOPK + GATHER-ATT kernel): whole units per CTA, units
    shared by neighbouring CTAs, units scored chunk by chunk through the workspace, empty selections; compared with the
    oracle on everything the step returns, then run three times on one workspace (the release counters must be back
    at zero after every call)."""
    cfg = wl.Config(name, 90 + len(name), B, lens, None, 0.02, n_q_heads=Hq, n_kv_heads=Hkv, sparsity=sparsity)
    w = wl.make_workload(cfg, DEV)
    n_sink, n_local = windows
    before = ha.ha_kernel_launches()
    r = _run_step(w, n_sink=n_sink, n_local=n_local, pipelined=True)
    assert ha.ha_kernel_launches() - before == 3            # prompt signatures, ENCODE of the step, the pipelined kernel
    Kc = oracle_key_codes(w["K"], w["map_k"], w["lens"])
    ref = oracle.decode_step(u16(w["q"]), u16(w["k_new"]), u16(w["K"]), u16(w["V"]), Kc.copy(),
                             wl.mapping_numpy(w["map_q"]), wl.mapping_numpy(w["map_k"]), w["lens"], w["ks"],
                             sm_scale=w["sm_scale"], n_threads=4, n_sink=n_sink, n_local=n_local)
    assert np.array_equal(codes_np(r["qc"]), ref["qcodes"])
    assert np.array_equal(r["cnt"].cpu().numpy(), ref["count"])
    assert np.array_equal(r["idx"].cpu().numpy(), ref["idx"])
    assert_out_close(u16(r["out"]), ref["out"])
    got_lse = r["lse"].cpu().numpy().astype(np.float64)
    finite = np.isfinite(ref["lse"])
    assert np.array_equal(np.isneginf(got_lse), ~finite)
    assert np.max(np.abs(got_lse[finite] - ref["lse"][finite]), initial=0.0) < 1e-3
    # the same step three times in a row on ONE workspace: every call must find the counters at zero
    shape = ha.make_shape(B, Hq, Hkv, w["sm_scale"], n_sink=n_sink, n_local=n_local)
    k_max = w["k_max"] + n_sink + n_local
    ws = ha.alloc_workspace(shape, w["n_cap"], k_max)
    mq, mk = ha.Mapping(w["map_q"]), ha.Mapping(w["map_k"])
    for _ in range(3):
        idx = torch.full((B, Hkv, k_max), 7, dtype=torch.int32, device=DEV)
        cnt = torch.full((B, Hkv), 7, dtype=torch.int32, device=DEV)
        out = torch.full((B, Hq, 128), 3.0, dtype=torch.bfloat16, device=DEV)
        qc = torch.zeros(B, Hq, dtype=torch.int32, device=DEV)
        ha.ha_sparse_decode_pipelined(shape, mq, mk, w["q"], w["k_new"], w["K"], w["V"], r["kc"], w["seq_lens"], w["k_per_seq"],
                                      0, w["n_cap"], k_max, qc, idx, cnt, out, ws)
        torch.cuda.synchronize()
        assert ha.ha_read_device_status(ws) == 0
        assert torch.equal(idx, r["idx"]) and torch.equal(cnt, r["cnt"]) and torch.equal(out, r["out"])
    # ... and ha_sparse_decode itself (fused or three kernels) returns the same lists
    r2 = _run_step(w, n_sink=n_sink, n_local=n_local)
    assert torch.equal(r2["idx"], r["idx"]) and torch.equal(r2["cnt"], r["cnt"]) and torch.equal(r2["qc"], r["qc"])
    assert max_abs_diff_bf16(u16(r2["out"]), u16(r["out"])) <= OUT_AIM


def test_k_equals_n_sparse_step_equals_dense_kernel():
    cfg = wl.Config("k=n", 52, 2, [1500, 900], None, 0.0, n_q_heads=8, n_kv_heads=2, sparsity=1)
    w = wl.make_workload(cfg, DEV)
    r = _run_step(w)
    shape = ha.make_shape(2, 8, 2, w["sm_scale"])
    ws = ha.alloc_workspace(shape, w["n_cap"], w["n_cap"])
    dense = torch.zeros_like(r["out"])
    ha.ha_dense_decode(shape, w["q"], w["K"], w["V"], w["seq_lens"], w["n_cap"], dense, ws)
    assert_out_close(u16(dense), u16(r["out"]))
    assert r["cnt"].cpu().tolist() == [[1500, 1500], [900, 900]]


@pytest.mark.parametrize("reps", [1, 5, 12, 40])     # 8 / 40 units: fused kernel, clusters of 8 / 4; 96 and 320 units: three-kernel path
def test_step_edge_cases_empty_sequence_budget_above_length_and_no_new_key(reps):
    # one launch covers: an empty sequence, a one-token sequence, k > n, k = 0; then the same without a new key
    cfg = wl.Config("edges", 53, 4 * reps, [0, 1, 37, 2500] * reps, 64, 0.0, n_q_heads=8, n_kv_heads=2)
    w = wl.make_workload(cfg, DEV)
    w["ks"] = [5, 9, 64, 0] * reps
    w["k_per_seq"] = torch.tensor(w["ks"], dtype=torch.int32, device=DEV)
    w["k_max"] = 64
    B, Hq, Hkv = 4 * reps, 8, 2
    shape = ha.make_shape(B, Hq, Hkv, w["sm_scale"])
    ws = ha.alloc_workspace(shape, w["n_cap"], w["k_max"])
    mq, mk = ha.Mapping(w["map_q"]), ha.Mapping(w["map_k"])
    Kc = oracle_key_codes(w["K"], w["map_k"], w["lens"])
    for with_key in (True, False):
        kc = torch.from_numpy(np.pad(Kc, ((0, 0), (0, 0), (0, (-Kc.shape[2]) % 4))).view(np.int32)).to(DEV)
        if with_key:
            for b in range(B):
                if w["lens"][b] > 0:
                    kc[b, :, w["lens"][b] - 1] = 0x0BADF00D
        qc = torch.zeros(B, Hq, dtype=torch.int32, device=DEV)
        idx = torch.full((B, Hkv, 64), 7, dtype=torch.int32, device=DEV)
        cnt = torch.full((B, Hkv), 7, dtype=torch.int32, device=DEV)
        out = torch.full((B, Hq, 128), 3.0, dtype=torch.bfloat16, device=DEV)
        lse = torch.zeros(B, Hq, device=DEV)
        ha.ha_sparse_decode(shape, mq, mk if with_key else None, w["q"], w["k_new"] if with_key else None, w["K"], w["V"],
                            kc, w["seq_lens"], w["k_per_seq"], 0, w["n_cap"], 64, qc, idx, cnt, out, ws, lse=lse)
        torch.cuda.synchronize()
        ref = oracle.decode_step(u16(w["q"]), u16(w["k_new"]) if with_key else None, u16(w["K"]), u16(w["V"]), Kc.copy(),
                                 wl.mapping_numpy(w["map_q"]), wl.mapping_numpy(w["map_k"]), w["lens"], w["ks"],
                                 sm_scale=w["sm_scale"])
        assert np.array_equal(codes_np(kc)[:, :, :Kc.shape[2]], Kc)          # appended slots rewritten (or untouched)
        assert np.array_equal(codes_np(qc), ref["qcodes"])
        assert np.array_equal(cnt.cpu().numpy(), ref["count"]) and cnt.cpu().numpy().tolist() == [[0, 0], [1, 1], [37, 37], [0, 0]] * reps
        assert np.array_equal(idx.cpu().numpy(), ref["idx"])
        assert_out_close(u16(out), ref["out"])
        got = lse.cpu().numpy().astype(np.float64)
        fin = np.isfinite(ref["lse"])
        assert np.array_equal(np.isneginf(got), ~fin) and np.max(np.abs(got[fin] - ref["lse"][fin]), initial=0.0) < 1e-3
        assert not u16(out)[0::4].any() and not u16(out)[3::4].any()          # empty selections give zeros


@pytest.mark.parametrize("B", [1, 6, 40, 90])   # fused clusters of 8 / of 4 / three kernels (80 and 180 units)
def test_append_by_a_separate_encode_call_and_consecutive_steps_on_one_cache(B):
    """Library kernels start while the library kernel in front of them is finishing, and request signatures before they
    wait for it.  Two sequences of calls in which that kernel writes a signature the next one needs: (1) the Section 4.1
    append done by its own ha_encode call (slot = seq_len - 1) followed by a step without k_new; (2) two layer-steps back
    to back on the same cache for lengths n and n + 1, the second of which needs the signature the first appended."""
    lens = [2000 + 37 * b for b in range(B)]
    cfg = wl.Config("append", 57, B, [n + 1 for n in lens], 128, 0.02, n_q_heads=8, n_kv_heads=2)
    w = wl.make_workload(cfg, DEV)                                      # caches of n + 1 tokens per sequence
    Hq, Hkv, n_cap = 8, 2, w["n_cap"]
    shape = ha.make_shape(B, Hq, Hkv, w["sm_scale"])
    ws = ha.alloc_workspace(shape, n_cap, 128)
    mq, mk = ha.Mapping(w["map_q"]), ha.Mapping(w["map_k"])
    Kc = oracle_key_codes(w["K"], w["map_k"], [n + 1 for n in lens])
    clean = torch.from_numpy(np.pad(Kc, ((0, 0), (0, 0), (0, (-Kc.shape[2]) % 4))).view(np.int32)).to(DEV)
    stale = clean.clone()
    ar = torch.arange(B, device=DEV)
    len1 = torch.tensor(lens, dtype=torch.int32, device=DEV)            # first step: n tokens, appended token n - 1
    len2 = len1 + 1                                                     # second step: n + 1 tokens, appended token n
    slot1 = len1 - 1
    stale[ar, :, len1.long() - 1] = 0x5A5A5A5A
    stale[ar, :, len2.long() - 1] = 0x0F0F0F0F
    k1 = w["K"][ar, :, len1.long() - 1].contiguous()
    k2 = w["K"][ar, :, len2.long() - 1].contiguous()
    kc = stale.clone()
    qc = torch.zeros(B, Hq, dtype=torch.int32, device=DEV)
    idx = torch.zeros(B, Hkv, 128, dtype=torch.int32, device=DEV)
    cnt = torch.zeros(B, Hkv, dtype=torch.int32, device=DEV)
    out = torch.zeros(B, Hq, 128, dtype=torch.bfloat16, device=DEV)
    qu, Ku, Vu = u16(w["q"]), u16(w["K"]), u16(w["V"])
    mqn, mkn = wl.mapping_numpy(w["map_q"]), wl.mapping_numpy(w["map_k"])
    ref1 = oracle.decode_step(qu, None, Ku, Vu, Kc.copy(), mqn, mkn, lens, [128] * B, sm_scale=w["sm_scale"], n_threads=4)
    ref2 = oracle.decode_step(qu, None, Ku, Vu, Kc.copy(), mqn, mkn, [n + 1 for n in lens], [128] * B,
                              sm_scale=w["sm_scale"], n_threads=4)
    for _ in range(10):
        # (1) append by ha_encode, then the step without a new key
        kc.copy_(stale)
        ha.ha_encode(mk, 1, k1, kc, slot=slot1)
        ha.ha_sparse_decode(shape, mq, None, w["q"], None, w["K"], w["V"], kc, len1, None, 128, n_cap, 128, qc, idx, cnt, out, ws)
        torch.cuda.synchronize()
        assert np.array_equal(idx.cpu().numpy(), ref1["idx"]) and np.array_equal(cnt.cpu().numpy(), ref1["count"])
        assert_out_close(u16(out), ref1["out"])
        # (2) two steps back to back: n tokens, then n + 1 tokens
        kc.copy_(stale)
        ha.ha_sparse_decode(shape, mq, mk, w["q"], k1, w["K"], w["V"], kc, len1, None, 128, n_cap, 128, qc, idx, cnt, out, ws)
        ha.ha_sparse_decode(shape, mq, mk, w["q"], k2, w["K"], w["V"], kc, len2, None, 128, n_cap, 128, qc, idx, cnt, out, ws)
        torch.cuda.synchronize()
        assert torch.equal(kc, clean)                                   # both appended signatures are in place
        assert np.array_equal(idx.cpu().numpy(), ref2["idx"]) and np.array_equal(cnt.cpu().numpy(), ref2["count"])
        assert_out_close(u16(out), ref2["out"])
    assert ha.ha_read_device_status(ws) == 0


# ---------------------------------------------------------------- wide signatures (SCORE-latency table)

def _wide_codes(rng, n, W):
    return rng.integers(0, 2**63, size=(n, W), dtype=np.uint64) * np.uint64(2) + rng.integers(0, 2, size=(n, W), dtype=np.uint64)


@pytest.mark.parametrize("n_bits", [64, 128, 256, 512])
@pytest.mark.parametrize("n", [1, 2, 3, 1000, 100003, 1 << 20])
def test_score_wide_is_bit_exact(n_bits, n):
    """Every score of the stand-alone wide-signature pass equals the oracle's bit-by-bit count: single tokens,
    odd counts (the 64-bit case packs two tokens per load), several CTA iterations and a ragged tail."""
    W = n_bits // 64
    rng = np.random.default_rng(9000 + n_bits + n % 97)
    q, k = _wide_codes(rng, 1, W)[0], _wide_codes(rng, n, W)
    if n >= 3:
        k[0] = q          # a full match and a complement among the tokens
        k[2] = ~q
    dq = torch.from_numpy(q.view(np.int64)).to(DEV)
    dk = torch.from_numpy(k.view(np.int64)).to(DEV)
    out = torch.full((n + 3,), -7, dtype=torch.int16, device=DEV)
    ha.ha_score_wide(dq, dk, n_bits, out[:n])
    torch.cuda.synchronize()
    got = out.cpu().numpy()
    assert np.array_equal(got[:n].astype(np.int32), oracle.score_wide(q, k))
    assert np.all(got[n:] == -7)                       # nothing written past the last token
    if n >= 3:
        assert got[0] == n_bits and got[2] == 0


@pytest.mark.parametrize("n,stride", [(1, 128), (77, 128), (5000, 136), (200003, 128)])
def test_inner_products_match_the_oracle(n, stride):
    g = torch.Generator(DEV).manual_seed(n)
    K = torch.randn(n, stride, device=DEV, generator=g).to(torch.bfloat16)[:, :128]
    q = torch.randn(128, device=DEV, generator=g).to(torch.bfloat16)
    dots = torch.full((n + 1,), 123.0, device=DEV)
    ha.ha_inner_products(q, K, dots[:n])
    torch.cuda.synchronize()
    ref = oracle.inner_products(u16(q), u16(K.contiguous()))
    got = dots.cpu().numpy().astype(np.float64)
    # 128 products of magnitude ~1 accumulated in fp32: error far below 1e-3
    assert np.max(np.abs(got[:n] - ref)) < 1e-3
    assert got[n] == 123.0


# ---------------------------------------------------------------- wide signatures through ENCODE -> SCORE -> TOPK

def _wide_mapping(hkv, n_bits, seed):
    g = torch.Generator(DEV).manual_seed(seed)
    m = wl.make_mapping(hkv, g, DEV)
    bound = 1.0 / np.sqrt(128)
    m["w3"] = ((torch.rand(hkv, 128, n_bits, device=DEV, generator=g) * 2 - 1) * bound).to(torch.bfloat16)
    m["b3"] = (torch.rand(hkv, n_bits, device=DEV, generator=g) * 2 - 1) * bound
    return m


@pytest.mark.parametrize("n_bits", [64, 128, 256, 512])
@pytest.mark.parametrize("T", [1, 77, 300])
def test_encode_wide_is_bit_exact(n_bits, T):
    """ha_encode_wide against the oracle's Eq. 2 with a 128 x b last layer: every word of every signature, for the
    query side (heads sharing a network) and strided inputs, and the append into a token slot."""
    B, Hkv, G, W = 2, 2, 2, n_bits // 64
    m = _wide_mapping(Hkv, n_bits, 900 + n_bits)
    mp = ha.MappingWide(m)
    mn = wl.mapping_numpy(m)
    g = torch.Generator(DEV).manual_seed(77 + T)
    xs = torch.randn(B, Hkv * G, T + 3, 128, device=DEV, generator=g).to(torch.bfloat16)
    x = xs[:, :, 1:T + 1]                                         # strided view
    codes = torch.zeros(B, Hkv * G, T, W, dtype=torch.int64, device=DEV)
    ha.ha_encode_wide(mp, G, x, codes)
    torch.cuda.synchronize()
    got = codes.cpu().numpy().view(np.uint64)
    xu = u16(x.contiguous())
    for b in range(B):
        for h in range(Hkv * G):
            net = h // G
            ref = oracle.encode_wide(xu[b, h], mn["w1"][net], mn["w2"][net], mn["w3"][net], mn["b1"][net], mn["b2"][net], mn["b3"][net])
            assert np.array_equal(got[b, h], ref), (b, h)
    if T == 1:                                                    # append: one new vector per (sequence, head) into slot[b]
        cache = torch.full((B, Hkv * G, 9, W), -1, dtype=torch.int64, device=DEV)
        slot = torch.tensor([4, -1], dtype=torch.int32, device=DEV)
        ha.ha_encode_wide(mp, G, x[:, :, 0], cache, slot=slot)
        torch.cuda.synchronize()
        c = cache.cpu().numpy()
        assert np.array_equal(c[0, :, 4].view(np.uint64), got[0, :, 0]) and (c[1] == -1).all() and (c[0, :, :4] == -1).all()


def _check_score_topk_wide(n_bits, qc, kc, lens, ks, Hq, Hkv, n_sink=0, n_local=0):
    B, W, G = len(lens), n_bits // 64, Hq // Hkv
    n_cap = kc.shape[2]
    k_max = max(max(ks), 1) + n_sink + n_local
    shape = ha.make_shape(B, Hq, Hkv, 1.0, n_sink=n_sink, n_local=n_local)
    ws = ha.alloc_workspace_wide(shape, n_cap)
    idx = torch.full((B, Hkv, k_max), 7, dtype=torch.int32, device=DEV)
    cnt = torch.full((B, Hkv), 7, dtype=torch.int32, device=DEV)
    hist = torch.full((B, Hkv, n_bits + 1), -1, dtype=torch.int32, device=DEV)
    for _ in range(2):                                            # twice on one workspace: the histograms are cleared per call
        ha.ha_score_topk_wide(shape, n_bits, torch.from_numpy(qc.view(np.int64)).to(DEV), torch.from_numpy(kc.view(np.int64)).to(DEV),
                              torch.tensor(lens, dtype=torch.int32, device=DEV), torch.tensor(ks, dtype=torch.int32, device=DEV),
                              0, n_cap, k_max, idx, cnt, ws, hist_out=hist)
    torch.cuda.synchronize()
    idx_np, cnt_np, hist_np = idx.cpu().numpy(), cnt.cpu().numpy(), hist.cpu().numpy()
    for b, n in enumerate(lens):
        for g in range(Hkv):
            s = oracle.score_wide_group(qc[b, g * G:(g + 1) * G], kc[b, g, :n]) if n else np.zeros(0, np.int32)
            ref = oracle.topk_windows(s, ks[b], n_sink, n_local) if (n_sink or n_local) else oracle.topk(s, ks[b])
            assert cnt_np[b, g] == len(ref), (b, g, cnt_np[b, g], len(ref))
            assert np.array_equal(idx_np[b, g, :len(ref)], ref), (b, g)
            assert (idx_np[b, g, len(ref):] == -1).all()
            others = np.ones(n, bool)
            others[:min(n_sink, n)] = False
            others[max(n - n_local, min(n_sink, n)):] = False
            assert np.array_equal(hist_np[b, g], np.bincount(s[others], minlength=n_bits + 1))
    return idx_np


@pytest.mark.parametrize("n_bits", [64, 128, 256, 512])
@pytest.mark.parametrize("G", [1, 4])
def test_score_topk_wide_sizes_ragged_tail_budgets_and_ties(n_bits, G):
    rng = np.random.default_rng(n_bits + G)
    W, Hkv = n_bits // 64, 2
    lens = [0, 1, 15, 4097, 20000, 70001]
    ks = [3, 5, 20, 300, 0, 9000]
    n_cap = max(lens) + 5
    kc = _wide_codes(rng, len(lens) * Hkv * n_cap, W).reshape(len(lens), Hkv, n_cap, W)
    qc = _wide_codes(rng, len(lens) * Hkv * G, W).reshape(len(lens), Hkv * G, W)
    kc[3, :, 100:400] = kc[3, :, 99:100]                          # a block of equal signatures: ties decided by token index
    kc[5, 0, 5000] = qc[5, 0]                                     # an exact match: the top level b
    flip = rng.integers(0, 64, size=(n_cap,))                     # near matches at every distance from 1 on
    kc[5, 1, :] = qc[5, G]
    for t in range(0, 3000):
        kc[5, 1, t, (t // 64) % W] ^= np.uint64(((1 << (t % 64 + 1)) - 1) & (2**64 - 1))
    _check_score_topk_wide(n_bits, qc, kc, lens, ks, Hkv * G, Hkv)


@pytest.mark.parametrize("n_sink,n_local", [(128, 128), (3, 0), (5000, 70000)])
def test_score_topk_wide_with_always_kept_windows(n_sink, n_local):
    rng = np.random.default_rng(7)
    n_bits, W, Hkv, G = 128, 2, 2, 2
    lens = [100, 6000, 150001]
    ks = [10, 700, 2000]
    n_cap = max(lens)
    kc = _wide_codes(rng, len(lens) * Hkv * n_cap, W).reshape(len(lens), Hkv, n_cap, W)
    qc = _wide_codes(rng, len(lens) * Hkv * G, W).reshape(len(lens), Hkv * G, W)
    _check_score_topk_wide(n_bits, qc, kc, lens, ks, Hkv * G, Hkv, n_sink, n_local)


@pytest.mark.parametrize("n_bits", [64, 256])
def test_step_from_entry_points_at_wide_signatures(n_bits):
    """ENCODE -> SCORE -> TOPK -> GATHER-ATT chained through the wide entry points against the same chain of oracle
    functions (Section 4 recipe at b = 64 / 256 bits): the index lists of ha_score_topk_wide feed ha_gather_attn."""
    cfg = wl.Config("wide-chain", 59, 3, [300, 5000, 1], None, 0.02, n_q_heads=8, n_kv_heads=2, sparsity=8)
    w = wl.make_workload(cfg, DEV)
    B, Hq, Hkv, G, W = 3, 8, 2, 4, n_bits // 64
    mq, mk = _wide_mapping(Hkv, n_bits, 31), _wide_mapping(Hkv, n_bits, 32)
    n_cap, k_max = w["n_cap"], w["k_max"]
    kc = torch.zeros(B, Hkv, n_cap, W, dtype=torch.int64, device=DEV)
    qc = torch.zeros(B, Hq, 1, W, dtype=torch.int64, device=DEV)
    ha.ha_encode_wide(ha.MappingWide(mk), 1, w["K"], kc)
    ha.ha_encode_wide(ha.MappingWide(mq), G, w["q"], qc)
    shape = ha.make_shape(B, Hq, Hkv, w["sm_scale"])
    idx = torch.zeros(B, Hkv, k_max, dtype=torch.int32, device=DEV)
    cnt = torch.zeros(B, Hkv, dtype=torch.int32, device=DEV)
    out = torch.zeros(B, Hq, 128, dtype=torch.bfloat16, device=DEV)
    ha.ha_score_topk_wide(shape, n_bits, qc.reshape(B, Hq, W), kc, w["seq_lens"], w["k_per_seq"], 0, n_cap, k_max, idx, cnt,
                          ha.alloc_workspace_wide(shape, n_cap))
    ha.ha_gather_attn(shape, w["q"], w["K"], w["V"], w["seq_lens"], idx, cnt, k_max, out, ha.alloc_workspace(shape, n_cap, k_max))
    torch.cuda.synchronize()
    qu, Ku, Vu = u16(w["q"]), u16(w["K"]), u16(w["V"])
    mqn, mkn = wl.mapping_numpy(mq), wl.mapping_numpy(mk)
    idx_np, cnt_np = idx.cpu().numpy(), cnt.cpu().numpy()
    for b, n in enumerate(w["lens"]):
        for g in range(Hkv):
            kcodes = oracle.encode_wide(Ku[b, g, :n], mkn["w1"][g], mkn["w2"][g], mkn["w3"][g], mkn["b1"][g], mkn["b2"][g], mkn["b3"][g])
            qcodes = oracle.encode_wide(qu[b, g * G:(g + 1) * G], mqn["w1"][g], mqn["w2"][g], mqn["w3"][g], mqn["b1"][g], mqn["b2"][g], mqn["b3"][g])
            assert np.array_equal(kc[b, g, :n].cpu().numpy().view(np.uint64), kcodes)
            ref = oracle.topk(oracle.score_wide_group(qcodes, kcodes), w["ks"][b])
            assert cnt_np[b, g] == len(ref) and np.array_equal(idx_np[b, g, :len(ref)], ref)
            for j in range(G):
                eo, _, _ = oracle.gather_attn(qu[b, g * G + j], Ku[b, g], Vu[b, g], ref, sm_scale=w["sm_scale"], n_valid=n)
                assert_out_close(u16(out[b, g * G + j]), eo)


# ---------------------------------------------------------------- paged signature cache

def _page_codes(codes_np, lens, page_size, rng):
    """Scatter contiguous signatures [B, Hkv, n_cap] over a pool [n_pages, Hkv, page_size]; returns (pool, block table)."""
    B, Hkv, n_cap = codes_np.shape
    pps = (n_cap + page_size - 1) // page_size
    perm = rng.permutation(B * pps + 5)[:B * pps].reshape(B, pps).astype(np.int32)
    pool = np.full((B * pps + 5, Hkv, page_size), 0x7BADC0DE, np.uint32)
    padded = np.pad(codes_np, ((0, 0), (0, 0), (0, pps * page_size - n_cap)))
    for b in range(B):
        pool[perm[b]] = padded[b].reshape(Hkv, pps, page_size).transpose(1, 0, 2)
    return pool, perm


@pytest.mark.parametrize("page_size", [1, 2, 16, 64])
def test_score_topk_over_a_paged_signature_cache(page_size):
    """ha_score_topk_paged and ha_score_topk_per_head_paged: lists, counts and histograms bit-identical to the oracle's
    on the un-paged signatures (paging is storage only), for ragged lengths, windows and ties."""
    rng = np.random.default_rng(100 + page_size)
    B, Hq, Hkv, G = 4, 8, 2, 4
    lens = [0, 37, 4100, 9000]
    ks = [4, 10, 300, 1000]
    n_cap = 9003
    codes = rng.integers(0, 2**32, size=(B, Hkv, n_cap), dtype=np.uint64).astype(np.uint32)
    codes[2, :, 500:900] = codes[2, :, 499:500]                         # a tie block
    qc = rng.integers(0, 2**32, size=(B, Hq), dtype=np.uint64).astype(np.uint32)
    pool, table = _page_codes(codes, lens, page_size, rng)
    for b in range(B):                                                  # the pool round-trips through the oracle's reader
        for h in range(Hkv):
            assert np.array_equal(oracle.unpage_codes(pool, table[b], page_size, h, lens[b]), codes[b, h, :lens[b]])
    pool_t = torch.from_numpy(pool.view(np.int32)).to(DEV)
    table_t = torch.from_numpy(table).to(DEV)
    qc_t = torch.from_numpy(qc.view(np.int32)).to(DEV)
    sl = torch.tensor(lens, dtype=torch.int32, device=DEV)
    kp = torch.tensor(ks, dtype=torch.int32, device=DEV)
    for n_sink, n_local in ((0, 0), (3, 40)):
        k_max = max(ks) + n_sink + n_local
        shape = ha.make_shape(B, Hq, Hkv, 1.0, n_sink=n_sink, n_local=n_local)
        pick = lambda s, k: oracle.topk_windows(s, k, n_sink, n_local) if (n_sink or n_local) else oracle.topk(s, k)
        # grouped (maximum over the group)
        ws = ha.alloc_workspace(shape, n_cap, k_max)
        idx = torch.full((B, Hkv, k_max), 5, dtype=torch.int32, device=DEV)
        cnt = torch.full((B, Hkv), 5, dtype=torch.int32, device=DEV)
        ha.ha_score_topk_paged(shape, qc_t, pool_t, table_t, sl, kp, 0, n_cap, k_max, idx, cnt, ws)
        # one list per query head
        wsh = ha.alloc_workspace(ha.make_shape(B, Hq, Hq, 1.0), n_cap, k_max)
        idxh = torch.full((B, Hq, k_max), 5, dtype=torch.int32, device=DEV)
        cnth = torch.full((B, Hq), 5, dtype=torch.int32, device=DEV)
        ha.ha_score_topk_paged(shape, qc_t, pool_t, table_t, sl, kp, 0, n_cap, k_max, idxh, cnth, wsh, per_head=True)
        torch.cuda.synchronize()
        idx_np, cnt_np, idxh_np, cnth_np = idx.cpu().numpy(), cnt.cpu().numpy(), idxh.cpu().numpy(), cnth.cpu().numpy()
        for b, n in enumerate(lens):
            for g in range(Hkv):
                ref = pick(oracle.score(qc[b, g * G:(g + 1) * G], codes[b, g, :n]), ks[b])
                assert cnt_np[b, g] == len(ref) and np.array_equal(idx_np[b, g, :len(ref)], ref) and (idx_np[b, g, len(ref):] == -1).all()
                for j in range(G):
                    h = g * G + j
                    refh = pick(oracle.score(qc[b, h:h + 1], codes[b, g, :n]), ks[b])
                    assert cnth_np[b, h] == len(refh) and np.array_equal(idxh_np[b, h, :len(refh)], refh)


@pytest.mark.parametrize("page_size,B", [(1, 3), (16, 3), (16, 20)])
def test_whole_step_with_keys_values_and_signatures_all_paged(page_size, B):
    """ha_sparse_decode_paged_codes (K, V and signatures behind one block table, the appended signature written into the
    pool) returns the lists and outputs of ha_sparse_decode over the contiguous caches; ha_encode_append_paged and the
    per-head entries over the same pools agree with their contiguous forms."""
    lens = ([700, 2049, 33] + [500 + 61 * i for i in range(B)])[:B]
    cfg = wl.Config("all-paged", 63, B, lens, None, 0.02, n_q_heads=8, n_kv_heads=2, sparsity=8)
    w = wl.make_workload(cfg, DEV)
    Hq, Hkv, n_cap, k_max = 8, 2, w["n_cap"], w["k_max"]
    ref = _run_step(w)                                                  # contiguous caches (checked against the oracle elsewhere)
    rng = np.random.default_rng(5 + page_size)
    pps = (n_cap + page_size - 1) // page_size
    table = torch.from_numpy(rng.permutation(B * pps + 3)[:B * pps].reshape(B, pps).astype(np.int32)).to(DEV)

    def paged(X, fill):                                                 # [B, Hkv, n_cap, ...] -> pool [pages, Hkv, page_size, ...]
        tail = X.shape[3:]
        P = torch.full((B * pps + 3, Hkv, page_size) + tuple(tail), fill, dtype=X.dtype, device=DEV)
        pad = torch.zeros((B, Hkv, pps * page_size - n_cap) + tuple(tail), dtype=X.dtype, device=DEV)
        Xp = torch.cat([X, pad], dim=2).reshape((B, Hkv, pps, page_size) + tuple(tail)).transpose(1, 2)
        P[table.reshape(-1).long()] = Xp.reshape((B * pps, Hkv, page_size) + tuple(tail))
        return P

    Kp, Vp = paged(w["K"], 0), paged(w["V"], 0)
    kc_clean = ref["kc"][:, :, :n_cap]
    stale = kc_clean.clone()
    for b in range(B):
        stale[b, :, lens[b] - 1] = 0x0BADF00D                           # the step must write the appended signature into the pool
    Cp = paged(stale, 0x11111111)
    shape = ha.make_shape(B, Hq, Hkv, w["sm_scale"])
    ws = ha.alloc_workspace(shape, n_cap, k_max)
    mq, mk = ha.Mapping(w["map_q"]), ha.Mapping(w["map_k"])
    qc = torch.zeros(B, Hq, dtype=torch.int32, device=DEV)
    idx = torch.zeros(B, Hkv, k_max, dtype=torch.int32, device=DEV)
    cnt = torch.zeros(B, Hkv, dtype=torch.int32, device=DEV)
    out = torch.zeros(B, Hq, 128, dtype=torch.bfloat16, device=DEV)
    ha.ha_sparse_decode_paged_codes(shape, mq, mk, w["q"], w["k_new"], Kp, Vp, Cp, table, w["seq_lens"], w["k_per_seq"], 0, n_cap,
                                    k_max, qc, idx, cnt, out, ws)
    torch.cuda.synchronize()
    assert ha.ha_read_device_status(ws) == 0
    assert torch.equal(idx, ref["idx"]) and torch.equal(cnt, ref["cnt"]) and torch.equal(qc, ref["qc"])
    assert max_abs_diff_bf16(u16(out), u16(ref["out"])) <= OUT_AIM
    assert torch.equal(Cp, paged(kc_clean, 0x11111111))                 # every appended signature sits in its page slot
    # the stand-alone append into the pool
    Cp2 = paged(stale, 0x11111111)
    ha.ha_encode_append_paged(mk, w["k_new"], Cp2, table, w["seq_lens"])
    torch.cuda.synchronize()
    assert torch.equal(Cp2, Cp)
    # one list per query head over the pools against the contiguous per-head entries
    idxh = torch.zeros(B, Hq, k_max, dtype=torch.int32, device=DEV)
    cnth = torch.zeros(B, Hq, dtype=torch.int32, device=DEV)
    idxr, cntr = torch.zeros_like(idxh), torch.zeros_like(cnth)
    outh, outr = torch.zeros_like(out), torch.zeros_like(out)
    wsh = ha.alloc_workspace(ha.make_shape(B, Hq, Hq, w["sm_scale"]), n_cap, k_max)
    ha.ha_score_topk_paged(shape, qc, Cp, table, w["seq_lens"], w["k_per_seq"], 0, n_cap, k_max, idxh, cnth, wsh, per_head=True)
    ha.ha_gather_attn_per_head_paged(shape, w["q"], Kp, Vp, table, page_size, w["seq_lens"], idxh, cnth, k_max, outh, wsh)
    kc_c = torch.nn.functional.pad(kc_clean, (0, (-n_cap) % 4)).contiguous()
    ha.ha_score_topk_per_head(shape, qc, kc_c, w["seq_lens"], w["k_per_seq"], 0, k_max, idxr, cntr)
    ha.ha_gather_attn_per_head(shape, w["q"], w["K"], w["V"], w["seq_lens"], idxr, cntr, k_max, outr, wsh)
    torch.cuda.synchronize()
    assert torch.equal(idxh, idxr) and torch.equal(cnth, cntr) and torch.equal(outh, outr)
