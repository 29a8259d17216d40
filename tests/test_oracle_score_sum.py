"""Pins for the oracle's alternative GQA reduction: Eq. 1 per query head, summed over the heads of the group
(the contract of the layer-step takes the maximum instead).  CPU only.

None of the pins shares the oracle's formulation:
  * +-1 vectors: the sum of the per-head scores is (32 G + <sum_j s_qj, s_k>) / 2 (Eq. 1 with the bitcount
    identity of Section 4.1, added over the heads), computed with a float matrix product;
  * Python integers: the G query codes concatenated into one 32 G-bit number against the key code repeated
    G times, xor and count of one bits;
  * special cases: one head is Eq. 1 itself (the already pinned score); equal heads give G times the single
    score; a head and its complement add up to 32 whatever the key;
  * relations to the maximum: max <= sum <= G max, with equality patterns;
  * top-k over the summed scores against brute force with Python's sort on tiny inputs.
"""
import numpy as np
import pytest

import oracle

GROUPS = [1, 2, 4, 8]


def _pm1(codes):
    bits = np.unpackbits(np.ascontiguousarray(codes, dtype="<u4").view(np.uint8).reshape(len(codes), 4), axis=1,
                         bitorder="little")
    return bits.astype(np.float64) * 2.0 - 1.0


@pytest.mark.parametrize("G", GROUPS)
def test_sum_score_is_half_of_bits_plus_inner_product_with_the_summed_sign_vectors(G):
    rng = np.random.default_rng(7 + G)
    q = rng.integers(0, 2**32, size=G, dtype=np.uint64).astype(np.uint32)
    k = rng.integers(0, 2**32, size=2500, dtype=np.uint64).astype(np.uint32)
    s = oracle.score_sum(q, k)
    dots = _pm1(k) @ _pm1(q).sum(axis=0)
    assert np.array_equal(s, ((32 * G + dots) / 2).astype(np.int64))
    assert s.min() >= 0 and s.max() <= 32 * G


@pytest.mark.parametrize("G", GROUPS)
def test_sum_score_equals_bitcount_of_concatenated_signatures(G):
    rng = np.random.default_rng(70 + G)
    q = [int(v) for v in rng.integers(0, 2**32, size=G, dtype=np.uint64)]
    k = [int(v) for v in rng.integers(0, 2**32, size=400, dtype=np.uint64)]
    big_q = sum(v << (32 * j) for j, v in enumerate(q))
    want = []
    for kv in k:
        big_k = sum(kv << (32 * j) for j in range(G))
        want.append(32 * G - bin(big_q ^ big_k).count("1"))
    got = oracle.score_sum(np.array(q, dtype=np.uint32), np.array(k, dtype=np.uint32))
    assert got.tolist() == want


def test_one_head_is_eq_1_and_equal_heads_multiply():
    rng = np.random.default_rng(3)
    k = rng.integers(0, 2**32, size=1000, dtype=np.uint64).astype(np.uint32)
    q = rng.integers(0, 2**32, size=1, dtype=np.uint64).astype(np.uint32)
    single = oracle.score(q, k)
    assert np.array_equal(oracle.score_sum(q, k), single)
    for G in (2, 4, 8):
        assert np.array_equal(oracle.score_sum(np.repeat(q, G), k), G * single)


def test_a_head_and_its_complement_add_up_to_32():
    rng = np.random.default_rng(4)
    k = rng.integers(0, 2**32, size=500, dtype=np.uint64).astype(np.uint32)
    q = np.uint32(0x9e3779b9)
    s = oracle.score_sum(np.array([q, ~q], dtype=np.uint32), k)
    assert np.all(s == 32)
    # special values: key equal to the only head / to its complement
    assert oracle.score_sum(np.array([q], dtype=np.uint32), np.array([q, ~q], dtype=np.uint32)).tolist() == [32, 0]


@pytest.mark.parametrize("G", [2, 4, 8])
def test_sum_lies_between_max_and_g_times_max_and_adds_over_heads(G):
    rng = np.random.default_rng(50 + G)
    q = rng.integers(0, 2**32, size=G, dtype=np.uint64).astype(np.uint32)
    k = rng.integers(0, 2**32, size=3000, dtype=np.uint64).astype(np.uint32)
    s, m = oracle.score_sum(q, k), oracle.score(q, k)
    assert np.all(m <= s) and np.all(s <= G * m)
    per_head = sum(oracle.score(q[j:j + 1], k) for j in range(G))     # the pinned single-head score, added up
    assert np.array_equal(s, per_head)
    # the order of the heads does not matter; a flip mask common to all codes does not either
    assert np.array_equal(oracle.score_sum(q[::-1], k), s)
    mask = np.uint32(0x0f0f1234)
    assert np.array_equal(oracle.score_sum(q ^ mask, k ^ mask), s)


def test_single_bit_flips_lower_the_sum_by_one_per_head_that_had_the_bit_right():
    q = np.array([0x00000000, 0xffffffff, 0x0000ffff, 0xffff0000], dtype=np.uint32)
    base = np.uint32(0x0000ffff)
    s0 = int(oracle.score_sum(q, np.array([base], dtype=np.uint32))[0])
    assert s0 == 16 + 16 + 32 + 0
    for bit in range(32):
        flipped = np.array([base ^ np.uint32(1 << bit)], dtype=np.uint32)
        agree_before = sum(1 for v in q.tolist() if ((v >> bit) & 1) == ((int(base) >> bit) & 1))
        assert int(oracle.score_sum(q, flipped)[0]) == s0 - agree_before + (4 - agree_before)


@pytest.mark.parametrize("seed", range(6))
def test_topk_over_summed_scores_against_python_sort(seed):
    rng = np.random.default_rng(900 + seed)
    G, n = (2, 4, 8, 4, 2, 8)[seed], 60 + 13 * seed
    q = rng.integers(0, 2**32, size=G, dtype=np.uint64).astype(np.uint32)
    # keys near one of the heads, so that the scores spread over many levels and ties are frequent
    k = (q[rng.integers(0, G, size=n)] ^ (np.uint32(1) << rng.integers(0, 32, size=n).astype(np.uint32))
         ^ np.where(rng.random(n) < 0.5, rng.integers(0, 2**32, size=n, dtype=np.uint64).astype(np.uint32), 0)).astype(np.uint32)
    s = oracle.score_sum(q, k)
    for kk in (0, 1, 7, n // 2, n, n + 5):
        order = sorted(range(n), key=lambda i: (-int(s[i]), i))[:min(kk, n)]
        assert oracle.topk(s, kk).tolist() == sorted(order)
