"""Pins for the oracle's wide-signature score (the setting of the paper's SCORE-latency table: one query
signature of 64 .. 512 bits against n key signatures, kept as packed 64-bit integers) and for the
inner-product comparator of the same table.  CPU only.

The score is pinned by what the mathematics fixes, none of which shares the oracle's formulation:
  * the relation between agreeing bits and the inner product of the +-1 vectors (Eq. 1 with the
    bitcount identity of Section 4.1: <s_q, s_k> = b - 2 Hamming, so score = (b + <s_q, s_k>) / 2),
    computed with a float matrix product;
  * Python's arbitrary-precision integers (xor of the whole b-bit numbers, count of one bits);
  * special values (equal signatures, complement, single flipped bits at every position, which fixes
    the bit and word order) and invariances (common flip mask, word permutation);
  * additivity over words, with each word's contribution given by the already pinned 32-bit score.
"""
import numpy as np
import pytest

import oracle

WORDS = [1, 2, 4, 8]   # 64, 128, 256, 512 bits


def _codes(rng, n, W):
    return rng.integers(0, 2**63, size=(n, W), dtype=np.uint64) * np.uint64(2) + rng.integers(0, 2, size=(n, W), dtype=np.uint64)


def _pm1(codes):
    """uint64 [n, W] -> float64 [n, 64 W] of +-1 (bit j of the signature = bit j % 64 of word j / 64)."""
    bits = np.unpackbits(codes.astype("<u8").view(np.uint8).reshape(codes.shape[0], -1), axis=1, bitorder="little")
    return bits.astype(np.float64) * 2.0 - 1.0


@pytest.mark.parametrize("W", WORDS)
def test_score_is_half_of_bits_plus_inner_product_of_sign_vectors(W):
    rng = np.random.default_rng(100 + W)
    q, k = _codes(rng, 1, W), _codes(rng, 3000, W)
    s = oracle.score_wide(q[0], k)
    dots = _pm1(k) @ _pm1(q)[0]                       # <s_q, s_k>, exact in float64
    assert np.array_equal(s, ((64 * W + dots) / 2).astype(np.int64))
    assert s.min() >= 0 and s.max() <= 64 * W


@pytest.mark.parametrize("W", WORDS)
def test_score_equals_big_integer_xor_popcount(W):
    rng = np.random.default_rng(200 + W)
    q, k = _codes(rng, 1, W), _codes(rng, 500, W)
    big = lambda row: sum(int(w) << (64 * j) for j, w in enumerate(row))
    qq = big(q[0])
    expect = [64 * W - bin(big(row) ^ qq).count("1") for row in k]
    assert oracle.score_wide(q[0], k).tolist() == expect


@pytest.mark.parametrize("W", WORDS)
def test_special_values_fix_the_bit_and_word_order(W):
    rng = np.random.default_rng(300 + W)
    q = _codes(rng, 1, W)[0]
    b = 64 * W
    assert oracle.score_wide(q, q[None, :])[0] == b
    assert oracle.score_wide(q, (~q)[None, :])[0] == 0
    # one flipped bit at every position: b - 1; two different flipped bits: b - 2
    flips = np.tile(q, (b, 1))
    for j in range(b):
        flips[j, j // 64] ^= np.uint64(1) << np.uint64(j % 64)
    assert np.all(oracle.score_wide(q, flips) == b - 1)
    # the lowest m bits flipped: b - m (a wrong word order or bit order would not give a ramp)
    ramp = np.tile(q, (b + 1, 1))
    for m in range(b + 1):
        for j in range(m):
            ramp[m, j // 64] ^= np.uint64(1) << np.uint64(j % 64)
    assert oracle.score_wide(q, ramp).tolist() == [b - m for m in range(b + 1)]


@pytest.mark.parametrize("W", [2, 8])
def test_invariances_and_additivity_over_words(W):
    rng = np.random.default_rng(400 + W)
    q, k = _codes(rng, 1, W)[0], _codes(rng, 800, W)
    base = oracle.score_wide(q, k)
    mask = _codes(rng, 1, W)[0]
    assert np.array_equal(oracle.score_wide(q ^ mask, k ^ mask), base)            # common flip mask
    perm = rng.permutation(W)
    assert np.array_equal(oracle.score_wide(q[perm], k[:, perm]), base)           # common word permutation
    # symmetric in its arguments
    assert all(int(oracle.score_wide(k[i], q[None, :])[0]) == int(base[i]) for i in range(40))
    # a signature's score is the sum of its 32-bit halves' scores (Eq. 1 at 32 bits, pinned separately)
    q32, k32 = q.astype("<u8").view(np.uint32), k.astype("<u8").view(np.uint32).reshape(k.shape[0], -1)
    parts = sum(oracle.score([q32[j]], np.ascontiguousarray(k32[:, j])) for j in range(2 * W))
    assert np.array_equal(base, parts)


def test_inner_products_match_float64_numpy_and_closed_forms():
    rng = np.random.default_rng(500)
    K = (rng.standard_normal((700, 128)).astype(np.float32).view(np.uint32) >> 16).astype(np.uint16)   # bf16 by truncation
    q = (rng.standard_normal(128).astype(np.float32).view(np.uint32) >> 16).astype(np.uint16)
    f = lambda a: (a.astype(np.uint32) << 16).view(np.float32).astype(np.float64)
    got = oracle.inner_products(q, K)
    assert np.allclose(got, f(K) @ f(q), rtol=1e-12, atol=1e-12)
    one = np.uint16(0x3F80)                                                       # bf16 1.0
    e3 = np.zeros(128, np.uint16); e3[3] = one
    assert np.array_equal(oracle.inner_products(e3, K), f(K)[:, 3])               # unit vector picks a component
    assert np.all(oracle.inner_products(np.zeros(128, np.uint16), K) == 0.0)
    ones = np.full(128, one, np.uint16)
    assert np.allclose(oracle.inner_products(ones, K), f(K).sum(axis=1), rtol=1e-12, atol=1e-12)
