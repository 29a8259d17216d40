"""Pins for the oracle's ENCODE at signatures of 64 to 512 bits (Eq. 2 with a wider last layer; the widths of the
bit-width study and of the SCORE-latency table): closed forms that fix bit and word order, the pinned 32-bit ENCODE on
the first 32 outputs, and an independent float64 evaluation.  CPU only."""
import numpy as np
import pytest
import torch

import oracle

D, HID = 128, 128


def bf16(a):
    t = torch.as_tensor(np.asarray(a, dtype=np.float32)).to(torch.bfloat16)
    return t.view(torch.int16).numpy().view(np.uint16).copy()


def bit(codes_row, j):
    return (int(codes_row[j // 64]) >> (j % 64)) & 1


@pytest.mark.parametrize("n_bits", [64, 128, 256, 512])
def test_signed_copies_of_the_input_fix_bit_and_word_order(n_bits):
    """W1 = W2 = I on a non-negative input, last layer column j = +e_(j mod 128) for even j // 128 and -e_(j mod 128)
    for odd ones, bias b3[j] = -t_j: bit j of the signature is (x[j mod 128] > t_j) or (-x[j mod 128] > t_j)."""
    rng = np.random.default_rng(11 + n_bits)
    x = np.abs(rng.standard_normal((40, D))).astype(np.float32)       # ReLU keeps non-negative inputs as they are
    xb = bf16(x)
    xv = oracle.bf16_bits_to_f64(xb)
    w3 = np.zeros((HID, n_bits), np.float32)
    for j in range(n_bits):
        w3[j % 128, j] = 1.0 if (j // 128) % 2 == 0 else -1.0
    thr = rng.choice([0.25, 0.5, 1.0, -0.5], size=n_bits).astype(np.float32)
    codes = oracle.encode_wide(xb, bf16(np.eye(D)), bf16(np.eye(HID)), bf16(w3), None, None, -thr)
    assert codes.shape == (40, n_bits // 64) and codes.dtype == np.uint64
    for r in range(40):
        for j in range(n_bits):
            val = xv[r, j % 128] * (1.0 if (j // 128) % 2 == 0 else -1.0)
            assert bit(codes[r], j) == int(np.float32(val) - thr[j] > 0), (r, j)


@pytest.mark.parametrize("n_bits", [64, 512])
def test_zero_weights_give_the_sign_pattern_of_the_last_bias(n_bits):
    rng = np.random.default_rng(5)
    b3 = rng.standard_normal(n_bits).astype(np.float32)
    b3[3] = 0.0
    b3[n_bits - 1] = -0.0
    z = np.zeros
    codes = oracle.encode_wide(bf16(rng.standard_normal((3, D))), z((D, HID), np.uint16), z((HID, HID), np.uint16),
                               z((HID, n_bits), np.uint16), None, None, b3)
    for r in range(3):
        assert [bit(codes[r], j) for j in range(n_bits)] == [int(b3[j] > 0) for j in range(n_bits)]


@pytest.mark.parametrize("n_bits", [64, 256])
def test_every_block_of_32_outputs_is_the_pinned_32_bit_encode(n_bits):
    """Output j depends on column j of the last layer alone: bits 32 c .. 32 c + 31 of the wide signature are the
    32-bit signature of the (pinned) ora_encode run on those 32 columns."""
    rng = np.random.default_rng(21)
    bound = 1.0 / np.sqrt(D)
    w1 = bf16(rng.uniform(-bound, bound, (D, HID)))
    w2 = bf16(rng.uniform(-bound, bound, (HID, HID)))
    w3 = bf16(rng.uniform(-bound, bound, (HID, n_bits)))
    b1, b2 = (rng.uniform(-bound, bound, HID).astype(np.float32) for _ in range(2))
    b3 = rng.uniform(-bound, bound, n_bits).astype(np.float32)
    x = bf16(rng.standard_normal((50, D)))
    wide = oracle.encode_wide(x, w1, w2, w3, b1, b2, b3)
    for c in range(n_bits // 32):
        narrow = oracle.encode(x, w1, w2, np.ascontiguousarray(w3[:, 32 * c:32 * c + 32]), b1, b2, b3[32 * c:32 * c + 32])
        got = (wide[:, c // 2] >> np.uint64(32 * (c % 2))) & np.uint64(0xFFFFFFFF)
        assert np.array_equal(got.astype(np.uint32), narrow)


def test_float64_evaluation_agrees_outside_a_margin():
    rng = np.random.default_rng(31)
    n_bits = 128
    bound = 1.0 / np.sqrt(D)
    ws = [rng.uniform(-bound, bound, s) for s in ((D, HID), (HID, HID), (HID, n_bits))]
    bs = [rng.uniform(-bound, bound, s).astype(np.float32) for s in (HID, HID, n_bits)]
    wb = [bf16(w) for w in ws]
    x = bf16(rng.standard_normal((200, D)))
    codes, z3 = oracle.encode_wide(x, *wb, *bs, return_z3=True)
    f = lambda a: oracle.bf16_bits_to_f64(a)
    h = np.maximum(f(x) @ f(wb[0]) + bs[0], 0.0)
    h = np.maximum(h @ f(wb[1]) + bs[1], 0.0)
    z = h @ f(wb[2]) + bs[2]
    assert np.max(np.abs(z - z3)) < 1e-4
    for r in range(200):
        for j in range(n_bits):
            if abs(z[r, j]) > 1e-4:
                assert bit(codes[r], j) == int(z[r, j] > 0)


def test_group_score_is_the_maximum_of_the_pinned_single_query_scores():
    rng = np.random.default_rng(41)
    W = 2
    k = rng.integers(0, 2**63, size=(300, W), dtype=np.uint64)
    q = rng.integers(0, 2**63, size=(4, W), dtype=np.uint64)
    q[2] = k[17]                                                       # an exact match: score 128 for token 17
    s = oracle.score_wide_group(q, k)
    assert s[17] == 64 * W
    per_head = np.stack([oracle.score_wide(q[j], k) for j in range(4)])
    assert np.array_equal(s, per_head.max(axis=0))
    assert np.array_equal(oracle.score_wide_group(q[:1], k), per_head[0])
