"""Pins for the oracle's ENCODE (Eq. 2 with the Section 5.2 network): closed forms and an
independent float64 evaluation.  CPU only."""
import numpy as np
import torch

import oracle

D, HID, BITS = 128, 128, 32


def bf16(a):
    """float array -> bf16 bit patterns (round to nearest even, via torch)."""
    t = torch.as_tensor(np.asarray(a, dtype=np.float32)).to(torch.bfloat16)
    return t.view(torch.int16).numpy().view(np.uint16).copy()


def zeros_w():
    return (np.zeros((D, HID), np.uint16), np.zeros((HID, HID), np.uint16), np.zeros((HID, BITS), np.uint16))


def eye_w():
    return bf16(np.eye(D, HID)), bf16(np.eye(HID, HID)), bf16(np.eye(HID, BITS))


def unit(k, scale=1.0):
    x = np.zeros(D, np.float32)
    x[k] = scale
    return bf16(x)[None, :]


def test_identity_weights_give_sign_bits_of_input():
    rng = np.random.default_rng(1)
    x = rng.standard_normal((64, D)).astype(np.float32)
    x[0, :8] = 0.0                       # sign(0) -> bit 0
    xb = bf16(x)
    w1, w2, w3 = eye_w()
    codes = oracle.encode(xb, w1, w2, w3)
    xv = oracle.bf16_bits_to_f64(xb)
    for r in range(x.shape[0]):
        expect = 0
        for o in range(BITS):
            if xv[r, o] > 0:
                expect |= 1 << o
        assert int(codes[r]) == expect


def test_zero_weights_code_is_sign_pattern_of_last_bias():
    w1, w2, w3 = zeros_w()
    rng = np.random.default_rng(2)
    b3 = rng.standard_normal(BITS).astype(np.float32)
    b3[5] = 0.0
    b3[6] = -0.0
    x = bf16(rng.standard_normal((3, D)))
    codes = oracle.encode(x, w1, w2, w3, None, None, b3)
    expect = sum(1 << o for o in range(BITS) if b3[o] > 0)
    assert all(int(c) == expect for c in codes)


def test_zero_input_zero_bias_gives_zero_code():
    rng = np.random.default_rng(3)
    w1, w2, w3 = bf16(rng.standard_normal((D, HID))), bf16(rng.standard_normal((HID, HID))), bf16(rng.standard_normal((HID, BITS)))
    codes = oracle.encode(np.zeros((2, D), np.uint16), w1, w2, w3)
    assert codes.tolist() == [0, 0]


def test_single_path_pins_weight_orientation():
    # W[in][out]: x = e_k0 -> hidden o0 -> hidden p0 -> bit r0, all indices distinct and asymmetric
    k0, o0, p0, r0 = 3, 77, 101, 19
    w1, w2, w3 = (np.zeros((D, HID), np.float32), np.zeros((HID, HID), np.float32), np.zeros((HID, BITS), np.float32))
    w1[k0, o0] = 1.0
    w2[o0, p0] = 1.0
    w3[p0, r0] = 1.0
    codes = oracle.encode(unit(k0), bf16(w1), bf16(w2), bf16(w3))
    assert int(codes[0]) == 1 << r0
    # any other input coordinate reaches nothing
    assert int(oracle.encode(unit(o0), bf16(w1), bf16(w2), bf16(w3))[0]) == 0
    # transposed weights must NOT work with these asymmetric indices
    codes_t = oracle.encode(unit(k0), bf16(w1.T.copy()), bf16(w2.T.copy()), bf16(w3))
    assert int(codes_t[0]) == 0


def test_relu_sits_after_layer1_and_layer2_only():
    k0, o0, p0, r0 = 5, 9, 33, 2
    z = lambda: (np.zeros((D, HID), np.float32), np.zeros((HID, HID), np.float32), np.zeros((HID, BITS), np.float32))
    # layer-1 ReLU: z1 = -1 is clipped, so the (-1)(-1) path of a linear net never appears
    w1, w2, w3 = z()
    w1[k0, o0], w2[o0, p0], w3[p0, r0] = 1.0, -1.0, 1.0
    assert int(oracle.encode(unit(k0, -1.0), bf16(w1), bf16(w2), bf16(w3))[0]) == 0
    # layer-2 ReLU: z2 = -1 is clipped before the last layer
    w1, w2, w3 = z()
    w1[k0, o0], w2[o0, p0], w3[p0, r0] = 1.0, -1.0, -1.0
    assert int(oracle.encode(unit(k0, 1.0), bf16(w1), bf16(w2), bf16(w3))[0]) == 0
    # no activation after layer 3: a negative output is simply bit 0, a positive one bit 1
    w1, w2, w3 = z()
    w1[k0, o0], w2[o0, p0], w3[p0, r0], w3[p0, r0 + 1] = 1.0, 1.0, -1.0, 1.0
    assert int(oracle.encode(unit(k0, 1.0), bf16(w1), bf16(w2), bf16(w3))[0]) == 1 << (r0 + 1)


def test_biases_enter_every_layer():
    o0, p0, r0 = 11, 120, 31
    w1, w2, w3 = np.zeros((D, HID), np.float32), np.zeros((HID, HID), np.float32), np.zeros((HID, BITS), np.float32)
    w2[o0, p0], w3[p0, r0] = 1.0, 1.0
    b1 = np.zeros(HID, np.float32); b1[o0] = 1.0
    x0 = np.zeros((1, D), np.uint16)
    assert int(oracle.encode(x0, bf16(w1), bf16(w2), bf16(w3), b1, None, None)[0]) == 1 << r0
    b2 = np.zeros(HID, np.float32); b2[p0] = 0.5
    assert int(oracle.encode(x0, bf16(w1), bf16(w2), bf16(w3), None, b2, None)[0]) == 1 << r0
    b3 = np.zeros(BITS, np.float32); b3[7] = 1e-30
    assert int(oracle.encode(x0, bf16(w1), bf16(w2), bf16(w3), None, None, b3)[0]) == 1 << 7


def test_positive_homogeneity_without_bias():
    rng = np.random.default_rng(4)
    s = 1.0 / np.sqrt(D)
    w1, w2, w3 = bf16(rng.uniform(-s, s, (D, HID))), bf16(rng.uniform(-s, s, (HID, HID))), bf16(rng.uniform(-s, s, (HID, BITS)))
    x = rng.standard_normal((200, D)).astype(np.float32)
    c1 = oracle.encode(bf16(x), w1, w2, w3)
    c2 = oracle.encode(bf16(2.0 * oracle.bf16_bits_to_f64(bf16(x))), w1, w2, w3)   # x2 is exact in bf16 and fp32
    assert np.array_equal(c1, c2)
    assert len(set(c1.tolist())) > 1      # not a degenerate mapping


def test_matches_float64_matmul_outside_rounding_margin():
    rng = np.random.default_rng(5)
    s = 1.0 / np.sqrt(D)
    ws = [bf16(rng.uniform(-s, s, shp)) for shp in ((D, HID), (HID, HID), (HID, BITS))]
    bs = [rng.uniform(-s, s, n).astype(np.float32) for n in (HID, HID, BITS)]
    x = bf16(rng.standard_normal((512, D)))
    codes, z3 = oracle.encode(x, *ws, *bs, return_z3=True)
    W = [oracle.bf16_bits_to_f64(w) for w in ws]
    h = oracle.bf16_bits_to_f64(x)
    h = np.maximum(h @ W[0] + bs[0].astype(np.float64), 0.0)
    h = np.maximum(h @ W[1] + bs[1].astype(np.float64), 0.0)
    z = h @ W[2] + bs[2].astype(np.float64)
    assert np.max(np.abs(z - z3.astype(np.float64))) < 1e-4
    bits = (codes[:, None] >> np.arange(BITS, dtype=np.uint32)[None, :]) & 1
    safe = np.abs(z) > 1e-4
    assert safe.mean() > 0.95
    assert np.array_equal(bits[safe], (z > 0)[safe].astype(bits.dtype))


def test_bit_o_is_output_o_lsb_first():
    w1, w2, w3 = zeros_w()
    for o in (0, 1, 15, 31):
        b3 = np.full(BITS, -1.0, np.float32)
        b3[o] = 1.0
        c = oracle.encode(np.zeros((1, D), np.uint16), w1, w2, w3, None, None, b3)
        assert int(c[0]) == (1 << o)


def test_single_layer_sign_projection_special_case():
    # with identity hidden layers and non-negative inputs the net is x -> sign(x W3'), i.e. random
    # signed projections of the first layer's pass-through (Section 4.3 / LSH ablation)
    rng = np.random.default_rng(6)
    x = np.abs(rng.standard_normal((50, D))).astype(np.float32)
    w3 = rng.standard_normal((HID, BITS)).astype(np.float32)
    codes = oracle.encode(bf16(x), bf16(np.eye(D)), bf16(np.eye(D)), bf16(w3))
    z = oracle.bf16_bits_to_f64(bf16(x)) @ oracle.bf16_bits_to_f64(bf16(w3))
    bits = (codes[:, None] >> np.arange(BITS, dtype=np.uint32)[None, :]) & 1
    safe = np.abs(z) > 1e-3
    assert np.array_equal(bits[safe], (z > 0)[safe].astype(bits.dtype))
