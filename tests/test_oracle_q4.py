"""Pins for the oracle's bf16 rounding, 4-bit dequantisation, quantiser and quantised matmul.

Each check compares the C oracle with something fixed by the format or by
arithmetic: a library conversion, exact rational arithmetic, a brute-force
product with an explicit float matrix, or an invariant.
"""
from fractions import Fraction

import numpy as np
import torch

import npref
from oracle import q4d_oracle as orc
from workload import gen


# ------------------------------------------------------------------- bf16

def test_bf16_matches_library_conversion_on_fp32_inputs():
    rng = np.random.default_rng(1)
    v = np.concatenate([
        rng.standard_normal(20000).astype(np.float32),
        (rng.standard_normal(2000) * 1e-39).astype(np.float32),     # bf16 subnormals
        (rng.standard_normal(2000) * 1e37).astype(np.float32),
        np.array([0.0, -0.0, 1.0, -1.0, 3.3895314e38, 3.4e38, np.inf, -np.inf], dtype=np.float32),
    ])
    want = torch.from_numpy(v).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)
    got = orc.bf16_round(v.astype(np.float64))
    assert np.array_equal(got, want)


def test_bf16_ties_and_single_rounding():
    one = 0x3F80
    assert orc.bf16_round(np.array([1.0 + 2.0 ** -8]))[0] == one            # tie -> even (down)
    assert orc.bf16_round(np.array([1.0 + 3 * 2.0 ** -8]))[0] == one + 2    # tie -> even (up)
    assert orc.bf16_round(np.array([1.0 + 2.0 ** -8 + 2.0 ** -30]))[0] == one + 1  # above the tie: up
    assert orc.bf16_round(np.array([1.0 + 2.0 ** -8 - 2.0 ** -30]))[0] == one
    assert orc.bf16_round(np.array([-(1.0 + 2.0 ** -8 + 2.0 ** -30)]))[0] == 0x8000 | (one + 1)
    assert orc.bf16_round(np.array([float(2 ** 128)]))[0] == 0x7F80
    nan = orc.bf16_round(np.array([np.nan]))[0]
    assert (nan & 0x7F80) == 0x7F80 and (nan & 0x7F) != 0


def test_bf16_matches_integer_bit_rounding_on_doubles():
    rng = np.random.default_rng(2)
    v = rng.standard_normal(50000) * np.exp(rng.uniform(-20, 20, 50000))
    assert np.array_equal(orc.bf16_round(v), npref.bf16_bits(v))


def test_bf16_roundtrip_is_identity():
    bits = np.arange(0, 0x7F80, 7, dtype=np.uint16)
    assert np.array_equal(orc.bf16_round(orc.bf16_to_f64(bits)), bits)


# ----------------------------------------------------------------- dequant

def _bf(x):
    return int(torch.tensor(x, dtype=torch.float32).to(torch.bfloat16).view(torch.int16).item()) & 0xFFFF


def _f32_neighbours(w):
    w = np.float32(w)
    return np.nextafter(w, np.float32(np.inf)), np.nextafter(w, np.float32(-np.inf))


def test_dequant_is_correctly_rounded_scale_times_code_plus_bias():
    scales = [1.0, 0.0, -0.5, 3.140625, 1e-3, 2.0 ** -126, 2.0 ** -130, 1e30, 0.00665283203125]
    biases = [0.0, -0.0, 1.0, -0.0498046875, 1e-3, -3.0, 2.0 ** -127, 7.5e29, 255.0]
    for s in scales:
        for b in biases:
            sb, bb = _bf(s), _bf(b)
            q = np.zeros((1, 8), dtype=np.uint32)
            q[0, 0], q[0, 1] = 0x76543210, 0xFEDCBA98   # codes 0..15 in element order
            S = np.full((1, 1), sb, dtype=np.uint16)
            B = np.full((1, 1), bb, dtype=np.uint16)
            w = orc.dequant_q4(q, S, B)[0]
            sv = Fraction(float(orc.bf16_to_f64(np.array([sb]))[0]))
            bv = Fraction(float(orc.bf16_to_f64(np.array([bb]))[0]))
            for code in range(16):
                exact = sv * code + bv
                got = w[code]
                up, dn = _f32_neighbours(got)
                err = abs(Fraction(float(got)) - exact)
                assert err <= abs(Fraction(float(up)) - exact), (s, b, code)
                assert err <= abs(Fraction(float(dn)) - exact), (s, b, code)
            assert np.all(w[16:] == np.float32(float(bv)))  # code 0 -> bias exactly


def test_nibble_order_lowest_nibble_first_and_group_indexing():
    K = 128
    q = np.zeros((2, K // 8), dtype=np.uint32)
    for k in range(K):
        q[0, k >> 3] |= np.uint32((k % 16) << (4 * (k & 7)))
        q[1, k >> 3] |= np.uint32(((k * 7 + 3) % 16) << (4 * (k & 7)))
    S = np.array([[_bf(1.0), _bf(2.0)], [_bf(0.5), _bf(-1.0)]], dtype=np.uint16)
    B = np.array([[_bf(0.0), _bf(100.0)], [_bf(-4.0), _bf(0.25)]], dtype=np.uint16)
    w = orc.dequant_q4(q, S, B)
    k = np.arange(K)
    assert np.array_equal(w[0], np.where(k < 64, k % 16, 2.0 * (k % 16) + 100.0).astype(np.float32))
    c1 = (k * 7 + 3) % 16
    assert np.array_equal(w[1], np.where(k < 64, 0.5 * c1 - 4.0, -1.0 * c1 + 0.25).astype(np.float32))
    assert np.array_equal(npref.unpack_codes(q)[1], c1)


# --------------------------------------------------------------- quantiser

def test_quantiser_roundtrip_error_bound_and_flat_group():
    rng = np.random.default_rng(3)
    w = (rng.standard_normal((24, 256)) * 0.02).astype(np.float32)
    w[3, 64:128] = 0.0123          # flat group
    w[5, :64] = 0.0                # flat at zero
    q, s, b = orc.quantize_q4(w)
    d = orc.dequant_q4(q, s, b).astype(np.float64)
    sv = np.repeat(orc.bf16_to_f64(s), 64, axis=1)
    bv = np.repeat(orc.bf16_to_f64(b), 64, axis=1)
    codes = npref.unpack_codes(q)
    g = w.reshape(24, 4, 64).astype(np.float64)
    # interior codes are the nearest grid point: half a step, plus fp32 rounding slack
    interior = (codes > 0) & (codes < 15)
    err = np.abs(d - w)
    assert np.all(err[interior] <= 0.5 * sv[interior] * (1 + 1e-5) + 1e-9)
    # edge codes: the grid was built from bf16-rounded min and step, so allow their rounding error too
    lo, hi = g.min(-1), g.max(-1)
    slack = np.repeat(np.abs(orc.bf16_to_f64(b) - lo) + 15 * np.abs(orc.bf16_to_f64(s) - (hi - lo) / 15), 64, axis=1)
    assert np.all(err <= 0.5 * sv + slack + 1e-9)
    assert np.all(codes[3, 64:128] == 0) and s[3, 1] == 0x3F80
    assert np.allclose(d[3, 64:128], orc.bf16_to_f64(b)[3, 1])
    assert np.all(d[5, :64] == 0.0)
    assert codes.min() == 0 and codes.max() == 15


def test_workload_quantiser_is_bit_identical_to_oracle_quantiser():
    g = torch.Generator().manual_seed(5)
    w = torch.randn(96, 512, generator=g) * 0.02
    w[7, 128:192] = -0.5
    w[9] = w[9] * 1e-30
    q, s, b = gen.quantize_q4(w)
    qo, so, bo = orc.quantize_q4(w.numpy())
    assert np.array_equal(orc.to_np(q, np.uint32), qo)
    assert np.array_equal(orc.to_np(s), so)
    assert np.array_equal(orc.to_np(b), bo)


# ------------------------------------------------------------------ matmul

def test_matmul_equals_brute_force_with_explicit_float_matrix():
    q, s, b = (orc.to_np(t) for t in gen.random_q4(24, 192, "cpu", "pin-matmul"))
    q = q.view(np.uint32)
    rng = np.random.default_rng(4)
    x = orc.bf16_round(rng.standard_normal((3, 192)))
    W = orc.dequant_q4(q, s, b).astype(np.float64)     # explicit matrix
    X = orc.bf16_to_f64(x)
    want = np.zeros((3, 24))
    for r in range(3):
        for j in range(24):
            acc = 0.0
            for k in range(192):
                acc += W[j, k] * X[r, k]
            want[r, j] = acc
    got = orc.q4_matmul(q, s, b, x)
    assert np.array_equal(got, want)                   # same order, same precision: identical
    assert np.allclose(got, X @ npref.dense_matrix((q, s, b)).T, rtol=1e-13, atol=1e-15)


def test_matmul_one_hot_activation_selects_single_weights():
    q, s, b = (orc.to_np(t) for t in gen.random_q4(32, 128, "cpu", "pin-onehot"))
    q = q.view(np.uint32)
    W = orc.dequant_q4(q, s, b)
    for k in (0, 1, 7, 8, 63, 64, 127):
        x = np.zeros((2, 128))
        x[0, k] = 1.0
        x[1, k] = -2.0
        out = orc.q4_matmul(q, s, b, orc.bf16_round(x))
        assert np.array_equal(out[0], W[:, k].astype(np.float64))
        assert np.array_equal(out[1], -2.0 * W[:, k].astype(np.float64))


def test_matmul_batch_rows_are_independent():
    q, s, b = (orc.to_np(t) for t in gen.random_q4(48, 256, "cpu", "pin-batch"))
    q = q.view(np.uint32)
    rng = np.random.default_rng(6)
    x = orc.bf16_round(rng.standard_normal((16, 256)))
    full = orc.q4_matmul(q, s, b, x)
    for r in (0, 5, 15):
        assert np.array_equal(orc.q4_matmul(q, s, b, x[r:r + 1])[0], full[r])
