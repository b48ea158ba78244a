"""Pins for the oracle's quantizer, packing, calibration, integer GEMM and
dequantizer (no GPU): error bounds, closed forms, brute force, library cross-checks."""
import itertools

import numpy as np
import pytest

from oracle import smoothrot_oracle as orc


# ------------------------------------------------------------------ quantizer
def _rows(seed, R=7, C=256, scale=1.0):
    rng = np.random.default_rng(seed)
    v = (rng.standard_normal((R, C)) * scale).astype(np.float32)
    v[0, 3] = 90.0 * scale   # an outlier row
    return v


def test_weight_quantizer_error_at_most_half_step():
    v = _rows(0)
    codes, step = orc.quantize_rows(v, 1.0)
    assert codes.dtype == np.int8 and step.dtype == np.float32
    assert codes.min() >= -7 and codes.max() <= 7          # clip 1.0 never reaches -8
    assert np.all(np.abs(codes).max(axis=1) == 7)          # the row maximum maps to +-7
    err = np.abs(orc.dequantize_rows(codes, step) - v.astype(np.float64))
    assert np.all(err <= 0.5 * step[:, None].astype(np.float64) * (1 + 1e-6))
    assert np.allclose(step, np.abs(v).max(axis=1) / 7.0, rtol=1e-6)


def test_activation_quantizer_clip_and_saturation():
    v = _rows(1)
    clip = 0.9
    codes, step = orc.quantize_rows(v, clip)
    assert np.allclose(step, 0.9 * np.abs(v).max(axis=1) / 7.0, rtol=1e-6)
    assert codes.min() >= -8 and codes.max() <= 7
    t = v.astype(np.float64) / step[:, None].astype(np.float64)
    inside = (t >= -8.5) & (t <= 7.5)
    err = np.abs(orc.dequantize_rows(codes, step) - v.astype(np.float64))
    assert np.all(err[inside] <= 0.5 * step[:, None].astype(np.float64).repeat(v.shape[1], 1)[inside] * (1 + 1e-6))
    # beyond the representable range the code saturates
    assert np.all(codes[t > 7.5] == 7) and np.all(codes[t < -8.5] == -8)
    # the row maximum sits at 7 / 0.9 = 7.78 steps: +7 if positive, -8 if negative
    for r in range(v.shape[0]):
        j = np.abs(v[r]).argmax()
        assert codes[r, j] == (7 if v[r, j] > 0 else -8)


def test_quantizer_rounds_half_to_even_and_uses_signed_range():
    # step = 1 exactly: max = 7, clip 1.0
    v = np.array([[7.0, 0.5, 1.5, 2.5, -0.5, -1.5, -2.5, 3.49, -3.51, 6.5, -6.5, 0.0]], np.float32)
    codes, step = orc.quantize_rows(v, 1.0)
    assert step[0] == np.float32(1.0)
    assert codes[0].tolist() == [7, 0, 2, 2, 0, -2, -2, 3, -4, 6, -6, 0]
    # with clip 0.5 values beyond +-7.5 / -8.5 steps saturate at 7 / -8
    v = np.array([[14.0, -14.0, 7.0, -7.0, 8.4, -8.4, 1.0, -1.0]], np.float32)
    codes, step = orc.quantize_rows(v, 0.5)
    assert step[0] == np.float32(1.0)
    assert codes[0].tolist() == [7, -8, 7, -7, 7, -8, 1, -1]


def test_quantizer_all_zero_row_and_idempotence():
    v = _rows(2)
    v[3] = 0.0
    codes, step = orc.quantize_rows(v, 0.9)
    assert step[3] == np.float32(1.0) and np.all(codes[3] == 0)
    # re-quantizing the dequantized weights (clip 1.0) gives the same codes
    cw, sw = orc.quantize_rows(v, 1.0)
    deq = orc.dequantize_rows(cw, sw).astype(np.float32)
    cw2, sw2 = orc.quantize_rows(deq, 1.0)
    keep = np.abs(cw).max(axis=1) == 7
    assert np.array_equal(cw[keep], cw2[keep])


def test_quantizer_scale_equivariance():
    v = _rows(3)
    c1, s1 = orc.quantize_rows(v, 0.9)
    c2, s2 = orc.quantize_rows(v * np.float32(4.0), 0.9)    # exact power of two
    assert np.array_equal(c1, c2) and np.array_equal(s1 * np.float32(4.0), s2)
    c3, _ = orc.quantize_rows(-v, 1.0)
    c4, _ = orc.quantize_rows(v, 1.0)
    assert np.array_equal(c3, -c4)                          # odd symmetry when -8 is not reached


# -------------------------------------------------------------------- packing
def test_pack_layout_and_round_trip_over_all_bytes():
    pairs = np.array(list(itertools.product(range(-8, 8), repeat=2)), dtype=np.int8)  # (lo, hi)
    packed = orc.pack_codes(pairs)
    assert packed.shape == (256, 1) and len(set(packed[:, 0].tolist())) == 256
    for (lo, hi), b in zip(pairs.tolist(), packed[:, 0].tolist()):
        assert b & 0xF == lo % 16 and (b >> 4) == hi % 16
    assert np.array_equal(orc.unpack_codes(packed), pairs)
    allbytes = np.arange(256, dtype=np.uint8).reshape(1, 256)
    assert np.array_equal(orc.pack_codes(orc.unpack_codes(allbytes)), allbytes)
    # code 2i in the low nibble of byte i
    c = np.array([[1, -1, 7, -8]], np.int8)
    assert orc.pack_codes(c).tolist() == [[0xF1, 0x87]]


# ---------------------------------------------------------------- calibration
def test_calibration_closed_forms():
    rng = np.random.default_rng(4)
    X = (rng.standard_normal((50, 64)) * 3).astype(np.float16)
    W = (rng.standard_normal((40, 64)) * 0.05).astype(np.float16)
    amax = np.abs(X.astype(np.float64)).max(axis=0)
    wmax = np.abs(W.astype(np.float64)).max(axis=0)
    a0, s0 = orc.calibrate(X, W, 0.0)
    assert np.array_equal(a0, amax.astype(np.float32))
    assert np.allclose(s0, 1.0 / wmax, rtol=1e-6)
    _, s1 = orc.calibrate(X, W, 1.0)
    assert np.allclose(s1, amax, rtol=1e-6)
    _, sh = orc.calibrate(X, W, 0.5)
    assert np.allclose(sh, np.sqrt(amax / wmax), rtol=1e-6)
    assert np.allclose(sh.astype(np.float64) ** 2, s0.astype(np.float64) * s1, rtol=1e-5)
    _, s3 = orc.calibrate(X, W, 0.3)
    assert np.allclose(s3, np.exp(0.3 * np.log(amax) - 0.7 * np.log(wmax)), rtol=1e-6)
    # amax == wmax and alpha = 1/2  =>  s = 1
    _, su = orc.calibrate(W, W, 0.5)
    assert np.allclose(su, 1.0, rtol=1e-6)


def test_calibration_symmetries():
    rng = np.random.default_rng(5)
    X = (rng.standard_normal((30, 32)) * 2).astype(np.float16)
    W = (rng.standard_normal((20, 32)) * 0.1).astype(np.float16)
    alpha = 0.45
    _, s = orc.calibrate(X, W, alpha)
    _, s4 = orc.calibrate(X * np.float16(4.0), W, alpha)
    assert np.allclose(s4, s * 4.0 ** alpha, rtol=1e-6)
    perm = rng.permutation(32)
    _, sp = orc.calibrate(X[:, perm], W[:, perm], alpha)
    assert np.array_equal(sp, s[perm])
    # token order and batching do not matter (max is associative): bit-exact
    a_full = orc.channel_absmax(X)
    a_run = np.maximum(orc.channel_absmax(X[17:]), orc.channel_absmax(X[:17][::-1]))
    assert np.array_equal(a_full, a_run)
    # guards: dead channels do not produce inf or nan
    X0 = X.copy(); X0[:, 3] = 0
    W0 = W.copy(); W0[:, 5] = 0
    _, sg = orc.calibrate(X0, W0, 0.5)
    assert np.all(np.isfinite(sg)) and np.all(sg >= 1e-5)
    assert np.isclose(sg[3], np.sqrt(1e-5 / np.abs(W[:, 3].astype(np.float64)).max()), rtol=1e-5)


# ----------------------------------------------------------------------- GEMM
def test_gemm_brute_force_tiny():
    rng = np.random.default_rng(6)
    xq = rng.integers(-8, 8, (5, 12), dtype=np.int8)
    wq = rng.integers(-8, 8, (4, 12), dtype=np.int8)
    want = [[sum(int(xq[m, k]) * int(wq[n, k]) for k in range(12)) for n in range(4)] for m in range(5)]
    assert orc.gemm_i32(xq, wq).tolist() == want
    assert orc.gemm_i32_numpy(xq, wq).tolist() == want


def test_gemm_extremes_and_library_cross_check():
    K = 14336
    lo = np.full((3, K), -8, np.int8)
    hi = np.full((2, K), 7, np.int8)
    assert np.all(orc.gemm_i32(lo, lo) == 64 * K)
    assert np.all(orc.gemm_i32(lo, hi) == -56 * K)
    rng = np.random.default_rng(7)
    xq = rng.integers(-8, 8, (33, 1000), dtype=np.int8)
    wq = rng.integers(-8, 8, (47, 1000), dtype=np.int8)
    got = orc.gemm_i32(xq, wq)
    assert got.dtype == np.int32 and got.shape == (33, 47)
    assert np.array_equal(got, xq.astype(np.int64) @ wq.astype(np.int64).T)
    # transposed operands give the transposed result; the sum is bilinear
    assert np.array_equal(orc.gemm_i32(wq, xq), got.T)
    e = np.zeros((1, 1000), np.int8); e[0, 123] = 1
    assert np.array_equal(orc.gemm_i32(e, wq)[0], wq[:, 123].astype(np.int32))
    assert orc.gemm_i32(np.zeros((0, 8), np.int8), np.zeros((3, 8), np.int8)).shape == (0, 3)


# -------------------------------------------------------------------- dequant
def test_dequant_output_is_the_rounded_exact_product():
    acc = np.array([[3, -5], [1000, 917504]], np.int32)
    dx = np.array([0.5, 0.001], np.float32)
    dw = np.array([0.25, 2.0 ** -10], np.float32)
    y = orc.dequant_output(acc, dx, dw)
    assert y.dtype == np.float16
    assert float(y[0, 0]) == 0.375 and float(y[0, 1]) == -5 * 0.5 * 2.0 ** -10
    exact = acc.astype(np.float64) * dx.astype(np.float64)[:, None] * dw.astype(np.float64)[None, :]
    assert np.all(np.abs(y.astype(np.float64) - exact) <= np.abs(exact) * 2.0 ** -11)
    big = orc.dequant_output(np.array([[917504]], np.int32), np.array([1.0], np.float32), np.array([1.0], np.float32))
    assert np.isinf(big[0, 0])                              # IEEE overflow, not saturation


# ---------------------------------------------------------------- the quantizer without a rotation
def test_plain_activation_quantizer_worked_example_and_relation_to_the_rotated_path():
    # one row, maximum 7: with clip 1 the step is 1 and the codes are the rounded values themselves
    x = np.array([[7.0, -7.0, 0.49, 0.5, 1.5, 2.5, -0.5, -3.4]], np.float16)
    packed, step, v = orc.quant_act_plain(x, None, 1.0)
    assert step[0] == np.float32(1.0) and v.dtype == np.float32
    assert list(orc.unpack_codes(packed)[0]) == [7, -7, 0, 0, 2, 2, 0, -3]       # halves go to the even neighbour
    # clip 0.9: step 0.9, the maximum lands at 7.78 steps and saturates
    packed, step, _ = orc.quant_act_plain(x, None, 0.9)
    assert step[0] == np.float32(np.float32(0.9) * np.float32(7.0)) / np.float32(7.0)
    assert list(orc.unpack_codes(packed)[0][:2]) == [7, -8]
    # the diagonal multiplies before the quantizer: doubling every channel doubles the step, same codes
    rng = np.random.default_rng(0)
    X = rng.standard_normal((5, 64)).astype(np.float16)
    p1, s1, _ = orc.quant_act_plain(X, None, 0.9)
    p2, s2, _ = orc.quant_act_plain(X, np.full(64, 2.0, np.float32), 0.9)
    assert np.array_equal(p1, p2) and np.array_equal(s2, 2 * s1)
    # against the rotated path: rotating first and quantizing plainly is quant_act
    K = 128
    X = rng.standard_normal((4, K)).astype(np.float16)
    q_rot, s_rot, xr = orc.quant_act(X, None, K, 0.9)
    codes, s_plain = orc.quantize_rows(xr, 0.9)
    assert np.array_equal(orc.pack_codes(codes), q_rot) and np.array_equal(s_plain, s_rot)
    # a zero row and a per-channel diagonal with signs
    X = np.zeros((1, 16), np.float16)
    packed, step, _ = orc.quant_act_plain(X, None, 0.9)
    assert step[0] == np.float32(1.0) and not packed.any()
    X = np.ones((1, 8), np.float16)
    pre = np.array([1, -1, 2, -2, 3.5, -3.5, 7, -7], np.float32)
    packed, step, _ = orc.quant_act_plain(X, pre, 1.0)
    assert list(orc.unpack_codes(packed)[0]) == [1, -1, 2, -2, 4, -4, 7, -7]     # 3.5 -> 4 (even), -3.5 -> -4
