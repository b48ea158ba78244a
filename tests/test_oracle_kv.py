"""Pins for the oracle's KV-cache quantizer (Eq. 1, asymmetric form; group 128, clip 0.95).  CPU only."""
import numpy as np

from oracle import smoothrot_oracle as orc


def test_values_on_the_grid_are_reproduced_exactly():
    # lo = -1, step = 0.25, 16 levels: -1, -0.75, ..., 2.75; clip 1 keeps the range
    levels = -1.0 + 0.25 * np.arange(16)
    x = np.tile(levels, 8).astype(np.float16)[None, :]            # one group of 128
    codes, step, zero = orc.kv_quantize(x, clip=1.0)
    assert step[0, 0] == np.float32(0.25) and zero[0, 0] == np.float32(4.0)     # -(-1 / 0.25)
    assert np.array_equal(codes[0], np.tile(np.arange(16), 8))
    assert np.array_equal(orc.kv_dequantize(codes, step, zero)[0], x[0].astype(np.float64))


def test_error_bound_inside_the_clipped_range_and_saturation_outside():
    rng = np.random.default_rng(0)
    x = rng.standard_normal((7, 512)).astype(np.float16)
    x[2, 5] = 40.0
    for clip in (1.0, 0.95, 0.7):
        codes, step, zero = orc.kv_quantize(x, clip)
        assert codes.min() >= 0 and codes.max() <= 15
        assert np.array_equal(zero, np.rint(zero))
        deq = orc.kv_dequantize(codes, step, zero)
        xv = x.astype(np.float64).reshape(7, 4, 128)
        d = np.abs(deq.reshape(7, 4, 128) - xv)
        st = step.astype(np.float64)[:, :, None]
        lo_rep = (0 - zero.astype(np.float64))[:, :, None] * st       # smallest representable value
        hi_rep = (15 - zero.astype(np.float64))[:, :, None] * st
        inside = (xv >= lo_rep - st / 2) & (xv <= hi_rep + st / 2)
        assert np.all(d[inside] <= st.repeat(128, axis=2)[inside] * (0.5 + 1e-6))
        # outside the representable range the code saturates at an end
        c3 = codes.reshape(7, 4, 128)
        assert np.all(c3[xv > hi_rep + st / 2] == 15) and np.all(c3[xv < lo_rep - st / 2] == 0)
        if clip == 1.0:
            assert inside.all()        # without clipping every value is inside (up to rounding of the ends)


def test_groups_are_independent_and_the_step_follows_eq1():
    rng = np.random.default_rng(1)
    x = rng.standard_normal((3, 256)).astype(np.float16)
    c_all, s_all, z_all = orc.kv_quantize(x, 0.95)
    for g in range(2):
        c, s, z = orc.kv_quantize(x[:, 128 * g:128 * (g + 1)], 0.95)
        assert np.array_equal(c, c_all[:, 128 * g:128 * (g + 1)])
        assert np.array_equal(s[:, 0], s_all[:, g]) and np.array_equal(z[:, 0], z_all[:, g])
    xv = x.astype(np.float64).reshape(3, 2, 128)
    want = 0.95 * (xv.max(axis=2) - xv.min(axis=2)) / 15
    assert np.allclose(s_all, want, rtol=1e-6)
    assert np.allclose(z_all, -np.rint(0.95 * xv.min(axis=2) / s_all), atol=1.0)


def test_degenerate_groups():
    x = np.zeros((1, 256), np.float16)
    x[0, 128:] = 3.0                                        # a constant non-zero group
    codes, step, zero = orc.kv_quantize(x, 0.95)
    assert step[0, 0] == 1.0 and zero[0, 0] == 0.0 and np.all(codes[0, :128] == 0)
    assert step[0, 1] == 1.0
    deq = orc.kv_dequantize(codes, step, zero)
    assert np.all(deq[0, :128] == 0.0)
    # constant group c = 3 with step 1: lo = 2.85 -> zero = -3, code = clamp(3 - 3) = 0 -> dequantized 3
    assert zero[0, 1] == -3.0 and np.all(codes[0, 128:] == 0) and np.all(deq[0, 128:] == 3.0)


def test_half_to_even_and_nibble_packing():
    # step 1 (lo = 0, hi = 15): x = 0.5, 1.5, 2.5 round to 0, 2, 2
    x = np.zeros((1, 128), np.float16)
    x[0, :4] = [15.0, 0.5, 1.5, 2.5]
    codes, step, zero = orc.kv_quantize(x, 1.0)
    assert step[0, 0] == 1.0 and zero[0, 0] == 0.0
    assert list(codes[0, :4]) == [15, 0, 2, 2]
    all_codes = np.arange(256, dtype=np.uint8)[None, :] % 16
    packed = orc.pack_nibbles(all_codes)
    assert packed.shape == (1, 128) and packed[0, 0] == (0 | (1 << 4)) and packed[0, 7] == (14 | (15 << 4))
    assert np.array_equal(orc.unpack_nibbles(packed), all_codes)
