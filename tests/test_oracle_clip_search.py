"""Pins for the oracle's weight clip-ratio search (Experimental settings, "Quantization":
the ratio with the least squared quantization error among a scan of candidates).  CPU only."""
import numpy as np

from oracle import smoothrot_oracle as orc


def test_grid():
    r = orc.clip_ratios()
    assert r.dtype == np.float32 and len(r) == 51 and r[0] == np.float32(1.0) and r[-1] == np.float32(0.5)
    assert np.allclose(np.diff(r.astype(np.float64)), -0.01, atol=1e-7)


def _brute_force(row, ratios):
    """Plain Python loops, float32 decisions redone here step by step."""
    amax = np.float32(max(abs(float(x)) for x in row))
    errs = []
    for ratio in ratios:
        step = np.float32(np.float32(ratio) * amax) / np.float32(7.0)
        e = 0.0
        for x in row:
            q = np.rint(np.float32(x) / step)
            q = min(max(float(q), -8.0), 7.0)
            e += (float(np.float32(x)) - q * float(step)) ** 2
        errs.append(e)
    best = min(range(len(ratios)), key=lambda i: (errs[i], i))
    return best, errs


def test_search_equals_brute_force_on_small_rows():
    rng = np.random.default_rng(0)
    ratios = orc.clip_ratios()
    v = rng.standard_normal((6, 48)).astype(np.float32)
    v[1, 5] = 9.0          # one large value: clipping pays
    v[2] *= 1e-3
    codes, step, best, errs = orc.clip_search_rows(v, ratios)
    for r in range(v.shape[0]):
        b, e = _brute_force(v[r], ratios)
        assert b == best[r]
        assert np.allclose(errs[r], e, rtol=1e-12)
        want_codes, want_step = orc.quantize_rows(v[r:r + 1], ratios[b])
        assert np.array_equal(codes[r], want_codes[0]) and step[r] == want_step[0]


def test_ratio_one_is_plain_rtn_and_error_is_the_dequantization_error():
    rng = np.random.default_rng(1)
    v = rng.standard_normal((4, 256)).astype(np.float32)
    ratios = orc.clip_ratios()
    _, _, _, errs = orc.clip_search_rows(v, ratios)
    codes, step = orc.quantize_rows(v, 1.0)
    e = ((v.astype(np.float64) - orc.dequantize_rows(codes, step)) ** 2).sum(axis=1)
    assert np.allclose(errs[:, 0], e, rtol=1e-12)


def test_equal_magnitudes_keep_ratio_one_and_outliers_choose_a_smaller_ratio():
    ratios = orc.clip_ratios()
    flat = np.array([[3.5, -3.5] * 32], np.float32)          # +-max everywhere, step 0.5: exact at ratio 1
    codes, step, best, errs = orc.clip_search_rows(flat, ratios)
    assert best[0] == 0 and errs[0, 0] == 0.0 and set(np.unique(codes)) == {-7, 7}
    rng = np.random.default_rng(2)
    heavy = rng.standard_normal((1, 4096)).astype(np.float32)
    heavy[0, 17] = 25.0                                      # one far outlier among 4096 Gaussians
    _, _, best, errs = orc.clip_search_rows(heavy, ratios)
    assert best[0] > 0 and errs[0, best[0]] < errs[0, 0]
    # the chosen ratio is a true minimum of the sampled error curve
    assert errs[0, best[0]] == errs[0].min()


def test_search_is_scale_equivariant():
    rng = np.random.default_rng(3)
    v = rng.standard_normal((3, 512)).astype(np.float32)
    ratios = orc.clip_ratios()
    c1, s1, b1, e1 = orc.clip_search_rows(v, ratios)
    c2, s2, b2, e2 = orc.clip_search_rows(v * np.float32(4.0), ratios)     # exact scaling by a power of two
    assert np.array_equal(b1, b2) and np.array_equal(c1, c2)
    assert np.array_equal(s2, s1 * np.float32(4.0)) and np.allclose(e2, 16.0 * e1, rtol=1e-12)


def test_fuse_weights_search_reduces_to_fuse_weights_at_the_chosen_ratio():
    rng = np.random.default_rng(4)
    K = 256
    W = (rng.standard_normal((5, K)) * 0.02).astype(np.float16)
    W[3, 9] = 0.9
    pre = rng.uniform(0.5, 2.0, K).astype(np.float32)
    ratios = orc.clip_ratios()
    packed, step, best, errs, wr = orc.fuse_weights_search(W, pre, K, ratios)
    for r in range(W.shape[0]):
        p2, s2, _ = orc.fuse_weights(W[r:r + 1], pre, K, float(ratios[best[r]]))
        assert np.array_equal(packed[r], p2[0]) and step[r] == s2[0]
    assert np.all(errs.min(axis=1) == errs[np.arange(5), best])
