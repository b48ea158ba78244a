"""Pins for the oracle's head-mixing rotation (the online Hadamard transform in front of the
attention output projection; Methodology section, by reference to QuaRot).  CPU only."""
import numpy as np

from oracle import smoothrot_oracle as orc


def test_worked_example_two_heads_of_two():
    # heads (a, b) and (c, d): the transform adds and subtracts the heads, value by value
    x = np.array([[1.0, 2.0, 10.0, 20.0]])
    y = orc.rotate_heads(x, None, 2)
    want = np.array([[11.0, 22.0, -9.0, -18.0]]) / np.sqrt(2.0)
    assert np.allclose(y, want, rtol=0, atol=1e-15)
    # the per-head factor works inside each head instead
    z = orc.rotate_per_head(x, 2)
    assert np.allclose(z, np.array([[3.0, -1.0, 30.0, -10.0]]) / np.sqrt(2.0), rtol=0, atol=1e-15)


def test_equals_the_dense_kronecker_product():
    rng = np.random.default_rng(1)
    for n_heads, head_dim in ((4, 3), (8, 5), (2, 7)):
        K = n_heads * head_dim
        x = rng.standard_normal((6, K))
        pre = rng.uniform(0.5, 2.0, K)
        Hh = np.array([[(-1) ** bin(i & j).count("1") for j in range(n_heads)] for i in range(n_heads)], float)
        dense = np.kron(Hh, np.eye(head_dim)) / np.sqrt(n_heads)
        assert np.allclose(orc.rotate_heads(x, pre, n_heads), (x * pre) @ dense, rtol=1e-13, atol=1e-13)
        # the wrong factor order would be I (x) H: it must differ
        wrong = np.kron(np.eye(head_dim), Hh) / np.sqrt(n_heads)
        assert not np.allclose(orc.rotate_heads(x, pre, n_heads), (x * pre) @ wrong, atol=1e-3)


def test_product_of_the_two_factors_is_the_full_rotation():
    # (I (x) H_dh)(H_h (x) I) = H_h (x) H_dh = the Sylvester matrix of order h * dh
    rng = np.random.default_rng(2)
    for n_heads, head_dim in ((8, 16), (32, 128), (4, 64)):
        K = n_heads * head_dim
        x = rng.standard_normal((3, K))
        both = orc.rotate_heads(orc.rotate_per_head(x, head_dim), None, n_heads)
        other_order = orc.rotate_per_head(orc.rotate_heads(x, None, n_heads), head_dim)
        full = orc.rotate(x, None, K)
        assert np.allclose(both, full, rtol=1e-12, atol=1e-12)
        assert np.allclose(other_order, full, rtol=1e-12, atol=1e-12)


def test_orthogonal_and_an_involution():
    rng = np.random.default_rng(3)
    x = rng.standard_normal((5, 32 * 128))
    y = orc.rotate_heads(x, None, 32)
    assert np.allclose(np.linalg.norm(y, axis=1), np.linalg.norm(x, axis=1), rtol=1e-12)
    assert np.allclose(orc.rotate_heads(y, None, 32), x, rtol=1e-12, atol=1e-12)     # H symmetric, H H = n I
    assert np.array_equal(orc.rotate_heads(x, None, 1), x)                            # one head: nothing to mix


def test_a_spike_in_one_head_spreads_over_all_heads_at_the_same_position():
    n_heads, head_dim = 32, 128
    x = np.zeros((1, n_heads * head_dim))
    x[0, 5 * head_dim + 17] = 64.0
    y = orc.rotate_heads(x, None, n_heads).reshape(n_heads, head_dim)
    assert np.allclose(np.abs(y[:, 17]), 64.0 / np.sqrt(32.0), rtol=1e-15)
    y[:, 17] = 0
    assert not y.any()
    # signs: column 5 of the Sylvester matrix
    signs = np.sign(orc.rotate_heads(x, None, n_heads).reshape(n_heads, head_dim)[:, 17])
    assert np.array_equal(signs, orc.sylvester(32)[5].astype(float))


def test_quant_act_heads_is_the_row_quantizer_on_the_mixed_heads():
    rng = np.random.default_rng(4)
    n_heads, head_dim = 8, 16
    X = rng.standard_normal((9, n_heads * head_dim)).astype(np.float16)
    X[3, 2 * head_dim + 1] = 300.0
    packed, step, xr = orc.quant_act_heads(X, None, n_heads, 0.9)
    assert xr.dtype == np.float32 and packed.shape == (9, 64)
    amax = np.abs(xr).max(axis=1)
    assert np.allclose(step, np.float32(0.9) * amax / 7, rtol=1e-6)
    codes = orc.unpack_codes(packed)
    assert codes.min() >= -8 and codes.max() <= 7
    inside = np.abs(xr) <= 7.5 * step[:, None]
    assert np.all(np.abs(codes * step[:, None] - xr)[inside] <= step[:, None].repeat(xr.shape[1], 1)[inside] * 0.5000001)
    # the spike row: every head carries +-300 / sqrt(8) at position 1, clipped to the ends of the code range
    assert set(np.unique(codes[3].reshape(n_heads, head_dim)[:, 1])) <= {-8, 7}
