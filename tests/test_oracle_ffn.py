"""Pins for the oracle's feed-forward block (Fig. 2: up/gate projection -> sigma(gate) (.) up ->
hadamard -> quantize -> down projection, Lambda^-1 in the up-projection and Lambda in the
down-projection, section "Methodology").  CPU only."""
import numpy as np
import pytest
from scipy.special import expit

from oracle import smoothrot_oracle as orc


def _block(seed, M, K1, I, N, outliers=True):
    rng = np.random.default_rng(seed)
    X = rng.standard_normal((M, K1)).astype(np.float16)
    Wg = (rng.standard_normal((I, K1)) * 0.05).astype(np.float16)
    Wu = (rng.standard_normal((I, K1)) * 0.05).astype(np.float16)
    Wd = (rng.standard_normal((N, I)) * 0.02).astype(np.float16)
    if outliers:                      # two channels of the gated product far above the rest
        Wu[[3, I - 5]] *= 40.0
        Wg[[3, I - 5]] *= 6.0
    d = np.where(rng.random(I) < 0.5, -1.0, 1.0).astype(np.float32)
    return X, Wg, Wu, Wd, d


def test_absorb_into_up_hand_example():
    W = np.array([[2.0, -4.0], [3.0, 9.0]])
    s = np.array([2.0, 3.0])
    assert np.array_equal(orc.absorb_into_up(W, s), np.array([[1.0, -2.0], [1.0, 3.0]]))
    assert orc.absorb_into_up(W.astype(np.float16), s.astype(np.float32)).dtype == np.float64


@pytest.mark.parametrize("I", [512, 28 * 16])
def test_transformed_block_equals_plain_block_before_quantization(I):
    """Eq. 2 through the channel-wise product: Lambda^-1 in W_up, Lambda (and the signs, and the
    rotation) in W_down leave the block's function unchanged, to 1e-10 in float64."""
    X, Wg, Wu, Wd, d = _block(1, 9, 128, I, 24)
    rng = np.random.default_rng(2)
    s = rng.uniform(0.05, 20.0, I)
    want = orc.ffn_plain_fp64(X, Wg, Wu, Wd)
    got = orc.ffn_transformed_fp64(X, Wg, Wu, Wd, s, d)
    assert np.abs(got - want).max() <= 1e-10 * np.abs(want).max()
    got1 = orc.ffn_transformed_fp64(X, Wg, Wu, Wd, s, None)
    assert np.abs(got1 - want).max() <= 1e-10 * np.abs(want).max()


def test_scaling_the_gate_half_instead_breaks_the_block():
    """The diagonal may only go into the up half: SiLU is not homogeneous, so Lambda^-1 in the gate
    projection does not give the gated product divided by s."""
    X, Wg, Wu, Wd, d = _block(3, 7, 128, 256, 16)
    rng = np.random.default_rng(4)
    s = rng.uniform(0.2, 5.0, 256)
    want = orc.ffn_plain_fp64(X, Wg, Wu, Wd)
    X64 = X.astype(np.float64)
    h_wrong = orc.glu_product(X64 @ orc.absorb_into_up(Wg, s).T, X64 @ Wu.astype(np.float64).T)
    wr = orc.rotate(Wd.astype(np.float64), s * d.astype(np.float64), 256)
    wrong = orc.rotate(h_wrong, d.astype(np.float64), 256) @ wr.T
    assert np.abs(wrong - want).max() > 1e-2 * np.abs(want).max()
    # written out independently of glu_product: silu(g / s) * u  !=  silu(g) * u / s
    g, u, sj = 1.5, -0.75, 3.0
    assert abs((g / sj) * expit(g / sj) * u - g * expit(g) * u / sj) > 0.05


def test_row_scaling_commutes_with_the_per_channel_quantizer():
    """Dividing an output channel by a power of two changes its step by that factor and none of
    its codes: absorbing Lambda^-1 into the up-projection costs no accuracy by itself."""
    rng = np.random.default_rng(5)
    W = (rng.standard_normal((12, 256)) * 0.05).astype(np.float16)
    c = 2.0 ** rng.integers(-3, 1, 12)     # dividing by c <= 1 keeps every fp16 weight normal
    q0, s0, _ = orc.fuse_weights(W, None, 256, 1.0)
    q1, s1, _ = orc.fuse_weights((W.astype(np.float64) / c[:, None]).astype(np.float16), None, 256, 1.0)
    assert np.array_equal(q0, q1)
    assert np.array_equal(s1, (s0.astype(np.float64) / c).astype(np.float32))


def test_ffn_calibrate_uses_the_gated_product_and_the_original_down_projection():
    X, Wg, Wu, Wd, _ = _block(6, 40, 128, 256, 16)
    h16, amax, s = orc.ffn_calibrate(X, Wg, Wu, Wd, 0.5)
    X64 = X.astype(np.float64)
    g, u = X64 @ Wg.astype(np.float64).T, X64 @ Wu.astype(np.float64).T
    h = g * expit(g) * u
    assert np.array_equal(h16, h.astype(np.float16))
    assert np.array_equal(amax, np.abs(h16.astype(np.float32)).max(axis=0))
    wmax = np.abs(Wd.astype(np.float64)).max(axis=0)
    want = np.sqrt(np.maximum(amax.astype(np.float64), orc.EPS) / np.maximum(wmax, orc.EPS))
    assert np.allclose(s, want, rtol=1e-6)
    # the outlier channels of the gated product get the largest scales
    assert set(np.argsort(s)[-2:]) == {3, 256 - 5}


def test_ffn_block_stages_and_output():
    X, Wg, Wu, Wd, d = _block(7, 24, 128, 256, 32)
    _, _, s = orc.ffn_calibrate(_block(8, 64, 128, 256, 32)[0], Wg, Wu, Wd, 0.5)
    r = orc.ffn_block(X, Wg, Wu, Wd, s, d)
    I = 256
    # the up half of the fused gate/up layer carries Lambda^-1, the gate half does not
    assert np.array_equal(r["W_up_abs"], (Wu.astype(np.float64) / s.astype(np.float64)[:, None]).astype(np.float16))
    wq_g, dw_g, _ = orc.fuse_weights(Wg, None, 128, 1.0)
    assert np.array_equal(r["wq_gu"][:I], wq_g) and np.array_equal(r["dw_gu"][:I], dw_g)
    # gate/up outputs approximate the unquantized projections (4-bit: coarse, but correlated)
    X64 = X.astype(np.float64)
    G = X64 @ Wg.astype(np.float64).T
    U = X64 @ orc.absorb_into_up(Wu, s).T
    Ygu = r["Y_gu"].astype(np.float64)
    assert np.linalg.norm(Ygu[:, :I] - G) < 0.3 * np.linalg.norm(G)
    assert np.linalg.norm(Ygu[:, I:] - U) < 0.3 * np.linalg.norm(U)
    # the online edge consumes exactly those fp16 halves, with the sign diagonal only
    hq, dh, _ = orc.quant_act_glu(r["Y_gu"][:, :I], r["Y_gu"][:, I:], d, I, 0.9)
    assert np.array_equal(hq, r["hq"]) and np.array_equal(dh, r["dh"])
    # the down-projection carries Lambda, the signs and the rotation
    assert np.array_equal(r["pre_w"], (s.astype(np.float64) * d).astype(np.float32))
    # end to end against the unquantized block
    want = orc.ffn_plain_fp64(X, Wg, Wu, Wd)
    err = np.linalg.norm(r["Y"].astype(np.float64) - want) / np.linalg.norm(want)
    assert err < 0.5


def test_smoothing_lowers_the_block_error_on_outlier_channels():
    """The direction of the paper's claim on the block as a whole: with massive outliers in the
    gated product, smoothing (alpha = 0.5) plus rotation gives a lower output error than rotation
    alone (s = 1)."""
    X, Wg, Wu, Wd, d = _block(9, 48, 128, 256, 32)
    Xc = _block(10, 96, 128, 256, 32)[0]
    _, _, s = orc.ffn_calibrate(Xc, Wg, Wu, Wd, 0.5)
    want = orc.ffn_plain_fp64(X, Wg, Wu, Wd)
    err = {}
    for name, sv in (("smooth", s), ("rotation only", np.ones_like(s))):
        r = orc.ffn_block(X, Wg, Wu, Wd, sv, d)
        err[name] = np.linalg.norm(r["Y"].astype(np.float64) - want) / np.linalg.norm(want)
    assert err["smooth"] < err["rotation only"]
