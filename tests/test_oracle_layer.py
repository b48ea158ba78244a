"""Whole-layer pins for the oracle (no GPU): the quantized layer approximates
the fp64 layer, and smoothing before rotation helps on massive outliers, which
is the direction the paper's central claim takes."""
import numpy as np

from oracle import smoothrot_oracle as orc
from paper_2506_05413_b200 import synth


def _layer_err(case, alpha, use_s=True):
    K = case.K
    X, W = case.X, case.W
    amax, s = orc.calibrate(case.X_calib, W, alpha)
    if not use_s:
        s = np.ones_like(s)
    d = case.d
    wq, dw, wr = orc.fuse_weights(W, (s * d).astype(np.float32), K, case.clip_w)
    xq, dx, xr = orc.quant_act(X, (d / s).astype(np.float32), K, case.clip_a)
    Y = orc.linear(xq, dx, wq, dw).astype(np.float64)
    Yref = X.astype(np.float64) @ W.astype(np.float64).T
    return np.linalg.norm(Y - Yref) / np.linalg.norm(Yref), np.abs(xr).max(), xr, wr, Yref


def test_config0_layer_is_close_to_fp64_and_preserves_function():
    case = synth.config0()
    err, xmax, xr, wr, Yref = _layer_err(case, 0.5)
    assert err < 0.25
    # before quantization the transformed pair reproduces X W^T (Eq. 2); xr, wr are float32
    Y1 = xr.astype(np.float64) @ wr.astype(np.float64).T
    assert np.abs(Y1 - Yref).max() <= 1e-5 * np.abs(Yref).max()
    out = orc.smoothrot_layer(case.X, case.X_calib, case.W, case.d, 0.5)
    assert out["Y"].shape == (64, 256) and out["Y"].dtype == np.float16
    assert out["xq"].shape == (64, 64) and out["wq"].shape == (256, 64)
    assert np.array_equal(out["acc"], orc.gemm_i32_numpy(orc.unpack_codes(out["xq"]), orc.unpack_codes(out["wq"])))


def test_smoothing_before_rotation_beats_rotation_alone_on_massive_outliers():
    case = synth.config0()
    e_smooth, m_smooth, *_ = _layer_err(case, 0.5, use_s=True)
    e_rot, m_rot, *_ = _layer_err(case, 0.5, use_s=False)
    assert e_smooth < e_rot
    case1 = synth.config1(M=64, N=128)
    # the outlier tokens are the ones the method is about: measure on them
    e1s, *_ = _layer_err(case1, 0.5, True)
    e1r, *_ = _layer_err(case1, 0.5, False)
    assert e1s < e1r
