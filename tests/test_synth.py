"""The seeded input generator: shapes, determinism, outlier structure (no GPU)."""
import numpy as np

from paper_2506_05413_b200 import synth


def test_config0_shape_and_outliers():
    a, b = synth.config0(), synth.config0()
    assert a.X.shape == (64, 128) and a.W.shape == (256, 128) and a.X_calib.shape == (128, 128)
    assert a.X.dtype == np.float16 and a.W.dtype == np.float16 and a.d.dtype == np.float32
    assert np.array_equal(a.X, b.X) and np.array_equal(a.W, b.W) and np.array_equal(a.d, b.d)
    assert set(np.unique(a.d)) == {-1.0, 1.0}
    x = np.abs(a.X.astype(np.float32))
    assert x[:4][:, [7, 93]].min() > 20 and np.median(x) < 1.0
    assert x[4:].max() < 10
    assert 0.015 < a.W.astype(np.float32).std() < 0.025


def test_larger_configs_reduced():
    c1 = synth.config1(M=200, N=16)
    assert c1.K == 4096 and len(c1.outlier_channels) == 4 and len(c1.outlier_tokens) == 2
    x = np.abs(c1.X.astype(np.float32))
    assert x[np.ix_(c1.outlier_tokens, c1.outlier_channels)].max() > 100
    c2 = synth.config2(M=100, N=8)
    assert c2.K == 14336 and np.array_equal(c2.d[:512], c2.d[512:1024]) and len(c2.outlier_channels) == 2
    assert np.isfinite(c2.X.astype(np.float32)).all()
    c4 = synth.config4("k_v", 4)
    assert c4.X.shape == (4, 4096) and c4.W.shape == (1024, 4096)
    # weights do not depend on the token count
    assert np.array_equal(synth.config1(M=8, N=16).W, c1.W)
