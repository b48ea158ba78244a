"""Pins for the oracle's gated-linear-unit input path (Fig. 2: sigma(gate) (.) up feeds the
online Hadamard and quantizer).  CPU only."""
import numpy as np
from scipy.special import expit

from oracle import smoothrot_oracle as orc


def test_silu_against_library_logistic_and_closed_forms():
    g = np.linspace(-30, 30, 2001)
    assert np.allclose(orc.silu(g), g * expit(g), rtol=1e-14, atol=1e-300)
    assert orc.silu(np.array([0.0]))[0] == 0.0
    # sigma(g) + sigma(-g) = 1  =>  silu(g) - silu(-g) = g
    assert np.allclose(orc.silu(g) - orc.silu(-g), g, rtol=0, atol=1e-13)
    # large arguments: silu(g) -> g, silu(-g) -> 0 from below
    assert abs(orc.silu(np.array([40.0]))[0] - 40.0) < 1e-15 * 40 + 1e-14
    assert -1e-15 < orc.silu(np.array([-40.0]))[0] <= 0.0
    # the minimum of silu sits near g = -1.2785 with value -0.27846
    grid = np.linspace(-2, -1, 100001)
    i = np.argmin(orc.silu(grid))
    assert abs(grid[i] + 1.27846) < 1e-4 and abs(orc.silu(grid)[i] + 0.278465) < 1e-6
    # no overflow warnings or NaNs at the ends of the fp16 range
    assert np.isfinite(orc.silu(np.array([-65504.0, 65504.0]))).all()


def test_glu_product_is_elementwise_and_uses_unrounded_values():
    rng = np.random.default_rng(0)
    g = rng.standard_normal((3, 8)).astype(np.float16)
    u = rng.standard_normal((3, 8)).astype(np.float16)
    want = np.array([[float(a) * expit(float(a)) * float(b) for a, b in zip(gr, ur)] for gr, ur in zip(g, u)])
    assert np.allclose(orc.glu_product(g, u), want, rtol=1e-14)
    assert orc.glu_product(g, u).dtype == np.float64


def test_quant_act_glu_reduces_to_quant_act_where_the_product_is_exact():
    """With gate = +30 (sigma = 1 to 1e-13) the gated product is 30 * up; choosing up so that
    30 * up is an fp16 number makes the fused path agree with quant_act on that fp16 matrix."""
    rng = np.random.default_rng(1)
    K = 512
    up = (rng.integers(-64, 65, size=(5, K)) / 32.0).astype(np.float16)      # multiples of 1/32
    gate = np.full((5, K), 30.0, np.float16)
    X = (30.0 * up.astype(np.float64)).astype(np.float16)
    assert np.array_equal(X.astype(np.float64), 30.0 * up.astype(np.float64))   # exact in fp16
    pre = rng.uniform(0.5, 2.0, K).astype(np.float32)
    q1, s1, r1 = orc.quant_act_glu(gate, up, pre, K, 0.9)
    q2, s2, r2 = orc.quant_act(X, pre, K, 0.9)
    assert np.allclose(r1, r2, rtol=1e-6, atol=1e-6)
    assert np.allclose(s1, s2, rtol=1e-6)
    assert (orc.unpack_codes(q1) != orc.unpack_codes(q2)).mean() < 1e-3


def test_quant_act_glu_zero_gate_or_zero_up_gives_zero_rows():
    K = 128
    z = np.zeros((2, K), np.float16)
    x = np.ones((2, K), np.float16)
    for gate, up in ((z, x), (x, z)):
        q, step, r = orc.quant_act_glu(gate, up, None, K, 0.9)
        assert np.all(r == 0) and np.all(step == 1.0) and np.all(orc.unpack_codes(q) == 0)


def test_quant_act_glu_single_active_channel_closed_form():
    """One non-zero product c at channel j: every rotated entry is +-c / sqrt(K), so with clip 0.9
    every code is +7 or -8 with the sign pattern of row j of H."""
    K, j = 256, 37
    gate = np.zeros((1, K), np.float16); up = np.zeros((1, K), np.float16)
    gate[0, j] = 2.0; up[0, j] = -3.0
    c = 2.0 * expit(2.0) * -3.0
    q, step, r = orc.quant_act_glu(gate, up, None, K, 0.9)
    H = orc.hadamard_matrix(K)
    assert np.allclose(r[0], c * H[j] / np.sqrt(K), rtol=1e-6)
    codes = orc.unpack_codes(q)[0]
    assert np.array_equal(codes == -8, H[j] > 0) and set(np.unique(codes)) <= {7, -8}
    assert abs(step[0] - np.float32(0.9 * abs(c) / np.sqrt(K)) / np.float32(7)) <= 1e-6 * step[0]
