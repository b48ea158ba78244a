"""GPU-vs-oracle parity of the activation quantizer without a rotation (smoothrot_quant_act_plain),
through the C-ABI binding.  The scaled values are products of an fp16 and an fp32 number rounded to
fp32 on both sides, so the steps must agree to 1e-6 and the codes may differ (by one) only where
x / step lands within an ulp of a rounding boundary: at most 1e-4 of them."""
import numpy as np
import pytest

from oracle import smoothrot_oracle as orc
from paper_2506_05413_b200 import synth

pytestmark = pytest.mark.gpu

TOL_SCALE = 1e-6
TOL_CODES = 1e-4


@pytest.fixture(scope="module")
def gu():
    from paper_2506_05413_b200 import build
    build.build()
    import gpu_util
    return gpu_util


def _acts(seed, M, K):
    rng = np.random.default_rng(seed)
    ch = np.sort(rng.choice(K, size=min(3, K), replace=False))
    return synth.activations(rng, M, K, law="normal", outlier_channels=ch, outlier_gain=300.0,
                             outlier_tokens=np.arange(0, M, 11))


def _pre(seed, K):
    rng = np.random.default_rng(seed)
    return (rng.uniform(0.02, 8.0, K) * (rng.integers(0, 2, K) * 2 - 1)).astype(np.float32)


@pytest.mark.parametrize("K,M", [(4096, 301), (4096, 1), (128, 64), (8, 5), (1000, 33), (5120, 40), (8192, 7),
                                 (14336, 19), (16384, 3), (4096, 2500)])
@pytest.mark.parametrize("use_pre", [False, True])
def test_plain_codes_match_oracle(gu, K, M, use_pre):
    from paper_2506_05413_b200 import binding as sr
    X = _acts(K + M, M, K)
    pre = _pre(K, K) if use_pre else None
    q, step = gu.gpu_quantize(sr.quant_act_plain, X, pre, 0.9)
    q_ref, step_ref, _ = orc.quant_act_plain(X, pre, 0.9)
    assert np.abs(step / step_ref - 1).max() <= TOL_SCALE
    frac, worst = gu.code_mismatch(q, q_ref)
    assert worst <= 1 and frac <= max(TOL_CODES, 1.5 / q.size / 2)
    if not use_pre:
        assert np.array_equal(step, step_ref)          # no arithmetic before the maximum: identical
    codes = orc.unpack_codes(q)
    assert codes.min() >= -8 and codes.max() <= 7


@pytest.mark.parametrize("clip", [0.5, 0.8, 0.83, 1.0])
def test_plain_quantizer_clip_ratios_and_edge_rows(gu, clip):
    import torch
    from paper_2506_05413_b200 import binding as sr
    K = 4096
    X = _acts(int(100 * clip), 23, K)
    X[1, :] = 0
    X[2, :] = 65504.0
    X[3, :] = 0
    X[3, 77] = -3.0
    q, step = gu.gpu_quantize(sr.quant_act_plain, X, None, clip)
    q_ref, step_ref, _ = orc.quant_act_plain(X, None, clip)
    assert np.array_equal(step, step_ref)
    frac, worst = gu.code_mismatch(q, q_ref)
    assert worst <= 1 and frac <= TOL_CODES
    codes = orc.unpack_codes(q)
    assert step[1] == np.float32(1.0) and not codes[1].any()
    assert np.all(codes[2] == 7) and codes[3, 77] == (-8 if clip < 0.95 else -7) and np.count_nonzero(codes[3]) == 1
    # rows further apart than they are long
    big = torch.zeros((23, K + 64), dtype=torch.float16, device=gu.DEV)
    big[:, :K] = gu.dev(X)
    q2 = torch.empty((23, K // 2), dtype=torch.uint8, device=gu.DEV)
    s2 = torch.empty(23, dtype=torch.float32, device=gu.DEV)
    sr.quant_act_plain(big[:, :K], None, clip, q2, s2)
    torch.cuda.synchronize()
    assert np.array_equal(q2.cpu().numpy(), q) and np.array_equal(s2.cpu().numpy(), step)


def test_plain_quantizer_at_full_size_on_sampled_rows(gu):
    from paper_2506_05413_b200 import binding as sr
    M, K = 8192, 4096
    X = _acts(31, M, K)
    pre = _pre(32, K)
    q, step = gu.gpu_quantize(sr.quant_act_plain, X, pre, 0.9)
    rows = np.unique(np.concatenate([[0, 1, 3, 4, 295, 296, 1183, 1184, M - 2, M - 1],
                                     np.random.default_rng(5).integers(0, M, 54)]))
    q_ref, step_ref, _ = orc.quant_act_plain(X[rows], pre, 0.9)
    assert np.abs(step[rows] / step_ref - 1).max() <= TOL_SCALE
    frac, worst = gu.code_mismatch(q[rows], q_ref)
    assert worst <= 1 and frac <= TOL_CODES
    assert np.all(step > 0) and np.all(np.isfinite(step))
