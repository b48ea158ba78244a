"""GPU-vs-oracle parity of the head-mixing online transform (smoothrot_quant_act_heads and its
rotation export), through the C-ABI binding.  Tolerances as in test_gpu_parity.py:
rotation 1e-5 of the row maximum, step sizes 1e-6, at most 1e-4 of the codes off by one."""
import numpy as np
import pytest

from oracle import smoothrot_oracle as orc
from paper_2506_05413_b200 import synth

pytestmark = pytest.mark.gpu

TOL_ROT = 1e-5
TOL_SCALE = 1e-6
TOL_CODES = 1e-4

SHAPES = [  # (n_heads, head_dim, M)
    (32, 128, 301),   # the 8B-class models: 32 heads of 128
    (32, 128, 1),
    (8, 64, 37),      # one warp per row
    (16, 256, 50),    # four warps per row
    (64, 128, 21),
    (8, 128, 2500),   # more rows than one pass of the grid
    (32, 64, 1200),
]


@pytest.fixture(scope="module")
def gu():
    from paper_2506_05413_b200 import build
    build.build()
    import gpu_util
    return gpu_util


def _attn_out(seed, M, K):
    """Attention outputs: N(0,1) with a few strong channels on a subset of the tokens."""
    rng = np.random.default_rng(seed)
    ch = np.sort(rng.choice(K, size=3, replace=False))
    return synth.activations(rng, M, K, law="normal", outlier_channels=ch, outlier_gain=200.0,
                             outlier_tokens=np.arange(0, M, 13))


def _pre(seed, K):
    rng = np.random.default_rng(seed)
    return (rng.uniform(0.05, 4.0, K) * (rng.integers(0, 2, K) * 2 - 1)).astype(np.float32)


def _gpu_rotate(gu, X, n_heads, pre):
    import torch
    from paper_2506_05413_b200 import binding as sr
    Xd = gu.dev(X)
    Y = torch.full(Xd.shape, float("nan"), dtype=torch.float32, device=gu.DEV)
    sr.debug_hadamard_heads(Xd, n_heads, gu.dev(pre) if pre is not None else None, Y)
    torch.cuda.synchronize()
    return Y.cpu().numpy()


def _gpu_quant(gu, X, n_heads, pre, clip):
    import torch
    from paper_2506_05413_b200 import binding as sr
    Xd = gu.dev(X)
    M, K = Xd.shape
    q = torch.full((M, K // 2), 0x5A, dtype=torch.uint8, device=gu.DEV)
    step = torch.full((M,), float("nan"), dtype=torch.float32, device=gu.DEV)
    sr.quant_act_heads(Xd, n_heads, gu.dev(pre) if pre is not None else None, clip, q, step)
    torch.cuda.synchronize()
    return q.cpu().numpy(), step.cpu().numpy()


@pytest.mark.parametrize("n_heads,head_dim,M", SHAPES)
@pytest.mark.parametrize("use_pre", [False, True])
def test_head_rotation_matches_oracle(gu, n_heads, head_dim, M, use_pre):
    K = n_heads * head_dim
    X = _attn_out(K + M, M, K)
    pre = _pre(K, K) if use_pre else None
    got = _gpu_rotate(gu, X, n_heads, pre)
    want = orc.rotate_heads(X, pre, n_heads)
    assert gu.rowwise_rel(got, want) <= TOL_ROT


@pytest.mark.parametrize("n_heads,head_dim,M", SHAPES)
@pytest.mark.parametrize("use_pre", [False, True])
def test_head_codes_match_oracle(gu, n_heads, head_dim, M, use_pre):
    K = n_heads * head_dim
    X = _attn_out(3 * K + M, M, K)
    pre = _pre(K + 1, K) if use_pre else None
    q, step = _gpu_quant(gu, X, n_heads, pre, 0.9)
    q_ref, step_ref, _ = orc.quant_act_heads(X, pre, n_heads, 0.9)
    assert np.abs(step / step_ref - 1).max() <= TOL_SCALE
    frac, worst = gu.code_mismatch(q, q_ref)
    assert worst <= 1 and frac <= max(TOL_CODES, 1.5 / q.size / 2)
    codes = orc.unpack_codes(q)
    assert codes.min() >= -8 and codes.max() <= 7


@pytest.mark.parametrize("clip", [0.5, 0.8, 0.83, 1.0])
def test_head_quantizer_clip_ratios_including_two_sided_saturation(gu, clip):
    n_heads, head_dim = 32, 128
    X = _attn_out(int(100 * clip), 29, n_heads * head_dim)
    q, step = _gpu_quant(gu, X, n_heads, None, clip)
    q_ref, step_ref, _ = orc.quant_act_heads(X, None, n_heads, clip)
    assert np.abs(step / step_ref - 1).max() <= TOL_SCALE
    frac, worst = gu.code_mismatch(q, q_ref)
    assert worst <= 1 and frac <= TOL_CODES
    if clip <= 0.8:
        assert orc.unpack_codes(q_ref).min() == -8 and orc.unpack_codes(q_ref).max() == 7


def test_head_quantizer_edge_rows_and_row_stride(gu):
    import torch
    from paper_2506_05413_b200 import binding as sr
    n_heads, head_dim = 32, 128
    K = n_heads * head_dim
    X = np.zeros((4, K), np.float16)
    X[1, 5 * head_dim + 17] = -2.0         # one value: every head gets +-2 / sqrt(32) at position 17
    X[2, :] = 65504.0                      # largest fp16 everywhere: head 0 collects all of it
    X[3] = _attn_out(9, 1, K)[0]
    q, step = _gpu_quant(gu, X, n_heads, None, 0.9)
    codes = orc.unpack_codes(q).reshape(4, n_heads, head_dim)
    assert step[0] == np.float32(1.0) and not codes[0].any()
    assert set(np.unique(codes[1][:, 17])) <= {7, -8} and not np.delete(codes[1], 17, axis=1).any()
    assert np.array_equal(codes[1][:, 17] == -8, orc.sylvester(n_heads)[5] > 0)
    assert np.all(codes[2][0] == 7) and not codes[2][1:].any() and np.all(np.isfinite(step))
    q_ref, step_ref, _ = orc.quant_act_heads(X, None, n_heads, 0.9)
    assert np.abs(step / step_ref - 1).max() <= TOL_SCALE
    # rows that are 64 values further apart than they are long
    big = torch.zeros((4, K + 64), dtype=torch.float16, device=gu.DEV)
    big[:, :K] = gu.dev(X)
    q2 = torch.empty((4, K // 2), dtype=torch.uint8, device=gu.DEV)
    s2 = torch.empty(4, dtype=torch.float32, device=gu.DEV)
    sr.quant_act_heads(big[:, :K], n_heads, None, 0.9, q2, s2)
    torch.cuda.synchronize()
    assert np.array_equal(q2.cpu().numpy(), q) and np.array_equal(s2.cpu().numpy(), step)


def test_head_codes_at_full_size_on_sampled_rows(gu):
    """8192 tokens of 32 heads x 128, the launch the sweep times (a grid of 2 CTAs per SM, every
    row group taking several rows): whole rows sampled across the range against the oracle, and
    properties that hold for every row."""
    n_heads, head_dim, M = 32, 128, 8192
    K = n_heads * head_dim
    X = _attn_out(2024, M, K)
    q, step = _gpu_quant(gu, X, n_heads, None, 0.9)
    assert np.all(np.isfinite(step)) and np.all(step > 0)
    rng = np.random.default_rng(11)
    rows = np.unique(np.concatenate([[0, 1, 3, 4, 295, 296, 1183, 1184, 1185, M - 2, M - 1],
                                     np.arange(0, M, 13)[:8], rng.integers(0, M, 48)]))
    q_ref, step_ref, _ = orc.quant_act_heads(X[rows], None, n_heads, 0.9)
    assert np.abs(step[rows] / step_ref - 1).max() <= TOL_SCALE
    frac, worst = gu.code_mismatch(q[rows], q_ref)
    assert worst <= 1 and frac <= TOL_CODES
    codes = orc.unpack_codes(q[::61])
    assert codes.min() >= -8 and codes.max() <= 7
    # the largest magnitude of a row lands on +7 or -8 (clip 0.9 puts it at 7.78 steps)
    assert np.all(np.abs(codes.astype(np.int16)).max(axis=1) >= 7)


def test_head_transform_then_per_head_factor_is_the_full_rotation(gu):
    """The two factors of the rotation, one on the GPU and one from the oracle, against the full
    rotation on the GPU: (I (x) H_dh)(H_h (x) I) = H_{h dh}."""
    n_heads, head_dim = 32, 128
    K = n_heads * head_dim
    X = _attn_out(77, 12, K)
    mixed = _gpu_rotate(gu, X, n_heads, None)
    full = gu.gpu_hadamard(X, None)
    assert gu.rowwise_rel(orc.rotate_per_head(mixed, head_dim), full.astype(np.float64)) <= 2 * TOL_ROT


def test_head_entry_points_reject_bad_arguments(gu):
    import torch
    from paper_2506_05413_b200 import binding as sr
    X = torch.zeros((4, 12 * 128), dtype=torch.float16, device=gu.DEV)
    q = torch.empty((4, 6 * 128), dtype=torch.uint8, device=gu.DEV)
    s = torch.empty(4, dtype=torch.float32, device=gu.DEV)
    with pytest.raises(sr.SmoothRotError) as e:
        sr.quant_act_heads(X, 12, None, 0.9, q, s)          # 12 heads: no Sylvester matrix
    assert e.value.status == -2
    X = torch.zeros((4, 32 * 128), dtype=torch.float16, device=gu.DEV)
    q = torch.empty((4, 16 * 128), dtype=torch.uint8, device=gu.DEV)
    with pytest.raises(sr.SmoothRotError) as e:
        sr.quant_act_heads(X, 32, None, 1.5, q, s)
    assert e.value.status == -1
    sr.quant_act_heads(X[:0], 32, None, 0.9, q[:0], s[:0])   # no rows: nothing to do
