"""GPU-vs-oracle parity of the fused decode layer (smoothrot_linear_decode: quant_act and linear in
one kernel for M <= 4 tokens of K = 4096), through the C-ABI binding.  Staged like the other parity
tests: the exported codes and steps against the oracle's activation path (steps 1e-6, at most 1e-4
of the codes off by one), the fp16 outputs against the oracle's layer fed the exported codes (2e-3
of the row maximum)."""
import numpy as np
import pytest

from oracle import smoothrot_oracle as orc
from paper_2506_05413_b200 import synth

pytestmark = pytest.mark.gpu

TOL_SCALE = 1e-6
TOL_CODES = 1e-4
TOL_OUT = 2e-3
K = 4096


@pytest.fixture(scope="module")
def gu():
    from paper_2506_05413_b200 import build
    build.build()
    import gpu_util
    return gpu_util


def _acts(seed, M):
    rng = np.random.default_rng(seed)
    ch = np.sort(rng.choice(K, size=4, replace=False))
    return synth.activations(rng, M, K, law="normal", outlier_channels=ch, outlier_gain=1000.0,
                             outlier_tokens=np.arange(0, M, 2))


def _weights(seed, N, width=K):
    rng = np.random.default_rng(seed)
    wq = orc.pack_codes(synth.random_codes(seed, N, width))
    dw = rng.uniform(1e-4, 4e-3, N).astype(np.float32)
    return wq, dw


def _run(gu, X, pre, clip, wq, dw, export=True, rotation=True):
    import torch
    from paper_2506_05413_b200 import binding as sr
    M, N = X.shape[0], wq.shape[0]
    Y = torch.full((M, N), float("nan"), dtype=torch.float16, device=gu.DEV)
    xq = torch.full((M, K // 2), 0x5A, dtype=torch.uint8, device=gu.DEV) if export else None
    dx = torch.full((M,), float("nan"), dtype=torch.float32, device=gu.DEV) if export else None
    sr.linear_decode(gu.dev(X), gu.dev(pre) if pre is not None else None, clip, gu.dev(wq), gu.dev(dw), Y, xq, dx,
                     rotation=rotation)
    torch.cuda.synchronize()
    return (Y.cpu().numpy(), xq.cpu().numpy() if export else None, dx.cpu().numpy() if export else None)


@pytest.mark.parametrize("M", [1, 2, 3, 4])
@pytest.mark.parametrize("N", [4096, 1000, 8, 14336])
@pytest.mark.parametrize("use_pre", [False, True])
def test_fused_decode_codes_and_outputs(gu, M, N, use_pre):
    X = _acts(10 * M + N, M)
    rng = np.random.default_rng(N)
    pre = (rng.uniform(0.02, 8.0, K) * (rng.integers(0, 2, K) * 2 - 1)).astype(np.float32) if use_pre else None
    wq, dw = _weights(N + M, N)
    Y, xq, dx = _run(gu, X, pre, 0.9, wq, dw)
    q_ref, step_ref, _ = orc.quant_act(X, pre, K, 0.9)
    assert np.abs(dx / step_ref - 1).max() <= TOL_SCALE
    frac, worst = gu.code_mismatch(xq, q_ref)
    assert worst <= 1 and frac <= max(TOL_CODES, 1.5 / xq.size / 2)
    want = orc.linear(xq, dx, wq, dw)                     # the oracle's layer on the kernel's own codes
    assert np.isfinite(Y.astype(np.float32)).all()
    assert gu.rowwise_rel(Y, want) <= TOL_OUT


def test_fused_decode_equals_the_two_call_path_on_its_own_codes(gu):
    """smoothrot_linear fed the codes and steps the fused kernel exports returns the same fp16
    outputs bit for bit (integer sums, same dequantization)."""
    import torch
    from paper_2506_05413_b200 import binding as sr
    M, N = 4, 4104
    X = _acts(5, M)
    wq, dw = _weights(6, N)
    Y, xq, dx = _run(gu, X, None, 0.9, wq, dw)
    Y2 = torch.empty((M, N), dtype=torch.float16, device=gu.DEV)
    sr.linear(gu.dev(xq), gu.dev(dx), gu.dev(wq), gu.dev(dw), Y2)
    torch.cuda.synchronize()
    assert np.array_equal(Y, Y2.cpu().numpy())
    # and without the optional exports the outputs are the same
    Y3, _, _ = _run(gu, X, None, 0.9, wq, dw, export=False)
    assert np.array_equal(Y, Y3)


@pytest.mark.parametrize("clip", [0.5, 0.8, 1.0])
def test_fused_decode_clip_ratios_and_edge_rows(gu, clip):
    X = _acts(77, 4)
    X[1, :] = 0                                # all zero: step 1, codes 0, outputs 0
    X[2, :] = 0
    X[2, 9] = -2.0                             # a unit vector: every code is +7 or -8
    wq, dw = _weights(8, 264)
    Y, xq, dx = _run(gu, X, None, clip, wq, dw)
    q_ref, step_ref, _ = orc.quant_act(X, None, K, clip)
    assert np.abs(dx / step_ref - 1).max() <= TOL_SCALE
    frac, worst = gu.code_mismatch(xq, q_ref)
    assert worst <= 1 and frac <= TOL_CODES
    codes = orc.unpack_codes(xq)
    assert dx[1] == np.float32(1.0) and not codes[1].any() and not Y[1].any()
    # the unit vector: |x^| / step = 7 / clip everywhere, so +-7 without clipping, +7 / -8 once it saturates
    assert set(np.unique(codes[2])) <= ({7, -7} if clip == 1.0 else {7, -8})
    assert gu.rowwise_rel(Y, orc.linear(xq, dx, wq, dw)) <= TOL_OUT


@pytest.mark.parametrize("M", [1, 3, 4, 8])
@pytest.mark.parametrize("N,width", [(4096, 4096), (1000, 4096), (14336, 4096), (264, 2048), (72, 1024)])
@pytest.mark.parametrize("use_pre", [False, True])
def test_fused_decode_without_rotation(gu, M, N, width, use_pre):
    """rotation = 0: the tokens take smoothrot_quant_act_plain's path; codes identical to the oracle's
    (correctly rounded quotient), outputs against the oracle's layer on those codes."""
    rng = np.random.default_rng(M + N + width)
    ch = np.sort(rng.choice(width, size=3, replace=False))
    X = synth.activations(rng, M, width, law="normal", outlier_channels=ch, outlier_gain=300.0,
                          outlier_tokens=np.arange(0, M, 3))
    X[M - 1, :] = 0 if M > 2 else X[M - 1, :]
    pre = (rng.uniform(0.02, 8.0, width) * (rng.integers(0, 2, width) * 2 - 1)).astype(np.float32) if use_pre else None
    wq, dw = _weights(N + M, N, width)
    import torch
    from paper_2506_05413_b200 import binding as sr
    Y = torch.full((M, N), float("nan"), dtype=torch.float16, device=gu.DEV)
    xq = torch.full((M, width // 2), 0x5A, dtype=torch.uint8, device=gu.DEV)
    dx = torch.full((M,), float("nan"), dtype=torch.float32, device=gu.DEV)
    sr.linear_decode(gu.dev(X), gu.dev(pre) if pre is not None else None, 0.9, gu.dev(wq), gu.dev(dw), Y, xq, dx,
                     rotation=False)
    torch.cuda.synchronize()
    Y, xq, dx = Y.cpu().numpy(), xq.cpu().numpy(), dx.cpu().numpy()
    q_ref, step_ref, _ = orc.quant_act_plain(X, pre, 0.9)
    assert np.abs(dx / step_ref - 1).max() <= TOL_SCALE
    frac, worst = gu.code_mismatch(xq, q_ref)
    assert worst <= 1 and frac <= max(TOL_CODES, 1.5 / xq.size / 2)
    assert np.isfinite(Y.astype(np.float32)).all()
    assert gu.rowwise_rel(Y, orc.linear(xq, dx, wq, dw)) <= TOL_OUT
    # the two-call path on the same inputs gives the same outputs bit for bit when the codes agree
    q2 = torch.empty((M, width // 2), dtype=torch.uint8, device=gu.DEV)
    s2 = torch.empty(M, dtype=torch.float32, device=gu.DEV)
    Y2 = torch.empty((M, N), dtype=torch.float16, device=gu.DEV)
    sr.quant_act_plain(gu.dev(X), gu.dev(pre) if pre is not None else None, 0.9, q2, s2)
    sr.linear(q2, s2, gu.dev(wq), gu.dev(dw), Y2)
    torch.cuda.synchronize()
    assert np.array_equal(q2.cpu().numpy(), xq) and np.array_equal(s2.cpu().numpy(), dx)
    assert np.array_equal(Y2.cpu().numpy(), Y)


@pytest.mark.parametrize("M", [1, 2, 3, 4])
@pytest.mark.parametrize("N", [4096, 1000, 14336])
@pytest.mark.parametrize("use_pre", [False, True])
def test_fused_decode_with_the_head_mixing_transform(gu, M, N, use_pre):
    """smoothrot_linear_decode_heads: the tokens take smoothrot_quant_act_heads' path (32 heads of 128)."""
    import torch
    from paper_2506_05413_b200 import binding as sr
    X = _acts(7 * M + N, M)
    rng = np.random.default_rng(N + 1)
    pre = (rng.uniform(0.05, 4.0, K) * (rng.integers(0, 2, K) * 2 - 1)).astype(np.float32) if use_pre else None
    wq, dw = _weights(N + 2 * M, N)
    pre_d = gu.dev(pre) if pre is not None else None
    Y = torch.full((M, N), float("nan"), dtype=torch.float16, device=gu.DEV)
    xq = torch.full((M, K // 2), 0x5A, dtype=torch.uint8, device=gu.DEV)
    dx = torch.full((M,), float("nan"), dtype=torch.float32, device=gu.DEV)
    sr.linear_decode_heads(gu.dev(X), 32, pre_d, 0.9, gu.dev(wq), gu.dev(dw), Y, xq, dx)
    torch.cuda.synchronize()
    Yh, xqh, dxh = Y.cpu().numpy(), xq.cpu().numpy(), dx.cpu().numpy()
    q_ref, step_ref, _ = orc.quant_act_heads(X, pre, 32, 0.9)
    assert np.abs(dxh / step_ref - 1).max() <= TOL_SCALE
    frac, worst = gu.code_mismatch(xqh, q_ref)
    assert worst <= 1 and frac <= max(TOL_CODES, 1.5 / xqh.size / 2)
    assert np.isfinite(Yh.astype(np.float32)).all()
    assert gu.rowwise_rel(Yh, orc.linear(xqh, dxh, wq, dw)) <= TOL_OUT
    # the two-call path (same arithmetic, call by call) gives the same codes and outputs
    q2 = torch.empty((M, K // 2), dtype=torch.uint8, device=gu.DEV)
    s2 = torch.empty(M, dtype=torch.float32, device=gu.DEV)
    Y2 = torch.empty((M, N), dtype=torch.float16, device=gu.DEV)
    sr.quant_act_heads(gu.dev(X), 32, pre_d, 0.9, q2, s2)
    sr.linear(q2, s2, gu.dev(wq), gu.dev(dw), Y2)
    torch.cuda.synchronize()
    assert np.array_equal(q2.cpu().numpy(), xqh) and np.array_equal(s2.cpu().numpy(), dxh)
    assert np.array_equal(Y2.cpu().numpy(), Yh)


def test_fused_decode_rejects_what_it_does_not_cover(gu):
    import torch
    from paper_2506_05413_b200 import binding as sr
    wq = torch.zeros((16, 2048), dtype=torch.uint8, device=gu.DEV)
    dw = torch.ones(16, device=gu.DEV)
    X5 = torch.zeros((5, K), dtype=torch.float16, device=gu.DEV)
    with pytest.raises(sr.SmoothRotError) as e:
        sr.linear_decode(X5, None, 0.9, wq, dw, torch.empty((5, 16), dtype=torch.float16, device=gu.DEV))
    assert e.value.status == -1                # more than 4 tokens
    X2 = torch.zeros((2, 2048), dtype=torch.float16, device=gu.DEV)
    wq2 = torch.zeros((16, 1024), dtype=torch.uint8, device=gu.DEV)
    with pytest.raises(sr.SmoothRotError) as e:
        sr.linear_decode(X2, None, 0.9, wq2, dw, torch.empty((2, 16), dtype=torch.float16, device=gu.DEV))
    assert e.value.status == -2                # K other than 4096
