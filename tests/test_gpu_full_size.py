"""Parity at the full workload sizes, in the launch configuration the benchmark times.

The oracle cannot redo a whole 8192 x 28672 x 4096 layer in seconds, so every stage is
checked on what it can compute one by one (staged: each oracle stage is fed the GPU's
upstream outputs, as in test_gpu_parity.py):

  * calibration: the per-channel maxima in full (exact), the scales in full (1e-6);
  * fuse_weights / quant_act: a seeded sample of whole rows (rows are independent),
    always including rows that carry the massive outliers: step sizes to 1e-6,
    codes equal except at most 1e-4 of them off by one;
  * the GEMM: the int32 accumulators of 64 whole rows and 64 whole columns of the output,
    chosen to include the first and last row/column of tiles, bit-exact;
  * the fp16 output: the same rows (within 2e-3 of the row maximum) and columns (each entry
    within one fp16 rounding of the exact product);
  * properties that hold at any size: every output finite, every step size positive.

The token-count sweep (decode shapes) is checked in full for every M it covers here.
"""
import numpy as np
import pytest

from oracle import smoothrot_oracle as orc
from paper_2506_05413_b200 import synth

pytestmark = pytest.mark.gpu

TOL_SCALE = 1e-6
TOL_CODES = 1e-4
TOL_OUT = 2e-3


@pytest.fixture(scope="module")
def env():
    import torch
    from paper_2506_05413_b200 import build, binding as sr
    build.build()
    sr.load()
    return torch, sr


def _t(torch, a):
    return torch.from_numpy(np.ascontiguousarray(a)).to("cuda:0")


def _run_layer(torch, sr, case):
    """The bench step on the device, plus the int32 export of the GEMM; returns device tensors."""
    dev = "cuda:0"
    M, N, K = case.M, case.N, case.K
    X, Xc, W, d = (_t(torch, a) for a in (case.X, case.X_calib, case.W, case.d))
    f32 = lambda n: torch.empty(n, dtype=torch.float32, device=dev)
    amax = torch.zeros(K, dtype=torch.float32, device=dev)
    s, pre_w, pre_x, dw, dx = f32(K), f32(K), f32(K), f32(N), f32(M)
    wq = torch.empty((N, K // 2), dtype=torch.uint8, device=dev)
    xq = torch.empty((M, K // 2), dtype=torch.uint8, device=dev)
    Y = torch.full((M, N), float("nan"), dtype=torch.float16, device=dev)
    need = sr.workspace_bytes(M, N, K)
    ws = torch.empty(need, dtype=torch.uint8, device=dev) if need else None
    sr.calibrate(Xc, amax, W=W, alpha=case.alpha, s_out=s, d=d, pre_w_out=pre_w, pre_x_out=pre_x)
    sr.fuse_weights(W, pre_w, case.clip_w, wq, dw)
    sr.quant_act(X, pre_x, case.clip_a, xq, dx)
    sr.linear(xq, dx, wq, dw, Y, ws)
    acc = torch.full((M, N), -7777, dtype=torch.int32, device=dev)
    sr.debug_gemm_i32(xq, wq, acc, ws)
    torch.cuda.synchronize()
    assert sr.device_status() == 0
    return dict(amax=amax, s=s, pre_w=pre_w, pre_x=pre_x, wq=wq, dw=dw, xq=xq, dx=dx, Y=Y, acc=acc)


def _sample(rng, n, count, always=()):
    """`count` indices below n: tile edges, the given ones, and a seeded rest."""
    edges = [0, 1, 31, 32, 127, 128, 129, 255, 256, 257, n - 257, n - 256, n - 129, n - 128, n - 2, n - 1]
    picked = {int(i) for i in list(always) + edges if 0 <= i < n}
    for i in rng.permutation(n):
        if len(picked) >= min(count, n):
            break
        picked.add(int(i))
    return np.array(sorted(picked), dtype=np.int64)


def _codes_ok(got_packed, ref_packed):
    a = orc.unpack_codes(got_packed).astype(np.int16)
    b = orc.unpack_codes(ref_packed).astype(np.int16)
    diff = np.abs(a - b)
    return int(diff.max()), float((diff != 0).mean())


def _rowwise_rel(got, want):
    g, w = np.asarray(got, np.float64), np.asarray(want, np.float64)
    den = np.abs(w).max(axis=1)
    den = np.where(den == 0, 1.0, den)
    return float((np.abs(g - w).max(axis=1) / den).max())


def _check_full_size(torch, sr, case, seed):
    g = _run_layer(torch, sr, case)
    M, N, K = case.M, case.N, case.K
    rng = np.random.default_rng(seed)
    # calibration in full
    amax_ref, s_ref = orc.calibrate(case.X_calib, case.W, case.alpha)
    assert np.array_equal(g["amax"].cpu().numpy(), amax_ref)
    assert np.abs(g["s"].cpu().numpy() / s_ref - 1).max() <= TOL_SCALE
    pre_w, pre_x = g["pre_w"].cpu().numpy(), g["pre_x"].cpu().numpy()
    # sampled whole rows of both quantizers
    rows_x = _sample(rng, M, 48, always=case.outlier_tokens[:8])
    rows_w = _sample(rng, N, 48)
    for which, rows, src, pre, clip, q_dev, step_dev in (
            ("act", rows_x, case.X, pre_x, case.clip_a, g["xq"], g["dx"]),
            ("weight", rows_w, case.W, pre_w, case.clip_w, g["wq"], g["dw"])):
        fn = orc.quant_act if which == "act" else orc.fuse_weights
        q_ref, step_ref, _ = fn(src[rows], pre, K, clip)
        idx = torch.from_numpy(rows).to("cuda:0")
        q_got = q_dev[idx].cpu().numpy()
        step_got = step_dev[idx].cpu().numpy()
        assert np.abs(step_got / step_ref - 1).max() <= TOL_SCALE, which
        worst, frac = _codes_ok(q_got, q_ref)
        assert worst <= 1 and frac <= TOL_CODES, (which, worst, frac)
    # properties at any size
    assert bool(torch.isfinite(g["Y"]).all())
    assert bool((g["dx"] > 0).all()) and bool((g["dw"] > 0).all())
    # 64 whole rows and 64 whole columns of the accumulators and of the output
    rows = _sample(rng, M, 64, always=case.outlier_tokens[:4])
    cols = _sample(rng, N, 64)
    ridx, cidx = torch.from_numpy(rows).to("cuda:0"), torch.from_numpy(cols).to("cuda:0")
    xq_all = orc.unpack_codes(g["xq"].cpu().numpy())
    wq_all = orc.unpack_codes(g["wq"].cpu().numpy())
    dx, dw = g["dx"].cpu().numpy(), g["dw"].cpu().numpy()
    acc_rows = orc.gemm_i32(xq_all[rows], wq_all)               # [64, N]
    acc_cols = orc.gemm_i32(xq_all, wq_all[cols])               # [M, 64]
    assert np.array_equal(g["acc"][ridx].cpu().numpy(), acc_rows)
    assert np.array_equal(g["acc"][:, cidx].cpu().numpy(), acc_cols)
    Y_rows = orc.dequant_output(acc_rows, dx[rows], dw)
    Y_cols = orc.dequant_output(acc_cols, dx, dw[cols])
    assert _rowwise_rel(g["Y"][ridx].cpu().numpy(), Y_rows) <= TOL_OUT
    # columns: the row maxima of unsampled rows are not known here, so each entry is held to one
    # fp16 rounding of the exact product (2^-10 relative, or one subnormal step near zero)
    got_cols = g["Y"][:, cidx].cpu().numpy().astype(np.float64)
    assert np.allclose(got_cols, Y_cols.astype(np.float64), rtol=TOL_OUT, atol=1.2e-7)


def test_config1_full_size(env):
    torch, sr = env
    _check_full_size(torch, sr, synth.config1(), seed=101)


def test_config2_full_size(env):
    torch, sr = env
    _check_full_size(torch, sr, synth.config2(), seed=102)


def test_config3_full_size(env):
    torch, sr = env
    _check_full_size(torch, sr, synth.config3(), seed=103)


@pytest.mark.parametrize("shape", [name for name, _, _ in synth.BLOCK_SHAPES])
def test_token_sweep_decode_shapes_in_full(env, shape):
    """configs[4]: M = 1, 4, 16, 32, 64, 128 for each linear shape of the block, every output checked."""
    torch, sr = env
    for M in (1, 4, 16, 32, 64, 128):
        case = synth.config4(shape, M)
        g = _run_layer(torch, sr, case)
        xq, wq = g["xq"].cpu().numpy(), g["wq"].cpu().numpy()
        dx, dw = g["dx"].cpu().numpy(), g["dw"].cpu().numpy()
        q_ref, step_ref, _ = orc.quant_act(case.X, g["pre_x"].cpu().numpy(), case.K, case.clip_a)
        assert np.abs(dx / step_ref - 1).max() <= TOL_SCALE
        worst, frac = _codes_ok(xq, q_ref)
        assert worst <= 1 and frac <= max(TOL_CODES, 1.5 / (2 * xq.size))
        acc_ref = orc.gemm_i32(orc.unpack_codes(xq), orc.unpack_codes(wq))
        assert np.array_equal(g["acc"].cpu().numpy(), acc_ref)
        Y_ref = orc.dequant_output(acc_ref, dx, dw)
        assert _rowwise_rel(g["Y"].cpu().numpy(), Y_ref) <= TOL_OUT


@pytest.mark.parametrize("shape,M", [("q_o", 512), ("q_o", 2048), ("q_o", 8192), ("k_v", 512), ("k_v", 2048),
                                     ("k_v", 8192), ("gate_up", 512), ("gate_up", 2048), ("gate_up", 8192),
                                     ("down", 512), ("down", 2048),
                                     ("q_o", 256), ("k_v", 256), ("k_v", 768), ("down", 256)])
def test_token_sweep_prefill_shapes_sampled(env, shape, M):
    """configs[4] at the prefill end of the sweep: every linear shape of the block at M = 512, 2048 and
    8192 tokens, and points at 256 and 768 tokens where the kernel choice changes (the streaming
    kernel with k-splits, the two-CTA kernel with and without its split-K reduction), checked like the full-size workloads: calibration in full, sampled whole rows of both
    quantizers, 64 whole rows and 64 whole columns of the accumulators and of the output."""
    torch, sr = env
    _check_full_size(torch, sr, synth.config4(shape, M), seed=400 + M + len(shape))
