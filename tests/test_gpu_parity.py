"""GPU-vs-oracle parity, call by call, through the C-ABI binding.

Tolerances (written here once):
  * rotation (debug export): per row ||y_gpu - y_oracle||_inf / ||y_oracle||_inf <= 1e-5
  * step sizes and smoothing scales: <= 1e-6 relative
  * packed codes: at most 1e-4 of the codes differ from the oracle's and every
    difference is +-1 (rounding ties moved by fp32 summation order)
  * int32 accumulators: bit-exact, and identical from run to run
  * fp16 outputs: per row <= 2e-3 relative to the row maximum of the oracle fed the GPU's codes
"""
import numpy as np
import pytest

from oracle import smoothrot_oracle as orc
from paper_2506_05413_b200 import synth

pytestmark = pytest.mark.gpu

TOL_ROT = 1e-5
TOL_SCALE = 1e-6
TOL_CODES = 1e-4
TOL_OUT = 2e-3


@pytest.fixture(scope="module")
def gu():
    from paper_2506_05413_b200 import build
    build.build()
    import gpu_util
    return gpu_util


def _acts(seed, M, K, gain=1000.0):
    rng = np.random.default_rng(seed)
    tok = np.arange(0, M, 17)
    ch = np.sort(rng.choice(K, size=3, replace=False))
    return synth.activations(rng, M, K, law="normal", outlier_channels=ch, outlier_gain=gain,
                             outlier_tokens=tok)


def _pre(seed, K):
    rng = np.random.default_rng(seed)
    return (rng.uniform(0.02, 8.0, K) * (rng.integers(0, 2, K) * 2 - 1)).astype(np.float32)


# ------------------------------------------------------------------ rotation
@pytest.mark.parametrize("K,M", [(128, 64), (256, 5), (512, 33), (1024, 7), (2048, 3), (4096, 37),
                                 (4096, 4), (8192, 2), (28 * 8, 9), (28 * 64, 5), (14336, 11),
                                 (12 * 8, 6), (12 * 256, 5), (20 * 16, 9), (20 * 256, 4), (28 * 1024, 2)])
@pytest.mark.parametrize("use_pre", [False, True])
def test_rotation_matches_oracle(gu, K, M, use_pre):
    X = _acts(K + M, M, K)
    pre = _pre(K, K) if use_pre else None
    got = gu.gpu_hadamard(X, pre)
    want = orc.rotate(X, pre, K)
    assert gu.rowwise_rel(got, want) <= TOL_ROT


def test_rotation_closed_forms_on_gpu(gu):
    for K in (128, 4096, 14336):
        X = np.zeros((2, K), np.float16)
        X[0, 5] = 3.0
        X[1, :] = 0.5
        got = gu.gpu_hadamard(X, None)
        assert np.allclose(np.abs(got[0]), 3.0 / np.sqrt(K), rtol=1e-6)
        if K != 14336:
            want = np.zeros(K); want[0] = 0.5 * np.sqrt(K)
            assert np.allclose(got[1], want, atol=1e-4)


def test_rotation_with_row_stride(gu):
    import torch
    from paper_2506_05413_b200 import binding as sr
    K, M = 4096, 6
    X = _acts(3, M, K)
    big = torch.zeros((M, K + 64), dtype=torch.float16, device=gu.DEV)
    big[:, :K] = gu.dev(X)
    Y = torch.empty((M, K), dtype=torch.float32, device=gu.DEV)
    sr.debug_hadamard(big[:, :K], None, Y)
    torch.cuda.synchronize()
    assert gu.rowwise_rel(Y.cpu().numpy(), orc.rotate(X, None, K)) <= TOL_ROT


# ------------------------------------------------------- quantize + pack
@pytest.mark.parametrize("K,M", [(128, 64), (512, 21), (4096, 301), (4096, 1), (8192, 3), (28 * 16, 10), (14336, 19),
                                 (12 * 256, 17), (20 * 256, 13), (28 * 1024, 3)])
@pytest.mark.parametrize("which", ["act", "weight"])
def test_quantized_codes_match_oracle(gu, K, M, which):
    from paper_2506_05413_b200 import binding as sr
    X = _acts(7 * K + M, M, K) if which == "act" else \
        (np.random.default_rng(K).standard_normal((M, K)) * 0.02).astype(np.float16)
    pre = _pre(K + 1, K)
    clip = 0.9 if which == "act" else 1.0
    fn = sr.quant_act if which == "act" else sr.fuse_weights
    q, step = gu.gpu_quantize(fn, X, pre, clip)
    ofn = orc.quant_act if which == "act" else orc.fuse_weights
    q_ref, step_ref, _ = ofn(X, pre, K, clip)
    assert np.abs(step / step_ref - 1).max() <= TOL_SCALE
    frac, worst = gu.code_mismatch(q, q_ref)
    assert worst <= 1 and frac <= max(TOL_CODES, 1.5 / q.size / 2)
    codes = orc.unpack_codes(q)
    assert codes.min() >= -8 and codes.max() <= 7


@pytest.mark.parametrize("K", [512, 4096, 14336])
@pytest.mark.parametrize("clip", [0.5, 0.8, 0.83, 1.0])
def test_quantizer_clip_ratios_including_two_sided_saturation(gu, K, clip):
    """Below clip = 7/8.5 values can fall under -8.5 steps and must saturate at -8."""
    from paper_2506_05413_b200 import binding as sr
    X = _acts(K + int(100 * clip), 23, K, gain=30.0)
    q, step = gu.gpu_quantize(sr.quant_act, X, None, clip)
    q_ref, step_ref, _ = orc.quant_act(X, None, K, clip)
    assert np.abs(step / step_ref - 1).max() <= TOL_SCALE
    frac, worst = gu.code_mismatch(q, q_ref)
    assert worst <= 1 and frac <= TOL_CODES
    if clip <= 0.8:
        assert orc.unpack_codes(q_ref).min() == -8 and orc.unpack_codes(q_ref).max() == 7


def test_quantizer_edge_rows(gu):
    from paper_2506_05413_b200 import binding as sr
    for K in (128, 4096, 14336):
        X = np.zeros((3, K), np.float16)
        X[1, 9] = -2.0                     # unit vector: every |x^| equal -> codes +7 / -8
        X[2, :] = 65504.0                  # largest fp16 everywhere
        q, step = gu.gpu_quantize(sr.quant_act, X, None, 0.9)
        codes = orc.unpack_codes(q)
        assert step[0] == np.float32(1.0) and np.all(codes[0] == 0)
        assert set(np.unique(codes[1])) <= {7, -8}
        H = orc.hadamard_matrix(K)
        assert np.array_equal(codes[1] == -8, H[9] > 0)      # x^ = -2 H[9] / sqrt(K)
        assert np.all(np.isfinite(step))
        q_ref, step_ref, _ = orc.quant_act(X, None, K, 0.9)
        assert np.abs(step / step_ref - 1).max() <= TOL_SCALE


# ------------------------------------------------------------- calibration
@pytest.mark.parametrize("K,T,N,batches", [(128, 128, 256, 1), (4096, 300, 77, 3), (14336, 65, 130, 2)])
def test_calibration_matches_oracle(gu, K, T, N, batches):
    rng = np.random.default_rng(K + T)
    Xc = _acts(K, T, K)
    W = (rng.standard_normal((N, K)) * 0.02).astype(np.float16)
    W[:, 3] = 0                                            # dead weight channel -> eps guard
    d = synth.sign_vector(rng, K)
    for alpha in (0.5, 0.45, 0.0, 1.0):
        amax, s, pre_w, pre_x = gu.gpu_calibrate(Xc, W, alpha, d, batches)
        amax_ref, s_ref = orc.calibrate(Xc, W, alpha)
        assert np.array_equal(amax, amax_ref)
        assert np.abs(s / s_ref - 1).max() <= TOL_SCALE
        assert np.array_equal(pre_w, s * d)
        assert np.array_equal(pre_x, (d.astype(np.float64) / s.astype(np.float64)).astype(np.float32))


# --------------------------------------------------------------------- GEMM
GEMM_SHAPES = [
    (64, 256, 128),      # config 0
    # few tokens: the decode kernel (plain loads, warp-level integer MMA, K split between the warps of a CTA)
    (1, 1024, 4096),
    (4, 4096, 4096),
    (2, 1000, 1024),     # ragged channels (N % 16 == 8)
    (3, 4104, 3072),
    (4, 264, 14336),     # long rows: the double-buffered loop
    (1, 8, 1024),
    (3, 1000, 1152),     # fewer 64-byte chunks than a batch holds
    (8, 1024, 4096),
    (6, 4096, 4096),
    (7, 72, 128),        # one chunk: seven of the eight warps have nothing to add
    (16, 136, 512),      # two token tiles
    (9, 264, 14336),     # two token tiles, long rows, 16 warps
    (16, 1000, 8192),
    (13, 520, 4224),     # long rows with a partial last batch
    (8, 256, 16384),
    (17, 64, 256),       # four token tiles
    (20, 520, 4096),
    (24, 256, 16384),
    (32, 8200, 512),     # four token tiles, many channels: two row groups per CTA, double-buffered
    (25, 8456, 1152),
    (33, 72, 384),       # eight token tiles
    (40, 136, 2048),
    (64, 1000, 4096),
    (50, 264, 14336),
    # the streaming kernel (128-token tiles)
    (64, 8200, 4096),    # 64 tokens, but too many weights for the decode kernel
    (100, 264, 256),
    (128, 64, 128),
    (70, 1000, 1024),    # 2 k-splits added up inside a cluster, ragged channels
    (80, 520, 4096),     # 8 k-splits in a cluster
    (128, 1024, 4096),
    (128, 6144, 4096),   # 48 channel tiles: 2 k-splits keep the CTAs in one wave
    (100, 256, 16384),   # few channels, long K: k-splits through the workspace
    (128, 256, 8192),
    (300, 1024, 2048),   # 3 token tiles of the streaming kernel, ragged
    (512, 520, 1024),
    (512, 1024, 14336),  # long K
    (130, 136, 640),     # two token tiles, ragged both ways
    (200, 1000, 2048),
    (300, 136, 640),     # few channels, 3 token tiles
    (257, 8, 128),
    # one CTA per SM, both operands through shared memory (more than 512 tokens, fewer than 256 channels)
    (600, 136, 640),     # BN = 128
    (520, 8, 128),       # BN = 64
    (1030, 200, 1024),
    # the two-CTA kernel
    (256, 256, 128),     # one pair tile
    (300, 520, 1152),    # several tiles and a ragged tail
    (100, 12296, 512),   # fewer than 256 tokens, but enough channels to fill the SM pairs
    (200, 10240, 256),
    (600, 776, 512),     # ragged in both directions
    (257, 3200, 8192),   # two k-splits through the workspace
    (300, 2560, 8192),   # few enough 128-token tiles for the streaming kernel with 2 k-splits in a cluster
    (520, 2568, 8192),   # ... ragged in both directions
]


@pytest.mark.parametrize("M,N,K", GEMM_SHAPES)
def test_gemm_accumulators_bit_exact(gu, M, N, K):
    xq = synth.random_codes(M * 31 + K, M, K)
    wq = synth.random_codes(N * 17 + K + 1, N, K)
    got = gu.gpu_gemm_i32(orc.pack_codes(xq), orc.pack_codes(wq))
    want = orc.gemm_i32(xq, wq)
    assert np.array_equal(got, want)
    again = gu.gpu_gemm_i32(orc.pack_codes(xq), orc.pack_codes(wq))
    assert np.array_equal(got, again)


def test_gemm_extreme_codes(gu):
    K = 14336
    xq = np.full((130, K), -8, np.int8)
    wq = np.full((264, K), -8, np.int8)
    wq[1::2] = 7
    got = gu.gpu_gemm_i32(orc.pack_codes(xq), orc.pack_codes(wq))
    assert np.all(got[:, 0::2] == 64 * K) and np.all(got[:, 1::2] == -56 * K)


@pytest.mark.parametrize("M,N,K", [(64, 256, 128), (3, 1024, 4096), (200, 264, 512), (130, 520, 4096),
                                   (300, 520, 640), (1024, 768, 4096), (16, 1000, 2048), (128, 520, 1024),
                                   (100, 256, 16384), (4, 1000, 14336), (1, 4096, 4096), (6, 1024, 4096), (16, 520, 14336),
                                   (30, 8200, 1024), (64, 520, 4096), (64, 8200, 4096), (96, 12288, 1024), (160, 520, 2048),
                                   (12, 4104, 2048), (32, 1024, 4096), (300, 2568, 8192), (520, 2568, 8192)])
def test_linear_output_matches_oracle_on_gpu_codes(gu, M, N, K):
    rng = np.random.default_rng(M + N + K)
    xq = orc.pack_codes(synth.random_codes(M, M, K))
    wq = orc.pack_codes(synth.random_codes(N + 1, N, K))
    dx = rng.uniform(0.01, 0.3, M).astype(np.float32)
    dw = rng.uniform(1e-4, 4e-3, N).astype(np.float32)
    got = gu.gpu_linear(xq, dx, wq, dw)
    want = orc.linear(xq, dx, wq, dw)
    assert np.isfinite(got.astype(np.float32)).all()
    assert gu.rowwise_rel(got, want) <= TOL_OUT


def test_prefill_k_split_is_optional_and_changes_nothing(gu):
    """For M >= 256 the workspace only lets the two-CTA kernel split K over idle SM pairs: without
    it the call runs unsplit and, the sums being integers, returns the same fp16 outputs."""
    import torch
    from paper_2506_05413_b200 import binding as sr
    M, N, K = 520, 2568, 8192
    assert sr.workspace_bytes(M, N, K) > 0
    rng = np.random.default_rng(5)
    xq = gu.dev(orc.pack_codes(synth.random_codes(1, M, K)))
    wq = gu.dev(orc.pack_codes(synth.random_codes(2, N, K)))
    dx = gu.dev(rng.uniform(0.01, 0.3, M).astype(np.float32))
    dw = gu.dev(rng.uniform(1e-4, 4e-3, N).astype(np.float32))
    ws = torch.empty(sr.workspace_bytes(M, N, K), dtype=torch.uint8, device=gu.DEV)
    Y_split = torch.full((M, N), float("nan"), dtype=torch.float16, device=gu.DEV)
    Y_plain = torch.full((M, N), float("nan"), dtype=torch.float16, device=gu.DEV)
    Y_short = torch.full((M, N), float("nan"), dtype=torch.float16, device=gu.DEV)
    sr.linear(xq, dx, wq, dw, Y_split, ws)
    sr.linear(xq, dx, wq, dw, Y_plain, None)
    sr.linear(xq, dx, wq, dw, Y_short, ws[:1024])
    torch.cuda.synchronize()
    assert sr.device_status() == 0
    assert torch.equal(Y_split, Y_plain) and torch.equal(Y_split, Y_short)
    assert bool(torch.isfinite(Y_split).all())


# ------------------------------------------------------------- whole layer
def _layer_on_gpu(gu, case):
    from paper_2506_05413_b200 import binding as sr
    amax, s, pre_w, pre_x = gu.gpu_calibrate(case.X_calib, case.W, case.alpha, case.d)
    wq, dw = gu.gpu_quantize(sr.fuse_weights, case.W, pre_w, case.clip_w)
    xq, dx = gu.gpu_quantize(sr.quant_act, case.X, pre_x, case.clip_a)
    Y = gu.gpu_linear(xq, dx, wq, dw)
    return dict(amax=amax, s=s, pre_w=pre_w, pre_x=pre_x, wq=wq, dw=dw, xq=xq, dx=dx, Y=Y)


def _check_layer(gu, case, g):
    K = case.K
    amax_ref, s_ref = orc.calibrate(case.X_calib, case.W, case.alpha)
    assert np.array_equal(g["amax"], amax_ref)
    assert np.abs(g["s"] / s_ref - 1).max() <= TOL_SCALE
    # staged: each oracle stage is fed the GPU's upstream outputs
    wq_ref, dw_ref, _ = orc.fuse_weights(case.W, g["pre_w"], K, case.clip_w)
    xq_ref, dx_ref, _ = orc.quant_act(case.X, g["pre_x"], K, case.clip_a)
    assert np.abs(g["dw"] / dw_ref - 1).max() <= TOL_SCALE
    assert np.abs(g["dx"] / dx_ref - 1).max() <= TOL_SCALE
    for got, ref in ((g["wq"], wq_ref), (g["xq"], xq_ref)):
        frac, worst = gu.code_mismatch(got, ref)
        assert worst <= 1 and frac <= TOL_CODES
    Y_ref = orc.linear(g["xq"], g["dx"], g["wq"], g["dw"])
    assert gu.rowwise_rel(g["Y"], Y_ref) <= TOL_OUT


def test_config0_whole_layer(gu):
    case = synth.config0()
    g = _layer_on_gpu(gu, case)
    _check_layer(gu, case, g)
    Yfp = case.X.astype(np.float64) @ case.W.astype(np.float64).T
    err = np.linalg.norm(g["Y"].astype(np.float64) - Yfp) / np.linalg.norm(Yfp)
    assert err < 0.25


@pytest.mark.parametrize("maker,M,N", [(synth.config1, 160, 264), (synth.config2, 130, 136), (synth.config3, 40, 520)])
def test_reduced_configs_whole_layer(gu, maker, M, N):
    case = maker(M=M, N=N)
    _check_layer(gu, case, _layer_on_gpu(gu, case))


@pytest.mark.parametrize("K", [3072, 5120])
def test_whole_layer_on_other_widths(gu, K):
    """Widths 12 * 256 and 20 * 256 (Paley factors of order 12 and 20): the whole path, staged
    against the oracle like the named configurations."""
    case = synth.make_layer(f"width_{K}", seed=100 + K, M=70, K=K, N=264, T=96, law="normal",
                            w_std=0.02, n_outlier_channels=3, outlier_gain=800.0)
    _check_layer(gu, case, _layer_on_gpu(gu, case))


# ------------------------------------------------ gated-linear-unit input path
@pytest.mark.parametrize("K,M", [(128, 9), (512, 21), (4096, 5), (28 * 16, 10), (14336, 1), (14336, 37)])
@pytest.mark.parametrize("use_pre", [False, True])
def test_glu_quantized_codes_match_oracle(gu, K, M, use_pre):
    import torch
    from paper_2506_05413_b200 import binding as sr
    rng = np.random.default_rng(K + M)
    gate = (rng.standard_normal((M, K)) * 2.0).astype(np.float16)
    up = rng.standard_normal((M, K)).astype(np.float16)
    gate[0, :7] = [0.0, -65504.0, 65504.0, 30.0, -30.0, 11.0, -11.0]     # the ends of the SiLU
    up[min(1, M - 1), 3] = 2000.0                                        # a massive outlier
    pre = _pre(K + 3, K) if use_pre else None
    q = torch.empty((M, K // 2), dtype=torch.uint8, device=gu.DEV)
    step = torch.empty(M, dtype=torch.float32, device=gu.DEV)
    sr.quant_act_glu(gu.dev(gate), gu.dev(up), gu.dev(pre) if use_pre else None, 0.9, q, step)
    torch.cuda.synchronize()
    assert sr.device_status() == 0
    q_ref, step_ref, _ = orc.quant_act_glu(gate, up, pre, K, 0.9)
    # the kernel evaluates the SiLU in fp32 (library exponential, IEEE division): the stated budgets hold
    assert np.abs(step.cpu().numpy() / step_ref - 1).max() <= TOL_SCALE
    frac, worst = gu.code_mismatch(q.cpu().numpy(), q_ref)
    assert worst <= 1 and frac <= max(TOL_CODES, 1.5 / q.numel() / 2)


def test_glu_path_equals_plain_path_when_the_product_is_exact_in_fp16(gu):
    """gate = 30 makes SiLU(gate) = 30 to fp32 precision; with up a multiple of 1/32 the product is an
    fp16 number, so the fused call and quant_act on that fp16 matrix must agree."""
    import torch
    from paper_2506_05413_b200 import binding as sr
    rng = np.random.default_rng(5)
    for K in (512, 14336):
        M = 6
        up = (rng.integers(-64, 65, size=(M, K)) / 32.0).astype(np.float16)
        gate = np.full((M, K), 30.0, np.float16)
        X = (30.0 * up.astype(np.float64)).astype(np.float16)
        outs = []
        for call in ("glu", "plain"):
            q = torch.empty((M, K // 2), dtype=torch.uint8, device=gu.DEV)
            step = torch.empty(M, dtype=torch.float32, device=gu.DEV)
            if call == "glu":
                sr.quant_act_glu(gu.dev(gate), gu.dev(up), None, 0.9, q, step)
            else:
                sr.quant_act(gu.dev(X), None, 0.9, q, step)
            torch.cuda.synchronize()
            outs.append((q.cpu().numpy(), step.cpu().numpy()))
        assert np.abs(outs[0][1] / outs[1][1] - 1).max() <= TOL_SCALE
        frac, worst = gu.code_mismatch(outs[0][0], outs[1][0])
        assert worst <= 1 and frac <= max(2 * TOL_CODES, 1.5 / outs[0][0].size / 2)   # two GPU paths, each within TOL_CODES of the oracle


# ------------------------------------------------ weight clip-ratio search
@pytest.mark.parametrize("K,N,slices", [(128, 40, 1), (4096, 33, 1), (4096, 9, 4), (14336, 10, 1), (28 * 16, 12, 3)])
def test_weight_clip_search_matches_oracle(gu, K, N, slices):
    import torch
    from paper_2506_05413_b200 import binding as sr
    rng = np.random.default_rng(K + N)
    W = (rng.standard_normal((N, K)) * 0.02).astype(np.float16)
    W[1, 5] = 0.9                                   # a row with a far outlier: clipping pays
    W[2, :] = 0                                     # an all-zero row
    W[3, :] = 0; W[3, 7] = 0.25                     # a single entry: flat after rotation, ratio 1 is exact
    pre = _pre(K + 11, K)
    ratios = orc.clip_ratios(51, 0.5)
    q = torch.empty((N, K // 2), dtype=torch.uint8, device=gu.DEV)
    step = torch.empty(N, dtype=torch.float32, device=gu.DEV)
    best = torch.full((N,), -1, dtype=torch.int32, device=gu.DEV)
    full = sr.fuse_weights_search_workspace_bytes(N, K)
    assert full == N * K * 4
    ws_bytes = full if slices == 1 else (N // slices + 1) * K * 4 + 64     # not a multiple of a row on purpose
    ws = torch.empty(ws_bytes, dtype=torch.uint8, device=gu.DEV)
    sr.fuse_weights_search(gu.dev(W), gu.dev(pre), 0.5, 51, q, step, best, ws)
    torch.cuda.synchronize()
    q, step, best = q.cpu().numpy(), step.cpu().numpy(), best.cpu().numpy()
    packed_ref, step_ref, best_ref, errs, wr = orc.fuse_weights_search(W, pre, K, ratios)
    assert best.min() >= 0 and best.max() < 51
    rows = np.arange(N)
    # the chosen ratio minimises the oracle's error curve (up to the fp32 noise of the rotation)
    assert np.all(errs[rows, best] <= errs.min(axis=1) * (1 + 1e-4) + 1e-30)
    # wherever the GPU took another ratio than the oracle, the oracle's own two errors are a tie up
    # to the fp32 noise of the rotation: its error curve decides, not a share of rows
    differ = best != best_ref
    e_gpu, e_ref = errs[rows, best], errs[rows, best_ref]
    assert np.all(np.abs(e_gpu[differ] - e_ref[differ]) <= 1e-6 * e_ref[differ] + 1e-30), (e_gpu[differ], e_ref[differ])
    assert best[2] == 0 and step[2] == np.float32(1.0) and best[3] == 0
    # staged: the oracle's quantizer at the ratio the GPU chose
    for r in rows:
        codes_r, step_r = orc.quantize_rows(wr[r:r + 1], ratios[best[r]])
        assert abs(step[r] / step_r[0] - 1) <= TOL_SCALE
        a = orc.unpack_codes(q[r:r + 1]).astype(int)
        diff = np.abs(a - codes_r.astype(int))
        assert diff.max() <= 1 and (diff != 0).mean() <= max(TOL_CODES, 1.5 / K)
    assert best[1] > 0          # the outlier row took a smaller ratio


# ------------------------------------------------ KV-cache quantizer
@pytest.mark.parametrize("R,C", [(1, 128), (7, 1024), (300, 512), (4099, 256)])
@pytest.mark.parametrize("clip", [0.95, 1.0, 0.6])
def test_kv_quantizer_matches_oracle_and_round_trips(gu, R, C, clip):
    """Steps and zero points come from the same fp32 operations on both sides and must be identical.
    The codes are decided in fp32 on both sides too, but the kernel multiplies by the rounded
    reciprocal of the step where the oracle divides: at most 1e-4 of them may differ, by one.
    The dequantizer is checked on the GPU's own codes, within one fp16 rounding."""
    import torch
    from paper_2506_05413_b200 import binding as sr
    rng = np.random.default_rng(R + C)
    X = rng.standard_normal((R, C)).astype(np.float16)
    X[0, :128] = 2.5                                  # a constant group
    if R > 2:
        X[1, :] = 0                                   # all zero
        X[2, 5] = 300.0                               # an outlier: the clip ratio saturates it
        X[2, 128 * (C // 128 - 1):] = np.abs(X[2, 128 * (C // 128 - 1):]) + 1   # a group that does not straddle zero
    pad = torch.zeros((R, C + 8), dtype=torch.float16, device=gu.DEV)      # a strided input
    pad[:, :C] = gu.dev(X)
    q = torch.empty((R, C // 2), dtype=torch.uint8, device=gu.DEV)
    step = torch.empty((R, C // 128), dtype=torch.float32, device=gu.DEV)
    zero = torch.empty((R, C // 128), dtype=torch.float32, device=gu.DEV)
    sr.kv_quant(pad[:, :C], clip, q, step, zero)
    Y = torch.empty((R, C), dtype=torch.float16, device=gu.DEV)
    sr.kv_dequant(q, step, zero, Y)
    torch.cuda.synchronize()
    codes_ref, step_ref, zero_ref = orc.kv_quantize(X, clip)
    assert np.array_equal(step.cpu().numpy(), step_ref)
    assert np.array_equal(zero.cpu().numpy(), zero_ref)
    codes_gpu = orc.unpack_nibbles(q.cpu().numpy())
    diff = np.abs(codes_gpu.astype(int) - codes_ref.astype(int))
    assert diff.max() <= 1 and (diff != 0).mean() <= TOL_CODES
    want = orc.kv_dequantize(codes_gpu, step_ref, zero_ref)
    got = Y.cpu().numpy().astype(np.float64)
    assert np.allclose(got, want, rtol=1e-3, atol=1e-7)


def test_kv_quantizer_rejects_bad_arguments(gu):
    import torch
    from paper_2506_05413_b200 import binding as sr
    X = torch.zeros((2, 192), dtype=torch.float16, device=gu.DEV)           # not a multiple of 128
    q = torch.empty((2, 96), dtype=torch.uint8, device=gu.DEV)
    s = torch.empty((2, 1), dtype=torch.float32, device=gu.DEV)
    with pytest.raises(sr.SmoothRotError):
        sr.kv_quant(X, 0.95, q, s, s.clone())


# ------------------------------------------------ tensor-core rotation kernels (no diagonal, many rows)
@pytest.mark.parametrize("K,M,diag", [(4096, 512, None), (4096, 777, None), (4096, 7200, None), (4096, 7992, None), (14336, 256, None),
                                      (14336, 301, None), (14336, 1030, None), (4096, 1024, "smooth"),
                                      (4096, 1101, "wide"), (4096, 6150, "smooth"), (4096, 1027, "tiny")])
def test_tensor_core_rotation_and_codes_match_oracle(gu, K, M, diag):
    """Without a diagonal and with a few hundred rows or more, K = 4096 and K = 14336 run their Walsh
    factor of order 128 / 256 on tcgen05: the rotation export, the steps and the codes against the
    oracle, on rows that include massive outliers, an all-zero row, the ends of the fp16 range, a
    single spike and a row a thousand times smaller than the rest, with a row stride larger than K
    and a ragged last batch.  The same rows with diagonals (smoothing-like with a dead channel, six
    decades wide with random signs, uniformly tiny) take the register kernel at these row counts."""
    import torch
    from paper_2506_05413_b200 import binding as sr
    rng = np.random.default_rng(K + M)
    pre = None
    if diag == "smooth":
        pre = (rng.uniform(0.08, 0.3, K) * rng.choice([-1.0, 1.0], K)).astype(np.float32)
        pre[rng.choice(K, 4, replace=False)] = 0.004          # channels that carry the outliers
        pre[5] = 89.0                                         # a dead channel
    elif diag == "wide":
        pre = (10.0 ** rng.uniform(-3, 3, K) * rng.choice([-1.0, 1.0], K)).astype(np.float32)
    elif diag == "tiny":
        pre = (rng.uniform(1.0, 2.0, K) * 3e-7).astype(np.float32)
    ld = K + 24
    Xfull = np.zeros((M, ld), np.float16)
    X = rng.standard_normal((M, K)).astype(np.float32)
    X[::17, rng.choice(K, 3, replace=False)] *= 1500.0        # massive outliers on some tokens
    X[1] = 0.0
    X[2] = 65504.0
    X[3] = -65504.0
    X[4] = 0.0
    X[4, K // 3] = 3.0                                        # a single spike
    X[M - 1] *= 1e-3                                          # a small row at the ragged end
    Xfull[:, :K] = np.clip(X, -65504, 65504).astype(np.float16)
    Xd = gu.dev(Xfull)[:, :K]                                 # strided view
    Xh = Xfull[:, :K]
    # rotation alone
    Y = torch.empty((M, K), dtype=torch.float32, device=gu.DEV)
    pre_d = gu.dev(pre) if pre is not None else None
    sr.debug_hadamard(Xd, pre_d, Y)
    torch.cuda.synchronize()
    assert sr.device_status() == 0
    rows = np.unique(np.concatenate([np.arange(8), [M - 2, M - 1], rng.choice(M, 24, replace=False)]))
    ref = orc.rotate(Xh[rows], pre, K)
    assert gu.rowwise_rel(Y.cpu().numpy()[rows], ref) <= TOL_ROT
    # quantized, two clip ratios (0.8 reaches the two-sided clamp)
    for clip in (0.9, 0.8):
        q = torch.empty((M, K // 2), dtype=torch.uint8, device=gu.DEV)
        step = torch.empty(M, dtype=torch.float32, device=gu.DEV)
        sr.quant_act(Xd, pre_d, clip, q, step)
        torch.cuda.synchronize()
        assert sr.device_status() == 0
        q_ref, step_ref, _ = orc.quant_act(Xh[rows], pre, K, clip)
        assert np.abs(step.cpu().numpy()[rows] / step_ref - 1).max() <= TOL_SCALE
        frac, worst = gu.code_mismatch(q.cpu().numpy()[rows], q_ref)
        assert worst <= 1 and frac <= TOL_CODES, (clip, frac, worst)
        assert step.cpu().numpy()[1] == np.float32(1.0) and not q.cpu().numpy()[1].any()
