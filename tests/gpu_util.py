"""Helpers for the GPU parity tests: move seeded inputs to the device, run the
library through its binding, bring results back as numpy."""
import numpy as np
import torch

from paper_2506_05413_b200 import binding as sr

DEV = "cuda:0"


def dev(a):
    return torch.from_numpy(np.ascontiguousarray(a)).to(DEV)


def gpu_calibrate(X_calib, W, alpha, d=None, batches=1):
    K = W.shape[1]
    amax = torch.zeros(K, dtype=torch.float32, device=DEV)
    s = torch.empty(K, dtype=torch.float32, device=DEV)
    pre_w = torch.empty(K, dtype=torch.float32, device=DEV)
    pre_x = torch.empty(K, dtype=torch.float32, device=DEV)
    Xc, Wd = dev(X_calib), dev(W)
    dd = dev(d) if d is not None else None
    T = Xc.shape[0]
    edges = np.linspace(0, T, batches + 1).astype(int)
    for i in range(batches - 1):
        sr.calibrate(Xc[edges[i]:edges[i + 1]], amax)
    sr.calibrate(Xc[edges[batches - 1]:], amax, W=Wd, alpha=alpha, s_out=s, d=dd,
                 pre_w_out=pre_w if d is not None else None, pre_x_out=pre_x if d is not None else None)
    torch.cuda.synchronize()
    return amax.cpu().numpy(), s.cpu().numpy(), pre_w.cpu().numpy(), pre_x.cpu().numpy()


def gpu_quantize(fn, X, pre, clip):
    Xd = dev(X)
    R, K = Xd.shape
    q = torch.empty((R, K // 2), dtype=torch.uint8, device=DEV)
    step = torch.empty(R, dtype=torch.float32, device=DEV)
    fn(Xd, dev(pre) if pre is not None else None, clip, q, step)
    torch.cuda.synchronize()
    return q.cpu().numpy(), step.cpu().numpy()


def gpu_hadamard(X, pre):
    Xd = dev(X)
    Y = torch.empty(Xd.shape, dtype=torch.float32, device=DEV)
    sr.debug_hadamard(Xd, dev(pre) if pre is not None else None, Y)
    torch.cuda.synchronize()
    return Y.cpu().numpy()


def _workspace(M, N, K):
    need = sr.workspace_bytes(M, N, K)
    return torch.empty(need, dtype=torch.uint8, device=DEV) if need else None


def gpu_gemm_i32(xq_packed, wq_packed):
    xd, wd = dev(xq_packed), dev(wq_packed)
    M, N, K = xd.shape[0], wd.shape[0], xd.shape[1] * 2
    acc = torch.full((M, N), -7777, dtype=torch.int32, device=DEV)
    sr.debug_gemm_i32(xd, wd, acc, _workspace(M, N, K))
    torch.cuda.synchronize()
    assert sr.device_status() == 0
    return acc.cpu().numpy()


def gpu_linear(xq_packed, dx, wq_packed, dw):
    xd, wd = dev(xq_packed), dev(wq_packed)
    M, N, K = xd.shape[0], wd.shape[0], xd.shape[1] * 2
    Y = torch.full((M, N), float("nan"), dtype=torch.float16, device=DEV)
    sr.linear(xd, dev(dx), wd, dev(dw), Y, _workspace(M, N, K))
    torch.cuda.synchronize()
    assert sr.device_status() == 0
    return Y.cpu().numpy()


def code_mismatch(packed_gpu, packed_ref):
    """(fraction of codes that differ, max |difference|) between two packed tensors."""
    from oracle import smoothrot_oracle as orc
    a = orc.unpack_codes(packed_gpu).astype(np.int16)
    b = orc.unpack_codes(packed_ref).astype(np.int16)
    diff = np.abs(a - b)
    return float((diff != 0).mean()) if diff.size else 0.0, int(diff.max()) if diff.size else 0


def rowwise_rel(got, want):
    """max over rows of ||got - want||_inf / ||want||_inf (float64)."""
    g, w = np.asarray(got, np.float64), np.asarray(want, np.float64)
    if g.size == 0:
        return 0.0
    den = np.abs(w).max(axis=1)
    num = np.abs(g - w).max(axis=1)
    den = np.where(den == 0, 1.0, den)
    return float((num / den).max())
