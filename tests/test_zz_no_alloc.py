"""smoothrot_linear_static_scratch: the entry point for callers that cannot
provide (or allocate) a split-K workspace, e.g. a plug-in whose host process
forbids cudaMalloc after start-up.  Its scratch is a fixed array inside the
library, shared by all calls on a device.

Collected last on purpose: a run that stops at the first failure has then
already run every other test.  The check: two calls in a row, on different
inputs, each equal to what smoothrot_linear (caller-provided workspace)
returns for the same inputs; the second call must not be disturbed by what the
first left in the array.  Also: a shape beyond the built-in size is refused.
"""
import numpy as np
import pytest

pytestmark = pytest.mark.gpu

TOL_OUT = 2e-3   # same bound as the other fp16-output parity tests


def _case(seed, M, N, K):
    from oracle import smoothrot_oracle as orc
    from paper_2506_05413_b200 import synth
    rng = np.random.default_rng(seed)
    xq = orc.pack_codes(synth.random_codes(seed, M, K))
    wq = orc.pack_codes(synth.random_codes(seed + 1, N, K))
    dx = rng.uniform(0.01, 0.3, M).astype(np.float32)
    dw = rng.uniform(1e-4, 4e-3, N).astype(np.float32)
    return xq, dx, wq, dw


def test_static_scratch_entry_point_matches_linear_twice_in_a_row():
    import torch
    from paper_2506_05413_b200 import build, binding as sr
    build.build()
    dev = "cuda:0"
    t = lambda a: torch.from_numpy(np.ascontiguousarray(a)).to(dev)
    # few output channels and a long K: the shapes whose k-splits still go through scratch memory
    shapes = [(100, 256, 16384), (65, 256, 16384)]
    for call, (M, N, K) in enumerate(shapes):
        need = sr.workspace_bytes(M, N, K)
        assert 0 < need <= sr.STATIC_SCRATCH_BYTES
        xq, dx, wq, dw = (t(a) for a in _case(100 + call, M, N, K))
        ws = torch.empty(need, dtype=torch.uint8, device=dev)
        Y_ref = torch.empty((M, N), dtype=torch.float16, device=dev)
        sr.linear(xq, dx, wq, dw, Y_ref, ws)
        Y = torch.full((M, N), float("nan"), dtype=torch.float16, device=dev)
        sr.linear_static_scratch(xq, dx, wq, dw, Y)
        torch.cuda.synchronize()
        assert sr.device_status() == 0
        got, want = Y.cpu().numpy().astype(np.float64), Y_ref.cpu().numpy().astype(np.float64)
        assert np.isfinite(got).all()
        rel = (np.abs(got - want).max(axis=1) / np.abs(want).max(axis=1)).max()
        assert rel <= TOL_OUT, (call, rel)
        assert np.array_equal(got, want)               # same kernels, same order of integer sums
        # and directly against the CPU oracle on the same codes and steps
        from oracle import smoothrot_oracle as orc
        xq_h, dx_h, wq_h, dw_h = _case(100 + call, M, N, K)
        Y_orc = orc.linear(xq_h, dx_h, wq_h, dw_h).astype(np.float64)
        rel_orc = (np.abs(got - Y_orc).max(axis=1) / np.abs(Y_orc).max(axis=1)).max()
        assert rel_orc <= TOL_OUT, (call, rel_orc)


def test_static_scratch_entry_point_refuses_oversized_shapes_and_needs_no_scratch_for_prefill():
    import torch
    from paper_2506_05413_b200 import build, binding as sr
    build.build()
    dev = "cuda:0"
    M, N, K = 128, 256, 37888                           # split-K partials beyond the built-in array
    assert sr.workspace_bytes(M, N, K) > sr.STATIC_SCRATCH_BYTES
    xq = torch.zeros((M, K // 2), dtype=torch.uint8, device=dev)
    wq = torch.zeros((N, K // 2), dtype=torch.uint8, device=dev)
    dx = torch.ones(M, device=dev)
    dw = torch.ones(N, device=dev)
    Y = torch.empty((M, N), dtype=torch.float16, device=dev)
    with pytest.raises(sr.SmoothRotError) as err:
        sr.linear_static_scratch(xq, dx, wq, dw, Y)
    assert err.value.status == -7
    # a prefill shape needs no scratch at all and goes straight through
    M, N, K = 256, 256, 256
    assert sr.workspace_bytes(M, N, K) == 0
    t = lambda a: torch.from_numpy(np.ascontiguousarray(a)).to(dev)
    xq, dx, wq, dw = (t(a) for a in _case(7, M, N, K))
    Y0 = torch.empty((M, N), dtype=torch.float16, device=dev)
    Y1 = torch.empty((M, N), dtype=torch.float16, device=dev)
    sr.linear(xq, dx, wq, dw, Y0)
    sr.linear_static_scratch(xq, dx, wq, dw, Y1)
    torch.cuda.synchronize()
    assert torch.equal(Y0, Y1)


def test_static_scratch_entry_point_on_prefill_shapes_whose_k_split_is_optional():
    """M >= 256 with few tiles and a long K: smoothrot_linear splits K through the workspace.  The
    no-allocation entry point does the same inside its array when the partial sums fit, and runs
    unsplit when they do not; either way the outputs equal smoothrot_linear's bit for bit."""
    import torch
    from paper_2506_05413_b200 import build, binding as sr
    build.build()
    dev = "cuda:0"
    t = lambda a: torch.from_numpy(np.ascontiguousarray(a)).to(dev)
    for call, (M, N, K, fits) in enumerate([(257, 3200, 8192, True), (512, 4096, 8192, False)]):
        need = sr.workspace_bytes(M, N, K)
        assert need > 0 and (need <= sr.STATIC_SCRATCH_BYTES) == fits
        xq, dx, wq, dw = (t(a) for a in _case(300 + call, M, N, K))
        ws = torch.empty(need, dtype=torch.uint8, device=dev)
        Y_ref = torch.empty((M, N), dtype=torch.float16, device=dev)
        sr.linear(xq, dx, wq, dw, Y_ref, ws)
        Y = torch.full((M, N), float("nan"), dtype=torch.float16, device=dev)
        sr.linear_static_scratch(xq, dx, wq, dw, Y)
        torch.cuda.synchronize()
        assert sr.device_status() == 0
        assert torch.equal(Y, Y_ref)
