"""The bounded device-side waits: a wait that nobody satisfies runs out, the kernel returns, the
status word names the place, and the library keeps working.  Nothing here hangs or faults: the
probe waits on a barrier with a limit of one millisecond and then leaves normally."""
import time

import numpy as np
import pytest

from oracle import smoothrot_oracle as orc
from paper_2506_05413_b200 import synth

pytestmark = pytest.mark.gpu


def test_a_wait_that_runs_out_is_reported_and_the_library_stays_usable():
    import torch
    from paper_2506_05413_b200 import build, binding as sr
    build.build()
    sr.load()
    dev = "cuda:0"
    torch.cuda.synchronize()
    assert sr.device_status() == 0
    sr.debug_set_wait_limit_ns(1_000_000)            # one millisecond instead of two seconds
    try:
        t0 = time.perf_counter()
        sr.debug_wait_expiry()
        torch.cuda.synchronize()
        elapsed = time.perf_counter() - t0
        assert elapsed < 1.0, elapsed                # far below the default limit: the short one was used
        assert sr.device_status(clear=False) == 7    # the probe's site code
        assert sr.device_status(clear=True) == 7
        assert sr.device_status() == 0               # cleared
    finally:
        sr.debug_set_wait_limit_ns(0)                # back to the default
    # the next ordinary calls are exact: a tcgen05 GEMM and the rotation kernels
    M, N, K = 512, 2560, 256
    xq = orc.pack_codes(synth.random_codes(11, M, K))
    wq = orc.pack_codes(synth.random_codes(12, N, K))
    t = lambda a: torch.from_numpy(np.ascontiguousarray(a)).to(dev)
    acc = torch.full((M, N), -7777, dtype=torch.int32, device=dev)
    need = sr.workspace_bytes(M, N, K)
    sr.debug_gemm_i32(t(xq), t(wq), acc, torch.empty(need, dtype=torch.uint8, device=dev) if need else None)
    torch.cuda.synchronize()
    assert sr.device_status() == 0
    assert np.array_equal(acc.cpu().numpy(), orc.gemm_i32(orc.unpack_codes(xq), orc.unpack_codes(wq)))
    rng = np.random.default_rng(13)
    X = rng.standard_normal((600, 4096)).astype(np.float16)
    q = torch.empty((600, 2048), dtype=torch.uint8, device=dev)
    step = torch.empty(600, dtype=torch.float32, device=dev)
    sr.quant_act(t(X), None, 0.9, q, step)
    torch.cuda.synchronize()
    assert sr.device_status() == 0
    q_ref, step_ref, _ = orc.quant_act(X, None, 4096, 0.9)
    assert np.abs(step.cpu().numpy() / step_ref - 1).max() <= 1e-6
    a = orc.unpack_codes(q.cpu().numpy()).astype(int)
    b = orc.unpack_codes(q_ref).astype(int)
    assert np.abs(a - b).max() <= 1 and (a != b).mean() <= 1e-4
