"""The C-ABI boundary without a GPU: the library loads, exports every symbol
the header declares, and rejects bad arguments before touching the device."""
import ctypes
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
HEADER = os.path.join(ROOT, "include", "smoothrot.h")


@pytest.fixture(scope="module")
def lib():
    from paper_2506_05413_b200 import build, binding
    build.build()
    return binding.load()


def _declared():
    text = open(HEADER).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(smoothrot_[a-z0-9_]+)\s*\(", text)))


def test_every_declared_symbol_is_exported_and_bound(lib):
    from paper_2506_05413_b200 import binding
    names = _declared()
    assert "smoothrot_quant_act" in names and "smoothrot_linear" in names and len(names) >= 11
    for n in names:
        assert hasattr(lib, n), n
        assert n in binding.SIGNATURES, f"{n} has no ctypes signature"
    assert sorted(binding.SIGNATURES) == names


def test_status_strings(lib):
    from paper_2506_05413_b200 import binding
    assert binding.status_string(0) == "ok"
    texts = {binding.status_string(c) for c in range(-6, 1)}
    assert len(texts) == 7 and binding.status_string(-99) == "unknown status"


def test_host_side_rejections(lib):
    dummy = ctypes.c_void_p(0x1000)   # never dereferenced: each call fails validation first
    odd = ctypes.c_void_p(0x1008)
    q = lib.smoothrot_quant_act
    assert q(dummy, 4, 100, 104, None, 0.9, dummy, dummy, None) == -2        # unsupported K
    assert q(dummy, 4, 64, 64, None, 0.9, dummy, dummy, None) == -2          # 2^6 too small
    assert q(dummy, 4, 28 * 2048, 28 * 2048, None, 0.9, dummy, dummy, None) == -2
    assert q(dummy, -1, 128, 128, None, 0.9, dummy, dummy, None) == -1       # negative rows
    assert q(None, 4, 128, 128, None, 0.9, dummy, dummy, None) == -1         # null input
    assert q(dummy, 4, 128, 64, None, 0.9, dummy, dummy, None) == -1         # ld < K
    assert q(odd, 4, 128, 128, None, 0.9, dummy, dummy, None) == -3          # misaligned
    assert q(dummy, 4, 128, 132, None, 0.9, dummy, dummy, None) == -3        # ld not multiple of 8
    assert q(dummy, 4, 128, 128, None, 0.0, dummy, dummy, None) == -1        # clip out of range
    assert q(dummy, 4, 128, 128, None, 1.5, dummy, dummy, None) == -1
    assert q(dummy, 0, 128, 128, None, 0.9, None, None, None) == 0           # empty input is fine
    assert lib.smoothrot_fuse_weights(dummy, 4, 88, 88, None, 1.0, dummy, dummy, None) == -2
    qp = lib.smoothrot_quant_act_plain
    assert qp(dummy, 4, 100, 104, None, 0.9, dummy, dummy, None) == -2           # K % 8
    assert qp(dummy, 4, 32768, 32768, None, 0.9, dummy, dummy, None) == -2       # K too long
    assert qp(dummy, 4, 128, 64, None, 0.9, dummy, dummy, None) == -1            # ldx < K
    assert qp(odd, 4, 128, 128, None, 0.9, dummy, dummy, None) == -3
    assert qp(dummy, 0, 128, 128, None, 0.9, None, None, None) == 0
    qh = lib.smoothrot_quant_act_heads
    assert qh(dummy, 4, 12, 128, 1536, None, 0.9, dummy, dummy, None) == -2      # 12 heads: not a power of two
    assert qh(dummy, 4, 32, 96, 3072, None, 0.9, dummy, dummy, None) == -2       # head_dim 96
    assert qh(dummy, 4, 32, 128, 4000, None, 0.9, dummy, dummy, None) == -1      # ldx < K
    assert qh(dummy, 4, 32, 128, 4096, None, 0.0, dummy, dummy, None) == -1
    assert qh(odd, 4, 32, 128, 4096, None, 0.9, dummy, dummy, None) == -3
    assert qh(dummy, 0, 32, 128, 4096, None, 0.9, None, None, None) == 0
    ld = lib.smoothrot_linear_decode
    assert ld(dummy, 5, 4096, 4096, 1, None, 0.9, dummy, dummy, 16, dummy, 16, None, None, None) == -1    # M > 4, rotated
    assert ld(dummy, 9, 4096, 4096, 0, None, 0.9, dummy, dummy, 16, dummy, 16, None, None, None) == -1    # M > 8, plain
    assert ld(dummy, 2, 2048, 2048, 1, None, 0.9, dummy, dummy, 16, dummy, 16, None, None, None) == -2    # rotated: K = 4096 only
    assert ld(dummy, 2, 8192, 8192, 0, None, 0.9, dummy, dummy, 16, dummy, 16, None, None, None) == -2    # plain: K <= 4096
    assert ld(dummy, 2, 4096, 4096, 2, None, 0.9, dummy, dummy, 16, dummy, 16, None, None, None) == -1    # rotation flag
    assert ld(dummy, 2, 4096, 4096, 1, None, 0.9, dummy, dummy, 12, dummy, 16, None, None, None) == -1    # N % 8
    assert ld(odd, 2, 4096, 4096, 0, None, 0.9, dummy, dummy, 16, dummy, 16, None, None, None) == -3
    assert ld(dummy, 0, 4096, 4096, 1, None, 0.9, dummy, dummy, 16, dummy, 16, None, None, None) == 0
    ldh = lib.smoothrot_linear_decode_heads
    assert ldh(dummy, 5, 32, 128, 4096, None, 0.9, dummy, dummy, 16, dummy, 16, None, None, None) == -1   # M > 4
    assert ldh(dummy, 2, 16, 128, 2048, None, 0.9, dummy, dummy, 16, dummy, 16, None, None, None) == -2   # 32 x 128 only
    assert ldh(dummy, 2, 32, 128, 4000, None, 0.9, dummy, dummy, 16, dummy, 16, None, None, None) == -1   # ldx < K
    assert ldh(dummy, 0, 32, 128, 4096, None, 0.9, dummy, dummy, 16, dummy, 16, None, None, None) == 0
    lin = lib.smoothrot_linear
    assert lin(dummy, dummy, 4, dummy, dummy, 8, 100, dummy, 8, None, 0, None) == -2   # K % 128
    assert lin(dummy, dummy, 4, dummy, dummy, 12, 128, dummy, 16, None, 0, None) == -1  # N % 8
    assert lin(dummy, dummy, 4, dummy, dummy, 8, 128, dummy, 4, None, 0, None) == -1   # ldy < N
    assert lin(odd, dummy, 4, dummy, dummy, 8, 128, dummy, 8, None, 0, None) == -3
    assert lin(dummy, dummy, 0, dummy, dummy, 8, 128, dummy, 8, None, 0, None) == 0
    # a shape that splits K needs a workspace
    need = lib.smoothrot_workspace_bytes(100, 256, 16384)
    assert need > 0 and need % (4 * 256 * 4) == 0
    assert lin(dummy, dummy, 100, dummy, dummy, 256, 16384, dummy, 256, None, 0, None) == -4
    assert lin(dummy, dummy, 100, dummy, dummy, 256, 16384, dummy, 256, dummy, need - 1, None) == -4
    assert lib.smoothrot_workspace_bytes(128, 1024, 4096) == 0   # k-splits reduced inside a cluster
    assert lib.smoothrot_workspace_bytes(32, 256, 16384) == 0    # few tokens: the decode kernel splits K inside a CTA
    assert lib.smoothrot_workspace_bytes(2048, 6144, 4096) == 0
    cal = lib.smoothrot_calibrate
    assert cal(dummy, 4, 128, 128, None, 0, 0, 0.5, 1, dummy, dummy, None, None, None, None) == -1  # finalize, no W
    assert cal(dummy, 4, 128, 128, dummy, 4, 128, 1.5, 1, dummy, dummy, None, None, None, None) == -1  # alpha
    assert cal(dummy, 4, 128, 128, None, 0, 0, 0.5, 0, None, None, None, None, None, None) == -1
    assert lib.smoothrot_paley28(None) == -1
    assert lib.smoothrot_base_matrix(12, None) == -1
    assert lib.smoothrot_device_status(None, 0) == -1


def test_library_paley_table_equals_oracle_table(lib):
    import numpy as np
    from oracle import smoothrot_oracle as orc
    from paper_2506_05413_b200 import binding
    assert np.array_equal(np.array(binding.paley28(), dtype=np.int8), orc.paley28())
    for order in (12, 20, 28):
        assert np.array_equal(np.array(binding.base_matrix(order), dtype=np.int8), orc.base_matrix(order))
    assert lib.smoothrot_base_matrix(16, None) == -1
