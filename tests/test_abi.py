"""The C-ABI library builds, loads, exports every symbol the header declares, and rejects bad arguments
before touching a device (no GPU needed: these calls return before any CUDA work)."""
import ctypes
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def L():
    from paper_2412_07174_b200 import build
    build.build()
    from paper_2412_07174_b200 import binding
    return binding.lib()


def declared_symbols():
    text = open(os.path.join(ROOT, "include", "scap.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(scap_[a-z_0-9]+)\s*\(", text)))


def test_every_declared_symbol_is_exported(L):
    from paper_2412_07174_b200 import binding
    syms = declared_symbols()
    assert len(syms) >= 16
    for s in syms:
        assert hasattr(L, s), s
    assert sorted(binding.EXPORTS) == syms


def test_status_strings_and_version(L):
    assert L.scap_status_string(0) == b"SCAP_OK"
    assert L.scap_status_string(4) == b"SCAP_ERR_ALIGN"
    assert L.scap_version() >= 1000


def test_workspace_queries_without_a_device(L):
    assert L.scap_fc_workspace(1, 11008, 4096) > 0
    assert L.scap_glu_workspace(16, 4096, 14336) > L.scap_glu_workspace(1, 4096, 14336)
    assert L.scap_fc_workspace(17, 64, 64) == 0 and L.scap_fc_workspace(1, 0, 64) == 0
    assert L.scap_glu_workspace(8, 4096, 11008) > 0
    assert L.scap_moe_workspace(4, 4096, 14336, 8, 2) > 0
    assert L.scap_moe_workspace(4, 4096, 14336, 8, 9) == 0
    assert L.scap_calibrate_workspace(2048, 14336, 2048) > 0
    assert L.scap_fc_host_workspace(1, 1024, 1024) > L.scap_fc_workspace(1, 1024, 1024)


def test_argument_validation_returns_codes(L):
    P = 0x10000  # a fake, 16-byte aligned, never dereferenced address
    ws = L.scap_fc_workspace(1, 64, 64)
    call = lambda **kw: L.scap_sparse_fc(*[kw.get(k, v) for k, v in dict(
        x=P, W=P, m=None, tau=P, b=None, y=P, B=1, K=64, N=64, dt=1, idx=None, nnz=None, ws=P, wsb=ws, st=None).items()])
    assert call(x=None) == 1                      # SCAP_ERR_INVALID_ARG
    assert call(tau=None) == 1
    assert call(B=0) == 2 and call(B=17) == 2     # SCAP_ERR_SHAPE
    assert call(K=0) == 2 and call(K=(1 << 20) + 1) == 2
    assert call(dt=7) == 3                        # SCAP_ERR_DTYPE
    assert call(N=60) == 4 and call(W=P + 2) == 4  # SCAP_ERR_ALIGN
    assert call(wsb=ws - 1) == 5                  # SCAP_ERR_WORKSPACE
    assert L.scap_tune(b"no_such_key", 1) == 1
    assert L.scap_tune(b"split_k", 9) == 1
    assert L.scap_tune(b"split_k", 0) == 0
    assert L.scap_tune(b"fma_rows", 3) == 1
    assert L.scap_tune(b"fma_rows", 2) == 0
    assert L.scap_tune(b"fma_rows", 4) == 0
    assert L.scap_tune(b"l2_hints", 0) == 0
    assert L.scap_tune(b"l2_hints", 1) == 0
    assert L.scap_tune(b"cal_strip", 24) == 1
    assert L.scap_tune(b"cal_strip", 32) == 0
    assert L.scap_tune(b"cal_strip", 16) == 0
    assert L.scap_tune(b"tcgen05", 3) == 1
    assert L.scap_tune(b"tcgen05", -1) == 1
    for v in (0, 2, 1):  # leaves the default
        assert L.scap_tune(b"tcgen05", v) == 0
    assert L.scap_calibrate(P, 16, 12, 1, 0.5, 16, P, P, P, 1 << 20, None) == 4   # K not a multiple of 8
    assert L.scap_calibrate(P, 16, 16, 1, 1.5, 16, P, P, P, 1 << 20, None) == 1   # sparsity outside [0, 1)
    assert L.scap_glu_ffn(P, P, P, None, P, None, None, P, None, P, 1, 64, 60, 1, None, None, None, None, None, P,
                          1 << 30, None) == 4
    assert L.scap_moe_ffn(P, P, None, 8, 2, P, 1, 64, 64, 1, None, None, P, 1 << 30, None) == 1
