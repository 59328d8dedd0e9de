"""Host-side checks of the C-ABI library: it loads, exports every declared symbol, sizes agree with
the oracle's layout, and argument validation returns error codes before any launch (no GPU needed)."""

import ctypes
import os
import re

import pytest

import paper_2510_19482_b200 as elutq
from oracle import layout

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _declared_symbols():
    text = open(os.path.join(ROOT, "include", "elutq.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(elutq_[a-z0-9_]+)\s*\(", text)))


def test_library_exports_every_declared_symbol():
    names = _declared_symbols()
    assert "elutq_pack" in names and "elutq_lut_gemm" in names and "elutq_lut_gemm_bias" in names
    handle = ctypes.CDLL(elutq.library_path())
    for n in names:
        assert hasattr(handle, n), f"{n} declared in elutq.h but not exported"


def test_binding_has_the_same_names():
    for n in _declared_symbols():
        assert hasattr(elutq, n), f"binding lacks {n}"


@pytest.mark.parametrize("q,G,N,K", [(2, 128, 4096, 4096), (3, 64, 21, 640), (4, 32, 5, 96), (1, 128, 28672, 4096)])
def test_packed_bytes_equals_reference_layout(q, G, N, K):
    assert elutq.elutq_packed_bytes(q, G, N, K) == layout.packed_bytes(q, G, N, K)


def test_shape_validation_codes():
    L = elutq.lib()
    out = ctypes.c_size_t(0)
    assert L.elutq_packed_bytes(0, 128, 16, 512, ctypes.byref(out)) == -2       # q out of range
    assert L.elutq_packed_bytes(5, 128, 16, 512, ctypes.byref(out)) == -2
    assert L.elutq_packed_bytes(2, 100, 16, 500, ctypes.byref(out)) == -2       # unsupported G
    assert L.elutq_packed_bytes(2, 128, 16, 500, ctypes.byref(out)) == -2       # K % G != 0
    assert L.elutq_packed_bytes(2, 128, 0, 512, ctypes.byref(out)) == -1
    assert L.elutq_packed_bytes(2, 128, 16, 512, None) == -1
    assert L.elutq_workspace_bytes(0, 16, 512, ctypes.byref(out)) == -1
    assert L.elutq_workspace_bytes(1, 16, 512, ctypes.byref(out)) == 0 and out.value == 256   # one chunk: counters only


def test_pointer_validation_happens_before_any_launch():
    L = elutq.lib()
    before = elutq.elutq_launch_count()
    assert L.elutq_pack(None, None, None, 2, 128, 16, 512, None, 0, None) == -1
    assert L.elutq_pack(8, 8, 8, 2, 128, 16, 512, 16, 10, None) == -4            # packed buffer too small
    assert L.elutq_pack(4, 8, 8, 2, 128, 16, 512, 16, 1 << 20, None) == -3       # planes not 8-byte aligned
    assert L.elutq_pack(8, 8, 8, 2, 128, 16, 512, 24, 1 << 20, None) == -3       # packed not 16-byte aligned
    assert L.elutq_lut_gemm(None, None, None, 1, 16, 512, None) == -1
    assert L.elutq_lut_gemm(16, 16, 16, 0, 16, 512, None) == -1
    assert L.elutq_lut_gemm(8, 16, 16, 1, 16, 512, None) == -3
    assert L.elutq_lut_gemm_ws(16, 16, 16, 1, 16, 512, 0x3, 16, 1 << 20, None) == -1   # skip-offset + offset-only
    assert L.elutq_lut_gemm_ws(16, 16, 16, 1, 16, 512, 0x400, 16, 1 << 20, None) == -1
    assert L.elutq_lut_gemm_ws(16, 16, 16, 4, 16, 512, 0x300, 16, 1 << 20, None) == -1      # fp16 + int8 tables
    assert L.elutq_lut_gemm_ws(16, 16, 16, 1, 16, 512, 0x50, 16, 1 << 20, None) == -1       # plain g4 + mirror
    assert L.elutq_hlq_fit(None, 2, 128, 16, 512, 10, None, None, None, None, None) == -1
    assert L.elutq_hlq_fit(16, 2, 128, 16, 512, 0, 16, 16, 16, None, None) == -1          # t_max < 1
    assert L.elutq_hlq_fit(16, 5, 128, 16, 512, 10, 16, 16, 16, None, None) == -2         # q out of range
    assert L.elutq_hlq_fit(16, 2, 128, 16, 500, 10, 16, 16, 16, None, None) == -2         # K % G != 0
    assert L.elutq_hlq_fit(17, 2, 128, 16, 512, 10, 16, 16, 16, None, None) == -3         # W not 2-byte aligned
    assert L.elutq_hlq_fit(16, 2, 128, 16, 512, 10, 16, 16, 16, 4, None) == -3            # trace not 8-byte aligned
    assert L.elutq_workspace_init(None, 16, None) == -1
    assert L.elutq_forget(None) == -1
    assert elutq.elutq_launch_count() == before
    assert elutq.elutq_status_string(-4) == "buffer too small"


def test_chain_argument_validation_happens_on_the_host():
    L = elutq.lib()
    out = ctypes.c_size_t(0)
    before = elutq.elutq_launch_count()
    good = (elutq.GemvCall * 2)(elutq.GemvCall(16, 16, 16, 64, 1024, 0), elutq.GemvCall(32, 32, 32, 4096, 4096, 0x4))
    assert L.elutq_chain_plan_bytes(good, 2, ctypes.byref(out)) == 0
    # control block + counters + descriptors + CTA shares + three scratch regions of 8 chunks x 4096 rows x 8 bytes
    assert out.value > 3 * 8 * 4096 * 8
    assert L.elutq_chain_plan_bytes(None, 2, ctypes.byref(out)) == -1
    assert L.elutq_chain_plan_bytes(good, 0, ctypes.byref(out)) == -1
    assert L.elutq_chain_plan_bytes(good, 5000, ctypes.byref(out)) == -1
    bad = (elutq.GemvCall * 1)(elutq.GemvCall(16, 16, 0, 64, 1024, 0))
    assert L.elutq_chain_plan_bytes(bad, 1, ctypes.byref(out)) == -1          # null Y
    bad = (elutq.GemvCall * 1)(elutq.GemvCall(8, 16, 16, 64, 1024, 0))
    assert L.elutq_chain_plan_bytes(bad, 1, ctypes.byref(out)) == -3          # X not 16-byte aligned
    bad = (elutq.GemvCall * 1)(elutq.GemvCall(16, 16, 16, 64, 1024, 0x1))
    assert L.elutq_chain_plan_bytes(bad, 1, ctypes.byref(out)) == -5          # term flags are not offered by the chain
    bad = (elutq.GemvCall * 1)(elutq.GemvCall(16, 16, 16, 64, 1024, 0x800))
    assert L.elutq_chain_plan_bytes(bad, 1, ctypes.byref(out)) == -1          # unknown flag
    assert L.elutq_chain_plan(good, 2, None, 0, None) == -1
    assert L.elutq_chain_plan(good, 2, 128, 1 << 30, None) == -3              # plan buffer not 256-byte aligned
    assert L.elutq_chain_plan(good, 2, 256, 16, None) == -4                   # plan buffer too small
    assert L.elutq_chain_run(None, 2, None) == -1
    assert L.elutq_chain_run(256, 2, None) == -2                              # a buffer that was never planned
    assert L.elutq_chain_status(None, None, None) == -1
    # the host-buffer form: a null pointer with a non-zero size is refused before anything is copied or launched
    assert L.elutq_chain_run_host(256, 2, None, 4096, 64, 512, 8192, 64, None) == -1
    assert L.elutq_chain_run_host(256, 2, 512, 4096, 64, 512, None, 64, None) == -1
    assert L.elutq_chain_run_host(256, 2, None, None, 0, None, None, 0, None) == -2      # no copies asked for: a plain run of an unplanned buffer
    assert L.elutq_reserve(0, 16, 512, None) == -1
    assert L.elutq_scratch_address(None, 9, None, None) == -1
    assert elutq.elutq_launch_count() == before
