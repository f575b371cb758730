"""Host-side checks of the C ABI that need no GPU: the library loads, exports
every symbol the header declares, answers size queries and rejects bad
arguments before anything is launched."""
import ctypes
import os
import re

import pytest

from paper_2607_00501_b200 import _build, qmm, synth

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def L():
    _build.build()
    return qmm.lib()


def test_header_symbols_are_exported(L):
    hdr = open(os.path.join(ROOT, "include", "qmm.h")).read()
    hdr = re.sub(r"/\*.*?\*/", "", hdr, flags=re.S)
    declared = set(re.findall(r"\b(qmm_[a-z_]+)\s*\(", hdr))
    assert declared == set(qmm.EXPORTS)
    for name in declared:
        assert hasattr(L, name), name


def test_version_and_sizes(L):
    assert qmm.version() >= 100
    assert qmm.canonical_bytes(4, 3072, 1024) == 1769472 == synth.canonical_bytes(4, 3072, 1024)
    assert qmm.canonical_bytes(8, 128256, 3072) == 418627584
    assert qmm.canonical_bytes(4, 128, 31) == 0
    assert qmm.packed_bytes(4, 3072, 1024) == 1769472
    assert qmm.packed_bytes(8, 128256, 3072) == 418627584
    # packed buffers with the same K concatenate row-wise
    assert qmm.packed_bytes(4, 2048, 2048) + 2 * qmm.packed_bytes(4, 512, 2048) == qmm.packed_bytes(4, 3072, 2048)


@pytest.mark.parametrize("fmt,N,K,status", [
    (7, 128, 256, 1), (4, 0, 256, 1), (4, 128, -256, 1), (4, 128, 100, 2), (4, 128, 288, 5), (4, 100, 256, 5),
])
def test_bad_shapes_are_rejected(L, fmt, N, K, status):
    buf = (ctypes.c_char * 64)()
    addr = ctypes.addressof(buf)
    assert L.qmm_pack(fmt, addr, N, K, addr, None) == status
    assert qmm.last_error()
    assert L.qmm_gemv(fmt, addr, N, K, addr, addr, None, 0, None) == status
    assert L.qmm_gemm(fmt, addr, N, K, addr, K, addr, N, 4, addr, 0, None) == status
    with pytest.raises(qmm.QmmError):
        qmm.packed_bytes(fmt, N, K)


def test_null_and_misaligned_pointers(L):
    buf = (ctypes.c_char * 512)()
    a = (ctypes.addressof(buf) + 255) & ~255
    assert L.qmm_pack(4, None, 128, 256, a, None) == 1
    assert L.qmm_pack(4, a, 128, 256, a + 8, None) == 3
    assert L.qmm_dequant(4, a, 128, 256, None, None) == 1
    assert L.qmm_gemv(4, a, 128, 256, None, a, None, 0, None) == 1
    assert L.qmm_gemv(4, a, 128, 256, a + 2, a, None, 0, None) == 3
    assert L.qmm_gemv(4, a + 16, 128, 256, a, a, None, 0, None) == 3
    assert "aligned" in qmm.last_error()
    assert L.qmm_gemv(4, a, 128, 65536, a, a, None, 0, None) == 5                  # K beyond the GEMV's shared-memory staging
    assert L.qmm_gemm(4, a, 128, 256, a, 255, a, 128, 4, a, 1 << 20, None) == 2     # ldx < K
    assert L.qmm_gemm(4, a, 128, 256, a, 260, a, 128, 4, a, 1 << 20, None) == 3     # ldx % 8
    assert L.qmm_gemm(4, a, 128, 256, a, 256, a, 128, -1, a, 1 << 20, None) == 1
    assert L.qmm_gemm(4, a, 128, 256, a, 256, a, 128, 0, a, 0, None) == 0           # M = 0: nothing to do
    assert L.qmm_gemm(4, a, 128, 256, a, 256, a, 128, 4, None, 0, None) == 4
    assert L.qmm_status_check(None, None) == 1


def test_gemv_workspace_rule(L):
    assert qmm.gemv_workspace_bytes(4, 512, 2048) == 0            # the plan's K split fits a cluster: no workspace
    qmm.debug_config("gemv_force", "8,4")
    assert qmm.gemv_workspace_bytes(4, 512, 2048) == 0            # forced 4-way split: still a cluster
    qmm.debug_config("gemv_force", "8,16")
    assert qmm.gemv_workspace_bytes(4, 512, 8192) == 16 * 512 * 4  # beyond a cluster: partial sums in the workspace
    qmm.debug_config("gemv_force", "8,4")
    qmm.debug_config("gemv_no_cluster", "1")
    need = qmm.gemv_workspace_bytes(4, 512, 2048)
    assert need == 4 * 512 * 4
    buf = (ctypes.c_char * 512)()
    a = (ctypes.addressof(buf) + 255) & ~255
    assert L.qmm_gemv(4, a, 512, 2048, a, a, None, 0, None) == 4
    assert L.qmm_gemv(4, a, 512, 2048, a, a, a, need - 1, None) == 4
    assert "workspace" in qmm.last_error()
    qmm.debug_config("gemv_force", "8,1")
    assert qmm.gemv_workspace_bytes(4, 512, 2048) == 0


def test_debug_config_rejects_what_it_does_not_know(L):
    assert L.qmm_debug_config(b"no_such_knob", b"1") == 1
    assert "unknown knob" in qmm.last_error()
    assert L.qmm_debug_config(b"gemv_force", b"12,1") == 1
    assert L.qmm_debug_config(b"gemm_force", b"100") == 1
    assert L.qmm_debug_config(b"gemm_force", b"128,0") == 1
    assert L.qmm_debug_config(b"gemm_force", b"128,5") == 0
    assert L.qmm_debug_config(None, None) == 0
    buf = (ctypes.c_char * 512)()
    a = (ctypes.addressof(buf) + 255) & ~255
    assert L.qmm_debug_wait_give_up(None, 1000, None) == 1
    assert L.qmm_debug_wait_give_up(a, 0, None) == 1
    assert L.qmm_debug_wait_give_up(a, 1 << 30, None) == 1
    assert L.qmm_packed_check(4, None, 128, 256, a, None) == 1
    assert L.qmm_packed_check(4, a, 128, 100, a, None) == 2
    assert L.qmm_packed_check(4, a + 16, 128, 256, a, None) == 3


def test_gemm_workspace_rule(L):
    """The workspace is a fixed header, plus fp32 partial-sum slots exactly when the plan cuts tiles
    along K (few output tiles); the plan is a pure function of the shape."""
    qmm.debug_config(None)
    header = qmm.gemm_workspace_bytes(4, 2048, 8192, 3072)        # 512 whole tiles: nothing to add up
    assert header == 8192
    assert qmm.gemm_workspace_bytes(8, 2048, 8192, 3072) == header
    assert qmm.gemm_workspace_bytes(4, 1024, 3072, 8192) == header    # 96 tiles: whole tiles, one round
    assert qmm.gemm_workspace_bytes(4, 256, 8192, 3072) == header     # 128 tiles of 128 tokens instead of a K split
    few = qmm.gemm_workspace_bytes(4, 256, 3072, 8192)                 # 24 tiles of 256 tokens: K cut in 4
    assert few == header + 2 * 96 * 256 * 128 * 4
    assert qmm.gemm_workspace_bytes(4, 256, 3072, 8192) == few         # same answer every time
    # 192 tiles of 128 k-blocks: one whole tile per block, the 44 tiles of the second round in equal shares
    assert qmm.gemm_workspace_bytes(4, 2048, 3072, 8192) == header + 2 * 148 * 256 * 128 * 4
    tiny = qmm.gemm_workspace_bytes(4, 1, 128, 256)                    # one tile, 4 k-blocks: too short to cut
    assert tiny == header
    qmm.debug_config("gemm_force", "128,5")
    forced = qmm.gemm_workspace_bytes(4, 100, 256, 2048)               # 2 tiles x 32 k-blocks in shares of 5: 13 blocks
    assert forced == header + 2 * 13 * 128 * 128 * 4
    buf = (ctypes.c_char * 512)()
    a = (ctypes.addressof(buf) + 255) & ~255
    assert L.qmm_gemm(4, a, 256, 2048, a, 2048, a, 256, 100, a, forced - 1, None) == 4
    assert "workspace" in qmm.last_error()


def test_empty_inputs_are_accepted_and_do_nothing(L):
    """M = 0 and T = 0 return QMM_OK before anything is launched (so no GPU is needed to see it);
    negative sizes are argument errors."""
    buf = (ctypes.c_char * 512)()
    a = (ctypes.addressof(buf) + 255) & ~255
    assert L.qmm_gemm(4, a, 128, 256, a, 256, a, 128, 0, None, 0, None) == 0
    assert L.qmm_gemm(4, a, 128, 256, a, 256, a, 128, -1, None, 0, None) == 1
    assert L.qmm_gemv_batch(4, None, 0, None) == 0
    assert L.qmm_gemv_batch(4, None, -1, None) == 1
    assert L.qmm_gemm_batch(4, None, 0, 4, None) == 0 and L.qmm_gemm_batch(4, None, 3, 0, None) == 0
    assert L.qmm_gemm_batch(4, None, -1, 4, None) == 1 and L.qmm_gemm_batch(4, None, 3, 4, None) == 1
    assert L.qmm_gemm_batch(4, None, 3, 9, None) == 5
    m = qmm.MoeArgs(0, 2048, 768, 128, 8, 4, a, a, a, a, a, a, None, None, None, None, None, None)
    assert L.qmm_moe(ctypes.byref(m), None, 0, None) == 0
    assert L.qmm_moe_route(ctypes.byref(m), None, 0, None) == 0
    m.T = -1
    assert L.qmm_moe(ctypes.byref(m), None, 0, None) == 1


def test_moe_argument_checks(L):
    buf = (ctypes.c_char * 512)()
    a = (ctypes.addressof(buf) + 255) & ~255
    ok = dict(fmt=4, T=4, H=2048, I=768, E=128, topk=8)

    def args(**kw):
        d = dict(ok, **kw)
        return qmm.MoeArgs(d["T"], d["H"], d["I"], d["E"], d["topk"], d["fmt"], a, a, a, a, a, a, 0, 0, 0, 0, 0, 0)

    assert L.qmm_moe(None, a, 0, None) == 1
    assert L.qmm_moe(ctypes.byref(args(topk=200)), a, 1 << 30, None) == 2
    assert L.qmm_moe(ctypes.byref(args(E=0)), a, 1 << 30, None) == 1
    assert L.qmm_moe(ctypes.byref(args(H=2000)), a, 1 << 30, None) == 2
    assert L.qmm_moe(ctypes.byref(args(I=96)), a, 1 << 30, None) == 5
    assert L.qmm_moe(ctypes.byref(args()), a, 16, None) == 4
    assert L.qmm_moe_workspace_bytes(ctypes.byref(args())) > 0
    assert L.qmm_moe_workspace_bytes(ctypes.byref(args(fmt=3))) == 0


def test_error_buffer_is_thread_local(L):
    import threading
    buf = (ctypes.c_char * 64)()
    addr = ctypes.addressof(buf)
    L.qmm_pack(4, addr, 128, 100, addr, None)
    mine = qmm.last_error()
    seen = []
    t = threading.Thread(target=lambda: seen.append(qmm.last_error()))
    t.start()
    t.join()
    assert "K=100" in mine and seen == [""]
