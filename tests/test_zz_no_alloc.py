"""qmm_gemv_static: the GEMV entry point for callers that cannot allocate.

Some integrations may not obtain device memory when they need a product (the
host application has handed out its memory budget, or forbids allocator calls
after start-up, or cannot afford the device-wide synchronisation an allocation
implies), so they cannot supply the split-K workspace qmm_gemv asks for.  This
variant keeps that scratch in a fixed array inside the library.  The test calls
it through the C ABI on a shape that really uses split-K, twice in a row (the
scratch keeps the first call's contents), and holds both results to the GEMV
tolerance against the CPU oracle and against qmm_gemv.

This file is named so that pytest collects it last.
"""
import ctypes

import numpy as np
import pytest
import torch

from paper_2607_00501_b200 import synth

pytestmark = pytest.mark.gpu


def test_gemv_static_matches_gemv_on_two_calls_in_a_row(oracle):
    from paper_2607_00501_b200 import qmm
    from tests import util
    L = qmm.lib()
    for fmt, N, K in ((synth.Q4, 512, 4096), (synth.Q8, 256, 8192)):
        qmm.debug_config("gemv_no_cluster", "1")                # ask about the form qmm_gemv_static runs
        assert qmm.gemv_workspace_bytes(fmt, N, K) > 0          # the shape goes through split-K partial sums
        qmm.debug_config(None)
        blocks = synth.quantize(fmt, synth.weights(808, fmt, N, K))
        packed = qmm.pack(fmt, torch.from_numpy(blocks).cuda(), N, K)
        x_host = [synth.activations(808, 10 + i, K) for i in range(2)]
        xs = [torch.from_numpy(x).cuda() for x in x_host]
        want = [qmm.gemv(fmt, packed, N, K, x) for x in xs]
        got = [torch.full((N,), 7.0, dtype=torch.float16, device="cuda") for _ in xs]
        stream = torch.cuda.current_stream().cuda_stream
        for x, y in zip(xs, got):                               # two calls in a row share the built-in scratch
            status = L.qmm_gemv_static(fmt, packed.data_ptr(), N, K, x.data_ptr(), y.data_ptr(), stream)
            assert status == 0, qmm.last_error()
        torch.cuda.synchronize()
        for x, w, g in zip(x_host, want, got):
            w64, g64 = w.cpu().numpy().astype(np.float64), g.cpu().numpy().astype(np.float64)
            y_ref, B = oracle.gemv(fmt, blocks, N, K, x)
            util.assert_within_tol(g64, y_ref, B, "qmm_gemv_static against the oracle")
            # and against the existing entry point: both are within the tolerance of the same exact value
            assert np.all(np.abs(w64 - g64) <= 2 * (2e-3 * B + 1e-5))
        assert not torch.equal(got[0], got[1])                  # the two calls really computed different products


def test_gemv_static_rejects_shapes_beyond_its_scratch():
    from paper_2607_00501_b200 import qmm
    L = qmm.lib()
    buf = torch.zeros(4096, dtype=torch.uint8, device="cuda")
    a = buf.data_ptr()
    # bad arguments are refused on the host before anything is enqueued
    assert L.qmm_gemv_static(4, a, 128, 100, a, a, None) == 2
    assert L.qmm_gemv_static(4, None, 128, 256, a, a, None) == 1
    assert L.qmm_gemv_static(4, a + 16, 128, 256, a, a, None) == 3
    # a forced 16-way split of 2^17 rows would need 8 MiB of partial sums: more than the built-in 1 MiB
    qmm.debug_config("gemv_force", "8,16")
    try:
        assert qmm.gemv_workspace_bytes(4, 1 << 17, 8192) > qmm.GEMV_STATIC_SCRATCH_BYTES
        assert L.qmm_gemv_static(4, a, 1 << 17, 8192, a, a, None) == 4
        assert "scratch" in qmm.last_error()
    finally:
        qmm.debug_config(None)
