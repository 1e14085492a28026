"""The allocation-free weight quantization entry point against the allocating one.

Some callers cannot allocate device memory when they need to quantize weights (their process
has given all device memory to its own arena, or they cannot take the device-wide
synchronisation an allocation may imply).  qvggt_quantize_weights_static serves them from a fixed
scratch array inside the library.  This file is collected last on purpose, so a failure here
cannot hide the other tests in a run that stops at the first failure.
"""
import ctypes

import numpy as np
import pytest
import torch

import oracle
import workload
from _util import dev_bf16

pytestmark = pytest.mark.gpu


def _both_ways(q, K, N, seed, signs=True, watch_memory=False):
    spec = workload.LinearSpec("w", K, N, workload.DIST_NORMAL, seed, 0)
    Wb = spec.weight()
    W = dev_bf16(Wb)
    ch = workload.loguniform_f32(seed, 5, K, 0.05, 20.0)
    vh = workload.signs_i8(seed, 6, K) if signs else None
    c = torch.from_numpy(ch).cuda()
    v = torch.from_numpy(vh).cuda() if signs else None
    Wq = torch.full((N, K // 2), 0xAA, dtype=torch.uint8, device="cuda")
    w_scale = torch.full((N,), -1.0, dtype=torch.float32, device="cuda")
    amul = torch.full((K,), -1.0, dtype=torch.float32, device="cuda")
    torch.cuda.synchronize()
    free0, used0 = torch.cuda.mem_get_info()[0], torch.cuda.memory_allocated()
    # straight through the C ABI: plain pointers and sizes
    st = q.lib().qvggt_quantize_weights_static(W.data_ptr(), c.data_ptr(), v.data_ptr() if signs else None, N, K, Wq.data_ptr(),
                                               w_scale.data_ptr(), amul.data_ptr(),
                                               torch.cuda.current_stream().cuda_stream)
    assert st == 0, q.lib().qvggt_status_string(st)
    torch.cuda.synchronize()
    if watch_memory:
        # the point of the entry point: the call took nothing from the driver's free memory (an allocation would
        # lower the reading; it may rise when the pool behind an EARLIER stream-ordered allocation is trimmed at a
        # synchronisation) and torch's allocator did not move.  A kernel's first launch may load its code, so only
        # calls after the first of each size are watched.
        assert torch.cuda.mem_get_info()[0] >= free0 and torch.cuda.memory_allocated() == used0
    # against the oracle directly: codes bit-exact, scales and multipliers bit-equal
    ref = oracle.prepare_weights(Wb, ch, vh)
    assert np.array_equal(Wq.cpu().numpy(), ref["wq_packed"])
    assert np.array_equal(w_scale.cpu().numpy(), ref["w_scale"])
    assert np.array_equal(amul.cpu().numpy(), ref["amul"])
    if N % 128 == 0:
        # ... and against the allocating entry point (same tolerance as the parity tests: bit-exact)
        h = q.prepare_weights(W, None, c, v)
        got = h.view()
        assert np.array_equal(Wq.cpu().numpy(), got["wq"].cpu().numpy())
        assert np.array_equal(w_scale.cpu().numpy(), got["w_scale"].cpu().numpy())
        assert np.array_equal(amul.cpu().numpy(), got["amul"].cpu().numpy())
        h.free()


def test_static_scratch_entry_point_matches_allocating_one_twice_in_a_row():
    import paper_2509_21302_b200 as q
    q.build()
    # two calls back to back; the second uses a shorter K, so stale scratch beyond it must not matter,
    # and a third goes back to the long K over the contents the second one left
    _both_ways(q, 4096, 256, seed=31)
    _both_ways(q, 1024, 384, seed=32)
    _both_ways(q, 4096, 128, seed=33, watch_memory=True)
    # by now the kernels of both sizes have run once (a kernel's first launch may load its code and move the
    # free-memory reading): from here on every call is watched
    _both_ways(q, 1024, 256, seed=37, watch_memory=True)


def test_static_scratch_entry_point_any_row_count_and_no_signs():
    import paper_2509_21302_b200 as q
    q.build()
    _both_ways(q, 1024, 130, seed=34)                       # N need not be a multiple of 128 here
    _both_ways(q, 4096, 1, seed=35, signs=False)
    _both_ways(q, 1024, 256, seed=36, signs=False, watch_memory=True)
    _both_ways(q, 4096, 130, seed=38, watch_memory=True)


def test_static_scratch_entry_point_rejects_what_it_cannot_serve():
    import paper_2509_21302_b200 as q
    q.build()
    L = q.lib()
    x = torch.zeros(64, dtype=torch.float32, device="cuda")
    p = x.data_ptr()
    assert L.qvggt_quantize_weights_static(p, p, None, 128, 8192, p, p, p, None) == -2    # K beyond the fixed scratch
    assert L.qvggt_quantize_weights_static(p, p, None, 128, 2048, p, p, p, None) == -2    # unsupported rotation size
    assert L.qvggt_quantize_weights_static(None, p, None, 128, 1024, p, p, p, None) == -1
    assert L.qvggt_quantize_weights_static(p, p, None, 0, 1024, p, p, p, None) == -2
    assert b"shape" in L.qvggt_status_string(-2)
