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

import workload
from _util import dev_bf16

pytestmark = pytest.mark.gpu


def _both_ways(q, K, N, seed):
    spec = workload.LinearSpec("w", K, N, workload.DIST_NORMAL, seed, 0)
    W = dev_bf16(spec.weight())
    c = torch.from_numpy(workload.loguniform_f32(seed, 5, K, 0.05, 20.0)).cuda()
    v = torch.from_numpy(workload.signs_i8(seed, 6, K)).cuda()
    ref = q.prepare_weights(W, None, c, v).view()
    Wq = torch.full((N, K // 2), 0xAA, dtype=torch.uint8, device="cuda")
    w_scale = torch.full((N,), -1.0, dtype=torch.float32, device="cuda")
    amul = torch.full((K,), -1.0, dtype=torch.float32, device="cuda")
    # straight through the C ABI: plain pointers and sizes
    st = q.lib().qvggt_quantize_weights_static(W.data_ptr(), c.data_ptr(), v.data_ptr(), N, K, Wq.data_ptr(),
                                               w_scale.data_ptr(), amul.data_ptr(),
                                               torch.cuda.current_stream().cuda_stream)
    assert st == 0, q.lib().qvggt_status_string(st)
    torch.cuda.synchronize()
    # same tolerance as the parity tests: codes bit-exact, scales bit-equal
    assert np.array_equal(Wq.cpu().numpy(), ref["wq"].cpu().numpy())
    assert np.array_equal(w_scale.cpu().numpy(), ref["w_scale"].cpu().numpy())
    assert np.array_equal(amul.cpu().numpy(), ref["amul"].cpu().numpy())


def test_static_scratch_entry_point_matches_allocating_one_twice_in_a_row():
    import paper_2509_21302_b200 as q
    q.build()
    # two calls back to back; the second uses a shorter K, so stale scratch beyond it must not matter,
    # and a third goes back to the long K over the contents the second one left
    _both_ways(q, 4096, 256, seed=31)
    _both_ways(q, 1024, 384, seed=32)
    _both_ways(q, 4096, 128, seed=33)


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
