"""The bounded device-side waits, exercised from the host without faulting, trapping or hanging anything.

A test hook launches the GEMM with its TMA producers switched off and every wait limited to about half a
millisecond: no operand ever arrives, the first wait runs out, the kernel records which wait gave up, all of its
roles fall through to the common exit, tensor memory is released and the launch completes.  Nothing asynchronous
is in flight at that point.  The context must stay usable: a normal run on a fresh handle afterwards is bit-exact.
"""
import ctypes

import numpy as np
import pytest
import torch

import oracle
import workload
from _util import dev_bf16, host_bits

pytestmark = pytest.mark.gpu

DEV_TIMEOUT_FULL, DEV_TIMEOUT_ACCUM = 1, 3      # operands never arrived / the accumulator was never published
ERR_DEVICE_TIMEOUT = -6


@pytest.mark.parametrize("M,N", [(256, 256), (3000, 1024), (8 * workload.TOKENS_PER_FRAME, 1024)])
def test_starved_gemm_reports_a_timeout_and_leaves_the_context_usable(M, N):
    import paper_2509_21302_b200 as q
    q.build()
    K = 1024
    spec = workload.LinearSpec("starved", K, N, workload.DIST_NORMAL, 77, 0)
    W, b, X = spec.weight(), spec.bias(), spec.x_rows(0, M)
    c = oracle.smooth_factors(spec.x_calib(128), W)
    cd = torch.from_numpy(c).cuda()
    h = q.prepare_weights(dev_bf16(W), dev_bf16(b), cd, None, c8="only")
    Xq8, a_scale = q.rotate_smooth_quantize_c8(h, dev_bf16(X))
    assert h.device_status() == 0
    Y = torch.full((M, N), -3.0, dtype=torch.bfloat16, device="cuda")
    t0, t1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    t0.record()
    assert q.debug_starved_linear_c8(h, Xq8, a_scale, Y, 1_000_000) == 0        # the launch itself succeeds
    t1.record()
    torch.cuda.synchronize()                                                       # ... and completes
    assert t0.elapsed_time(t1) < 200.0, "the starved launch should give up after about a millisecond per work item"
    code = ctypes.c_int(0)
    st = q.lib().qvggt_device_status(h.handle, torch.cuda.current_stream().cuda_stream, ctypes.byref(code))
    assert st == ERR_DEVICE_TIMEOUT and code.value in (DEV_TIMEOUT_FULL, DEV_TIMEOUT_ACCUM)
    assert b"wait expired" in q.lib().qvggt_status_string(st)
    assert torch.all(Y == -3.0), "a starved launch must not write outputs"
    # the limits are validated on the host
    assert q.debug_starved_linear_c8(h, Xq8, a_scale, Y, 10) == -2
    assert q.debug_starved_linear_c8(h, Xq8, a_scale, Y, 3_000_000_000) == -2
    h.free()
    # a fresh handle, a normal launch: bit-exact against the oracle, status clean
    h2 = q.prepare_weights(dev_bf16(W), dev_bf16(b), cd, None, c8="only")
    acc = torch.zeros((M, N), dtype=torch.int32, device="cuda")
    Y2 = q.w4a4_linear_c8(h2, Xq8, a_scale, acc_debug=acc)
    ref = oracle.w4a4_linear(X, oracle.prepare_weights(W, c), b, 0)
    assert h2.device_status() == 0
    assert np.array_equal(acc.cpu().numpy(), ref["acc"])
    assert np.array_equal(host_bits(Y2), ref["y"])
    h2.free()
