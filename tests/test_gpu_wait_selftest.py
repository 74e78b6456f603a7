"""The give-up path of the bounded device waits, run on purpose and harmlessly.

Every barrier wait inside the kernels has a time limit; when it runs out the waiting role writes a code to the
workspace's status word and the kernel returns.  dirotq_wait_selftest makes one small kernel take that path (a warp
waits, with the library's own wait routine, on a barrier in its shared memory that nothing arrives on).  Nothing
faults, traps or spins without a limit, and the context stays usable: the same workspace serves a normal call next.
"""
import numpy as np
import pytest
import torch

from paper_2605_16732_b200 import binding as dq
from paper_2605_16732_b200 import synth

pytestmark = pytest.mark.gpu


def _bf(bits):
    return torch.from_numpy(np.ascontiguousarray(bits).view(np.int16)).cuda().view(torch.bfloat16)


def test_a_wait_that_runs_out_is_reported_and_the_workspace_serves_the_next_call():
    spec = synth.LayerSpec(K=512, N=384, r=32, G=64, model=synth.PIXART, seed=31, calib_tokens=512)
    M = 200
    inp = synth.make_layer_inputs(spec, M)
    layer = dq.dirotq_prepare_layer(torch.from_numpy(inp["W"]).cuda(), torch.from_numpy(inp["Q"]).cuda(), spec.r, spec.G,
                                    bias=_bf(inp["bias"]))
    x = _bf(inp["x"])
    ws = dq.alloc_workspace(layer, M)
    ref = torch.zeros((M, spec.N), dtype=torch.bfloat16, device="cuda")
    dq.dirotq_linear(x, layer, ref, ws)
    assert dq.dirotq_workspace_status(ws) == 0

    t0, t1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    t0.record()
    dq.dirotq_wait_selftest(ws, limit_us=2000)
    t1.record()
    code = dq.ctypes.c_int(0)
    st = dq.lib().dirotq_workspace_status(ws.data_ptr(), torch.cuda.current_stream().cuda_stream, dq.ctypes.byref(code))
    assert st == 6 and code.value == 5  # DIROTQ_ERR_DEVICE_TIMEOUT, written by the self-test's wait
    # it waited about as long as it was told to, not for the kernels' one-second limit
    assert 1.5 <= t0.elapsed_time(t1) <= 200.0

    ws[:256].zero_()
    out = torch.zeros_like(ref)
    dq.dirotq_linear(x, layer, out, ws)
    assert dq.dirotq_workspace_status(ws) == 0
    assert torch.equal(out.view(torch.int16), ref.view(torch.int16))
    layer.close()


def test_selftest_rejects_bad_arguments():
    ws = torch.zeros(256, dtype=torch.uint8, device="cuda")
    L = dq.lib()
    assert L.dirotq_wait_selftest(None, 1000, None) == 1
    assert L.dirotq_wait_selftest(ws.data_ptr(), 0, None) == 1
    assert L.dirotq_wait_selftest(ws.data_ptr(), 200000, None) == 1
