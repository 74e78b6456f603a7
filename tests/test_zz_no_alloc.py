"""The allocation-free entry point against the ordinary one.

dirotq_linear_noalloc exists for callers that cannot allocate device memory where they run (a
plug-in inside a runtime that owns the memory, code on a captured stream, a fixed-memory loop):
its workspace is an array inside the library.  It must give exactly what dirotq_linear gives --
the same two kernels run -- on consecutive calls that reuse the shared array, including a call
with a different shape in between, and it must refuse a problem that does not fit.

This file sorts last on purpose: a run that stops at the first failure has then run everything else.
"""
import numpy as np
import pytest
import torch

from paper_2605_16732_b200 import binding as dq
from paper_2605_16732_b200 import synth

pytestmark = pytest.mark.gpu


def _bf(bits):
    return torch.from_numpy(np.ascontiguousarray(bits).view(np.int16)).cuda().view(torch.bfloat16)


def _layer(K, N, r, G, seed):
    spec = synth.LayerSpec(K=K, N=N, r=r, G=G, model=synth.PIXART, seed=seed, calib_tokens=512)
    W, bias = synth.make_weights(spec)
    # any orthogonal matrix will do here: a seeded Householder reflection
    g = np.random.default_rng(seed)
    v = g.standard_normal(K)
    v /= np.linalg.norm(v)
    Q = np.eye(K) - 2.0 * np.outer(v, v)
    layer = dq.dirotq_prepare_layer(torch.from_numpy(W).cuda(), torch.from_numpy(Q).cuda(), r, G, bias=_bf(bias))
    return spec, layer


def test_noalloc_matches_linear_on_consecutive_calls():
    spec, layer = _layer(512, 768, 32, 64, seed=21)
    spec2, layer2 = _layer(256, 272, 16, 128, seed=22)
    status = torch.full((1,), -1, dtype=torch.int32, device="cuda")
    for call, (sp, ly, M) in enumerate([(spec, layer, 300), (spec, layer, 300), (spec2, layer2, 77), (spec, layer, 129)]):
        x = _bf(synth.make_tokens(sp, M, batch_seed=100 + call))
        ref = torch.zeros((M, sp.N), dtype=torch.bfloat16, device="cuda")
        ws = dq.alloc_workspace(ly, M)
        dq.dirotq_linear(x, ly, ref, ws)
        assert dq.dirotq_workspace_status(ws) == 0
        out = torch.zeros_like(ref)
        before = torch.cuda.memory_allocated()
        dq.dirotq_linear_noalloc(x, ly, out, status)
        assert torch.cuda.memory_allocated() == before  # nothing went through torch's allocator either
        torch.cuda.synchronize()
        assert int(status.item()) == 0
        # same kernels, same inputs: identical bits (tighter than the 1e-2 rms bound of the parity tests)
        assert torch.equal(out.view(torch.int16), ref.view(torch.int16)), f"call {call} differs"
    layer.close()
    layer2.close()


def test_noalloc_rejects_what_does_not_fit():
    spec, layer = _layer(512, 768, 32, 64, seed=23)
    M = 40000  # 40000 x 512 bytes of codes alone exceed the 16 MiB array
    x = torch.zeros((M, spec.K), dtype=torch.bfloat16, device="cuda")
    y = torch.zeros((M, spec.N), dtype=torch.bfloat16, device="cuda")
    st = dq.lib().dirotq_linear_noalloc(x.data_ptr(), M, layer.handle, y.data_ptr(), None,
                                        torch.cuda.current_stream().cuda_stream)
    assert st == 3  # DIROTQ_ERR_BUFFER_TOO_SMALL
    assert dq.lib().dirotq_linear_noalloc(None, 8, layer.handle, y.data_ptr(), None, None) == 1
    torch.cuda.synchronize()
    layer.close()


def test_noalloc_matches_linear_for_every_layer_format():
    K, N, r, G, M = 512, 400, 32, 64, 260
    spec = synth.LayerSpec(K=K, N=N, r=r, G=G, model=synth.FLUX, seed=24, calib_tokens=1024)
    W, bias = synth.make_weights(spec)
    g = np.random.default_rng(24)
    v = g.standard_normal(K)
    v /= np.linalg.norm(v)
    Q = torch.from_numpy(np.eye(K) - 2.0 * np.outer(v, v)).cuda()
    Wd, Uh, b = torch.from_numpy(W).cuda(), Q[:, :r].contiguous(), _bf(bias)
    x = _bf(synth.make_tokens(spec, M, batch_seed=5))
    layers = {
        "int4_asym": dq.dirotq_prepare_layer_asym(Wd, Q, r, G, bias=b),
        "w4a8": dq.dirotq_prepare_layer_w4a8(Wd, Q, r, bias=b),
        "nvfp4": dq.dirotq_prepare_layer_nvfp4(Wd, Q, r, -8, bias=b),
        "int4_ph": dq.dirotq_prepare_layer_ph(Wd, Uh, G, bias=b),
        "nvfp4_ph": dq.dirotq_prepare_layer_nvfp4_ph(Wd, Uh, -8, bias=b),
    }
    status = torch.full((1,), -1, dtype=torch.int32, device="cuda")
    for name, ly in layers.items():
        ref = torch.zeros((M, N), dtype=torch.bfloat16, device="cuda")
        ws = dq.alloc_workspace(ly, M)
        dq.dirotq_linear(x, ly, ref, ws)
        assert dq.dirotq_workspace_status(ws) == 0
        out = torch.zeros_like(ref)
        dq.dirotq_linear_noalloc(x, ly, out, status)
        torch.cuda.synchronize()
        assert int(status.item()) == 0, name
        assert torch.equal(out.view(torch.int16), ref.view(torch.int16)), name
        assert float(ref.float().abs().max()) > 0
        ly.close()


@pytest.mark.parametrize("fmt", ["int4_ph", "nvfp4_ph"])
def test_noalloc_with_the_split_first_step_of_the_projection_form(fmt):
    """K = 2048 with few token rows: the projection form's first step splits its reduction and parks the ranges' partial
    sums in the code region of the workspace, which the second pass then overwrites -- here that region is the shared
    array, still holding what another layer's call left there."""
    K, N, r, G, M = 2048, 256, 32, 64, 512
    spec = synth.LayerSpec(K=K, N=N, r=r, G=G, model=synth.FLUX, seed=41, calib_tokens=512)
    W, bias = synth.make_weights(spec)
    g = np.random.default_rng(41)
    Uh = torch.from_numpy(np.linalg.qr(g.standard_normal((K, r)))[0]).cuda().contiguous()
    Wd, b = torch.from_numpy(W).cuda(), _bf(bias)
    layer = (dq.dirotq_prepare_layer_ph(Wd, Uh, G, bias=b) if fmt == "int4_ph"
             else dq.dirotq_prepare_layer_nvfp4_ph(Wd, Uh, -6, bias=b))
    _, other = _layer(512, 768, 32, 64, seed=42)
    spec_o = synth.LayerSpec(K=512, N=768, r=32, G=64, model=synth.PIXART, seed=42, calib_tokens=512)
    x = _bf(synth.make_tokens(spec, M, batch_seed=6))
    xo = _bf(synth.make_tokens(spec_o, 300, batch_seed=7))
    ref = torch.zeros((M, N), dtype=torch.bfloat16, device="cuda")
    ws = dq.alloc_workspace(layer, M)
    assert ws.numel() <= 16 << 20
    dq.dirotq_linear(x, layer, ref, ws)
    assert dq.dirotq_workspace_status(ws) == 0
    status = torch.full((1,), -1, dtype=torch.int32, device="cuda")
    yo = torch.zeros((300, 768), dtype=torch.bfloat16, device="cuda")
    for call in range(2):
        dq.dirotq_linear_noalloc(xo, other, yo, status)  # leaves its own codes and scales in the shared array
        out = torch.zeros_like(ref)
        dq.dirotq_linear_noalloc(x, layer, out, status)
        torch.cuda.synchronize()
        assert int(status.item()) == 0
        assert torch.equal(out.view(torch.int16), ref.view(torch.int16)), f"{fmt} call {call}"
    layer.close()
    other.close()
