"""Parity of the CUDA library against the CPU oracle, element by element, through the C ABI."""
import numpy as np
import pytest
import torch

from oracle import dirotq_oracle as orc
from paper_2605_16732_b200 import binding as dq
from paper_2605_16732_b200 import synth

from parity_utils import (bf16_tensor_to_bits, bits_to_bf16_tensor, check_activation_side, check_layer_output,
                          check_weight_side)

pytestmark = pytest.mark.gpu


def _run_case(spec: synth.LayerSpec, M: int, with_bias=True, x_override=None, check_rot=True):
    inp = synth.make_layer_inputs(spec, M, with_bias=with_bias)
    if x_override is not None:
        inp["x"] = x_override(inp["x"])
    lo = orc.prepare_layer(inp["W"], inp["Q"], spec.r, spec.G, want_t=True)
    oo = orc.linear_deployed(inp["x"], lo, bias=inp["bias"])

    dev = "cuda"
    W = torch.from_numpy(inp["W"]).to(dev)
    Q = torch.from_numpy(inp["Q"]).to(dev)
    bias = bits_to_bf16_tensor(inp["bias"]) if with_bias else None
    layer = dq.dirotq_prepare_layer(W, Q, spec.r, spec.G, bias=bias)
    check_weight_side(dq.dirotq_layer_export(layer), lo)

    x = bits_to_bf16_tensor(inp["x"])
    ws = dq.alloc_workspace(layer, M)
    xrot = torch.zeros((M, spec.K), dtype=torch.float32, device=dev) if check_rot else None
    dq.dirotq_rotate_quantize(x, layer, ws, xrot)
    assert dq.dirotq_workspace_status(ws) == 0
    xh, codes, scales = dq.dirotq_workspace_export(layer, M, ws)
    xh_b, codes_n, scales_b = bf16_tensor_to_bits(xh), codes.cpu().numpy(), bf16_tensor_to_bits(scales)
    stats = check_activation_side(xrot.cpu().numpy() if check_rot else None, xh_b, codes_n, scales_b, oo, spec.r,
                                  spec.G)

    # integer GEMM on the oracle's codes: bit exact
    padded = np.zeros((M, layer.K_lp), dtype=np.int8)
    padded[:, :spec.K_l] = oo["codes"]
    P = dq.dirotq_int_gemm_debug(torch.from_numpy(padded).to(dev), layer, ws)
    assert dq.dirotq_workspace_status(ws) == 0
    assert np.array_equal(P.cpu().numpy(), oo["P"]), "int32 group sums differ"

    # whole layer
    y = torch.zeros((M, spec.N), dtype=torch.bfloat16, device=dev)
    dq.dirotq_linear(x, layer, y, ws)
    assert dq.dirotq_workspace_status(ws) == 0
    stats.update(check_layer_output(bf16_tensor_to_bits(y), xh_b, codes_n, scales_b, lo, oo, inp["bias"]))
    # a second call on the same workspace gives the same bits (the integer path is deterministic)
    y2 = torch.zeros_like(y)
    dq.dirotq_linear(x, layer, y2, ws)
    torch.cuda.synchronize()
    assert torch.equal(y.view(torch.int16), y2.view(torch.int16))
    layer.close()
    return stats


def test_small_single_tile():
    spec = synth.LayerSpec(K=256, N=256, r=32, G=64, model=synth.PIXART, seed=1, calib_tokens=512)
    print(_run_case(spec, M=100))


def test_config1_pixart_attention_projection():
    spec = synth.LayerSpec(K=1152, N=1152, r=32, G=64, model=synth.PIXART, seed=2)
    print(_run_case(spec, M=256))


def test_ragged_m_and_n_group128():
    spec = synth.LayerSpec(K=512, N=400, r=16, G=128, model=synth.FLUX, seed=3, calib_tokens=1024)
    print(_run_case(spec, M=300))


def test_rank64_no_ragged_group_half_kblock():
    spec = synth.LayerSpec(K=640, N=512, r=64, G=64, model=synth.FLUX, seed=4, calib_tokens=1024)
    print(_run_case(spec, M=129, with_bias=False))


def test_rank128_group128_two_lowrank_chunks():
    spec = synth.LayerSpec(K=768, N=272, r=128, G=128, model=synth.PIXART, seed=5, calib_tokens=1024)
    print(_run_case(spec, M=257))


def test_rank48():
    spec = synth.LayerSpec(K=384, N=256, r=48, G=64, model=synth.PIXART, seed=8, calib_tokens=1024)
    print(_run_case(spec, M=64))


def test_single_token():
    spec = synth.LayerSpec(K=256, N=256, r=32, G=64, model=synth.PIXART, seed=6, calib_tokens=512)
    print(_run_case(spec, M=1))


def test_many_tiles_per_cta():
    # more tiles than SMs in both kernels: exercises the persistent loops and the TMEM ping-pong parity
    spec = synth.LayerSpec(K=512, N=2304, r=32, G=64, model=synth.FLUX, seed=9, calib_tokens=1024)
    print(_run_case(spec, M=2500, check_rot=True))


def test_zero_tokens_give_zero_scales():
    spec = synth.LayerSpec(K=256, N=256, r=32, G=64, model=synth.PIXART, seed=7, calib_tokens=512)

    def zero_some(x):
        x = x.copy()
        x[3] = 0
        x[17] = 0
        return x

    print(_run_case(spec, M=40, x_override=zero_some))


def test_argument_errors_on_device():
    spec = synth.LayerSpec(K=256, N=256, r=32, G=64, model=synth.PIXART, seed=1, calib_tokens=512)
    inp = synth.make_layer_inputs(spec, 8)
    W = torch.from_numpy(inp["W"]).cuda()
    Q = torch.from_numpy(inp["Q"]).cuda()
    layer = dq.dirotq_prepare_layer(W, Q, spec.r, spec.G)
    ws = dq.alloc_workspace(layer, 8)
    x = bits_to_bf16_tensor(inp["x"])
    y = torch.empty((8, spec.N), dtype=torch.bfloat16, device="cuda")
    L = dq.lib()
    s = torch.cuda.current_stream().cuda_stream
    assert L.dirotq_linear(x.data_ptr(), 8, layer.handle, y.data_ptr(), ws.data_ptr(), 16, s) == 3  # too small
    assert L.dirotq_linear(x.data_ptr() + 2, 8, layer.handle, y.data_ptr(), ws.data_ptr(), ws.numel(), s) == 1
    assert L.dirotq_linear(x.data_ptr(), 0, layer.handle, y.data_ptr(), ws.data_ptr(), ws.numel(), s) == 1
    torch.cuda.synchronize()


def test_wait_counters_are_reported():
    spec = synth.LayerSpec(K=512, N=1024, r=32, G=64, model=synth.PIXART, seed=12, calib_tokens=512)
    inp = synth.make_layer_inputs(spec, 700)
    layer = dq.dirotq_prepare_layer(torch.from_numpy(inp["W"]).cuda(), torch.from_numpy(inp["Q"]).cuda(), spec.r, spec.G)
    ws = dq.alloc_workspace(layer, 700)
    x = bits_to_bf16_tensor(inp["x"])
    y = torch.empty((700, spec.N), dtype=torch.bfloat16, device="cuda")
    dq.dirotq_linear(x, layer, y, ws)
    c = dq.dirotq_workspace_wait_counters(ws)
    assert dq.dirotq_workspace_status(ws) == 0
    assert c["mma_role_total"] > 0 and c["epilogue_total"] > 0
    assert c["epilogue_wait_accumulator"] <= c["epilogue_total"]
    assert c["mma_wait_operands"] + c["mma_wait_accumulator"] <= c["mma_role_total"]
    layer.close()


@pytest.mark.parametrize("G", [64, 128])
def test_group_sums_exact_on_codes_built_to_lose_low_bits(G):
    """The group sums come out of a floating-point accumulator (products of small integers, scaled by a power
    of two): they must still equal the integer sums bit for bit when the sum is as large as it can get and
    single +-1 products are added to or cancelled against long runs of +-49."""
    K, N, r, M = 2 * 128 + 128, 256, 128, 128
    K_l = K - r
    rng = np.random.default_rng(5)
    # identity rotation: the folded weight is W itself; every |w| equal in a group -> every weight code is +-7
    Q = np.eye(K)
    sign = rng.choice([-1.0, 1.0], size=(K, N))
    sign[:, :64] = 1.0  # a block of columns with all codes +7
    W = (0.02 * sign).astype(np.float32)
    lo = orc.prepare_layer(W, Q, r, G, want_t=True)
    assert np.all(np.abs(lo["wcodes"]) == 7)
    layer = dq.dirotq_prepare_layer(torch.from_numpy(W).cuda(), torch.from_numpy(Q).cuda(), r, G)
    codes = np.zeros((M, K_l), dtype=np.int8)
    codes[0:16] = 7                                             # largest sum: G * 49
    codes[16:32] = -7
    for m in range(32, 64):                                     # a long run of 7s, then 1s
        codes[m] = 7
        codes[m, K_l - 1 - (m - 32):] = 1
    for m in range(64, 96):                                     # cancellation down to a small remainder
        codes[m, 0::2] = 7
        codes[m, 1::2] = -7
        codes[m, 2 * (m - 64)] = 6
    codes[96:] = rng.integers(-7, 8, size=(M - 96, K_l))
    ws = dq.alloc_workspace(layer, M)
    padded = np.zeros((M, layer.K_lp), dtype=np.int8)
    padded[:, :K_l] = codes
    P = dq.dirotq_int_gemm_debug(torch.from_numpy(padded).cuda(), layer, ws)
    assert dq.dirotq_workspace_status(ws) == 0
    ref = orc.int_gemm(codes, lo["wcodes"], G)
    assert int(np.abs(ref).max()) == G * 49
    assert np.array_equal(P.cpu().numpy(), ref)
    layer.close()


@pytest.mark.parametrize("M", [300, 2500, 4608])
def test_host_entry_point_equals_device_entry_point(M):
    """dirotq_linear_host (pinned host buffers; row chunks pipelined over copy streams for large M) gives the same
    bits as dirotq_linear on device buffers, twice in a row (re-use of the staging buffers and events)."""
    spec = synth.LayerSpec(K=512, N=384, r=32, G=64, model=synth.PIXART, seed=9, calib_tokens=1024)
    inp = synth.make_layer_inputs(spec, M)
    layer = dq.dirotq_prepare_layer(torch.from_numpy(inp["W"]).cuda(), torch.from_numpy(inp["Q"]).cuda(), spec.r, spec.G,
                                    bias=bits_to_bf16_tensor(inp["bias"]))
    x = bits_to_bf16_tensor(inp["x"])
    ws = dq.alloc_workspace(layer, M)
    y = torch.zeros((M, spec.N), dtype=torch.bfloat16, device="cuda")
    dq.dirotq_linear(x, layer, y, ws)
    torch.cuda.synchronize()
    xh = x.cpu().pin_memory()
    yh = torch.zeros((M, spec.N), dtype=torch.bfloat16).pin_memory()
    x_dev, y_dev = torch.empty_like(x), torch.empty_like(y)
    for _ in range(2):
        yh.zero_()
        dq.dirotq_linear_host(xh, layer, yh, x_dev, y_dev, ws)
        torch.cuda.current_stream().synchronize()
        assert torch.equal(yh.view(torch.int16), y.cpu().view(torch.int16))
    assert dq.dirotq_workspace_status(ws) == 0
    layer.close()


def test_shared_rotation_across_linears_with_the_same_input():
    """Linears that read the same activations and were calibrated on them have the same rotation (Sec. 4.2: the basis
    depends only on the input's statistics), so one rotate/quantize pass serves them all: dirotq_rotate_quantize once,
    then dirotq_w4a4_gemm per layer on the same workspace.  Must equal each layer's own dirotq_linear bit for bit."""
    spec = synth.LayerSpec(K=1152, N=1152, r=32, G=64, model=synth.PIXART, seed=11)
    M = 520
    inp = synth.make_layer_inputs(spec, M)
    Q = torch.from_numpy(inp["Q"]).cuda()
    x = bits_to_bf16_tensor(inp["x"])
    rng = np.random.default_rng(3)
    layers, own = [], []
    for i in range(3):  # q, k, v projections: same input, different weights
        W = (0.02 * rng.standard_normal((spec.K, spec.N))).astype(np.float32)
        layer = dq.dirotq_prepare_layer(torch.from_numpy(W).cuda(), Q, spec.r, spec.G)
        ws = dq.alloc_workspace(layer, M)
        y = torch.zeros((M, spec.N), dtype=torch.bfloat16, device="cuda")
        dq.dirotq_linear(x, layer, y, ws)
        layers.append(layer)
        own.append(y)
    ws = dq.alloc_workspace(layers[0], M)
    dq.dirotq_rotate_quantize(x, layers[0], ws)
    for layer, y_own in zip(layers, own):
        y = torch.zeros_like(y_own)
        dq.dirotq_w4a4_gemm(M, layer, ws, y)
        torch.cuda.synchronize()
        assert torch.equal(y.view(torch.int16), y_own.view(torch.int16))
    assert dq.dirotq_workspace_status(ws) == 0
    for layer in layers:
        layer.close()


def test_host_entry_point_on_concurrent_streams():
    """Two independent layers through dirotq_linear_host on two streams at once (the library's copy streams and events
    are shared by all calls on a device): both results equal the device entry point's."""
    M = 3000
    cases = []
    for seed, (K, N) in enumerate([(512, 384), (384, 640)]):
        spec = synth.LayerSpec(K=K, N=N, r=32, G=64, model=synth.PIXART, seed=20 + seed, calib_tokens=1024)
        inp = synth.make_layer_inputs(spec, M)
        layer = dq.dirotq_prepare_layer(torch.from_numpy(inp["W"]).cuda(), torch.from_numpy(inp["Q"]).cuda(), spec.r, spec.G,
                                        bias=bits_to_bf16_tensor(inp["bias"]))
        x = bits_to_bf16_tensor(inp["x"])
        ws = dq.alloc_workspace(layer, M)
        y = torch.zeros((M, N), dtype=torch.bfloat16, device="cuda")
        dq.dirotq_linear(x, layer, y, ws)
        cases.append({"layer": layer, "ws": ws, "y": y, "xh": x.cpu().pin_memory(),
                      "yh": torch.zeros((M, N), dtype=torch.bfloat16).pin_memory(), "x_dev": torch.empty_like(x),
                      "y_dev": torch.empty_like(y), "stream": torch.cuda.Stream()})
    torch.cuda.synchronize()
    for _ in range(3):
        for c in cases:
            c["yh"].zero_()
        for c in cases:
            dq.dirotq_linear_host(c["xh"], c["layer"], c["yh"], c["x_dev"], c["y_dev"], c["ws"], stream=c["stream"])
        for c in cases:
            c["stream"].synchronize()
            assert torch.equal(c["yh"].view(torch.int16), c["y"].cpu().view(torch.int16))
    for c in cases:
        assert dq.dirotq_workspace_status(c["ws"]) == 0
        c["layer"].close()


def test_layer_chain_replayed_from_a_cuda_graph_gives_the_same_bits():
    # the entry points only enqueue work on the caller's stream (no allocation, no synchronisation), so a chain of
    # layers can be captured once and replayed; small layers are launch-bound without this
    specs = [synth.LayerSpec(K=256, N=512, r=32, G=64, model=synth.PIXART, seed=41, calib_tokens=512),
             synth.LayerSpec(K=512, N=384, r=16, G=128, model=synth.PIXART, seed=42, calib_tokens=512),
             synth.LayerSpec(K=384, N=256, r=32, G=64, model=synth.PIXART, seed=43, calib_tokens=512)]
    M, dev = 200, "cuda"
    layers, bufs = [], []
    for spec in specs:
        inp = synth.make_layer_inputs(spec, M, with_bias=True)
        layers.append(dq.dirotq_prepare_layer(torch.from_numpy(inp["W"]).to(dev), torch.from_numpy(inp["Q"]).to(dev),
                                              spec.r, spec.G, bias=bits_to_bf16_tensor(inp["bias"])))
        bufs.append(torch.zeros((M, spec.N), dtype=torch.bfloat16, device=dev))
    x0 = bits_to_bf16_tensor(synth.make_layer_inputs(specs[0], M)["x"])
    wss = [dq.alloc_workspace(l, M) for l in layers]

    def chain():
        cur = x0
        for l, y, ws in zip(layers, bufs, wss):
            dq.dirotq_linear(cur, l, y, ws)
            cur = y

    chain()
    torch.cuda.synchronize()
    eager = [b.view(torch.int16).clone() for b in bufs]
    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    with torch.cuda.stream(side):
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph, stream=side):
            chain()
    torch.cuda.current_stream().wait_stream(side)
    for b in bufs:
        b.zero_()
    for _ in range(3):
        graph.replay()
    torch.cuda.synchronize()
    for ws in wss:
        assert dq.dirotq_workspace_status(ws) == 0
    for b, e in zip(bufs, eager):
        assert torch.equal(b.view(torch.int16), e)
    for l in layers:
        l.close()


def test_dependent_launch_on_and_off_give_the_same_bits():
    # the second kernel of a layer (and the first kernel of the next) is scheduled early and orders itself with
    # griddepcontrol.wait; a chain on ONE workspace is the case where an early writer would be caught
    specs = [synth.LayerSpec(K=512, N=512, r=32, G=64, model=synth.PIXART, seed=61, calib_tokens=512),
             synth.LayerSpec(K=512, N=512, r=16, G=128, model=synth.PIXART, seed=62, calib_tokens=512)]
    M, dev = 700, "cuda"
    layers = []
    for spec in specs:
        inp = synth.make_layer_inputs(spec, M, with_bias=True)
        layers.append(dq.dirotq_prepare_layer(torch.from_numpy(inp["W"]).to(dev), torch.from_numpy(inp["Q"]).to(dev),
                                              spec.r, spec.G, bias=bits_to_bf16_tensor(inp["bias"])))
    x0 = bits_to_bf16_tensor(synth.make_layer_inputs(specs[0], M)["x"])
    ws = dq.alloc_workspace(layers[0], M)
    assert ws.numel() >= dq.alloc_workspace(layers[1], M).numel()
    bufs = [torch.zeros((M, 512), dtype=torch.bfloat16, device=dev) for _ in range(2)]
    outs = {}
    try:
        for on in (False, True):
            dq.dirotq_set_dependent_launch(on)
            for b in bufs:
                b.zero_()
            for _ in range(4):      # ping-pong through both layers, same workspace throughout
                dq.dirotq_linear(x0, layers[0], bufs[0], ws)
                dq.dirotq_linear(bufs[0], layers[1], bufs[1], ws)
            torch.cuda.synchronize()
            assert dq.dirotq_workspace_status(ws) == 0
            outs[on] = [b.view(torch.int16).clone() for b in bufs]
        assert all(torch.equal(a, b) for a, b in zip(outs[False], outs[True]))
    finally:
        dq.dirotq_set_dependent_launch(True)
    for l in layers:
        l.close()


def test_sibling_layers_without_their_own_rotation():
    # q / k / v-style group: one layer owns the rotation, the others are prepared without a copy of it and consume
    # the owner's rotated workspace; they must give the bits of fully prepared layers
    spec = synth.LayerSpec(K=512, N=384, r=32, G=64, model=synth.PIXART, seed=95, calib_tokens=1024)
    M, dev = 333, "cuda"
    base = synth.make_layer_inputs(spec, M, with_bias=True)
    Q = torch.from_numpy(base["Q"]).to(dev)
    x = bits_to_bf16_tensor(base["x"])
    rng = np.random.default_rng(5)
    Ws = [torch.from_numpy((rng.standard_normal((spec.K, spec.N)) * 0.02).astype(np.float32)).to(dev) for _ in range(3)]
    bias = bits_to_bf16_tensor(base["bias"])
    for asym in (False, True):
        prep = dq.dirotq_prepare_layer_asym if asym else dq.dirotq_prepare_layer
        full = [prep(W, Q, spec.r, spec.G, bias=bias) for W in Ws]
        sibs = [dq.dirotq_prepare_layer_sibling(W, Q, spec.r, spec.G, bias=bias, asym=asym) for W in Ws[1:]]
        assert all(s.blob.numel() <= f.blob.numel() - 2 * spec.K * spec.K for s, f in zip(sibs, full[1:]))
        ws = dq.alloc_workspace(full[0], M)
        dq.dirotq_rotate_quantize(x, full[0], ws)
        for i, sib in enumerate(sibs, start=1):
            y_ref = torch.zeros((M, spec.N), dtype=torch.bfloat16, device=dev)
            dq.dirotq_linear(x, full[i], y_ref, dq.alloc_workspace(full[i], M))
            y = torch.zeros_like(y_ref)
            dq.dirotq_w4a4_gemm(M, sib, ws, y)
            torch.cuda.synchronize()
            assert dq.dirotq_workspace_status(ws) == 0
            assert torch.equal(y.view(torch.int16), y_ref.view(torch.int16))
            # what a sibling cannot do is refused before any launch
            with pytest.raises(dq.DirotqError):
                dq.dirotq_linear(x, sib, y, ws)
            with pytest.raises(dq.DirotqError):
                dq.dirotq_rotate_quantize(x, sib, ws)
            with pytest.raises(dq.DirotqError):
                dq.dirotq_layer_export(sib)
        for l in full + sibs:
            l.close()
