"""Parity of the projection form (U_h only + block-Hadamard residual, a cheaper first stage that is NOT the paper's
Eq. 5) against its CPU reference, stage by stage: prepared weights, x~_h, codes and scales of the rotated residual,
integer group sums, output."""
import numpy as np
import pytest
import torch

from oracle import dirotq_oracle as orc
from paper_2605_16732_b200 import binding as dq
from paper_2605_16732_b200 import synth

from parity_utils import bf16_tensor_to_bits, bits_to_bf16_tensor, check_activation_side, check_layer_output

pytestmark = pytest.mark.gpu


def _run_case(spec: synth.LayerSpec, M: int, with_bias=True):
    inp = synth.make_layer_inputs(spec, M, with_bias=with_bias)
    Uh = np.ascontiguousarray(np.asarray(inp["Q"], dtype=np.float64)[:, :spec.r])
    lo = orc.prepare_layer_ph(inp["W"], Uh, spec.G)
    oo = orc.linear_deployed_ph(inp["x"], lo, bias=inp["bias"])

    dev = "cuda"
    W = torch.from_numpy(inp["W"]).to(dev)
    bias = bits_to_bf16_tensor(inp["bias"]) if with_bias else None
    layer = dq.dirotq_prepare_layer_ph(W, torch.from_numpy(Uh).to(dev), spec.G, bias=bias)
    assert (layer.K_l, layer.n_g) == (spec.K, spec.K // spec.G)

    # weight side: the rounded projection, V = bf16(U_hb^T H+-), the 16-bit rows (V H+-^T / G) W, scales and codes of
    # H^T W (exact ties may differ)
    assert np.array_equal(bf16_tensor_to_bits(dq.dirotq_layer_export_uh(layer)), lo["Uhb"])
    assert np.array_equal(bf16_tensor_to_bits(dq.dirotq_layer_export_v(layer)), lo["V"])
    wcodes = torch.empty((spec.K, spec.N), dtype=torch.int8, device=dev)
    wscales = torch.empty((layer.n_g, spec.N), dtype=torch.bfloat16, device=dev)
    wh = torch.empty((spec.r, spec.N), dtype=torch.bfloat16, device=dev)
    dq._check(dq.lib().dirotq_layer_export(layer.handle, wcodes.data_ptr(), wscales.data_ptr(), wh.data_ptr(), None, None),
              "dirotq_layer_export")
    torch.cuda.synchronize()
    assert np.array_equal(bf16_tensor_to_bits(wh), lo["Wh"])
    assert np.array_equal(bf16_tensor_to_bits(wscales), lo["wscales"])
    bad = wcodes.cpu().numpy() != lo["wcodes"]
    if bad.any():
        t = lo["wt"][bad]
        assert bad.sum() <= 4 and np.all(np.abs(np.abs(t - np.floor(t)) - 0.5) < 1e-9)
    lo_gpu = dict(lo)
    lo_gpu["wcodes"] = wcodes.cpu().numpy()

    x = bits_to_bf16_tensor(inp["x"])
    ws = dq.alloc_workspace(layer, M)
    dq.dirotq_rotate_quantize(x, layer, ws)
    assert dq.dirotq_workspace_status(ws) == 0
    xh, codes, scales = dq.dirotq_workspace_export(layer, M, ws)
    xh_b, codes_n, scales_b = bf16_tensor_to_bits(xh), codes.cpu().numpy(), bf16_tensor_to_bits(scales)
    assert codes_n.shape == (M, spec.K)
    # x~_h: within one bf16 step of the reference where the fp32 sum lands on a rounding boundary
    xh_g, xh_o = orc.bf16_to_f64(xh_b), orc.bf16_to_f64(oo["xh"])
    xnorm = np.linalg.norm(orc.bf16_to_f64(inp["x"]), axis=1, keepdims=True)
    assert np.all(np.abs(xh_g - xh_o) <= np.maximum(np.abs(xh_o), 2.0 ** -126) * 2.0 ** -7 + 1e-5 * xnorm)
    # The residual is DEFINED through the rounded x~_h, so a token whose x~_h differs in one element has a different
    # (equally valid) residual: codes and scales are held to the reference's second step run on the library's own x~_h,
    # with the same protocol as for the rotation (equal except at rounding boundaries).
    _, xl_ref = orc.residual_ph(inp["x"], lo, spec.G, xh_bits=xh_b)
    sq_ref = orc.split_quantize(xl_ref, 0, spec.G, want_t=True)
    same_xh = np.all(xh_b == oo["xh"], axis=1)
    assert np.array_equal(sq_ref["codes"][same_xh], oo["codes"][same_xh])      # consistency of the re-run
    prot = {"xt": np.concatenate([xh_g, xl_ref], axis=1), "xh": xh_b, "scales": sq_ref["scales"], "codes": sq_ref["codes"]}
    stats = check_activation_side(None, xh_b, codes_n, scales_b, prot, spec.r, spec.G)
    stats["xh_exact_frac"] = float(np.mean(xh_b == oo["xh"]))

    padded = np.ascontiguousarray(oo["codes"])
    P = dq.dirotq_int_gemm_debug(torch.from_numpy(padded).to(dev), layer, ws)
    assert dq.dirotq_workspace_status(ws) == 0
    assert np.array_equal(P.cpu().numpy(), orc.int_gemm(oo["codes"], lo_gpu["wcodes"], spec.G)), "int32 group sums differ"

    y = torch.zeros((M, spec.N), dtype=torch.bfloat16, device=dev)
    dq.dirotq_linear(x, layer, y, ws)
    assert dq.dirotq_workspace_status(ws) == 0
    stats.update(check_layer_output(bf16_tensor_to_bits(y), xh_b, codes_n, scales_b, lo_gpu, oo, inp["bias"]))
    y2 = torch.zeros_like(y)
    dq.dirotq_linear(x, layer, y2, ws)
    torch.cuda.synchronize()
    assert torch.equal(y.view(torch.int16), y2.view(torch.int16))
    with pytest.raises(dq.DirotqError):
        dq.dirotq_layer_export(layer)          # asks for the K x K rotation, which this form does not have
    layer.close()
    return stats


def test_projection_form_small():
    spec = synth.LayerSpec(K=256, N=256, r=32, G=64, model=synth.PIXART, seed=101, calib_tokens=512)
    print(_run_case(spec, M=100))


def test_projection_form_pixart_projection():
    spec = synth.LayerSpec(K=1152, N=1152, r=32, G=64, model=synth.PIXART, seed=102)
    print(_run_case(spec, M=256))


def test_projection_form_ragged_rows_columns_group128():
    spec = synth.LayerSpec(K=512, N=400, r=16, G=128, model=synth.FLUX, seed=103, calib_tokens=1024)
    print(_run_case(spec, M=300))


def test_projection_form_rank_112_no_bias():
    spec = synth.LayerSpec(K=1152, N=384, r=112, G=64, model=synth.PIXART, seed=104)
    print(_run_case(spec, M=257, with_bias=False))


def test_projection_form_through_the_other_entry_points():
    # host entry (pipelined copies, M >= 2048 so that it cuts the rows into chunks), the built-in workspace, the two
    # kernels called separately, a CUDA graph and every tile knob: all give the bits of dirotq_linear
    spec = synth.LayerSpec(K=512, N=384, r=32, G=64, model=synth.PIXART, seed=105, calib_tokens=1024)
    M, dev = 2300, "cuda"
    inp = synth.make_layer_inputs(spec, M, with_bias=True)
    Uh = np.ascontiguousarray(np.asarray(inp["Q"], dtype=np.float64)[:, :spec.r])
    layer = dq.dirotq_prepare_layer_ph(torch.from_numpy(inp["W"]).to(dev), torch.from_numpy(Uh).to(dev), spec.G,
                                       bias=bits_to_bf16_tensor(inp["bias"]))
    x = bits_to_bf16_tensor(inp["x"])
    ws = dq.alloc_workspace(layer, M)
    y = torch.zeros((M, spec.N), dtype=torch.bfloat16, device=dev)
    dq.dirotq_linear(x, layer, y, ws)
    torch.cuda.synchronize()
    ref = y.view(torch.int16).clone()

    x_host = x.cpu().pin_memory()
    y_host = torch.zeros((M, spec.N), dtype=torch.bfloat16).pin_memory()
    xd, yd = torch.empty_like(x), torch.empty_like(y)
    dq.dirotq_linear_host(x_host, layer, y_host, xd, yd, ws)
    torch.cuda.synchronize()
    assert torch.equal(y_host.view(torch.int16), ref.cpu())

    m_small = 200                                    # the built-in workspace is small
    y_small = torch.zeros((m_small, spec.N), dtype=torch.bfloat16, device=dev)
    dq.dirotq_linear_noalloc(x[:m_small].contiguous(), layer, y_small)
    torch.cuda.synchronize()
    assert torch.equal(y_small.view(torch.int16), ref[:m_small])

    y.zero_()
    dq.dirotq_rotate_quantize(x, layer, ws)
    dq.dirotq_w4a4_gemm(M, layer, ws, y)
    torch.cuda.synchronize()
    assert torch.equal(y.view(torch.int16), ref)

    try:
        for tile, plan, pdl in [(128, 1, False), (256, 3, True), (0, 2, True)]:
            dq.dirotq_set_gemm_tile(tile)
            dq.dirotq_set_rotation_tile(plan)       # the projection form has its own fixed plans: must be unaffected
            dq.dirotq_set_dependent_launch(pdl)
            y.zero_()
            dq.dirotq_linear(x, layer, y, ws)
            torch.cuda.synchronize()
            assert torch.equal(y.view(torch.int16), ref)
    finally:
        dq.dirotq_set_gemm_tile(0)
        dq.dirotq_set_rotation_tile(0)
        dq.dirotq_set_dependent_launch(True)

    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    with torch.cuda.stream(side):
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph, stream=side):
            dq.dirotq_linear(x, layer, y, ws)
    torch.cuda.current_stream().wait_stream(side)
    y.zero_()
    graph.replay()
    torch.cuda.synchronize()
    assert torch.equal(y.view(torch.int16), ref) and dq.dirotq_workspace_status(ws) == 0
    with pytest.raises(dq.DirotqError):
        dq.dirotq_rotate_quantize(x, layer, ws, torch.empty((M, spec.K), dtype=torch.float32, device=dev))
    layer.close()


# ------------------------------------------------------------------ NVFP4 operands behind the projection form

from parity_utils import check_activation_side_nvfp4, check_layer_output_nvfp4, check_weight_side_nvfp4


def _run_case_nvfp4(spec: synth.LayerSpec, M: int, with_bias=True):
    inp = synth.make_layer_inputs(spec, M, with_bias=with_bias)
    Uh = np.ascontiguousarray(np.asarray(inp["Q"], dtype=np.float64)[:, :spec.r])
    lo = orc.nvfp4_prepare_layer_ph(inp["W"], Uh, want_t=True)
    _, xl = orc.nvfp4_residual(inp["x"], lo)
    ex = orc.nvfp4_global_exponent(float(np.abs(xl).max()))          # calibration of the power-of-two scale: this batch
    oo = orc.nvfp4_linear_deployed_ph(inp["x"], lo, ex, bias=inp["bias"])

    dev = "cuda"
    bias = bits_to_bf16_tensor(inp["bias"]) if with_bias else None
    layer = dq.dirotq_prepare_layer_nvfp4_ph(torch.from_numpy(inp["W"]).to(dev), torch.from_numpy(Uh).to(dev), ex, bias=bias)
    lo_chk = dict(lo)
    lo_chk["Qb"] = lo["Uhb"]                 # the export returns U_hb in the rotation's place
    stats = check_weight_side_nvfp4(dq.dirotq_layer_export_nvfp4(layer), lo_chk)
    assert np.array_equal(bf16_tensor_to_bits(dq.dirotq_layer_export_v(layer)), lo["V"])

    x = bits_to_bf16_tensor(inp["x"])
    ws = dq.alloc_workspace(layer, M)
    y = torch.zeros((M, spec.N), dtype=torch.bfloat16, device=dev)
    dq.dirotq_linear(x, layer, y, ws)
    assert dq.dirotq_workspace_status(ws) == 0
    xh, codes, sf = dq.dirotq_workspace_export_nvfp4(layer, M, ws)
    xh_b, codes_n, sf_n = bf16_tensor_to_bits(xh), codes.cpu().numpy(), sf.cpu().numpy()
    assert codes_n.shape == (M, spec.K)
    # codes and block scales against the reference's second step on the library's own x~_h (the residual is defined
    # through the rounded x~_h), with the NVFP4 protocol
    _, xl_ref = orc.nvfp4_residual(inp["x"], lo, xh_bits=xh_b)
    xt_ref = np.ascontiguousarray(np.concatenate([orc.bf16_to_f64(xh_b), xl_ref], axis=1))
    sq_ref = orc.nvfp4_split_quantize(xt_ref, spec.r, ex, want_t=True)
    prot = {"xt": xt_ref, "xh": sq_ref["xh"], "codes": sq_ref["codes"], "sf": sq_ref["sf"], "t": sq_ref["t"]}
    stats.update(check_activation_side_nvfp4(None, xh_b, codes_n, sf_n, prot, spec.r, ex))
    xh_g, xh_o = orc.bf16_to_f64(xh_b), orc.bf16_to_f64(oo["xh"])
    xnorm = np.linalg.norm(orc.bf16_to_f64(inp["x"]), axis=1, keepdims=True)
    assert np.all(np.abs(xh_g - xh_o) <= np.maximum(np.abs(xh_o), 2.0 ** -126) * 2.0 ** -7 + 1e-5 * xnorm)
    stats.update(check_layer_output_nvfp4(bf16_tensor_to_bits(y), xh_b, codes_n, sf_n, ex, lo, oo, inp["bias"]))
    y2 = torch.zeros_like(y)
    dq.dirotq_linear(x, layer, y2, ws)
    torch.cuda.synchronize()
    assert torch.equal(y.view(torch.int16), y2.view(torch.int16))
    layer.close()
    return stats


def test_nvfp4_projection_form_small():
    spec = synth.LayerSpec(K=256, N=256, r=32, G=64, model=synth.PIXART, seed=111, calib_tokens=512)
    print(_run_case_nvfp4(spec, M=100))


def test_nvfp4_projection_form_pixart_projection():
    spec = synth.LayerSpec(K=1152, N=1152, r=32, G=64, model=synth.PIXART, seed=112)
    print(_run_case_nvfp4(spec, M=256))


def test_nvfp4_projection_form_ragged_rank64_no_bias():
    spec = synth.LayerSpec(K=768, N=400, r=64, G=64, model=synth.FLUX, seed=113, calib_tokens=1024)
    print(_run_case_nvfp4(spec, M=300, with_bias=False))


@pytest.mark.parametrize("split", [False, True])
def test_first_step_split_on_and_off(split):
    # M = 300: 3 row tiles, so the reduction is split when the knob is on; both settings must satisfy the same checks
    dq.dirotq_set_first_step_split(split)
    try:
        spec = synth.LayerSpec(K=2048, N=512, r=32, G=64, model=synth.FLUX, seed=114, calib_tokens=4096)
        print(_run_case(spec, M=300))
        print(_run_case_nvfp4(spec, M=300))
    finally:
        dq.dirotq_set_first_step_split(True)
