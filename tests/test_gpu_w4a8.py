"""Parity of the W4A8 variant (per-token INT8 activations, per-channel INT4 weights) against the CPU oracle."""
import numpy as np
import pytest
import torch

from oracle import dirotq_oracle as orc
from paper_2605_16732_b200 import binding as dq
from paper_2605_16732_b200 import synth

from parity_utils import (bf16_tensor_to_bits, bits_to_bf16_tensor, check_activation_side_w4a8, check_layer_output_w4a8,
                          check_weight_side)

pytestmark = pytest.mark.gpu


def _run_case(spec: synth.LayerSpec, M: int, with_bias=True, check_rot=True):
    inp = synth.make_layer_inputs(spec, M, with_bias=with_bias)
    lo = orc.prepare_layer_w4a8(inp["W"], inp["Q"], spec.r, want_t=True)
    oo = orc.linear_deployed_w4a8(inp["x"], lo, bias=inp["bias"])

    dev = "cuda"
    W = torch.from_numpy(inp["W"]).to(dev)
    Q = torch.from_numpy(inp["Q"]).to(dev)
    bias = bits_to_bf16_tensor(inp["bias"]) if with_bias else None
    layer = dq.dirotq_prepare_layer_w4a8(W, Q, spec.r, bias=bias)
    check_weight_side(dq.dirotq_layer_export(layer), lo)

    x = bits_to_bf16_tensor(inp["x"])
    ws = dq.alloc_workspace(layer, M)
    xrot = torch.zeros((M, spec.K), dtype=torch.float32, device=dev) if check_rot else None
    dq.dirotq_rotate_quantize(x, layer, ws, xrot)
    assert dq.dirotq_workspace_status(ws) == 0
    xh, codes, scales = dq.dirotq_workspace_export_w4a8(layer, M, ws)
    xh_b, codes_n, scales_b = bf16_tensor_to_bits(xh), codes.cpu().numpy(), bf16_tensor_to_bits(scales)
    stats = check_activation_side_w4a8(xrot.cpu().numpy() if check_rot else None, xh_b, codes_n, scales_b, oo, spec.r)

    # integer sums over the whole of K on the oracle's codes: bit exact
    padded = np.zeros((M, layer.K_lp), dtype=np.int8)
    padded[:, :spec.K_l] = oo["codes"]
    P = dq.dirotq_int_gemm_debug(torch.from_numpy(padded).to(dev), layer, ws)
    assert dq.dirotq_workspace_status(ws) == 0
    assert np.array_equal(P[0].cpu().numpy(), oo["P"]), "int32 sums differ"

    y = torch.zeros((M, spec.N), dtype=torch.bfloat16, device=dev)
    dq.dirotq_linear(x, layer, y, ws)
    assert dq.dirotq_workspace_status(ws) == 0
    stats.update(check_layer_output_w4a8(bf16_tensor_to_bits(y), xh_b, codes_n, scales_b, lo, oo, inp["bias"]))
    y2 = torch.zeros_like(y)
    dq.dirotq_linear(x, layer, y2, ws)
    torch.cuda.synchronize()
    assert torch.equal(y.view(torch.int16), y2.view(torch.int16))
    layer.close()
    return stats


def test_w4a8_small_single_tile():
    spec = synth.LayerSpec(K=256, N=256, r=32, G=64, model=synth.PIXART, seed=1, calib_tokens=512)
    print(_run_case(spec, M=100))


def test_w4a8_config1_pixart_attention_projection():
    spec = synth.LayerSpec(K=1152, N=1152, r=32, G=64, model=synth.PIXART, seed=2)
    print(_run_case(spec, M=256))


def test_w4a8_ragged_m_and_n_rank16():
    spec = synth.LayerSpec(K=512, N=400, r=16, G=64, model=synth.FLUX, seed=3, calib_tokens=1024)
    print(_run_case(spec, M=300))


def test_w4a8_rank128_no_bias_padded_k():
    # K_l = 640 - 128 = 512... use K = 704: K_l = 576, padded to 640 codes per row
    spec = synth.LayerSpec(K=704, N=384, r=128, G=64, model=synth.FLUX, seed=5, calib_tokens=1024)
    print(_run_case(spec, M=257, with_bias=False))


def test_w4a8_many_tiles_wide_k():
    spec = synth.LayerSpec(K=3072, N=768, r=32, G=64, model=synth.FLUX, seed=8)
    print(_run_case(spec, M=520, check_rot=False))
