"""Parity of the NVFP4 variant (E2M1 elements, blocks of 16, E4M3 scales) against the CPU oracle."""
import numpy as np
import pytest
import torch

from oracle import dirotq_oracle as orc
from paper_2605_16732_b200 import binding as dq
from paper_2605_16732_b200 import synth

from parity_utils import (bf16_tensor_to_bits, bits_to_bf16_tensor, check_activation_side_nvfp4,
                          check_layer_output_nvfp4, check_weight_side_nvfp4)

pytestmark = pytest.mark.gpu


def _run_case(spec: synth.LayerSpec, M: int, with_bias=True, ex_shift=0, check_rot=True):
    inp = synth.make_layer_inputs(spec, M, with_bias=with_bias)
    lo = orc.nvfp4_prepare_layer(inp["W"], inp["Q"], spec.r, want_t=True)
    # calibration of the activations' power-of-two scale: on this batch, by the oracle
    xt = orc.rotate(inp["x"], lo["Qb"])
    ex = orc.nvfp4_global_exponent(float(np.abs(xt[:, spec.r:]).max())) + ex_shift
    oo = orc.nvfp4_linear_deployed(inp["x"], lo, ex, bias=inp["bias"])

    dev = "cuda"
    W = torch.from_numpy(inp["W"]).to(dev)
    Q = torch.from_numpy(inp["Q"]).to(dev)
    bias = bits_to_bf16_tensor(inp["bias"]) if with_bias else None
    layer = dq.dirotq_prepare_layer_nvfp4(W, Q, spec.r, ex, bias=bias)
    stats = check_weight_side_nvfp4(dq.dirotq_layer_export_nvfp4(layer), lo)

    x = bits_to_bf16_tensor(inp["x"])
    ws = dq.alloc_workspace(layer, M)
    xrot = torch.zeros((M, spec.K), dtype=torch.float32, device=dev) if check_rot else None
    dq.dirotq_rotate_quantize(x, layer, ws, xrot)
    assert dq.dirotq_workspace_status(ws) == 0
    xh, codes, sf = dq.dirotq_workspace_export_nvfp4(layer, M, ws)
    xh_b, codes_n, sf_n = bf16_tensor_to_bits(xh), codes.cpu().numpy(), sf.cpu().numpy()
    stats.update(check_activation_side_nvfp4(xrot.cpu().numpy() if check_rot else None, xh_b, codes_n, sf_n, oo, spec.r, ex))

    y = torch.zeros((M, spec.N), dtype=torch.bfloat16, device=dev)
    dq.dirotq_linear(x, layer, y, ws)
    assert dq.dirotq_workspace_status(ws) == 0
    stats.update(check_layer_output_nvfp4(bf16_tensor_to_bits(y), xh_b, codes_n, sf_n, ex, lo, oo, inp["bias"]))
    y2 = torch.zeros_like(y)
    dq.dirotq_linear(x, layer, y2, ws)
    torch.cuda.synchronize()
    assert torch.equal(y.view(torch.int16), y2.view(torch.int16))
    layer.close()
    return stats


def test_nvfp4_small_single_tile():
    spec = synth.LayerSpec(K=256, N=256, r=32, G=64, model=synth.PIXART, seed=1, calib_tokens=512)
    print(_run_case(spec, M=100))


def test_nvfp4_config1_pixart_attention_projection():
    spec = synth.LayerSpec(K=1152, N=1152, r=32, G=64, model=synth.PIXART, seed=2)
    print(_run_case(spec, M=256))


def test_nvfp4_ragged_m_and_n_rank16():
    # K_l = 496: the last block of 64 is half padding, the last k-block of 256 mostly so
    spec = synth.LayerSpec(K=512, N=400, r=16, G=64, model=synth.FLUX, seed=3, calib_tokens=1024)
    print(_run_case(spec, M=300))


def test_nvfp4_rank64_no_bias():
    spec = synth.LayerSpec(K=640, N=512, r=64, G=64, model=synth.FLUX, seed=4, calib_tokens=1024)
    print(_run_case(spec, M=129, with_bias=False))


def test_nvfp4_rank128_two_rank_chunks():
    spec = synth.LayerSpec(K=768, N=384, r=128, G=64, model=synth.FLUX, seed=5, calib_tokens=1024)
    print(_run_case(spec, M=257))


def test_nvfp4_saturating_activation_scale():
    # a per-tensor exponent 3 below the calibrated one: block scales saturate at 448, codes at +-6
    spec = synth.LayerSpec(K=512, N=256, r=32, G=64, model=synth.PIXART, seed=6, calib_tokens=1024)
    print(_run_case(spec, M=192, ex_shift=-3))


def test_nvfp4_int4_entry_points_reject_the_layer():
    spec = synth.LayerSpec(K=256, N=256, r=32, G=64, model=synth.PIXART, seed=1, calib_tokens=512)
    inp = synth.make_layer_inputs(spec, 16)
    layer = dq.dirotq_prepare_layer_nvfp4(torch.from_numpy(inp["W"]).cuda(), torch.from_numpy(inp["Q"]).cuda(), spec.r, 0)
    with pytest.raises(dq.DirotqError):
        dq.dirotq_layer_export(layer)
    layer.close()
