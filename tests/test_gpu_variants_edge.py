"""Degenerate inputs through the three format variants: all-zero tokens (zero scales, zero codes, output = bias) and
constant tokens, next to ordinary ones."""
import numpy as np
import pytest
import torch

from oracle import dirotq_oracle as orc
from paper_2605_16732_b200 import binding as dq
from paper_2605_16732_b200 import synth

from parity_utils import bf16_tensor_to_bits, bits_to_bf16_tensor

pytestmark = pytest.mark.gpu


def _inputs():
    spec = synth.LayerSpec(K=256, N=256, r=32, G=64, model=synth.PIXART, seed=7, calib_tokens=512)
    inp = synth.make_layer_inputs(spec, 40)
    x = inp["x"].copy()
    x[3] = 0
    x[17] = 0
    inp["x"] = x
    return spec, inp


def _check_zero_rows(y, bias_bits):
    yb = bf16_tensor_to_bits(y)
    for m in (3, 17):
        assert np.array_equal(yb[m], bias_bits), "an all-zero token must give exactly the bias"


def test_zero_tokens_nvfp4():
    spec, inp = _inputs()
    lo = orc.nvfp4_prepare_layer(inp["W"], inp["Q"], spec.r)
    xt = orc.rotate(inp["x"], lo["Qb"])
    ex = orc.nvfp4_global_exponent(float(np.abs(xt[:, spec.r:]).max()))
    layer = dq.dirotq_prepare_layer_nvfp4(torch.from_numpy(inp["W"]).cuda(), torch.from_numpy(inp["Q"]).cuda(), spec.r, ex,
                                          bias=bits_to_bf16_tensor(inp["bias"]))
    ws = dq.alloc_workspace(layer, 40)
    y = torch.zeros((40, spec.N), dtype=torch.bfloat16, device="cuda")
    dq.dirotq_linear(bits_to_bf16_tensor(inp["x"]), layer, y, ws)
    assert dq.dirotq_workspace_status(ws) == 0
    _, codes, sf = dq.dirotq_workspace_export_nvfp4(layer, 40, ws)
    assert not (codes[[3, 17]].cpu().numpy() & 7).any() and not sf[[3, 17]].cpu().numpy().any()
    _check_zero_rows(y, inp["bias"])
    layer.close()


def test_zero_tokens_asym():
    spec, inp = _inputs()
    layer = dq.dirotq_prepare_layer_asym(torch.from_numpy(inp["W"]).cuda(), torch.from_numpy(inp["Q"]).cuda(), spec.r, spec.G,
                                         bias=bits_to_bf16_tensor(inp["bias"]))
    ws = dq.alloc_workspace(layer, 40)
    y = torch.zeros((40, spec.N), dtype=torch.bfloat16, device="cuda")
    dq.dirotq_linear(bits_to_bf16_tensor(inp["x"]), layer, y, ws)
    assert dq.dirotq_workspace_status(ws) == 0
    _, codes, scales, zeros = dq.dirotq_workspace_export_asym(layer, 40, ws)
    for t in (codes, scales.view(torch.int16), zeros.view(torch.int16)):
        assert not t[[3, 17]].cpu().numpy().any()
    _check_zero_rows(y, inp["bias"])
    layer.close()


def test_zero_tokens_w4a8():
    spec, inp = _inputs()
    layer = dq.dirotq_prepare_layer_w4a8(torch.from_numpy(inp["W"]).cuda(), torch.from_numpy(inp["Q"]).cuda(), spec.r,
                                         bias=bits_to_bf16_tensor(inp["bias"]))
    ws = dq.alloc_workspace(layer, 40)
    y = torch.zeros((40, spec.N), dtype=torch.bfloat16, device="cuda")
    dq.dirotq_linear(bits_to_bf16_tensor(inp["x"]), layer, y, ws)
    assert dq.dirotq_workspace_status(ws) == 0
    _, codes, scales = dq.dirotq_workspace_export_w4a8(layer, 40, ws)
    assert not codes[[3, 17]].cpu().numpy().any() and not scales.view(torch.int16)[[3, 17]].cpu().numpy().any()
    _check_zero_rows(y, inp["bias"])
    layer.close()
