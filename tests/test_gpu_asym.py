"""Parity of the layer with asymmetric activation codes (Eq. 1 with z = min X) against the CPU oracle."""
import numpy as np
import pytest
import torch

from oracle import dirotq_oracle as orc
from paper_2605_16732_b200 import binding as dq
from paper_2605_16732_b200 import synth

from parity_utils import (bf16_tensor_to_bits, bits_to_bf16_tensor, check_activation_side_asym, check_layer_output_asym,
                          check_weight_side)

pytestmark = pytest.mark.gpu


def _run_case(spec: synth.LayerSpec, M: int, with_bias=True, shift=0.0, check_rot=True):
    inp = synth.make_layer_inputs(spec, M, with_bias=with_bias)
    if shift:
        # move the activations off-centre (what asymmetric codes are for): add a constant along every channel
        x = orc.bf16_to_f64(inp["x"]) + shift
        inp["x"] = orc.bf16_round(x)
    lo = orc.prepare_layer(inp["W"], inp["Q"], spec.r, spec.G, want_t=True)
    oo = orc.linear_deployed_asym(inp["x"], lo, bias=inp["bias"])

    dev = "cuda"
    W = torch.from_numpy(inp["W"]).to(dev)
    Q = torch.from_numpy(inp["Q"]).to(dev)
    bias = bits_to_bf16_tensor(inp["bias"]) if with_bias else None
    layer = dq.dirotq_prepare_layer_asym(W, Q, spec.r, spec.G, bias=bias)
    check_weight_side(dq.dirotq_layer_export(layer), lo)
    # zero-point term of the weight side: s_w * sum of the group's codes, exact
    n_g = layer.n_g
    csum = np.stack([lo["wcodes"][g * spec.G:(g + 1) * spec.G].astype(np.int64).sum(axis=0) for g in range(n_g)])
    d_ref = (orc.bf16_to_f64(lo["wscales"]) * csum).astype(np.float32)
    assert np.array_equal(dq.dirotq_layer_export_zero_term(layer).cpu().numpy(), d_ref), "zero-point term differs"

    x = bits_to_bf16_tensor(inp["x"])
    ws = dq.alloc_workspace(layer, M)
    xrot = torch.zeros((M, spec.K), dtype=torch.float32, device=dev) if check_rot else None
    dq.dirotq_rotate_quantize(x, layer, ws, xrot)
    assert dq.dirotq_workspace_status(ws) == 0
    xh, codes, scales, zeros = dq.dirotq_workspace_export_asym(layer, M, ws)
    xh_b, codes_n = bf16_tensor_to_bits(xh), codes.cpu().numpy()
    scales_b, zeros_b = bf16_tensor_to_bits(scales), bf16_tensor_to_bits(zeros)
    stats = check_activation_side_asym(xrot.cpu().numpy() if check_rot else None, xh_b, codes_n, scales_b, zeros_b, oo,
                                       spec.r, spec.G)

    # integer group sums on the oracle's unsigned codes: bit exact
    ws2 = dq.alloc_workspace(layer, M)
    padded = np.zeros((M, layer.K_lp), dtype=np.int8)
    padded[:, :spec.K_l] = oo["codes"].astype(np.int8)
    P = dq.dirotq_int_gemm_debug(torch.from_numpy(padded).to(dev), layer, ws2)
    assert dq.dirotq_workspace_status(ws2) == 0
    assert np.array_equal(P.cpu().numpy(), oo["P"]), "int32 group sums differ"

    y = torch.zeros((M, spec.N), dtype=torch.bfloat16, device=dev)
    dq.dirotq_linear(x, layer, y, ws)
    assert dq.dirotq_workspace_status(ws) == 0
    stats.update(check_layer_output_asym(bf16_tensor_to_bits(y), xh_b, codes_n, scales_b, zeros_b, lo, oo, inp["bias"]))
    y2 = torch.zeros_like(y)
    dq.dirotq_linear(x, layer, y2, ws)
    torch.cuda.synchronize()
    assert torch.equal(y.view(torch.int16), y2.view(torch.int16))
    with pytest.raises(dq.DirotqError):
        dq.dirotq_workspace_export(layer, M, ws)  # the symmetric export does not apply
    layer.close()
    return stats


def test_asym_small_single_tile():
    spec = synth.LayerSpec(K=256, N=256, r=32, G=64, model=synth.PIXART, seed=1, calib_tokens=512)
    print(_run_case(spec, M=100))


def test_asym_config1_pixart_attention_projection():
    spec = synth.LayerSpec(K=1152, N=1152, r=32, G=64, model=synth.PIXART, seed=2)
    print(_run_case(spec, M=256))


def test_asym_shifted_activations():
    spec = synth.LayerSpec(K=512, N=256, r=32, G=64, model=synth.PIXART, seed=7, calib_tokens=1024)
    print(_run_case(spec, M=192, shift=2.5))


def test_asym_ragged_m_and_n_group128():
    spec = synth.LayerSpec(K=512, N=400, r=16, G=128, model=synth.FLUX, seed=3, calib_tokens=1024)
    print(_run_case(spec, M=300))


def test_asym_rank128_no_bias():
    spec = synth.LayerSpec(K=768, N=384, r=128, G=64, model=synth.FLUX, seed=5, calib_tokens=1024)
    print(_run_case(spec, M=257, with_bias=False))


def test_asym_many_groups_wide_k():
    # n_g = 48: 144 zero-point columns, four 64-wide chunks on the bf16 branch
    spec = synth.LayerSpec(K=3072, N=512, r=32, G=64, model=synth.FLUX, seed=8)
    print(_run_case(spec, M=200, check_rot=False))
