"""Calibration of the NVFP4 activations' power-of-two scale through the C ABI against the reference's rule (App. E: the
largest block scale must fit E4M3): the exponent the library picks from a batch equals the one the CPU reference gives
for its own rotated (or Hadamard-rotated residual) coefficients of the same tokens."""
import numpy as np
import pytest
import torch

from oracle import dirotq_oracle as orc
from paper_2605_16732_b200 import binding as dq
from paper_2605_16732_b200 import synth

pytestmark = pytest.mark.gpu


def _check(got, amax_ref):
    want = orc.nvfp4_global_exponent(amax_ref)
    # the library works in fp32: at most one step apart, and only when the maximum sits on a power-of-two boundary
    assert abs(got - want) <= 1
    if got != want:
        assert abs(np.log2(amax_ref / 1536.0) - round(np.log2(amax_ref / 1536.0))) < 1e-3


@pytest.mark.parametrize("K,r,model", [(256, 32, synth.PIXART), (512, 16, synth.FLUX), (1152, 64, synth.FLUX)])
def test_projection_form_exponent(K, r, model):
    spec = synth.LayerSpec(K=K, N=64, r=r, G=64, model=model, seed=70 + r, calib_tokens=1024)
    inp = synth.make_layer_inputs(spec, 200, with_bias=False)
    Uh = np.ascontiguousarray(np.asarray(inp["Q"], dtype=np.float64)[:, :r])
    lay = orc.nvfp4_prepare_layer_ph(inp["W"], Uh)
    _, xl = orc.nvfp4_residual(inp["x"], lay)
    x = torch.from_numpy(np.ascontiguousarray(inp["x"]).view(np.int16)).cuda().view(torch.bfloat16)
    for uh in (torch.from_numpy(Uh).cuda(), torch.from_numpy(Uh.astype(np.float32)).cuda()):
        _check(dq.dirotq_act_scale_log2_ph(x, uh), float(np.abs(xl).max()))


def test_dense_rotation_exponent():
    spec = synth.LayerSpec(K=512, N=64, r=32, G=64, model=synth.FLUX, seed=75, calib_tokens=1024)
    inp = synth.make_layer_inputs(spec, 300, with_bias=False)
    xt = orc.rotate(inp["x"], orc.bf16_round(inp["Q"]))
    xrot = torch.from_numpy(xt.astype(np.float32)).cuda()
    _check(dq.dirotq_act_scale_log2_from_rotated(xrot, spec.r), float(np.abs(xt[:, spec.r:]).max()))
    assert dq.dirotq_act_scale_log2_from_rotated(torch.zeros((4, 64), dtype=torch.float32, device="cuda"), 16) == 0
