"""Host-side calibration helper of the NVFP4 projection form against the reference: the power-of-two activation scale
it picks from a batch (plain torch ops on the CPU here) is the one the reference's rule (App. E: the largest block scale
must fit E4M3) gives for the reference's own Hadamard-rotated residual of the same tokens."""
import numpy as np
import torch

from oracle import dirotq_oracle as orc
from paper_2605_16732_b200 import synth
from paper_2605_16732_b200.suite import residual_exponent


def test_residual_exponent_matches_the_reference_rule():
    for seed, (K, r, model) in enumerate([(256, 32, synth.PIXART), (512, 16, synth.FLUX), (384, 64, synth.FLUX)]):
        spec = synth.LayerSpec(K=K, N=64, r=r, G=64, model=model, seed=70 + seed, calib_tokens=1024)
        inp = synth.make_layer_inputs(spec, 200, with_bias=False)
        Uh = np.ascontiguousarray(np.asarray(inp["Q"], dtype=np.float64)[:, :r])
        lay = orc.nvfp4_prepare_layer_ph(inp["W"], Uh)
        _, xl = orc.nvfp4_residual(inp["x"], lay)
        want = orc.nvfp4_global_exponent(float(np.abs(xl).max()))
        x = torch.from_numpy(np.ascontiguousarray(inp["x"]).view(np.int16)).view(torch.bfloat16)
        got = residual_exponent(x, torch.from_numpy(Uh), rows=200)
        # the helper works in fp32: at most one step apart, and only when the maximum sits on a power-of-two boundary
        assert abs(got - want) <= 1
        if got != want:
            amax = float(np.abs(xl).max())
            assert abs(np.log2(amax / 1536.0) - round(np.log2(amax / 1536.0))) < 1e-3
