"""Pins of the oracle's NVFP4 pieces (Sec. 5.1: E2M1 elements, blocks of 16, FP8 E4M3 scales).

  * E4M3 decode/round against torch.float8_e4m3fn (an independent implementation of the format);
  * E2M1: the eight magnitudes of a 2-exponent/1-mantissa float (q_max = 6, Sec. 3), rounding =
    brute-force nearest value with ties to the even code, saturation at 6;
  * block quantizer: scale = E4M3 nearest to absmax/6 (relative to the tensor's power-of-two),
    the absmax element maps to +-6 (or saturates), error bounded by half the local spacing;
  * whole layer: with nothing quantized the path reduces to x W (Eq. 4); the dequantized
    formulation equals a plain fp64 product of the dequantized operands.
"""
import itertools

import numpy as np
import torch

from oracle import dirotq_oracle as orc
from paper_2605_16732_b200 import synth


def test_e4m3_decode_matches_torch_for_all_bytes():
    b = np.arange(256, dtype=np.uint8)
    ref = torch.from_numpy(b).view(torch.float8_e4m3fn).to(torch.float64).numpy()
    ours = orc.e4m3_to_f64(b)
    finite = np.isfinite(ref)  # 0x7F / 0xFF are NaN in the format
    assert np.array_equal(ours[finite], ref[finite])
    assert ours[0x7E] == 448.0 and ours[0x01] == 2.0 ** -9 and ours[0x08] == 2.0 ** -6


def test_e4m3_round_matches_torch_and_saturates():
    g = np.random.default_rng(0)
    v = np.abs(g.standard_normal(50000) * np.exp(g.uniform(-8, 6, 50000)))
    v = v[v < 448.0].astype(np.float32).astype(np.float64)  # float32-exact inputs: torch rounds from float32
    ours = np.array([orc._load().dq_e4m3_round(float(x)) for x in v], dtype=np.uint8)
    ref = torch.from_numpy(v.astype(np.float32)).to(torch.float8_e4m3fn).view(torch.uint8).numpy()
    assert np.array_equal(ours, ref)
    assert orc._load().dq_e4m3_round(1e9) == 0x7E and orc._load().dq_e4m3_round(0.0) == 0
    assert orc._load().dq_e4m3_round(2.0 ** -11) == 0           # below half of the smallest subnormal
    # ties: 1 + 1/16 is midway between 1.0 (even mantissa 000) and 1.125 -> 1.0
    assert orc._load().dq_e4m3_round(1.0625) == 0x38


def test_e2m1_values_and_rounding_bruteforce():
    vals = orc.e2m1_to_f64(np.arange(16, dtype=np.uint8))
    assert vals[:8].tolist() == [0.0, 0.5, 1.0, 1.5, 2.0, 3.0, 4.0, 6.0]
    assert vals[8:].tolist() == [-0.0, -0.5, -1.0, -1.5, -2.0, -3.0, -4.0, -6.0]
    # 1 sign, 2 exponent (bias 1), 1 mantissa bit: subnormal 0.5, then (1 + m/2) 2^(e-1)
    for c in range(8):
        e, m = c >> 1, c & 1
        assert vals[c] == (0.5 * m if e == 0 else (1 + m / 2) * 2.0 ** (e - 1))
    g = np.random.default_rng(1)
    for t in np.concatenate([g.uniform(-7, 7, 5000), [0.25, 0.75, 1.25, 1.75, 2.5, 3.5, 5.0, -2.5, 6.5, 100.0, -9.0]]):
        c = orc._load().dq_e2m1_round(float(t))
        d = np.abs(np.abs(t) - vals[:8])
        best = np.flatnonzero(d == d.min())
        if len(best) == 1:
            assert (c & 7) == best[0]
        else:
            assert (c & 7) in best and (c & 1) == 0      # tie -> even code
        assert bool(c & 8) == (t < 0)
    # the documented ties
    assert [orc._load().dq_e2m1_round(x) & 7 for x in (0.25, 0.75, 1.25, 1.75, 2.5, 3.5, 5.0)] == [0, 2, 2, 4, 4, 6, 6]


def test_block_quantizer_properties():
    g = np.random.default_rng(2)
    for trial in range(400):
        n = int(g.integers(1, 17))
        v = g.standard_normal(n) * 10.0 ** g.uniform(-2, 2)
        e = int(g.integers(-12, 4))
        sf, codes, t = orc.nvfp4_quantize_block(v, e)
        a = np.abs(v).max()
        target = a / 6.0 / 2.0 ** e
        ref_sf = torch.tensor([min(target, 448.0)], dtype=torch.float32).to(torch.float8_e4m3fn).view(torch.uint8).item()
        # float32 input rounding can move a value across an E4M3 boundary: allow the neighbour in that rare case
        assert abs(int(sf) - int(ref_sf)) <= 1
        s = float(orc.e4m3_to_f64(np.array([sf], dtype=np.uint8))[0]) * 2.0 ** e
        if s == 0.0:
            assert not codes.any()
            continue
        deq = orc.e2m1_to_f64(codes) * s
        # nearest representable value: error at most half the spacing around the value (spacing <= 2 s), saturation aside
        inside = np.abs(v) <= 6.0 * s
        assert np.all(np.abs(v - deq)[inside] <= 1.0 * s * (1 + 1e-12))
        small = np.abs(v) <= 2.0 * s
        assert np.all(np.abs(v - deq)[small] <= 0.25 * s * (1 + 1e-12))
        k = int(np.argmax(np.abs(v)))
        if target < 448.0 and sf > 8:  # normal scale: relative rounding error <= 1/16, so |t_max| in [6/1.0625, 6*1.0625]
            assert (codes[k] & 7) == 7


def test_global_exponent_puts_largest_block_scale_below_256():
    for amax in (1e-3, 0.37, 5.0, 900.0):
        e = orc.nvfp4_global_exponent(amax)
        assert amax / 6.0 / 2.0 ** e <= 256.0 < amax / 6.0 / 2.0 ** (e - 1)
    assert orc.nvfp4_global_exponent(0.0) == 0


def test_nvfp4_layer_is_a_product_of_dequantized_operands():
    spec = synth.LayerSpec(K=128, N=40, r=16, G=16, model=synth.PIXART, seed=4, calib_tokens=256)
    inp = synth.make_layer_inputs(spec, 12)
    layer = orc.nvfp4_prepare_layer(inp["W"], inp["Q"], spec.r)
    xc = synth.bf16_bits_to_f32(synth.make_tokens(spec, 256, 1_000_003)).astype(np.float64)
    ex = orc.nvfp4_global_exponent(np.abs((xc @ orc.bf16_to_f64(layer["Qb"]))[:, spec.r:]).max())
    out = orc.nvfp4_linear_deployed(inp["x"], layer, ex, bias=inp["bias"])
    nb = -(-spec.K_l // 16)
    xq = orc.e2m1_to_f64(out["codes"]) * np.repeat(orc.e4m3_to_f64(out["sf"]), 16, axis=1)[:, :spec.K_l] * 2.0 ** ex
    wq = orc.e2m1_to_f64(layer["wcodes"]) * np.repeat(orc.e4m3_to_f64(layer["wsf"]), 16, axis=0)[:spec.K_l] * 2.0 ** layer["ew"]
    ref = xq @ wq + orc.bf16_to_f64(out["xh"]) @ orc.bf16_to_f64(layer["Wh"]) + orc.bf16_to_f64(inp["bias"])[None, :]
    assert np.abs(out["y64"] - ref).max() <= 1e-12 * np.abs(ref).max()
    # and it approximates x W (the method's claim): 4-bit float error of a few percent of the output scale
    x = synth.bf16_bits_to_f32(inp["x"]).astype(np.float64)
    exact = x @ inp["W"].astype(np.float64) + orc.bf16_to_f64(inp["bias"])[None, :]
    assert np.linalg.norm(out["y64"] - exact) / np.linalg.norm(exact) < 0.1
    # blocks are counted from the first low-precision coefficient: the high block never enters a scale
    assert out["sf"].shape == (12, nb)
