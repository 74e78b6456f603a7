"""The oracle against the constants the paper prints for its number formats (tests/golden/quantizer_constants.txt)."""
import os

import numpy as np

from oracle import dirotq_oracle as orc

_HERE = os.path.dirname(os.path.abspath(__file__))


def _constants():
    out = {}
    for line in open(os.path.join(_HERE, "golden", "quantizer_constants.txt")):
        line = line.split("#")[0].split()
        if len(line) == 2:
            out[line[0]] = int(line[1])
    return out


def test_symmetric_int4_reaches_exactly_qmax():
    c = _constants()
    rng = np.random.default_rng(0)
    G = c["int4_group_size"]
    xt = rng.standard_normal((8, 16 + 3 * G))
    sq = orc.split_quantize(xt, 16, G)
    per_group = np.abs(sq["codes"]).reshape(8, 3, G).max(axis=2)
    assert np.all(per_group == c["int4_symmetric_qmax"])
    # and nothing beyond it, even when the bf16 rounding of the scale makes x / s exceed q_max
    assert np.abs(sq["codes"]).max() == c["int4_symmetric_qmax"]


def test_asymmetric_int4_spans_qmin_to_qmax():
    c = _constants()
    rng = np.random.default_rng(1)
    G = c["int4_group_size"]
    xt = rng.standard_normal((8, 16 + 2 * G)) + 3.0
    sq = orc.split_quantize_asym(xt, 16, G)
    codes = sq["codes"].reshape(8, 2, G)
    assert np.all(codes.min(axis=2) == c["int4_asymmetric_qmin"])
    assert np.all(codes.max(axis=2) == c["int4_asymmetric_qmax"])


def test_int8_activations_reach_exactly_qmax():
    c = _constants()
    rng = np.random.default_rng(2)
    sq = orc.split_quantize_a8(rng.standard_normal((8, 16 + 200)), 16)
    assert np.all(np.abs(sq["codes"]).max(axis=1) == c["int8_symmetric_qmax"])


def test_fp4_grid_tops_out_at_qmax_and_blocks_have_sixteen_elements():
    c = _constants()
    values = orc.e2m1_to_f64(np.arange(16, dtype=np.uint8))
    assert values.max() == c["fp4_qmax"] and values.min() == -c["fp4_qmax"]
    assert len(set(np.abs(values))) == 8          # 1 sign, 2 exponent, 1 mantissa bit: eight magnitudes
    rng = np.random.default_rng(3)
    xt = rng.standard_normal((4, 16 + 4 * c["nvfp4_group_size"]))
    ex = orc.nvfp4_global_exponent(float(np.abs(xt[:, 16:]).max()))
    sq = orc.nvfp4_split_quantize(xt, 16, ex)
    assert sq["sf"].shape == (4, 4)               # one scale per block of 16
    # the largest element of every block lands on the largest or second-largest magnitude (the E4M3 scale is rounded)
    mags = np.abs(orc.e2m1_to_f64(sq["codes"])).reshape(4, 4, c["nvfp4_group_size"]).max(axis=2)
    assert np.all(mags >= 4.0) and np.all(mags <= c["fp4_qmax"])
