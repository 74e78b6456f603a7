"""Pins of the oracle's asymmetric activation quantizer (Sec. 3, Eq. 1 with z = min X, q in 0..15) and of the
combination with its zero-point term.  None of them re-types the oracle's formula: they check it against a
nearest-level search, closed-form special cases, invariances, and the plain dequantize-then-multiply product."""
import numpy as np
import pytest

from oracle import dirotq_oracle as orc


def _bf(bits):
    return orc.bf16_to_f64(np.asarray(bits, dtype=np.uint16))


def test_codes_are_the_nearest_of_the_sixteen_levels():
    rng = np.random.default_rng(0)
    for trial in range(200):
        n = int(rng.integers(2, 65))
        v = rng.standard_normal(n) * rng.choice([0.01, 1.0, 50.0]) + rng.choice([0.0, 3.0, -20.0])
        sb, zb, codes, t = orc.quantize_group_asym(v)
        s, z = float(_bf([sb])[0]), float(_bf([zb])[0])
        levels = z + s * np.arange(16)
        brute = np.argmin(np.abs(v[:, None] - levels[None, :]), axis=1)
        tie = np.abs(np.abs(t - np.floor(t)) - 0.5) < 1e-9
        assert np.array_equal(codes[~tie], brute[~tie])
        assert codes.min() >= 0 and codes.max() <= 15


def test_scale_and_zero_point_follow_the_range():
    # values chosen so that min and (max - min)/15 are exact in bf16: z = -2, s = 0.5, levels -2, -1.5, ..., 5.5
    v = np.array([-2.0, 5.5, 0.26, 0.24, 3.0, -1.76])
    sb, zb, codes, t = orc.quantize_group_asym(v)
    assert _bf([zb])[0] == -2.0 and _bf([sb])[0] == 0.5
    assert list(codes) == [0, 15, 5, 4, 10, 0]
    # ties go to the even code: -1.75 is exactly between levels 0 (-2) and 1 (-1.5); -0.75 between 2 and 3
    _, _, c2, _ = orc.quantize_group_asym(np.array([-2.0, 5.5, -1.75, -0.75]))
    assert list(c2) == [0, 15, 0, 2]


def test_minimum_maps_to_zero_and_maximum_to_fifteen_and_error_is_half_a_step():
    rng = np.random.default_rng(1)
    for trial in range(100):
        v = rng.standard_normal(64) * 3.0
        sb, zb, codes, _ = orc.quantize_group_asym(v)
        s, z = float(_bf([sb])[0]), float(_bf([zb])[0])
        assert codes[np.argmin(v)] == 0 and codes[np.argmax(v)] == 15
        deq = z + s * codes
        # half a step, plus what the bf16 rounding of z and s moves the grid by
        slack = abs(z - v.min()) + 15 * abs(s - (v.max() - v.min()) / 15.0)
        assert np.all(np.abs(deq - v) <= 0.5 * s + slack + 1e-12)


def test_constant_group_and_single_element():
    sb, zb, codes, _ = orc.quantize_group_asym(np.full(16, 1.25))
    assert sb == 0 and _bf([zb])[0] == 1.25 and not codes.any()
    sb, zb, codes, _ = orc.quantize_group_asym(np.array([-7.0]))
    assert sb == 0 and _bf([zb])[0] == -7.0 and codes[0] == 0


def test_shift_by_a_representable_constant_moves_only_the_zero_point():
    rng = np.random.default_rng(2)
    v = np.round(rng.standard_normal(32) * 4.0) / 4.0          # multiples of 0.25, |v| < 32
    v[0], v[1] = -3.0, 4.5                                      # fixes min and max: range 7.5, s = 0.5 exactly
    sb0, zb0, c0, _ = orc.quantize_group_asym(v)
    sb1, zb1, c1, _ = orc.quantize_group_asym(v + 8.0)
    assert sb0 == sb1 and np.array_equal(c0, c1)
    assert _bf([zb1])[0] - _bf([zb0])[0] == 8.0


def test_split_quantize_places_groups_and_handles_the_ragged_tail():
    rng = np.random.default_rng(3)
    M, K, r, G = 5, 16 + 40, 16, 16          # K_l = 40: groups of 16, 16 and a ragged one of 8
    xt = rng.standard_normal((M, K)) * 2.0 + 1.0
    sq = orc.split_quantize_asym(xt, r, G)
    assert sq["codes"].shape == (M, 40) and sq["scales"].shape == (M, 3) and sq["zeros"].shape == (M, 3)
    for m in range(M):
        for g, (a, b) in enumerate([(0, 16), (16, 32), (32, 40)]):
            sb, zb, codes, _ = orc.quantize_group_asym(xt[m, r + a:r + b])
            assert sq["scales"][m, g] == sb and sq["zeros"][m, g] == zb
            assert np.array_equal(sq["codes"][m, a:b], codes)
    assert np.array_equal(sq["xh"], orc.bf16_round(xt[:, :r]))


def test_integer_path_with_zero_point_term_equals_dequantize_then_multiply():
    rng = np.random.default_rng(4)
    M, K, N, r, G = 7, 16 + 72, 12, 16, 32    # K_l = 72: two full groups and a ragged one of 8
    Q = np.linalg.qr(rng.standard_normal((K, K)))[0]
    W = rng.standard_normal((K, N)) * 0.02
    layer = orc.prepare_layer(W, Q, r, G)
    xt = rng.standard_normal((M, K)) * 2.0 + 0.7
    sq = orc.split_quantize_asym(xt, r, G)
    P = orc.int_gemm_u(sq["codes"], layer["wcodes"], G)
    bias = orc.bf16_round(rng.standard_normal(N) * 0.02)
    y64, yb = orc.combine_asym(P, sq["scales"], sq["zeros"], layer, sq["xh"], bias)
    # plain route: dequantize both sides element by element, then one fp64 product
    K_l = K - r
    gi = np.arange(K_l) // G
    xq = _bf(sq["scales"])[:, gi] * sq["codes"] + _bf(sq["zeros"])[:, gi]
    wq = _bf(layer["wscales"])[gi, :] * layer["wcodes"]
    ref = xq @ wq + _bf(sq["xh"]) @ _bf(layer["Wh"]) + _bf(bias)[None, :]
    assert np.max(np.abs(y64 - ref)) <= 1e-12 * max(1.0, np.max(np.abs(ref)))
    assert np.array_equal(yb, orc.bf16_round(y64))
    # brute-force integer sums on a few entries
    for (g, m, n) in [(0, 0, 0), (2, 6, 11), (1, 3, 5)]:
        j0, j1 = g * G, min((g + 1) * G, K_l)
        assert P[g, m, n] == sum(int(sq["codes"][m, j]) * int(layer["wcodes"][j, n]) for j in range(j0, j1))


def test_asymmetric_codes_beat_symmetric_ones_on_shifted_activations():
    # the reason the paper quantizes activations asymmetrically: a group that sits off-centre wastes half of a
    # symmetric grid.  Same data, same group size: the asymmetric reconstruction error must be clearly smaller.
    rng = np.random.default_rng(5)
    xt = np.abs(rng.standard_normal((64, 16 + 256))) + 0.5       # all low-precision coefficients positive
    a = orc.split_quantize_asym(xt, 16, 64)
    s = orc.split_quantize(xt, 16, 64)
    gi = np.arange(256) // 64
    xa = _bf(a["scales"])[:, gi] * a["codes"] + _bf(a["zeros"])[:, gi]
    xs = _bf(s["scales"])[:, gi] * s["codes"]
    ea, es = np.mean((xa - xt[:, 16:]) ** 2), np.mean((xs - xt[:, 16:]) ** 2)
    assert ea < 0.3 * es
