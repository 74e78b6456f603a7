"""Pins of the oracle's W4A8 functions (Sec. 5.1: per-token INT8 activations, per-channel INT4 weights)."""
import numpy as np

from oracle import dirotq_oracle as orc


def _bf(bits):
    return orc.bf16_to_f64(np.asarray(bits, dtype=np.uint16))


def test_token_codes_are_nearest_levels_and_absmax_maps_to_127():
    rng = np.random.default_rng(0)
    M, K, r = 9, 16 + 300, 16
    xt = rng.standard_normal((M, K)) * rng.choice([0.01, 1.0, 30.0], size=(M, 1))
    sq = orc.split_quantize_a8(xt, r)
    s = _bf(sq["scales"])
    for m in range(M):
        low = xt[m, r:]
        levels = s[m] * np.arange(-127, 128)
        brute = np.argmin(np.abs(low[:, None] - levels[None, :]), axis=1) - 127
        tie = np.abs(np.abs(sq["t"][m] - np.floor(sq["t"][m])) - 0.5) < 1e-9
        assert np.array_equal(sq["codes"][m][~tie], brute[~tie])
        assert abs(int(sq["codes"][m][np.argmax(np.abs(low))])) == 127
        # error at most half a step (a hair more where the bf16 rounding of the scale clips the largest element)
        assert np.all(np.abs(s[m] * sq["codes"][m] - low) <= 0.5 * s[m] + np.abs(low).max() * 2.0 ** -8)
    assert np.array_equal(sq["xh"], orc.bf16_round(xt[:, :r]))


def test_scale_is_one_per_token_over_all_low_coefficients():
    xt = np.zeros((2, 8 + 40))
    xt[0, 8 + 37] = -254.0       # s = 2 exactly, code -127
    xt[0, 8 + 3] = 5.0           # 2.5 -> tie -> even code 2
    xt[0, 8 + 4] = 7.0           # 3.5 -> tie -> even code 4
    xt[0, 2] = 1000.0            # a high-precision coefficient does not enter the scale
    sq = orc.split_quantize_a8(xt, 8)
    assert _bf(sq["scales"])[0] == 2.0 and sq["scales"][1] == 0
    assert sq["codes"][0, 37] == -127 and sq["codes"][0, 3] == 2 and sq["codes"][0, 4] == 4
    assert not sq["codes"][1].any()


def test_weights_have_one_scale_per_output_channel():
    rng = np.random.default_rng(1)
    K, N, r = 48, 5, 16
    Q = np.linalg.qr(rng.standard_normal((K, K)))[0]
    W = rng.standard_normal((K, N)) * 0.02
    lo = orc.prepare_layer_w4a8(W, Q, r)
    assert lo["wscales"].shape == (1, N) and lo["wcodes"].shape == (K - r, N)
    Wt = orc.fold(Q, W)
    assert np.array_equal(lo["wscales"][0], orc.bf16_round(np.abs(Wt[r:]).max(axis=0) / 7.0))
    assert np.all(np.abs(lo["wcodes"]).max(axis=0) == 7)


def test_integer_path_equals_dequantize_then_multiply():
    rng = np.random.default_rng(2)
    M, K, N, r = 6, 16 + 80, 7, 16
    Q = np.linalg.qr(rng.standard_normal((K, K)))[0]
    W = rng.standard_normal((K, N)) * 0.02
    lo = orc.prepare_layer_w4a8(W, Q, r)
    x_bits = orc.bf16_round(rng.standard_normal((M, K)) * 2.0)
    bias = orc.bf16_round(rng.standard_normal(N) * 0.02)
    out = orc.linear_deployed_w4a8(x_bits, lo, bias=bias)
    xq = _bf(out["scales"])[:, None] * out["codes"]
    wq = _bf(lo["wscales"]) * lo["wcodes"]
    ref = xq @ wq + _bf(out["xh"]) @ _bf(lo["Wh"]) + _bf(bias)[None, :]
    assert np.max(np.abs(out["y64"] - ref)) <= 1e-12 * max(1.0, np.max(np.abs(ref)))
    for (m, n) in [(0, 0), (5, 6), (3, 2)]:
        assert out["P"][m, n] == sum(int(out["codes"][m, j]) * int(lo["wcodes"][j, n]) for j in range(K - r))


def test_eight_bit_activations_are_closer_to_the_unquantized_product_than_four_bit_ones():
    rng = np.random.default_rng(3)
    M, K, N, r = 32, 16 + 256, 24, 16
    Q = np.linalg.qr(rng.standard_normal((K, K)))[0]
    W = rng.standard_normal((K, N)) * 0.02
    x = rng.standard_normal((M, K))
    x_bits = orc.bf16_round(x)
    ideal = orc.linear_ideal(orc.bf16_to_f64(x_bits), Q, W, r)
    # same per-channel 4-bit weights on both sides; only the activation format differs
    lo = orc.prepare_layer_w4a8(W, Q, r)
    y8 = orc.linear_deployed_w4a8(x_bits, lo)["y64"]
    y4 = orc.linear_deployed(x_bits, lo)["y64"]       # 4-bit activations, one group spanning the row
    assert np.mean((y8 - ideal) ** 2) < np.mean((y4 - ideal) ** 2)
