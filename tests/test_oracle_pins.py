"""Pins of the CPU oracle against facts fixed by the paper and by arithmetic -- none of them
re-types the oracle's own formula.

  * Lemma (App. C) / Sec. 4.2: the combined rotation is orthogonal.
  * Eq. 4: with nothing quantized, [xU_h, x~_l][W~_h; W~_l] == x W.
  * App. B: the PCA basis diagonalises the calibration second moment, eigenvalues descending.
  * Eq. 1 (symmetric): the code is the nearest of the 15 levels q*s (brute-force search), the
    absmax element maps to +-7, the error is at most s/2.
  * Integer products: exhaustive enumeration for K <= 2, Python big-int dot products for K <= 8.
  * Special case V = I, r = 0, one group: textbook per-token / per-column RTN W4A4.
  * Integer path == dequantized path.
"""
import itertools

import numpy as np
import pytest
import torch

from oracle import dirotq_oracle as orc
from paper_2605_16732_b200 import synth


def _f64(bits):
    return orc.bf16_to_f64(bits)


# ---------------------------------------------------------------- bf16 rounding


def test_bf16_known_values():
    assert orc._load().dq_double_to_bf16(1.0) == 0x3F80
    assert orc._load().dq_double_to_bf16(-2.0) == 0xC000
    # ties: 1 + 2^-8 lies midway between 1 and 1 + 2^-7 -> even mantissa (1.0)
    assert orc._load().dq_double_to_bf16(1.0 + 2.0 ** -8) == 0x3F80
    # 1 + 3*2^-8 lies midway between 0x3F81 and 0x3F82 -> even (0x3F82)
    assert orc._load().dq_double_to_bf16(1.0 + 3 * 2.0 ** -8) == 0x3F82
    # just above / below the tie
    assert orc._load().dq_double_to_bf16(1.0 + 2.0 ** -8 + 2.0 ** -40) == 0x3F81
    assert orc._load().dq_double_to_bf16(1.0 + 2.0 ** -8 - 2.0 ** -40) == 0x3F80
    # a carry into the next binade
    assert orc._load().dq_double_to_bf16(1.998046875 + 2.0 ** -9) == 0x4000
    assert orc._load().dq_double_to_bf16(0.0) == 0


def test_bf16_matches_torch_on_float32_inputs():
    g = np.random.default_rng(0)
    a = (g.standard_normal(200000) * np.exp(g.uniform(-30, 30, 200000))).astype(np.float32)
    ours = orc.bf16_round(a.astype(np.float64))
    ref = torch.from_numpy(a).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)
    assert np.array_equal(ours, ref)
    # the generator's own rounding helper agrees too (it feeds both sides)
    assert np.array_equal(synth.bf16_bits(a), ref)


def test_bf16_direct_rounding_has_no_double_rounding():
    # 1 + 2^-8 + 2^-30 is above the tie; rounding through float32 first would land on the tie
    v = 1.0 + 2.0 ** -8 + 2.0 ** -30
    assert orc._load().dq_double_to_bf16(v) == 0x3F81
    assert synth.bf16_bits(np.array([v]))[0] == 0x3F81


# ---------------------------------------------------------------- Eq. 1 quantizer


def test_quantizer_hand_example():
    # a = 7 -> s = 1; -3.5 and 2.5 are ties -> even codes -4 and 2; 0.4 -> 0
    sb, codes, t = orc.quantize_group([7.0, -3.5, 0.4, 2.5, -0.5, 6.5])
    assert sb == 0x3F80
    assert codes.tolist() == [7, -4, 0, 2, 0, 6]
    assert np.allclose(t, [7.0, -3.5, 0.4, 2.5, -0.5, 6.5])


def test_quantizer_zero_group():
    sb, codes, _ = orc.quantize_group(np.zeros(5))
    assert sb == 0 and not codes.any()


def test_quantizer_is_nearest_level_bruteforce():
    g = np.random.default_rng(1)
    levels = np.arange(-7, 8, dtype=np.float64)
    for trial in range(300):
        n = int(g.integers(1, 9))
        v = g.standard_normal(n) * 10.0 ** g.uniform(-3, 3)
        if trial % 7 == 0:
            v[g.integers(0, n)] = 0.0
        sb, codes, t = orc.quantize_group(v)
        s = float(_f64(np.array([sb], dtype=np.uint16))[0])
        a = np.abs(v).max()
        if a == 0.0:
            assert sb == 0 and not codes.any()
            continue
        # scale is the bf16 nearest to a/7 (torch as an independent rounding routine)
        ref_s = torch.tensor([a / 7.0], dtype=torch.float64).to(torch.float32).to(torch.bfloat16)
        assert abs(s - float(ref_s)) <= 2.0 ** -7 * s  # at most the neighbouring bf16 (double rounding)
        assert abs(s - a / 7.0) <= 2.0 ** -8 * (a / 7.0) * (1 + 1e-12)
        # brute force: nearest level, ties towards the even code
        d = np.abs(v[:, None] - levels[None, :] * s)
        best = d.min(axis=1)
        for i in range(n):
            cand = levels[np.isclose(d[i], best[i], rtol=0, atol=0)]
            if len(cand) == 1:
                assert codes[i] == cand[0]
            else:
                assert codes[i] in cand and codes[i] % 2 == 0
        # the absmax element maps to +-7 and the error bound of a uniform quantizer holds
        k = int(np.argmax(np.abs(v)))
        assert abs(codes[k]) == 7
        inside = np.abs(v) <= 7.5 * s
        assert np.all(np.abs(v - codes * s)[inside] <= s / 2 * (1 + 1e-12))


def test_quantizer_clip_range():
    # a scale rounded *down* in bf16 pushes the absmax quotient slightly above 7: still code 7
    v = np.array([7.0 * (1 + 2.0 ** -9) * 1.0001, 1.0])
    _, codes, t = orc.quantize_group(v)
    assert codes[0] == 7 and t[0] > 7.0
    assert np.all(np.abs(codes) <= 7)


# ---------------------------------------------------------------- integer GEMM


def test_int_gemm_exhaustive_K1_K2():
    vals = np.arange(-7, 8, dtype=np.int8)
    # K = 1: all 225 pairs at once (M = N = 15)
    P = orc.int_gemm(vals[:, None], vals[None, :], G=64)
    assert np.array_equal(P[0], vals.astype(np.int32)[:, None] * vals.astype(np.int32)[None, :])
    # K = 2: every (a0,a1) x (b0,b1)
    pairs = np.array(list(itertools.product(range(-7, 8), repeat=2)), dtype=np.int8)  # [225, 2]
    P = orc.int_gemm(pairs, pairs.T.copy(), G=64)
    for i, (a0, a1) in enumerate(pairs.tolist()):
        row = [a0 * b0 + a1 * b1 for (b0, b1) in pairs.tolist()]
        assert P[0, i].tolist() == row


@pytest.mark.parametrize("K_l,G", [(3, 2), (5, 4), (8, 3), (8, 8), (7, 64)])
def test_int_gemm_python_ints_and_group_ranges(K_l, G):
    g = np.random.default_rng(K_l * 100 + G)
    M, N = 4, 5
    qx = g.integers(-7, 8, (M, K_l)).astype(np.int8)
    qw = g.integers(-7, 8, (K_l, N)).astype(np.int8)
    P = orc.int_gemm(qx, qw, G)
    n_g = -(-K_l // G)
    assert P.shape == (n_g, M, N)
    for gi in range(n_g):
        for m in range(M):
            for n in range(N):
                ref = sum(int(qx[m, j]) * int(qw[j, n]) for j in range(gi * G, min(K_l, (gi + 1) * G)))
                assert int(P[gi, m, n]) == ref


def test_int_gemm_extreme_magnitude():
    qx = np.full((1, 128), -7, dtype=np.int8)
    qw = np.full((128, 1), 7, dtype=np.int8)
    assert orc.int_gemm(qx, qw, 128)[0, 0, 0] == -49 * 128


# ---------------------------------------------------------------- rotation and Eq. 4


@pytest.fixture(scope="module")
def small_layer():
    spec = synth.LayerSpec(K=128, N=48, r=16, G=32, model=synth.PIXART, seed=3, calib_tokens=512)
    inp = synth.make_layer_inputs(spec, M=20)
    return spec, inp


def test_rotation_is_orthogonal(small_layer):
    spec, inp = small_layer
    Q = inp["Q"]
    assert np.abs(Q.T @ Q - np.eye(spec.K)).max() < 1e-10
    assert np.abs(Q @ Q.T - np.eye(spec.K)).max() < 1e-10


def test_pca_basis_diagonalises_second_moment(small_layer):
    spec, inp = small_layer
    xc = synth.bf16_bits_to_f32(synth.make_tokens(spec, spec.calib_tokens, 1_000_003)).astype(np.float64)
    sigma = xc.T @ xc / spec.calib_tokens
    Uh = inp["Q"][:, :spec.r]
    lam = np.diag(Uh.T @ sigma @ Uh)
    off = Uh.T @ sigma @ Uh - np.diag(lam)
    assert np.abs(off).max() < 1e-8 * lam.max()
    assert np.all(np.diff(lam) <= 1e-9 * lam.max())
    # the high block carries the planted energy: every remaining direction has less variance
    rest = inp["Q"][:, spec.r:]
    assert np.diag(rest.T @ sigma @ rest).max() <= lam.min() * (1 + 1e-9)


def test_eq4_identity_ideal_mode(small_layer):
    spec, inp = small_layer
    x = synth.bf16_bits_to_f32(inp["x"]).astype(np.float64)
    W = inp["W"].astype(np.float64)
    ref = x @ W
    scale = np.abs(ref).max()
    for r in (0, spec.r, spec.K):
        y = orc.linear_ideal(x, inp["Q"], W, r)
        assert np.abs(y - ref).max() <= 1e-9 * scale


def test_fold_uses_transpose(small_layer):
    # a transposed operand in the fold would break this: (Q^T W)[i,:] = sum_k Q[k,i] W[k,:]
    spec, inp = small_layer
    W = inp["W"].astype(np.float64)
    Wt = orc.fold(inp["Q"], W)
    assert np.abs(Wt - inp["Q"].T @ W).max() < 1e-12
    assert np.abs(Wt - inp["Q"] @ W).max() > 1e-3


def test_rotate_matches_numpy(small_layer):
    spec, inp = small_layer
    Qb = orc.bf16_round(inp["Q"])
    xt = orc.rotate(inp["x"], Qb)
    ref = synth.bf16_bits_to_f32(inp["x"]).astype(np.float64) @ _f64(Qb)
    assert np.abs(xt - ref).max() <= 1e-12 * np.abs(ref).max()


# ---------------------------------------------------------------- grouping conventions


def test_groups_count_from_first_low_column_and_ragged_tail():
    # K = 12, r = 2, G = 4: K_l = 10 -> groups [2..5], [6..9], [10..11] (ragged, 2 wide)
    M, K, r, G = 1, 12, 2, 4
    xt = np.zeros((M, K))
    xt[0, 0] = 1000.0            # high column: must not influence any scale
    xt[0, 2:6] = [1, 2, 3, 7]    # group 0, s = 1
    xt[0, 6:10] = [14, 0, -2, 4]  # group 1, s = 2
    xt[0, 10:12] = [0.5, -3.5]   # ragged group 2, s = 0.5
    out = orc.split_quantize(xt, r, G)
    assert _f64(out["scales"]).tolist() == [[1.0, 2.0, 0.5]]
    assert out["codes"].tolist() == [[1, 2, 3, 7, 7, 0, -1, 2, 1, -7]]
    assert _f64(out["xh"]).tolist() == [[1000.0, 0.0]]


def test_weight_groups_run_along_K_per_output_column():
    K, N, r, G = 10, 2, 2, 4
    Wt = np.zeros((K, N))
    Wt[0] = [5.0, 6.0]
    Wt[2:6, 0] = [7, 1, 1, 1]
    Wt[2:6, 1] = [14, 2, 2, 2]
    Wt[6:10, 0] = [0, 0, 0, 3.5]
    out = orc.prepare_weights(Wt, r, G)
    assert _f64(out["wscales"]).tolist() == [[1.0, 2.0], [0.5, 0.0]]
    assert out["wcodes"][:, 0].tolist() == [7, 1, 1, 1, 0, 0, 0, 7]
    assert out["wcodes"][:, 1].tolist() == [7, 1, 1, 1, 0, 0, 0, 0]
    assert _f64(out["Wh"]).tolist() == [[5.0, 6.0], [0.0, 0.0]]


# ---------------------------------------------------------------- whole layer


def test_integer_path_equals_dequantized_path(small_layer):
    spec, inp = small_layer
    layer = orc.prepare_layer(inp["W"], inp["Q"], spec.r, spec.G)
    out = orc.linear_deployed(inp["x"], layer, bias=inp["bias"])
    sx = _f64(out["scales"])
    sw = _f64(layer["wscales"])
    xq = out["codes"].astype(np.float64) * np.repeat(sx, spec.G, axis=1)[:, :spec.K_l]
    wq = layer["wcodes"].astype(np.float64) * np.repeat(sw, spec.G, axis=0)[:spec.K_l]
    ref = xq @ wq + _f64(out["xh"]) @ _f64(layer["Wh"]) + _f64(inp["bias"])[None, :]
    assert np.abs(out["y64"] - ref).max() <= 1e-12 * np.abs(ref).max()
    # final rounding is bf16 nearest of that value
    assert np.array_equal(out["y"], orc.bf16_round(out["y64"]))


def test_textbook_rtn_special_case():
    """V = I, r = 0, one group spanning K: per-token activation scale, per-column weight scale."""
    g = np.random.default_rng(5)
    M, K, N = 6, 24, 7
    x_bits = synth.bf16_bits(g.standard_normal((M, K)) * 3)
    W = g.standard_normal((K, N)) * 0.02
    layer = orc.prepare_layer(W, np.eye(K), r=0, G=K)
    out = orc.linear_deployed(x_bits, layer)

    def bf(a):
        return torch.tensor(a, dtype=torch.float64).to(torch.float32).to(torch.bfloat16).to(torch.float64).numpy()

    x = synth.bf16_bits_to_f32(x_bits).astype(np.float64)
    sx = bf(np.abs(x).max(axis=1, keepdims=True) / 7)
    sw = bf(np.abs(W).max(axis=0, keepdims=True) / 7)
    xq = np.clip(np.round(x / sx), -7, 7) * sx   # np.round is half-to-even
    wq = np.clip(np.round(W / sw), -7, 7) * sw
    ref = xq @ wq
    assert np.abs(out["y64"] - ref).max() <= 1e-12 * np.abs(ref).max()


def test_quantization_error_shrinks_with_structure(small_layer):
    """Qualitative check of the method's claim (Fig. 1, Table 2): on outlier-heavy activations,
    plain RTN < PCA split < PCA split + R in output fidelity."""
    spec, inp = small_layer
    x = synth.bf16_bits_to_f32(inp["x"]).astype(np.float64)
    W = inp["W"].astype(np.float64)
    ref = x @ W

    def err(Q, r):
        layer = orc.prepare_layer(W, Q, r, spec.G)
        y = orc.linear_deployed(inp["x"], layer)["y64"]
        return np.linalg.norm(y - ref) / np.linalg.norm(ref)

    K = spec.K
    e_rtn = err(np.eye(K), 0)
    Q = inp["Q"]
    # undo R: plain PCA basis ordering is recovered from the calibration second moment
    xc = synth.bf16_bits_to_f32(synth.make_tokens(spec, spec.calib_tokens, 1_000_003)).astype(np.float64)
    evals, evecs = np.linalg.eigh(xc.T @ xc)
    U = evecs[:, ::-1]
    e_pca = err(U, spec.r)
    e_full = err(Q, spec.r)
    assert e_full < e_pca < e_rtn
