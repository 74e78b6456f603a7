"""Pins of the oracle's projection form (only U_h applied densely, the residual rotated by a block Hadamard): the
reference for the cheaper first stage.  What the construction fixes: the Hadamard blocks
are orthonormal; the decomposition x H+- = sqrt(G) x~_l + x~_h V is exact for ANY U_h and any rounding of V because
x~_l is defined as that difference, so without quantization the layer is x W; up to the rounding of V the low-precision
coefficients are the block-Hadamard transform of the rounded projection's residual; the integer path equals
dequantize-then-multiply; with no
projection it reduces to group-wise rounding of the Hadamard-rotated operands; and on activations with outlier
directions the projection is what keeps the error down."""
import numpy as np
import pytest

from oracle import dirotq_oracle as orc
from paper_2605_16732_b200 import synth


def _bf(bits):
    return orc.bf16_to_f64(np.asarray(bits, dtype=np.uint16))


def test_hadamard_blocks_are_orthonormal_and_the_two_transforms_cancel():
    for n in (1, 2, 8, 64, 128):
        H = orc.hadamard(n)
        assert np.allclose(H @ H.T, np.eye(n), atol=1e-12) and np.array_equal(H, H.T)
        assert set(np.unique(np.round(np.abs(H) * np.sqrt(n), 12))) == {1.0}
    rng = np.random.default_rng(0)
    A, B = rng.standard_normal((7, 192)), rng.standard_normal((192, 5))
    assert np.allclose(orc.block_hadamard_cols(A, 64) @ orc.block_hadamard_rows(B, 64), A @ B, atol=1e-10)
    # a constant group has all its energy in the block's first coefficient
    c = orc.block_hadamard_cols(np.full((1, 64), 3.0), 64)
    assert np.isclose(c[0, 0], 3.0 * 8.0) and np.allclose(c[0, 1:], 0.0, atol=1e-12)
    # the +-1 form: entry (i, j) is (-1)^popcount(i & j); the block product is that matrix applied group by group
    for n in (4, 64, 128):
        S = orc.hadamard_signs(n)
        assert all(S[i, j] == (-1.0) ** bin(i & j).count("1") for i in range(n) for j in range(0, n, 7))
        assert np.array_equal(S @ S.T, n * np.eye(n))
    A = np.round(rng.standard_normal((3, 128)) * 64.0)
    ref = np.array([[sum(A[m, 64 * b + j] * (-1.0) ** bin(j & c).count("1") for j in range(64)) for b in range(2) for c in range(64)]
                    for m in range(3)])
    assert np.array_equal(orc.block_signs_cols(A, 64), ref)


@pytest.mark.parametrize("G", [64, 128])
def test_decomposition_is_exact_for_any_projection(G):
    rng = np.random.default_rng(1)
    K, N, r, M = 256, 48, 32, 33
    W = rng.standard_normal((K, N)) * 0.02
    x_bits = orc.bf16_round(rng.standard_normal((M, K)) * rng.choice([0.1, 1.0, 20.0], size=(1, K)))
    x = _bf(x_bits)
    for Uh in (np.linalg.qr(rng.standard_normal((K, r)))[0], rng.standard_normal((K, r)) * 0.3):   # orthonormal or not
        lay = orc.prepare_layer_ph(W, Uh, G)
        out = orc.linear_deployed_ph(x_bits, lay)
        Uhb, V, xh = _bf(lay["Uhb"]), _bf(lay["V"]), _bf(out["xh"])
        S = np.kron(np.eye(K // G), orc.hadamard_signs(G))             # H+- written out
        assert np.array_equal(lay["Uhb"], orc.bf16_round(Uh)) and np.array_equal(lay["V"], orc.bf16_round(Uhb.T @ S))
        assert np.array_equal(out["xh"], orc.bf16_round(x @ Uhb))
        assert np.allclose(np.sqrt(G) * out["xl"] + xh @ V, x @ S, rtol=0, atol=1e-12 * np.abs(x @ S).max())
        # unquantized: x~_h ((V H+-^T / G) W) + x~_l (H^T W) = x W
        back = V @ S.T / G
        ideal = xh @ (back @ W) + out["xl"] @ orc.block_hadamard_rows(W, G)
        assert np.allclose(ideal, x @ W, rtol=1e-10, atol=1e-10)
        # up to the rounding of V (2^-9 relative per entry), x~_l is the transformed residual of the rounded projection
        plain = orc.block_hadamard_cols(x - xh @ Uhb.T, G)
        bound = (np.abs(xh) @ (np.abs(V) * 2.0 ** -9)) / np.sqrt(G)
        assert np.all(np.abs(out["xl"] - plain) <= bound + 1e-12) and np.abs(out["xl"] - plain).max() > 0
        # the high rows of the prepared weight are bf16((V H+-^T / G) W), the low rows the K transformed rows
        assert np.array_equal(lay["Wh"], orc.bf16_round(back @ W))
        assert lay["wcodes"].shape == (K, N) and out["codes"].shape == (M, K)


def test_integer_path_equals_dequantize_then_multiply():
    spec = synth.LayerSpec(K=256, N=80, r=32, G=64, model=synth.PIXART, seed=3, calib_tokens=1024)
    inp = synth.make_layer_inputs(spec, 24, with_bias=True)
    Q = np.asarray(inp["Q"], dtype=np.float64)
    lay = orc.prepare_layer_ph(inp["W"], Q[:, :spec.r], spec.G)
    out = orc.linear_deployed_ph(inp["x"], lay, bias=inp["bias"])
    sx = np.repeat(_bf(out["scales"]), spec.G, axis=1)
    sw = np.repeat(_bf(lay["wscales"]), spec.G, axis=0)
    ref = (sx * out["codes"]) @ (sw * lay["wcodes"]) + _bf(out["xh"]) @ _bf(lay["Wh"]) + _bf(inp["bias"])[None, :]
    assert np.allclose(out["y64"], ref, rtol=1e-12, atol=1e-12)
    assert np.array_equal(out["y"], orc.bf16_round(out["y64"]))


def test_without_projection_it_is_group_rounding_of_the_hadamard_rotated_operands():
    rng = np.random.default_rng(4)
    K, N, G, M = 128, 16, 64, 9
    W = rng.standard_normal((K, N)) * 0.02
    x_bits = orc.bf16_round(rng.standard_normal((M, K)))
    lay = orc.prepare_layer_ph(W, np.zeros((K, 16)), G)          # sixteen null directions: x~_h = 0, d = x
    out = orc.linear_deployed_ph(x_bits, lay)
    assert not out["xh"].any() and not lay["V"].any()
    xr = orc.block_hadamard_cols(_bf(x_bits), G)
    for m in range(M):
        for g in range(K // G):
            sb, codes, _ = orc.quantize_group(xr[m, g * G:(g + 1) * G])
            assert sb == out["scales"][m, g] and np.array_equal(codes, out["codes"][m, g * G:(g + 1) * G])
    rtn = orc.prepare_weights(orc.block_hadamard_rows(W, G), 0, G)
    assert np.array_equal(lay["wcodes"], rtn["wcodes"]) and np.array_equal(lay["wscales"], rtn["wscales"])


def test_error_matches_the_dense_rotation_and_the_projection_is_what_removes_the_outliers():
    spec = synth.LayerSpec(K=512, N=96, r=32, G=64, model=synth.PIXART, seed=5, calib_tokens=2048)
    inp = synth.make_layer_inputs(spec, 160, with_bias=False)
    Q = np.asarray(inp["Q"], dtype=np.float64)
    x = _bf(inp["x"])
    ideal = x @ np.asarray(inp["W"], dtype=np.float64)

    def err(y):
        return float(np.sqrt(np.mean((y - ideal) ** 2) / np.mean(ideal ** 2)))

    e_paper = err(orc.linear_deployed(inp["x"], orc.prepare_layer(inp["W"], inp["Q"], spec.r, spec.G))["y64"])
    e_proj = err(orc.linear_deployed_ph(inp["x"], orc.prepare_layer_ph(inp["W"], Q[:, :spec.r], spec.G))["y64"])
    e_none = err(orc.linear_deployed_ph(inp["x"], orc.prepare_layer_ph(inp["W"], np.zeros((spec.K, spec.r)), spec.G))["y64"])
    print(e_paper, e_proj, e_none)
    assert 0.8 < e_proj / e_paper < 1.25          # same error as the paper's dense rotation on these activations
    assert e_none > 3.0 * e_proj                  # a Hadamard alone does not remove the planted outlier directions


def test_nvfp4_projection_form_shares_the_decomposition_and_matches_the_dense_form():
    spec = synth.LayerSpec(K=256, N=64, r=32, G=64, model=synth.PIXART, seed=6, calib_tokens=1024)
    inp = synth.make_layer_inputs(spec, 48, with_bias=True)
    Q = np.asarray(inp["Q"], dtype=np.float64)
    x = _bf(inp["x"])
    lay = orc.nvfp4_prepare_layer_ph(inp["W"], np.ascontiguousarray(Q[:, :spec.r]), want_t=True)
    xh_bits, xl = orc.nvfp4_residual(inp["x"], lay)
    # same exact decomposition as the INT4 projection form, Hadamard blocks of 64
    S = np.kron(np.eye(spec.K // 64), orc.hadamard_signs(64))
    assert np.allclose(8.0 * xl + _bf(xh_bits) @ _bf(lay["V"]), x @ S, rtol=0, atol=1e-12 * np.abs(x @ S).max())
    ref = orc.prepare_layer_ph(inp["W"], np.ascontiguousarray(Q[:, :spec.r]), 64)
    assert np.array_equal(lay["V"], ref["V"]) and np.array_equal(lay["Uhb"], ref["Uhb"]) and np.array_equal(lay["Wh"], ref["Wh"])
    ex = orc.nvfp4_global_exponent(float(np.abs(xl).max()))
    out = orc.nvfp4_linear_deployed_ph(inp["x"], lay, ex, bias=inp["bias"])
    # block-scaled product = dequantize-then-multiply of the codes it returns
    mag = np.array([0, 0.5, 1, 1.5, 2, 3, 4, 6], dtype=np.float64)
    deq = lambda c: np.where(c & 8, -1.0, 1.0) * mag[c & 7]
    xs = np.repeat(orc.e4m3_to_f64(out["sf"]), 16, axis=1) * 2.0 ** ex * deq(out["codes"])
    ws = np.repeat(orc.e4m3_to_f64(lay["wsf"]), 16, axis=0) * 2.0 ** lay["ew"] * deq(lay["wcodes"])
    ref = xs @ ws + _bf(out["xh"]) @ _bf(lay["Wh"]) + _bf(inp["bias"])[None, :]
    assert np.allclose(out["y64"], ref, rtol=1e-9, atol=1e-9)
    # and its error is that of the dense NVFP4 form on these activations
    ideal = x @ np.asarray(inp["W"], dtype=np.float64) + _bf(inp["bias"])[None, :]
    lo = orc.nvfp4_prepare_layer(inp["W"], inp["Q"], spec.r)
    ex2 = orc.nvfp4_global_exponent(float(np.abs(orc.rotate(inp["x"], lo["Qb"])[:, spec.r:]).max()))
    dense = orc.nvfp4_linear_deployed(inp["x"], lo, ex2, bias=inp["bias"])
    e = lambda y: float(np.sqrt(np.mean((y - ideal) ** 2) / np.mean(ideal ** 2)))
    assert 0.8 < e(out["y64"]) / e(dense["y64"]) < 1.25


@pytest.mark.parametrize("n_outlier,magnitude,spread", [(0, 1.0, 0.0), (48, 30.0, 0.0), (48, 30.0, 1.0), (96, 100.0, 1.0)])
def test_residuals_that_are_not_white(n_outlier, magnitude, spread):
    """The synthetic layer generator leaves a white residual.  Here the residual is far from white: log-normal channel
    scales and more axis-aligned outlier channels than the r directions U_h can take (PCA of calibration tokens picks
    the largest).  A per-group Hadamard spreads a leftover outlier over its 64 neighbours only, the dense random
    rotation over all K - r coefficients; with one scale per group of 64 the output errors come out alike."""
    K, N, r, G, T, M = 512, 96, 32, 64, 2048, 160
    g = np.random.default_rng(40 + n_outlier)
    sig = np.exp(spread * g.standard_normal(K))
    idx = g.choice(K, n_outlier, replace=False)
    sig[idx] *= magnitude * g.uniform(0.3, 1.0, n_outlier)
    calib = np.random.default_rng(1).standard_normal((T, K)) * sig
    _, V = np.linalg.eigh(calib.T @ calib)
    V = V[:, ::-1]                                                  # PCA directions, largest first (Sec. 4.1)
    R, _ = np.linalg.qr(g.standard_normal((K - r, K - r)))         # the random rotation of the residual (Eq. 5)
    Q = np.concatenate([V[:, :r], V[:, r:] @ R], axis=1)
    W = 0.02 * g.standard_normal((K, N))
    xb = orc.bf16_round(np.random.default_rng(2).standard_normal((M, K)) * sig)
    ideal = _bf(xb) @ W

    def err(y):
        return float(np.sqrt(np.mean((y - ideal) ** 2) / np.mean(ideal ** 2)))

    e_paper = err(orc.linear_deployed(xb, orc.prepare_layer(W, Q, r, G))["y64"])
    e_proj = err(orc.linear_deployed_ph(xb, orc.prepare_layer_ph(W, np.ascontiguousarray(Q[:, :r]), G))["y64"])
    print(n_outlier, magnitude, spread, e_paper, e_proj)
    assert e_proj < 1.15 * e_paper
