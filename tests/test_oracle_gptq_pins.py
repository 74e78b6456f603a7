"""Pins of the oracle's GPTQ rounding of the residual weight (Sec. 4.1, App. F.1: damping 0.01, block 128).

The checks use only what the method fixes: with an uncorrelated Hessian no error is fed forward, so the codes are
round-to-nearest; once every earlier row is fixed, the last row of a problem must be the best of its 15 levels for
the damped objective tr(E^T H E) (brute force); the blocked form equals the row-by-row form; and on correlated
calibration tokens the activation-weighted error falls below that of round-to-nearest.
"""
import numpy as np

from oracle import dirotq_oracle as orc


def _bf(bits):
    return orc.bf16_to_f64(np.asarray(bits, dtype=np.uint16))


def _objective(W, codes, scales, H, G):
    s = np.repeat(_bf(scales), G, axis=0)[: W.shape[0]]
    E = W - s * codes
    return float(np.trace(E.T @ H @ E))


def _correlated_tokens(rng, T, K_l, rank=6, noise=0.15):
    # strongly correlated columns: a few shared factors plus a little independent noise
    return rng.standard_normal((T, rank)) @ rng.standard_normal((rank, K_l)) + noise * rng.standard_normal((T, K_l))


def test_uncorrelated_hessian_reduces_to_round_to_nearest():
    rng = np.random.default_rng(1)
    K_l, N, G = 200, 24, 64                      # ragged last group of 8 rows
    W = rng.standard_normal((K_l, N)) * 0.02
    rtn = orc.prepare_weights(W, 0, G)
    for H in (3.7 * np.eye(K_l), np.diag(rng.uniform(0.5, 4.0, K_l))):
        codes, scales = orc.gptq_quantize(W, H, G)
        assert np.array_equal(codes, rtn["wcodes"]) and np.array_equal(scales, rtn["wscales"])


def test_first_group_scales_and_first_row_codes_are_round_to_nearest():
    # nothing has been fed forward when the first group starts, and the first row is rounded as it stands
    rng = np.random.default_rng(2)
    K_l, N, G = 128, 16, 64
    W = rng.standard_normal((K_l, N)) * 0.02
    X = _correlated_tokens(rng, 400, K_l)
    codes, scales = orc.gptq_quantize(W, X.T @ X, G)
    rtn = orc.prepare_weights(W, 0, G)
    assert np.array_equal(scales[0], rtn["wscales"][0])
    assert np.array_equal(codes[0], rtn["wcodes"][0])
    assert not np.array_equal(codes, rtn["wcodes"])      # the feedback does change later rows


def test_last_row_is_the_best_level_given_the_earlier_rows():
    rng = np.random.default_rng(3)
    damp = 0.01
    for trial in range(40):
        K_l = int(rng.integers(2, 7))
        N = 5
        W = rng.standard_normal((K_l, N))
        X = _correlated_tokens(rng, 50, K_l, rank=2, noise=0.3)
        H = X.T @ X
        codes, scales = orc.gptq_quantize(W, H, G=8, damp=damp, block=8)
        Hd = H + damp * np.mean(np.diag(H)) * np.eye(K_l)
        s = _bf(scales)[0]
        for n in range(N):
            best, best_q = None, None
            for q in range(-7, 8):
                c = codes[:, n].astype(np.float64).copy()
                c[-1] = q
                e = W[:, n] - s[n] * c
                val = e @ Hd @ e
                if best is None or val < best:
                    best, best_q = val, q
            assert int(codes[-1, n]) == best_q, (trial, n)


def test_two_rows_closed_form():
    # K_l = 2: the second row is rounded after adding (H01/H11) * (error of the first row), H the damped Hessian
    rng = np.random.default_rng(4)
    for _ in range(50):
        W = rng.standard_normal((2, 3))
        A = rng.standard_normal((2, 2))
        H = A @ A.T + 0.1 * np.eye(2)
        codes, scales = orc.gptq_quantize(W, H, G=2, damp=0.0, block=2)
        s = _bf(scales)[0]
        e0 = W[0] - s * codes[0]
        target = W[1] + (H[0, 1] / H[1, 1]) * e0
        expect = np.clip(np.rint(target / s), -7, 7)
        near_tie = np.abs(np.abs(target / s - np.floor(target / s)) - 0.5) < 1e-9
        assert np.array_equal(codes[1][~near_tie], expect[~near_tie].astype(np.int8))


def test_blocked_form_equals_row_by_row_form():
    rng = np.random.default_rng(5)
    K_l, N, G = 320, 12, 64
    W = rng.standard_normal((K_l, N)) * 0.02
    X = _correlated_tokens(rng, 600, K_l, rank=12)
    H = X.T @ X
    c1, s1 = orc.gptq_quantize(W, H, G, block=128, lazy=True)
    c2, s2 = orc.gptq_quantize(W, H, G, block=128, lazy=False)
    c3, s3 = orc.gptq_quantize(W, H, G, block=64, lazy=True)
    # identical up to the rare code that sits on a rounding boundary to within fp64 rounding order
    assert np.mean(c1 != c2) < 1e-3 and np.mean(c1 != c3) < 1e-3
    assert np.mean(s1 != s2) < 1e-3 and np.mean(s1 != s3) < 1e-3


def test_activation_weighted_error_beats_round_to_nearest():
    rng = np.random.default_rng(6)
    K_l, N, G = 256, 32, 64
    W = rng.standard_normal((K_l, N)) * 0.02
    X = _correlated_tokens(rng, 1024, K_l, rank=8)
    H = X.T @ X
    codes, scales = orc.gptq_quantize(W, H, G)
    rtn = orc.prepare_weights(W, 0, G)
    e_gptq = _objective(W, codes, scales, H, G)
    e_rtn = _objective(W, rtn["wcodes"], rtn["wscales"], H, G)
    assert e_gptq < 0.5 * e_rtn
    # and this is the output error on the calibration tokens themselves: ||X W - X W^||_F^2
    s = np.repeat(_bf(scales), G, axis=0)
    assert np.isclose(e_gptq, np.sum((X @ W - X @ (s * codes)) ** 2), rtol=1e-9)
    assert np.abs(codes).max() <= 7


def test_dead_column_gets_zero_codes():
    rng = np.random.default_rng(7)
    K_l, N, G = 64, 4, 64
    W = rng.standard_normal((K_l, N))
    X = rng.standard_normal((100, K_l))
    X[:, 10] = 0.0
    codes, _ = orc.gptq_quantize(W, X.T @ X, G)
    assert not codes[10].any()


def test_hessian_and_layer_driver():
    rng = np.random.default_rng(8)
    X = rng.standard_normal((30, 17))
    assert np.allclose(orc.gptq_hessian(X), X.T @ X, rtol=1e-12, atol=1e-12)
    K, N, r, G = 128, 16, 32, 32
    Q, _ = np.linalg.qr(rng.standard_normal((K, K)))
    W = rng.standard_normal((K, N)) * 0.02
    calib = orc.bf16_round(_correlated_tokens(rng, 256, K, rank=5))
    lay = orc.prepare_layer_gptq(W, Q, calib, r, G)
    ref = orc.prepare_layer(W, Q, r, G)
    assert np.array_equal(lay["Wh"], ref["Wh"]) and np.array_equal(lay["Qb"], ref["Qb"])
    assert np.array_equal(lay["wcodes_rtn"], ref["wcodes"])
    xt = orc.rotate(calib, lay["Qb"])[:, r:]
    assert np.allclose(lay["H"], xt.T @ xt, rtol=1e-10, atol=1e-10)
    e_g = _objective(lay["Wt_low"], lay["wcodes"], lay["wscales"], lay["H"], G)
    e_r = _objective(lay["Wt_low"], ref["wcodes"], ref["wscales"], lay["H"], G)
    assert e_g < e_r
