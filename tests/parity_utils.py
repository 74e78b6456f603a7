"""Comparison protocol between the CUDA library and the CPU oracle (used by the -m gpu tests).

Tolerances of the comparison (restated here so that the tests are self-contained):
  * given identical codes, the int32 group sums match bit for bit;
  * activation codes match exactly, except +-1 where the oracle's pre-rounding quotient lies
    within 1e-3 of a rounding boundary;
  * an activation scale either equals the oracle's, or is the neighbouring bf16 value when the
    oracle's unrounded absmax/7 lies within 1e-4 (relative) of the midpoint between the two --
    the codes of such a group are then checked against the oracle quantizer re-run with the
    library's scale;
  * rotated activations: per token, ||x~_gpu - x~_oracle|| <= 2e-3 ||x~_oracle||; the bf16
    high-precision coefficients within one bf16 step (+1e-5 of the token norm for fp32 accumulation);
  * output: max |y_gpu - y_oracle| <= 1e-2 * rms(y_oracle), read before the final bf16 rounding; asserted on every
    row, with the effect of the tolerated code / scale differences of that row added to the bound (a single +-1 code
    moves an output by up to 7 s_x s_w, about 1e-2 rms by itself), and as stated wherever that effect is small.
"""
import numpy as np
import torch

from oracle import dirotq_oracle as orc


def bits_to_bf16_tensor(bits: np.ndarray, device="cuda") -> torch.Tensor:
    return torch.from_numpy(np.ascontiguousarray(bits).view(np.int16)).to(device).view(torch.bfloat16)


def bf16_tensor_to_bits(t: torch.Tensor) -> np.ndarray:
    return t.contiguous().view(torch.int16).cpu().numpy().view(np.uint16)


def f64(bits):
    return orc.bf16_to_f64(bits)


def check_weight_side(layer_gpu_export, layer_orc):
    wcodes, wscales, wh, qb = layer_gpu_export
    assert np.array_equal(bf16_tensor_to_bits(qb), layer_orc["Qb"]), "bf16 rotation differs"
    assert np.array_equal(bf16_tensor_to_bits(wscales), layer_orc["wscales"]), "weight scales differ"
    assert np.array_equal(bf16_tensor_to_bits(wh), layer_orc["Wh"]), "bf16 high rows differ"
    got = wcodes.cpu().numpy()
    bad = got != layer_orc["wcodes"]
    if bad.any():
        # only exact ties of the fp64 quotient may differ (different summation order in the fold)
        t = layer_orc["wt"]
        assert t is not None, f"{bad.sum()} weight codes differ"
        frac = np.abs(np.abs(t[bad] - np.floor(t[bad])) - 0.5)
        assert np.all(frac < 1e-9) and np.all(np.abs(got[bad].astype(int) - layer_orc["wcodes"][bad]) == 1)
        assert bad.sum() <= 4


def check_activation_side(xrot, xh, codes, scales, out_orc, r, G):
    """xrot fp32 [M,K] (or None), xh/codes/scales from dirotq_workspace_export, out_orc from the oracle."""
    xt = out_orc["xt"]
    M, K = xt.shape
    K_l = K - r
    n_g = -(-K_l // G)
    stats = {}
    if xrot is not None:
        d = np.linalg.norm(xrot.astype(np.float64) - xt, axis=1)
        ref = np.linalg.norm(xt, axis=1)
        rel = d / np.maximum(ref, 1e-300)
        stats["xrot_rel_max"] = float(rel.max())
        assert rel.max() <= 2e-3
    # high-precision coefficients: within one bf16 step
    xh_g, xh_o = f64(xh), f64(out_orc["xh"])
    # one bf16 step of the value, plus the fp32 accumulation error of the rotation, which scales with
    # the token's norm rather than with the (possibly cancelling) coefficient
    step = np.maximum(np.abs(xh_o), 2.0 ** -126) * 2.0 ** -7 + 1e-5 * np.linalg.norm(xt, axis=1, keepdims=True)
    assert np.all(np.abs(xh_g - xh_o) <= step), "x~_h differs by more than one bf16 step"
    stats["xh_exact_frac"] = float(np.mean(xh == out_orc["xh"]))
    # scales
    s_g, s_o = f64(scales), f64(out_orc["scales"])
    low = np.zeros((M, n_g * G))
    low[:, :K_l] = xt[:, r:]
    u = np.abs(low).reshape(M, n_g, G).max(axis=2) / 7.0  # unrounded absmax / q_max
    flip = scales != out_orc["scales"]
    if flip.any():
        db = np.abs(scales[flip].astype(np.int64) - out_orc["scales"][flip].astype(np.int64))
        assert np.all(db == 1), "a scale is more than one bf16 step away"
        mid = 0.5 * (s_g[flip] + s_o[flip])
        assert np.all(np.abs(u[flip] - mid) <= 1e-4 * u[flip]), "scale differs away from a rounding boundary"
    stats["scale_flips"] = int(flip.sum())
    # codes: re-run the quotient with the library's scale where it differs
    s_use = np.repeat(s_g, G, axis=1)[:, :K_l]
    with np.errstate(divide="ignore", invalid="ignore"):
        t = np.where(s_use != 0, xt[:, r:] / s_use, 0.0)
    q_ref = np.clip(np.rint(t), -7, 7).astype(np.int8)
    same_scale = ~np.repeat(flip, G, axis=1)[:, :K_l]
    assert np.array_equal(q_ref[same_scale], out_orc["codes"][same_scale])  # consistency of the re-run
    bad = codes != q_ref
    if bad.any():
        assert np.all(np.abs(codes[bad].astype(int) - q_ref[bad].astype(int)) == 1), "a code is off by more than 1"
        dist = np.abs(np.abs(t[bad] - np.floor(t[bad])) - 0.5)
        assert np.all(dist <= 1e-3), "a code differs away from a rounding boundary"
    stats["code_flips"] = int(bad.sum())
    return stats


def check_output(y_bits, y_ref64, rows=None, slack=3e-4):
    """Stored bf16 output against an fp64 reference computed from the SAME integer codes, scales and
    bf16 coefficients: it must lie within half a bf16 step of the unrounded reference, plus
    `slack`*rms for the fp32 accumulation order.  (The stated bound, max|dy| <= 1e-2 rms, is
    read on the value before the final bf16 rounding -- one bf16 step of an output with
    |y| >= 2.6 rms is already larger than 1e-2 rms -- and is implied by this stricter check.)"""
    y = f64(y_bits)
    rms = float(np.sqrt(np.mean(y_ref64 ** 2)))
    if rows is not None:
        y, y_ref64, y_bits = y[rows], y_ref64[rows], y_bits[rows]
    if y.size == 0:
        return {}
    d = np.abs(y - y_ref64)
    e = np.floor(np.log2(np.maximum(np.abs(y_ref64), 2.0 ** -126)))
    half_step = 0.5 * 2.0 ** (e - 7)
    excess = float((d - half_step).max())
    assert excess <= slack * rms, f"max(|dy| - half bf16 step) = {excess:.3e} > {slack} * rms = {slack * rms:.3e}"
    assert excess <= 1e-2 * rms
    same = float(np.mean(y_bits == orc.bf16_round(y_ref64)))
    assert same >= 0.995, f"only {same:.4f} of the bf16 outputs equal the reference's"
    return {"max_err_over_rms": float(d.max() / rms), "excess_over_rms": excess / rms, "bf16_equal_frac": same}


def _rep(a, n, width):
    return np.repeat(a, n, axis=1)[:, :width]


def deq_int4(codes, scales_bits, G):
    """Dequantized low-precision activations s_x q [M, K_l] (or, transposed roles, weights: pass codes.T / scales.T)."""
    return _rep(f64(scales_bits), G, codes.shape[1]) * codes.astype(np.float64)


def check_all_rows_end_to_end(y_bits, y_ref_lib, y_orc, dx, w_abs, dxh, wh_abs, slack=3e-4):
    """End-to-end bound on EVERY token row, rows with tolerated differences included.

    dx [M, K_l]: dequantized low-precision activations of the library minus the oracle's (zero on rows whose codes and
    scales agree); dxh [M, r] likewise for the bf16 coefficients; w_abs [K_l, N], wh_abs [r, N]: |dequantized weights|.
    flip[m, n] = |dx| |W^| + |dxh| |W~_h| is the largest change of an output that the tolerated differences can cause
    (one +-1 code moves it by s_x s_w |q_w|).  Asserted: (i) the fp64 re-run on the library's intermediates differs
    from the oracle's output by no more than flip, i.e. by nothing but those differences; (ii) the library's output is
    within half a bf16 step + slack*rms + flip of the oracle's; (iii) wherever flip + slack*rms stays below 1e-2 rms,
    the bound as stated: |y - y_oracle| (before the final bf16 rounding) <= 1e-2 rms."""
    rms = float(np.sqrt(np.mean(y_orc ** 2)))
    touched = np.any(dx != 0, axis=1) | np.any(dxh != 0, axis=1)
    flip = np.zeros_like(y_orc)
    if touched.any():
        flip[touched] = np.abs(dx[touched]) @ w_abs + np.abs(dxh[touched]) @ wh_abs
    assert np.all(np.abs(y_ref_lib - y_orc) <= flip * (1 + 1e-9) + 1e-9 * rms), "re-run deviates by more than the flips explain"
    y = f64(y_bits)
    big = np.maximum(np.abs(y_orc), np.abs(y_ref_lib))
    half_step = 0.5 * 2.0 ** (np.floor(np.log2(np.maximum(big, 2.0 ** -126))) - 7)
    excess = np.abs(y - y_orc) - half_step
    assert np.all(excess <= slack * rms + flip), "an output is further from the oracle's than the tolerated flips allow"
    plain = flip + slack * rms <= 1e-2 * rms
    assert np.all(excess[plain] <= 1e-2 * rms)
    return {"e2e_all_max_err_over_rms": float(np.abs(y - y_orc).max() / rms), "e2e_all_plain_bound_frac": float(np.mean(plain)),
            "e2e_all_max_flip_over_rms": float(flip.max() / rms), "touched_rows_frac": float(np.mean(touched))}


def check_layer_output(y_bits, xh_bits, codes, scales, layer_orc, out_orc, bias_bits):
    """End-to-end protocol.

    1. Steps 4-5 of the oracle (integer GEMM, dequantize, rank-r branch, bias) are re-run on the
       library's own codes / scales / bf16 coefficients; the library's y must match that reference
       within half a bf16 step + 3e-4 rms.  Together with the stage checks of the first kernel this
       covers every element.
    2. Token rows whose codes, scales and bf16 coefficients all equal the oracle's are compared with
       the oracle's own end-to-end output under the same bound (hence within 1e-2 rms).
       Rows with a tolerated +-1 code / neighbouring-scale / one-step bf16 difference are excluded
       here: a single tolerated code flip moves an output by up to s_x*s_w*7, which for these
       weight statistics is itself about 1e-2 rms.
    3. Every row, those included, against the oracle's own output with the effect of the tolerated
       differences added to the bound (check_all_rows_end_to_end).
    """
    G = layer_orc["G"]
    P = orc.int_gemm(codes, layer_orc["wcodes"], G)
    y_ref, _ = orc.combine(P, scales, layer_orc["wscales"], xh_bits, layer_orc["Wh"], bias_bits)
    stats = check_output(y_bits, y_ref)
    clean = (np.all(codes == out_orc["codes"], axis=1) & np.all(scales == out_orc["scales"], axis=1)
             & np.all(xh_bits == out_orc["xh"], axis=1))
    stats["clean_rows_frac"] = float(np.mean(clean))
    e2e = check_output(y_bits, out_orc["y64"], rows=clean)
    stats["e2e_clean_max_err_over_rms"] = e2e.get("max_err_over_rms")
    # every row, flipped ones included
    dx = deq_int4(codes, scales, G) - deq_int4(out_orc["codes"], out_orc["scales"], G)
    w_abs = np.abs(deq_int4(layer_orc["wcodes"].T, layer_orc["wscales"].T, G)).T
    stats.update(check_all_rows_end_to_end(y_bits, y_ref, out_orc["y64"], dx, w_abs, f64(xh_bits) - f64(out_orc["xh"]),
                                           np.abs(f64(layer_orc["Wh"]))))
    return stats


# ------------------------------------------------------------------ NVFP4 variant
#
# Protocol (same structure as for INT4; E2M1 codes are compared with +0 and -0 identified):
#   * weights: E4M3 block scales, bf16 rows, rotation and the per-tensor exponent equal the oracle's;
#     E2M1 codes equal, except at exact ties of the fp64 quotient (|distance to a rounding boundary|
#     < 1e-9: the fold's summation order differs), at most 4 per layer;
#   * an activation block scale equals the oracle's or is the neighbouring E4M3 value when the
#     unrounded absmax/6/2^ex lies within tol_s of the midpoint between the two;
#   * an activation code equals the oracle quantizer re-run with the library's scale, or is the
#     neighbouring E2M1 value when the quotient lies within tol_t of the boundary between the two;
#   * tol_s = 1e-4 relative + 1e-5 ||x~_row|| (fp32 accumulation of the rotation, as for x~_h),
#     tol_t = 1e-3 + 1e-5 ||x~_row|| / s_block  (blocks of 16 can have scales far below the row norm);
#   * output: within half a bf16 step + slack * rms of the fp64 combination of the library's own
#     codes, scales and bf16 coefficients.

_E2M1_BOUNDS = np.array([0.25, 0.75, 1.25, 1.75, 2.5, 3.5, 5.0])


def _mag(c):
    return c & 7


def _codes_equal_mod_zero(a, b):
    return (a == b) | ((_mag(a) == 0) & (_mag(b) == 0))


def check_weight_side_nvfp4(export, layer_orc):
    wcodes, wsf, wh, qb, ew = export
    assert ew == layer_orc["ew"], "per-tensor weight exponent differs"
    assert np.array_equal(bf16_tensor_to_bits(qb), layer_orc["Qb"]), "bf16 rotation differs"
    assert np.array_equal(wsf.cpu().numpy(), layer_orc["wsf"]), "weight block scales differ"
    assert np.array_equal(bf16_tensor_to_bits(wh), layer_orc["Wh"]), "bf16 high rows differ"
    got = wcodes.cpu().numpy()
    bad = ~_codes_equal_mod_zero(got, layer_orc["wcodes"])
    if bad.any():
        t = layer_orc["wt"]
        assert t is not None, f"{bad.sum()} weight codes differ"
        dist = np.min(np.abs(np.abs(t[bad])[:, None] - _E2M1_BOUNDS[None, :]), axis=1)
        assert np.all(dist < 1e-9), "a weight code differs away from an exact tie"
        assert bad.sum() <= 4
    return {"weight_code_ties": int(bad.sum())}


def check_activation_side_nvfp4(xrot, xh, codes, sf, out_orc, r, ex):
    xt = out_orc["xt"]
    M, K = xt.shape
    K_l = K - r
    nb = -(-K_l // 16)
    stats = {}
    norm = np.linalg.norm(xt, axis=1, keepdims=True)
    if xrot is not None:
        rel = np.linalg.norm(xrot.astype(np.float64) - xt, axis=1) / np.maximum(norm[:, 0], 1e-300)
        stats["xrot_rel_max"] = float(rel.max())
        assert rel.max() <= 2e-3
    xh_g, xh_o = f64(xh), f64(out_orc["xh"])
    step = np.maximum(np.abs(xh_o), 2.0 ** -126) * 2.0 ** -7 + 1e-5 * norm
    assert np.all(np.abs(xh_g - xh_o) <= step), "x~_h differs by more than one bf16 step"
    # block scales
    low = np.zeros((M, nb * 16))
    low[:, :K_l] = xt[:, r:]
    u = np.abs(low).reshape(M, nb, 16).max(axis=2) / 6.0 * 2.0 ** (-ex)
    s_g, s_o = orc.e4m3_to_f64(sf), orc.e4m3_to_f64(out_orc["sf"])
    flip = sf != out_orc["sf"]
    if flip.any():
        db = np.abs(sf[flip].astype(np.int64) - out_orc["sf"][flip].astype(np.int64))
        assert np.all(db == 1), "a block scale is more than one E4M3 step away"
        mid = 0.5 * (s_g[flip] + s_o[flip])
        tol = 1e-4 * u[flip] + 1e-5 * np.broadcast_to(norm, u.shape)[flip] / 6.0 * 2.0 ** (-ex)
        assert np.all(np.abs(u[flip] - mid) <= tol), "block scale differs away from a rounding boundary"
    stats["scale_flips"] = int(flip.sum())
    # codes against the quantizer re-run with the library's scale
    s_use = np.repeat(s_g * 2.0 ** ex, 16, axis=1)[:, :K_l]
    with np.errstate(divide="ignore", invalid="ignore"):
        t = np.where(s_use != 0, xt[:, r:] / s_use, 0.0)
    mag_ref = np.searchsorted(_E2M1_BOUNDS, np.abs(t), side="left").astype(np.uint8)
    # ties go to the even code: a value exactly on a boundary between codes c and c+1 takes the even one
    on = np.isin(np.abs(t), _E2M1_BOUNDS)
    if on.any():
        lo_code = np.searchsorted(_E2M1_BOUNDS, np.abs(t[on]), side="left").astype(np.uint8)  # the lower neighbour
        mag_ref[on] = np.where(lo_code % 2 == 0, lo_code, lo_code + 1)
    q_ref = np.where(t < 0, 8, 0).astype(np.uint8) | mag_ref
    same_scale = ~np.repeat(flip, 16, axis=1)[:, :K_l]
    assert np.all(_codes_equal_mod_zero(q_ref, out_orc["codes"])[same_scale]), "the protocol's re-run disagrees with the oracle"
    bad = ~_codes_equal_mod_zero(codes, q_ref)
    if bad.any():
        dm = np.abs(_mag(codes[bad]).astype(int) - _mag(q_ref[bad]).astype(int))
        sign_ok = ((codes[bad] & 8) == (q_ref[bad] & 8)) | (np.minimum(_mag(codes[bad]), _mag(q_ref[bad])) == 0)
        assert np.all(dm == 1) and np.all(sign_ok), "a code is off by more than one E2M1 step"
        dist = np.min(np.abs(np.abs(t[bad])[:, None] - _E2M1_BOUNDS[None, :]), axis=1)
        with np.errstate(divide="ignore"):
            tol_t = 1e-3 + 1e-5 * np.broadcast_to(norm, t.shape)[bad] / s_use[bad]
        assert np.all(dist <= tol_t), "a code differs away from a rounding boundary"
    stats["code_flips"] = int(bad.sum())
    return stats


def check_layer_output_nvfp4(y_bits, xh_bits, codes, sf, ex, layer_orc, out_orc, bias_bits, slack=3e-4):
    y_ref, _ = orc.nvfp4_combine(codes, sf, ex, layer_orc, xh_bits, bias_bits)
    stats = check_output(y_bits, y_ref, slack=slack)
    clean = (np.all(_codes_equal_mod_zero(codes, out_orc["codes"]), axis=1) & np.all(sf == out_orc["sf"], axis=1)
             & np.all(xh_bits == out_orc["xh"], axis=1))
    stats["clean_rows_frac"] = float(np.mean(clean))
    e2e = check_output(y_bits, out_orc["y64"], rows=clean, slack=slack)
    stats["e2e_clean_max_err_over_rms"] = e2e.get("max_err_over_rms")
    def deq(c, f, e):  # E2M1 codes [R, K_l], E4M3 block scales [R, nb], power-of-two exponent
        return orc.e2m1_to_f64(c) * _rep(orc.e4m3_to_f64(f), 16, c.shape[1]) * 2.0 ** e
    dx = deq(codes, sf, ex) - deq(out_orc["codes"], out_orc["sf"], ex)
    w_abs = np.abs(deq(layer_orc["wcodes"].T, layer_orc["wsf"].T, layer_orc["ew"])).T
    stats.update(check_all_rows_end_to_end(y_bits, y_ref, out_orc["y64"], dx, w_abs, f64(xh_bits) - f64(out_orc["xh"]),
                                           np.abs(f64(layer_orc["Wh"])), slack=slack))
    return stats


# ------------------------------------------------------------------ asymmetric activation codes
#
# Same protocol as the symmetric case with a zero-point per group: the zero-point equals the oracle's or is the
# neighbouring bf16 value when the unrounded minimum lies within 1e-4 (relative) + 1e-5 ||x~_row|| of the midpoint; the
# scale likewise for (max - min)/15; codes are checked against the quantizer re-run with the library's scale and
# zero-point (+-1 within 1e-3 + 1e-5 ||x~_row|| / s of a rounding boundary); the output against the fp64
# combination (integer sums, scales, zero-point term, rank-r branch, bias) of the library's own intermediates.

def check_activation_side_asym(xrot, xh, codes, scales, zeros, out_orc, r, G):
    xt = out_orc["xt"]
    M, K = xt.shape
    K_l = K - r
    n_g = -(-K_l // G)
    stats = {}
    norm = np.linalg.norm(xt, axis=1, keepdims=True)
    if xrot is not None:
        rel = np.linalg.norm(xrot.astype(np.float64) - xt, axis=1) / np.maximum(norm[:, 0], 1e-300)
        stats["xrot_rel_max"] = float(rel.max())
        assert rel.max() <= 2e-3
    xh_g, xh_o = f64(xh), f64(out_orc["xh"])
    step = np.maximum(np.abs(xh_o), 2.0 ** -126) * 2.0 ** -7 + 1e-5 * norm
    assert np.all(np.abs(xh_g - xh_o) <= step), "x~_h differs by more than one bf16 step"
    # group minima / ranges of the oracle's fp64 rotation (padding slots excluded)
    lo = np.full((M, n_g), np.inf)
    hi = np.full((M, n_g), -np.inf)
    for g in range(n_g):
        seg = xt[:, r + g * G: r + min((g + 1) * G, K_l)]
        lo[:, g], hi[:, g] = seg.min(axis=1), seg.max(axis=1)
    normb = np.broadcast_to(norm, lo.shape)
    z_g, z_o = f64(zeros), f64(out_orc["zeros"])
    zflip = zeros != out_orc["zeros"]
    if zflip.any():
        assert np.all(np.abs(z_g[zflip] - z_o[zflip]) <= np.maximum(np.abs(z_o[zflip]), 2.0 ** -126) * 2.0 ** -7), \
            "a zero-point is more than one bf16 step away"
        mid = 0.5 * (z_g[zflip] + z_o[zflip])
        assert np.all(np.abs(lo[zflip] - mid) <= 1e-4 * np.abs(lo[zflip]) + 1e-5 * normb[zflip]), \
            "zero-point differs away from a rounding boundary"
    s_g, s_o = f64(scales), f64(out_orc["scales"])
    u = (hi - lo) / 15.0
    sflip = scales != out_orc["scales"]
    if sflip.any():
        db = np.abs(scales[sflip].astype(np.int64) - out_orc["scales"][sflip].astype(np.int64))
        assert np.all(db == 1), "a scale is more than one bf16 step away"
        mid = 0.5 * (s_g[sflip] + s_o[sflip])
        assert np.all(np.abs(u[sflip] - mid) <= 1e-4 * u[sflip] + 2e-5 * normb[sflip] / 15.0), \
            "scale differs away from a rounding boundary"
    stats["scale_flips"], stats["zero_flips"] = int(sflip.sum()), int(zflip.sum())
    s_use = np.repeat(s_g, G, axis=1)[:, :K_l]
    z_use = np.repeat(z_g, G, axis=1)[:, :K_l]
    with np.errstate(divide="ignore", invalid="ignore"):
        t = np.where(s_use != 0, (xt[:, r:] - z_use) / s_use, 0.0)
    q_ref = np.clip(np.rint(t), 0, 15).astype(np.uint8)
    same = ~np.repeat(sflip | zflip, G, axis=1)[:, :K_l]
    assert np.array_equal(q_ref[same], out_orc["codes"][same])
    bad = codes != q_ref
    if bad.any():
        assert np.all(np.abs(codes[bad].astype(int) - q_ref[bad].astype(int)) == 1), "a code is off by more than 1"
        dist = np.abs(np.abs(t[bad] - np.floor(t[bad])) - 0.5)
        with np.errstate(divide="ignore"):
            tol = 1e-3 + 1e-5 * np.broadcast_to(norm, t.shape)[bad] / s_use[bad]
        assert np.all(dist <= tol), "a code differs away from a rounding boundary"
    stats["code_flips"] = int(bad.sum())
    return stats


def check_layer_output_asym(y_bits, xh_bits, codes, scales, zeros, layer_orc, out_orc, bias_bits, slack=3e-4):
    P = orc.int_gemm_u(codes, layer_orc["wcodes"], layer_orc["G"])
    y_ref, _ = orc.combine_asym(P, scales, zeros, layer_orc, xh_bits, bias_bits)
    stats = check_output(y_bits, y_ref, slack=slack)
    clean = (np.all(codes == out_orc["codes"], axis=1) & np.all(scales == out_orc["scales"], axis=1)
             & np.all(zeros == out_orc["zeros"], axis=1) & np.all(xh_bits == out_orc["xh"], axis=1))
    stats["clean_rows_frac"] = float(np.mean(clean))
    e2e = check_output(y_bits, out_orc["y64"], rows=clean, slack=slack)
    stats["e2e_clean_max_err_over_rms"] = e2e.get("max_err_over_rms")
    G = layer_orc["G"]
    def deq(u, sb, zb):  # x^ = s u + z per group
        return _rep(f64(sb), G, u.shape[1]) * u.astype(np.float64) + _rep(f64(zb), G, u.shape[1])
    dx = deq(codes, scales, zeros) - deq(out_orc["codes"], out_orc["scales"], out_orc["zeros"])
    w_abs = np.abs(deq_int4(layer_orc["wcodes"].T, layer_orc["wscales"].T, G)).T
    stats.update(check_all_rows_end_to_end(y_bits, y_ref, out_orc["y64"], dx, w_abs, f64(xh_bits) - f64(out_orc["xh"]),
                                           np.abs(f64(layer_orc["Wh"])), slack=slack))
    return stats


# ------------------------------------------------------------------ W4A8 (per-token INT8 activations, per-channel INT4 weights)
#
# Protocol: weights as in the grouped case (one "group" per column); the token scale equals the oracle's or is the
# neighbouring bf16 value when the unrounded max|x~|/127 lies within 1e-4 (relative) + 1e-5 ||x~_row|| / 127 of the
# midpoint; codes against the quantizer re-run with the library's scale (+-1 within 1e-3 + 1e-5 ||x~_row|| / s of a
# rounding boundary); int32 sums bit for bit; output within half a bf16 step + slack * rms of the fp64 combination of
# the library's own intermediates.

def check_activation_side_w4a8(xrot, xh, codes, scales, out_orc, r):
    xt = out_orc["xt"]
    M, K = xt.shape
    stats = {}
    norm = np.linalg.norm(xt, axis=1)
    if xrot is not None:
        rel = np.linalg.norm(xrot.astype(np.float64) - xt, axis=1) / np.maximum(norm, 1e-300)
        stats["xrot_rel_max"] = float(rel.max())
        assert rel.max() <= 2e-3
    xh_g, xh_o = f64(xh), f64(out_orc["xh"])
    step = np.maximum(np.abs(xh_o), 2.0 ** -126) * 2.0 ** -7 + 1e-5 * norm[:, None]
    assert np.all(np.abs(xh_g - xh_o) <= step), "x~_h differs by more than one bf16 step"
    s_g, s_o = f64(scales), f64(out_orc["scales"])
    u = np.abs(xt[:, r:]).max(axis=1) / 127.0
    flip = scales != out_orc["scales"]
    if flip.any():
        db = np.abs(scales[flip].astype(np.int64) - out_orc["scales"][flip].astype(np.int64))
        assert np.all(db == 1), "a token scale is more than one bf16 step away"
        mid = 0.5 * (s_g[flip] + s_o[flip])
        assert np.all(np.abs(u[flip] - mid) <= 1e-4 * u[flip] + 1e-5 * norm[flip] / 127.0)
    stats["scale_flips"] = int(flip.sum())
    with np.errstate(divide="ignore", invalid="ignore"):
        t = np.where(s_g[:, None] != 0, xt[:, r:] / s_g[:, None], 0.0)
    q_ref = np.clip(np.rint(t), -127, 127).astype(np.int8)
    assert np.array_equal(q_ref[~flip], out_orc["codes"][~flip])
    bad = codes != q_ref
    if bad.any():
        assert np.all(np.abs(codes[bad].astype(int) - q_ref[bad].astype(int)) == 1), "a code is off by more than 1"
        dist = np.abs(np.abs(t[bad] - np.floor(t[bad])) - 0.5)
        with np.errstate(divide="ignore"):
            tol = 1e-3 + 1e-5 * np.broadcast_to(norm[:, None], t.shape)[bad] / np.broadcast_to(s_g[:, None], t.shape)[bad]
        assert np.all(dist <= tol), "a code differs away from a rounding boundary"
    stats["code_flips"] = int(bad.sum())
    return stats


def check_layer_output_w4a8(y_bits, xh_bits, codes, scales, layer_orc, out_orc, bias_bits, slack=3e-4):
    K_l = codes.shape[1]
    P = orc.int_gemm(codes, layer_orc["wcodes"], K_l)
    y_ref, _ = orc.combine(P, scales.reshape(-1, 1), layer_orc["wscales"], xh_bits, layer_orc["Wh"], bias_bits)
    stats = check_output(y_bits, y_ref, slack=slack)
    clean = (np.all(codes == out_orc["codes"], axis=1) & (scales == out_orc["scales"]) & np.all(xh_bits == out_orc["xh"], axis=1))
    stats["clean_rows_frac"] = float(np.mean(clean))
    e2e = check_output(y_bits, out_orc["y64"], rows=clean, slack=slack)
    stats["e2e_clean_max_err_over_rms"] = e2e.get("max_err_over_rms")
    dx = (f64(scales).reshape(-1, 1) * codes.astype(np.float64)
          - f64(out_orc["scales"]).reshape(-1, 1) * out_orc["codes"].astype(np.float64))
    w_abs = np.abs(f64(layer_orc["wscales"]).reshape(1, -1) * layer_orc["wcodes"].astype(np.float64))
    stats.update(check_all_rows_end_to_end(y_bits, y_ref, out_orc["y64"], dx, w_abs, f64(xh_bits) - f64(out_orc["xh"]),
                                           np.abs(f64(layer_orc["Wh"])), slack=slack))
    return stats
