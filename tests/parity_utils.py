"""Comparison protocol between the CUDA library and the CPU oracle (used by the -m gpu tests).

Tolerances (from the benchmark spec, restated here so that the tests are self-contained):
  * given identical codes, the int32 group sums match bit for bit;
  * activation codes match exactly, except +-1 where the oracle's pre-rounding quotient lies
    within 1e-3 of a rounding boundary;
  * an activation scale either equals the oracle's, or is the neighbouring bf16 value when the
    oracle's unrounded absmax/7 lies within 1e-4 (relative) of the midpoint between the two --
    the codes of such a group are then checked against the oracle quantizer re-run with the
    library's scale;
  * rotated activations: per token, ||x~_gpu - x~_oracle|| <= 2e-3 ||x~_oracle||; the bf16
    high-precision coefficients within one bf16 step;
  * output: max |y_gpu - y_oracle| <= 1e-2 * rms(y_oracle).
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
    step = np.maximum(np.abs(xh_o), 2.0 ** -126) * 2.0 ** -7
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


def check_output(y_bits, y_oracle64):
    y = f64(y_bits)
    rms = float(np.sqrt(np.mean(y_oracle64 ** 2)))
    err = float(np.abs(y - y_oracle64).max())
    assert err <= 1e-2 * rms, f"max |dy| = {err:.3e} > 1e-2 * rms = {1e-2 * rms:.3e}"
    return err / rms
