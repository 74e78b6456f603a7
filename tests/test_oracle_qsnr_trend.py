"""Activation QSNR of the rotated, split and quantized representation, computed by the oracle on the synthetic
activation model.  What the paper reports and these inputs reproduce in kind (not in value): rotating into the
calibrated basis and keeping the leading coefficients in 16 bits lifts the QSNR far above plain per-group
round-to-nearest (its per-block figures show 5-10 dB on real activations), and the gain from a larger 16-bit
subspace is steep until that subspace covers the dominant directions and nearly flat beyond (Sec. 5, rank ablation:
less than 0.5 dB per further 5 % of the coefficients)."""
import numpy as np

from oracle import dirotq_oracle as orc
from paper_2605_16732_b200 import synth


def _qsnr_db(x, xhat):
    return 10.0 * np.log10(np.sum(x ** 2) / np.sum((x - xhat) ** 2))


def _dequantized(sq, G, width):
    s = np.repeat(orc.bf16_to_f64(sq["scales"]), G, axis=1)[:, :width]
    return s * sq["codes"]


def _qsnr(K, model, r, G=64, T=384):
    spec = synth.LayerSpec(K=K, N=64, r=max(r, 16), G=G, model=model, seed=5, calib_tokens=2048)
    x = orc.bf16_to_f64(synth.make_tokens(spec, T, batch_seed=3))
    if r == 0:      # no rotation, nothing kept in 16 bits: Eq. 1 applied to the activations as they are
        return _qsnr_db(x, _dequantized(orc.split_quantize(x, 0, G, want_t=False), G, K))
    Q = np.asarray(synth.make_rotation(spec), dtype=np.float64)
    sq = orc.split_quantize(x @ Q, r, G, want_t=False)
    xt_hat = np.concatenate([orc.bf16_to_f64(sq["xh"]), _dequantized(sq, G, K - r)], axis=1)
    return _qsnr_db(x, xt_hat @ Q.T)      # Q is orthogonal: the error norm is the same in either basis


def test_rotation_and_split_beat_plain_rounding_and_saturate_with_rank():
    # PixArt-like generator: 8 outlier channels + a rank-16 shared component = 24 dominant directions
    ranks = [0, 16, 32, 64, 128]      # 0, 3, 6, 12.5 and 25 % of K = 512
    q = [_qsnr(512, synth.PIXART, r) for r in ranks]
    print(dict(zip(ranks, np.round(q, 2))))
    assert q[2] - q[0] > 10.0                      # far above plain round-to-nearest once the structure is covered
    assert all(b >= a - 0.05 for a, b in zip(q[1:], q[2:]))   # a larger 16-bit subspace never hurts
    assert q[2] - q[1] > 2.0                       # steep while the subspace is still too small (16 < 24 directions)
    step = 0.05 * 512                              # and nearly flat beyond: under 0.5 dB per further 5 % of K
    assert (q[3] - q[2]) / ((64 - 32) / step) < 0.5 and (q[4] - q[3]) / ((128 - 64) / step) < 0.5


def test_orthogonal_rotation_alone_changes_no_norm():
    spec = synth.LayerSpec(K=256, N=64, r=32, G=64, model=synth.FLUX, seed=6, calib_tokens=1024)
    x = orc.bf16_to_f64(synth.make_tokens(spec, 64, batch_seed=4))
    Q = np.asarray(synth.make_rotation(spec), dtype=np.float64)
    assert np.allclose(np.linalg.norm(x @ Q, axis=1), np.linalg.norm(x, axis=1), rtol=1e-10)
