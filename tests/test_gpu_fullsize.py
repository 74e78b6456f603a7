"""Parity at the full sizes of the benchmarked configurations (PixArt- and FLUX-shaped layers), in the launch configuration bench.py times
(persistent 148-CTA grids, many tiles per CTA), on sampled outputs the oracle can compute one by one.

Token rows are independent (per-token scales, row-wise GEMM) and so are output columns of the weight
side, hence comparing a seeded sample of rows x columns is exact, not approximate.  Per case:
  * prepared weights (codes, scales, bf16 rows) of the sampled columns, and the whole bf16 rotation,
    against the oracle's fold + quantizer;
  * activation codes / scales / bf16 coefficients of the sampled rows against the oracle's
    rotation + quantizer (tolerated: +-1 code at a rounding boundary, neighbouring bf16 scale at a
    boundary, see parity_utils);
  * int32 group sums of a 128-row slice on the sampled columns, bit exact;
  * the bf16 output of the sampled rows x columns.
"""
import numpy as np
import pytest
import torch

from oracle import dirotq_oracle as orc
from paper_2605_16732_b200 import binding as dq
from paper_2605_16732_b200 import synth

from parity_utils import (bf16_tensor_to_bits, bits_to_bf16_tensor, check_activation_side, check_layer_output)

pytestmark = pytest.mark.gpu

_ROT = {}


def _rotation(spec):
    key = (spec.K, spec.r, spec.model.name, spec.seed)
    if key not in _ROT:
        _ROT.clear()  # keep at most one K x K fp64 matrix alive
        _ROT[key] = synth.make_rotation(spec, device="cuda")
    return _ROT[key]


def _run(M, K, N, r, G, model, n_rows=24, n_cols=96, seed=0):
    spec = synth.LayerSpec(K=K, N=N, r=r, G=G, model=model, seed=seed)
    Q = _rotation(spec)
    W, bias = synth.make_weights(spec)
    x_bits = synth.make_tokens(spec, M, batch_seed=3)
    g = np.random.default_rng(K * 7 + N)
    rows = np.sort(g.choice(M, size=min(n_rows, M), replace=False))
    rows[-1] = M - 1  # always include the last row of the ragged last token block
    cols = np.sort(g.choice(N, size=n_cols, replace=False))
    cols[-1] = N - 1

    # ---- oracle on the sample
    lo = orc.prepare_layer(W[:, cols], Q, r, G, want_t=True)
    bias_s = bias[cols]
    oo = orc.linear_deployed(x_bits[rows], lo, bias=bias_s)

    # ---- library on everything
    Qd = torch.from_numpy(Q).cuda()
    layer = dq.dirotq_prepare_layer(torch.from_numpy(W).cuda(), Qd, r, G, bias=bits_to_bf16_tensor(bias))
    del Qd
    wcodes, wscales, wh, qb = dq.dirotq_layer_export(layer)
    assert np.array_equal(bf16_tensor_to_bits(qb), lo["Qb"]), "bf16 rotation differs"
    del qb
    cols_t = torch.from_numpy(cols).cuda()
    assert np.array_equal(bf16_tensor_to_bits(wscales[:, cols_t]), lo["wscales"])
    assert np.array_equal(bf16_tensor_to_bits(wh[:, cols_t]), lo["Wh"])
    wc = wcodes[:, cols_t].cpu().numpy()
    bad = wc != lo["wcodes"]
    assert bad.sum() <= 2 and np.all(np.abs(np.abs(lo["wt"][bad] - np.floor(lo["wt"][bad])) - 0.5) < 1e-9)
    del wcodes, wscales, wh

    x = bits_to_bf16_tensor(x_bits)
    y = torch.zeros((M, N), dtype=torch.bfloat16, device="cuda")
    ws = dq.alloc_workspace(layer, M)
    dq.dirotq_linear(x, layer, y, ws)
    assert dq.dirotq_workspace_status(ws) == 0
    xh, codes, scales = dq.dirotq_workspace_export(layer, M, ws)
    rows_t = torch.from_numpy(rows).cuda()
    xh_b = bf16_tensor_to_bits(xh[rows_t])
    codes_n = codes[rows_t].cpu().numpy()
    scales_b = bf16_tensor_to_bits(scales[rows_t])
    stats = check_activation_side(None, xh_b, codes_n, scales_b, oo, r, G)
    y_s = bf16_tensor_to_bits(y[rows_t][:, cols_t])
    stats.update(check_layer_output(y_s, xh_b, codes_n, scales_b, lo, oo, bias_s))

    # ---- int32 group sums, bit exact, on a 128-row slice that spans a token-block boundary
    m0 = max(0, min(M - 128, (M // 2) - 37))
    msub = min(128, M)
    sl = codes[m0:m0 + msub]
    padded = torch.zeros((msub, layer.K_lp), dtype=torch.int8, device="cuda")
    padded[:, :layer.K_l] = sl
    ws2 = dq.alloc_workspace(layer, msub)
    P = dq.dirotq_int_gemm_debug(padded, layer, ws2)
    assert dq.dirotq_workspace_status(ws2) == 0
    P_ref = orc.int_gemm(sl.cpu().numpy(), lo["wcodes"], G)
    assert np.array_equal(P[:, :, cols_t].cpu().numpy(), P_ref), "int32 group sums differ"
    layer.close()
    return stats


# config 3: FLUX.1-dev-shaped linears at M = 4608 (the benchmark's workload)
@pytest.mark.parametrize("K,N", [(3072, 9216), (3072, 3072), (3072, 12288), (12288, 3072)])
def test_config3_flux_linears(K, N):
    print(_run(4608, K, N, 32, 64, synth.FLUX))


# config 2: PixArt-Sigma-shaped block linears at M = 4096
@pytest.mark.parametrize("K,N", [(1152, 1152), (1152, 4608), (4608, 1152)])
def test_config2_pixart_linears(K, N):
    print(_run(4096, K, N, 32, 64, synth.PIXART))


# config 4: batch 4 (M = 18432), rank and group sweep (a subset that covers every r and both G)
@pytest.mark.parametrize("K,N,r,G", [(3072, 9216, 16, 64), (3072, 9216, 64, 128), (3072, 9216, 128, 64),
                                     (12288, 3072, 128, 128)])
def test_config4_rank_group_sweep(K, N, r, G):
    print(_run(18432, K, N, r, G, synth.FLUX))


# the paper's own rank (about a tenth of K kept in 16 bits, Sec. 4.2) on two FLUX linears at M = 4608
@pytest.mark.parametrize("K,N,r", [(3072, 9216, 320), (12288, 3072, 1232)])
def test_flux_linears_at_ten_percent_rank(K, N, r):
    print(_run(4608, K, N, r, 64, synth.FLUX))


# config 5: the two single-stream shapes that the other configs do not contain
@pytest.mark.parametrize("K,N", [(3072, 21504), (15360, 3072)])
def test_config5_single_stream_shapes(K, N):
    print(_run(4608, K, N, 32, 64, synth.FLUX))


# ------------------------------------------------------------------ NVFP4 variant at the benchmark's sizes

def _run_nvfp4(M, K, N, r, model, n_rows=24, n_cols=96, seed=0):
    from parity_utils import check_activation_side_nvfp4, check_layer_output_nvfp4, _codes_equal_mod_zero
    spec = synth.LayerSpec(K=K, N=N, r=r, G=64, model=model, seed=seed)
    Q = _rotation(spec)
    W, bias = synth.make_weights(spec)
    x_bits = synth.make_tokens(spec, M, batch_seed=3)
    g = np.random.default_rng(K * 7 + N + 1)
    rows = np.sort(g.choice(M, size=min(n_rows, M), replace=False))
    rows[-1] = M - 1
    cols = np.sort(g.choice(N, size=n_cols, replace=False))
    cols[-1] = N - 1

    # The weights' per-tensor exponent depends on ALL columns (max |W~_l|): the oracle folds the whole weight.
    lo_full = orc.nvfp4_prepare_layer(W, Q, r, want_t=True)
    lo = dict(lo_full)
    lo["wcodes"], lo["wsf"], lo["Wh"] = lo_full["wcodes"][:, cols], lo_full["wsf"][:, cols], lo_full["Wh"][:, cols]
    bias_s = bias[cols]
    xt = orc.rotate(x_bits[rows], lo["Qb"])
    ex = orc.nvfp4_global_exponent(float(np.abs(xt[:, r:]).max()))
    oo = orc.nvfp4_linear_deployed(x_bits[rows], lo, ex, bias=bias_s)

    Qd = torch.from_numpy(Q).cuda()
    layer = dq.dirotq_prepare_layer_nvfp4(torch.from_numpy(W).cuda(), Qd, r, ex, bias=bits_to_bf16_tensor(bias))
    del Qd
    wcodes, wsf, wh, qb, ew = dq.dirotq_layer_export_nvfp4(layer)
    assert ew == lo_full["ew"]
    assert np.array_equal(bf16_tensor_to_bits(qb), lo["Qb"]), "bf16 rotation differs"
    del qb
    cols_t = torch.from_numpy(cols).cuda()
    assert np.array_equal(wsf[:, cols_t].cpu().numpy(), lo["wsf"])
    assert np.array_equal(bf16_tensor_to_bits(wh[:, cols_t]), lo["Wh"])
    bad = ~_codes_equal_mod_zero(wcodes[:, cols_t].cpu().numpy(), lo["wcodes"])
    assert bad.sum() <= 2
    del wcodes, wsf, wh

    x = bits_to_bf16_tensor(x_bits)
    y = torch.zeros((M, N), dtype=torch.bfloat16, device="cuda")
    ws = dq.alloc_workspace(layer, M)
    dq.dirotq_linear(x, layer, y, ws)
    assert dq.dirotq_workspace_status(ws) == 0
    xh, codes, sf = dq.dirotq_workspace_export_nvfp4(layer, M, ws)
    rows_t = torch.from_numpy(rows).cuda()
    xh_b = bf16_tensor_to_bits(xh[rows_t])
    codes_n = codes[rows_t].cpu().numpy()
    sf_n = sf[rows_t].cpu().numpy()
    stats = check_activation_side_nvfp4(None, xh_b, codes_n, sf_n, oo, r, ex)
    y_s = bf16_tensor_to_bits(y[rows_t][:, cols_t])
    stats.update(check_layer_output_nvfp4(y_s, xh_b, codes_n, sf_n, ex, lo, oo, bias_s))
    layer.close()
    return stats


@pytest.mark.parametrize("K,N", [(3072, 9216), (12288, 3072)])
def test_nvfp4_flux_linears(K, N):
    print(_run_nvfp4(4608, K, N, 32, synth.FLUX))


def test_nvfp4_batch4_rank128():
    print(_run_nvfp4(18432, 3072, 9216, 128, synth.FLUX))


# ------------------------------------------------------------------ asymmetric activation codes at the benchmark's sizes

def _run_asym(M, K, N, r, G, model, n_rows=24, n_cols=96, seed=0):
    from parity_utils import check_activation_side_asym, check_layer_output_asym
    spec = synth.LayerSpec(K=K, N=N, r=r, G=G, model=model, seed=seed)
    Q = _rotation(spec)
    W, bias = synth.make_weights(spec)
    x_bits = synth.make_tokens(spec, M, batch_seed=3)
    g = np.random.default_rng(K * 7 + N + 2)
    rows = np.sort(g.choice(M, size=min(n_rows, M), replace=False))
    rows[-1] = M - 1
    cols = np.sort(g.choice(N, size=n_cols, replace=False))
    cols[-1] = N - 1
    lo = orc.prepare_layer(W[:, cols], Q, r, G, want_t=True)
    bias_s = bias[cols]
    oo = orc.linear_deployed_asym(x_bits[rows], lo, bias=bias_s)

    Qd = torch.from_numpy(Q).cuda()
    layer = dq.dirotq_prepare_layer_asym(torch.from_numpy(W).cuda(), Qd, r, G, bias=bits_to_bf16_tensor(bias))
    del Qd
    cols_t = torch.from_numpy(cols).cuda()
    n_g = layer.n_g
    csum = np.stack([lo["wcodes"][gi * G:(gi + 1) * G].astype(np.int64).sum(axis=0) for gi in range(n_g)])
    d_ref = (orc.bf16_to_f64(lo["wscales"]) * csum).astype(np.float32)
    d = dq.dirotq_layer_export_zero_term(layer)[:, cols_t].cpu().numpy()
    # a weight code may differ from the oracle's at an exact tie of the fp64 quotient (different summation order in
    # the fold): compare the zero-point term on the columns whose codes all agree
    wc = dq.dirotq_layer_export(layer)[0][:, cols_t].cpu().numpy()
    agree = np.all(wc == lo["wcodes"], axis=0)
    assert agree.sum() >= n_cols - 2 and np.array_equal(d[:, agree], d_ref[:, agree]), "zero-point term differs"

    x = bits_to_bf16_tensor(x_bits)
    y = torch.zeros((M, N), dtype=torch.bfloat16, device="cuda")
    ws = dq.alloc_workspace(layer, M)
    dq.dirotq_linear(x, layer, y, ws)
    assert dq.dirotq_workspace_status(ws) == 0
    xh, codes, scales, zeros = dq.dirotq_workspace_export_asym(layer, M, ws)
    rows_t = torch.from_numpy(rows).cuda()
    xh_b = bf16_tensor_to_bits(xh[rows_t])
    codes_n = codes[rows_t].cpu().numpy()
    scales_b, zeros_b = bf16_tensor_to_bits(scales[rows_t]), bf16_tensor_to_bits(zeros[rows_t])
    stats = check_activation_side_asym(None, xh_b, codes_n, scales_b, zeros_b, oo, r, G)
    lo_lib = dict(lo)
    lo_lib["wcodes"] = wc  # the output check uses the library's own weight codes
    y_s = bf16_tensor_to_bits(y[rows_t][:, cols_t])
    stats.update(check_layer_output_asym(y_s, xh_b, codes_n, scales_b, zeros_b, lo_lib, oo, bias_s))
    layer.close()
    return stats


@pytest.mark.parametrize("K,N", [(3072, 9216), (12288, 3072)])
def test_asym_flux_linears(K, N):
    print(_run_asym(4608, K, N, 32, 64, synth.FLUX))


def test_asym_batch4_rank64_group128():
    print(_run_asym(18432, 3072, 9216, 64, 128, synth.FLUX))


# ------------------------------------------------------------------ W4A8 at the benchmark's sizes

def _run_w4a8(M, K, N, r, model, n_rows=24, n_cols=96, seed=0):
    from parity_utils import check_activation_side_w4a8, check_layer_output_w4a8
    spec = synth.LayerSpec(K=K, N=N, r=r, G=64, model=model, seed=seed)
    Q = _rotation(spec)
    W, bias = synth.make_weights(spec)
    x_bits = synth.make_tokens(spec, M, batch_seed=3)
    g = np.random.default_rng(K * 7 + N + 3)
    rows = np.sort(g.choice(M, size=min(n_rows, M), replace=False))
    rows[-1] = M - 1
    cols = np.sort(g.choice(N, size=n_cols, replace=False))
    cols[-1] = N - 1
    lo = orc.prepare_layer_w4a8(W[:, cols], Q, r, want_t=True)   # one scale per column: columns are independent
    bias_s = bias[cols]
    oo = orc.linear_deployed_w4a8(x_bits[rows], lo, bias=bias_s)

    Qd = torch.from_numpy(Q).cuda()
    layer = dq.dirotq_prepare_layer_w4a8(torch.from_numpy(W).cuda(), Qd, r, bias=bits_to_bf16_tensor(bias))
    del Qd
    wcodes, wscales, wh, qb = dq.dirotq_layer_export(layer)
    assert np.array_equal(bf16_tensor_to_bits(qb), lo["Qb"]), "bf16 rotation differs"
    del qb
    cols_t = torch.from_numpy(cols).cuda()
    assert np.array_equal(bf16_tensor_to_bits(wscales[:, cols_t]), lo["wscales"])
    assert np.array_equal(bf16_tensor_to_bits(wh[:, cols_t]), lo["Wh"])
    wc = wcodes[:, cols_t].cpu().numpy()
    bad = wc != lo["wcodes"]
    assert bad.sum() <= 2 and np.all(np.abs(np.abs(lo["wt"][bad] - np.floor(lo["wt"][bad])) - 0.5) < 1e-9)
    del wcodes, wscales, wh

    x = bits_to_bf16_tensor(x_bits)
    y = torch.zeros((M, N), dtype=torch.bfloat16, device="cuda")
    ws = dq.alloc_workspace(layer, M)
    dq.dirotq_linear(x, layer, y, ws)
    assert dq.dirotq_workspace_status(ws) == 0
    xh, codes, scales = dq.dirotq_workspace_export_w4a8(layer, M, ws)
    rows_t = torch.from_numpy(rows).cuda()
    xh_b = bf16_tensor_to_bits(xh[rows_t])
    codes_n = codes[rows_t].cpu().numpy()
    scales_b = bf16_tensor_to_bits(scales[rows_t])
    stats = check_activation_side_w4a8(None, xh_b, codes_n, scales_b, oo, r)
    lo_lib = dict(lo)
    lo_lib["wcodes"] = wc
    y_s = bf16_tensor_to_bits(y[rows_t][:, cols_t])
    stats.update(check_layer_output_w4a8(y_s, xh_b, codes_n, scales_b, lo_lib, oo, bias_s))
    layer.close()
    return stats


@pytest.mark.parametrize("K,N", [(3072, 9216), (12288, 3072)])
def test_w4a8_flux_linears(K, N):
    print(_run_w4a8(4608, K, N, 32, synth.FLUX))


# ------------------------------------------------------------------ projection form at the benchmark's sizes

def _run_ph(M, K, N, r, G, model, n_rows=24, n_cols=96, seed=0):
    """Sampled parity of the projection form: the reference's steps on a sample of token rows (all K columns, since the
    Hadamard blocks and the groups need them) and a sample of output columns."""
    from parity_utils import check_activation_side, check_output
    spec = synth.LayerSpec(K=K, N=N, r=r, G=G, model=model, seed=seed)
    rng = np.random.default_rng(1234 + seed)
    rows = np.sort(rng.choice(M, size=n_rows, replace=False))
    cols = np.sort(rng.choice(N, size=n_cols, replace=False))
    Q = synth.make_rotation(spec, device="cuda")
    Uh = np.ascontiguousarray(np.asarray(Q, dtype=np.float64)[:, :r])
    W, bias = synth.make_weights(spec)
    x_bits = synth.make_tokens(spec, M, batch_seed=7)
    dev = "cuda"
    layer = dq.dirotq_prepare_layer_ph(torch.from_numpy(W).to(dev), torch.from_numpy(Uh).to(dev), G, bias=bits_to_bf16_tensor(bias))
    x = bits_to_bf16_tensor(x_bits)
    ws = dq.alloc_workspace(layer, M)
    y = torch.zeros((M, N), dtype=torch.bfloat16, device=dev)
    dq.dirotq_linear(x, layer, y, ws)
    torch.cuda.synchronize()
    assert dq.dirotq_workspace_status(ws) == 0
    xh, codes, scales = dq.dirotq_workspace_export(layer, M, ws)
    xh_b = bf16_tensor_to_bits(xh)[rows]
    codes_n, scales_b = codes.cpu().numpy()[rows], bf16_tensor_to_bits(scales)[rows]
    lo = orc.prepare_layer_ph(np.ascontiguousarray(W[:, cols]), Uh, G)
    oo = orc.linear_deployed_ph(np.ascontiguousarray(x_bits[rows]), lo, bias=np.ascontiguousarray(bias[cols]))
    xh_g = orc.bf16_to_f64(xh_b)
    _, xl_ref = orc.residual_ph(np.ascontiguousarray(x_bits[rows]), lo, G, xh_bits=xh_b)
    sq_ref = orc.split_quantize(xl_ref, 0, G, want_t=True)
    prot = {"xt": np.concatenate([xh_g, xl_ref], axis=1), "xh": xh_b, "scales": sq_ref["scales"], "codes": sq_ref["codes"]}
    stats = check_activation_side(None, xh_b, codes_n, scales_b, prot, r, G)
    xnorm = np.linalg.norm(orc.bf16_to_f64(x_bits[rows]), axis=1, keepdims=True)
    xh_o = orc.bf16_to_f64(oo["xh"])
    assert np.all(np.abs(xh_g - xh_o) <= np.maximum(np.abs(xh_o), 2.0 ** -126) * 2.0 ** -7 + 1e-5 * xnorm)
    # output on the sample: the reference's last steps on the library's own codes, scales and x~_h
    wcodes = torch.empty((K, N), dtype=torch.int8, device=dev)
    dq._check(dq.lib().dirotq_layer_export(layer.handle, wcodes.data_ptr(), None, None, None, None), "dirotq_layer_export")
    torch.cuda.synchronize()
    wc = wcodes.cpu().numpy()[:, cols]
    bad = wc != lo["wcodes"]
    assert bad.sum() <= 4
    P = orc.int_gemm(codes_n, np.ascontiguousarray(wc), G)
    y_ref, _ = orc.combine(P, scales_b, lo["wscales"], xh_b, lo["Wh"], np.ascontiguousarray(bias[cols]))
    y_s = bf16_tensor_to_bits(y)[np.ix_(rows, cols)]
    stats.update(check_output(y_s, y_ref))
    layer.close()
    return stats


@pytest.mark.parametrize("K,N", [(3072, 9216), (12288, 3072)])
def test_projection_form_flux_linears(K, N):
    print(_run_ph(4608, K, N, 32, 64, synth.FLUX))


def test_projection_form_batch4_group128_rank128():
    print(_run_ph(18432, 3072, 3072, 128, 128, synth.FLUX))


# ------------------------------------------------------------------ NVFP4 operands behind the projection form, full size

def _run_nvfp4_ph(M, K, N, r, model, n_rows=24, n_cols=96, seed=0):
    from parity_utils import check_activation_side_nvfp4, check_layer_output_nvfp4, _codes_equal_mod_zero
    spec = synth.LayerSpec(K=K, N=N, r=r, G=64, model=model, seed=seed)
    Uh = np.ascontiguousarray(np.asarray(synth.make_rotation(spec, device="cuda"), dtype=np.float64)[:, :r])
    W, bias = synth.make_weights(spec)
    x_bits = synth.make_tokens(spec, M, batch_seed=3)
    g = np.random.default_rng(K * 7 + N + 2)
    rows = np.sort(g.choice(M, size=min(n_rows, M), replace=False))
    rows[-1] = M - 1
    cols = np.sort(g.choice(N, size=n_cols, replace=False))
    cols[-1] = N - 1

    # the weights' per-tensor exponent depends on all columns: the reference folds the whole weight
    lo_full = orc.nvfp4_prepare_layer_ph(W, Uh, want_t=True)
    lo = dict(lo_full)
    lo["wcodes"], lo["wsf"], lo["Wh"] = lo_full["wcodes"][:, cols], lo_full["wsf"][:, cols], lo_full["Wh"][:, cols]
    if lo_full["wt"] is not None:
        lo["wt"] = lo_full["wt"][:, cols]
    bias_s = np.ascontiguousarray(bias[cols])
    xs = np.ascontiguousarray(x_bits[rows])
    ex = orc.nvfp4_global_exponent(float(np.abs(orc.nvfp4_residual(xs, lo)[1]).max()))
    oo = orc.nvfp4_linear_deployed_ph(xs, lo, ex, bias=bias_s)

    layer = dq.dirotq_prepare_layer_nvfp4_ph(torch.from_numpy(W).cuda(), torch.from_numpy(Uh).cuda(), ex,
                                             bias=bits_to_bf16_tensor(bias))
    wcodes, wsf, wh, uhb, ew = dq.dirotq_layer_export_nvfp4(layer)
    assert ew == lo_full["ew"]
    assert np.array_equal(bf16_tensor_to_bits(uhb), lo["Uhb"])
    cols_t = torch.from_numpy(cols).cuda()
    assert np.array_equal(wsf[:, cols_t].cpu().numpy(), lo["wsf"])
    assert np.array_equal(bf16_tensor_to_bits(wh[:, cols_t]), lo["Wh"])
    bad = ~_codes_equal_mod_zero(wcodes[:, cols_t].cpu().numpy(), lo["wcodes"])
    assert bad.sum() <= 2
    del wcodes, wsf, wh

    x = bits_to_bf16_tensor(x_bits)
    y = torch.zeros((M, N), dtype=torch.bfloat16, device="cuda")
    ws = dq.alloc_workspace(layer, M)
    dq.dirotq_linear(x, layer, y, ws)
    assert dq.dirotq_workspace_status(ws) == 0
    xh, codes, sf = dq.dirotq_workspace_export_nvfp4(layer, M, ws)
    rows_t = torch.from_numpy(rows).cuda()
    xh_b = bf16_tensor_to_bits(xh[rows_t])
    codes_n, sf_n = codes[rows_t].cpu().numpy(), sf[rows_t].cpu().numpy()
    _, xl_ref = orc.nvfp4_residual(xs, lo, xh_bits=xh_b)
    xt_ref = np.ascontiguousarray(np.concatenate([orc.bf16_to_f64(xh_b), xl_ref], axis=1))
    sq_ref = orc.nvfp4_split_quantize(xt_ref, r, ex, want_t=True)
    prot = {"xt": xt_ref, "xh": sq_ref["xh"], "codes": sq_ref["codes"], "sf": sq_ref["sf"], "t": sq_ref["t"]}
    stats = check_activation_side_nvfp4(None, xh_b, codes_n, sf_n, prot, r, ex)
    y_s = bf16_tensor_to_bits(y[rows_t][:, cols_t])
    stats.update(check_layer_output_nvfp4(y_s, xh_b, codes_n, sf_n, ex, lo, oo, bias_s))
    layer.close()
    return stats


@pytest.mark.parametrize("K,N", [(3072, 9216), (12288, 3072)])
def test_nvfp4_projection_form_flux_linears(K, N):
    print(_run_nvfp4_ph(4608, K, N, 32, synth.FLUX))


def test_nvfp4_projection_form_batch4_rank128():
    print(_run_nvfp4_ph(18432, 3072, 3072, 128, synth.FLUX))
