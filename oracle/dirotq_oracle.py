"""ctypes front end of the plain-C DiRotQ oracle (TEST INFRASTRUCTURE, not a product path).

Only the tests, the smoke check and the benchmark's CPU-baseline leg may import
this module.  It compiles ``dirotq_oracle.c`` with gcc on first use and exposes
the steps of the method one by one, in the order of the paper's Eq. 5:

    prepare (offline):  W~ = Q^T W;  rows < r -> bf16;  rows >= r -> INT4 codes + bf16 scales
    rotate:             x~ = x Q_b           (Q_b = bf16(Q), fp64 accumulation)
    split/quantize:     x~_h -> bf16;  x~_l -> per token, per group INT4 codes + bf16 scales (Eq. 1, z = 0)
    int_gemm:           P_g = q_x q_w per group (int32)
    combine:            y = bf16( sum_g s_x s_w P_g + x~_h W~_h + bias )
"""
from __future__ import annotations

import ctypes
import os
import subprocess
import threading

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "dirotq_oracle.c")
_LIB = os.path.join(_HERE, "libdirotq_oracle.so")
_lock = threading.Lock()
_lib = None


def build(force: bool = False) -> str:
    """Compile the oracle with gcc (OpenMP over rows).  Returns the library path."""
    with _lock:
        if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
            tmp = _LIB + f".{os.getpid()}.tmp"
            subprocess.check_call(["gcc", "-O2", "-fopenmp", "-fPIC", "-shared", "-ffp-contract=off",
                                   "-o", tmp, _SRC, "-lm"])
            os.replace(tmp, _LIB)
    return _LIB


def _load():
    global _lib
    if _lib is None:
        build()
        _lib = ctypes.CDLL(_LIB)
        _lib.dq_bf16_to_double.restype = ctypes.c_double
        _lib.dq_bf16_to_double.argtypes = [ctypes.c_uint16]
        _lib.dq_double_to_bf16.restype = ctypes.c_uint16
        _lib.dq_double_to_bf16.argtypes = [ctypes.c_double]
        _lib.dq_num_threads.restype = ctypes.c_int
        _lib.dq_e4m3_to_double.restype = ctypes.c_double
        _lib.dq_e4m3_to_double.argtypes = [ctypes.c_uint8]
        _lib.dq_e4m3_round.restype = ctypes.c_uint8
        _lib.dq_e4m3_round.argtypes = [ctypes.c_double]
        _lib.dq_e2m1_to_double.restype = ctypes.c_double
        _lib.dq_e2m1_to_double.argtypes = [ctypes.c_uint8]
        _lib.dq_e2m1_round.restype = ctypes.c_uint8
        _lib.dq_e2m1_round.argtypes = [ctypes.c_double]
        _lib.dq_nvfp4_global_exponent.restype = ctypes.c_int
        _lib.dq_nvfp4_global_exponent.argtypes = [ctypes.c_double]
        _lib.dq_nvfp4_prepare_weights.restype = ctypes.c_int
    return _lib


def _p(a: np.ndarray | None):
    return None if a is None else a.ctypes.data_as(ctypes.c_void_p)


def _c(a, dtype):
    return np.ascontiguousarray(a, dtype=dtype)


def num_threads() -> int:
    return int(_load().dq_num_threads())


def bf16_round(a) -> np.ndarray:
    """fp64 -> bf16 bits (uint16), nearest, ties to even."""
    a = _c(a, np.float64)
    out = np.empty(a.shape, dtype=np.uint16)
    _load().dq_round_bf16(_p(a), _p(out), ctypes.c_int64(a.size))
    return out


def bf16_to_f64(bits) -> np.ndarray:
    bits = np.asarray(bits, dtype=np.uint16)
    return (bits.astype(np.uint32) << 16).view(np.float32).astype(np.float64)


def quantize_group(v):
    """Eq. 1 (symmetric, 4 bit) on one group.  Returns (scale_bits, codes, t)."""
    v = _c(v, np.float64).ravel()
    n = v.size
    sb = ctypes.c_uint16(0)
    codes = np.zeros(n, dtype=np.int8)
    t = np.zeros(n, dtype=np.float64)
    _load().dq_quantize_group(_p(v), ctypes.c_int(n), ctypes.c_int64(1), ctypes.byref(sb), _p(codes),
                              ctypes.c_int64(1), _p(t), ctypes.c_int64(1))
    return int(sb.value), codes, t


def fold(Q, W) -> np.ndarray:
    """W~ = Q^T W in fp64 (Eq. 5).  Q [K,K] (unrounded), W [K,N]."""
    Q = _c(Q, np.float64)
    W = _c(W, np.float64)
    K, N = W.shape
    assert Q.shape == (K, K)
    Wt = np.empty((K, N), dtype=np.float64)
    _load().dq_fold(_p(Q), _p(W), _p(Wt), ctypes.c_int(K), ctypes.c_int(N))
    return Wt


def prepare_weights(Wt, r: int, G: int, want_t: bool = False):
    """Split the folded weight at row r; bf16 high rows, INT4 codes + bf16 scales for the rest."""
    Wt = _c(Wt, np.float64)
    K, N = Wt.shape
    K_l = K - r
    n_g = -(-K_l // G)
    Wh = np.empty((r, N), dtype=np.uint16)
    wcodes = np.empty((K_l, N), dtype=np.int8)
    wscales = np.empty((n_g, N), dtype=np.uint16)
    wt = np.empty((K_l, N), dtype=np.float64) if want_t else None
    _load().dq_prepare_weights(_p(Wt), ctypes.c_int(K), ctypes.c_int(N), ctypes.c_int(r), ctypes.c_int(G),
                               _p(Wh), _p(wcodes), _p(wscales), _p(wt))
    return {"Wh": Wh, "wcodes": wcodes, "wscales": wscales, "wt": wt}


def rotate(x_bits, Qb_bits) -> np.ndarray:
    """x~ = x Q_b with fp64 accumulation over bf16 inputs."""
    x_bits = _c(x_bits, np.uint16)
    Qb_bits = _c(Qb_bits, np.uint16)
    M, K = x_bits.shape
    assert Qb_bits.shape == (K, K)
    xt = np.empty((M, K), dtype=np.float64)
    _load().dq_rotate(_p(x_bits), _p(Qb_bits), _p(xt), ctypes.c_int(M), ctypes.c_int(K))
    return xt


def split_quantize(xt, r: int, G: int, want_t: bool = True):
    xt = _c(xt, np.float64)
    M, K = xt.shape
    K_l = K - r
    n_g = -(-K_l // G)
    xh = np.empty((M, r), dtype=np.uint16)
    codes = np.empty((M, K_l), dtype=np.int8)
    scales = np.empty((M, n_g), dtype=np.uint16)
    t = np.empty((M, K_l), dtype=np.float64) if want_t else None
    _load().dq_split_quantize(_p(xt), ctypes.c_int(M), ctypes.c_int(K), ctypes.c_int(r), ctypes.c_int(G),
                              _p(xh), _p(codes), _p(scales), _p(t))
    return {"xh": xh, "codes": codes, "scales": scales, "t": t}


def int_gemm(qx, qw, G: int) -> np.ndarray:
    """P[g,m,n] = sum over group g of qx[m,j] qw[j,n]  (int32)."""
    qx = _c(qx, np.int8)
    qw = _c(qw, np.int8)
    M, K_l = qx.shape
    N = qw.shape[1]
    assert qw.shape[0] == K_l
    n_g = -(-K_l // G)
    P = np.empty((n_g, M, N), dtype=np.int32)
    _load().dq_int_gemm(_p(qx), _p(qw), _p(P), ctypes.c_int(M), ctypes.c_int(K_l), ctypes.c_int(N), ctypes.c_int(G))
    return P


def combine(P, sx, sw, xh, Wh, bias):
    P = _c(P, np.int32)
    n_g, M, N = P.shape
    sx = _c(sx, np.uint16)
    sw = _c(sw, np.uint16)
    xh = _c(xh, np.uint16)
    Wh = _c(Wh, np.uint16)
    r = xh.shape[1]
    assert sx.shape == (M, n_g) and sw.shape == (n_g, N) and Wh.shape == (r, N)
    bias = None if bias is None else _c(bias, np.uint16)
    y64 = np.empty((M, N), dtype=np.float64)
    yb = np.empty((M, N), dtype=np.uint16)
    _load().dq_combine(_p(P), _p(sx), _p(sw), _p(xh), _p(Wh), _p(bias), ctypes.c_int(M), ctypes.c_int(N),
                       ctypes.c_int(r), ctypes.c_int(n_g), _p(y64), _p(yb))
    return y64, yb


def matmul(A, B) -> np.ndarray:
    A = _c(A, np.float64)
    B = _c(B, np.float64)
    M, K = A.shape
    N = B.shape[1]
    C = np.empty((M, N), dtype=np.float64)
    _load().dq_matmul(_p(A), _p(B), _p(C), ctypes.c_int(M), ctypes.c_int(K), ctypes.c_int(N))
    return C


# ---------------------------------------------------------------------------------------------
# whole-layer drivers


def prepare_layer(W, Q, r: int, G: int, want_t: bool = False):
    """Offline part: fold with the *unrounded* Q, quantize, and round Q to bf16 for the online GEMM."""
    Q = _c(Q, np.float64)
    out = prepare_weights(fold(Q, np.asarray(W, dtype=np.float64)), r, G, want_t=want_t)
    out["Qb"] = bf16_round(Q)
    out["r"], out["G"] = r, G
    return out


def linear_deployed(x_bits, layer, bias=None, want_t: bool = True):
    """Online part on bf16 inputs.  Returns every intermediate the parity tests look at."""
    r, G = layer["r"], layer["G"]
    xt = rotate(x_bits, layer["Qb"])
    sq = split_quantize(xt, r, G, want_t=want_t)
    P = int_gemm(sq["codes"], layer["wcodes"], G)
    y64, yb = combine(P, sq["scales"], layer["wscales"], sq["xh"], layer["Wh"], bias)
    return {"xt": xt, "xh": sq["xh"], "codes": sq["codes"], "scales": sq["scales"], "t": sq["t"],
            "P": P, "y64": y64, "y": yb}


# ---------------------------------------------------------------------------------------------
# Projection form with a structured rotation: NOT the paper's Eq. 5 but the cheaper formulation its remarks on the cost
# of the online rotation point towards (Sec. 4.2 keeps only the top-r directions in 16 bits; App. E notes that the
# rotation's cost and memory grow with the layer width).  Only U_h is applied densely, and the residual is taken in
# the Hadamard domain so that both of its terms are plain matrix products:
#     U_hb = bf16(U_h),   V = bf16(U_hb^T H+-)            [r, K]   (H+- = sqrt(G) H: block-diagonal, entries +-1)
#     x~_h = bf16(x U_hb)
#     x~_l = (x H+-  -  x~_h V) / sqrt(G)
#     y    = x~_h ((V H+-^T / G) W)  +  Q4(x~_l) Q4(H^T W)  +  bias
# with H block-diagonal, one orthonormal Hadamard block per quantization group.  x H+- = sqrt(G) x~_l + x~_h V holds by
# construction, and H+- H+-^T = G I, so x = x~_l H^T + x~_h (V H+-^T / G): the layer equals x W when nothing is
# quantized, for any U_h and whatever the rounding of V.  (With V unrounded, x~_l is the block-Hadamard transform of the
# residual x - x~_h U_hb^T of the rounded projection.)  These functions are the reference the library's projection-form
# layers are held to.

def hadamard_signs(n: int) -> np.ndarray:
    """Sylvester-Hadamard matrix of order n (a power of two) with entries +-1: symmetric, H+- H+-^T = n I."""
    assert n >= 1 and n & (n - 1) == 0
    H = np.ones((1, 1), dtype=np.float64)
    while H.shape[0] < n:
        H = np.block([[H, H], [H, -H]])
    return H


def hadamard(n: int) -> np.ndarray:
    """Orthonormal Sylvester-Hadamard matrix of order n: entries +-1/sqrt(n), symmetric."""
    return hadamard_signs(n) / np.sqrt(float(n))


def block_signs_cols(A, G: int) -> np.ndarray:
    """A H+-: every group of G consecutive COLUMNS of A multiplied by the +-1 Hadamard block (sums only: exact in fp64
    for operands of a few significant bits)."""
    A = _c(A, np.float64)
    M, K = A.shape
    assert K % G == 0
    return (A.reshape(M, K // G, G) @ hadamard_signs(G)).reshape(M, K)


def block_hadamard_rows(A, G: int) -> np.ndarray:
    """H^T A for the block-diagonal H with blocks of order G: every group of G consecutive ROWS of A is transformed."""
    A = _c(A, np.float64)
    K = A.shape[0]
    assert K % G == 0
    H = hadamard(G)
    return (H.T @ A.reshape(K // G, G, -1)).reshape(A.shape)


def block_hadamard_cols(A, G: int) -> np.ndarray:
    """A H: every group of G consecutive COLUMNS of A is transformed."""
    A = _c(A, np.float64)
    return block_hadamard_rows(np.ascontiguousarray(A.T), G).T.copy()


def projection_operands_ph(Uh, G: int):
    """U_hb = bf16(U_h) [K, r] and V = bf16(U_hb^T H+-) [r, K], both as bf16 bit patterns."""
    Uh = _c(Uh, np.float64)
    Uhb = bf16_round(Uh)
    V = bf16_round(block_signs_cols(np.ascontiguousarray(bf16_to_f64(Uhb).T), G))
    return Uhb, V


def folded_high_rows_ph(V_bits, W, G: int) -> np.ndarray:
    """(V H+-^T / G) W [r, N] in fp64: the weight the 16-bit coefficients x~_h multiply."""
    back = block_signs_cols(bf16_to_f64(V_bits), G) / float(G)      # V H+-^T / G (H+- is symmetric); exact
    return matmul(np.ascontiguousarray(back), _c(W, np.float64))


def residual_ph(x_bits, layer, G: int, xh_bits=None):
    """x~_h (bf16 bits) and x~_l = (x H+- - x~_h V) / sqrt(G); xh_bits overrides the reference's own x~_h."""
    x = bf16_to_f64(_c(x_bits, np.uint16))
    if xh_bits is None:
        xh_bits = bf16_round(matmul(x, bf16_to_f64(layer["Uhb"])))
    xl = (block_signs_cols(x, G) - matmul(bf16_to_f64(xh_bits), bf16_to_f64(layer["V"]))) / np.sqrt(float(G))
    return xh_bits, xl


def prepare_layer_ph(W, Uh, G: int):
    """Offline part of the projection form.  W [K, N]; Uh [K, r] (the leading principal directions, unrounded)."""
    W = _c(W, np.float64)
    Uh = _c(Uh, np.float64)
    K, N = W.shape
    r = Uh.shape[1]
    assert Uh.shape[0] == K and K % G == 0
    Uhb, V = projection_operands_ph(Uh, G)                      # what runs online
    Wt = np.concatenate([folded_high_rows_ph(V, W, G), block_hadamard_rows(W, G)], axis=0)
    out = prepare_weights(Wt, r, G, want_t=True)               # rows < r -> bf16, the K transformed rows -> INT4 groups
    out["Uhb"], out["V"] = Uhb, V
    out["r"], out["G"], out["K"] = r, G, K
    return out


def linear_deployed_ph(x_bits, layer, bias=None, want_t: bool = True):
    """Online part of the projection form on bf16 inputs; every intermediate is returned."""
    G = layer["G"]
    xh_bits, xl = residual_ph(x_bits, layer, G)
    sq = split_quantize(np.concatenate([np.zeros((xl.shape[0], 0)), xl], axis=1), 0, G, want_t=want_t)
    P = int_gemm(sq["codes"], layer["wcodes"], G)
    y64, yb = combine(P, sq["scales"], layer["wscales"], xh_bits, layer["Wh"], bias)
    return {"xh": xh_bits, "xl": xl, "codes": sq["codes"], "scales": sq["scales"], "t": sq["t"], "P": P,
            "y64": y64, "y": yb}


def nvfp4_prepare_layer_ph(W, Uh, want_t: bool = False):
    """Projection form with NVFP4 operands: rows (V H+-^T / G) W in 16 bits, the rows of H^T W (Hadamard blocks of 64) as
    E2M1 codes with E4M3 block scales and a per-tensor power of two, exactly as nvfp4_prepare_layer quantizes its low rows."""
    W = _c(W, np.float64)
    Uh = _c(Uh, np.float64)
    K, N = W.shape
    r = Uh.shape[1]
    assert Uh.shape[0] == K and K % 64 == 0
    Uhb, V = projection_operands_ph(Uh, 64)
    Wt = np.ascontiguousarray(np.concatenate([folded_high_rows_ph(V, W, 64), block_hadamard_rows(W, 64)], axis=0))
    nb = K // 16
    Wh = np.empty((r, N), dtype=np.uint16)
    wcodes = np.empty((K, N), dtype=np.uint8)
    wsf = np.empty((nb, N), dtype=np.uint8)
    wt = np.empty((K, N), dtype=np.float64) if want_t else None
    ew = _load().dq_nvfp4_prepare_weights(_p(Wt), ctypes.c_int(K + r), ctypes.c_int(N), ctypes.c_int(r), _p(Wh), _p(wcodes),
                                          _p(wsf), _p(wt))
    return {"Wh": Wh, "wcodes": wcodes, "wsf": wsf, "ew": int(ew), "wt": wt, "Uhb": Uhb, "V": V, "r": r, "K": K}


def nvfp4_residual(x_bits, layer, xh_bits=None):
    """residual_ph with the NVFP4 form's Hadamard blocks of 64."""
    return residual_ph(x_bits, layer, 64, xh_bits=xh_bits)


def nvfp4_linear_deployed_ph(x_bits, layer, ex: int, bias=None, want_t: bool = True):
    r = layer["r"]
    xh_bits, xl = nvfp4_residual(x_bits, layer)
    xt = np.ascontiguousarray(np.concatenate([bf16_to_f64(xh_bits), xl], axis=1))
    sq = nvfp4_split_quantize(xt, r, ex, want_t=want_t)
    assert np.array_equal(sq["xh"], xh_bits)
    y64, yb = nvfp4_combine(sq["codes"], sq["sf"], ex, layer, sq["xh"], bias)
    return {"xt": xt, "xh": sq["xh"], "xl": xl, "codes": sq["codes"], "sf": sq["sf"], "t": sq["t"], "y64": y64, "y": yb}


# ---------------------------------------------------------------------------------------------
# GPTQ rounding of the residual weight (Sec. 4.1: the rounding minimises ||X W - X W^||_F^2 rather than the
# layer-wise surrogate; App. F.1: damping 0.01, block size 128).  The steps are those of the published GPTQ
# algorithm, on the residual weight W~_l whose rows are the rotated low columns: the Hessian is
# H = X~_l^T X~_l of the calibration tokens, rows are rounded in order, and the rounding error of each row is
# spread over the rows not yet rounded, weighted by the upper Cholesky factor of H^-1.

def gptq_hessian(xt_low) -> np.ndarray:
    """H = X~_l^T X~_l  [K_l, K_l] in fp64 for calibration tokens X~_l [T, K_l] (already rotated and split)."""
    xt_low = _c(xt_low, np.float64)
    return matmul(np.ascontiguousarray(xt_low.T), xt_low)


def gptq_quantize(Wt_low, H, G: int, damp: float = 0.01, block: int = 128, lazy: bool = True):
    """INT4 codes [K_l, N] and bf16 scale bits [n_g, N] for the residual weight Wt_low [K_l, N].

    Group scales are those of Eq. 1 (bf16(absmax/7) per group of G rows and output column), taken from the
    rows as they stand when the group starts, i.e. after the feedback of every earlier row.  `lazy` applies
    the feedback beyond the current block once per block (the published blocked form); lazy=False applies it
    row by row.  Both are the same arithmetic up to rounding order.
    """
    W = np.array(Wt_low, dtype=np.float64, copy=True)
    H = np.array(H, dtype=np.float64, copy=True)
    K_l, N = W.shape
    assert H.shape == (K_l, K_l) and block % G == 0
    n_g = -(-K_l // G)
    dead = np.diag(H) == 0.0                       # a column no calibration token excites
    H[dead, dead] = 1.0
    W[dead, :] = 0.0
    H[np.diag_indices(K_l)] += damp * np.mean(np.diag(H))
    Hinv = np.linalg.inv(H)
    Hinv = 0.5 * (Hinv + Hinv.T)
    U = np.linalg.cholesky(Hinv).T                 # upper, H^-1 = U^T U
    codes = np.zeros((K_l, N), dtype=np.int8)
    scales = np.zeros((n_g, N), dtype=np.uint16)
    s = np.zeros(N, dtype=np.float64)
    for b0 in range(0, K_l, block):
        b1 = min(b0 + block, K_l)
        E = np.zeros((b1 - b0, N), dtype=np.float64)
        for j in range(b0, b1):
            if j % G == 0:
                g1 = min(j + G, K_l)
                sb = bf16_round(np.max(np.abs(W[j:g1, :]), axis=0) / 7.0)
                scales[j // G, :] = sb
                s = bf16_to_f64(sb)
            safe = np.where(s > 0.0, s, 1.0)
            q = np.where(s > 0.0, np.clip(np.rint(W[j, :] / safe), -7.0, 7.0), 0.0)
            codes[j, :] = q.astype(np.int8)
            err = (W[j, :] - s * q) / U[j, j]
            end = b1 if lazy else K_l
            W[j + 1:end, :] -= np.outer(U[j, j + 1:end], err)
            E[j - b0, :] = err
        if lazy and b1 < K_l:
            W[b1:, :] -= U[b0:b1, b1:].T @ E
    return codes, scales


def prepare_layer_gptq(W, Q, calib_bits, r: int, G: int, damp: float = 0.01, block: int = 128):
    """Offline part with GPTQ rounding: like prepare_layer, but the residual codes and scales come from
    gptq_quantize with the Hessian of the rotated calibration tokens (bf16 bits [T, K])."""
    Q = _c(Q, np.float64)
    Wt = fold(Q, np.asarray(W, dtype=np.float64))
    out = prepare_weights(Wt, r, G, want_t=False)
    out["Qb"] = bf16_round(Q)
    out["r"], out["G"] = r, G
    xt = rotate(calib_bits, out["Qb"])
    H = gptq_hessian(xt[:, r:])
    out["wcodes_rtn"], out["wscales_rtn"] = out["wcodes"], out["wscales"]
    out["wcodes"], out["wscales"] = gptq_quantize(Wt[r:, :], H, G, damp=damp, block=block)
    out["H"], out["Wt_low"] = H, Wt[r:, :]
    return out


# ---------------------------------------------------------------------------------------------
# Asymmetric activation quantization (Sec. 3, Eq. 1 with z = min X; Sec. 5.1: the paper's INT4 setting)

def quantize_group_asym(v):
    v = _c(v, np.float64).ravel()
    n = v.size
    sb, zb = ctypes.c_uint16(0), ctypes.c_uint16(0)
    codes = np.zeros(n, dtype=np.uint8)
    t = np.zeros(n, dtype=np.float64)
    _load().dq_quantize_group_asym(_p(v), ctypes.c_int(n), ctypes.c_int64(1), ctypes.byref(sb), ctypes.byref(zb), _p(codes),
                                   ctypes.c_int64(1), _p(t), ctypes.c_int64(1))
    return int(sb.value), int(zb.value), codes, t


def split_quantize_asym(xt, r: int, G: int, want_t: bool = True):
    xt = _c(xt, np.float64)
    M, K = xt.shape
    K_l = K - r
    n_g = -(-K_l // G)
    xh = np.empty((M, r), dtype=np.uint16)
    codes = np.empty((M, K_l), dtype=np.uint8)
    scales = np.empty((M, n_g), dtype=np.uint16)
    zeros = np.empty((M, n_g), dtype=np.uint16)
    t = np.empty((M, K_l), dtype=np.float64) if want_t else None
    _load().dq_split_quantize_asym(_p(xt), ctypes.c_int(M), ctypes.c_int(K), ctypes.c_int(r), ctypes.c_int(G), _p(xh),
                                   _p(codes), _p(scales), _p(zeros), _p(t))
    return {"xh": xh, "codes": codes, "scales": scales, "zeros": zeros, "t": t}


def int_gemm_u(ux, qw, G: int) -> np.ndarray:
    """P[g,m,n] = sum over group g of u[m,j] qw[j,n] with unsigned activation codes (int32)."""
    ux = _c(ux, np.uint8)
    qw = _c(qw, np.int8)
    M, K_l = ux.shape
    N = qw.shape[1]
    n_g = -(-K_l // G)
    P = np.empty((n_g, M, N), dtype=np.int32)
    _load().dq_int_gemm_u(_p(ux), _p(qw), _p(P), ctypes.c_int(M), ctypes.c_int(K_l), ctypes.c_int(N), ctypes.c_int(G))
    return P


def combine_asym(P, sx, zx, layer, xh, bias):
    P = _c(P, np.int32)
    n_g, M, N = P.shape
    sx, zx, xh = _c(sx, np.uint16), _c(zx, np.uint16), _c(xh, np.uint16)
    sw, qw, Wh = _c(layer["wscales"], np.uint16), _c(layer["wcodes"], np.int8), _c(layer["Wh"], np.uint16)
    bias = None if bias is None else _c(bias, np.uint16)
    y64 = np.empty((M, N), dtype=np.float64)
    yb = np.empty((M, N), dtype=np.uint16)
    _load().dq_combine_asym(_p(P), _p(sx), _p(zx), _p(sw), _p(qw), _p(xh), _p(Wh), _p(bias), ctypes.c_int(M),
                            ctypes.c_int(N), ctypes.c_int(qw.shape[0]), ctypes.c_int(xh.shape[1]), ctypes.c_int(layer["G"]),
                            _p(y64), _p(yb))
    return y64, yb


def linear_deployed_asym(x_bits, layer, bias=None, want_t: bool = True):
    """Online part with asymmetric activation codes (the layer is prepared as for the symmetric case)."""
    r, G = layer["r"], layer["G"]
    xt = rotate(x_bits, layer["Qb"])
    sq = split_quantize_asym(xt, r, G, want_t=want_t)
    P = int_gemm_u(sq["codes"], layer["wcodes"], G)
    y64, yb = combine_asym(P, sq["scales"], sq["zeros"], layer, sq["xh"], bias)
    return {"xt": xt, "xh": sq["xh"], "codes": sq["codes"], "scales": sq["scales"], "zeros": sq["zeros"], "t": sq["t"],
            "P": P, "y64": y64, "y": yb}


# ---------------------------------------------------------------------------------------------
# W4A8 (Sec. 5.1): per-token INT8 activations, per-output-channel INT4 weights

def prepare_layer_w4a8(W, Q, r: int, want_t: bool = False):
    """The weight side is Eq. 1 with a single group spanning the column: prepare_layer with G = K - r."""
    K = np.asarray(Q).shape[0]
    return prepare_layer(W, Q, r, K - r, want_t=want_t)


def split_quantize_a8(xt, r: int, want_t: bool = True):
    xt = _c(xt, np.float64)
    M, K = xt.shape
    K_l = K - r
    xh = np.empty((M, r), dtype=np.uint16)
    codes = np.empty((M, K_l), dtype=np.int8)
    scales = np.empty((M,), dtype=np.uint16)
    t = np.empty((M, K_l), dtype=np.float64) if want_t else None
    _load().dq_split_quantize_a8(_p(xt), ctypes.c_int(M), ctypes.c_int(K), ctypes.c_int(r), _p(xh), _p(codes), _p(scales),
                                 _p(t))
    return {"xh": xh, "codes": codes, "scales": scales, "t": t}


def linear_deployed_w4a8(x_bits, layer, bias=None, want_t: bool = True):
    r = layer["r"]
    xt = rotate(x_bits, layer["Qb"])
    sq = split_quantize_a8(xt, r, want_t=want_t)
    K_l = xt.shape[1] - r
    P = int_gemm(sq["codes"], layer["wcodes"], K_l)                      # one "group": the whole row
    y64, yb = combine(P, sq["scales"].reshape(-1, 1), layer["wscales"], sq["xh"], layer["Wh"], bias)
    return {"xt": xt, "xh": sq["xh"], "codes": sq["codes"], "scales": sq["scales"], "t": sq["t"], "P": P[0], "y64": y64,
            "y": yb}


def linear_ideal(x, Q, W, r: int):
    """Eq. 4 with nothing quantized and nothing rounded: [xU_h, x~_l] [W~_h; W~_l] in fp64."""
    x = _c(x, np.float64)
    Q = _c(Q, np.float64)
    Wt = fold(Q, np.asarray(W, dtype=np.float64))
    xt = matmul(x, Q)
    return matmul(xt[:, :r], Wt[:r]) + matmul(xt[:, r:], Wt[r:])


# ---------------------------------------------------------------------------------------------
# NVFP4 variant (Sec. 5.1): E2M1 elements, blocks of 16 with an E4M3 scale, one power-of-two scale per tensor

E2M1_VALUES = np.array([0.0, 0.5, 1.0, 1.5, 2.0, 3.0, 4.0, 6.0])


def e4m3_to_f64(b) -> np.ndarray:
    b = np.asarray(b, dtype=np.uint8)
    e = ((b >> 3) & 0xF).astype(np.int64)
    m = (b & 7).astype(np.float64)
    v = np.where(e == 0, np.ldexp(m, -9), np.ldexp(1.0 + m / 8.0, e - 7))
    return np.where(b & 0x80, -v, v)


def e2m1_to_f64(c) -> np.ndarray:
    c = np.asarray(c, dtype=np.uint8)
    v = E2M1_VALUES[c & 7]
    return np.where(c & 8, -v, v)


def nvfp4_global_exponent(amax: float) -> int:
    return int(_load().dq_nvfp4_global_exponent(ctypes.c_double(float(amax))))


def nvfp4_quantize_block(v, e_global: int):
    v = _c(v, np.float64).ravel()
    n = v.size
    sf = ctypes.c_uint8(0)
    codes = np.zeros(n, dtype=np.uint8)
    t = np.zeros(n, dtype=np.float64)
    _load().dq_nvfp4_quantize_block(_p(v), ctypes.c_int(n), ctypes.c_int64(1), ctypes.c_int(e_global), ctypes.byref(sf),
                                    _p(codes), ctypes.c_int64(1), _p(t), ctypes.c_int64(1))
    return int(sf.value), codes, t


def nvfp4_prepare_layer(W, Q, r: int, want_t: bool = False):
    Q = _c(Q, np.float64)
    Wt = fold(Q, np.asarray(W, dtype=np.float64))
    K, N = Wt.shape
    K_l = K - r
    nb = -(-K_l // 16)
    Wh = np.empty((r, N), dtype=np.uint16)
    wcodes = np.empty((K_l, N), dtype=np.uint8)
    wsf = np.empty((nb, N), dtype=np.uint8)
    wt = np.empty((K_l, N), dtype=np.float64) if want_t else None
    ew = _load().dq_nvfp4_prepare_weights(_p(Wt), ctypes.c_int(K), ctypes.c_int(N), ctypes.c_int(r), _p(Wh), _p(wcodes),
                                          _p(wsf), _p(wt))
    return {"Wh": Wh, "wcodes": wcodes, "wsf": wsf, "ew": int(ew), "wt": wt, "Qb": bf16_round(Q), "r": r}


def nvfp4_split_quantize(xt, r: int, ex: int, want_t: bool = True):
    xt = _c(xt, np.float64)
    M, K = xt.shape
    K_l = K - r
    nb = -(-K_l // 16)
    xh = np.empty((M, r), dtype=np.uint16)
    codes = np.empty((M, K_l), dtype=np.uint8)
    sf = np.empty((M, nb), dtype=np.uint8)
    t = np.empty((M, K_l), dtype=np.float64) if want_t else None
    _load().dq_nvfp4_split_quantize(_p(xt), ctypes.c_int(M), ctypes.c_int(K), ctypes.c_int(r), ctypes.c_int(ex), _p(xh),
                                    _p(codes), _p(sf), _p(t))
    return {"xh": xh, "codes": codes, "sf": sf, "t": t}


def nvfp4_combine(xcodes, xsf, ex: int, layer, xh, bias):
    xcodes = _c(xcodes, np.uint8)
    xsf = _c(xsf, np.uint8)
    xh = _c(xh, np.uint16)
    M, K_l = xcodes.shape
    N = layer["wcodes"].shape[1]
    r = xh.shape[1]
    bias = None if bias is None else _c(bias, np.uint16)
    y64 = np.empty((M, N), dtype=np.float64)
    yb = np.empty((M, N), dtype=np.uint16)
    _load().dq_nvfp4_combine(_p(xcodes), _p(xsf), ctypes.c_int(ex), _p(_c(layer["wcodes"], np.uint8)),
                             _p(_c(layer["wsf"], np.uint8)), ctypes.c_int(layer["ew"]), _p(xh), _p(_c(layer["Wh"], np.uint16)),
                             _p(bias), ctypes.c_int(M), ctypes.c_int(N), ctypes.c_int(K_l), ctypes.c_int(r), _p(y64), _p(yb))
    return y64, yb


def nvfp4_linear_deployed(x_bits, layer, ex: int, bias=None, want_t: bool = True):
    xt = rotate(x_bits, layer["Qb"])
    sq = nvfp4_split_quantize(xt, layer["r"], ex, want_t=want_t)
    y64, yb = nvfp4_combine(sq["codes"], sq["sf"], ex, layer, sq["xh"], bias)
    return {"xt": xt, "xh": sq["xh"], "codes": sq["codes"], "sf": sq["sf"], "t": sq["t"], "y64": y64, "y": yb}
