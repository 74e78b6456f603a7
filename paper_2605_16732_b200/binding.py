"""ctypes binding of libdirotq: argument marshalling only.

Function names mirror the C ABI in ``include/dirotq.h``.  Tensors are torch tensors used as
device memory; every step of the layer runs inside the CUDA library.  If the library is not
built, importing the entry points raises: there is no fallback path.
"""
from __future__ import annotations

import ctypes
import os

import torch

from . import build as _build

# DIROTQ_LIBRARY: another build of the same library to load instead (the integer-path fallback, build.build_i8())
_LIB_PATH = os.environ.get("DIROTQ_LIBRARY") or os.path.join(os.path.dirname(os.path.abspath(__file__)), "libdirotq.so")

DIROTQ_OK = 0
STATUS_NAMES = {0: "ok", 1: "invalid argument", 2: "unsupported shape", 3: "buffer too small",
                4: "device is not sm_100", 5: "CUDA error", 6: "device-side wait timed out"}
DTYPE_F32, DTYPE_BF16, DTYPE_F64 = 0, 1, 2
LAYOUT_KN, LAYOUT_NK = 0, 1

EXPORTED = [
    "dirotq_status_string", "dirotq_version", "dirotq_last_error", "dirotq_layer_bytes",
    "dirotq_prepare_scratch_bytes", "dirotq_workspace_bytes", "dirotq_prepare_layer", "dirotq_layer_destroy",
    "dirotq_layer_info", "dirotq_linear", "dirotq_linear_host", "dirotq_workspace_status",
    "dirotq_rotate_quantize", "dirotq_w4a4_gemm", "dirotq_workspace_wait_counters", "dirotq_workspace_export", "dirotq_int_gemm_debug", "dirotq_layer_export",
    "dirotq_mma_rate_probe", "dirotq_linear_noalloc", "dirotq_wait_selftest", "dirotq_act_scale_log2_from_rotated", "dirotq_act_scale_log2_ph",
    "dirotq_layer_bytes_nvfp4", "dirotq_prepare_layer_nvfp4", "dirotq_workspace_export_nvfp4", "dirotq_layer_export_nvfp4",
    "dirotq_layer_bytes_w4a8", "dirotq_prepare_layer_w4a8", "dirotq_workspace_export_w4a8",
    "dirotq_prepare_layer_codes", "dirotq_prepare_scratch_bytes_gptq", "dirotq_prepare_layer_gptq", "dirotq_layer_bytes_ph", "dirotq_prepare_scratch_bytes_ph", "dirotq_prepare_layer_ph",
    "dirotq_layer_export_uh", "dirotq_layer_export_v", "dirotq_layer_bytes_nvfp4_ph", "dirotq_prepare_layer_nvfp4_ph", "dirotq_layer_bytes_sibling", "dirotq_prepare_layer_sibling", "dirotq_set_gemm_tile", "dirotq_set_dependent_launch", "dirotq_set_rotation_tile", "dirotq_set_first_step_split", "dirotq_layer_bytes_asym", "dirotq_prepare_layer_asym", "dirotq_workspace_export_asym", "dirotq_layer_export_zero_term",
]


class DirotqError(RuntimeError):
    def __init__(self, status: int, where: str, detail: str = ""):
        self.status = status
        super().__init__(f"{where}: {STATUS_NAMES.get(status, status)}" + (f" ({detail})" if detail else ""))


_lib = None


def use_library(path: str) -> None:
    """Makes the binding load another build of the library (before its first use): the integer-path fallback or the
    diagnostic build of paper_2605_16732_b200.build."""
    global _LIB_PATH
    if _lib is not None:
        raise RuntimeError("a library is loaded already")
    _LIB_PATH = path


def lib() -> ctypes.CDLL:
    """Loads libdirotq.so (must have been built: ``python -m paper_2605_16732_b200.build``)."""
    global _lib
    if _lib is None:
        if not os.path.exists(_LIB_PATH):
            raise ImportError(f"{_LIB_PATH} is missing: build it with paper_2605_16732_b200.build.build()")
        L = ctypes.CDLL(_LIB_PATH)
        vp, i, sz = ctypes.c_void_p, ctypes.c_int, ctypes.c_size_t
        pi, psz = ctypes.POINTER(ctypes.c_int), ctypes.POINTER(ctypes.c_size_t)
        L.dirotq_status_string.restype = ctypes.c_char_p
        L.dirotq_status_string.argtypes = [i]
        L.dirotq_version.restype = i
        L.dirotq_last_error.restype = ctypes.c_char_p
        L.dirotq_layer_bytes.argtypes = [i, i, i, i, psz]
        L.dirotq_prepare_scratch_bytes.argtypes = [i, i, psz]
        L.dirotq_workspace_bytes.argtypes = [vp, i, psz]
        L.dirotq_prepare_layer.argtypes = [vp, i, i, vp, i, vp, i, i, i, i, vp, sz, vp, sz, vp, ctypes.POINTER(vp)]
        L.dirotq_layer_destroy.argtypes = [vp]
        L.dirotq_layer_info.argtypes = [vp, pi, pi, pi, pi, pi, pi]
        L.dirotq_linear.argtypes = [vp, i, vp, vp, vp, sz, vp]
        L.dirotq_linear_host.argtypes = [vp, i, vp, vp, vp, vp, vp, sz, vp]
        L.dirotq_workspace_status.argtypes = [vp, vp, pi]
        L.dirotq_rotate_quantize.argtypes = [vp, i, vp, vp, sz, vp, vp]
        L.dirotq_w4a4_gemm.argtypes = [i, vp, vp, sz, vp, vp]
        L.dirotq_workspace_wait_counters.argtypes = [vp, vp, ctypes.POINTER(ctypes.c_ulonglong)]
        L.dirotq_workspace_export.argtypes = [vp, i, vp, vp, vp, vp, vp]
        L.dirotq_int_gemm_debug.argtypes = [vp, i, vp, vp, vp, sz, vp]
        L.dirotq_layer_export.argtypes = [vp, vp, vp, vp, vp, vp]
        L.dirotq_linear_noalloc.argtypes = [vp, i, vp, vp, vp, vp]
        L.dirotq_mma_rate_probe.argtypes = [i, i, vp, ctypes.POINTER(ctypes.c_float), vp]
        L.dirotq_wait_selftest.argtypes = [vp, ctypes.c_uint, vp]
        L.dirotq_act_scale_log2_from_rotated.argtypes = [vp, i, i, i, vp, pi, vp]
        L.dirotq_act_scale_log2_ph.argtypes = [vp, i, vp, i, i, i, vp, sz, pi, vp]
        L.dirotq_layer_bytes_nvfp4.argtypes = [i, i, i, psz]
        L.dirotq_prepare_layer_nvfp4.argtypes = [vp, i, i, vp, i, vp, i, i, i, i, vp, sz, vp, sz, vp, ctypes.POINTER(vp)]
        L.dirotq_workspace_export_nvfp4.argtypes = [vp, i, vp, vp, vp, vp, vp]
        L.dirotq_layer_export_nvfp4.argtypes = [vp, vp, vp, vp, vp, vp, vp]
        L.dirotq_layer_bytes_w4a8.argtypes = [i, i, i, psz]
        L.dirotq_prepare_layer_w4a8.argtypes = [vp, i, i, vp, i, vp, i, i, i, vp, sz, vp, sz, vp, ctypes.POINTER(vp)]
        L.dirotq_workspace_export_w4a8.argtypes = [vp, i, vp, vp, vp, vp, vp]
        L.dirotq_layer_bytes_asym.argtypes = [i, i, i, i, psz]
        L.dirotq_prepare_layer_asym.argtypes = [vp, i, i, vp, i, vp, i, i, i, i, vp, sz, vp, sz, vp, ctypes.POINTER(vp)]
        L.dirotq_layer_bytes_sibling.argtypes = [i, i, i, i, i, ctypes.POINTER(sz)]
        L.dirotq_prepare_layer_sibling.argtypes = [vp, i, i, vp, i, vp, i, i, i, i, i, vp, sz, vp, sz, vp, ctypes.POINTER(vp)]
        L.dirotq_layer_bytes_ph.argtypes = [i, i, i, i, ctypes.POINTER(sz)]
        L.dirotq_prepare_scratch_bytes_ph.argtypes = [i, i, i, ctypes.POINTER(sz)]
        L.dirotq_prepare_layer_ph.argtypes = [vp, i, i, vp, i, vp, i, i, i, i, vp, sz, vp, sz, vp, ctypes.POINTER(vp)]
        L.dirotq_layer_export_uh.argtypes = [vp, vp, vp]
        L.dirotq_layer_export_v.argtypes = [vp, vp, vp]
        L.dirotq_layer_bytes_nvfp4_ph.argtypes = [i, i, i, ctypes.POINTER(sz)]
        L.dirotq_prepare_layer_nvfp4_ph.argtypes = [vp, i, i, vp, i, vp, i, i, i, i, vp, sz, vp, sz, vp, ctypes.POINTER(vp)]
        L.dirotq_set_gemm_tile.argtypes = [i]
        L.dirotq_set_dependent_launch.argtypes = [i]
        L.dirotq_set_rotation_tile.argtypes = [i]
        L.dirotq_set_first_step_split.argtypes = [i]
        L.dirotq_prepare_scratch_bytes_gptq.argtypes = [i, i, i, i, psz]
        L.dirotq_prepare_layer_gptq.argtypes = [vp, i, i, vp, i, vp, vp, i, ctypes.c_double, i, i, i, i, i, i, vp, sz, vp, sz,
                                                vp, ctypes.POINTER(vp)]
        L.dirotq_prepare_layer_codes.argtypes = [vp, i, i, vp, i, vp, vp, vp, i, i, i, i, i, vp, sz, vp, sz, vp,
                                                 ctypes.POINTER(vp)]
        L.dirotq_workspace_export_asym.argtypes = [vp, i, vp, vp, vp, vp, vp, vp]
        L.dirotq_layer_export_zero_term.argtypes = [vp, vp, vp]
        for name in EXPORTED:
            if name not in ("dirotq_status_string", "dirotq_version", "dirotq_last_error"):
                getattr(L, name).restype = i
        _lib = L
    return _lib


def _check(st: int, where: str):
    if st != DIROTQ_OK:
        raise DirotqError(st, where, lib().dirotq_last_error().decode())


def _stream(stream=None) -> int:
    s = torch.cuda.current_stream() if stream is None else stream
    return s.cuda_stream


def _ptr(t):
    return None if t is None else t.data_ptr()


def dirotq_layer_bytes(K: int, N: int, r: int, group: int) -> int:
    out = ctypes.c_size_t(0)
    _check(lib().dirotq_layer_bytes(K, N, r, group, ctypes.byref(out)), "dirotq_layer_bytes")
    return out.value


def dirotq_prepare_scratch_bytes(K: int, N: int) -> int:
    out = ctypes.c_size_t(0)
    _check(lib().dirotq_prepare_scratch_bytes(K, N, ctypes.byref(out)), "dirotq_prepare_scratch_bytes")
    return out.value


class Layer:
    """Owner of one prepared layer: the device blob (a torch uint8 tensor) and the host handle."""

    def __init__(self, handle: int, blob: torch.Tensor, K: int, N: int, r: int, group: int, fmt: str = "int4"):
        self.handle, self.blob = handle, blob
        self.K, self.N, self.r, self.group = K, N, r, group
        self.fmt = fmt
        self.K_l = K if fmt in ("int4_ph", "nvfp4_ph") else K - r      # projection form: all K residual coefficients are low-precision
        self.n_g = -(-self.K_l // group)
        self.K_lp = self.n_g * group

    def close(self):
        if self.handle:
            lib().dirotq_layer_destroy(self.handle)
            self.handle = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass


def _alloc_bytes(nbytes: int, device, zero: bool = False) -> torch.Tensor:
    # torch's caching allocator returns 512-byte aligned blocks; over-allocate to align to 1024
    f = torch.zeros if zero else torch.empty
    raw = f(nbytes + 1024, dtype=torch.uint8, device=device)
    off = (-raw.data_ptr()) % 1024
    return raw[off:off + nbytes]


def dirotq_prepare_layer(W: torch.Tensor, Q: torch.Tensor, r: int, group: int, bias: torch.Tensor | None = None,
                         w_layout: int = LAYOUT_KN, stream=None) -> Layer:
    """W: cuda float32/bfloat16 [K,N] (or [N,K] with LAYOUT_NK); Q: cuda float64/float32 [K,K]; bias: cuda bf16 [N]."""
    assert W.is_cuda and Q.is_cuda and W.is_contiguous() and Q.is_contiguous()
    K = Q.shape[0]
    N = W.shape[1] if w_layout == LAYOUT_KN else W.shape[0]
    w_dtype = {torch.float32: DTYPE_F32, torch.bfloat16: DTYPE_BF16}[W.dtype]
    q_dtype = {torch.float64: DTYPE_F64, torch.float32: DTYPE_F32}[Q.dtype]
    blob = _alloc_bytes(dirotq_layer_bytes(K, N, r, group), W.device)
    scratch_bytes = dirotq_prepare_scratch_bytes(K, N)
    scratch = _alloc_bytes(scratch_bytes, W.device)
    handle = ctypes.c_void_p(0)
    st = lib().dirotq_prepare_layer(_ptr(W), w_dtype, w_layout, _ptr(Q), q_dtype, _ptr(bias), K, N, r, group,
                                    blob.data_ptr(), blob.numel(), scratch.data_ptr(), scratch_bytes, _stream(stream),
                                    ctypes.byref(handle))
    _check(st, "dirotq_prepare_layer")
    torch.cuda.current_stream().synchronize()  # scratch is released when this function returns
    return Layer(handle.value, blob, K, N, r, group)


def dirotq_workspace_bytes(layer: Layer, M: int) -> int:
    out = ctypes.c_size_t(0)
    _check(lib().dirotq_workspace_bytes(layer.handle, M, ctypes.byref(out)), "dirotq_workspace_bytes")
    return out.value


def alloc_workspace(layer: Layer, M: int) -> torch.Tensor:
    return _alloc_bytes(dirotq_workspace_bytes(layer, M), layer.blob.device, zero=True)


def dirotq_linear(x: torch.Tensor, layer: Layer, y: torch.Tensor, workspace: torch.Tensor, stream=None) -> None:
    M = x.shape[0]
    _check(lib().dirotq_linear(x.data_ptr(), M, layer.handle, y.data_ptr(), workspace.data_ptr(), workspace.numel(),
                               _stream(stream)), "dirotq_linear")


def dirotq_linear_host(x_host: torch.Tensor, layer: Layer, y_host: torch.Tensor, x_dev: torch.Tensor,
                       y_dev: torch.Tensor, workspace: torch.Tensor, stream=None) -> None:
    M = x_host.shape[0]
    _check(lib().dirotq_linear_host(x_host.data_ptr(), M, layer.handle, y_host.data_ptr(), x_dev.data_ptr(),
                                    y_dev.data_ptr(), workspace.data_ptr(), workspace.numel(), _stream(stream)),
           "dirotq_linear_host")


def dirotq_workspace_status(workspace: torch.Tensor, stream=None) -> int:
    code = ctypes.c_int(0)
    st = lib().dirotq_workspace_status(workspace.data_ptr(), _stream(stream), ctypes.byref(code))
    if st not in (0, 6):
        _check(st, "dirotq_workspace_status")
    return code.value


def dirotq_rotate_quantize(x: torch.Tensor, layer: Layer, workspace: torch.Tensor, xrot: torch.Tensor | None = None,
                           stream=None) -> None:
    _check(lib().dirotq_rotate_quantize(x.data_ptr(), x.shape[0], layer.handle, workspace.data_ptr(),
                                        workspace.numel(), _ptr(xrot), _stream(stream)), "dirotq_rotate_quantize")


def dirotq_w4a4_gemm(M: int, layer: Layer, workspace: torch.Tensor, y: torch.Tensor, stream=None) -> None:
    _check(lib().dirotq_w4a4_gemm(M, layer.handle, workspace.data_ptr(), workspace.numel(), y.data_ptr(),
                                  _stream(stream)), "dirotq_w4a4_gemm")


WAIT_COUNTER_NAMES = ("producer_wait_stage", "mma_wait_operands", "mma_wait_accumulator", "unpack_wait_tma",
                      "epilogue_wait_accumulator", "epilogue_wait_scales", "epilogue_total", "mma_role_total")


def dirotq_workspace_wait_counters(workspace: torch.Tensor, stream=None) -> dict:
    """Per-role blocked-cycle counters of the W4A4 kernel (summed over CTAs and calls since the workspace was zeroed)."""
    out = (ctypes.c_ulonglong * 8)()
    _check(lib().dirotq_workspace_wait_counters(workspace.data_ptr(), _stream(stream), out),
           "dirotq_workspace_wait_counters")
    return dict(zip(WAIT_COUNTER_NAMES, [int(v) for v in out]))


def dirotq_workspace_export(layer: Layer, M: int, workspace: torch.Tensor, stream=None):
    dev = workspace.device
    xh = torch.empty((M, layer.r), dtype=torch.bfloat16, device=dev)
    codes = torch.empty((M, layer.K_l), dtype=torch.int8, device=dev)
    scales = torch.empty((M, layer.n_g), dtype=torch.bfloat16, device=dev)
    _check(lib().dirotq_workspace_export(layer.handle, M, workspace.data_ptr(), xh.data_ptr(), codes.data_ptr(),
                                         scales.data_ptr(), _stream(stream)), "dirotq_workspace_export")
    return xh, codes, scales


def dirotq_int_gemm_debug(act_codes: torch.Tensor, layer: Layer, workspace: torch.Tensor, stream=None) -> torch.Tensor:
    """act_codes: cuda int8 [M, K_lp] (zero in columns >= K - r).  Returns int32 [n_g, M, N]."""
    M = act_codes.shape[0]
    assert act_codes.shape[1] == layer.K_lp and act_codes.is_contiguous()
    P = torch.empty((1 if layer.fmt == "w4a8" else layer.n_g, M, layer.N), dtype=torch.int32, device=act_codes.device)
    _check(lib().dirotq_int_gemm_debug(act_codes.data_ptr(), M, layer.handle, P.data_ptr(), workspace.data_ptr(),
                                       workspace.numel(), _stream(stream)), "dirotq_int_gemm_debug")
    return P


def dirotq_layer_export(layer: Layer, stream=None):
    dev = layer.blob.device
    wcodes = torch.empty((layer.K_l, layer.N), dtype=torch.int8, device=dev)
    wscales = torch.empty((1 if layer.fmt == "w4a8" else layer.n_g, layer.N), dtype=torch.bfloat16, device=dev)
    wh = torch.empty((layer.r, layer.N), dtype=torch.bfloat16, device=dev)
    qb = torch.empty((layer.K, layer.K), dtype=torch.bfloat16, device=dev)
    _check(lib().dirotq_layer_export(layer.handle, wcodes.data_ptr(), wscales.data_ptr(), wh.data_ptr(), qb.data_ptr(),
                                     _stream(stream)), "dirotq_layer_export")
    return wcodes, wscales, wh, qb


def dirotq_mma_rate_probe(kind: int, iters: int = 20000, stream=None) -> float:
    """Measured tensor-pipe rate in tera-ops/s.  kind 0: int8 (kind::i8), 1: bf16 (kind::f16), 2: E4M3 (kind::f8f6f4)."""
    status = torch.zeros(64, dtype=torch.int32, device="cuda")
    out = ctypes.c_float(0.0)
    _check(lib().dirotq_mma_rate_probe(kind, iters, status.data_ptr(), ctypes.byref(out), _stream(stream)),
           "dirotq_mma_rate_probe")
    if int(status[0].item()) != 0:
        raise DirotqError(6, "dirotq_mma_rate_probe")
    return float(out.value)


def dirotq_act_scale_log2_from_rotated(xrot: torch.Tensor, r: int, stream=None) -> int:
    """Exponent of the NVFP4 activations' power-of-two scale from fp32 rotated calibration activations [M, K]."""
    assert xrot.is_cuda and xrot.is_contiguous() and xrot.dtype == torch.float32
    word = torch.zeros(1, dtype=torch.int32, device=xrot.device)
    out = ctypes.c_int(0)
    _check(lib().dirotq_act_scale_log2_from_rotated(xrot.data_ptr(), xrot.shape[0], xrot.shape[1], int(r), word.data_ptr(),
                                                    ctypes.byref(out), _stream(stream)), "dirotq_act_scale_log2_from_rotated")
    return out.value


def dirotq_act_scale_log2_ph(x: torch.Tensor, Uh: torch.Tensor, stream=None) -> int:
    """Projection form: the same exponent from calibration tokens x (bf16 [M, K]) and U_h ([K, r], f64 or f32)."""
    assert x.is_cuda and x.is_contiguous() and x.dtype == torch.bfloat16 and Uh.is_cuda and Uh.is_contiguous()
    uh_dtype = {torch.float64: DTYPE_F64, torch.float32: DTYPE_F32}[Uh.dtype]
    K, r = Uh.shape
    scratch = torch.empty(16 + 4 * r * K, dtype=torch.uint8, device=x.device)
    out = ctypes.c_int(0)
    _check(lib().dirotq_act_scale_log2_ph(x.data_ptr(), x.shape[0], Uh.data_ptr(), uh_dtype, K, r, scratch.data_ptr(),
                                          scratch.numel(), ctypes.byref(out), _stream(stream)), "dirotq_act_scale_log2_ph")
    return out.value


def dirotq_wait_selftest(workspace: torch.Tensor, limit_us: int = 1000, stream=None) -> None:
    """Runs the bounded-wait give-up path on purpose (see the header); the status word of `workspace` then reads 5."""
    _check(lib().dirotq_wait_selftest(workspace.data_ptr(), int(limit_us), _stream(stream)), "dirotq_wait_selftest")


def dirotq_linear_noalloc(x: torch.Tensor, layer: Layer, y: torch.Tensor, device_status: torch.Tensor | None = None,
                          stream=None) -> None:
    """dirotq_linear on the library's built-in 16 MiB workspace: for callers that may not allocate.

    device_status: optional cuda int32 tensor (1 element) that receives this call's device status word."""
    _check(lib().dirotq_linear_noalloc(x.data_ptr(), x.shape[0], layer.handle, y.data_ptr(), _ptr(device_status),
                                       _stream(stream)), "dirotq_linear_noalloc")


# ------------------------------------------------------------------ NVFP4 variant

def dirotq_layer_bytes_nvfp4(K: int, N: int, r: int) -> int:
    out = ctypes.c_size_t(0)
    _check(lib().dirotq_layer_bytes_nvfp4(K, N, r, ctypes.byref(out)), "dirotq_layer_bytes_nvfp4")
    return out.value


def dirotq_prepare_layer_nvfp4(W: torch.Tensor, Q: torch.Tensor, r: int, act_scale_log2: int,
                               bias: torch.Tensor | None = None, w_layout: int = LAYOUT_KN, stream=None) -> Layer:
    """As dirotq_prepare_layer, for the NVFP4 format; act_scale_log2 is the activations' calibrated exponent."""
    assert W.is_cuda and Q.is_cuda and W.is_contiguous() and Q.is_contiguous()
    K = Q.shape[0]
    N = W.shape[1] if w_layout == LAYOUT_KN else W.shape[0]
    w_dtype = {torch.float32: DTYPE_F32, torch.bfloat16: DTYPE_BF16}[W.dtype]
    q_dtype = {torch.float64: DTYPE_F64, torch.float32: DTYPE_F32}[Q.dtype]
    blob = _alloc_bytes(dirotq_layer_bytes_nvfp4(K, N, r), W.device, zero=True)
    scratch_bytes = dirotq_prepare_scratch_bytes(K, N)
    scratch = _alloc_bytes(scratch_bytes, W.device)
    handle = ctypes.c_void_p(0)
    st = lib().dirotq_prepare_layer_nvfp4(_ptr(W), w_dtype, w_layout, _ptr(Q), q_dtype, _ptr(bias), K, N, r,
                                          int(act_scale_log2), blob.data_ptr(), blob.numel(), scratch.data_ptr(),
                                          scratch_bytes, _stream(stream), ctypes.byref(handle))
    _check(st, "dirotq_prepare_layer_nvfp4")
    torch.cuda.current_stream().synchronize()
    return Layer(handle.value, blob, K, N, r, 16, fmt="nvfp4")


def dirotq_workspace_export_nvfp4(layer: Layer, M: int, workspace: torch.Tensor, stream=None):
    dev = workspace.device
    nb = -(-layer.K_l // 16)
    xh = torch.empty((M, layer.r), dtype=torch.bfloat16, device=dev)
    codes = torch.empty((M, layer.K_l), dtype=torch.uint8, device=dev)
    scales = torch.empty((M, nb), dtype=torch.uint8, device=dev)
    _check(lib().dirotq_workspace_export_nvfp4(layer.handle, M, workspace.data_ptr(), xh.data_ptr(), codes.data_ptr(),
                                               scales.data_ptr(), _stream(stream)), "dirotq_workspace_export_nvfp4")
    return xh, codes, scales


def dirotq_layer_export_nvfp4(layer: Layer, stream=None):
    dev = layer.blob.device
    nb = -(-layer.K_l // 16)
    wcodes = torch.empty((layer.K_l, layer.N), dtype=torch.uint8, device=dev)
    wscales = torch.empty((nb, layer.N), dtype=torch.uint8, device=dev)
    wh = torch.empty((layer.r, layer.N), dtype=torch.bfloat16, device=dev)
    # the projection form holds U_hb instead of a K x K rotation: returned in the rotation's place
    qb = None if layer.fmt == "nvfp4_ph" else torch.empty((layer.K, layer.K), dtype=torch.bfloat16, device=dev)
    ew = torch.zeros(1, dtype=torch.int32, device=dev)
    _check(lib().dirotq_layer_export_nvfp4(layer.handle, wcodes.data_ptr(), wscales.data_ptr(), wh.data_ptr(),
                                           _ptr(qb), ew.data_ptr(), _stream(stream)), "dirotq_layer_export_nvfp4")
    if qb is None:
        qb = dirotq_layer_export_uh(layer, stream)
    return wcodes, wscales, wh, qb, int(ew.item())


# ------------------------------------------------------------------ asymmetric activation codes

def dirotq_layer_bytes_asym(K: int, N: int, r: int, group: int) -> int:
    out = ctypes.c_size_t(0)
    _check(lib().dirotq_layer_bytes_asym(K, N, r, group, ctypes.byref(out)), "dirotq_layer_bytes_asym")
    return out.value


def dirotq_prepare_layer_asym(W: torch.Tensor, Q: torch.Tensor, r: int, group: int, bias: torch.Tensor | None = None,
                              w_layout: int = LAYOUT_KN, stream=None) -> Layer:
    """As dirotq_prepare_layer, for a layer whose activations are quantized asymmetrically (codes 0..15, zero-point)."""
    assert W.is_cuda and Q.is_cuda and W.is_contiguous() and Q.is_contiguous()
    K = Q.shape[0]
    N = W.shape[1] if w_layout == LAYOUT_KN else W.shape[0]
    w_dtype = {torch.float32: DTYPE_F32, torch.bfloat16: DTYPE_BF16}[W.dtype]
    q_dtype = {torch.float64: DTYPE_F64, torch.float32: DTYPE_F32}[Q.dtype]
    blob = _alloc_bytes(dirotq_layer_bytes_asym(K, N, r, group), W.device)
    scratch_bytes = dirotq_prepare_scratch_bytes(K, N)
    scratch = _alloc_bytes(scratch_bytes, W.device)
    handle = ctypes.c_void_p(0)
    st = lib().dirotq_prepare_layer_asym(_ptr(W), w_dtype, w_layout, _ptr(Q), q_dtype, _ptr(bias), K, N, r, group,
                                         blob.data_ptr(), blob.numel(), scratch.data_ptr(), scratch_bytes, _stream(stream),
                                         ctypes.byref(handle))
    _check(st, "dirotq_prepare_layer_asym")
    torch.cuda.current_stream().synchronize()
    return Layer(handle.value, blob, K, N, r, group, fmt="int4_asym")


def dirotq_layer_bytes_sibling(K: int, N: int, r: int, group: int, asym: bool = False) -> int:
    out = ctypes.c_size_t(0)
    _check(lib().dirotq_layer_bytes_sibling(K, N, r, group, int(asym), ctypes.byref(out)), "dirotq_layer_bytes_sibling")
    return out.value


def dirotq_prepare_layer_sibling(W: torch.Tensor, Q: torch.Tensor, r: int, group: int, bias: torch.Tensor | None = None,
                                 asym: bool = False, w_layout: int = LAYOUT_KN, stream=None) -> Layer:
    """A layer without its own copy of the rotation: used through dirotq_w4a4_gemm on a sibling's rotated workspace."""
    assert W.is_cuda and Q.is_cuda and W.is_contiguous() and Q.is_contiguous()
    K = Q.shape[0]
    N = W.shape[1] if w_layout == LAYOUT_KN else W.shape[0]
    w_dtype = {torch.float32: DTYPE_F32, torch.bfloat16: DTYPE_BF16}[W.dtype]
    q_dtype = {torch.float64: DTYPE_F64, torch.float32: DTYPE_F32}[Q.dtype]
    blob = _alloc_bytes(dirotq_layer_bytes_sibling(K, N, r, group, asym), W.device)
    scratch_bytes = dirotq_prepare_scratch_bytes(K, N)
    scratch = _alloc_bytes(scratch_bytes, W.device)
    handle = ctypes.c_void_p(0)
    st = lib().dirotq_prepare_layer_sibling(_ptr(W), w_dtype, w_layout, _ptr(Q), q_dtype, _ptr(bias), int(asym), K, N, r, group,
                                            blob.data_ptr(), blob.numel(), scratch.data_ptr(), scratch_bytes, _stream(stream),
                                            ctypes.byref(handle))
    _check(st, "dirotq_prepare_layer_sibling")
    torch.cuda.current_stream().synchronize()
    return Layer(handle.value, blob, K, N, r, group, fmt="int4_asym" if asym else "int4")


def dirotq_prepare_layer_ph(W: torch.Tensor, Uh: torch.Tensor, group: int, bias: torch.Tensor | None = None,
                            w_layout: int = LAYOUT_KN, stream=None) -> Layer:
    """Projection form: Uh [K, r] (fp64 or fp32, row-major) is the only dense part of the first stage."""
    assert W.is_cuda and Uh.is_cuda and W.is_contiguous() and Uh.is_contiguous()
    K, r = Uh.shape
    N = W.shape[1] if w_layout == LAYOUT_KN else W.shape[0]
    w_dtype = {torch.float32: DTYPE_F32, torch.bfloat16: DTYPE_BF16}[W.dtype]
    uh_dtype = {torch.float64: DTYPE_F64, torch.float32: DTYPE_F32}[Uh.dtype]
    nb, ns = ctypes.c_size_t(0), ctypes.c_size_t(0)
    _check(lib().dirotq_layer_bytes_ph(K, N, r, group, ctypes.byref(nb)), "dirotq_layer_bytes_ph")
    _check(lib().dirotq_prepare_scratch_bytes_ph(K, N, r, ctypes.byref(ns)), "dirotq_prepare_scratch_bytes_ph")
    blob = _alloc_bytes(nb.value, W.device)
    scratch = _alloc_bytes(ns.value, W.device)
    handle = ctypes.c_void_p(0)
    st = lib().dirotq_prepare_layer_ph(_ptr(W), w_dtype, w_layout, _ptr(Uh), uh_dtype, _ptr(bias), K, N, r, group,
                                       blob.data_ptr(), blob.numel(), scratch.data_ptr(), ns.value, _stream(stream),
                                       ctypes.byref(handle))
    _check(st, "dirotq_prepare_layer_ph")
    torch.cuda.current_stream().synchronize()
    return Layer(handle.value, blob, K, N, r, group, fmt="int4_ph")


def dirotq_prepare_layer_nvfp4_ph(W: torch.Tensor, Uh: torch.Tensor, act_scale_log2: int, bias: torch.Tensor | None = None,
                                  w_layout: int = LAYOUT_KN, stream=None) -> Layer:
    """Projection form with NVFP4 operands."""
    assert W.is_cuda and Uh.is_cuda and W.is_contiguous() and Uh.is_contiguous()
    K, r = Uh.shape
    N = W.shape[1] if w_layout == LAYOUT_KN else W.shape[0]
    w_dtype = {torch.float32: DTYPE_F32, torch.bfloat16: DTYPE_BF16}[W.dtype]
    uh_dtype = {torch.float64: DTYPE_F64, torch.float32: DTYPE_F32}[Uh.dtype]
    nb, ns = ctypes.c_size_t(0), ctypes.c_size_t(0)
    _check(lib().dirotq_layer_bytes_nvfp4_ph(K, N, r, ctypes.byref(nb)), "dirotq_layer_bytes_nvfp4_ph")
    _check(lib().dirotq_prepare_scratch_bytes_ph(K, N, r, ctypes.byref(ns)), "dirotq_prepare_scratch_bytes_ph")
    blob = _alloc_bytes(nb.value, W.device)
    scratch = _alloc_bytes(ns.value, W.device)
    handle = ctypes.c_void_p(0)
    st = lib().dirotq_prepare_layer_nvfp4_ph(_ptr(W), w_dtype, w_layout, _ptr(Uh), uh_dtype, _ptr(bias), K, N, r,
                                             int(act_scale_log2), blob.data_ptr(), blob.numel(), scratch.data_ptr(), ns.value,
                                             _stream(stream), ctypes.byref(handle))
    _check(st, "dirotq_prepare_layer_nvfp4_ph")
    torch.cuda.current_stream().synchronize()
    return Layer(handle.value, blob, K, N, r, 16, fmt="nvfp4_ph")


def dirotq_layer_export_uh(layer: Layer, stream=None) -> torch.Tensor:
    uh = torch.empty((layer.K, layer.r), dtype=torch.bfloat16, device=layer.blob.device)
    _check(lib().dirotq_layer_export_uh(layer.handle, uh.data_ptr(), _stream(stream)), "dirotq_layer_export_uh")
    return uh


def dirotq_layer_export_v(layer: Layer, stream=None) -> torch.Tensor:
    """V = bf16(U_hb^T H+-) [r, K] of a projection-form layer."""
    v = torch.empty((layer.r, layer.K), dtype=torch.bfloat16, device=layer.blob.device)
    _check(lib().dirotq_layer_export_v(layer.handle, v.data_ptr(), _stream(stream)), "dirotq_layer_export_v")
    return v


def dirotq_set_gemm_tile(columns: int) -> None:
    """Output columns per tile of the INT4 and NVFP4 second kernels: 0 automatic, 128 or 256 forced (process-wide)."""
    _check(lib().dirotq_set_gemm_tile(int(columns)), "dirotq_set_gemm_tile")


def dirotq_set_rotation_tile(plan: int) -> None:
    """Tile plan of the rotation kernel: 0 automatic, 1 = 128x128, 2 = 128x256, 3 = 256x256, 4 = 256x256 per pair of CTAs sharing
    every MMA (process-wide)."""
    _check(lib().dirotq_set_rotation_tile(int(plan)), "dirotq_set_rotation_tile")


def dirotq_set_first_step_split(enabled: bool) -> None:
    """Projection form: split the first step's reduction over K into ranges when there are few row tiles (default on)."""
    _check(lib().dirotq_set_first_step_split(int(bool(enabled))), "dirotq_set_first_step_split")


def dirotq_set_dependent_launch(enabled: bool) -> None:
    """Programmatic dependent launch of each layer's second kernel: on (default) or off, process-wide."""
    _check(lib().dirotq_set_dependent_launch(int(bool(enabled))), "dirotq_set_dependent_launch")


def dirotq_prepare_layer_codes(W: torch.Tensor, Q: torch.Tensor, wcodes: torch.Tensor, wscales: torch.Tensor, r: int,
                               group: int, bias: torch.Tensor | None = None, asym: bool = False,
                               w_layout: int = LAYOUT_KN, stream=None) -> Layer:
    """As dirotq_prepare_layer(_asym), with the residual codes int8 [K-r,N] and bf16 scales [n_g,N] given by the caller."""
    assert W.is_cuda and Q.is_cuda and W.is_contiguous() and Q.is_contiguous()
    K = Q.shape[0]
    N = W.shape[1] if w_layout == LAYOUT_KN else W.shape[0]
    n_g = -(-(K - r) // group)
    assert wcodes.is_cuda and wcodes.is_contiguous() and wcodes.dtype == torch.int8 and tuple(wcodes.shape) == (K - r, N)
    assert wscales.is_cuda and wscales.is_contiguous() and wscales.dtype == torch.bfloat16 and tuple(wscales.shape) == (n_g, N)
    w_dtype = {torch.float32: DTYPE_F32, torch.bfloat16: DTYPE_BF16}[W.dtype]
    q_dtype = {torch.float64: DTYPE_F64, torch.float32: DTYPE_F32}[Q.dtype]
    nbytes = dirotq_layer_bytes_asym(K, N, r, group) if asym else dirotq_layer_bytes(K, N, r, group)
    blob = _alloc_bytes(nbytes, W.device)
    scratch_bytes = dirotq_prepare_scratch_bytes(K, N)
    scratch = _alloc_bytes(scratch_bytes, W.device)
    handle = ctypes.c_void_p(0)
    st = lib().dirotq_prepare_layer_codes(_ptr(W), w_dtype, w_layout, _ptr(Q), q_dtype, _ptr(bias), wcodes.data_ptr(),
                                          wscales.data_ptr(), int(asym), K, N, r, group, blob.data_ptr(), blob.numel(),
                                          scratch.data_ptr(), scratch_bytes, _stream(stream), ctypes.byref(handle))
    _check(st, "dirotq_prepare_layer_codes")
    torch.cuda.current_stream().synchronize()
    return Layer(handle.value, blob, K, N, r, group, fmt="int4_asym" if asym else "int4")


def dirotq_prepare_layer_gptq(W: torch.Tensor, Q: torch.Tensor, calib_x: torch.Tensor, r: int, group: int,
                              bias: torch.Tensor | None = None, asym: bool = False, damp: float = 0.01, block: int = 128,
                              w_layout: int = LAYOUT_KN, stream=None) -> Layer:
    """As dirotq_prepare_layer(_asym), with the residual rows rounded by GPTQ on the calibration tokens calib_x (bf16 [T,K])."""
    assert W.is_cuda and Q.is_cuda and W.is_contiguous() and Q.is_contiguous()
    K = Q.shape[0]
    N = W.shape[1] if w_layout == LAYOUT_KN else W.shape[0]
    assert calib_x.is_cuda and calib_x.is_contiguous() and calib_x.dtype == torch.bfloat16 and calib_x.shape[1] == K
    w_dtype = {torch.float32: DTYPE_F32, torch.bfloat16: DTYPE_BF16}[W.dtype]
    q_dtype = {torch.float64: DTYPE_F64, torch.float32: DTYPE_F32}[Q.dtype]
    nbytes = dirotq_layer_bytes_asym(K, N, r, group) if asym else dirotq_layer_bytes(K, N, r, group)
    blob = _alloc_bytes(nbytes, W.device)
    need = ctypes.c_size_t(0)
    _check(lib().dirotq_prepare_scratch_bytes_gptq(K, N, r, calib_x.shape[0], ctypes.byref(need)), "dirotq_prepare_scratch_bytes_gptq")
    scratch = _alloc_bytes(need.value, W.device)
    handle = ctypes.c_void_p(0)
    st = lib().dirotq_prepare_layer_gptq(_ptr(W), w_dtype, w_layout, _ptr(Q), q_dtype, _ptr(bias), calib_x.data_ptr(),
                                         calib_x.shape[0], float(damp), int(block), int(asym), K, N, r, group, blob.data_ptr(),
                                         blob.numel(), scratch.data_ptr(), need.value, _stream(stream), ctypes.byref(handle))
    _check(st, "dirotq_prepare_layer_gptq")
    torch.cuda.current_stream().synchronize()
    return Layer(handle.value, blob, K, N, r, group, fmt="int4_asym" if asym else "int4")


def dirotq_workspace_export_asym(layer: Layer, M: int, workspace: torch.Tensor, stream=None):
    dev = workspace.device
    xh = torch.empty((M, layer.r), dtype=torch.bfloat16, device=dev)
    codes = torch.empty((M, layer.K_l), dtype=torch.uint8, device=dev)
    scales = torch.empty((M, layer.n_g), dtype=torch.bfloat16, device=dev)
    zeros = torch.empty((M, layer.n_g), dtype=torch.bfloat16, device=dev)
    _check(lib().dirotq_workspace_export_asym(layer.handle, M, workspace.data_ptr(), xh.data_ptr(), codes.data_ptr(),
                                              scales.data_ptr(), zeros.data_ptr(), _stream(stream)),
           "dirotq_workspace_export_asym")
    return xh, codes, scales, zeros


def dirotq_layer_export_zero_term(layer: Layer, stream=None) -> torch.Tensor:
    d = torch.empty((layer.n_g, layer.N), dtype=torch.float32, device=layer.blob.device)
    _check(lib().dirotq_layer_export_zero_term(layer.handle, d.data_ptr(), _stream(stream)), "dirotq_layer_export_zero_term")
    return d


# ------------------------------------------------------------------ W4A8

def dirotq_layer_bytes_w4a8(K: int, N: int, r: int) -> int:
    out = ctypes.c_size_t(0)
    _check(lib().dirotq_layer_bytes_w4a8(K, N, r, ctypes.byref(out)), "dirotq_layer_bytes_w4a8")
    return out.value


def dirotq_prepare_layer_w4a8(W: torch.Tensor, Q: torch.Tensor, r: int, bias: torch.Tensor | None = None,
                              w_layout: int = LAYOUT_KN, stream=None) -> Layer:
    """Per-token INT8 activations, per-channel INT4 weights (Layer.group is the packing granularity, 128)."""
    assert W.is_cuda and Q.is_cuda and W.is_contiguous() and Q.is_contiguous()
    K = Q.shape[0]
    N = W.shape[1] if w_layout == LAYOUT_KN else W.shape[0]
    w_dtype = {torch.float32: DTYPE_F32, torch.bfloat16: DTYPE_BF16}[W.dtype]
    q_dtype = {torch.float64: DTYPE_F64, torch.float32: DTYPE_F32}[Q.dtype]
    blob = _alloc_bytes(dirotq_layer_bytes_w4a8(K, N, r), W.device)
    scratch_bytes = dirotq_prepare_scratch_bytes(K, N)
    scratch = _alloc_bytes(scratch_bytes, W.device)
    handle = ctypes.c_void_p(0)
    st = lib().dirotq_prepare_layer_w4a8(_ptr(W), w_dtype, w_layout, _ptr(Q), q_dtype, _ptr(bias), K, N, r, blob.data_ptr(),
                                         blob.numel(), scratch.data_ptr(), scratch_bytes, _stream(stream),
                                         ctypes.byref(handle))
    _check(st, "dirotq_prepare_layer_w4a8")
    torch.cuda.current_stream().synchronize()
    return Layer(handle.value, blob, K, N, r, 128, fmt="w4a8")


def dirotq_workspace_export_w4a8(layer: Layer, M: int, workspace: torch.Tensor, stream=None):
    dev = workspace.device
    xh = torch.empty((M, layer.r), dtype=torch.bfloat16, device=dev)
    codes = torch.empty((M, layer.K_l), dtype=torch.int8, device=dev)
    scales = torch.empty((M,), dtype=torch.bfloat16, device=dev)
    _check(lib().dirotq_workspace_export_w4a8(layer.handle, M, workspace.data_ptr(), xh.data_ptr(), codes.data_ptr(),
                                              scales.data_ptr(), _stream(stream)), "dirotq_workspace_export_w4a8")
    return xh, codes, scales
