"""Host-side checks of the C ABI that need no GPU: the library loads, exports every symbol the
header declares, and validates arguments before touching CUDA."""
import ctypes
import os
import re

import pytest

from paper_2605_16732_b200 import binding

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def L():
    from paper_2605_16732_b200 import build
    build.build()
    return binding.lib()


def test_every_declared_symbol_is_exported(L):
    header = open(os.path.join(ROOT, "include", "dirotq.h")).read()
    declared = sorted(set(re.findall(r"DIROTQ_API\s+[\w\s\*]+?\b(dirotq_\w+)\s*\(", header)))
    assert len(declared) >= 16
    assert sorted(binding.EXPORTED) == declared
    for name in declared:
        assert getattr(L, name) is not None


def test_status_strings(L):
    assert L.dirotq_status_string(0) == b"ok"
    assert L.dirotq_status_string(6) == b"device-side wait timed out"
    assert L.dirotq_version() >= 100


def test_layer_bytes_and_shape_validation(L):
    n = ctypes.c_size_t(0)
    assert L.dirotq_layer_bytes(1152, 1152, 32, 64, ctypes.byref(n)) == 0
    K, N, r, G = 1152, 1152, 32, 64
    n_g = -(-(K - r) // G)
    floor = K * K * 2 + N * n_g * G // 2 + n_g * N * 4 + N * 64 * 2 + N * 4
    assert floor <= n.value <= floor + 6 * 1024
    # unsupported shapes are refused
    for bad in [(1100, 1152, 32, 64), (1152, 1150, 32, 64), (1152, 1152, 24, 64), (1152, 1152, 32, 32),
                (12288, 1152, 4112, 64), (64, 64, 64, 64), (192, 64, 32, 128)]:
        assert L.dirotq_layer_bytes(*bad, ctypes.byref(n)) == 2, bad
    assert L.dirotq_layer_bytes(-1, 64, 32, 64, ctypes.byref(n)) == 1
    assert L.dirotq_layer_bytes(1152, 1152, 32, 64, None) == 1


def test_scratch_bytes(L):
    n = ctypes.c_size_t(0)
    assert L.dirotq_prepare_scratch_bytes(3072, 9216, ctypes.byref(n)) == 0
    assert n.value == 3072 * 9216 * 8


def test_null_and_bad_handles_are_rejected(L):
    n = ctypes.c_size_t(0)
    assert L.dirotq_workspace_bytes(None, 16, ctypes.byref(n)) == 1
    assert L.dirotq_layer_destroy(None) == 1
    assert L.dirotq_linear(None, 1, None, None, None, 0, None) == 1
    assert L.dirotq_rotate_quantize(None, 1, None, None, 0, None, None) == 1
    assert L.dirotq_int_gemm_debug(None, 1, None, None, None, 0, None) == 1
    assert L.dirotq_layer_export(None, None, None, None, None, None) == 1
    h = ctypes.c_void_p(0)
    # NULL tensors: refused before any CUDA call
    assert L.dirotq_prepare_layer(None, 0, 0, None, 2, None, 128, 64, 32, 64, None, 0, None, 0, None,
                                  ctypes.byref(h)) == 1
    # a fake handle (wrong magic) is refused too
    fake = ctypes.create_string_buffer(4096)
    assert L.dirotq_workspace_bytes(fake, 16, ctypes.byref(n)) == 1


def test_knobs_validate_their_argument_without_a_gpu(L):
    for ok in (0, 64, 66, 128, 192, 256, 512, 0):
        assert L.dirotq_set_gemm_tile(ok) == 0
    for bad in (-1, 96, 160, 384, 1024):
        assert L.dirotq_set_gemm_tile(bad) == 1
    assert L.dirotq_set_dependent_launch(0) == 0 and L.dirotq_set_dependent_launch(1) == 0
    assert L.dirotq_set_first_step_split(0) == 0 and L.dirotq_set_first_step_split(1) == 0


def test_prepare_from_codes_rejects_null_arguments(L):
    h = ctypes.c_void_p(0)
    # codes without scales (or neither) are refused before any CUDA call
    assert L.dirotq_prepare_layer_codes(None, 0, 0, None, 2, None, None, None, 0, 128, 64, 32, 64, None, 0, None, 0, None,
                                        ctypes.byref(h)) == 1
    assert not h.value


def test_sibling_layer_is_smaller_by_the_rotation(L):
    full, sib = ctypes.c_size_t(0), ctypes.c_size_t(0)
    for K, N, r, G, asym in [(1152, 1152, 32, 64, 0), (3072, 9216, 320, 128, 0), (1152, 4608, 112, 64, 1)]:
        fn = L.dirotq_layer_bytes_asym if asym else L.dirotq_layer_bytes
        assert fn(K, N, r, G, ctypes.byref(full)) == 0
        assert L.dirotq_layer_bytes_sibling(K, N, r, G, asym, ctypes.byref(sib)) == 0
        assert 0 <= full.value - sib.value - 2 * K * K <= 1024          # the bf16 rotation, up to the section alignment
    assert L.dirotq_layer_bytes_sibling(1100, 1152, 32, 64, 0, ctypes.byref(sib)) == 2


def test_memory_report_runs_without_a_gpu(capsys):
    import json
    from paper_2605_16732_b200 import suite
    suite.memory_report()
    rows = [json.loads(l) for l in capsys.readouterr().out.splitlines()]
    assert len(rows) == 18
    for row in rows:
        assert row["layer_bytes"] - row["layer_bytes_without_rotation"] >= 2 * row["K"] ** 2
        assert 2.5 < row["x_smaller_than_bf16_without_rotation"] < 3.6


def test_the_other_builds_export_the_same_interface():
    # the integer-path fallback and the diagnostic build are the same sources with one definition each: same symbols
    from paper_2605_16732_b200 import build
    for path in (build.build_i8(), build.build_trace()):
        other = ctypes.CDLL(path)
        for name in binding.EXPORTED:
            assert getattr(other, name) is not None, (path, name)
        other.dirotq_version.restype = ctypes.c_int
        assert other.dirotq_version() >= 100
