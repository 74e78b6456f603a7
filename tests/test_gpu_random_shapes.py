"""Seeded random sweep over shapes, formats, tile widths and launch modes: every case goes through the same
stage-by-stage parity protocol as the hand-picked ones.  Small cases cover ragged rows, columns and groups in all
combinations; the large-M cases give every CTA several tiles (more tiles than SMs)."""
import random

import pytest

from paper_2605_16732_b200 import binding as dq
from paper_2605_16732_b200 import synth

import test_gpu_asym
import test_gpu_nvfp4
import test_gpu_parity
import test_gpu_projection_form
import test_gpu_w4a8

pytestmark = pytest.mark.gpu


def _one(rng, big, fmt=None):
    fmt = fmt or rng.choice(["int4", "int4", "asym", "nvfp4", "w4a8", "ph"])
    if big:
        M = rng.choice([19000, 20001, 25000])
        K = 64 * rng.randint(2, 4)
        N = 16 * rng.randint(4, 30)
        r = 16 * rng.randint(1, 3)
    else:
        M = rng.choice([1, 7, 64, 128, 129, 200, 257, 300, 513, 700])
        K = 64 * rng.randint(2, 20)
        N = 16 * rng.randint(1, 60)
        r = 16 * rng.randint(1, max(1, min(K // 16 - 2, 20)))
    G = rng.choice([64, 128])
    if K % G:
        G = 64
    tile = rng.choice([0, 0, 128, 256])
    pdl = rng.choice([True, True, False])
    plan = rng.choice([0, 0, 1, 2, 3, 4])  # tile plan of the rotation kernel (4: CTA pairs)
    if not big and rng.random() < 0.3:
        r = 16 * rng.randint(1, max(1, K // 32))      # up to half of K in 16 bits
    bias = rng.random() < 0.7
    model = rng.choice([synth.PIXART, synth.FLUX])
    spec = synth.LayerSpec(K=K, N=N, r=r, G=G if fmt in ("int4", "asym", "ph") else 64, model=model, seed=rng.randint(1, 10 ** 6),
                           calib_tokens=max(512, 2 * K))
    desc = dict(fmt=fmt, M=M, K=K, N=N, r=r, G=spec.G, tile=tile, pdl=pdl, bias=bias, plan=plan)
    dq.dirotq_set_gemm_tile(tile)
    dq.dirotq_set_dependent_launch(pdl)
    dq.dirotq_set_rotation_tile(plan)
    try:
        if fmt == "int4":
            test_gpu_parity._run_case(spec, M=M, with_bias=bias, check_rot=not big)
        elif fmt == "asym":
            test_gpu_asym._run_case(spec, M=M, with_bias=bias, shift=rng.choice([0.0, 1.5]), check_rot=not big)
        elif fmt == "ph":
            test_gpu_projection_form._run_case(spec, M=M, with_bias=bias)
        elif fmt == "nvfp4_ph":
            test_gpu_projection_form._run_case_nvfp4(spec, M=M, with_bias=bias)
        elif fmt == "nvfp4":
            test_gpu_nvfp4._run_case(spec, M=M, with_bias=bias, check_rot=not big)
        else:
            test_gpu_w4a8._run_case(spec, M=M, with_bias=bias, check_rot=not big)
    except AssertionError as e:
        raise AssertionError(f"{desc}: {e}") from e
    finally:
        dq.dirotq_set_gemm_tile(0)
        dq.dirotq_set_dependent_launch(True)
        dq.dirotq_set_rotation_tile(0)


def test_random_small_shapes():
    rng = random.Random(20251)
    for _ in range(60):
        _one(rng, big=False)


def test_random_large_m_shapes():
    rng = random.Random(20252)
    for _ in range(6):
        _one(rng, big=True)


def test_random_nvfp4_projection_form_shapes():
    rng = random.Random(20253)
    for _ in range(25):
        _one(rng, big=False, fmt="nvfp4_ph")
    for _ in range(2):
        _one(rng, big=True, fmt="nvfp4_ph")
