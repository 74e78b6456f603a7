"""The paper's own operating point keeps about a tenth of the rotated coefficients in 16 bits (Sec. 4.2, App. E):
ranks far above the 16..128 of the benchmark configurations, i.e. several 64-wide chunks on the bf16 branch and
several all-high tiles in the rotation kernel's epilogue."""
import pytest

from paper_2605_16732_b200 import synth

import test_gpu_asym
import test_gpu_nvfp4
import test_gpu_parity
import test_gpu_w4a8

pytestmark = pytest.mark.gpu


def test_int4_rank_a_quarter_of_k():
    spec = synth.LayerSpec(K=1024, N=512, r=256, G=64, model=synth.PIXART, seed=71, calib_tokens=1024)
    print(test_gpu_parity._run_case(spec, M=300))


def test_int4_flux_width_rank_320_group128():
    # K = 3072, r = 320 (10.4 %): K_l = 2752 = 21.5 groups of 128 -> ragged last group
    spec = synth.LayerSpec(K=3072, N=384, r=320, G=128, model=synth.FLUX, seed=72)
    print(test_gpu_parity._run_case(spec, M=200, check_rot=False))


def test_int4_rank_not_a_multiple_of_64():
    spec = synth.LayerSpec(K=1152, N=640, r=112, G=64, model=synth.PIXART, seed=73)
    print(test_gpu_parity._run_case(spec, M=257, with_bias=False))


def test_asym_rank_192():
    spec = synth.LayerSpec(K=1024, N=400, r=192, G=64, model=synth.FLUX, seed=74, calib_tokens=1024)
    print(test_gpu_asym._run_case(spec, M=150, shift=1.0))


def test_nvfp4_rank_256():
    spec = synth.LayerSpec(K=1024, N=384, r=256, G=64, model=synth.PIXART, seed=75, calib_tokens=1024)
    print(test_gpu_nvfp4._run_case(spec, M=200))


def test_w4a8_rank_320():
    spec = synth.LayerSpec(K=1536, N=512, r=320, G=64, model=synth.FLUX, seed=76, calib_tokens=1024)
    print(test_gpu_w4a8._run_case(spec, M=190))
