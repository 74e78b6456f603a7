"""The INT4 second kernel with 64- (one epilogue warpgroup, for calls with few token rows), 128-, 192- (three epilogue warpgroups) and 256-column tiles: both forced through dirotq_set_gemm_tile, on shapes the
automatic choice would send one way only.  Parity with the oracle under each setting, and bit-equal outputs and
integer group sums between the two (every output element is accumulated in the same order)."""
import numpy as np
import pytest
import torch

from paper_2605_16732_b200 import binding as dq
from paper_2605_16732_b200 import synth

import test_gpu_asym
import test_gpu_parity
from parity_utils import bits_to_bf16_tensor

pytestmark = pytest.mark.gpu


@pytest.fixture
def tile(request):
    dq.dirotq_set_gemm_tile(request.param)
    yield request.param
    dq.dirotq_set_gemm_tile(0)


@pytest.mark.parametrize("tile", [64, 66, 128, 192, 256], indirect=True)
def test_parity_group64_ragged_everything(tile):
    # N = 400: ragged in both tile widths; M = 300: ragged rows; K_l = 496: ragged last group
    spec = synth.LayerSpec(K=512, N=400, r=16, G=64, model=synth.FLUX, seed=31, calib_tokens=1024)
    print(tile, test_gpu_parity._run_case(spec, M=300))


@pytest.mark.parametrize("tile", [64, 66, 128, 192, 256], indirect=True)
def test_parity_group128_rank128(tile):
    spec = synth.LayerSpec(K=768, N=640, r=128, G=128, model=synth.FLUX, seed=32, calib_tokens=1024)
    print(tile, test_gpu_parity._run_case(spec, M=257, with_bias=False))


@pytest.mark.parametrize("tile", [64, 66, 128, 192, 256], indirect=True)
def test_parity_pixart_projection_many_tiles(tile):
    # 8 row blocks x 9 (or 5) column blocks: several tiles per CTA are not reached on one GPU with 148 SMs, but the
    # tile -> (row block, column block) mapping and the ring phases across k-blocks are
    spec = synth.LayerSpec(K=1152, N=1152, r=32, G=64, model=synth.PIXART, seed=33)
    print(tile, test_gpu_parity._run_case(spec, M=1024, check_rot=False))


@pytest.mark.parametrize("tile", [64, 66, 128, 192, 256], indirect=True)
def test_parity_asymmetric_codes(tile):
    spec = synth.LayerSpec(K=640, N=400, r=32, G=64, model=synth.PIXART, seed=34, calib_tokens=1024)
    print(tile, test_gpu_asym._run_case(spec, M=200, shift=1.5))


def test_both_widths_give_the_same_bits_and_automatic_choice_is_one_of_them():
    spec = synth.LayerSpec(K=1152, N=1152, r=32, G=64, model=synth.PIXART, seed=35)
    M = 4096 + 77
    inp = synth.make_layer_inputs(spec, M, with_bias=True)
    dev = "cuda"
    layer = dq.dirotq_prepare_layer(torch.from_numpy(inp["W"]).to(dev), torch.from_numpy(inp["Q"]).to(dev), spec.r, spec.G,
                                    bias=bits_to_bf16_tensor(inp["bias"]))
    x = bits_to_bf16_tensor(inp["x"])
    ws = dq.alloc_workspace(layer, M)
    outs = {}
    try:
        for cols in (0, 64, 66, 128, 192, 256):
            dq.dirotq_set_gemm_tile(cols)
            y = torch.zeros((M, spec.N), dtype=torch.bfloat16, device=dev)
            dq.dirotq_linear(x, layer, y, ws)
            torch.cuda.synchronize()
            assert dq.dirotq_workspace_status(ws) == 0
            outs[cols] = y.view(torch.int16).clone()
        # several tiles per CTA here (33 row blocks x 9 column blocks on 148 SMs)
        assert torch.equal(outs[128], outs[256]) and torch.equal(outs[192], outs[256]) and torch.equal(outs[0], outs[128])
        assert torch.equal(outs[64], outs[256]) and torch.equal(outs[66], outs[256])  # 66 applies to calls with few tiles only
        with pytest.raises(dq.DirotqError):
            dq.dirotq_set_gemm_tile(96)
    finally:
        dq.dirotq_set_gemm_tile(0)
    layer.close()


# ------------------------------------------------------------------ NVFP4 second kernel: 128- and 256-column tiles, and
# 256 rows x 256 columns per pair of CTAs (knob value 512)

import test_gpu_nvfp4


@pytest.mark.parametrize("tile", [128, 256, 512], indirect=True)
def test_nvfp4_ragged_columns_two_blocks_in_last_tile(tile):
    # N = 400: four 128-column blocks, the last one ragged
    spec = synth.LayerSpec(K=512, N=400, r=16, G=64, model=synth.FLUX, seed=51, calib_tokens=1024)
    print(tile, test_gpu_nvfp4._run_case(spec, M=300))


@pytest.mark.parametrize("tile", [128, 256, 512], indirect=True)
def test_nvfp4_odd_number_of_column_blocks(tile):
    # N = 384: three 128-column blocks, so the second 256-column tile has no second block (its scale atoms do not exist)
    spec = synth.LayerSpec(K=768, N=384, r=32, G=64, model=synth.PIXART, seed=52, calib_tokens=1024)
    print(tile, test_gpu_nvfp4._run_case(spec, M=257, with_bias=False))


@pytest.mark.parametrize("tile", [128, 256, 512], indirect=True)
def test_nvfp4_single_column_block_and_two_rank_chunks(tile):
    spec = synth.LayerSpec(K=640, N=128, r=128, G=64, model=synth.FLUX, seed=53, calib_tokens=1024)
    print(tile, test_gpu_nvfp4._run_case(spec, M=130))


def test_nvfp4_both_widths_give_the_same_bits():
    from oracle import dirotq_oracle as orc
    spec = synth.LayerSpec(K=1152, N=1152, r=32, G=64, model=synth.PIXART, seed=54)
    M = 4096 + 77
    inp = synth.make_layer_inputs(spec, M, with_bias=True)
    dev = "cuda"
    W, Q = torch.from_numpy(inp["W"]).to(dev), torch.from_numpy(inp["Q"]).to(dev)
    x = bits_to_bf16_tensor(inp["x"])
    probe = dq.dirotq_prepare_layer_nvfp4(W, Q, spec.r, 0)
    xrot = torch.empty((256, spec.K), dtype=torch.float32, device=dev)
    dq.dirotq_rotate_quantize(x[:256], probe, dq.alloc_workspace(probe, 256), xrot)
    ex = orc.nvfp4_global_exponent(float(xrot[:, spec.r:].abs().max().item()))
    probe.close()
    layer = dq.dirotq_prepare_layer_nvfp4(W, Q, spec.r, ex, bias=bits_to_bf16_tensor(inp["bias"]))
    ws = dq.alloc_workspace(layer, M)
    outs = {}
    try:
        for cols in (0, 128, 256, 512):
            dq.dirotq_set_gemm_tile(cols)
            y = torch.zeros((M, spec.N), dtype=torch.bfloat16, device=dev)
            dq.dirotq_linear(x, layer, y, ws)
            torch.cuda.synchronize()
            assert dq.dirotq_workspace_status(ws) == 0
            outs[cols] = y.view(torch.int16).clone()
        # the accumulation order inside the tensor core does not depend on the tile width: same bits
        assert torch.equal(outs[128], outs[256]) and torch.equal(outs[0], outs[128]) and torch.equal(outs[512], outs[256])
    finally:
        dq.dirotq_set_gemm_tile(0)
    layer.close()


# ------------------------------------------------------------------ W4A8 second kernel: 128- and 256-column tiles

import test_gpu_w4a8


@pytest.mark.parametrize("tile", [128, 256], indirect=True)
def test_w4a8_ragged_rows_and_columns(tile):
    spec = synth.LayerSpec(K=768, N=400, r=32, G=64, model=synth.FLUX, seed=81, calib_tokens=1024)
    print(tile, test_gpu_w4a8._run_case(spec, M=300))


@pytest.mark.parametrize("tile", [128, 256], indirect=True)
def test_w4a8_pixart_projection_many_tiles(tile):
    spec = synth.LayerSpec(K=1152, N=1152, r=32, G=64, model=synth.PIXART, seed=82)
    print(tile, test_gpu_w4a8._run_case(spec, M=1024, check_rot=False))


# ------------------------------------------------------------------ rotation kernel: the tile plans (4 = CTA pairs, 5 = 64-column
# tiles for calls with few token rows; with groups of 128 plan 5 falls back to plan 1)

@pytest.fixture
def rot_plan(request):
    dq.dirotq_set_rotation_tile(request.param)
    yield request.param
    dq.dirotq_set_rotation_tile(0)


@pytest.mark.parametrize("rot_plan", [1, 2, 3, 4, 5], indirect=True)
def test_rotation_plans_int4_ragged(rot_plan):
    # M = 300: the second 128-row block of a 256-row tile is ragged; K_l = 496: ragged last group
    spec = synth.LayerSpec(K=512, N=256, r=16, G=64, model=synth.FLUX, seed=91, calib_tokens=1024)
    print(rot_plan, test_gpu_parity._run_case(spec, M=300))


@pytest.mark.parametrize("rot_plan", [1, 2, 3, 4, 5], indirect=True)
def test_rotation_plans_group128_many_row_blocks(rot_plan):
    spec = synth.LayerSpec(K=768, N=128, r=128, G=128, model=synth.PIXART, seed=92, calib_tokens=1024)
    print(rot_plan, test_gpu_parity._run_case(spec, M=1100, with_bias=False))


@pytest.mark.parametrize("rot_plan", [3, 4, 5], indirect=True)
def test_rotation_256_row_tiles_other_formats(rot_plan):
    spec = synth.LayerSpec(K=640, N=256, r=32, G=64, model=synth.FLUX, seed=93, calib_tokens=1024)
    print(test_gpu_asym._run_case(spec, M=385, shift=1.0))
    print(test_gpu_nvfp4._run_case(spec, M=385))
    print(test_gpu_w4a8._run_case(spec, M=385))


def test_rotation_plans_give_the_same_codes_and_outputs():
    spec = synth.LayerSpec(K=1152, N=256, r=32, G=64, model=synth.PIXART, seed=94)
    M = 5000      # 40 row blocks x 5 column blocks: several tiles per CTA under every plan
    inp = synth.make_layer_inputs(spec, M, with_bias=True)
    dev = "cuda"
    layer = dq.dirotq_prepare_layer(torch.from_numpy(inp["W"]).to(dev), torch.from_numpy(inp["Q"]).to(dev), spec.r, spec.G,
                                    bias=bits_to_bf16_tensor(inp["bias"]))
    x = bits_to_bf16_tensor(inp["x"])
    ws = dq.alloc_workspace(layer, M)
    outs = {}
    try:
        for plan in (0, 1, 2, 3, 4, 5):
            dq.dirotq_set_rotation_tile(plan)
            y = torch.zeros((M, spec.N), dtype=torch.bfloat16, device=dev)
            dq.dirotq_linear(x, layer, y, ws)
            torch.cuda.synchronize()
            assert dq.dirotq_workspace_status(ws) == 0
            xh, codes, scales = dq.dirotq_workspace_export(layer, M, ws)
            outs[plan] = (y.view(torch.int16).clone(), codes.clone(), scales.view(torch.int16).clone(), xh.view(torch.int16).clone())
        for plan in (0, 1, 3, 4, 5):
            for a, b in zip(outs[plan], outs[2]):
                assert torch.equal(a, b)
        with pytest.raises(dq.DirotqError):
            dq.dirotq_set_rotation_tile(6)
    finally:
        dq.dirotq_set_rotation_tile(0)
    layer.close()


# ------------------------------------------------------------------ few token rows: the automatic choice is the 64-column plans

@pytest.mark.parametrize("M", [1, 100, 256, 300])
def test_few_token_rows_take_the_narrow_plans(M):
    # 1152 -> 1152: with up to three row blocks even 128-column tiles would use 27 of 148 SMs; both kernels then run with
    # 64-column tiles (nothing forced here)
    spec = synth.LayerSpec(K=1152, N=1152, r=32, G=64, model=synth.PIXART, seed=95)
    print(M, test_gpu_parity._run_case(spec, M=M))


def test_split_reduction_against_one_cta_per_tile():
    # knob 66: the K-groups of a 128 x 64 tile cut over a cluster of CTAs whose partial tiles meet in one of them through
    # distributed shared memory.  The partial sums are added in another order than one CTA adds the groups, so the outputs
    # agree to fp32 rounding (a bf16 step where a value sits on a rounding boundary), not bit for bit.
    spec = synth.LayerSpec(K=1152, N=1152, r=32, G=64, model=synth.PIXART, seed=97)
    for M in (256, 130):
        inp = synth.make_layer_inputs(spec, M, with_bias=True)
        dev = "cuda"
        layer = dq.dirotq_prepare_layer(torch.from_numpy(inp["W"]).to(dev), torch.from_numpy(inp["Q"]).to(dev), spec.r, spec.G,
                                        bias=bits_to_bf16_tensor(inp["bias"]))
        x = bits_to_bf16_tensor(inp["x"])
        ws = dq.alloc_workspace(layer, M)
        outs = {}
        try:
            for cols in (64, 66):
                dq.dirotq_set_gemm_tile(cols)
                y = torch.zeros((M, spec.N), dtype=torch.bfloat16, device=dev)
                for _ in range(3):  # consecutive calls: the barriers and the landing area start afresh every launch
                    dq.dirotq_linear(x, layer, y, ws)
                torch.cuda.synchronize()
                assert dq.dirotq_workspace_status(ws) == 0
                outs[cols] = y.float().clone()
        finally:
            dq.dirotq_set_gemm_tile(0)
        a, b = outs[64], outs[66]
        rms = float(a.pow(2).mean().sqrt())
        assert float((a - b).abs().max()) <= 2.0 ** -7 * float(a.abs().max()) + 1e-6 * rms  # at most one bf16 step of the largest value
        assert float((a != b).float().mean()) < 0.02
        layer.close()


def test_few_token_rows_other_formats():
    spec = synth.LayerSpec(K=640, N=320, r=32, G=64, model=synth.FLUX, seed=96, calib_tokens=1024)
    print(test_gpu_asym._run_case(spec, M=130, shift=1.0))
    print(test_gpu_nvfp4._run_case(spec, M=130))
    print(test_gpu_w4a8._run_case(spec, M=130))
