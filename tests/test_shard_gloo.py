"""world_size-2 checks on CPU (gloo) of the multi-rank host logic: row shards cover the batch, the
timing reduction takes the max over ranks, and -- the property that lets the path shard without any
collective -- the layer evaluated on a rank's rows equals the same rows of the full-batch result."""
import os
import sys

import numpy as np
import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def test_row_shard_covers_and_balances():
    from paper_2605_16732_b200.shard import row_shard
    for M in (0, 1, 7, 128, 4608, 18433):
        for world in (1, 2, 3, 8):
            spans = [row_shard(M, r, world) for r in range(world)]
            assert spans[0][0] == 0 and spans[-1][1] == M
            assert all(spans[i][1] == spans[i + 1][0] for i in range(world - 1))
            sizes = [hi - lo for lo, hi in spans]
            assert max(sizes) - min(sizes) <= 1
    with pytest.raises(ValueError):
        row_shard(10, 2, 2)


def _worker(rank, world, port, out_dir):
    sys.path.insert(0, ROOT)
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    from oracle import dirotq_oracle as orc
    from paper_2605_16732_b200 import synth
    from paper_2605_16732_b200.shard import aggregate_throughput, max_over_ranks, row_shard

    spec = synth.LayerSpec(K=128, N=64, r=16, G=32, model=synth.PIXART, seed=5, calib_tokens=256)
    M = 37
    inp = synth.make_layer_inputs(spec, M)           # same seeds on both ranks: the layer is replicated
    layer = orc.prepare_layer(inp["W"], inp["Q"], spec.r, spec.G)
    lo, hi = row_shard(M, rank, world)
    y_mine = orc.linear_deployed(inp["x"][lo:hi], layer, bias=inp["bias"])["y"]
    y_full = orc.linear_deployed(inp["x"], layer, bias=inp["bias"])["y"]
    assert np.array_equal(y_mine, y_full[lo:hi])     # rows are independent: no exchange needed
    # timing rule: max over ranks
    t = max_over_ranks(10.0 + 5.0 * rank)
    assert t == 10.0 + 5.0 * (world - 1)
    assert aggregate_throughput(100.0, t, world) == world * 100.0 / (t * 1e-3)
    # gather the shards on rank 0 only to prove that they tile the batch (test-side collective)
    parts = [None] * world
    dist.all_gather_object(parts, (lo, hi, y_mine))
    if rank == 0:
        parts.sort(key=lambda p: p[0])
        assert np.array_equal(np.concatenate([p[2] for p in parts], axis=0), y_full)
        open(os.path.join(out_dir, "ok"), "w").write("ok")
    dist.destroy_process_group()


def test_two_rank_row_sharding_gloo(tmp_path):
    from oracle import dirotq_oracle as orc
    orc.build()  # compile once before the ranks start
    port = 29500 + (os.getpid() % 2000)
    mp.spawn(_worker, args=(2, port, str(tmp_path)), nprocs=2, join=True)
    assert (tmp_path / "ok").read_text() == "ok"
