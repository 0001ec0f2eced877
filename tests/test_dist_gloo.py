"""Multi-process host logic on CPU (gloo, world_size 2): batch sharding covers every image exactly
once, the job-wide step time is the maximum over ranks, and sharded oracle results tile the full result."""
import os
import socket

import numpy as np
import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from paper_2405_18425_b200 import dist as vdist
from paper_2405_18425_b200 import synth


def _free_port():
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    port = s.getsockname()[1]
    s.close()
    return port


def _worker(rank, world, port, out_dir):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        import oracle

        cfg = synth.BiglaConfig("dist", B=5, H=2, L=23, dk=8, dv=16, dtype="bf16", gate_mean=0.0, seed=9)
        mine = vdist.shard_range(cfg.B, rank, world)
        units = slice(mine.start * cfg.H, mine.stop * cfg.H)
        x = synth.make_inputs(cfg, units=units)
        f = {n: synth.stored_to_f64(a, cfg.dtype) for n, a in x.items()}
        o = oracle.bigla_fwd(f["q"], f["k"], f["v"], oracle.gate_prep(f["g_fwd"]), oracle.gate_prep(f["g_bwd"]))
        np.save(os.path.join(out_dir, f"o{rank}.npy"), o)
        # every image is owned exactly once
        owned = torch.zeros(cfg.B, dtype=torch.int64)
        owned[mine.start:mine.stop] = 1
        dist.all_reduce(owned)
        assert owned.tolist() == [1] * cfg.B
        # job-wide time = slowest rank
        ms = vdist.max_over_ranks(10.0 + 5.0 * rank, dist)
        assert ms == 10.0 + 5.0 * (world - 1)
        assert vdist.job_throughput(100.0, ms, world) == pytest.approx(world * 100.0 / (ms * 1e-3))
    finally:
        dist.destroy_process_group()


def test_two_rank_batch_sharding(tmp_path, oracle):
    world = 2
    mp.spawn(_worker, args=(world, _free_port(), str(tmp_path)), nprocs=world, join=True)
    cfg = synth.BiglaConfig("dist", B=5, H=2, L=23, dk=8, dv=16, dtype="bf16", gate_mean=0.0, seed=9)
    x = synth.make_inputs(cfg)
    f = {n: synth.stored_to_f64(a, cfg.dtype) for n, a in x.items()}
    full = oracle.bigla_fwd(f["q"], f["k"], f["v"], oracle.gate_prep(f["g_fwd"]), oracle.gate_prep(f["g_bwd"]))
    parts = [np.load(tmp_path / f"o{r}.npy") for r in range(world)]
    tiled = np.concatenate(parts, axis=0).reshape(full.shape)
    np.testing.assert_array_equal(tiled, full)


def test_shard_range_properties():
    for n in (0, 1, 7, 64, 128):
        for world in (1, 2, 3, 8):
            parts = [vdist.shard_range(n, r, world) for r in range(world)]
            assert [i for p in parts for i in p] == list(range(n))
            sizes = [len(p) for p in parts]
            assert max(sizes) - min(sizes) <= 1
    with pytest.raises(ValueError):
        vdist.shard_range(4, 2, 2)
    assert vdist.max_over_ranks(3.5) == 3.5
