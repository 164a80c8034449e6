"""World-size-2 checks of the multi-GPU host logic, run as gloo ranks on CPU."""
import os
import socket

import numpy as np
import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

import oracle
from paper_2401_05391_b200 import sharding
from paper_2401_05391_b200 import workloads as wl


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, out_dir):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        w = wl.Workload("mp", 2, 3, 4, 2, 16, 9, 5, "f16", "uniform", True, 70)
        t = w.steps - 1
        par = wl.make_parents(w)
        kp, vp = wl.make_prompt(w)
        steps = [wl.make_step(w, s) for s in range(w.steps)]
        q = steps[t][0]
        kr = torch.stack([s[1] for s in steps]); vr = torch.stack([s[2] for s in steps])
        slopes = wl.alibi_slopes(w.heads)

        # --- head sharding: each rank evaluates its kv heads only, nothing is exchanged on the data path
        sub, hq, hk = sharding.shard_heads(w, rank, world)
        mine = oracle.decode_sdpa(w.dtype, w.batch, w.beams, sub.heads, sub.kv_heads, w.head_dim,
                                  wl.to_bits(q[:, hq]), wl.to_bits(kp[:, :, hk]), wl.to_bits(vp[:, :, hk]),
                                  wl.to_bits(kr[:, :, hk]), wl.to_bits(vr[:, :, hk]), par, t,
                                  slopes=slopes[hq].numpy())
        parts = [torch.zeros_like(torch.from_numpy(mine)) for _ in range(world)]
        dist.all_gather(parts, torch.from_numpy(mine))
        if rank == 0:
            full = oracle.decode_sdpa(w.dtype, w.batch, w.beams, w.heads, w.kv_heads, w.head_dim, wl.to_bits(q),
                                      wl.to_bits(kp), wl.to_bits(vp), wl.to_bits(kr), wl.to_bits(vr), par, t,
                                      slopes=slopes.numpy())
            assert np.array_equal(torch.cat(parts, dim=1).numpy(), full)

        # --- weak scaling: ranks hold different requests of the same shape; timing is the max over ranks
        mine_w = sharding.rank_workload(w, rank, world)
        seeds = [torch.zeros(1, dtype=torch.int64) for _ in range(world)]
        dist.all_gather(seeds, torch.tensor([mine_w.seed]))
        assert len({int(s) for s in seeds}) == world
        assert (mine_w.batch, mine_w.heads, mine_w.prompt_len) == (w.batch, w.heads, w.prompt_len)
        slow = sharding.max_over_ranks(1.0 + rank)
        assert slow == float(world)
        assert sharding.whole_job_rate(10.0, world, slow) == 10.0 * world / world
        dist.barrier()
        open(os.path.join(out_dir, f"ok{rank}"), "w").close()
    finally:
        dist.destroy_process_group()


def test_two_gloo_ranks(tmp_path):
    oracle.build()
    world = 2
    mp.spawn(_worker, args=(world, _free_port(), str(tmp_path)), nprocs=world, join=True)
    assert all((tmp_path / f"ok{r}").exists() for r in range(world))


def test_shard_heads_rejects_uneven_split():
    with pytest.raises(ValueError):
        sharding.shard_heads(wl.CONFIGS[3], 0, 3)
    sub, hq, hk = sharding.shard_heads(wl.CONFIGS[3], 1, 2)
    assert (sub.heads, sub.kv_heads, hq, hk) == (28, 28, slice(28, 56), slice(28, 56))
    assert sharding.max_over_ranks(3.5) == 3.5
