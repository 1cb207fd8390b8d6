"""The N > 1 path of the bench on CPU: two ``gloo`` ranks run the replica protocol (disjoint prompt
shards, barrier, maximum over ranks, whole-job throughput)."""
import os
import socket
import sys

import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

from paper_2510_04147_b200 import replicas, workloads as wl


def _free_port() -> int:
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    p = s.getsockname()[1]
    s.close()
    return p


def _worker(rank: int, world: int, port: int, out_dir: str):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world),
                      LOCAL_RANK=str(rank))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        assert replicas.rank_world_local() == (rank, world, rank)
        w = wl.LLADA_8B.replace(batch=2)
        mine = replicas.shard_prompts(w, rank, world)
        assert mine.shape == (2, w.prompt_len)
        # every rank sees every shard: disjoint rows of one seeded set, rank 0 = the single-GPU prompts
        gathered = [torch.zeros_like(mine) for _ in range(world)]
        dist.all_gather(gathered, mine)
        assert torch.equal(torch.cat(gathered), wl.make_prompts(w, batch=2 * world))
        assert torch.equal(gathered[0], wl.make_prompts(w, batch=2))
        assert not torch.equal(gathered[0], gathered[1])
        # timing protocol: the slowest rank decides
        dist.barrier()
        ms = replicas.max_over_ranks(10.0 + 5.0 * rank, dist)
        assert ms == 10.0 + 5.0 * (world - 1)
        tps = replicas.job_tokens_per_s(world, 2, w.gen_len, ms)
        assert abs(tps - world * 2 * w.gen_len / (ms * 1e-3)) < 1e-9
        dist.barrier()
        with open(os.path.join(out_dir, f"ok{rank}"), "w") as f:
            f.write(f"{tps}")
    finally:
        dist.destroy_process_group()


def test_two_gloo_ranks_replica_protocol(tmp_path):
    world = 2
    mp.spawn(_worker, args=(world, _free_port(), str(tmp_path)), nprocs=world, join=True)
    vals = [float(open(tmp_path / f"ok{r}").read()) for r in range(world)]
    assert vals[0] == vals[1]            # every rank derives the same whole-job number


def test_single_process_defaults():
    assert replicas.max_over_ranks(3.5) == 3.5
    assert replicas.job_tokens_per_s(1, 1, 256, 1000.0) == 256.0
    with pytest.raises(ValueError):
        replicas.shard_prompts(wl.TINY, 2, 2)
    assert torch.equal(replicas.shard_prompts(wl.TINY, 0, 1), wl.make_prompts(wl.TINY))
