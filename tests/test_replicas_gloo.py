"""The N > 1 path of the benchmark on CPU: two gloo ranks stand in for two GPUs.  The speculative step does not
shard (sequences are independent; every GPU runs a replica on its own prompts), so what N > 1 adds is only the
split of the prompt set and the max / sum reductions of the timing -- exercised here without a GPU."""
import os
import socket
import sys

import numpy as np
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)


def _free_port() -> int:
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _rank_main(rank: int, world: int, port: int, out_dir: str):
    import bench
    from workload import configs, corpus
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        cfg = configs.get(0)
        per_rank = 3
        prompts_all = corpus.make_prompts(cfg, per_rank * world)
        mine = bench.shard_prompts(prompts_all, rank, per_rank)
        assert mine.shape == (per_rank, cfg.prompt_len)
        # every rank regenerates the same global prompt set and takes a disjoint slice
        gathered = [torch.zeros((per_rank, cfg.prompt_len), dtype=torch.int32) for _ in range(world)]
        dist.all_gather(gathered, torch.from_numpy(mine.copy()))
        assert np.array_equal(torch.cat(gathered).numpy(), prompts_all)
        dev = torch.device("cpu")
        assert bench.reduce_over_ranks(1.5 + rank, "max", world, dev) == 1.5 + (world - 1)
        assert bench.reduce_over_ranks(1.0 + rank, "sum", world, dev) == sum(1.0 + r for r in range(world))
        # rank r commits 100 * (r + 1) tokens in 10 * (r + 1) ms: the job's rate is all tokens over the slowest rank
        value, ms = bench.whole_job_throughput(100.0 * (rank + 1), 10.0 * (rank + 1), world, dev)
        assert ms == 10.0 * world
        assert abs(value - sum(100.0 * (r + 1) for r in range(world)) / (10.0 * world * 1e-3)) < 1e-6
        open(os.path.join(out_dir, f"ok{rank}"), "w").write("ok")
    finally:
        dist.destroy_process_group()


def test_two_replica_ranks_split_prompts_and_reduce_timing(tmp_path):
    world = 2
    mp.spawn(_rank_main, args=(world, _free_port(), str(tmp_path)), nprocs=world, join=True)
    assert sorted(os.listdir(tmp_path)) == ["ok0", "ok1"]


def test_single_rank_reductions_are_identities():
    import bench
    assert bench.reduce_over_ranks(3.25, "max", 1, None) == 3.25
    assert bench.whole_job_throughput(50.0, 5.0, 1, None) == (50.0 / 5e-3, 5.0)
