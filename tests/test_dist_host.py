"""The multi-GPU path is replicas only; its host logic (max-over-ranks aggregation) is covered
here with two gloo ranks on CPU."""
import os
import sys

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _worker(rank, world, port, q):
    sys.path.insert(0, ROOT)
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    import importlib.util
    spec = importlib.util.spec_from_file_location("csd_dist", os.path.join(ROOT, "paper_2312_11462_b200", "dist.py"))
    mod = importlib.util.module_from_spec(spec)
    spec.loader.exec_module(mod)
    # rank 1 is the slow one: both figures must come from its times
    dev_ms, br_ms = (1000.0, 1100.0) if rank == 0 else (2000.0, 2500.0)
    out = mod.aggregate_tokens_per_s(256 * 4, dev_ms, br_ms, 4, dist)
    q.put((rank, out, mod.replica_prompt_seed(1000, rank)))
    dist.barrier()
    dist.destroy_process_group()


def test_two_rank_aggregation():
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    port = 29500 + os.getpid() % 2000
    procs = [ctx.Process(target=_worker, args=(r, 2, port, q)) for r in range(2)]
    for p in procs:
        p.start()
    res = [q.get(timeout=120) for _ in procs]
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    seeds = set()
    for rank, (value, e2e, ms), seed in res:
        assert abs(value - 2 * 1024 / 2.0) < 1e-9       # all tokens / slowest device time
        assert abs(e2e - 2 * 1024 / 2.5) < 1e-9
        assert abs(ms - 2500.0 / 4) < 1e-9
        seeds.add(seed)
    assert seeds == {1000, 1001}


def test_single_process():
    sys.path.insert(0, ROOT)
    import importlib.util
    spec = importlib.util.spec_from_file_location("csd_dist", os.path.join(ROOT, "paper_2312_11462_b200", "dist.py"))
    mod = importlib.util.module_from_spec(spec)
    spec.loader.exec_module(mod)
    assert mod.aggregate_tokens_per_s(512, 1000.0, 2000.0, 2) == (512.0, 256.0, 1000.0)
