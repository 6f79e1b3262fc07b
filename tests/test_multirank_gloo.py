"""The path shards by (batch, head) with no exchange step.  Two CPU ranks (gloo) each draw and plan
their own batch element; the union must equal what one process computes for the whole batch, and the
bench's aggregation rule (max over ranks of the step time, layers summed) is exercised."""
import os
import socket
import sys

import numpy as np
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, out):
    sys.path.insert(0, ROOT)
    from oracle import scope_oracle as orc
    from paper_2608_12780_b200 import inputs

    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    cfg = inputs.CONFIGS["tiny"]
    Q, K, V = inputs.make_qkv(cfg, seed=0, threads=1, batch_offset=rank)  # this rank's batch element
    plans = orc.plan_layer(Q, K, cfg)
    k_head = torch.tensor([p.k_head for p in plans], dtype=torch.int64)
    pairs = torch.tensor([int((p.n_c.astype(np.int64) * p.r_c).sum()) for p in plans], dtype=torch.int64)
    gathered = [torch.zeros_like(k_head) for _ in range(world)]
    dist.all_gather(gathered, k_head)  # reporting only: nothing in the path depends on another rank
    step_ms = torch.tensor([10.0 + rank], dtype=torch.float64)
    dist.all_reduce(step_ms, op=dist.ReduceOp.MAX)
    total_pairs = pairs.sum().clone()
    dist.all_reduce(total_pairs)
    if rank == 0:
        out.put((torch.stack(gathered).numpy(), float(step_ms), int(total_pairs)))
    dist.barrier()
    dist.destroy_process_group()


def test_batch_sharded_ranks_reproduce_the_single_process_result():
    sys.path.insert(0, ROOT)
    from oracle import scope_oracle as orc
    from paper_2608_12780_b200 import inputs

    world = 2
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_worker, args=(r, world, port, out)) for r in range(world)]
    for p in procs:
        p.start()
    k_heads, step_ms, total_pairs = out.get(timeout=300)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    cfg = inputs.CONFIGS["tiny"].replace(B=world)
    Q, K, V = inputs.make_qkv(cfg, seed=0, threads=1)
    ref = orc.plan_layer(Q, K, cfg)
    ref_k = np.array([p.k_head for p in ref]).reshape(world, cfg.H)
    assert np.array_equal(k_heads, ref_k)
    assert total_pairs == sum(int((p.n_c.astype(np.int64) * p.r_c).sum()) for p in ref)
    assert step_ms == 11.0  # the slowest rank defines the step
    # whole-job metric of the bench: step time divided by the layers all ranks processed
    assert step_ms / world == 5.5
