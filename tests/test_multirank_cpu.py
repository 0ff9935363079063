"""The N > 1 path on CPU: two gloo ranks shard the chains (no data-path collective), each runs its
own chain ids, and the union equals the single-process run - chain results depend only on the
chain id.  The per-rank work here is done by the oracle (the CUDA library needs a GPU); what is
under test is the sharding rule and the max-over-ranks / sum-over-ranks reduction bench.py uses."""
import os
import sys
import tempfile

import numpy as np
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

import workloads
from oracle import asd as oasd, denoisers as oden

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _rank_main(rank, world, init_file, n_per_rank, out_dir):
    sys.path.insert(0, ROOT)
    dist.init_process_group("gloo", init_method=f"file://{init_file}", rank=rank, world_size=world)
    wl = workloads.make("cfg1_gmm2d", K=30)
    g, sch = oden.from_workload(wl), oasd.make_schedule(wl.t)
    base = rank * n_per_rank                       # the rule bench.py applies: chain_id_base = rank * n
    ys = np.stack([oasd.asd_sample(g, sch, wl.seed, base + j, j, wl.window, d=wl.d, keep_records=False).y
                   for j in range(n_per_rank)])
    t = torch.tensor([10.0 + rank, float(n_per_rank)], dtype=torch.float64)   # (fake ms, samples)
    tmax, tsum = t.clone(), t.clone()
    dist.all_reduce(tmax, op=dist.ReduceOp.MAX)
    dist.all_reduce(tsum, op=dist.ReduceOp.SUM)
    gathered = [torch.zeros(n_per_rank, wl.d, dtype=torch.float64) for _ in range(world)]
    dist.all_gather(gathered, torch.from_numpy(ys))
    if rank == 0:
        np.save(os.path.join(out_dir, "all.npy"), torch.cat(gathered).numpy())
        np.save(os.path.join(out_dir, "red.npy"), np.array([tmax[0].item(), tsum[1].item()]))
    dist.barrier()
    dist.destroy_process_group()


def test_two_ranks_shard_chains_without_collectives():
    world, n = 2, 3
    with tempfile.TemporaryDirectory() as tmp:
        init_file = os.path.join(tmp, "init")
        mp.spawn(_rank_main, args=(world, init_file, n, tmp), nprocs=world, join=True)
        allys = np.load(os.path.join(tmp, "all.npy"))
        red = np.load(os.path.join(tmp, "red.npy"))
    wl = workloads.make("cfg1_gmm2d", K=30)
    g, sch = oden.from_workload(wl), oasd.make_schedule(wl.t)
    # the single-process run of chain ids 0..5 (slot only matters for conditioned networks)
    ref = np.stack([oasd.asd_sample(g, sch, wl.seed, c, 0, wl.window, d=wl.d, keep_records=False).y
                    for c in range(world * n)])
    assert np.array_equal(allys, ref)
    assert red[0] == 11.0 and red[1] == world * n       # max over ranks of time, sum of samples
