"""World-size-2 check (gloo, CPU) of how the path shards over ranks.

Every rank owns B consecutive samples and passes sample_offset = rank * B to the sampler, so the
masks are those of the unsharded batch; dX and X_keep stay local, dW and db are partial sums
whose all-reduce equals the gradient of the whole batch (rows are independent, Sec. 3.2.1).
The step time a multi-rank benchmark reports is the maximum over ranks.  The rank logic under test is the
benchmark's own (`bench.sample_offset_of`, `bench.max_over_ranks`), run here over gloo.
"""
import os
import socket

import numpy as np
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

import bench
import oracle
from paper_2210_00129_b200 import synth

B_PER_RANK, H, W, C_IN, C_OUT, R = 3, 4, 5, 8, 12, 0.5


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _rank_main(rank, world, port, out):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    N = H * W
    M_all = world * B_PER_RANK * N
    X, Wt, dY = synth.layer_inputs("f32", M_all, C_IN, C_OUT, 77, 1.0, 0.1, 1.0)     # same seeded batch on every rank
    lo, hi = rank * B_PER_RANK * N, (rank + 1) * B_PER_RANK * N
    keep, offs = oracle.sample_keep(oracle.MASK_RANDOM, B_PER_RANK, H, W, R, seed=5, step=2,
                                    sample_offset=bench.sample_offset_of(rank, B_PER_RANK))
    g = oracle.linear_backward(oracle.forward_cache(X[lo:hi], keep).astype(np.float64), dY[lo:hi], Wt, keep)
    dW = torch.from_numpy(g["dW"].copy()); db = torch.from_numpy(g["db"].copy())
    dist.all_reduce(dW); dist.all_reduce(db)                                         # the only exchange of DP training
    rows = [torch.zeros(len(keep), dtype=torch.int64) for _ in range(world)]
    dist.all_gather(rows, torch.from_numpy(keep.astype(np.int64)) + lo)
    tmax = bench.max_over_ranks(1.0 + rank, "cpu")                                     # pretend step times
    if rank == 0:
        out.put((torch.cat(rows).numpy(), dW.numpy(), db.numpy(), g["dX"], tmax))
    dist.barrier()
    dist.destroy_process_group()


def test_two_ranks_reproduce_the_unsharded_batch():
    world = 2
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_rank_main, args=(r, world, port, out)) for r in range(world)]
    for p in procs:
        p.start()
    rows, dW, db, dX0, tmax = out.get(timeout=120)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    N = H * W
    M_all = world * B_PER_RANK * N
    X, Wt, dY = synth.layer_inputs("f32", M_all, C_IN, C_OUT, 77, 1.0, 0.1, 1.0)
    keep_all, _ = oracle.sample_keep(oracle.MASK_RANDOM, world * B_PER_RANK, H, W, R, seed=5, step=2)
    assert rows.tolist() == keep_all.tolist()                       # masks do not depend on the sharding
    whole = oracle.linear_backward(oracle.forward_cache(X, keep_all).astype(np.float64), dY, Wt, keep_all)
    assert np.allclose(dW, whole["dW"], rtol=1e-12, atol=1e-12)     # summed partials = whole-batch gradient
    assert np.allclose(db, whole["db"], rtol=1e-12, atol=1e-12)
    assert np.array_equal(dX0, whole["dX"][: B_PER_RANK * N])       # dX is local to the shard
    assert tmax == 2.0


def test_single_process_rank_logic_and_config_keys():
    assert bench.sample_offset_of(0, 64) == 0 and bench.sample_offset_of(3, 64) == 192
    assert bench.max_over_ranks(1.25, "cpu") == 1.25                  # no process group: the rank's own time
    w = bench.WORKLOADS[bench.DEFAULT_WORKLOAD]
    cfg = bench.config_of(bench.DEFAULT_WORKLOAD, w, 4)
    assert cfg["workload"] == "vit_b16_block_b128" and cfg["B_per_gpu"] == 128 and cfg["parallelism"].startswith("dp4")
    assert cfg["layers"] == ["qkv:768->2304", "proj:768->768", "fc1:768->3072", "fc2:3072->768"]
    assert cfg["keep_ratio_sweep"] == [0.25, 0.5, 0.75, 1.0]
    # FLOPs of the default step at keep ratio 0.5: 4 * 12544 * (768*2304 + 768*768 + 768*3072 + 3072*768)
    assert bench.flops_of(w, 12544) == 4.0 * 12544 * 7077888
