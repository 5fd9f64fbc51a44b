"""World-size-2 check (gloo, CPU) of the only multi-rank logic the path has: sequences are sharded over
ranks with replicated heads and no data-path collective; a host scheduler may gather the accepted-prefix
lengths; the benchmark takes the maximum time over ranks."""
import os
import socket

import numpy as np
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from oracle import csd_oracle as orc
from paper_2411_11925_b200 import inputs as gen


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, B, q):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    torch.set_num_threads(2)
    wl = gen.Workload(**{**gen.WORKLOADS["tiny_fp32"].__dict__, "B": B, "cfg": True, "cfg_scale": 2.0, "T": 4})
    inp = gen.make_round_inputs(wl)                       # same seed on every rank: replicated heads + inputs
    mine = gen.shard_sequences(B, world, rank)
    out = orc.round_from_inputs(gen.select_sequences(inp, mine))
    sp_local = orc.single_path_from_inputs(gen.select_sequences(inp, mine))["logratio"]   # Eq. 2 shards the same way
    n_local = torch.full((B,), -1, dtype=torch.int32)
    n_local[mine.start:mine.stop] = torch.from_numpy(out["n_accept"])
    dist.all_reduce(n_local, op=dist.ReduceOp.MAX)        # gather for a host-side AR scheduler
    t = torch.tensor([0.010 * (rank + 1)], dtype=torch.float64)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)              # benchmark timing: max over ranks
    if rank == 0:
        q.put((n_local.numpy(), float(t), out["logratio"], sp_local))
    dist.barrier()
    dist.destroy_process_group()


def test_two_ranks_shard_sequences_without_exchange():
    B, world = 5, 2
    assert [list(gen.shard_sequences(B, world, r)) for r in range(world)] == [[0, 1, 2], [3, 4]]
    assert sum(len(gen.shard_sequences(64, 8, r)) for r in range(8)) == 64
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_worker, args=(r, world, port, B, q)) for r in range(world)]
    for p in procs:
        p.start()
    n_all, tmax, lr0, sp0 = q.get(timeout=240)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    wl = gen.Workload(**{**gen.WORKLOADS["tiny_fp32"].__dict__, "B": B, "cfg": True, "cfg_scale": 2.0, "T": 4})
    full = orc.round_from_inputs(gen.make_round_inputs(wl))
    np.testing.assert_array_equal(n_all, full["n_accept"])          # sharded == unsharded
    np.testing.assert_allclose(lr0, full["logratio"][:3], rtol=1e-9)
    np.testing.assert_allclose(sp0, orc.single_path_from_inputs(gen.make_round_inputs(wl))["logratio"][:3], rtol=1e-9)
    assert abs(tmax - 0.020) < 1e-12
