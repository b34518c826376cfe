"""Host side of the multi-GPU path on CPU: two gloo ranks shard the tables (independent problems, no
data-path collective), each evaluates its shard, rank 0 reassembles the decision table; timings are
reduced with MAX.  The shard evaluation itself is done by the CPU oracle here (no GPU in this test)."""
import os
import socket

import numpy as np
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from paper_cs_0408034_b200 import workloads as wl


def _free_port():
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    port = s.getsockname()[1]
    s.close()
    return port


def _decide_tables(w):
    from oracle import plogp_oracle as po
    sg = po.SGrid(w.s_list)
    out = []
    for t in range(w.n_tables):
        tab = po.Table(w.table_sizes(t), w.gaps[t], w.latency[t])
        d = po.select_grid(w.strategy_mask, po.predict_grid(tab, w.strategy_mask, w.P_values(), w.m, sg))
        out.append(np.stack([d.strategy.astype(np.float64), d.s.astype(np.float64), d.time]))
    return np.stack(out)  # [tables][3][2][P][m]


def _rank(rank, world, port, q):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        import bench
        full = wl.config4(n_tables=5, P_hi=12, n_m=9, n_s=6)   # 5 tables over 2 ranks: ragged shards
        mine = wl.shard_tables(full, rank, world)
        part = torch.from_numpy(_decide_tables(mine))
        counts = [torch.zeros(1, dtype=torch.int64) for _ in range(world)]
        dist.all_gather(counts, torch.tensor([mine.n_tables]))
        sizes = [int(c.item()) for c in counts]
        gathered = []
        for r in range(world):   # shards may differ in size: one broadcast per shard
            buf = part.clone() if r == rank else torch.zeros((sizes[r],) + tuple(part.shape[1:]), dtype=part.dtype)
            dist.broadcast(buf, src=r)
            gathered.append(buf)
        slowest = bench.max_over_ranks(1.0 + rank, world, "cpu")
        if rank == 0:
            whole = torch.cat(gathered).numpy()
            ref = _decide_tables(full)
            q.put((sizes, bool(np.array_equal(whole, ref)), slowest))
    finally:
        dist.destroy_process_group()


def test_two_ranks_shard_tables_and_reassemble():
    world, port = 2, _free_port()
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    procs = [ctx.Process(target=_rank, args=(r, world, port, q)) for r in range(world)]
    for p in procs:
        p.start()
    sizes, same, slowest = q.get(timeout=120)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    assert sizes == [2, 3] and same
    assert slowest == 2.0


def test_shards_partition_the_tables():
    w = wl.config4(n_tables=11, P_hi=4, n_m=3, n_s=2)
    for world in (1, 2, 3, 4, 8):
        parts = [wl.shard_tables(w, r, world) for r in range(world)]
        assert sum(p.n_tables for p in parts) == w.n_tables
        assert np.array_equal(np.concatenate([p.gaps for p in parts]), w.gaps)
        assert np.array_equal(np.concatenate([p.latency for p in parts]), w.latency)
