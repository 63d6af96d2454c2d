"""The N > 1 host logic on CPU: two gloo ranks shard KV heads with no data exchange, each runs
the oracle on its shard, and the timing/throughput reduction takes the max over ranks."""
import os
import socket

import numpy as np
import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from paper_2502_00299_b200.sharding import partition


def test_partition_is_balanced_and_covers_everything():
    for n in (0, 1, 7, 8, 80, 81):
        for world in (1, 2, 3, 8):
            spans = [partition(n, world, r) for r in range(world)]
            assert spans[0][0] == 0 and spans[-1][1] == n
            assert all(a[1] == b[0] for a, b in zip(spans, spans[1:]))
            sizes = [e - b for b, e in spans]
            assert max(sizes) - min(sizes) <= 1
    with pytest.raises(ValueError):
        partition(4, 2, 2)


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, q):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        from oracle import chunkkv_oracle as ora
        from paper_2502_00299_b200.sharding import gather_index_shards, job_throughput, max_over_ranks
        from workloads import CONFIGS, make_layer, scaled
        wl = scaled(CONFIGS[2], L=600, budget=92)
        x = make_layer(wl)
        G = wl.Hq // wl.Hkv
        h0, h1 = partition(wl.Hkv, world, rank)
        # a rank's shard: its KV heads and the query heads that map onto them
        res = ora.compress_layer(x.q_obs[h0 * G:h1 * G], x.K[h0:h1], x.V[h0:h1], (h1 - h0) * G, h1 - h0,
                                 wl.w, wl.c, wl.budget)
        shards = gather_index_shards(torch.from_numpy(res["idx"]), world)
        full = torch.cat(shards, dim=0).numpy()
        ms_local = 10.0 * (rank + 1)
        thr, ms = job_throughput(1000.0, ms_local)
        q.put((rank, full, max_over_ranks(ms_local), thr, ms))
    finally:
        dist.destroy_process_group()


def test_two_ranks_shard_heads_without_exchange():
    world, port = 2, _free_port()
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    procs = [ctx.Process(target=_worker, args=(r, world, port, q)) for r in range(world)]
    for p in procs:
        p.start()
    got = [q.get(timeout=180) for _ in range(world)]
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    from oracle import chunkkv_oracle as ora
    from workloads import CONFIGS, make_layer, scaled
    wl = scaled(CONFIGS[2], L=600, budget=92)
    x = make_layer(wl)
    ref = ora.compress_layer(x.q_obs, x.K, x.V, wl.Hq, wl.Hkv, wl.w, wl.c, wl.budget)["idx"]
    for rank, full, mx, thr, ms in got:
        assert np.array_equal(full, ref)          # head-sharded result == unsharded result
        assert mx == 20.0 and ms == 20.0          # max over ranks
        assert thr == pytest.approx(2000.0 / 0.020)
