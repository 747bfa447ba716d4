"""The multi-GPU path is token-sharded replicas; its host logic is checked with two gloo ranks on CPU."""
import os
import socket

import numpy as np
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from paper_2410_07348_b200.replicas import token_shard, whole_job_rate


def test_token_shards_partition_the_batch():
    for T in (0, 1, 7, 32768, 32769):
        for world in (1, 2, 3, 8):
            cuts = [token_shard(T, r, world) for r in range(world)]
            assert cuts[0][0] == 0 and cuts[-1][1] == T
            assert all(a[1] == b[0] for a, b in zip(cuts, cuts[1:]))
            sizes = [e - b for b, e in cuts]
            assert max(sizes) - min(sizes) <= 1


def _worker(rank, world, port, out):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    # each rank "processes" its shard; rank 1 is slower
    b, e = token_shard(1001, rank, world)
    rate, ms = whole_job_rate(float(e - b), 10.0 * (rank + 1))
    # sharded oracle run: the layer on a shard equals the shard of the layer on the whole batch
    import oracle
    o = oracle.Oracle("f64")
    rng = np.random.default_rng(0)
    s_all = oracle.LayerShape(T=40, D=16, F=24, n_ffn=3, n_zero=1, n_copy=1, n_const=1)
    x = rng.standard_normal((40, 16)).astype(np.float32)
    W_r = rng.standard_normal((6, 16)).astype(np.float32)
    W_c, v = rng.standard_normal((1, 2, 16)).astype(np.float32), rng.standard_normal((1, 16)).astype(np.float32)
    Wg, Wu, Wd = (rng.standard_normal(sh).astype(np.float32) * 0.2 for sh in ((3, 24, 16), (3, 24, 16), (3, 16, 24)))
    full = o.layer_forward(s_all, x, W_r, W_c=W_c, v=v, W_gate=Wg, W_up=Wu, W_down=Wd)["y"]
    tb, te = token_shard(40, rank, world)
    s_part = oracle.LayerShape(T=te - tb, D=16, F=24, n_ffn=3, n_zero=1, n_copy=1, n_const=1)
    part = o.layer_forward(s_part, x[tb:te], W_r, W_c=W_c, v=v, W_gate=Wg, W_up=Wu, W_down=Wd)["y"]
    ok = bool(np.array_equal(part, full[tb:te]))
    gathered = [None] * world
    dist.all_gather_object(gathered, (rate, ms, ok))
    if rank == 0:
        torch.save(gathered, out)
    dist.destroy_process_group()


def test_two_ranks_aggregate_with_the_slowest_time(tmp_path):
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        port = s.getsockname()[1]
    out = str(tmp_path / "res.pt")
    mp.spawn(_worker, args=(2, port, out), nprocs=2, join=True)
    res = torch.load(out)
    for rate, ms, ok in res:
        assert ok
        assert ms == 20.0  # max over ranks
        assert abs(rate - 1001 / 20e-3) < 1e-6  # all units over the slowest rank's time
