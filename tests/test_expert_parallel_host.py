"""Host logic of the expert-parallel forward (paper_2410_07348_b200/expert_parallel.py), CPU only.

The planning arithmetic against a brute-force walk over tagged rows, and the two collectives (count exchange, row
exchange out and back) between two gloo ranks: every FFN row reaches the rank that owns its expert, is regrouped
expert-major, and returns to the position it was sent from.  No kernel runs here.
"""
import os
import socket

import numpy as np
import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from paper_2410_07348_b200 import expert_parallel as EP


def _random_offsets(rng, n_ffn, max_rows):
    counts = rng.integers(0, max_rows, size=n_ffn)
    counts[rng.integers(0, n_ffn)] = 0  # an expert nobody picked
    return np.concatenate([[0], np.cumsum(counts)]).astype(np.int32)


def test_send_counts_and_regroup_plan_by_brute_force():
    rng = np.random.default_rng(1)
    for world, n_ffn in ((1, 4), (2, 8), (4, 8), (4, 16)):
        n_local = EP.experts_per_rank(n_ffn, world)
        offs = [_random_offsets(rng, n_ffn, 9) for _ in range(world)]
        sc = [EP.send_counts(o, world) for o in offs]
        for r in range(world):
            assert sc[r].shape == (world, n_local) and sc[r].sum() == offs[r][-1]
        for dst in range(world):
            # rows as they arrive at `dst`: for every source, its segment for dst, tagged (src, global expert, k)
            arrival = []
            for src in range(world):
                for e in range(dst * n_local, (dst + 1) * n_local):
                    arrival += [(src, e, k) for k in range(offs[src][e + 1] - offs[src][e])]
            plan = EP.regroup_plan(np.stack([sc[src][dst] for src in range(world)]))
            assert plan.recv_splits == [int(sc[src][dst].sum()) for src in range(world)]
            em = [arrival[i] for i in plan.to_expert_major]
            # expert-major, and inside an expert by source then by the source's own order
            assert em == sorted(arrival, key=lambda t: (t[1], t[0], t[2]))
            for j in range(n_local):
                seg = em[plan.expert_offsets[j]:plan.expert_offsets[j + 1]]
                assert all(t[1] == dst * n_local + j for t in seg)
            assert [em[i] for i in plan.to_arrival] == arrival  # the way back


def test_uneven_expert_split_is_refused():
    with pytest.raises(ValueError):
        EP.experts_per_rank(6, 4)


def _worker(rank, world, port, out):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    n_ffn, D = 6, 4
    n_local = n_ffn // world
    rng = np.random.default_rng(10 + rank)
    off = _random_offsets(rng, n_ffn, 7)
    m_send = int(off[-1])
    # a row carries (sender, expert, position in the sender's buffer, 0)
    send = torch.zeros(m_send, D, dtype=torch.float32)
    for e in range(n_ffn):
        for p in range(off[e], off[e + 1]):
            send[p] = torch.tensor([rank, e, p, 0.0])
    sc = EP.send_counts(off, world)
    rc = EP.exchange_counts(sc)
    plan = EP.regroup_plan(rc)
    send_splits = [int(v) for v in sc.sum(axis=1)]
    recv = EP.exchange_rows(send, send_splits, plan.recv_splits)
    ok = recv.shape[0] == plan.expert_offsets[-1]
    ok = ok and bool(((recv[:, 1] >= rank * n_local) & (recv[:, 1] < (rank + 1) * n_local)).all())  # only my experts
    em = recv[torch.as_tensor(plan.to_expert_major, dtype=torch.long)]
    for j in range(n_local):
        seg = em[plan.expert_offsets[j]:plan.expert_offsets[j + 1]]
        ok = ok and bool((seg[:, 1] == rank * n_local + j).all())
    worked = em.clone()
    worked[:, 3] = 1.0  # "the expert ran"
    back_src = worked[torch.as_tensor(plan.to_arrival, dtype=torch.long)]
    back = EP.exchange_rows(back_src, plan.recv_splits, send_splits)
    ok = ok and back.shape == send.shape and bool((back[:, :3] == send[:, :3]).all()) and bool((back[:, 3] == 1).all())
    gathered = [None] * world
    dist.all_gather_object(gathered, bool(ok))
    if rank == 0:
        torch.save(gathered, out)
    dist.destroy_process_group()


def test_two_gloo_ranks_dispatch_and_return(tmp_path):
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        port = s.getsockname()[1]
    out = str(tmp_path / "res.pt")
    mp.spawn(_worker, args=(2, port, out), nprocs=2, join=True)
    assert all(torch.load(out))
