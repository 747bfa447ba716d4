"""The expert-parallel forward with all ranks of a job emulated in one process on one GPU.

`forward_emulated` runs the per-rank phases of paper_2410_07348_b200/expert_parallel.py (route and permute on the
rank's tokens, dispatch of the FFN rows to the owners of their experts, regrouping, grouped FFN on the local experts,
return, local combine with the zero-computation experts) for 2 or 4 ranks, with device copies where a job of several
processes would call all-to-all.  A token's result does not depend on which other rows share its GEMM tile, so the
sharded outputs must be the same bits as the single-GPU layer on the whole batch; one float32 case is also compared
with the oracle directly.
"""
import numpy as np
import pytest
import torch

from harness import max_abs, oracle_inputs, shape_of
from paper_2410_07348_b200 import binding as B
from paper_2410_07348_b200 import expert_parallel as EP
from paper_2410_07348_b200 import workloads as W

pytestmark = pytest.mark.gpu


def _single_gpu(spec, wd, x, prev):
    cfg = B.config_from_spec(spec)
    ws = torch.empty(B.moepp_workspace_bytes(cfg), dtype=torch.uint8, device="cuda")
    y = torch.empty_like(x)
    logits = torch.empty(spec.T, spec.N, device="cuda")
    B.moepp_layer_forward(cfg, wd, x, prev, y, logits, ws)
    return y, logits


def _sharded(spec, wd, x, prev, world, cuts):
    n_local = spec.n_ffn // world
    ranks, xs, prevs = [], [], []
    for r in range(world):
        b, e = cuts[r], cuts[r + 1]
        sub = W.LayerSpec(e - b, spec.D, spec.F, spec.n_ffn, spec.n_zero, spec.n_copy, spec.n_const, spec.top_k, spec.dtype)
        local = dict(wd)
        for name in ("W_gate", "W_up", "W_down"):
            local[name] = wd[name][r * n_local:(r + 1) * n_local].contiguous()
        ranks.append(EP.EpRank(r, world, B.config_from_spec(sub), local))
        xs.append(x[b:e].contiguous())
        prevs.append(prev[b:e].contiguous())
    ys = EP.forward_emulated(ranks, xs, prevs)
    torch.cuda.synchronize()
    assert B.moepp_device_error() == 0
    return torch.cat(ys), torch.cat([r.logits for r in ranks]), ranks


@pytest.mark.parametrize("world,dtype,T", [(2, "bf16", 3000), (4, "bf16", 5000), (8, "bf16", 2500), (2, "f32", 900)])
def test_emulated_ranks_reproduce_the_single_gpu_layer(world, dtype, T):
    spec = W.LayerSpec(T=T, D=264, F=392, n_ffn=8, n_zero=1, n_copy=1, n_const=2, top_k=2, dtype=dtype)
    lt = W.make_layer(spec, seed=23, with_prev=True, w_std=0.05)
    wd = B.weights_from_tensors(lt)
    x, prev = lt.x.cuda(), lt.prev.cuda()
    y_full, lg_full = _single_gpu(spec, wd, x, prev)
    rng = np.random.default_rng(world)
    inner = np.sort(rng.choice(np.arange(1, T), size=world - 1, replace=False))  # uneven token shards
    cuts = [0] + [int(v) for v in inner] + [T]
    y, lg, ranks = _sharded(spec, wd, x, prev, world, cuts)
    assert torch.equal(lg, lg_full)
    assert torch.equal(y, y_full)
    # only FFN rows travelled: what every rank sent is its FFN slot count, less than all its slots
    for r in ranks:
        sent = sum(r.send_splits)
        assert sent == int(r.counts[:spec.n_ffn].sum().item())
        assert sent < r.cfg.T * spec.top_k


def test_emulated_ranks_against_the_oracle(oracle64):
    spec = W.LayerSpec(T=500, D=64, F=96, n_ffn=4, n_zero=1, n_copy=1, n_const=1, top_k=2, dtype="f32")
    lt = W.make_layer(spec, seed=29, with_prev=True, w_std=0.1)
    wd = B.weights_from_tensors(lt)
    x, prev = lt.x.cuda(), lt.prev.cuda()
    y, lg, ranks = _sharded(spec, wd, x, prev, 2, [0, 180, 500])
    idx = torch.cat([r.idx for r in ranks]).cpu().numpy()
    oi = oracle_inputs(lt)
    ref = oracle64.layer_forward(shape_of(spec), oi["x"], oi["W_r"], oi["W_g"], oi["prev"], oi["bias"], oi["W_c"], oi["v"],
                                 oi["W_gate"], oi["W_up"], oi["W_down"], forced_idx=idx)
    assert max_abs(lg.cpu().numpy(), ref["logits"]) <= 2e-4
    assert max_abs(y.cpu().numpy(), ref["y"]) <= 1e-4


def test_distributed_driver_with_a_single_nccl_rank():
    """forward_distributed itself (counts all-to-all, rows out, rows back through torch.distributed / NCCL) with a
    world of one rank: the collectives degenerate to self-sends, the result must equal the single-GPU layer."""
    import socket

    import torch.distributed as dist
    spec = W.LayerSpec(T=1200, D=128, F=256, n_ffn=4, n_zero=1, n_copy=1, n_const=1, top_k=2, dtype="bf16")
    lt = W.make_layer(spec, seed=31, with_prev=True, w_std=0.05)
    wd = B.weights_from_tensors(lt)
    x, prev = lt.x.cuda(), lt.prev.cuda()
    y_full, _ = _single_gpu(spec, wd, x, prev)
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        port = s.getsockname()[1]
    dist.init_process_group("nccl", init_method="tcp://127.0.0.1:%d" % port, rank=0, world_size=1,
                            device_id=torch.device("cuda:0"))
    try:
        rank = EP.EpRank(0, 1, B.config_from_spec(spec), wd)
        y = EP.forward_distributed(rank, x, prev)
        torch.cuda.synchronize()
    finally:
        dist.destroy_process_group()
    assert torch.equal(y, y_full)
