"""Expert-parallel forward of one MoE++ layer: FFN experts spread over the ranks, zero-computation experts on every rank.

The paper's deployment argument (Sec. 3.4): the FFN experts of a layer live on different GPUs, the zero, copy and
constant experts are replicated on each of them, so a token routed to a zero-computation expert never leaves its GPU
and only the FFN slots cross the interconnect.  Here that becomes, per rank and layer:

  1. route + permute on the rank's own tokens (all N experts are candidates; only FFN slots get a grouped row);
     the grouped buffer is expert-major, and rank r owns the contiguous expert block [r n_local, (r + 1) n_local),
     so the rows bound for rank r are one contiguous segment of x_perm -- it is the send buffer as it stands;
  2. an all-to-all of the per-expert row counts, then an all-to-all-v of the rows (FFN slots only);
  3. the received rows arrive source-major; `moepp_gather_rows` regroups them expert-major, the grouped FFN runs on
     the local experts, a second gather puts the results back in arrival order;
  4. the reverse all-to-all-v returns every result row to the rank that sent it, into its y_perm;
  5. combine on the rank's own tokens, with the zero-computation experts applied locally (Eq. 3-5).

Planning is plain integer arithmetic on the host (one device-to-host read of the expert offsets per layer, which the
variable-size all-to-all needs anyway).  `forward_distributed` runs one rank per process over torch.distributed;
`forward_emulated` runs the same per-rank phases for all ranks of a job inside one process, moving the segments with
device copies in the place of the collective, so that the sharding logic can be checked on a single GPU.
"""
from __future__ import annotations

from dataclasses import dataclass
from typing import List, Optional

import numpy as np
import torch

from . import binding as B


# --------------------------------------------------------------------------------------------------
# host-side planning (no device work)
# --------------------------------------------------------------------------------------------------
def experts_per_rank(n_ffn: int, world: int) -> int:
    if world < 1 or n_ffn % world != 0:
        raise ValueError("the FFN experts (%d) must divide evenly over the ranks (%d)" % (n_ffn, world))
    return n_ffn // world


def send_counts(expert_offsets: np.ndarray, world: int) -> np.ndarray:
    """[world, n_local]: rows this rank sends to each rank, per expert of that rank, from its dense
    (row_align 1) expert offsets."""
    off = np.asarray(expert_offsets, np.int64)
    n_local = experts_per_rank(len(off) - 1, world)
    return np.diff(off).reshape(world, n_local)


@dataclass
class Regroup:
    """Received rows arrive source-major (for every source rank, its rows in expert order)."""
    to_expert_major: np.ndarray   # int32 [M_recv]: arrival position of the row at each expert-major position
    to_arrival: np.ndarray        # int32 [M_recv]: the inverse permutation
    expert_offsets: np.ndarray    # int32 [n_local + 1]: segments of the local experts in expert-major order
    recv_splits: List[int]        # rows received from each source rank


def regroup_plan(recv_counts: np.ndarray) -> Regroup:
    """recv_counts [world (source), n_local]: rows each source rank sends for each local expert."""
    rc = np.asarray(recv_counts, np.int64)
    world, n_local = rc.shape
    flat_base = np.concatenate([[0], np.cumsum(rc.reshape(-1))])[:-1].reshape(world, n_local)  # arrival start of (src, e)
    order = []
    for e in range(n_local):
        for src in range(world):
            order.append(flat_base[src, e] + np.arange(rc[src, e], dtype=np.int64))
    to_em = np.concatenate(order) if order else np.zeros(0, np.int64)
    to_arr = np.empty_like(to_em)
    to_arr[to_em] = np.arange(len(to_em), dtype=np.int64)
    offs = np.concatenate([[0], np.cumsum(rc.sum(axis=0))])
    return Regroup(to_em.astype(np.int32), to_arr.astype(np.int32), offs.astype(np.int32),
                   [int(v) for v in rc.sum(axis=1)])


# --------------------------------------------------------------------------------------------------
# collectives (one rank per process)
# --------------------------------------------------------------------------------------------------
def exchange_counts(sc: np.ndarray, group=None, device="cpu") -> np.ndarray:
    """All-to-all of the count matrix: row r of `sc` goes to rank r; returns [world (source), n_local]."""
    import torch.distributed as dist
    send = torch.as_tensor(np.ascontiguousarray(sc), dtype=torch.int64, device=device)
    recv = torch.empty_like(send)
    dist.all_to_all_single(recv, send, group=group)
    return recv.cpu().numpy()


def exchange_rows(send: torch.Tensor, send_splits: List[int], recv_splits: List[int], group=None) -> torch.Tensor:
    """All-to-all-v of rows (dim 0): segment r of `send` goes to rank r."""
    import torch.distributed as dist
    recv = torch.empty((sum(recv_splits),) + tuple(send.shape[1:]), dtype=send.dtype, device=send.device)
    dist.all_to_all_single(recv, send, output_split_sizes=recv_splits, input_split_sizes=send_splits, group=group)
    return recv


# --------------------------------------------------------------------------------------------------
# one rank's device work, in phases
# --------------------------------------------------------------------------------------------------
class EpRank:
    """State of one rank for one layer.  `weights`: the router-side tensors of the full layer (W_r, W_g, W_c, v,
    router_bias) and the FFN weights of the LOCAL experts only (W_gate, W_up [n_local, F, D], W_down [n_local, D, F])."""

    def __init__(self, rank: int, world: int, cfg: B.Config, weights: dict, device="cuda"):
        if cfg.row_align != 1 or cfg.capacity_factor > 0:
            raise ValueError("expert parallelism here uses dense segments and no capacity limit")
        self.rank, self.world, self.cfg, self.w, self.dev = rank, world, cfg, weights, device
        self.n_local = experts_per_rank(cfg.n_ffn, world)
        T, N, K = cfg.T, cfg.N, cfg.top_k
        self.td = torch.bfloat16 if cfg.dtype == B.MOEPP_BF16 else torch.float32
        new = lambda *shape, dtype=torch.float32: torch.empty(*shape, dtype=dtype, device=device)
        self.logits, self.idx, self.wk = new(T, N), new(T, K, dtype=torch.int32), new(T, K)
        self.counts, self.offsets = new(N, dtype=torch.int32), new(cfg.n_ffn + 1, dtype=torch.int32)
        self.alpha = new(T, max(cfg.n_const, 1), 2)
        self.ros, self.sor = new(T, K, dtype=torch.int32), new(max(cfg.M_cap, 1), dtype=torch.int32)
        self.x_perm = new(max(cfg.M_cap, 1), cfg.D, dtype=self.td)
        self.y_perm = new(max(cfg.M_cap, 1), cfg.D, dtype=self.td)

    # 1. local routing and grouping; returns the [world, n_local] send counts
    def route_permute(self, x: torch.Tensor, prev: Optional[torch.Tensor]) -> np.ndarray:
        c, w = self.cfg, self.w
        self.x = x
        B.moepp_route(c, x, w["W_r"], w["W_g"], prev if w["W_g"] is not None else None, w["router_bias"], w["W_c"],
                      self.logits, self.idx, self.wk, self.counts, self.offsets, self.alpha if c.n_const else None)
        B.moepp_permute(c, x, self.idx, self.offsets, self.ros, self.sor, self.x_perm)
        self.off_host = self.offsets.cpu().numpy().astype(np.int64)  # the one device-to-host read of the layer
        self.sc = send_counts(self.off_host, self.world)
        self.send_splits = [int(v) for v in self.sc.sum(axis=1)]
        return self.sc

    def send_segment(self, dst: int) -> torch.Tensor:
        b = int(self.off_host[dst * self.n_local])
        return self.x_perm[b:b + self.send_splits[dst]]

    def send_buffer(self) -> torch.Tensor:
        return self.x_perm[:int(self.off_host[-1])]

    # 2. sizes of what arrives
    def prepare(self, recv_counts: np.ndarray) -> None:
        self.plan = regroup_plan(recv_counts)
        m = int(self.plan.expert_offsets[-1])
        self.m_recv = m
        self.x_recv = torch.empty(max(m, 1), self.cfg.D, dtype=self.td, device=self.dev)

    # 3. regroup expert-major, grouped FFN on the local experts, back to arrival order
    def ffn(self) -> torch.Tensor:
        m, c = self.m_recv, self.cfg
        y_send = torch.empty(max(m, 1), c.D, dtype=self.td, device=self.dev)
        if m == 0:
            return y_send[:0]
        dev = self.dev
        to_em = torch.as_tensor(self.plan.to_expert_major, device=dev)
        to_arr = torch.as_tensor(self.plan.to_arrival, device=dev)
        offs = torch.as_tensor(self.plan.expert_offsets, device=dev)
        x_em = torch.empty(m, c.D, dtype=self.td, device=dev)
        B.moepp_gather_rows(self.x_recv[:m], to_em, x_em)
        ffn_cfg = B.Config(T=m, D=c.D, F=c.F, n_ffn=self.n_local, top_k=1, dtype=c.dtype, flags=c.flags)
        h = torch.empty(m, c.F, dtype=self.td, device=dev)
        y_em = torch.empty(m, c.D, dtype=self.td, device=dev)
        B.moepp_grouped_ffn(ffn_cfg, x_em, offs, self.w["W_gate"], self.w["W_up"], self.w["W_down"], h, y_em)
        B.moepp_gather_rows(y_em, to_arr, y_send[:m])
        return y_send[:m]

    # 5. local combine (zero-computation experts never left the rank)
    def combine(self) -> torch.Tensor:
        c, w = self.cfg, self.w
        y = torch.empty_like(self.x)
        B.moepp_combine(c, self.x, self.y_perm, self.idx, self.wk, self.ros, self.alpha if c.n_const else None,
                        w["W_c"], w["v"], y)
        return y


def forward_distributed(rank_state: EpRank, x: torch.Tensor, prev: Optional[torch.Tensor], group=None) -> torch.Tensor:
    """One rank of a torch.distributed job (NCCL for CUDA tensors); collectives: counts, rows out, rows back."""
    r = rank_state
    sc = r.route_permute(x, prev)
    r.prepare(exchange_counts(sc, group, device=r.dev))
    m_send = int(r.off_host[-1])
    recv = exchange_rows(r.send_buffer(), r.send_splits, r.plan.recv_splits, group)
    r.x_recv[:r.m_recv].copy_(recv)
    y_send = r.ffn()
    back = exchange_rows(y_send, r.plan.recv_splits, r.send_splits, group)
    r.y_perm[:m_send].copy_(back)
    return r.combine()


def forward_emulated(ranks: List[EpRank], xs: List[torch.Tensor], prevs: List[Optional[torch.Tensor]]) -> List[torch.Tensor]:
    """All ranks of a job in one process: the same phases, device copies in the place of the collectives."""
    world = len(ranks)
    sc = [r.route_permute(x, p) for r, x, p in zip(ranks, xs, prevs)]
    for dst, r in enumerate(ranks):
        r.prepare(np.stack([sc[src][dst] for src in range(world)]))
    for dst, r in enumerate(ranks):  # rows out
        pos = 0
        for src in range(world):
            n = ranks[src].send_splits[dst]
            r.x_recv[pos:pos + n].copy_(ranks[src].send_segment(dst))
            pos += n
    results = [r.ffn() for r in ranks]
    for owner, r in enumerate(ranks):  # rows back: segment `src` of the owner's results returns to rank src
        pos = 0
        for src in range(world):
            n = ranks[src].send_splits[owner]
            b = int(ranks[src].off_host[owner * ranks[src].n_local])
            ranks[src].y_perm[b:b + n].copy_(results[owner][pos:pos + n])
            pos += n
    return [r.combine() for r in ranks]
