"""Seeded synthetic inputs for the MoE++ layer (arXiv 2410.07348).

This module only draws random tensors with the shapes and value distributions of the paper's MoE
sizes (Table 2) and of the five benchmark configurations, and rounds them to the storage type.
It holds none of the layer's arithmetic: both the CUDA library's callers and the CPU oracle's
callers take their inputs from here, and neither implementation is used here.

The one piece of numerics is the router-bias calibration used to shape the load (share of routing
slots on zero-computation experts, Zipf imbalance over FFN experts): the bias is an *input* that is
not part of the paper's method, and it is found with ordinary torch ops on a sample of tokens.

All tensors are torch CPU tensors unless ``device`` is given.  For bf16 workloads ``x`` and the FFN
weights are rounded to bf16 once here, so every consumer sees the same stored values.
"""
from __future__ import annotations

import math
from dataclasses import dataclass, field
from typing import Optional

import torch


@dataclass
class LayerSpec:
    """Sizes and storage type of one layer.  Expert index order: FFN | zero | copy | constant."""
    T: int
    D: int
    F: int
    n_ffn: int
    n_zero: int = 1
    n_copy: int = 1
    n_const: int = 2
    top_k: int = 2
    dtype: str = "bf16"  # "f32" or "bf16": storage of x, y, FFN weights and the staged activations

    @property
    def N(self) -> int:
        return self.n_ffn + self.n_zero + self.n_copy + self.n_const

    @property
    def n_zc(self) -> int:
        return self.n_zero + self.n_copy + self.n_const

    def vanilla(self) -> "LayerSpec":
        """The equal-size all-FFN MoE (Eq. 2): same T, D, F, n_ffn, K and no zero-computation experts."""
        return LayerSpec(self.T, self.D, self.F, self.n_ffn, 0, 0, 0, self.top_k, self.dtype)


@dataclass
class LayerTensors:
    spec: LayerSpec
    x: torch.Tensor  # [T,D] storage dtype
    W_r: torch.Tensor  # [N,D] f32
    W_g: Optional[torch.Tensor]  # [N,N] f32
    prev: Optional[torch.Tensor]  # [T,N] f32 previous layer's router logits
    bias: Optional[torch.Tensor]  # [N] f32 (benchmark skew only)
    W_c: Optional[torch.Tensor]  # [n_const,2,D] f32
    v: Optional[torch.Tensor]  # [n_const,D] f32
    W_gate: torch.Tensor  # [n_ffn,F,D] storage dtype
    W_up: torch.Tensor  # [n_ffn,F,D]
    W_down: torch.Tensor  # [n_ffn,D,F]
    meta: dict = field(default_factory=dict)


# The five benchmark configurations (sizes only; see make_* below for the values).
CONFIGS = {
    "cfg1_tiny_f32": LayerSpec(T=512, D=256, F=512, n_ffn=8, dtype="f32"),
    "cfg2_bf16_8e": LayerSpec(T=16384, D=1024, F=2816, n_ffn=8),
    "cfg3_bf16_16e_skew": LayerSpec(T=32768, D=1536, F=4096, n_ffn=16),
    "cfg4_7b_stack": LayerSpec(T=32768, D=4096, F=2816, n_ffn=16),
    "cfg5_sweep": LayerSpec(T=32768, D=4096, F=2816, n_ffn=16),
    # the paper's 2B/(32+8)E model (Table 2): hidden 768, intermediate 2048, 32 FFN + 1/1/6 zero-computation
    # experts; a second router shape (40 experts, 52 stacked rows)
    "paper_2b_32p8e": LayerSpec(T=32768, D=768, F=2048, n_ffn=32, n_zero=1, n_copy=1, n_const=6),
    # the other two small models of Table 2 (same hidden and intermediate size, 1/1/2 zero-computation experts);
    # the 7B/(16+4)E model (hidden 1536, intermediate 4096) has cfg3's sizes
    "paper_06b_8p4e": LayerSpec(T=32768, D=768, F=2048, n_ffn=8, n_zero=1, n_copy=1, n_const=2),
    "paper_1b_16p4e": LayerSpec(T=32768, D=768, F=2048, n_ffn=16, n_zero=1, n_copy=1, n_const=2),
}
CFG4_LAYERS = 4
CFG5_ZC_SHARES = (0.0, 0.15, 0.30, 0.50, 0.75)
CFG5_TOKENS = (128, 2048, 32768, 131072)


def torch_dtype(name: str) -> torch.dtype:
    return {"f32": torch.float32, "bf16": torch.bfloat16}[name]


def _randn(gen, shape, std, dtype, device):
    """N(0, std) drawn in fp32 on the generator's device, rounded once to the storage dtype.
    Large tensors are drawn slab by slab along dim 0 to bound peak memory."""
    out = torch.empty(shape, dtype=dtype, device=device)
    if out.numel() == 0:
        return out
    slab = max(1, (1 << 26) // max(1, out[0].numel()))
    for i in range(0, shape[0], slab):
        n = min(slab, shape[0] - i)
        t = torch.randn((n,) + tuple(shape[1:]), generator=gen, dtype=torch.float32, device=gen.device)
        out[i:i + n] = (t * std).to(dtype).to(device)
    return out


def make_layer(spec: LayerSpec, seed: int = 0, *, with_prev: bool = True, w_std: float = 0.02,
               device: str = "cpu", gen_device: str = "cpu") -> LayerTensors:
    """x~N(0,1); W_r, W_g, W_c, FFN weights ~N(0,w_std); v~N(0,1); previous logits ~N(0,1)."""
    gen = torch.Generator(device=gen_device)
    gen.manual_seed(seed)
    sd = torch_dtype(spec.dtype)
    f32 = torch.float32
    N, D, F = spec.N, spec.D, spec.F
    x = _randn(gen, (spec.T, D), 1.0, sd, device)
    W_r = _randn(gen, (N, D), w_std, f32, device)
    W_g = _randn(gen, (N, N), w_std, f32, device) if with_prev else None
    prev = _randn(gen, (spec.T, N), 1.0, f32, device) if with_prev else None
    W_c = _randn(gen, (spec.n_const, 2, D), w_std, f32, device) if spec.n_const else None
    v = _randn(gen, (spec.n_const, D), 1.0, f32, device) if spec.n_const else None
    W_gate = _randn(gen, (spec.n_ffn, F, D), w_std, sd, device)
    W_up = _randn(gen, (spec.n_ffn, F, D), w_std, sd, device)
    W_down = _randn(gen, (spec.n_ffn, D, F), w_std, sd, device)
    return LayerTensors(spec, x, W_r, W_g, prev, None, W_c, v, W_gate, W_up, W_down, meta={"seed": seed})


def make_stack(spec: LayerSpec, n_layers: int = CFG4_LAYERS, *, device: str = "cpu", gen_device: str = "cpu"):
    """Chained layers: layer j (1-based) uses seed j-1 and weight std 0.02/sqrt(j).  Layer 1 has no gating
    residual (Eq. 6, case j=1); later layers carry W_g and receive the previous layer's logits at run time.
    Only layer 1's x is an input; the others' x is produced by the layer below."""
    layers = []
    for j in range(1, n_layers + 1):
        lt = make_layer(spec if j == 1 else LayerSpec(0, spec.D, spec.F, spec.n_ffn, spec.n_zero, spec.n_copy,
                                                      spec.n_const, spec.top_k, spec.dtype),
                        seed=j - 1, with_prev=False, w_std=0.02 / math.sqrt(j), device=device, gen_device=gen_device)
        if j > 1:
            g = torch.Generator(device=gen_device)
            g.manual_seed(1000 + j)
            lt.W_g = _randn(g, (spec.N, spec.N), 0.02 / math.sqrt(j), torch.float32, device)
            lt.spec = spec
        layers.append(lt)
    return layers


# --------------------------------------------------------------------------------------------------
# Router-bias calibration (load shaping; the bias is an input, not part of the method)
# --------------------------------------------------------------------------------------------------
def _sample_logits(lt: LayerTensors, max_tokens: int = 8192) -> torch.Tensor:
    n = min(lt.spec.T, max_tokens)
    x = lt.x[:n].float().cpu()
    G = x @ lt.W_r.float().cpu().t()
    if lt.W_g is not None and lt.prev is not None:
        G = G + lt.prev[:n].float().cpu() @ lt.W_g.float().cpu().t()
    return G


def _slot_shares(G: torch.Tensor, bias: torch.Tensor, k: int) -> torch.Tensor:
    picks = torch.topk(G + bias, k, dim=1).indices.reshape(-1)
    return torch.bincount(picks, minlength=G.shape[1]).double() / picks.numel()


def calibrate_zc_share(lt: LayerTensors, p_target: float, tol: float = 0.005) -> torch.Tensor:
    """Bias that adds one common offset to every zero-computation expert (the zero expert gets a little
    more, as the paper's load plots show it the busiest of them) so that a share p_target of the routing
    slots lands on zero-computation experts."""
    s = lt.spec
    G = _sample_logits(lt)
    sigma = float(G.std())
    bias = torch.zeros(s.N)
    if s.n_zc == 0:
        return bias
    lo, hi = -12.0 * sigma - 5.0, 12.0 * sigma + 5.0
    for _ in range(60):
        mid = 0.5 * (lo + hi)
        bias[s.n_ffn:] = mid
        if s.n_zero:
            bias[s.n_ffn:s.n_ffn + s.n_zero] = mid + 0.25 * sigma
        p = float(_slot_shares(G, bias, s.top_k)[s.n_ffn:].sum())
        if abs(p - p_target) < tol * 0.2:
            break
        if p < p_target:
            lo = mid
        else:
            hi = mid
    lt.meta["zc_share_sampled"] = p
    return bias


def calibrate_zipf(lt: LayerTensors, p_target: float = 0.30, exponent: float = 1.1) -> torch.Tensor:
    """Bias for the skewed configuration: FFN expert of rank r (1-based, expert index r-1) gets
    beta*ln(r^-exponent); zero-computation experts get a common offset.  beta is chosen so that the FFN
    loads fit r^-exponent in least squares, the offset so that the zero-computation share is p_target."""
    s = lt.spec
    G = _sample_logits(lt)
    ranks = torch.arange(1, s.n_ffn + 1, dtype=torch.float64)
    zipf = ranks.pow(-exponent)
    zipf = zipf / zipf.sum()
    base = (-exponent * ranks.log()).float()

    def with_beta(beta, zc_bias):
        b = torch.zeros(s.N)
        b[:s.n_ffn] = beta * base
        b[s.n_ffn:] = zc_bias[s.n_ffn:]
        return b

    zc_bias = torch.zeros(s.N)
    beta = 1.0
    for _ in range(4):
        # 1-D search for beta (coarse to fine) at the current zero-computation offset
        lo, hi = 0.0, 6.0
        for _ in range(5):
            grid = torch.linspace(lo, hi, 13)
            errs = []
            for b in grid:
                sh = _slot_shares(G, with_beta(float(b), zc_bias), s.top_k)[:s.n_ffn]
                sh = sh / sh.sum().clamp_min(1e-12)
                errs.append(float(((sh - zipf) ** 2).sum()))
            i = int(torch.tensor(errs).argmin())
            beta = float(grid[i])
            step = float(grid[1] - grid[0])
            lo, hi = max(0.0, beta - step), beta + step
        # bisection on the zero-computation offset at this beta
        sigma = float(G.std())
        l2, h2 = -12.0 * sigma - 10.0, 12.0 * sigma + 10.0
        for _ in range(60):
            mid = 0.5 * (l2 + h2)
            zc_bias[s.n_ffn:] = mid
            if s.n_zero:
                zc_bias[s.n_ffn:s.n_ffn + s.n_zero] = mid + 0.25 * sigma
            p = float(_slot_shares(G, with_beta(beta, zc_bias), s.top_k)[s.n_ffn:].sum())
            if p < p_target:
                l2 = mid
            else:
                h2 = mid
    bias = with_beta(beta, zc_bias)
    lt.meta.update(zipf_beta=beta, zc_share_sampled=p)
    return bias


def make_config(name: str, *, device: str = "cpu", gen_device: str = "cpu", T: Optional[int] = None,
                zc_share: Optional[float] = None) -> LayerTensors:
    """One layer of a named configuration (cfg4's stack is built by make_stack)."""
    spec = CONFIGS[name]
    if T is not None:
        spec = LayerSpec(T, spec.D, spec.F, spec.n_ffn, spec.n_zero, spec.n_copy, spec.n_const, spec.top_k, spec.dtype)
    if name == "cfg5_sweep" and zc_share == 0.0:
        spec = spec.vanilla()
    lt = make_layer(spec, seed=0, device=device, gen_device=gen_device)
    if name == "cfg3_bf16_16e_skew":
        lt.bias = calibrate_zipf(lt, 0.30, 1.1).to(device)
    elif name == "cfg5_sweep" and zc_share:
        lt.bias = calibrate_zc_share(lt, zc_share).to(device)
    return lt
