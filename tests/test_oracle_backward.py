"""Pins for the oracle's backward pass.

Two independent referees: (1) central finite differences of the oracle's own forward pass (picks held fixed),
for every input and parameter group; (2) torch autograd (float64) on the layer's definition written with torch
ops, which derives the gradient by itself.  CPU only.
"""
import numpy as np
import pytest
import torch

from oracle import LayerShape

rng = np.random.default_rng(7)


def _rand(*shape, std=1.0):
    return (rng.standard_normal(shape) * std).astype(np.float32)


def _problem(T=6, D=8, F=10, n_ffn=3, n_const=2, K=2, **over):
    s = LayerShape(T=T, D=D, F=F, n_ffn=n_ffn, n_zero=1, n_copy=1, n_const=n_const, top_k=K, **over)
    p = dict(x=_rand(T, D), W_r=_rand(s.N, D, std=0.4), W_g=_rand(s.N, s.N, std=0.3), prev=_rand(T, s.N),
             bias=_rand(s.N, std=0.2), W_c=_rand(n_const, 2, D, std=0.4), v=_rand(n_const, D),
             W_gate=_rand(n_ffn, F, D, std=0.4), W_up=_rand(n_ffn, F, D, std=0.4), W_down=_rand(n_ffn, D, F, std=0.4))
    return s, p


def _forward_loss(o, s, p, idx, R, Q):
    r = o.layer_forward(s, p["x"], p["W_r"], p["W_g"], p["prev"], p["bias"], p["W_c"], p["v"], p["W_gate"], p["W_up"],
                        p["W_down"], forced_idx=idx)
    return float((r["y"].astype(np.float64) * R).sum() + (r["logits"].astype(np.float64) * Q).sum())


@pytest.mark.parametrize("over", [dict(), dict(renorm_topk=1, add_residual=1), dict(capacity_factor=0.6, tau=0.5),
                                  dict(K=3)])
def test_backward_matches_finite_differences(oracle64, over):
    over = dict(over)
    K = over.pop("K", 2)
    s, p = _problem(K=K, **over)
    # picks that cover every expert kind, fixed for all evaluations
    idx = np.stack([rng.permutation(s.N)[:K] for _ in range(s.T)]).astype(np.int32)
    idx[0, :2] = [0, s.n_ffn]          # FFN + zero
    idx[1, :2] = [s.n_ffn + 1, s.n_ffn + 2]  # copy + constant
    R, Q = rng.standard_normal((s.T, s.D)), rng.standard_normal((s.T, s.N)) * 0.5
    g = oracle64.layer_backward(s, p["x"], p["W_r"], idx, R.astype(np.float32), p["W_g"], p["prev"], p["bias"], p["W_c"],
                                p["v"], p["W_gate"], p["W_up"], p["W_down"], dlogits=Q.astype(np.float32))
    names = dict(x="dx", prev="dprev", W_r="dW_r", W_g="dW_g", bias="dbias", W_c="dW_c", v="dv", W_gate="dW_gate",
                 W_up="dW_up", W_down="dW_down")
    eps = 2e-3
    R32, Q32 = R.astype(np.float32).astype(np.float64), Q.astype(np.float32).astype(np.float64)
    for key, gname in names.items():
        grad = g[gname]
        scale = max(float(np.abs(grad).max()), 1e-3)
        flat = p[key].reshape(-1)
        for pos in rng.choice(flat.size, size=min(12, flat.size), replace=False):
            keep = flat[pos]
            flat[pos] = keep + eps
            hi = _forward_loss(oracle64, s, p, idx, R32, Q32)
            flat[pos] = keep - eps
            lo = _forward_loss(oracle64, s, p, idx, R32, Q32)
            flat[pos] = keep
            step = float(np.float32(keep + eps)) - float(np.float32(keep - eps))
            fd = (hi - lo) / step
            assert abs(fd - float(grad.reshape(-1)[pos])) <= 5e-3 * scale + 2e-4, (key, pos, fd, grad.reshape(-1)[pos])


def _torch_layer(s, p, idx, t64):
    """The layer's definition (Eq. 1-6, SwiGLU experts) with torch ops and fixed picks; autograd does the rest."""
    x, W_r, W_g, prev, bias, W_c, v, Wg, Wu, Wd = (t64[k] for k in ("x", "W_r", "W_g", "prev", "bias", "W_c", "v",
                                                                     "W_gate", "W_up", "W_down"))
    G = x @ W_r.T + prev @ W_g.T + bias
    P = torch.softmax(G, dim=1)
    zero0, copy0, const0 = s.n_ffn, s.n_ffn + s.n_zero, s.n_ffn + s.n_zero + s.n_copy
    ys = []
    for t in range(s.T):
        w = P[t, torch.as_tensor(idx[t], dtype=torch.long)]
        if s.renorm_topk:
            w = w / w.sum()
        acc = x[t].clone() if s.add_residual else torch.zeros_like(x[t])
        for k, e in enumerate(idx[t]):
            if e < zero0:
                out = Wd[e] @ (torch.nn.functional.silu(Wg[e] @ x[t]) * (Wu[e] @ x[t]))
            elif e < copy0:
                out = torch.zeros_like(x[t])
            elif e < const0:
                out = x[t]
            else:
                a = torch.softmax(W_c[e - const0] @ x[t], dim=0)
                out = a[0] * x[t] + a[1] * v[e - const0]
            acc = acc + w[k] * out
        ys.append(acc)
    return torch.stack(ys), G


@pytest.mark.parametrize("over", [dict(), dict(renorm_topk=1, add_residual=1)])
def test_backward_matches_torch_autograd(oracle64, over):
    s, p = _problem(T=9, D=12, F=14, **over)
    idx = np.stack([rng.permutation(s.N)[:2] for _ in range(s.T)]).astype(np.int32)
    R, Q = _rand(s.T, s.D), _rand(s.T, s.N, std=0.5)
    t64 = {k: torch.tensor(a, dtype=torch.float64, requires_grad=True) for k, a in p.items()}
    y, G = _torch_layer(s, p, idx, t64)
    ((y * torch.tensor(R, dtype=torch.float64)).sum() + (G * torch.tensor(Q, dtype=torch.float64)).sum()).backward()
    g = oracle64.layer_backward(s, p["x"], p["W_r"], idx, R, p["W_g"], p["prev"], p["bias"], p["W_c"], p["v"],
                                p["W_gate"], p["W_up"], p["W_down"], dlogits=Q)
    names = dict(x="dx", prev="dprev", W_r="dW_r", W_g="dW_g", bias="dbias", W_c="dW_c", v="dv", W_gate="dW_gate",
                 W_up="dW_up", W_down="dW_down")
    for key, gname in names.items():
        ref = t64[key].grad.numpy()
        np.testing.assert_allclose(g[gname], ref, rtol=2e-4, atol=2e-5 * max(1.0, float(np.abs(ref).max())), err_msg=key)


def test_backward_special_cases(oracle64, oracle32):
    s, p = _problem()
    zero, copy = s.n_ffn, s.n_ffn + 1
    R = _rand(s.T, s.D)
    # every pick on the zero expert: the layer is constant, all gradients vanish (no residual, no logits gradient)
    idx = np.full((s.T, 2), zero, np.int32)
    idx[:, 1] = zero  # the same expert twice is not a legal top-K result, but a legal forced input
    g = oracle64.layer_backward(s, p["x"], p["W_r"], idx, R, p["W_g"], p["prev"], p["bias"], p["W_c"], p["v"],
                                p["W_gate"], p["W_up"], p["W_down"])
    for k, a in g.items():
        assert a is None or np.all(a == 0), k
    # first layer (no gating residual): dprev and dW_g are not produced
    s1 = LayerShape(**{**s.__dict__})
    idx = np.tile(np.array([[0, copy]], np.int32), (s.T, 1))
    g1 = oracle64.layer_backward(s1, p["x"], p["W_r"], idx, R, None, None, None, p["W_c"], p["v"], p["W_gate"],
                                 p["W_up"], p["W_down"])
    assert g1["dprev"] is None and g1["dW_g"] is None
    assert np.all(g1["dW_gate"][1:] == 0) and np.any(g1["dW_gate"][0] != 0)  # only the expert in use learns
    assert np.all(g1["dv"] == 0) and np.all(g1["dW_c"] == 0)
    # float and double arithmetic agree
    g32 = oracle32.layer_backward(s1, p["x"], p["W_r"], idx, R, None, None, None, p["W_c"], p["v"], p["W_gate"],
                                  p["W_up"], p["W_down"])
    for k in ("dx", "dW_r", "dW_gate", "dW_down"):
        assert np.abs(g32[k] - g1[k]).max() <= 1e-4 * max(1.0, np.abs(g1[k]).max())
