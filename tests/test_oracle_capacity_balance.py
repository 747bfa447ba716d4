"""Pins for the oracle's heterogeneous capacity (Eq. 8) and load-balance statistics (Eq. 7).

Checked against things that are not the oracle: hand arithmetic on the paper's printed formulas, an
independent slot-by-slot brute force in Python, torch's float64 softmax, and special cases.  CPU only.
"""
import math

import numpy as np
import pytest
import torch

from oracle import LayerShape

rng = np.random.default_rng(99)


def _rand(*shape, std=1.0):
    return (rng.standard_normal(shape) * std).astype(np.float32)


# ------------------------------------------------------------------------------------------------
# Eq. 8
# ------------------------------------------------------------------------------------------------
def test_capacity_formula_by_hand(oracle64):
    # 16 FFN + 4 zero-computation experts, tau = 0.75, gamma = 1.1, 1000 tokens, top-1:
    # denominator 0.75*16 + 4 = 16; FFN: 1.1*0.75*1000/16 = 51.5625 -> 52; ZC: 1.1*1000/16 = 68.75 -> 69
    s = LayerShape(T=1000, D=8, F=8, n_ffn=16, n_zero=1, n_copy=1, n_const=2, top_k=1, tau=0.75, capacity_factor=1.1)
    assert oracle64.capacities(s) == (52, 69)
    # top-2 doubles the slots that are shared out
    s.top_k = 2
    assert oracle64.capacities(s) == (104, 138)
    # a vanilla MoE (no zero-computation experts): gamma * slots / N_FFN, whatever tau is
    sv = LayerShape(T=640, D=8, F=8, n_ffn=8, top_k=2, tau=0.3, capacity_factor=1.25)
    assert oracle64.capacities(sv)[0] == 200  # (the other value is unused: there is no such expert)
    # tau = 1: every expert gets the same share; smaller tau moves capacity to the zero-computation experts
    s1 = LayerShape(T=1200, D=8, F=8, n_ffn=8, n_zero=4, top_k=1, tau=1.0, capacity_factor=1.0)
    assert oracle64.capacities(s1) == (100, 100)
    s1.tau = 0.5
    cf, cz = oracle64.capacities(s1)
    assert (cf, cz) == (75, 150) and cz == 2 * cf
    # total capacity = gamma * slots (up to the rounding up of each expert)
    assert abs(8 * cf + 4 * cz - 1200) <= 12
    # no factor -> no limit
    s1.capacity_factor = 0.0
    assert oracle64.capacities(s1) == (2**31 - 1, 2**31 - 1)


def _brute_tables(idx, N, n_ffn, cap_ffn, cap_zc):
    """Independent restatement: walk the slots in order, serve each expert's first `cap` slots."""
    flat = idx.reshape(-1)
    kept_counts = [min(int((flat == e).sum()), cap_ffn) for e in range(n_ffn)]
    offsets = np.concatenate([[0], np.cumsum(kept_counts)]).astype(np.int32)
    seen = [0] * N
    ros = np.empty(len(flat), np.int32)
    for s, e in enumerate(flat):
        cap = cap_ffn if e < n_ffn else cap_zc
        if seen[e] >= cap:
            ros[s] = -2
        elif e < n_ffn:
            ros[s] = offsets[e] + seen[e]
        else:
            ros[s] = -1
        seen[e] += 1
    return offsets, ros


@pytest.mark.parametrize("gamma,tau", [(1.1, 0.75), (0.5, 1.0), (1.0, 0.1), (4.0, 0.75)])
def test_tables_with_capacity_against_brute_force(oracle64, gamma, tau):
    s = LayerShape(T=257, D=4, F=4, n_ffn=5, n_zero=1, n_copy=1, n_const=1, top_k=2, tau=tau, capacity_factor=gamma)
    G = _rand(s.T, s.N, std=2.0)
    G[:, 0] += 1.5  # one crowded FFN expert
    G[:, 5] += 1.0  # and a crowded zero expert
    idx, _ = oracle64.gate_topk(s, G)
    counts, offsets, ros, sor = oracle64.tables(s, idx)
    cap_ffn, cap_zc = oracle64.capacities(s)
    off_b, ros_b = _brute_tables(idx, s.N, s.n_ffn, cap_ffn, cap_zc)
    assert np.array_equal(offsets, off_b)
    assert np.array_equal(ros.reshape(-1), ros_b)
    assert np.array_equal(counts, np.bincount(idx.reshape(-1), minlength=s.N))  # selection counts, not capped
    rows = ros.reshape(-1)
    kept = rows >= 0
    assert np.array_equal(sor[rows[kept]], np.nonzero(kept)[0])
    assert (sor >= 0).sum() == kept.sum() == offsets[-1]
    if gamma >= 4.0:
        assert not np.any(rows == -2)  # generous capacity: nothing is dropped
    else:
        assert np.any(rows == -2)


def test_layer_with_capacity_drops_in_slot_order(oracle64):
    s = LayerShape(T=64, D=16, F=24, n_ffn=3, n_zero=1, n_copy=1, n_const=1, top_k=2, tau=0.75, capacity_factor=0.6)
    x, W_r, W_c, v = _rand(s.T, s.D), _rand(s.N, s.D, std=0.4), _rand(1, 2, s.D, std=0.3), _rand(1, s.D)
    Wg, Wu, Wd = (_rand(3, 24, 16, std=0.2), _rand(3, 24, 16, std=0.2), _rand(3, 16, 24, std=0.2))
    kw = dict(W_c=W_c, v=v, W_gate=Wg, W_up=Wu, W_down=Wd)
    r = oracle64.layer_forward(s, x, W_r, **kw)
    free = LayerShape(**{**s.__dict__, "capacity_factor": 0.0})
    r0 = oracle64.layer_forward(free, x, W_r, **kw)
    assert np.array_equal(r["idx"], r0["idx"]) and np.array_equal(r["w"], r0["w"])  # routing itself is unchanged
    _, _, ros, _ = oracle64.tables(s, r["idx"])
    dropped = ros == -2
    assert dropped.any() and not dropped.all()
    untouched = ~dropped.any(axis=1)
    np.testing.assert_array_equal(r["y"][untouched], r0["y"][untouched])
    both = dropped.all(axis=1)
    if both.any():
        assert np.all(r["y"][both] == 0)  # the token passes on through the residual stream only
    # a token with exactly one dropped pick keeps exactly the other pick's contribution:
    # rerun without capacity but with the dropped picks forced onto the zero expert (Eq. 3 contributes nothing)
    forced = np.where(dropped, s.n_ffn, r["idx"]).astype(np.int32)
    one = dropped.sum(axis=1) == 1
    rz = oracle64.layer_forward(free, x, W_r, forced_idx=forced, **kw)
    # weights differ (forced picks read their own softmax value), so compare only the surviving pick's term
    keep_k = np.argmax(~dropped, axis=1)
    for t in np.nonzero(one)[0][:10]:
        solo = np.full((s.T, 2), s.n_ffn, np.int32)
        solo[t, 0] = r["idx"][t, keep_k[t]]
        ys = oracle64.layer_forward(free, x, W_r, forced_idx=solo, **kw)["y"][t]
        np.testing.assert_allclose(r["y"][t], ys, rtol=1e-6, atol=1e-7)
    # staged pipeline = definition, with dropping
    counts, offsets, ros, sor = oracle64.tables(s, r["idx"])
    xp = oracle64.permute_rows(s, x, sor)
    kept_counts = np.diff(offsets)
    yp = oracle64.grouped_ffn(s, xp, offsets, kept_counts, Wg, Wu, Wd)
    y = oracle64.combine(s, x, yp, r["idx"], r["w"], ros, oracle64.const_alpha(s, x, W_c), v)
    np.testing.assert_allclose(y, r["y"], rtol=2e-6, atol=2e-6)


# ------------------------------------------------------------------------------------------------
# Eq. 7
# ------------------------------------------------------------------------------------------------
def test_balance_stats_closed_forms(oracle64):
    # all logits equal: P_i = 1/N for every token; ties go to the lowest indices, so experts 0..K-1 are
    # selected by every token (f = 1) and nobody else is: L_b = sum_{i<K} eta_i / N
    s = LayerShape(T=50, D=1, F=1, n_ffn=1, n_zero=1, n_copy=1, n_const=1, top_k=2, tau=0.25)
    G = np.zeros((s.T, s.N), np.float32)
    idx, _ = oracle64.gate_topk(s, G)
    f, P, L = oracle64.balance_stats(s, G, idx)
    np.testing.assert_allclose(P, 0.25, atol=1e-7)
    np.testing.assert_allclose(f, [1, 1, 0, 0], atol=0)
    assert abs(L - (1.0 + 0.25) / 4) < 1e-7  # eta = 1 for the FFN expert, tau for the zero expert
    # perfectly balanced selection with uniform probabilities: L_b = (K/N^2) (N_FFN + tau N_ZC)
    s = LayerShape(T=12, D=1, F=1, n_ffn=4, n_zero=2, top_k=1, tau=0.5)
    G = np.zeros((s.T, s.N), np.float32)
    idx = (np.arange(12) % 6).astype(np.int32).reshape(12, 1)
    f, P, L = oracle64.balance_stats(s, G, idx)
    np.testing.assert_allclose(f, 1 / 6, atol=1e-7)
    assert abs(L - (1 / 36) * (4 + 0.5 * 2)) < 1e-7


def test_balance_stats_against_torch(oracle64, oracle32):
    s = LayerShape(T=300, D=1, F=1, n_ffn=8, n_zero=1, n_copy=1, n_const=2, top_k=2, tau=0.75)
    G = _rand(s.T, s.N, std=2.0)
    idx, _ = oracle64.gate_topk(s, G)
    f, P, L = oracle64.balance_stats(s, G, idx)
    Pt = torch.softmax(torch.from_numpy(G).double(), 1).mean(0).numpy()
    ft = np.bincount(idx.reshape(-1), minlength=s.N) / s.T
    np.testing.assert_allclose(P, Pt, atol=1e-6)
    np.testing.assert_allclose(f, ft, atol=1e-7)
    assert abs(f.sum() - s.top_k) < 1e-6 and abs(P.sum() - 1) < 1e-6
    eta = np.array([1.0] * 8 + [0.75] * 4)
    assert abs(L - float((eta * ft * Pt).sum())) < 1e-6
    # tau only weighs the zero-computation experts
    s1 = LayerShape(**{**s.__dict__, "tau": 1.0})
    _, _, L1 = oracle64.balance_stats(s1, G, idx)
    assert abs((L1 - L) - float((0.25 * ft[8:] * Pt[8:]).sum())) < 1e-6
    f32_, P32, L32 = oracle32.balance_stats(s, G, idx)
    assert abs(L32 - L) < 1e-5


# ------------------------------------------------------------------------------------------------
# Eq. 7 differentiated with respect to the logits (f held fixed)
# ------------------------------------------------------------------------------------------------
def _balance_problem(T=9, n_ffn=3, n_zero=1, n_copy=1, n_const=1, K=2, tau=0.6):
    s = LayerShape(T=T, D=8, F=8, n_ffn=n_ffn, n_zero=n_zero, n_copy=n_copy, n_const=n_const, top_k=K, tau=tau)
    G = _rand(T, s.N)
    idx = np.stack([rng.permutation(s.N)[:K] for _ in range(T)]).astype(np.int32)
    return s, G, idx


def test_balance_backward_matches_finite_differences(oracle64):
    s, G, idx = _balance_problem()
    f, _, _ = oracle64.balance_stats(s, G, idx)
    dG = oracle64.balance_backward(s, G, f, scale=0.7)
    eps = 1e-2
    for t, j in [(0, 0), (3, 2), (8, 5), (4, 4), (7, 1)]:
        keep = G[t, j]
        G[t, j] = keep + eps
        hi = oracle64.balance_stats(s, G, idx)[2]
        G[t, j] = keep - eps
        lo = oracle64.balance_stats(s, G, idx)[2]
        G[t, j] = keep
        step = float(np.float32(keep + eps)) - float(np.float32(keep - eps))
        assert abs(0.7 * (hi - lo) / step - dG[t, j]) < 2e-5, (t, j)


def test_balance_backward_matches_torch_autograd(oracle64):
    s, G, idx = _balance_problem(T=17, n_ffn=5, n_const=2, tau=0.25)
    f, _, _ = oracle64.balance_stats(s, G, idx)
    g = torch.tensor(G, dtype=torch.float64, requires_grad=True)
    eta = torch.tensor([1.0] * s.n_ffn + [0.25] * (s.N - s.n_ffn), dtype=torch.float64)
    loss = (eta * torch.tensor(f, dtype=torch.float64) * torch.softmax(g, dim=1).mean(dim=0)).sum()
    loss.backward()
    dG = oracle64.balance_backward(s, G, f, scale=1.0)
    assert np.abs(dG - g.grad.numpy()).max() < 1e-8
    # every row sums to zero: a constant added to a token's logits changes nothing
    assert np.abs(dG.sum(axis=1)).max() < 1e-8
    # accumulation adds to what is there
    base = _rand(s.T, s.N)
    acc = oracle64.balance_backward(s, G, f, scale=2.0, into=base)
    assert np.abs(acc - (base + 2.0 * dG)).max() < 1e-6


def test_balance_backward_closed_form_for_equal_logits(oracle64):
    # equal logits: P = 1/N everywhere, so dG[t, j] = scale / (T N) * (c_j - mean(c)), c_i = eta_i f_i
    s, _, idx = _balance_problem(T=6, tau=0.5)
    G = np.full((s.T, s.N), 0.3, np.float32)
    f, _, _ = oracle64.balance_stats(s, G, idx)
    c = np.array([1.0] * s.n_ffn + [0.5] * (s.N - s.n_ffn)) * f.astype(np.float64)
    want = 3.0 / (s.T * s.N) * (c - c.mean())
    dG = oracle64.balance_backward(s, G, f, scale=3.0)
    assert np.abs(dG - want[None, :]).max() < 1e-8
