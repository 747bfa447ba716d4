"""Pins for the CPU oracle: closed forms, invariants, brute force and library referees.

Every check here compares the oracle with something that is NOT the oracle: the paper's closed forms
(Eq. 3-5), a hand-derived vector (tests/golden/hand_vector.txt), exhaustive enumeration, or torch's
float64 matmul/softmax used as an independent referee.  CPU only.
"""
import itertools
import math
import os

import numpy as np
import pytest
import torch

from oracle import LayerShape

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")
rng = np.random.default_rng(1234)


def _rand(*shape, std=1.0):
    return (rng.standard_normal(shape) * std).astype(np.float32)


def _ffn_weights(s, std=0.2):
    return _rand(s.n_ffn, s.F, s.D, std=std), _rand(s.n_ffn, s.F, s.D, std=std), _rand(s.n_ffn, s.D, s.F, std=std)


def _torch_ffn(x, Wg, Wu, Wd):
    """SwiGLU FFN with torch float64 library routines (independent referee)."""
    x, Wg, Wu, Wd = (torch.from_numpy(np.asarray(a)).double() for a in (x, Wg, Wu, Wd))
    return ((torch.nn.functional.silu(x @ Wg.T) * (x @ Wu.T)) @ Wd.T).numpy()


# ------------------------------------------------------------------------------------------------
# hand-derived vector (Eq. 1, 3, 4, 5)
# ------------------------------------------------------------------------------------------------
def _read_golden(name):
    out = {}
    with open(os.path.join(GOLDEN, name)) as f:
        for line in f:
            if line.startswith("#") or not line.strip():
                continue
            k, *vals = line.split()
            out[k] = np.array([float(v) for v in vals])
    return out


@pytest.mark.parametrize("arith", ["oracle32", "oracle64"])
def test_hand_vector(arith, request):
    o = request.getfixturevalue(arith)
    g = _read_golden("hand_vector.txt")
    s = LayerShape(T=1, D=2, F=0, n_ffn=0, n_zero=1, n_copy=1, n_const=2, top_k=2)
    x = np.array([[1.0, 2.0]], np.float32)
    W_r = np.array([[0, 0], [math.log(4.0), 0], [math.log(2.0), 0], [0, 0]], np.float32)
    W_c = np.zeros((2, 2, 2), np.float32)
    v = np.array([[3.0, -1.0], [7.0, 7.0]], np.float32)
    r = o.layer_forward(s, x, W_r, W_c=W_c, v=v)
    assert r["idx"].tolist() == [g["idx"].astype(int).tolist()]
    np.testing.assert_allclose(r["w"][0], g["w"], rtol=1e-6)
    np.testing.assert_allclose(r["y"][0], g["y"], rtol=1e-6)
    _, _, P = o.gate_topk(s, r["logits"], want_probs=True)
    np.testing.assert_allclose(P[0], g["P"], rtol=1e-6)
    s.renorm_topk = 1
    r = o.layer_forward(s, x, W_r, W_c=W_c, v=v)
    np.testing.assert_allclose(r["y"][0], g["y_renorm"], rtol=1e-6)
    np.testing.assert_allclose(r["w"][0].sum(), 1.0, rtol=1e-6)


# ------------------------------------------------------------------------------------------------
# routing: brute force over all K-subsets, softmax invariants (Eq. 1)
# ------------------------------------------------------------------------------------------------
@pytest.mark.parametrize("N,K", [(3, 1), (5, 2), (8, 3), (6, 6)])
def test_topk_brute_force(oracle64, N, K):
    T = 64
    s = LayerShape(T=T, D=1, F=0, n_ffn=0, n_zero=N, top_k=K)
    G = _rand(T, N)
    idx, w = oracle64.gate_topk(s, G)
    for t in range(T):
        best = max(itertools.combinations(range(N), K), key=lambda c: sum(float(G[t, i]) for i in c))
        assert set(idx[t].tolist()) == set(best)
        picked = G[t, idx[t]]
        assert np.all(picked[:-1] >= picked[1:])  # descending order of the K picks
        # every expert left out is no larger than the smallest pick
        rest = np.delete(G[t], idx[t])
        assert rest.size == 0 or rest.max() <= picked.min()


def test_topk_ties_take_lower_index(oracle64):
    s = LayerShape(T=3, D=1, F=0, n_ffn=0, n_zero=5, top_k=2)
    G = np.array([[1, 1, 1, 1, 1], [0, 2, 2, 0, 2], [-0.0, 0.0, -1, 0.0, -1]], np.float32)
    idx, w = oracle64.gate_topk(s, G)
    assert idx.tolist() == [[0, 1], [1, 2], [0, 1]]


def test_softmax_invariants(oracle64):
    T, N, K = 128, 12, 2
    s = LayerShape(T=T, D=1, F=0, n_ffn=8, n_zero=1, n_copy=1, n_const=2, top_k=K)
    s.F = 1
    G = _rand(T, N, std=3.0)
    idx, w, P = oracle64.gate_topk(s, G, want_probs=True)
    np.testing.assert_allclose(P.sum(1), 1.0, atol=1e-6)
    # shift invariance
    idx2, w2, P2 = oracle64.gate_topk(s, G + np.float32(8.0), want_probs=True)
    assert np.array_equal(idx, idx2)
    np.testing.assert_allclose(P, P2, atol=2e-6)
    # torch float64 softmax as referee; gate weight is the softmax value at the picked index
    Pt = torch.softmax(torch.from_numpy(G).double(), dim=1).numpy()
    np.testing.assert_allclose(P, Pt, atol=1e-6)
    np.testing.assert_allclose(w, np.take_along_axis(Pt, idx, 1), atol=1e-6)
    # without renormalisation the K weights sum to less than one (N > K, finite logits)
    assert np.all(w.sum(1) < 1.0)
    s.renorm_topk = 1
    _, wr = oracle64.gate_topk(s, G)
    np.testing.assert_allclose(wr.sum(1), 1.0, atol=1e-6)
    np.testing.assert_allclose(wr, w / w.sum(1, keepdims=True), atol=1e-6)


# ------------------------------------------------------------------------------------------------
# zero / copy / constant experts: closed forms (Eq. 3, 4, 5) with routing forced through the bias
# ------------------------------------------------------------------------------------------------
def _force_bias(N, first, second):
    b = np.full(N, -40.0, np.float32)
    b[first] = 40.0
    b[second] = 39.0
    return b


def _mini(T=16, D=32, F=48):
    s = LayerShape(T=T, D=D, F=F, n_ffn=3, n_zero=1, n_copy=1, n_const=2, top_k=2)
    x = _rand(T, D)
    W_r = _rand(s.N, D, std=0.005)
    W_c = _rand(2, 2, D, std=0.3)
    v = _rand(2, D)
    Wg, Wu, Wd = _ffn_weights(s)
    return s, x, W_r, W_c, v, Wg, Wu, Wd


def test_zero_plus_copy_bypasses_layer(oracle64):
    s, x, W_r, W_c, v, Wg, Wu, Wd = _mini()
    zero, copy = s.n_ffn, s.n_ffn + 1
    r = oracle64.layer_forward(s, x, W_r, bias=_force_bias(s.N, copy, zero), W_c=W_c, v=v, W_gate=Wg, W_up=Wu,
                               W_down=Wd)
    assert np.all(r["idx"] == [copy, zero])
    np.testing.assert_allclose(r["y"], r["w"][:, :1] * x, rtol=1e-6, atol=1e-7)  # y = g_copy * x


def test_zero_degrades_top2_to_top1(oracle64):
    s, x, W_r, W_c, v, Wg, Wu, Wd = _mini()
    zero = s.n_ffn
    r2 = oracle64.layer_forward(s, x, W_r, bias=_force_bias(s.N, 1, zero), W_c=W_c, v=v, W_gate=Wg, W_up=Wu,
                                W_down=Wd)
    assert np.all(r2["idx"] == [1, zero])
    s1 = LayerShape(**{**s.__dict__, "top_k": 1})
    r1 = oracle64.layer_forward(s1, x, W_r, bias=_force_bias(s.N, 1, zero), W_c=W_c, v=v, W_gate=Wg, W_up=Wu,
                                W_down=Wd)
    np.testing.assert_allclose(r2["y"], r1["y"], rtol=1e-6, atol=1e-7)
    # and both equal g * FFN_1(x) with the FFN from torch
    ref = r2["w"][:, :1].astype(np.float64) * _torch_ffn(x, Wg[1], Wu[1], Wd[1])
    np.testing.assert_allclose(r2["y"], ref, rtol=1e-5, atol=1e-6)


def test_constant_expert_closed_forms(oracle64):
    s, x, W_r, W_c, v, Wg, Wu, Wd = _mini()
    zero, copy, cA, cB = s.n_ffn, s.n_ffn + 1, s.n_ffn + 2, s.n_ffn + 3
    bias = _force_bias(s.N, cA, zero)
    kw = dict(W_gate=Wg, W_up=Wu, W_down=Wd)
    # W_c = 0 -> alpha = (1/2, 1/2)
    Wc0 = np.zeros_like(W_c)
    r = oracle64.layer_forward(s, x, W_r, bias=bias, W_c=Wc0, v=v, **kw)
    np.testing.assert_allclose(r["y"], r["w"][:, :1] * (0.5 * x + 0.5 * v[0]), rtol=1e-6, atol=1e-7)
    np.testing.assert_allclose(oracle64.const_alpha(s, x, Wc0), 0.5, atol=1e-7)
    # alpha -> (1, 0): the constant expert turns into the copy expert; (0, 1): into the bare vector v
    xp = np.abs(x) + 0.5
    Wc_hi = np.zeros_like(W_c)
    Wc_hi[0, 0, 3] = 60.0
    r = oracle64.layer_forward(s, xp, W_r, bias=bias, W_c=Wc_hi, v=v, **kw)
    np.testing.assert_allclose(r["y"], r["w"][:, :1] * xp, rtol=1e-6, atol=1e-7)
    Wc_lo = np.zeros_like(W_c)
    Wc_lo[0, 1, 3] = 60.0
    r = oracle64.layer_forward(s, xp, W_r, bias=bias, W_c=Wc_lo, v=v, **kw)
    np.testing.assert_allclose(r["y"], r["w"][:, :1] * np.broadcast_to(v[0], xp.shape), rtol=1e-6, atol=1e-7)
    # general W_c: alpha from torch softmax; E = a1 x + a2 v
    a = torch.softmax(torch.from_numpy(x).double() @ torch.from_numpy(W_c[0]).double().T, dim=1).numpy()
    r = oracle64.layer_forward(s, x, W_r, bias=bias, W_c=W_c, v=v, **kw)
    np.testing.assert_allclose(r["y"], r["w"][:, :1] * (a[:, :1] * x + a[:, 1:] * v[0]), rtol=1e-5, atol=1e-6)
    np.testing.assert_allclose(oracle64.const_alpha(s, x, W_c)[:, 0, :], a, atol=1e-6)
    # second constant expert uses ITS OWN W_c and v
    biasB = _force_bias(s.N, cB, zero)
    aB = torch.softmax(torch.from_numpy(x).double() @ torch.from_numpy(W_c[1]).double().T, dim=1).numpy()
    r = oracle64.layer_forward(s, x, W_r, bias=biasB, W_c=W_c, v=v, **kw)
    np.testing.assert_allclose(r["y"], r["w"][:, :1] * (aB[:, :1] * x + aB[:, 1:] * v[1]), rtol=1e-5, atol=1e-6)


def test_ffn_plus_constant_is_linear_in_v(oracle64):
    """FFN + constant expert = FFN output adjusted by a vector: y is affine in v with slope w*alpha2."""
    s, x, W_r, W_c, v, Wg, Wu, Wd = _mini()
    cA = s.n_ffn + 2
    bias = _force_bias(s.N, 0, cA)
    kw = dict(W_gate=Wg, W_up=Wu, W_down=Wd)
    y0 = oracle64.layer_forward(s, x, W_r, bias=bias, W_c=W_c, v=np.zeros_like(v), **kw)
    y1 = oracle64.layer_forward(s, x, W_r, bias=bias, W_c=W_c, v=v, **kw)
    y2 = oracle64.layer_forward(s, x, W_r, bias=bias, W_c=W_c, v=2 * v, **kw)
    np.testing.assert_allclose(y2["y"] - y1["y"], y1["y"] - y0["y"], rtol=1e-4, atol=1e-6)
    a = oracle64.const_alpha(s, x, W_c)
    np.testing.assert_allclose(y1["y"] - y0["y"], (y1["w"][:, 1] * a[:, 0, 1])[:, None] * v[0], rtol=1e-4, atol=1e-6)


# ------------------------------------------------------------------------------------------------
# gating residual (Eq. 6)
# ------------------------------------------------------------------------------------------------
def test_gating_residual_special_cases(oracle64):
    T, D, N = 40, 24, 7
    s = LayerShape(T=T, D=D, F=1, n_ffn=4, n_zero=1, n_copy=1, n_const=1)
    x, W_r, prev = _rand(T, D), _rand(N, D, std=0.3), _rand(T, N)
    G_plain = oracle64.router_logits(s, x, W_r)
    ref = (torch.from_numpy(x).double() @ torch.from_numpy(W_r).double().T).numpy()
    np.testing.assert_allclose(G_plain, ref, rtol=1e-5, atol=1e-6)  # Eq. 2 against a library matmul
    # W_g = 0 -> the vanilla router
    G0 = oracle64.router_logits(s, x, W_r, np.zeros((N, N), np.float32), prev)
    np.testing.assert_array_equal(G0, G_plain)
    # W_g = I and W_r = 0 -> the logits repeat
    Gi = oracle64.router_logits(s, x, np.zeros_like(W_r), np.eye(N, dtype=np.float32), prev)
    np.testing.assert_allclose(Gi, prev, rtol=0, atol=0)
    # W_g is applied as W_g @ G_prev (not its transpose)
    W_g = _rand(N, N, std=0.5)
    Gg = oracle64.router_logits(s, x, W_r, W_g, prev)
    ref = ref + (torch.from_numpy(prev).double() @ torch.from_numpy(W_g).double().T).numpy()
    np.testing.assert_allclose(Gg, ref, rtol=1e-5, atol=1e-5)
    # bias is added last
    b = _rand(N)
    np.testing.assert_allclose(oracle64.router_logits(s, x, W_r, W_g, prev, b), ref + b, rtol=1e-5, atol=1e-5)


def test_three_layer_logit_chain(oracle64):
    """G3 = W3 x3 + Wg3 (W2 x2 + Wg2 W1 x1), expanded with torch matmuls."""
    T, D, N = 10, 16, 6
    s = LayerShape(T=T, D=D, F=1, n_ffn=6)
    xs = [_rand(T, D) for _ in range(3)]
    Ws = [_rand(N, D, std=0.3) for _ in range(3)]
    Wgs = [None, _rand(N, N, std=0.5), _rand(N, N, std=0.5)]
    G = oracle64.router_logits(s, xs[0], Ws[0])
    for j in (1, 2):
        G = oracle64.router_logits(s, xs[j], Ws[j], Wgs[j], G)
    t = lambda a: torch.from_numpy(a).double()
    G1 = t(xs[0]) @ t(Ws[0]).T
    G2 = t(xs[1]) @ t(Ws[1]).T + G1 @ t(Wgs[1]).T
    G3 = t(xs[2]) @ t(Ws[2]).T + G2 @ t(Wgs[2]).T
    np.testing.assert_allclose(G, G3.numpy(), rtol=1e-5, atol=1e-5)


# ------------------------------------------------------------------------------------------------
# FFN expert and dense mixture against torch (library referee)
# ------------------------------------------------------------------------------------------------
@pytest.mark.parametrize("arith,tol", [("oracle64", 1e-6), ("oracle32", 2e-4)])
def test_single_ffn_expert_is_three_matmuls(arith, tol, request):
    o = request.getfixturevalue(arith)
    s = LayerShape(T=24, D=40, F=56, n_ffn=1, top_k=1)
    x, W_r = _rand(s.T, s.D), _rand(1, s.D)
    Wg, Wu, Wd = _ffn_weights(s)
    r = o.layer_forward(s, x, W_r, W_gate=Wg, W_up=Wu, W_down=Wd)
    np.testing.assert_allclose(r["w"], 1.0)
    ref = _torch_ffn(x, Wg[0], Wu[0], Wd[0])
    np.testing.assert_allclose(r["y"], ref, rtol=tol, atol=tol * np.abs(ref).max())
    np.testing.assert_allclose(o.ffn_token(s, x[3], Wg[0], Wu[0], Wd[0]), ref[3], rtol=tol, atol=tol * np.abs(ref).max())


def test_k_equals_n_is_dense_mixture(oracle64):
    """K = N: Eq. 1 has no mask left; y = sum_i P_i E_i(x), computed here without any top-k code."""
    s = LayerShape(T=12, D=20, F=28, n_ffn=3, n_zero=1, n_copy=1, n_const=1, top_k=6)
    x, W_r, W_c, v = _rand(s.T, s.D), _rand(s.N, s.D, std=0.3), _rand(1, 2, s.D, std=0.3), _rand(1, s.D)
    Wg, Wu, Wd = _ffn_weights(s)
    r = oracle64.layer_forward(s, x, W_r, W_c=W_c, v=v, W_gate=Wg, W_up=Wu, W_down=Wd)
    xt = torch.from_numpy(x).double()
    P = torch.softmax(xt @ torch.from_numpy(W_r).double().T, dim=1).numpy()
    a = torch.softmax(xt @ torch.from_numpy(W_c[0]).double().T, dim=1).numpy()
    ref = sum(P[:, i:i + 1] * _torch_ffn(x, Wg[i], Wu[i], Wd[i]) for i in range(3))
    ref = ref + P[:, 4:5] * x + P[:, 5:6] * (a[:, :1] * x + a[:, 1:] * v[0])  # zero expert (index 3) adds nothing
    np.testing.assert_allclose(r["y"], ref, rtol=1e-5, atol=1e-6)


def test_bf16_weight_path_equals_widened_floats(oracle64):
    s = LayerShape(T=8, D=32, F=48, n_ffn=2, n_zero=1, top_k=2)
    x, W_r = _rand(s.T, s.D), _rand(s.N, s.D, std=0.3)
    ws = [torch.from_numpy(w).to(torch.bfloat16) for w in _ffn_weights(s)]
    as_f32 = [w.float().numpy() for w in ws]
    as_bits = [w.view(torch.int16).numpy().view(np.uint16) for w in ws]
    ra = oracle64.layer_forward(s, x, W_r, W_gate=as_f32[0], W_up=as_f32[1], W_down=as_f32[2])
    rb = oracle64.layer_forward(s, x, W_r, W_gate=as_bits[0], W_up=as_bits[1], W_down=as_bits[2])
    np.testing.assert_array_equal(ra["y"], rb["y"])


# ------------------------------------------------------------------------------------------------
# vanilla MoE (Eq. 2) == MoE++ whose zero-computation experts can never be picked
# ------------------------------------------------------------------------------------------------
def test_vanilla_equals_masked_moepp(oracle64):
    s = LayerShape(T=64, D=32, F=40, n_ffn=6, n_zero=1, n_copy=1, n_const=2, top_k=2)
    x, W_r, W_c, v = _rand(s.T, s.D), _rand(s.N, s.D, std=0.3), _rand(2, 2, s.D), _rand(2, s.D)
    Wg, Wu, Wd = _ffn_weights(s)
    bias = np.zeros(s.N, np.float32)
    bias[s.n_ffn:] = -1e30
    r = oracle64.layer_forward(s, x, W_r, bias=bias, W_c=W_c, v=v, W_gate=Wg, W_up=Wu, W_down=Wd)
    sv = LayerShape(T=s.T, D=s.D, F=s.F, n_ffn=6, top_k=2)
    rv = oracle64.layer_forward(sv, x, W_r[:6], W_gate=Wg, W_up=Wu, W_down=Wd)
    assert np.array_equal(r["idx"], rv["idx"])
    np.testing.assert_allclose(r["w"], rv["w"], rtol=1e-6)
    np.testing.assert_allclose(r["y"], rv["y"], rtol=1e-6, atol=1e-7)


# ------------------------------------------------------------------------------------------------
# grouping tables
# ------------------------------------------------------------------------------------------------
@pytest.mark.parametrize("row_align", [1, 8, 128])
def test_table_invariants(oracle64, row_align):
    s = LayerShape(T=300, D=8, F=8, n_ffn=5, n_zero=1, n_copy=1, n_const=2, top_k=2, row_align=row_align)
    G = _rand(s.T, s.N)
    G[:7, s.n_ffn:] += 50.0  # a few tokens routed only to zero-computation experts
    idx, w = oracle64.gate_topk(s, G)
    counts, offsets, row_of_slot, slot_of_row = oracle64.tables(s, idx)
    flat = idx.reshape(-1)
    assert counts.sum() == s.T * s.top_k
    assert np.array_equal(counts, np.bincount(flat, minlength=s.N))
    assert offsets[0] == 0
    seg = np.diff(offsets)
    assert np.all(seg >= counts[:s.n_ffn]) and np.all(seg % row_align == 0) and np.all(seg - counts[:s.n_ffn] < row_align)
    if row_align == 1:
        assert offsets[-1] == (flat < s.n_ffn).sum()
    ros = row_of_slot.reshape(-1)
    ffn_slots = np.nonzero(flat < s.n_ffn)[0]
    assert np.all(ros[flat >= s.n_ffn] == -1)  # zero-computation slots own no row
    assert np.all(ros[:7 * s.top_k] == -1)  # tokens routed only to zero-computation experts: no FFN work
    rows = ros[ffn_slots]
    assert len(set(rows.tolist())) == len(rows)  # injective
    assert np.array_equal(slot_of_row[rows], ffn_slots)  # inverse
    assert (slot_of_row >= 0).sum() == len(ffn_slots)  # everything else is a pad row
    for e in range(s.n_ffn):
        seg_slots = slot_of_row[offsets[e]:offsets[e] + counts[e]]
        assert np.all(flat[seg_slots] == e)
        assert np.all(np.diff(seg_slots) > 0)  # ascending slot id inside an expert
        assert np.all(slot_of_row[offsets[e] + counts[e]:offsets[e + 1]] == -1)
    xp = oracle64.permute_rows(s, _x := _rand(s.T, s.D), slot_of_row)
    live = slot_of_row >= 0
    np.testing.assert_array_equal(xp[live], _x[slot_of_row[live] // s.top_k])
    assert np.all(xp[~live] == 0)


def test_staged_pipeline_equals_definition(oracle64):
    """tables + permute + grouped FFN + combine must reproduce the ungrouped definition."""
    for align in (1, 16):
        s = LayerShape(T=96, D=24, F=40, n_ffn=4, n_zero=1, n_copy=1, n_const=2, top_k=2, row_align=align)
        x, W_r, W_c, v = _rand(s.T, s.D), _rand(s.N, s.D, std=0.4), _rand(2, 2, s.D, std=0.3), _rand(2, s.D)
        W_g, prev = _rand(s.N, s.N, std=0.3), _rand(s.T, s.N)
        Wg, Wu, Wd = _ffn_weights(s)
        r = oracle64.layer_forward(s, x, W_r, W_g, prev, None, W_c, v, Wg, Wu, Wd)
        G = oracle64.router_logits(s, x, W_r, W_g, prev)
        np.testing.assert_array_equal(G, r["logits"])
        idx, w = oracle64.gate_topk(s, G)
        assert np.array_equal(idx, r["idx"])
        np.testing.assert_array_equal(w, r["w"])
        counts, offsets, row_of_slot, slot_of_row = oracle64.tables(s, idx)
        xp = oracle64.permute_rows(s, x, slot_of_row)
        yp = oracle64.grouped_ffn(s, xp, offsets, counts, Wg, Wu, Wd)
        alpha = oracle64.const_alpha(s, x, W_c)
        y = oracle64.combine(s, x, yp, idx, w, row_of_slot, alpha, v)
        np.testing.assert_allclose(y, r["y"], rtol=2e-6, atol=2e-6)


def test_token_permutation_equivariance_and_subset(oracle64):
    s = LayerShape(T=50, D=16, F=24, n_ffn=3, n_zero=1, n_copy=1, n_const=1, top_k=2, add_residual=1)
    x, W_r, W_c, v = _rand(s.T, s.D), _rand(s.N, s.D, std=0.4), _rand(1, 2, s.D, std=0.3), _rand(1, s.D)
    Wg, Wu, Wd = _ffn_weights(s)
    r = oracle64.layer_forward(s, x, W_r, W_c=W_c, v=v, W_gate=Wg, W_up=Wu, W_down=Wd)
    perm = rng.permutation(s.T)
    rp = oracle64.layer_forward(s, x[perm], W_r, W_c=W_c, v=v, W_gate=Wg, W_up=Wu, W_down=Wd)
    np.testing.assert_array_equal(rp["y"], r["y"][perm])
    toks = np.array([7, 0, 33, 49], np.int32)
    rs = oracle64.layer_forward(s, x, W_r, W_c=W_c, v=v, W_gate=Wg, W_up=Wu, W_down=Wd, tokens=toks)
    np.testing.assert_array_equal(rs["y"], r["y"][toks])
    # add_residual adds x once
    s0 = LayerShape(**{**s.__dict__, "add_residual": 0})
    r0 = oracle64.layer_forward(s0, x, W_r, W_c=W_c, v=v, W_gate=Wg, W_up=Wu, W_down=Wd)
    np.testing.assert_allclose(r["y"], r0["y"] + x, rtol=1e-6, atol=1e-6)


def test_forced_idx_uses_own_softmax(oracle64):
    s = LayerShape(T=20, D=16, F=24, n_ffn=3, n_zero=1, n_copy=1, n_const=1, top_k=2)
    x, W_r, W_c, v = _rand(s.T, s.D), _rand(s.N, s.D, std=0.4), _rand(1, 2, s.D, std=0.3), _rand(1, s.D)
    Wg, Wu, Wd = _ffn_weights(s)
    forced = np.tile(np.array([[4, 3]], np.int32), (s.T, 1))  # copy, zero
    r = oracle64.layer_forward(s, x, W_r, W_c=W_c, v=v, W_gate=Wg, W_up=Wu, W_down=Wd, forced_idx=forced)
    P = torch.softmax(torch.from_numpy(r["logits"]).double(), 1).numpy()
    np.testing.assert_allclose(r["w"], P[:, [4, 3]], rtol=1e-6)
    np.testing.assert_allclose(r["y"], P[:, 4:5] * x, rtol=1e-6, atol=1e-7)


def test_f32_and_f64_arithmetic_agree(oracle32, oracle64):
    s = LayerShape(T=64, D=256, F=512, n_ffn=8, n_zero=1, n_copy=1, n_const=2, top_k=2)
    x, W_r = _rand(s.T, s.D), _rand(s.N, s.D, std=0.02)
    W_g, prev, W_c, v = _rand(s.N, s.N, std=0.02), _rand(s.T, s.N), _rand(2, 2, s.D, std=0.02), _rand(2, s.D)
    Wg, Wu, Wd = _ffn_weights(s, std=0.02)
    a = oracle32.layer_forward(s, x, W_r, W_g, prev, None, W_c, v, Wg, Wu, Wd)
    b = oracle64.layer_forward(s, x, W_r, W_g, prev, None, W_c, v, Wg, Wu, Wd)
    same = np.all(a["idx"] == b["idx"], axis=1)
    assert same.mean() > 0.97
    assert np.abs(a["y"][same] - b["y"][same]).max() <= 1e-5
    assert np.abs(a["logits"] - b["logits"]).max() <= 1e-5
