"""Per-call GPU parity against the CPU oracle, through the C-ABI (route, permute, grouped FFN, combine).

Integer results (top-K indices on clear-gap tokens, counts, offsets, both permutation tables, gathered
rows) must be bit-exact; float results must be within the stated tolerances:
  float32 storage: max-abs 1e-4;  bf16 storage: per-token relative error 2e-2 against the float oracle.
"""
import numpy as np
import pytest
import torch

from harness import (clear_gap_tokens, f32, bits_or_f32, max_abs, oracle_inputs, rel_err_per_token, shape_of)
from paper_2410_07348_b200 import binding as B
from paper_2410_07348_b200 import workloads as W

pytestmark = pytest.mark.gpu

F32_ABS_TOL = 1e-4
BF16_REL_TOL = 2e-2


def dev(t, dtype=None):
    if t is None:
        return None
    if isinstance(t, np.ndarray):
        t = torch.from_numpy(t)
    t = t.cuda()
    return t.to(dtype).contiguous() if dtype is not None else t.contiguous()


def small_spec(dtype, T=777, D=328, F=392, n_ffn=5, n_const=2, top_k=2):
    return W.LayerSpec(T=T, D=D, F=F, n_ffn=n_ffn, n_zero=1, n_copy=1, n_const=n_const, top_k=top_k, dtype=dtype)


def run_route(cfg, lt, logits_in=None, want_alpha=True):
    T, N, K = cfg.T, cfg.N, cfg.top_k
    logits = torch.empty(T, N, device="cuda") if logits_in is None else dev(logits_in)
    idx = torch.empty(T, K, dtype=torch.int32, device="cuda")
    w = torch.empty(T, K, device="cuda")
    counts = torch.full((N,), -7, dtype=torch.int32, device="cuda")
    offsets = torch.full((cfg.n_ffn + 1,), -7, dtype=torch.int32, device="cuda")
    alpha = torch.empty(T, max(cfg.n_const, 1), 2, device="cuda") if (want_alpha and cfg.n_const) else None
    B.moepp_route(cfg, dev(lt.x), dev(lt.W_r), dev(lt.W_g), dev(lt.prev), dev(lt.bias), dev(lt.W_c), logits, idx, w,
                  counts, offsets, alpha)
    torch.cuda.synchronize()
    return dict(logits=logits.cpu().numpy(), idx=idx.cpu().numpy(), w=w.cpu().numpy(), counts=counts.cpu().numpy(),
                offsets=offsets.cpu().numpy(), alpha=None if alpha is None else alpha.cpu().numpy())


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
@pytest.mark.parametrize("shape", [dict(), dict(T=1), dict(T=33, n_ffn=40, n_const=8, top_k=4, D=64, F=64),
                                   dict(T=300, n_ffn=0, D=128), dict(T=257, n_ffn=3, n_const=0, D=1032)])
def test_route(oracle64, dtype, shape):
    spec = small_spec(dtype, **shape)
    lt = W.make_layer(spec, seed=3)
    cfg = B.config_from_spec(spec)
    s, oi = shape_of(spec), oracle_inputs(lt)
    G = oracle64.router_logits(s, oi["x"], oi["W_r"], oi["W_g"], oi["prev"])
    idx_o, w_o = oracle64.gate_topk(s, G)
    counts_o, offsets_o, _, _ = oracle64.tables(s, idx_o)

    r = run_route(cfg, lt)
    assert max_abs(r["logits"], G) <= F32_ABS_TOL
    clear = clear_gap_tokens(G, spec.top_k)
    if spec.T >= 100:
        assert clear.mean() > 0.8
    assert np.array_equal(r["idx"][clear], idx_o[clear])
    assert max_abs(r["w"][clear], w_o[clear]) <= 1e-5
    if spec.n_const:
        assert max_abs(r["alpha"], oracle64.const_alpha(s, oi["x"], oi["W_c"])) <= 1e-5
    # the tables are exact functions of the GPU's own picks
    c2, o2, _, _ = oracle64.tables(s, r["idx"])
    assert np.array_equal(r["counts"], c2) and np.array_equal(r["offsets"], o2)

    # fed the oracle's logits, the picks, counts and offsets are bit-exact on every token
    cfg_given = B.config_from_spec(spec, flags=B.FLAG_LOGITS_GIVEN)
    rg = run_route(cfg_given, lt, logits_in=G)
    assert np.array_equal(rg["idx"], idx_o)
    assert np.array_equal(rg["counts"], counts_o) and np.array_equal(rg["offsets"], offsets_o)
    assert max_abs(rg["w"], w_o) <= 1e-6
    assert np.array_equal(rg["logits"], G)  # untouched
    if spec.n_const:
        assert max_abs(rg["alpha"], oracle64.const_alpha(s, oi["x"], oi["W_c"])) <= 1e-5


def test_route_variants(oracle64):
    """Bias, first layer (no gating residual), renormalised weights, row_align, exact ties."""
    spec = small_spec("bf16")
    lt = W.make_layer(spec, seed=5, with_prev=False)
    lt.bias = torch.linspace(-0.5, 0.5, spec.N)
    for over in (dict(), dict(renorm_topk=1), dict(row_align=128), dict(row_align=8, renorm_topk=1)):
        cfg = B.config_from_spec(spec, **over)
        s, oi = shape_of(spec, **over), oracle_inputs(lt)
        G = oracle64.router_logits(s, oi["x"], oi["W_r"], None, None, oi["bias"])
        r = run_route(cfg, lt)
        assert max_abs(r["logits"], G) <= F32_ABS_TOL
        cfg_g = B.config_from_spec(spec, flags=B.FLAG_LOGITS_GIVEN, **over)
        rg = run_route(cfg_g, lt, logits_in=G)
        idx_o, w_o = oracle64.gate_topk(s, G)
        counts_o, offsets_o, _, _ = oracle64.tables(s, idx_o)
        assert np.array_equal(rg["idx"], idx_o) and max_abs(rg["w"], w_o) <= 1e-6
        assert np.array_equal(rg["counts"], counts_o) and np.array_equal(rg["offsets"], offsets_o)
        if over.get("renorm_topk"):
            np.testing.assert_allclose(rg["w"].sum(1), 1.0, atol=1e-6)
    # exact ties: equal logits go to the lower index
    G = np.zeros((spec.T, spec.N), np.float32)
    G[:, 4] = 1.0
    rg = run_route(B.config_from_spec(spec, flags=B.FLAG_LOGITS_GIVEN), lt, logits_in=G)
    assert np.all(rg["idx"] == [4, 0])


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
@pytest.mark.parametrize("row_align", [1, 8, 128])
@pytest.mark.parametrize("T", [1, 777, 5000])
def test_permute(oracle64, dtype, row_align, T):
    spec = small_spec(dtype, T=T)
    lt = W.make_layer(spec, seed=7)
    cfg = B.config_from_spec(spec, row_align=row_align)
    s, oi = shape_of(spec, row_align=row_align), oracle_inputs(lt)
    G = oracle64.router_logits(s, oi["x"], oi["W_r"], oi["W_g"], oi["prev"])
    if T >= 100:
        G[:9, spec.n_ffn:] += 30.0  # some tokens routed only to zero-computation experts
        G[:, 2] -= 30.0  # an FFN expert nobody picks
    idx_o, _ = oracle64.gate_topk(s, G)
    counts_o, offsets_o, ros_o, sor_o = oracle64.tables(s, idx_o)
    xp_o = oracle64.permute_rows(s, oi["x"], sor_o)

    ros = torch.full((T, spec.top_k), -9, dtype=torch.int32, device="cuda")
    sor = torch.full((cfg.M_cap,), -9, dtype=torch.int32, device="cuda")
    xp = torch.full((cfg.M_cap, spec.D), 3.0, dtype=W.torch_dtype(dtype), device="cuda")
    B.moepp_permute(cfg, dev(lt.x), dev(idx_o), dev(offsets_o), ros, sor, xp)
    torch.cuda.synchronize()
    assert np.array_equal(ros.cpu().numpy(), ros_o)
    assert np.array_equal(sor.cpu().numpy(), sor_o)
    used = int(offsets_o[-1])
    assert np.array_equal(xp[:used].float().cpu().numpy(), xp_o[:used])  # a gather is exact in any dtype
    assert torch.all(xp[used:].float() == 3.0)  # rows beyond the rows in use are not touched


def ffn_case(oracle64, dtype, flags=0, row_align=1, T=777, **shape):
    spec = small_spec(dtype, T=T, **shape)
    lt = W.make_layer(spec, seed=11, w_std=0.05)
    cfg = B.config_from_spec(spec, row_align=row_align, flags=flags)
    s, oi = shape_of(spec, row_align=row_align), oracle_inputs(lt)
    G = oracle64.router_logits(s, oi["x"], oi["W_r"], oi["W_g"], oi["prev"])
    if spec.n_ffn >= 4 and T >= 100:
        G[:, 1] -= 30.0  # empty expert
        G[:, 0] += 1.0   # a crowded one: several row tiles
    idx_o, _ = oracle64.gate_topk(s, G)
    counts_o, offsets_o, ros_o, sor_o = oracle64.tables(s, idx_o)
    xp_o = oracle64.permute_rows(s, oi["x"], sor_o)
    yp_o = oracle64.grouped_ffn(s, xp_o, offsets_o, counts_o, oi["W_gate"], oi["W_up"], oi["W_down"])

    td = W.torch_dtype(dtype)
    xp = dev(xp_o, td)
    if cfg.M_cap > int(offsets_o[-1]):  # rows beyond the rows in use hold garbage in real life
        xp[int(offsets_o[-1]):] = float("nan")
    h = torch.full((cfg.M_cap, spec.F), float("nan"), dtype=td, device="cuda")
    yp = torch.full((cfg.M_cap, spec.D), 5.0, dtype=td, device="cuda")
    B.moepp_grouped_ffn(cfg, xp, dev(offsets_o), dev(lt.W_gate), dev(lt.W_up), dev(lt.W_down), h, yp)
    torch.cuda.synchronize()
    assert B.moepp_device_error() == 0
    live = sor_o >= 0
    got = yp.float().cpu().numpy()
    if dtype == "f32":
        assert max_abs(got[live], yp_o[live]) <= F32_ABS_TOL
        assert rel_err_per_token(got[live], yp_o[live]) <= 1e-4
    else:
        assert rel_err_per_token(got[live], yp_o[live]) <= BF16_REL_TOL
    # rows at or beyond the rows in use are never written
    assert torch.all(yp[int(offsets_o[-1]):].float() == 5.0)
    return rel_err_per_token(got[live], yp_o[live])


@pytest.mark.parametrize("row_align", [1, 128])
def test_grouped_ffn_f32(oracle64, row_align):
    ffn_case(oracle64, "f32", row_align=row_align)


@pytest.mark.parametrize("row_align", [1, 128])
def test_grouped_ffn_bf16_fma_path(oracle64, row_align):
    ffn_case(oracle64, "bf16", flags=B.FLAG_SIMT_FFN, row_align=row_align)


@pytest.mark.parametrize("row_align", [1, 128])
@pytest.mark.parametrize("shape", [dict(), dict(D=256, F=512), dict(T=1, D=64, F=64), dict(T=40, D=1024, F=136),
                                   dict(T=3000, D=512, F=1024, n_ffn=3)])
def test_grouped_ffn_bf16_tensor_cores(oracle64, row_align, shape):
    ffn_case(oracle64, "bf16", row_align=row_align, **shape)  # CTA pairs, 256 x 256 tiles
    ffn_case(oracle64, "bf16", row_align=row_align, flags=B.FLAG_FFN_SINGLE_CTA, **shape)  # single CTAs, 128 x 256


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
@pytest.mark.parametrize("alpha_given", [True, False])
@pytest.mark.parametrize("add_residual", [0, 1])
def test_combine(oracle64, dtype, alpha_given, add_residual):
    spec = small_spec(dtype, top_k=3)
    lt = W.make_layer(spec, seed=13)
    cfg = B.config_from_spec(spec, add_residual=add_residual)
    s, oi = shape_of(spec, add_residual=add_residual), oracle_inputs(lt)
    G = oracle64.router_logits(s, oi["x"], oi["W_r"], oi["W_g"], oi["prev"])
    G[:, spec.n_ffn:] += 0.3  # plenty of zero-computation picks of every kind
    idx_o, w_o = oracle64.gate_topk(s, G)
    counts_o, offsets_o, ros_o, sor_o = oracle64.tables(s, idx_o)
    td = W.torch_dtype(dtype)
    yp_t = (torch.randn(cfg.M_cap, spec.D, generator=torch.Generator().manual_seed(1)) * 0.5).to(td)
    alpha_o = oracle64.const_alpha(s, oi["x"], oi["W_c"])
    y_o = oracle64.combine(s, oi["x"], f32(yp_t), idx_o, w_o, ros_o, alpha_o, oi["v"])

    y = torch.empty(spec.T, spec.D, dtype=td, device="cuda")
    B.moepp_combine(cfg, dev(lt.x), dev(yp_t), dev(idx_o), dev(w_o), dev(ros_o),
                    dev(alpha_o) if alpha_given else None, dev(lt.W_c), dev(lt.v), y)
    torch.cuda.synchronize()
    got = y.float().cpu().numpy()
    if dtype == "f32":
        assert max_abs(got, y_o) <= F32_ABS_TOL
    else:
        assert rel_err_per_token(got, y_o) <= BF16_REL_TOL
    # closed forms on the GPU result itself: tokens routed to {copy, zero} only come out as g_copy * x
    zero, copy = spec.n_ffn, spec.n_ffn + 1
    only = np.all((idx_o == zero) | (idx_o == copy), axis=1)
    if only.any() and dtype == "f32":
        g = (w_o * (idx_o == copy)).sum(1) + add_residual
        assert max_abs(got[only], g[only, None] * oi["x"][only]) <= 1e-5


def test_argument_errors_on_device():
    spec = small_spec("bf16")
    cfg = B.config_from_spec(spec)
    x = torch.zeros(spec.T, spec.D, dtype=torch.bfloat16, device="cuda")
    with pytest.raises(B.MoeppError) as ei:  # missing outputs
        B.moepp_route(cfg, x, None, None, None, None, None, None, None, None, None, None, None)
    assert ei.value.status == 1
    ws = torch.empty(1024, dtype=torch.uint8, device="cuda")
    lt = W.make_layer(W.LayerSpec(T=8, D=64, F=64, n_ffn=2), seed=0)
    wd = B.weights_from_tensors(lt)
    c8 = B.config_from_spec(lt.spec)
    y = torch.empty(8, 64, dtype=torch.bfloat16, device="cuda")
    with pytest.raises(B.MoeppError) as ei:  # workspace too small
        B.moepp_layer_forward(c8, wd, lt.x.cuda(), lt.prev.cuda(), y, None, ws)
    assert ei.value.status == 4
    with pytest.raises(B.MoeppError) as ei:  # misaligned activation pointer
        buf = torch.zeros(8 * 64 + 8, dtype=torch.bfloat16, device="cuda")
        big = torch.empty(B.moepp_workspace_bytes(c8), dtype=torch.uint8, device="cuda")
        B.moepp_layer_forward(c8, wd, buf[1:1 + 8 * 64].view(8, 64), lt.prev.cuda(), y, None, big)
    assert ei.value.status == 3
