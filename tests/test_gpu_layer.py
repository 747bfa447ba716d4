"""Whole-layer GPU parity against the CPU oracle on the benchmark configurations, through the C-ABI.

For every configuration: logits within 1e-4 of the oracle, top-K picks bit-exact on every token whose
leading logits are more than 1e-3 apart, and the layer output compared with the oracle run on the
GPU's own picks (so that every token's arithmetic is checked even where a near-tie went the other way):
float32 within max-abs 1e-4, bf16 within per-token relative error 2e-2.  Large configurations are
checked on a token sample (tokens are independent through the layer and through a stack).
"""
import math

import numpy as np
import pytest
import torch

from harness import clear_gap_tokens, f32, max_abs, oracle_inputs, rel_err_per_token, sample_tokens, shape_of
from paper_2410_07348_b200 import binding as B
from paper_2410_07348_b200 import workloads as W

pytestmark = pytest.mark.gpu

F32_ABS_TOL = 1e-4
BF16_REL_TOL = 2e-2
LOGIT_TOL = 2e-4


def gpu_layer(cfg, wd, x, prev, host=False):
    """Runs moepp_layer_forward (or its host-buffer variant) and, with the same inputs, moepp_route to
    expose the picks the layer used."""
    T, N, K = cfg.T, cfg.N, cfg.top_k
    td = torch.bfloat16 if cfg.dtype == B.MOEPP_BF16 else torch.float32
    if host:
        ws = torch.empty(B.moepp_workspace_bytes(cfg, host=True), dtype=torch.uint8, device="cuda")
        xh = x.cpu().pin_memory()
        ph = None if prev is None else prev.cpu().pin_memory()
        yh = torch.empty(T, cfg.D, dtype=td).pin_memory()
        lh = torch.empty(T, N).pin_memory()
        B.moepp_layer_forward_host(cfg, wd, xh, ph, yh, lh, ws)
        torch.cuda.synchronize()
        y, logits = yh.cuda(), lh.cuda()
    else:
        ws = torch.empty(B.moepp_workspace_bytes(cfg), dtype=torch.uint8, device="cuda")
        y = torch.empty(T, cfg.D, dtype=td, device="cuda")
        logits = torch.empty(T, N, device="cuda")
        B.moepp_layer_forward(cfg, wd, x, prev, y, logits, ws)
    idx = torch.empty(T, K, dtype=torch.int32, device="cuda")
    w = torch.empty(T, K, device="cuda")
    counts = torch.empty(N, dtype=torch.int32, device="cuda")
    offsets = torch.empty(cfg.n_ffn + 1, dtype=torch.int32, device="cuda")
    lg2 = torch.empty(T, N, device="cuda")
    B.moepp_route(cfg, x, wd["W_r"], wd["W_g"], prev, wd["router_bias"], None, lg2, idx, w, counts, offsets, None)
    torch.cuda.synchronize()
    assert B.moepp_device_error() == 0
    assert torch.equal(lg2, logits)
    return y, logits, idx.cpu().numpy(), counts.cpu().numpy()


def check_layer(oracle64, lt, n_sample, host=False, **over):
    spec = lt.spec
    cfg = B.config_from_spec(spec, **over)
    wd = B.weights_from_tensors(lt)
    x, prev = lt.x.cuda(), None if lt.prev is None else lt.prev.cuda()
    y, logits, idx_g, counts = gpu_layer(cfg, wd, x, prev, host=host)
    s, oi = shape_of(spec, **{k: v for k, v in over.items()
                              if k in ("renorm_topk", "row_align", "add_residual", "tau", "capacity_factor")}), \
        oracle_inputs(lt)
    toks = None if n_sample is None else sample_tokens(idx_g, spec.N, n_sample)
    r = oracle64.layer_forward(s, oi["x"], oi["W_r"], oi["W_g"], oi["prev"], oi["bias"], oi["W_c"], oi["v"],
                               oi["W_gate"], oi["W_up"], oi["W_down"], forced_idx=idx_g, tokens=toks)
    lg = logits.cpu().numpy()
    assert max_abs(lg, r["logits"]) <= LOGIT_TOL
    idx_o, _ = oracle64.gate_topk(s, r["logits"])
    clear = clear_gap_tokens(r["logits"], spec.top_k)
    assert np.array_equal(idx_g[clear], idx_o[clear])
    if spec.T >= 200:
        assert clear.mean() > 0.9
    got = y.float().cpu().numpy()
    got = got if toks is None else got[toks]
    if spec.dtype == "f32":
        assert max_abs(got, r["y"]) <= F32_ABS_TOL
    else:
        assert rel_err_per_token(got, r["y"]) <= BF16_REL_TOL
    assert counts.sum() == spec.T * spec.top_k
    return dict(zc_share=float(counts[spec.n_ffn:].sum()) / max(1, counts.sum()), counts=counts)


def test_cfg1_tiny_f32(oracle64, oracle32):
    lt = W.make_config("cfg1_tiny_f32")
    info = check_layer(oracle64, lt, None)
    assert 0.2 < info["zc_share"] < 0.5
    check_layer(oracle64, lt, None, renorm_topk=1, add_residual=1, row_align=128)
    check_layer(oracle64, lt, None, host=True)


def test_cfg1_vanilla_and_first_layer(oracle64):
    lt = W.make_layer(W.CONFIGS["cfg1_tiny_f32"].vanilla(), seed=0, with_prev=False)
    check_layer(oracle64, lt, None)


def test_cfg2_bf16(oracle64):
    lt = W.make_config("cfg2_bf16_8e", gen_device="cuda", device="cuda")
    info = check_layer(oracle64, lt, 192)
    assert 0.2 < info["zc_share"] < 0.5
    check_layer(oracle64, lt, 64, host=True)
    check_layer(oracle64, lt, 64, flags=B.FLAG_SIMT_FFN)
    check_layer(oracle64, lt, 64, flags=B.FLAG_FFN_SINGLE_CTA)  # 128 x 256 tiles on single CTAs
    check_layer(oracle64, lt, 64, flags=B.FLAG_FUSED_GATHER)  # GEMM 1 gathers its rows from x


def test_cfg3_bf16_skewed(oracle64):
    lt = W.make_config("cfg3_bf16_16e_skew", gen_device="cuda", device="cuda")
    info = check_layer(oracle64, lt, 96)
    assert abs(info["zc_share"] - 0.30) < 0.02
    c = info["counts"][:16].astype(np.float64)
    assert c[0] > 8 * c[15]  # Zipf(1.1) over 16 experts: rank 1 carries about 21x rank 16


@pytest.mark.parametrize("seed", range(8))
def test_random_shapes(oracle64, seed):
    """Seeded random small configurations: sizes, expert mix, top-k, padding, capacity, both storage types."""
    rng = np.random.default_rng(1000 + seed)
    dtype = "bf16" if seed % 2 == 0 else "f32"
    n_ffn = int(rng.integers(1, 12))
    n_zero, n_copy, n_const = int(rng.integers(0, 3)), int(rng.integers(0, 3)), int(rng.integers(0, 4))
    N = n_ffn + n_zero + n_copy + n_const
    spec = W.LayerSpec(T=int(rng.integers(1, 1500)), D=8 * int(rng.integers(1, 70)), F=8 * int(rng.integers(1, 70)),
                       n_ffn=n_ffn, n_zero=n_zero, n_copy=n_copy, n_const=n_const,
                       top_k=int(rng.integers(1, min(N, 4) + 1)), dtype=dtype)
    lt = W.make_layer(spec, seed=seed, with_prev=bool(seed & 2), w_std=0.05)
    over = dict(row_align=int(rng.choice([1, 8, 128])), add_residual=int(rng.integers(0, 2)),
                renorm_topk=int(rng.integers(0, 2)))
    if seed % 3 == 0:
        over.update(capacity_factor=float(rng.choice([0.7, 1.1])), tau=float(rng.choice([0.5, 0.75, 1.0])))
    check_layer(oracle64, lt, None, **over)


def test_tiny_dims_bf16(oracle64):
    """d_model and d_ffn far below one tile (8 and 16)."""
    spec = W.LayerSpec(T=300, D=8, F=16, n_ffn=3, dtype="bf16")
    check_layer(oracle64, W.make_layer(spec, seed=4, w_std=0.3), None)


def test_paper_2b_shape_32_plus_8_experts(oracle64):
    """The paper's 2B/(32+8)E layer (Table 2): 40 experts, six constant experts, 52 stacked router rows."""
    lt = W.make_config("paper_2b_32p8e", gen_device="cuda", device="cuda")
    info = check_layer(oracle64, lt, 160)
    assert 0.1 < info["zc_share"] < 0.35
    assert np.all(info["counts"] > 0)


@pytest.mark.parametrize("name", ["paper_06b_8p4e", "paper_1b_16p4e"])
def test_paper_small_model_shapes(oracle64, name):
    """The 0.6B/(8+4)E and 1B/(16+4)E layers of Table 2 (hidden 768, intermediate 2048)."""
    lt = W.make_config(name, gen_device="cuda", device="cuda")
    info = check_layer(oracle64, lt, 96)
    assert np.all(info["counts"] > 0)


def test_cfg4_stack_of_four(oracle64):
    """Free-running 4-layer stack on all 32768 tokens; the oracle follows the same picks on a token sample."""
    spec = W.CONFIGS["cfg4_7b_stack"]
    n_tok = 48
    rng = np.random.default_rng(0)
    toks = np.sort(rng.choice(spec.T, n_tok, replace=False)).astype(np.int32)
    sub = W.LayerSpec(n_tok, spec.D, spec.F, spec.n_ffn, spec.n_zero, spec.n_copy, spec.n_const, spec.top_k, "bf16")
    cfg = B.config_from_spec(spec, add_residual=1)
    ws = torch.empty(B.moepp_workspace_bytes(cfg), dtype=torch.uint8, device="cuda")
    x = None
    prev = None
    x_o = None
    prev_o = None
    s_sub = shape_of(sub, add_residual=1)
    kept, x_first = [], None
    for j in range(1, 5):
        # build one layer at a time to bound memory: same recipe as workloads.make_stack
        lt = W.make_layer(spec if j == 1 else W.LayerSpec(0, spec.D, spec.F, spec.n_ffn, dtype="bf16"), seed=j - 1,
                          with_prev=False, w_std=0.02 / math.sqrt(j), device="cuda", gen_device="cuda")
        if j == 1:
            x = lt.x
            x_first = x
            x_o = f32(x)[toks]
        else:
            g = torch.Generator(device="cuda").manual_seed(1000 + j)
            lt.W_g = W._randn(g, (spec.N, spec.N), 0.02 / math.sqrt(j), torch.float32, "cuda")
        lt.spec = spec
        wd = B.weights_from_tensors(lt)
        y = torch.empty_like(x)
        logits = torch.empty(spec.T, spec.N, device="cuda")
        B.moepp_layer_forward(cfg, wd, x, prev, y, logits, ws)
        idx = torch.empty(spec.T, spec.top_k, dtype=torch.int32, device="cuda")
        wk = torch.empty(spec.T, spec.top_k, device="cuda")
        cnt = torch.empty(spec.N, dtype=torch.int32, device="cuda")
        off = torch.empty(spec.n_ffn + 1, dtype=torch.int32, device="cuda")
        lg2 = torch.empty_like(logits)
        B.moepp_route(cfg, x, wd["W_r"], wd["W_g"], prev, None, None, lg2, idx, wk, cnt, off, None)
        torch.cuda.synchronize()
        assert B.moepp_device_error() == 0
        idx_g = idx.cpu().numpy()[toks]
        # oracle on the sampled tokens, float activations carried from layer to layer
        lt.x = None
        lt.prev = None
        oi = oracle_inputs(lt)
        r = oracle64.layer_forward(s_sub, x_o, oi["W_r"], oi["W_g"], prev_o, None, oi["W_c"], oi["v"], oi["W_gate"],
                                   oi["W_up"], oi["W_down"], forced_idx=idx_g)
        got = y.float().cpu().numpy()[toks]
        assert rel_err_per_token(got, r["y"]) <= BF16_REL_TOL, "layer %d" % j
        lg = logits.cpu().numpy()[toks]
        assert max_abs(lg, r["logits"]) <= 5e-2  # inputs differ by the bf16 rounding carried down the stack
        idx_o, _ = oracle64.gate_topk(s_sub, r["logits"])
        clear = clear_gap_tokens(r["logits"], spec.top_k, gap=0.1)
        assert np.array_equal(idx_g[clear], idx_o[clear])
        x, prev = y, logits
        x_o, prev_o = r["y"], r["logits"]
        kept.append(wd)
        del lt
    # the call bench.py times: the whole stack in one moepp_stack_forward, same bits as the chained calls
    ws2 = torch.empty(B.moepp_stack_workspace_bytes(cfg, 4), dtype=torch.uint8, device="cuda")
    y2 = torch.empty_like(x)
    lg2 = torch.empty(spec.T, spec.N, device="cuda")
    B.moepp_stack_forward(cfg, kept, x_first, None, y2, lg2, ws2)
    torch.cuda.synchronize()
    assert B.moepp_device_error() == 0
    assert torch.equal(y2, x) and torch.equal(lg2, prev)


def test_stack_call_equals_chained_layer_calls(oracle64):
    """moepp_stack_forward (and its host-buffer form) = the same layers called one after another."""
    spec = W.LayerSpec(T=1500, D=512, F=768, n_ffn=6, dtype="bf16")
    layers = W.make_stack(spec, 3, device="cuda", gen_device="cuda")
    cfg = B.config_from_spec(spec, add_residual=1)
    wds = [B.weights_from_tensors(lt) for lt in layers]
    x = layers[0].x
    ws = torch.empty(B.moepp_workspace_bytes(cfg), dtype=torch.uint8, device="cuda")
    cur, prev = x, None
    for wd in wds:
        y = torch.empty_like(x)
        lg = torch.empty(spec.T, spec.N, device="cuda")
        B.moepp_layer_forward(cfg, wd, cur, prev if wd["W_g"] is not None else None, y, lg, ws)
        cur, prev = y, lg
    ws2 = torch.empty(B.moepp_stack_workspace_bytes(cfg, 3, host=True), dtype=torch.uint8, device="cuda")
    y2 = torch.empty_like(x)
    lg2 = torch.empty(spec.T, spec.N, device="cuda")
    B.moepp_stack_forward(cfg, wds, x, None, y2, lg2, ws2)
    torch.cuda.synchronize()
    assert torch.equal(y2, cur) and torch.equal(lg2, prev)
    xh, yh, lh = x.cpu().pin_memory(), torch.empty_like(x, device="cpu").pin_memory(), torch.empty(spec.T, spec.N).pin_memory()
    B.moepp_stack_forward_host(cfg, wds, xh, None, yh, lh, ws2)
    torch.cuda.synchronize()
    assert torch.equal(yh.cuda(), cur) and torch.equal(lh.cuda(), prev)
    assert B.moepp_device_error() == 0
    # against the oracle: free-running chain on all tokens, following the GPU's picks layer by layer
    s = shape_of(spec, add_residual=1)
    x_o, prev_o = f32(x), None
    cur, prev = x, None
    for wd, lt in zip(wds, layers):
        idx = torch.empty(spec.T, spec.top_k, dtype=torch.int32, device="cuda")
        tmp = [torch.empty(spec.T, spec.top_k, device="cuda"), torch.empty(spec.N, dtype=torch.int32, device="cuda"),
               torch.empty(spec.n_ffn + 1, dtype=torch.int32, device="cuda"), torch.empty(spec.T, spec.N, device="cuda")]
        B.moepp_route(cfg, cur, wd["W_r"], wd["W_g"], prev if wd["W_g"] is not None else None, None, None, tmp[3], idx,
                      tmp[0], tmp[1], tmp[2], None)
        y = torch.empty_like(x)
        lg = torch.empty(spec.T, spec.N, device="cuda")
        B.moepp_layer_forward(cfg, wd, cur, prev if wd["W_g"] is not None else None, y, lg, ws)
        torch.cuda.synchronize()
        lt.x, lt.prev = None, None
        oi = oracle_inputs(lt)
        r = oracle64.layer_forward(s, x_o, oi["W_r"], oi["W_g"], prev_o if oi["W_g"] is not None else None, None,
                                   oi["W_c"], oi["v"], oi["W_gate"], oi["W_up"], oi["W_down"],
                                   forced_idx=idx.cpu().numpy())
        assert rel_err_per_token(y.float().cpu().numpy(), r["y"]) <= BF16_REL_TOL
        cur, prev, x_o, prev_o = y, lg, r["y"], r["logits"]


@pytest.mark.parametrize("T", [5000, 20000])
def test_host_stack_call_chunks_tokens(T):
    """The host-buffer stack call cuts large batches into token chunks that overlap copies with compute; the
    result must be the same bits as the device call on the whole batch."""
    spec = W.LayerSpec(T=T, D=256, F=384, n_ffn=6, dtype="bf16")
    layers = W.make_stack(spec, 2, device="cuda", gen_device="cuda")
    cfg = B.config_from_spec(spec, add_residual=1)
    wds = [B.weights_from_tensors(lt) for lt in layers]
    x = layers[0].x
    ws = torch.empty(B.moepp_stack_workspace_bytes(cfg, 2), dtype=torch.uint8, device="cuda")
    y = torch.empty_like(x)
    lg = torch.empty(T, spec.N, device="cuda")
    B.moepp_stack_forward(cfg, wds, x, None, y, lg, ws)
    wsh = torch.empty(B.moepp_stack_workspace_bytes(cfg, 2, host=True), dtype=torch.uint8, device="cuda")
    xh = x.cpu().pin_memory()
    for _ in range(2):  # twice in a row: the second call must wait for nothing it should not and reuse cleanly
        yh = torch.zeros_like(x, device="cpu").pin_memory()
        lh = torch.zeros(T, spec.N).pin_memory()
        B.moepp_stack_forward_host(cfg, wds, xh, None, yh, lh, wsh)
        torch.cuda.current_stream().synchronize()
        assert torch.equal(yh, y.cpu()) and torch.equal(lh, lg.cpu())
    assert B.moepp_device_error() == 0


def test_cfg4_teacher_forced_layers(oracle64):
    """Each layer of the stack fed the oracle's own state (rounded once to bf16): picks exact, outputs in tolerance."""
    spec = W.CONFIGS["cfg4_7b_stack"]
    T = 256
    sub = W.LayerSpec(T, spec.D, spec.F, spec.n_ffn, spec.n_zero, spec.n_copy, spec.n_const, spec.top_k, "bf16")
    s = shape_of(sub, add_residual=1)
    cfg = B.config_from_spec(sub, add_residual=1)
    x_o = None
    prev_o = None
    for j in range(1, 5):
        lt = W.make_layer(sub if j == 1 else W.LayerSpec(0, spec.D, spec.F, spec.n_ffn, dtype="bf16"), seed=j - 1,
                          with_prev=False, w_std=0.02 / math.sqrt(j), device="cuda", gen_device="cuda")
        if j == 1:
            x_t = lt.x
        else:
            g = torch.Generator(device="cuda").manual_seed(1000 + j)
            lt.W_g = W._randn(g, (spec.N, spec.N), 0.02 / math.sqrt(j), torch.float32, "cuda")
            x_t = torch.from_numpy(x_o).to(torch.bfloat16).cuda()
        lt.spec, lt.x = sub, x_t
        lt.prev = None if prev_o is None else torch.from_numpy(prev_o).cuda()
        check_layer(oracle64, lt, 32, add_residual=1)
        oi = oracle_inputs(lt)
        r = oracle64.layer_forward(s, oi["x"], oi["W_r"], oi["W_g"], oi["prev"], None, oi["W_c"], oi["v"], oi["W_gate"],
                                   oi["W_up"], oi["W_down"], tokens=np.arange(T, dtype=np.int32))
        x_o, prev_o = r["y"], r["logits"]


@pytest.mark.parametrize("T,share", [(128, 0.0), (128, 0.5), (2048, 0.15), (2048, 0.75), (32768, 0.30)])
def test_cfg5_sweep_points(oracle64, T, share):
    lt = W.make_config("cfg5_sweep", T=T, zc_share=share, gen_device="cuda", device="cuda")
    info = check_layer(oracle64, lt, 48)
    assert abs(info["zc_share"] - share) < 0.03


def test_empty_and_degenerate(oracle64):
    # T = 0 is valid and does nothing
    spec = W.LayerSpec(T=0, D=64, F=64, n_ffn=2, dtype="bf16")
    lt = W.make_layer(spec, seed=0)
    cfg = B.config_from_spec(spec)
    ws = torch.empty(B.moepp_workspace_bytes(cfg), dtype=torch.uint8, device="cuda")
    y = torch.empty(0, 64, dtype=torch.bfloat16, device="cuda")
    B.moepp_layer_forward(cfg, B.weights_from_tensors(lt), lt.x.cuda(), lt.prev.cuda(), y, None, ws)
    torch.cuda.synchronize()
    # a layer of zero-computation experts only (no FFN expert at all)
    spec = W.LayerSpec(T=100, D=64, F=0, n_ffn=0, n_zero=1, n_copy=1, n_const=2, dtype="f32")
    check_layer(oracle64, W.make_layer(spec, seed=1), None)
    # every slot on zero-computation experts although FFN experts exist: no FFN work at all
    spec = W.LayerSpec(T=300, D=128, F=256, n_ffn=4, dtype="bf16")
    lt = W.make_layer(spec, seed=2)
    lt.bias = torch.tensor([-50.0] * 4 + [50.0] * 4)
    info = check_layer(oracle64, lt, None)
    assert info["zc_share"] == 1.0
    # top-1 and top-4
    for k in (1, 4):
        spec = W.LayerSpec(T=200, D=128, F=256, n_ffn=6, top_k=k, dtype="bf16")
        check_layer(oracle64, W.make_layer(spec, seed=3), None)


@pytest.mark.parametrize("gamma,tau", [(1.1, 0.75), (0.6, 0.5), (8.0, 0.75)])
def test_capacity_limited_layer(oracle64, gamma, tau):
    """Eq. 8: slots beyond an expert's capacity are dropped in slot order (no row, no FFN work, no contribution)."""
    spec = W.LayerSpec(T=3000, D=256, F=384, n_ffn=6, dtype="bf16")
    lt = W.make_layer(spec, seed=21)
    lt.bias = torch.tensor([0.8, 0.0, -0.2, 0.0, 0.0, 0.0, 0.6, 0.0, 0.0, 0.0])  # crowd FFN expert 0 and the zero expert
    info = check_layer(oracle64, lt, None, tau=tau, capacity_factor=gamma)
    check_layer(oracle64, lt, None, tau=tau, capacity_factor=gamma, row_align=128, add_residual=1)
    # tables of the capacity-limited permutation, bit-exact
    cfg = B.config_from_spec(spec, tau=tau, capacity_factor=gamma)
    s = shape_of(spec, tau=tau, capacity_factor=gamma)
    oi = oracle_inputs(lt)
    G = oracle64.router_logits(s, oi["x"], oi["W_r"], oi["W_g"], oi["prev"], oi["bias"])
    idx_o, _ = oracle64.gate_topk(s, G)
    counts_o, offsets_o, ros_o, sor_o = oracle64.tables(s, idx_o)
    d = lambda a: torch.from_numpy(a).cuda()
    lg = d(G)
    idx = torch.empty(spec.T, 2, dtype=torch.int32, device="cuda")
    w = torch.empty(spec.T, 2, device="cuda")
    cnt = torch.empty(spec.N, dtype=torch.int32, device="cuda")
    off = torch.empty(spec.n_ffn + 1, dtype=torch.int32, device="cuda")
    cfg_g = B.config_from_spec(spec, tau=tau, capacity_factor=gamma, flags=B.FLAG_LOGITS_GIVEN)
    B.moepp_route(cfg_g, lt.x.cuda(), None, None, None, None, None, lg, idx, w, cnt, off, None)
    ros = torch.empty(spec.T, 2, dtype=torch.int32, device="cuda")
    sor = torch.empty(cfg.M_cap, dtype=torch.int32, device="cuda")
    xp = torch.empty(cfg.M_cap, spec.D, dtype=torch.bfloat16, device="cuda")
    B.moepp_permute(cfg, lt.x.cuda(), idx, off, ros, sor, xp)
    torch.cuda.synchronize()
    assert np.array_equal(idx.cpu().numpy(), idx_o)
    assert np.array_equal(cnt.cpu().numpy(), counts_o) and np.array_equal(off.cpu().numpy(), offsets_o)
    assert np.array_equal(ros.cpu().numpy(), ros_o) and np.array_equal(sor.cpu().numpy(), sor_o)
    dropped = (ros_o == -2).mean()
    assert (dropped == 0) if gamma >= 8 else (dropped > 0.02)


def test_balance_stats(oracle64):
    """Eq. 7 statistics from the router's own outputs."""
    for spec, tau in ((W.CONFIGS["cfg1_tiny_f32"], 0.75), (W.LayerSpec(T=5000, D=128, F=64, n_ffn=40, n_const=8), 0.1)):
        lt = W.make_layer(spec, seed=5)
        cfg = B.config_from_spec(spec, tau=tau)
        s, oi = shape_of(spec, tau=tau), oracle_inputs(lt)
        T, N, K = spec.T, spec.N, spec.top_k
        lg = torch.empty(T, N, device="cuda")
        idx = torch.empty(T, K, dtype=torch.int32, device="cuda")
        w = torch.empty(T, K, device="cuda")
        cnt = torch.empty(N, dtype=torch.int32, device="cuda")
        off = torch.empty(spec.n_ffn + 1, dtype=torch.int32, device="cuda")
        B.moepp_route(cfg, lt.x.cuda(), lt.W_r.cuda(), lt.W_g.cuda(), lt.prev.cuda(), None, None, lg, idx, w, cnt, off, None)
        f = torch.empty(N, device="cuda")
        P = torch.empty(N, device="cuda")
        loss = torch.empty(1, device="cuda")
        B.moepp_balance_stats(cfg, lg, cnt, f, P, loss)
        torch.cuda.synchronize()
        f_o, P_o, L_o = oracle64.balance_stats(s, lg.cpu().numpy(), idx.cpu().numpy())
        assert max_abs(f.cpu().numpy(), f_o) <= 1e-6
        assert max_abs(P.cpu().numpy(), P_o) <= 1e-6
        assert abs(float(loss.item()) - L_o) <= 1e-6
        assert abs(float(f.sum().item()) - K) <= 1e-5
        # reproducible bit for bit
        P2 = torch.empty(N, device="cuda")
        loss2 = torch.empty(1, device="cuda")
        B.moepp_balance_stats(cfg, lg, cnt, f, P2, loss2)
        torch.cuda.synchronize()
        assert torch.equal(P, P2) and torch.equal(loss, loss2)


def test_balance_backward(oracle64):
    """Gradient of the Eq. 7 loss with respect to the logits (f held fixed): overwrite and accumulate forms."""
    for spec, tau in ((W.CONFIGS["cfg1_tiny_f32"], 0.75), (W.LayerSpec(T=3001, D=64, F=64, n_ffn=40, n_const=8), 0.1)):
        cfg = B.config_from_spec(spec, tau=tau)
        s = shape_of(spec, tau=tau)
        T, N = spec.T, spec.N
        gen = torch.Generator().manual_seed(3)
        lg = 2.0 * torch.randn(T, N, generator=gen)
        f = torch.rand(N, generator=gen)
        base = torch.randn(T, N, generator=gen)
        out = torch.full((T, N), float("nan"), device="cuda")
        B.moepp_balance_backward(cfg, lg.cuda(), f.cuda(), 0.01, out)
        acc = base.cuda()
        B.moepp_balance_backward(cfg, lg.cuda(), f.cuda(), 0.01, acc, accumulate=True)
        torch.cuda.synchronize()
        ref = oracle64.balance_backward(s, lg.numpy(), f.numpy(), scale=0.01)
        scale = float(np.abs(ref).max())
        assert max_abs(out.cpu().numpy(), ref) <= 1e-5 * scale + 1e-12
        assert max_abs(acc.cpu().numpy(), base.numpy().astype(np.float64) + ref) <= 1e-6
