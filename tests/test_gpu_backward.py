"""GPU parity of the layer's backward pass (moepp_layer_backward) against the CPU oracle, through the C-ABI.

The forward call fills its workspace, the backward call reads it; the oracle differentiates the same layer in
float64 with the GPU's own picks held fixed.  Every gradient tensor is compared element by element, the error
measured against that tensor's largest magnitude: float32 storage within 2e-4, bf16 storage within 2e-2 (the
grouped intermediates dL/dE, the SwiGLU pre-activations and their gradients are rounded to bf16 on the way).
"""
import numpy as np
import pytest
import torch

from harness import f32, oracle_inputs, shape_of
from paper_2410_07348_b200 import binding as B
from paper_2410_07348_b200 import workloads as W

pytestmark = pytest.mark.gpu

TOL = {"f32": 2e-4, "bf16": 2e-2}
GRADS = ("dx", "dprev", "dW_r", "dW_g", "dbias", "dW_c", "dv", "dW_gate", "dW_up", "dW_down")


def gpu_backward(cfg, wd, x, prev, dy, dlogits):
    T, N, K = cfg.T, cfg.N, cfg.top_k
    dev = "cuda"
    ws = torch.empty(B.moepp_workspace_bytes(cfg), dtype=torch.uint8, device=dev)
    y = torch.empty(T, cfg.D, dtype=x.dtype, device=dev)
    logits = torch.empty(T, N, device=dev)
    B.moepp_layer_forward(cfg, wd, x, prev, y, logits, ws)
    idx = torch.empty(T, K, dtype=torch.int32, device=dev)
    w = torch.empty(T, K, device=dev)
    counts = torch.empty(N, dtype=torch.int32, device=dev)
    offsets = torch.empty(cfg.n_ffn + 1, dtype=torch.int32, device=dev)
    lg2 = torch.empty(T, N, device=dev)
    B.moepp_route(cfg, x, wd["W_r"], wd["W_g"], prev, wd["router_bias"], None, lg2, idx, w, counts, offsets, None)
    nan = lambda *shape, dtype=torch.float32: torch.full(shape, float("nan"), dtype=dtype, device=dev)
    g = dict(dx=nan(T, cfg.D, dtype=x.dtype), dprev=nan(T, N) if prev is not None else None, dW_r=nan(N, cfg.D),
             dW_g=nan(N, N) if prev is not None else None, dbias=nan(N), dW_c=nan(max(cfg.n_const, 1), 2, cfg.D),
             dv=nan(max(cfg.n_const, 1), cfg.D), dW_gate=nan(max(cfg.n_ffn, 1), cfg.F, cfg.D),
             dW_up=nan(max(cfg.n_ffn, 1), cfg.F, cfg.D), dW_down=nan(max(cfg.n_ffn, 1), cfg.D, cfg.F))
    bws = torch.empty(B.moepp_backward_workspace_bytes(cfg), dtype=torch.uint8, device=dev)
    B.moepp_layer_backward(cfg, wd, x, prev, logits, dy, dlogits, ws, g, bws)
    torch.cuda.synchronize()
    assert B.moepp_device_error() == 0
    return {k: (None if v is None else v.float().cpu().numpy()) for k, v in g.items()}, idx.cpu().numpy()


def check_backward(oracle64, lt, seed=0, with_dlogits=True, **over):
    spec = lt.spec
    cfg = B.config_from_spec(spec, **over)
    wd = B.weights_from_tensors(lt)
    x, prev = lt.x.cuda(), None if lt.prev is None else lt.prev.cuda()
    gen = torch.Generator().manual_seed(77 + seed)
    dy = torch.randn(spec.T, spec.D, generator=gen).to(x.dtype)
    dlogits = (0.1 * torch.randn(spec.T, spec.N, generator=gen)) if with_dlogits else None
    got, idx_g = gpu_backward(cfg, wd, x, prev, dy.cuda(), None if dlogits is None else dlogits.cuda())
    s = shape_of(spec, **{k: v for k, v in over.items()
                          if k in ("renorm_topk", "row_align", "add_residual", "tau", "capacity_factor")})
    oi = oracle_inputs(lt)
    ref = oracle64.layer_backward(s, oi["x"], oi["W_r"], idx_g, f32(dy), oi["W_g"], oi["prev"], oi["bias"], oi["W_c"],
                                  oi["v"], f32(lt.W_gate), f32(lt.W_up), f32(lt.W_down), dlogits=f32(dlogits))
    tol = TOL[spec.dtype]
    worst = {}
    for name in GRADS:
        r = ref[name]
        if r is None or r.size == 0 or got[name] is None:
            continue
        gq = got[name].reshape(-1)[:r.size].reshape(r.shape)
        assert np.isfinite(gq).all(), name
        scale = max(float(np.abs(r).max()), 1e-6)
        worst[name] = float(np.abs(gq.astype(np.float64) - r).max()) / scale
        assert worst[name] <= tol, (name, worst[name], scale)
    return worst


def test_backward_cfg1_f32(oracle64):
    lt = W.make_config("cfg1_tiny_f32")
    check_backward(oracle64, lt)
    check_backward(oracle64, lt, renorm_topk=1, add_residual=1, row_align=128)
    check_backward(oracle64, lt, with_dlogits=False)


def test_backward_first_layer_vanilla(oracle64):
    lt = W.make_layer(W.CONFIGS["cfg1_tiny_f32"].vanilla(), seed=0, with_prev=False)
    check_backward(oracle64, lt)


@pytest.mark.parametrize("dtype,row_align", [("f32", 128), ("bf16", 128), ("bf16", 1), ("bf16", 8)])
def test_backward_several_tiles(oracle64, dtype, row_align):
    """Several 64-row tiles per expert with ragged tails, all four expert kinds; padded segments, and dense ones
    whose last weight-gradient k tile reaches into the next expert's rows (cleared in shared memory)."""
    spec = W.LayerSpec(T=1900, D=264, F=392, n_ffn=5, n_zero=1, n_copy=1, n_const=2, top_k=2, dtype=dtype)
    lt = W.make_layer(spec, seed=3, with_prev=True, w_std=0.05)
    check_backward(oracle64, lt, row_align=row_align, add_residual=1)


@pytest.mark.parametrize("seed", range(6))
def test_backward_random_shapes(oracle64, seed):
    rng = np.random.default_rng(2000 + seed)
    dtype = "bf16" if seed % 2 == 0 else "f32"
    n_ffn = int(rng.integers(1, 9))
    n_zero, n_copy, n_const = int(rng.integers(0, 3)), int(rng.integers(0, 3)), int(rng.integers(0, 4))
    N = n_ffn + n_zero + n_copy + n_const
    spec = W.LayerSpec(T=int(rng.integers(1, 900)), D=8 * int(rng.integers(1, 40)), F=8 * int(rng.integers(1, 40)),
                       n_ffn=n_ffn, n_zero=n_zero, n_copy=n_copy, n_const=n_const,
                       top_k=int(rng.integers(1, min(N, 4) + 1)), dtype=dtype)
    lt = W.make_layer(spec, seed=seed, with_prev=bool(seed & 2), w_std=0.05)
    over = dict(row_align=int(rng.choice([1, 8, 128])), add_residual=int(rng.integers(0, 2)),
                renorm_topk=int(rng.integers(0, 2)))
    if seed % 3 == 0:
        over.update(capacity_factor=float(rng.choice([0.7, 1.1])), tau=float(rng.choice([0.5, 0.75, 1.0])))
    check_backward(oracle64, lt, seed=seed, **over)


@pytest.mark.parametrize("dtype,flags", [("f32", 0), ("bf16", 0), ("bf16", B.FLAG_SIMT_FFN)])
def test_backward_with_kept_pre_activations(oracle64, dtype, flags):
    """MOEPP_FLAG_SAVE_PREACT: the forward pass stores gate and up, the backward pass reads them instead of
    recomputing; same oracle, same tolerance, and the forward output is unchanged by the flag."""
    spec = W.LayerSpec(T=1500, D=200, F=328, n_ffn=4, n_zero=1, n_copy=1, n_const=1, top_k=2, dtype=dtype)
    lt = W.make_layer(spec, seed=11, with_prev=True, w_std=0.05)
    check_backward(oracle64, lt, row_align=64, flags=flags | B.FLAG_SAVE_PREACT)
    wd = B.weights_from_tensors(lt)
    x, prev = lt.x.cuda(), lt.prev.cuda()
    ys = []
    for fl in (flags, flags | B.FLAG_SAVE_PREACT):
        cfg = B.config_from_spec(spec, row_align=64, flags=fl)
        ws = torch.empty(B.moepp_workspace_bytes(cfg), dtype=torch.uint8, device="cuda")
        y = torch.empty_like(x)
        B.moepp_layer_forward(cfg, wd, x, prev, y, None, ws)
        ys.append(y)
    torch.cuda.synchronize()
    assert torch.equal(ys[0], ys[1])


def test_backward_experts_without_rows_on_tensor_cores(oracle64):
    """Fewer slots than experts: the weight-gradient tiles of an expert nobody picked have an empty k range and must
    come out as exact zeros (bf16, 64-row segments, so the tensor-core kernels run)."""
    spec = W.LayerSpec(T=5, D=128, F=256, n_ffn=12, n_zero=1, n_copy=1, n_const=1, top_k=2, dtype="bf16")
    lt = W.make_layer(spec, seed=2, with_prev=True, w_std=0.05)
    check_backward(oracle64, lt, row_align=64)
    cfg = B.config_from_spec(spec, row_align=64)
    wd = B.weights_from_tensors(lt)
    dy = torch.ones(spec.T, spec.D, dtype=torch.bfloat16, device="cuda")
    got, idx = gpu_backward(cfg, wd, lt.x.cuda(), lt.prev.cuda(), dy, None)
    unused = [e for e in range(spec.n_ffn) if not (idx == e).any()]
    assert unused
    for e in unused:
        for name in ("dW_gate", "dW_up", "dW_down"):
            assert not np.any(got[name][e]), (name, e)


def test_backward_through_two_chained_layers(oracle64):
    """Two layers joined by the residual stream and the gating residual (Eq. 6): layer 2's dx is layer 1's dy and
    layer 2's dprev is the dlogits layer 1 receives.  GPU chain against the oracle's chain, float32."""
    spec = W.LayerSpec(T=300, D=96, F=160, n_ffn=4, n_zero=1, n_copy=1, n_const=2, top_k=2, dtype="f32")
    l1 = W.make_layer(spec, seed=21, with_prev=True, w_std=0.05)
    l2 = W.make_layer(spec, seed=22, with_prev=True, w_std=0.05)
    cfg = B.config_from_spec(spec, add_residual=1)
    w1, w2 = B.weights_from_tensors(l1), B.weights_from_tensors(l2)
    dev = "cuda"
    x, prev = l1.x.cuda(), l1.prev.cuda()
    T, N, D = spec.T, spec.N, spec.D
    new = lambda *shape: torch.empty(*shape, device=dev)
    ws1 = torch.empty(B.moepp_workspace_bytes(cfg), dtype=torch.uint8, device=dev)
    ws2 = torch.empty_like(ws1)
    bws = torch.empty(B.moepp_backward_workspace_bytes(cfg), dtype=torch.uint8, device=dev)
    y1, g1, y2, g2 = new(T, D), new(T, N), new(T, D), new(T, N)
    B.moepp_layer_forward(cfg, w1, x, prev, y1, g1, ws1)
    B.moepp_layer_forward(cfg, w2, y1, g1, y2, g2, ws2)
    gen = torch.Generator().manual_seed(5)
    R, Q = torch.randn(T, D, generator=gen), 0.1 * torch.randn(T, N, generator=gen)

    def grads():
        return dict(dx=new(T, D), dprev=new(T, N), dW_r=new(N, D), dW_g=new(N, N), dbias=new(N),
                    dW_c=new(spec.n_const, 2, D), dv=new(spec.n_const, D), dW_gate=new(spec.n_ffn, spec.F, D),
                    dW_up=new(spec.n_ffn, spec.F, D), dW_down=new(spec.n_ffn, D, spec.F))

    ga, gb = grads(), grads()
    B.moepp_layer_backward(cfg, w2, y1, g1, g2, R.cuda(), Q.cuda(), ws2, gb, bws)
    B.moepp_layer_backward(cfg, w1, x, prev, g1, gb["dx"], gb["dprev"], ws1, ga, bws)
    idx = []
    for (w, xin, pin) in ((w1, x, prev), (w2, y1, g1)):
        i_ = torch.empty(T, spec.top_k, dtype=torch.int32, device=dev)
        B.moepp_route(cfg, xin, w["W_r"], w["W_g"], pin, w["router_bias"], None, new(T, N), i_, new(T, spec.top_k),
                      torch.empty(N, dtype=torch.int32, device=dev),
                      torch.empty(spec.n_ffn + 1, dtype=torch.int32, device=dev), None)
        idx.append(i_.cpu().numpy())
    torch.cuda.synchronize()

    # the oracle's own chain from the same x: forward both layers, backward both layers
    s = shape_of(spec, add_residual=1)
    o1, o2 = oracle_inputs(l1), oracle_inputs(l2)
    f1 = oracle64.layer_forward(s, o1["x"], o1["W_r"], o1["W_g"], o1["prev"], o1["bias"], o1["W_c"], o1["v"], o1["W_gate"],
                                o1["W_up"], o1["W_down"], forced_idx=idx[0])
    b2 = oracle64.layer_backward(s, f1["y"], o2["W_r"], idx[1], f32(R), o2["W_g"], f1["logits"], o2["bias"], o2["W_c"],
                                 o2["v"], o2["W_gate"], o2["W_up"], o2["W_down"], dlogits=f32(Q))
    b1 = oracle64.layer_backward(s, o1["x"], o1["W_r"], idx[0], b2["dx"], o1["W_g"], o1["prev"], o1["bias"], o1["W_c"],
                                 o1["v"], o1["W_gate"], o1["W_up"], o1["W_down"], dlogits=b2["dprev"])
    for got, ref in ((gb, b2), (ga, b1)):
        for name in GRADS:
            r = ref[name]
            scale = max(float(np.abs(r).max()), 1e-6)
            err = float(np.abs(got[name].cpu().numpy().astype(np.float64) - r).max()) / scale
            assert err <= 5e-4, (name, err)


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_backward_at_the_expert_count_limits(oracle64, dtype):
    """N = 64 experts, 16 of them constant experts (96 router rows), top-8: the widest tables every kernel takes."""
    spec = W.LayerSpec(T=700, D=264, F=72, n_ffn=40, n_zero=4, n_copy=4, n_const=16, top_k=8, dtype=dtype)
    lt = W.make_layer(spec, seed=13, with_prev=True, w_std=0.05)
    check_backward(oracle64, lt, row_align=64, renorm_topk=1, add_residual=1)


def test_backward_full_size_layer_on_sampled_tokens(oracle64):
    """The benchmark's layer shape and launch configuration (T = 32768, d_model 4096, d_ffn 2816, 16 + 4 experts, bf16,
    64-row segments, kept pre-activations).  dy and dlogits are non-zero on 20 sampled tokens only, so every gradient
    is the sum of those tokens' contributions, which the oracle computes from the 20-token sub-batch (tokens are
    independent without a capacity limit); all other tokens must get an exactly zero dx."""
    spec = W.CONFIGS["cfg4_7b_stack"]
    lt = W.make_layer(spec, seed=1, with_prev=True, w_std=0.02, device="cuda", gen_device="cuda")
    cfg = B.config_from_spec(spec, add_residual=1, row_align=64, flags=B.FLAG_SAVE_PREACT)
    wd = B.weights_from_tensors(lt)
    n_tok = 20
    rng = np.random.default_rng(4)
    toks = np.sort(rng.choice(spec.T, n_tok, replace=False))
    gen = torch.Generator().manual_seed(44)
    dy_s = torch.randn(n_tok, spec.D, generator=gen).to(torch.bfloat16)
    dl_s = 0.1 * torch.randn(n_tok, spec.N, generator=gen)
    dy = torch.zeros(spec.T, spec.D, dtype=torch.bfloat16, device="cuda")
    dl = torch.zeros(spec.T, spec.N, device="cuda")
    tk = torch.as_tensor(toks, device="cuda")
    dy[tk] = dy_s.cuda()
    dl[tk] = dl_s.cuda()
    got, idx_g = gpu_backward(cfg, wd, lt.x, lt.prev, dy, dl)

    sub = W.LayerSpec(n_tok, spec.D, spec.F, spec.n_ffn, spec.n_zero, spec.n_copy, spec.n_const, spec.top_k, "bf16")
    s = shape_of(sub, add_residual=1, row_align=64)
    x_s, prev_s = f32(lt.x[tk]), f32(lt.prev[tk])
    lt.x, lt.prev = None, None
    oi = oracle_inputs(lt)
    ref = oracle64.layer_backward(s, x_s, oi["W_r"], idx_g[toks], f32(dy_s), oi["W_g"], prev_s, oi["bias"], oi["W_c"],
                                  oi["v"], f32(lt.W_gate), f32(lt.W_up), f32(lt.W_down), dlogits=f32(dl_s))
    for name in GRADS:
        r, g = ref[name], got[name]
        if name in ("dx", "dprev"):
            rest = np.ones(spec.T, bool)
            rest[toks] = False
            assert not np.any(g[rest]), name  # untouched tokens: exact zeros
            g = g[toks]
        scale = max(float(np.abs(r).max()), 1e-6)
        err = float(np.abs(g.reshape(r.shape).astype(np.float64) - r).max()) / scale
        assert err <= TOL["bf16"], (name, err)


@pytest.mark.parametrize("dtype,row_align", [("f32", 1), ("bf16", 64), ("bf16", 8)])
def test_backward_gradient_accumulation(dtype, row_align):
    """MOEPP_FLAG_ACCUM_GRADS: two calls into zeroed buffers give exactly twice the weight gradients of one plain call
    (g + g is exact in float); dx and dprev are overwritten, not added to."""
    spec = W.LayerSpec(T=1300, D=264, F=200, n_ffn=5, n_zero=1, n_copy=1, n_const=2, top_k=2, dtype=dtype)
    lt = W.make_layer(spec, seed=17, with_prev=True, w_std=0.05)
    wd = B.weights_from_tensors(lt)
    x, prev = lt.x.cuda(), lt.prev.cuda()
    gen = torch.Generator().manual_seed(3)
    dy = torch.randn(spec.T, spec.D, generator=gen).to(x.dtype).cuda()
    dev = "cuda"
    outs = []
    for flags, calls in ((0, 1), (B.FLAG_ACCUM_GRADS, 2)):
        cfg = B.config_from_spec(spec, row_align=row_align, flags=flags)
        ws = torch.empty(B.moepp_workspace_bytes(cfg), dtype=torch.uint8, device=dev)
        bws = torch.empty(B.moepp_backward_workspace_bytes(cfg), dtype=torch.uint8, device=dev)
        y, logits = torch.empty_like(x), torch.empty(spec.T, spec.N, device=dev)
        B.moepp_layer_forward(cfg, wd, x, prev, y, logits, ws)
        z = lambda *shape, dt=torch.float32: torch.zeros(*shape, dtype=dt, device=dev)
        N, D, F = spec.N, spec.D, spec.F
        g = dict(dx=z(spec.T, D, dt=x.dtype), dprev=z(spec.T, N), dW_r=z(N, D), dW_g=z(N, N), dbias=z(N),
                 dW_c=z(spec.n_const, 2, D), dv=z(spec.n_const, D), dW_gate=z(spec.n_ffn, F, D),
                 dW_up=z(spec.n_ffn, F, D), dW_down=z(spec.n_ffn, D, F))
        for _ in range(calls):
            B.moepp_layer_backward(cfg, wd, x, prev, logits, dy, None, ws, g, bws)
        torch.cuda.synchronize()
        outs.append(g)
    one, two = outs
    for name in GRADS:
        if name in ("dx", "dprev"):
            assert torch.equal(one[name], two[name]), name
        else:
            assert torch.equal(2 * one[name], two[name]), name
            assert one[name].abs().max() > 0, name


def test_backward_no_tokens():
    spec = W.LayerSpec(T=0, D=64, F=96, n_ffn=2, n_zero=1, n_copy=1, n_const=1, top_k=2, dtype="f32")
    lt = W.make_layer(spec, seed=0, with_prev=True)
    cfg = B.config_from_spec(spec)
    wd = B.weights_from_tensors(lt)
    got, _ = gpu_backward(cfg, wd, lt.x.cuda(), lt.prev.cuda(), torch.empty(0, 64, device="cuda"), None)
    for name in GRADS[2:]:
        assert not np.any(got[name]), name


def test_backward_tensor_core_path_matches_fma_path():
    """At a size the oracle cannot cover in seconds: the tensor-core GEMMs against the FMA kernels (forced by flag)
    on the same forward state, with padded (128) and dense (1) segments; both paths were checked against the oracle
    at smaller sizes above."""
    spec = W.LayerSpec(T=6000, D=1032, F=1416, n_ffn=6, n_zero=1, n_copy=1, n_const=1, top_k=2, dtype="bf16")
    lt = W.make_layer(spec, seed=5, with_prev=True, w_std=0.03)
    wd = B.weights_from_tensors(lt)
    x, prev = lt.x.cuda(), lt.prev.cuda()
    gen = torch.Generator().manual_seed(9)
    dy = torch.randn(spec.T, spec.D, generator=gen).to(x.dtype).cuda()
    for row_align in (128, 1):
        res = []
        for flags in (0, B.FLAG_SIMT_FFN):
            cfg = B.config_from_spec(spec, row_align=row_align, flags=flags)
            res.append(gpu_backward(cfg, wd, x, prev, dy, None)[0])
        for name in GRADS:
            a, b = res[0][name], res[1][name]
            scale = max(float(np.abs(b).max()), 1e-6)
            assert float(np.abs(a - b).max()) / scale <= 1e-2, (name, row_align)
