"""GPU parity of the differentiable stack (moepp_stack_forward_train + moepp_stack_backward) through the C-ABI.

(1) float32, three chained layers, with the Eq. 7 loss of every layer added at weight beta: every layer's gradients
    against the oracle's own chain (forward with the GPU's picks, then layer by layer backwards, each layer's
    logit gradient being the next layer's dprev plus beta times the balance gradient).
(2) bf16 on the tensor-core path with kept pre-activations: the stack calls against the same chain made of
    single-layer calls, bit for bit (they run the same kernels on the same values).
"""
import numpy as np
import pytest
import torch

from harness import f32, oracle_inputs, shape_of
from paper_2410_07348_b200 import binding as B
from paper_2410_07348_b200 import workloads as W

pytestmark = pytest.mark.gpu

WEIGHT_GRADS = ("dW_r", "dW_g", "dbias", "dW_c", "dv", "dW_gate", "dW_up", "dW_down")


def _new_grads(spec, dev, dtype, with_wg):
    z = lambda *shape, dt=torch.float32: torch.full(shape, float("nan"), dtype=dt, device=dev)
    N, D, F = spec.N, spec.D, spec.F
    return dict(dx=z(spec.T, D, dt=dtype), dprev=z(spec.T, N), dW_r=z(N, D), dW_g=z(N, N) if with_wg else None,
                dbias=z(N), dW_c=z(max(spec.n_const, 1), 2, D), dv=z(max(spec.n_const, 1), D),
                dW_gate=z(spec.n_ffn, F, D), dW_up=z(spec.n_ffn, F, D), dW_down=z(spec.n_ffn, D, F))


def _stack_run(spec, layers, cfg, dy, dlogits_last, beta):
    dev = "cuda"
    L = len(layers)
    wds = [B.weights_from_tensors(lt) for lt in layers]
    x = layers[0].x.cuda()
    tws = torch.empty(B.moepp_stack_train_workspace_bytes(cfg, L), dtype=torch.uint8, device=dev)
    bws = torch.empty(B.moepp_stack_backward_workspace_bytes(cfg, L), dtype=torch.uint8, device=dev)
    y = torch.empty_like(x)
    lg = torch.empty(spec.T, spec.N, device=dev)
    B.moepp_stack_forward_train(cfg, wds, x, None, y, lg, tws)
    grads = [_new_grads(spec, dev, x.dtype, wd["W_g"] is not None) for wd in wds]
    losses = torch.full((L,), float("nan"), device=dev)
    B.moepp_stack_backward(cfg, wds, x, None, dy, dlogits_last, beta, losses if beta else None, tws, grads, bws)
    torch.cuda.synchronize()
    assert B.moepp_device_error() == 0
    return wds, x, y, lg, grads, losses


def _layer_chain(spec, wds, cfg, x, dy, dlogits_last):
    """The same stack made of single-layer calls; returns outputs, per-layer picks, logits and gradients."""
    dev = "cuda"
    T, N, K = spec.T, spec.N, spec.top_k
    wss, xs, lgs, idxs = [], [x], [None], []
    for wd in wds:
        ws = torch.empty(B.moepp_workspace_bytes(cfg), dtype=torch.uint8, device=dev)
        yj, gj = torch.empty_like(x), torch.empty(T, N, device=dev)
        prev = lgs[-1] if wd["W_g"] is not None else None
        B.moepp_layer_forward(cfg, wd, xs[-1], prev, yj, gj, ws)
        ij = torch.empty(T, K, dtype=torch.int32, device=dev)
        B.moepp_route(cfg, xs[-1], wd["W_r"], wd["W_g"], prev, wd["router_bias"], None, torch.empty(T, N, device=dev), ij,
                      torch.empty(T, K, device=dev), torch.empty(N, dtype=torch.int32, device=dev),
                      torch.empty(spec.n_ffn + 1, dtype=torch.int32, device=dev), None)
        wss.append(ws); xs.append(yj); lgs.append(gj); idxs.append(ij.cpu().numpy())
    bws = torch.empty(B.moepp_backward_workspace_bytes(cfg), dtype=torch.uint8, device=dev)
    grads = [None] * len(wds)
    cur_dy, cur_dl = dy, dlogits_last
    for j in reversed(range(len(wds))):
        wd = wds[j]
        g = _new_grads(spec, dev, x.dtype, wd["W_g"] is not None)
        prev = lgs[j] if wd["W_g"] is not None else None
        B.moepp_layer_backward(cfg, wd, xs[j], prev, lgs[j + 1], cur_dy, cur_dl, wss[j], g, bws)
        grads[j] = g
        cur_dy, cur_dl = g["dx"], (g["dprev"] if wd["W_g"] is not None else None)
    torch.cuda.synchronize()
    return xs, lgs, idxs, grads


@pytest.mark.parametrize("gamma", [0.0, 0.9])
def test_stack_backward_f32_against_oracle_chain_with_balance_loss(oracle64, gamma):
    spec = W.LayerSpec(T=260, D=72, F=120, n_ffn=4, n_zero=1, n_copy=1, n_const=2, top_k=2, dtype="f32")
    layers = W.make_stack(spec, 3)
    for lt in layers:  # larger weights than the benchmark recipe, so that the gradients are not tiny
        lt.W_r, lt.W_gate, lt.W_up, lt.W_down = lt.W_r * 4, lt.W_gate * 3, lt.W_up * 3, lt.W_down * 3
    tau, beta = 0.75, 0.05
    cfg = B.config_from_spec(spec, add_residual=1, tau=tau, capacity_factor=gamma)  # gamma > 0: Eq. 8 drops slots
    gen = torch.Generator().manual_seed(31)
    dy = torch.randn(spec.T, spec.D, generator=gen)
    dl_last = 0.1 * torch.randn(spec.T, spec.N, generator=gen)
    wds, x, y, lg, grads, losses = _stack_run(spec, layers, cfg, dy.cuda(), dl_last.cuda(), beta)
    _, _, idxs, _ = _layer_chain(spec, wds, cfg, x, dy.cuda(), dl_last.cuda())

    s = shape_of(spec, add_residual=1, tau=tau, capacity_factor=gamma)
    ois = [oracle_inputs(lt) for lt in layers]
    fw, xin, prev = [], ois[0]["x"], None
    for j, o in enumerate(ois):
        pj = prev if o["W_g"] is not None else None
        r = oracle64.layer_forward(s, xin, o["W_r"], o["W_g"], pj, o["bias"], o["W_c"], o["v"], o["W_gate"], o["W_up"],
                                   o["W_down"], forced_idx=idxs[j])
        fw.append((xin, pj, r["logits"]))
        xin, prev = r["y"], r["logits"]
    assert np.abs(y.cpu().numpy() - xin).max() <= 1e-4
    cur_dy, cur_dl = f32(dy), f32(dl_last)
    for j in reversed(range(3)):
        o = ois[j]
        xj, pj, lj = fw[j]
        fj, _, Lj = oracle64.balance_stats(s, lj, idxs[j])
        assert abs(float(losses[j].item()) - Lj) <= 1e-5
        dl = oracle64.balance_backward(s, lj, fj, scale=beta, into=cur_dl)
        ref = oracle64.layer_backward(s, xj, o["W_r"], idxs[j], cur_dy, o["W_g"], pj, o["bias"], o["W_c"], o["v"],
                                      o["W_gate"], o["W_up"], o["W_down"], dlogits=dl)
        names = WEIGHT_GRADS + (("dx",) if j == 0 else ())
        for name in names:
            r_ = ref[name]
            if r_ is None or grads[j][name] is None:
                continue
            scale = max(float(np.abs(r_).max()), 1e-6)
            err = float(np.abs(grads[j][name].cpu().numpy().astype(np.float64) - r_).max()) / scale
            assert err <= 5e-4, (j, name, err)
        cur_dy, cur_dl = ref["dx"], ref["dprev"]


def test_stack_backward_bf16_equals_chain_of_layer_calls():
    spec = W.LayerSpec(T=2100, D=256, F=384, n_ffn=6, n_zero=1, n_copy=1, n_const=2, top_k=2, dtype="bf16")
    layers = W.make_stack(spec, 3)
    cfg = B.config_from_spec(spec, add_residual=1, row_align=64, flags=B.FLAG_SAVE_PREACT)
    gen = torch.Generator().manual_seed(32)
    dy = torch.randn(spec.T, spec.D, generator=gen).to(torch.bfloat16).cuda()
    wds, x, y, lg, grads, _ = _stack_run(spec, layers, cfg, dy, None, 0.0)
    xs, lgs, _, ref = _layer_chain(spec, wds, cfg, x, dy, None)
    assert torch.equal(y, xs[-1]) and torch.equal(lg, lgs[-1])
    for j in range(3):
        for name in WEIGHT_GRADS + (("dx",) if j == 0 else ()):
            if ref[j][name] is None:
                continue
            assert torch.equal(grads[j][name], ref[j][name]), (j, name)
            assert torch.isfinite(grads[j][name].float()).all(), (j, name)
