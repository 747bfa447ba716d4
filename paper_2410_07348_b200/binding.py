"""Thin ctypes binding of the C-ABI library declared in ``include/moepp.h``.

Argument marshalling only: every function here has the name of the C call it forwards to, takes torch
CUDA tensors (or ``None`` for optional pointers), passes their data pointers and the current torch
stream, and raises ``MoeppError`` on a non-zero status.  No step of the layer runs in Python, and
there is no fallback: if ``libmoepp.so`` is missing or fails to load, every call raises.
"""
from __future__ import annotations

import ctypes
import os
from dataclasses import dataclass

import torch

_LIB_PATH = os.path.join(os.path.dirname(os.path.abspath(__file__)), "libmoepp.so")
_lib = None

MOEPP_F32, MOEPP_BF16 = 0, 1
FLAG_LOGITS_GIVEN, FLAG_SIMT_FFN, FLAG_FFN_SINGLE_CTA, FLAG_FUSED_GATHER, FLAG_SAVE_PREACT, FLAG_ACCUM_GRADS = 1, 2, 4, 8, 16, 32
STATUS = {0: "MOEPP_OK", 1: "MOEPP_ERR_INVALID_ARG", 2: "MOEPP_ERR_UNSUPPORTED", 3: "MOEPP_ERR_ALIGN",
          4: "MOEPP_ERR_WORKSPACE", 5: "MOEPP_ERR_CUDA", 6: "MOEPP_ERR_TIMEOUT"}

EXPORTS = ("moepp_status_string", "moepp_workspace_bytes", "moepp_workspace_bytes_host", "moepp_route",
           "moepp_permute", "moepp_grouped_ffn", "moepp_combine", "moepp_layer_forward",
           "moepp_layer_forward_host", "moepp_device_error", "moepp_grouped_ffn_static",
           "moepp_stack_workspace_bytes", "moepp_stack_forward", "moepp_stack_workspace_bytes_host",
           "moepp_stack_forward_host", "moepp_balance_stats", "moepp_backward_workspace_bytes",
           "moepp_layer_backward", "moepp_balance_backward", "moepp_stack_train_workspace_bytes",
           "moepp_stack_forward_train", "moepp_stack_backward_workspace_bytes", "moepp_stack_backward",
           "moepp_gather_rows")
STATIC_SCRATCH_BYTES = 32 << 20


class MoeppError(RuntimeError):
    def __init__(self, status: int, call: str):
        self.status = status
        super().__init__("%s returned %s" % (call, STATUS.get(status, status)))


class moepp_config(ctypes.Structure):
    _fields_ = [(n, ctypes.c_int32) for n in (
        "T", "D", "F", "n_ffn", "n_zero", "n_copy", "n_const", "top_k", "dtype", "renorm_topk", "row_align",
        "add_residual", "flags")] + [("tau", ctypes.c_float), ("capacity_factor", ctypes.c_float)]


class moepp_weights(ctypes.Structure):
    _fields_ = [(n, ctypes.c_void_p) for n in ("W_r", "W_g", "W_c", "v", "router_bias", "W_gate", "W_up", "W_down")]


class moepp_grads(ctypes.Structure):
    _fields_ = [(n, ctypes.c_void_p) for n in ("dx", "dprev", "dW_r", "dW_g", "dbias", "dW_c", "dv", "dW_gate",
                                               "dW_up", "dW_down")]


def lib() -> ctypes.CDLL:
    """Loads libmoepp.so (built in-tree by build.py).  A missing library is a hard error."""
    global _lib
    if _lib is None:
        if not os.path.exists(_LIB_PATH):
            raise RuntimeError("libmoepp.so is not built: run `python -m paper_2410_07348_b200.build` "
                               "(there is no fallback path)")
        _lib = ctypes.CDLL(_LIB_PATH)
        _lib.moepp_status_string.restype = ctypes.c_char_p
        for name in EXPORTS[1:]:
            getattr(_lib, name).restype = ctypes.c_int
    return _lib


@dataclass
class Config:
    T: int
    D: int
    F: int
    n_ffn: int
    n_zero: int = 0
    n_copy: int = 0
    n_const: int = 0
    top_k: int = 2
    dtype: int = MOEPP_BF16
    renorm_topk: int = 0
    row_align: int = 1
    add_residual: int = 0
    flags: int = 0
    tau: float = 1.0
    capacity_factor: float = 0.0

    @property
    def N(self):
        return self.n_ffn + self.n_zero + self.n_copy + self.n_const

    @property
    def M_cap(self):
        return self.T * self.top_k + self.n_ffn * (self.row_align - 1)

    def c(self):
        return moepp_config(self.T, self.D, self.F, self.n_ffn, self.n_zero, self.n_copy, self.n_const, self.top_k,
                            self.dtype, self.renorm_topk, self.row_align, self.add_residual, self.flags, self.tau,
                            self.capacity_factor)


def _p(t):
    if t is None:
        return ctypes.c_void_p(0)
    if isinstance(t, int):
        return ctypes.c_void_p(t)
    assert t.is_contiguous(), "tensors handed to the library must be contiguous"
    return ctypes.c_void_p(t.data_ptr())


def _stream():
    return ctypes.c_void_p(torch.cuda.current_stream().cuda_stream)


def _check(status, call):
    if status != 0:
        raise MoeppError(status, call)


def _weights(w: dict) -> moepp_weights:
    return moepp_weights(*[(w.get(k).data_ptr() if w.get(k) is not None else None) for k in
                           ("W_r", "W_g", "W_c", "v", "router_bias", "W_gate", "W_up", "W_down")])


def moepp_workspace_bytes(cfg: Config, host: bool = False) -> int:
    n = ctypes.c_size_t(0)
    c = cfg.c()
    fn = lib().moepp_workspace_bytes_host if host else lib().moepp_workspace_bytes
    _check(fn(ctypes.byref(c), ctypes.byref(n)), "moepp_workspace_bytes")
    return int(n.value)


def moepp_route(cfg, x, W_r, W_g, prev_logits, router_bias, W_c, logits, topk_idx, topk_w, expert_counts,
                expert_offsets, alpha):
    c = cfg.c()
    _check(lib().moepp_route(ctypes.byref(c), _p(x), _p(W_r), _p(W_g), _p(prev_logits), _p(router_bias), _p(W_c),
                             _p(logits), _p(topk_idx), _p(topk_w), _p(expert_counts), _p(expert_offsets), _p(alpha),
                             _stream()), "moepp_route")


def moepp_permute(cfg, x, topk_idx, expert_offsets, row_of_slot, slot_of_row, x_perm):
    c = cfg.c()
    _check(lib().moepp_permute(ctypes.byref(c), _p(x), _p(topk_idx), _p(expert_offsets), _p(row_of_slot),
                               _p(slot_of_row), _p(x_perm), _stream()), "moepp_permute")


def moepp_grouped_ffn(cfg, x_perm, expert_offsets, W_gate, W_up, W_down, h_ws, y_perm):
    c = cfg.c()
    _check(lib().moepp_grouped_ffn(ctypes.byref(c), _p(x_perm), _p(expert_offsets), _p(W_gate), _p(W_up), _p(W_down),
                                   _p(h_ws), _p(y_perm), _stream()), "moepp_grouped_ffn")


def moepp_grouped_ffn_static(cfg, x_perm, expert_offsets, W_gate, W_up, W_down, y_perm):
    """moepp_grouped_ffn for callers that own no scratch memory: the intermediate sits in a fixed
    STATIC_SCRATCH_BYTES array inside the library.  Calls share that array, so do not overlap them."""
    c = cfg.c()
    _check(lib().moepp_grouped_ffn_static(ctypes.byref(c), _p(x_perm), _p(expert_offsets), _p(W_gate), _p(W_up),
                                          _p(W_down), _p(y_perm), _stream()), "moepp_grouped_ffn_static")


def moepp_combine(cfg, x, y_perm, topk_idx, topk_w, row_of_slot, alpha, W_c, v, y):
    c = cfg.c()
    _check(lib().moepp_combine(ctypes.byref(c), _p(x), _p(y_perm), _p(topk_idx), _p(topk_w), _p(row_of_slot),
                               _p(alpha), _p(W_c), _p(v), _p(y), _stream()), "moepp_combine")


def moepp_layer_forward(cfg, weights: dict, x, prev_logits, y, logits_out, workspace):
    c, w = cfg.c(), _weights(weights)
    _check(lib().moepp_layer_forward(ctypes.byref(c), ctypes.byref(w), _p(x), _p(prev_logits), _p(y), _p(logits_out),
                                     _p(workspace), ctypes.c_size_t(workspace.numel() * workspace.element_size()),
                                     _stream()), "moepp_layer_forward")


def moepp_layer_forward_host(cfg, weights: dict, x_host, prev_logits_host, y_host, logits_out_host, workspace):
    """x_host, prev_logits_host, y_host, logits_out_host: pinned CPU tensors; weights and workspace: CUDA."""
    c, w = cfg.c(), _weights(weights)
    _check(lib().moepp_layer_forward_host(ctypes.byref(c), ctypes.byref(w), _p(x_host), _p(prev_logits_host),
                                          _p(y_host), _p(logits_out_host), _p(workspace),
                                          ctypes.c_size_t(workspace.numel() * workspace.element_size()), _stream()),
           "moepp_layer_forward_host")


def moepp_backward_workspace_bytes(cfg: Config) -> int:
    n = ctypes.c_size_t(0)
    c = cfg.c()
    _check(lib().moepp_backward_workspace_bytes(ctypes.byref(c), ctypes.byref(n)), "moepp_backward_workspace_bytes")
    return int(n.value)


def moepp_layer_backward(cfg, weights: dict, x, prev_logits, logits, dy, dlogits_next, fwd_workspace, grads: dict,
                         bwd_workspace):
    """grads: dict of CUDA tensors named like the fields of moepp_grads (absent or None = NULL)."""
    c, w = cfg.c(), _weights(weights)
    g = moepp_grads()
    for name, _ in moepp_grads._fields_:
        setattr(g, name, _p(grads.get(name)))
    nbytes = lambda t: ctypes.c_size_t(t.numel() * t.element_size())
    _check(lib().moepp_layer_backward(ctypes.byref(c), ctypes.byref(w), _p(x), _p(prev_logits), _p(logits), _p(dy),
                                      _p(dlogits_next), _p(fwd_workspace), nbytes(fwd_workspace), ctypes.byref(g),
                                      _p(bwd_workspace), nbytes(bwd_workspace), _stream()), "moepp_layer_backward")


def moepp_balance_stats(cfg, logits, expert_counts, f, P, loss):
    c = cfg.c()
    _check(lib().moepp_balance_stats(ctypes.byref(c), _p(logits), _p(expert_counts), _p(f), _p(P), _p(loss),
                                     _stream()), "moepp_balance_stats")


def moepp_gather_rows(src, row_index, dst):
    """dst[i, :] = src[row_index[i], :] (zeros for a negative index); src, dst: 2-D CUDA tensors of one dtype."""
    assert src.dtype == dst.dtype and src.shape[1] == dst.shape[1] and row_index.dtype == torch.int32
    dt = MOEPP_BF16 if src.dtype == torch.bfloat16 else MOEPP_F32
    _check(lib().moepp_gather_rows(_p(src), _p(row_index), ctypes.c_int64(dst.shape[0]), ctypes.c_int32(src.shape[1]),
                                   ctypes.c_int32(dt), _p(dst), _stream()), "moepp_gather_rows")


def _grads(grads: dict) -> moepp_grads:
    g = moepp_grads()
    for name, _ in moepp_grads._fields_:
        setattr(g, name, _p(grads.get(name)))
    return g


def moepp_stack_train_workspace_bytes(cfg: Config, n_layers: int) -> int:
    n = ctypes.c_size_t(0)
    c = cfg.c()
    _check(lib().moepp_stack_train_workspace_bytes(ctypes.byref(c), ctypes.c_int32(n_layers), ctypes.byref(n)),
           "moepp_stack_train_workspace_bytes")
    return int(n.value)


def moepp_stack_backward_workspace_bytes(cfg: Config, n_layers: int) -> int:
    n = ctypes.c_size_t(0)
    c = cfg.c()
    _check(lib().moepp_stack_backward_workspace_bytes(ctypes.byref(c), ctypes.c_int32(n_layers), ctypes.byref(n)),
           "moepp_stack_backward_workspace_bytes")
    return int(n.value)


def moepp_stack_forward_train(cfg, weights_list, x, prev_logits, y, logits_out, workspace):
    c, arr = cfg.c(), _weights_array(weights_list)
    _check(lib().moepp_stack_forward_train(ctypes.byref(c), arr, ctypes.c_int32(len(weights_list)), _p(x),
                                           _p(prev_logits), _p(y), _p(logits_out), _p(workspace),
                                           ctypes.c_size_t(workspace.numel() * workspace.element_size()), _stream()),
           "moepp_stack_forward_train")


def moepp_stack_backward(cfg, weights_list, x, prev_logits, dy, dlogits_last, balance_scale, balance_loss_out,
                         train_workspace, grads_list, bwd_workspace):
    """grads_list: one dict per layer (fields of moepp_grads); dx / dprev are read from the first only."""
    c, arr = cfg.c(), _weights_array(weights_list)
    garr = (moepp_grads * len(grads_list))()
    for i, g in enumerate(grads_list):
        garr[i] = _grads(g)
    nbytes = lambda t: ctypes.c_size_t(t.numel() * t.element_size())
    _check(lib().moepp_stack_backward(ctypes.byref(c), arr, ctypes.c_int32(len(weights_list)), _p(x), _p(prev_logits),
                                      _p(dy), _p(dlogits_last), ctypes.c_float(balance_scale), _p(balance_loss_out),
                                      _p(train_workspace), nbytes(train_workspace), garr, _p(bwd_workspace),
                                      nbytes(bwd_workspace), _stream()), "moepp_stack_backward")


def moepp_balance_backward(cfg, logits, f, scale, dlogits, accumulate=False):
    c = cfg.c()
    _check(lib().moepp_balance_backward(ctypes.byref(c), _p(logits), _p(f), ctypes.c_float(scale),
                                        ctypes.c_int32(1 if accumulate else 0), _p(dlogits), _stream()),
           "moepp_balance_backward")


def _weights_array(weights_list):
    arr = (moepp_weights * len(weights_list))()
    for i, w in enumerate(weights_list):
        arr[i] = _weights(w)
    return arr


def moepp_stack_workspace_bytes(cfg: Config, n_layers: int, host: bool = False) -> int:
    n = ctypes.c_size_t(0)
    c = cfg.c()
    fn = lib().moepp_stack_workspace_bytes_host if host else lib().moepp_stack_workspace_bytes
    _check(fn(ctypes.byref(c), ctypes.c_int32(n_layers), ctypes.byref(n)), "moepp_stack_workspace_bytes")
    return int(n.value)


def moepp_stack_forward(cfg, weights_list, x, prev_logits, y, logits_out, workspace):
    c, arr = cfg.c(), _weights_array(weights_list)
    _check(lib().moepp_stack_forward(ctypes.byref(c), arr, ctypes.c_int32(len(weights_list)), _p(x), _p(prev_logits),
                                     _p(y), _p(logits_out), _p(workspace),
                                     ctypes.c_size_t(workspace.numel() * workspace.element_size()), _stream()),
           "moepp_stack_forward")


def moepp_stack_forward_host(cfg, weights_list, x_host, prev_logits_host, y_host, logits_out_host, workspace):
    """x_host, prev_logits_host, y_host, logits_out_host: pinned CPU tensors; weights and workspace: CUDA."""
    c, arr = cfg.c(), _weights_array(weights_list)
    _check(lib().moepp_stack_forward_host(ctypes.byref(c), arr, ctypes.c_int32(len(weights_list)), _p(x_host),
                                          _p(prev_logits_host), _p(y_host), _p(logits_out_host), _p(workspace),
                                          ctypes.c_size_t(workspace.numel() * workspace.element_size()), _stream()),
           "moepp_stack_forward_host")


def moepp_device_error() -> int:
    code = ctypes.c_int32(0)
    st = lib().moepp_device_error(ctypes.byref(code))
    if st not in (0, 6):
        raise MoeppError(st, "moepp_device_error")
    return int(code.value)


# ---- conveniences for callers that hold workloads.LayerTensors (still marshalling only) -----------
def config_from_spec(spec, **over) -> Config:
    kw = dict(T=spec.T, D=spec.D, F=spec.F, n_ffn=spec.n_ffn, n_zero=spec.n_zero, n_copy=spec.n_copy,
              n_const=spec.n_const, top_k=spec.top_k, dtype=MOEPP_BF16 if spec.dtype == "bf16" else MOEPP_F32)
    kw.update(over)
    return Config(**kw)


def weights_from_tensors(lt, device="cuda") -> dict:
    """Moves a LayerTensors' weights to the device and returns the dict the layer calls take."""
    mv = lambda t: None if t is None else t.to(device).contiguous()
    return dict(W_r=mv(lt.W_r), W_g=mv(lt.W_g), W_c=mv(lt.W_c), v=mv(lt.v), router_bias=mv(lt.bias),
                W_gate=mv(lt.W_gate), W_up=mv(lt.W_up), W_down=mv(lt.W_down))
