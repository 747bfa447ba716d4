"""ctypes front end of the CPU oracle (TEST INFRASTRUCTURE ONLY).

The oracle is the paper's definition of one MoE++ layer (arXiv 2410.07348, Eq. 1-6) written out
token by token in C (``moepp_oracle.c``).  Only the tests, the smoke check and the benchmark's CPU
baseline leg may import this package; the CUDA library never does, and this package never imports
the CUDA library.

``Oracle("f64")`` does all arithmetic in double (the referee); ``Oracle("f32")`` in float.
All arrays are numpy, C-contiguous; activations and router weights are float32, FFN weights are
float32 or bf16 bit patterns held in uint16.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from dataclasses import dataclass

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_LIB_PATH = os.path.join(_HERE, "liboracle.so")


def build(force: bool = False) -> str:
    """Compile the oracle with gcc (twice: float and double arithmetic) into liboracle.so."""
    src = os.path.join(_HERE, "moepp_oracle.c")
    hdr = os.path.join(_HERE, "moepp_oracle.h")
    if (not force and os.path.exists(_LIB_PATH)
            and os.path.getmtime(_LIB_PATH) >= max(os.path.getmtime(src), os.path.getmtime(hdr))):
        return _LIB_PATH
    common = ["gcc", "-O2", "-fopenmp", "-fPIC", "-std=c11", "-Wall", "-Wno-maybe-uninitialized", "-c", src]
    o32 = os.path.join(_HERE, "oracle_f32.o")
    o64 = os.path.join(_HERE, "oracle_f64.o")
    subprocess.check_call(common + ["-DORACLE_REAL=float", "-DORACLE_PFX=oracle_f32_", "-DORACLE_MAIN_TU", "-o", o32])
    subprocess.check_call(common + ["-DORACLE_REAL=double", "-DORACLE_PFX=oracle_f64_", "-o", o64])
    subprocess.check_call(["gcc", "-shared", "-fopenmp", "-o", _LIB_PATH, o32, o64, "-lm"])
    return _LIB_PATH


class _Cfg(ctypes.Structure):
    _fields_ = [(n, ctypes.c_int32) for n in (
        "T", "D", "F", "n_ffn", "n_zero", "n_copy", "n_const", "top_k", "renorm_topk", "row_align",
        "add_residual", "ffn_w_bf16")] + [("tau", ctypes.c_float), ("capacity_factor", ctypes.c_float)]


@dataclass
class LayerShape:
    """Sizes of one layer.  Expert index order: FFN | zero | copy | constant."""
    T: int
    D: int
    F: int
    n_ffn: int
    n_zero: int = 0
    n_copy: int = 0
    n_const: int = 0
    top_k: int = 2
    renorm_topk: int = 0
    row_align: int = 1
    add_residual: int = 0
    tau: float = 1.0  # Eq. 7 / Eq. 8
    capacity_factor: float = 0.0  # Eq. 8 gamma; 0 = no limit

    @property
    def N(self) -> int:
        return self.n_ffn + self.n_zero + self.n_copy + self.n_const

    @property
    def M_cap(self) -> int:
        return self.T * self.top_k + self.n_ffn * (self.row_align - 1)


def _f32(a):
    return None if a is None else np.ascontiguousarray(a, dtype=np.float32)


def _i32(a):
    return None if a is None else np.ascontiguousarray(a, dtype=np.int32)


def _ptr(a):
    return None if a is None else a.ctypes.data_as(ctypes.c_void_p)


def _ffn_w(a):
    """FFN weights: float32 array, or uint16 array of bf16 bit patterns.  Returns (array, is_bf16)."""
    if a is None:
        return None, 0
    if a.dtype == np.uint16:
        return np.ascontiguousarray(a), 1
    return np.ascontiguousarray(a, dtype=np.float32), 0


class Oracle:
    def __init__(self, arithmetic: str = "f64"):
        if arithmetic not in ("f32", "f64"):
            raise ValueError("arithmetic must be 'f32' or 'f64'")
        self.arithmetic = arithmetic
        self._lib = ctypes.CDLL(build())
        self._lib.oracle_num_threads.restype = ctypes.c_int
        self._pfx = "oracle_%s_" % arithmetic

    def num_threads(self) -> int:
        return int(self._lib.oracle_num_threads())

    def _call(self, name, *args):
        fn = getattr(self._lib, self._pfx + name)
        fn.restype = ctypes.c_int
        rc = fn(*args)
        if rc != 0:
            raise RuntimeError("oracle %s failed with code %d" % (name, rc))

    def _cfg(self, s: LayerShape, ffn_w_bf16: int = 0):
        return ctypes.byref(_Cfg(s.T, s.D, s.F, s.n_ffn, s.n_zero, s.n_copy, s.n_const, s.top_k, s.renorm_topk,
                                 s.row_align, s.add_residual, ffn_w_bf16, s.tau, s.capacity_factor))

    # Eq. 2 / Eq. 6
    def router_logits(self, s, x, W_r, W_g=None, prev=None, bias=None):
        x, W_r, W_g, prev, bias = _f32(x), _f32(W_r), _f32(W_g), _f32(prev), _f32(bias)
        G = np.empty((s.T, s.N), np.float32)
        self._call("router_logits", self._cfg(s), _ptr(x), _ptr(W_r), _ptr(W_g), _ptr(prev), _ptr(bias), _ptr(G))
        return G

    # Eq. 1 gate
    def gate_topk(self, s, G, want_probs=False):
        G = _f32(G)
        idx = np.empty((s.T, s.top_k), np.int32)
        w = np.empty((s.T, s.top_k), np.float32)
        P = np.empty((s.T, s.N), np.float32) if want_probs else None
        self._call("gate_topk", self._cfg(s), _ptr(G), _ptr(idx), _ptr(w), _ptr(P))
        return (idx, w, P) if want_probs else (idx, w)

    def tables(self, s, idx):
        idx = _i32(idx)
        counts = np.empty(s.N, np.int32)
        offsets = np.empty(s.n_ffn + 1, np.int32)
        row_of_slot = np.empty((s.T, s.top_k), np.int32)
        slot_of_row = np.empty(max(s.M_cap, 1), np.int32)
        self._call("tables", self._cfg(s), _ptr(idx), _ptr(counts), _ptr(offsets), _ptr(row_of_slot),
                   _ptr(slot_of_row))
        return counts, offsets, row_of_slot, slot_of_row[:s.M_cap]

    def capacities(self, s):
        """(cap_ffn, cap_zc) of Eq. 8 in routing slots."""
        a, b = ctypes.c_int32(0), ctypes.c_int32(0)
        self._lib.oracle_capacities(self._cfg(s), ctypes.byref(a), ctypes.byref(b))
        return int(a.value), int(b.value)

    # Eq. 7
    def balance_stats(self, s, G, idx):
        G, idx = _f32(G), _i32(idx)
        f, P, loss = np.empty(s.N, np.float32), np.empty(s.N, np.float32), np.empty(1, np.float32)
        self._call("balance_stats", self._cfg(s), _ptr(G), _ptr(idx), _ptr(f), _ptr(P), _ptr(loss))
        return f, P, float(loss[0])

    def balance_backward(self, s, G, f, scale=1.0, into=None):
        """d(scale * L_b)/dG of Eq. 7 with f held fixed; added to `into` (float32 [T, N]) if given."""
        G, f = _f32(G), _f32(f)
        dG = np.zeros((s.T, s.N), np.float32) if into is None else np.ascontiguousarray(into, np.float32).copy()
        self._call("balance_backward", self._cfg(s), _ptr(G), _ptr(f), ctypes.c_float(scale),
                   ctypes.c_int(0 if into is None else 1), _ptr(dG))
        return dG

    def permute_rows(self, s, x, slot_of_row):
        x, slot_of_row = _f32(x), _i32(slot_of_row)
        out = np.empty((len(slot_of_row), s.D), np.float32)
        self._call("permute_rows", self._cfg(s), _ptr(x), _ptr(slot_of_row), ctypes.c_int64(len(slot_of_row)),
                   _ptr(out))
        return out

    # Eq. 5 mixing weights
    def const_alpha(self, s, x, W_c):
        x, W_c = _f32(x), _f32(W_c)
        alpha = np.empty((s.T, s.n_const, 2), np.float32)
        self._call("const_alpha", self._cfg(s), _ptr(x), _ptr(W_c), _ptr(alpha))
        return alpha

    def ffn_token(self, s, x_row, Wg_e, Wu_e, Wd_e):
        x_row = _f32(x_row)
        (Wg_e, b), (Wu_e, _), (Wd_e, _) = _ffn_w(Wg_e), _ffn_w(Wu_e), _ffn_w(Wd_e)
        out = np.empty(s.D, np.float32)
        self._call("ffn_token", self._cfg(s, b), _ptr(x_row), _ptr(Wg_e), _ptr(Wu_e), _ptr(Wd_e), _ptr(out))
        return out

    def grouped_ffn(self, s, x_perm, offsets, counts, W_gate, W_up, W_down):
        x_perm, offsets, counts = _f32(x_perm), _i32(offsets), _i32(counts)
        (W_gate, b), (W_up, _), (W_down, _) = _ffn_w(W_gate), _ffn_w(W_up), _ffn_w(W_down)
        y_perm = np.zeros_like(x_perm)
        self._call("grouped_ffn", self._cfg(s, b), _ptr(x_perm), _ptr(offsets), _ptr(counts), _ptr(W_gate),
                   _ptr(W_up), _ptr(W_down), _ptr(y_perm))
        return y_perm

    # Eq. 1 sum with Eq. 3-5
    def combine(self, s, x, y_perm, idx, w, row_of_slot, alpha=None, v=None):
        x, y_perm, idx, w = _f32(x), _f32(y_perm), _i32(idx), _f32(w)
        row_of_slot, alpha, v = _i32(row_of_slot), _f32(alpha), _f32(v)
        y = np.empty((s.T, s.D), np.float32)
        self._call("combine", self._cfg(s), _ptr(x), _ptr(y_perm), _ptr(idx), _ptr(w), _ptr(row_of_slot),
                   _ptr(alpha), _ptr(v), _ptr(y))
        return y

    def layer_forward(self, s, x, W_r, W_g=None, prev=None, bias=None, W_c=None, v=None, W_gate=None, W_up=None,
                      W_down=None, forced_idx=None, tokens=None):
        """Returns dict(logits [T,N], idx [T,K], w [T,K], y [T or len(tokens), D])."""
        x, W_r, W_g, prev, bias = _f32(x), _f32(W_r), _f32(W_g), _f32(prev), _f32(bias)
        W_c, v = _f32(W_c), _f32(v)
        (W_gate, b), (W_up, _), (W_down, _) = _ffn_w(W_gate), _ffn_w(W_up), _ffn_w(W_down)
        forced_idx, tokens = _i32(forced_idx), _i32(tokens)
        n_out = s.T if tokens is None else len(tokens)
        logits = np.empty((s.T, s.N), np.float32)
        idx = np.empty((s.T, s.top_k), np.int32)
        w = np.empty((s.T, s.top_k), np.float32)
        y = np.empty((n_out, s.D), np.float32)
        self._call("layer_forward", self._cfg(s, b), _ptr(x), _ptr(W_r), _ptr(W_g), _ptr(prev), _ptr(bias),
                   _ptr(W_c), _ptr(v), _ptr(W_gate), _ptr(W_up), _ptr(W_down), _ptr(forced_idx), _ptr(tokens),
                   ctypes.c_int32(0 if tokens is None else len(tokens)), _ptr(logits), _ptr(idx), _ptr(w), _ptr(y))
        return dict(logits=logits, idx=idx, w=w, y=y)

    def layer_backward(self, s, x, W_r, idx, dy, W_g=None, prev=None, bias=None, W_c=None, v=None, W_gate=None,
                       W_up=None, W_down=None, dlogits=None):
        """Gradients of a scalar L given dy = dL/dy (and dlogits = dL/dlogits from the next layer), with the picks
        `idx` held fixed.  Returns a dict with dx, dprev, dW_r, dW_g, dbias, dW_c, dv, dW_gate, dW_up, dW_down."""
        x, W_r, W_g, prev, bias, W_c, v = _f32(x), _f32(W_r), _f32(W_g), _f32(prev), _f32(bias), _f32(W_c), _f32(v)
        W_gate, W_up, W_down, dy, dlogits, idx = _f32(W_gate), _f32(W_up), _f32(W_down), _f32(dy), _f32(dlogits), _i32(idx)
        z = lambda *shape: np.zeros(shape, np.float32)
        out = dict(dx=z(s.T, s.D), dprev=z(s.T, s.N) if W_g is not None else None, dW_r=z(s.N, s.D),
                   dW_g=z(s.N, s.N) if W_g is not None else None, dbias=z(s.N), dW_c=z(max(s.n_const, 0), 2, s.D),
                   dv=z(max(s.n_const, 0), s.D), dW_gate=z(s.n_ffn, s.F, s.D), dW_up=z(s.n_ffn, s.F, s.D),
                   dW_down=z(s.n_ffn, s.D, s.F))
        self._call("layer_backward", self._cfg(s), _ptr(x), _ptr(W_r), _ptr(W_g), _ptr(prev), _ptr(bias), _ptr(W_c),
                   _ptr(v), _ptr(W_gate), _ptr(W_up), _ptr(W_down), _ptr(idx), _ptr(dy), _ptr(dlogits),
                   _ptr(out["dx"]), _ptr(out["dprev"]), _ptr(out["dW_r"]), _ptr(out["dW_g"]), _ptr(out["dbias"]),
                   _ptr(out["dW_c"]), _ptr(out["dv"]), _ptr(out["dW_gate"]), _ptr(out["dW_up"]), _ptr(out["dW_down"]))
        return out
