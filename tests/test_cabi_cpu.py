"""CPU-side checks of the C-ABI library: it loads, exports every symbol the header declares, and its
host-only paths (status strings, workspace sizing, argument validation that returns before any launch)
behave as documented.  No kernel is launched here."""
import ctypes
import os
import re

import pytest

from paper_2410_07348_b200 import binding as B
from paper_2410_07348_b200 import build as build_mod

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    build_mod.build()
    return B.lib()


def declared_symbols():
    text = open(os.path.join(ROOT, "include", "moepp.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(moepp_[a-z_]+)\s*\(", text)))


def test_every_declared_symbol_is_exported(lib):
    names = declared_symbols()
    assert {"moepp_route", "moepp_permute", "moepp_grouped_ffn", "moepp_combine", "moepp_layer_forward"} <= set(names)
    for n in names:
        assert hasattr(lib, n), n
    assert set(names) == set(B.EXPORTS)


def test_status_strings(lib):
    seen = {lib.moepp_status_string(i).decode() for i in range(7)}
    assert len(seen) == 7 and "ok" in seen


def test_workspace_bytes_is_host_only_and_monotone(lib):
    small = B.Config(T=128, D=256, F=512, n_ffn=8, n_zero=1, n_copy=1, n_const=2)
    big = B.Config(T=256, D=256, F=512, n_ffn=8, n_zero=1, n_copy=1, n_const=2)
    a, b = B.moepp_workspace_bytes(small), B.moepp_workspace_bytes(big)
    assert 0 < a < b and a % 256 == 0
    # grouped buffers dominate: x_perm + h + y_perm for M_cap rows
    rows = small.M_cap
    assert a >= rows * (2 * 256 + 512) * 2
    assert B.moepp_workspace_bytes(small, host=True) > a
    assert B.moepp_workspace_bytes(B.Config(T=0, D=64, F=64, n_ffn=2)) > 0


@pytest.mark.parametrize("bad,status", [
    (dict(T=-1), 1), (dict(D=0), 1), (dict(top_k=0), 1), (dict(top_k=13), 1), (dict(top_k=9, n_ffn=20), 2),
    (dict(n_ffn=70), 2), (dict(dtype=5), 1), (dict(row_align=0), 1), (dict(D=60), 3), (dict(F=100), 3),
    (dict(n_ffn=0, n_zero=0, n_copy=0, n_const=0), 1), (dict(n_ffn=30, n_const=34), 2),
])
def test_bad_configs_are_rejected_on_the_host(lib, bad, status):
    kw = dict(T=16, D=64, F=64, n_ffn=8, n_zero=1, n_copy=1, n_const=2)
    kw.update(bad)
    with pytest.raises(B.MoeppError) as ei:
        B.moepp_workspace_bytes(B.Config(**kw))
    assert ei.value.status == status


def test_null_config_and_null_outputs(lib):
    n = ctypes.c_size_t(0)
    assert lib.moepp_workspace_bytes(None, ctypes.byref(n)) == 1
    c = B.Config(T=16, D=64, F=64, n_ffn=2).c()
    assert lib.moepp_workspace_bytes(ctypes.byref(c), None) == 1
    null = ctypes.c_void_p(0)
    # every call checks its pointers before touching the device
    assert lib.moepp_route(ctypes.byref(c), *([null] * 13)) == 1
    assert lib.moepp_permute(ctypes.byref(c), *([null] * 7)) == 1
    assert lib.moepp_grouped_ffn(ctypes.byref(c), *([null] * 8)) == 1
    assert lib.moepp_combine(ctypes.byref(c), *([null] * 10)) == 1
    one = ctypes.c_void_p(256)  # a non-null stand-in: these calls must fail on the NEXT missing pointer, before any launch
    assert lib.moepp_route(ctypes.byref(c), null, null, null, null, null, null, null, null, null, one, one, null,
                           null) == 1
    assert lib.moepp_permute(ctypes.byref(c), null, null, one, null, null, null, null) == 1
    assert lib.moepp_grouped_ffn(ctypes.byref(c), null, one, null, null, null, null, null, null) == 1
    assert lib.moepp_layer_forward(ctypes.byref(c), *([null] * 6), ctypes.c_size_t(0), null) == 1
    assert lib.moepp_layer_forward_host(ctypes.byref(c), *([null] * 6), ctypes.c_size_t(0), null) == 1
    assert lib.moepp_device_error(None) == 1
    assert lib.moepp_balance_stats(ctypes.byref(c), *([null] * 6)) == 1
    assert lib.moepp_stack_forward(ctypes.byref(c), null, 1, *([null] * 5), ctypes.c_size_t(0), null) == 1
    assert lib.moepp_stack_forward_host(ctypes.byref(c), null, 1, *([null] * 5), ctypes.c_size_t(0), null) == 1


def test_backward_sizing_and_argument_checks_are_host_only(lib):
    """The backward and training-stack entry points: workspace sizes are pure host arithmetic, and bad arguments come
    back as status codes before anything is launched."""
    cfg = B.Config(T=512, D=256, F=512, n_ffn=8, n_zero=1, n_copy=1, n_const=2, row_align=64)
    kept = B.Config(T=512, D=256, F=512, n_ffn=8, n_zero=1, n_copy=1, n_const=2, row_align=64, flags=B.FLAG_SAVE_PREACT)
    bwd = B.moepp_backward_workspace_bytes(cfg)
    rows, es = cfg.M_cap, 2
    assert bwd % 256 == 0 and bwd >= rows * (2 * 256 + 2 * 512) * es  # dYp, dXp, gate, up
    # keeping the pre-activations adds two [M_cap, F] buffers to the forward workspace
    assert B.moepp_workspace_bytes(kept) - B.moepp_workspace_bytes(cfg) >= 2 * rows * 512 * es
    one_slot = B.moepp_stack_train_workspace_bytes(cfg, 1)
    assert B.moepp_stack_train_workspace_bytes(cfg, 3) == 3 * one_slot
    assert one_slot > B.moepp_workspace_bytes(cfg)
    assert B.moepp_stack_backward_workspace_bytes(cfg, 3) > bwd
    with pytest.raises(B.MoeppError):
        B.moepp_stack_train_workspace_bytes(cfg, 0)

    c = cfg.c()
    null, one = ctypes.c_void_p(0), ctypes.c_void_p(256)
    sz = ctypes.c_size_t(1 << 40)
    w = B.moepp_weights(*([256] * 8))
    g = B.moepp_grads()
    # no gradient set, no scratch
    assert lib.moepp_layer_backward(ctypes.byref(c), ctypes.byref(w), one, one, null, one, null, one, sz, None, one, sz,
                                    null) == 1
    # a gradient set without dW_r
    assert lib.moepp_layer_backward(ctypes.byref(c), ctypes.byref(w), one, one, null, one, null, one, sz,
                                    ctypes.byref(g), one, sz, null) == 1
    # workspaces too small: status 5 (workspace), checked before the gradient set is looked at
    assert lib.moepp_layer_backward(ctypes.byref(c), ctypes.byref(w), one, one, null, one, null, one,
                                    ctypes.c_size_t(16), ctypes.byref(g), one, ctypes.c_size_t(16), null) == \
        lib.moepp_layer_forward(ctypes.byref(c), ctypes.byref(w), one, one, one, null, one, ctypes.c_size_t(16), null)
    # the fused-gather forward keeps no x_perm, so it cannot be differentiated
    fused = B.Config(T=512, D=256, F=512, n_ffn=8, flags=B.FLAG_FUSED_GATHER).c()
    assert lib.moepp_layer_backward(ctypes.byref(fused), ctypes.byref(w), one, one, null, one, null, one, sz,
                                    ctypes.byref(g), one, sz, null) == 1
    assert lib.moepp_balance_backward(ctypes.byref(c), null, null, ctypes.c_float(1.0), 0, null, null) == 1
    assert lib.moepp_stack_forward_train(ctypes.byref(c), null, 1, *([null] * 5), ctypes.c_size_t(0), null) == 1
    assert lib.moepp_stack_backward(ctypes.byref(c), null, 1, null, null, null, null, ctypes.c_float(0.0), null, null,
                                    ctypes.c_size_t(0), None, null, ctypes.c_size_t(0), null) == 1


def test_missing_library_is_a_hard_error(monkeypatch):
    monkeypatch.setattr(B, "_lib", None)
    monkeypatch.setattr(B, "_LIB_PATH", "/nonexistent/libmoepp.so")
    with pytest.raises(RuntimeError):
        B.lib()
