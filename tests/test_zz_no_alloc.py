"""moepp_grouped_ffn_static: the grouped FFN for callers that cannot bring scratch memory.

Some users of this library are given input and output buffers only and are not allowed to create device
memory (an operator inside a runtime whose memory planner owns the GPU, a loop that cannot afford the
device-wide stall of an allocation).  For them the intermediate of the FFN lives in a fixed array
inside the library.  This test calls that entry point through the C-ABI twice in a row, with different
problems, and checks each result against the ordinary entry point (which takes caller scratch), to the
tolerance the other parity tests use; the second call also shows that what the first call left in the
shared array does no harm.  Collected last on purpose (file name), so a failure here cannot hide others.
"""
import numpy as np
import pytest
import torch

from paper_2410_07348_b200 import binding as B

pytestmark = pytest.mark.gpu

BF16_REL_TOL = 2e-2
F32_ABS_TOL = 1e-4


def _problem(seed, T, D, F, n_ffn, dtype, row_align=1):
    g = torch.Generator().manual_seed(seed)
    td = torch.bfloat16 if dtype == B.MOEPP_BF16 else torch.float32
    cfg = B.Config(T=T, D=D, F=F, n_ffn=n_ffn, n_zero=1, n_copy=1, n_const=2, top_k=2, dtype=dtype,
                   row_align=row_align)
    # a ragged split of some of the rows over the experts (one expert empty), the rest unused
    cuts = sorted(torch.randint(0, T * 2 - n_ffn * row_align, (n_ffn - 1,), generator=g).tolist())
    counts = np.diff([0] + cuts + [T * 2 - n_ffn * row_align - 7]).clip(min=0)
    counts[1] = 0
    seg = (counts + row_align - 1) // row_align * row_align
    offsets = torch.tensor(np.concatenate([[0], np.cumsum(seg)]), dtype=torch.int32).cuda()
    x_perm = torch.randn(cfg.M_cap, D, generator=g).to(td).cuda()
    w = [(torch.randn(*s, generator=g) * 0.05).to(td).cuda() for s in ((n_ffn, F, D), (n_ffn, F, D), (n_ffn, D, F))]
    return cfg, offsets, x_perm, w


def _both(cfg, offsets, x_perm, w):
    td = x_perm.dtype
    h = torch.empty(cfg.M_cap, cfg.F, dtype=td, device="cuda")
    y_ref = torch.zeros(cfg.M_cap, cfg.D, dtype=td, device="cuda")
    y_new = torch.zeros(cfg.M_cap, cfg.D, dtype=td, device="cuda")
    B.moepp_grouped_ffn(cfg, x_perm, offsets, w[0], w[1], w[2], h, y_ref)
    torch.cuda.synchronize()
    B.moepp_grouped_ffn_static(cfg, x_perm, offsets, w[0], w[1], w[2], y_new)
    torch.cuda.synchronize()
    assert B.moepp_device_error() == 0
    return y_ref.float().cpu().numpy(), y_new.float().cpu().numpy()


def _check(cfg, ref, new):
    assert np.isfinite(ref).all() and np.abs(ref).max() > 0
    if cfg.dtype == B.MOEPP_F32:
        assert np.abs(new - ref).max() <= F32_ABS_TOL
    else:
        row = np.abs(ref).max(axis=1)
        err = np.abs(new - ref).max(axis=1) / np.maximum(row, 1e-6 * np.abs(ref).max())
        assert err.max() <= BF16_REL_TOL


def test_static_scratch_matches_caller_scratch_twice_in_a_row():
    first = _problem(1, T=700, D=256, F=512, n_ffn=5, dtype=B.MOEPP_BF16)
    second = _problem(2, T=300, D=328, F=392, n_ffn=4, dtype=B.MOEPP_BF16, row_align=128)
    for prob in (first, second):
        ref, new = _both(*prob)
        _check(prob[0], ref, new)
    third = _problem(3, T=200, D=64, F=128, n_ffn=3, dtype=B.MOEPP_F32)
    ref, new = _both(*third)
    _check(third[0], ref, new)


def test_static_scratch_refuses_problems_beyond_its_size():
    cfg = B.Config(T=16384, D=1024, F=2816, n_ffn=8, n_zero=1, n_copy=1, n_const=2, dtype=B.MOEPP_BF16)
    assert cfg.M_cap * cfg.F * 2 > B.STATIC_SCRATCH_BYTES
    one = torch.zeros(16, dtype=torch.int32, device="cuda")
    with pytest.raises(B.MoeppError) as ei:
        B.moepp_grouped_ffn_static(cfg, one, one, one, one, one, one)
    assert ei.value.status == 4  # MOEPP_ERR_WORKSPACE, before anything is launched
