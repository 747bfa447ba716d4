"""Conversion of seeded workload tensors into the numpy arrays the oracle takes (TEST INFRASTRUCTURE ONLY).

Duck-typed on purpose: nothing from the CUDA library or its package is imported here.  bf16 tensors are
handed over as their bit patterns, so the oracle sees exactly the stored values.
"""
from __future__ import annotations

import numpy as np
import torch

from . import LayerShape


def bits_or_f32(t: torch.Tensor) -> np.ndarray:
    """FFN weights for the oracle: bf16 tensors as uint16 bit patterns, float tensors as float32."""
    t = t.detach().cpu().contiguous()
    if t.dtype == torch.bfloat16:
        return t.view(torch.int16).numpy().view(np.uint16)
    return t.float().numpy()


def f32(t):
    return None if t is None else t.detach().cpu().float().contiguous().numpy()


def shape_of(spec, **over) -> LayerShape:
    kw = dict(T=spec.T, D=spec.D, F=spec.F, n_ffn=spec.n_ffn, n_zero=spec.n_zero, n_copy=spec.n_copy,
              n_const=spec.n_const, top_k=spec.top_k)
    kw.update(over)
    return LayerShape(**kw)


def oracle_inputs(lt) -> dict:
    """The same stored values the CUDA side sees, widened for the oracle."""
    return dict(x=f32(lt.x), W_r=f32(lt.W_r), W_g=f32(lt.W_g), prev=f32(lt.prev), bias=f32(lt.bias), W_c=f32(lt.W_c),
                v=f32(lt.v), W_gate=bits_or_f32(lt.W_gate), W_up=bits_or_f32(lt.W_up), W_down=bits_or_f32(lt.W_down))
