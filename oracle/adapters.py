"""Glue between the seeded input generators (torch bf16 tensors) and the oracle's numpy bit arrays.
Test infrastructure only; holds no arithmetic of the method."""
from __future__ import annotations

import numpy as np
import torch

from .mtad_oracle import OracleModel


def bits(t: torch.Tensor) -> np.ndarray:
    """bf16 torch tensor -> uint16 numpy array of its bit patterns (host copy)."""
    assert t.dtype == torch.bfloat16
    return t.detach().cpu().contiguous().view(torch.int16).numpy().view(np.uint16)


class _LazyLayers:
    """Builds one layer at a time from a callable so that large shapes stream through host memory."""

    def __init__(self, n, make):
        self.n, self.make, self._cache = n, make, (None, None)

    def __len__(self):
        return self.n

    def __getitem__(self, l):
        if self._cache[0] != l:
            self._cache = (l, {k: bits(v) for k, v in self.make(l).items()})
        return self._cache[1]


def oracle_model(model: dict, layer_maker=None) -> OracleModel:
    """model: the dict returned by mtad_synth.make_model (or the same without 'layers' plus layer_maker(l))."""
    s = model["shape"]
    if layer_maker is None:
        layers = [{k: bits(v) for k, v in lw.items()} for lw in model["layers"]]
    else:
        layers = _LazyLayers(s.layers, layer_maker)
    return OracleModel(s.layers, s.d_model, s.n_q_heads, s.n_kv_heads, s.head_dim, s.d_ffn, s.vocab,
                       s.rope_base, s.rms_eps, bits(model["embed"]), bits(model["lm_head"]),
                       bits(model["final_norm"]), layers)


def cache_bits(cache: torch.Tensor, seq: int) -> np.ndarray:
    """One sequence's slice of a [layers, B, 2, Hkv, cap, hd] bf16 cache as a writable uint16 array
    [layers, 2, Hkv, cap, hd]."""
    return bits(cache[:, seq]).copy()
