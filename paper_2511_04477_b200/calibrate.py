"""Threshold calibration on top of ``spqt_calibrate_threshold`` (the paper's calibration tool, Sec. 5).

Two modes, as in the paper:

* ``unified(pools, sparsity)``: one global sparsity level for every site; each site's threshold is the
  nearest-rank order statistic of |x| over that site's calibration activations.
* ``grouped(pools, matrix_sparsity, groups)``: per-matrix sparsity levels (the paper takes them from a
  greedy search on trained models, which needs data that is not here: they are an input) are averaged
  over the matrices that share an input -- {q, k, v} and {gate, up} -- so that each group shares one
  threshold and therefore one index collection per token.

``pools`` maps a site name to a CUDA float16 tensor holding that site's calibration activations
(any number of tokens, concatenated).  Only argument handling happens here: the order statistic is
computed on the device by the library.
"""
from __future__ import annotations

from typing import Dict, Iterable, Mapping

import torch

from . import binding

# matrices of a Llama-style decoder layer by the input they read
LLAMA_GROUPS = {"attn_in": ("q", "k", "v"), "attn_out": ("o",), "mlp_in": ("gate", "up"), "mlp_mid": ("down",)}


def unified(pools: Mapping[str, torch.Tensor], sparsity: float) -> Dict[str, float]:
    """site -> threshold for one global sparsity level."""
    return grouped(pools, {site: sparsity for site in pools}, {site: (site,) for site in pools})


def grouped(pools: Mapping[str, torch.Tensor], matrix_sparsity: Mapping[str, float],
            groups: Mapping[str, Iterable[str]] = None) -> Dict[str, float]:
    """site -> threshold; the sparsity of a site is the mean of the sparsities of the matrices that read it."""
    groups = LLAMA_GROUPS if groups is None else groups
    out, ws, t = {}, None, None
    for site, pool in pools.items():
        names = tuple(groups[site])
        level = sum(float(matrix_sparsity[nm]) for nm in names) / len(names)
        if ws is None:
            ws = binding.new_calibration_workspace(pool.device)
            t = torch.empty(1, dtype=torch.float32, device=pool.device)
        binding.spqt_calibrate_threshold(pool.reshape(-1), level, ws, t)
        out[site] = float(t.item())
    return out
