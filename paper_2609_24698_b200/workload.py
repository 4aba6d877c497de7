"""Timing workloads: device-resident caches and per-cycle input sets for a named config,
plus the algorithmic work (bytes, FLOPs) of one verify cycle.

For timing, cache CONTENTS are drawn directly (synth.direct_cache) instead of compressing a
drawn prefix: timing does not depend on the values, and the product path has no prefill
kernel to run.  Parity tests build their caches from compressed prefixes instead.
"""
from __future__ import annotations

from dataclasses import dataclass
from typing import Dict, List

import numpy as np
import torch

from . import binding as tsv
from . import harness as hz
from . import synth


direct_arrays = synth.direct_arrays      # (kept under this name for the callers of this module)


@dataclass
class Workload:
    cfg: synth.Config
    lengths: np.ndarray
    engine: hz.VerifyEngine
    inputs: List[hz.InputSet]


def build(cfg: synth.Config, cycles_headroom: int, n_sets: int = 3, flags: int = 0, device="cuda", page_tokens: int = 0) -> Workload:
    sh = cfg.shape
    lengths = synth.prefix_lengths(cfg)
    ccap, hcap = hz.capacities(sh, lengths, cycles_headroom * sh.D)
    max_L = int(lengths.max()) + (cycles_headroom + 1) * sh.D
    eng = hz.VerifyEngine(sh, cfg.layers, ccap, hcap, max_L, flags=flags, want_topk=False, device=device, page_tokens=page_tokens)
    for l in range(cfg.layers):
        for b in range(sh.B):
            hz.fill_cache(eng.caches[l], sh, b, int(lengths[b]), direct_arrays(cfg, l, b, int(lengths[b])))
    sets = []
    for c in range(n_sets):
        nodes = [synth.node_inputs(cfg, l, c) for l in range(cfg.layers)]
        parent, n_nodes = synth.trees(cfg, c)
        draft, target = synth.tokens(cfg, c, parent, n_nodes)
        sets.append(hz.InputSet.from_numpy(sh, nodes, parent, n_nodes, draft, target, device))
    return Workload(cfg, lengths, eng, sets)


def algorithmic_work(sh: synth.Shape, n_layers: int, lengths: np.ndarray, parents: np.ndarray) -> Dict[str, float]:
    """Compulsory bytes and FLOPs of ONE verify cycle (all layers), from the shapes alone.

    attention (per sequence-layer): distinct CSA rows read (all of them when n_csa <= topk, else the
    expected union of D independent selections), HCA rows, window rows, tree rows, q in, out;
    selection: all indexer keys, only when a node has more candidates than topk;
    state build / refresh: per-node compression inputs, scratch states, committed rows."""
    es = 2 if sh.dtype == "bf16" else 4
    D, H, d, di = sh.D, sh.H, sh.d, sh.di
    attn_cache = sel_bytes = attn_flops = sel_flops = 0.0
    depth = np.zeros_like(parents)
    for n in range(1, D):
        depth[:, n] = depth[np.arange(parents.shape[0]), parents[:, n]] + 1
    for b, L in enumerate(np.asarray(lengths, dtype=np.int64)):
        n_csa, n_hca, nw = L // sh.m_csa, L // sh.m_hca, min(L, sh.window)
        k_eff = min(sh.topk, n_csa)
        U = n_csa if n_csa <= sh.topk else n_csa * (1.0 - (1.0 - sh.topk / n_csa) ** D)
        attn_cache += (U + n_hca + nw + D) * d * es
        keys = sum(k_eff + n_hca + max(0, nw - 1 - int(depth[b, n])) + int(depth[b, n]) + 1 for n in range(D))
        attn_flops += 4.0 * H * d * keys
        if n_csa > sh.topk:
            sel_bytes += n_csa * di * es
            sel_flops += 2.0 * D * sh.HI * di * n_csa
    B = len(lengths)
    q_out = 2.0 * B * D * H * d * es
    node_small = B * D * ((3 * d + di + sh.HI * di) * es + (2 + sh.HI) * 4)
    state_rw = B * D * (2 * d + di) * 4 * 2 + B * D * (2 * d + di) * es      # scratch states written + read at commit, entries
    per_layer_attn = attn_cache + q_out + B * D * d * es
    return {
        "attn_bytes_per_layer": per_layer_attn,
        "attn_flops_per_layer": attn_flops,
        "cache_bytes": n_layers * (attn_cache + sel_bytes),
        "full_bytes": n_layers * (per_layer_attn + sel_bytes + node_small + state_rw),
        "flops": n_layers * (attn_flops + sel_flops),
    }
