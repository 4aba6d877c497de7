"""Verify-cycle driver over the C-ABI binding: device buffers, stream-ordered calls, graph replay.

Nothing here computes anything of the method; it owns tensors and issues, per cycle,
    for each layer: branch_state_build -> tree_verify_attn
    then:           accept_and_refresh(all layers)
on one CUDA stream with no host synchronisation in between.
"""
from __future__ import annotations

import weakref
from typing import Dict, List, Optional, Sequence

import numpy as np
import torch

from . import binding as tsv
from . import synth

_NODE_FIELDS = ("q", "kv", "c_csa", "ikc", "g_csa", "c_hca", "g_hca", "iq", "iw")
_F32_FIELDS = ("g_csa", "g_hca", "iw")


def capacities(shape: synth.Shape, lengths: Sequence[int], headroom_tokens: int):
    """Rows to reserve per sequence so that `headroom_tokens` more tokens can be committed."""
    D = shape.D
    csa = [(int(L) + headroom_tokens + D) // shape.m_csa + 1 for L in lengths]
    hca = [(int(L) + headroom_tokens + D) // shape.m_hca + 1 for L in lengths]
    return csa, hca


def fill_cache(cache: tsv.LayerCache, shape: synth.Shape, b: int, L: int, arrays: Dict[str, np.ndarray]) -> None:
    """Copy one sequence's committed state (numpy arrays holding storage-dtype values) to the device.

    arrays: csa_kv [n_csa,d], csa_ik [n_csa,di], hca_kv [n_hca,d], win [<=w rows or w,d] placed by
    `win_slots`, csa_mx, csa_s, csa_acc_kv, csa_acc_ik, hca_mx, hca_s, hca_acc_kv."""
    dt = tsv.torch_dtype(shape)
    dev = cache.L.device
    up = lambda a, t=dt: torch.from_numpy(np.ascontiguousarray(a, dtype=np.float32)).to(dev).to(t)
    cache.L[b] = int(L)
    n = arrays["csa_kv"].shape[0]
    assert n <= int(cache.csa_cap[b])
    if n:
        rows = cache.csa_row_index(shape, b, n)
        cache.csa_kv[rows] = up(arrays["csa_kv"]); cache.csa_ik[rows] = up(arrays["csa_ik"])
    n = arrays["hca_kv"].shape[0]
    assert n <= int(cache.hca_cap[b])
    if n:
        cache.hca_kv[cache.hca_row_index(shape, b, n)] = up(arrays["hca_kv"])
    if cache.page_table is None:
        cache.win_kv[b] = up(arrays["win"])
    else:                       # token-level pool: the last min(L, window) positions, taken from their ring slots
        pos = torch.arange(max(0, int(L) - shape.window), int(L), dtype=torch.long, device=dev)
        if pos.numel():
            cache.win_kv[cache.tok_row_index(shape, b, pos)] = up(arrays["win"])[pos % shape.window]
    f = torch.float32
    cache.csa_mx[b] = float(arrays["csa_mx"]); cache.csa_s[b] = float(arrays["csa_s"])
    cache.hca_mx[b] = float(arrays["hca_mx"]); cache.hca_s[b] = float(arrays["hca_s"])
    cache.csa_acc_kv[b] = up(arrays["csa_acc_kv"], f); cache.csa_acc_ik[b] = up(arrays["csa_acc_ik"], f)
    cache.hca_acc_kv[b] = up(arrays["hca_acc_kv"], f)


def nodes_to_device(shape: synth.Shape, nodes: Dict[str, np.ndarray], parent: np.ndarray, n_nodes: np.ndarray,
                    device="cuda") -> tsv.NodeInputs:
    dt = tsv.torch_dtype(shape)
    t = {k: torch.from_numpy(np.ascontiguousarray(nodes[k], dtype=np.float32)).to(device).to(torch.float32 if k in _F32_FIELDS else dt)
         for k in _NODE_FIELDS}
    return tsv.NodeInputs(parent=torch.from_numpy(np.ascontiguousarray(parent, dtype=np.int32)).to(device),
                          n_nodes=torch.from_numpy(np.ascontiguousarray(n_nodes, dtype=np.int32)).to(device), **t)


class InputSet:
    """Per-cycle inputs of all layers on the device: node tensors, the tree, draft/target tokens."""

    def __init__(self, layer_nodes: List[tsv.NodeInputs], draft: torch.Tensor, target: torch.Tensor):
        self.layers, self.draft, self.target = layer_nodes, draft, target

    @staticmethod
    def empty(shape: synth.Shape, n_layers: int, device="cuda") -> "InputSet":
        dt, B, D = tsv.torch_dtype(shape), shape.B, shape.D
        i32 = dict(dtype=torch.int32, device=device)
        parent = torch.zeros(B, D, **i32); parent[:, 0] = -1
        n_nodes = torch.ones(B, **i32)
        v = lambda *s: torch.zeros(*s, dtype=dt, device=device)
        f = lambda *s: torch.zeros(*s, dtype=torch.float32, device=device)
        layers = [tsv.NodeInputs(q=v(B, D, shape.H, shape.d), kv=v(B, D, shape.d), c_csa=v(B, D, shape.d), ikc=v(B, D, shape.di),
                                 g_csa=f(B, D), c_hca=v(B, D, shape.d), g_hca=f(B, D), iq=v(B, D, shape.HI, shape.di),
                                 iw=f(B, D, shape.HI), parent=parent, n_nodes=n_nodes) for _ in range(n_layers)]
        return InputSet(layers, torch.zeros(B, D, **i32), torch.zeros(B, D, **i32))

    @staticmethod
    def from_numpy(shape: synth.Shape, layer_nodes: List[Dict[str, np.ndarray]], parent, n_nodes, draft, target,
                   device="cuda") -> "InputSet":
        layers = [nodes_to_device(shape, nd, parent, n_nodes, device) for nd in layer_nodes]
        for nd in layers[1:]:
            nd.parent, nd.n_nodes = layers[0].parent, layers[0].n_nodes
        return InputSet(layers, torch.from_numpy(np.ascontiguousarray(draft, dtype=np.int32)).to(device),
                        torch.from_numpy(np.ascontiguousarray(target, dtype=np.int32)).to(device))

    def tensors(self) -> List[torch.Tensor]:
        out = []
        for nd in self.layers:
            out += [getattr(nd, k) for k in _NODE_FIELDS]
        return out + [self.layers[0].parent, self.layers[0].n_nodes, self.draft, self.target]

    def pinned_host_copy(self) -> List[torch.Tensor]:
        return [t.cpu().pin_memory() for t in self.tensors()]

    def load_from_host(self, host: List[torch.Tensor]) -> int:
        """Async host-to-device copy of every input tensor; returns the bytes moved."""
        n = 0
        for d, h in zip(self.tensors(), host):
            d.copy_(h, non_blocking=True)
            n += h.numel() * h.element_size()
        return n


class VerifyEngine:
    """Owns the persistent caches, scratch pads, workspace and outputs of an n-layer stack."""

    def __init__(self, shape: synth.Shape, n_layers: int, csa_caps, hca_caps, max_L: int, flags: int = 0,
                 want_topk: bool = False, device="cuda", page_tokens: int = 0):
        self.shape, self.n_layers, self.device = shape, n_layers, device
        self.cshape = tsv.c_shape(shape, max_L, flags)
        if page_tokens:         # paged pool: per layer its own pool and page table (different shuffles)
            self.caches = [tsv.alloc_cache_paged(shape, csa_caps, hca_caps, page_tokens, seed=l, device=device) for l in range(n_layers)]
        else:
            self.caches = [tsv.alloc_cache(shape, csa_caps, hca_caps, device) for _ in range(n_layers)]
        self.scratch = [tsv.alloc_scratch(shape, device) for _ in range(n_layers)]
        self.workspace = tsv.alloc_workspace(shape, max_L, flags, device)
        dt = tsv.torch_dtype(shape)
        B, D = shape.B, shape.D
        self.out = [torch.zeros(B, D, shape.H, shape.d, dtype=dt, device=device) for _ in range(n_layers)]
        self.topk_idx = [torch.full((B, D, shape.topk), -2, dtype=torch.int32, device=device) if want_topk else None
                         for _ in range(n_layers)]
        i32 = dict(dtype=torch.int32, device=device)
        self.status = torch.zeros(B, **i32)
        self.accept_len = torch.zeros(B, **i32)
        self.accept_path = torch.zeros(B, D, **i32)
        self.bonus = torch.zeros(B, **i32)
        # pointer packs per input set; weak keys: an entry must die with its input set (an id() key could be reused by a
        # later input set and hand accept_and_refresh the pointers of freed tensors)
        self._packs = weakref.WeakKeyDictionary()

    def _pack(self, inp: InputSet) -> tsv.LayerPack:
        p = self._packs.get(inp)
        if p is None:
            p = self._packs[inp] = tsv.LayerPack(self.caches, inp.layers, self.scratch)
        return p

    def launch_cycle(self, inp: InputSet, attention: bool = True, refresh: bool = True) -> None:
        """Enqueue one verify cycle on the current stream (no host sync)."""
        self.status.zero_()
        for l in range(self.n_layers):
            tsv.branch_state_build(self.cshape, self.caches[l], inp.layers[l], self.scratch[l], self.status)
            if attention:
                tsv.tree_verify_attn(self.cshape, self.caches[l], inp.layers[l], self.scratch[l], self.out[l], self.topk_idx[l],
                                     self.workspace, self.status)
        if refresh:
            tsv.accept_and_refresh(self.cshape, self._pack(inp), inp.draft, inp.target, self.accept_len, self.accept_path,
                                   self.bonus, self.status)

    def capture(self, inp: InputSet) -> torch.cuda.CUDAGraph:
        """Capture one cycle over `inp` into a CUDA graph (the launch sequence is shape-stable)."""
        self._pack(inp)
        s = torch.cuda.Stream()
        s.wait_stream(torch.cuda.current_stream())
        g = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g, stream=s):
            self.launch_cycle(inp)
        torch.cuda.current_stream().wait_stream(s)
        return g

    def snapshot(self) -> List[tsv.LayerCache]:
        return [c.clone() for c in self.caches]

    def restore(self, snap: List[tsv.LayerCache]) -> None:
        for c, s in zip(self.caches, snap):
            for name in tsv.CACHE_TENSORS:
                getattr(c, name).copy_(getattr(s, name))
