"""Thin ctypes binding over the C-ABI library (include/tsv.h).  Argument marshalling only.

Torch tensors provide device memory and streams; every step of the path runs in the CUDA
kernels behind `branch_state_build`, `tree_verify_attn` and `accept_and_refresh`.
Importing this module without a built library raises: there is no CPU fallback.
"""
from __future__ import annotations

import ctypes as C
import os
from dataclasses import dataclass
from typing import List, Optional, Sequence

import torch

from . import synth

_PKG = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_PKG, "libtsv.so")

if not os.path.exists(LIB_PATH):
    raise ImportError(f"{LIB_PATH} is missing: build it with `python -m paper_2609_24698_b200.build` "
                      "(no CPU fallback exists for the tree-verify path)")
_lib = C.CDLL(LIB_PATH)

TSV_FP32, TSV_BF16 = 0, 1
FLAG_FORCE_SIMT, FLAG_HCA_DEFERRED = 1, 2
STAGE_SELECT, STAGE_ATTENTION, STAGE_ATTENTION_KERNELS = 1, 2, 4    # stages of tree_verify_attn for bench_tree_verify_attn_stages (4: without the tile plan)
ST_NODES, ST_PARENT, ST_LENGTH, ST_CSA_CAP, ST_HCA_CAP, ST_INTERNAL = 1, 2, 4, 8, 16, 32
ERR_NULL, ERR_ALIGN, ERR_SHAPE, ERR_WORKSPACE, ERR_CUDA, ERR_LIMIT = -1, -2, -3, -4, -5, -6

_p = C.c_void_p


class CShape(C.Structure):
    _fields_ = [("dtype", C.c_int32), ("B", C.c_int32), ("D", C.c_int32), ("H", C.c_int32), ("d", C.c_int32),
                ("m_csa", C.c_int32), ("topk", C.c_int32), ("HI", C.c_int32), ("di", C.c_int32),
                ("m_hca", C.c_int32), ("window", C.c_int32), ("sm_scale", C.c_float), ("max_L", C.c_int64),
                ("flags", C.c_int32), ("reserved", C.c_int32)]


CACHE_TENSORS = ("L", "csa_kv", "csa_ik", "csa_row0", "csa_cap", "hca_kv", "hca_row0", "hca_cap",
                 "win_kv", "csa_mx", "csa_s", "csa_acc_kv", "csa_acc_ik", "hca_mx", "hca_s", "hca_acc_kv")


class CCache(C.Structure):
    _fields_ = [(n, _p) for n in CACHE_TENSORS] + [("csa_rows", C.c_int64), ("hca_rows", C.c_int64),
                                                   ("page_table", _p), ("page_tokens", C.c_int32), ("max_pages", C.c_int32), ("tok_rows", C.c_int64)]


class CNodes(C.Structure):
    _fields_ = [(n, _p) for n in ("q", "kv", "c_csa", "ikc", "g_csa", "c_hca", "g_hca", "iq", "iw", "parent", "n_nodes")]


class CScratch(C.Structure):
    _fields_ = [(n, _p) for n in ("csa_mx", "csa_s", "csa_acc_kv", "csa_acc_ik", "hca_mx", "hca_s", "hca_acc_kv",
                                  "new_csa_kv", "new_csa_ik", "new_hca_kv", "csa_done", "hca_done")]


_lib.tsv_version.restype = C.c_int
_lib.tsv_kernel_launches.restype = C.c_uint64
_lib.tsv_error_string.restype = C.c_char_p
_lib.tsv_error_string.argtypes = [C.c_int]
_lib.tsv_workspace_bytes.restype = C.c_size_t
_lib.tsv_workspace_bytes.argtypes = [C.POINTER(CShape)]
_lib.branch_state_build.restype = C.c_int
_lib.branch_state_build.argtypes = [C.POINTER(CShape), C.POINTER(CCache), C.POINTER(CNodes), C.POINTER(CScratch), _p, _p]
_lib.tree_verify_attn.restype = C.c_int
_lib.tree_verify_attn.argtypes = [C.POINTER(CShape), C.POINTER(CCache), C.POINTER(CNodes), C.POINTER(CScratch),
                                  _p, _p, _p, C.c_size_t, _p, _p]
_lib.accept_and_refresh.restype = C.c_int
_lib.accept_and_refresh.argtypes = [C.POINTER(CShape), C.c_int32, C.POINTER(C.POINTER(CCache)), C.POINTER(C.POINTER(CNodes)),
                                    C.POINTER(C.POINTER(CScratch)), _p, _p, _p, _p, _p, _p, _p]


class TsvError(RuntimeError):
    def __init__(self, code: int, where: str):
        self.code = code
        super().__init__(f"{where}: {_lib.tsv_error_string(code).decode()} ({code})")


def version() -> int:
    return _lib.tsv_version()


def kernel_launches() -> int:
    """Kernels launched by the library in this process so far."""
    return int(_lib.tsv_kernel_launches())


def torch_dtype(shape: synth.Shape) -> torch.dtype:
    return torch.bfloat16 if shape.dtype == "bf16" else torch.float32


def c_shape(shape: synth.Shape, max_L: int, flags: int = 0) -> CShape:
    return CShape(TSV_BF16 if shape.dtype == "bf16" else TSV_FP32, shape.B, shape.D, shape.H, shape.d, shape.m_csa,
                  shape.topk, shape.HI, shape.di, shape.m_hca, shape.window, float(shape.sm_scale), int(max_L), flags, 0)


def _ptr(t: Optional[torch.Tensor]) -> Optional[int]:
    return None if t is None else t.data_ptr()


def _stream(stream) -> int:
    return (torch.cuda.current_stream() if stream is None else stream).cuda_stream


@dataclass
class LayerCache:
    """Persistent per-layer state (device tensors); rows of sequence b start at *_row0[b]."""
    L: torch.Tensor
    csa_kv: torch.Tensor
    csa_ik: torch.Tensor
    csa_row0: torch.Tensor
    csa_cap: torch.Tensor
    hca_kv: torch.Tensor
    hca_row0: torch.Tensor
    hca_cap: torch.Tensor
    win_kv: torch.Tensor
    csa_mx: torch.Tensor
    csa_s: torch.Tensor
    csa_acc_kv: torch.Tensor
    csa_acc_ik: torch.Tensor
    hca_mx: torch.Tensor
    hca_s: torch.Tensor
    hca_acc_kv: torch.Tensor
    page_table: Optional[torch.Tensor] = None      # [B, max_pages] int32: paged pool (csa_row0 / hca_row0 unused then)
    page_tokens: int = 0

    def struct(self) -> CCache:
        pt = self.page_table
        return CCache(*[_ptr(getattr(self, n)) for n in CACHE_TENSORS], int(self.csa_kv.shape[0]), int(self.hca_kv.shape[0]),
                      _ptr(pt), int(self.page_tokens), 0 if pt is None else int(pt.shape[1]),
                      0 if pt is None else int(self.win_kv.shape[0]))

    def clone(self) -> "LayerCache":
        return LayerCache(*[getattr(self, n).clone() for n in CACHE_TENSORS], page_table=self.page_table, page_tokens=self.page_tokens)

    def csa_row_index(self, shape: synth.Shape, b: int, n: int) -> torch.Tensor:
        """Physical rows of CSA entries 0 .. n-1 of sequence b (slab, or through the page table)."""
        return self._rows(b, n, self.csa_row0, shape.m_csa)

    def hca_row_index(self, shape: synth.Shape, b: int, n: int) -> torch.Tensor:
        return self._rows(b, n, self.hca_row0, shape.m_hca)

    def tok_row_index(self, shape: synth.Shape, b: int, positions: torch.Tensor) -> torch.Tensor:
        """Physical rows of win_kv that hold the token-level KV of the given positions of sequence b."""
        if self.page_table is None:
            return b * shape.window + positions % shape.window       # rows of win_kv viewed as [B * window, d]
        return self.page_table[b].long()[positions // self.page_tokens] * self.page_tokens + positions % self.page_tokens

    def _rows(self, b: int, n: int, row0: torch.Tensor, block: int) -> torch.Tensor:
        e = torch.arange(n, dtype=torch.long, device=self.L.device)
        if self.page_table is None:
            return int(row0[b]) + e
        per = self.page_tokens // block
        return self.page_table[b].long()[e // per] * per + e % per


@dataclass
class NodeInputs:
    q: torch.Tensor
    kv: torch.Tensor
    c_csa: torch.Tensor
    ikc: torch.Tensor
    g_csa: torch.Tensor
    c_hca: torch.Tensor
    g_hca: torch.Tensor
    iq: torch.Tensor
    iw: torch.Tensor
    parent: torch.Tensor
    n_nodes: torch.Tensor

    def struct(self) -> CNodes:
        return CNodes(*[_ptr(getattr(self, n)) for n, _ in CNodes._fields_])


@dataclass
class Scratch:
    csa_mx: torch.Tensor
    csa_s: torch.Tensor
    csa_acc_kv: torch.Tensor
    csa_acc_ik: torch.Tensor
    hca_mx: torch.Tensor
    hca_s: torch.Tensor
    hca_acc_kv: torch.Tensor
    new_csa_kv: torch.Tensor
    new_csa_ik: torch.Tensor
    new_hca_kv: torch.Tensor
    csa_done: torch.Tensor
    hca_done: torch.Tensor

    def struct(self) -> CScratch:
        return CScratch(*[_ptr(getattr(self, n)) for n, _ in CScratch._fields_])


def alloc_cache(shape: synth.Shape, csa_caps: Sequence[int], hca_caps: Sequence[int], device="cuda") -> LayerCache:
    """Empty caches (L = 0) with the given per-sequence row capacities, packed back to back."""
    dt, B = torch_dtype(shape), shape.B
    i32 = dict(dtype=torch.int32, device=device)
    f32 = dict(dtype=torch.float32, device=device)
    ccap = torch.tensor(list(csa_caps), dtype=torch.int64)
    hcap = torch.tensor(list(hca_caps), dtype=torch.int64)
    crow0 = torch.cumsum(ccap, 0) - ccap
    hrow0 = torch.cumsum(hcap, 0) - hcap
    nc, nh = max(1, int(ccap.sum())), max(1, int(hcap.sum()))
    return LayerCache(
        L=torch.zeros(B, **i32),
        csa_kv=torch.zeros(nc, shape.d, dtype=dt, device=device), csa_ik=torch.zeros(nc, shape.di, dtype=dt, device=device),
        csa_row0=crow0.to(device), csa_cap=ccap.to(torch.int32).to(device),
        hca_kv=torch.zeros(nh, shape.d, dtype=dt, device=device), hca_row0=hrow0.to(device), hca_cap=hcap.to(torch.int32).to(device),
        win_kv=torch.zeros(B, shape.window, shape.d, dtype=dt, device=device),
        csa_mx=torch.zeros(B, **f32), csa_s=torch.zeros(B, **f32),
        csa_acc_kv=torch.zeros(B, shape.d, **f32), csa_acc_ik=torch.zeros(B, shape.di, **f32),
        hca_mx=torch.zeros(B, **f32), hca_s=torch.zeros(B, **f32), hca_acc_kv=torch.zeros(B, shape.d, **f32))


def alloc_cache_paged(shape: synth.Shape, csa_caps: Sequence[int], hca_caps: Sequence[int], page_tokens: int, seed: int = 0,
                      device="cuda") -> LayerCache:
    """Empty caches over a paged pool: every sequence gets the pages its capacities ask for, drawn from one pool in a
    shuffled order (pages of different sequences interleave), and ONE page table serves the three physical layers: CSA
    entries, HCA entries and the token-level KV (win_kv becomes a pool of page_tokens rows per page)."""
    import numpy as np
    assert page_tokens % shape.m_csa == 0 and page_tokens % shape.m_hca == 0
    epp, hpp = page_tokens // shape.m_csa, page_tokens // shape.m_hca
    need = [max(-(-int(c) // epp), -(-int(h) // hpp), 1) for c, h in zip(csa_caps, hca_caps)]
    n_pages, max_pages = sum(need), max(need)
    perm = np.random.default_rng(seed).permutation(n_pages)
    table = np.full((shape.B, max_pages), -1, dtype=np.int32)
    k = 0
    for lp in range(max_pages):                       # page by page over the sequences: neighbours in a sequence are far apart
        for b in range(shape.B):
            if lp < need[b]:
                table[b, lp] = perm[k]; k += 1
    flat = alloc_cache(shape, [n_pages * epp], [n_pages * hpp], device)     # one slab per layer = the pool
    B = shape.B
    i32 = dict(dtype=torch.int32, device=device)
    f32 = dict(dtype=torch.float32, device=device)
    dt = torch_dtype(shape)
    return LayerCache(
        L=torch.zeros(B, **i32), csa_kv=flat.csa_kv, csa_ik=flat.csa_ik,
        csa_row0=torch.zeros(B, dtype=torch.int64, device=device), csa_cap=torch.tensor([n * epp for n in need], **i32),
        hca_kv=flat.hca_kv, hca_row0=torch.zeros(B, dtype=torch.int64, device=device), hca_cap=torch.tensor([n * hpp for n in need], **i32),
        win_kv=torch.zeros(n_pages * page_tokens, shape.d, dtype=dt, device=device),     # token-level pool, rows by position
        csa_mx=torch.zeros(B, **f32), csa_s=torch.zeros(B, **f32),
        csa_acc_kv=torch.zeros(B, shape.d, **f32), csa_acc_ik=torch.zeros(B, shape.di, **f32),
        hca_mx=torch.zeros(B, **f32), hca_s=torch.zeros(B, **f32), hca_acc_kv=torch.zeros(B, shape.d, **f32),
        page_table=torch.from_numpy(table).to(device), page_tokens=page_tokens)


def alloc_scratch(shape: synth.Shape, device="cuda") -> Scratch:
    dt, B, D = torch_dtype(shape), shape.B, shape.D
    f = lambda *s: torch.zeros(*s, dtype=torch.float32, device=device)
    v = lambda *s: torch.zeros(*s, dtype=dt, device=device)
    u8 = lambda *s: torch.zeros(*s, dtype=torch.uint8, device=device)
    return Scratch(f(B, D), f(B, D), f(B, D, shape.d), f(B, D, shape.di), f(B, D), f(B, D), f(B, D, shape.d),
                   v(B, D, shape.d), v(B, D, shape.di), v(B, D, shape.d), u8(B, D), u8(B, D))


def workspace_bytes(shape: synth.Shape, max_L: int, flags: int = 0) -> int:
    cs = c_shape(shape, max_L, flags)
    return int(_lib.tsv_workspace_bytes(C.byref(cs)))


def alloc_workspace(shape: synth.Shape, max_L: int, flags: int = 0, device="cuda") -> torch.Tensor:
    n = workspace_bytes(shape, max_L, flags)
    if n == 0:
        raise TsvError(ERR_SHAPE, "tsv_workspace_bytes")
    return torch.empty(n + 256, dtype=torch.uint8, device=device)


def _aligned(ws: torch.Tensor) -> (int, int):
    base = ws.data_ptr()
    a = (base + 255) & ~255
    return a, ws.numel() - (a - base)


def branch_state_build(shape: CShape, cache: LayerCache, nodes: NodeInputs, scratch: Scratch, status: torch.Tensor, stream=None) -> None:
    cs, ns, ss = cache.struct(), nodes.struct(), scratch.struct()
    r = _lib.branch_state_build(C.byref(shape), C.byref(cs), C.byref(ns), C.byref(ss), _ptr(status), _stream(stream))
    if r:
        raise TsvError(r, "branch_state_build")


def tree_verify_attn(shape: CShape, cache: LayerCache, nodes: NodeInputs, scratch: Scratch, out: torch.Tensor,
                     topk_idx: Optional[torch.Tensor], workspace: torch.Tensor, status: torch.Tensor, stream=None) -> None:
    cs, ns, ss = cache.struct(), nodes.struct(), scratch.struct()
    wp, wn = _aligned(workspace)
    r = _lib.tree_verify_attn(C.byref(shape), C.byref(cs), C.byref(ns), C.byref(ss), _ptr(out), _ptr(topk_idx), wp, wn,
                              _ptr(status), _stream(stream))
    if r:
        raise TsvError(r, "tree_verify_attn")


_lib.tsv_bench_tree_verify_attn_stages.restype = C.c_int
_lib.tsv_bench_tree_verify_attn_stages.argtypes = [C.POINTER(CShape), C.POINTER(CCache), C.POINTER(CNodes), C.POINTER(CScratch),
                                                   _p, _p, _p, C.c_size_t, _p, _p, C.c_int]


def bench_tree_verify_attn_stages(shape: CShape, cache: LayerCache, nodes: NodeInputs, scratch: Scratch, out: torch.Tensor,
                                  topk_idx: Optional[torch.Tensor], workspace: torch.Tensor, status: torch.Tensor, stages: int,
                                  stream=None) -> None:
    """Per-stage timing aid of the benchmark (an export of the library outside its public header): tree_verify_attn
    restricted to `stages` (STAGE_SELECT | STAGE_ATTENTION).  The attention stage alone reuses the selection that a
    full call on the same inputs left in `workspace`."""
    cs, ns, ss = cache.struct(), nodes.struct(), scratch.struct()
    wp, wn = _aligned(workspace)
    r = _lib.tsv_bench_tree_verify_attn_stages(C.byref(shape), C.byref(cs), C.byref(ns), C.byref(ss), _ptr(out), _ptr(topk_idx),
                                               wp, wn, _ptr(status), _stream(stream), stages)
    if r:
        raise TsvError(r, "tsv_bench_tree_verify_attn_stages")


class LayerPack:
    """Host arrays of per-layer struct pointers for accept_and_refresh, built once and reused."""

    def __init__(self, caches: List[LayerCache], nodes: List[NodeInputs], scratch: List[Scratch]):
        n = len(caches)
        self.n = n
        self._keep = ([c.struct() for c in caches], [x.struct() for x in nodes], [s.struct() for s in scratch])
        self.caches = (C.POINTER(CCache) * n)(*[C.pointer(x) for x in self._keep[0]])
        self.nodes = (C.POINTER(CNodes) * n)(*[C.pointer(x) for x in self._keep[1]])
        self.scratch = (C.POINTER(CScratch) * n)(*[C.pointer(x) for x in self._keep[2]])


def accept_and_refresh(shape: CShape, pack: LayerPack, draft_tok: torch.Tensor, target_tok: torch.Tensor,
                       accept_len: torch.Tensor, accept_path: torch.Tensor, bonus_tok: torch.Tensor,
                       status: torch.Tensor, stream=None) -> None:
    r = _lib.accept_and_refresh(C.byref(shape), pack.n, pack.caches, pack.nodes, pack.scratch, _ptr(draft_tok), _ptr(target_tok),
                                _ptr(accept_len), _ptr(accept_path), _ptr(bonus_tok), _ptr(status), _stream(stream))
    if r:
        raise TsvError(r, "accept_and_refresh")


STATIC_WORKSPACE_BYTES = 16 << 20
_lib.tree_verify_attn_static.restype = C.c_int
_lib.tree_verify_attn_static.argtypes = [C.POINTER(CShape), C.POINTER(CCache), C.POINTER(CNodes), C.POINTER(CScratch),
                                         _p, _p, _p, _p]


def tree_verify_attn_static(shape: CShape, cache: LayerCache, nodes: NodeInputs, scratch: Scratch, out: torch.Tensor,
                            topk_idx: Optional[torch.Tensor], status: torch.Tensor, stream=None) -> None:
    """tree_verify_attn for callers that cannot allocate device memory (a serving engine that owns
    the whole memory pool, a plug-in, a latency-critical loop): the workspace is an array built into
    the library, so no workspace tensor is passed and the call allocates nothing.  Shapes that need
    more than STATIC_WORKSPACE_BYTES raise TsvError(ERR_LIMIT).  Calls share that array: do not let
    two of them overlap on the GPU, and make the first call on a device outside stream capture."""
    cs, ns, ss = cache.struct(), nodes.struct(), scratch.struct()
    r = _lib.tree_verify_attn_static(C.byref(shape), C.byref(cs), C.byref(ns), C.byref(ss), _ptr(out), _ptr(topk_idx),
                                     _ptr(status), _stream(stream))
    if r:
        raise TsvError(r, "tree_verify_attn_static")
