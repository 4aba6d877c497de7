"""Seeded synthetic inputs for tree-verify over compressed attention.

This module only DRAWS inputs (random vectors, gate logits, trees, token ids,
prefix lengths) and quantises them to the storage dtype.  It holds none of the
method's arithmetic: no compression, no scoring, no attention, no acceptance.
Both the CPU oracle's tests and the CUDA path's tests/bench read their inputs
from here, so the two sides see identical bits.

Every draw comes from a counter-based Philox stream keyed by
(seed, config id, tensor id, layer, sequence, cycle), so any tensor can be
regenerated on demand instead of being stored.

Workload recipe (stands in for the paper's GSM8K / MBPP / ShareGPT runs, whose
shapes only are used: budgets D=5..8, batches 1..64, short math/code-like and
chat-like variable prefix lengths; Section "Setup and Metrics"):
  * q, kv, c_csa, c_hca, ikc, iq ~ N(0,1)/sqrt(dim of the vector)
  * gate logits g_csa, g_hca ~ N(0,1)
  * indexer head weights iw = |N(0,1)|/sqrt(HI)
  * draft tokens uniform in [0, vocab); siblings are made distinct
  * target token of an internal node: with probability p the draft token of one
    of its children (picked uniformly), else uniform; leaves uniform
  * random trees: node n>=1 picks its parent uniformly among earlier nodes of
    depth <= 4
"""
from __future__ import annotations

from dataclasses import dataclass, field, replace
from typing import Dict, Optional, Tuple

import numpy as np

VOCAB = 32000

# tensor ids (part of the Philox key)
_T_LEN, _T_TREE, _T_TOK, _T_P = 1, 2, 3, 4
_T_PREFIX, _T_NODES, _T_DIRECT = 10, 11, 12


@dataclass(frozen=True)
class Shape:
    """Problem shape of one attention layer (names follow the paper's C4/C128/SWA split)."""
    dtype: str            # "fp32" | "bf16": storage type of vectors and caches
    B: int                # sequences
    D: int                # tree nodes per sequence, root included (verification budget)
    H: int                # query heads (one shared KV head)
    d: int                # shared KV dim (key == value)
    m_csa: int            # CSA block (C4)
    topk: int             # CSA entries selected per node
    HI: int               # indexer heads
    di: int               # indexer dim
    m_hca: int            # HCA block (C128)
    window: int           # sliding window of uncompressed tokens
    sm_scale: float = 0.0  # 0 -> 1/sqrt(d)

    @property
    def scale(self) -> float:
        return self.sm_scale if self.sm_scale > 0 else 1.0 / float(np.sqrt(self.d))


@dataclass(frozen=True)
class Config:
    """One synthetic workload: shape + how prefixes, trees and acceptance are drawn."""
    name: str
    cfg_id: int
    shape: Shape
    layers: int = 1
    cycles: int = 1
    L_min: int = 1024
    L_max: int = 1024                 # inclusive; L ~ U[L_min, L_max]
    tree: str = "random"              # "random" | "chain" | "fixed"
    fixed_parent: Tuple[int, ...] = ()
    p_lo: float = 0.7
    p_hi: float = 0.7                 # acceptance p ~ U[p_lo, p_hi] per sequence
    seed: int = 0


def _cfgs() -> Dict[str, Config]:
    big = dict(H=64, d=512, m_csa=4, HI=4, di=128, m_hca=128, window=128)
    c = {}
    c["cfg1"] = Config("cfg1", 1, Shape("fp32", 1, 5, 16, 128, 4, 64, 1, 64, 128, 128),
                       L_min=1024, L_max=1024, tree="fixed", fixed_parent=(-1, 0, 0, 1, 1))
    c["cfg2"] = Config("cfg2", 2, Shape("bf16", 1, 8, topk=512, **big), L_min=4096, L_max=4096)
    c["cfg2_chain"] = replace(c["cfg2"], name="cfg2_chain", tree="chain")
    c["cfg3"] = Config("cfg3", 3, Shape("bf16", 16, 8, topk=512, **big), L_min=512, L_max=8192,
                       p_lo=0.5, p_hi=0.8)
    c["cfg4"] = Config("cfg4", 4, Shape("bf16", 64, 8, topk=512, **big), layers=8, cycles=50,
                       L_min=256, L_max=2048)
    c["cfg5"] = Config("cfg5", 5, Shape("bf16", 4, 8, topk=2048, **big), cycles=100,
                       L_min=131072, L_max=131072, p_lo=0.6, p_hi=0.6)
    return c


CONFIGS: Dict[str, Config] = _cfgs()


# --------------------------------------------------------------------------- streams
def stream(cfg: Config, tensor_id: int, layer: int = 0, seq: int = 0, cycle: int = 0) -> np.random.Generator:
    """Philox generator keyed by (seed, config, tensor, layer, sequence, cycle)."""
    ss = np.random.SeedSequence([cfg.seed, cfg.cfg_id, tensor_id, layer, seq, cycle])
    return np.random.Generator(np.random.Philox(key=ss.generate_state(2, dtype=np.uint64)))


def quantize(x: np.ndarray, dtype: str) -> np.ndarray:
    """Round drawn values once to the storage dtype; returned as float32 holding those values."""
    x32 = np.asarray(x, dtype=np.float32)
    if dtype == "fp32":
        return x32
    if dtype != "bf16":
        raise ValueError(dtype)
    u = x32.view(np.uint32).astype(np.uint64)
    u = (u + 0x7FFF + ((u >> 16) & 1)) & 0xFFFF0000
    return u.astype(np.uint32).view(np.float32).reshape(x32.shape)


# --------------------------------------------------------------------------- draws
def prefix_lengths(cfg: Config) -> np.ndarray:
    g = stream(cfg, _T_LEN)
    return g.integers(cfg.L_min, cfg.L_max + 1, size=cfg.shape.B).astype(np.int64)


def accept_prob(cfg: Config) -> np.ndarray:
    g = stream(cfg, _T_P)
    return g.uniform(cfg.p_lo, cfg.p_hi, size=cfg.shape.B)


def prefix_tokens(cfg: Config, layer: int, seq: int, L: int) -> Dict[str, np.ndarray]:
    """Per-token cache-side inputs of a committed prefix of L tokens (one layer, one sequence)."""
    s = cfg.shape
    g = stream(cfg, _T_PREFIX, layer, seq)
    out = {
        "kv": quantize(g.standard_normal((L, s.d), dtype=np.float32) / np.sqrt(s.d), s.dtype),
        "c_csa": quantize(g.standard_normal((L, s.d), dtype=np.float32) / np.sqrt(s.d), s.dtype),
        "ikc": quantize(g.standard_normal((L, s.di), dtype=np.float32) / np.sqrt(s.di), s.dtype),
        "c_hca": quantize(g.standard_normal((L, s.d), dtype=np.float32) / np.sqrt(s.d), s.dtype),
        "g_csa": g.standard_normal(L, dtype=np.float32),
        "g_hca": g.standard_normal(L, dtype=np.float32),
    }
    return out


def node_inputs(cfg: Config, layer: int, cycle: int) -> Dict[str, np.ndarray]:
    """Per-node inputs of one verify cycle for one layer, all sequences: arrays [B, D, ...]."""
    s = cfg.shape
    g = stream(cfg, _T_NODES, layer, 0, cycle)
    B, D = s.B, s.D
    n = lambda *sh: g.standard_normal(sh, dtype=np.float32)
    return {
        "q": quantize(n(B, D, s.H, s.d) / np.sqrt(s.d), s.dtype),
        "kv": quantize(n(B, D, s.d) / np.sqrt(s.d), s.dtype),
        "c_csa": quantize(n(B, D, s.d) / np.sqrt(s.d), s.dtype),
        "ikc": quantize(n(B, D, s.di) / np.sqrt(s.di), s.dtype),
        "g_csa": n(B, D),
        "c_hca": quantize(n(B, D, s.d) / np.sqrt(s.d), s.dtype),
        "g_hca": n(B, D),
        "iq": quantize(n(B, D, s.HI, s.di) / np.sqrt(s.di), s.dtype),
        "iw": np.abs(n(B, D, s.HI)) / np.float32(np.sqrt(s.HI)),
    }


def random_parent(g: np.random.Generator, D: int, max_parent_depth: int = 4) -> np.ndarray:
    parent = np.full(D, -1, dtype=np.int32)
    depth = np.zeros(D, dtype=np.int32)
    for n in range(1, D):
        cand = [j for j in range(n) if depth[j] <= max_parent_depth]
        parent[n] = cand[int(g.integers(0, len(cand)))]
        depth[n] = depth[parent[n]] + 1
    return parent


def trees(cfg: Config, cycle: int = 0) -> Tuple[np.ndarray, np.ndarray]:
    """parent [B, D] (root = node 0, parent -1) and n_nodes [B] for one cycle."""
    s = cfg.shape
    g = stream(cfg, _T_TREE, 0, 0, cycle)
    parent = np.zeros((s.B, s.D), dtype=np.int32)
    for b in range(s.B):
        if cfg.tree == "fixed":
            parent[b] = np.asarray(cfg.fixed_parent, dtype=np.int32)
        elif cfg.tree == "chain":
            parent[b] = np.arange(-1, s.D - 1, dtype=np.int32)
        else:
            parent[b] = random_parent(g, s.D)
    return parent, np.full(s.B, s.D, dtype=np.int32)


def tokens(cfg: Config, cycle: int, parent: np.ndarray, n_nodes: np.ndarray,
           p: Optional[np.ndarray] = None) -> Tuple[np.ndarray, np.ndarray]:
    """draft_tok, target_tok [B, D] int32 for the given trees."""
    s = cfg.shape
    g = stream(cfg, _T_TOK, 0, 0, cycle)
    p = accept_prob(cfg) if p is None else p
    draft = g.integers(0, VOCAB, size=(s.B, s.D)).astype(np.int32)
    target = g.integers(0, VOCAB, size=(s.B, s.D)).astype(np.int32)
    for b in range(s.B):
        nn = int(n_nodes[b])
        kids = [[c for c in range(1, nn) if parent[b, c] == u] for u in range(nn)]
        for u in range(nn):
            seen = set()
            for c in kids[u]:                      # siblings get distinct draft tokens
                while int(draft[b, c]) in seen:
                    draft[b, c] = (int(draft[b, c]) + 1) % VOCAB
                seen.add(int(draft[b, c]))
        for u in range(nn):
            hit = g.uniform() < p[b]
            pick = int(g.integers(0, max(1, len(kids[u]))))
            if kids[u] and hit:
                target[b, u] = draft[b, kids[u][pick]]
    return draft, target


def direct_cache(cfg: Config, layer: int, seq: int, L: int) -> Dict[str, np.ndarray]:
    """Cache CONTENTS drawn directly (no compression run), for timing only.

    Entries are drawn with the per-element spread that pooling m unit-variance/sqrt(dim)
    vectors under softmax weights of N(0,1) gates produces (about 0.65 of the token spread
    for m=4 and 0.13 for m=128); partial states are drawn as a one-token fold.  Timing does
    not depend on these values beyond which entries the indexer ranks first.
    """
    s = cfg.shape
    g = stream(cfg, _T_DIRECT, layer, seq)
    n_csa, n_hca, nw = L // s.m_csa, L // s.m_hca, min(L, s.window)
    f = lambda rows, dim, sd: quantize(g.standard_normal((rows, dim), dtype=np.float32) * np.float32(sd / np.sqrt(dim)), s.dtype)
    return {
        "csa_kv": f(n_csa, s.d, 0.65), "csa_ik": f(n_csa, s.di, 0.65),
        "hca_kv": f(n_hca, s.d, 0.13), "win_kv": f(nw, s.d, 1.0),
        "csa_acc_kv": g.standard_normal(s.d, dtype=np.float32) / np.float32(np.sqrt(s.d)),
        "csa_acc_ik": g.standard_normal(s.di, dtype=np.float32) / np.float32(np.sqrt(s.di)),
        "hca_acc_kv": g.standard_normal(s.d, dtype=np.float32) / np.float32(np.sqrt(s.d)),
        "gates": g.standard_normal(2, dtype=np.float32),
    }


def direct_arrays(cfg: Config, layer: int, b: int, L: int) -> Dict[str, np.ndarray]:
    """direct_cache laid out as a committed per-sequence state: window rows placed at their ring slots (pos % w), the
    open-block states as a one-token fold (max gate = the drawn gate, weight sum 1).  Layout only."""
    sh = cfg.shape
    dc = direct_cache(cfg, layer, b, L)
    win = np.zeros((sh.window, sh.d), dtype=np.float32)
    nw = dc["win_kv"].shape[0]
    for i, pos in enumerate(range(L - nw, L)):
        win[pos % sh.window] = dc["win_kv"][i]
    return {"csa_kv": dc["csa_kv"], "csa_ik": dc["csa_ik"], "hca_kv": dc["hca_kv"], "win": win,
            "csa_mx": float(dc["gates"][0]), "csa_s": 1.0, "csa_acc_kv": dc["csa_acc_kv"], "csa_acc_ik": dc["csa_acc_ik"],
            "hca_mx": float(dc["gates"][1]), "hca_s": 1.0, "hca_acc_kv": dc["hca_acc_kv"]}


def small_config(name: str = "tiny", dtype: str = "fp32", B: int = 2, D: int = 6, H: int = 4, d: int = 16,
                 m_csa: int = 2, topk: int = 3, HI: int = 2, di: int = 8, m_hca: int = 3, window: int = 4,
                 L_min: int = 0, L_max: int = 12, seed: int = 0, cfg_id: int = 100, layers: int = 1,
                 cycles: int = 1, tree: str = "random", sm_scale: float = 0.0, p: float = 0.7) -> Config:
    """Small configs for brute-force pins and edge-case parity tests."""
    return Config(name, cfg_id, Shape(dtype, B, D, H, d, m_csa, topk, HI, di, m_hca, window, sm_scale),
                  layers=layers, cycles=cycles, L_min=L_min, L_max=L_max, tree=tree, p_lo=p, p_hi=p, seed=seed)
