"""CPU oracle (fp64, numpy) for tree verification over online-compressed attention.

TEST INFRASTRUCTURE ONLY.  Nothing here is part of the product: only tests/, the
smoke check and the benchmark's CPU-baseline leg may import it.  It shares no code
with the CUDA path and is deliberately plain and slow.

What the paper fixes (Sections "Branch-Aware Causal Verification and Isolation",
"Compressed-State Consistency and Accepted-Path Refresh", "Three-Stage Speculative
Forward", "Temporary Branch States and Compressed-State Handling"): tree verification
is an exact re-organisation of sequential decoding.  A node sees the accepted context
and its own ancestors only; branches compress independently after they split; nothing
speculative touches the persistent state; after acceptance, token history, KV and the
CSA/HCA compression states all describe the same prefix.  The oracle is therefore
DEFINED by the sequential single-token step `decode_step`, and the tree functions are
written to reproduce it along every root-to-node path (the tests check exactly that).

The paper does not print the layer arithmetic; the readings used here are:
  * compression = softmax-gated pooling over non-overlapping position-aligned blocks,
    one scalar gate logit per token per cache; the CSA indexer key is pooled with the
    same weights as the CSA entry;
  * indexer score of entry e for a query token: sum_h iw_h * relu(iq_h . ik_e);
    top-k by score, ties to the lower block index, k_eff = min(k, #candidates);
  * one joint softmax over selected CSA entries, all HCA entries, the window of
    uncompressed tokens (positions p-w+1 .. p, self included) -- key == value (MQA);
  * attention at position p happens BEFORE token p is folded into the compression
    state, so a block closed by token p is first visible at position p+1;
  * a closed entry is rounded once to the storage dtype and that rounded value is what
    every later reader sees; partial accumulators stay unrounded (fp32 on the GPU);
  * greedy acceptance: walk from the root, follow the lowest-index child whose draft
    token equals the target argmax at the current node.

Parity status: all functions are pinned (brute force, closed forms, library routines)
in tests/test_oracle_*.py.  Fidelity of the readings above to the real DeepSeek-V4
layer is unpinned (its report is not available to this build).
"""
from __future__ import annotations

import math
from dataclasses import dataclass, field
from typing import Dict, List, Optional, Sequence, Tuple

import numpy as np


# ----------------------------------------------------------------------------- storage rounding
def round_storage(x: np.ndarray, dtype: str) -> np.ndarray:
    """Round fp64 values to the storage dtype (RNE) and return them as fp64."""
    x = np.asarray(x, dtype=np.float64)
    f = x.astype(np.float32)
    if dtype == "fp32":
        return f.astype(np.float64)
    assert dtype == "bf16"
    bits = f.view(np.uint32).astype(np.int64)
    lsb = (bits >> 16) & 1
    bits = (bits + 0x7FFF + lsb) & ~np.int64(0xFFFF)
    return bits.astype(np.uint32).view(np.float32).astype(np.float64).reshape(x.shape)


# ----------------------------------------------------------------------------- state
@dataclass
class Partial:
    """Running state of one open compression block: max gate, sum of weights, weighted sums."""
    mx: float = 0.0
    s: float = 0.0
    acc: List[np.ndarray] = field(default_factory=list)   # [acc_kv] or [acc_kv, acc_ik]

    def copy(self) -> "Partial":
        return Partial(self.mx, self.s, [a.copy() for a in self.acc])


def empty_partial(dims: Sequence[int]) -> Partial:
    return Partial(0.0, 0.0, [np.zeros(n) for n in dims])


@dataclass
class SeqState:
    """Persistent state of one sequence in one layer (the committed prefix)."""
    L: int
    csa_kv: np.ndarray        # [n_csa, d]
    csa_ik: np.ndarray        # [n_csa, di]
    hca_kv: np.ndarray        # [n_hca, d]
    win: np.ndarray           # [w, d] ring, slot = position % w
    csa_part: Partial
    hca_part: Partial

    def copy(self) -> "SeqState":
        return SeqState(self.L, self.csa_kv.copy(), self.csa_ik.copy(), self.hca_kv.copy(),
                        self.win.copy(), self.csa_part.copy(), self.hca_part.copy())


def empty_state(sh) -> SeqState:
    return SeqState(0, np.zeros((0, sh.d)), np.zeros((0, sh.di)), np.zeros((0, sh.d)),
                    np.zeros((sh.window, sh.d)), empty_partial([sh.d, sh.di]), empty_partial([sh.d]))


# ----------------------------------------------------------------------------- compression
def fold(part: Partial, is_empty: bool, g: float, vecs: Sequence[np.ndarray]) -> Partial:
    """Add one token (gate g, vectors vecs) to an open block; emptiness is known from the
    position count, never from the stored numbers."""
    g = float(g)
    if is_empty:
        return Partial(g, 1.0, [np.asarray(v, dtype=np.float64).copy() for v in vecs])
    mx2 = max(part.mx, g)
    a = math.exp(part.mx - mx2)
    b = math.exp(g - mx2)
    return Partial(mx2, part.s * a + b, [acc * a + b * np.asarray(v, dtype=np.float64)
                                         for acc, v in zip(part.acc, vecs)])


def close(part: Partial, dtype: str) -> List[np.ndarray]:
    """Entry of a finished block: weighted mean, rounded once to the storage dtype."""
    return [round_storage(acc / part.s, dtype) for acc in part.acc]


def pool_block(g: np.ndarray, c: np.ndarray) -> np.ndarray:
    """Two-pass softmax pooling of one block: sum_i softmax_i(g_i) c_i."""
    g = np.asarray(g, dtype=np.float64)
    w = np.exp(g - g.max())
    w = w / w.sum()
    return w @ np.asarray(c, dtype=np.float64)


def recompress_from_scratch(sh, toks: Dict[str, np.ndarray]) -> SeqState:
    """Build the persistent state of a committed token list directly from the block
    definition (two-pass pooling per block, no online form).  Used for checking and for
    building the prefix caches of the tests."""
    L = int(toks["kv"].shape[0])
    m, mh, w = sh.m_csa, sh.m_hca, sh.window
    n_csa, n_hca = L // m, L // mh
    csa_kv = np.zeros((n_csa, sh.d)); csa_ik = np.zeros((n_csa, sh.di)); hca_kv = np.zeros((n_hca, sh.d))
    if n_csa:
        g = np.asarray(toks["g_csa"][:n_csa * m], dtype=np.float64).reshape(n_csa, m)
        wgt = np.exp(g - g.max(axis=1, keepdims=True)); wgt /= wgt.sum(axis=1, keepdims=True)
        csa_kv = round_storage(np.einsum("bm,bmd->bd", wgt, np.asarray(toks["c_csa"][:n_csa * m], dtype=np.float64).reshape(n_csa, m, sh.d)), sh.dtype)
        csa_ik = round_storage(np.einsum("bm,bmd->bd", wgt, np.asarray(toks["ikc"][:n_csa * m], dtype=np.float64).reshape(n_csa, m, sh.di)), sh.dtype)
    for b in range(n_hca):
        hca_kv[b] = round_storage(pool_block(toks["g_hca"][b * mh:(b + 1) * mh], toks["c_hca"][b * mh:(b + 1) * mh]), sh.dtype)

    def tail(gname, cnames, blk):
        lo = (L // blk) * blk
        dims = [toks[c].shape[1] for c in cnames]
        if lo == L:
            return empty_partial(dims)
        g = np.asarray(toks[gname][lo:L], dtype=np.float64)
        mx = float(g.max()); e = np.exp(g - mx)
        return Partial(mx, float(e.sum()), [e @ np.asarray(toks[c][lo:L], dtype=np.float64) for c in cnames])

    win = np.zeros((w, sh.d))
    for p in range(max(0, L - w), L):
        win[p % w] = toks["kv"][p]
    return SeqState(L, csa_kv, csa_ik, hca_kv, win, tail("g_csa", ["c_csa", "ikc"], m), tail("g_hca", ["c_hca"], mh))


# ----------------------------------------------------------------------------- selection / attention
def indexer_scores(iq: np.ndarray, iw: np.ndarray, ik: np.ndarray) -> np.ndarray:
    """score_e = sum_h iw_h * relu(iq_h . ik_e);  iq [HI, di], iw [HI], ik [n, di] -> [n]."""
    if ik.shape[0] == 0:
        return np.zeros(0)
    dots = np.asarray(iq, dtype=np.float64) @ np.asarray(ik, dtype=np.float64).T
    return np.asarray(iw, dtype=np.float64) @ np.maximum(dots, 0.0)


def select_topk(scores: np.ndarray, k: int) -> np.ndarray:
    """Positions of the k_eff = min(k, n) largest scores, ties to the lower position, ascending."""
    n = scores.shape[0]
    if n <= k:
        return np.arange(n, dtype=np.int64)
    order = np.lexsort((np.arange(n), -scores))     # primary: score descending; secondary: index ascending
    return np.sort(order[:k]).astype(np.int64)


def attend(q: np.ndarray, keys: np.ndarray, scale: float) -> np.ndarray:
    """o_h = sum_j softmax_j(scale * q_h . K_j) K_j   (key == value);  q [H, d], keys [N, d]."""
    logits = scale * (np.asarray(q, dtype=np.float64) @ keys.T)
    logits -= logits.max(axis=1, keepdims=True)
    p = np.exp(logits)
    p /= p.sum(axis=1, keepdims=True)
    return p @ keys


def _window_rows(S: SeqState, p: int, w: int) -> np.ndarray:
    """Uncompressed committed tokens a query at position p sees: positions max(0, p-w+1) .. L-1."""
    lo = max(0, p - w + 1)
    if lo >= S.L:
        return np.zeros((0, S.win.shape[1]))
    return S.win[[pos % w for pos in range(lo, S.L)]]


# ----------------------------------------------------------------------------- sequential semantics
def decode_step(S: SeqState, sh, tok: Dict[str, np.ndarray]):
    """One ordinary decode step at position p = S.L: attention first, then the state update.
    Returns (out [H, d], selected CSA block indices)."""
    p, m, mh, w = S.L, sh.m_csa, sh.m_hca, sh.window
    sel = select_topk(indexer_scores(tok["iq"], tok["iw"], S.csa_ik), sh.topk)
    keys = np.concatenate([S.csa_kv[sel], S.hca_kv, _window_rows(S, p, w),
                           np.asarray(tok["kv"], dtype=np.float64)[None, :]], axis=0)
    out = attend(tok["q"], keys, sh.scale)
    # update
    S.win[p % w] = tok["kv"]
    S.csa_part = fold(S.csa_part, p % m == 0, tok["g_csa"], [tok["c_csa"], tok["ikc"]])
    if (p + 1) % m == 0:
        e_kv, e_ik = close(S.csa_part, sh.dtype)
        S.csa_kv = np.concatenate([S.csa_kv, e_kv[None]], 0)
        S.csa_ik = np.concatenate([S.csa_ik, e_ik[None]], 0)
        S.csa_part = empty_partial([sh.d, sh.di])
    S.hca_part = fold(S.hca_part, p % mh == 0, tok["g_hca"], [tok["c_hca"]])
    if (p + 1) % mh == 0:
        (e,) = close(S.hca_part, sh.dtype)
        S.hca_kv = np.concatenate([S.hca_kv, e[None]], 0)
        S.hca_part = empty_partial([sh.d])
    S.L = p + 1
    return out, sel


# ----------------------------------------------------------------------------- tree functions
def tree_depth(parent: np.ndarray, n_nodes: int) -> np.ndarray:
    depth = np.zeros(n_nodes, dtype=np.int64)
    for n in range(1, n_nodes):
        depth[n] = depth[int(parent[n])] + 1
    return depth


def strict_ancestors(parent: np.ndarray, n: int) -> List[int]:
    """Root-first list of the strict ancestors of node n."""
    out = []
    a = int(parent[n])
    while a >= 0:
        out.append(a)
        a = int(parent[a])
    return out[::-1]


@dataclass
class Scratch:
    """Branch-private temporary state of one sequence in one layer (the scratch pad)."""
    csa_part: List[Partial]
    hca_part: List[Partial]
    new_csa_kv: np.ndarray    # [D, d]   valid where csa_done
    new_csa_ik: np.ndarray    # [D, di]
    new_hca_kv: np.ndarray    # [D, d]   valid where hca_done
    csa_done: np.ndarray      # [D] bool
    hca_done: np.ndarray


def branch_state_build(S: SeqState, sh, nodes: Dict[str, np.ndarray], parent: np.ndarray, n_nodes: int) -> Scratch:
    """Chain-private compression: each node folds its own token into the state inherited
    from its parent (the root inherits the persistent partial state); a node that closes
    a block emits the entry into the scratch pad and leaves an empty state behind."""
    D = parent.shape[0]
    depth = tree_depth(parent, n_nodes)
    sc = Scratch([empty_partial([sh.d, sh.di]) for _ in range(D)], [empty_partial([sh.d]) for _ in range(D)],
                 np.zeros((D, sh.d)), np.zeros((D, sh.di)), np.zeros((D, sh.d)),
                 np.zeros(D, dtype=bool), np.zeros(D, dtype=bool))
    for n in range(n_nodes):
        p = S.L + int(depth[n])
        src_c = S.csa_part if n == 0 else sc.csa_part[int(parent[n])]
        src_h = S.hca_part if n == 0 else sc.hca_part[int(parent[n])]
        st = fold(src_c, p % sh.m_csa == 0, nodes["g_csa"][n], [nodes["c_csa"][n], nodes["ikc"][n]])
        if (p + 1) % sh.m_csa == 0:
            sc.new_csa_kv[n], sc.new_csa_ik[n] = close(st, sh.dtype)
            sc.csa_done[n] = True
            st = empty_partial([sh.d, sh.di])
        sc.csa_part[n] = st
        st = fold(src_h, p % sh.m_hca == 0, nodes["g_hca"][n], [nodes["c_hca"][n]])
        if (p + 1) % sh.m_hca == 0:
            (sc.new_hca_kv[n],) = close(st, sh.dtype)
            sc.hca_done[n] = True
            st = empty_partial([sh.d])
        sc.hca_part[n] = st
    return sc


def tree_verify_attn(S: SeqState, sh, nodes: Dict[str, np.ndarray], parent: np.ndarray, n_nodes: int,
                     sc: Scratch, forced_sel: Optional[Sequence[np.ndarray]] = None):
    """Branch-aware causal attention of every tree node over the committed prefix plus its
    own ancestors.  Returns (out [D, H, d], sel: list of ascending logical CSA block
    indices per node).  Logical index >= n_csa names the entry closed inside the tree at
    the strict ancestor whose position falls in that block.  `forced_sel` replaces the
    top-k decision (used to re-evaluate with a selection that differs inside the tie band)."""
    D = parent.shape[0]
    depth = tree_depth(parent, n_nodes)
    n_csa = S.csa_kv.shape[0]
    out = np.zeros((D, sh.H, sh.d))
    sels: List[np.ndarray] = []
    for n in range(n_nodes):
        p = S.L + int(depth[n])
        anc = strict_ancestors(parent, n)
        new_c = [a for a in anc if sc.csa_done[a]]           # root-first == ascending block index
        new_h = [a for a in anc if sc.hca_done[a]]
        if forced_sel is None:
            # candidates = prefix entries 0..n_csa-1 followed by the in-tree entries of this path
            scores = np.concatenate([indexer_scores(nodes["iq"][n], nodes["iw"][n], S.csa_ik),
                                     indexer_scores(nodes["iq"][n], nodes["iw"][n], sc.new_csa_ik[new_c])])
            sel = select_topk(scores, sh.topk)
        else:
            sel = np.asarray(forced_sel[n], dtype=np.int64)
            sel = sel[sel >= 0]
        sel_kv = np.concatenate([S.csa_kv[sel[sel < n_csa]],
                                 sc.new_csa_kv[[new_c[int(i) - n_csa] for i in sel[sel >= n_csa]]]], 0)
        tree_kv = np.asarray(nodes["kv"], dtype=np.float64)[[a for a in anc if depth[n] - depth[a] <= sh.window - 1] + [n]]
        keys = np.concatenate([sel_kv, S.hca_kv, sc.new_hca_kv[new_h], _window_rows(S, p, sh.window), tree_kv], 0)
        out[n] = attend(nodes["q"][n], keys, sh.scale)
        sels.append(sel)
    return out, sels


def accept_walk(parent: np.ndarray, n_nodes: int, draft: np.ndarray, target: np.ndarray):
    """Greedy acceptance: the root is always accepted; from the current node go to the
    lowest-index child whose draft token equals the target token at the current node.
    Returns (path as list of node ids, bonus token = target at the last accepted node)."""
    cur, path = 0, [0]
    while True:
        nxt = -1
        for c in range(cur + 1, n_nodes):
            if int(parent[c]) == cur and int(draft[c]) == int(target[cur]):
                nxt = c
                break
        if nxt < 0:
            break
        path.append(nxt)
        cur = nxt
    return path, int(target[cur])


def refresh(S: SeqState, sh, nodes: Dict[str, np.ndarray], sc: Scratch, path: Sequence[int]) -> None:
    """Commit the accepted path into the persistent state and drop everything else."""
    for i, n in enumerate(path):
        pos = S.L + i
        S.win[pos % sh.window] = nodes["kv"][n]
        if sc.csa_done[n]:
            S.csa_kv = np.concatenate([S.csa_kv, sc.new_csa_kv[n][None]], 0)
            S.csa_ik = np.concatenate([S.csa_ik, sc.new_csa_ik[n][None]], 0)
        if sc.hca_done[n]:
            S.hca_kv = np.concatenate([S.hca_kv, sc.new_hca_kv[n][None]], 0)
    last = path[-1]
    S.csa_part = sc.csa_part[last].copy()
    S.hca_part = sc.hca_part[last].copy()
    S.L += len(path)


# ----------------------------------------------------------------------------- whole cycle (convenience)
def verify_cycle(states: List[List[SeqState]], sh, nodes_per_layer: List[Dict[str, np.ndarray]],
                 parent: np.ndarray, n_nodes: np.ndarray, draft: np.ndarray, target: np.ndarray,
                 want_out: bool = True):
    """One verify cycle over all layers and sequences.  states[layer][seq] are mutated.
    Returns (outs[layer][seq] or None, sels[layer][seq], paths[seq], bonus[seq])."""
    n_layers, B = len(states), len(states[0])
    outs = [[None] * B for _ in range(n_layers)]
    sels = [[None] * B for _ in range(n_layers)]
    scs = [[None] * B for _ in range(n_layers)]
    for l in range(n_layers):
        for b in range(B):
            nb = {k: v[b] for k, v in nodes_per_layer[l].items()}
            scs[l][b] = branch_state_build(states[l][b], sh, nb, parent[b], int(n_nodes[b]))
            if want_out:
                outs[l][b], sels[l][b] = tree_verify_attn(states[l][b], sh, nb, parent[b], int(n_nodes[b]), scs[l][b])
    paths, bonus = [], []
    for b in range(B):
        path, bt = accept_walk(parent[b], int(n_nodes[b]), draft[b], target[b])
        paths.append(path); bonus.append(bt)
        for l in range(n_layers):
            nb = {k: v[b] for k, v in nodes_per_layer[l].items()}
            refresh(states[l][b], sh, nb, scs[l][b], path)
    return outs, sels, paths, bonus
