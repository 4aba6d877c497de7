"""Shared test helpers: build oracle states from the seeded generators (no method arithmetic here)."""
from __future__ import annotations

import itertools
from typing import Dict, List

import numpy as np

from oracle import tsv_oracle as O
from paper_2609_24698_b200 import synth


def oracle_states(cfg: synth.Config, lengths=None) -> List[List[O.SeqState]]:
    """states[layer][seq]: prefix tokens from the generator, compressed by the oracle from scratch."""
    lengths = synth.prefix_lengths(cfg) if lengths is None else lengths
    return [[O.recompress_from_scratch(cfg.shape, synth.prefix_tokens(cfg, l, b, int(lengths[b])))
             for b in range(cfg.shape.B)] for l in range(cfg.layers)]


def per_seq(nodes: Dict[str, np.ndarray], b: int) -> Dict[str, np.ndarray]:
    return {k: v[b] for k, v in nodes.items()}


def token_of(nodes_b: Dict[str, np.ndarray], n: int) -> Dict[str, np.ndarray]:
    return {k: v[n] for k, v in nodes_b.items()}


def all_parent_arrays(D: int):
    """Every valid parent array with parent[0] = -1 and 0 <= parent[n] < n."""
    for tail in itertools.product(*[range(n) for n in range(1, D)]):
        yield np.asarray((-1,) + tail, dtype=np.int32)


def path_to(parent: np.ndarray, n: int) -> List[int]:
    out = [n]
    while parent[out[-1]] >= 0:
        out.append(int(parent[out[-1]]))
    return out[::-1]


def states_close(a: O.SeqState, b: O.SeqState, tol: float = 1e-12) -> None:
    assert a.L == b.L
    assert a.csa_kv.shape == b.csa_kv.shape and a.hca_kv.shape == b.hca_kv.shape and a.csa_ik.shape == b.csa_ik.shape
    for x, y in [(a.csa_kv, b.csa_kv), (a.csa_ik, b.csa_ik), (a.hca_kv, b.hca_kv), (a.win, b.win)]:
        if x.size:
            assert np.max(np.abs(x - y)) <= tol
    for pa, pb in [(a.csa_part, b.csa_part), (a.hca_part, b.hca_part)]:
        assert pa.mx == pb.mx
        assert abs(pa.s - pb.s) <= tol * max(1.0, abs(pb.s))
        for x, y in zip(pa.acc, pb.acc):
            assert np.max(np.abs(x - y)) <= tol * max(1.0, np.max(np.abs(y)))


# ----------------------------------------------------------------------------- oracle <-> device plumbing
def state_arrays(S: O.SeqState) -> Dict[str, np.ndarray]:
    """Oracle state -> plain arrays in the layout harness.fill_cache uploads."""
    return {"csa_kv": S.csa_kv, "csa_ik": S.csa_ik, "hca_kv": S.hca_kv, "win": S.win,
            "csa_mx": S.csa_part.mx, "csa_s": S.csa_part.s, "csa_acc_kv": S.csa_part.acc[0], "csa_acc_ik": S.csa_part.acc[1],
            "hca_mx": S.hca_part.mx, "hca_s": S.hca_part.s, "hca_acc_kv": S.hca_part.acc[0]}


def rel_err(got: np.ndarray, ref: np.ndarray) -> float:
    """max |got - ref| relative to the reference tensor's max magnitude."""
    ref = np.asarray(ref, dtype=np.float64)
    got = np.asarray(got, dtype=np.float64)
    if ref.size == 0:
        return 0.0
    return float(np.max(np.abs(got - ref)) / max(np.max(np.abs(ref)), 1e-30))


def check_topk(shape, S: O.SeqState, nodes_b, parent_b, n: int, sc: O.Scratch, got_idx: np.ndarray, ref_sel: np.ndarray,
               band: float = 1e-4) -> bool:
    """True if the device's selection is the oracle's; otherwise asserts that the two differ only by
    candidates whose score lies within `band` (relative) of the oracle's k-th score, and returns False."""
    got = got_idx[got_idx >= 0]
    assert np.all(np.diff(got) > 0), "selection must be ascending and duplicate-free"
    assert np.all(got_idx[len(got):] == -1)
    assert len(got) == len(ref_sel)
    if np.array_equal(got, ref_sel):
        return True
    n_csa = S.csa_kv.shape[0]
    anc = O.strict_ancestors(parent_b, n)
    new_c = [a for a in anc if sc.csa_done[a]]
    scores = np.concatenate([O.indexer_scores(nodes_b["iq"][n], nodes_b["iw"][n], S.csa_ik),
                             O.indexer_scores(nodes_b["iq"][n], nodes_b["iw"][n], sc.new_csa_ik[new_c])])
    tau = np.sort(scores)[::-1][len(ref_sel) - 1]
    for i in set(got.tolist()) ^ set(ref_sel.tolist()):
        assert abs(scores[i] - tau) <= band * abs(tau) + 1e-30, f"top-k differs outside the tie band at candidate {i}"
    return False
