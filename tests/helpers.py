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
