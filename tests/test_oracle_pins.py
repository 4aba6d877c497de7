"""Pins for the CPU oracle: brute force, closed forms, library routines, invariants.

None of these compares the oracle with a retyped copy of itself: the references are
sequential decoding (the definition), hand-derived values (tests/golden), library
softmax / scaled-dot-product attention, plain sorting and exhaustive enumeration.
"""
import json
import math
import os

import numpy as np
import pytest
import scipy.special
import torch

from oracle import tsv_oracle as O
from paper_2609_24698_b200 import synth
from tests.helpers import all_parent_arrays, oracle_states, path_to, per_seq, states_close, token_of

GOLD = json.load(open(os.path.join(os.path.dirname(__file__), "golden", "hand_worked.json")))


def tiny(**kw):
    return synth.small_config(**kw)


# ------------------------------------------------------------------ golden, hand-derived
def test_golden_pool():
    g = GOLD["pool_two_tokens"]
    assert np.allclose(O.pool_block(np.array(g["gates"]), np.array(g["c"])), g["entry"], atol=1e-15)
    # the online form reaches the same entry
    p = O.fold(O.empty_partial([2]), True, g["gates"][0], [np.array(g["c"][0])])
    p = O.fold(p, False, g["gates"][1], [np.array(g["c"][1])])
    assert np.allclose(p.acc[0] / p.s, g["entry"], atol=1e-15)


def test_golden_attend():
    g = GOLD["attend_two_keys"]
    assert np.allclose(O.attend(np.array(g["q"]), np.array(g["keys"]), g["scale"]), g["out"], atol=1e-15)


def test_golden_indexer():
    g = GOLD["indexer_relu"]
    s = O.indexer_scores(np.array(g["iq"]), np.array(g["iw"]), np.array(g["ik"]))
    assert np.allclose(s, g["scores"], atol=1e-15)
    assert list(O.select_topk(s, 1)) == [0]          # exact tie -> lower index


def test_golden_in_tree_entry():
    g = GOLD["in_tree_entry_visible_to_descendants"]
    sh = synth.Shape(**g["shape"])
    S = O.recompress_from_scratch(sh, {k: np.array(v, dtype=np.float64) for k, v in g["prefix"].items()})
    nodes = {k: np.array(v, dtype=np.float64) for k, v in g["nodes"].items()}
    parent = np.array(g["parent"], dtype=np.int32)
    sc = O.branch_state_build(S, sh, nodes, parent, 3)
    e = g["expect"]
    assert list(sc.csa_done) == e["csa_done"]
    assert np.allclose(sc.new_csa_kv[0], e["new_csa_kv_root"], atol=1e-7)      # fp32 storage rounding
    assert np.allclose(sc.new_csa_ik[0], e["new_csa_ik_root"], atol=1e-7)
    out, sel = O.tree_verify_attn(S, sh, nodes, parent, 3, sc)
    assert [list(map(int, s)) for s in sel] == e["sel"]
    assert np.allclose(out, np.array(e["out"]), atol=1e-7)


# ------------------------------------------------------------------ compression closed forms
def test_pool_equal_gates_is_mean_and_shift_invariant():
    rng = np.random.default_rng(1)
    c = rng.standard_normal((5, 7))
    assert np.allclose(O.pool_block(np.full(5, 0.3), c), c.mean(axis=0), atol=1e-14)
    g = rng.standard_normal(5)
    assert np.allclose(O.pool_block(g, c), O.pool_block(g + 11.5, c), atol=1e-13)
    g2 = g.copy(); g2[3] = 80.0
    assert np.allclose(O.pool_block(g2, c), c[3], atol=1e-12)


def test_online_fold_matches_library_softmax():
    rng = np.random.default_rng(2)
    for m in (1, 2, 4, 9):
        g = rng.standard_normal(m) * 3
        c = rng.standard_normal((m, 6)); k = rng.standard_normal((m, 3))
        p = O.empty_partial([6, 3])
        for i in range(m):
            p = O.fold(p, i == 0, g[i], [c[i], k[i]])
        w = scipy.special.softmax(g)
        assert p.mx == g.max()
        assert np.allclose(p.acc[0] / p.s, w @ c, atol=1e-13)
        assert np.allclose(p.acc[1] / p.s, w @ k, atol=1e-13)


def test_fold_ignores_garbage_when_empty():
    junk = O.Partial(float("nan"), float("inf"), [np.full(3, np.nan)])
    p = O.fold(junk, True, 0.25, [np.arange(3.0)])
    assert p.mx == 0.25 and p.s == 1.0 and np.array_equal(p.acc[0], np.arange(3.0))


def test_round_storage_bf16():
    x = np.array([1.0, 1.0 + 2 ** -8, 1.0 + 2 ** -7, 1.0 + 3 * 2 ** -8, -0.1, 3.3895313892515355e38])
    r = O.round_storage(x, "bf16")
    # ties to even: 1+2^-8 -> 1 ; 1+3*2^-8 -> 1+2^-6
    assert r[0] == 1.0 and r[1] == 1.0 and r[2] == 1.0 + 2 ** -7 and r[3] == 1.0 + 2 ** -6
    assert np.array_equal(r, torch.tensor(x, dtype=torch.float64).to(torch.float32).to(torch.bfloat16).to(torch.float64).numpy())
    y = np.random.default_rng(0).standard_normal(1000)
    assert np.array_equal(O.round_storage(y, "bf16"),
                          torch.tensor(y).to(torch.float32).to(torch.bfloat16).to(torch.float64).numpy())
    assert np.array_equal(O.round_storage(y, "fp32"), y.astype(np.float32).astype(np.float64))


# ------------------------------------------------------------------ top-k
def test_topk_against_plain_sort():
    rng = np.random.default_rng(3)
    for n in (0, 1, 5, 17):
        for k in (1, 3, 17, 40):
            s = np.round(rng.standard_normal(n), 1)          # coarse values -> many exact ties
            want = sorted(sorted(range(n), key=lambda i: (-s[i], i))[:min(k, n)])
            assert list(O.select_topk(s, k)) == want


# ------------------------------------------------------------------ sequential semantics == tree (brute force)
def _seq_state_by_decoding(cfg, layer, b, L):
    """Prefix state obtained by running decode_step token by token from an empty state."""
    sh = cfg.shape
    toks = synth.prefix_tokens(cfg, layer, b, L)
    rng = np.random.default_rng(1234 + L)
    S = O.empty_state(sh)
    for p in range(L):
        t = {k: v[p] for k, v in toks.items()}
        t.update(q=rng.standard_normal((sh.H, sh.d)), iq=rng.standard_normal((sh.HI, sh.di)), iw=np.abs(rng.standard_normal(sh.HI)))
        O.decode_step(S, sh, t)
    return S, toks


@pytest.mark.parametrize("dtype", ["fp32", "bf16"])
def test_online_prefix_equals_recompression(dtype):
    cfg = tiny(dtype=dtype)
    for L in range(0, 14):
        S, toks = _seq_state_by_decoding(cfg, 0, 0, L)
        states_close(S, O.recompress_from_scratch(cfg.shape, toks))


@pytest.mark.parametrize("L", list(range(0, 13)))
def test_every_node_equals_sequential_decode_along_its_path(L):
    """All tree shapes with D=5 (24 of them) on small blocks so that CSA and HCA blocks
    close inside the tree and the window slides over the tree."""
    cfg = tiny(B=1, D=5, m_csa=2, m_hca=3, window=3, topk=2, L_min=L, L_max=L, sm_scale=1.5)
    sh = cfg.shape
    S0 = O.recompress_from_scratch(sh, synth.prefix_tokens(cfg, 0, 0, L))
    nodes = per_seq(synth.node_inputs(cfg, 0, L), 0)
    for parent in all_parent_arrays(sh.D):
        sc = O.branch_state_build(S0, sh, nodes, parent, sh.D)
        out, sel = O.tree_verify_attn(S0, sh, nodes, parent, sh.D, sc)
        for n in range(sh.D):
            S = S0.copy()
            for j in path_to(parent, n):
                o, s_ = O.decode_step(S, sh, token_of(nodes, j))
            assert np.max(np.abs(o - out[n])) <= 1e-12
            assert list(s_) == list(sel[n])
            # the node's branch-private state equals the sequential state after its path
            assert S.csa_part.mx == sc.csa_part[n].mx and abs(S.csa_part.s - sc.csa_part[n].s) <= 1e-12
            assert np.max(np.abs(S.csa_part.acc[0] - sc.csa_part[n].acc[0])) <= 1e-12
            assert np.max(np.abs(S.hca_part.acc[0] - sc.hca_part[n].acc[0])) <= 1e-12


def test_deeper_trees_and_partial_node_counts():
    cfg = tiny(B=3, D=6, m_csa=2, m_hca=3, window=4, topk=3, L_min=0, L_max=12, seed=5)
    sh = cfg.shape
    lengths = synth.prefix_lengths(cfg)
    states = oracle_states(cfg, lengths)[0]
    rng = np.random.default_rng(0)
    for cyc in range(6):
        nodes = synth.node_inputs(cfg, 0, cyc)
        parent, _ = synth.trees(cfg, cyc)
        for b in range(sh.B):
            nn = int(rng.integers(1, sh.D + 1))
            nb = per_seq(nodes, b)
            sc = O.branch_state_build(states[b], sh, nb, parent[b], nn)
            out, sel = O.tree_verify_attn(states[b], sh, nb, parent[b], nn, sc)
            for n in range(nn):
                S = states[b].copy()
                for j in path_to(parent[b], n):
                    o, s_ = O.decode_step(S, sh, token_of(nb, j))
                assert np.max(np.abs(o - out[n])) <= 1e-12 and list(s_) == list(sel[n])
            assert not out[nn:].any()


def test_single_chain_is_linear_verification_and_refresh_is_recompression():
    """A chain tree = D ordinary decode steps; after committing the accepted path the state
    equals recompressing the committed token list from scratch, cycle after cycle."""
    cfg = tiny(B=2, D=5, m_csa=2, m_hca=3, window=4, topk=3, L_min=0, L_max=7, tree="chain", cycles=8, seed=9)
    sh = cfg.shape
    lengths = synth.prefix_lengths(cfg)
    states = oracle_states(cfg, lengths)
    committed = [dict(synth.prefix_tokens(cfg, 0, b, int(lengths[b]))) for b in range(sh.B)]
    for cyc in range(cfg.cycles):
        nodes = synth.node_inputs(cfg, 0, cyc)
        parent, n_nodes = synth.trees(cfg, cyc)
        draft, target = synth.tokens(cfg, cyc, parent, n_nodes)
        for b in range(sh.B):                                    # chain == sequential
            nb = per_seq(nodes, b)
            sc = O.branch_state_build(states[0][b], sh, nb, parent[b], sh.D)
            out, _ = O.tree_verify_attn(states[0][b], sh, nb, parent[b], sh.D, sc)
            S = states[0][b].copy()
            for n in range(sh.D):
                o, _s = O.decode_step(S, sh, token_of(nb, n))
                assert np.max(np.abs(o - out[n])) <= 1e-12
        _, _, paths, _ = O.verify_cycle(states, sh, [nodes], parent, n_nodes, draft, target)
        for b in range(sh.B):
            for k in committed[b]:
                committed[b][k] = np.concatenate([committed[b][k], nodes[k][b][paths[b]]], 0)
            states_close(states[0][b], O.recompress_from_scratch(sh, committed[b]))
            assert states[0][b].L == committed[b]["kv"].shape[0]


@pytest.mark.parametrize("dtype", ["fp32", "bf16"])
def test_refresh_equals_recompression_random_trees(dtype):
    cfg = tiny(dtype=dtype, B=3, D=6, m_csa=2, m_hca=3, window=4, topk=2, L_min=0, L_max=9, cycles=10, seed=11, layers=2)
    sh = cfg.shape
    lengths = synth.prefix_lengths(cfg)
    states = oracle_states(cfg, lengths)
    committed = [[dict(synth.prefix_tokens(cfg, l, b, int(lengths[b]))) for b in range(sh.B)] for l in range(cfg.layers)]
    tot = 0
    for cyc in range(cfg.cycles):
        nodes = [synth.node_inputs(cfg, l, cyc) for l in range(cfg.layers)]
        parent, n_nodes = synth.trees(cfg, cyc)
        draft, target = synth.tokens(cfg, cyc, parent, n_nodes)
        before = [[s.L for s in row] for row in states]
        _, _, paths, _ = O.verify_cycle(states, sh, nodes, parent, n_nodes, draft, target, want_out=False)
        for l in range(cfg.layers):
            for b in range(sh.B):
                for k in committed[l][b]:
                    committed[l][b][k] = np.concatenate([committed[l][b][k], nodes[l][k][b][paths[b]]], 0)
                S = states[l][b]
                states_close(S, O.recompress_from_scratch(sh, committed[l][b]), tol=1e-12 if dtype == "fp32" else 1e-12)
                # consistency of token history, caches and open-block counts with the same prefix
                assert S.L == before[l][b] + len(paths[b])
                assert S.csa_kv.shape[0] == S.L // sh.m_csa and S.hca_kv.shape[0] == S.L // sh.m_hca
        tot += sum(len(p) for p in paths)
    assert tot > cfg.cycles * sh.B          # some drafts were accepted


# ------------------------------------------------------------------ reductions to library attention
def _sdpa(q, keys, mask, scale):
    """torch's scaled_dot_product_attention in fp64 on CPU; q [M, d], keys [N, d], mask [M, N] bool."""
    qt = torch.tensor(q, dtype=torch.float64)[None]
    kt = torch.tensor(keys, dtype=torch.float64)[None]
    o = torch.nn.functional.scaled_dot_product_attention(qt, kt, kt, attn_mask=torch.tensor(mask)[None], scale=scale)
    return o[0].numpy()


def test_short_prefix_reduces_to_tree_masked_dense_attention():
    """L < m, L < m' and w >= L + D: nothing is compressed, the window covers everything, so
    the result is ordinary softmax attention with a tree mask over [prefix tokens ; nodes]."""
    cfg = tiny(B=1, D=6, H=3, d=8, m_csa=64, m_hca=64, window=32, L_min=9, L_max=9, sm_scale=0.7)
    sh = cfg.shape
    toks = synth.prefix_tokens(cfg, 0, 0, 9)
    S = O.recompress_from_scratch(sh, toks)
    nodes = per_seq(synth.node_inputs(cfg, 0, 0), 0)
    for parent in list(all_parent_arrays(sh.D))[::7]:
        sc = O.branch_state_build(S, sh, nodes, parent, sh.D)
        out, _ = O.tree_verify_attn(S, sh, nodes, parent, sh.D, sc)
        keys = np.concatenate([toks["kv"], nodes["kv"]], 0).astype(np.float64)
        for n in range(sh.D):
            mask = np.zeros((sh.H, 9 + sh.D), dtype=bool)
            mask[:, :9] = True
            mask[:, [9 + j for j in path_to(parent, n)]] = True
            assert np.max(np.abs(out[n] - _sdpa(nodes["q"][n], keys, mask, sh.scale))) <= 1e-12


def test_large_k_reduces_to_dense_attention_over_all_entries():
    cfg = tiny(B=1, D=1, H=2, d=8, m_csa=2, m_hca=4, window=3, topk=1000, L_min=21, L_max=21)
    sh = cfg.shape
    toks = synth.prefix_tokens(cfg, 0, 0, 21)
    S = O.recompress_from_scratch(sh, toks)
    nodes = per_seq(synth.node_inputs(cfg, 0, 0), 0)
    sc = O.branch_state_build(S, sh, nodes, np.array([-1], dtype=np.int32), 1)
    out, sel = O.tree_verify_attn(S, sh, nodes, np.array([-1], dtype=np.int32), 1, sc)
    assert list(sel[0]) == list(range(10))
    # entries from library softmax pooling; window = positions 19, 20 (w=3, self included)
    ck = np.stack([scipy.special.softmax(toks["g_csa"][2 * i:2 * i + 2].astype(np.float64)) @ toks["c_csa"][2 * i:2 * i + 2].astype(np.float64) for i in range(10)])
    hk = np.stack([scipy.special.softmax(toks["g_hca"][4 * i:4 * i + 4].astype(np.float64)) @ toks["c_hca"][4 * i:4 * i + 4].astype(np.float64) for i in range(5)])
    keys = np.concatenate([O.round_storage(ck, "fp32"), O.round_storage(hk, "fp32"), toks["kv"][19:21], nodes["kv"][:1]], 0)
    ref = _sdpa(nodes["q"][0], keys, np.ones((sh.H, keys.shape[0]), dtype=bool), sh.scale)
    assert np.max(np.abs(out[0] - ref)) <= 1e-12


# ------------------------------------------------------------------ invariants from the paper
def _snapshot(S):
    return (S.L, S.csa_kv.tobytes(), S.csa_ik.tobytes(), S.hca_kv.tobytes(), S.win.tobytes(),
            S.csa_part.mx, S.csa_part.s, tuple(a.tobytes() for a in S.csa_part.acc),
            S.hca_part.mx, S.hca_part.s, tuple(a.tobytes() for a in S.hca_part.acc))


def test_isolation_non_ancestors_do_not_matter_and_persistent_state_is_untouched():
    cfg = tiny(B=1, D=6, m_csa=2, m_hca=3, window=4, topk=2, L_min=7, L_max=7)
    sh = cfg.shape
    S = oracle_states(cfg)[0][0]
    snap = _snapshot(S)
    nodes = per_seq(synth.node_inputs(cfg, 0, 0), 0)
    parent = np.array([-1, 0, 0, 1, 2, 1], dtype=np.int32)
    sc = O.branch_state_build(S, sh, nodes, parent, sh.D)
    out, sel = O.tree_verify_attn(S, sh, nodes, parent, sh.D, sc)
    assert _snapshot(S) == snap                                  # nothing speculative reaches the cache
    rng = np.random.default_rng(0)
    for n in range(sh.D):
        keep = set(path_to(parent, n))
        pert = {k: v.copy() for k, v in nodes.items()}
        for j in range(sh.D):
            if j not in keep:
                for k in pert:
                    pert[k][j] = rng.standard_normal(pert[k][j].shape)
        sc2 = O.branch_state_build(S, sh, pert, parent, sh.D)
        out2, sel2 = O.tree_verify_attn(S, sh, pert, parent, sh.D, sc2)
        assert np.array_equal(out2[n], out[n]) and list(sel2[n]) == list(sel[n])
        assert np.array_equal(sc2.csa_part[n].acc[0], sc.csa_part[n].acc[0]) and sc2.hca_part[n].s == sc.hca_part[n].s


def test_relabelling_nodes_permutes_outputs():
    cfg = tiny(B=1, D=5, m_csa=2, m_hca=3, window=4, topk=2, L_min=5, L_max=5)
    sh = cfg.shape
    S = oracle_states(cfg)[0][0]
    nodes = per_seq(synth.node_inputs(cfg, 0, 0), 0)
    parent = np.array([-1, 0, 0, 1, 2], dtype=np.int32)
    perm = [0, 2, 1, 4, 3]                       # new label -> old label, parents still first
    inv = {old: new for new, old in enumerate(perm)}
    parent2 = np.array([-1] + [inv[int(parent[perm[n]])] for n in range(1, 5)], dtype=np.int32)
    nodes2 = {k: v[perm] for k, v in nodes.items()}
    out, _ = O.tree_verify_attn(S, sh, nodes, parent, 5, O.branch_state_build(S, sh, nodes, parent, 5))
    out2, _ = O.tree_verify_attn(S, sh, nodes2, parent2, 5, O.branch_state_build(S, sh, nodes2, parent2, 5))
    assert np.max(np.abs(out2 - out[perm])) <= 1e-13


# ------------------------------------------------------------------ acceptance
def _accepted_set_brute_force(parent, nn, draft, target):
    """A node is accepted iff it is the root, or its parent is accepted, its draft token equals the
    parent's target token, and no lower-index sibling does."""
    acc = [False] * nn
    acc[0] = True
    for n in range(1, nn):
        p = int(parent[n])
        first = min([c for c in range(1, nn) if parent[c] == p and draft[c] == target[p]], default=-1)
        acc[n] = acc[p] and first == n
    return [n for n in range(nn) if acc[n]]


def test_accept_walk_special_cases_and_brute_force():
    chain = np.arange(-1, 7, dtype=np.int32)
    t = np.arange(100, 108, dtype=np.int32)
    d_all = np.concatenate([[7], t[:-1]]).astype(np.int32)
    assert O.accept_walk(chain, 8, d_all, t) == (list(range(8)), 107)
    assert O.accept_walk(chain, 8, d_all + 1, t) == ([0], 100)
    assert O.accept_walk(chain, 3, d_all, t) == ([0, 1, 2], 102)         # padding nodes are never visited
    # two matching siblings -> lowest index
    par = np.array([-1, 0, 0, 1, 2], dtype=np.int32)
    assert O.accept_walk(par, 5, np.array([0, 9, 9, 5, 5], dtype=np.int32), np.array([9, 5, 5, 1, 1], dtype=np.int32))[0] == [0, 1, 3]
    cfg = tiny(B=8, D=6, seed=3)
    for cyc in range(20):
        parent, n_nodes = synth.trees(cfg, cyc)
        draft, target = synth.tokens(cfg, cyc, parent, n_nodes)
        for b in range(cfg.shape.B):
            path, bonus = O.accept_walk(parent[b], 6, draft[b], target[b])
            assert path == _accepted_set_brute_force(parent[b], 6, draft[b], target[b])
            assert bonus == target[b][path[-1]]


def test_chain_accept_length_statistics():
    """Independent per-step acceptance p on a chain of D: E[len] = (1 - p^D) / (1 - p)."""
    cfg = tiny(B=64, D=8, tree="chain", p=0.7, seed=1)
    tot, cnt = 0, 0
    for cyc in range(40):
        parent, n_nodes = synth.trees(cfg, cyc)
        draft, target = synth.tokens(cfg, cyc, parent, n_nodes)
        for b in range(64):
            tot += len(O.accept_walk(parent[b], 8, draft[b], target[b])[0]); cnt += 1
    want = (1 - 0.7 ** 8) / (1 - 0.7)
    assert abs(tot / cnt - want) < 0.15
