"""GPU parity: the CUDA path through the C-ABI against the fp64 oracle, element by element,
on identical seeded inputs.  Tolerances (stated by the benchmark spec): attention outputs and
compressed states within max|err| <= 2e-2 (bf16 storage) / 1e-5 (fp32 storage) of each tensor's
max magnitude; accepted paths, committed lengths and cache indices bit-exact; CSA top-k sets
bit-exact except for candidates within 1e-4 (relative) of the k-th score.
"""
import numpy as np
import pytest
import torch

from oracle import tsv_oracle as O
from paper_2609_24698_b200 import synth
from tests.helpers import check_topk, oracle_states, per_seq, rel_err, state_arrays, states_close

pytestmark = pytest.mark.gpu

TOL = {"fp32": 1e-5, "bf16": 2e-2}
TOL_STATE = 2e-5          # fp32 accumulators on both storage dtypes


def _np(t):
    return t.detach().to(torch.float32).cpu().numpy().astype(np.float64)


def lockstep(cfg, cycles, flags=0, lengths=None, n_nodes_fn=None, out_pairs=None, check_recompress=False,
             parent_fn=None, return_engine=False, plant=None, graph=False, recompress_pairs=None, on_cycle=None,
             per_row=False, incremental_caches=False, page_tokens=0, exact_topk=False, want_topk=True):
    """Advance oracle and device cycle by cycle from the same prefix; compare everything each cycle.
    out_pairs: None = compare attention outputs of every (layer, seq); else callable cycle -> iterable of pairs.
    plant: callable(states, lengths) editing the oracle's prefix states in place before they are uploaded.
    graph: the device cycle is ONE CUDA graph captured over a fixed input slot and replayed every cycle (the way the
           benchmark runs it); the inputs of a cycle are copied into the slot before the replay.
    check_recompress: True = every cycle, "final" = after the last cycle; recompress_pairs: callable cycle -> pairs
           checked against recompression from scratch (None = all pairs).
    on_cycle: callable(cycle, engine, states) for extra bookkeeping.
    incremental_caches: per cycle compare only the cache rows appended in that cycle (plus lengths, window, open-block
           states); all rows are compared after the last cycle and every tenth cycle.
    page_tokens: the persistent caches live in a paged pool with pages of that many tokens (shuffled page tables).
    exact_topk: the device's selection must BE the oracle's (for inputs whose scores tie exactly, where the tie band of the
           usual check would accept a wrong tie-break).
    want_topk: False = the call gets no buffer for the index lists (the way the benchmark calls it: selection kernels may
           then skip work nobody reads); the outputs are compared with the oracle's own selection.
    per_row: also require every (node, head) output row to be within the tolerance of ITS OWN max magnitude (for inputs
           where a few rows are far larger than the rest, so that the tensor-wide bound would say little about the others)."""
    from paper_2609_24698_b200 import binding as tsv, harness as hz
    sh = cfg.shape
    lengths = synth.prefix_lengths(cfg) if lengths is None else np.asarray(lengths)
    states = oracle_states(cfg, lengths)
    if plant is not None:
        plant(states, lengths)
    committed = None
    if check_recompress:
        committed = [[{k: [v] for k, v in synth.prefix_tokens(cfg, l, b, int(lengths[b])).items()} for b in range(sh.B)]
                     for l in range(cfg.layers)]                 # per tensor: list of pieces, joined when checked
    ccap, hcap = hz.capacities(sh, lengths, cycles * sh.D)
    max_L = int(lengths.max()) + (cycles + 1) * sh.D
    eng = hz.VerifyEngine(sh, cfg.layers, ccap, hcap, max_L, flags=flags, want_topk=want_topk, page_tokens=page_tokens)
    for l in range(cfg.layers):
        for b in range(sh.B):
            hz.fill_cache(eng.caches[l], sh, b, int(lengths[b]), state_arrays(states[l][b]))
    tol = TOL[sh.dtype]
    worst = 0.0
    n_deferred, n_timely = [0], [0]
    slot = graph_obj = None
    for cyc in range(cycles):
        nodes = [synth.node_inputs(cfg, l, cyc) for l in range(cfg.layers)]
        parent, n_nodes = synth.trees(cfg, cyc)
        if parent_fn is not None:
            parent = parent_fn(cyc, parent)
        if n_nodes_fn is not None:
            n_nodes = n_nodes_fn(cyc, n_nodes)
        draft, target = synth.tokens(cfg, cyc, parent, n_nodes)
        inp = hz.InputSet.from_numpy(sh, nodes, parent, n_nodes, draft, target)
        if graph:
            if slot is None:
                slot = hz.InputSet.empty(sh, cfg.layers)
                for d_, s_ in zip(slot.tensors(), inp.tensors()):
                    d_.copy_(s_)
                snap = eng.snapshot()
                eng.launch_cycle(slot)                     # eager warm-up on the same inputs, then back to the prefix
                torch.cuda.synchronize()
                eng.restore(snap)
                graph_obj = eng.capture(slot)
            for d_, s_ in zip(slot.tensors(), inp.tensors()):
                d_.copy_(s_)
            graph_obj.replay()
            torch.cuda.synchronize()
        else:
            before = eng.snapshot()
            eng.launch_cycle(inp, refresh=False)
            torch.cuda.synchronize()
            # isolation: the first two calls leave every persistent byte unchanged
            for c0, c1 in zip(before, eng.caches):
                for name in tsv.CACHE_TENSORS:
                    assert torch.equal(getattr(c0, name), getattr(c1, name)), f"{name} changed before acceptance"
            tsv.accept_and_refresh(eng.cshape, eng._pack(inp), inp.draft, inp.target, eng.accept_len, eng.accept_path,
                                   eng.bonus, eng.status)
            torch.cuda.synchronize()
        assert int(eng.status.abs().sum()) == 0, f"cycle {cyc}: status flags {eng.status.cpu().tolist()}"
        prev_L = [[S.L for S in states[l]] for l in range(cfg.layers)]
        pairs = [(l, b) for l in range(cfg.layers) for b in range(sh.B)] if out_pairs is None else list(out_pairs(cyc))
        g_alen, g_path, g_bonus = eng.accept_len.cpu().numpy(), eng.accept_path.cpu().numpy(), eng.bonus.cpu().numpy()
        scs = {}
        for l in range(cfg.layers):
            s_ = eng.scratch[l]
            g = {k: _np(getattr(s_, k)) for k in ("csa_mx", "csa_s", "csa_acc_kv", "csa_acc_ik", "hca_mx", "hca_s", "hca_acc_kv",
                                                  "new_csa_kv", "new_csa_ik", "new_hca_kv")}
            g_cd, g_hd = s_.csa_done.cpu().numpy(), s_.hca_done.cpu().numpy()
            for b in range(sh.B):
                nb, nn = per_seq(nodes[l], b), int(n_nodes[b])
                sc = scs[(l, b)] = O.branch_state_build(states[l][b], sh, nb, parent[b], nn)
                assert np.array_equal(g_cd[b].astype(bool), sc.csa_done) and np.array_equal(g_hd[b].astype(bool), sc.hca_done)
                assert np.array_equal(g["csa_mx"][b], [p.mx for p in sc.csa_part])
                assert rel_err(g["csa_s"][b], [p.s for p in sc.csa_part]) <= TOL_STATE
                assert rel_err(g["csa_acc_kv"][b], np.stack([p.acc[0] for p in sc.csa_part])) <= TOL_STATE
                assert rel_err(g["csa_acc_ik"][b], np.stack([p.acc[1] for p in sc.csa_part])) <= TOL_STATE
                assert rel_err(g["new_csa_kv"][b], sc.new_csa_kv) <= tol and rel_err(g["new_csa_ik"][b], sc.new_csa_ik) <= tol
                # C128-deferred schedule: no HCA branch states exist for a sequence in which no HCA block can close inside
                # the tree (the committed state is compared after the refresh, like every cycle)
                if (flags & tsv.FLAG_HCA_DEFERRED) and (states[l][b].L % sh.m_hca) + sh.D < sh.m_hca:
                    n_deferred[0] += 1
                    continue
                n_timely[0] += 1
                assert np.array_equal(g["hca_mx"][b], [p.mx for p in sc.hca_part])
                assert rel_err(g["hca_s"][b], [p.s for p in sc.hca_part]) <= TOL_STATE
                assert rel_err(g["hca_acc_kv"][b], np.stack([p.acc[0] for p in sc.hca_part])) <= TOL_STATE
                assert rel_err(g["new_hca_kv"][b], sc.new_hca_kv) <= tol
        for (l, b) in pairs:
            nb, nn = per_seq(nodes[l], b), int(n_nodes[b])
            ref_out, ref_sel = O.tree_verify_attn(states[l][b], sh, nb, parent[b], nn, scs[(l, b)])
            same = True
            if want_topk:
                g_idx = eng.topk_idx[l][b].cpu().numpy()
                same = all([check_topk(sh, states[l][b], nb, parent[b], n, scs[(l, b)], g_idx[n], ref_sel[n]) for n in range(nn)])
                assert np.all(g_idx[nn:] == -1)
                assert same or not exact_topk, f"cycle {cyc} layer {l} seq {b}: selection differs from the oracle's"
            if not same:       # inside the tie band: evaluate the oracle with the device's selection
                ref_out, _ = O.tree_verify_attn(states[l][b], sh, nb, parent[b], nn, scs[(l, b)], forced_sel=[g_idx[n] for n in range(nn)])
            e = rel_err(_np(eng.out[l][b]), ref_out)
            if per_row:
                g_out = _np(eng.out[l][b])
                for n in range(nn):
                    for h in range(sh.H):
                        er = rel_err(g_out[n, h], ref_out[n, h])
                        assert er <= tol, f"cycle {cyc} layer {l} seq {b} node {n} head {h}: row error {er:.3e} > {tol}"
            worst = max(worst, e)
            assert e <= tol, f"cycle {cyc} layer {l} seq {b}: attention output error {e:.3e} > {tol}"
            assert not _np(eng.out[l][b])[nn:].any()
        # acceptance + refresh
        for b in range(sh.B):
            path, bonus = O.accept_walk(parent[b], int(n_nodes[b]), draft[b], target[b])
            assert int(g_alen[b]) == len(path) and list(g_path[b][:len(path)]) == path and np.all(g_path[b][len(path):] == -1)
            assert int(g_bonus[b]) == bonus
            for l in range(cfg.layers):
                O.refresh(states[l][b], sh, per_seq(nodes[l], b), scs[(l, b)], path)
                if committed is not None:
                    for k in committed[l][b]:
                        committed[l][b][k].append(nodes[l][k][b][path])
        rp = None if recompress_pairs is None else set(recompress_pairs(cyc))
        full = not incremental_caches or cyc == cycles - 1 or cyc % 10 == 9
        compare_caches(eng, states, sh, tol, committed if (check_recompress is True or cyc == cycles - 1) else None,
                       None if cyc == cycles - 1 else rp, None if full else prev_L)
        if on_cycle is not None:
            on_cycle(cyc, eng, states)
    if flags & tsv.FLAG_HCA_DEFERRED:
        assert n_deferred[0] > 0 and n_timely[0] > 0, "the run is meant to take both HCA refresh schedules"
    return (worst, eng, states) if return_engine else worst


def compare_caches(eng, states, sh, tol, committed=None, recompress_pairs=None, prev_L=None):
    """Device caches against the oracle states.  prev_L[l][b] (committed lengths before this cycle): compare only the
    entries appended since then (full-size runs; a later full comparison covers the untouched rows)."""
    for l, cache in enumerate(eng.caches):
        Ls = cache.L.cpu().numpy()
        r0c, r0h = cache.csa_row0.cpu().numpy(), cache.hca_row0.cpu().numpy()
        win = _np(cache.win_kv)
        f = {k: _np(getattr(cache, k)) for k in ("csa_mx", "csa_s", "csa_acc_kv", "csa_acc_ik", "hca_mx", "hca_s", "hca_acc_kv")}
        lo_c = [0 if prev_L is None else prev_L[l][b] // sh.m_csa for b in range(sh.B)]
        lo_h = [0 if prev_L is None else prev_L[l][b] // sh.m_hca for b in range(sh.B)]
        if cache.page_table is not None:                                        # paged pool: physical rows through the page table
            tab = cache.page_table.cpu().numpy().astype(np.int64)
            epp, hpp = cache.page_tokens // sh.m_csa, cache.page_tokens // sh.m_hca
            phys_c = lambda b, i: int(tab[b, i // epp]) * epp + i % epp
            phys_h = lambda b, i: int(tab[b, i // hpp]) * hpp + i % hpp
        else:
            phys_c = lambda b, i: int(r0c[b]) + i
            phys_h = lambda b, i: int(r0h[b]) + i
        if prev_L is None:
            ckv, cik, hkv = _np(cache.csa_kv), _np(cache.csa_ik), _np(cache.hca_kv)
            row_c, row_h = phys_c, phys_h
        else:                                                                     # gather only the appended rows
            ic = [phys_c(b, i) for b, S in enumerate(states[l]) for i in range(lo_c[b], S.L // sh.m_csa)]
            ih = [phys_h(b, i) for b, S in enumerate(states[l]) for i in range(lo_h[b], S.L // sh.m_hca)]
            tc_ = torch.tensor(ic, dtype=torch.long, device=cache.csa_kv.device)
            th_ = torch.tensor(ih, dtype=torch.long, device=cache.csa_kv.device)
            ckv, cik, hkv = _np(cache.csa_kv[tc_]), _np(cache.csa_ik[tc_]), _np(cache.hca_kv[th_])
            pc_, ph_ = {r: j for j, r in enumerate(ic)}, {r: j for j, r in enumerate(ih)}
            row_c = lambda b, i: pc_[phys_c(b, i)]
            row_h = lambda b, i: ph_[phys_h(b, i)]
        for b, S in enumerate(states[l]):
            assert int(Ls[b]) == S.L                                            # committed length: exact
            n_csa, n_hca = S.L // sh.m_csa, S.L // sh.m_hca
            assert S.csa_kv.shape[0] == n_csa and S.hca_kv.shape[0] == n_hca      # entry indices: exact
            rc = [row_c(b, i) for i in range(lo_c[b], n_csa)]
            rh = [row_h(b, i) for i in range(lo_h[b], n_hca)]
            assert rel_err(ckv[rc], S.csa_kv[lo_c[b]:]) <= tol and rel_err(cik[rc], S.csa_ik[lo_c[b]:]) <= tol
            assert rel_err(hkv[rh], S.hca_kv[lo_h[b]:]) <= tol
            if cache.page_table is None:
                assert np.array_equal(win[b], S.win)                             # token-level KV: copies, exact
            else:                                                                # token pool: the window's positions, by page
                for pos in range(max(0, S.L - sh.window), S.L):
                    r = int(tab[b, pos // cache.page_tokens]) * cache.page_tokens + pos % cache.page_tokens
                    assert np.array_equal(win[r], S.win[pos % sh.window])
            assert f["csa_mx"][b] == S.csa_part.mx and f["hca_mx"][b] == S.hca_part.mx
            assert abs(f["csa_s"][b] - S.csa_part.s) <= TOL_STATE * max(1.0, S.csa_part.s)
            assert abs(f["hca_s"][b] - S.hca_part.s) <= TOL_STATE * max(1.0, S.hca_part.s)
            assert rel_err(f["csa_acc_kv"][b], S.csa_part.acc[0]) <= TOL_STATE or not S.csa_part.acc[0].any()
            assert rel_err(f["csa_acc_ik"][b], S.csa_part.acc[1]) <= TOL_STATE or not S.csa_part.acc[1].any()
            assert rel_err(f["hca_acc_kv"][b], S.hca_part.acc[0]) <= TOL_STATE or not S.hca_part.acc[0].any()
            if committed is not None and (recompress_pairs is None or (l, b) in recompress_pairs):   # oracle state == recompression from scratch
                states_close(S, O.recompress_from_scratch(sh, {k: np.concatenate(v, 0) for k, v in committed[l][b].items()}), tol=1e-9)


# ------------------------------------------------------------------------------------------------ small shapes, every edge
@pytest.mark.parametrize("dtype", ["fp32", "bf16"])
def test_tiny_blocks_close_inside_tree(dtype):
    """m=2, m'=3, w=8 (>= D): CSA and HCA blocks close inside the tree on every cycle; ragged L from 0."""
    cfg = synth.small_config(dtype=dtype, B=5, D=8, H=4, d=16, m_csa=2, topk=3, HI=2, di=8, m_hca=3, window=8,
                             L_min=0, L_max=14, layers=2, seed=21, sm_scale=1.0)
    lockstep(cfg, cycles=6, check_recompress=True)


def test_tiny_partial_node_counts_and_chains():
    cfg = synth.small_config(dtype="fp32", B=6, D=7, H=3, d=24, m_csa=3, topk=2, HI=1, di=16, m_hca=5, window=9,
                             L_min=0, L_max=20, layers=1, seed=22, sm_scale=2.0)
    rng = np.random.default_rng(5)
    lockstep(cfg, cycles=5, n_nodes_fn=lambda c, nn: rng.integers(1, 8, size=nn.shape).astype(np.int32), check_recompress=True)
    chain = synth.small_config(dtype="fp32", B=3, D=8, H=2, d=8, m_csa=2, topk=4, HI=2, di=8, m_hca=4, window=8,
                               L_min=1, L_max=9, tree="chain", seed=23, p=0.9)
    lockstep(chain, cycles=6, check_recompress=True)


@pytest.mark.parametrize("dtype,scale", [("fp32", 0.0), ("fp32", 6.0), ("bf16", 0.0), ("bf16", 6.0)])
def test_medium_multi_split_and_peaked_softmax(dtype, scale):
    """Enough keys for several key tiles and splits with a ragged tail; peaked softmax (scale 6 on
    unit-ish logits) makes a single wrongly masked key visible above the tolerance."""
    cfg = synth.small_config(dtype=dtype, B=3, D=8, H=20, d=64, m_csa=4, topk=48, HI=4, di=32, m_hca=16, window=40,
                             L_min=130, L_max=700, layers=1, seed=31, sm_scale=scale)
    lockstep(cfg, cycles=3)


# ------------------------------------------------------------------------------------------------ the named configs
def test_cfg1_fp32_and_block_closing_variants():
    cfg = synth.CONFIGS["cfg1"]
    w = lockstep(cfg, cycles=3)
    assert w <= 1e-5
    # the config as written never closes a block inside the tree: shift L so CSA (m=4) and HCA (m'=128) do
    for L in (1023, 1022, 1021, 1149, 1150, 1151):
        lockstep(cfg, cycles=2, lengths=[L])


@pytest.mark.parametrize("name", ["cfg2", "cfg2_chain"])
def test_cfg2_bf16(name):
    lockstep(synth.CONFIGS[name], cycles=2)
    lockstep(synth.CONFIGS[name], cycles=1, lengths=[4096 + 125])


def test_cfg2_tree_and_chain_share_prefix_and_root():
    """Tree and chain of 8 on identical prefix caches: the root sees the same context, so its output matches bit for bit."""
    from paper_2609_24698_b200 import harness as hz
    outs = []
    for name in ("cfg2", "cfg2_chain"):
        cfg = synth.CONFIGS[name]
        _, eng, _ = lockstep(cfg, cycles=1, return_engine=True)
        outs.append(eng.out[0][0, 0].clone())
    assert torch.equal(outs[0], outs[1])


def test_cfg3_ragged_batch16():
    lockstep(synth.CONFIGS["cfg3"], cycles=2)


def test_cfg3_peaked():
    from dataclasses import replace
    cfg = synth.CONFIGS["cfg3"]
    cfg = replace(cfg, shape=replace(cfg.shape, B=4, sm_scale=1.5), cfg_id=33, L_min=600, L_max=3000)
    lockstep(cfg, cycles=2)


def test_cfg4_full_size_stack_50_cycles():
    """8 layers x 64 sequences, the launch configuration the benchmark times, 50 verify cycles back to back.  Every
    cycle: branch states and closed entries, acceptance, committed lengths, appended cache rows, window and open-block
    states of ALL 512 (layer, sequence) pairs; the refreshed state of a rotating sample of 48 pairs (all pairs after
    the last cycle) against recompression of the committed tokens from scratch; attention outputs of all pairs on the
    first and the last cycle (by then several sequences have more than top-k candidates and rank) and of a rotating
    sample of 16 pairs plus the longest sequence in between."""
    cfg = synth.CONFIGS["cfg4"]
    sh = cfg.shape
    rng = np.random.default_rng(4)
    longest = int(np.argmax(synth.prefix_lengths(cfg)))
    everyone = [(l, b) for l in range(cfg.layers) for b in range(sh.B)]
    def pairs(cyc):
        if cyc in (0, cfg.cycles - 1):
            return everyone
        return [(int(rng.integers(0, cfg.layers)), int(rng.integers(0, sh.B))) for _ in range(16)] + [(cyc % cfg.layers, longest)]
    def rpairs(cyc):
        return [(int(rng.integers(0, cfg.layers)), int(rng.integers(0, sh.B))) for _ in range(48)]
    ranked = []
    def watch(cyc, eng, states):
        ranked.append(sum(S.L // sh.m_csa > sh.topk for S in states[0]))
    lockstep(cfg, cycles=cfg.cycles, out_pairs=pairs, check_recompress=True, recompress_pairs=rpairs, incremental_caches=True,
             on_cycle=watch)
    assert cfg.cycles == 50 and ranked[-1] >= 2, "the run is meant to end with sequences past top-k candidates"


def test_cfg4_as_the_benchmark_launches_it():
    """The benchmark workload in the benchmark's launch configuration: every cycle one replay of a CUDA graph captured
    over a fixed input slot, no buffer for the index lists.  20 cycles, so that the run ends with sequences whose nodes
    rank; branch states, acceptance and appended cache rows every cycle, attention outputs for all pairs on the first
    cycle and for a seeded sample plus the longest sequence afterwards.  (Four of the workload's eight layers, to bound
    the oracle's time: the layers are independent.)"""
    from dataclasses import replace
    cfg = replace(synth.CONFIGS["cfg4"], layers=4)
    sh = cfg.shape
    rng = np.random.default_rng(44)
    longest = int(np.argmax(synth.prefix_lengths(cfg)))
    everyone = [(l, b) for l in range(cfg.layers) for b in range(sh.B)]
    cycles = 20
    def pairs(cyc):
        if cyc == 0:
            return everyone
        if cyc == cycles - 1:                            # every layer of the longest (ranking) sequence and a sample of the others
            return [(l, longest) for l in range(cfg.layers)] + [(int(rng.integers(0, cfg.layers)), int(rng.integers(0, sh.B))) for _ in range(48)]
        return [(int(rng.integers(0, cfg.layers)), int(rng.integers(0, sh.B))) for _ in range(12)] + [(cyc % cfg.layers, longest)]
    ranked = []
    def watch(cyc, eng, states):
        ranked.append(sum(S.L // sh.m_csa > sh.topk for S in states[0]))
    lockstep(cfg, cycles=cycles, out_pairs=pairs, incremental_caches=True, on_cycle=watch, graph=True, want_topk=False)
    assert ranked[-1] >= 1, "the run is meant to end with a sequence past top-k candidates"


def test_cfg5_long_context_100_cycles():
    """131072-token prefixes, top-k 2048 of 32768 candidates, 100 verify-accept-refresh cycles: branch states,
    acceptance and caches every cycle; attention outputs and selections on cycles 0, 1, 2, then every 16th and the
    last; recompression from scratch after the last cycle.  The bytes the method must read per cycle are tracked
    from the evolving lengths and selections (they may only grow with the prefix)."""
    cfg = synth.CONFIGS["cfg5"]
    sh = cfg.shape
    everyone = [(0, b) for b in range(sh.B)]
    track = []
    def watch(cyc, eng, states):
        es = 2
        per_cycle = 0
        idx = eng.topk_idx[0].cpu().numpy()
        for b, S in enumerate(states[0]):
            union = np.unique(idx[b][idx[b] >= 0]).size
            n_csa_before = (S.L - int(eng.accept_len[b])) // sh.m_csa
            per_cycle += (n_csa_before * sh.di + (union + S.hca_kv.shape[0] + sh.window + sh.D) * sh.d) * es
        track.append(per_cycle)
    lockstep(cfg, cycles=cfg.cycles, out_pairs=lambda c: everyone if (c < 3 or c % 16 == 0 or c == cfg.cycles - 1) else [],
             check_recompress="final", incremental_caches=True, on_cycle=watch)
    assert cfg.cycles == 100 and len(track) == 100
    # indexer keys of all 32768+ entries and the union of the nodes' selections dominate: tens of MB, slowly growing
    assert 40e6 < track[0] < 120e6 and track[-1] >= track[0] - 8e6


@pytest.mark.parametrize("D,B", [(5, 1), (6, 2), (7, 64), (8, 4)])
def test_budget_and_batch_sweep(D, B):
    """The paper's budgets D=5..8 and batch sizes from 1 to 64 on the benchmark's head shape, short prefixes."""
    cfg = synth.Config(f"sweep_d{D}_b{B}", 60 + D, synth.Shape("bf16", B, D, 64, 512, 4, 512, 4, 128, 128, 128),
                       L_min=100, L_max=420, seed=D)
    lockstep(cfg, cycles=2)


@pytest.mark.parametrize("dtype", ["fp32", "bf16"])
def test_long_candidate_lists_generic_scoring(dtype):
    """More than 2048 candidates per node with indexer rows that are not 256 bytes wide: the thread-per-entry scoring
    kernel and both key paths of the per-node selection (up to 2304 candidates: keys in registers; beyond: re-read)."""
    cfg = synth.small_config(name="long_lists", dtype=dtype, B=3, D=6, H=4, d=16, m_csa=2, topk=24, HI=2, di=8, m_hca=32,
                             window=16, L_min=4200, L_max=5200, layers=1, seed=77, cfg_id=72)
    lockstep(cfg, cycles=2)


@pytest.mark.parametrize("D,HI", [(4, 8), (6, 2), (7, 1), (8, 4)])
def test_long_candidate_lists_tensor_core_scoring(D, HI):
    """More than 2048 candidates per node with 128-wide bf16 indexer rows: the scores of all nodes and heads come from
    the tcgen05 scoring kernel (every head count it is built for; ragged last tiles, sequences on both sides of the
    2304-candidate switch of the selection's key paths)."""
    cfg = synth.small_config(name=f"long_lists_tc_d{D}_hi{HI}", dtype="bf16", B=3, D=D, H=4, d=16, m_csa=2, topk=24, HI=HI,
                             di=128, m_hca=32, window=16, L_min=4200, L_max=5200, layers=1, seed=78 + HI, cfg_id=73)
    lockstep(cfg, cycles=2)


def _plant_tied_indexer_keys(every=60):
    """`plant` hook: every committed CSA entry gets the indexer key of entry 0, except each `every`-th one, so that the
    k-th largest score is shared by nearly all candidates and the selection is decided by the tie rule (lower index)."""
    def hook(states, lengths):
        for layer in states:
            for S in layer:
                keep = np.arange(S.csa_ik.shape[0]) % every == every - 1
                S.csa_ik[~keep] = S.csa_ik[0]
    return hook


@pytest.mark.parametrize("dtype,di", [("fp32", 8), ("bf16", 128)])
def test_long_candidate_lists_exact_ties_across_the_cluster(dtype, di):
    """Long lists are selected by a cluster of CTAs per node, each holding a share of the candidates: with nearly all
    scores equal, the threshold's ties span every CTA of the cluster and the lowest indices must win."""
    cfg = synth.small_config(name="long_ties", dtype=dtype, B=3, D=6, H=4, d=16, m_csa=2, topk=100, HI=2, di=di, m_hca=32,
                             window=16, L_min=4700, L_max=5600, layers=1, seed=91, cfg_id=74)
    lockstep(cfg, cycles=2, plant=_plant_tied_indexer_keys(), exact_topk=True)


@pytest.mark.parametrize("HI,topk,L_min,L_max", [(1, 40, 300, 1500), (2, 100, 900, 2400), (3, 7, 0, 60), (4, 3, 0, 24)])
def test_selection_inside_one_cta_head_counts_and_tiny_lists(HI, topk, L_min, L_max):
    """The one-CTA selection kernel for 128-wide bf16 indexer rows (scores by warp-level tensor-core products, keys in
    registers) with every head count it takes, on the CUDA-core attention path (no extra CTA column); the tiny cases have
    nodes that rank with no committed entry at all (only blocks closed inside the tree) and lists of a few candidates."""
    cfg = synth.small_config(name=f"fused_sel_hi{HI}", dtype="bf16", B=4, D=6, H=4, d=16, m_csa=2, topk=topk, HI=HI, di=128,
                             m_hca=32, window=16, L_min=L_min, L_max=L_max, layers=1, seed=93 + HI, cfg_id=77)
    lockstep(cfg, cycles=3)


def test_selection_inside_one_cta_exact_ties():
    """Nearly all candidates share one score: the threshold's ties are decided by index in the one-CTA selection kernel
    (keys strided over the threads, ordered write by warp shares)."""
    cfg = synth.small_config(name="fused_ties", dtype="bf16", B=3, D=6, H=4, d=16, m_csa=2, topk=100, HI=2, di=128, m_hca=32,
                             window=16, L_min=700, L_max=2600, layers=1, seed=97, cfg_id=78)
    lockstep(cfg, cycles=2, plant=_plant_tied_indexer_keys(every=40), exact_topk=True)


def test_candidate_lists_beyond_the_cluster_capacity():
    """More than 65536 candidates per node: the single-CTA selection that re-reads the score array pass after pass."""
    cfg = synth.small_config(name="huge_lists", dtype="bf16", B=1, D=4, H=4, d=16, m_csa=2, topk=40, HI=2, di=128, m_hca=64,
                             window=16, L_min=131500, L_max=131500, layers=1, seed=92, cfg_id=75)
    lockstep(cfg, cycles=1)


def test_tensor_core_shape_without_row_counts_takes_the_cuda_core_path(monkeypatch):
    """A cache handed over without the row counts of its arrays (csa_rows = 0) gives the library nothing to build tensor
    maps from: a shape of the tensor-core path then runs on the CUDA-core path, through the same workspace."""
    from paper_2609_24698_b200 import binding as tsv
    orig = tsv.LayerCache.struct

    def no_rows(self):
        st = orig(self)
        st.csa_rows = 0
        st.hca_rows = 0
        return st
    cfg = synth.Config("tc_no_rows", 76, synth.Shape("bf16", 3, 8, 64, 512, 4, 64, 4, 128, 128, 128), L_min=150, L_max=700, seed=12)
    _, forced, _ = lockstep(cfg, cycles=1, flags=tsv.FLAG_FORCE_SIMT, return_engine=True)
    monkeypatch.setattr(tsv.LayerCache, "struct", no_rows)
    _, eng, _ = lockstep(cfg, cycles=1, return_engine=True)
    for a, b in zip(eng.out, forced.out):                # bit for bit what the CUDA-core path gives when asked for by flag
        assert torch.equal(a, b)


def test_ranked_short_candidate_lists_bf16():
    """Benchmark head shape with a small top-k: every node ranks its candidates, the lists are short enough to be scored
    inside the selection kernel (256-byte indexer rows), and the committed runs lie on both sides of 2 x topk, so ranked
    tiles take the contiguous-run path with per-node masks as well as the gathered path."""
    cfg = synth.Config("ranked_short", 71, synth.Shape("bf16", 6, 8, 64, 512, 4, 128, 4, 128, 128, 128),
                       L_min=300, L_max=1400, seed=9)
    lockstep(cfg, cycles=2)



# ------------------------------------------------------------------------------------------------ tensor-core path, peaked softmax
BENCH_HEADS = dict(H=64, d=512, m_csa=4, HI=4, di=128, m_hca=128, window=128)


def _plant_peaks(cfg, gap_nats=14.0):
    """Returns a `plant` hook: into late window rows of every sequence it writes c * q/|q| of chosen (node, head) queries of
    cycle 0, c such that this key's logit lies `gap_nats` above the (near-zero) logits of all other keys.  The window run
    comes after the CSA run in a tile's key list, so these keys fall into the second or third 256-key piece of a chunk
    (or into a later chunk): the row's running maximum jumps by more than the kernel's rescale threshold there.
      position L-1    <- query of (node 3, head 5): visible to every node
      position L-126  <- query of (deepest node, head 7): visible to depths <= 1 only, i.e. MASKED for the row it matches
      position L-125  <- query of (root, head 9): visible to depths <= 2"""
    sh = cfg.shape
    def hook(states, lengths):
        parent, n_nodes = synth.trees(cfg, 0)
        for l in range(cfg.layers):
            nodes = synth.node_inputs(cfg, l, 0)
            for b, S in enumerate(states[l]):
                depth = O.tree_depth(parent[b], int(n_nodes[b]))
                deep = int(np.argmax(depth))
                assert depth[deep] >= 2
                for pos, (n, h) in ((S.L - 1, (3, 5)), (S.L - 126, (deep, 7)), (S.L - 125, (0, 9))):
                    q = nodes["q"][b, n, h].astype(np.float64)
                    c = gap_nats / (sh.scale * np.linalg.norm(q))
                    S.win[pos % sh.window] = synth.quantize(c * q / np.linalg.norm(q), sh.dtype).astype(np.float64)
    return hook


def test_tc_planted_peaks_reach_rescale_and_merge_paths():
    """Benchmark head shape.  Sequence lengths put the planted window keys into: the second piece of a single-chunk
    tile (1200), the third piece (2040), a later chunk of a multi-chunk tile on the contiguous-run path (3500:
    n_csa <= 2 topk), and a gathered tile (5000: n_csa > 2 topk)."""
    cfg = synth.Config("tc_peaks", 81, synth.Shape("bf16", 5, 8, topk=512, **BENCH_HEADS), L_min=1, L_max=1, seed=3)
    lockstep(cfg, cycles=1, lengths=[1200, 2040, 1660, 3500, 5000], plant=_plant_peaks(cfg), per_row=True)


def test_tc_planted_peaks_ranked_tiles():
    """Same planted keys with a small top-k, so that every node ranks: masked-run tiles (n_csa <= 2 topk) and
    gathered tiles, single- and multi-chunk."""
    cfg = synth.Config("tc_peaks_ranked", 82, synth.Shape("bf16", 4, 8, topk=256, **BENCH_HEADS), L_min=1, L_max=1, seed=4)
    lockstep(cfg, cycles=1, lengths=[1500, 2040, 2600, 4400], plant=_plant_peaks(cfg, gap_nats=16.0), per_row=True)


def test_tc_without_index_lists_ranked_and_unranked_sequences():
    """The call as the benchmark makes it: no buffer for the index lists.  Selection CTAs of nodes that cannot rank then
    leave after one load, tiles without ranking nodes are planned without waiting for the selection, tiles with ranking
    nodes finish their key masks after it.  Lengths: far below the ranking threshold (top-k 256 of L / 4 entries), just
    below it so that only deep nodes rank (entries closed inside the tree count as candidates) and the sequence crosses
    it while the cycles run, above it, and above twice the top-k (gathered tiles); sm_scale 8 makes a wrongly masked key
    visible."""
    cfg = synth.Config("tc_no_lists", 84, synth.Shape("bf16", 7, 8, topk=256, sm_scale=8.0, **BENCH_HEADS), L_min=1, L_max=1, seed=6)
    lockstep(cfg, cycles=4, lengths=[200, 900, 1003, 1015, 1023, 1500, 2300], want_topk=False, per_row=True)


@pytest.mark.parametrize("B", [200, 1030])
def test_tc_more_tiles_than_the_plan_ranks(B):
    """Many plan tiles.  1030 sequences x 2 tiles = more than 2048: the plan kernel then leaves the tile records in their
    natural order instead of ranking the tiles by key count.  200 sequences = 400 tiles: ranked, with more tiles than a plan
    CTA has threads (every thread sums over several tiles).  Short prefixes; branch states, acceptance and caches are
    compared for every sequence, the attention output for a sample (the first, the last, and some in between)."""
    cfg = synth.Config("tc_many_tiles", 85, synth.Shape("bf16", B, 8, topk=512, sm_scale=8.0, **BENCH_HEADS), L_min=40, L_max=200, seed=7)
    sample = [(0, b) for b in [0, B - 1] + list(range(97, B - 1, 103))]
    lockstep(cfg, cycles=1, out_pairs=lambda c: sample)


def test_tc_peaked_scale100():
    """sm_scale = 100 on the d = 512 path: logits are O(+-5) everywhere, so one wrongly masked or dropped key moves an
    output row by far more than the tolerance.  Lengths cover single-chunk, multi-chunk and gathered tiles."""
    cfg = synth.Config("tc_scale100", 83, synth.Shape("bf16", 6, 8, topk=512, sm_scale=100.0, **BENCH_HEADS), L_min=1, L_max=1, seed=5)
    lockstep(cfg, cycles=2, lengths=[300, 900, 1400, 2047, 3300, 4700], per_row=True)


@pytest.mark.parametrize("H,D,B", [(32, 16, 3), (128, 8, 3), (64, 12, 3), (64, 16, 2), (32, 5, 2)])
def test_tc_other_head_counts_and_budgets(H, D, B):
    """The tensor-core path takes H in {32, 64, 128} and budgets up to 32 nodes: 8, 4 or 2 nodes per 256-row tile, up to
    four tiles per sequence, partial last tiles; blocks closing inside the deeper trees."""
    sh = synth.Shape("bf16", B, D, H, 512, 4, 512, 4, 128, 128, 128, sm_scale=8.0)
    cfg = synth.Config(f"tc_h{H}_d{D}", 84, sh, L_min=250, L_max=2300, seed=H + D)
    lockstep(cfg, cycles=2, per_row=True)


@pytest.mark.parametrize("dtype", ["fp32", "bf16"])
def test_budgets_beyond_eight_cuda_core_path(dtype):
    """D = 12 and D = 16 on the CUDA-core path (d = 64): deeper trees close several CSA and HCA blocks inside the tree."""
    for D in (12, 16):
        cfg = synth.small_config(name=f"simt_d{D}", dtype=dtype, B=3, D=D, H=6, d=64, m_csa=2, topk=12, HI=2, di=16, m_hca=5,
                                 window=20, L_min=30, L_max=200, layers=1, seed=90 + D, cfg_id=85, sm_scale=3.0)
        lockstep(cfg, cycles=3, check_recompress=True)






def test_refresh_skips_copies_nobody_reads():
    """The refresh moves only what a later reader can see: when the last accepted node closes a CSA (HCA) block, the open
    block is empty afterwards and its stored accumulator is never read, so it is not copied (the persistent accumulator
    keeps its old bits); rejected branches are never copied at all.  Parity with the oracle holds through such cycles."""
    cfg = synth.small_config(name="refresh_skip", dtype="bf16", B=8, D=8, H=4, d=32, m_csa=2, topk=8, HI=2, di=16, m_hca=4, window=10,
                             L_min=0, L_max=40, layers=1, seed=95, cfg_id=95, p=0.8)
    seen = {"csa": 0, "hca": 0}
    prev = {}
    def watch(cyc, eng, states):
        c = eng.caches[0]
        L = c.L.cpu().numpy()
        for b in range(cfg.shape.B):
            if cyc in prev:
                if L[b] % cfg.shape.m_csa == 0 and L[b] != prev[cyc]["L"][b]:
                    assert torch.equal(c.csa_acc_kv[b], prev[cyc]["csa"][b]); seen["csa"] += 1
                if L[b] % cfg.shape.m_hca == 0 and L[b] != prev[cyc]["L"][b]:
                    assert torch.equal(c.hca_acc_kv[b], prev[cyc]["hca"][b]); seen["hca"] += 1
        prev[cyc + 1] = {"L": L.copy(), "csa": c.csa_acc_kv.clone(), "hca": c.hca_acc_kv.clone()}
    lockstep(cfg, cycles=10, check_recompress=True, on_cycle=watch)
    assert seen["csa"] > 5 and seen["hca"] > 2


# ------------------------------------------------------------------------------------------------ paged pool
@pytest.mark.parametrize("dtype", ["fp32", "bf16"])
def test_paged_pool_small(dtype):
    """Caches in a paged pool (pages of 12 tokens = 6 CSA entries = 4 HCA entries, one shuffled page table for both
    physical layers, pages of different sequences interleaved), CUDA-core path: ranked selections, blocks closing in the
    tree, entries appended across page boundaries by the refresh; recompression check every cycle."""
    cfg = synth.small_config(name="paged", dtype=dtype, B=5, D=7, H=4, d=32, m_csa=2, topk=8, HI=2, di=16, m_hca=3, window=9,
                             L_min=0, L_max=80, layers=2, seed=93, cfg_id=93, sm_scale=2.0)
    lockstep(cfg, cycles=8, check_recompress=True, page_tokens=12)


@pytest.mark.parametrize("page_tokens,m_csa,topk,lengths", [(128, 4, 512, [300, 1100, 2040, 2500, 3900]), (128, 4, 128, [600, 900, 1500, 2600]),
                                                            (256, 4, 512, [700, 1300, 2040]), (128, 16, 64, [900, 1500, 4000])])
def test_paged_pool_tensor_core_path(page_tokens, m_csa, topk, lengths):
    """Benchmark head shape over a paged pool.  128-token pages hold exactly one 32-row TMA box of CSA entries (m = 4) and
    one HCA entry: contiguous-run tiles fetch page by page (single- and multi-chunk), ranked and long tiles gather by
    pointer; 256-token pages hold two boxes; with m = 16 a page holds 8 CSA entries and every tile gathers by pointer."""
    heads = dict(BENCH_HEADS, m_csa=m_csa)
    cfg = synth.Config(f"paged_tc_{page_tokens}_{m_csa}_{topk}", 94, synth.Shape("bf16", len(lengths), 8, topk=topk, **heads), layers=1,
                       L_min=1, L_max=1, seed=page_tokens + topk)
    lockstep(cfg, cycles=3, lengths=lengths, page_tokens=page_tokens, check_recompress="final")


def test_paged_pool_tensor_core_path_without_index_lists():
    """The paged pool called the way the benchmark calls it (no buffer for the index lists): sequences that cannot rank,
    one at the ranking threshold, ranked contiguous-run tiles and a gathered one."""
    cfg = synth.Config("paged_tc_no_lists", 95, synth.Shape("bf16", 5, 8, topk=256, sm_scale=8.0, **BENCH_HEADS), layers=1, L_min=1, L_max=1, seed=9)
    lockstep(cfg, cycles=3, lengths=[300, 1015, 1023, 1700, 2600], page_tokens=128, want_topk=False, per_row=True)

# ------------------------------------------------------------------------------------------------ refresh schedules
@pytest.mark.parametrize("dtype", ["fp32", "bf16"])
def test_c128_deferred_refresh_schedule_small(dtype):
    """C128-deferred schedule on small shapes: with m' = 20 and D = 6 about two thirds of the (sequence, cycle) pairs defer
    the HCA update to the commit, the others (a block can close inside the tree) build HCA branch states as usual; the
    committed caches equal the oracle's and recompression from scratch after every cycle."""
    from paper_2609_24698_b200 import binding as tsv
    cfg = synth.small_config(name="hca_deferred", dtype=dtype, B=6, D=6, H=4, d=32, m_csa=2, topk=6, HI=2, di=16, m_hca=20, window=10,
                             L_min=0, L_max=70, layers=2, seed=91, cfg_id=91, sm_scale=2.0)
    lockstep(cfg, cycles=12, flags=tsv.FLAG_HCA_DEFERRED, check_recompress=True)


def test_c128_deferred_refresh_schedule_bench_shape_bit_identical():
    """Benchmark head shape (m' = 128: nearly every cycle defers), 2 layers, 10 cycles against the oracle; the committed
    caches are then bit-identical to those of the timely schedule on the same inputs."""
    from paper_2609_24698_b200 import binding as tsv
    cfg = synth.Config("hca_deferred_tc", 92, synth.Shape("bf16", 8, 8, topk=512, **BENCH_HEADS), layers=2, L_min=100, L_max=1500, seed=10)
    lengths = synth.prefix_lengths(cfg).copy()
    lengths[0] = 128 * 5 - 3                      # one sequence closes an HCA block inside the tree on the first cycle
    _, eng_d, _ = lockstep(cfg, cycles=10, lengths=lengths, flags=tsv.FLAG_HCA_DEFERRED, return_engine=True, check_recompress="final")
    _, eng_t, _ = lockstep(cfg, cycles=10, lengths=lengths, return_engine=True)
    for l in range(cfg.layers):
        for name in ("L", "hca_mx", "hca_s", "hca_kv", "csa_kv", "csa_ik", "win_kv", "csa_mx", "csa_s"):
            assert torch.equal(getattr(eng_d.caches[l], name), getattr(eng_t.caches[l], name)), name
        open_h = (eng_t.caches[l].L % cfg.shape.m_hca) != 0           # (an empty block's stored numbers are not defined)
        assert torch.equal(eng_d.caches[l].hca_acc_kv[open_h], eng_t.caches[l].hca_acc_kv[open_h])
        assert torch.equal(eng_d.out[l], eng_t.out[l])

# ------------------------------------------------------------------------------------------------ variants
@pytest.mark.parametrize("dtype,big", [("fp32", False), ("bf16", False), ("bf16", True)])
def test_variant_without_hca_cache(dtype, big):
    """A layer with no HCA cache (the CSA-only variant the paper's discussion names): an HCA block length beyond any
    sequence length keeps n_hca at 0 for ever; CUDA-core path (small d) and tensor-core path (bench head shape)."""
    no_hca = 1 << 30
    if big:
        cfg = synth.Config("no_hca_tc", 88, synth.Shape("bf16", 4, 8, 64, 512, 4, 256, 4, 128, no_hca, 128), L_min=200, L_max=2300, seed=8)
        lockstep(cfg, cycles=3, check_recompress=True)
    else:
        cfg = synth.small_config(name="no_hca", dtype=dtype, B=4, D=8, H=6, d=64, m_csa=2, topk=10, HI=2, di=16, m_hca=no_hca, window=12,
                                 L_min=0, L_max=90, layers=2, seed=87, cfg_id=87, sm_scale=2.0)
        lockstep(cfg, cycles=5, check_recompress=True)

# ------------------------------------------------------------------------------------------------ the cycle as the benchmark runs it
@pytest.mark.parametrize("want_topk", [True, False])
def test_graph_replayed_cycles_match_oracle_and_eager(want_topk):
    """One CUDA graph captured over a fixed input slot and replayed for four cycles (fresh inputs copied into the slot each
    time), 2 layers on the benchmark head shape: branch states, outputs, selections, acceptance and refreshed caches
    against the oracle every cycle; then bit-equality of outputs, selections, acceptance and caches with an engine that
    ran the same four cycles eagerly.  Once with and once without a buffer for the index lists (the benchmark's call)."""
    cfg = synth.Config("graph_cycle", 86, synth.Shape("bf16", 6, 8, topk=512, **BENCH_HEADS), layers=2, L_min=200, L_max=2600, seed=6)
    _, eng_g, _ = lockstep(cfg, cycles=4, graph=True, return_engine=True, check_recompress=True, want_topk=want_topk)
    _, eng_e, _ = lockstep(cfg, cycles=4, return_engine=True, want_topk=want_topk)
    from paper_2609_24698_b200 import binding as tsv
    for l in range(cfg.layers):
        assert torch.equal(eng_g.out[l], eng_e.out[l]) and (not want_topk or torch.equal(eng_g.topk_idx[l], eng_e.topk_idx[l]))
        for name in tsv.CACHE_TENSORS:
            assert torch.equal(getattr(eng_g.caches[l], name), getattr(eng_e.caches[l], name)), name
    assert torch.equal(eng_g.accept_path, eng_e.accept_path) and torch.equal(eng_g.accept_len, eng_e.accept_len)

# ------------------------------------------------------------------------------------------------ status / error paths
@pytest.mark.parametrize("path", ["cuda_cores", "tensor_cores_without_index_lists"])
def test_device_detected_errors_commit_nothing(path):
    """Flagged sequences (parent array out of order, node count out of range, no room for a closing entry) next to a good
    one: status bits, zero outputs, nothing committed.  Once on a small fp32 shape (CUDA-core attention) and once on the
    benchmark head shape without a buffer for the index lists (selection CTAs that leave early, the tile plan's empty
    records, the paired kernel's zero fill)."""
    from paper_2609_24698_b200 import binding as tsv, harness as hz
    if path == "cuda_cores":
        cfg = synth.small_config(dtype="fp32", B=4, D=6, H=2, d=16, m_csa=2, topk=3, HI=1, di=8, m_hca=3, window=8,
                                 L_min=4, L_max=9, layers=2, seed=40)
    else:
        cfg = synth.Config("tc_flagged", 86, synth.Shape("bf16", 4, 8, topk=512, **BENCH_HEADS), L_min=300, L_max=900, seed=8)
    sh = cfg.shape
    lengths = synth.prefix_lengths(cfg)
    states = oracle_states(cfg, lengths)
    ccap, hcap = hz.capacities(sh, lengths, 64)
    ccap[3] = int(lengths[3]) // sh.m_csa            # sequence 3: no room for the entry a deep path could close
    eng = hz.VerifyEngine(sh, cfg.layers, ccap, hcap, int(lengths.max()) + 64, want_topk=(path == "cuda_cores"))
    for l in range(cfg.layers):
        for b in range(sh.B):
            hz.fill_cache(eng.caches[l], sh, b, int(lengths[b]), state_arrays(states[l][b]))
    nodes = [synth.node_inputs(cfg, l, 0) for l in range(cfg.layers)]
    parent, n_nodes = synth.trees(cfg, 0)
    parent[1, 3] = 3                                  # not a parent-before-child array
    n_nodes[2] = 0                                    # node count out of range
    draft, target = synth.tokens(cfg, 0, np.where(parent < np.arange(sh.D), parent, 0), np.maximum(n_nodes, 1))
    inp = hz.InputSet.from_numpy(sh, nodes, parent, n_nodes, draft, target)
    before = eng.snapshot()
    for o in eng.out:
        o.fill_(7.0)
    eng.launch_cycle(inp)
    torch.cuda.synchronize()
    st = eng.status.cpu().numpy()
    assert st[0] == 0 and st[1] & tsv.ST_PARENT and st[2] & tsv.ST_NODES and st[3] & tsv.ST_CSA_CAP
    alen = eng.accept_len.cpu().numpy()
    assert alen[0] >= 1 and list(alen[1:]) == [0, 0, 0]
    for l in range(cfg.layers):
        assert int(eng.caches[l].L[0]) == int(lengths[0]) + int(alen[0])
        for b in (1, 2, 3):                            # all-or-nothing: nothing of a flagged sequence is committed
            assert int(eng.caches[l].L[b]) == int(lengths[b])
            assert torch.equal(eng.caches[l].win_kv[b], before[l].win_kv[b])
            assert torch.equal(eng.caches[l].csa_acc_kv[b], before[l].csa_acc_kv[b])
            assert not eng.out[l][b].any()            # outputs of flagged sequences are zero-filled
        assert eng.out[l][0].any()


def test_determinism_same_inputs_same_bits():
    cfg = synth.small_config(dtype="bf16", B=3, D=8, H=20, d=64, m_csa=4, topk=48, HI=4, di=32, m_hca=16, window=40,
                             L_min=130, L_max=700, layers=1, seed=32)
    _, eng1, _ = lockstep(cfg, cycles=2, return_engine=True)
    _, eng2, _ = lockstep(cfg, cycles=2, return_engine=True)
    assert torch.equal(eng1.out[0], eng2.out[0]) and torch.equal(eng1.topk_idx[0], eng2.topk_idx[0])
    assert torch.equal(eng1.caches[0].csa_kv, eng2.caches[0].csa_kv)
