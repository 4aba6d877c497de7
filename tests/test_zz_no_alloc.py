"""tree_verify_attn_static: the entry point for callers that cannot allocate device memory
(engines that own the whole device pool, plug-ins, latency-critical loops).  Its workspace is an
array built into the library; this test checks, through the C-ABI, that it gives what
tree_verify_attn gives with a caller-provided workspace -- on two calls in a row, because the
built-in array is shared and keeps the previous call's contents --, that it matches the oracle on
the tensor-core path (whose plan leaves counters and tile records in the shared array between
calls), that the second call leaves the device's free memory as it was, and that shapes beyond
the built-in size are refused.
"""
import numpy as np
import pytest
import torch

from paper_2609_24698_b200 import synth

pytestmark = pytest.mark.gpu


def _setup(cfg, cycle):
    from paper_2609_24698_b200 import harness as hz, workload as W
    sh = cfg.shape
    lengths = synth.prefix_lengths(cfg)
    ccap, hcap = hz.capacities(sh, lengths, 4 * sh.D)
    eng = hz.VerifyEngine(sh, 1, ccap, hcap, int(lengths.max()) + 5 * sh.D, want_topk=True)
    for b in range(sh.B):
        hz.fill_cache(eng.caches[0], sh, b, int(lengths[b]), W.direct_arrays(cfg, 0, b, int(lengths[b])))
    parent, n_nodes = synth.trees(cfg, cycle)
    draft, target = synth.tokens(cfg, cycle, parent, n_nodes)
    inp = hz.InputSet.from_numpy(sh, [synth.node_inputs(cfg, 0, cycle)], parent, n_nodes, draft, target)
    return eng, inp


def test_static_workspace_matches_caller_workspace_twice():
    from paper_2609_24698_b200 import binding as tsv
    # ranked selection (n_csa > topk), several key splits, blocks closing inside the tree
    cfg = synth.small_config(name="noalloc", dtype="bf16", B=3, D=8, H=20, d=64, m_csa=4, topk=48, HI=4, di=32, m_hca=16,
                             window=40, L_min=130, L_max=700, seed=77, cfg_id=177)
    sh = cfg.shape
    for cycle in (0, 1):                       # second call: the built-in array still holds the first call's data
        eng, inp = _setup(cfg, cycle)
        tsv.branch_state_build(eng.cshape, eng.caches[0], inp.layers[0], eng.scratch[0], eng.status)
        tsv.tree_verify_attn(eng.cshape, eng.caches[0], inp.layers[0], eng.scratch[0], eng.out[0], eng.topk_idx[0],
                             eng.workspace, eng.status)
        torch.cuda.synchronize()
        ref_out, ref_idx = eng.out[0].clone(), eng.topk_idx[0].clone()
        out2 = torch.full_like(ref_out, 3.0)
        idx2 = torch.full_like(ref_idx, -7)
        tsv.tree_verify_attn_static(eng.cshape, eng.caches[0], inp.layers[0], eng.scratch[0], out2, idx2, eng.status)
        torch.cuda.synchronize()
        assert int(eng.status.sum()) == 0
        assert torch.equal(idx2, ref_idx)
        ref = ref_out.float().cpu().numpy()
        err = np.max(np.abs(out2.float().cpu().numpy() - ref)) / np.max(np.abs(ref))
        assert err <= 2e-2, err                # the tolerance of the bf16 parity tests; in practice the bits agree
        assert ref_out.any()


def test_static_workspace_tensor_core_path_matches_oracle_and_allocates_nothing():
    """bf16, d = 512 (tcgen05 kernels, single- and multi-chunk tiles), small enough for the built-in array: two cycles in
    a row against the oracle at the tolerance of the bf16 parity tests; free device memory unchanged across the second call."""
    from oracle import tsv_oracle as O
    from paper_2609_24698_b200 import binding as tsv, harness as hz
    from tests.helpers import oracle_states, per_seq, state_arrays
    cfg = synth.Config("noalloc_tc", 179, synth.Shape("bf16", 2, 8, 64, 512, 4, 512, 4, 128, 128, 128), L_min=300, L_max=1400, seed=12)
    sh = cfg.shape
    lengths = synth.prefix_lengths(cfg)
    states = oracle_states(cfg, lengths)
    ccap, hcap = hz.capacities(sh, lengths, 4 * sh.D)
    max_L = 1500
    assert tsv.workspace_bytes(sh, max_L) <= tsv.STATIC_WORKSPACE_BYTES
    eng = hz.VerifyEngine(sh, 1, ccap, hcap, max_L, want_topk=True)
    for b in range(sh.B):
        hz.fill_cache(eng.caches[0], sh, b, int(lengths[b]), state_arrays(states[0][b]))
    for cycle in (0, 1):
        nodes = synth.node_inputs(cfg, 0, cycle)
        parent, n_nodes = synth.trees(cfg, cycle)
        draft, target = synth.tokens(cfg, cycle, parent, n_nodes)
        inp = hz.InputSet.from_numpy(sh, [nodes], parent, n_nodes, draft, target)
        out = torch.full_like(eng.out[0], 3.0)
        tsv.branch_state_build(eng.cshape, eng.caches[0], inp.layers[0], eng.scratch[0], eng.status)
        torch.cuda.synchronize()
        free_before = torch.cuda.mem_get_info()[0]
        tsv.tree_verify_attn_static(eng.cshape, eng.caches[0], inp.layers[0], eng.scratch[0], out, eng.topk_idx[0], eng.status)
        torch.cuda.synchronize()
        if cycle == 1:
            assert torch.cuda.mem_get_info()[0] == free_before, "the call changed the device's free memory"
        assert int(eng.status.sum()) == 0
        got = out.float().cpu().numpy().astype(np.float64)
        for b in range(sh.B):
            nb = per_seq(nodes, b)
            sc = O.branch_state_build(states[0][b], sh, nb, parent[b], int(n_nodes[b]))
            ref, _ = O.tree_verify_attn(states[0][b], sh, nb, parent[b], int(n_nodes[b]), sc)
            err = np.max(np.abs(got[b] - ref)) / np.max(np.abs(ref))
            assert err <= 2e-2, (cycle, b, err)


def test_static_workspace_refuses_oversized_shapes():
    from paper_2609_24698_b200 import binding as tsv
    cfg = synth.small_config(name="noalloc_big", dtype="bf16", B=8, D=8, H=20, d=64, m_csa=4, topk=48, HI=4, di=32, m_hca=16,
                             window=40, L_min=130, L_max=700, seed=78, cfg_id=178)
    eng, inp = _setup(cfg, 0)
    big = tsv.c_shape(cfg.shape, 1 << 22)       # ranking scores for 4M-token prefixes: far beyond the built-in array
    assert tsv.workspace_bytes(cfg.shape, 1 << 22) > tsv.STATIC_WORKSPACE_BYTES
    out = torch.zeros_like(eng.out[0])
    with pytest.raises(tsv.TsvError) as ei:
        tsv.tree_verify_attn_static(big, eng.caches[0], inp.layers[0], eng.scratch[0], out, None, eng.status)
    assert ei.value.code == tsv.ERR_LIMIT
    torch.cuda.synchronize()
    assert not out.any()                        # nothing was enqueued
