#!/usr/bin/env python
"""Benchmark of the verify-side hot path (one step = one full verify cycle over all layers:
branch_state_build + tree_verify_attn per layer, then accept_and_refresh).

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference] [--workload cfg4]

Prints ONE JSON line (rank 0).  `value` is verified tree tokens per second (B*D tokens per cycle)
with inputs resident in HBM and the cycle replayed from a CUDA graph; `e2e` is the same metric
with every step's inputs copied from pinned host memory and the acceptance result read back
(within a step the copy of the next layer's inputs runs under the current layer's kernels; steps do
not overlap).
N > 1 runs N independent replicas (the path has no exchange step): weak scaling, no collective
on the data path; only the barrier and the MAX-over-ranks of the device time use the process group.
"""
from __future__ import annotations

import argparse
import json
import os
import subprocess
import sys
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import numpy as np  # noqa: E402

# Measured DRAM traffic (ncu: dram__bytes_read.sum + dram__bytes_write.sum), per workload: the dominant kernel of the
# attention stage with the bytes of ONE of its launches (one layer), and, where captured, the sum over all kernels of one
# verify cycle.  The captures are summarised under profiles/; workloads without a capture report null.
NCU_DRAM = {
    "cfg4": {"kernel": "tc_attn_pair_kernel", "launch_bytes": 66_239_168, "cycle_bytes": None},   # 65.48 MB read + 0.76 MB written
    # cfg5: tc_attn_pair_kernel 61.11 MB read + 1.70 MB written; all kernels of one cycle 138.1 MB (cold cache per kernel)
    "cfg5": {"kernel": "tc_attn_pair_kernel", "launch_bytes": 62_808_320, "cycle_bytes": 138_081_792},
}
ATTN_KERNEL = {"cfg1": "attn_simt_kernel (fp32 CUDA-core path)", "cfg2": "tc_attn_pair_kernel + tc_combine_pair_kernel",
               "cfg2_chain": "tc_attn_pair_kernel + tc_combine_pair_kernel",
               "cfg3": "tc_attn_pair_kernel (contiguous-run and gathered tiles) + tc_combine_pair_kernel", "cfg4": "tc_attn_pair_kernel",
               "cfg5": "tc_attn_pair_kernel (gathered tiles) + tc_combine_pair_kernel"}


def peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        j = json.load(open(p))
        return {"hbm_gbs": float(j["hbm_gbs"]), "bf16_tflops": float(j["bf16_tflops"]),
                "bf16_tflops_sustained": float(j.get("bf16_tflops_sustained", j["bf16_tflops"])), "source": "measured"}
    return {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0, "source": "fallback"}


class ClockSampler:
    """nvidia-smi clock / throttle-reason samples taken while the timed region runs."""
    Q = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,clocks_event_reasons.hw_slowdown,"
         "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index: int):
        self.idx, self.proc = gpu_index, None

    def start(self):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", f"--query-gpu={self.Q}", "--format=csv,noheader,nounits", "-lms", "100",
                                          "-i", str(self.idx)], stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
        except OSError:
            self.proc = None

    def stop(self):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        time.sleep(0.15)
        self.proc.terminate()
        try:
            out, _ = self.proc.communicate(timeout=5)
        except subprocess.TimeoutExpired:
            self.proc.kill(); out = ""
        sm, mx, reasons = [], [], set()
        for line in out.strip().splitlines():
            f = [x.strip() for x in line.split(",")]
            if len(f) < 9:
                continue
            try:
                sm.append(float(f[1])); mx.append(float(f[2]))
            except ValueError:
                continue
            for name, v in zip(("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"), f[5:9]):
                if v.lower().startswith("active"):
                    reasons.add(name)
        return {"sm_mhz": float(np.median(sm)) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "samples": len(sm), "reasons": sorted(reasons)}


# ------------------------------------------------------------------------------------------ oracle arm
def oracle_sample(cfg, n_layers_sample: int, n_seq_sample: int, steps: int, warmup: int):
    """Times the CPU oracle (as it stands) on a bounded sample of the workload: the first
    n_seq_sample sequences x n_layers_sample layers of the same seeded inputs, one verify cycle per step.
    Returns verified tokens/s scaled to the full layer count, and a description of the sample."""
    from oracle import tsv_oracle as O
    from paper_2609_24698_b200 import synth      # (synth only: the CUDA library is not loaded into the oracle's process)
    direct_arrays = synth.direct_arrays
    sh = cfg.shape
    lengths = synth.prefix_lengths(cfg)

    def fresh_states():
        st = []
        for l in range(n_layers_sample):
            row = []
            for b in range(n_seq_sample):
                a = direct_arrays(cfg, l, b, int(lengths[b]))
                row.append(O.SeqState(int(lengths[b]), a["csa_kv"].astype(np.float64), a["csa_ik"].astype(np.float64),
                                      a["hca_kv"].astype(np.float64), a["win"].astype(np.float64),
                                      O.Partial(a["csa_mx"], a["csa_s"], [a["csa_acc_kv"].astype(np.float64), a["csa_acc_ik"].astype(np.float64)]),
                                      O.Partial(a["hca_mx"], a["hca_s"], [a["hca_acc_kv"].astype(np.float64)])))
            st.append(row)
        return st

    states = fresh_states()
    times, cpu_times = [], []
    n_sets = min(3, warmup + steps)
    node_sets = [[{k: v[:n_seq_sample] for k, v in synth.node_inputs(cfg, l, c).items()} for l in range(n_layers_sample)]
                 for c in range(n_sets)]
    for it in range(warmup + steps):
        c = it % n_sets
        nodes = node_sets[c]
        parent, n_nodes = synth.trees(cfg, c)
        draft, target = synth.tokens(cfg, c, parent, n_nodes)
        t0, c0 = time.perf_counter(), time.process_time()
        O.verify_cycle(states, sh, nodes, parent[:n_seq_sample], n_nodes[:n_seq_sample], draft[:n_seq_sample], target[:n_seq_sample])
        dt, dc = time.perf_counter() - t0, time.process_time() - c0
        if it >= warmup:
            times.append(dt); cpu_times.append(dc)
    t_cycle_full_layers = float(np.mean(times)) * cfg.layers / n_layers_sample
    tok_s = n_seq_sample * sh.D / t_cycle_full_layers
    # cores the oracle keeps busy: CPU time of the process (all threads) over wall time; the oracle is mostly Python loops
    # around numpy calls, so this is close to 1 however many threads the BLAS pool holds
    cores = max(1, int(round(float(np.sum(cpu_times)) / max(float(np.sum(times)), 1e-9))))
    sample = (f"{n_seq_sample} of {sh.B} sequences x {n_layers_sample} of {cfg.layers} layers of {cfg.name}, "
              f"{steps} verify cycles (mean {np.mean(times):.3f} s each), time scaled to {cfg.layers} layers")
    return tok_s, float(np.mean(times)) * 1e3, cores, sample


def run_reference(args, cfg):
    """Reference arm = the fp64 CPU oracle on the host cores, bounded sample, same metric and config."""
    from paper_2609_24698_b200 import dist as D
    rank, _, world = D.env_world()
    if rank != 0:
        return
    steps, warmup = max(1, min(args.steps, 5)), max(0, min(args.warmup, 1))
    tok_s, ms, cores, sample = oracle_sample(cfg, n_layers_sample=min(2, cfg.layers), n_seq_sample=min(32, cfg.shape.B), steps=steps, warmup=warmup)
    line = {"impl": "reference", "metric": "verified_tree_tokens_per_s", "value": tok_s, "unit": "tokens/s", "n_gpus": args.gpus,
            "steps": steps, "warmup": warmup, "ms_per_step": ms, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
            "dtype": "f64", "data": "synthetic", "config": workload_config(cfg, args),
            "cpu_baseline": {"value": tok_s, "unit": "tokens/s", "cores": cores, "kind": "oracle", "sample": sample},
            "e2e": {"value": tok_s, "unit": "tokens/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}}
    print(json.dumps(line), flush=True)


def workload_config(cfg, args):
    sh = cfg.shape
    return {"workload": f"{cfg.name}: {cfg.layers}-layer stack, {sh.dtype}, batch {sh.B}, D={sh.D} random trees, prefixes "
                        f"U[{cfg.L_min},{cfg.L_max}], H={sh.H}, d={sh.d}, CSA m={sh.m_csa} top-k={sh.topk} (indexer {sh.HI}x{sh.di}), "
                        f"HCA m'={sh.m_hca}, window {sh.window}",
            "global_batch": sh.B * max(1, args.gpus), "tree_nodes": sh.D, "layers": cfg.layers,
            "parallelism": "single GPU" if args.gpus <= 1 else f"{args.gpus} independent replicas (no collective)",
            "l2_policy": "inputs larger than L2: every cycle reads a different input set (q alone is 268 MB per cycle)",
            "launch": "one CUDA graph replay per cycle", "hca_refresh_schedule": getattr(args, "schedule", "timely"),
            "cache_layout": (f"paged pool, {args.page_tokens}-token pages, one page table for the CSA and HCA layers"
                             if getattr(args, "page_tokens", 0) else "flat slab per sequence"),
            "topk_idx": "not requested (tree_verify_attn's optional output; the selection is used by the attention only)"}


# ------------------------------------------------------------------------------------------ our arm
def run_ours(args, cfg):
    import torch
    from paper_2609_24698_b200 import binding as tsv, dist as D, synth, workload as W

    rank, local_rank, world = D.env_world()
    if not torch.cuda.is_available():
        raise SystemExit("bench.py: no CUDA device; the tree-verify path has no CPU fallback")
    torch.cuda.set_device(local_rank if world > 1 else 0)
    dev = torch.device("cuda", torch.cuda.current_device())
    D.init("nccl")
    if world > 1:                                     # replicas differ only by seed
        from dataclasses import replace
        cfg = replace(cfg, seed=cfg.seed + rank)
    sh = cfg.shape
    K, Wm = args.steps, max(3, args.warmup)
    n_sets = 3
    lib_flags = tsv.FLAG_HCA_DEFERRED if args.schedule == "c128-deferred" else 0
    wl = W.build(cfg, cycles_headroom=2 * (K + Wm) + 8, n_sets=n_sets, flags=lib_flags, device=dev, page_tokens=args.page_tokens)
    eng = wl.engine
    snap = eng.snapshot()
    stream = torch.cuda.current_stream()

    # ---- launch bookkeeping (our kernels per cycle) and graphs
    n0 = tsv.kernel_launches()
    eng.launch_cycle(wl.inputs[0])
    torch.cuda.synchronize()
    launches_per_cycle = tsv.kernel_launches() - n0
    assert int(eng.status.sum()) == 0, "workload flagged by the device-side validation"
    eng.restore(snap)
    graphs = [eng.capture(inp) for inp in wl.inputs] if not args.no_graph else None

    def step(i):
        if graphs is not None:
            graphs[i % n_sets].replay()
        else:
            eng.launch_cycle(wl.inputs[i % n_sets])

    # ---- timed region: K cycles, inputs resident in HBM
    for i in range(Wm):
        step(i)
    torch.cuda.synchronize(); D.barrier(); torch.cuda.synchronize()
    clk = ClockSampler(torch.cuda.current_device()); clk.start()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record(stream)
    for i in range(K):
        step(Wm + i)
    e1.record(stream)
    torch.cuda.synchronize(); D.barrier(); torch.cuda.synchronize()
    clocks = clk.stop()
    sec_local = e0.elapsed_time(e1) * 1e-3
    accepted = float(eng.accept_len.sum().item())
    assert int(eng.status.sum()) == 0
    value, sec = D.whole_job_throughput(sh.B * sh.D * K, sec_local, dev)

    # ---- per-stage pass: each stage of the cycle captured alone in a CUDA graph (all layers) and replayed, timed with
    # CUDA events on the launching stream.  Graph replay keeps the host out of the measurement; the attention stage is
    # tree_verify_attn without its selection step (tile plan + paired attention kernel + merge of multi-chunk tiles).
    eng.restore(snap)
    inp0 = wl.inputs[0]
    eng.launch_cycle(inp0, refresh=False)           # scratch pads and selections of inp0 are in place for the partial graphs
    torch.cuda.synchronize()

    def stage_fn(name):
        def f():
            for l in range(eng.n_layers):
                if name == "branch_state_build":
                    tsv.branch_state_build(eng.cshape, eng.caches[l], inp0.layers[l], eng.scratch[l], eng.status)
                elif name == "select":
                    tsv.bench_tree_verify_attn_stages(eng.cshape, eng.caches[l], inp0.layers[l], eng.scratch[l], eng.out[l], None,
                                                      eng.workspace, eng.status, tsv.STAGE_SELECT)
                elif name == "attention":
                    tsv.bench_tree_verify_attn_stages(eng.cshape, eng.caches[l], inp0.layers[l], eng.scratch[l], eng.out[l], None,
                                                      eng.workspace, eng.status, tsv.STAGE_ATTENTION)
                elif name == "attention_kernels":    # the stage without its tile plan (the plan of the call before is used again)
                    tsv.bench_tree_verify_attn_stages(eng.cshape, eng.caches[l], inp0.layers[l], eng.scratch[l], eng.out[l], None,
                                                      eng.workspace, eng.status, tsv.STAGE_ATTENTION_KERNELS)
        return f

    t_parts = {}
    for name in ("branch_state_build", "select", "attention", "attention_kernels"):
        sg = torch.cuda.Stream(); sg.wait_stream(stream)
        g = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g, stream=sg):
            stage_fn(name)()
        stream.wait_stream(sg)
        for _ in range(Wm):
            g.replay()
        s0, s1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        s0.record(stream)
        for _ in range(K):
            g.replay()
        s1.record(stream)
        torch.cuda.synchronize()
        t_parts[name] = s0.elapsed_time(s1) / K / eng.n_layers          # ms per layer-call
    a0, a1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    a0.record(stream)
    tsv.accept_and_refresh(eng.cshape, eng._pack(inp0), inp0.draft, inp0.target, eng.accept_len, eng.accept_path, eng.bonus, eng.status)
    a1.record(stream)
    torch.cuda.synchronize()
    t_parts["accept_and_refresh"] = a0.elapsed_time(a1)
    attn_ms = float(t_parts["attention"])
    kern_ms = float(t_parts["attention_kernels"])

    # ---- algorithmic work and roofline of the dominant kernel (attention)
    parents = wl.inputs[0].layers[0].parent.cpu().numpy()
    work = W.algorithmic_work(sh, cfg.layers, wl.lengths, parents)
    pk = peaks()
    # the dominant kernel is the attention kernel (with the merge kernel where a workload launches one): its duration is that
    # of the attention stage replayed without the tile plan; the stage with its plan kernel is reported next to it (in a
    # full cycle the plan runs under the tails of the state build and the selection, replayed alone it cannot)
    attn_gbs = work["attn_bytes_per_layer"] / (kern_ms * 1e-3) / 1e9
    attn_tf = work["attn_flops_per_layer"] / (kern_ms * 1e-3) / 1e12
    hbm = {"achieved": attn_gbs, "peak": pk["hbm_gbs"], "unit": "GB/s", "frac": attn_gbs / pk["hbm_gbs"],
           "algorithmic_bytes_per_launch": work["attn_bytes_per_layer"]}
    tensor = {"achieved": attn_tf, "peak": pk["bf16_tflops_sustained"], "unit": "TFLOP/s", "frac": attn_tf / pk["bf16_tflops_sustained"],
              "flops_per_launch": work["attn_flops_per_layer"]}
    # which roof governs: the stage's FLOP per algorithmic byte against the ridge of the measured peaks (fp32 storage runs
    # on the CUDA cores and is judged against the memory roof)
    ridge = pk["bf16_tflops_sustained"] * 1e12 / (pk["hbm_gbs"] * 1e9)
    intensity = work["attn_flops_per_layer"] / work["attn_bytes_per_layer"]
    bound = "tensor" if (sh.dtype == "bf16" and intensity > ridge) else "hbm"
    cap = NCU_DRAM.get(cfg.name)
    roofline = {"bound": bound, "kernel": f"tree_verify_attn: {ATTN_KERNEL.get(cfg.name, 'attention kernels')}, one layer, all sequences",
                **(tensor if bound == "tensor" else hbm),
                "traffic": cap["launch_bytes"] if cap else None,
                "traffic_note": (f"ncu DRAM read+write of one {cap['kernel']} launch on this workload" if cap else "no ncu capture for this workload"),
                "peak_source": pk["source"], "launch_ms": kern_ms,
                # the same work over the duration of the stage replayed with its tile plan kernel
                "with_tile_plan": {"launch_ms": attn_ms, "frac_hbm": attn_gbs * kern_ms / attn_ms / pk["hbm_gbs"],
                                   "frac_tensor": attn_tf * kern_ms / attn_ms / pk["bf16_tflops_sustained"]},
                "flop_per_byte": intensity, "ridge_flop_per_byte": ridge,
                "lengths": "algorithmic bytes and FLOPs from the initial prefix lengths (the caches grow by the accepted tokens while timed)",
                "hbm": hbm, "tensor": tensor}
    cycle_s = sec / K
    cycle = {"full_bytes": work["full_bytes"], "cache_bytes": work["cache_bytes"], "flops": work["flops"],
             "frac_hbm_full": work["full_bytes"] / cycle_s / 1e9 / pk["hbm_gbs"],
             "frac_hbm_cache": work["cache_bytes"] / cycle_s / 1e9 / pk["hbm_gbs"],
             "frac_tensor_sustained": work["flops"] / cycle_s / 1e12 / pk["bf16_tflops_sustained"],
             "measured_dram_bytes": cap["cycle_bytes"] if cap else None,
             "stage_ms_per_layer_call": {k: float(v) for k, v in t_parts.items()},
             "accepted_tokens_per_cycle_last": accepted}

    # ---- end to end: host buffers in, acceptance result out, every step
    eng.restore(snap)
    host_sets = [inp.pinned_host_copy() for inp in wl.inputs]
    slot = wl.inputs[0]
    res_dev = [eng.accept_len, eng.accept_path, eng.bonus, eng.status]
    res_host = [torch.empty_like(t, device="cpu").pin_memory() for t in res_dev]
    h2d = d2h = 0

    # Within a step the copy of layer l + 1's inputs runs (on a second stream) under layer l's kernels: a layer's calls wait
    # only for that layer's tensors.  Steps are not overlapped with each other (a real verify cycle builds its tree from
    # the previous cycle's result), so every step ends with the result on the host.
    copy_stream = torch.cuda.Stream()
    n_fields = len(slot.tensors()) - 4                       # per-layer node tensors, then parent, n_nodes, draft, target
    per_layer = n_fields // cfg.layers
    dev_t = slot.tensors()

    def e2e_step(i):
        nonlocal h2d, d2h
        host = host_sets[i % n_sets]
        h2d = 0
        copy_stream.wait_stream(stream)
        events = []
        with torch.cuda.stream(copy_stream):
            for d_, h_ in zip(dev_t[n_fields:], host[n_fields:]):
                d_.copy_(h_, non_blocking=True); h2d += h_.numel() * h_.element_size()
            for l in range(cfg.layers):
                for d_, h_ in zip(dev_t[l * per_layer:(l + 1) * per_layer], host[l * per_layer:(l + 1) * per_layer]):
                    d_.copy_(h_, non_blocking=True); h2d += h_.numel() * h_.element_size()
                ev = torch.cuda.Event(); ev.record(copy_stream); events.append(ev)
        eng.status.zero_()
        for l in range(cfg.layers):
            stream.wait_event(events[l])
            tsv.branch_state_build(eng.cshape, eng.caches[l], slot.layers[l], eng.scratch[l], eng.status)
            tsv.tree_verify_attn(eng.cshape, eng.caches[l], slot.layers[l], eng.scratch[l], eng.out[l], eng.topk_idx[l],
                                 eng.workspace, eng.status)
        tsv.accept_and_refresh(eng.cshape, eng._pack(slot), slot.draft, slot.target, eng.accept_len, eng.accept_path,
                               eng.bonus, eng.status)
        d2h = 0
        for hdst, dsrc in zip(res_host, res_dev):
            hdst.copy_(dsrc, non_blocking=True)
            d2h += dsrc.numel() * dsrc.element_size()
        torch.cuda.synchronize()

    for i in range(Wm):
        e2e_step(i)
    torch.cuda.synchronize(); D.barrier(); torch.cuda.synchronize()
    e0.record(stream)
    for i in range(K):
        e2e_step(Wm + i)
    e1.record(stream)
    torch.cuda.synchronize(); D.barrier(); torch.cuda.synchronize()
    e2e_value, _ = D.whole_job_throughput(sh.B * sh.D * K, e0.elapsed_time(e1) * 1e-3, dev)

    line = {"metric": "verified_tree_tokens_per_s", "value": value, "unit": "tokens/s", "n_gpus": world, "steps": K, "warmup": Wm,
            "ms_per_step": sec / K * 1e3, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
            "dtype": sh.dtype, "data": "synthetic", "config": workload_config(cfg, args), "clocks": clocks,
            "e2e": {"value": e2e_value, "unit": "tokens/s", "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h},
            "gpu_launches": int(launches_per_cycle * K), "roofline": roofline, "cycle": cycle}
    if rank == 0:
        if world == 1 and not args.no_cpu_baseline:
            tok_s, ms, cores, sample = oracle_sample(cfg, n_layers_sample=min(2, cfg.layers), n_seq_sample=min(32, sh.B), steps=4, warmup=1)
            line["cpu_baseline"] = {"value": tok_s, "unit": "tokens/s", "cores": cores, "kind": "oracle", "sample": sample}
        print(json.dumps(line), flush=True)
    D.finalize()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=50)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="cfg4")
    ap.add_argument("--no-graph", action="store_true", help="launch every call eagerly instead of replaying a CUDA graph")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--page-tokens", type=int, default=0,
                    help="keep the persistent caches in a paged pool with pages of this many tokens (0: flat slabs per sequence)")
    ap.add_argument("--schedule", default="timely", choices=["timely", "c128-deferred"],
                    help="refresh schedule of the HCA (C128) cache: per-node branch states (timely) or folded at commit time")
    args = ap.parse_args()
    from paper_2609_24698_b200 import synth
    cfg = synth.CONFIGS[args.workload]
    if args.impl == "reference":
        run_reference(args, cfg)
    else:
        run_ours(args, cfg)


if __name__ == "__main__":
    main()
