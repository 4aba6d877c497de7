"""Verification budget and batch sweep, tree against chain (the study the paper runs end to end with a real model,
"Experiments": budgets 5-8, batch sizes 1-64, tree against linear drafts; here on the verify-side path alone).

    python -m paper_2609_24698_b200.sweep [--budgets 5 6 7 8] [--batches 1 4 16 64] [--layers 8] [--steps 20]

For every (budget D, batch B) the same verify cycle (branch_state_build + tree_verify_attn per layer, then
accept_and_refresh) is timed on seeded synthetic inputs of the benchmark's head shape and prefix mix, once with random
trees of D nodes and once with chains of D nodes.  What the path can answer is what verifying a tree costs relative to
verifying a chain of the same budget; how many more tokens a tree gets accepted depends on the draft and target models
and is not modelled (the synthetic acceptance rule accepts a child of a node with the same probability in both shapes).
Prints a markdown table; timing as in bench.py (cycles replayed from CUDA graphs over rotating input sets, CUDA events).
"""
from __future__ import annotations

import argparse

import torch

from . import synth
from . import workload as W


def time_cycles(cfg: synth.Config, steps: int, warmup: int = 3, n_sets: int = 3):
    wl = W.build(cfg, cycles_headroom=2 * (steps + warmup) + 8, n_sets=n_sets)
    eng = wl.engine
    graphs = [eng.capture(inp) for inp in wl.inputs]
    for i in range(warmup):
        graphs[i % n_sets].replay()
    torch.cuda.synchronize()
    acc = torch.zeros((), dtype=torch.int64, device="cuda")
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for i in range(steps):
        graphs[(warmup + i) % n_sets].replay()
        acc += eng.accept_len.sum()
    e1.record()
    torch.cuda.synchronize()
    if int(eng.status.abs().sum()) != 0:
        raise RuntimeError(f"{cfg.name}: status flags raised")
    ms = e0.elapsed_time(e1) / steps
    return ms, float(acc) / (steps * cfg.shape.B)


def main() -> None:
    ap = argparse.ArgumentParser()
    ap.add_argument("--budgets", type=int, nargs="+", default=[5, 6, 7, 8])
    ap.add_argument("--batches", type=int, nargs="+", default=[1, 4, 16, 64])
    ap.add_argument("--layers", type=int, default=8)
    ap.add_argument("--steps", type=int, default=20)
    args = ap.parse_args()
    # one throw-away configuration first: module load, first-use costs of every kernel and of the graph machinery
    time_cycles(synth.Config("sweep_warm", 80, synth.Shape("bf16", 2, 5, 64, 512, 4, 512, 4, 128, 128, 128), layers=args.layers,
                             L_min=256, L_max=2048, seed=1), 3)
    print("| D | B | tree ms/cycle | chain ms/cycle | tree / chain | tree verified tok/s | mean accepted length tree / chain |")
    print("|---|---|---|---|---|---|---|")
    for D in args.budgets:
        for B in args.batches:
            res = {}
            for tree in ("random", "chain"):
                cfg = synth.Config(f"sweep_{tree}_d{D}_b{B}", 80 + D, synth.Shape("bf16", B, D, 64, 512, 4, 512, 4, 128, 128, 128),
                                   layers=args.layers, L_min=256, L_max=2048, tree=tree, seed=100 * D + B)
                res[tree] = time_cycles(cfg, args.steps)
                torch.cuda.empty_cache()
            (tm, ta), (cm, ca) = res["random"], res["chain"]
            print(f"| {D} | {B} | {tm:.3f} | {cm:.3f} | {tm / cm:.2f} | {B * D / tm * 1e3:,.0f} | {ta:.2f} / {ca:.2f} |", flush=True)


if __name__ == "__main__":
    main()
