"""Device time per call of small-batch race sampling and sequence verification.

    python -m paper_2504_15475_b200.latency [--V 128256] [--k 5] [--batches 1,2,4,8,16,32]
    python -m paper_2504_15475_b200.latency --trees [--batches 1,2,4]     # draft trees, batch drafting

Calls of a few rows are bound by latency, not by bandwidth, and a Python caller cannot issue
them faster than about ten microseconds apart; so the calls are captured into a CUDA graph (30
calls on rotating inputs) and the graph is replayed: the time per call is the device's own,
launch gaps included.  One JSON line per (entry, batch, kernel) with kernel = "streaming" or
"cluster" (opts.kernel_path 1 and 2) and "default" (what the library picks by itself).
"""
from __future__ import annotations

import argparse
import json

import torch

from . import binding
from . import workloads as wl

PATHS = {"default": 0, "streaming": 1, "cluster": 2}


def graph_time_us(call, calls_per_graph=30, replays=20):
    """Mean device time of call(i, stream), i = 0.. rotating, measured by graph replay."""
    st = torch.cuda.Stream()
    st.wait_stream(torch.cuda.current_stream())
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    with torch.cuda.stream(st):
        for i in range(6):
            call(i, st)
        torch.cuda.synchronize()
        g = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g, stream=st):
            for i in range(calls_per_graph):
                call(i, st)
        for _ in range(3):
            g.replay()
        torch.cuda.synchronize()
        e0.record(st)
        for _ in range(replays):
            g.replay()
        e1.record(st)
        torch.cuda.synchronize()
    return e0.elapsed_time(e1) * 1e3 / (calls_per_graph * replays)


def time_trees(args):
    """ersd_verify_tree on the draft-tree shapes of the workloads module."""
    V = args.V
    shapes = (("root with 4 children, chains to depth 4", wl.TREE_4x4), ("SpecInfer shape", wl.TREE_SPECINFER),
              ("star of 8", wl.star_parent(8)), ("chain of 16", wl.chain_parent(16)))
    for name, parent in shapes:
        n = len(parent)
        for B in [int(x) for x in args.batches.split(",")]:
            gen = torch.Generator().manual_seed(2000 + B)
            sets = []
            for _ in range(min(args.sets, 4)):
                t = wl.zipf_rows(B * n, V, gen, "cpu").view(B, n, V)
                d = t + torch.randn(B, n, V, generator=gen)
                sets.append((t.to(torch.bfloat16).cuda(), d.to(torch.bfloat16).cuda()))
            seeds = wl.make_seeds(78, B, B).cuda()
            D = binding.ersd_tree_depth(parent)
            tok = torch.empty(B, D + 1, dtype=torch.int32, device="cuda")
            acc = torch.empty(B, dtype=torch.int32, device="cuda")
            ws = torch.zeros(binding.ersd_workspace_bytes(B, n), dtype=torch.uint8, device="cuda")
            binding.ersd_workspace_init(ws)
            for kernel, path in PATHS.items():
                opts = binding.make_opts(workspace=ws, kernel_path=path, split_v=args.split if path else 0)

                def call(i, st):
                    t, d = sets[i % len(sets)]
                    binding.ersd_verify_tree(t, d, parent, seeds, 1.0, tok, acc, opts, st)

                try:
                    call(0, torch.cuda.current_stream())
                except binding.ErsdError:                     # this kernel does not take the call
                    continue
                if args.plain:
                    for i in range(args.plain):
                        call(i, torch.cuda.current_stream())
                    torch.cuda.synchronize()
                    continue
                print(json.dumps({"entry": "ersd_verify_tree", "tree": name, "nodes": n, "B": B, "V": V,
                                  "dtype": "bf16", "kernel": kernel, "launch": binding.ersd_last_launch(),
                                  "us_per_call": round(graph_time_us(call), 2),
                                  "timing": "CUDA graph replay, 30 calls per graph"}), flush=True)


def time_batch_drafting(args, c=8):
    """ersd_race_sample with top_c = c: the first c arrivals of one race per sequence."""
    V = args.V
    for B in [int(x) for x in args.batches.split(",")]:
        gen = torch.Generator().manual_seed(3000 + B)
        rows = [wl.zipf_rows(B, V, gen, "cpu").view(B, 1, V).to(torch.bfloat16).cuda() for _ in range(min(args.sets, 4))]
        seeds = wl.make_seeds(79, B, B).cuda()
        tok = torch.empty(B, 1, c, dtype=torch.int32, device="cuda")
        ws = torch.zeros(binding.ersd_workspace_bytes(B, 1), dtype=torch.uint8, device="cuda")
        binding.ersd_workspace_init(ws)
        for kernel, path in PATHS.items():
            opts = binding.make_opts(workspace=ws, kernel_path=path, top_c=c, split_v=args.split if path else 0)

            def draft(i, st):
                binding.ersd_race_sample(rows[i % len(rows)], seeds, 1.0, tok, opts, st)

            try:
                draft(0, torch.cuda.current_stream())
            except binding.ErsdError:                         # this kernel does not take the call
                continue
            if args.plain:
                for i in range(args.plain):
                    draft(i, torch.cuda.current_stream())
                torch.cuda.synchronize()
                continue
            print(json.dumps({"entry": "ersd_race_sample", "top_c": c, "B": B, "V": V, "dtype": "bf16",
                              "kernel": kernel, "launch": binding.ersd_last_launch(),
                              "us_per_call": round(graph_time_us(draft), 2),
                              "timing": "CUDA graph replay, 30 calls per graph"}), flush=True)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--V", type=int, default=128256)
    ap.add_argument("--k", type=int, default=5, help="drafted positions per sequence (verification)")
    ap.add_argument("--batches", default="1,2,4,8,16,32")
    ap.add_argument("--sets", type=int, default=6, help="distinct inputs rotated between calls")
    ap.add_argument("--split", type=int, default=0, help="thread blocks per row / per cluster (0: library default)")
    ap.add_argument("--trees", action="store_true",
                    help="time ersd_verify_tree on draft trees, and batch drafting, instead of the two entries above")
    ap.add_argument("--plain", type=int, default=0,
                    help="issue this many plain calls per case instead of replaying a graph and print no "
                         "times (for a profiler's launch list)")
    args = ap.parse_args()
    binding.lib()
    if not torch.cuda.is_available():
        raise SystemExit("needs a CUDA device")
    V, k = args.V, args.k
    if args.trees:
        time_trees(args)
        time_batch_drafting(args)
        return
    for B in [int(x) for x in args.batches.split(",")]:
        gen = torch.Generator().manual_seed(1000 + B)
        sets = []
        for _ in range(args.sets):
            t = wl.zipf_rows(B * (k + 1), V, gen, "cpu").view(B, k + 1, V)
            d = t[:, :k] + torch.randn(B, k, V, generator=gen)
            sets.append((t.to(torch.bfloat16).cuda(), d.to(torch.bfloat16).cuda().contiguous()))
        seeds = wl.make_seeds(77, B, B).cuda()
        ws = torch.zeros(binding.ersd_workspace_bytes(B, k + 1), dtype=torch.uint8, device="cuda")
        binding.ersd_workspace_init(ws)
        tok1 = torch.empty(B, 1, 1, dtype=torch.int32, device="cuda")
        tok = torch.empty(B, k + 1, dtype=torch.int32, device="cuda")
        acc = torch.empty(B, dtype=torch.int32, device="cuda")
        rows1 = [s[1][:, :1].contiguous() for s in sets]          # one draft row per sequence
        for name, path in PATHS.items():
            opts = binding.make_opts(workspace=ws, kernel_path=path, split_v=args.split if path else 0)

            def sample(i, st):
                binding.ersd_race_sample(rows1[i % len(sets)], seeds, 1.0, tok1, opts, st)

            def verify(i, st):
                t, d = sets[i % len(sets)]
                binding.ersd_verify(t, d, seeds, 1.0, tok, acc, opts, st)

            for entry, fn, rows in (("ersd_race_sample", sample, B), ("ersd_verify", verify, B * (2 * k + 1))):
                if args.plain:
                    for i in range(args.plain):
                        fn(i, torch.cuda.current_stream())
                    torch.cuda.synchronize()
                    continue
                us = graph_time_us(fn)
                print(json.dumps({"entry": entry, "B": B, "k": None if fn is sample else k, "V": V, "dtype": "bf16",
                                  "kernel": name, "split": args.split if path else 0, "us_per_call": round(us, 2), "logit_rows_per_call": rows,
                                  "timing": "CUDA graph replay, 30 calls per graph"}), flush=True)


if __name__ == "__main__":
    main()
