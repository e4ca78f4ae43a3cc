#!/usr/bin/env python
"""Throughput of libersd's verify path on synthetic Zipf-shaped logits.

A step is one pass of the whole hot path (race variables, race keys, draft and
target winners, accepted-prefix scan: ONE kernel launch) over one batch.  The
default workload is the serving-scale sequence configuration (B=256, k=5,
V=128256, bf16, per-row Zipf exponents, per-sequence temperatures); three
distinct input sets are rotated so that every launch reads data the previous one
did not touch (each set, 722 MB, is larger than the 126 MB L2 anyway).

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload c5|c3|c4|c2] [--impl reference]

With N > 1 (under torch.distributed.run) every rank runs an independent replica
on its own GPU -- the path has no exchange step -- and rank 0 reports the total.
`--impl reference` times the CPU oracle, as it stands, on the host cores.
Prints one JSON line.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

# profiles/: dram bytes (read + write) per algorithmic byte of one launch, and the library version
# the counters were taken at
DRAM_BYTES_PER_ALGORITHMIC_BYTE = 1.016
TRAFFIC_AT_VERSION = 111  # (the counters were taken at this library version; another version reports traffic null)
SM_COUNT = 148

METRIC = "race-verified logit rows/s at V=128256 bf16 (B*(k+1) rows)"
UNIT = "rows/s"


def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            return float(json.load(f)["hbm_gbs"]), "measured"
    return 6650.0, "fallback"


class ClockSampler:
    """Samples nvidia-smi clocks and throttle reasons of one GPU while the timed region runs."""
    FIELDS = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
              "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
              "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index = index
        self.rows = []
        self.proc = None
        self.thread = None

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", "-i", str(self.index), "--query-gpu=" + self.FIELDS,
                 "--format=csv,noheader,nounits", "-lms", "50"],
                stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
        except OSError:
            self.proc = None
            return
        self.thread = threading.Thread(target=self._read, daemon=True)
        self.thread.start()

    def _read(self):
        for line in self.proc.stdout:
            self.rows.append((time.time(), [c.strip() for c in line.split(",")]))

    def stop(self, t0: float, t1: float):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        time.sleep(0.15)
        self.proc.terminate()
        try:
            self.proc.wait(timeout=2)
        except subprocess.TimeoutExpired:
            self.proc.kill()
        inside = [r for t, r in self.rows if t0 - 0.05 <= t <= t1 + 0.15] or [r for _, r in self.rows]
        sm, smax, reasons = [], [], set()
        for r in inside:
            try:
                sm.append(float(r[0]))
                smax.append(float(r[1]))
            except (ValueError, IndexError):
                continue
            for name, val in zip(("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"),
                                 r[4:8]):
                if val.lower().startswith("active"):
                    reasons.add(name)
        return {"sm_mhz": statistics.median(sm) if sm else None,
                "sm_max_mhz": max(smax) if smax else None, "reasons": sorted(reasons),
                "samples": len(inside)}


def algorithmic_bytes(w, inp, entry="verify"):
    """Bytes one verify launch must read: every target row, every draft row that has children
    (token-given verification reads target rows only)."""
    es = inp["target"].element_size()
    if entry == "gsd":
        return (w.B * (w.rows_target + w.k) + 2 * w.B) * w.V * es
    if entry == "tokens":
        rows = w.B * w.rows_target
    elif w.is_tree:
        parent = inp["parent"]
        internal = len({p for p in parent if p >= 0})
        rows = w.B * (w.rows_target + internal)
    else:
        rows = w.B * (w.rows_target + w.k)
    return rows * w.V * es


def oracle_rate(w, inp, n_seq, reps=1):
    """rows/s of the CPU oracle on the first n_seq sequences of inp (host copies made here)."""
    import oracle
    from paper_2504_15475_b200 import workloads as wl
    tgt = wl.as_numpy_logits(inp["target"][:n_seq])
    drf = wl.as_numpy_logits(inp["draft"][:n_seq])
    seeds = wl.seeds_as_u64(inp["seeds"][:n_seq])
    temps = None if inp.get("temps") is None else inp["temps"][:n_seq].cpu().numpy()
    best, ref = None, None
    for _ in range(reps):
        t0 = time.perf_counter()
        if w.is_tree:
            ref = oracle.verify_tree(tgt, drf, inp["parent"], seeds, T=inp["T"], temps=temps)
        else:
            ref = oracle.verify(tgt, drf, seeds, T=inp["T"], temps=temps)
        dt = time.perf_counter() - t0
        best = dt if best is None else min(best, dt)
    return n_seq * w.rows_target / best, best, oracle.max_threads(), ref


def parity_report(w, inp, n_seq, ref):
    """The library's result on the oracle's sample against the oracle's: target winners of every
    row, accepted lengths and emitted tokens.  A row counts as a near-tie when the oracle's two
    best keys are closer than 1e-5 (either winner is right there)."""
    import numpy as np
    from paper_2504_15475_b200 import binding
    out = binding.verify(inp["target"][:n_seq], inp["draft"][:n_seq], inp["seeds"][:n_seq], inp["T"],
                         temps=None if inp.get("temps") is None else inp["temps"][:n_seq].contiguous(),
                         parent=inp.get("parent"), want_rows=True)
    ttok = out["target_tok"].cpu().numpy()
    gap = ref["target_key"][..., 1] - ref["target_key"][..., 0]
    differ = ttok != ref["target_tok"]
    acc_same = out["accept_len"].cpu().numpy() == ref["accept_len"]
    tok_same = (out["tokens"].cpu().numpy() == ref["tokens"]).all(axis=1)
    key_err = float(np.abs(out["target_key"].cpu().numpy()[~differ] - ref["target_key"][..., 0][~differ]).max())
    return {"sequences_checked": int(n_seq), "target_rows_checked": int(ttok.size),
            "oracle_near_tie_rows": int((gap < 1e-5).sum()),
            "winner_mismatches": int(differ.sum()),
            "winner_mismatches_outside_near_ties": int((differ & ~(gap < 1e-5)).sum()),
            "sequences_with_other_accept_len_or_tokens": int((~(acc_same & tok_same)).sum()),
            "max_winner_key_error": key_err}


def run_reference(args, w):
    """The oracle as the reference arm: rank 0 only, bounded sample per step."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    import oracle
    from paper_2504_15475_b200 import workloads as wl
    n_seq = max(1, min(w.B, args.ref_seqs))
    inp = wl.make_inputs(wl.scaled(w, B=n_seq), call=0)
    for _ in range(args.warmup):
        oracle_rate(w, inp, n_seq)
    t0 = time.perf_counter()
    for _ in range(args.steps):
        oracle_rate(w, inp, n_seq)
    dt = (time.perf_counter() - t0) / args.steps
    value = n_seq * w.rows_target / dt
    sample = "%d of %d sequences of %s per step (%d logit rows)" % (n_seq, w.B, w.name,
                                                                     n_seq * (w.rows_target + w.k))
    print(json.dumps({
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": dt * 1e3, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": workload_config(w, "oracle sample"),
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": oracle.max_threads(), "kind": "oracle",
                         "sample": sample},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0}))


L2_BYTES = 126e6


def l2_note(bytes_per_launch, n_sets):
    """How the timed launches relate to the L2: what the timing rules ask a bench line to say."""
    mb = bytes_per_launch / 1e6
    if bytes_per_launch > L2_BYTES:
        return "inputs larger than L2 (%.0f MB per launch); %d input sets rotated" % (mb, n_sets)
    if bytes_per_launch * n_sets > L2_BYTES:
        return ("one input set (%.1f MB) fits the L2, the %d sets rotated between launches together do not"
                % (mb, n_sets))
    return ("inputs fit the L2 (%.2f MB per launch, %d sets): a latency figure, not an HBM one; "
            "pass --sets N for more sets than the L2 holds" % (mb, n_sets))


def workload_config(w, l2_note):
    return {"workload": "%s: B=%d k=%d V=%d %s %s" % (w.name, w.B, w.k, w.V, w.dtype,
                                                     "tree" if w.is_tree else "sequence"),
            "B": w.B, "k": w.k, "V": w.V, "rows_per_step": w.B * w.rows_target,
            "l2": l2_note, "parallelism": "replicas only (no exchange step)"}


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=1000)
    ap.add_argument("--warmup", type=int, default=10)
    ap.add_argument("--workload", default="c5")
    ap.add_argument("--entry", default="verify", choices=["verify", "tokens", "gsd"],
                    help="verify: ersd_verify / ersd_verify_tree (the headline path); tokens: "
                         "ersd_verify_tokens on tokens drafted before the timed region; gsd: the "
                         "comparison verifier ersd_gsd_verify (Algorithm 1) on tokens drafted before it")
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--sets", type=int, default=3, help="distinct input sets rotated between launches")
    ap.add_argument("--e2e-steps", type=int, default=4)
    ap.add_argument("--ref-seqs", type=int, default=64, help="sequences per oracle step (reference arm)")
    ap.add_argument("--cpu-seqs", type=int, default=0, help="sequences of the oracle sample (cpu_baseline); 0 = all")
    ap.add_argument("--cpu-passes", type=int, default=8, help="passes of the oracle over its sample (cpu_baseline)")
    ap.add_argument("--split", type=int, default=0, help="thread blocks per row (0: library default)")
    ap.add_argument("--threads", type=int, default=0, help="threads per block of the kernel (0: library default)")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--sigma", type=float, default=None)
    ap.add_argument("--temperature", type=float, default=None)
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3)

    from paper_2504_15475_b200 import workloads as wl
    w = wl.CONFIGS[args.workload]
    if args.impl == "reference":
        run_reference(args, w)
        return

    import torch
    from paper_2504_15475_b200 import binding, replicas
    binding.lib()  # fail loudly if the CUDA library is missing
    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device (no CPU fallback)")
    torch.cuda.set_device(local_rank)
    dist = None
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=torch.device("cuda", local_rank))

    # ---- inputs: resident in HBM before the timed region; every rank has its own replica
    sets = []
    for s in range(max(1, args.sets)):
        sets.append(wl.make_inputs(w, call=replicas.replica_call_index(rank, s), device="cuda", sigma=args.sigma,
                                   T=args.temperature))
    D = w.k if not w.is_tree else binding.ersd_tree_depth(w.parent)
    tokens = torch.empty(w.B, D + 1, dtype=torch.int32, device="cuda")
    accept = torch.empty(w.B, dtype=torch.int32, device="cuda")
    stream = torch.cuda.current_stream()

    def opts_for(inp):
        kw = dict(split_v=args.split, block_threads=args.threads)
        if inp.get("temps") is not None:
            kw.update(temps=inp["temps"], temp_strides=(inp["temps"].stride(0), inp["temps"].stride(1)))
        return binding.make_opts(**kw)

    all_opts = [opts_for(inp) for inp in sets]

    drafted = None
    if args.entry in ("tokens", "gsd"):
        if w.is_tree:
            raise SystemExit("--entry %s takes a sequence workload" % args.entry)
        drafted = []
        for inp, o in zip(sets, all_opts):     # drafting happens before the timed region
            d = torch.empty(w.B, w.k, 1, dtype=torch.int32, device="cuda")
            kw = {}
            if inp.get("temps") is not None:
                t_d = inp["temps"][:, :w.k].contiguous()
                kw = dict(temps=t_d, temp_strides=(t_d.stride(0), t_d.stride(1)))
                inp["temps_draft"] = t_d
            binding.ersd_race_sample(inp["draft"], inp["seeds"], inp["T"], d, binding.make_opts(**kw), stream)
            drafted.append(d[..., 0].contiguous())
        torch.cuda.synchronize()

    def step(i):
        inp = sets[i % len(sets)]
        if drafted is not None and args.entry == "gsd":
            binding.ersd_gsd_verify(inp["target"], inp["draft"], drafted[i % len(sets)], inp["seeds"], inp["T"],
                                    tokens, accept, all_opts[i % len(sets)], stream)
        elif drafted is not None:
            binding.ersd_verify_tokens(inp["target"], drafted[i % len(sets)], inp["seeds"], inp["T"], tokens,
                                       accept, all_opts[i % len(sets)], stream)
        elif w.is_tree:
            binding.ersd_verify_tree(inp["target"], inp["draft"], inp["parent"], inp["seeds"], inp["T"],
                                     tokens, accept, all_opts[i % len(sets)], stream)
        else:
            binding.ersd_verify(inp["target"], inp["draft"], inp["seeds"], inp["T"], tokens, accept,
                                all_opts[i % len(sets)], stream)

    def barrier():
        if dist is not None:
            dist.barrier()
        torch.cuda.synchronize()

    for i in range(args.warmup):
        step(i)
    barrier()
    sampler = ClockSampler(local_rank)
    sampler.start()
    time.sleep(0.25)
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    barrier()
    # profiler range = the timed region (a no-op unless a profiler asked for --profile-from-start off)
    torch.cuda.cudart().cudaProfilerStart()
    t_wall0 = time.time()
    ev0.record(stream)
    for i in range(args.steps):
        step(i)
    ev1.record(stream)
    barrier()
    t_wall1 = time.time()
    torch.cuda.cudart().cudaProfilerStop()
    clocks = sampler.stop(t_wall0, t_wall1)
    rows_per_step = w.B * w.rows_target
    value, ms_step = replicas.whole_job_rate(rows_per_step, args.steps, ev0.elapsed_time(ev1), dist, "cuda")
    launched = "ersd_gsd_verify: statistics, scan, race and merge kernels" if args.entry == "gsd" else binding.ersd_last_launch()
    mean_accept = float(accept.float().mean().item())

    # ---- roofline of the one kernel a step launches
    peak, peak_kind = load_peaks()
    alg_bytes = algorithmic_bytes(w, sets[0], args.entry)
    achieved = alg_bytes / (ms_step * 1e-3) / 1e9
    # DRAM traffic per launch from the ncu capture summarised in profiles/ (dram read + write bytes
    # over algorithmic bytes, taken on this workload); void once the kernel has changed since
    traffic = None
    if binding.ersd_version() == TRAFFIC_AT_VERSION and args.entry == "verify" and args.workload == "c5":
        traffic = DRAM_BYTES_PER_ALGORITHMIC_BYTE * alg_bytes
    # the other roof: every vocabulary index needs a quarter of a Philox4x32-10 call, 4.5 wide
    # multiplies and 4.75 three-input xors on the integer path (64 lanes per clock and SM)
    n_index = w.B * w.rows_target * w.V
    t_alu_ms = n_index * 9.25 / (64.0 * SM_COUNT * (clocks["sm_max_mhz"] or 1965.0) * 1e6) * 1e3
    t_hbm_ms = alg_bytes / (peak * 1e9) * 1e3
    roofline = {"bound": "hbm", "achieved": achieved, "peak": peak, "unit": "GB/s", "frac": achieved / peak,
                "traffic": traffic, "peak_kind": peak_kind + " copy bandwidth",
                "algorithmic_bytes_per_launch": alg_bytes, "kernel": launched,
                "kernel_ms": ms_step, "t_hbm_ms": t_hbm_ms, "t_int_ms": t_alu_ms,
                "note": "t_int_ms: Philox integer work alone at the nominal 64 int lanes/clk/SM"}
    if t_alu_ms > t_hbm_ms and args.entry != "gsd":
        # fewer bytes per index than integer work (target rows only): the integer path is the roof
        int_ops = n_index * 9.25
        peak_ops = 64.0 * SM_COUNT * (clocks["sm_max_mhz"] or 1965.0) * 1e6 / 1e9
        roofline.update(bound="alu", achieved=int_ops / (ms_step * 1e-3) / 1e9, peak=peak_ops, unit="Gop/s",
                        frac=t_alu_ms / ms_step, traffic=None,
                        peak_kind="64 integer lanes per clock and SM x 148 SMs x max SM clock")

    # ---- end to end: host buffers in pinned memory, copies inside the timed region
    e2e = None
    if not args.no_e2e and args.entry == "verify":
        h = sets[0]
        host_t = h["target"].cpu().pin_memory()
        host_d = h["draft"].cpu().pin_memory()
        host_s = h["seeds"].cpu().pin_memory()
        host_temps = None if h.get("temps") is None else h["temps"].cpu().pin_memory()
        for _ in range(2):
            binding.verify_host(host_t, host_d, host_s, h["T"], temps=host_temps, parent=h.get("parent"))
        barrier()
        t0 = time.perf_counter()
        for _ in range(args.e2e_steps):
            tok_h, acc_h = binding.verify_host(host_t, host_d, host_s, h["T"], temps=host_temps,
                                               parent=h.get("parent"))
        torch.cuda.synchronize()
        dt = (time.perf_counter() - t0) / args.e2e_steps
        dt = replicas.max_over_ranks(dt, dist, "cuda")
        h2d = sum(x.numel() * x.element_size() for x in (host_t, host_d, host_s) if x is not None)
        if host_temps is not None:
            h2d += host_temps.numel() * 4
        e2e = {"value": world * rows_per_step / dt, "unit": UNIT, "h2d_bytes_per_step": h2d,
               "d2h_bytes_per_step": tok_h.numel() * 4 + acc_h.numel() * 4, "ms_per_step": dt * 1e3,
               "steps": args.e2e_steps}

    # ---- the oracle on the host cores, on a bounded sample of the same workload (rank 0, N = 1)
    cpu, parity = None, None
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        n_seq = w.B if args.cpu_seqs <= 0 else max(1, min(w.B, args.cpu_seqs))
        t_cpu0 = time.perf_counter()
        rates = [oracle_rate(w, sets[0], n_seq) for _ in range(max(1, args.cpu_passes))]
        parity = parity_report(w, sets[0], n_seq, rates[-1][3]) if args.entry == "verify" else None
        t_cpu = time.perf_counter() - t_cpu0
        rate = statistics.median(r[0] for r in rates)
        cores = rates[0][2]
        cpu = {"value": rate, "unit": UNIT, "cores": cores, "kind": "oracle",
               "sample": "first %d of %d sequences of input set 0 (%d logit rows), median of %d passes, "
                         "%.1f s of wall time in all" % (n_seq, w.B, n_seq * (w.rows_target + w.k),
                                                         len(rates), t_cpu)}

    if rank == 0:
        print(json.dumps({
            "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": ms_step, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "f32 screen + f64 decision, u32 Philox", "data": "synthetic",
            "config": dict(workload_config(w, l2_note(alg_bytes, len(sets))),
                           entry={"tokens": "ersd_verify_tokens", "gsd": "ersd_gsd_verify"}.get(
                               args.entry, "ersd_verify_tree" if w.is_tree else "ersd_verify")),
            "clocks": clocks, "e2e": e2e, "gpu_launches": args.steps * (4 if args.entry == "gsd" else 1),
            "roofline": roofline,
            "cpu_baseline": cpu, "parity_on_cpu_sample": parity, "mean_accept_len": mean_accept}))
    if dist is not None:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
