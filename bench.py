#!/usr/bin/env python
"""Benchmark of the routed decode path: one step = one decode step of the whole
model through the cache (for every layer: append on owners, then decode
attention that reads the owner's pages), on seeded synthetic inputs of the
Llama-3-8B attention shape (32 layers, 32 q / 8 kv heads, head_dim 128, every
second layer owns, batch 32, lengths uniform in [1024, 4096], page_size 16,
random page permutation).

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl reference] [--workload NAME] [--only LEGS]

Prints ONE JSON line.  `value` is algorithmic GB/s of the whole job (bytes the
method must move: the owner layer's K,V of every attended token plus Q and out
per attention call, plus the appended rows) with inputs resident in HBM, for the
step as a decoder runs it: layer by layer through skv_append / skv_decode_attn,
each layer's query computed from the previous layer's output.  `inputs_up_front`
is skv_decode_step (all queries known before the step), `e2e` the host-buffer
entry point with the copies timed.  Every figure is the median over repeated
timed regions of `steps` steps; `spread` gives the range.
"""
from __future__ import annotations

import argparse
import json
import os
import subprocess
import sys
import threading
import time

import torch

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import workloads as W  # noqa: E402

METRIC = "decode_attn_hbm_gbs"
UNIT = "GB/s"
NOMINAL_HBM_GBS = 8000.0
FALLBACK_HBM_GBS = 6650.0
# dram__bytes_read.sum + dram__bytes_write.sum per launch of the split-K kernel of a stand-alone attention
# call (decode_cta_kernel), mean of the two launches of the ncu capture summarised in
# profiles/decode_cta_llama3_8b.md (taken on the two-layer form of the workload, which issues the same call)
NCU_TRAFFIC_BYTES = {"llama3_8b": 346880000, "llama3_8b_2layers": 346880000}
DEFAULT_L2_KEEP = 35     # the library's default share of each block range kept in L2 for the next layer


def _peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(path) as f:
            return float(json.load(f)["hbm_gbs"]), "measured"
    except Exception:
        return FALLBACK_HBM_GBS, "fallback"


class ClockSampler:
    """Samples SM clocks and throttle reasons with nvidia-smi while the timed regions run.  Every sample
    carries the host time at which it was read, so a leg can be given the median clock of its own window."""
    FIELDS = ("clocks.sm,clocks.max.sm,clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
              "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")
    NAMES = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]

    def __init__(self, index: int):
        self.index, self.rows, self.proc = index, [], None

    def __enter__(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--id={self.index}", f"--query-gpu={self.FIELDS}", "--format=csv,noheader,nounits",
                 "-lms", "25"], stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._read, daemon=True)
            self.thread.start()
        except Exception:
            self.proc = None
        return self

    def _read(self):
        for line in self.proc.stdout:
            self.rows.append((time.time(), [x.strip() for x in line.split(",")]))

    def wait_first(self, timeout_s: float = 5.0):
        """nvidia-smi needs a moment to start: wait for its first sample before the timed work begins."""
        t0 = time.time()
        while self.proc and not self.rows and time.time() - t0 < timeout_s:
            time.sleep(0.05)

    def __exit__(self, *a):
        if self.proc:
            self.proc.terminate()
            try:
                self.proc.wait(timeout=5)
            except Exception:
                self.proc.kill()
            self.thread.join(timeout=2)

    def summary(self, t0: float = 0.0, t1: float = float("inf")):
        """Median SM clock, maximum clock and the throttle reasons seen in samples read within [t0, t1]."""
        sm, mx, reasons = [], 0, set()
        for when, r in list(self.rows):
            if not (t0 <= when <= t1):
                continue
            try:
                sm.append(int(float(r[0])))
                mx = max(mx, int(float(r[1])))
            except Exception:
                continue
            for n, v in zip(self.NAMES, r[2:6]):
                if v.lower().startswith("active"):
                    reasons.add(n)
        sm.sort()
        return {"sm_mhz": sm[len(sm) // 2] if sm else None, "sm_max_mhz": mx or None,
                "reasons": sorted(reasons), "samples": len(sm)}


def _dist_env():
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    return rank, world, local


def _oracle_sample(w, dw_lens, r, n_seqs):
    """Oracle over the first n_seqs sequences of the workload, layer 1 reading its owner's store."""
    from oracle import Oracle
    layer = 1 if w.n_layers > 1 else 0
    src = r[layer]
    lens = dw_lens[:n_seqs].clone()
    o = Oracle(w.n_layers, r, w.q_heads, w.kv_heads, w.head_dim, n_seqs, int(lens.max()))
    si, pos = W.token_index(lens)
    K, V = W.draw_kv(w, src, si, pos)
    o.append(src, K, V, si, pos)
    Q = W.draw_q(w, layer, batch=n_seqs)
    nbytes = int(lens.to(torch.int64).sum()) * w.kv_heads * w.head_dim * 4 + 2 * n_seqs * w.q_heads * w.head_dim * 2
    return o, layer, Q, lens, nbytes


def run_reference(args, w):
    """The oracle as it stands, on host cores; each step is one decode-attention call over a bounded sample."""
    rank, world, _ = _dist_env()
    if rank != 0:
        return
    r = W.routing_map(w)
    lens = W.seq_lens(w)
    n_seqs = min(w.batch, args.ref_seqs)
    o, layer, Q, sl, nbytes = _oracle_sample(w, lens, r, n_seqs)
    cores = torch.get_num_threads() if False else (os.cpu_count() or 1)
    for _ in range(args.warmup):
        o.decode_attn(layer, Q, sl)
    t0 = time.perf_counter()
    for _ in range(args.steps):
        o.decode_attn(layer, Q, sl)
    dt = (time.perf_counter() - t0) / args.steps
    val = nbytes / dt / 1e9
    sample = f"1 decode-attention call (layer {layer} reading layer {r[layer]}) over the first {n_seqs} sequences ({int(sl.sum())} tokens) per step"
    print(json.dumps({
        "impl": "reference", "metric": METRIC, "value": val, "unit": UNIT, "n_gpus": args.gpus, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": dt * 1e3, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": w.name, "family": w.family, "sample": sample},
        "cpu_baseline": {"value": val, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": sample},
        "e2e": {"value": val, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }))


def rank_workload(w, rank: int, world: int):
    """Weak scaling: every rank holds its own batch of the same shape (rank-specific seed), no exchange."""
    if world <= 1:
        return w
    import dataclasses
    return dataclasses.replace(w, seed=w.seed + 1000 * rank)


def max_over_ranks(values, world: int, device):
    """Element-wise maximum of a list of floats over all ranks (identity for one rank)."""
    if world <= 1:
        return [float(v) for v in values]
    import torch.distributed as dist
    t = torch.tensor(list(values), dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return [float(v) for v in t]


def whole_job_rate(units_per_rank_per_step: float, steps: int, ms_max_over_ranks: float, world: int) -> float:
    """Units all ranks processed divided by the slowest rank's time (units per second)."""
    return world * units_per_rank_per_step * steps / (ms_max_over_ranks * 1e-3)


def median(xs):
    xs = sorted(xs)
    n = len(xs)
    return xs[n // 2] if n % 2 else 0.5 * (xs[n // 2 - 1] + xs[n // 2])


class Timer:
    """Times `fn` as repeated regions of args.steps calls each (CUDA events on the current stream, a barrier
    and a device synchronize on both sides of every region, maximum over ranks per region) until the regions
    add up to about `min_total_ms` of GPU work, and keeps the median region."""

    def __init__(self, args, world, dev, clocks, min_total_ms=1000.0, min_regions=5, max_regions=60):
        self.args, self.world, self.dev, self.clocks = args, world, dev, clocks
        self.min_total_ms, self.min_regions, self.max_regions = min_total_ms, min_regions, max_regions

    def barrier(self):
        if self.world > 1:
            import torch.distributed as dist
            dist.barrier()
        torch.cuda.synchronize(self.dev)

    def region(self, fn):
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        self.barrier()
        e0.record()
        for _ in range(self.args.steps):
            fn()
        e1.record()
        self.barrier()
        return max_over_ranks([e0.elapsed_time(e1)], self.world, self.dev)[0]

    def __call__(self, fn):
        for _ in range(self.args.warmup):
            fn()
        t0 = time.time()
        regions = [self.region(fn)]
        want = int(self.min_total_ms / max(regions[0], 1e-3)) + 1
        want = max(self.min_regions, min(self.max_regions, want))
        while len(regions) < want:
            regions.append(self.region(fn))
        t1 = time.time()
        clk = self.clocks.summary(t0, t1)
        return {"ms": median(regions), "ms_min": min(regions), "ms_max": max(regions), "regions": len(regions),
                "sm_mhz": clk["sm_mhz"], "reasons": clk["reasons"]}


def spread_of(leg, steps):
    return {"regions": leg["regions"], "ms_per_step_min": leg["ms_min"] / steps, "ms_per_step_max": leg["ms_max"] / steps,
            "sm_mhz": leg["sm_mhz"]}


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="skv", choices=["skv", "reference"])
    ap.add_argument("--workload", default="llama3_8b")
    ap.add_argument("--ref-seqs", type=int, default=32, help="sequences in the oracle's bounded sample")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--variant", type=int, default=0)
    ap.add_argument("--tuning", default="", help="warps,stages,ctas_per_sm of the split-K kernel")
    ap.add_argument("--overlap", type=int, default=-1, help="1 = overlappable (chained) launches, 0 = plain launches")
    ap.add_argument("--l2-keep", type=int, default=-1, help="percent of each block range kept in L2 for the next layer")
    ap.add_argument("--worker", default="", help="mode[,consumers,stages] of skv_set_decode_worker")
    ap.add_argument("--early-fetch", type=int, default=1, help="per-layer legs: split-K launches fill their rings "
                    "before waiting for the kernel before them (legal in a decoder, see skv_set_decode_early_fetch)")
    ap.add_argument("--fp8", action="store_true", help="run the main legs on FP8 pages (profiling the FP8 kernel); "
                    "the byte counts are then those of the FP8 cache")
    ap.add_argument("--no-sweep", action="store_true", help="skip the sharing-ratio sweep (owner fractions 1, 1/2, 1/4, 1/8)")
    ap.add_argument("--only", default="", help="comma-separated legs to run beside the headline leg "
                    "(up_front, roofline, single_call, e2e, sweep, prefill, fp8, small_batch); default: all")
    ap.add_argument("--batch", type=int, default=0, help="another number of sequences for the workload (a probe, not the benchmark)")
    ap.add_argument("--merge", type=int, default=-1, help="skv_set_decode_merge: 0 auto, 1 merge kernel, 2 inside the split-K kernel")
    ap.add_argument("--graph", type=int, default=1, help="1: the per-layer loop is captured into a CUDA graph and "
                    "replayed (GPU-bound timing); 0: issued from Python every step")
    ap.add_argument("--region-ms", type=float, default=1000.0, help="GPU work per leg over which the median is taken")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3)
    w = W.get_workload(args.workload)
    if args.batch > 0:
        import dataclasses
        w = dataclasses.replace(w, name=f"{w.name}_b{args.batch}", batch=args.batch)
    if args.impl == "reference":
        return run_reference(args, w)
    only = set(x for x in args.only.split(",") if x)
    if args.no_sweep:
        only = (only or {"up_front", "roofline", "single_call", "e2e", "prefill", "fp8", "small_batch"}) - {"sweep"}

    def wanted(leg):
        return not only or leg in only

    rank, world, local = _dist_env()
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the CUDA library is the product, there is no CPU fallback")
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=dev)

    from paper_2604_22782_b200 import harness
    w = rank_workload(w, rank, world)
    dw = harness.setup(w, device=dev, fp8=args.fp8)
    dw.retune(variant=args.variant or None,
              tuning=[int(x) for x in args.tuning.split(",")] if args.tuning else None,
              overlap=args.overlap if args.overlap >= 0 else None,
              l2_keep=args.l2_keep if args.l2_keep >= 0 else None,
              worker=tuple(int(x) for x in args.worker.split(",")) if args.worker else None,
              merge=args.merge if args.merge >= 0 else None)
    l2_keep = args.l2_keep if args.l2_keep >= 0 else DEFAULT_L2_KEEP
    harness.prefill(dw, upto_offset=-1)
    t = harness.step_tensors(dw)
    L, n_own = w.n_layers, len(dw.owners)
    attn_bytes = dw.kv_bytes_per_call()
    step_bytes = L * attn_bytes + n_own * dw.append_bytes_per_call()
    cache = dw.cache

    step_per_layer, step_without_attention, step_up_front = make_steps(dw, t)
    step_coop = make_steps(dw, t, query_kernel=cooperating_query_kernel())[0] if wanted("roofline") else None

    with ClockSampler(local) as clocks:
        clocks.wait_first()
        timer = Timer(args, world, dev, clocks, min_total_ms=args.region_ms)
        # (1) the headline: the per-layer loop under the method's data dependence, library defaults plus early fetch
        t["out"].zero_()
        dw.retune(early_fetch=args.early_fetch)
        launches0 = cache.skv_launch_count()
        step_per_layer()
        launches = cache.skv_launch_count() - launches0
        torch.cuda.synchronize(dev)
        out_eager = t["out"].clone()
        if args.graph:
            run_main, how_main, graph_main = as_graph(step_per_layer, dev)
        else:
            run_main, how_main, graph_main = step_per_layer, "eager", None
        leg_main = timer(run_main)
        torch.cuda.synchronize(dev)
        out_per_layer = t["out"].clone()
        if not torch.equal(out_eager.view(torch.int16), out_per_layer.view(torch.int16)):
            raise SystemExit("graph replay and plain launches of the per-layer loop disagree")
        # (2) the roofline leg: the same loop with L2 reuse between layers off, so that every attention
        # launch streams all of its pages from HBM; and the loop without its attention calls, to show what
        # the query kernel and the updates cost inside it
        def leg_of(fn):
            run, _, keep_alive = as_graph(fn, dev) if args.graph else (fn, "eager", None)
            res = timer(run)
            del keep_alive
            return res

        dw.retune(l2_keep=0)
        leg_hbm = leg_of(step_per_layer)
        leg_rest = leg_of(step_without_attention)
        dw.retune(l2_keep=l2_keep, early_fetch=0)
        leg_wait_first = leg_of(step_per_layer) if wanted("roofline") else None
        leg_eager = timer(step_per_layer) if (wanted("roofline") and args.graph) else None
        dw.retune(early_fetch=args.early_fetch)
        # the same loop when the caller's query kernel takes part in programmatic launches (the stand-in from
        # the test-hook library): the next layer's attention kernel then moves in while this layer's drains
        leg_coop = leg_coop_hbm = None
        if step_coop is not None and args.early_fetch:
            leg_coop = leg_of(step_coop)
            torch.cuda.synchronize(dev)
            if not torch.equal(t["out"].view(torch.int16), out_per_layer.view(torch.int16)):
                close = ((t["out"].float() - out_per_layer.float()).abs() <= 1e-2 + 1e-2 * out_per_layer.float().abs()).all()
                if not bool(close):
                    raise SystemExit("the per-layer loop with the cooperating query kernel disagrees")
            dw.retune(l2_keep=0)
            leg_coop_hbm = leg_of(step_coop)
            dw.retune(l2_keep=l2_keep)

        # (3) whole steps with every layer's query given up front (skv_decode_step): the library then chains
        # the attention launches so that layer l+1 streams while layer l drains -- an overlap a decoder's own
        # data flow does not offer; reported for comparison only
        leg_up = leg_up_hbm = None
        if wanted("up_front"):
            leg_up = timer(step_up_front)
            torch.cuda.synchronize(dev)
            if not torch.equal(t["out"].view(torch.int16), out_per_layer.view(torch.int16)):
                close = ((t["out"].float() - out_per_layer.float()).abs() <= 1e-2 + 1e-2 * out_per_layer.float().abs()).all()
                if not bool(close):
                    raise SystemExit("per-layer loop and skv_decode_step disagree")
            dw.retune(l2_keep=0)
            leg_up_hbm = timer(step_up_front)
            dw.retune(l2_keep=l2_keep)

        # (4) one attention call at a time between two events (nothing before it to overlap with)
        call_ms_owner = call_ms_reader = None
        if wanted("single_call"):
            pairs = []
            for _ in range(max(2, args.steps // 4)):
                for l in range(L):
                    if dw.r[l] == l:
                        i = dw.owners.index(l)
                        cache.skv_append(l, t["K"][i], t["V"][i], dw.slot_new)
                    a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                    a.record()
                    cache.skv_decode_attn(l, t["Q"][l], dw.page_table, dw.seq_lens, t["out"][l], dw.workspace)
                    b.record()
                    pairs.append((l, a, b))
            torch.cuda.synchronize(dev)
            per = [(l, a.elapsed_time(b)) for l, a, b in pairs[L:]]
            own = [x for l, x in per if dw.r[l] == l]
            non = [x for l, x in per if dw.r[l] != l]
            call_ms_owner = median(own)
            call_ms_reader = median(non) if non else None

        # (5) end to end: host buffers in, host buffer out, copies inside the timed region
        leg_e2e = None
        hb = harness.step_tensors(dw, device="cpu", pin=True)
        h_slot = dw.slot_new.cpu().pin_memory()
        h_pt = dw.page_table_cpu.contiguous().pin_memory()
        h_len = dw.lens_cpu.contiguous().pin_memory()
        if wanted("e2e"):
            staging = torch.empty(cache.skv_decode_step_staging_bytes(dw.batch, w.q_heads, h_pt.shape[1]),
                                  dtype=torch.uint8, device=dev)

            def step_host():
                cache.skv_decode_step_host(hb["Q"], hb["K"], hb["V"], h_slot, h_pt, h_len, hb["out"], staging)

            leg_e2e = timer(step_host)
            torch.cuda.synchronize(dev)
            ref16, got = out_per_layer.cpu().float(), hb["out"].float()
            if not bool(((got - ref16).abs() <= 1e-2 + 1e-2 * ref16.abs()).all()):
                raise SystemExit("host-buffer step and per-layer loop disagree")
            del staging
        all_clocks = clocks.summary()
    status = cache.skv_get_status()
    if status != 0:
        raise SystemExit(f"device status {status}")
    if rank != 0:
        return

    peak, peak_kind = _peaks()
    K = args.steps
    value = whole_job_rate(step_bytes, K, leg_main["ms"], world) / 1e9
    us_per_launch = leg_hbm["ms"] * 1e3 / (K * L)
    achieved = attn_bytes / (us_per_launch * 1e-6) / 1e9
    us_rest = leg_rest["ms"] * 1e3 / (K * L)
    h2d = sum(hb[k].numel() * 2 for k in ("Q", "K", "V")) + h_slot.numel() * 8 + h_pt.numel() * 4 + h_len.numel() * 4
    d2h = hb["out"].numel() * 2

    def call_fig(leg):
        us = leg["ms"] * 1e3 / (K * L)
        g = attn_bytes / (us * 1e-6) / 1e9
        return {"us_per_call": us, "gbs": g, "frac": g / peak, "frac_of_nominal_8TBs": g / NOMINAL_HBM_GBS,
                **spread_of(leg, K)}

    worker_mode = int(args.worker.split(",")[0]) if args.worker else 0
    kernel_name = ("decode_fp8_umma_kernel" if (args.fp8 and w.head_dim == 128 and args.variant != 2)
                   else "decode_splitk_kernel" if worker_mode == 1 else "decode_cta_kernel")
    line = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": K, "warmup": args.warmup,
        "ms_per_step": leg_main["ms"] / K, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "e4m3 pages" if args.fp8 else "bf16", "data": "synthetic",
        "config": {"workload": w.name, "family": w.family, "n_layers": L, "owners": n_own, "batch": dw.batch,
                   "tokens": int(dw.lens_cpu.sum()), "q_heads": w.q_heads, "kv_heads": w.kv_heads,
                   "head_dim": w.head_dim, "page_size": w.page_size, "early_fetch": args.early_fetch, "l2_keep": l2_keep,
                   "l2": ("inputs larger than L2: every attention call streams %.0f MB of pages" % (attn_bytes / 1e6))
                         if attn_bytes > 126e6 else
                         ("a call's pages (%.2f MB) fit the L2 cache and are not flushed between calls: a small case, "
                          "not a bandwidth figure" % (attn_bytes / 1e6)),
                   "step": "per layer: query kernel (reads the previous layer's output), skv_append on owners, "
                           "skv_decode_attn (split-K + merge); one stream, no events inside",
                   "value_is": "algorithmic GB/s (bytes the method must move / time), not DRAM traffic: with L2 reuse "
                               "on, part of a reader layer's bytes come from L2",
                   "launch": how_main,
                   "timing": "median over repeated regions of `steps` steps each"},
        "spread": spread_of(leg_main, K),
        "steps_per_s": world * K / (leg_main["ms"] * 1e-3),
        "attn_calls_per_s": world * L * K / (leg_main["ms"] * 1e-3),
        "frac_of_nominal_8TBs": value / world / NOMINAL_HBM_GBS,
        "clocks": all_clocks,
        "gpu_launches": int(launches) * K,
        "roofline": {"bound": "hbm", "kernel": kernel_name, "achieved": achieved, "peak": peak,
                     "peak_kind": peak_kind, "unit": "GB/s", "frac": achieved / peak,
                     "frac_of_nominal_8TBs": achieved / NOMINAL_HBM_GBS, "us_per_launch": us_per_launch,
                     "bytes_per_launch": attn_bytes,
                     "how": "the per-layer loop with L2 reuse between layers off; region time / split-K launches in it, "
                            "so the query kernel, the updates and the merge launches are charged to it",
                     "us_per_launch_minus_rest": us_per_launch - us_rest,
                     "us_query_kernel_and_update_per_layer": us_rest,
                     "traffic": NCU_TRAFFIC_BYTES.get(w.name) if kernel_name == "decode_cta_kernel" else None,
                     "traffic_from": "committed ncu profile (profiles/), not this run",
                     **spread_of(leg_hbm, K)},
        "per_layer_api": {"early_fetch_on": call_fig(leg_main) if args.early_fetch else None,
                          "early_fetch_on_l2_reuse_off": call_fig(leg_hbm) if args.early_fetch else None,
                          "early_fetch_off": call_fig(leg_wait_first) if leg_wait_first else None,
                          "early_fetch_off_issued_from_python": call_fig(leg_eager) if leg_eager else None,
                          "cooperating_query_kernel": {
                              **call_fig(leg_coop), "l2_reuse_off": call_fig(leg_coop_hbm),
                              "how": "early fetch on; the caller's query kernel is launched with the programmatic "
                                     "attribute, releases its dependents first and then waits (test-hook stand-in "
                                     "for a decoder's own kernel): not the headline, which keeps a kernel that "
                                     "knows nothing of programmatic launches"} if leg_coop else None,
                          "launch": how_main,
                          "how": "region time / attention calls in it; Q of every layer depends on the previous layer's output"},
    }
    if leg_e2e:
        line["e2e"] = {"value": whole_job_rate(step_bytes, K, leg_e2e["ms"], world) / 1e9, "unit": UNIT,
                       "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h, "ms_per_step": leg_e2e["ms"] / K,
                       "how": "skv_decode_step_host: pinned host buffers in and out, all copies timed; the step's "
                              "queries are host inputs, so they exist up front by the nature of the call",
                       **spread_of(leg_e2e, K)}
    if leg_up:
        line["inputs_up_front"] = {
            "value": whole_job_rate(step_bytes, K, leg_up["ms"], world) / 1e9, "unit": UNIT,
            "ms_per_step": leg_up["ms"] / K, "l2_reuse_off": call_fig(leg_up_hbm), **spread_of(leg_up, K),
            "how": "skv_decode_step with all layers' queries given before the step: chained launches overlap "
                   "consecutive layers; not available to a decoder, whose next query depends on this output"}
    if call_ms_owner is not None:
        line["single_call"] = {"us_owner_layers": call_ms_owner * 1e3,
                               "us_reader_layers": None if call_ms_reader is None else call_ms_reader * 1e3,
                               "gbs_owner_layers": attn_bytes / (call_ms_owner * 1e-3) / 1e9,
                               "how": "skv_decode_attn (split-K + merge) alone between two events (median); "
                                      "includes what an event pair itself costs"}
    if not args.no_cpu_baseline and world == 1:
        line["cpu_baseline"] = cpu_baseline(args, w, dw)
    if world == 1:
        del dw, cache, t, hb, step_per_layer, step_without_attention, step_up_front
        torch.cuda.empty_cache()
        if wanted("sweep") and not args.fp8:
            line["sharing_sweep"] = sharing_sweep(args, dev)
        if wanted("small_batch") and not args.fp8:
            line["small_batch_l2"] = small_batch_leg(args, dev)
        if wanted("prefill") and not args.fp8:
            line["prefill"] = prefill_leg(args, dev)
        if wanted("fp8") and not args.fp8:
            line["fp8_pages"] = fp8_leg(args, dev)
    print(json.dumps(line))
    if world > 1:
        import torch.distributed as dist
        dist.destroy_process_group()


def cooperating_query_kernel():
    """The stand-in for a decoder's own query kernel that takes part in programmatic launches
    (include/skv_test_hooks.h): a function (q_in, prev_out, q_out) that launches it on the current stream."""
    import ctypes
    from paper_2604_22782_b200 import build
    lib = ctypes.CDLL(build.build_test_hooks())
    fn = lib.skv_test_query_kernel
    fn.restype = ctypes.c_int
    fn.argtypes = [ctypes.c_void_p, ctypes.c_void_p, ctypes.c_void_p, ctypes.c_longlong, ctypes.c_void_p]

    def launch(q_in, prev_out, q_out):
        rc = fn(q_in.data_ptr(), prev_out.data_ptr(), q_out.data_ptr(), q_in.numel(),
                torch.cuda.current_stream().cuda_stream)
        if rc != 0:
            raise SystemExit(f"skv_test_query_kernel: {rc}")
    return launch


def make_steps(dw, t, query_kernel=None):
    """The decode step three ways.  (1) As a decoder runs it (Algorithm 2): layer by layer through the
    per-layer entry points, the query of layer l computed FROM THE OUTPUT of layer l-1 (of the last layer of
    the previous step for layer 0) by a kernel of the caller's, here an element-wise torch kernel, so that
    no attention call can read its query before the call before it has finished; one stream, no events
    inside.  (2) The same loop without its attention calls.  (3) skv_decode_step, which is given every
    layer's query before the step starts."""
    cache, L = dw.cache, dw.w.n_layers
    q_in = [t["Q"][l] for l in range(L)]
    q_dep = [torch.empty_like(t["Q"][l]) for l in range(L)]
    outs = [t["out"][l] for l in range(L)]
    kv_of = {l: (t["K"][i], t["V"][i]) for i, l in enumerate(dw.owners)}
    if query_kernel is None:
        def query_kernel(a, prev, out):
            torch.add(a, prev, alpha=0.0, out=out)

    def step_per_layer():
        for l in range(L):
            query_kernel(q_in[l], outs[l - 1], q_dep[l])                    # "Compute Query Q_l"
            if l in kv_of:
                cache.skv_append(l, kv_of[l][0], kv_of[l][1], dw.slot_new)  # "Update" (owners only)
            cache.skv_decode_attn(l, q_dep[l], dw.page_table, dw.seq_lens, outs[l], dw.workspace)   # "Load + Attn"

    def step_without_attention():
        for l in range(L):
            query_kernel(q_in[l], outs[l - 1], q_dep[l])
            if l in kv_of:
                cache.skv_append(l, kv_of[l][0], kv_of[l][1], dw.slot_new)

    def step_up_front():
        cache.skv_decode_step(t["Q"], t["K"], t["V"], dw.slot_new, dw.page_table, dw.seq_lens, t["out"], dw.workspace)

    return step_per_layer, step_without_attention, step_up_front


def as_graph(fn, dev):
    """fn captured once into a CUDA graph (its kernels, with the programmatic launch dependencies between
    them, on one capture stream) and a function that replays it: what is then timed is the GPU's work on
    the step, not Python issuing ~100 launches per step.  Returns (replay, "cuda graph replay"), or
    (fn, "eager: ...") when the capture is refused."""
    try:
        side = torch.cuda.Stream(device=dev)
        side.wait_stream(torch.cuda.current_stream(dev))
        with torch.cuda.stream(side):
            fn()
            fn()
        torch.cuda.current_stream(dev).wait_stream(side)
        torch.cuda.synchronize(dev)
        g = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g, stream=side):
            fn()
        torch.cuda.synchronize(dev)
        return g.replay, "cuda graph replay", g
    except Exception as e:          # noqa: BLE001  (report, fall back to plain launches)
        torch.cuda.synchronize(dev)
        return fn, f"eager: {type(e).__name__}: {e}"[:200], None


def simple_time(fn, dev, warmup, n):
    """Milliseconds per call of fn: `warmup` untimed calls, then n calls between two events."""
    for _ in range(warmup):
        fn()
    torch.cuda.synchronize(dev)
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(n):
        fn()
    e1.record()
    torch.cuda.synchronize(dev)
    return e0.elapsed_time(e1) / n


def small_batch_leg(args, dev):
    """Table 4's shape (Section 4.3): Qwen3-8B heads, groups of four layers, one sequence of 2 048 / 8 192
    prompt tokens (+128 generated).  An owner layer's K,V (8.9 / 34.1 MB) fit in the L2 cache, so the
    three reader layers of a group can take them from there (the paper's suggestion for a backend: keep
    the shared K,V on chip across consecutive layers).  The per-layer loop under the data dependence of
    a decoder, with the library's L2 reuse on and off."""
    from paper_2604_22782_b200 import harness
    rows = []
    for name in ("qwen3_8b_b1_2k", "qwen3_8b_b1_8k"):
        w = W.get_workload(name)
        dw = harness.setup(w, device=dev)
        harness.prefill(dw, upto_offset=-1)
        t = harness.step_tensors(dw)
        dw.retune(early_fetch=args.early_fetch)
        step_per_layer, step_rest, _ = make_steps(dw, t)
        n = max(20, args.steps * 5)
        row = {"workload": name, "tokens": int(dw.lens_cpu.sum()), "bytes_per_owner_layer": dw.kv_bytes_per_call()}
        for keep, key in ((DEFAULT_L2_KEEP, "l2_reuse_on"), (0, "l2_reuse_off")):
            dw.retune(l2_keep=keep)
            run, how, keep_alive = as_graph(step_per_layer, dev) if args.graph else (step_per_layer, "eager", None)
            ms = simple_time(run, dev, args.warmup, n)
            us = ms * 1e3 / w.n_layers
            row[key] = {"us_per_call": us, "algorithmic_gbs": dw.kv_bytes_per_call() / (us * 1e-6) / 1e9, "launch": how}
            del run, keep_alive
        run, how, keep_alive = as_graph(step_rest, dev) if args.graph else (step_rest, "eager", None)
        row["us_query_kernel_and_update_per_layer"] = simple_time(run, dev, args.warmup, n) * 1e3 / w.n_layers
        del run, keep_alive
        if dw.cache.skv_get_status() != 0:
            raise SystemExit("device status after the small-batch leg")
        rows.append(row)
        del dw, t, step_per_layer, step_rest
        torch.cuda.empty_cache()
    return rows


def cpu_baseline(args, w, dw):
    """The oracle as it stands on the host cores: one decode-attention call over the first --ref-seqs
    sequences of the workload, best of 3; for a larger batch also the linear extrapolation in tokens
    (the oracle's work is exactly linear in the number of attended tokens)."""
    n_seqs = min(w.batch, args.ref_seqs)
    o, layer, Q, sl, nbytes = _oracle_sample(w, dw.lens_cpu, dw.r, n_seqs)
    best = float("inf")
    for _ in range(3):
        t0 = time.perf_counter()
        o.decode_attn(layer, Q, sl)
        best = min(best, time.perf_counter() - t0)
    tokens, all_tokens = int(sl.sum()), int(dw.lens_cpu.sum())
    res = {"value": nbytes / best / 1e9, "unit": UNIT, "cores": os.cpu_count() or 1, "kind": "oracle",
           "sample": f"1 decode-attention call (layer {layer} reading layer {dw.r[layer]}) over the first {n_seqs} "
                     f"sequences ({tokens} tokens), best of 3, {best * 1e3:.1f} ms",
           "ms_per_call_sample": best * 1e3}
    if n_seqs < w.batch:
        res["ms_per_call_full_batch_extrapolated"] = best * 1e3 * all_tokens / max(tokens, 1)
        res["extrapolation"] = f"linear in attended tokens: {tokens} measured -> {all_tokens} in the full batch"
    return res


def prefill_leg(args, dev):
    """Pre-fill (the phase before decoding): Llama-3-8B head shape, 8 prompts of 4096 tokens.  Times the
    multi-token update of the owner layer and the causal attention of all prompt tokens over the routed
    owner's pages (layer 1 reads layer 0), for the tcgen05 kernel and the mma.sync kernel.  A dense
    contraction: the bound is the tensor core, flops = 4 * q_heads * head_dim * sum over rows of (pos + 1)."""
    from paper_2604_22782_b200 import harness
    B, T = 8, 4096
    w = W.Workload("prefill_llama3_8b", 2, 32, 8, 128, 16, B, T, T, "groups", group=2, seed=1, family="Llama-3-8B")
    lens = torch.full((B,), T, dtype=torch.int32)
    dw = harness.setup(w, device=dev, lens=lens)
    seq_idx, pos = W.token_index(lens)
    slots = W.slot_map_for(dw.page_table_cpu, seq_idx, pos, w.page_size).to(dev)
    K, V = W.draw_kv(w, 0, seq_idx, pos, device=dev)
    n_rep = max(3, args.steps // 2)

    def timed(fn):
        for _ in range(args.warmup):
            fn()
        torch.cuda.synchronize(dev)
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for _ in range(n_rep):
            fn()
        e1.record()
        torch.cuda.synchronize(dev)
        return e0.elapsed_time(e1) / n_rep

    ms_append = timed(lambda: dw.cache.skv_append(0, K, V, slots))
    inp = harness.prefill_inputs(dw, 1, lens)
    out = torch.empty_like(inp["Q"])
    flops = 4.0 * w.q_heads * w.head_dim * B * (T * (T + 1) / 2)
    res = {"workload": w.name, "batch": B, "prompt_tokens": T, "flops_per_call": flops,
           "append_ms": ms_append, "append_gbs": 2 * K.numel() * 2 * 2 / (ms_append * 1e-3) / 1e9}
    try:
        with open(os.path.join(ROOT, "MEASURED_PEAKS.json")) as f:
            peak = float(json.load(f)["bf16_tflops"])
            peak_kind = "measured"
    except Exception:
        peak, peak_kind = 1590.0, "fallback"
    for variant, name in ((2, "tcgen05"), (1, "mma_sync")):
        dw.cache.skv_set_prefill_variant(variant)
        ms = timed(lambda: dw.cache.skv_prefill_attn(1, inp["Q"], inp["cu_q_lens"], dw.page_table, dw.seq_lens, out, T))
        res[name] = {"ms_per_call": ms, "tflops": flops / (ms * 1e-3) / 1e12,
                     "tokens_per_s": B * T / (ms * 1e-3)}
    res["roofline"] = {"bound": "tensor", "kernel": "prefill_umma_kernel", "achieved": res["tcgen05"]["tflops"],
                       "peak": peak, "peak_kind": peak_kind, "unit": "TFLOP/s",
                       "frac": res["tcgen05"]["tflops"] / peak}
    if dw.cache.skv_get_status() != 0:
        raise SystemExit("device status after the pre-fill leg")
    # the same prompts on FP8 pages: quantising append and the mma.sync kernel that converts the codes on the way in
    del dw
    torch.cuda.empty_cache()
    dq = harness.setup(w, device=dev, lens=lens, fp8=True)
    ms_append8 = timed(lambda: dq.cache.skv_append(0, K, V, slots))
    st8 = dq.cache.skv_cache_stats()
    ms8 = timed(lambda: dq.cache.skv_prefill_attn(1, inp["Q"], inp["cu_q_lens"], dq.page_table, dq.seq_lens, out, T))
    res["fp8_pages"] = {"append_ms": ms_append8,
                        "append_gbs": (K.numel() * 2 * 2 + st8["page_bytes"] * dq.total_pages) / (ms_append8 * 1e-3) / 1e9,
                        "mma_sync": {"ms_per_call": ms8, "tflops": flops / (ms8 * 1e-3) / 1e12, "tokens_per_s": B * T / (ms8 * 1e-3)}}
    # ... and with a scratch area: the pages turned into bf16 (one more launch, timed with the call), then the tcgen05 kernel
    area = torch.empty(dq.cache.skv_prefill_scratch_bytes(), dtype=torch.uint8, device=dev)
    dq.cache.skv_set_prefill_scratch(area)
    ms8s = timed(lambda: dq.cache.skv_prefill_attn(1, inp["Q"], inp["cu_q_lens"], dq.page_table, dq.seq_lens, out, T))
    res["fp8_pages"]["tcgen05_via_bf16_scratch"] = {"ms_per_call": ms8s, "tflops": flops / (ms8s * 1e-3) / 1e12,
                                                    "tokens_per_s": B * T / (ms8s * 1e-3),
                                                    "frac_of_bf16_tcgen05": res["tcgen05"]["ms_per_call"] / ms8s}
    dq.cache.skv_set_prefill_scratch(None)
    if dq.cache.skv_get_status() != 0:
        raise SystemExit("device status after the FP8 pre-fill leg")
    return res


def fp8_leg(args, dev):
    """The benchmark's workload with FP8 pages (E4M3 codes + one fp32 scale per token and kv head): whole
    decode steps (at head_dim 128 the tcgen05 kernel that runs both contractions on the stored codes), cache bytes
    per token, and the rate in tokens attended per microsecond, to be read next to the bf16 cache's."""
    from paper_2604_22782_b200 import harness
    w = W.get_workload("llama3_8b")
    dw = harness.setup(w, device=dev, fp8=True)
    harness.prefill(dw, upto_offset=-1)
    t = harness.step_tensors(dw)
    cache = dw.cache

    step_per_layer, _, step_up_front = make_steps(dw, t)
    n = max(3, args.steps // 2)
    run, how, keep_alive = as_graph(step_per_layer, dev) if args.graph else (step_per_layer, "eager", None)
    ms_loop = simple_time(run, dev, args.warmup, n)
    ms = simple_time(step_up_front, dev, args.warmup, n)
    del run, keep_alive
    step_coop = make_steps(dw, t, query_kernel=cooperating_query_kernel())[0]
    run, _, keep_alive = as_graph(step_coop, dev) if args.graph else (step_coop, "eager", None)
    ms_coop = simple_time(run, dev, args.warmup, n)
    del run, keep_alive
    if cache.skv_get_status() != 0:
        raise SystemExit("device status after the FP8 leg")
    st = cache.skv_cache_stats()
    tokens = int(dw.lens_cpu.sum())
    return {"workload": w.name, "kv_bytes_per_token": st["bytes_per_token"],
            "per_layer_loop": {"ms_per_step": ms_loop, "us_per_attn_call": ms_loop * 1e3 / w.n_layers,
                               "attn_gbs": w.n_layers * dw.kv_bytes_per_call() / (ms_loop * 1e-3) / 1e9,
                               "tokens_attended_per_us": w.n_layers * tokens / (ms_loop * 1e3), "launch": how,
                               "us_per_attn_call_cooperating_query_kernel": ms_coop * 1e3 / w.n_layers},
            "inputs_up_front": {"ms_per_step": ms, "us_per_attn_call": ms * 1e3 / w.n_layers,
                                "attn_gbs": w.n_layers * dw.kv_bytes_per_call() / (ms * 1e-3) / 1e9,
                                "tokens_attended_per_us": w.n_layers * tokens / (ms * 1e3)}}


def sharing_sweep(args, dev):
    """Llama-3-8B shape, batch 128, lengths U[512,2048]: owner fractions 1, 1/2, 1/4, 1/8 (evenly spaced
    owners).  Per ratio: cache bytes, the largest batch a 120e9-byte KV budget holds, whole decode steps per
    second (per layer: query kernel that reads the previous layer's output, update on owners, attention -- the
    loop of make_steps, replayed as a CUDA graph) and the time per attention call; beside it the same step through
    skv_decode_step, which is given all queries up front."""
    from paper_2604_22782_b200 import harness
    rows = []
    budget = 120e9
    for g in (1, 2, 4, 8):
        w = W.sweep_workload(g)
        dw = harness.setup(w, device=dev)
        harness.prefill(dw, upto_offset=-1)
        t = harness.step_tensors(dw)
        cache = dw.cache

        dw.retune(early_fetch=args.early_fetch)
        step_per_layer, _, step_up_front = make_steps(dw, t)
        n = max(3, args.steps // 2)
        run, how, keep_alive = as_graph(step_per_layer, dev) if args.graph else (step_per_layer, "eager", None)
        ms = simple_time(run, dev, args.warmup, n)                  # the step as a decoder runs it (see make_steps)
        ms_up_front = simple_time(step_up_front, dev, args.warmup, n)
        del run, keep_alive
        # the same loop with a query kernel of the caller's that takes part in programmatic launches
        step_coop = make_steps(dw, t, query_kernel=cooperating_query_kernel())[0]
        run, _, keep_alive = as_graph(step_coop, dev) if args.graph else (step_coop, "eager", None)
        ms_coop = simple_time(run, dev, args.warmup, n)
        del run, keep_alive, step_coop
        st = cache.skv_cache_stats()
        pages = (dw.lens_cpu.to(torch.int64) + w.page_size - 1) // w.page_size
        per_seq_mean = st["n_owners"] * float(pages.double().mean()) * st["page_bytes"]
        per_seq_worst = st["n_owners"] * ((w.len_hi + w.page_size - 1) // w.page_size) * st["page_bytes"]
        tokens = int(dw.lens_cpu.sum())
        rows.append({
            "owner_fraction": 1.0 / g, "owners": st["n_owners"], "kv_bytes_per_token": st["bytes_per_token"],
            "kv_bytes_tokens": st["bytes_per_token"] * tokens, "kv_bytes_pages": st["kv_bytes"],
            "max_batch_120e9_mean_len": int(budget // per_seq_mean),
            "max_batch_120e9_max_len": int(budget // per_seq_worst),
            "ms_per_step": ms, "steps_per_s": 1e3 / ms, "us_per_attn_call": ms * 1e3 / w.n_layers,
            "attn_gbs": w.n_layers * dw.kv_bytes_per_call() / (ms * 1e-3) / 1e9, "launch": how,
            "cooperating_query_kernel": {"ms_per_step": ms_coop, "steps_per_s": 1e3 / ms_coop,
                                         "us_per_attn_call": ms_coop * 1e3 / w.n_layers,
                                         "attn_gbs": w.n_layers * dw.kv_bytes_per_call() / (ms_coop * 1e-3) / 1e9},
            "inputs_up_front": {"ms_per_step": ms_up_front, "steps_per_s": 1e3 / ms_up_front,
                                "attn_gbs": w.n_layers * dw.kv_bytes_per_call() / (ms_up_front * 1e-3) / 1e9},
        })
        if cache.skv_get_status() != 0:
            raise SystemExit("device status after the sweep")
        del dw, cache, t, step_per_layer, step_up_front
        torch.cuda.empty_cache()
    return rows


if __name__ == "__main__":
    main()
