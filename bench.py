#!/usr/bin/env python
"""Benchmark of the routed decode path: one step = one decode step of the whole
model through the cache (for every layer: append on owners, then decode
attention that reads the owner's pages), on seeded synthetic inputs of the
Llama-3-8B attention shape (32 layers, 32 q / 8 kv heads, head_dim 128, every
second layer owns, batch 32, lengths uniform in [1024, 4096], page_size 16,
random page permutation).

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl reference] [--workload NAME]

Prints ONE JSON line.  `value` is algorithmic GB/s of the whole job (bytes the
method must move: the owner layer's K,V of every attended token plus Q and out
per attention call, plus the appended rows) with inputs resident in HBM; `e2e`
is the same through the host-buffer entry point with the copies timed.
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
# dram__bytes_read.sum + dram__bytes_write.sum per launch of the split-K kernel,
# from the ncu capture summarised under profiles/ (None until captured)
NCU_TRAFFIC_BYTES = {"llama3_8b": None}


def _peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(path) as f:
            return float(json.load(f)["hbm_gbs"]), "measured"
    except Exception:
        return FALLBACK_HBM_GBS, "fallback"


class ClockSampler:
    """Samples SM clocks and throttle reasons with nvidia-smi while the timed region runs."""
    FIELDS = ("clocks.sm,clocks.max.sm,clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
              "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index, self.rows, self.proc = index, [], None

    def __enter__(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--id={self.index}", f"--query-gpu={self.FIELDS}", "--format=csv,noheader,nounits",
                 "-lms", "100"], stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._read, daemon=True)
            self.thread.start()
        except Exception:
            self.proc = None
        return self

    def _read(self):
        for line in self.proc.stdout:
            self.rows.append([x.strip() for x in line.split(",")])

    def __exit__(self, *a):
        if self.proc:
            self.proc.terminate()
            try:
                self.proc.wait(timeout=5)
            except Exception:
                self.proc.kill()
            self.thread.join(timeout=2)

    def summary(self):
        sm, mx, reasons = [], 0, set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for r in self.rows:
            try:
                sm.append(int(float(r[0])))
                mx = max(mx, int(float(r[1])))
            except Exception:
                continue
            for n, v in zip(names, r[2:6]):
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
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3)
    w = W.get_workload(args.workload)
    if args.impl == "reference":
        return run_reference(args, w)

    rank, world, local = _dist_env()
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the CUDA library is the product, there is no CPU fallback")
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=dev)

    from paper_2604_22782_b200 import harness
    # weak scaling: every rank holds its own batch of the same shape (rank-specific seed), no exchange
    if world > 1:
        import dataclasses
        w = dataclasses.replace(w, seed=w.seed + 1000 * rank)
    dw = harness.setup(w, device=dev)
    dw.retune(variant=args.variant or None,
              tuning=[int(x) for x in args.tuning.split(",")] if args.tuning else None,
              overlap=args.overlap if args.overlap >= 0 else None,
              l2_keep=args.l2_keep if args.l2_keep >= 0 else None)
    harness.prefill(dw, upto_offset=-1)
    t = harness.step_tensors(dw)
    L, n_own = w.n_layers, len(dw.owners)
    step_bytes = L * dw.kv_bytes_per_call() + n_own * dw.append_bytes_per_call()
    cache = dw.cache

    def step():
        cache.skv_decode_step(t["Q"], t["K"], t["V"], dw.slot_new, dw.page_table, dw.seq_lens, t["out"], dw.workspace)

    def barrier():
        if world > 1:
            import torch.distributed as dist
            dist.barrier()
        torch.cuda.synchronize(dev)

    for _ in range(args.warmup):
        step()
    barrier()
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    launches0 = cache.skv_launch_count()
    with ClockSampler(local) as clocks:
        barrier()
        ev0.record()
        for _ in range(args.steps):
            step()
        ev1.record()
        barrier()
        ms = ev0.elapsed_time(ev1)
        launches = cache.skv_launch_count() - launches0

        # the dominant kernel alone: the same layers through the per-layer entry points, an event pair
        # around every attention launch (events between launches also keep them from overlapping)
        pairs = []
        for _ in range(args.steps):
            for l in range(L):
                if dw.r[l] == l:
                    cache.skv_append(l, t["K"][dw.owners.index(l)], t["V"][dw.owners.index(l)], dw.slot_new)
                a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                a.record()
                cache.skv_decode_attn(l, t["Q"][l], dw.page_table, dw.seq_lens, t["out"][l], dw.workspace)
                b.record()
                pairs.append((l, a, b))
        torch.cuda.synchronize(dev)
        per = [(l, a.elapsed_time(b)) for l, a, b in pairs]
        kern_ms = sum(x for _, x in per) / len(per)
        own = [x for l, x in per if dw.r[l] == l]
        non = [x for l, x in per if dw.r[l] != l]
        kern_ms_owner = sum(own) / len(own)
        kern_ms_reader = sum(non) / len(non) if non else None

        # end to end: host buffers in, host buffer out, copies inside the timed region
        hb = harness.step_tensors(dw, device="cpu", pin=True)
        h_slot = dw.slot_new.cpu().pin_memory()
        h_pt = dw.page_table_cpu.contiguous().pin_memory()
        h_len = dw.lens_cpu.contiguous().pin_memory()
        staging = torch.empty(cache.skv_decode_step_staging_bytes(dw.batch, w.q_heads, h_pt.shape[1]),
                              dtype=torch.uint8, device=dev)

        def step_host():
            cache.skv_decode_step_host(hb["Q"], hb["K"], hb["V"], h_slot, h_pt, h_len, hb["out"], staging)

        for _ in range(args.warmup):
            step_host()
        barrier()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for _ in range(args.steps):
            step_host()
        e1.record()
        barrier()
        ms_e2e = e0.elapsed_time(e1)
    status = cache.skv_get_status()
    if status != 0:
        raise SystemExit(f"device status {status}")
    if not torch.equal(hb["out"].view(torch.int16), t["out"].cpu().view(torch.int16)):
        raise SystemExit("host-buffer step and device-resident step disagree")

    times = torch.tensor([ms, ms_e2e], dtype=torch.float64, device=dev)
    if world > 1:
        import torch.distributed as dist
        dist.all_reduce(times, op=dist.ReduceOp.MAX)
    ms, ms_e2e = float(times[0]), float(times[1])
    if rank != 0:
        return

    peak, peak_kind = _peaks()
    value = world * step_bytes * args.steps / (ms * 1e-3) / 1e9
    e2e_value = world * step_bytes * args.steps / (ms_e2e * 1e-3) / 1e9
    # the roofline figure is taken on the owner layers' launches: their pages were last touched a whole
    # model pass ago, so nothing of them is in L2 (a layer that re-reads its predecessor's owner can be faster)
    achieved = dw.kv_bytes_per_call() / (kern_ms_owner * 1e-3) / 1e9
    h2d = sum(hb[k].numel() * 2 for k in ("Q", "K", "V")) + h_slot.numel() * 8 + h_pt.numel() * 4 + h_len.numel() * 4
    d2h = hb["out"].numel() * 2
    line = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps, "warmup": args.warmup,
        "ms_per_step": ms / args.steps, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "bf16", "data": "synthetic",
        "config": {"workload": w.name, "family": w.family, "n_layers": L, "owners": n_own, "batch": dw.batch,
                   "tokens": int(dw.lens_cpu.sum()), "q_heads": w.q_heads, "kv_heads": w.kv_heads,
                   "head_dim": w.head_dim, "page_size": w.page_size,
                   "l2": "inputs larger than L2: every attention call streams %.0f MB of pages" % (dw.kv_bytes_per_call() / 1e6),
                   "step": "append (owners) + decode attention for every layer"},
        "steps_per_s": world * args.steps / (ms * 1e-3),
        "attn_calls_per_s": world * L * args.steps / (ms * 1e-3),
        "frac_of_nominal_8TBs": value / world / NOMINAL_HBM_GBS,
        "clocks": clocks.summary(),
        "e2e": {"value": e2e_value, "unit": UNIT, "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h,
                "ms_per_step": ms_e2e / args.steps},
        "gpu_launches": int(launches),
        "roofline": {"bound": "hbm", "kernel": "decode_splitk_kernel", "achieved": achieved, "peak": peak,
                     "peak_kind": peak_kind, "unit": "GB/s", "frac": achieved / peak,
                     "frac_of_nominal_8TBs": achieved / NOMINAL_HBM_GBS, "us_per_launch": kern_ms_owner * 1e3,
                     "us_per_launch_all_layers": kern_ms * 1e3,
                     "us_per_launch_reader_layers": None if kern_ms_reader is None else kern_ms_reader * 1e3,
                     "bytes_per_launch": dw.kv_bytes_per_call(),
                     "traffic": NCU_TRAFFIC_BYTES.get(w.name)},
    }
    if not args.no_cpu_baseline and world == 1:
        n_seqs = min(w.batch, args.ref_seqs)
        o, layer, Q, sl, nbytes = _oracle_sample(w, dw.lens_cpu, dw.r, n_seqs)
        best = float("inf")
        for _ in range(3):
            t0 = time.perf_counter()
            o.decode_attn(layer, Q, sl)
            best = min(best, time.perf_counter() - t0)
        line["cpu_baseline"] = {
            "value": nbytes / best / 1e9, "unit": UNIT, "cores": os.cpu_count() or 1, "kind": "oracle",
            "sample": f"1 decode-attention call (layer {layer} reading layer {dw.r[layer]}) over the first {n_seqs} "
                      f"sequences ({int(sl.sum())} tokens), best of 3, {best * 1e3:.1f} ms"}
    print(json.dumps(line))
    if world > 1:
        import torch.distributed as dist
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
