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
NCU_TRAFFIC_BYTES = {"llama3_8b": 343470000}
DEFAULT_L2_KEEP = 35     # the library's default share of each block range kept in L2 for the next layer


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
                 "-lms", "25"], stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._read, daemon=True)
            self.thread.start()
        except Exception:
            self.proc = None
        return self

    def _read(self):
        for line in self.proc.stdout:
            self.rows.append([x.strip() for x in line.split(",")])

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
    ap.add_argument("--fp8", action="store_true", help="run the main legs on FP8 pages (profiling the FP8 kernel); "
                    "the byte counts are then those of the FP8 cache")
    ap.add_argument("--no-sweep", action="store_true", help="skip the sharing-ratio sweep (owner fractions 1, 1/2, 1/4, 1/8)")
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
    w = rank_workload(w, rank, world)
    dw = harness.setup(w, device=dev, fp8=args.fp8)
    dw.retune(variant=args.variant or None,
              tuning=[int(x) for x in args.tuning.split(",")] if args.tuning else None,
              overlap=args.overlap if args.overlap >= 0 else None,
              l2_keep=args.l2_keep if args.l2_keep >= 0 else None)
    harness.prefill(dw, upto_offset=-1)
    t = harness.step_tensors(dw)
    L, n_own = w.n_layers, len(dw.owners)
    attn_bytes = dw.kv_bytes_per_call()
    step_bytes = L * attn_bytes + n_own * dw.append_bytes_per_call()
    cache = dw.cache

    def step():
        cache.skv_decode_step(t["Q"], t["K"], t["V"], dw.slot_new, dw.page_table, dw.seq_lens, t["out"], dw.workspace)

    def barrier():
        if world > 1:
            import torch.distributed as dist
            dist.barrier()
        torch.cuda.synchronize(dev)

    def timed_steps(fn):
        """args.warmup untimed calls, then args.steps calls between two events (barrier + synchronize on
        both sides); returns milliseconds for the args.steps calls."""
        for _ in range(args.warmup):
            fn()
        barrier()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for _ in range(args.steps):
            fn()
        e1.record()
        barrier()
        return e0.elapsed_time(e1)

    with ClockSampler(local) as clocks:
        clocks.wait_first()
        # (1) the headline: whole decode steps, inputs resident in HBM, library defaults
        launches0 = cache.skv_launch_count()
        ms = timed_steps(step)
        launches = (cache.skv_launch_count() - launches0) * args.steps // (args.steps + args.warmup)
        out_default = t["out"].clone()

        # (2) the roofline leg: the same steps with L2 reuse between layers switched off, so that every
        # attention launch streams all of its pages from HBM.  The split-K kernel's average launch
        # duration is taken as (time of the timed region) / (split-K launches in it): its launches
        # overlap each other and the small merge and update kernels, so they cannot be bracketed one
        # by one without changing what is measured; the quotient charges those kernels to it.
        dw.retune(l2_keep=0)
        ms_hbm = timed_steps(step)
        dw.retune(l2_keep=args.l2_keep if args.l2_keep >= 0 else DEFAULT_L2_KEEP)

        # (3) one attention call at a time (no overlap between calls): per-layer entry points with an
        # event pair around every skv_decode_attn (split-K + merge)
        pairs = []
        for _ in range(max(2, args.steps // 4)):
            for l in range(L):
                if dw.r[l] == l:
                    cache.skv_append(l, t["K"][dw.owners.index(l)], t["V"][dw.owners.index(l)], dw.slot_new)
                a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                a.record()
                cache.skv_decode_attn(l, t["Q"][l], dw.page_table, dw.seq_lens, t["out"][l], dw.workspace)
                b.record()
                pairs.append((l, a, b))
        torch.cuda.synchronize(dev)
        per = [(l, a.elapsed_time(b)) for l, a, b in pairs[L:]]
        own = [x for l, x in per if dw.r[l] == l]
        non = [x for l, x in per if dw.r[l] != l]
        call_ms_owner = sum(own) / len(own)
        call_ms_reader = sum(non) / len(non) if non else None

        # (4) end to end: host buffers in, host buffer out, copies inside the timed region
        hb = harness.step_tensors(dw, device="cpu", pin=True)
        h_slot = dw.slot_new.cpu().pin_memory()
        h_pt = dw.page_table_cpu.contiguous().pin_memory()
        h_len = dw.lens_cpu.contiguous().pin_memory()
        staging = torch.empty(cache.skv_decode_step_staging_bytes(dw.batch, w.q_heads, h_pt.shape[1]),
                              dtype=torch.uint8, device=dev)

        def step_host():
            cache.skv_decode_step_host(hb["Q"], hb["K"], hb["V"], h_slot, h_pt, h_len, hb["out"], staging)

        ms_e2e = timed_steps(step_host)
    status = cache.skv_get_status()
    if status != 0:
        raise SystemExit(f"device status {status}")
    if not torch.equal(hb["out"].view(torch.int16), out_default.cpu().view(torch.int16)):
        raise SystemExit("host-buffer step and device-resident step disagree")

    ms, ms_hbm, ms_e2e = max_over_ranks([ms, ms_hbm, ms_e2e], world, dev)
    if rank != 0:
        return

    peak, peak_kind = _peaks()
    value = whole_job_rate(step_bytes, args.steps, ms, world) / 1e9
    e2e_value = whole_job_rate(step_bytes, args.steps, ms_e2e, world) / 1e9
    us_per_launch = ms_hbm * 1e3 / (args.steps * L)
    achieved = attn_bytes / (us_per_launch * 1e-6) / 1e9
    h2d = sum(hb[k].numel() * 2 for k in ("Q", "K", "V")) + h_slot.numel() * 8 + h_pt.numel() * 4 + h_len.numel() * 4
    d2h = hb["out"].numel() * 2
    line = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps, "warmup": args.warmup,
        "ms_per_step": ms / args.steps, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "e4m3 pages" if args.fp8 else "bf16", "data": "synthetic",
        "config": {"workload": w.name, "family": w.family, "n_layers": L, "owners": n_own, "batch": dw.batch,
                   "tokens": int(dw.lens_cpu.sum()), "q_heads": w.q_heads, "kv_heads": w.kv_heads,
                   "head_dim": w.head_dim, "page_size": w.page_size,
                   "l2": "inputs larger than L2: every attention call streams %.0f MB of pages" % (attn_bytes / 1e6),
                   "step": "update of every owner layer + decode attention (split-K + merge) for every layer"},
        "steps_per_s": world * args.steps / (ms * 1e-3),
        "attn_calls_per_s": world * L * args.steps / (ms * 1e-3),
        "frac_of_nominal_8TBs": value / world / NOMINAL_HBM_GBS,
        "clocks": clocks.summary(),
        "e2e": {"value": e2e_value, "unit": UNIT, "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h,
                "ms_per_step": ms_e2e / args.steps},
        "gpu_launches": int(launches),
        "roofline": {"bound": "hbm", "kernel": "decode_splitk_kernel", "achieved": achieved, "peak": peak,
                     "peak_kind": peak_kind, "unit": "GB/s", "frac": achieved / peak,
                     "frac_of_nominal_8TBs": achieved / NOMINAL_HBM_GBS, "us_per_launch": us_per_launch,
                     "bytes_per_launch": attn_bytes,
                     "how": "whole steps with L2 reuse between layers off; timed region / split-K launches in it",
                     "traffic": None if args.fp8 else NCU_TRAFFIC_BYTES.get(w.name)},
        "single_call": {"us_owner_layers": call_ms_owner * 1e3,
                        "us_reader_layers": None if call_ms_reader is None else call_ms_reader * 1e3,
                        "gbs_owner_layers": attn_bytes / (call_ms_owner * 1e-3) / 1e9,
                        "how": "skv_decode_attn (split-K + merge) alone between two events, nothing overlapping it"},
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
    if not args.no_sweep and world == 1:
        del dw, cache, t, hb, staging
        torch.cuda.empty_cache()
        line["sharing_sweep"] = sharing_sweep(args, dev)
        line["prefill"] = prefill_leg(args, dev)
        line["fp8_pages"] = fp8_leg(args, dev)
    print(json.dumps(line))
    if world > 1:
        import torch.distributed as dist
        dist.destroy_process_group()


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
    ms8 = timed(lambda: dq.cache.skv_prefill_attn(1, inp["Q"], inp["cu_q_lens"], dq.page_table, dq.seq_lens, out, T))
    res["fp8_pages"] = {"append_ms": ms_append8, "ms_per_call": ms8, "tflops": flops / (ms8 * 1e-3) / 1e12,
                        "tokens_per_s": B * T / (ms8 * 1e-3)}
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

    def step():
        cache.skv_decode_step(t["Q"], t["K"], t["V"], dw.slot_new, dw.page_table, dw.seq_lens, t["out"], dw.workspace)

    for _ in range(args.warmup):
        step()
    torch.cuda.synchronize(dev)
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    n = max(3, args.steps // 2)
    e0.record()
    for _ in range(n):
        step()
    e1.record()
    torch.cuda.synchronize(dev)
    ms = e0.elapsed_time(e1) / n
    if cache.skv_get_status() != 0:
        raise SystemExit("device status after the FP8 leg")
    st = cache.skv_cache_stats()
    tokens = int(dw.lens_cpu.sum())
    return {"workload": w.name, "kv_bytes_per_token": st["bytes_per_token"], "ms_per_step": ms,
            "us_per_attn_call": ms * 1e3 / w.n_layers,
            "attn_gbs": w.n_layers * dw.kv_bytes_per_call() / (ms * 1e-3) / 1e9,
            "tokens_attended_per_us": w.n_layers * tokens / (ms * 1e3)}


def sharing_sweep(args, dev):
    """Llama-3-8B shape, batch 128, lengths U[512,2048]: owner fractions 1, 1/2, 1/4, 1/8 (evenly spaced
    owners).  Per ratio: cache bytes, the largest batch a 120e9-byte KV budget holds, whole decode steps per
    second (update of the owners + attention of all 32 layers) and the time per attention call."""
    from paper_2604_22782_b200 import harness
    rows = []
    budget = 120e9
    for g in (1, 2, 4, 8):
        w = W.sweep_workload(g)
        dw = harness.setup(w, device=dev)
        harness.prefill(dw, upto_offset=-1)
        t = harness.step_tensors(dw)
        cache = dw.cache

        def step():
            cache.skv_decode_step(t["Q"], t["K"], t["V"], dw.slot_new, dw.page_table, dw.seq_lens, t["out"],
                                  dw.workspace)

        for _ in range(args.warmup):
            step()
        torch.cuda.synchronize(dev)
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        n = max(3, args.steps // 2)
        e0.record()
        for _ in range(n):
            step()
        e1.record()
        torch.cuda.synchronize(dev)
        ms = e0.elapsed_time(e1) / n
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
            "attn_gbs": w.n_layers * dw.kv_bytes_per_call() / (ms * 1e-3) / 1e9,
        })
        if cache.skv_get_status() != 0:
            raise SystemExit("device status after the sweep")
        del dw, cache, t
        torch.cuda.empty_cache()
    return rows


if __name__ == "__main__":
    main()
