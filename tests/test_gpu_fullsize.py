"""The five full-size workloads, in the launch configurations the benchmark times: the step layer by layer
through skv_append / skv_decode_attn with early fetch on (each layer's query written by a kernel that reads
the previous layer's output), and the whole step through skv_decode_step.  The Llama-3-8B workload is
compared with the oracle in full (every sequence, every layer).  The oracle cannot hold the others whole, so:
  - cache contents are compared bit for bit for EVERY token of EVERY owner layer, on the device,
    against the rows the generator draws (the update is a pure copy);
  - attention outputs are compared with the oracle, element by element within
    |out - ref| <= 1e-2 + 1e-2 |ref|, for a sample of sequences (shortest, longest, seeded picks;
    full length, all heads) on a sample of layers (first owner, its first reader, last owner, last layer);
  - every other output row must be finite and lie inside the convex-combination bound
    |out| <= max |V| of the generator's value table.
The Llama-3-8B and Qwen3-8B workloads also run on FP8 pages (codes and scales of the sampled sequences bit for
bit against the oracle's quantiser, their outputs within the same tolerance)."""
import pytest
import torch

import workloads as W

pytestmark = pytest.mark.gpu

ATOL, RTOL = 1e-2, 1e-2


def _sample_sequences(lens, k, seed):
    order = torch.argsort(lens.to(torch.int64), stable=True)
    picks = [int(order[0]), int(order[-1])]
    g = torch.Generator().manual_seed(seed)
    for i in torch.randperm(lens.numel(), generator=g).tolist():
        if len(picks) >= k:
            break
        if i not in picks:
            picks.append(i)
    return picks[:k]


def _sample_layers(r):
    L = len(r)
    owners = [l for l in range(L) if r[l] == l]
    first_reader = next((l for l in range(L) if r[l] != l), 0)
    return sorted({0, first_reader, owners[-1], L - 1})


def _check_workload(w, n_seqs, all_layers=False):
    from oracle import Oracle
    from paper_2604_22782_b200 import harness
    dw = harness.setup(w)
    harness.prefill(dw, upto_offset=-1)
    t = harness.step_tensors(dw)
    t["out"].fill_(float("nan"))
    dw.cache.skv_decode_step(t["Q"], t["K"], t["V"], dw.slot_new, dw.page_table, dw.seq_lens, t["out"], dw.workspace)
    torch.cuda.synchronize()
    assert dw.cache.skv_get_status() == 0
    # the same step as a decoder issues it: per layer a kernel that makes the query from the previous layer's
    # output, the update (owners), the attention call with early fetch on (the benchmark's headline leg)
    dw.retune(early_fetch=1)
    loop_out = torch.full_like(t["out"], float("nan"))
    q_dep = torch.empty_like(t["Q"][0])
    for l in range(w.n_layers):
        torch.add(t["Q"][l], t["out"][l - 1], alpha=0.0, out=q_dep)
        if dw.r[l] == l:
            i = dw.owners.index(l)
            dw.cache.skv_append(l, t["K"][i], t["V"][i], dw.slot_new)
        dw.cache.skv_decode_attn(l, q_dep, dw.page_table, dw.seq_lens, loop_out[l], dw.workspace)
    torch.cuda.synchronize()
    assert dw.cache.skv_get_status() == 0
    dw.retune(early_fetch=0)
    a, b = loop_out.float(), t["out"].float()
    assert bool(((a - b).abs() <= 2 * ATOL + RTOL * b.abs()).all()), "per-layer loop and whole-step call disagree"

    # byte accounting scales exactly with the owner count
    stats = dw.cache.skv_cache_stats()
    assert stats["n_owners"] == len(dw.owners)
    assert stats["bytes_per_token"] == 2 * len(dw.owners) * w.kv_heads * w.head_dim * 2
    assert stats["kv_bytes"] == len(dw.owners) * dw.total_pages * (2 * w.page_size * w.kv_heads * w.head_dim * 2)

    # cache: every token of every owner layer, bit for bit, against what the generator draws
    seq_idx, pos = W.token_index(dw.lens_cpu)
    slots = W.slot_map_for(dw.page_table_cpu, seq_idx, pos, w.page_size)
    chunk = 1 << 16
    for l in dw.owners:
        for s in range(0, seq_idx.numel(), chunk):
            e = min(seq_idx.numel(), s + chunk)
            Kd, Vd = W.draw_kv(w, l, seq_idx[s:e], pos[s:e], device=dw.device)
            Kg, Vg = torch.empty_like(Kd), torch.empty_like(Vd)
            dw.cache.skv_gather(l, slots[s:e].to(dw.device), Kg, Vg)
            assert torch.equal(Kg.view(torch.int16), Kd.view(torch.int16)), f"K of layer {l}, tokens {s}..{e}"
            assert torch.equal(Vg.view(torch.int16), Vd.view(torch.int16)), f"V of layer {l}, tokens {s}..{e}"

    # attention outputs of the sampled sequences on the sampled layers against the oracle
    seqs = _sample_sequences(dw.lens_cpu, n_seqs, w.seed + 7)
    layers = list(range(w.n_layers)) if all_layers else _sample_layers(dw.r)
    sub_lens = dw.lens_cpu[seqs]
    o = Oracle(w.n_layers, dw.r, w.q_heads, w.kv_heads, w.head_dim, len(seqs), int(sub_lens.max()))
    local, lpos = W.token_index(sub_lens)
    glob = torch.as_tensor(seqs, dtype=torch.int64)[local]
    for src in sorted({dw.r[l] for l in layers}):
        for s in range(0, local.numel(), chunk):     # drawn on the device (same bits as on the CPU), used on the CPU
            e = min(local.numel(), s + chunk)
            K, V = W.draw_kv(w, src, glob[s:e], lpos[s:e], device=dw.device)
            o.append(src, K.cpu(), V.cpu(), local[s:e], lpos[s:e])
    worst = 0.0
    for l in layers:
        Q = t["Q"][l].cpu()[seqs]
        ref = o.decode_attn(l, Q, sub_lens)
        for name, res in (("skv_decode_step", t["out"]), ("per-layer loop", loop_out)):
            got = res[l].cpu()[seqs].double()
            err = (got - ref).abs()
            assert bool((err <= ATOL + RTOL * ref.abs()).all()), f"{name}, layer {l}: max abs err {err.max().item()}"
            worst = max(worst, err.max().item())
    o.close()

    # every row: finite and inside the convex-combination bound
    vmax = 5.0 * w.kv_std            # the generator's table ends below 4.5 standard deviations
    for res in (t["out"], loop_out):
        out = res.float()
        assert torch.isfinite(out).all()
        assert out.abs().max().item() <= vmax
    return worst


def test_llama3_8b_full_size():
    """Config 2: 32 layers, 32q/8kv, D=128, 16 owners, batch 32, lengths U[1024,4096]: every sequence on
    every layer against the oracle (16 source stores of 32 x 4096 tokens on the host)."""
    _check_workload(W.get_workload("llama3_8b"), n_seqs=32, all_layers=True)


@pytest.mark.parametrize("name", ["qwen3_8b_b1_2k", "qwen3_8b_b1_8k"])
def test_table4_shape_one_sequence(name):
    """Table 4's shape: Qwen3-8B heads, groups of four layers, ONE sequence of 2 048 / 8 192 + 128 tokens (an
    owner layer's cache fits in L2 and is loaded with normal priority for the group's reader layers): every
    layer against the oracle."""
    _check_workload(W.get_workload(name), n_seqs=1, all_layers=True)


def test_qwen3_8b_full_size():
    """Config 3: 36 layers in groups of 4 (9 owners), batch 64, lengths U[2048,8192], Q std 0.5."""
    _check_workload(W.get_workload("qwen3_8b"), n_seqs=4)


def test_llama2_7b_32k_full_size():
    """Config 4: MHA 32/32, stochastic routing map, batch 8 x 32768 tokens (the CUDA-core kernel)."""
    w = W.get_workload("llama2_7b_32k")
    free, _ = torch.cuda.mem_get_info()
    from paper_2604_22782_b200.binding import skv_cache_pool_bytes
    need = skv_cache_pool_bytes(W.routing_map(w), w.kv_heads, w.head_dim, w.page_size, 8 * 2048)
    if free < need + (8 << 30):
        pytest.skip(f"needs {need / 1e9:.0f} GB of device memory for the pool")
    _check_workload(w, n_seqs=2)


@pytest.mark.parametrize("group", [1, 2, 4, 8])
def test_sharing_sweep_full_size(group):
    """Config 5: Llama-3-8B shape, batch 128, lengths U[512,2048], owner fraction 1/group."""
    _check_workload(W.sweep_workload(group), n_seqs=4)


def _check_workload_fp8(w, n_seqs):
    """The same whole step on FP8 pages (library defaults: the tcgen05 kernel at head_dim 128): codes and
    scales of every token of the sampled sequences on the sampled source layers bit for bit against the oracle's
    quantiser, their attention outputs element by element, every other row finite and inside the bound."""
    from oracle import Oracle
    from paper_2604_22782_b200 import harness
    dw = harness.setup(w, fp8=True)
    harness.prefill(dw, upto_offset=-1)
    t = harness.step_tensors(dw)
    t["out"].fill_(float("nan"))
    dw.cache.skv_decode_step(t["Q"], t["K"], t["V"], dw.slot_new, dw.page_table, dw.seq_lens, t["out"], dw.workspace)
    torch.cuda.synchronize()
    assert dw.cache.skv_get_status() == 0
    stats = dw.cache.skv_cache_stats()
    assert stats["bytes_per_token"] == 2 * len(dw.owners) * w.kv_heads * (w.head_dim + 4)

    seqs = _sample_sequences(dw.lens_cpu, n_seqs, w.seed + 7)
    layers = _sample_layers(dw.r)
    sub_lens = dw.lens_cpu[seqs]
    o = Oracle(w.n_layers, dw.r, w.q_heads, w.kv_heads, w.head_dim, len(seqs), int(sub_lens.max()))
    local, lpos = W.token_index(sub_lens)
    glob = torch.as_tensor(seqs, dtype=torch.int64)[local]
    slots = W.slot_map_for(dw.page_table_cpu, glob, lpos, w.page_size)
    chunk = 1 << 15
    for src in sorted({dw.r[l] for l in layers}):
        for s in range(0, local.numel(), chunk):
            e = min(local.numel(), s + chunk)
            K, V = W.draw_kv(w, src, glob[s:e], lpos[s:e], device=dw.device)
            okc, ovc, oks, ovs = o.append_fp8(src, K.cpu(), V.cpu(), local[s:e], lpos[s:e])
            n = e - s
            kc = torch.zeros((n, w.kv_heads, w.head_dim), dtype=torch.uint8, device=dw.device)
            vc = torch.zeros_like(kc)
            ks = torch.zeros((n, w.kv_heads), dtype=torch.float32, device=dw.device)
            vs = torch.zeros_like(ks)
            dw.cache.skv_gather_fp8(src, slots[s:e].to(dw.device), kc, vc, ks, vs)
            assert torch.equal(kc.cpu(), okc) and torch.equal(vc.cpu(), ovc), f"codes of layer {src}, tokens {s}..{e}"
            assert torch.equal(ks.cpu().view(torch.int32), oks.view(torch.int32)), f"K scales of layer {src}"
            assert torch.equal(vs.cpu().view(torch.int32), ovs.view(torch.int32)), f"V scales of layer {src}"
    for l in layers:
        Q = t["Q"][l].cpu()[seqs]
        ref = o.decode_attn(l, Q, sub_lens)
        got = t["out"][l].cpu()[seqs].double()
        err = (got - ref).abs()
        assert bool((err <= ATOL + RTOL * ref.abs()).all()), f"layer {l}: max abs err {err.max().item()}"
    o.close()
    out = t["out"].float()
    assert torch.isfinite(out).all()
    assert out.abs().max().item() <= 5.0 * w.kv_std * 1.07      # E4M3 rounding can lift a value by 1/16


def test_llama3_8b_full_size_fp8():
    _check_workload_fp8(W.get_workload("llama3_8b"), n_seqs=4)


def test_qwen3_8b_full_size_fp8():
    _check_workload_fp8(W.get_workload("qwen3_8b"), n_seqs=3)


def test_sharing_sweep_cache_bytes_scale_exactly():
    """Pool bytes of the four sweep points are in the ratio 32:16:8:4 (same pages, fewer owner layers)."""
    from paper_2604_22782_b200.binding import skv_cache_pool_bytes
    lens = W.seq_lens(W.sweep_workload(1))
    pages = int(((lens.to(torch.int64) + 15) // 16).sum())
    sizes = [skv_cache_pool_bytes(W.routing_map(W.sweep_workload(g)), 8, 128, 16, pages) - 256 for g in (1, 2, 4, 8)]
    assert [s * g for s, g in zip(sizes, (1, 2, 4, 8))] == [sizes[0]] * 4


@pytest.mark.parametrize("group", [1, 2, 4, 8])
def test_largest_batch_of_a_kv_budget_is_a_cache_that_can_be_created(group):
    """The sweep's "largest batch in a 120e9-byte KV budget" (worst-case length 2048 = 128 pages per sequence) is a
    closed form in bench.py; here the same arithmetic is checked against a real cache: a pool of exactly the bytes
    the library asks for at that batch fits the budget, one sequence more does not, the cache is created on it and
    its last page can be written and read back.  At a tenth of the budget for every ratio (12e9 bytes), and at the
    whole 120e9 bytes for the owner fraction 1/8 when the GPU has the room."""
    from paper_2604_22782_b200 import binding as skv
    w = W.sweep_workload(group)
    r = W.routing_map(w)
    pages_per_seq = (w.len_hi + w.page_size - 1) // w.page_size
    one_seq = skv.skv_cache_pool_bytes(r, w.kv_heads, w.head_dim, w.page_size, pages_per_seq) - 256
    assert one_seq == (32 // group) * pages_per_seq * w.kv_heads * 2 * 16 * w.head_dim * 2
    budgets = [12e9]
    free, _ = torch.cuda.mem_get_info()
    if group == 8 and free > 150e9:
        budgets.append(120e9)
    for budget in budgets:
        max_batch = int(budget // one_seq)
        need = skv.skv_cache_pool_bytes(r, w.kv_heads, w.head_dim, w.page_size, max_batch * pages_per_seq)
        assert need - 256 <= budget < need - 256 + one_seq
        if budget == 120e9:
            assert max_batch == {1: 447, 2: 894, 4: 1788, 8: 3576}[group]      # the figures the benchmark prints
        pool = torch.empty(need, dtype=torch.uint8, device="cuda")
        cache = skv.SkvCache(r, w.kv_heads, w.head_dim, w.page_size, max_batch * pages_per_seq, device_pool=pool)
        assert cache.skv_cache_stats()["kv_bytes"] == need - 256
        # the very last slot of the very last page, on the last owner layer
        last_owner = max(l for l in range(w.n_layers) if r[l] == l)
        slot = torch.tensor([max_batch * pages_per_seq * w.page_size - 1], dtype=torch.int64, device="cuda")
        K = torch.randn((1, w.kv_heads, w.head_dim), device="cuda").to(torch.bfloat16)
        V = torch.randn((1, w.kv_heads, w.head_dim), device="cuda").to(torch.bfloat16)
        cache.skv_append(last_owner, K, V, slot)
        Kg, Vg = torch.zeros_like(K), torch.zeros_like(V)
        cache.skv_gather(last_owner, slot, Kg, Vg)
        torch.cuda.synchronize()
        assert torch.equal(Kg.view(torch.int16), K.view(torch.int16)) and torch.equal(Vg.view(torch.int16), V.view(torch.int16))
        assert cache.skv_get_status() == 0
        cache.close()
        del cache, pool
        torch.cuda.empty_cache()
