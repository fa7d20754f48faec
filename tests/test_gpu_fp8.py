"""FP8 pages (E4M3 codes + one fp32 scale per (token, kv head) row): cache contents bit for bit against
the oracle's quantiser, decode attention against the oracle's attention over the dequantised values."""
import pytest
import torch

import workloads as W

pytestmark = pytest.mark.gpu

ATOL, RTOL = 1e-2, 1e-2


def _setup(w, lens, poison=False):
    from paper_2604_22782_b200 import harness
    dw = harness.setup(w, lens=lens, fp8=True)
    if poison:       # every byte 0x7f: NaN codes and NaN scales in every slot that is never written
        dw.cache.pool[256:].fill_(0x7F)
    harness.prefill(dw, upto_offset=0)
    return harness, dw


def _oracle(dw, layers):
    """Oracle with the source layers appended through its quantiser; also returns their codes and scales."""
    from oracle import Oracle
    w = dw.w
    o = Oracle(w.n_layers, dw.r, w.q_heads, w.kv_heads, w.head_dim, dw.batch, max(1, int(dw.lens_cpu.max())))
    si, pos = W.token_index(dw.lens_cpu)
    stored = {}
    for src in sorted({dw.r[l] for l in layers}):
        K, V = W.draw_kv(w, src, si, pos)
        stored[src] = o.append_fp8(src, K, V, si, pos)
    return o, stored, si, pos


@pytest.mark.parametrize("variant", [0, 2])      # 0: tcgen05 kernel where it applies (head_dim 128), 2: mma.sync kernel
@pytest.mark.parametrize("Hq,Hkv,D", [(8, 2, 128), (4, 4, 128), (8, 1, 128), (6, 2, 128), (6, 2, 64), (4, 2, 64), (2, 2, 64)])
def test_cache_codes_and_decode_outputs(Hq, Hkv, D, variant):
    if variant == 2 and D == 64:
        pytest.skip("head_dim 64 runs the mma.sync kernel under either setting")
    lens = torch.tensor([1, 5, 16, 17, 31, 33, 47, 100, 3, 700, 2049, 129, 256, 112], dtype=torch.int32)
    w = W.Workload("fp8", 3, Hq, Hkv, D, 16, lens.numel(), 0, 0, "explicit", explicit_r=(0, 0, 2), seed=97, kv_std=1.7)
    harness, dw = _setup(w, lens, poison=True)
    dw.retune(variant=variant)
    o, stored, si, pos = _oracle(dw, range(3))
    # cache: codes and scales of every token of every owner layer, bit for bit
    slots = W.slot_map_for(dw.page_table_cpu, si, pos, w.page_size).to(dw.device)
    n = si.numel()
    for l in dw.owners:
        kc = torch.zeros((n, Hkv, D), dtype=torch.uint8, device=dw.device)
        vc = torch.zeros_like(kc)
        ks = torch.zeros((n, Hkv), dtype=torch.float32, device=dw.device)
        vs = torch.zeros_like(ks)
        dw.cache.skv_gather_fp8(l, slots, kc, vc, ks, vs)
        torch.cuda.synchronize()
        okc, ovc, oks, ovs = stored[l]
        assert torch.equal(kc.cpu(), okc) and torch.equal(vc.cpu(), ovc)
        assert torch.equal(ks.cpu().view(torch.int32), oks.view(torch.int32))
        assert torch.equal(vs.cpu().view(torch.int32), ovs.view(torch.int32))
    # attention of every layer
    for l in range(3):
        Q = harness.step_inputs(dw, l)["Q"]
        out = torch.full((dw.batch, Hq, D), float("nan"), dtype=torch.bfloat16, device=dw.device)
        dw.cache.skv_decode_attn(l, Q, dw.page_table, dw.seq_lens, out, dw.workspace)
        torch.cuda.synchronize()
        ref = o.decode_attn(l, Q.cpu(), dw.lens_cpu)
        err = (out.cpu().double() - ref).abs()
        assert bool((err <= ATOL + RTOL * ref.abs()).all()), f"layer {l}: max abs err {err.max().item()}"
    assert dw.cache.skv_get_status() == 0
    st = dw.cache.skv_cache_stats()
    assert st["bytes_per_token"] == 2 * len(dw.owners) * Hkv * (D + 4)
    assert st["page_bytes"] == Hkv * (2 * 16 * D + 128)


@pytest.mark.parametrize("Hq,Hkv,D,variant", [(6, 2, 64, 0), (8, 2, 128, 2)])
def test_decode_merged_inside_the_cta_kernel(Hq, Hkv, D, variant):
    """FP8 pages through the CTA-per-range kernel (head_dim 64, or the mma.sync variant at head_dim 128) with the
    segments cut by range ends finished inside the kernel (skv_set_decode_merge(2)), early fetch on and off."""
    lens = torch.tensor([1, 5, 16, 17, 31, 33, 47, 100, 3, 700, 2049, 129, 256, 112, 0, 4100], dtype=torch.int32)
    w = W.Workload("fp8_merge", 2, Hq, Hkv, D, 16, lens.numel(), 0, 0, "explicit", explicit_r=(0, 0), seed=98, kv_std=1.7)
    harness, dw = _setup(w, lens, poison=True)
    o, stored, si, pos = _oracle(dw, range(2))
    for early in (0, 1):
        dw.retune(variant=variant, merge=2, early_fetch=early)
        for l in range(2):
            Q = harness.step_inputs(dw, l)["Q"]
            out = torch.full((dw.batch, Hq, D), float("nan"), dtype=torch.bfloat16, device=dw.device)
            before = dw.cache.skv_launch_count()
            dw.cache.skv_decode_attn(l, Q, dw.page_table, dw.seq_lens, out, dw.workspace)
            torch.cuda.synchronize()
            assert dw.cache.skv_launch_count() == before + 1          # no merge launch
            ref = o.decode_attn(l, Q.cpu(), dw.lens_cpu)
            err = (out.cpu().double() - ref).abs()
            assert bool((err <= ATOL + RTOL * ref.abs()).all()), f"layer {l} early {early}: max abs err {err.max().item()}"
    assert dw.cache.skv_get_status() == 0


def test_rows_of_very_different_magnitude():
    """Per-row scales spanning 2^-20 .. 2^12 in one sequence: the scales are applied outside the f16
    contractions, so neither overflow nor flush-to-zero may show.  With such a spread an output element
    is a sum of terms thousands of times larger than itself wherever the big rows cancel, so the bound
    here is taken relative to the largest element of the output row, not element by element."""
    from paper_2604_22782_b200 import harness
    from oracle import Oracle
    lens = torch.tensor([300, 40], dtype=torch.int32)
    w = W.Workload("fp8_mag", 1, 8, 2, 128, 16, 2, 0, 0, "explicit", explicit_r=(0,), seed=101)
    dw = harness.setup(w, lens=lens, fp8=True)
    si, pos = W.token_index(lens)
    K, V = W.draw_kv(w, 0, si, pos)
    g = torch.Generator().manual_seed(1)
    mag = torch.exp2(torch.randint(-20, 13, (si.numel(), 1, 1), generator=g).float())
    V = (V.float() * mag).to(torch.bfloat16)
    K = (K.float() * torch.exp2(torch.randint(-3, 3, (si.numel(), 1, 1), generator=g).float())).to(torch.bfloat16)
    slots = W.slot_map_for(dw.page_table_cpu, si, pos, w.page_size).to(dw.device)
    dw.cache.skv_append(0, K.to(dw.device), V.to(dw.device), slots)
    o = Oracle(1, [0], 8, 2, 128, 2, 300)
    o.append_fp8(0, K, V, si, pos)
    Q = harness.step_inputs(dw, 0)["Q"]
    out = torch.empty((2, 8, 128), dtype=torch.bfloat16, device=dw.device)
    dw.cache.skv_decode_attn(0, Q, dw.page_table, dw.seq_lens, out, dw.workspace)
    torch.cuda.synchronize()
    ref = o.decode_attn(0, Q.cpu(), lens)
    err = (out.cpu().double() - ref).abs()
    assert torch.isfinite(out.float()).all()
    row_max = ref.abs().amax(dim=-1, keepdim=True)
    assert bool((err <= ATOL + RTOL * row_max).all()), f"max abs err {err.max().item()} at |ref| up to {ref.abs().max().item()}"


@pytest.mark.parametrize("n_extra", [0, 700])     # below and above the size at which the page-granular update kernel takes over
def test_update_with_arbitrary_slot_maps(n_extra):
    """skv_append on FP8 pages with slot maps that mix whole pages at odd positions of the call, pages in reverse
    order, pages with a skipped token, scattered single slots and runs of whole pages: every written slot reads
    back as the oracle quantiser's codes and scales, for both update kernels."""
    from oracle import quantize_e4m3
    from paper_2604_22782_b200 import harness
    Hkv, D = 2, 128
    n_pages = 120
    lens = torch.tensor([n_pages * 16], dtype=torch.int32)
    w = W.Workload("fp8_slots", 1, 4, Hkv, D, 16, 1, 0, 0, "explicit", explicit_r=(0,), seed=113)
    dw = harness.setup(w, lens=lens, fp8=True)
    g = torch.Generator().manual_seed(17)
    pages = torch.randperm(n_pages, generator=g).tolist()
    page = lambda: pages.pop() * 16
    parts = [torch.tensor([page() + 3, page() + 9, page()])]                       # three loose tokens first: pages start at odd positions
    parts.append(page() + torch.arange(16))                                        # a whole page in order
    parts.append(page() + torch.arange(15, -1, -1))                                # a page in reverse order
    hole = page() + torch.arange(16); hole[5] = -1; parts.append(hole)             # a page with a skipped token
    parts.append(torch.cat([page() + torch.arange(16) for _ in range(12)]))        # a run of whole pages
    parts.append(torch.tensor([page() + i for i in (1, 15, 7)]))                   # loose tokens of one page
    parts.append(page() + torch.arange(8))                                         # half a page
    parts.append(torch.cat([page() + torch.arange(16) for _ in range(3)]))
    if n_extra:
        rest = torch.cat([page() + torch.arange(16) for _ in range(n_extra // 16)])
        parts.append(rest[torch.randperm(rest.numel(), generator=g)][: n_extra // 2])    # scattered
        parts.append(torch.cat([page() + torch.arange(16) for _ in range(20)]))
    slots = torch.cat(parts).to(torch.int64)
    n = slots.numel()
    K = (torch.randn((n, Hkv, D), generator=g) * 1.5).to(torch.bfloat16)
    V = (torch.randn((n, Hkv, D), generator=g) * torch.exp2(torch.randint(-6, 7, (n, 1, 1), generator=g).float())).to(torch.bfloat16)
    dw.cache.skv_append(0, K.to(dw.device), V.to(dw.device), slots.to(dw.device))
    torch.cuda.synchronize()
    assert dw.cache.skv_get_status() == 0
    keep = slots >= 0
    kc = torch.zeros((int(keep.sum()), Hkv, D), dtype=torch.uint8, device=dw.device)
    vc = torch.zeros_like(kc)
    ks = torch.zeros((kc.shape[0], Hkv), dtype=torch.float32, device=dw.device)
    vs = torch.zeros_like(ks)
    dw.cache.skv_gather_fp8(0, slots[keep].to(dw.device), kc, vc, ks, vs)
    torch.cuda.synchronize()
    okc, oks = quantize_e4m3(K[keep])
    ovc, ovs = quantize_e4m3(V[keep])
    assert torch.equal(kc.cpu(), okc) and torch.equal(vc.cpu(), ovc)
    assert torch.equal(ks.cpu().view(torch.int32), oks.view(torch.int32))
    assert torch.equal(vs.cpu().view(torch.int32), ovs.view(torch.int32))


def test_many_short_sequences():
    """Hundreds of sequences of at most one tile (128 tokens), more (sequence, kv head) segments than workers: every
    worker of the tcgen05 kernel goes through several one-tile runs back to back, the case in which its roles are
    furthest apart (queries of the run after next being prepared while the softmax is still on this one)."""
    g = torch.Generator().manual_seed(5)
    lens = torch.randint(1, 129, (320,), generator=g, dtype=torch.int32)
    lens[::7] = 128
    lens[3::11] = 0
    w = W.Workload("fp8_short", 2, 8, 4, 128, 16, lens.numel(), 0, 0, "explicit", explicit_r=(0, 0), seed=107)
    harness, dw = _setup(w, lens)
    o, _, _, _ = _oracle(dw, range(2))
    Q = harness.step_inputs(dw, 1)["Q"]
    ref = o.decode_attn(1, Q.cpu(), dw.lens_cpu)
    for overlap in (1, 0):
        dw.retune(overlap=overlap)
        for rep in range(5):
            out = torch.full((dw.batch, 8, 128), float("nan"), dtype=torch.bfloat16, device=dw.device)
            dw.cache.skv_decode_attn(1, Q, dw.page_table, dw.seq_lens, out, dw.workspace)
            torch.cuda.synchronize()
            assert dw.cache.skv_get_status() == 0
            err = (out.cpu().double() - ref).abs()
            assert bool((err <= ATOL + RTOL * ref.abs()).all()), f"overlap {overlap} rep {rep}: {err.max().item()}"


@pytest.mark.parametrize("trial", range(6))
def test_random_shapes_whole_steps(trial):
    """Seeded random batch, lengths and group size through whole decode steps (three layers reading layer 0: forward
    and backward walks, chained launches) against the oracle."""
    g = torch.Generator().manual_seed(200 + trial)
    Hkv = (1, 2, 4, 8, 2, 4)[trial]
    G = (8, 4, 3, 1, 2, 4)[trial]
    B = int(torch.randint(1, 14, (1,), generator=g))
    lens = torch.randint(0, (130, 700, 300, 140, 1200, 260)[trial], (B,), generator=g).to(torch.int32)
    lens[0] = max(int(lens[0]), 1)
    w = W.Workload("fp8_rand", 3, G * Hkv, Hkv, 128, 16, B, 0, 0, "explicit", explicit_r=(0, 0, 0), seed=300 + trial)
    from paper_2604_22782_b200 import harness
    dw = harness.setup(w, lens=lens, fp8=True)
    harness.prefill(dw, upto_offset=-1)
    t = harness.step_tensors(dw)
    o, _, _, _ = _oracle(dw, range(3))
    for rep in range(2):
        t["out"].fill_(float("nan"))
        dw.cache.skv_decode_step(t["Q"], t["K"], t["V"], dw.slot_new, dw.page_table, dw.seq_lens, t["out"], dw.workspace)
        torch.cuda.synchronize()
        assert dw.cache.skv_get_status() == 0
        for l in range(3):
            ref = o.decode_attn(l, t["Q"][l].cpu(), dw.lens_cpu)
            err = (t["out"][l].cpu().double() - ref).abs()
            assert bool((err <= ATOL + RTOL * ref.abs()).all()), f"rep {rep} layer {l}: {err.max().item()}"


def test_whole_step_and_unsupported_calls():
    from paper_2604_22782_b200 import harness
    from paper_2604_22782_b200.binding import SKV_ERR_UNSUPPORTED, SkvError
    lens = torch.tensor([700, 33, 1, 256, 1023, 90, 0, 15], dtype=torch.int32)
    w = W.Workload("fp8_step", 4, 8, 2, 128, 16, lens.numel(), 0, 0, "explicit", explicit_r=(0, 0, 2, 2), seed=103)
    dw = harness.setup(w, lens=lens, fp8=True)
    harness.prefill(dw, upto_offset=-1)
    t = harness.step_tensors(dw)
    o, _, _, _ = _oracle(dw, range(4))
    for rep in range(3):
        dw.retune(l2_keep=(35, 0, 60)[rep])      # layers 1 and 3 walk backward unless L2 reuse is off
        t["out"].fill_(float("nan"))
        dw.cache.skv_decode_step(t["Q"], t["K"], t["V"], dw.slot_new, dw.page_table, dw.seq_lens, t["out"], dw.workspace)
        torch.cuda.synchronize()
        for l in range(4):
            ref = o.decode_attn(l, t["Q"][l].cpu(), dw.lens_cpu)
            err = (t["out"][l].cpu().double() - ref).abs()
            assert bool((err <= ATOL + RTOL * ref.abs()).all()), f"rep {rep} layer {l}: {err.max().item()}"
    assert dw.cache.skv_get_status() == 0
    with pytest.raises(SkvError) as e:
        dw.cache.skv_gather(0, dw.slot_new, t["K"][0], t["V"][0])
    assert e.value.status == SKV_ERR_UNSUPPORTED
    dw.cache.skv_set_prefill_variant(2)              # the tcgen05 pre-fill kernel reads bf16 pages only
    inp = harness.prefill_inputs(dw, 0, torch.ones(lens.numel(), dtype=torch.int32))
    with pytest.raises(SkvError) as e:
        dw.cache.skv_prefill_attn(0, inp["Q"], inp["cu_q_lens"], dw.page_table, dw.seq_lens, torch.empty_like(inp["Q"]), 1)
    assert e.value.status == SKV_ERR_UNSUPPORTED


@pytest.mark.parametrize("scratch", [False, True])
@pytest.mark.parametrize("Hq,Hkv,D", [(8, 2, 128), (4, 4, 128), (8, 1, 128), (6, 2, 64), (6, 2, 128)])
def test_prefill_on_fp8_pages(Hq, Hkv, D, scratch):
    """Pre-fill attention over FP8 pages (whole prompts, chunks, single rows) against the oracle's rows over the
    dequantised values; unused slots of the pool hold NaN codes and NaN scales.  Without a scratch area: the
    mma.sync kernel that converts the codes on the way in; with one: the pages the call reaches are turned into
    bf16 there and the tcgen05 kernel runs on them (where it applies: head_dim 128, group sizes that divide 128)."""
    lens = torch.tensor([1, 15, 16, 17, 63, 64, 65, 100, 257, 700], dtype=torch.int32)
    w = W.Workload("fp8_pf", 3, Hq, Hkv, D, 16, lens.numel(), 0, 0, "explicit", explicit_r=(0, 0, 2), seed=109, kv_std=1.3)
    harness, dw = _setup(w, lens, poison=True)
    if scratch:
        need = dw.cache.skv_prefill_scratch_bytes()
        assert need == dw.total_pages * 2 * 16 * Hkv * D * 2
        area = torch.empty(need, dtype=torch.uint8, device=dw.device)
        area.view(torch.int16).fill_(0x7FC1)                    # NaN patterns: only converted pages may be read
        dw.cache.skv_set_prefill_scratch(area)
        launches = dw.cache.skv_launch_count()
    o, _, _, _ = _oracle(dw, range(3))
    v_abs_max = 4.5 * w.kv_std * (1 + 2.0 ** -4)          # the generator's largest value, after E4M3 rounding
    for layer, q_lens in ((0, lens), (1, lens), (2, lens), (1, torch.tensor([1, 7, 16, 1, 40, 0, 65, 3, 200, 129], dtype=torch.int32)),
                          (2, torch.ones(lens.numel(), dtype=torch.int32))):
        inp = harness.prefill_inputs(dw, layer, q_lens)
        out = torch.full_like(inp["Q"], float("nan"))
        dw.cache.skv_prefill_attn(layer, inp["Q"], inp["cu_q_lens"], dw.page_table, dw.seq_lens, out, max(1, int(q_lens.max())))
        torch.cuda.synchronize()
        ref = o.attn_rows(layer, inp["Q"].cpu(), inp["q_seq"], inp["q_pos"])
        err = (out.cpu().double() - ref).abs()
        # On the scratch path every dequantised value (code x scale, which the oracle sums exactly) is rounded to
        # bf16 once more before it is summed: up to 2^-9 of the largest |V| on top of the usual tolerance, which
        # shows where the terms of a row cancel (|ref| small beside the values summed).
        extra = (2.0 ** -9) * v_abs_max if scratch else 0.0
        assert bool((err <= ATOL + RTOL * ref.abs() + extra).all()), f"layer {layer}: max abs err {err.max().item()}"
        assert torch.isfinite(out.float()).all()
    assert dw.cache.skv_get_status() == 0
    if scratch:
        two_launches = D == 128 and 128 % (Hq // Hkv) == 0      # conversion + tcgen05 kernel; else the mma.sync kernel alone
        assert dw.cache.skv_launch_count() - launches == (10 if two_launches else 5)
        dw.cache.skv_set_prefill_scratch(None)
