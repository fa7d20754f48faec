"""Parity of the CUDA path (through the C ABI) against the CPU oracle, element by
element on the same seeded inputs.  Cache contents: bit-exact.  Attention
outputs: |out - ref| <= 1e-2 + 1e-2*|ref| (bf16 in, fp32 accumulate)."""
import pytest
import torch

import workloads as W

pytestmark = pytest.mark.gpu

ATOL, RTOL = 1e-2, 1e-2


def _within_tol(out_bf16, ref64):
    out = out_bf16.detach().cpu().double()
    err = (out - ref64).abs()
    bound = ATOL + RTOL * ref64.abs()
    worst = (err - bound).max().item()
    return worst <= 0.0, err.max().item()


def _make(w, **kw):
    from paper_2604_22782_b200 import harness
    return harness, harness.setup(w, **kw)


def _oracle_for(dw, seqs, layers_needed, upto_offset=0):
    """Oracle holding sequences `seqs` (their full lengths) for the given layers' own stores."""
    from oracle import Oracle
    w = dw.w
    sub_lens = dw.lens_cpu[seqs]
    o = Oracle(w.n_layers, dw.r, w.q_heads, w.kv_heads, w.head_dim, len(seqs), max(1, int(sub_lens.max())))
    local, pos = W.token_index(sub_lens, upto_offset)
    glob = torch.as_tensor(seqs, dtype=torch.int64)[local]
    for l in layers_needed:
        K, V = W.draw_kv(w, l, glob, pos)
        o.append(l, K, V, local, pos)
    return o


def _decode_layer(dw, layer, Q=None, scale=0.0):
    from paper_2604_22782_b200 import harness
    w = dw.w
    if Q is None:
        Q = harness.step_inputs(dw, layer)["Q"]
    out = torch.full((dw.batch, w.q_heads, w.head_dim), float("nan"), dtype=torch.bfloat16, device=dw.device)
    dw.cache.skv_decode_attn(layer, Q, dw.page_table, dw.seq_lens, out, dw.workspace, scale=scale)
    torch.cuda.synchronize()
    assert dw.cache.skv_get_status() == 0
    return Q, out


def _full_step_check(w, lens=None, r=None, variant=0, tuning=None, poison=False, permute=None, check_cache=True,
                     overlap=None, l2_keep=None, early_fetch=None, worker=None, merge=None):
    """One decode step of every layer: prefill n-1 tokens, append the last one, attend; compare all."""
    harness, dw = _make(w, lens=lens, r=r, permute=permute)
    if poison:   # every byte of the page area becomes a bf16 NaN pattern (0x7FC1)
        dw.pool_view = dw.cache.pool[256:].view(torch.int16)
        dw.pool_view.fill_(0x7FC1)
    dw.retune(variant=variant or None, tuning=tuning, overlap=overlap, l2_keep=l2_keep, early_fetch=early_fetch,
              worker=worker, merge=merge)
    B = dw.batch
    harness.prefill(dw, upto_offset=-1)
    seqs = list(range(B))
    o = _oracle_for(dw, seqs, range(w.n_layers), upto_offset=0)    # every layer keeps its own store
    worst = 0.0
    for l in range(w.n_layers):
        inp = harness.step_inputs(dw, l)
        before = dw.cache.skv_launch_count()
        dw.cache.skv_append(l, inp["K"], inp["V"], dw.slot_new)
        if dw.r[l] != l:
            assert dw.cache.skv_launch_count() == before      # non-owner: nothing launched
        Q, out = _decode_layer(dw, l, inp["Q"])
        ref = o.decode_attn(l, Q.cpu(), dw.lens_cpu)
        ok, err = _within_tol(out, ref)
        worst = max(worst, err)
        assert ok, f"layer {l}: max abs err {err}"
        assert torch.isfinite(out.float()).all()
    if check_cache:
        seq_idx, pos = W.token_index(dw.lens_cpu)
        slots = W.slot_map_for(dw.page_table_cpu, seq_idx, pos, w.page_size).to(dw.device)
        n = seq_idx.numel()
        for l in dw.owners:
            Kg = torch.zeros((n, w.kv_heads, w.head_dim), dtype=torch.bfloat16, device=dw.device)
            Vg = torch.zeros_like(Kg)
            dw.cache.skv_gather(l, slots, Kg, Vg)
            torch.cuda.synchronize()
            Kg, Vg = Kg.cpu().view(torch.int16), Vg.cpu().view(torch.int16)
            for i in range(0, n, max(1, n // 97)):
                k, v = o.read(l, int(seq_idx[i]), int(pos[i]))
                assert torch.equal(k.view(torch.int16), Kg[i]) and torch.equal(v.view(torch.int16), Vg[i])
            Kd, Vd = W.draw_kv(w, l, seq_idx, pos)            # what was appended, all rows
            assert torch.equal(Kd.view(torch.int16), Kg) and torch.equal(Vd.view(torch.int16), Vg)
    assert dw.cache.skv_get_status() == 0
    return worst


def test_tiny_config_every_layer():
    """Config 1: 4 layers r=[0,0,2,2], 4 q / 2 kv heads, D=64, lens {37,128}, contiguous pages."""
    w = W.get_workload("tiny")
    assert W.routing_map(w) == [0, 0, 2, 2] and W.seq_lens(w).tolist() == [37, 128]
    _full_step_check(w)


@pytest.mark.parametrize("Hq,Hkv,D", [(4, 4, 128), (4, 4, 64), (4, 2, 128), (8, 2, 128), (8, 2, 64), (8, 1, 128),
                                       (6, 2, 64), (3, 1, 128)])
def test_all_short_lengths(Hq, Hkv, D):
    """Every length 0..3*page_size (one sequence each; odd batch) for G in {1,2,3,4,8}, D in {64,128}."""
    lens = torch.arange(0, 3 * 16 + 1, dtype=torch.int32)
    w = W.Workload("short", 3, Hq, Hkv, D, 16, lens.numel(), 0, 48, "explicit", explicit_r=(0, 0, 2), seed=11)
    _full_step_check(w, lens=lens)


@pytest.mark.parametrize("Hq,Hkv,D", [(4, 4, 128), (8, 2, 128), (8, 2, 64), (3, 1, 128)])
def test_all_short_lengths_with_early_fetch(Hq, Hkv, D):
    """The same lengths with the split-K launch filling its rings before it waits for the kernel before it
    (the append of the step's token, or the kernel that produced Q): same outputs, same cache."""
    lens = torch.arange(0, 3 * 16 + 1, dtype=torch.int32)
    w = W.Workload("short", 3, Hq, Hkv, D, 16, lens.numel(), 0, 48, "explicit", explicit_r=(0, 0, 2), seed=11)
    _full_step_check(w, lens=lens, early_fetch=1)


def test_poisoned_pool_never_leaks():
    """Unused slots hold NaN patterns: tokens past seq_len must contribute nothing."""
    lens = torch.tensor([1, 5, 16, 17, 31, 33, 47, 100, 3], dtype=torch.int32)
    for Hq, Hkv in ((8, 2), (2, 2)):
        w = W.Workload("poison", 2, Hq, Hkv, 128, 16, lens.numel(), 0, 0, "explicit", explicit_r=(0, 0), seed=5)
        _full_step_check(w, lens=lens, poison=True, check_cache=False)


@pytest.mark.parametrize("variant,Hq,Hkv", [(2, 4, 4), (1, 4, 4), (2, 16, 4)])
def test_forced_variants_and_launch_shapes(variant, Hq, Hkv):
    """Tensor-core kernel on MHA, CUDA-core kernel, and other warps/stages/CTAs-per-SM settings."""
    lens = torch.tensor([700, 33, 1, 256, 1023, 90, 15], dtype=torch.int32)
    w = W.Workload("variants", 2, Hq, Hkv, 128, 16, lens.numel(), 0, 0, "explicit", explicit_r=(0, 0), seed=6)
    for tuning in ((4, 3, 2), (1, 2, 1), (8, 2, 1), (2, 6, 2), (3, 4, 3), (2, 2, 4), (1, 1, 8), (8, 1, 1)):
        _full_step_check(w, lens=lens, variant=variant, tuning=tuning, check_cache=False, worker=1)


@pytest.mark.parametrize("variant,Hq,Hkv,D", [(0, 8, 2, 128), (0, 4, 4, 128), (2, 4, 4, 64), (0, 16, 2, 64), (0, 3, 1, 128)])
def test_cta_worker_shapes(variant, Hq, Hkv, D):
    """The CTA-per-range kernel with other numbers of consumer warps and ring depths (ranges that hold many
    whole segments, segments cut by range ends, consumers without a block in a run), with and without
    early fetch, against the oracle; and the warp-per-range kernel on the same inputs."""
    lens = torch.tensor([700, 33, 1, 256, 1023, 90, 15, 0, 4100, 17, 16], dtype=torch.int32)
    w = W.Workload("cta", 3, Hq, Hkv, D, 16, lens.numel(), 0, 0, "explicit", explicit_r=(0, 0, 2), seed=67)
    for worker, early in (((2, 8, 0), 0), ((2, 1, 2), 0), ((2, 3, 5), 1), ((2, 5, 7), 0), ((2, 7, 4), 1),
                          ((2, 8, 20), 1), ((2, 2, 26), 0), ((3, 8, 0), 1), ((3, 3, 2), 0), ((3, 6, 4), 0),
                          ((2, 4, 0, 2), 1), ((2, 4, 6, 2), 0), ((2, 2, 4, 4), 1), ((2, 8, 0, 1), 0),
                          (1, 0), (1, 1)):
        _full_step_check(w, lens=lens, variant=variant, check_cache=False, worker=worker, early_fetch=early)


@pytest.mark.parametrize("Hq,Hkv,D", [(8, 2, 128), (16, 2, 64), (3, 1, 128)])
def test_merge_inside_the_cta_kernel(Hq, Hkv, D):
    """skv_set_decode_merge(2): segments cut by range ends are finished by the CTAs themselves, partials handed from
    range to range.  Few long segments (one spans dozens of ranges: a long chain of hand-overs), forward and
    backward walks (layers 0 and 1 read one owner), an empty sequence (its rows must be zeros), with and without
    early fetch, other consumer counts and ring depths; then a block list shorter than the number of CTAs (every
    range a single block); the calls of one handle reuse one workspace, so tags of earlier calls are in it."""
    lens = torch.tensor([700, 33, 1, 256, 1023, 90, 15, 0, 4100, 17, 16], dtype=torch.int32)
    w = W.Workload("cta_merge", 3, Hq, Hkv, D, 16, lens.numel(), 0, 0, "explicit", explicit_r=(0, 0, 2), seed=71)
    for worker, early in (((2, 8, 0), 0), ((2, 8, 0), 1), ((2, 3, 5), 1), ((2, 7, 4), 0), ((3, 6, 4), 1)):
        _full_step_check(w, lens=lens, check_cache=False, worker=worker, early_fetch=early, merge=2)
    short = torch.tensor([40, 17, 3, 0, 49], dtype=torch.int32)
    w2 = W.Workload("cta_merge_short", 3, Hq, Hkv, D, 16, short.numel(), 0, 0, "explicit", explicit_r=(0, 0, 2), seed=72)
    for early in (0, 1):
        _full_step_check(w2, lens=short, check_cache=False, worker=(2, 8, 0), early_fetch=early, merge=2)
    # (one launch per call then, not two)
    from paper_2604_22782_b200 import harness
    dw = harness.setup(w2, lens=short)
    dw.retune(merge=2)
    harness.prefill(dw, upto_offset=0)
    before = dw.cache.skv_launch_count()
    _decode_layer(dw, 0)
    assert dw.cache.skv_launch_count() == before + 1
    dw.retune(merge=1)
    _decode_layer(dw, 0)
    assert dw.cache.skv_launch_count() == before + 3
    # many short sequences: more segments than CTAs, the default picks in-kernel merging by itself
    many = torch.randint(1, 300, (200,), generator=torch.Generator().manual_seed(5), dtype=torch.int32)
    w3 = W.Workload("cta_merge_many", 2, Hq, Hkv, D, 16, many.numel(), 0, 0, "explicit", explicit_r=(0, 0), seed=73)
    _full_step_check(w3, lens=many, check_cache=False, early_fetch=1)
    _full_step_check(w3, lens=many, check_cache=False, early_fetch=0, merge=1)


def test_merge_inside_the_kernel_replayed_from_a_graph():
    """A call captured into a CUDA graph carries the same tag value in every replay: the tags of one replay must
    not pass for those of the next.  The query changes between replays; every replay is checked against the oracle."""
    from paper_2604_22782_b200 import harness
    lens = torch.tensor([700, 33, 1, 256, 1023, 90, 15, 0, 4100, 17, 16], dtype=torch.int32)
    w = W.Workload("cta_graph", 2, 8, 2, 128, 16, lens.numel(), 0, 0, "explicit", explicit_r=(0, 0), seed=74)
    dw = harness.setup(w, lens=lens)
    dw.retune(merge=2, early_fetch=1)
    harness.prefill(dw, upto_offset=0)
    o = _oracle_for(dw, list(range(dw.batch)), range(w.n_layers), upto_offset=0)
    Q = harness.step_inputs(dw, 1)["Q"].clone()
    out = torch.empty_like(Q)
    side = torch.cuda.Stream(device=dw.device)
    side.wait_stream(torch.cuda.current_stream(dw.device))
    with torch.cuda.stream(side):
        dw.cache.skv_decode_attn(1, Q, dw.page_table, dw.seq_lens, out, dw.workspace)
    torch.cuda.current_stream(dw.device).wait_stream(side)
    torch.cuda.synchronize()
    g = torch.cuda.CUDAGraph()
    with torch.cuda.graph(g, stream=side):
        dw.cache.skv_decode_attn(1, Q, dw.page_table, dw.seq_lens, out, dw.workspace)
    gen = torch.Generator(device="cpu").manual_seed(9)
    for rep in range(4):
        Q.copy_((torch.randn(Q.shape, generator=gen) * (0.5 + rep)).to(torch.bfloat16))
        out.fill_(float("nan"))
        g.replay()
        torch.cuda.synchronize()
        ref = o.decode_attn(1, Q.cpu(), dw.lens_cpu)
        ok, err = _within_tol(out, ref)
        assert ok, f"replay {rep}: max abs err {err}"
    assert dw.cache.skv_get_status() == 0


def test_cta_worker_long_segments_and_reverse_walks():
    """Segments much longer than a range (every CTA holds a piece of one segment and writes a partial), walked
    forwards and backwards with part of the stream kept in L2."""
    lens = torch.tensor([60000, 9000, 5], dtype=torch.int32)
    for Hq, Hkv in ((8, 2), (2, 2)):
        w = W.Workload("cta_long", 4, Hq, Hkv, 128, 16, lens.numel(), 0, 0, "explicit", explicit_r=(0, 0, 0, 3), seed=69)
        _full_step_check(w, lens=lens, check_cache=False, l2_keep=35, early_fetch=1)
        _full_step_check(w, lens=lens, check_cache=False, l2_keep=35, early_fetch=1, worker=(2, 4, 0, 2))


@pytest.mark.parametrize("overlap,l2_keep,early", [(1, 0, 0), (0, 0, 0), (1, 30, 0), (0, 100, 0), (1, 1, 0),
                                                   (1, 0, 1), (1, 35, 1), (0, 0, 1)])
def test_overlap_and_walk_directions(overlap, l2_keep, early):
    """Plain vs overlappable launches; forward-only walks vs alternating directions with part of each
    range kept in L2 (layers 0,1,2 read owner 0, layer 3 owns); rings filled before or after the wait
    on the previous kernel."""
    lens = torch.tensor([5000, 33, 1, 256, 1023, 0, 90, 15, 2048], dtype=torch.int32)
    for Hq, Hkv in ((8, 2), (2, 2)):
        w = W.Workload("walks", 4, Hq, Hkv, 128, 16, lens.numel(), 0, 0, "explicit", explicit_r=(0, 0, 0, 3), seed=31)
        _full_step_check(w, lens=lens, check_cache=False, overlap=overlap, l2_keep=l2_keep, early_fetch=early)


def test_early_fetch_sees_the_token_appended_just_before():
    """A decoder's order of events, repeated: a kernel writes Q, the update appends one token per sequence,
    the attention call follows at once with its rings filled early.  The newest token must be attended
    (it carries nearly all the weight here) although the launch started before the update finished, and
    the partials of the previous call must not be disturbed while its merge still reads them."""
    from paper_2604_22782_b200 import harness
    lens = torch.tensor([16, 17, 1, 33, 4000, 250, 64], dtype=torch.int32)
    w = W.Workload("early", 2, 8, 2, 128, 16, lens.numel(), 0, 0, "explicit", explicit_r=(0, 0), seed=61)
    dw = harness.setup(w, lens=lens)
    dw.retune(early_fetch=1)
    harness.prefill(dw, upto_offset=-1)
    o = _oracle_for(dw, list(range(dw.batch)), range(w.n_layers), upto_offset=-1)
    b = torch.arange(dw.batch, dtype=torch.int64)
    last = dw.lens_cpu.to(torch.int64) - 1
    shape = (dw.batch, w.q_heads, w.head_dim)
    outs, refs = [], []
    for rep in range(4):
        # the new token's K is a large multiple of the query direction, so it dominates the softmax
        Q = W.draw_rows(w.seed + rep, W.KIND_Q, 0, b, last, w.q_heads, w.head_dim, 1.0, dw.device)
        K = (Q[:, ::w.q_heads // w.kv_heads, :].float() * 4.0).to(torch.bfloat16).contiguous()
        V = W.draw_rows(w.seed + rep, W.KIND_V, 0, b, last, w.kv_heads, w.head_dim, 1.0, dw.device)
        o.append(0, K.cpu(), V.cpu(), b, last)
        out0 = torch.full(shape, float("nan"), dtype=torch.bfloat16, device=dw.device)
        out1 = torch.full(shape, float("nan"), dtype=torch.bfloat16, device=dw.device)
        Qd = torch.add(Q, out0.nan_to_num(0.0), alpha=0.0)       # Q comes out of a kernel of its own
        dw.cache.skv_append(0, K, V, dw.slot_new)
        dw.cache.skv_decode_attn(0, Qd, dw.page_table, dw.seq_lens, out0, dw.workspace)
        dw.cache.skv_decode_attn(1, Qd, dw.page_table, dw.seq_lens, out1, dw.workspace)   # back to back, same workspace
        outs.append((out0, out1))
        refs.append(o.decode_attn(0, Q.cpu(), dw.lens_cpu))
    torch.cuda.synchronize()
    assert dw.cache.skv_get_status() == 0
    for rep, ((out0, out1), ref) in enumerate(zip(outs, refs)):
        for out in (out0, out1):
            ok, err = _within_tol(out, ref)
            assert ok, f"rep {rep}: max abs err {err}"


def test_length_beyond_the_page_table_row_is_cut_and_flagged():
    """seq_lens[b] that needs more pages than a page_table row holds: no id is read past the row; the
    length is cut to the row and the device status says SKV_ERR_BOUNDS (decode and pre-fill)."""
    from paper_2604_22782_b200 import harness
    from paper_2604_22782_b200.binding import SKV_ERR_BOUNDS
    lens = torch.tensor([40, 64, 7], dtype=torch.int32)
    for fp8 in (False, True):
        w = W.Workload("ptrow", 1, 8, 2, 128, 16, lens.numel(), 0, 0, "explicit", explicit_r=(0,), seed=71)
        dw = harness.setup(w, lens=lens, fp8=fp8)
        harness.prefill(dw, upto_offset=0)
        width = dw.page_table.shape[1]
        assert width == 4
        Q = harness.step_inputs(dw, 0)["Q"]
        good = torch.full((dw.batch, w.q_heads, w.head_dim), float("nan"), dtype=torch.bfloat16, device=dw.device)
        dw.cache.skv_decode_attn(0, Q, dw.page_table, dw.seq_lens, good, dw.workspace)
        assert dw.cache.skv_get_status() == 0
        too_long = dw.seq_lens.clone()
        too_long[2] = width * 16 + 1            # the LAST row: ids past it would lie outside the tensor
        out = torch.full_like(good, float("nan"))
        dw.cache.skv_decode_attn(0, Q, dw.page_table, too_long, out, dw.workspace)
        assert dw.cache.skv_get_status() == SKV_ERR_BOUNDS
        ok, err = _within_tol(out[:2], good[:2].cpu().double())                       # the other rows are unaffected
        assert ok, err
        assert torch.isfinite(out.float()).all()
        cu = torch.tensor([0, 1, 2, 3], dtype=torch.int32, device=dw.device)
        pout = torch.full_like(good, float("nan"))
        dw.cache.skv_prefill_attn(0, Q, cu, dw.page_table, too_long, pout, 1)
        assert dw.cache.skv_get_status() == SKV_ERR_BOUNDS
        assert torch.isnan(pout[2].float()).all()                # rows of the offending sequence are left untouched
        assert torch.isfinite(pout[:2].float()).all()


def test_workspace_query_matches_the_launch_after_retuning():
    """skv_decode_workspace_bytes is what the launches check against, whatever the variant and launch shape."""
    from paper_2604_22782_b200 import harness
    lens = torch.tensor([300, 77, 512, 129], dtype=torch.int32)
    for fp8 in (False, True):
        w = W.Workload("wsq", 1, 32, 8, 128, 16, lens.numel(), 0, 0, "explicit", explicit_r=(0,), seed=73)
        dw = harness.setup(w, lens=lens, fp8=fp8)
        harness.prefill(dw, upto_offset=0)
        Q = harness.step_inputs(dw, 0)["Q"]
        first = None
        for variant, tuning in ((0, None), (2, None), (2, (1, 2, 1)), (2, (4, 2, 3)), (0, (2, 2, 8))):
            dw.cache.skv_set_decode_variant(variant)
            if tuning:
                dw.cache.skv_set_decode_tuning(*tuning)
            need = dw.cache.skv_decode_workspace_bytes(dw.batch, w.q_heads)
            ws = torch.empty(need, dtype=torch.uint8, device=dw.device)      # exactly what the query says
            out = torch.full((dw.batch, w.q_heads, w.head_dim), float("nan"), dtype=torch.bfloat16, device=dw.device)
            dw.cache.skv_decode_attn(0, Q, dw.page_table, dw.seq_lens, out, ws)
            assert dw.cache.skv_get_status() == 0
            first = out if first is None else first
            ok, err = _within_tol(out, first.cpu().double())
            assert ok, (fp8, variant, tuning, err)
            if need > 256:
                with pytest.raises(Exception):
                    dw.cache.skv_decode_attn(0, Q, dw.page_table, dw.seq_lens, out, ws[:need - 256])


@pytest.mark.parametrize("overlap,l2_keep", [(1, 0), (1, 40), (0, 0)])
@pytest.mark.parametrize("Hq,Hkv,D", [(8, 2, 128), (4, 4, 128), (4, 2, 64)])
def test_whole_step_entry_points_match_the_oracle(overlap, l2_keep, Hq, Hkv, D):
    """skv_decode_step (all updates first, then the chained attention launches) and skv_decode_step_host
    against the oracle for every layer, and against each other bit for bit, repeated to reuse both
    workspace buffers."""
    from paper_2604_22782_b200 import harness
    lens = torch.tensor([700, 33, 1, 256, 1023, 90, 0, 15, 3000, 16, 17], dtype=torch.int32)
    w = W.Workload("step", 5, Hq, Hkv, D, 16, lens.numel(), 0, 0, "explicit", explicit_r=(0, 0, 2, 2, 2), seed=43)
    dw = harness.setup(w, lens=lens)
    dw.retune(overlap=overlap, l2_keep=l2_keep)
    harness.prefill(dw, upto_offset=-1)
    t = harness.step_tensors(dw)
    o = _oracle_for(dw, list(range(dw.batch)), range(w.n_layers))
    refs = [o.decode_attn(l, t["Q"][l].cpu(), dw.lens_cpu) for l in range(w.n_layers)]
    for rep in range(3):
        t["out"].fill_(float("nan"))
        dw.cache.skv_decode_step(t["Q"], t["K"], t["V"], dw.slot_new, dw.page_table, dw.seq_lens, t["out"],
                                 dw.workspace)
        torch.cuda.synchronize()
        assert dw.cache.skv_get_status() == 0
        for l in range(w.n_layers):
            ok, err = _within_tol(t["out"][l], refs[l])
            assert ok, f"rep {rep} layer {l}: max abs err {err}"
    hb = harness.step_tensors(dw, device="cpu", pin=True)
    staging = torch.empty(dw.cache.skv_decode_step_staging_bytes(dw.batch, w.q_heads, dw.page_table_cpu.shape[1]),
                          dtype=torch.uint8, device=dw.device)
    h_slot, h_pt, h_len = (dw.slot_new.cpu().pin_memory(), dw.page_table_cpu.contiguous().pin_memory(),
                           dw.lens_cpu.contiguous().pin_memory())
    pageable_out = torch.empty_like(hb["out"], pin_memory=False)
    # every cut of the step, into pinned or pageable result buffers: one answer
    for groups, direct, h_out in ((4, 1, hb["out"]), (4, 0, hb["out"]), (1, 1, hb["out"]), (8, 1, hb["out"]),
                                  (3, 0, hb["out"]), (5, 1, pageable_out)):
        dw.cache.skv_set_host_step(groups, direct)
        h_out.fill_(float("nan"))
        dw.cache.skv_decode_step_host(hb["Q"], hb["K"], hb["V"], h_slot, h_pt, h_len, h_out, staging)
        torch.cuda.synchronize()
        assert dw.cache.skv_get_status() == 0
        assert torch.equal(h_out.view(torch.int16), t["out"].cpu().view(torch.int16)), (groups, direct)
    # the updates really happened: the newest token of every owner layer reads back bit-exactly
    has = dw.slot_new >= 0
    for i, l in enumerate(dw.owners):
        Kg = torch.zeros_like(t["K"][i])
        Vg = torch.zeros_like(Kg)
        dw.cache.skv_gather(l, dw.slot_new, Kg, Vg)
        torch.cuda.synchronize()
        assert torch.equal(Kg[has].view(torch.int16), t["K"][i][has].view(torch.int16))
        assert torch.equal(Vg[has].view(torch.int16), t["V"][i][has].view(torch.int16))


def test_repeated_calls_leave_the_workspace_reusable():
    """The control words return to zero after every launch: many calls on one workspace give one answer."""
    from paper_2604_22782_b200 import harness
    lens = torch.tensor([3000, 100, 777, 16, 1], dtype=torch.int32)
    w = W.Workload("repeat", 1, 8, 2, 128, 16, lens.numel(), 0, 0, "explicit", explicit_r=(0,), seed=37)
    dw = harness.setup(w, lens=lens)
    harness.prefill(dw, upto_offset=0)
    first = _decode_layer(dw, 0)[1].clone()
    for _ in range(20):
        again = _decode_layer(dw, 0)[1]
        assert torch.equal(first.view(torch.int16), again.view(torch.int16))


def test_page_permutation_does_not_change_outputs():
    lens = torch.tensor([300, 77, 512, 129], dtype=torch.int32)
    w = W.Workload("perm", 2, 8, 2, 128, 16, lens.numel(), 0, 0, "explicit", explicit_r=(0, 0), seed=8)
    from paper_2604_22782_b200 import harness
    outs = []
    for permute in (False, True):
        dw = harness.setup(w, lens=lens, permute=permute, extra_pages=13)
        harness.prefill(dw, upto_offset=0)
        outs.append(_decode_layer(dw, 1)[1].cpu())
    assert torch.equal(outs[0].view(torch.int16), outs[1].view(torch.int16))


def test_non_owner_append_is_a_noop_and_null_inputs_are_fine():
    from paper_2604_22782_b200 import harness
    w = W.get_workload("tiny")
    dw = harness.setup(w)
    harness.prefill(dw, upto_offset=0)
    snap = dw.cache.pool.clone()
    count = dw.cache.skv_launch_count()
    for l in (1, 3):
        inp = harness.step_inputs(dw, l)
        dw.cache.skv_append(l, inp["K"], inp["V"], dw.slot_new)
        dw.cache.skv_append(l, None, None, None, n_tokens=dw.batch)
    torch.cuda.synchronize()
    assert dw.cache.skv_launch_count() == count
    assert torch.equal(snap, dw.cache.pool)
    with pytest.raises(Exception):
        dw.cache.skv_append(0, None, None, dw.slot_new)       # an owner needs real K,V


@pytest.mark.parametrize("D", [128, 64])
@pytest.mark.parametrize("n_extra", [0, 700])     # below and above the size at which the page-granular update kernel takes over
def test_update_with_arbitrary_slot_maps(n_extra, D):
    """skv_append with slot maps that mix whole pages at odd positions of the call, pages in reverse order,
    pages with a skipped token, scattered single slots, runs of whole pages and a ragged end: every written
    slot reads back bit for bit, nothing else is touched, for both update kernels."""
    from paper_2604_22782_b200 import harness
    Hkv = 2
    n_pages = 120
    lens = torch.tensor([n_pages * 16], dtype=torch.int32)
    w = W.Workload("slots", 1, 4, Hkv, D, 16, 1, 0, 0, "explicit", explicit_r=(0,), seed=113)
    dw = harness.setup(w, lens=lens)
    g = torch.Generator().manual_seed(17)
    pages = torch.randperm(n_pages, generator=g).tolist()
    page = lambda: pages.pop() * 16
    parts = [torch.tensor([page() + 3, page() + 9, page()])]                       # three loose tokens first: pages start at odd positions
    parts.append(page() + torch.arange(16))                                        # a whole page in order
    parts.append(page() + torch.arange(15, -1, -1))                                # a page in reverse order
    hole = page() + torch.arange(16); hole[5] = -1; parts.append(hole)             # a page with a skipped token
    parts.append(torch.tensor([-1]))                                               # realign: whole pages on group boundaries from here
    parts.append(torch.cat([page() + torch.arange(16) for _ in range(12)]))        # a run of whole pages
    parts.append(torch.tensor([page() + i for i in (1, 15, 7)]))                   # loose tokens of one page
    parts.append(page() + torch.arange(8))                                         # half a page
    parts.append(torch.cat([page() + torch.arange(16) for _ in range(3)]))
    if n_extra:
        rest = torch.cat([page() + torch.arange(16) for _ in range(n_extra // 16)])
        parts.append(rest[torch.randperm(rest.numel(), generator=g)][: n_extra // 2])    # scattered
        pad = (-sum(x.numel() for x in parts)) % 16
        parts.append(torch.full((pad,), -1))
        parts.append(torch.cat([page() + torch.arange(16) for _ in range(20)]))    # whole pages on group boundaries
        parts.append(page() + torch.arange(5))                                     # ragged end of the call
    slots = torch.cat(parts).to(torch.int64)
    n = slots.numel()
    K = torch.randn((n, Hkv, D), generator=g).to(torch.bfloat16)
    V = torch.randn((n, Hkv, D), generator=g).to(torch.bfloat16)
    before = dw.cache.pool.clone()
    dw.cache.skv_append(0, K.to(dw.device), V.to(dw.device), slots.to(dw.device))
    torch.cuda.synchronize()
    assert dw.cache.skv_get_status() == 0
    keep = slots >= 0
    Kg = torch.zeros((int(keep.sum()), Hkv, D), dtype=torch.bfloat16, device=dw.device)
    Vg = torch.zeros_like(Kg)
    dw.cache.skv_gather(0, slots[keep].to(dw.device), Kg, Vg)
    torch.cuda.synchronize()
    assert torch.equal(Kg.cpu().view(torch.int16), K[keep].view(torch.int16))
    assert torch.equal(Vg.cpu().view(torch.int16), V[keep].view(torch.int16))
    # nothing but the named slots changed: every other slot of the layer reads back as before (zeros)
    others = torch.ones(n_pages * 16, dtype=torch.bool)
    others[slots[keep]] = False
    idx = torch.nonzero(others).flatten().to(dw.device)
    Ko = torch.ones((idx.numel(), Hkv, D), dtype=torch.bfloat16, device=dw.device)
    Vo = torch.ones_like(Ko)
    dw.cache.skv_gather(0, idx, Ko, Vo)
    torch.cuda.synchronize()
    assert torch.count_nonzero(Ko.view(torch.int16)) == 0 and torch.count_nonzero(Vo.view(torch.int16)) == 0
    assert torch.equal(before[:256], dw.cache.pool[:256])
    # a slot past the pool in a large call is flagged and skipped
    if n_extra:
        from paper_2604_22782_b200.binding import SKV_ERR_BOUNDS
        bad = slots.clone()
        bad[40] = n_pages * 16 + 3
        dw.cache.skv_append(0, K.to(dw.device), V.to(dw.device), bad.to(dw.device))
        assert dw.cache.skv_get_status() == SKV_ERR_BOUNDS


def test_out_of_range_ids_are_flagged_not_followed():
    """Bad slot / page ids raise the device status word; nothing is read or written out of bounds."""
    from paper_2604_22782_b200 import harness
    from paper_2604_22782_b200.binding import SKV_ERR_BOUNDS
    w = W.get_workload("tiny")
    dw = harness.setup(w)
    harness.prefill(dw, upto_offset=0)
    inp = harness.step_inputs(dw, 0)
    bad = dw.slot_new.clone()
    bad[0] = dw.total_pages * w.page_size + 5
    dw.cache.skv_append(0, inp["K"], inp["V"], bad)
    assert dw.cache.skv_get_status() == SKV_ERR_BOUNDS
    assert dw.cache.skv_get_status() == 0                      # reading clears it
    pt = dw.page_table.clone()
    pt[1, 2] = dw.total_pages + 7
    out = torch.zeros((dw.batch, w.q_heads, w.head_dim), dtype=torch.bfloat16, device=dw.device)
    dw.cache.skv_decode_attn(0, inp["Q"], pt, dw.seq_lens, out, dw.workspace)
    assert dw.cache.skv_get_status() == SKV_ERR_BOUNDS


def test_medium_llama3_shape_ragged():
    """Llama-3-8B head shape, 12 ragged sequences spanning many pages and several workers' ranges."""
    lens = torch.tensor([1000, 17, 640, 333, 2049, 1, 16, 999, 1500, 48, 777, 1211], dtype=torch.int32)
    w = W.Workload("medium", 4, 32, 8, 128, 16, lens.numel(), 0, 0, "groups", group=2, seed=21)
    _full_step_check(w, lens=lens)


def test_medium_mha_long_sequence_split_and_merge():
    """MHA, one 20k-token sequence + short ones: one segment is split over many workers and merged."""
    lens = torch.tensor([20000, 5, 300], dtype=torch.int32)
    w = W.Workload("mha_long", 2, 4, 4, 128, 16, lens.numel(), 0, 0, "explicit", explicit_r=(0, 0), seed=23)
    _full_step_check(w, lens=lens, check_cache=False)


def test_explicit_scale_is_used():
    from paper_2604_22782_b200 import harness
    lens = torch.tensor([200, 31], dtype=torch.int32)
    w = W.Workload("scale", 1, 8, 2, 128, 16, 2, 0, 0, "explicit", explicit_r=(0,), seed=29)
    dw = harness.setup(w, lens=lens)
    harness.prefill(dw, upto_offset=0)
    o = _oracle_for(dw, [0, 1], [0])
    Q, out = _decode_layer(dw, 0, scale=0.031)
    ok, err = _within_tol(out, o.decode_attn(0, Q.cpu(), dw.lens_cpu, 0.031))
    assert ok, err
    ok_default, _ = _within_tol(out, o.decode_attn(0, Q.cpu(), dw.lens_cpu))
    assert not ok_default


@pytest.mark.parametrize("B,Hq,Hkv,hi", [(300, 4, 1, 40), (3000, 4, 2, 48), (700, 8, 8, 33)])
def test_many_short_sequences(B, Hq, Hkv, hi):
    """Large batches of very short sequences (some empty): fewer blocks than workers in the first case
    (every worker holds at most one block), several whole segments per worker in the others."""
    g = torch.Generator().manual_seed(B)
    lens = torch.randint(0, hi + 1, (B,), generator=g, dtype=torch.int32)
    w = W.Workload("short_many", 2, Hq, Hkv, 128, 16, B, 0, hi, "explicit", explicit_r=(0, 0), seed=51)
    _full_step_check(w, lens=lens, check_cache=False)


def test_all_sequences_empty():
    """Nothing cached anywhere: every output row is zero and nothing is read."""
    from paper_2604_22782_b200 import harness
    lens = torch.zeros(5, dtype=torch.int32)
    w = W.Workload("empty", 1, 8, 2, 128, 16, 5, 0, 0, "explicit", explicit_r=(0,), seed=53)
    dw = harness.setup(w, lens=lens)
    _, out = _decode_layer(dw, 0)
    assert torch.count_nonzero(out.view(torch.int16)) == 0
