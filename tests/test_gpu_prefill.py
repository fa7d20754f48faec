"""Pre-fill attention (many query tokens per sequence, causal, over the routed owner's pages) through the
C ABI against the oracle's pre-fill rows, element by element: |out - ref| <= 1e-2 + 1e-2 |ref|."""
import pytest
import torch

import workloads as W

pytestmark = pytest.mark.gpu

ATOL, RTOL = 1e-2, 1e-2


def _setup(w, lens, poison=False, variant=0):
    from paper_2604_22782_b200 import harness
    dw = harness.setup(w, lens=lens)
    dw.cache.skv_set_prefill_variant(variant)
    if poison:
        dw.cache.pool[256:].view(torch.int16).fill_(0x7FC1)
    harness.prefill(dw, upto_offset=0)               # every token of every owner layer is cached
    return harness, dw


def _oracle(dw, layers):
    from oracle import Oracle
    w = dw.w
    o = Oracle(w.n_layers, dw.r, w.q_heads, w.kv_heads, w.head_dim, dw.batch, max(1, int(dw.lens_cpu.max())))
    si, pos = W.token_index(dw.lens_cpu)
    for src in sorted({dw.r[l] for l in layers}):
        K, V = W.draw_kv(w, src, si, pos)
        o.append(src, K, V, si, pos)
    return o


def _run(harness, dw, layer, q_lens, scale=0.0, rows=None):
    inp = harness.prefill_inputs(dw, layer, q_lens)
    out = torch.full_like(inp["Q"], float("nan"))
    dw.cache.skv_prefill_attn(layer, inp["Q"], inp["cu_q_lens"], dw.page_table, dw.seq_lens, out,
                              max(1, int(q_lens.max())), scale=scale)
    torch.cuda.synchronize()
    return inp, out


def _check(o, layer, inp, out, rows=None, scale=None):
    sel = slice(None) if rows is None else rows
    ref = o.attn_rows(layer, inp["Q"].cpu()[sel], inp["q_seq"][sel], inp["q_pos"][sel], scale)
    got = out.cpu()[sel].double()
    err = (got - ref).abs()
    assert bool((err <= ATOL + RTOL * ref.abs()).all()), f"layer {layer}: max abs err {err.max().item()}"
    return err.max().item()


@pytest.mark.parametrize("variant", [1, 0])       # the mma.sync kernel; automatic (tcgen05 kernel where it applies)
@pytest.mark.parametrize("Hq,Hkv,D", [(8, 2, 128), (4, 4, 128), (8, 1, 128), (6, 2, 64), (4, 2, 64), (2, 1, 128), (6, 2, 128)])
def test_whole_prompts_ragged(Hq, Hkv, D, variant):
    """Every token of every sequence is a query (q_len = seq_len): lengths around page and tile edges."""
    lens = torch.tensor([1, 15, 16, 17, 63, 64, 65, 100, 257, 700], dtype=torch.int32)
    w = W.Workload("pf", 3, Hq, Hkv, D, 16, lens.numel(), 0, 0, "explicit", explicit_r=(0, 0, 2), seed=61)
    harness, dw = _setup(w, lens, variant=variant)
    o = _oracle(dw, range(3))
    for layer in range(3):
        inp, out = _run(harness, dw, layer, lens)
        _check(o, layer, inp, out)
        assert torch.isfinite(out.float()).all()
    assert dw.cache.skv_get_status() == 0


@pytest.mark.parametrize("variant", [1, 2])
def test_chunks_of_a_prompt_and_single_rows(variant):
    """Chunked pre-fill (the last q_len tokens only), sequences with no query at all, and one row per
    sequence, which must agree with the decode step's entry point."""
    lens = torch.tensor([900, 33, 128, 2049, 5, 300], dtype=torch.int32)
    w = W.Workload("pf_chunk", 2, 8, 2, 128, 16, lens.numel(), 0, 0, "explicit", explicit_r=(0, 0), seed=67)
    harness, dw = _setup(w, lens, poison=True, variant=variant)
    o = _oracle(dw, [1])
    for q_lens in ([100, 33, 0, 513, 1, 17], [1, 1, 1, 1, 1, 1], [0, 0, 128, 0, 5, 0]):
        ql = torch.tensor(q_lens, dtype=torch.int32)
        inp, out = _run(harness, dw, 1, ql)
        _check(o, 1, inp, out)
        assert torch.isfinite(out.float()).all()
    # one row per sequence = Algorithm 2's decode attention
    ones = torch.ones(lens.numel(), dtype=torch.int32)
    inp, out = _run(harness, dw, 1, ones)
    dec = torch.empty_like(out)
    dw.cache.skv_decode_attn(1, inp["Q"], dw.page_table, dw.seq_lens, dec, dw.workspace)
    torch.cuda.synchronize()
    assert bool(((out.float() - dec.float()).abs() <= ATOL + RTOL * dec.float().abs()).all())
    assert dw.cache.skv_get_status() == 0


@pytest.mark.parametrize("variant", [1, 2])
def test_explicit_scale_and_bad_lengths(variant):
    from paper_2604_22782_b200.binding import SKV_ERR_BOUNDS
    lens = torch.tensor([70, 40], dtype=torch.int32)
    w = W.Workload("pf_scale", 1, 4, 2, 128, 16, 2, 0, 0, "explicit", explicit_r=(0,), seed=71)
    harness, dw = _setup(w, lens, variant=variant)
    o = _oracle(dw, [0])
    inp, out = _run(harness, dw, 0, lens, scale=0.05)
    _check(o, 0, inp, out, scale=0.05)
    assert dw.cache.skv_get_status() == 0
    # more query rows than cached tokens: flagged, rows untouched
    cu = torch.tensor([0, 80, 120], dtype=torch.int32, device=dw.device)
    Q = torch.zeros((120, 4, 128), dtype=torch.bfloat16, device=dw.device)
    out = torch.full_like(Q, 7.0)
    dw.cache.skv_prefill_attn(0, Q, cu, dw.page_table, dw.seq_lens, out, 80)
    assert dw.cache.skv_get_status() == SKV_ERR_BOUNDS
    assert bool((out[:80] == 7.0).all())


@pytest.mark.parametrize("variant", [1, 2])
def test_llama3_8b_shape_prompts_sampled_rows(variant):
    """Llama-3-8B head shape, 4 prompts of 1024..4096 tokens in layer 1 (reads layer 0): sampled rows
    (first, last, tile edges, seeded picks of every sequence) against the oracle; all rows finite and bounded."""
    w0 = W.get_workload("llama3_8b")
    w = W.Workload("pf_l3", 2, w0.q_heads, w0.kv_heads, w0.head_dim, 16, 4, 1024, 4096, "groups", group=2, seed=73)
    lens = W.seq_lens(w)
    harness, dw = _setup(w, lens, variant=variant)
    inp, out = _run(harness, dw, 1, lens)
    assert dw.cache.skv_get_status() == 0
    from oracle import Oracle
    o = Oracle(w.n_layers, dw.r, w.q_heads, w.kv_heads, w.head_dim, dw.batch, int(lens.max()))
    si, pos = W.token_index(lens)
    K, V = W.draw_kv(w, 0, si, pos, device=dw.device)
    o.append(0, K.cpu(), V.cpu(), si, pos)
    g = torch.Generator().manual_seed(5)
    rows, start = [], 0
    for n in lens.tolist():
        picks = {0, 1, 15, 16, 17, n // 2, n - 17, n - 16, n - 2, n - 1} | set(torch.randint(0, n, (6,), generator=g).tolist())
        rows += [start + i for i in sorted(picks)]
        start += n
    _check(o, 1, inp, out, rows=torch.tensor(rows))
    f = out.float()
    assert torch.isfinite(f).all() and f.abs().max().item() <= 5.0


def test_tcgen05_variant_is_refused_where_it_does_not_apply():
    from paper_2604_22782_b200.binding import SKV_ERR_UNSUPPORTED, SkvError
    lens = torch.tensor([20], dtype=torch.int32)
    w = W.Workload("pf_no", 1, 6, 2, 64, 16, 1, 0, 0, "explicit", explicit_r=(0,), seed=79)     # head_dim 64, G = 3
    harness, dw = _setup(w, lens, variant=2)
    inp = harness.prefill_inputs(dw, 0, lens)
    with pytest.raises(SkvError) as e:
        dw.cache.skv_prefill_attn(0, inp["Q"], inp["cu_q_lens"], dw.page_table, dw.seq_lens, torch.empty_like(inp["Q"]), 20)
    assert e.value.status == SKV_ERR_UNSUPPORTED


@pytest.mark.parametrize("Hq,Hkv", [(4, 4), (8, 2)])
def test_tcgen05_repeated_calls_stay_correct(Hq, Hkv):
    """The warps of the tcgen05 kernel run far apart (softmax, tensor-core issue, copies): many calls on
    tiles of one and two key blocks (where a warp that is a phase early shows up) must all give the
    oracle's rows, and the same bits every time."""
    lens = torch.tensor([1, 15, 16, 17, 63, 64, 65, 100, 257, 700], dtype=torch.int32)
    w = W.Workload("pf_rep", 2, Hq, Hkv, 128, 16, lens.numel(), 0, 0, "explicit", explicit_r=(0, 0), seed=83)
    harness, dw = _setup(w, lens, variant=2)
    o = _oracle(dw, [1])
    inp, first = _run(harness, dw, 1, lens)
    _check(o, 1, inp, first)
    for _ in range(40):
        _, again = _run(harness, dw, 1, lens)
        assert torch.equal(again.view(torch.int16), first.view(torch.int16))
    assert dw.cache.skv_get_status() == 0


@pytest.mark.parametrize("sampler", ["rcla", "rdcla"])
def test_training_time_routed_forward(sampler):
    """Section 3.2: one forward pass in which every layer draws its K,V source.  Every layer keeps its own
    K,V (identity map in the cache); layer l attends the layer the sampler gave it.  The oracle applies the
    sampled map by indexing (it may send a layer to a layer that itself reads elsewhere)."""
    from oracle import Oracle
    from paper_2604_22782_b200 import skv_routing_rcla, skv_routing_rdcla
    L, Hq, Hkv, D = 8, 8, 2, 128
    lens = torch.tensor([200, 77, 513], dtype=torch.int32)
    w = W.Workload("train_fwd", L, Hq, Hkv, D, 16, lens.numel(), 0, 0, "explicit", explicit_r=tuple(range(L)), seed=89)
    harness, dw = _setup(w, lens)
    si, pos = W.token_index(lens)
    g = torch.Generator().manual_seed(11)
    for trial in range(3):
        u, v = torch.rand(L, generator=g, dtype=torch.float64).tolist(), torch.rand(L, generator=g, dtype=torch.float64).tolist()
        m = skv_routing_rcla(0.4, u, v) if sampler == "rcla" else skv_routing_rdcla(4, 0.4, u)
        assert any(s != l for l, s in enumerate(m))                 # the pass really routes somewhere
        o = Oracle(L, m, Hq, Hkv, D, lens.numel(), int(lens.max()))
        for src in sorted(set(m)):
            K, V = W.draw_kv(w, src, si, pos)
            o.append(src, K, V, si, pos)
        for l in range(L):
            inp = harness.prefill_inputs(dw, l, lens)
            out = torch.full_like(inp["Q"], float("nan"))
            dw.cache.skv_prefill_attn_src(m[l], inp["Q"], inp["cu_q_lens"], dw.page_table, dw.seq_lens, out, int(lens.max()))
            torch.cuda.synchronize()
            _check(o, l, inp, out)
    assert dw.cache.skv_get_status() == 0
