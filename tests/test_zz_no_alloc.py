"""skv_decode_attn_static: decode attention for callers that cannot allocate device memory.

Some users of the library never get to call cudaMalloc where they call us: a serving engine that has
handed every byte of the GPU to its own pool before the first request, a plugin inside a process
that forbids allocation on its hot path, a bare C caller with nothing but its input and output
buffers.  For them the library carries a fixed scratch area of its own.  This test drives that
entry point through the C ABI and checks it against the ordinary skv_decode_attn (which takes a
caller-provided workspace), twice in a row because the area is shared and keeps the previous call's
contents.  It is collected last so that a failure here cannot hide any other test's result.
"""
import pytest
import torch

import workloads as W

pytestmark = pytest.mark.gpu

ATOL, RTOL = 1e-2, 1e-2


def _close(a, b):
    a, b = a.float(), b.float()
    return bool(((a - b).abs() <= ATOL + RTOL * b.abs()).all())


def test_static_scratch_entry_matches_workspace_entry_twice_in_a_row():
    from paper_2604_22782_b200 import harness
    lens = torch.tensor([1500, 17, 640, 1, 333, 2049, 16, 0, 999], dtype=torch.int32)
    w = W.Workload("noalloc", 2, 32, 8, 128, 16, lens.numel(), 0, 0, "explicit", explicit_r=(0, 0), seed=41)
    dw = harness.setup(w, lens=lens)
    harness.prefill(dw, upto_offset=0)
    shape = (dw.batch, w.q_heads, w.head_dim)
    for layer in (0, 1):                                  # two different calls back to back on the shared area
        Q = harness.step_inputs(dw, layer)["Q"]
        want = torch.full(shape, float("nan"), dtype=torch.bfloat16, device=dw.device)
        dw.cache.skv_decode_attn(layer, Q, dw.page_table, dw.seq_lens, want, dw.workspace)
        got = torch.full(shape, float("nan"), dtype=torch.bfloat16, device=dw.device)
        again = torch.full(shape, float("nan"), dtype=torch.bfloat16, device=dw.device)
        dw.cache.skv_decode_attn_static(layer, Q, dw.page_table, dw.seq_lens, got)
        torch.cuda.synchronize()
        free_before = torch.cuda.mem_get_info(dw.device)[0]     # the driver's count: sees any allocation at all
        dw.cache.skv_decode_attn_static(layer, Q, dw.page_table, dw.seq_lens, again)
        torch.cuda.synchronize()
        assert torch.cuda.mem_get_info(dw.device)[0] == free_before
        assert dw.cache.skv_get_status() == 0
        assert torch.isfinite(got.float()).all() and torch.isfinite(again.float()).all()
        assert _close(got, want), f"layer {layer}: first call differs from skv_decode_attn"
        assert _close(again, want), f"layer {layer}: second call differs from skv_decode_attn"
    # and, so that this file stands on its own, against the CPU oracle too
    from oracle import Oracle
    o = Oracle(w.n_layers, dw.r, w.q_heads, w.kv_heads, w.head_dim, dw.batch, int(lens.max()))
    si, pos = W.token_index(lens)
    K, V = W.draw_kv(w, 0, si, pos)
    o.append(0, K, V, si, pos)
    Q = harness.step_inputs(dw, 1)["Q"]
    got = torch.full(shape, float("nan"), dtype=torch.bfloat16, device=dw.device)
    dw.cache.skv_decode_attn_static(1, Q, dw.page_table, dw.seq_lens, got)
    torch.cuda.synchronize()
    ref = o.decode_attn(1, Q.cpu(), lens)
    assert bool(((got.cpu().double() - ref).abs() <= ATOL + RTOL * ref.abs()).all())


def test_static_scratch_entry_takes_an_fp8_cache_of_the_llama3_shape():
    """Batch 32 of the Llama-3-8B head shape on FP8 pages needs about 3 MB of scratch: it must fit the built-in
    area (the size check uses the worker count of the kernel that really runs), and agree with the
    workspace entry point on two calls in a row."""
    from paper_2604_22782_b200 import harness
    from paper_2604_22782_b200.binding import SKV_STATIC_SCRATCH_BYTES
    g = torch.Generator().manual_seed(5)
    lens = torch.randint(1, 700, (32,), generator=g, dtype=torch.int32)
    w = W.Workload("noalloc8", 2, 32, 8, 128, 16, lens.numel(), 0, 0, "explicit", explicit_r=(0, 0), seed=43)
    dw = harness.setup(w, lens=lens, fp8=True)
    harness.prefill(dw, upto_offset=0)
    assert dw.cache.skv_decode_workspace_bytes(dw.batch, w.q_heads) <= SKV_STATIC_SCRATCH_BYTES
    shape = (dw.batch, w.q_heads, w.head_dim)
    for layer in (0, 1):
        Q = harness.step_inputs(dw, layer)["Q"]
        want = torch.full(shape, float("nan"), dtype=torch.bfloat16, device=dw.device)
        dw.cache.skv_decode_attn(layer, Q, dw.page_table, dw.seq_lens, want, dw.workspace)
        for _ in range(2):
            got = torch.full(shape, float("nan"), dtype=torch.bfloat16, device=dw.device)
            dw.cache.skv_decode_attn_static(layer, Q, dw.page_table, dw.seq_lens, got)
            torch.cuda.synchronize()
            assert dw.cache.skv_get_status() == 0
            assert _close(got, want)


def test_static_scratch_entry_refuses_what_does_not_fit():
    from paper_2604_22782_b200 import harness
    from paper_2604_22782_b200.binding import SKV_ERR_TOO_LARGE, SKV_STATIC_SCRATCH_BYTES, SkvError
    w = W.get_workload("tiny")
    dw = harness.setup(w)
    big = 16384                                           # largest batch the library takes
    assert dw.cache.skv_decode_workspace_bytes(big, w.q_heads) > SKV_STATIC_SCRATCH_BYTES
    Q = torch.zeros((big, w.q_heads, w.head_dim), dtype=torch.bfloat16, device=dw.device)
    pt = torch.zeros((big, 1), dtype=torch.int32, device=dw.device)
    sl = torch.zeros((big,), dtype=torch.int32, device=dw.device)
    out = torch.zeros_like(Q)
    launches = dw.cache.skv_launch_count()
    with pytest.raises(SkvError) as e:
        dw.cache.skv_decode_attn_static(0, Q, pt, sl, out)
    assert e.value.status == SKV_ERR_TOO_LARGE
    assert dw.cache.skv_launch_count() == launches       # refused on the host, nothing ran
