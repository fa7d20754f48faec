"""The per-layer loop when every kernel between two attention calls takes part in programmatic launches:
the caller's query kernel (a stand-in from the test-hook library, include/skv_test_hooks.h) releases its
dependents first and waits second, and so do the library's decode-step update kernels, so that with early
fetch the attention kernel of layer l+1 is on the SMs while that of layer l still runs.  Every output is
compared with the oracle; an output buffer starts as NaN and the query of layer l+1 is computed FROM the
output of layer l, so a kernel that read its input before the kernel ahead of it was done would poison
everything after it."""
import ctypes

import pytest
import torch

import workloads as W
from test_gpu_parity import _oracle_for, _within_tol


def _hooks_lib():
    from paper_2604_22782_b200 import build
    lib = ctypes.CDLL(build.build_test_hooks())
    lib.skv_test_query_kernel.restype = ctypes.c_int
    lib.skv_test_query_kernel.argtypes = [ctypes.c_void_p, ctypes.c_void_p, ctypes.c_void_p, ctypes.c_longlong,
                                          ctypes.c_void_p]
    return lib


def test_the_product_library_does_not_export_the_query_kernel():
    from paper_2604_22782_b200 import binding
    assert not hasattr(binding.lib, "skv_test_query_kernel")
    assert hasattr(_hooks_lib(), "skv_test_query_kernel")


def test_query_kernel_rejects_bad_arguments():
    hooks = _hooks_lib()
    assert hooks.skv_test_query_kernel(None, None, None, 8, None) != 0
    assert hooks.skv_test_query_kernel(16, 32, 48, 12, None) != 0          # not a multiple of 8 elements
    assert hooks.skv_test_query_kernel(16, 32, 50, 8, None) != 0           # not 16-byte aligned
    assert hooks.skv_test_query_kernel(16, 32, 48, 0, None) == 0           # nothing to do, nothing launched


@pytest.mark.gpu
@pytest.mark.parametrize("Hq,Hkv,D,worker", [
    (8, 2, 128, None),       # tensor-core states, CTA per range with a combining warp
    (4, 4, 128, None),       # one query head per kv head: CUDA-core states, no combining warp, merge launch
    (8, 2, 64, None),        # head_dim 64
    (8, 1, 128, None),       # eight query heads share a kv head
    (8, 2, 128, 1),          # the warp-per-range kernel
])
@pytest.mark.parametrize("fp8", [False, True])
@pytest.mark.parametrize("merge", [1, 2])
def test_chained_programmatic_launches_match_the_oracle(merge, fp8, Hq, Hkv, D, worker):
    from paper_2604_22782_b200 import harness
    hooks = _hooks_lib()
    lens = torch.tensor([16, 17, 1, 33, 4000, 250, 64, 1200, 2047, 5, 900, 3100], dtype=torch.int32)
    r = (0, 0, 2, 2, 2, 5)
    w = W.Workload("chain", len(r), Hq, Hkv, D, 16, lens.numel(), 0, 0, "explicit", explicit_r=r, seed=67)
    dw = harness.setup(w, lens=lens, fp8=fp8)
    dw.retune(early_fetch=1, merge=merge, worker=worker)
    harness.prefill(dw, upto_offset=-1)
    owners = [l for l in range(w.n_layers) if r[l] == l]
    if fp8:
        o = None
    else:
        o = _oracle_for(dw, list(range(dw.batch)), owners, upto_offset=-1)
    b = torch.arange(dw.batch, dtype=torch.int64)
    last = dw.lens_cpu.to(torch.int64) - 1
    shape = (dw.batch, w.q_heads, w.head_dim)
    stream = torch.cuda.current_stream().cuda_stream
    G = w.q_heads // w.kv_heads
    prev = torch.zeros(shape, dtype=torch.bfloat16, device=dw.device)
    runs = []
    for rep in range(3):
        for l in range(w.n_layers):
            Q = W.draw_rows(w.seed + 10 * rep, W.KIND_Q, l, b, last, w.q_heads, w.head_dim, 1.0, dw.device)
            Qd = torch.full(shape, float("nan"), dtype=torch.bfloat16, device=dw.device)
            out = torch.full(shape, float("nan"), dtype=torch.bfloat16, device=dw.device)
            K = V = None
            if l in owners:
                # the new token's K points along the query, so the token the update has just written carries weight
                K = (Q[:, ::G, :].float() * 2.0).to(torch.bfloat16).contiguous()
                V = W.draw_rows(w.seed + 10 * rep, W.KIND_V, l, b, last, w.kv_heads, w.head_dim, 1.0, dw.device)
            runs.append((rep, l, Q, Qd, out, K, V, prev))
            prev = out
    torch.cuda.synchronize()
    # the whole chain goes out without anything between its launches
    for rep, l, Q, Qd, out, K, V, before in runs:
        assert hooks.skv_test_query_kernel(Q.data_ptr(), before.data_ptr(), Qd.data_ptr(), Q.numel(), stream) == 0
        if K is not None:
            dw.cache.skv_append(l, K, V, dw.slot_new)
        dw.cache.skv_decode_attn(l, Qd, dw.page_table, dw.seq_lens, out, dw.workspace)
    torch.cuda.synchronize()
    assert dw.cache.skv_get_status() == 0
    for rep, l, Q, Qd, out, K, V, before in runs:
        assert torch.equal(Qd.view(torch.int16), Q.view(torch.int16)), f"rep {rep} layer {l}: query kernel"
        assert not torch.isnan(out.float()).any(), f"rep {rep} layer {l}"
    if fp8:
        # FP8 pages: the same chain with a synchronisation after every launch is the reference
        # (the oracle comparison of FP8 decode is test_gpu_fp8's)
        dw2 = harness.setup(w, lens=lens, fp8=True)
        dw2.retune(early_fetch=0, merge=1)
        harness.prefill(dw2, upto_offset=-1)
        for rep, l, Q, Qd, out, K, V, before in runs:
            if K is not None:
                dw2.cache.skv_append(l, K, V, dw2.slot_new)
                torch.cuda.synchronize()
            ref = torch.empty_like(out)
            dw2.cache.skv_decode_attn(l, Q, dw2.page_table, dw2.seq_lens, ref, dw2.workspace)
            torch.cuda.synchronize()
            ok, err = _within_tol(out, ref.cpu().double())
            assert ok, f"rep {rep} layer {l}: max abs err {err}"
        return
    for rep, l, Q, Qd, out, K, V, before in runs:
        if K is not None:
            o.append(l, K.cpu(), V.cpu(), b, last)
        ref = o.decode_attn(l, Q.cpu(), dw.lens_cpu)
        ok, err = _within_tol(out, ref)
        assert ok, f"rep {rep} layer {l}: max abs err {err}"
