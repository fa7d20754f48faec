"""A bounded device wait that runs out: the library reports SKV_ERR_TIMEOUT through the status word and stays
usable.  The expiry is made by a test-only entry point (include/skv_test_hooks.h) that exists only in a
library built with -DSKV_TEST_HOOKS: a one-thread kernel waits, through the attention kernels' own
bounded-wait routine, for bytes that no copy delivers.  Nothing faults, nothing spins without a limit and
no copy is in flight when the kernel leaves."""
import ctypes

import pytest
import torch

import workloads as W


def _hooks_lib():
    from paper_2604_22782_b200 import build
    return ctypes.CDLL(build.build_test_hooks())


def test_the_product_library_does_not_export_the_hook():
    from paper_2604_22782_b200 import binding
    assert not hasattr(binding.lib, "skv_test_wait_expires")
    hooks = _hooks_lib()
    assert hasattr(hooks, "skv_test_wait_expires")
    for name in binding.exported_symbols():              # and it is the whole library otherwise
        assert hasattr(hooks, name), name


@pytest.mark.gpu
def test_expired_wait_is_reported_and_the_next_call_is_clean():
    from paper_2604_22782_b200 import harness
    from paper_2604_22782_b200.binding import SKV_ERR_TIMEOUT
    hooks = _hooks_lib()
    hooks.skv_test_wait_expires.argtypes = [ctypes.c_void_p, ctypes.c_int, ctypes.c_void_p]
    w = W.get_workload("tiny")
    dw = harness.setup(w)
    harness.prefill(dw, upto_offset=0)
    assert dw.cache.skv_get_status() == 0
    stream = torch.cuda.current_stream().cuda_stream
    rc = hooks.skv_test_wait_expires(dw.cache.pool.data_ptr(), 3, stream)     # the status word heads the pool
    assert rc == 0
    assert dw.cache.skv_get_status() == SKV_ERR_TIMEOUT                       # synchronises the stream
    assert dw.cache.skv_get_status() == 0                                     # reading cleared it
    # an ordinary call afterwards: same result as before the expiry, clean status
    Q = harness.step_inputs(dw, 1)["Q"]
    out = torch.full((dw.batch, w.q_heads, w.head_dim), float("nan"), dtype=torch.bfloat16, device=dw.device)
    dw.cache.skv_decode_attn(1, Q, dw.page_table, dw.seq_lens, out, dw.workspace)
    assert dw.cache.skv_get_status() == 0
    from oracle import Oracle
    o = Oracle(w.n_layers, dw.r, w.q_heads, w.kv_heads, w.head_dim, dw.batch, int(dw.lens_cpu.max()))
    si, pos = W.token_index(dw.lens_cpu)
    K, V = W.draw_kv(w, 0, si, pos)
    o.append(0, K, V, si, pos)
    ref = o.decode_attn(1, Q.cpu(), dw.lens_cpu)
    assert bool(((out.cpu().double() - ref).abs() <= 1e-2 + 1e-2 * ref.abs()).all())
    assert hooks.skv_test_wait_expires(None, 3, stream) != 0                  # argument checks
    assert hooks.skv_test_wait_expires(dw.cache.pool.data_ptr(), 5000, stream) != 0
