"""ctypes binding of ``libskv.so``: same names as the C entry points, argument
marshalling only.  Tensors are torch CUDA tensors (torch is used for device
memory and streams, nothing else)."""
from __future__ import annotations

import ctypes
import os
import re
from typing import List, Optional, Sequence

import torch

from . import build as _build

_HERE = os.path.dirname(os.path.abspath(__file__))
_HEADER = os.path.join(_HERE, "..", "include", "skv.h")

SKV_OK = 0
SKV_ERR_ARG, SKV_ERR_ROUTING, SKV_ERR_UNSUPPORTED, SKV_ERR_NOMEM = -1, -2, -3, -4
SKV_ERR_LAYER, SKV_ERR_CUDA, SKV_ERR_TIMEOUT, SKV_ERR_BOUNDS = -5, -6, -7, -8
SKV_ERR_TOO_LARGE = -9
SKV_STATIC_SCRATCH_BYTES = 8 << 20


def lib_path() -> str:
    return _build.LIB


def _load() -> ctypes.CDLL:
    path = _build.LIB
    if not os.path.exists(path):
        try:
            _build.build()
        except Exception as e:  # no silent fallback: the CUDA library is the product
            raise ImportError(f"libskv.so is missing and could not be built with nvcc: {e}") from e
    return ctypes.CDLL(path)


lib = _load()

_vp, _i32p, _i64p, _szp = ctypes.c_void_p, ctypes.c_void_p, ctypes.c_void_p, ctypes.POINTER(ctypes.c_size_t)
_int, _i64, _f32, _sz = ctypes.c_int, ctypes.c_int64, ctypes.c_float, ctypes.c_size_t

lib.skv_strerror.restype = ctypes.c_char_p
lib.skv_strerror.argtypes = [_int]
lib.skv_routing_from_owners.argtypes = [_int, _i32p, _int, _i32p]
lib.skv_routing_groups.argtypes = [_int, _int, _i32p]
lib.skv_routing_rcla.argtypes = [_int, ctypes.c_double, _vp, _vp, _i32p]
lib.skv_routing_rdcla.argtypes = [_int, _int, ctypes.c_double, _vp, _i32p]
lib.skv_cache_pool_bytes.argtypes = [_int, _i32p, _int, _int, _int, _i64, _szp]
lib.skv_cache_create.argtypes = [ctypes.POINTER(_vp), _int, _i32p, _int, _int, _int, _i64, _vp, _sz, _vp]
lib.skv_cache_create_fp8.argtypes = lib.skv_cache_create.argtypes
lib.skv_cache_pool_bytes_fp8.argtypes = [_int, _i32p, _int, _int, _int, _i64, _szp]
lib.skv_gather_fp8.argtypes = [_vp, _int, _i64p, _i64, _vp, _vp, _vp, _vp, _vp]
lib.skv_cache_destroy.restype = None
lib.skv_cache_destroy.argtypes = [_vp]
lib.skv_layer_owner.argtypes = [_vp, _int]
lib.skv_is_owner.argtypes = [_vp, _int]
lib.skv_cache_stats.argtypes = [_vp, ctypes.POINTER(_int), _szp, _szp, _szp]
lib.skv_append.argtypes = [_vp, _int, _vp, _vp, _i64p, _i64, _vp]
lib.skv_gather.argtypes = [_vp, _int, _i64p, _i64, _vp, _vp, _vp]
lib.skv_decode_workspace_bytes.argtypes = [_vp, _int, _int, _szp]
lib.skv_decode_attn.argtypes = [_vp, _int, _vp, _i32p, _i32p, _vp, _int, _int, _int, _f32, _vp, _sz, _vp]
lib.skv_decode_attn_static.argtypes = [_vp, _int, _vp, _i32p, _i32p, _vp, _int, _int, _int, _f32, _vp]
lib.skv_prefill_attn.argtypes = [_vp, _int, _vp, _i32p, _i32p, _i32p, _vp, _int, _int, _int, _int, _f32, _vp]
lib.skv_prefill_attn_src.argtypes = [_vp, _int, _vp, _i32p, _i32p, _i32p, _vp, _int, _int, _int, _int, _f32, _vp]
lib.skv_decode_splitk.argtypes = [_vp, _int, _vp, _i32p, _i32p, _int, _int, _int, _f32, _vp, _sz, _vp]
lib.skv_decode_merge.argtypes = [_vp, _vp, _int, _int, _vp, _sz, _vp]
lib.skv_decode_step.argtypes = [_vp, _vp, _vp, _vp, _i64p, _i32p, _i32p, _vp, _int, _int, _int, _f32, _vp, _sz, _vp]
lib.skv_decode_step_staging_bytes.argtypes = [_vp, _int, _int, _int, _szp]
lib.skv_decode_step_host.argtypes = [_vp, _vp, _vp, _vp, _i64p, _i32p, _i32p, _vp, _int, _int, _int, _f32,
                                     _vp, _sz, _vp]
lib.skv_get_status.argtypes = [_vp, _vp, ctypes.POINTER(_int)]
lib.skv_set_decode_variant.argtypes = [_vp, _int]
lib.skv_set_decode_tuning.argtypes = [_vp, _int, _int, _int]
lib.skv_set_prefill_variant.argtypes = [_vp, _int]
lib.skv_prefill_scratch_bytes.argtypes = [_vp, _szp]
lib.skv_set_prefill_scratch.argtypes = [_vp, _vp, _sz]
lib.skv_set_decode_overlap.argtypes = [_vp, _int]
lib.skv_set_decode_l2_reuse.argtypes = [_vp, _int]
lib.skv_set_decode_early_fetch.argtypes = [_vp, _int]
lib.skv_set_decode_worker.argtypes = [_vp, _int, _int, _int, _int]
lib.skv_set_decode_merge.argtypes = [_vp, _int]
lib.skv_set_host_step.argtypes = [_vp, _int, _int]
lib.skv_set_trace_buffer.argtypes = [_vp, _vp, _sz]
lib.skv_decode_worker_count.argtypes = [_vp]
lib.skv_launch_count.argtypes = [_vp, ctypes.POINTER(_i64)]
lib.skv_plan_worker_range.argtypes = [_i64, _int, _int, ctypes.POINTER(_i64), ctypes.POINTER(_i64)]
lib.skv_plan_worker_of.argtypes = [_i64, _int, _i64]


def exported_symbols() -> List[str]:
    """Names of the functions ``include/skv.h`` declares."""
    with open(_HEADER) as f:
        text = f.read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(skv_[a-z_0-9]+)\s*\(", text)))


class SkvError(RuntimeError):
    def __init__(self, status: int, what: str):
        self.status = status
        super().__init__(f"{what}: {skv_strerror(status)} ({status})")


def skv_strerror(status: int) -> str:
    return lib.skv_strerror(status).decode()


def _check(rc: int, what: str) -> None:
    if rc != SKV_OK:
        raise SkvError(rc, what)


def _i32_array(xs: Sequence[int]):
    return (ctypes.c_int32 * len(xs))(*[int(x) for x in xs])


def skv_routing_from_owners(n_layers: int, owners: Sequence[int]) -> List[int]:
    out = (ctypes.c_int32 * max(n_layers, 1))()
    _check(lib.skv_routing_from_owners(n_layers, _i32_array(list(owners)), len(owners), out), "skv_routing_from_owners")
    return list(out)[:n_layers]


def skv_routing_groups(n_layers: int, g: int) -> List[int]:
    out = (ctypes.c_int32 * max(n_layers, 1))()
    _check(lib.skv_routing_groups(n_layers, g, out), "skv_routing_groups")
    return list(out)[:n_layers]


def _f64_array(xs: Sequence[float]):
    return (ctypes.c_double * len(xs))(*xs)


def skv_routing_rcla(p_self: float, u: Sequence[float], v: Sequence[float]) -> List[int]:
    n = len(u)
    out = (ctypes.c_int32 * n)()
    _check(lib.skv_routing_rcla(n, p_self, _f64_array(list(u)), _f64_array(list(v)), out), "skv_routing_rcla")
    return list(out)


def skv_routing_rdcla(k: int, p_self: float, u: Sequence[float]) -> List[int]:
    n = len(u)
    out = (ctypes.c_int32 * n)()
    _check(lib.skv_routing_rdcla(n, k, p_self, _f64_array(list(u)), out), "skv_routing_rdcla")
    return list(out)


def skv_cache_pool_bytes(r: Sequence[int], kv_heads: int, head_dim: int, page_size: int, max_pages: int) -> int:
    out = ctypes.c_size_t(0)
    _check(lib.skv_cache_pool_bytes(len(r), _i32_array(r), kv_heads, head_dim, page_size, max_pages,
                                    ctypes.byref(out)), "skv_cache_pool_bytes")
    return out.value


def skv_cache_pool_bytes_fp8(r: Sequence[int], kv_heads: int, head_dim: int, page_size: int, max_pages: int) -> int:
    out = _sz(0)
    _check(lib.skv_cache_pool_bytes_fp8(len(r), _i32_array(r), kv_heads, head_dim, page_size, max_pages,
                                        ctypes.byref(out)), "skv_cache_pool_bytes_fp8")
    return out.value


def skv_plan_worker_range(n_blocks: int, n_workers: int, w: int):
    b, e = _i64(0), _i64(0)
    _check(lib.skv_plan_worker_range(n_blocks, n_workers, w, ctypes.byref(b), ctypes.byref(e)),
           "skv_plan_worker_range")
    return b.value, e.value


def skv_plan_worker_of(n_blocks: int, n_workers: int, x: int) -> int:
    rc = lib.skv_plan_worker_of(n_blocks, n_workers, x)
    if rc < 0:
        raise SkvError(rc, "skv_plan_worker_of")
    return rc


def _stream_ptr(stream) -> int:
    if stream is None:
        return torch.cuda.current_stream().cuda_stream if torch.cuda.is_available() else 0
    if isinstance(stream, int):
        return stream
    return stream.cuda_stream


def _ptr(t: Optional[torch.Tensor]) -> Optional[int]:
    return None if t is None else t.data_ptr()


def _arg(name: str, t: Optional[torch.Tensor], dtype, shape=None, min_numel: Optional[int] = None,
         cuda: Optional[bool] = True) -> Optional[torch.Tensor]:
    """Checks a tensor argument before its raw pointer goes to the library: dtype, device (cuda=None: either),
    contiguity, and an exact shape or a minimum number of elements.  The kernels trust the sizes they are
    given, so a wrong one here would be an out-of-bounds access there."""
    if t is None:
        return None
    if t.dtype != dtype:
        raise TypeError(f"{name}: expected {dtype}, got {t.dtype}")
    if cuda is not None and t.is_cuda != cuda:
        raise ValueError(f"{name}: expected a {'CUDA' if cuda else 'host'} tensor")
    if not t.is_contiguous():
        raise ValueError(f"{name}: must be contiguous")
    if shape is not None and tuple(t.shape) != tuple(shape):
        raise ValueError(f"{name}: expected shape {tuple(shape)}, got {tuple(t.shape)}")
    if min_numel is not None and t.numel() < min_numel:
        raise ValueError(f"{name}: needs at least {min_numel} elements, has {t.numel()}")
    return t


def _nbytes(t: torch.Tensor) -> int:
    return t.numel() * t.element_size()


class SkvCache:
    """Handle of one routed cache.  ``device_pool`` is a torch uint8 CUDA tensor
    of at least ``skv_cache_pool_bytes`` bytes that the caller keeps alive; pass
    ``allocate=True`` to let this wrapper allocate it with torch, or
    ``accounting_only=True`` for a handle without device memory."""

    def __init__(self, r: Sequence[int], kv_heads: int, head_dim: int, page_size: int, max_pages: int,
                 device_pool: Optional[torch.Tensor] = None, allocate: bool = False,
                 accounting_only: bool = False, stream=None, fp8: bool = False):
        self.fp8 = fp8
        create = lib.skv_cache_create_fp8 if fp8 else lib.skv_cache_create
        self.r = [int(x) for x in r]
        self.n_layers = len(self.r)
        self.kv_heads, self.head_dim, self.page_size, self.max_pages = kv_heads, head_dim, page_size, max_pages
        self._h = _vp()
        self.pool = None
        if accounting_only:
            rc = create(ctypes.byref(self._h), self.n_layers, _i32_array(self.r), kv_heads, head_dim,
                        page_size, max_pages, None, 0, None)
            _check(rc, "skv_cache_create")
            return
        need = (skv_cache_pool_bytes_fp8 if fp8 else skv_cache_pool_bytes)(self.r, kv_heads, head_dim, page_size, max_pages)
        if device_pool is None:
            if not allocate:
                raise ValueError("pass device_pool, allocate=True or accounting_only=True")
            device_pool = torch.empty(need, dtype=torch.uint8, device="cuda")
        assert device_pool.is_cuda and device_pool.dtype == torch.uint8 and device_pool.is_contiguous()
        self.pool = device_pool
        rc = create(ctypes.byref(self._h), self.n_layers, _i32_array(self.r), kv_heads, head_dim,
                    page_size, max_pages, device_pool.data_ptr(), device_pool.numel(), _stream_ptr(stream))
        _check(rc, "skv_cache_create")

    # -- lifetime
    def close(self):
        if getattr(self, "_h", None):
            lib.skv_cache_destroy(self._h)
            self._h = None

    __del__ = close

    # -- introspection
    def skv_layer_owner(self, layer: int) -> int:
        rc = lib.skv_layer_owner(self._h, layer)
        if rc < 0:
            raise SkvError(rc, "skv_layer_owner")
        return rc

    def skv_is_owner(self, layer: int) -> bool:
        rc = lib.skv_is_owner(self._h, layer)
        if rc < 0:
            raise SkvError(rc, "skv_is_owner")
        return bool(rc)

    def skv_cache_stats(self) -> dict:
        n = _int(0)
        pb, kb, bt = _sz(0), _sz(0), _sz(0)
        _check(lib.skv_cache_stats(self._h, ctypes.byref(n), ctypes.byref(pb), ctypes.byref(kb), ctypes.byref(bt)),
               "skv_cache_stats")
        return {"n_owners": n.value, "page_bytes": pb.value, "kv_bytes": kb.value, "bytes_per_token": bt.value}

    # -- Update
    def skv_append(self, layer: int, K: Optional[torch.Tensor], V: Optional[torch.Tensor],
                   slot_map: Optional[torch.Tensor], n_tokens: Optional[int] = None, stream=None) -> None:
        if n_tokens is None:
            n_tokens = 0 if slot_map is None else slot_map.numel()
        row = (n_tokens, self.kv_heads, self.head_dim)
        _arg("K", K, torch.bfloat16, row)
        _arg("V", V, torch.bfloat16, row)
        _arg("slot_map", slot_map, torch.int64, min_numel=n_tokens)
        rc = lib.skv_append(self._h, layer, _ptr(K), _ptr(V), _ptr(slot_map), n_tokens, _stream_ptr(stream))
        _check(rc, "skv_append")

    def skv_gather(self, layer: int, slot_ids: torch.Tensor, K_out: torch.Tensor, V_out: torch.Tensor,
                   stream=None) -> None:
        n = slot_ids.numel()
        _arg("slot_ids", slot_ids, torch.int64)
        _arg("K_out", K_out, torch.bfloat16, (n, self.kv_heads, self.head_dim))
        _arg("V_out", V_out, torch.bfloat16, (n, self.kv_heads, self.head_dim))
        rc = lib.skv_gather(self._h, layer, _ptr(slot_ids), slot_ids.numel(), _ptr(K_out), _ptr(V_out),
                            _stream_ptr(stream))
        _check(rc, "skv_gather")

    def skv_gather_fp8(self, layer: int, slot_ids: torch.Tensor, K_codes: torch.Tensor, V_codes: torch.Tensor,
                       K_scales: torch.Tensor, V_scales: torch.Tensor, stream=None) -> None:
        rc = lib.skv_gather_fp8(self._h, layer, _ptr(slot_ids), slot_ids.numel(), _ptr(K_codes), _ptr(V_codes),
                                _ptr(K_scales), _ptr(V_scales), _stream_ptr(stream))
        _check(rc, "skv_gather_fp8")

    # -- Load + Attn
    def _decode_args(self, Q, page_table, seq_lens, out):
        """Shapes of one decode-attention call: Q, out [batch][q_heads][head_dim] bf16; page_table
        [batch][width] int32; seq_lens [batch] int32, all on the device."""
        if Q.dim() != 3 or Q.shape[2] != self.head_dim:
            raise ValueError(f"Q: expected [batch][q_heads][{self.head_dim}], got {tuple(Q.shape)}")
        batch, q_heads = Q.shape[0], Q.shape[1]
        _arg("Q", Q, torch.bfloat16)
        if out is not None:
            _arg("out", out, torch.bfloat16, Q.shape)
        _arg("page_table", page_table, torch.int32)
        if page_table.dim() != 2 or page_table.shape[0] != batch:
            raise ValueError(f"page_table: expected [{batch}][width], got {tuple(page_table.shape)}")
        _arg("seq_lens", seq_lens, torch.int32, (batch,))
        return batch, q_heads

    def skv_decode_workspace_bytes(self, batch: int, q_heads: int) -> int:
        out = _sz(0)
        _check(lib.skv_decode_workspace_bytes(self._h, batch, q_heads, ctypes.byref(out)),
               "skv_decode_workspace_bytes")
        return out.value

    def skv_decode_attn(self, layer: int, Q: torch.Tensor, page_table: torch.Tensor, seq_lens: torch.Tensor,
                        out: torch.Tensor, workspace: torch.Tensor, scale: float = 0.0, stream=None) -> None:
        batch, q_heads = self._decode_args(Q, page_table, seq_lens, out)
        _arg("workspace", workspace, torch.uint8)
        rc = lib.skv_decode_attn(self._h, layer, _ptr(Q), _ptr(page_table), _ptr(seq_lens), _ptr(out), batch,
                                 q_heads, page_table.shape[1], scale, _ptr(workspace), _nbytes(workspace),
                                 _stream_ptr(stream))
        _check(rc, "skv_decode_attn")

    def skv_decode_attn_static(self, layer: int, Q: torch.Tensor, page_table: torch.Tensor, seq_lens: torch.Tensor,
                               out: torch.Tensor, scale: float = 0.0, stream=None) -> None:
        """skv_decode_attn without a workspace argument, for callers that cannot allocate device memory:
        the scratch is a fixed SKV_STATIC_SCRATCH_BYTES area inside the library (shared by all calls on
        the device; calls that overlap on the GPU race on it)."""
        batch, q_heads = self._decode_args(Q, page_table, seq_lens, out)
        rc = lib.skv_decode_attn_static(self._h, layer, _ptr(Q), _ptr(page_table), _ptr(seq_lens), _ptr(out),
                                        batch, q_heads, page_table.shape[1], scale, _stream_ptr(stream))
        _check(rc, "skv_decode_attn_static")

    def _prefill_args(self, Q, cu_q_lens, page_table, seq_lens, out):
        if Q.dim() != 3 or Q.shape[2] != self.head_dim:
            raise ValueError(f"Q: expected [n_q][q_heads][{self.head_dim}], got {tuple(Q.shape)}")
        batch = seq_lens.shape[0]
        _arg("Q", Q, torch.bfloat16)
        _arg("out", out, torch.bfloat16, Q.shape)
        _arg("cu_q_lens", cu_q_lens, torch.int32, (batch + 1,))
        _arg("page_table", page_table, torch.int32)
        if page_table.dim() != 2 or page_table.shape[0] != batch:
            raise ValueError(f"page_table: expected [{batch}][width], got {tuple(page_table.shape)}")
        _arg("seq_lens", seq_lens, torch.int32, (batch,))
        return batch, Q.shape[1]

    def skv_prefill_attn(self, layer: int, Q: torch.Tensor, cu_q_lens: torch.Tensor, page_table: torch.Tensor,
                         seq_lens: torch.Tensor, out: torch.Tensor, max_q_len: int, scale: float = 0.0,
                         stream=None) -> None:
        batch, q_heads = self._prefill_args(Q, cu_q_lens, page_table, seq_lens, out)
        rc = lib.skv_prefill_attn(self._h, layer, _ptr(Q), _ptr(cu_q_lens), _ptr(page_table), _ptr(seq_lens),
                                  _ptr(out), batch, max_q_len, q_heads, page_table.shape[1], scale,
                                  _stream_ptr(stream))
        _check(rc, "skv_prefill_attn")

    def skv_prefill_attn_src(self, src_layer: int, Q: torch.Tensor, cu_q_lens: torch.Tensor, page_table: torch.Tensor,
                             seq_lens: torch.Tensor, out: torch.Tensor, max_q_len: int, scale: float = 0.0,
                             stream=None) -> None:
        batch, q_heads = self._prefill_args(Q, cu_q_lens, page_table, seq_lens, out)
        rc = lib.skv_prefill_attn_src(self._h, src_layer, _ptr(Q), _ptr(cu_q_lens), _ptr(page_table), _ptr(seq_lens),
                                      _ptr(out), batch, max_q_len, q_heads, page_table.shape[1], scale,
                                      _stream_ptr(stream))
        _check(rc, "skv_prefill_attn_src")

    def skv_decode_splitk(self, layer: int, Q: torch.Tensor, page_table: torch.Tensor, seq_lens: torch.Tensor,
                          workspace: torch.Tensor, scale: float = 0.0, stream=None) -> None:
        batch, q_heads = self._decode_args(Q, page_table, seq_lens, None)
        _arg("workspace", workspace, torch.uint8)
        rc = lib.skv_decode_splitk(self._h, layer, _ptr(Q), _ptr(page_table), _ptr(seq_lens), batch, q_heads,
                                   page_table.shape[1], scale, _ptr(workspace), _nbytes(workspace),
                                   _stream_ptr(stream))
        _check(rc, "skv_decode_splitk")

    def skv_decode_merge(self, out: torch.Tensor, workspace: torch.Tensor, stream=None) -> None:
        batch, q_heads = out.shape[0], out.shape[1]
        _arg("out", out, torch.bfloat16, (batch, q_heads, self.head_dim))
        _arg("workspace", workspace, torch.uint8)
        rc = lib.skv_decode_merge(self._h, _ptr(out), batch, q_heads, _ptr(workspace),
                                  _nbytes(workspace), _stream_ptr(stream))
        _check(rc, "skv_decode_merge")

    def skv_decode_step(self, Q: torch.Tensor, K: torch.Tensor, V: torch.Tensor, slot_map: torch.Tensor,
                        page_table: torch.Tensor, seq_lens: torch.Tensor, out: torch.Tensor,
                        workspace: torch.Tensor, scale: float = 0.0, stream=None) -> None:
        batch, q_heads = Q.shape[1], Q.shape[2]
        self._step_args(Q, K, V, slot_map, page_table, seq_lens, out, cuda=True)
        _arg("workspace", workspace, torch.uint8)
        rc = lib.skv_decode_step(self._h, _ptr(Q), _ptr(K), _ptr(V), _ptr(slot_map), _ptr(page_table),
                                 _ptr(seq_lens), _ptr(out), batch, q_heads, page_table.shape[1], scale,
                                 _ptr(workspace), _nbytes(workspace), _stream_ptr(stream))
        _check(rc, "skv_decode_step")

    def _step_args(self, Q, K, V, slot_map, page_table, seq_lens, out, cuda):
        """Shapes of one whole step: Q, out [n_layers][batch][q_heads][head_dim]; K, V
        [n_owners][batch][kv_heads][head_dim]; slot_map [batch] int64; page_table [batch][width]; seq_lens [batch]."""
        if Q.dim() != 4 or Q.shape[0] != self.n_layers or Q.shape[3] != self.head_dim:
            raise ValueError(f"Q: expected [{self.n_layers}][batch][q_heads][{self.head_dim}], got {tuple(Q.shape)}")
        batch = Q.shape[1]
        n_owners = sum(1 for l, s in enumerate(self.r) if s == l)
        _arg("Q", Q, torch.bfloat16, cuda=cuda)
        _arg("out", out, torch.bfloat16, Q.shape, cuda=cuda)
        _arg("K", K, torch.bfloat16, (n_owners, batch, self.kv_heads, self.head_dim), cuda=cuda)
        _arg("V", V, torch.bfloat16, (n_owners, batch, self.kv_heads, self.head_dim), cuda=cuda)
        _arg("slot_map", slot_map, torch.int64, (batch,), cuda=cuda)
        _arg("page_table", page_table, torch.int32, cuda=cuda)
        if page_table.dim() != 2 or page_table.shape[0] != batch:
            raise ValueError(f"page_table: expected [{batch}][width], got {tuple(page_table.shape)}")
        _arg("seq_lens", seq_lens, torch.int32, (batch,), cuda=cuda)

    def skv_decode_step_staging_bytes(self, batch: int, q_heads: int, pt_stride: int) -> int:
        out = _sz(0)
        _check(lib.skv_decode_step_staging_bytes(self._h, batch, q_heads, pt_stride, ctypes.byref(out)),
               "skv_decode_step_staging_bytes")
        return out.value

    def skv_decode_step_host(self, hQ: torch.Tensor, hK: torch.Tensor, hV: torch.Tensor, h_slot_map: torch.Tensor,
                             h_page_table: torch.Tensor, h_seq_lens: torch.Tensor, h_out: torch.Tensor,
                             staging: torch.Tensor, scale: float = 0.0, stream=None) -> None:
        batch, q_heads = hQ.shape[1], hQ.shape[2]
        self._step_args(hQ, hK, hV, h_slot_map, h_page_table, h_seq_lens, h_out, cuda=False)
        _arg("staging", staging, torch.uint8)
        rc = lib.skv_decode_step_host(self._h, _ptr(hQ), _ptr(hK), _ptr(hV), _ptr(h_slot_map), _ptr(h_page_table),
                                      _ptr(h_seq_lens), _ptr(h_out), batch, q_heads, h_page_table.shape[1], scale,
                                      _ptr(staging), _nbytes(staging), _stream_ptr(stream))
        _check(rc, "skv_decode_step_host")

    # -- status, tuning, counters
    def skv_get_status(self, stream=None) -> int:
        st = _int(0)
        _check(lib.skv_get_status(self._h, _stream_ptr(stream), ctypes.byref(st)), "skv_get_status")
        return st.value

    def skv_set_decode_variant(self, variant: int) -> None:
        _check(lib.skv_set_decode_variant(self._h, variant), "skv_set_decode_variant")

    def skv_set_decode_tuning(self, warps_per_cta: int = 0, stages: int = 0, ctas_per_sm: int = 0) -> None:
        _check(lib.skv_set_decode_tuning(self._h, warps_per_cta, stages, ctas_per_sm), "skv_set_decode_tuning")

    def skv_prefill_scratch_bytes(self) -> int:
        out = _sz(0)
        _check(lib.skv_prefill_scratch_bytes(self._h, ctypes.byref(out)), "skv_prefill_scratch_bytes")
        return out.value

    def skv_set_prefill_scratch(self, scratch: Optional[torch.Tensor]) -> None:
        """Give (or, with None, take back) the area in which pre-fill calls on an FP8 cache keep a bf16 copy of
        the pages they reach; the tensor must stay alive while it is set."""
        _arg("scratch", scratch, torch.uint8)
        self._prefill_scratch = scratch
        _check(lib.skv_set_prefill_scratch(self._h, _ptr(scratch), 0 if scratch is None else _nbytes(scratch)),
               "skv_set_prefill_scratch")

    def skv_set_prefill_variant(self, variant: int) -> None:
        _check(lib.skv_set_prefill_variant(self._h, variant), "skv_set_prefill_variant")

    def skv_set_decode_overlap(self, enabled: int) -> None:
        _check(lib.skv_set_decode_overlap(self._h, enabled), "skv_set_decode_overlap")

    def skv_set_decode_worker(self, mode: int, consumers: int = 0, stages: int = 0, ctas_per_sm: int = 0) -> None:
        _check(lib.skv_set_decode_worker(self._h, mode, consumers, stages, ctas_per_sm), "skv_set_decode_worker")

    def skv_set_decode_early_fetch(self, enabled: int) -> None:
        _check(lib.skv_set_decode_early_fetch(self._h, enabled), "skv_set_decode_early_fetch")

    def skv_set_decode_merge(self, mode: int) -> None:
        _check(lib.skv_set_decode_merge(self._h, mode), "skv_set_decode_merge")

    def skv_set_decode_l2_reuse(self, keep_percent: int) -> None:
        _check(lib.skv_set_decode_l2_reuse(self._h, keep_percent), "skv_set_decode_l2_reuse")

    def skv_set_host_step(self, groups: int, ramp: int) -> None:
        _check(lib.skv_set_host_step(self._h, groups, ramp), "skv_set_host_step")

    def skv_set_trace_buffer(self, buf: Optional[torch.Tensor]) -> None:
        _check(lib.skv_set_trace_buffer(self._h, _ptr(buf), 0 if buf is None else buf.numel() * buf.element_size()),
               "skv_set_trace_buffer")

    def skv_decode_worker_count(self) -> int:
        rc = lib.skv_decode_worker_count(self._h)
        if rc < 0:
            raise SkvError(rc, "skv_decode_worker_count")
        return rc

    def skv_launch_count(self) -> int:
        out = _i64(0)
        _check(lib.skv_launch_count(self._h, ctypes.byref(out)), "skv_launch_count")
        return out.value
