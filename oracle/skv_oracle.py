"""ctypes wrapper of ``skv_oracle.c`` (TEST INFRASTRUCTURE, see that file's header).

Argument marshalling only; every number is computed by the plain C code.
Tensors are torch CPU tensors: bf16 for Q/K/V (passed as their bit patterns),
float64 for outputs.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from typing import Optional, Sequence

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "skv_oracle.c")
_LIB = os.path.join(_HERE, "libskv_oracle.so")
_lib = None


def build_oracle(force: bool = False) -> str:
    """Compile the oracle with gcc (plain C, -O2, OpenMP for timing only)."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        tmp = _LIB + f".tmp{os.getpid()}"
        subprocess.check_call(["gcc", "-O2", "-std=c11", "-fopenmp", "-fPIC", "-shared",
                               "-o", tmp, _SRC, "-lm"])
        os.replace(tmp, _LIB)
    return _LIB


def _load():
    global _lib
    if _lib is None:
        lib = ctypes.CDLL(build_oracle())
        vp, i32p, i64p, u16p, f64p = (ctypes.c_void_p,) * 5
        lib.oracle_create.restype = ctypes.c_void_p
        lib.oracle_create.argtypes = [ctypes.c_int, i32p, ctypes.c_int, ctypes.c_int, ctypes.c_int,
                                      ctypes.c_int, ctypes.c_int64]
        lib.oracle_destroy.restype = None
        lib.oracle_destroy.argtypes = [vp]
        lib.oracle_append.argtypes = [vp, ctypes.c_int, u16p, u16p, i64p, i64p, ctypes.c_int64]
        lib.oracle_read.argtypes = [vp, ctypes.c_int, ctypes.c_int64, ctypes.c_int64, u16p, u16p]
        lib.oracle_attn_weights.argtypes = [vp, ctypes.c_int, u16p, ctypes.c_int, ctypes.c_int,
                                            ctypes.c_int64, ctypes.c_double, f64p]
        lib.oracle_decode_attn.argtypes = [vp, ctypes.c_int, u16p, i32p, ctypes.c_double, f64p]
        lib.oracle_attn_rows.argtypes = [vp, ctypes.c_int, u16p, i64p, i64p, ctypes.c_int64, ctypes.c_double, f64p]
        lib.oracle_quantize_e4m3.restype = None
        lib.oracle_quantize_e4m3.argtypes = [u16p, ctypes.c_int64, ctypes.c_int, vp, vp]
        lib.oracle_e4m3_value.restype = ctypes.c_double
        lib.oracle_e4m3_value.argtypes = [ctypes.c_int]
        lib.oracle_append_fp8.argtypes = [vp, ctypes.c_int, u16p, u16p, i64p, i64p, ctypes.c_int64, vp, vp, vp, vp]
        lib.oracle_rcla_map.argtypes = [ctypes.c_int, ctypes.c_double, f64p, f64p, i32p]
        lib.oracle_rdcla_map.argtypes = [ctypes.c_int, ctypes.c_int, ctypes.c_double, f64p, i32p]
        lib.oracle_mu.argtypes = [ctypes.c_int, i32p, ctypes.c_int, i32p]
        lib.oracle_group_map.argtypes = [ctypes.c_int, ctypes.c_int, i32p]
        lib.oracle_count_owners.argtypes = [ctypes.c_int, i32p]
        lib.oracle_cache_bytes.restype = ctypes.c_int64
        lib.oracle_cache_bytes.argtypes = [ctypes.c_int, i32p, ctypes.c_int, ctypes.c_int, ctypes.c_int,
                                           ctypes.c_int64]
        _lib = lib
    return _lib


def _i32(xs) -> torch.Tensor:
    return torch.as_tensor(list(xs) if not torch.is_tensor(xs) else xs, dtype=torch.int32).contiguous()


def _bf16_bits(x: torch.Tensor) -> torch.Tensor:
    assert x.dtype == torch.bfloat16 and x.device.type == "cpu"
    return x.contiguous().view(torch.int16)


def mu_from_owners(n_layers: int, owners: Sequence[int]):
    """Eq. (3.2), 0-based.  Returns the map as a list, or None if undefined."""
    ow = _i32(owners)
    out = torch.empty(n_layers, dtype=torch.int32)
    rc = _load().oracle_mu(n_layers, ow.data_ptr(), ow.numel(), out.data_ptr())
    return out.tolist() if rc == 0 else None


def quantize_e4m3(x: torch.Tensor):
    """FP8 E4M3 codes (uint8, same shape) and one fp32 scale per row (last dim) of a bf16 tensor."""
    xb = _bf16_bits(x)
    D = xb.shape[-1]
    n = xb.numel() // D
    codes = torch.empty(xb.shape, dtype=torch.uint8)
    scales = torch.empty(xb.shape[:-1], dtype=torch.float32)
    _load().oracle_quantize_e4m3(xb.data_ptr(), n, D, codes.data_ptr(), scales.data_ptr())
    return codes, scales


def e4m3_value(code: int) -> float:
    return float(_load().oracle_e4m3_value(int(code)))


def rcla_map(p_self: float, u: Sequence[float], v: Sequence[float]):
    """Section 3.2: one forward pass of R-CLA training (u: coins, v: choices, both in [0,1))."""
    uu = torch.as_tensor(list(u), dtype=torch.float64).contiguous()
    vv = torch.as_tensor(list(v), dtype=torch.float64).contiguous()
    out = torch.empty(uu.numel(), dtype=torch.int32)
    rc = _load().oracle_rcla_map(uu.numel(), p_self, uu.data_ptr(), vv.data_ptr(), out.data_ptr())
    return out.tolist() if rc == 0 else None


def rdcla_map(k: int, p_self: float, u: Sequence[float]):
    """Section 4.2 ablation, RD-CLA@k."""
    uu = torch.as_tensor(list(u), dtype=torch.float64).contiguous()
    out = torch.empty(uu.numel(), dtype=torch.int32)
    rc = _load().oracle_rdcla_map(uu.numel(), k, p_self, uu.data_ptr(), out.data_ptr())
    return out.tolist() if rc == 0 else None


def group_map(n_layers: int, g: int):
    out = torch.empty(n_layers, dtype=torch.int32)
    rc = _load().oracle_group_map(n_layers, g, out.data_ptr())
    assert rc == 0
    return out.tolist()


def count_owners(r: Sequence[int]) -> int:
    rr = _i32(r)
    return _load().oracle_count_owners(rr.numel(), rr.data_ptr())


def cache_bytes(r: Sequence[int], kv_heads: int, head_dim: int, bytes_per_elt: int, n_tokens: int) -> int:
    rr = _i32(r)
    return int(_load().oracle_cache_bytes(rr.numel(), rr.data_ptr(), kv_heads, head_dim,
                                          bytes_per_elt, n_tokens))


class Oracle:
    """Dense per-layer K/V stores + routed fp64 attention (see skv_oracle.c)."""

    def __init__(self, n_layers: int, r: Sequence[int], q_heads: int, kv_heads: int, head_dim: int,
                 batch: int, n_max: int):
        self.lib = _load()
        self.L, self.Hq, self.Hkv, self.D, self.B, self.n_max = n_layers, q_heads, kv_heads, head_dim, batch, n_max
        rr = _i32(r)
        assert rr.numel() == n_layers
        self.h = self.lib.oracle_create(n_layers, rr.data_ptr(), q_heads, kv_heads, head_dim, batch, n_max)
        if not self.h:
            raise ValueError("oracle_create rejected its arguments")

    def close(self):
        if getattr(self, "h", None):
            self.lib.oracle_destroy(self.h)
            self.h = None

    __del__ = close

    def append(self, layer: int, K: torch.Tensor, V: torch.Tensor, seq_idx: torch.Tensor, pos: torch.Tensor):
        kb, vb = _bf16_bits(K), _bf16_bits(V)
        n = kb.shape[0]
        assert kb.shape == (n, self.Hkv, self.D) and vb.shape == kb.shape
        s = seq_idx.to(torch.int64).contiguous()
        p = pos.to(torch.int64).contiguous()
        assert s.numel() == n and p.numel() == n
        rc = self.lib.oracle_append(self.h, layer, kb.data_ptr(), vb.data_ptr(), s.data_ptr(), p.data_ptr(), n)
        if rc != 0:
            raise RuntimeError(f"oracle_append failed: {rc}")

    def append_fp8(self, layer: int, K: torch.Tensor, V: torch.Tensor, seq_idx: torch.Tensor, pos: torch.Tensor):
        """Update through the FP8 quantiser; returns (K codes, V codes, K scales, V scales) of the rows."""
        kb, vb = _bf16_bits(K), _bf16_bits(V)
        n = kb.shape[0]
        assert kb.shape == (n, self.Hkv, self.D) and vb.shape == kb.shape
        s = seq_idx.to(torch.int64).contiguous()
        p = pos.to(torch.int64).contiguous()
        kc = torch.empty((n, self.Hkv, self.D), dtype=torch.uint8)
        vc = torch.empty_like(kc)
        ks = torch.empty((n, self.Hkv), dtype=torch.float32)
        vs = torch.empty_like(ks)
        rc = self.lib.oracle_append_fp8(self.h, layer, kb.data_ptr(), vb.data_ptr(), s.data_ptr(), p.data_ptr(), n,
                                        kc.data_ptr(), vc.data_ptr(), ks.data_ptr(), vs.data_ptr())
        if rc != 0:
            raise RuntimeError(f"oracle_append_fp8 failed: {rc}")
        return kc, vc, ks, vs

    def read(self, layer: int, b: int, t: int):
        k = torch.empty((self.Hkv, self.D), dtype=torch.int16)
        v = torch.empty_like(k)
        rc = self.lib.oracle_read(self.h, layer, b, t, k.data_ptr(), v.data_ptr())
        if rc != 0:
            raise RuntimeError(f"oracle_read failed: {rc}")
        return k.view(torch.bfloat16), v.view(torch.bfloat16)

    def attn_weights(self, layer: int, Q: torch.Tensor, b: int, h: int, n: int,
                     scale: Optional[float] = None) -> torch.Tensor:
        qb = _bf16_bits(Q)
        assert qb.shape == (self.B, self.Hq, self.D)
        scale = self.D ** -0.5 if scale is None else scale
        w = torch.empty(n, dtype=torch.float64)
        rc = self.lib.oracle_attn_weights(self.h, layer, qb.data_ptr(), b, h, n, scale, w.data_ptr())
        if rc != 0:
            raise RuntimeError(f"oracle_attn_weights failed: {rc}")
        return w

    def decode_attn(self, layer: int, Q: torch.Tensor, seq_lens: torch.Tensor,
                    scale: Optional[float] = None) -> torch.Tensor:
        qb = _bf16_bits(Q)
        assert qb.shape == (self.B, self.Hq, self.D)
        lens = seq_lens.to(torch.int32).contiguous()
        assert lens.numel() == self.B
        scale = self.D ** -0.5 if scale is None else scale
        out = torch.empty((self.B, self.Hq, self.D), dtype=torch.float64)
        rc = self.lib.oracle_decode_attn(self.h, layer, qb.data_ptr(), lens.data_ptr(), scale, out.data_ptr())
        if rc != 0:
            raise RuntimeError(f"oracle_decode_attn failed: {rc}")
        return out

    def attn_rows(self, layer: int, Q: torch.Tensor, q_seq: torch.Tensor, q_pos: torch.Tensor,
                  scale: Optional[float] = None) -> torch.Tensor:
        """Pre-fill: row i of Q [n_q, Hq, D] is a token of sequence q_seq[i] at position q_pos[i] and
        attends tokens 0..q_pos[i] of the source layer's store of that sequence."""
        qb = _bf16_bits(Q)
        n_q = qb.shape[0]
        assert qb.shape == (n_q, self.Hq, self.D)
        s = q_seq.to(torch.int64).contiguous()
        p = q_pos.to(torch.int64).contiguous()
        assert s.numel() == n_q and p.numel() == n_q
        scale = self.D ** -0.5 if scale is None else scale
        out = torch.empty((n_q, self.Hq, self.D), dtype=torch.float64)
        rc = self.lib.oracle_attn_rows(self.h, layer, qb.data_ptr(), s.data_ptr(), p.data_ptr(), n_q, scale,
                                       out.data_ptr())
        if rc != 0:
            raise RuntimeError(f"oracle_attn_rows failed: {rc}")
        return out
