"""Seeded synthetic inputs for the routed KV-cache decode path.

This module only *draws inputs*: tensor values, sequence lengths, page
permutations and the routing maps the workload descriptions spell out.  It
holds none of the method's arithmetic (no attention, no cache layout, no
owner lookup), so both the CPU oracle's tests and the CUDA path's tests may
import it without sharing anything that is under test.

Every value is a pure function of ``(seed, kind, layer, sequence, position,
head, dim)`` computed with 32-bit integer hashing in torch integer ops, which
give identical bits on CPU and on CUDA.  Any subset of a workload (one
sequence, one layer, one token) can therefore be drawn on either device
without materialising the rest.

The five workloads mirror the attention shapes of the model families the
paper evaluates (Llama-2-7B, Llama-3-8B, Qwen3-8B; Section 1 and Section 4.3);
they stand in for the paper's own QA workloads, which need datasets and trained
weights that are not available here.
"""
from __future__ import annotations

import dataclasses
import math
from typing import List, Optional, Sequence, Tuple

import torch

__all__ = [
    "Workload", "WORKLOADS", "get_workload", "sweep_workload", "routing_map",
    "seq_lens", "page_layout", "slot_map_for", "draw_rows", "draw_q", "draw_kv",
    "KIND_K", "KIND_V", "KIND_Q", "POS_STRIDE",
]

KIND_K, KIND_V, KIND_Q, _KIND_LEN, _KIND_ROUTE = 1, 2, 3, 4, 5
POS_STRIDE = 1 << 20          # positions per sequence in the element counter
_M32 = 0xFFFFFFFF


# --------------------------------------------------------------------------
# counter-based generator (integer only => same bits on every device)
# --------------------------------------------------------------------------
def _mul32(x: torch.Tensor, c: int) -> torch.Tensor:
    """(x * c) mod 2^32 for int64 tensors holding values < 2^32, no overflow."""
    lo, hi = c & 0xFFFF, (c >> 16) & 0xFFFF
    return (x * lo + (((x * hi) & 0xFFFF) << 16)) & _M32


def _mix32(x: torch.Tensor) -> torch.Tensor:
    """32-bit avalanche mixer (xor-shift / multiply rounds)."""
    x = x ^ (x >> 16)
    x = _mul32(x, 0x7FEB352D)
    x = x ^ (x >> 15)
    x = _mul32(x, 0x846CA68B)
    x = x ^ (x >> 16)
    return x


def _mix32_int(x: int) -> int:
    x &= _M32
    x ^= x >> 16
    x = (x * 0x7FEB352D) & _M32
    x ^= x >> 15
    x = (x * 0x846CA68B) & _M32
    x ^= x >> 16
    return x


def _stream_key(seed: int, kind: int, layer: int) -> int:
    k = _mix32_int(seed * 0x9E3779B1 + 0x1234567)
    k = _mix32_int(k ^ (kind * 0x85EBCA77))
    k = _mix32_int(k ^ (layer * 0xC2B2AE3D + 0x27D4EB2F))
    return k


def _hash_counter(counter: torch.Tensor, key: int) -> torch.Tensor:
    """int64 counters (< 2^63) -> 32 pseudo-random bits each (as int64)."""
    lo = counter & _M32
    hi = (counter >> 32) & _M32
    h = _mix32(hi ^ key)
    return _mix32(lo ^ h)


_TABLE_CACHE: dict = {}


def _normal_table(device: torch.device) -> torch.Tensor:
    """65536 standard-normal quantiles, fp32, always computed on the CPU."""
    key = str(device)
    if key not in _TABLE_CACHE:
        u = (torch.arange(65536, dtype=torch.float64) + 0.5) / 65536.0
        z = math.sqrt(2.0) * torch.special.erfinv(2.0 * u - 1.0)
        _TABLE_CACHE[key] = z.to(torch.float32).to(device)
    return _TABLE_CACHE[key]


def draw_rows(seed: int, kind: int, layer: int, seq_idx: torch.Tensor,
              pos: torch.Tensor, heads: int, dim: int, std: float = 1.0,
              device: Optional[torch.device] = None) -> torch.Tensor:
    """bf16 tensor ``[n, heads, dim]`` ~ N(0, std^2) for rows (seq_idx[i], pos[i]).

    The value of an element depends only on (seed, kind, layer, seq, pos, head,
    dim); it is bf16(std * z) with z one of 65536 normal quantiles picked by
    the low 16 bits of the element's hash.
    """
    device = torch.device(device) if device is not None else seq_idx.device
    seq_idx = seq_idx.to(device=device, dtype=torch.int64)
    pos = pos.to(device=device, dtype=torch.int64)
    n = seq_idx.numel()
    out = torch.empty((n, heads, dim), dtype=torch.bfloat16, device=device)
    if n == 0:
        return out
    table = _normal_table(device)
    key = _stream_key(seed, kind, layer)
    # one hash per row, then one mixing round per element of the row
    inner = _mul32(torch.arange(1, heads * dim + 1, dtype=torch.int64, device=device), 0x9E3779B1)
    rows_per_chunk = max(1, (1 << 22) // (heads * dim))
    for s in range(0, n, rows_per_chunk):
        e = min(n, s + rows_per_chunk)
        row_hash = _hash_counter(seq_idx[s:e] * POS_STRIDE + pos[s:e], key)
        bits = _mix32(row_hash[:, None] ^ inner[None, :]) & 0xFFFF
        out[s:e] = (table[bits] * std).to(torch.bfloat16).view(e - s, heads, dim)
    return out


# --------------------------------------------------------------------------
# workload descriptions
# --------------------------------------------------------------------------
@dataclasses.dataclass(frozen=True)
class Workload:
    name: str
    n_layers: int
    q_heads: int
    kv_heads: int
    head_dim: int
    page_size: int
    batch: int
    len_lo: int
    len_hi: int
    routing: str                 # "explicit", "groups", "stochastic"
    group: int = 1               # for "groups": r(l) = l - (l mod group)
    explicit_r: Tuple[int, ...] = ()
    explicit_lens: Tuple[int, ...] = ()
    seed: int = 0
    q_std: float = 1.0
    kv_std: float = 1.0
    permute_pages: bool = True
    family: str = ""

    @property
    def group_size(self) -> int:   # query heads per kv head
        return self.q_heads // self.kv_heads


WORKLOADS = {
    # 4 layers, r=[0,0,2,2], 4 q heads / 2 kv heads, D=64, lens {37,128}, contiguous pages
    "tiny": Workload("tiny", 4, 4, 2, 64, 16, 2, 37, 128, "explicit",
                     explicit_r=(0, 0, 2, 2), explicit_lens=(37, 128), seed=0,
                     permute_pages=False, family="tiny"),
    # Llama-3-8B attention shape, every second layer owns
    "llama3_8b": Workload("llama3_8b", 32, 32, 8, 128, 16, 32, 1024, 4096, "groups",
                          group=2, seed=1, family="Llama-3-8B"),
    # Qwen3-8B attention shape, groups of four
    "qwen3_8b": Workload("qwen3_8b", 36, 32, 8, 128, 16, 64, 2048, 8192, "groups",
                         group=4, seed=2, q_std=0.5, family="Qwen3-8B"),
    # Llama-2-7B MHA, long context, stochastic map
    "llama2_7b_32k": Workload("llama2_7b_32k", 32, 32, 32, 128, 16, 8, 32768, 32768,
                              "stochastic", seed=3, family="Llama-2-7B"),
}


# the same attention call as "llama3_8b" (same batch, lengths, page permutation) with only two
# layers, so that a profiler capture holds a few hundred MB instead of the whole model's cache
WORKLOADS["llama3_8b_2layers"] = dataclasses.replace(WORKLOADS["llama3_8b"], name="llama3_8b_2layers", n_layers=2)


def sweep_workload(group: int) -> Workload:
    """Sharing-ratio sweep on the Llama-3-8B shape: owner fraction 1/group."""
    return Workload(f"sweep_g{group}", 32, 32, 8, 128, 16, 128, 512, 2048, "groups",
                    group=group, seed=4, family="Llama-3-8B")


for _g in (1, 2, 4, 8):
    WORKLOADS[f"sweep_g{_g}"] = sweep_workload(_g)


# Table 4's shape (Section 4.3): the Qwen3-8B architecture with groups of four layers, ONE sequence, 2 048
# or 8 192 prompt tokens plus the 128 generated ones.  An owner layer's cache is 8.9 / 34.1 MB here,
# well inside the L2 cache: the three reader layers of a group re-read what the owner layer just
# streamed.  Four groups (16 layers) are enough to show that.
for _t in (2048, 8192):
    WORKLOADS[f"qwen3_8b_b1_{_t // 1024}k"] = Workload(
        f"qwen3_8b_b1_{_t // 1024}k", 16, 32, 8, 128, 16, 1, _t + 128, _t + 128, "groups", group=4,
        explicit_lens=(_t + 128,), seed=5, q_std=0.5, family="Qwen3-8B")


def get_workload(name: str) -> Workload:
    return WORKLOADS[name]


def routing_map(w: Workload) -> List[int]:
    """0-based routing map r[l] exactly as the workload description states it."""
    L = w.n_layers
    if w.routing == "explicit":
        return list(w.explicit_r)
    if w.routing == "groups":
        return [l - (l % w.group) for l in range(L)]
    if w.routing == "stochastic":
        # layer 0 owns; each later layer: with probability 1/2 it reads a
        # uniformly chosen preceding owner, otherwise it owns its cache.
        r = [0]
        owners = [0]
        for l in range(1, L):
            h = _mix32_int(_stream_key(w.seed, _KIND_ROUTE, l))
            if (h & 1) == 1:
                pick = (h >> 8) % len(owners)
                r.append(owners[pick])
            else:
                r.append(l)
                owners.append(l)
        return r
    raise ValueError(w.routing)


def seq_lens(w: Workload, batch: Optional[int] = None) -> torch.Tensor:
    """int32 ``[batch]`` lengths, uniform on [len_lo, len_hi] (inclusive)."""
    B = w.batch if batch is None else batch
    if w.explicit_lens:
        assert B == len(w.explicit_lens)
        return torch.tensor(list(w.explicit_lens), dtype=torch.int32)
    span = w.len_hi - w.len_lo + 1
    key = _stream_key(w.seed, _KIND_LEN, 0)
    h = _hash_counter(torch.arange(B, dtype=torch.int64), key)
    return (w.len_lo + (h % span)).to(torch.int32)


def page_layout(lens: torch.Tensor, page_size: int, permute: bool, seed: int,
                extra_pages: int = 0) -> Tuple[torch.Tensor, int]:
    """Physical page table ``[B, max_pages_per_seq]`` (int32, -1 = unused).

    Pages needed are handed out to (sequence, logical page) in order from a
    seeded random permutation of ``[0, total)`` (or the identity order).
    Returns (page_table, total_pages).
    """
    lens64 = lens.to(torch.int64)
    pages = (lens64 + page_size - 1) // page_size
    total = int(pages.sum().item()) + extra_pages
    B = lens.numel()
    width = max(1, int(pages.max().item()) if B else 1)
    if permute:
        g = torch.Generator(device="cpu")
        g.manual_seed(1000003 * (seed + 1) + 17)
        order = torch.randperm(total, generator=g, dtype=torch.int64)
    else:
        order = torch.arange(total, dtype=torch.int64)
    table = torch.full((B, width), -1, dtype=torch.int32)
    cur = 0
    for b in range(B):
        nb = int(pages[b])
        table[b, :nb] = order[cur:cur + nb].to(torch.int32)
        cur += nb
    return table, total


def slot_map_for(page_table: torch.Tensor, seq_idx: torch.Tensor, pos: torch.Tensor,
                 page_size: int) -> torch.Tensor:
    """int64 slot ids ``page * page_size + offset`` for tokens (seq_idx[i], pos[i])."""
    seq_idx = seq_idx.to(torch.int64)
    pos = pos.to(torch.int64)
    page = page_table.to(torch.int64)[seq_idx, pos // page_size]
    return page * page_size + pos % page_size


def token_index(lens: torch.Tensor, upto_offset: int = 0) -> Tuple[torch.Tensor, torch.Tensor]:
    """(seq_idx, pos) of every token t < lens[b] + upto_offset, sequence-major."""
    lens64 = (lens.to(torch.int64) + upto_offset).clamp(min=0)
    B = lens64.numel()
    seq_idx = torch.repeat_interleave(torch.arange(B, dtype=torch.int64), lens64)
    starts = torch.cumsum(lens64, 0) - lens64
    pos = torch.arange(int(lens64.sum()), dtype=torch.int64) - torch.repeat_interleave(starts, lens64)
    return seq_idx, pos


def draw_q(w: Workload, layer: int, batch: Optional[int] = None, step: int = 0,
           device="cpu") -> torch.Tensor:
    """Queries ``[B, q_heads, head_dim]`` bf16 for one layer of one decode step."""
    B = w.batch if batch is None else batch
    b = torch.arange(B, dtype=torch.int64)
    return draw_rows(w.seed, KIND_Q, layer, b, torch.full((B,), step, dtype=torch.int64),
                     w.q_heads, w.head_dim, w.q_std, device)


def draw_kv(w: Workload, layer: int, seq_idx: torch.Tensor, pos: torch.Tensor,
            device="cpu") -> Tuple[torch.Tensor, torch.Tensor]:
    """(K, V) rows ``[n, kv_heads, head_dim]`` bf16 of one layer."""
    k = draw_rows(w.seed, KIND_K, layer, seq_idx, pos, w.kv_heads, w.head_dim, w.kv_std, device)
    v = draw_rows(w.seed, KIND_V, layer, seq_idx, pos, w.kv_heads, w.head_dim, w.kv_std, device)
    return k, v
