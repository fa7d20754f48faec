"""Driving code shared by the GPU tests, the smoke check and the benchmark:
sets a workload up on the device through the binding (pool, page table, cache
pre-fill, per-step inputs).  It draws inputs from :mod:`workloads` and calls
the library; it contains no arithmetic of the method and never touches the
oracle."""
from __future__ import annotations

import dataclasses
from typing import Dict, List, Optional

import torch

import workloads as W

from .binding import SkvCache


@dataclasses.dataclass
class DeviceWorkload:
    w: W.Workload
    r: List[int]
    lens_cpu: torch.Tensor            # int32 [B], tokens attended in the decode step
    page_table_cpu: torch.Tensor      # int32 [B, width]
    total_pages: int
    cache: SkvCache
    page_table: torch.Tensor          # device copies
    seq_lens: torch.Tensor
    slot_new: torch.Tensor            # int64 [B] slot of each sequence's newest token (position n_b-1)
    workspace: torch.Tensor
    device: torch.device

    @property
    def batch(self) -> int:
        return int(self.lens_cpu.numel())

    @property
    def owners(self) -> List[int]:
        return [l for l in range(self.w.n_layers) if self.r[l] == l]

    def retune(self, variant=None, tuning=None, overlap=None, l2_keep=None, early_fetch=None, worker=None,
               merge=None) -> None:
        """Change kernel variant / launch shape / overlap / L2 reuse / early fetch, then size the workspace again."""
        if variant is not None:
            self.cache.skv_set_decode_variant(variant)
        if tuning is not None:
            self.cache.skv_set_decode_tuning(*tuning)
        if overlap is not None:
            self.cache.skv_set_decode_overlap(overlap)
        if l2_keep is not None:
            self.cache.skv_set_decode_l2_reuse(l2_keep)
        if early_fetch is not None:
            self.cache.skv_set_decode_early_fetch(early_fetch)
        if worker is not None:                       # mode, or (mode, consumers, stages, CTAs per SM)
            self.cache.skv_set_decode_worker(*((worker,) if isinstance(worker, int) else worker))
        if merge is not None:                        # 0 auto, 1 merge kernel, 2 inside the CTA-per-range kernel
            self.cache.skv_set_decode_merge(merge)
        need = self.cache.skv_decode_workspace_bytes(self.batch, self.w.q_heads)
        if need > self.workspace.numel():
            self.workspace = torch.empty(need, dtype=torch.uint8, device=self.device)

    def kv_bytes_per_call(self) -> int:
        """Algorithmic bytes of one decode-attention call: the owner layer's K,V of
        every attended token (bf16, or FP8 codes plus one fp32 scale per row), plus Q in and out out."""
        w = self.w
        tokens = int(self.lens_cpu.to(torch.int64).sum())
        row = (w.head_dim + 4) if self.cache.fp8 else w.head_dim * 2
        return tokens * w.kv_heads * row * 2 + 2 * self.batch * w.q_heads * w.head_dim * 2

    def append_bytes_per_call(self) -> int:
        """Algorithmic bytes of one owner-layer append of one token per sequence (read + write)."""
        w = self.w
        return 2 * (self.batch * w.kv_heads * w.head_dim * 2 * 2)


def setup(w: W.Workload, device="cuda", lens: Optional[torch.Tensor] = None, r: Optional[List[int]] = None,
          extra_pages: int = 0, permute: Optional[bool] = None, fp8: bool = False) -> DeviceWorkload:
    device = torch.device(device)
    r = W.routing_map(w) if r is None else list(r)
    lens_cpu = (W.seq_lens(w) if lens is None else lens).to(torch.int32)
    B = int(lens_cpu.numel())
    table, total = W.page_layout(lens_cpu, w.page_size, w.permute_pages if permute is None else permute, w.seed,
                                 extra_pages=extra_pages)
    total = max(total, 1)
    cache = SkvCache(r, w.kv_heads, w.head_dim, w.page_size, total, allocate=True, fp8=fp8)
    ws = torch.empty(cache.skv_decode_workspace_bytes(B, w.q_heads), dtype=torch.uint8, device=device)
    b = torch.arange(B, dtype=torch.int64)
    last = (lens_cpu.to(torch.int64) - 1)
    has = last >= 0
    slot_new = torch.full((B,), -1, dtype=torch.int64)
    if bool(has.any()):
        slot_new[has] = W.slot_map_for(table, b[has], last[has], w.page_size)
    return DeviceWorkload(w=w, r=r, lens_cpu=lens_cpu, page_table_cpu=table, total_pages=total, cache=cache,
                          page_table=table.to(device), seq_lens=lens_cpu.to(device),
                          slot_new=slot_new.to(device), workspace=ws, device=device)


def prefill(dw: DeviceWorkload, upto_offset: int = -1, layers: Optional[List[int]] = None,
            chunk_tokens: int = 1 << 16, draw_on=None) -> None:
    """Append tokens t < lens[b] + upto_offset of every owner layer.  The rows are drawn on the device
    unless `draw_on` names another one ("cpu": drawn on the host and copied over, so that the only
    kernels on the GPU are the library's; the generator gives the same bits on either)."""
    w = dw.w
    seq_idx, pos = W.token_index(dw.lens_cpu, upto_offset)
    slots = W.slot_map_for(dw.page_table_cpu, seq_idx, pos, w.page_size)
    for l in (dw.owners if layers is None else layers):
        if dw.r[l] != l:
            continue
        for s in range(0, seq_idx.numel(), chunk_tokens):
            e = min(seq_idx.numel(), s + chunk_tokens)
            K, V = W.draw_kv(w, l, seq_idx[s:e], pos[s:e], device=dw.device if draw_on is None else draw_on)
            dw.cache.skv_append(l, K.to(dw.device), V.to(dw.device), slots[s:e].to(dw.device))
    torch.cuda.synchronize(dw.device)


def step_inputs(dw: DeviceWorkload, layer: int, device=None) -> Dict[str, torch.Tensor]:
    """Q of `layer` and the newest token's K,V rows (position lens[b]-1) for this decode step."""
    w = dw.w
    device = dw.device if device is None else device
    B = dw.batch
    b = torch.arange(B, dtype=torch.int64)
    last = (dw.lens_cpu.to(torch.int64) - 1).clamp(min=0)
    K, V = W.draw_kv(w, layer, b, last, device=device)
    return {"Q": W.draw_q(w, layer, batch=B, device=device), "K": K, "V": V}


def step_tensors(dw: DeviceWorkload, device=None, pin: bool = False) -> Dict[str, torch.Tensor]:
    """Inputs of one whole decode step, stacked: Q [L,B,Hq,D]; K,V [n_owners,B,Hkv,D] (owner layers in
    increasing order); out buffer [L,B,Hq,D]."""
    w = dw.w
    device = dw.device if device is None else torch.device(device)
    qs, ks, vs = [], [], []
    for l in range(w.n_layers):
        inp = step_inputs(dw, l, device=device)
        qs.append(inp["Q"])
        if dw.r[l] == l:
            ks.append(inp["K"])
            vs.append(inp["V"])
    t = {"Q": torch.stack(qs).contiguous(), "K": torch.stack(ks).contiguous(), "V": torch.stack(vs).contiguous()}
    t["out"] = torch.zeros_like(t["Q"])
    if pin and device.type == "cpu":
        t = {k: v.pin_memory() for k, v in t.items()}
    return t


def prefill_inputs(dw: DeviceWorkload, layer: int, q_lens: torch.Tensor, device=None) -> Dict[str, torch.Tensor]:
    """Query rows of a pre-fill call: sequence b contributes its LAST q_lens[b] tokens (positions
    lens[b]-q_lens[b] .. lens[b]-1).  Returns Q [n_q,Hq,D] (drawn), cu_q_lens [B+1] (int32), and the rows'
    (sequence, position) as int64 CPU tensors."""
    w = dw.w
    device = dw.device if device is None else device
    q64 = q_lens.to(torch.int64)
    q_seq, i = W.token_index(q64)
    q_pos = (dw.lens_cpu.to(torch.int64) - q64)[q_seq] + i
    Q = W.draw_rows(w.seed, W.KIND_Q, layer, q_seq, q_pos, w.q_heads, w.head_dim, w.q_std, device)
    cu = torch.zeros(q64.numel() + 1, dtype=torch.int32)
    cu[1:] = torch.cumsum(q64, 0).to(torch.int32)
    return {"Q": Q, "cu_q_lens": cu.to(device), "q_seq": q_seq, "q_pos": q_pos}
