"""Marshalling of a synthetic SuffixCheckpoint into the CUDA library's argument structs.

Test and benchmark plumbing (used by the GPU tests, the smoke check and bench.py; the CPU checker's tests never
import it).  Holds no arithmetic of the method: it moves tensors to the device (or to pinned host memory),
allocates the output arrays and fills the POD structs of paper_2609_26219_b200.binding.
"""
from __future__ import annotations

from typing import Optional

import torch

import patchkv_inputs as pin
from paper_2609_26219_b200 import binding as pk


class StagedCheckpoint:
    """Device-side (or pinned-host) image of one session plus its selection outputs."""

    def __init__(self, ck: pin.SuffixCheckpoint, device="cuda:0", payload_on_host: bool = False):
        self.ck = ck
        self.device = torch.device(device)
        g = ck.geom
        L, NB = g.n_layers, ck.n_blocks
        dev = self.device
        self.tags = ck.tags.to(dev).contiguous()
        self.blk_off = ck.blk_off.to(dev).contiguous()
        self.block_table = ck.block_table.to(dev).contiguous()
        self.payload_on_host = payload_on_host
        if payload_on_host:
            self.payload = ck.payload if ck.payload.is_pinned() else ck.payload.cpu().pin_memory()
        else:
            self.payload = ck.payload.to(dev)
        base = self.payload.data_ptr()
        assert base % 256 == 0
        ptrs = torch.tensor([base + o for o in ck.layer_off], dtype=torch.int64)
        lbytes = torch.tensor(ck.layer_bytes, dtype=torch.int64)
        self.layer_ptrs_host, self.layer_bytes_host = ptrs, lbytes
        self.layer_ptrs, self.layer_bytes = ptrs.to(dev), lbytes.to(dev)
        self.mass = None if ck.mass is None else ck.mass.to(dev).contiguous()
        self.attn = None if ck.attn is None else ck.attn.to(dev)
        self.mass_out = torch.zeros((L, NB), dtype=torch.int64, device=dev)
        self.repair_mask = torch.full((L, NB), 255, dtype=torch.uint8, device=dev)
        self.repair_idx = torch.full((L, NB), -7, dtype=torch.int32, device=dev)
        self.reuse_idx = torch.full((L, NB), -7, dtype=torch.int32, device=dev)
        self.repair_cnt = torch.full((L,), -7, dtype=torch.int32, device=dev)
        self.reuse_cnt = torch.full((L,), -7, dtype=torch.int32, device=dev)
        self._host_lists = None

    # ---- structs
    def geom(self, inv_freq: Optional[torch.Tensor] = None) -> pk.Geom:
        g = self.ck.geom
        return pk.make_geom(g.n_layers, g.n_kv_heads, g.head_dim, g.rotary_dim, g.rope_style, g.rope_base,
                            g.block_tokens, g.page_tokens, g.group, inv_freq)

    def select_args(self, use_mass_out: bool = True, **over) -> pk.SelectArgs:
        ck = self.ck
        kw = dict(kind=pk.SCORE_ATTN_F16 if self.attn is not None else pk.SCORE_BLOCK_MASS,
                  n_layers=ck.geom.n_layers, n_suffix_tokens=ck.n_suffix_tokens, block_tokens=ck.geom.block_tokens,
                  dirty_tokens=ck.dirty_tokens, top_k=ck.top_k, layer_mode=ck.layer_mode,
                  repair_mask=self.repair_mask, repair_idx=self.repair_idx, repair_cnt=self.repair_cnt,
                  reuse_idx=self.reuse_idx, reuse_cnt=self.reuse_cnt, attn=self.attn, mass=self.mass,
                  mass_out=self.mass_out if (use_mass_out and self.attn is not None) else None)
        kw.update(over)
        return pk.select_args(**kw)

    def session(self, **over) -> pk.Session:
        ck = self.ck
        kw = dict(n_suffix_tokens=ck.n_suffix_tokens, delta=ck.delta, dst_shift=ck.dst_shift,
                  block_table=self.block_table, tags=self.tags, blk_off=self.blk_off,
                  layer_payload=self.layer_ptrs, layer_bytes=self.layer_bytes,
                  reuse_idx=self.reuse_idx, reuse_cnt=self.reuse_cnt)
        kw.update(over)
        return pk.make_session(**kw)

    def host_session(self, **over) -> pk.Session:
        """Session struct for restore_from_host: host copies of the directory and of the reuse lists (the
        device-to-host read of the selection result is part of the caller's resume path)."""
        ck = self.ck
        self._host_lists = dict(
            block_table=ck.block_table.cpu().contiguous(), tags=ck.tags.cpu().contiguous(),
            blk_off=ck.blk_off.cpu().contiguous(), reuse_idx=self.reuse_idx.cpu(), reuse_cnt=self.reuse_cnt.cpu())
        kw = dict(n_suffix_tokens=ck.n_suffix_tokens, delta=ck.delta, dst_shift=ck.dst_shift,
                  layer_payload=self.layer_ptrs_host, layer_bytes=self.layer_bytes_host, **self._host_lists)
        kw.update(over)
        self._host_keep = kw
        return pk.make_session(**kw)


def device_pool(ck: pin.SuffixCheckpoint, device="cuda:0", n_pages: Optional[int] = None):
    """Sentinel-filled K and V pools [L][page][slot][H][D] (int16 bit patterns) and the Pool struct."""
    n_pages = ck.n_pages if n_pages is None else n_pages
    k, v = pin.make_pool(ck.geom, n_pages, device=device)
    return k, v, pk.make_pool(k, v, n_pages, pin.pool_strides(ck.geom, n_pages))
