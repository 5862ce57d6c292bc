"""Shared test plumbing: run the CPU oracle on a synthetic checkpoint (numpy side only)."""
from __future__ import annotations

import numpy as np
import torch

import oracle
import patchkv_inputs as pin


def np_u16(t: torch.Tensor) -> np.ndarray:
    return t.detach().cpu().contiguous().view(torch.int16).numpy().view(np.uint16)


def oracle_select(ck: pin.SuffixCheckpoint):
    """Scores -> repair / reuse sets with the oracle.  Returns (mass u64 [L][NB], select dict)."""
    B = ck.geom.block_tokens
    if ck.attn is not None:
        rc, mass = oracle.block_mass(ck.attn.cpu().numpy(), B)
        assert rc == oracle.OK
    else:
        mass = ck.mass.cpu().numpy().astype(np.uint64)
    sel = oracle.select(mass, ck.n_suffix_tokens, B, ck.dirty_tokens, ck.top_k, ck.layer_mode)
    assert sel["status"] == oracle.OK
    return mass, sel


def layer_payloads(ck: pin.SuffixCheckpoint, layers=None):
    pay = ck.payload.cpu().numpy()
    layers = range(ck.geom.n_layers) if layers is None else layers
    return [pay[ck.layer_off[l]:ck.layer_off[l] + ck.layer_bytes[l]] for l in layers]


def oracle_restore(ck: pin.SuffixCheckpoint, reuse_idx, reuse_cnt, layers=None, n_threads=0, want_stats=False,
                   pools=None, **over):
    """Restore `layers` (default all) of a checkpoint into fresh sentinel pools [len(layers)][page][slot][H][D].

    Returns (status, k_pool u16, v_pool u16, stats).  `over` may override delta, dst_shift, block_table,
    n_pages, inv_freq, tags, blk_off.
    """
    g = ck.geom
    layers = list(range(g.n_layers)) if layers is None else list(layers)
    n_pages = over.get("n_pages", ck.n_pages)
    sub = pin.Geometry(len(layers), g.n_kv_heads, g.head_dim, g.rotary_dim, g.rope_style, g.rope_base,
                       g.block_tokens, g.page_tokens, g.group)
    if pools is None:
        shape = (len(layers), n_pages, g.page_tokens, g.n_kv_heads, g.head_dim)
        k_pool = np.full(shape, pin.SENTINEL, dtype=np.uint16)
        v_pool = np.full(shape, pin.SENTINEL, dtype=np.uint16)
    else:
        k_pool, v_pool = pools
    tags = np.asarray(over.get("tags", ck.tags.cpu().numpy()))[layers]
    blk_off = np.asarray(over.get("blk_off", ck.blk_off.cpu().numpy()))[layers]
    table = np.asarray(over.get("block_table", ck.block_table.cpu().numpy()), dtype=np.int32)
    rc, stats = oracle.restore(
        L=len(layers), H=g.n_kv_heads, D=g.head_dim, Dr=g.rotary_dim, rope_style=g.rope_style, rope_base=g.rope_base,
        B=g.block_tokens, P=g.page_tokens, G=g.group, k_pool=k_pool, v_pool=v_pool,
        strides=pin.pool_strides(sub, n_pages), n_pages=n_pages, n=ck.n_suffix_tokens,
        delta=over.get("delta", ck.delta), dst_shift=over.get("dst_shift", ck.dst_shift), block_table=table,
        tags=tags, blk_off=blk_off, layer_payload=layer_payloads(ck, layers),
        reuse_idx=np.asarray(reuse_idx)[layers], reuse_cnt=np.asarray(reuse_cnt)[layers],
        inv_freq=over.get("inv_freq"), n_threads=n_threads or oracle.max_threads(), want_stats=want_stats)
    return rc, k_pool, v_pool, stats


def bf16_bits_to_f64(u: np.ndarray) -> np.ndarray:
    return (u.astype(np.uint32) << 16).view(np.float32).astype(np.float64)


def bf16_ulp(x: np.ndarray) -> np.ndarray:
    """Spacing of bf16 numbers at magnitude |x| (8 significant bits), floored at the smallest normal binade."""
    ax = np.maximum(np.abs(x), 2.0 ** -126)
    return 2.0 ** (np.floor(np.log2(ax)) - 7)
