"""Seeded synthetic inputs for the PatchKV suffix-restore path.

This module only *produces inputs*: suffix KV checkpoints in the packed per-block
format, stored attention / block masses, block tables and paged pools.  It is the
one module that both the CPU oracle's tests and the CUDA library's tests and
benchmark consume.  It contains none of the restore or selection arithmetic
(no dequantisation, no RoPE, no placement, no scoring, no top-k); it does contain
an encoder, because a checkpoint has to be written by something before it can be
restored.  The paper's offload side gathers block rows, computes scales and packs
K8/V4, K8/V8 or full-precision payloads, clustered in same-representation runs
(Section IV-D); the encoder here is a plain torch statement of that, used only to
make inputs.

Checkpoint byte layout written here (the paper gives none):

* one payload per layer: all BF16-tag block records, then all INT8-tag records,
  then all INT4-tag records, then all K4V4 records, each group in ascending block
  index; every layer payload starts on a 256-byte boundary of one flat buffer;
* one block record = [K codes][K scales][V codes][V scales]; codes are
  [token][head][channel] row-major; bf16 codes are 2 bytes, int8 codes 1 byte
  (two's complement), int4 codes pack channel c (even) in bits 0-3 and c+1 in bits
  4-7 (two's complement nibbles); scales are fp16 [token][head][channel // group];
  a bf16 section has no scales; a partial last block is zero-padded to a whole block;
* directory: tags u8 [L][NB], blk_off u64 [L][NB] = byte offset of the record inside
  its layer payload.

Tags: 0 = K bf16 / V bf16, 1 = K int8 / V int8, 2 = K int8 / V int4 (the paper's
low-bit tier keeps keys at 8 bits), 3 = K int4 / V int4 (uniform-INT4 ablation).
"""
from __future__ import annotations

import math
from dataclasses import dataclass, field, replace
from typing import List, Optional

import numpy as np
import torch

TAG_BF16, TAG_INT8, TAG_INT4, TAG_K4V4 = 0, 1, 2, 3
FMT_BF16, FMT_INT8, FMT_INT4 = 0, 1, 2
ROPE_HALF, ROPE_INTERLEAVED = 0, 1
LAYERS_INDEPENDENT, LAYERS_SHARED = 0, 1
SENTINEL = 0xDEAD  # halfword the pools are pre-filled with

_K_FMT = {TAG_BF16: FMT_BF16, TAG_INT8: FMT_INT8, TAG_INT4: FMT_INT8, TAG_K4V4: FMT_INT4}
_V_FMT = {TAG_BF16: FMT_BF16, TAG_INT8: FMT_INT8, TAG_INT4: FMT_INT4, TAG_K4V4: FMT_INT4}


@dataclass(frozen=True)
class Geometry:
    n_layers: int
    n_kv_heads: int
    head_dim: int
    rotary_dim: int
    rope_style: int
    rope_base: float
    block_tokens: int
    page_tokens: int
    group: int


def section_bytes(fmt: int, g: Geometry) -> tuple[int, int]:
    """(code bytes, scale bytes) of one K or V section of a block record."""
    elems = g.block_tokens * g.n_kv_heads * g.head_dim
    scales = 2 * elems // g.group
    if fmt == FMT_BF16:
        return 2 * elems, 0
    if fmt == FMT_INT8:
        return elems, scales
    return elems // 2, scales


def record_bytes(tag: int, g: Geometry) -> int:
    kc, ks = section_bytes(_K_FMT[tag], g)
    vc, vs = section_bytes(_V_FMT[tag], g)
    return kc + ks + vc + vs


@dataclass
class SuffixCheckpoint:
    """One resumed session: the old checkpoint of its aligned suffix plus the plan inputs."""
    geom: Geometry
    n_suffix_tokens: int
    delta: int
    dst_shift: int
    tags: torch.Tensor            # u8  [L][NB]
    blk_off: torch.Tensor         # i64 [L][NB] (non-negative; read as u64)
    payload: torch.Tensor         # u8 flat; layer l occupies [layer_off[l], layer_off[l]+layer_bytes[l])
    layer_off: List[int]
    layer_bytes: List[int]
    block_table: torch.Tensor     # i32 [n_table]
    n_pages: int
    dirty_tokens: int
    top_k: int
    layer_mode: int = LAYERS_INDEPENDENT
    mass: Optional[torch.Tensor] = None   # i64 [L][NB] (units of 2^-24), or None when attn is given
    attn: Optional[torch.Tensor] = None   # fp16 [L][Hq][Q][n]
    name: str = ""
    raw_kv: Optional[list] = None         # [(K, V) fp32 [NB*B][H][D]] per layer, kept only on request

    @property
    def n_blocks(self) -> int:
        return -(-self.n_suffix_tokens // self.geom.block_tokens)


def pool_strides(g: Geometry, n_pages: int) -> tuple[int, int, int, int]:
    """Element strides (layer, page, token, head) of the benchmark pool layout [L][page][slot][H][D]."""
    s_head = g.head_dim
    s_token = g.n_kv_heads * g.head_dim
    s_page = g.page_tokens * s_token
    s_layer = n_pages * s_page
    return s_layer, s_page, s_token, s_head


def make_pool(g: Geometry, n_pages: int, device="cpu") -> tuple[torch.Tensor, torch.Tensor]:
    """Two sentinel-filled bf16 pools (K and V), returned as int16 bit patterns [L][page][slot][H][D]."""
    shape = (g.n_layers, n_pages, g.page_tokens, g.n_kv_heads, g.head_dim)
    fill = SENTINEL - 0x10000  # same 16 bits as a signed halfword
    k = torch.full(shape, fill, dtype=torch.int16, device=device)
    v = torch.full(shape, fill, dtype=torch.int16, device=device)
    return k, v


# --------------------------------------------------------------------------- encoder
def _quantise(x: torch.Tensor, group: int, qmax: int) -> tuple[torch.Tensor, torch.Tensor]:
    """Symmetric per-group codes: s = fp16(amax / qmax), q = clamp(rint(x / s), -qmax, qmax), s = 0 -> q = 0."""
    lead = x.shape[:-1]
    xg = x.reshape(*lead, x.shape[-1] // group, group)
    amax = xg.abs().amax(dim=-1, keepdim=True)
    s16 = (amax / float(qmax)).to(torch.float16)
    s = s16.to(torch.float32)
    q = torch.where(s > 0, torch.round(xg / torch.where(s > 0, s, torch.ones_like(s))), torch.zeros_like(xg))
    q = q.clamp_(-qmax, qmax).to(torch.int8).reshape(*lead, x.shape[-1])
    return q, s16.squeeze(-1)


def _section(x: torch.Tensor, fmt: int, group: int) -> List[torch.Tensor]:
    """x: [nb][B][H][D] fp32 -> [codes u8 [nb][*], scales u8 [nb][*]] for one K or V section."""
    nb = x.shape[0]
    if fmt == FMT_BF16:
        return [x.to(torch.bfloat16).contiguous().view(torch.uint8).reshape(nb, -1)]
    if fmt == FMT_INT8:
        q, s = _quantise(x, group, 127)
        return [q.contiguous().view(torch.uint8).reshape(nb, -1),
                s.contiguous().view(torch.uint8).reshape(nb, -1)]
    q, s = _quantise(x, group, 7)
    nib = (q.to(torch.int16) & 0xF).to(torch.uint8)
    packed = nib[..., 0::2] | (nib[..., 1::2] << 4)
    return [packed.contiguous().reshape(nb, -1), s.contiguous().view(torch.uint8).reshape(nb, -1)]


def encode_layer(k: torch.Tensor, v: torch.Tensor, tags_l: torch.Tensor, g: Geometry):
    """k, v: [NB*B][H][D] fp32 (zero-padded past the suffix); tags_l: u8 [NB].

    Returns (payload u8 [bytes], blk_off i64 [NB]) in the clustered layout described above.
    """
    nb_total = tags_l.numel()
    kb = k.reshape(nb_total, g.block_tokens, g.n_kv_heads, g.head_dim)
    vb = v.reshape(nb_total, g.block_tokens, g.n_kv_heads, g.head_dim)
    blk_off = torch.zeros(nb_total, dtype=torch.int64, device=k.device)
    parts, base = [], 0
    for tag in (TAG_BF16, TAG_INT8, TAG_INT4, TAG_K4V4):
        idx = torch.nonzero(tags_l == tag).flatten()
        if idx.numel() == 0:
            continue
        rec = torch.cat(_section(kb[idx], _K_FMT[tag], g.group) + _section(vb[idx], _V_FMT[tag], g.group), dim=1)
        assert rec.shape[1] == record_bytes(tag, g)
        blk_off[idx] = base + torch.arange(idx.numel(), device=k.device, dtype=torch.int64) * rec.shape[1]
        parts.append(rec.reshape(-1))
        base += rec.numel()
    payload = torch.cat(parts) if parts else torch.zeros(0, dtype=torch.uint8, device=k.device)
    return payload, blk_off


# --------------------------------------------------------------------------- generators
def _kv_layer(gen: torch.Generator, g: Geometry, n: int, n_outlier: int, outlier_scale: float, device):
    """K, V ~ N(0,1) fp32 [NB*B][H][D] with n_outlier channels per head scaled, rows >= n zeroed."""
    nb = -(-n // g.block_tokens)
    shape = (nb * g.block_tokens, g.n_kv_heads, g.head_dim)
    out = []
    for _ in range(2):
        x = torch.randn(shape, generator=gen, device=device, dtype=torch.float32)
        if n_outlier > 0:
            scale = torch.ones(g.n_kv_heads, g.head_dim, device=device)
            for h in range(g.n_kv_heads):
                ch = torch.randperm(g.head_dim, generator=gen, device=device)[:n_outlier]
                scale[h, ch] = outlier_scale
            x = x * scale
        x[n:] = 0
        out.append(x)
    return out[0], out[1]


def _draw_tags(gen, probs, shape, device) -> torch.Tensor:
    p = torch.tensor(probs, dtype=torch.float32, device=device)
    flat = torch.multinomial(p, int(np.prod(shape)), replacement=True, generator=gen)
    return flat.to(torch.uint8).reshape(shape)


def zipf_block_mass(gen, n_layers: int, n_blocks: int, device, exponent: float = 1.2) -> torch.Tensor:
    """Per layer a seeded permutation of ranks r; mass = floor(2^36 * (r+1)^-exponent) units of 2^-24."""
    rows = []
    for _ in range(n_layers):
        r = torch.randperm(n_blocks, generator=gen, device=device).to(torch.float64)
        rows.append(torch.floor((2.0 ** 36) * (r + 1.0) ** (-exponent)).to(torch.int64))
    return torch.stack(rows)


def softmax_attention(gen, n_layers, n_q_heads, n_queries, n, device, logit_std=2.0) -> torch.Tensor:
    """fp16 [L][Hq][Q][n]: row softmax (fp32) of logit_std * N(0,1) logits."""
    logits = logit_std * torch.randn((n_layers, n_q_heads, n_queries, n), generator=gen, device=device)
    return torch.softmax(logits, dim=-1).to(torch.float16)


def zipf_attention(gen, n_layers, n_q_heads, n_queries, n, device, exponent=1.2, noise=0.5) -> torch.Tensor:
    """fp16 [L][Hq][Q][n]: per layer, key weight (rank+1)^-exponent under a seeded permutation of key
    positions, times exp(noise * N(0,1)) per entry, row-normalised in fp32."""
    out = torch.empty((n_layers, n_q_heads, n_queries, n), dtype=torch.float16, device=device)
    for l in range(n_layers):
        r = torch.randperm(n, generator=gen, device=device).to(torch.float32)
        base_logit = -exponent * torch.log(r + 1.0)
        for h in range(n_q_heads):
            z = base_logit + noise * torch.randn((n_queries, n), generator=gen, device=device)
            out[l, h] = torch.softmax(z, dim=-1).to(torch.float16)
    return out


def make_checkpoint(*, name: str, seed: int, geom: Geometry, n: int, delta: int, dst_shift: int = 0,
                    tag_probs=(1 / 3, 1 / 3, 1 / 3, 0.0), tags_per_layer: bool = False,
                    n_outlier: int = 0, outlier_scale: float = 1.0,
                    n_pages: int, table: str = "permutation",
                    dirty_tokens: int, top_k: int, layer_mode: int = LAYERS_INDEPENDENT,
                    scores: str = "mass", n_q_heads: int = 0, n_queries: int = 0,
                    device="cpu", payload_device=None, pin_payload: bool = False,
                    keep_kv: bool = False, kv_seed: Optional[int] = None) -> SuffixCheckpoint:
    """Build one seeded session.

    table: "permutation" (first entries of a seeded permutation of all pages), "identity",
    or "free_list" (pages popped from a seeded shuffle in block order - the same thing, named
    for the 2x-oversized-pool configuration).
    scores: "mass" (Zipf block masses), "softmax_attn" or "zipf_attn" (fp16 attention).
    The payload is encoded on `device` and moved to `payload_device` (default: same), optionally
    into pinned host memory.  kv_seed, if given, seeds the K/V values on their own (everything else - tags,
    block table, scores - still follows `seed`).
    """
    g = geom
    gen = torch.Generator(device=device)
    gen.manual_seed(seed)
    nb = -(-n // g.block_tokens)
    L = g.n_layers
    if tags_per_layer:
        tags = _draw_tags(gen, tag_probs, (L, nb), device)
    else:
        tags = _draw_tags(gen, tag_probs, (1, nb), device).expand(L, nb).contiguous()

    # layer payloads, each starting on a 256-byte boundary of one flat buffer
    sizes = []
    for l in range(L):
        sizes.append(sum(record_bytes(int(t), g) * int((tags[l] == t).sum()) for t in range(4)))
    layer_off, total = [], 0
    for s in sizes:
        layer_off.append(total)
        total += -(-s // 256) * 256
    pdev = device if payload_device is None else payload_device
    if pin_payload:
        payload = torch.empty(max(total, 256), dtype=torch.uint8, device="cpu").pin_memory()
    else:
        payload = torch.empty(max(total, 256), dtype=torch.uint8, device=pdev)
    payload.zero_()
    blk_off = torch.empty((L, nb), dtype=torch.int64, device=device)
    raw = []
    gen_kv = gen
    if kv_seed is not None:
        gen_kv = torch.Generator(device=device)
        gen_kv.manual_seed(kv_seed)
    for l in range(L):
        k, v = _kv_layer(gen_kv, g, n, n_outlier, outlier_scale, device)
        pl, off = encode_layer(k, v, tags[l], g)
        assert pl.numel() == sizes[l]
        payload[layer_off[l]:layer_off[l] + sizes[l]].copy_(pl)
        blk_off[l] = off
        if keep_kv:
            raw.append((k.cpu(), v.cpu()))
        del k, v, pl

    n_table = -(-(nb * g.block_tokens + dst_shift) // g.page_tokens)
    assert n_table <= n_pages
    if table == "identity":
        block_table = torch.arange(n_table, dtype=torch.int32, device=device)
    else:
        block_table = torch.randperm(n_pages, generator=gen, device=device)[:n_table].to(torch.int32)

    mass = attn = None
    if scores == "mass":
        mass = zipf_block_mass(gen, L, nb, device)
    elif scores == "softmax_attn":
        attn = softmax_attention(gen, L, n_q_heads, n_queries, n, device)
    elif scores == "zipf_attn":
        attn = zipf_attention(gen, L, n_q_heads, n_queries, n, device)
    else:
        raise ValueError(scores)
    return SuffixCheckpoint(geom=g, n_suffix_tokens=n, delta=delta, dst_shift=dst_shift, tags=tags,
                            blk_off=blk_off, payload=payload, layer_off=layer_off, layer_bytes=sizes,
                            block_table=block_table, n_pages=n_pages, dirty_tokens=dirty_tokens,
                            top_k=top_k, layer_mode=layer_mode, mass=mass, attn=attn, name=name,
                            raw_kv=raw if keep_kv else None)


# --------------------------------------------------------------------------- the five workloads
MIX = (0.30, 0.50, 0.20, 0.0)  # bf16 / int8 / int4 shares of the 8B- and 7B-shaped workloads


def config_tiny(device="cpu", **over) -> SuffixCheckpoint:
    """2 layers, 4 KV heads, head_dim 64, base 1e4, 1024-token suffix in 16-token blocks, delta +137,
    4 of 64 channels x8, tags uniform per (layer, block), 6-block dirty window (90 tokens) + top-2,
    256-page pool with a random-permutation table; scores from fp16 softmax attention [2][8][16][1024]."""
    g = over.pop("geom", Geometry(2, 4, 64, 64, ROPE_HALF, 10000.0, 16, 16, 32))
    kw = dict(name="tiny", seed=1001, geom=g, n=1024, delta=137, tag_probs=(1 / 3, 1 / 3, 1 / 3, 0.0),
              tags_per_layer=True, n_outlier=4, outlier_scale=8.0, n_pages=256, dirty_tokens=90, top_k=2,
              scores="softmax_attn", n_q_heads=8, n_queries=16, device=device)
    kw.update(over)
    return make_checkpoint(**kw)


def config_llama8b(device="cpu", delta: Optional[int] = None, n_layers: int = 32, **over) -> SuffixCheckpoint:
    """32 layers, 8 KV heads, head_dim 128, base 5e5, 16384-token suffix, tags 30/50/20 per block,
    6 of 128 channels x10, repair set 15 % = 90-block dirty window (1440 tokens) + top-64 of Zipf masses,
    1280-page pool, random-permutation table.  delta None = seeded draw uniform in [-2048, 2048]."""
    g = Geometry(n_layers, 8, 128, 128, ROPE_HALF, 500000.0, 16, 16, 32)
    if delta is None:
        delta = int(np.random.default_rng(1002).integers(-2048, 2049))
    kw = dict(name="llama3-8b-shaped", seed=1002, geom=g, n=16384, delta=delta, tag_probs=MIX,
              n_outlier=6, outlier_scale=10.0, n_pages=1280, dirty_tokens=1440, top_k=64, device=device)
    kw.update(over)
    return make_checkpoint(**kw)


def config_7b_host(device="cpu", n_layers: int = 28, **over) -> SuffixCheckpoint:
    """28 layers, 4 KV heads, head_dim 128, base 1e6, 32768-token suffix, delta -3000, same tag mix,
    dirty 2880 tokens (180 blocks) + top-127; 4096-page pool (2x oversized), shuffled free list."""
    g = Geometry(n_layers, 4, 128, 128, ROPE_HALF, 1.0e6, 16, 16, 32)
    kw = dict(name="7b-4kvhead-host", seed=1003, geom=g, n=32768, delta=-3000, tag_probs=MIX,
              n_outlier=6, outlier_scale=10.0, n_pages=4096, table="free_list", dirty_tokens=2880,
              top_k=127, device=device)
    kw.update(over)
    return make_checkpoint(**kw)


def config_select_scale(device="cpu", n_layers: int = 32, n_q_heads: int = 32, n_queries: int = 64,
                        **over) -> SuffixCheckpoint:
    """Selection at scale: Zipf-skewed fp16 attention [32][32][64][16384], 40-block dirty window
    (640 tokens), top-32 per layer; the payload is the 8B-shaped one."""
    g = Geometry(n_layers, 8, 128, 128, ROPE_HALF, 500000.0, 16, 16, 32)
    delta = int(np.random.default_rng(1004).integers(-2048, 2049))
    kw = dict(name="select-at-scale", seed=1004, geom=g, n=16384, delta=delta, tag_probs=MIX,
              n_outlier=6, outlier_scale=10.0, n_pages=1280, dirty_tokens=640, top_k=32,
              scores="zipf_attn", n_q_heads=n_q_heads, n_queries=n_queries, device=device)
    kw.update(over)
    return make_checkpoint(**kw)


STRESS_INT4_SHARE = (0.10, 0.17, 0.24, 0.31, 0.38, 0.45, 0.52, 0.60)


def config_stress_session(i: int, device="cpu", n_layers: int = 80, n: int = 65536, n_pages: int = 4096,
                          **over) -> SuffixCheckpoint:
    """Session i of the 70B-shaped stress workload: 80 layers, 8 KV heads, head_dim 128, base 5e5,
    64k-token suffix, delta seeded in [-8192, 8192], int4 share STRESS_INT4_SHARE[i] with the rest
    split bf16:int8 = 3:5, dirty 5760 tokens + top-254.  The caller assigns pages of the shared pool
    (block_table here is a per-session permutation to be replaced)."""
    g = Geometry(n_layers, 8, 128, 128, ROPE_HALF, 500000.0, 16, 16, 32)
    p4 = STRESS_INT4_SHARE[i % 8]
    probs = ((1 - p4) * 3 / 8, (1 - p4) * 5 / 8, p4, 0.0)
    delta = int(np.random.default_rng(1005 + 17 * i).integers(-8192, 8193))
    kw = dict(name=f"stress-session{i}", seed=1005 + 17 * i, geom=g, n=n, delta=delta, tag_probs=probs,
              n_outlier=6, outlier_scale=10.0, n_pages=n_pages, dirty_tokens=5760, top_k=254, device=device)
    kw.update(over)
    return make_checkpoint(**kw)


STRESS_LAYERS = 80
STRESS_WAVE_LAYERS = 10


def stress_wave(w: int, device="cpu", layers: int = STRESS_WAVE_LAYERS, n: int = 65536, pin_payload: bool = True,
                n_sessions: int = 8, **over) -> List[SuffixCheckpoint]:
    """Layers [w * layers, (w + 1) * layers) of the 70B-shaped stress workload: the 8 sessions with their own
    delta and tag mix, pages drawn from one shared shuffled free list.  The whole workload (80 layers, 172 GB of
    pool, 103 GB of payload) does not fit next to itself, so it is produced and restored one wave of layers at a
    time.  Tags, delta, masses and pages of a session are the same in every wave (they come from the session's
    seed); only the K/V values are re-seeded per wave."""
    nb = -(-n // 16)
    sess = [config_stress_session(i, device=device, n_layers=layers, n=n, n_pages=nb, pin_payload=pin_payload,
                                  kv_seed=1005 + 17 * i + 1000 * w, **over)
            for i in range(n_sessions)]
    shared_free_list(1005, n_sessions * nb, sess)
    return sess


def shared_free_list(seed: int, n_pages: int, sessions: List[SuffixCheckpoint]) -> None:
    """Give every session pages popped from one seeded shuffle of a shared pool, round-robin per block
    so that the sessions' pages interleave.  Rewrites block_table and n_pages in place."""
    rng = np.random.default_rng(seed)
    free = rng.permutation(n_pages).astype(np.int32)
    need = [s.block_table.numel() for s in sessions]
    assert sum(need) <= n_pages
    tables = [np.empty(k, dtype=np.int32) for k in need]
    pos, cur = [0] * len(sessions), 0
    for step in range(max(need)):
        for si in range(len(sessions)):
            if pos[si] < need[si]:
                tables[si][pos[si]] = free[cur]
                pos[si] += 1
                cur += 1
    for s, t in zip(sessions, tables):
        s.block_table = torch.from_numpy(t).to(s.block_table.device)
        s.n_pages = n_pages
