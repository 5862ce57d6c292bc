"""ctypes front end of the CPU oracle (oracle/patchkv_oracle.c).

TEST INFRASTRUCTURE: only tests/, the smoke check and the benchmark's CPU-baseline leg may
import this package.  It never imports the CUDA library or its binding, and shares no code
with them.  Arrays are numpy; a restore call writes into numpy pools passed by the caller.
"""
from __future__ import annotations

import ctypes as C
import os
import subprocess
from typing import Optional, Sequence

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "patchkv_oracle.c")
_SO = os.path.join(_HERE, "libpatchkv_oracle.so")

OK, E_INVALID, E_BOUNDS, E_BADINPUT = 0, -1, -3, -7

_lib = None


def build(force: bool = False) -> str:
    """Compile the oracle with gcc: -O2, no FMA contraction, OpenMP for the timed baseline."""
    if force or not os.path.exists(_SO) or os.path.getmtime(_SO) < os.path.getmtime(_SRC):
        tmp = _SO + f".{os.getpid()}.tmp"
        subprocess.check_call(["gcc", "-O2", "-std=c11", "-ffp-contract=off", "-fopenmp", "-fPIC", "-shared",
                               "-o", tmp, _SRC, "-lm"])
        os.replace(tmp, _SO)
    return _SO


class _RestoreArgs(C.Structure):
    _fields_ = [
        ("L", C.c_int), ("H", C.c_int), ("D", C.c_int), ("Dr", C.c_int), ("rope_style", C.c_int),
        ("B", C.c_int), ("P", C.c_int), ("G", C.c_int),
        ("rope_base", C.c_double), ("inv_freq", C.c_void_p),
        ("k_pool", C.c_void_p), ("v_pool", C.c_void_p),
        ("stride_layer", C.c_int64), ("stride_page", C.c_int64), ("stride_token", C.c_int64), ("stride_head", C.c_int64),
        ("n_pages", C.c_int),
        ("n", C.c_int), ("delta", C.c_int), ("dst_shift", C.c_int),
        ("block_table", C.c_void_p), ("n_table", C.c_int),
        ("tags", C.c_void_p), ("blk_off", C.c_void_p), ("layer_payload", C.c_void_p), ("layer_bytes", C.c_void_p),
        ("reuse_idx", C.c_void_p), ("reuse_cnt", C.c_void_p),
        ("n_threads", C.c_int), ("k_stats", C.c_void_p),
    ]


class _GatherArgs(C.Structure):
    _fields_ = [
        ("L", C.c_int), ("H", C.c_int), ("D", C.c_int), ("B", C.c_int), ("P", C.c_int), ("G", C.c_int),
        ("k_pool", C.c_void_p), ("v_pool", C.c_void_p),
        ("stride_layer", C.c_int64), ("stride_page", C.c_int64), ("stride_token", C.c_int64), ("stride_head", C.c_int64),
        ("n_pages", C.c_int), ("n", C.c_int), ("src_shift", C.c_int),
        ("block_table", C.c_void_p), ("n_table", C.c_int),
        ("tags", C.c_void_p), ("blk_off", C.c_void_p), ("layer_payload", C.c_void_p), ("layer_bytes", C.c_void_p),
    ]


def lib():
    global _lib
    if _lib is None:
        l = C.CDLL(build())
        l.pkvo_fp16_to_f32.restype = C.c_float
        l.pkvo_fp16_to_f32.argtypes = [C.c_uint16]
        l.pkvo_bf16_to_f32.restype = C.c_float
        l.pkvo_bf16_to_f32.argtypes = [C.c_uint16]
        l.pkvo_f32_to_bf16.restype = C.c_uint16
        l.pkvo_f32_to_bf16.argtypes = [C.c_float]
        l.pkvo_f32_to_fp16.restype = C.c_uint16
        l.pkvo_f32_to_fp16.argtypes = [C.c_float]
        l.pkvo_record_bytes.restype = C.c_uint64
        l.pkvo_record_bytes.argtypes = [C.c_int] * 5
        l.pkvo_quantise_group.restype = None
        l.pkvo_quantise_group.argtypes = [C.c_void_p, C.c_int, C.c_int, C.c_void_p, C.c_void_p]
        l.pkvo_dequantise_group.restype = None
        l.pkvo_dequantise_group.argtypes = [C.c_void_p, C.c_int, C.c_uint16, C.c_void_p]
        l.pkvo_rope_table.restype = None
        l.pkvo_rope_table.argtypes = [C.c_int, C.c_double, C.c_void_p, C.c_int, C.c_void_p, C.c_void_p]
        l.pkvo_rotate_pair_f32.restype = None
        l.pkvo_rotate_pair_f32.argtypes = [C.c_float] * 4 + [C.c_void_p, C.c_void_p]
        l.pkvo_rotate_head_f32.restype = None
        l.pkvo_rotate_head_f32.argtypes = [C.c_void_p, C.c_int, C.c_int, C.c_int, C.c_void_p, C.c_void_p, C.c_void_p]
        for f in (l.pkvo_fp16_to_f32_n, l.pkvo_f32_to_bf16_n, l.pkvo_f32_to_fp16_n):
            f.restype = None
            f.argtypes = [C.c_void_p, C.c_int64, C.c_void_p]
        for f in (l.pkvo_block_mass, l.pkvo_block_mass_f64):
            f.restype = C.c_int
            f.argtypes = [C.c_void_p, C.c_int, C.c_int, C.c_int, C.c_int, C.c_int64, C.c_int64, C.c_int64,
                          C.c_int, C.c_void_p]
        l.pkvo_select.restype = C.c_int
        l.pkvo_select.argtypes = [C.c_void_p] + [C.c_int] * 6 + [C.c_void_p] * 5
        l.pkvo_normalise.restype = C.c_int
        l.pkvo_normalise.argtypes = [C.c_void_p, C.c_int, C.c_int, C.c_int, C.c_void_p]
        l.pkvo_restore.restype = C.c_int
        l.pkvo_restore.argtypes = [C.POINTER(_RestoreArgs)]
        l.pkvo_max_threads.restype = C.c_int
        l.pkvo_select_tokens.restype = C.c_int
        l.pkvo_select_tokens.argtypes = [C.c_void_p] + [C.c_int] * 6 + [C.c_void_p] * 6
        l.pkvo_plan_precision.restype = C.c_int
        l.pkvo_plan_precision.argtypes = [C.c_void_p, C.c_void_p, C.c_int, C.c_int, C.c_float, C.c_float, C.c_float,
                                          C.c_float, C.c_void_p, C.c_void_p]
        l.pkvo_plan_checkpoint.restype = C.c_int
        l.pkvo_plan_checkpoint.argtypes = [C.c_void_p] + [C.c_int] * 6 + [C.c_void_p, C.c_void_p]
        l.pkvo_quantize_gather.restype = C.c_int
        l.pkvo_quantize_gather.argtypes = [C.POINTER(_GatherArgs)]
        _lib = l
    return _lib


def _p(a: Optional[np.ndarray]):
    return None if a is None else a.ctypes.data


# ---------------------------------------------------------------- scalar helpers (vectorised by loops)
def fp16_to_f32(h: int) -> float:
    return lib().pkvo_fp16_to_f32(int(h))


def f32_to_bf16(x: float) -> int:
    return lib().pkvo_f32_to_bf16(C.c_float(x))


def f32_to_fp16(x: float) -> int:
    return lib().pkvo_f32_to_fp16(C.c_float(x))


def bf16_to_f32(b: int) -> float:
    return lib().pkvo_bf16_to_f32(int(b))


def record_bytes(tag: int, B: int, H: int, D: int, G: int) -> int:
    return int(lib().pkvo_record_bytes(tag, B, H, D, G))


def quantise_group(x: np.ndarray, qmax: int):
    x = np.ascontiguousarray(x, dtype=np.float32)
    q = np.zeros(x.size, dtype=np.int8)
    s = np.zeros(1, dtype=np.uint16)
    lib().pkvo_quantise_group(_p(x), x.size, qmax, _p(q), _p(s))
    return q, int(s[0])


def dequantise_group(q: np.ndarray, scale_fp16: int) -> np.ndarray:
    q = np.ascontiguousarray(q, dtype=np.int8)
    x = np.zeros(q.size, dtype=np.float32)
    lib().pkvo_dequantise_group(_p(q), q.size, int(scale_fp16), _p(x))
    return x


def rope_table(Dr: int, base: float, delta: int, inv_freq: Optional[np.ndarray] = None):
    c = np.zeros(Dr // 2, dtype=np.float32)
    s = np.zeros(Dr // 2, dtype=np.float32)
    if inv_freq is not None:
        inv_freq = np.ascontiguousarray(inv_freq, dtype=np.float32)
    lib().pkvo_rope_table(Dr, float(base), _p(inv_freq), int(delta), _p(c), _p(s))
    return c, s


def rotate_pair_f32(a: float, b: float, c: float, s: float):
    out = np.zeros(2, dtype=np.float32)
    lib().pkvo_rotate_pair_f32(C.c_float(a), C.c_float(b), C.c_float(c), C.c_float(s),
                               out.ctypes.data, out.ctypes.data + 4)
    return float(out[0]), float(out[1])


def rotate_head_f32(x: np.ndarray, Dr: int, rope_style: int, cos: np.ndarray, sin: np.ndarray) -> np.ndarray:
    """Rotate every row of x [..., D] (fp32) by the table; fp32 result before any bf16 rounding."""
    x = np.ascontiguousarray(x, dtype=np.float32)
    cos = np.ascontiguousarray(cos, dtype=np.float32)
    sin = np.ascontiguousarray(sin, dtype=np.float32)
    out = np.empty_like(x)
    D = x.shape[-1]
    rows_in, rows_out = x.reshape(-1, D), out.reshape(-1, D)
    for i in range(rows_in.shape[0]):
        lib().pkvo_rotate_head_f32(rows_in[i].ctypes.data, D, Dr, rope_style, _p(cos), _p(sin), rows_out[i].ctypes.data)
    return out


def fp16_to_f32_array(h: np.ndarray) -> np.ndarray:
    h = np.ascontiguousarray(h, dtype=np.uint16)
    out = np.empty(h.shape, dtype=np.float32)
    lib().pkvo_fp16_to_f32_n(_p(h), h.size, _p(out))
    return out


def f32_to_bf16_array(x: np.ndarray) -> np.ndarray:
    x = np.ascontiguousarray(x, dtype=np.float32)
    out = np.empty(x.shape, dtype=np.uint16)
    lib().pkvo_f32_to_bf16_n(_p(x), x.size, _p(out))
    return out


def f32_to_fp16_array(x: np.ndarray) -> np.ndarray:
    x = np.ascontiguousarray(x, dtype=np.float32)
    out = np.empty(x.shape, dtype=np.uint16)
    lib().pkvo_f32_to_fp16_n(_p(x), x.size, _p(out))
    return out


# ---------------------------------------------------------------- selection
def block_mass(attn: np.ndarray, B: int, as_double: bool = False):
    """attn: fp16 (or its uint16 bits) [L][Hq][Q][n], last axis contiguous.  Returns (status, mass [L][NB])."""
    a = attn.view(np.uint16) if attn.dtype == np.float16 else attn
    assert a.dtype == np.uint16 and a.ndim == 4 and a.strides[3] == 2
    L, Hq, Q, n = a.shape
    NB = -(-n // B)
    out = np.zeros((L, NB), dtype=np.float64 if as_double else np.uint64)
    f = lib().pkvo_block_mass_f64 if as_double else lib().pkvo_block_mass
    rc = f(_p(a), L, Hq, Q, n, a.strides[0] // 2, a.strides[1] // 2, a.strides[2] // 2, B, _p(out))
    return rc, out


def select(mass: np.ndarray, n: int, B: int, dirty_tokens: int, top_k: int, layer_mode: int = 0):
    """Returns dict(status, mask u8 [L][NB], repair_idx, repair_cnt, reuse_idx, reuse_cnt)."""
    mass = np.ascontiguousarray(mass, dtype=np.uint64)
    L = mass.shape[0]
    NB = -(-n // B)
    assert mass.shape == (L, NB)
    mask = np.zeros((L, NB), dtype=np.uint8)
    ri = np.zeros((L, NB), dtype=np.int32)
    fi = np.zeros((L, NB), dtype=np.int32)
    rc_ = np.zeros(L, dtype=np.int32)
    fc = np.zeros(L, dtype=np.int32)
    rc = lib().pkvo_select(_p(mass), L, n, B, dirty_tokens, top_k, layer_mode, _p(mask), _p(ri), _p(rc_), _p(fi), _p(fc))
    return dict(status=rc, mask=mask, repair_idx=ri, repair_cnt=rc_, reuse_idx=fi, reuse_cnt=fc)


def normalise(mass: np.ndarray, layer_mode: int = 0) -> np.ndarray:
    """Norm of Eq. 10 as the share of the total: mass u64 [L][NB] -> fp32 [L][NB] (independent) or [NB] (shared)."""
    mass = np.ascontiguousarray(mass, dtype=np.uint64)
    L, NB = mass.shape
    out = np.zeros((NB,) if layer_mode == 1 else (L, NB), dtype=np.float32)
    rc = lib().pkvo_normalise(_p(mass), L, NB, layer_mode, _p(out))
    assert rc == OK
    return out


def select_tokens(token_mass: np.ndarray, B: int, dirty_tokens: int, top_tokens: int, layer_mode: int = 1):
    """Token-level selection (the paper's printed form): token_mass u64 [L][n].  Returns dict(status, token_mask
    u8 [L][n], mask u8 [L][NB], repair_idx, repair_cnt, reuse_idx, reuse_cnt)."""
    token_mass = np.ascontiguousarray(token_mass, dtype=np.uint64)
    L, n = token_mass.shape
    NB = -(-n // B)
    tmask = np.zeros((L, n), dtype=np.uint8)
    mask = np.zeros((L, NB), dtype=np.uint8)
    ri = np.zeros((L, NB), dtype=np.int32)
    fi = np.zeros((L, NB), dtype=np.int32)
    rc_ = np.zeros(L, dtype=np.int32)
    fc = np.zeros(L, dtype=np.int32)
    rc = lib().pkvo_select_tokens(_p(token_mass), L, n, B, dirty_tokens, top_tokens, layer_mode, _p(tmask), _p(mask),
                                  _p(ri), _p(rc_), _p(fi), _p(fc))
    return dict(status=rc, token_mask=tmask, mask=mask, repair_idx=ri, repair_cnt=rc_, reuse_idx=fi, reuse_cnt=fc)


# ---------------------------------------------------------------- restore
def restore(*, L, H, D, Dr, rope_style, rope_base, B, P, G, k_pool: np.ndarray, v_pool: np.ndarray,
            strides: Sequence[int], n_pages: int, n: int, delta: int, dst_shift: int,
            block_table: np.ndarray, tags: np.ndarray, blk_off: np.ndarray,
            layer_payload: Sequence[np.ndarray], reuse_idx: np.ndarray, reuse_cnt: np.ndarray,
            inv_freq: Optional[np.ndarray] = None, n_threads: int = 1, want_stats: bool = False,
            layer_bytes: Optional[Sequence[int]] = None):
    """Restore one session into the uint16 (bf16 bit pattern) pools in place.

    layer_payload: one uint8 array per layer.  Returns (status, stats or None) where stats =
    [max abs difference between the fp32 recipe and the pair evaluated in double (after bf16
    rounding), number of K elements whose bf16 differs, number of rotated K elements].
    """
    assert k_pool.dtype == np.uint16 and v_pool.dtype == np.uint16
    NB = -(-n // B)
    tags = np.ascontiguousarray(tags, dtype=np.uint8).reshape(L, NB)
    blk_off = np.ascontiguousarray(blk_off).astype(np.uint64, copy=False).reshape(L, NB)
    reuse_idx = np.ascontiguousarray(reuse_idx, dtype=np.int32).reshape(L, NB)
    reuse_cnt = np.ascontiguousarray(reuse_cnt, dtype=np.int32).reshape(L)
    block_table = np.ascontiguousarray(block_table, dtype=np.int32)
    pays = [np.ascontiguousarray(p, dtype=np.uint8) for p in layer_payload]
    ptrs = (C.c_void_p * L)(*[p.ctypes.data if p.size else None for p in pays])
    lbytes = np.array([p.size for p in pays] if layer_bytes is None else list(layer_bytes), dtype=np.uint64)
    stats = np.zeros(3, dtype=np.float64) if want_stats else None
    if inv_freq is not None:
        inv_freq = np.ascontiguousarray(inv_freq, dtype=np.float32)
    a = _RestoreArgs(L=L, H=H, D=D, Dr=Dr, rope_style=rope_style, B=B, P=P, G=G, rope_base=float(rope_base),
                     inv_freq=_p(inv_freq), k_pool=_p(k_pool), v_pool=_p(v_pool),
                     stride_layer=strides[0], stride_page=strides[1], stride_token=strides[2], stride_head=strides[3],
                     n_pages=n_pages, n=n, delta=delta, dst_shift=dst_shift, block_table=_p(block_table),
                     n_table=block_table.size, tags=_p(tags), blk_off=_p(blk_off),
                     layer_payload=C.cast(ptrs, C.c_void_p), layer_bytes=_p(lbytes),
                     reuse_idx=_p(reuse_idx), reuse_cnt=_p(reuse_cnt), n_threads=n_threads, k_stats=_p(stats))
    rc = lib().pkvo_restore(C.byref(a))
    return rc, stats


def max_threads() -> int:
    return int(lib().pkvo_max_threads())


# ---------------------------------------------------------------- checkpoint writer (offload side)
def plan_checkpoint(tags: np.ndarray, B: int, H: int, D: int, G: int):
    """tags u8 [L][NB] -> (status, blk_off u64 [L][NB], layer_bytes u64 [L]) of the clustered layout."""
    tags = np.ascontiguousarray(tags, dtype=np.uint8)
    L, NB = tags.shape
    off = np.zeros((L, NB), dtype=np.uint64)
    lb = np.zeros(L, dtype=np.uint64)
    rc = lib().pkvo_plan_checkpoint(_p(tags), L, NB, B, H, D, G, _p(off), _p(lb))
    return rc, off, lb


def quantize_gather(*, L, H, D, B, P, G, k_pool: np.ndarray, v_pool: np.ndarray, strides: Sequence[int], n_pages: int,
                    n: int, src_shift: int, block_table: np.ndarray, tags: np.ndarray, blk_off: np.ndarray,
                    layer_payload: Sequence[np.ndarray]):
    """Encode every block of every layer from the uint16 (bf16 bit pattern) pools into the per-layer uint8 buffers
    `layer_payload` in place.  Returns the status."""
    assert k_pool.dtype == np.uint16 and v_pool.dtype == np.uint16
    NB = -(-n // B)
    tags = np.ascontiguousarray(tags, dtype=np.uint8).reshape(L, NB)
    blk_off = np.ascontiguousarray(blk_off).astype(np.uint64, copy=False).reshape(L, NB)
    block_table = np.ascontiguousarray(block_table, dtype=np.int32)
    for p_ in layer_payload:
        assert p_.dtype == np.uint8 and p_.flags["C_CONTIGUOUS"]
    ptrs = (C.c_void_p * L)(*[p_.ctypes.data if p_.size else None for p_ in layer_payload])
    lbytes = np.array([p_.size for p_ in layer_payload], dtype=np.uint64)
    a = _GatherArgs(L=L, H=H, D=D, B=B, P=P, G=G, k_pool=_p(k_pool), v_pool=_p(v_pool),
                    stride_layer=strides[0], stride_page=strides[1], stride_token=strides[2], stride_head=strides[3],
                    n_pages=n_pages, n=n, src_shift=src_shift, block_table=_p(block_table), n_table=block_table.size,
                    tags=_p(tags), blk_off=_p(blk_off), layer_payload=C.cast(ptrs, C.c_void_p), layer_bytes=_p(lbytes))
    return lib().pkvo_quantize_gather(C.byref(a))


def plan_precision(attn: np.ndarray, resid: np.ndarray, B: int, alpha: float, tau_L: float, tau_H: float, eps4: float):
    """Eqs. 13-14: per-token fp32 attention mass and low-bit residual -> (status, tags u8 [NB], risk fp32 [NB])."""
    attn = np.ascontiguousarray(attn, dtype=np.float32)
    resid = np.ascontiguousarray(resid, dtype=np.float32)
    n = attn.size
    NB = -(-n // B)
    tags = np.zeros(NB, dtype=np.uint8)
    risk = np.zeros(NB, dtype=np.float32)
    rc = lib().pkvo_plan_precision(_p(attn), _p(resid), n, B, alpha, tau_L, tau_H, eps4, _p(tags), _p(risk))
    return rc, tags, risk
