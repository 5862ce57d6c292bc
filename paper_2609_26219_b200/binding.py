"""ctypes binding of libpatchkv: argument marshalling only, every step of the path runs in the CUDA library.

The functions mirror the C ABI of include/patchkv.h one to one (same names without the prefix).  torch is used
for device memory and streams; no torch type crosses the ABI - only raw pointers, sizes and POD structs.
There is no fallback: if the shared library is missing, importing or calling raises.
"""
from __future__ import annotations

import ctypes as C
import os
from typing import List, Optional, Sequence

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libpatchkv.so")

OK, E_INVALID, E_CUDA, E_BOUNDS, E_NOMEM, E_TIMEOUT, E_UNSUPPORTED, E_BADINPUT = 0, -1, -2, -3, -4, -5, -6, -7
E_TOO_LARGE = -8
STATIC_MAX_MASS_ELEMS = 262144
TAG_BF16, TAG_INT8, TAG_INT4, TAG_K4V4 = 0, 1, 2, 3
ROPE_HALF, ROPE_INTERLEAVED = 0, 1
LAYERS_INDEPENDENT, LAYERS_SHARED = 0, 1
SCORE_ATTN_F16, SCORE_BLOCK_MASS, SCORE_TOKEN_MASS = 0, 1, 2
MAX_SESSIONS = 8
FLAG_DIRECT_LOADS = 1
FLAG_HOST_DIRECT = 2
FLAG_HOST_STAGED = 4


class Config(C.Structure):
    _fields_ = [("struct_size", C.c_uint32), ("device", C.c_int32), ("staging_slots", C.c_int32),
                ("flags", C.c_int32), ("merge_gap_bytes", C.c_uint64)]


class Geom(C.Structure):
    _fields_ = [("struct_size", C.c_uint32), ("n_layers", C.c_int32), ("n_kv_heads", C.c_int32),
                ("head_dim", C.c_int32), ("rotary_dim", C.c_int32), ("rope_style", C.c_int32),
                ("block_tokens", C.c_int32), ("page_tokens", C.c_int32), ("group", C.c_int32),
                ("rope_base", C.c_double), ("inv_freq", C.c_void_p)]


class Pool(C.Structure):
    _fields_ = [("struct_size", C.c_uint32), ("n_pages", C.c_int32), ("k_base", C.c_void_p), ("v_base", C.c_void_p),
                ("stride_layer", C.c_int64), ("stride_page", C.c_int64), ("stride_token", C.c_int64),
                ("stride_head", C.c_int64)]


class Session(C.Structure):
    """Layout shared by patchkv_session (device pointers) and patchkv_session_host (host pointers)."""
    _fields_ = [("struct_size", C.c_uint32), ("n_suffix_tokens", C.c_int32), ("delta", C.c_int32),
                ("dst_shift", C.c_int32), ("n_table", C.c_int32), ("reserved", C.c_int32),
                ("block_table", C.c_void_p), ("tags", C.c_void_p), ("blk_off", C.c_void_p),
                ("layer_payload", C.c_void_p), ("layer_bytes", C.c_void_p),
                ("reuse_idx", C.c_void_p), ("reuse_cnt", C.c_void_p)]


class SelectArgs(C.Structure):
    _fields_ = [("struct_size", C.c_uint32), ("kind", C.c_int32), ("n_layers", C.c_int32), ("n_q_heads", C.c_int32),
                ("n_queries", C.c_int32), ("n_suffix_tokens", C.c_int32), ("block_tokens", C.c_int32),
                ("dirty_tokens", C.c_int32), ("top_k", C.c_int32), ("layer_mode", C.c_int32),
                ("attn", C.c_void_p), ("attn_stride_layer", C.c_int64), ("attn_stride_head", C.c_int64),
                ("attn_stride_query", C.c_int64), ("mass", C.c_void_p), ("mass_out", C.c_void_p),
                ("repair_mask", C.c_void_p), ("repair_idx", C.c_void_p), ("repair_cnt", C.c_void_p),
                ("reuse_idx", C.c_void_p), ("reuse_cnt", C.c_void_p), ("score_out", C.c_void_p),
                ("host_repair_mask", C.c_void_p), ("host_repair_idx", C.c_void_p), ("host_repair_cnt", C.c_void_p),
                ("host_reuse_idx", C.c_void_p), ("host_reuse_cnt", C.c_void_p), ("sync_to_host", C.c_int32),
                ("reserved", C.c_int32)]


class RestoreStats(C.Structure):
    _fields_ = [("struct_size", C.c_uint32), ("n_copies", C.c_uint32), ("bytes_copied", C.c_uint64),
                ("bytes_useful", C.c_uint64), ("n_block_layers", C.c_uint64), ("bytes_direct", C.c_uint64)]


_lib = None


def lib():
    """Load libpatchkv.so (built in-tree by paper_2609_26219_b200.build).  Raises if it is missing."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise RuntimeError(f"{LIB_PATH} is missing: run `python -m paper_2609_26219_b200.build` "
                               "(there is no CPU or PyTorch fallback for the restore path)")
        l = C.CDLL(LIB_PATH)
        l.patchkv_create.argtypes = [C.POINTER(C.c_void_p), C.POINTER(Config)]
        l.patchkv_destroy.argtypes = [C.c_void_p]
        l.patchkv_last_error.argtypes = [C.c_void_p, C.c_char_p, C.c_size_t]
        l.patchkv_select_repair.argtypes = [C.c_void_p, C.POINTER(SelectArgs), C.c_void_p]
        l.patchkv_select_repair_tokens.argtypes = [C.c_void_p, C.POINTER(SelectArgs), C.c_void_p]
        l.patchkv_select_repair_tokens.restype = C.c_int
        l.patchkv_select_repair_static.argtypes = [C.POINTER(SelectArgs), C.c_void_p, C.c_void_p]
        l.patchkv_select_repair_static.restype = C.c_int
        l.patchkv_restore.argtypes = [C.c_void_p, C.POINTER(Geom), C.POINTER(Pool), C.c_void_p, C.c_int, C.c_void_p]
        l.patchkv_restore_from_host.argtypes = [C.c_void_p, C.POINTER(Geom), C.POINTER(Pool), C.c_void_p, C.c_int,
                                                C.c_void_p, C.POINTER(RestoreStats)]
        l.patchkv_plan_checkpoint.argtypes = [C.c_void_p, C.POINTER(Geom), C.c_int, C.c_void_p, C.c_void_p, C.c_void_p,
                                              C.c_void_p]
        l.patchkv_quantize_gather.argtypes = [C.c_void_p, C.POINTER(Geom), C.POINTER(Pool), C.POINTER(Session), C.c_void_p]
        l.patchkv_checkpoint_to_host.argtypes = [C.c_void_p, C.POINTER(Geom), C.POINTER(Pool), C.POINTER(Session),
                                                 C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p]
        l.patchkv_checkpoint_to_host.restype = C.c_int
        l.patchkv_plan_precision.argtypes = [C.c_void_p, C.c_void_p, C.c_void_p, C.c_int, C.c_int, C.c_float, C.c_float,
                                             C.c_float, C.c_float, C.c_void_p, C.c_void_p, C.c_void_p]
        l.patchkv_plan_precision.restype = C.c_int
        l.patchkv_query_status.argtypes = [C.c_void_p, C.POINTER(C.c_int)]
        l.patchkv_selftest_bounded_wait.argtypes = [C.c_void_p, C.c_uint32, C.c_void_p]
        l.patchkv_selftest_stall_next_launch.argtypes = [C.c_void_p, C.c_int32, C.c_uint32]
        l.patchkv_selftest_stall_next_launch.restype = C.c_int
        l.patchkv_record_bytes.argtypes = [C.c_int] * 5
        l.patchkv_record_bytes.restype = C.c_uint64
        for f in (l.patchkv_create, l.patchkv_destroy, l.patchkv_last_error, l.patchkv_select_repair,
                  l.patchkv_restore, l.patchkv_restore_from_host, l.patchkv_query_status,
                  l.patchkv_plan_checkpoint, l.patchkv_quantize_gather):
            f.restype = C.c_int
        _lib = l
    return _lib


class PatchKVError(RuntimeError):
    def __init__(self, code: int, text: str):
        super().__init__(f"patchkv status {code}: {text}")
        self.code = code


def _ptr(t: Optional[torch.Tensor]) -> Optional[int]:
    return None if t is None else t.data_ptr()


def _stream_handle(stream) -> Optional[int]:
    if stream is None:
        stream = torch.cuda.current_stream()
    return stream.cuda_stream if isinstance(stream, torch.cuda.Stream) else int(stream)


def make_geom(n_layers, n_kv_heads, head_dim, rotary_dim, rope_style, rope_base, block_tokens, page_tokens, group,
              inv_freq: Optional[torch.Tensor] = None) -> Geom:
    """inv_freq, if given, is a CPU float32 tensor [rotary_dim / 2] kept alive by the caller."""
    return Geom(C.sizeof(Geom), n_layers, n_kv_heads, head_dim, rotary_dim, rope_style, block_tokens, page_tokens,
                group, float(rope_base), _ptr(inv_freq))


def make_pool(k: torch.Tensor, v: torch.Tensor, n_pages: int, strides: Sequence[int]) -> Pool:
    return Pool(C.sizeof(Pool), n_pages, k.data_ptr(), v.data_ptr(), *[int(s) for s in strides])


def make_session(*, n_suffix_tokens, delta, dst_shift, block_table, tags, blk_off, layer_payload, layer_bytes,
                 reuse_idx, reuse_cnt) -> Session:
    """All tensor arguments on the device (patchkv_restore) or all on the host (patchkv_restore_from_host);
    layer_payload is an int64 tensor of L addresses, layer_bytes an int64 tensor [L]."""
    return Session(C.sizeof(Session), n_suffix_tokens, delta, dst_shift, block_table.numel(), 0,
                   _ptr(block_table), _ptr(tags), _ptr(blk_off), _ptr(layer_payload), _ptr(layer_bytes),
                   _ptr(reuse_idx), _ptr(reuse_cnt))


class Context:
    """Owns one patchkv_ctx.  Methods are the C entry points with the `patchkv_` prefix dropped."""

    def __init__(self, device: int = 0, staging_slots: int = 0, merge_gap_bytes: Optional[int] = None,
                 flags: int = 0):
        self._h = C.c_void_p()
        cfg = Config(C.sizeof(Config), device, staging_slots, flags,
                     0xFFFFFFFFFFFFFFFF if merge_gap_bytes is None else merge_gap_bytes)
        rc = lib().patchkv_create(C.byref(self._h), C.byref(cfg))
        if rc != OK:
            raise PatchKVError(rc, "patchkv_create failed")
        self.device = device

    def close(self):
        if getattr(self, "_h", None) and self._h.value and _lib is not None:
            try:
                _lib.patchkv_destroy(self._h)
            except Exception:       # interpreter shutdown: the process is going away anyway
                pass
            self._h = C.c_void_p()

    __del__ = close

    def last_error(self) -> str:
        buf = C.create_string_buffer(512)
        lib().patchkv_last_error(self._h, buf, 512)
        return buf.value.decode(errors="replace")

    def _check(self, rc: int, check: bool) -> int:
        if check and rc != OK:
            raise PatchKVError(rc, self.last_error())
        return rc

    def select_repair(self, args: SelectArgs, stream=None, check: bool = True) -> int:
        return self._check(lib().patchkv_select_repair(self._h, C.byref(args), _stream_handle(stream)), check)

    def select_repair_tokens(self, args: SelectArgs, stream=None, check: bool = True) -> int:
        return self._check(lib().patchkv_select_repair_tokens(self._h, C.byref(args), _stream_handle(stream)), check)

    def restore(self, geom: Geom, pool: Pool, sessions: List[Session], stream=None, check: bool = True) -> int:
        arr = (Session * max(len(sessions), 1))(*sessions)
        return self._check(lib().patchkv_restore(self._h, C.byref(geom), C.byref(pool), C.cast(arr, C.c_void_p),
                                                 len(sessions), _stream_handle(stream)), check)

    def restore_from_host(self, geom: Geom, pool: Pool, sessions: List[Session], stream=None, check: bool = True):
        arr = (Session * max(len(sessions), 1))(*sessions)
        stats = RestoreStats(C.sizeof(RestoreStats))
        rc = lib().patchkv_restore_from_host(self._h, C.byref(geom), C.byref(pool), C.cast(arr, C.c_void_p),
                                             len(sessions), _stream_handle(stream), C.byref(stats))
        return self._check(rc, check), stats

    def plan_checkpoint(self, geom: Geom, n_suffix_tokens: int, tags: torch.Tensor, blk_off: torch.Tensor,
                        layer_bytes: torch.Tensor, stream=None, check: bool = True) -> int:
        """tags u8 [L][NB] (device) -> blk_off i64 [L][NB], layer_bytes i64 [L] (device) of the clustered layout."""
        return self._check(lib().patchkv_plan_checkpoint(self._h, C.byref(geom), n_suffix_tokens, _ptr(tags),
                                                         _ptr(blk_off), _ptr(layer_bytes), _stream_handle(stream)), check)

    def quantize_gather(self, geom: Geom, pool: Pool, session: Session, stream=None, check: bool = True) -> int:
        return self._check(lib().patchkv_quantize_gather(self._h, C.byref(geom), C.byref(pool), C.byref(session),
                                                         _stream_handle(stream)), check)

    def checkpoint_to_host(self, geom: Geom, pool: Pool, session: Session, host_layer_ptrs: torch.Tensor,
                           host_layer_capacity: torch.Tensor, host_layer_bytes: torch.Tensor, stream=None,
                           check: bool = True) -> int:
        """host_layer_ptrs / host_layer_capacity / host_layer_bytes: CPU int64 tensors [L] (addresses of pinned buffers,
        their sizes, and the output sizes)."""
        return self._check(lib().patchkv_checkpoint_to_host(
            self._h, C.byref(geom), C.byref(pool), C.byref(session), _ptr(host_layer_ptrs), _ptr(host_layer_capacity),
            _ptr(host_layer_bytes), _stream_handle(stream)), check)

    def plan_precision(self, attn: torch.Tensor, resid: torch.Tensor, block_tokens: int, alpha: float, tau_L: float,
                       tau_H: float, eps4: float, tags: torch.Tensor, risk: Optional[torch.Tensor] = None,
                       stream=None, check: bool = True) -> int:
        """Eqs. 13-14: fp32 device tensors attn [n], resid [n] -> tags u8 [NB] (and risk fp32 [NB])."""
        return self._check(lib().patchkv_plan_precision(self._h, _ptr(attn), _ptr(resid), attn.numel(), block_tokens,
                                                        alpha, tau_L, tau_H, eps4, _ptr(tags), _ptr(risk),
                                                        _stream_handle(stream)), check)

    def selftest_bounded_wait(self, max_polls: int, stream=None, check: bool = True) -> int:
        """Runs the kernels' bounded barrier wait on a barrier that nothing completes; query_status() then reports E_TIMEOUT."""
        return self._check(lib().patchkv_selftest_bounded_wait(self._h, max_polls, _stream_handle(stream)), check)

    def selftest_stall_next_launch(self, after_units: int, max_polls: int, check: bool = True) -> int:
        """Arms the next pipeline launch on this context to stall one consumer group after `after_units` units with a
        wait limit of `max_polls` polls; that launch ends early and latches E_TIMEOUT."""
        return self._check(lib().patchkv_selftest_stall_next_launch(self._h, after_units, max_polls), check)

    def query_status(self) -> int:
        v = C.c_int(0)
        rc = lib().patchkv_query_status(self._h, C.byref(v))
        if rc != OK:
            raise PatchKVError(rc, self.last_error())
        return v.value


def select_repair_static(args: SelectArgs, stream=None, device_status: Optional[torch.Tensor] = None) -> int:
    """patchkv_select_repair_static: the selection for callers that cannot allocate device memory (an engine
    that has handed all of HBM to its KV pool, or a resume path that must not stall the device).  No context,
    no allocation; scratch is a fixed 2 MiB array inside the library, shared by all calls on the device, so
    calls must not overlap on the GPU.  Runs on the current device; returns the status code (E_TOO_LARGE when
    the problem does not fit the fixed scratch).  `device_status`: optional zeroed int32 device tensor."""
    return int(lib().patchkv_select_repair_static(C.byref(args), _stream_handle(stream), _ptr(device_status)))


def record_bytes(tag: int, block_tokens: int, n_kv_heads: int, head_dim: int, group: int) -> int:
    return int(lib().patchkv_record_bytes(tag, block_tokens, n_kv_heads, head_dim, group))


def select_args(*, kind, n_layers, n_suffix_tokens, block_tokens, dirty_tokens, top_k, layer_mode, repair_mask,
                repair_idx, repair_cnt, reuse_idx, reuse_cnt, attn: Optional[torch.Tensor] = None,
                mass: Optional[torch.Tensor] = None, mass_out: Optional[torch.Tensor] = None,
                score_out: Optional[torch.Tensor] = None, host_repair_mask: Optional[torch.Tensor] = None,
                host_repair_idx: Optional[torch.Tensor] = None, host_repair_cnt: Optional[torch.Tensor] = None,
                host_reuse_idx: Optional[torch.Tensor] = None, host_reuse_cnt: Optional[torch.Tensor] = None,
                sync_to_host: bool = False) -> SelectArgs:
    """attn: fp16 device tensor [L][Hq][Q][n] with unit stride on the last axis (any other strides);
    score_out: optional fp32 device tensor that receives the normalised importance (Norm of Eq. 10)."""
    a = SelectArgs()
    a.struct_size = C.sizeof(SelectArgs)
    a.kind, a.n_layers, a.n_suffix_tokens, a.block_tokens = kind, n_layers, n_suffix_tokens, block_tokens
    a.dirty_tokens, a.top_k, a.layer_mode = dirty_tokens, top_k, layer_mode
    if attn is not None:
        assert attn.dtype == torch.float16 and attn.dim() == 4 and (attn.shape[3] <= 1 or attn.stride(3) == 1)
        a.n_q_heads, a.n_queries = attn.shape[1], attn.shape[2]
        a.attn = attn.data_ptr()
        a.attn_stride_layer, a.attn_stride_head, a.attn_stride_query = attn.stride(0), attn.stride(1), attn.stride(2)
    a.mass, a.mass_out = _ptr(mass), _ptr(mass_out)
    a.repair_mask, a.repair_idx, a.repair_cnt = _ptr(repair_mask), _ptr(repair_idx), _ptr(repair_cnt)
    a.reuse_idx, a.reuse_cnt = _ptr(reuse_idx), _ptr(reuse_cnt)
    a.score_out = _ptr(score_out)
    for name, t in (("host_repair_mask", host_repair_mask), ("host_repair_idx", host_repair_idx),
                    ("host_repair_cnt", host_repair_cnt), ("host_reuse_idx", host_reuse_idx),
                    ("host_reuse_cnt", host_reuse_cnt)):
        if t is not None:
            assert t.device.type == "cpu" and t.is_pinned() and t.is_contiguous(), f"{name} must be pinned host memory"
        setattr(a, name, _ptr(t))
    a.sync_to_host = 1 if sync_to_host else 0
    return a
