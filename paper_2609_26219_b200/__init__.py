"""PatchKV suffix-restore hot path for NVIDIA B200: repair-set selection and fused restore
(dequantise by precision tag, RoPE phase correction of K, page placement) as a C-ABI CUDA library
(libpatchkv.so, sources in csrc/, declarations in include/patchkv.h) plus this thin ctypes binding."""
from .binding import *  # noqa: F401,F403
from .binding import Context, lib, make_geom, make_pool, make_session, select_args, record_bytes  # noqa: F401
