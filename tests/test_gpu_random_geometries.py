"""Seeded sweep over random geometries, suffix lengths, shifts and position deltas: restore (both kernels, device
and pinned-host payload) and the checkpoint writer (both kernels) against the oracle.  Small sizes; the point is
the combinations (odd head counts, groups of 8 to 128 channels, blocks that straddle pages, partial rotary
dimensions, ragged suffixes), not the volume."""
import numpy as np
import pytest
import torch

import oracle
import patchkv_inputs as pin
from gpu_common import new_context, run_select_and_restore
from test_gpu_writer import gpu_writer
from test_oracle_writer import _ck, pool_from_raw, run_writer

pytestmark = pytest.mark.gpu


def draw(seed: int, pow2_groups: bool = False):
    """One admissible configuration (the library's stated limits: D, G multiples of 8, G | D, rotary dimension a
    multiple of 16 (half) or 8 (interleaved), record sections multiples of 16 bytes, B * H <= 2048)."""
    rng = np.random.default_rng(1000 + seed)
    while True:
        H = int(rng.choice([1, 2, 3, 4, 6, 8]))
        D = int(rng.choice([16, 32, 48, 64, 96, 128]))
        G = int(rng.choice([g for g in ((8, 16, 32, 64, 128) if pow2_groups else (8, 16, 24, 32, 48, 64, 96, 128))
                            if D % g == 0]))
        B = int(rng.choice([8, 16, 24, 32, 48]))
        P = int(rng.choice([8, 16, 32]))
        style = int(rng.choice([pin.ROPE_HALF, pin.ROPE_INTERLEAVED]))
        step = 16 if style == pin.ROPE_HALF else 8
        Dr = int(rng.choice([d for d in range(0, D + 1, step)]))
        if (B * H * D) % 32 or (B * H * (D // G)) % 8:
            continue
        L = int(rng.integers(1, 4))
        n = int(rng.integers(1, 700))
        shift = int(rng.integers(0, P))
        delta = int(rng.choice([0, int(rng.integers(-5000, 5000))]))
        nb = -(-n // B)
        geom = pin.Geometry(L, H, D, Dr, style, float(rng.choice([1e4, 5e5, 1e6])), B, P, G)
        kw = dict(geom=geom, n=n, delta=delta, dst_shift=shift, n_pages=(n + shift) // P + 8,
                  dirty_tokens=int(rng.integers(0, n + 1)) // 3, top_k=int(rng.integers(0, max(1, nb // 3) + 1)),
                  tag_probs=(0.25, 0.25, 0.25, 0.25), seed=77 + seed)
        return kw


@pytest.fixture(scope="module", params=[0, 1], ids=["pipeline", "direct_loads"])
def ctx(request):
    c = new_context(flags=request.param)
    yield c
    c.close()


@pytest.mark.parametrize("seed", range(40))
def test_restore_random_configuration(ctx, seed):
    kw = draw(seed)
    ck = pin.config_tiny(**{**kw, "n_q_heads": 2, "n_queries": 3})
    run_select_and_restore(ctx, ck)
    run_select_and_restore(ctx, ck, host=True)


@pytest.mark.parametrize("seed", range(40))
def test_writer_random_configuration(ctx, seed):
    kw = draw(100 + seed, pow2_groups=True)                # the writer takes groups of 8, 16, 32, 64 or 128 channels
    for drop in ("delta", "dirty_tokens", "top_k", "seed"):
        kw.pop(drop)
    shift = kw.pop("dst_shift")
    ck = _ck(dst_shift=shift, **kw)
    kp, vp = pool_from_raw(ck, shift=shift)
    rc, rc2, off_o, lb_o, bufs_o = run_writer(ck, kp, vp, shift=shift)
    assert rc == oracle.OK and rc2 == oracle.OK
    off, sizes, bufs = gpu_writer(ctx, ck, kp, vp, shift=shift)
    assert ctx.query_status() == 0
    assert np.array_equal(off, off_o) and sizes == [int(x) for x in lb_o]
    for a, b in zip(bufs, bufs_o):
        assert np.array_equal(a, b)
