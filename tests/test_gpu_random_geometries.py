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


def draw(seed: int, writer: bool = False):
    """One configuration.  For restore: anything the format allows (even D and Dr, G dividing D) - two draws in three
    stay inside the vector kernels' limits, the third is unconstrained and lands in the element-wise kernel.  For the
    writer (`writer`): its stated limits (D multiple of 8, G in {8, 16, 32, 64, 128}, record sections multiples of 16 bytes)."""
    rng = np.random.default_rng(1000 + seed)
    free = not writer and seed % 3 == 2
    while True:
        H = int(rng.choice([1, 2, 3, 4, 6, 8]))
        if free:
            D = int(rng.choice([6, 10, 16, 24, 36, 40, 64, 100]))
            G = int(rng.choice([g for g in range(1, D + 1) if D % g == 0 and (g <= 4 or g % 2 == 0)]))
            B = int(rng.choice([3, 5, 8, 16, 20]))
        else:
            D = int(rng.choice([16, 32, 48, 64, 96, 128]))
            G = int(rng.choice([g for g in ((8, 16, 32, 64, 128) if writer else (8, 16, 24, 32, 48, 64, 96, 128)) if D % g == 0]))
            B = int(rng.choice([8, 16, 24, 32, 48]))
        P = int(rng.choice([8, 16, 32]))
        style = int(rng.choice([pin.ROPE_HALF, pin.ROPE_INTERLEAVED]))
        step = 2 if free else (16 if style == pin.ROPE_HALF else 8)
        Dr = int(rng.choice([d for d in range(0, D + 1, step)]))
        if not free and ((B * H * D) % 32 or (B * H * (D // G)) % 8):
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


@pytest.mark.parametrize("seed", range(60))
def test_restore_random_configuration(ctx, seed):
    kw = draw(seed)
    ck = pin.config_tiny(**{**kw, "n_q_heads": 2, "n_queries": 3})
    run_select_and_restore(ctx, ck)
    run_select_and_restore(ctx, ck, host=True)


@pytest.mark.parametrize("seed", range(40))
def test_writer_random_configuration(ctx, seed):
    kw = draw(100 + seed, writer=True)                     # the writer takes groups of 8, 16, 32, 64 or 128 channels
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


@pytest.fixture(scope="module")
def sctx():
    c = new_context()
    yield c
    c.close()


@pytest.mark.parametrize("seed", range(40))
def test_selection_random_configuration(sctx, seed):
    """Block form and token form, from masses full of ties and from small attention maps of odd shapes."""
    from gpu_common import DEV
    from paper_2609_26219_b200 import binding as pk
    rng = np.random.default_rng(5000 + seed)
    L = int(rng.integers(1, 5))
    n = int(rng.integers(1, 3000))
    B = int(rng.choice([1, 8, 16, 20, 32, 64]))
    NB = -(-n // B)
    d_hat = int(rng.integers(-5, n + 6))
    mode = int(rng.integers(0, 2))
    from_attn = bool(rng.integers(0, 2))
    if from_attn:
        Hq, Q = int(rng.integers(1, 4)), int(rng.integers(1, 20))
        bits = rng.integers(0, 0x3C01, size=(L, Hq, Q, n)).astype(np.uint16)          # [0, 1]
        bits[rng.random(bits.shape) < 0.7] = 0                                         # many zeros: ties
        attn = torch.from_numpy(bits.view(np.float16).copy()).to(DEV)
        rc, mass = oracle.block_mass(bits, B)
        rc, tmass = oracle.block_mass(bits, 1)
    else:
        tmass = rng.integers(0, 6, size=(L, n)).astype(np.uint64) << np.uint64(int(rng.integers(0, 40)))
        mass = np.zeros((L, NB), dtype=np.uint64)
        for j in range(NB):
            mass[:, j] = tmass[:, j * B:(j + 1) * B].sum(axis=1)

    def outputs():
        return dict(repair_mask=torch.full((L, NB), 9, dtype=torch.uint8, device=DEV),
                    repair_idx=torch.full((L, NB), -7, dtype=torch.int32, device=DEV),
                    repair_cnt=torch.full((L,), -7, dtype=torch.int32, device=DEV),
                    reuse_idx=torch.full((L, NB), -7, dtype=torch.int32, device=DEV),
                    reuse_cnt=torch.full((L,), -7, dtype=torch.int32, device=DEV))

    def check(out, sel):
        torch.cuda.synchronize()
        for name, key in (("repair_mask", "mask"), ("repair_idx", "repair_idx"), ("reuse_idx", "reuse_idx"),
                          ("repair_cnt", "repair_cnt"), ("reuse_cnt", "reuse_cnt")):
            assert np.array_equal(out[name].cpu().numpy(), sel[key]), name

    # block form
    k = int(rng.integers(0, NB + 3))
    out = outputs()
    common = dict(n_layers=L, n_suffix_tokens=n, block_tokens=B, dirty_tokens=d_hat, layer_mode=mode)
    if from_attn:
        a = pk.select_args(kind=pk.SCORE_ATTN_F16, top_k=k, attn=attn, **common, **out)
    else:
        a = pk.select_args(kind=pk.SCORE_BLOCK_MASS, top_k=k, mass=torch.from_numpy(mass.astype(np.int64)).to(DEV),
                           **common, **out)
    sctx.select_repair(a)
    check(out, oracle.select(mass, n, B, d_hat, k, mode))
    # token form
    kappa = int(rng.integers(0, n + 3))
    out = outputs()
    if from_attn:
        a = pk.select_args(kind=pk.SCORE_ATTN_F16, top_k=kappa, attn=attn, **common, **out)
    else:
        a = pk.select_args(kind=pk.SCORE_TOKEN_MASS, top_k=kappa, mass=torch.from_numpy(tmass.astype(np.int64)).to(DEV),
                           **common, **out)
    sctx.select_repair_tokens(a)
    check(out, oracle.select_tokens(tmass, B, d_hat, kappa, mode))
    assert sctx.query_status() == 0


@pytest.mark.parametrize("seed", range(24))
def test_token_selection_random_many_candidates(sctx, seed):
    """Token form with 4096 candidates or more (the ranking whose first cut is a code histogram by several CTAs): suffix
    lengths, block sizes, dirty windows and budgets at random, scores full of ties, spread over many octaves, or both."""
    from gpu_common import DEV
    from paper_2609_26219_b200 import binding as pk
    rng = np.random.default_rng(9000 + seed)
    L = int(rng.integers(1, 4))
    n = int(rng.integers(4200, 30000))
    B = int(rng.choice([1, 8, 16, 20, 32, 64]))
    NB = -(-n // B)
    d_hat = int(rng.integers(0, 100))
    mode = int(rng.integers(0, 2))
    kind = seed % 3
    if kind == 0:                                           # a handful of distinct values
        tmass = rng.integers(0, 6, size=(L, n)).astype(np.uint64) << np.uint64(int(rng.integers(0, 40)))
    elif kind == 1:                                         # twenty octaves, nearly all distinct
        tmass = (2.0 ** rng.uniform(0, 40, size=(L, n))).astype(np.uint64)
    else:                                                   # a crowd of near-equal scores with duplicates under a few large ones
        tmass = ((1 << 28) + (rng.integers(0, 300, size=(L, n)) << 8)).astype(np.uint64)
        tmass[:, rng.permutation(n)[:50]] <<= np.uint64(5)
    kappa = int(rng.choice([1, 17, n // 64, n // 7, n]))
    sel = oracle.select_tokens(np.ascontiguousarray(tmass), B, d_hat, kappa, mode)
    out = dict(repair_mask=torch.full((L, NB), 9, dtype=torch.uint8, device=DEV),
               repair_idx=torch.full((L, NB), -7, dtype=torch.int32, device=DEV),
               repair_cnt=torch.full((L,), -7, dtype=torch.int32, device=DEV),
               reuse_idx=torch.full((L, NB), -7, dtype=torch.int32, device=DEV),
               reuse_cnt=torch.full((L,), -7, dtype=torch.int32, device=DEV))
    a = pk.select_args(kind=pk.SCORE_TOKEN_MASS, n_layers=L, n_suffix_tokens=n, block_tokens=B, dirty_tokens=d_hat,
                       top_k=kappa, layer_mode=mode, mass=torch.from_numpy(tmass.view(np.int64)).to(DEV), **out)
    sctx.select_repair_tokens(a)
    torch.cuda.synchronize()
    for name, key in (("repair_mask", "mask"), ("repair_idx", "repair_idx"), ("reuse_idx", "reuse_idx"),
                      ("repair_cnt", "repair_cnt"), ("reuse_cnt", "reuse_cnt")):
        assert np.array_equal(out[name].cpu().numpy(), sel[key]), name
    assert sctx.query_status() == 0
