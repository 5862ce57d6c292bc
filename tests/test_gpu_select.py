"""GPU parity of patchkv_select_repair against the oracle: bit-exact masses, masks, lists and counts."""
import numpy as np
import pytest
import torch

import oracle
import patchkv_inputs as pin
from gpu_common import DEV, check_select, new_context, staged
from helpers import oracle_select

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def ctx():
    c = new_context()
    yield c
    c.close()


def _run(ctx, ck, **over):
    st = staged(ck)
    mass, sel = oracle_select(ck)
    ctx.select_repair(st.select_args(**over))
    check_select(st, sel, mass if (ck.attn is not None and over.get("use_mass_out", True)) else None)
    assert ctx.query_status() == 0
    return st, sel


def test_tiny_from_attention(ctx):
    st, sel = _run(ctx, pin.config_tiny())
    assert list(sel["reuse_cnt"]) == [56, 56]


@pytest.mark.parametrize("n,B,d_hat,k", [(1000, 16, 90, 2), (1024, 32, 64, 3), (1024, 8, 0, 5), (1019, 24, 100, 4),
                                         (1024, 16, -5, 0), (1024, 16, 5000, 3), (1024, 16, 90, 1000), (7, 16, 0, 1),
                                         (1024, 20, 33, 6)])
def test_attention_shapes_and_edge_parameters(ctx, n, B, d_hat, k):
    ck = pin.config_tiny(n=n, dirty_tokens=d_hat, top_k=k, n_pages=512)
    # the selection block size is independent of the payload geometry: only select is exercised here
    ck.geom = pin.Geometry(2, 4, 64, 64, pin.ROPE_HALF, 1e4, B, 16, 32)
    st = staged(ck)
    rc, mass = oracle.block_mass(ck.attn.numpy(), B)
    sel = oracle.select(mass, n, B, d_hat, k)
    ctx.select_repair(st.select_args())
    check_select(st, sel, mass)


def test_layers_shared(ctx):
    _run(ctx, pin.config_tiny(layer_mode=pin.LAYERS_SHARED, top_k=5))


def test_strided_and_unaligned_attention_uses_the_general_kernel(ctx):
    ck = pin.config_tiny()
    st = staged(ck)
    big = torch.zeros((2, 8, 16, 1024 + 3), dtype=torch.float16, device=DEV)
    big[..., 3:] = st.attn
    view = big[..., 3:]                  # rows start 6 bytes past a 16-byte boundary
    mass, sel = oracle_select(ck)
    ctx.select_repair(st.select_args(attn=view))
    check_select(st, sel, mass)
    wide = torch.zeros((2, 16, 16, 1024), dtype=torch.float16, device=DEV)
    wide[:, ::2] = st.attn
    ctx.select_repair(st.select_args(attn=wide[:, ::2]))      # strided heads, still 16-byte aligned rows
    check_select(st, sel, mass)


@pytest.mark.parametrize("Q", [5, 24])
def test_values_outside_the_unit_interval_and_bad_entries(ctx, Q):
    """Q = 24 takes the kernel's regular row loop (batches of eight rows inside one head), Q = 5 the general one."""
    rng = np.random.default_rng(3)
    bits = rng.integers(0, 0x7C00, size=(2, 3, Q, 512)).astype(np.uint16)     # whole finite fp16 range
    attn = torch.from_numpy(bits.view(np.float16).copy())
    g = pin.Geometry(2, 4, 64, 64, pin.ROPE_HALF, 1e4, 16, 16, 32)
    ck = pin.config_tiny(n=512, geom=g)
    ck.attn = attn
    _run(ctx, ck)
    bad = bits.copy()
    bad[0, 0, 0, 3] = 0xBC00
    bad[1, 1, 1, 40] = 0x7C00
    bad[1, 2, 4, 41] = 0x7E00
    bad[0, 0, 0, 4] = 0x8000
    ck.attn = torch.from_numpy(bad.view(np.float16).copy())
    st = staged(ck)
    rc, mass = oracle.block_mass(bad, 16)
    assert rc == oracle.E_BADINPUT
    sel = oracle.select(mass, 512, 16, ck.dirty_tokens, ck.top_k)
    ctx.select_repair(st.select_args())
    check_select(st, sel, mass)
    assert ctx.query_status() == -7
    assert ctx.query_status() == 0          # the latch clears on read


def test_ties_constant_mass_and_one_unit_difference(ctx):
    ck = pin.config_llama8b(n_layers=2)
    ck.mass = torch.full_like(ck.mass, 12345)
    ck.mass[1, 700] += 1
    st, sel = _run(ctx, ck)
    assert 700 in sel["repair_idx"][1, :sel["repair_cnt"][1]]


def test_zipf_masses_8b_shape_and_workspace_path(ctx):
    ck = pin.config_llama8b(n_layers=4)
    st, sel = _run(ctx, ck)
    assert list(sel["repair_cnt"]) == [154] * 4 and list(sel["reuse_cnt"]) == [870] * 4
    ck2 = pin.config_tiny()
    _run(ctx, ck2, use_mass_out=False)      # masses kept in the context's workspace


def test_many_blocks_many_ties(ctx):
    g = pin.Geometry(3, 8, 128, 128, pin.ROPE_HALF, 5e5, 16, 16, 32)
    rng = np.random.default_rng(4)
    NB = 5000
    mass = torch.from_numpy(rng.integers(0, 40, size=(3, NB)).astype(np.int64))
    sel = oracle.select(mass.numpy().astype(np.uint64), NB * 16, 16, 333, 777)
    ctxm = ctx
    from paper_2609_26219_b200 import binding as pk
    out = dict(repair_mask=torch.zeros((3, NB), dtype=torch.uint8, device=DEV),
               repair_idx=torch.zeros((3, NB), dtype=torch.int32, device=DEV),
               repair_cnt=torch.zeros(3, dtype=torch.int32, device=DEV),
               reuse_idx=torch.zeros((3, NB), dtype=torch.int32, device=DEV),
               reuse_cnt=torch.zeros(3, dtype=torch.int32, device=DEV))
    md = mass.to(DEV)
    a = pk.select_args(kind=pk.SCORE_BLOCK_MASS, n_layers=3, n_suffix_tokens=NB * 16, block_tokens=16,
                       dirty_tokens=333, top_k=777, layer_mode=0, mass=md, **out)
    ctxm.select_repair(a)
    torch.cuda.synchronize()
    assert np.array_equal(out["repair_idx"].cpu().numpy(), sel["repair_idx"])
    assert np.array_equal(out["reuse_idx"].cpu().numpy(), sel["reuse_idx"])
    assert np.array_equal(out["repair_mask"].cpu().numpy(), sel["mask"])


def test_selection_at_scale_full_size_sampled_layers(ctx):
    """Stored attention [32][32][64][16384] fp16 (2 GiB): masses and lists compared on sampled layers."""
    ck = pin.config_select_scale(device=DEV, n_layers=32)   # payload of 32 layers is built too (1.4 GB)
    st = staged(ck)
    ctx.select_repair(st.select_args())
    torch.cuda.synchronize()
    assert ctx.query_status() == 0
    for l in (0, 13, 31):
        rc, mass = oracle.block_mass(ck.attn[l:l + 1].cpu().numpy(), 16)
        assert rc == oracle.OK
        assert np.array_equal(st.mass_out[l].cpu().numpy().astype(np.uint64), mass[0])
        sel = oracle.select(mass, ck.n_suffix_tokens, 16, ck.dirty_tokens, ck.top_k)
        assert np.array_equal(st.repair_idx[l].cpu().numpy(), sel["repair_idx"][0])
        assert np.array_equal(st.reuse_idx[l].cpu().numpy(), sel["reuse_idx"][0])
        assert int(st.reuse_cnt[l]) == 952 and int(st.repair_cnt[l]) == 72
    # ... followed by the restore of the complement, driven by the lists just produced on the device
    from gpu_common import check_pools, gpu_pool
    from helpers import oracle_restore
    k, v, pool = gpu_pool(ck)
    ctx.restore(st.geom(), pool, [st.session()])
    torch.cuda.synchronize()
    assert ctx.query_status() == 0
    layers = [0, 13, 31]
    ridx, rcnt = st.reuse_idx.cpu().numpy(), st.reuse_cnt.cpu().numpy()
    rc, k_ref, v_ref, _ = oracle_restore(ck, ridx, rcnt, layers=layers)
    assert rc == oracle.OK
    check_pools(k[layers], v[layers], k_ref, v_ref, ck.geom)


@pytest.mark.parametrize("mode", [0, 1])
def test_normalised_score_output_matches_the_oracle_bit_for_bit(ctx, mode):
    """Norm of Eq. 10 (share of the row total): from stored attention and from given masses, per layer and request-level."""
    from paper_2609_26219_b200 import binding as pk
    ck = pin.config_tiny(n=1000, layer_mode=mode, top_k=3)
    rc, mass = oracle.block_mass(ck.attn.numpy(), 16)
    want = oracle.normalise(mass, mode)
    NB, L = mass.shape[1], mass.shape[0]
    sel = oracle.select(mass, 1000, 16, ck.dirty_tokens, 3, mode)
    for kind in ("attn", "mass"):
        out = dict(repair_mask=torch.zeros((L, NB), dtype=torch.uint8, device=DEV),
                   repair_idx=torch.zeros((L, NB), dtype=torch.int32, device=DEV),
                   repair_cnt=torch.zeros(L, dtype=torch.int32, device=DEV),
                   reuse_idx=torch.zeros((L, NB), dtype=torch.int32, device=DEV),
                   reuse_cnt=torch.zeros(L, dtype=torch.int32, device=DEV))
        score = torch.full((L, NB), -1.0, dtype=torch.float32, device=DEV)
        if kind == "attn":
            a = pk.select_args(kind=pk.SCORE_ATTN_F16, n_layers=L, n_suffix_tokens=1000, block_tokens=16,
                               dirty_tokens=ck.dirty_tokens, top_k=3, layer_mode=mode, attn=ck.attn.to(DEV),
                               score_out=score, **out)
        else:
            a = pk.select_args(kind=pk.SCORE_BLOCK_MASS, n_layers=L, n_suffix_tokens=1000, block_tokens=16,
                               dirty_tokens=ck.dirty_tokens, top_k=3, layer_mode=mode,
                               mass=torch.from_numpy(mass.astype(np.int64)).to(DEV), score_out=score, **out)
        ctx.select_repair(a)
        torch.cuda.synchronize()
        got = score.cpu().numpy()
        if mode == 1:
            assert np.array_equal(got[0].view(np.uint32), want.view(np.uint32))
            assert np.all(got[1:] == -1.0)                  # one row only
        else:
            assert np.array_equal(got.view(np.uint32), want.view(np.uint32))
        assert np.array_equal(out["repair_idx"].cpu().numpy(), sel["repair_idx"])
    assert ctx.query_status() == 0
    # an all-zero row gives zeros
    zero = torch.zeros((L, NB), dtype=torch.int64, device=DEV)
    score = torch.full((L, NB), -1.0, dtype=torch.float32, device=DEV)
    a = pk.select_args(kind=pk.SCORE_BLOCK_MASS, n_layers=L, n_suffix_tokens=1000, block_tokens=16, dirty_tokens=0,
                       top_k=3, layer_mode=0, mass=zero, score_out=score, **out)
    ctx.select_repair(a)
    torch.cuda.synchronize()
    assert np.all(score.cpu().numpy() == 0.0)


@pytest.mark.parametrize("sync", [True, False])
def test_host_mirrors_of_the_selection_outputs(ctx, sync):
    ck = pin.config_llama8b(n_layers=3)
    st = staged(ck)
    mass, sel = oracle_select(ck)
    L, NB = 3, ck.n_blocks
    mirrors = dict(host_repair_mask=torch.full((L, NB), 7, dtype=torch.uint8).pin_memory(),
                   host_repair_idx=torch.full((L, NB), -5, dtype=torch.int32).pin_memory(),
                   host_repair_cnt=torch.full((L,), -5, dtype=torch.int32).pin_memory(),
                   host_reuse_idx=torch.full((L, NB), -5, dtype=torch.int32).pin_memory(),
                   host_reuse_cnt=torch.full((L,), -5, dtype=torch.int32).pin_memory())
    ctx.select_repair(st.select_args(sync_to_host=sync, **mirrors))
    if not sync:
        torch.cuda.current_stream().synchronize()
    assert np.array_equal(mirrors["host_repair_mask"].numpy(), sel["mask"])
    assert np.array_equal(mirrors["host_repair_idx"].numpy(), sel["repair_idx"])
    assert np.array_equal(mirrors["host_reuse_idx"].numpy(), sel["reuse_idx"])
    assert np.array_equal(mirrors["host_repair_cnt"].numpy(), sel["repair_cnt"])
    assert np.array_equal(mirrors["host_reuse_cnt"].numpy(), sel["reuse_cnt"])
    check_select(st, sel)
    # a subset of the mirrors, through the token-level entry point
    from paper_2609_26219_b200 import binding as pk
    tm = pin.zipf_block_mass(torch.Generator().manual_seed(3), 2, 512, "cpu")
    want = oracle.select_tokens(tm.numpy().astype(np.uint64), 16, 40, 9, 1)
    out = dict(repair_mask=torch.zeros((2, 32), dtype=torch.uint8, device=DEV),
               repair_idx=torch.zeros((2, 32), dtype=torch.int32, device=DEV),
               repair_cnt=torch.zeros(2, dtype=torch.int32, device=DEV),
               reuse_idx=torch.zeros((2, 32), dtype=torch.int32, device=DEV),
               reuse_cnt=torch.zeros(2, dtype=torch.int32, device=DEV))
    h_idx = torch.full((2, 32), -5, dtype=torch.int32).pin_memory()
    h_cnt = torch.full((2,), -5, dtype=torch.int32).pin_memory()
    a = pk.select_args(kind=pk.SCORE_TOKEN_MASS, n_layers=2, n_suffix_tokens=512, block_tokens=16, dirty_tokens=40,
                       top_k=9, layer_mode=1, mass=tm.to(DEV), host_reuse_idx=h_idx, host_reuse_cnt=h_cnt,
                       sync_to_host=True, **out)
    ctx.select_repair_tokens(a)
    assert np.array_equal(h_idx.numpy(), want["reuse_idx"]) and np.array_equal(h_cnt.numpy(), want["reuse_cnt"])
