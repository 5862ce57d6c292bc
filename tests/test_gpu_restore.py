"""GPU parity of patchkv_restore / patchkv_restore_from_host against the oracle on the same seeded inputs:
V, placement and untouched pages bit-exact; rotated K within 2 bf16 ulp (and expected bit-exact)."""
import numpy as np
import pytest
import torch

import oracle
import patchkv_inputs as pin
from gpu_common import DEV, check_pools, gpu_pool, new_context, run_select_and_restore, staged
from helpers import np_u16, oracle_restore, oracle_select

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module", params=[0, 1], ids=["bulk_copy_pipeline", "direct_loads"])
def ctx(request):
    """Both restore kernels run every case: the shared-memory pipeline (where the geometry allows it) and the
    plain-load kernel (PATCHKV_FLAG_DIRECT_LOADS)."""
    c = new_context(flags=request.param)
    yield c
    c.close()


def test_tiny(ctx):
    run_select_and_restore(ctx, pin.config_tiny())


TINY_VARIANTS = {
    "delta0": dict(delta=0),
    "delta_neg": dict(delta=-137),
    "shift5": dict(dst_shift=5, n_pages=300),
    "P32": dict(geom=pin.Geometry(2, 4, 64, 64, pin.ROPE_HALF, 1e4, 16, 32, 32)),
    "P8_shift3": dict(geom=pin.Geometry(2, 4, 64, 64, pin.ROPE_HALF, 1e4, 16, 8, 32), dst_shift=3),
    "interleaved": dict(geom=pin.Geometry(2, 4, 64, 64, pin.ROPE_INTERLEAVED, 1e4, 16, 16, 32)),
    "partial_rotary_half": dict(geom=pin.Geometry(2, 4, 64, 32, pin.ROPE_HALF, 1e4, 16, 16, 32)),
    "partial_rotary_interleaved": dict(geom=pin.Geometry(2, 4, 64, 40, pin.ROPE_INTERLEAVED, 1e4, 16, 16, 32)),
    "ragged_n1000": dict(n=1000),
    "G64": dict(geom=pin.Geometry(2, 4, 64, 64, pin.ROPE_HALF, 1e4, 16, 16, 64)),
    "G8": dict(geom=pin.Geometry(2, 4, 64, 64, pin.ROPE_HALF, 1e4, 16, 16, 8)),
    "k4v4": dict(tag_probs=(0.25, 0.25, 0.25, 0.25)),
    "one_head_D128": dict(geom=pin.Geometry(3, 1, 128, 128, pin.ROPE_HALF, 5e5, 16, 16, 32)),
    "D72_odd_chunks": dict(geom=pin.Geometry(2, 2, 72, 48, pin.ROPE_HALF, 1e4, 16, 16, 24)),
    "D256": dict(geom=pin.Geometry(1, 2, 256, 256, pin.ROPE_HALF, 1e4, 16, 16, 128)),
    "B32_P16": dict(geom=pin.Geometry(2, 4, 64, 64, pin.ROPE_HALF, 1e4, 32, 16, 32)),
    "all_dirty": dict(dirty_tokens=10 ** 6),
    "nothing_dirty_k0": dict(dirty_tokens=0, top_k=0),
    "shared_layers": dict(layer_mode=pin.LAYERS_SHARED, top_k=4),
    # the geometry of the benchmark's paper-microbenchmark leg: 8 KV heads x 128, 32-token blocks and pages, one scale
    # per 128 channels, a ragged 8031-token suffix, all four formats
    "microbench_geometry": dict(geom=pin.Geometry(2, 8, 128, 128, pin.ROPE_HALF, 1e6, 32, 32, 128), n=8031, n_pages=300,
                                tag_probs=(0.25, 0.25, 0.25, 0.25), dirty_tokens=200, top_k=8),
}


@pytest.mark.parametrize("name", sorted(TINY_VARIANTS))
def test_tiny_variants(ctx, name):
    kw = dict(TINY_VARIANTS[name])
    kw.setdefault("n_pages", 256)
    run_select_and_restore(ctx, pin.config_tiny(**kw))


def test_inv_freq_override(ctx):
    inv = (1e4 ** (-2.0 * np.arange(32) / 64) / 8.0).astype(np.float32)      # a frequency-scaled variant
    run_select_and_restore(ctx, pin.config_tiny(), inv_freq=inv)


def test_empty_suffix_and_no_sessions(ctx):
    ck = pin.config_tiny()
    st = staged(ck)
    k, v, pool = gpu_pool(ck)
    assert ctx.restore(st.geom(), pool, []) == 0
    ctx.select_repair(st.select_args())
    assert ctx.restore(st.geom(), pool, [st.session(n_suffix_tokens=0)]) == 0
    torch.cuda.synchronize()
    assert bool((k == k[0, 0, 0, 0, 0]).all()) and bool((v == v[0, 0, 0, 0, 0]).all())


@pytest.mark.parametrize("what", ["page", "negative_page", "tag", "offset", "reuse_index", "table_short", "misaligned"])
def test_out_of_range_items_are_skipped_and_latched(ctx, what):
    ck = pin.config_tiny(tag_probs=(0.3, 0.4, 0.3, 0.0))
    st = staged(ck)
    _, sel = oracle_select(ck)
    ctx.select_repair(st.select_args())
    torch.cuda.synchronize()
    F0 = [int(x) for x in sel["reuse_idx"][0, :sel["reuse_cnt"][0]]]
    bad_block = F0[3]
    over_o, over_g = {}, {}
    table = ck.block_table.clone()
    tags = ck.tags.clone()
    off = ck.blk_off.clone()
    if what == "page":
        table[bad_block] = ck.n_pages
    elif what == "negative_page":
        table[bad_block] = -1
    elif what == "tag":
        tags[:, bad_block] = 9
    elif what == "offset":
        off[:, bad_block] = max(ck.layer_bytes) - 16
    elif what == "misaligned":
        off[:, bad_block] += 8
    elif what == "reuse_index":
        ridx = sel["reuse_idx"].copy()
        ridx[:, 3] = ck.n_blocks
        st.reuse_idx.copy_(torch.from_numpy(ridx))
        over_o["reuse_idx"] = ridx
    elif what == "table_short":
        bad_block = ck.n_blocks - 1
        table = table[:-1]
    over_o.update(block_table=table.numpy(), tags=tags.numpy(), blk_off=off.numpy())
    k, v, pool = gpu_pool(ck)
    sess = st.session(block_table=table.to(DEV), tags=tags.to(DEV), blk_off=off.to(DEV))
    assert ctx.restore(st.geom(), pool, [sess]) == 0
    torch.cuda.synchronize()
    assert ctx.query_status() == -3
    if what == "misaligned":
        # the oracle has no alignment rule; compare against a run without that block
        ridx = sel["reuse_idx"].copy()
        cnt = sel["reuse_cnt"].copy()
        for l in range(2):
            row = [x for x in ridx[l, :cnt[l]] if x != bad_block]
            ridx[l, :len(row)] = row
            cnt[l] = len(row)
        rc, k_ref, v_ref, _ = oracle_restore(ck, ridx, cnt)
    else:
        ridx = over_o.pop("reuse_idx", sel["reuse_idx"])
        rc, k_ref, v_ref, _ = oracle_restore(ck, ridx, sel["reuse_cnt"], **over_o)
        assert rc == oracle.E_BOUNDS
    check_pools(k, v, k_ref, v_ref, ck.geom)


def test_invalid_arguments_are_rejected_on_the_host(ctx):
    from paper_2609_26219_b200 import binding as pk
    ck = pin.config_tiny()
    st = staged(ck)
    ctx.select_repair(st.select_args())
    k, v, pool = gpu_pool(ck)
    g = st.geom()
    assert ctx.restore(g, pool, [st.session(dst_shift=16)], check=False) == pk.E_INVALID
    assert "dst_shift" in ctx.last_error()
    bad = st.geom(); bad.head_dim = 63
    assert ctx.restore(bad, pool, [st.session()], check=False) == pk.E_INVALID
    bad = st.geom(); bad.group = 5                                         # does not divide head_dim
    assert ctx.restore(bad, pool, [st.session()], check=False) == pk.E_INVALID
    bad = st.geom(); bad.rotary_dim = 23
    assert ctx.restore(bad, pool, [st.session()], check=False) == pk.E_INVALID
    badp = pk.make_pool(k, v, ck.n_pages, (-8, 8, 8, 8))
    assert ctx.restore(g, badp, [st.session()], check=False) == pk.E_INVALID
    assert ctx.restore(g, pool, [st.session()] * 9, check=False) == pk.E_INVALID
    a = st.select_args(); a.top_k = -1
    assert ctx.select_repair(a, check=False) == pk.E_INVALID
    # a pageable payload is not accepted by the host-resident entry point
    hs = st.host_session()
    pageable = torch.zeros(ck.payload.numel(), dtype=torch.uint8)
    ptrs = torch.tensor([pageable.data_ptr() // 256 * 256 + 256 + o for o in ck.layer_off], dtype=torch.int64)
    hs2 = st.host_session(layer_payload=ptrs)
    rc, _ = ctx.restore_from_host(g, pool, [hs2], check=False)
    assert rc == pk.E_INVALID
    torch.cuda.synchronize()
    assert bool((k == k[0, 0, 0, 0, 0]).all())


def test_two_sessions_in_one_call_share_a_pool(ctx):
    a = pin.config_tiny(n_pages=256)
    b = pin.config_tiny(seed=77, delta=-999, n=700, dirty_tokens=40, top_k=5, n_pages=256)
    pin.shared_free_list(5, 256, [a, b])
    sa, sb = staged(a), staged(b)
    ctx.select_repair(sa.select_args())
    ctx.select_repair(sb.select_args())
    k, v, pool = gpu_pool(a)
    ctx.restore(sa.geom(), pool, [sa.session(), sb.session()])
    torch.cuda.synchronize()
    assert ctx.query_status() == 0
    _, sela = oracle_select(a)
    _, selb = oracle_select(b)
    rc, k_ref, v_ref, _ = oracle_restore(a, sela["reuse_idx"], sela["reuse_cnt"])
    rc, k_ref, v_ref, _ = oracle_restore(b, selb["reuse_idx"], selb["reuse_cnt"], pools=(k_ref, v_ref))
    check_pools(k, v, k_ref, v_ref, a.geom)


def test_noncontiguous_pool_strides(ctx):
    """Pool laid out [page][L][slot][H][D+pad]: every stride differs from the benchmark layout."""
    from paper_2609_26219_b200 import binding as pk
    ck = pin.config_tiny()
    g = ck.geom
    st = staged(ck)
    ctx.select_repair(st.select_args())
    Dp = g.head_dim + 8
    shape = (ck.n_pages, g.n_layers, g.page_tokens, g.n_kv_heads, Dp)
    fill = pin.SENTINEL - 0x10000
    k = torch.full(shape, fill, dtype=torch.int16, device=DEV)
    v = torch.full(shape, fill, dtype=torch.int16, device=DEV)
    s_head, s_tok = Dp, g.n_kv_heads * Dp
    s_layer = g.page_tokens * s_tok
    s_page = g.n_layers * s_layer
    pool = pk.make_pool(k, v, ck.n_pages, (s_layer, s_page, s_tok, s_head))
    ctx.restore(st.geom(), pool, [st.session()])
    torch.cuda.synchronize()
    _, sel = oracle_select(ck)
    rc, k_ref, v_ref, _ = oracle_restore(ck, sel["reuse_idx"], sel["reuse_cnt"])
    kk = k.permute(1, 0, 2, 3, 4)
    check_pools(kk[..., :g.head_dim].contiguous(), v.permute(1, 0, 2, 3, 4)[..., :g.head_dim].contiguous(), k_ref, v_ref, g)
    assert bool((k[..., g.head_dim:] == fill).all()) and bool((v[..., g.head_dim:] == fill).all())


def test_tiny_from_pinned_host(ctx):
    run_select_and_restore(ctx, pin.config_tiny(), host=True)


@pytest.mark.parametrize("name", ["delta0", "shift5", "ragged_n1000", "k4v4", "all_dirty", "interleaved"])
def test_tiny_variants_from_pinned_host(ctx, name):
    kw = dict(TINY_VARIANTS[name])
    kw.setdefault("n_pages", 256)
    run_select_and_restore(ctx, pin.config_tiny(**kw), host=True)


@pytest.mark.parametrize("name", ["base", "delta0", "shift5", "ragged_n1000", "k4v4", "all_dirty", "interleaved"])
def test_tiny_variants_from_pinned_host_zero_copy(name):
    """PATCHKV_FLAG_HOST_DIRECT: no staging copies, the restore kernel reads the pinned payload itself."""
    from paper_2609_26219_b200 import binding as pk
    c = new_context(flags=pk.FLAG_HOST_DIRECT)
    try:
        kw = dict(TINY_VARIANTS.get(name, {}))
        kw.setdefault("n_pages", 256)
        st, sel, pools, _ = run_select_and_restore(c, pin.config_tiny(**kw), host=True)
    finally:
        c.close()


def test_stress_shape_zero_copy_and_7b_shape_zero_copy():
    from paper_2609_26219_b200 import binding as pk
    c = new_context(flags=pk.FLAG_HOST_DIRECT)
    try:
        stats = _run_stress(c, _stress_sessions(n_layers=2, n=8192), range(8), [0, 1])
        assert stats.n_copies == 0 and stats.bytes_copied == stats.bytes_useful
        run_select_and_restore(c, pin.config_7b_host(device=DEV, pin_payload=True, n_layers=6), layers=[0, 5], host=True)
    finally:
        c.close()


def test_host_restore_small_ring_and_no_merging():
    c = new_context(staging_slots=1, merge_gap_bytes=0)
    try:
        st, sel, pools, _ = run_select_and_restore(c, pin.config_tiny(), host=True)
        # twice in a row on the same context: the ring and the metadata arena are reused
        run_select_and_restore(c, pin.config_tiny(seed=9), host=True)
    finally:
        c.close()


def test_host_restore_stats_and_two_sessions(ctx):
    a = pin.config_tiny(n_pages=256)
    b = pin.config_tiny(seed=78, delta=-5, n=900, n_pages=256)
    pin.shared_free_list(6, 256, [a, b])
    sa, sb = staged(a, payload_on_host=True), staged(b, payload_on_host=True)
    ctx.select_repair(sa.select_args())
    ctx.select_repair(sb.select_args())
    k, v, pool = gpu_pool(a)
    rc, stats = ctx.restore_from_host(sa.geom(), pool, [sa.host_session(), sb.host_session()])
    torch.cuda.synchronize()
    assert ctx.query_status() == 0
    _, sela = oracle_select(a)
    _, selb = oracle_select(b)
    rc, k_ref, v_ref, _ = oracle_restore(a, sela["reuse_idx"], sela["reuse_cnt"])
    rc, k_ref, v_ref, _ = oracle_restore(b, selb["reuse_idx"], selb["reuse_cnt"], pools=(k_ref, v_ref))
    check_pools(k, v, k_ref, v_ref, a.geom)
    useful = 0
    for ck, sel in ((a, sela), (b, selb)):
        for l in range(2):
            for j in sel["reuse_idx"][l, :sel["reuse_cnt"][l]]:
                useful += pin.record_bytes(int(ck.tags[l, j]), ck.geom)
    assert stats.bytes_useful == useful
    assert stats.bytes_copied >= useful and (stats.n_copies >= 4 or stats.bytes_direct > 0)
    assert stats.n_block_layers == int(sela["reuse_cnt"].sum() + selb["reuse_cnt"].sum())


def test_llama8b_shape_full_size_sampled_layers(ctx):
    """The benchmark configuration (32 layers, 16384-token suffix, device-resident payload): every layer is
    restored on the GPU; sampled layers are compared in full, the rest by their untouched-page invariant."""
    for delta in (-2048, 0, 2048, None):
        ck = pin.config_llama8b(device=DEV, delta=delta)
        st, sel, (k, v), frac = run_select_and_restore(ctx, ck, layers=[0, 17, 31], oracle_threads=0)
        table = ck.block_table.cpu().numpy()
        fill = pin.SENTINEL - 0x10000
        for l in (5, 23):
            R = sel["repair_idx"][l, :sel["repair_cnt"][l]]
            untouched = np.setdiff1d(np.arange(ck.n_pages), table[np.setdiff1d(np.arange(1024), R)])
            idx = torch.from_numpy(untouched).to(DEV)
            assert bool((k[l, idx] == fill).all()) and bool((v[l, idx] == fill).all())
            Fp = torch.from_numpy(table[sel["reuse_idx"][l, :sel["reuse_cnt"][l]]].astype(np.int64)).to(DEV)
            assert not bool((v[l, Fp] == fill).all(dim=(1, 2, 3)).any())
        del st, k, v
        torch.cuda.empty_cache()


def test_7b_shape_from_pinned_host_sampled_layers(ctx):
    ck = pin.config_7b_host(device=DEV, pin_payload=True)
    run_select_and_restore(ctx, ck, layers=[0, 11, 27], host=True)


def _stress_sessions(n_layers, n, n_sessions=8):
    nb = -(-n // 16)
    sess = [pin.config_stress_session(i, device=DEV, n_layers=n_layers, n=n, n_pages=nb, pin_payload=True,
                                      dirty_tokens=min(5760, n // 8), top_k=min(254, nb // 16))
            for i in range(n_sessions)]
    pin.shared_free_list(1005, n_sessions * nb, sess)
    return sess


def _run_stress(ctx, sess, check_sessions, check_layers):
    sts = [staged(c, payload_on_host=True) for c in sess]
    for s in sts:
        ctx.select_repair(s.select_args())
    torch.cuda.synchronize()
    k, v, pool = gpu_pool(sess[0])
    rc, stats = ctx.restore_from_host(sts[0].geom(), pool, [s.host_session() for s in sts])
    torch.cuda.synchronize()
    assert ctx.query_status() == 0
    sels = [oracle_select(c)[1] for c in sess]
    for s, sel in zip(sts, sels):
        assert np.array_equal(s.reuse_idx.cpu().numpy(), sel["reuse_idx"])
    # the oracle restores every session into one shared pool (sampled layers), like the library did
    k_ref = v_ref = None
    for c, sel in zip(sess, sels):
        pools = None if k_ref is None else (k_ref, v_ref)
        rc, k_ref, v_ref, _ = oracle_restore(c, sel["reuse_idx"], sel["reuse_cnt"], layers=check_layers, pools=pools)
        assert rc == oracle.OK
    check_pools(k[check_layers], v[check_layers], k_ref, v_ref, sess[0].geom)
    assert stats.n_block_layers == sum(int(sel["reuse_cnt"].sum()) for sel in sels)
    return stats


def test_stress_shape_eight_sessions_reduced_suffix(ctx):
    """70B-shaped geometry, 8 concurrent sessions with their own delta and tag mix, interleaved pages of one
    shared pool, payloads in pinned host memory; 4096-token suffixes, 3 layers, compared in full."""
    sess = _stress_sessions(n_layers=3, n=4096)
    assert len({c.delta for c in sess}) == 8
    _run_stress(ctx, sess, range(8), [0, 1, 2])


def test_stress_shape_full_suffix_one_layer(ctx):
    """The same at the full 64k-token suffix per session (4096 blocks each, 32768 shared pages), one layer."""
    sess = _stress_sessions(n_layers=1, n=65536)
    _run_stress(ctx, sess, range(8), [0])


def test_select_and_restore_replay_from_a_cuda_graph(ctx):
    """select_repair + restore enqueue only stream work (a counter reset and kernels), so the pair can be captured
    once and replayed; the replayed result equals the eager one bit for bit."""
    ck = pin.config_tiny()
    st = staged(ck)
    k, v, pool = gpu_pool(ck)
    geom, sess, sel_args = st.geom(), st.session(), st.select_args()
    ctx.select_repair(sel_args)
    ctx.restore(geom, pool, [sess])           # eager once: sizes every workspace before the capture
    torch.cuda.synchronize()
    k_eager, v_eager = k.clone(), v.clone()
    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    g = torch.cuda.CUDAGraph()
    with torch.cuda.graph(g, stream=side):
        ctx.select_repair(sel_args, side)
        ctx.restore(geom, pool, [sess], side)
    for _ in range(3):
        k.fill_(pin.SENTINEL - 0x10000)
        v.fill_(pin.SENTINEL - 0x10000)
        st.reuse_cnt.fill_(-7)
        g.replay()
        torch.cuda.synchronize()
        assert torch.equal(k, k_eager) and torch.equal(v, v_eager)
    assert ctx.query_status() == 0


def test_restores_overlapping_on_two_streams_of_one_context(ctx):
    """Launches from one context may overlap on the GPU: each gets its own work counter."""
    a = pin.config_llama8b(device=DEV, n_layers=3, delta=77)
    b = pin.config_llama8b(device=DEV, n_layers=3, delta=-1234, seed=4321)
    sa, sb = staged(a), staged(b)
    ctx.select_repair(sa.select_args())
    ctx.select_repair(sb.select_args())
    ka, va, pa = gpu_pool(a)
    kb, vb, pb = gpu_pool(b)
    torch.cuda.synchronize()
    s1, s2 = torch.cuda.Stream(), torch.cuda.Stream()
    ga, gb = sa.geom(), sb.geom()
    sess_a, sess_b = sa.session(), sb.session()
    for _ in range(4):
        ctx.restore(ga, pa, [sess_a], s1)
        ctx.restore(gb, pb, [sess_b], s2)
    torch.cuda.synchronize()
    assert ctx.query_status() == 0
    for ck, k, v in ((a, ka, va), (b, kb, vb)):
        _, sel = oracle_select(ck)
        rc, k_ref, v_ref, _ = oracle_restore(ck, sel["reuse_idx"], sel["reuse_cnt"])
        check_pools(k, v, k_ref, v_ref, ck.geom)


def test_eight_device_resident_sessions_in_one_launch(ctx):
    sess = [pin.config_stress_session(i, device=DEV, n_layers=2, n=2048, n_pages=128, dirty_tokens=200, top_k=9)
            for i in range(8)]
    pin.shared_free_list(77, 8 * 128, sess)
    sts = [staged(c) for c in sess]
    for s in sts:
        ctx.select_repair(s.select_args())
    k, v, pool = gpu_pool(sess[0])
    ctx.restore(sts[0].geom(), pool, [s.session() for s in sts])
    torch.cuda.synchronize()
    assert ctx.query_status() == 0
    k_ref = v_ref = None
    for c in sess:
        _, sel = oracle_select(c)
        pools = None if k_ref is None else (k_ref, v_ref)
        rc, k_ref, v_ref, _ = oracle_restore(c, sel["reuse_idx"], sel["reuse_cnt"], pools=pools)
    check_pools(k, v, k_ref, v_ref, sess[0].geom)


def test_geometry_limits_block_vectors_and_rotary_dim(ctx):
    """block_tokens * n_kv_heads = 2048 is the largest block the vector kernels take (larger ones go to the element-wise
    kernel, see test_geometries_outside_the_vector_kernels); a rotary dimension beyond 256 is refused."""
    from paper_2609_26219_b200 import binding as pk
    g = pin.Geometry(1, 16, 16, 16, pin.ROPE_HALF, 1e4, 128, 128, 8)       # 128 tokens x 16 heads = 2048 vectors
    ck = pin.make_checkpoint(name="max", seed=3, geom=g, n=300, delta=19, tag_probs=(0.3, 0.3, 0.2, 0.2), tags_per_layer=True,
                             n_pages=8, dirty_tokens=0, top_k=1)
    run_select_and_restore(ctx, ck)
    st = staged(ck)
    k, v, pool = gpu_pool(ck)
    bad = st.geom(); bad.head_dim = 512; bad.rotary_dim = 512
    assert ctx.restore(bad, pool, [st.session()], check=False) == pk.E_UNSUPPORTED


def test_a_bounded_wait_runs_out_and_the_context_keeps_working(ctx):
    """The wait helper of the pipeline kernels, on a barrier that nothing completes and with a short limit: it gives
    up, the kernel latches E_TIMEOUT, the host reads it, and the next restore on the same context is correct."""
    import time
    t0 = time.time()
    ctx.selftest_bounded_wait(2000)
    assert ctx.query_status() == -5
    assert time.time() - t0 < 5.0
    assert ctx.query_status() == 0                       # the latch clears on read
    assert ctx.selftest_bounded_wait(0, check=False) == -1
    run_select_and_restore(ctx, pin.config_tiny(n_pages=256))


def test_restore_pipeline_leaves_cleanly_when_a_wait_runs_out():
    """The path a timeout takes inside the restore pipeline, end to end: one consumer group of every CTA withholds
    an `empty` arrival (a self-test switch armed for one launch), so the warp that feeds the ring gives up after a
    short limit with earlier copies already landed.  The launch must return, latch E_TIMEOUT, write nothing outside
    the reuse set and nothing wrong inside it, and the next launch on the same context must be bit-exact."""
    import time
    c = new_context()
    try:
        ck = pin.config_llama8b(device=DEV, n_layers=2, delta=77)
        st = staged(ck)
        _, sel = oracle_select(ck)
        c.select_repair(st.select_args())
        k, v, pool = gpu_pool(ck)
        geom, sess = st.geom(), st.session()
        torch.cuda.synchronize()
        rc, k_ref, v_ref, _ = oracle_restore(ck, sel["reuse_idx"], sel["reuse_cnt"])
        assert rc == oracle.OK
        t0 = time.time()
        c.selftest_stall_next_launch(2, 4096)
        c.restore(geom, pool, [sess])
        torch.cuda.synchronize()
        assert time.time() - t0 < 20.0
        assert c.query_status() == -5
        # every halfword is either what the full restore writes there or still the sentinel; some blocks are missing
        for got, ref in ((np_u16(k), k_ref), (np_u16(v), v_ref)):
            got = got.reshape(ref.shape)
            assert np.all((got == ref) | (got == pin.SENTINEL))
            assert (got != ref).any() and (got[ref != pin.SENTINEL] != pin.SENTINEL).any()
        # the switch was for one launch: the same context restores everything, bit for bit
        c.restore(geom, pool, [sess])
        torch.cuda.synchronize()
        assert c.query_status() == 0
        check_pools(k, v, k_ref, v_ref, ck.geom)
        assert c.selftest_stall_next_launch(-1, 10, check=False) == -1
        assert c.selftest_stall_next_launch(0, 0, check=False) == -1
    finally:
        c.close()


SMALL_RECORD_GEOMETRIES = {
    "H2_D128_B16": dict(geom=pin.Geometry(4, 2, 128, 128, pin.ROPE_HALF, 1e6, 16, 16, 32), n=16380),
    "H1_D128_B16": dict(geom=pin.Geometry(4, 1, 128, 128, pin.ROPE_HALF, 5e5, 16, 16, 32), n=32768),
    "H4_D64_B8_P16": dict(geom=pin.Geometry(4, 4, 64, 64, pin.ROPE_INTERLEAVED, 1e4, 8, 16, 32), n=16383, dst_shift=3),
    "H2_D64_B32_P16": dict(geom=pin.Geometry(3, 2, 64, 32, pin.ROPE_HALF, 1e4, 32, 16, 16), n=40000, dst_shift=5),
    "H4_D128_B16": dict(geom=pin.Geometry(3, 4, 128, 128, pin.ROPE_HALF, 1e6, 16, 16, 32), n=32768),
}


@pytest.mark.parametrize("name", sorted(SMALL_RECORD_GEOMETRIES))
def test_small_records_share_units(ctx, name):
    """Records far smaller than a stage of the pipeline travel several to a unit (neighbours of a same-tag run, one
    bulk copy, one token table); enough blocks per CTA that rounds hold several blocks, all four tags, a partial last
    block, pages that do not line up with blocks.  Compared in full with the oracle."""
    kw = dict(SMALL_RECORD_GEOMETRIES[name])
    g, n, shift = kw["geom"], kw["n"], kw.get("dst_shift", 0)
    ck = pin.make_checkpoint(name=name, seed=11, geom=g, n=n, delta=-777, dst_shift=shift, tag_probs=(0.3, 0.3, 0.2, 0.2),
                             n_outlier=3, outlier_scale=8.0, n_pages=-(-(n + shift) // g.page_tokens) + 37,
                             dirty_tokens=n // 20, top_k=max(1, n // g.block_tokens // 40), device=DEV)
    run_select_and_restore(ctx, ck)
    run_select_and_restore(ctx, ck, host=True)


@pytest.mark.parametrize("mode", ["hybrid", "staged", "zero_copy"])
def test_host_restore_modes_on_the_8b_shape(mode):
    """The three ways the pinned payload can travel, on six layers of the benchmark's 8B-shaped workload: long runs by the
    copy engine with short runs read by a side launch at the same time (the default), staging copies only, and no
    staging at all.  Same pools bit for bit; the byte counters say which way the records went."""
    from paper_2609_26219_b200 import binding as pk
    flags = {"hybrid": 0, "staged": pk.FLAG_HOST_STAGED, "zero_copy": pk.FLAG_HOST_DIRECT}[mode]
    c = new_context(flags=flags)
    try:
        ck = pin.config_llama8b(device=DEV, n_layers=6, delta=-1500, pin_payload=True)
        st = staged(ck, payload_on_host=True)
        _, sel = oracle_select(ck)
        c.select_repair(st.select_args())
        k, v, pool = gpu_pool(ck)
        for _ in range(2):                                  # twice: the arenas and the ring are reused
            rc, stats = c.restore_from_host(st.geom(), pool, [st.host_session()])
            torch.cuda.synchronize()
            assert c.query_status() == 0
        rc, k_ref, v_ref, _ = oracle_restore(ck, sel["reuse_idx"], sel["reuse_cnt"])
        check_pools(k, v, k_ref, v_ref, ck.geom)
        assert stats.n_block_layers == int(sel["reuse_cnt"].sum())
        if mode == "hybrid":
            assert stats.n_copies > 0 and 0 < stats.bytes_direct < stats.bytes_useful
            assert stats.bytes_copied == stats.bytes_useful          # nothing crosses the link that is not a reused record
        elif mode == "staged":
            assert stats.n_copies > 0 and stats.bytes_direct == 0 and stats.bytes_copied >= stats.bytes_useful
        else:
            assert stats.n_copies == 0 and stats.bytes_direct == stats.bytes_useful == stats.bytes_copied
    finally:
        c.close()


@pytest.mark.parametrize("flags", [0, 4], ids=["hybrid", "staged"])
def test_host_restore_latches_out_of_range_entries(flags):
    ck = pin.config_tiny(tag_probs=(0.3, 0.4, 0.3, 0.0))
    c = new_context(flags=flags)
    try:
        st = staged(ck, payload_on_host=True)
        _, sel = oracle_select(ck)
        c.select_repair(st.select_args())
        torch.cuda.synchronize()
        ridx = sel["reuse_idx"].copy()
        ridx[:, 3] = ck.n_blocks                              # not a block
        off = ck.blk_off.clone()
        bad_block = int(sel["reuse_idx"][0, 5])
        off[:, bad_block] = max(ck.layer_bytes) - 16          # a record that would end past its layer payload
        k, v, pool = gpu_pool(ck)
        hs = st.host_session(reuse_idx=torch.from_numpy(ridx), blk_off=off)
        rc, stats = c.restore_from_host(st.geom(), pool, [hs])
        torch.cuda.synchronize()
        assert c.query_status() == -3
        rc, k_ref, v_ref, _ = oracle_restore(ck, ridx, sel["reuse_cnt"], blk_off=off.numpy())
        assert rc == oracle.E_BOUNDS
        check_pools(k, v, k_ref, v_ref, ck.geom)
    finally:
        c.close()


ODD_GEOMETRIES = {
    "G4": dict(geom=pin.Geometry(2, 4, 64, 64, pin.ROPE_HALF, 1e4, 16, 16, 4)),
    "G2_interleaved": dict(geom=pin.Geometry(2, 2, 32, 32, pin.ROPE_INTERLEAVED, 1e4, 16, 16, 2)),
    "Dr24_half": dict(geom=pin.Geometry(2, 4, 64, 24, pin.ROPE_HALF, 1e4, 16, 16, 32)),
    "Dr6_interleaved": dict(geom=pin.Geometry(2, 3, 48, 6, pin.ROPE_INTERLEAVED, 1e4, 16, 16, 24)),
    "D50_G10_Dr30": dict(geom=pin.Geometry(2, 3, 50, 30, pin.ROPE_HALF, 1e4, 8, 16, 10), n=500, dst_shift=7),
    "D6_G2_B3": dict(geom=pin.Geometry(3, 1, 6, 4, pin.ROPE_HALF, 1e4, 3, 8, 2), n=100, dst_shift=5),
    "sections_not_16B": dict(geom=pin.Geometry(2, 1, 8, 8, pin.ROPE_HALF, 1e4, 3, 4, 8), n=50),
    "B130_H16_over_2048_vectors": dict(geom=pin.Geometry(1, 16, 16, 16, pin.ROPE_HALF, 1e4, 130, 128, 8), n=400, n_pages=8),
}


@pytest.mark.parametrize("name", sorted(ODD_GEOMETRIES))
def test_geometries_outside_the_vector_kernels(ctx, name):
    """Scale groups of 2 or 4 channels, rotary dimensions that are not multiples of 16, head dimensions that are not
    multiples of 8, record sections that are not multiples of 16 bytes, blocks of more than 2048 vectors: everything the
    format allows and the oracle accepts is restored (by the element-wise kernel), device- and host-resident, all tags."""
    kw = dict(ODD_GEOMETRIES[name])
    kw.setdefault("n_pages", 256)
    kw.setdefault("tag_probs", (0.25, 0.25, 0.25, 0.25))
    ck = pin.config_tiny(**{**kw, "n_q_heads": 2, "n_queries": 3})
    run_select_and_restore(ctx, ck)
    run_select_and_restore(ctx, ck, host=True)
    run_select_and_restore(ctx, pin.config_tiny(**{**kw, "n_q_heads": 2, "n_queries": 3, "delta": 0}))
