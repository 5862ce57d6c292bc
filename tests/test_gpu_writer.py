"""GPU parity of the checkpoint writer (patchkv_plan_checkpoint + patchkv_quantize_gather) against the oracle:
directory and payload bytes identical; and the round trip writer -> restore on the GPU."""
import numpy as np
import pytest
import torch

import oracle
import patchkv_inputs as pin
from gpu_common import DEV, check_pools, gpu_pool, new_context, staged
from helpers import np_u16, oracle_restore, oracle_select
from test_oracle_writer import _ck, pool_from_raw, run_writer, scale_raw

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module", params=[0, 1], ids=["pipeline", "direct_loads"])
def ctx(request):
    """Both writer kernels run every case: the bulk-copy pipeline, and one CTA per block with plain loads."""
    c = new_context(flags=request.param)
    yield c
    c.close()


def gpu_writer(ctx, ck, kp, vp, shift=0, fill=0xEE, table=None, blk_off=None, geom=None, strides=None):
    """Run plan + quantize_gather on the GPU for the pools kp, vp (uint16 numpy).  Returns (off, lb, payload bytes per layer).
    `geom` / `strides` override the checkpoint's geometry and the pool's element strides (a strided view of the pool)."""
    from paper_2609_26219_b200 import binding as pk
    g = ck.geom if geom is None else geom
    L, NB = g.n_layers, ck.n_blocks
    k = torch.from_numpy(kp.view(np.int16)).to(DEV)
    v = torch.from_numpy(vp.view(np.int16)).to(DEV)
    pool = pk.make_pool(k, v, ck.n_pages, pin.pool_strides(g, ck.n_pages) if strides is None else strides)
    geom = pk.make_geom(g.n_layers, g.n_kv_heads, g.head_dim, g.rotary_dim, g.rope_style, g.rope_base, g.block_tokens,
                        g.page_tokens, g.group)
    tags = ck.tags.to(DEV).contiguous()
    off = torch.full((L, NB), -1, dtype=torch.int64, device=DEV)
    lb = torch.zeros(L, dtype=torch.int64, device=DEV)
    ctx.plan_checkpoint(geom, ck.n_suffix_tokens, tags, off, lb)
    torch.cuda.synchronize()
    sizes = [int(x) for x in lb.cpu()]
    if blk_off is not None:
        off = torch.from_numpy(blk_off.astype(np.int64)).to(DEV)
    layer_off, total = [], 0
    for s in sizes:
        layer_off.append(total)
        total += -(-s // 256) * 256
    payload = torch.full((max(total, 256),), fill, dtype=torch.uint8, device=DEV)
    ptrs = torch.tensor([payload.data_ptr() + o for o in layer_off], dtype=torch.int64, device=DEV)
    tb = (ck.block_table if table is None else torch.from_numpy(table)).to(DEV).contiguous()
    sess = pk.make_session(n_suffix_tokens=ck.n_suffix_tokens, delta=0, dst_shift=shift, block_table=tb, tags=tags,
                           blk_off=off, layer_payload=ptrs, layer_bytes=lb, reuse_idx=None, reuse_cnt=None)
    ctx.quantize_gather(geom, pool, sess)
    torch.cuda.synchronize()
    pay = payload.cpu().numpy()
    return off.cpu().numpy().astype(np.uint64), sizes, [pay[o:o + s] for o, s in zip(layer_off, sizes)]


@pytest.mark.parametrize("kw", [dict(), dict(n=150), dict(n=150, dst_shift=5),
                                dict(geom=pin.Geometry(1, 4, 128, 128, pin.ROPE_HALF, 5e5, 16, 16, 128)),
                                dict(geom=pin.Geometry(2, 2, 64, 64, pin.ROPE_HALF, 1e4, 32, 16, 8), n=200, n_pages=40),
                                dict(geom=pin.Geometry(2, 3, 64, 64, pin.ROPE_HALF, 1e4, 16, 8, 64), n=100, n_pages=40),
                                dict(geom=pin.Geometry(2, 4, 64, 64, pin.ROPE_HALF, 1e4, 16, 16, 16), n=150, dst_shift=3),
                                dict(geom=pin.Geometry(2, 2, 128, 128, pin.ROPE_HALF, 1e4, 48, 16, 32), n=500, n_pages=40),
                                dict(geom=pin.Geometry(1, 1, 16, 16, pin.ROPE_HALF, 1e4, 16, 16, 8), n=40, n_pages=8),
                                dict(geom=pin.Geometry(1, 8, 128, 128, pin.ROPE_HALF, 1e6, 32, 32, 128), n=500, n_pages=20),
                                dict(geom=pin.Geometry(1, 2, 256, 256, pin.ROPE_HALF, 1e4, 16, 16, 256), n=100, n_pages=12)])
def test_writer_bytes_match_the_oracle(ctx, kw):
    ck = _ck(**kw)
    shift = ck.dst_shift
    kp, vp = pool_from_raw(ck, shift=shift)
    rc, rc2, off_o, lb_o, bufs_o = run_writer(ck, kp, vp, shift=shift)
    assert rc == oracle.OK and rc2 == oracle.OK
    off, sizes, bufs = gpu_writer(ctx, ck, kp, vp, shift=shift)
    assert ctx.query_status() == 0
    assert np.array_equal(off, off_o) and sizes == [int(x) for x in lb_o]
    for a, b in zip(bufs, bufs_o):
        assert np.array_equal(a, b)


@pytest.mark.parametrize("G", [16, 32])
def test_writer_reads_a_strided_view_of_the_pool(ctx, G):
    """Heads that are not contiguous in the pool: encode the first half of every head vector of a D = 64 pool
    (geometry D = 32, head stride 64), so that every row is gathered head by head."""
    full = pin.Geometry(2, 4, 64, 64, pin.ROPE_HALF, 1e4, 16, 16, 32)
    ck = _ck(geom=full, n=150, dst_shift=5)
    kp, vp = pool_from_raw(ck, shift=5)
    half = pin.Geometry(2, 4, 32, 32, pin.ROPE_HALF, 1e4, 16, 16, G)
    strides = pin.pool_strides(full, ck.n_pages)
    tags = ck.tags.numpy()
    rc, off_o, lb_o = oracle.plan_checkpoint(tags, 16, 4, 32, G)
    bufs_o = [np.full(int(x), 0xEE, dtype=np.uint8) for x in lb_o]
    rc2 = oracle.quantize_gather(L=2, H=4, D=32, B=16, P=16, G=G, k_pool=kp, v_pool=vp, strides=strides,
                                 n_pages=ck.n_pages, n=150, src_shift=5, block_table=ck.block_table.numpy(),
                                 tags=tags, blk_off=off_o, layer_payload=bufs_o)
    assert rc == oracle.OK and rc2 == oracle.OK
    off, sizes, bufs = gpu_writer(ctx, ck, kp, vp, shift=5, geom=half, strides=strides)
    assert ctx.query_status() == 0
    assert np.array_equal(off, off_o) and sizes == [int(x) for x in lb_o]
    for a, b in zip(bufs, bufs_o):
        assert np.array_equal(a, b)


@pytest.mark.parametrize("factor", [3e-5, 1e-6, 2e-8, 1e3])
def test_writer_subnormal_scales_and_large_values(ctx, factor):
    ck = scale_raw(_ck(), factor)
    kp, vp = pool_from_raw(ck)
    rc, rc2, off_o, lb_o, bufs_o = run_writer(ck, kp, vp)
    off, sizes, bufs = gpu_writer(ctx, ck, kp, vp)
    for a, b in zip(bufs, bufs_o):
        assert np.array_equal(a, b)


def test_writer_exact_ties_round_to_even(ctx):
    """Exact half-integer quotients against a non-power-of-two scale (4-bit codes: amax 10.5 gives s = 1.5 exactly):
    0.75 -> 0.5 -> 0, 2.25 -> 1.5 -> 2, -3.75 -> -2.5 -> -2, 5.25 -> 3.5 -> 4, 9.75 -> 6.5 -> 6."""
    g = pin.Geometry(1, 1, 64, 64, pin.ROPE_HALF, 1e4, 16, 16, 32)
    ck = _ck(geom=g, n=16, n_pages=2, table="identity", tag_probs=(0, 0, 0, 1.0))
    kp = np.zeros((1, 2, 16, 1, 64), dtype=np.uint16)
    vp = np.zeros_like(kp)
    vals = [10.5, 0.75, 2.25, -3.75, 5.25, -0.75, 1.5, 9.75]
    for c, x in enumerate(vals):
        bits = int(np.array([x], dtype=np.float32).view(np.uint32)[0])
        assert bits & 0xFFFF == 0                      # representable in bf16
        kp[0, 0, 2, 0, c] = bits >> 16
    rc, rc2, off_o, lb_o, bufs_o = run_writer(ck, kp, vp)
    rec = bufs_o[0]
    assert rec[512:512 + 64].view(np.float16).reshape(16, 2)[2, 0] == np.float16(1.5)
    by = rec[:512].reshape(16, 32)[2, :4]
    nib = []
    for b in by:
        nib += [int(b) & 15, int(b) >> 4]
    codes = [n - 16 if n >= 8 else n for n in nib]
    assert codes == [7, 0, 2, -2, 4, 0, 1, 6]
    off, sizes, bufs = gpu_writer(ctx, ck, kp, vp)
    assert np.array_equal(bufs[0], bufs_o[0])


def test_writer_every_bf16_maximum_and_many_ties(ctx):
    """Every finite positive bf16 value as the maximum of a scale group (so every scale the encoder can produce from
    one, subnormal and infinite fp16 scales included), in 8-bit and in 4-bit codes; the other channels of the group are
    fractions of the maximum with few significant bits (odd multiples of max/14, max/254, max/8 ... rounded to bf16,
    which land on exact half-integer quotients whenever the scale has few bits) and random values below it."""
    rng = np.random.default_rng(77)
    amax_bits = np.arange(1, 0x7F80, dtype=np.uint32)                       # 32 639 values
    n_groups = 32768
    amax = np.zeros(n_groups, dtype=np.float32)
    amax[:amax_bits.size] = (amax_bits << 16).view(np.float32)
    amax[amax_bits.size:] = 1.5
    x = np.zeros((n_groups, 32), dtype=np.float64)
    x[:, 0] = amax
    odd = rng.integers(0, 64, size=(n_groups, 15)) * 2 + 1
    den = rng.choice([14.0, 254.0, 8.0, 16.0, 28.0, 508.0], size=(n_groups, 15))
    x[:, 1:16] = amax[:, None].astype(np.float64) * np.minimum(odd / den, 1.0) * rng.choice([-1.0, 1.0], size=(n_groups, 15))
    x[:, 16:] = amax[:, None].astype(np.float64) * rng.uniform(-1.0, 1.0, size=(n_groups, 16))
    with np.errstate(over="ignore", invalid="ignore"):
        xf = x.astype(np.float32)
    bits = xf.view(np.uint32)
    bf = ((bits + 0x7FFF + ((bits >> 16) & 1)) >> 16).astype(np.uint16)    # round to nearest even bf16
    bf[:, 0] = (amax.view(np.uint32) >> 16).astype(np.uint16)
    mag = bf & 0x7FFF
    over = mag > mag[:, :1]                                                 # rounding must not exceed the maximum
    bf = np.where(over, (bf & 0x8000) | mag[:, :1], bf).astype(np.uint16)
    # layout: 1 head of 128 channels (4 groups per token), 16-token blocks: 64 groups per block, 512 blocks
    g = pin.Geometry(2, 1, 128, 128, pin.ROPE_HALF, 1e4, 16, 16, 32)
    n = n_groups // 4
    ck = _ck(geom=g, n=n, n_pages=n // 16, table="identity", tag_probs=(0, 1.0, 0, 0))
    ck.tags[1, :] = pin.TAG_K4V4
    kp = np.zeros((2, n // 16, 16, 1, 128), dtype=np.uint16)
    kp[0] = bf.reshape(n // 16, 16, 1, 128)
    kp[1] = kp[0]
    vp = kp[:, ::-1].copy()
    rc, rc2, off_o, lb_o, bufs_o = run_writer(ck, kp, vp)
    assert rc == oracle.OK and rc2 == oracle.OK
    off, sizes, bufs = gpu_writer(ctx, ck, kp, vp)
    assert ctx.query_status() == 0
    for a, b in zip(bufs, bufs_o):
        assert np.array_equal(a, b)


def test_plan_and_writer_replay_from_a_cuda_graph(ctx):
    """plan_checkpoint + quantize_gather enqueue kernels only (the encoder's work counters live in a slot of their own
    for a captured launch and are left zeroed), so the pair can be captured once and replayed: same bytes as the oracle
    on every replay."""
    from paper_2609_26219_b200 import binding as pk
    ck = _ck(n=150, dst_shift=5)
    kp, vp = pool_from_raw(ck, shift=5)
    rc, rc2, off_o, lb_o, bufs_o = run_writer(ck, kp, vp, shift=5)
    g = ck.geom
    L, NB = g.n_layers, ck.n_blocks
    k = torch.from_numpy(kp.view(np.int16)).to(DEV)
    v = torch.from_numpy(vp.view(np.int16)).to(DEV)
    pool = pk.make_pool(k, v, ck.n_pages, pin.pool_strides(g, ck.n_pages))
    geom = pk.make_geom(g.n_layers, g.n_kv_heads, g.head_dim, g.rotary_dim, g.rope_style, g.rope_base, g.block_tokens,
                        g.page_tokens, g.group)
    tags = ck.tags.to(DEV).contiguous()
    off = torch.zeros((L, NB), dtype=torch.int64, device=DEV)
    lb = torch.zeros(L, dtype=torch.int64, device=DEV)
    sizes = [int(x) for x in lb_o]
    starts = [sum(-(-s // 256) * 256 for s in sizes[:i]) for i in range(L)]
    payload = torch.zeros(starts[-1] + sizes[-1] + 256, dtype=torch.uint8, device=DEV)
    ptrs = torch.tensor([payload.data_ptr() + o for o in starts], dtype=torch.int64, device=DEV)
    table = ck.block_table.to(DEV).contiguous()           # (the session holds raw pointers: keep the tensors alive)
    sess = pk.make_session(n_suffix_tokens=ck.n_suffix_tokens, delta=0, dst_shift=5, block_table=table,
                           tags=tags, blk_off=off, layer_payload=ptrs, layer_bytes=lb, reuse_idx=None, reuse_cnt=None)
    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph, stream=side):
        ctx.plan_checkpoint(geom, ck.n_suffix_tokens, tags, off, lb, side)
        ctx.quantize_gather(geom, pool, sess, side)
    for _ in range(3):
        payload.fill_(0xEE)
        off.fill_(-1)
        graph.replay()
        torch.cuda.synchronize()
        pay = payload.cpu().numpy()
        assert np.array_equal(off.cpu().numpy().astype(np.uint64), off_o)
        for o, s_, b_ in zip(starts, sizes, bufs_o):
            assert np.array_equal(pay[o:o + s_], b_)
    assert ctx.query_status() == 0


def test_two_writers_on_two_streams_of_one_context(ctx):
    """Two checkpoints encoded at the same time on two streams of one context (each stream has its own work counters):
    both match the oracle, over several rounds without a synchronisation in between."""
    from paper_2609_26219_b200 import binding as pk
    jobs = []
    for seed, n in ((31, 640), (32, 1000)):
        g = pin.Geometry(3, 4, 64, 64, pin.ROPE_HALF, 1e4, 16, 16, 32)
        ck = _ck(geom=g, n=n, n_pages=n // 16 + 8, seed=seed)
        kp, vp = pool_from_raw(ck)
        rc, rc2, off_o, lb_o, bufs_o = run_writer(ck, kp, vp)
        L, NB = g.n_layers, ck.n_blocks
        k = torch.from_numpy(kp.view(np.int16)).to(DEV)
        v = torch.from_numpy(vp.view(np.int16)).to(DEV)
        pool = pk.make_pool(k, v, ck.n_pages, pin.pool_strides(g, ck.n_pages))
        geom = pk.make_geom(g.n_layers, g.n_kv_heads, g.head_dim, g.rotary_dim, g.rope_style, g.rope_base, g.block_tokens,
                            g.page_tokens, g.group)
        tags = ck.tags.to(DEV).contiguous()
        off = torch.from_numpy(off_o.astype(np.int64)).to(DEV)
        lb = torch.from_numpy(np.asarray(lb_o).astype(np.int64)).to(DEV)
        sizes = [int(x) for x in lb_o]
        starts = [sum(-(-s // 256) * 256 for s in sizes[:i]) for i in range(L)]
        payload = torch.zeros(starts[-1] + sizes[-1] + 256, dtype=torch.uint8, device=DEV)
        ptrs = torch.tensor([payload.data_ptr() + o for o in starts], dtype=torch.int64, device=DEV)
        table = ck.block_table.to(DEV).contiguous()
        sess = pk.make_session(n_suffix_tokens=ck.n_suffix_tokens, delta=0, dst_shift=0, block_table=table,
                               tags=tags, blk_off=off, layer_payload=ptrs, layer_bytes=lb, reuse_idx=None, reuse_cnt=None)
        jobs.append(dict(geom=geom, pool=pool, sess=sess, payload=payload, starts=starts, sizes=sizes, want=bufs_o,
                         stream=torch.cuda.Stream(), keep=(k, v, tags, off, lb, ptrs, table)))   # the session holds raw pointers
    torch.cuda.synchronize()
    for _ in range(6):
        for j in jobs:
            with torch.cuda.stream(j["stream"]):
                j["payload"].fill_(0xEE)
            ctx.quantize_gather(j["geom"], j["pool"], j["sess"], j["stream"])
    torch.cuda.synchronize()
    for j in jobs:
        pay = j["payload"].cpu().numpy()
        for o, s_, b_ in zip(j["starts"], j["sizes"], j["want"]):
            assert np.array_equal(pay[o:o + s_], b_)
    assert ctx.query_status() == 0


@pytest.mark.parametrize("what", ["page", "offset", "table_short"])
def test_writer_skips_out_of_range_blocks(ctx, what):
    ck = _ck()
    kp, vp = pool_from_raw(ck)
    _, _, off_o, lb_o, _ = run_writer(ck, kp, vp)
    table = ck.block_table.numpy().copy()
    off2 = off_o.copy()
    if what == "page":
        table[4] = ck.n_pages + 3
    elif what == "offset":
        off2[:, 4] = max(int(x) for x in lb_o)
    else:
        table = table[:-1]
    rc, rc2, _, _, bufs_o = run_writer(ck, kp, vp, table=table, blk_off=off2)
    assert rc2 == oracle.E_BOUNDS
    off, sizes, bufs = gpu_writer(ctx, ck, kp, vp, table=table, blk_off=off2)
    assert ctx.query_status() == -3
    for a, b in zip(bufs, bufs_o):
        assert np.array_equal(a, b)


def test_unknown_tag_in_plan_and_unsupported_group(ctx):
    from paper_2609_26219_b200 import binding as pk
    ck = _ck()
    ck.tags[0, 3] = 9
    kp, vp = pool_from_raw(ck)
    off, sizes, bufs = gpu_writer(ctx, ck, kp, vp)
    assert ctx.query_status() == -3
    assert off[0, 3] == np.uint64(2 ** 64 - 1)
    g24 = pin.Geometry(1, 2, 72, 48, pin.ROPE_HALF, 1e4, 16, 16, 24)
    ck2 = pin.config_tiny(geom=g24)
    st = staged(ck2)
    k, v, pool = gpu_pool(ck2)
    assert ctx.quantize_gather(st.geom(), pool, st.session(), check=False) == pk.E_UNSUPPORTED


def test_full_size_8b_shape_writer_then_restore_round_trip(ctx):
    """32-layer 8B-shaped pool -> checkpoint written on the GPU -> restored on the GPU with delta = 0 into a second
    pool: bf16-tag blocks come back bit-identical, quantised blocks within half a quantisation step; sampled
    layers of the written payload are compared byte for byte with the oracle's writer."""
    from paper_2609_26219_b200 import binding as pk
    ck = pin.config_llama8b(device=DEV, delta=0, dirty_tokens=0, top_k=0)
    g = ck.geom
    st = staged(ck)
    ctx.select_repair(st.select_args())
    k, v, pool = gpu_pool(ck)
    ctx.restore(st.geom(), pool, [st.session()])          # pool <- the synthetic checkpoint (all 1024 blocks)
    torch.cuda.synchronize()
    # write a second checkpoint from that pool with the same tags
    L, NB = g.n_layers, ck.n_blocks
    off = torch.zeros((L, NB), dtype=torch.int64, device=DEV)
    lb = torch.zeros(L, dtype=torch.int64, device=DEV)
    ctx.plan_checkpoint(st.geom(), ck.n_suffix_tokens, st.tags, off, lb)
    torch.cuda.synchronize()
    assert torch.equal(off, st.blk_off) and [int(x) for x in lb.cpu()] == ck.layer_bytes
    payload2 = torch.zeros_like(st.payload)
    ptrs2 = torch.tensor([payload2.data_ptr() + o for o in ck.layer_off], dtype=torch.int64, device=DEV)
    sess_w = st.session(layer_payload=ptrs2, blk_off=off, layer_bytes=lb)
    ctx.quantize_gather(st.geom(), pool, sess_w)
    torch.cuda.synchronize()
    assert ctx.query_status() == 0
    # sampled layers against the oracle's writer
    table = ck.block_table.cpu().numpy()
    tags_np = ck.tags.cpu().numpy()
    for l in (0, 19):
        sub = pin.Geometry(1, g.n_kv_heads, g.head_dim, g.rotary_dim, g.rope_style, g.rope_base, 16, 16, g.group)
        kp, vp = np_u16(k[l:l + 1]), np_u16(v[l:l + 1])
        buf = [np.zeros(ck.layer_bytes[l], dtype=np.uint8)]
        rc = oracle.quantize_gather(L=1, H=g.n_kv_heads, D=g.head_dim, B=16, P=16, G=g.group, k_pool=kp, v_pool=vp,
                                    strides=pin.pool_strides(sub, ck.n_pages), n_pages=ck.n_pages, n=ck.n_suffix_tokens,
                                    src_shift=0, block_table=table, tags=tags_np[l:l + 1],
                                    blk_off=off[l:l + 1].cpu().numpy(), layer_payload=buf)
        assert rc == oracle.OK
        got = payload2[ck.layer_off[l]:ck.layer_off[l] + ck.layer_bytes[l]].cpu().numpy()
        assert np.array_equal(got, buf[0])
    # restore the second checkpoint into a fresh pool and compare with the first pool
    k2, v2, pool2 = gpu_pool(ck)
    ctx.restore(st.geom(), pool2, [sess_w])
    torch.cuda.synchronize()
    bf = torch.from_numpy(np.isin(tags_np[0], [0])).to(DEV)
    pages_bf = st.block_table[:NB][bf].long()
    assert torch.equal(k2[:, pages_bf], k[:, pages_bf]) and torch.equal(v2[:, pages_bf], v[:, pages_bf])
    a = k.view(torch.bfloat16).float()
    b = k2.view(torch.bfloat16).float()
    amax = a.abs().reshape(*a.shape[:-1], -1, g.group).amax(dim=-1, keepdim=True)
    step = (amax / 127.0).expand(*amax.shape[:-1], g.group).reshape(a.shape)
    used = torch.zeros(ck.n_pages, dtype=torch.bool, device=DEV)
    used[st.block_table[:NB].long()] = True
    err = (a - b).abs()[:, used]
    bound = (0.5 * step * 1.01 + a.abs() * 2.0 ** -8 + amax.expand(*amax.shape[:-1], g.group).reshape(a.shape) * 2.0 ** -10)[:, used]
    assert bool((err <= bound).all())


@pytest.mark.parametrize("n,B", [(65536, 32), (1000, 16), (7, 16)])
def test_precision_planner_matches_the_oracle_bit_for_bit(ctx, n, B):
    rng = np.random.default_rng(n)
    attn = (rng.random(n) ** 4 / n * 8).astype(np.float32)
    resid = (rng.random(n) * 0.3).astype(np.float32)
    NB = -(-n // B)
    for alpha in (0.5, 0.0, 1.0):
        # thresholds at quantiles of the risk so that every tier occurs (the real ones come from calibration)
        _, _, r0 = oracle.plan_precision(attn, resid, B, alpha, 0.0, 1.0, 1.0)
        tl, th = (float(np.quantile(r0, 0.4)), float(np.quantile(r0, 0.8))) if NB > 4 else (1e-4, 1e-3)
        e4 = float(np.median(resid.reshape(-1)[:NB * B - (NB * B - n)].max())) * 0.97
        rc, tags_o, risk_o = oracle.plan_precision(attn, resid, B, alpha, tl, th, e4)
        assert rc == oracle.OK
        tags = torch.full((NB,), 9, dtype=torch.uint8, device=DEV)
        risk = torch.zeros(NB, dtype=torch.float32, device=DEV)
        ctx.plan_precision(torch.from_numpy(attn).to(DEV), torch.from_numpy(resid).to(DEV), B, alpha, tl, th, e4, tags, risk)
        torch.cuda.synchronize()
        assert np.array_equal(risk.cpu().numpy().view(np.uint32), risk_o.view(np.uint32))
        assert np.array_equal(tags.cpu().numpy(), tags_o)
        if n > 1000:
            assert len(set(tags_o)) == 3         # all three tiers occur


@pytest.mark.parametrize("slots", [1, 2, 4])
def test_checkpoint_to_host_streams_the_same_bytes(slots):
    """Plan + encode + device-to-host copy per layer through the staging ring: the pinned buffers end up holding
    exactly the oracle's payload, for ring depths below, at and above what overlaps."""
    from paper_2609_26219_b200 import binding as pk
    c = new_context(staging_slots=slots)
    try:
        g = pin.Geometry(5, 2, 64, 64, pin.ROPE_HALF, 1e4, 16, 16, 32)
        ck = _ck(geom=g, n=150, n_pages=24)
        kp, vp = pool_from_raw(ck)
        rc, rc2, off_o, lb_o, bufs_o = run_writer(ck, kp, vp)
        L, NB = g.n_layers, ck.n_blocks
        k = torch.from_numpy(kp.view(np.int16)).to(DEV)
        v = torch.from_numpy(vp.view(np.int16)).to(DEV)
        pool = pk.make_pool(k, v, ck.n_pages, pin.pool_strides(g, ck.n_pages))
        geom = pk.make_geom(g.n_layers, g.n_kv_heads, g.head_dim, g.rotary_dim, g.rope_style, g.rope_base,
                            g.block_tokens, g.page_tokens, g.group)
        tags = ck.tags.to(DEV).contiguous()
        off = torch.zeros((L, NB), dtype=torch.int64, device=DEV)
        lb = torch.zeros(L, dtype=torch.int64, device=DEV)
        sess = pk.make_session(n_suffix_tokens=ck.n_suffix_tokens, delta=0, dst_shift=0,
                               block_table=ck.block_table.to(DEV), tags=tags, blk_off=off, layer_payload=None,
                               layer_bytes=lb, reuse_idx=None, reuse_cnt=None)
        cap = NB * 16 * 2 * 64 * 4
        host = [torch.full((cap,), 0x55, dtype=torch.uint8).pin_memory() for _ in range(L)]
        ptrs = torch.tensor([h.data_ptr() for h in host], dtype=torch.int64)
        caps = torch.full((L,), cap, dtype=torch.int64)
        sizes = torch.zeros(L, dtype=torch.int64)
        for _ in range(2):                                   # twice: ring and events are reused
            c.checkpoint_to_host(geom, pool, sess, ptrs, caps, sizes)
            torch.cuda.synchronize()
            assert c.query_status() == 0
            assert [int(x) for x in sizes] == [int(x) for x in lb_o]
            assert np.array_equal(off.cpu().numpy().astype(np.uint64), off_o)
            for l in range(L):
                assert np.array_equal(host[l][:int(sizes[l])].numpy(), bufs_o[l])
                assert bool((host[l][int(sizes[l]):] == 0x55).all())
        small = torch.full((L,), 64, dtype=torch.int64)
        assert c.checkpoint_to_host(geom, pool, sess, ptrs, small, sizes, check=False) == pk.E_INVALID
    finally:
        c.close()


def test_writer_pipeline_leaves_cleanly_when_a_wait_runs_out():
    """The writer's twin of the restore pipeline's timeout path: consumer warp 0 of every CTA withholds one `empty`
    arrival, the producer warp gives up, waits for its copies in flight and leaves; E_TIMEOUT is latched, every
    payload byte is either the checker's or untouched, and the next launch on the context writes the whole payload."""
    import time
    c = new_context()
    try:
        g = pin.Geometry(2, 8, 128, 128, pin.ROPE_HALF, 5e5, 16, 16, 32)
        ck = _ck(geom=g, n=16384, n_pages=1100, tag_probs=(0.3, 0.5, 0.2, 0.0))
        kp, vp = pool_from_raw(ck)
        rc, rc2, off_o, lb_o, bufs_o = run_writer(ck, kp, vp)
        assert rc == oracle.OK and rc2 == oracle.OK
        t0 = time.time()
        c.selftest_stall_next_launch(2, 4096)
        off, sizes, bufs = gpu_writer(c, ck, kp, vp)
        assert time.time() - t0 < 30.0
        assert c.query_status() == -5
        missing = 0
        for a, b in zip(bufs, bufs_o):
            assert np.all((a == b) | (a == 0xEE))
            missing += int((a != b).sum())
        assert missing > 0
        off, sizes, bufs = gpu_writer(c, ck, kp, vp)
        assert c.query_status() == 0
        for a, b in zip(bufs, bufs_o):
            assert np.array_equal(a, b)
    finally:
        c.close()
