"""Pins of the oracle's checkpoint writer (offload side: gather block rows, per-group scales, pack by tag,
cluster same-representation runs).  The independent implementation it is compared with is the torch encoder
of the input generator; the round trip through the oracle's restore pins it against the error bound."""
import numpy as np
import pytest
import torch

import oracle
import patchkv_inputs as pin
from helpers import bf16_bits_to_f64, bf16_ulp, np_u16, oracle_restore


def _ck(**kw):
    g = kw.pop("geom", pin.Geometry(2, 2, 64, 64, pin.ROPE_HALF, 1e4, 16, 16, 32))
    args = dict(name="w", seed=31, geom=g, n=160, delta=0, tag_probs=(0.25, 0.25, 0.25, 0.25), tags_per_layer=True,
                n_outlier=4, outlier_scale=8.0, n_pages=24, table="permutation", dirty_tokens=0, top_k=0, keep_kv=True)
    args.update(kw)
    return pin.make_checkpoint(**args)


def pool_from_raw(ck, shift=0):
    """Scatter the bf16-rounded raw K, V of a checkpoint into sentinel pools through its block table."""
    g = ck.geom
    kp, vp = pin.make_pool(g, ck.n_pages)
    kp, vp = np_u16(kp).copy(), np_u16(vp).copy()
    table = ck.block_table.numpy()
    for l in range(g.n_layers):
        for pool, raw in ((kp, ck.raw_kv[l][0]), (vp, ck.raw_kv[l][1])):
            bits = raw.to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)
            for s in range(ck.n_suffix_tokens):
                u = s + shift
                pool[l, table[u // g.page_tokens], u % g.page_tokens] = bits[s]
    return kp, vp


def run_writer(ck, kp, vp, shift=0, tags=None, table=None, blk_off=None, sizes=None):
    g = ck.geom
    tags = ck.tags.numpy() if tags is None else tags
    rc, off, lb = oracle.plan_checkpoint(tags, g.block_tokens, g.n_kv_heads, g.head_dim, g.group)
    if blk_off is not None:
        off = blk_off
    sizes = [int(x) for x in lb] if sizes is None else sizes
    bufs = [np.full(s, 0xEE, dtype=np.uint8) for s in sizes]
    table = ck.block_table.numpy() if table is None else table
    rc2 = oracle.quantize_gather(L=g.n_layers, H=g.n_kv_heads, D=g.head_dim, B=g.block_tokens, P=g.page_tokens,
                                 G=g.group, k_pool=kp, v_pool=vp, strides=pin.pool_strides(g, ck.n_pages),
                                 n_pages=ck.n_pages, n=ck.n_suffix_tokens, src_shift=shift, block_table=table,
                                 tags=tags, blk_off=off, layer_payload=bufs)
    return rc, rc2, off, lb, bufs


@pytest.mark.parametrize("kw", [dict(), dict(n=150), dict(geom=pin.Geometry(1, 4, 128, 128, pin.ROPE_HALF, 5e5, 16, 16, 128)),
                                dict(geom=pin.Geometry(2, 2, 64, 64, pin.ROPE_HALF, 1e4, 32, 16, 8), n=200, n_pages=40)])
def test_writer_matches_the_generators_encoder_byte_for_byte(kw):
    ck = _ck(**kw)
    g = ck.geom
    kp, vp = pool_from_raw(ck)
    rc, rc2, off, lb, bufs = run_writer(ck, kp, vp)
    assert rc == oracle.OK and rc2 == oracle.OK
    for l in range(g.n_layers):
        k16 = ck.raw_kv[l][0].to(torch.bfloat16).float()
        v16 = ck.raw_kv[l][1].to(torch.bfloat16).float()
        want, want_off = pin.encode_layer(k16, v16, ck.tags[l], g)
        assert np.array_equal(off[l], want_off.numpy().astype(np.uint64))
        assert int(lb[l]) == want.numel()
        assert np.array_equal(bufs[l], want.numpy())


def test_plan_is_the_clustered_layout():
    tags = np.array([[2, 0, 1, 0, 3, 1, 2, 0]], dtype=np.uint8)
    rc, off, lb = oracle.plan_checkpoint(tags, 16, 4, 64, 32)
    r = [oracle.record_bytes(t, 16, 4, 64, 32) for t in range(4)]
    want = {1: 0, 3: r[0], 7: 2 * r[0], 2: 3 * r[0], 5: 3 * r[0] + r[1], 0: 3 * r[0] + 2 * r[1],
            6: 3 * r[0] + 2 * r[1] + r[2], 4: 3 * r[0] + 2 * r[1] + 2 * r[2]}
    assert {j: int(off[0, j]) for j in range(8)} == want
    assert int(lb[0]) == 3 * r[0] + 2 * r[1] + 2 * r[2] + r[3]
    bad = tags.copy()
    bad[0, 3] = 4
    assert oracle.plan_checkpoint(bad, 16, 4, 64, 32)[0] == oracle.E_INVALID


def test_round_trip_through_restore_stays_within_half_a_step():
    ck = _ck(table="identity", n_pages=10)
    g = ck.geom
    kp, vp = pool_from_raw(ck)
    rc, rc2, off, lb, bufs = run_writer(ck, kp, vp)
    NB = ck.n_blocks
    ridx = np.tile(np.arange(NB, dtype=np.int32), (g.n_layers, 1))
    rcnt = np.full(g.n_layers, NB, dtype=np.int32)
    k2 = np.full(kp.shape, pin.SENTINEL, dtype=np.uint16)
    v2 = np.full(vp.shape, pin.SENTINEL, dtype=np.uint16)
    rc3, _ = oracle.restore(L=g.n_layers, H=g.n_kv_heads, D=g.head_dim, Dr=g.rotary_dim, rope_style=g.rope_style,
                            rope_base=g.rope_base, B=g.block_tokens, P=g.page_tokens, G=g.group, k_pool=k2, v_pool=v2,
                            strides=pin.pool_strides(g, ck.n_pages), n_pages=ck.n_pages, n=ck.n_suffix_tokens, delta=0,
                            dst_shift=0, block_table=ck.block_table.numpy(), tags=ck.tags.numpy(), blk_off=off,
                            layer_payload=bufs, reuse_idx=ridx, reuse_cnt=rcnt)
    assert rc3 == oracle.OK
    tags = ck.tags.numpy()
    qmax = {1: (127, 127), 2: (127, 7), 3: (7, 7)}
    for l in range(g.n_layers):
        for j in range(NB):
            sl = slice(j * 16, min((j + 1) * 16, ck.n_suffix_tokens))
            for pool_in, pool_out, which in ((kp, k2, 0), (vp, v2, 1)):
                a = pool_in[l].reshape(-1, g.n_kv_heads, g.head_dim)[sl]
                b = pool_out[l].reshape(-1, g.n_kv_heads, g.head_dim)[sl]
                if tags[l, j] == 0:
                    assert np.array_equal(a, b)
                    continue
                x, y = bf16_bits_to_f64(a), bf16_bits_to_f64(b)
                qm = qmax[int(tags[l, j])][which]
                amax = np.abs(x.reshape(*x.shape[:-1], -1, g.group)).max(axis=-1, keepdims=True)
                step = np.repeat(amax / qm, g.group, axis=-1).reshape(x.shape)
                assert np.all(np.abs(x - y) <= 0.5 * step * (1 + 2.0 ** -9) + bf16_ulp(x) + amax.repeat(g.group, -1).reshape(x.shape) * 2.0 ** -10)


def test_closed_forms_single_value_zero_group_and_codes_in_range():
    g = pin.Geometry(1, 1, 64, 64, pin.ROPE_HALF, 1e4, 16, 16, 32)
    ck = _ck(geom=g, n=16, n_pages=2, table="identity", tag_probs=(0, 1.0, 0, 0))
    kp = np.zeros((1, 2, 16, 1, 64), dtype=np.uint16)
    vp = np.zeros_like(kp)
    kp[0, 0, 3, 0, 5] = 0x4040       # 3.0 alone in group 0 of token 3
    kp[0, 0, 3, 0, 40] = 0xC080      # -4.0 in group 1
    kp[0, 0, 3, 0, 41] = 0x3F80      # 1.0 in group 1
    rc, rc2, off, lb, bufs = run_writer(ck, kp, vp)
    rec = bufs[0]
    codes = rec[:1024].view(np.int8).reshape(16, 64)
    scales = rec[1024:1024 + 64].view(np.float16).reshape(16, 2)
    assert codes[3, 5] == 127 and scales[3, 0] == np.float16(3.0 / 127)
    assert codes[3, 40] == -127 and scales[3, 1] == np.float16(4.0 / 127)
    assert codes[3, 41] == int(np.rint(np.float32(1.0) / np.float32(np.float16(4.0 / 127))))
    assert not codes[0].any() and scales[0, 0] == 0
    ck4 = _ck(tag_probs=(0, 0, 0, 1.0))
    k4, v4 = pool_from_raw(ck4)
    _, _, _, _, bufs4 = run_writer(ck4, k4, v4)
    n_code = 16 * 2 * 64 // 2
    for j in range(ck4.n_blocks):
        o = int(ck4.blk_off[0, j])
        by = bufs4[0][o:o + n_code]
        for nib in (by & 15, by >> 4):
            assert np.all(nib != 8)          # the encoder never emits -8


def test_ragged_suffix_pads_with_zeros_and_shifted_source_pages():
    ck = _ck(n=150, dst_shift=5, n_pages=24)
    g = ck.geom
    kp, vp = pool_from_raw(ck, shift=5)
    rc, rc2, off, lb, bufs = run_writer(ck, kp, vp, shift=5)
    assert rc2 == oracle.OK
    for l in range(g.n_layers):
        k16 = ck.raw_kv[l][0].to(torch.bfloat16).float()
        v16 = ck.raw_kv[l][1].to(torch.bfloat16).float()
        want, _ = pin.encode_layer(k16, v16, ck.tags[l], g)
        assert np.array_equal(bufs[l], want.numpy())      # rows past token 150 are zero in both


@pytest.mark.parametrize("what", ["page", "offset", "table_short"])
def test_writer_skips_out_of_range_blocks(what):
    ck = _ck()
    kp, vp = pool_from_raw(ck)
    _, _, off, lb, good = run_writer(ck, kp, vp)
    table = ck.block_table.numpy().copy()
    off2 = off.copy()
    bad = 4
    if what == "page":
        table[bad] = ck.n_pages + 3
    elif what == "offset":
        off2[:, bad] = max(int(x) for x in lb)
    else:
        table = table[:-1]
        bad = ck.n_blocks - 1
    rc, rc2, _, _, bufs = run_writer(ck, kp, vp, table=table, blk_off=off2)
    assert rc2 == oracle.E_BOUNDS
    g = ck.geom
    for l in range(g.n_layers):
        o = int(off[l, bad])
        r = oracle.record_bytes(int(ck.tags[l, bad]), 16, g.n_kv_heads, g.head_dim, g.group)
        assert np.all(bufs[l][o:o + r] == 0xEE)
        keep = np.ones(bufs[l].size, dtype=bool)
        keep[o:o + r] = False
        assert np.array_equal(bufs[l][keep], good[l][keep])


def scale_raw(ck, factor):
    ck.raw_kv = [(k * factor, v * factor) for k, v in ck.raw_kv]
    return ck


@pytest.mark.parametrize("factor", [3e-5, 1e-6, 2e-8])
def test_tiny_magnitudes_with_subnormal_fp16_scales_match_the_generators_encoder(factor):
    """Groups whose amax / qmax falls in the fp16 subnormal range: the scale loses precision, codes can exceed qmax
    before the clamp, and many groups quantise to a zero scale."""
    ck = scale_raw(_ck(), factor)
    g = ck.geom
    kp, vp = pool_from_raw(ck)
    rc, rc2, off, lb, bufs = run_writer(ck, kp, vp)
    assert rc2 == oracle.OK
    for l in range(g.n_layers):
        k16 = ck.raw_kv[l][0].to(torch.bfloat16).float()
        v16 = ck.raw_kv[l][1].to(torch.bfloat16).float()
        want, _ = pin.encode_layer(k16, v16, ck.tags[l], g)
        assert np.array_equal(bufs[l], want.numpy())
