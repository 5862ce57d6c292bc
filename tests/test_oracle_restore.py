"""Pins of the oracle's dequantise + placement: error bound against the un-quantised data, dense gather,
page bijection, misaligned destination, ragged suffix, and error handling."""
import numpy as np
import pytest
import torch

import oracle
import patchkv_inputs as pin
from helpers import bf16_bits_to_f64, bf16_ulp, oracle_restore, oracle_select


def _ck(tag_probs, **kw):
    g = kw.pop("geom", pin.Geometry(2, 2, 64, 64, pin.ROPE_HALF, 1e4, 16, 16, 32))
    args = dict(name="t", seed=21, geom=g, n=160, delta=0, tag_probs=tag_probs, tags_per_layer=True,
                n_outlier=4, outlier_scale=8.0, n_pages=16, table="identity", dirty_tokens=0, top_k=0, keep_kv=True)
    args.update(kw)
    return pin.make_checkpoint(**args)


def _dense(pool, ck, layer=0):
    g = ck.geom
    return pool[layer].reshape(-1, g.n_kv_heads, g.head_dim)[:ck.n_suffix_tokens]


@pytest.mark.parametrize("tag,qmax_k,qmax_v", [(pin.TAG_INT8, 127, 127), (pin.TAG_INT4, 127, 7), (pin.TAG_K4V4, 7, 7)])
def test_dequantised_values_are_within_half_a_step_of_the_original(tag, qmax_k, qmax_v):
    """Identity table, delta 0: the restored dense tensor is the original within s/2 per group plus one bf16
    rounding.  A wrong scale index, nibble order, sign extension or section offset breaks the bound because
    outlier channels make neighbouring groups' scales differ by 8x."""
    probs = [0.0] * 4
    probs[tag] = 1.0
    ck = _ck(tuple(probs))
    g = ck.geom
    _, sel = oracle_select(ck)
    rc, kp, vp, _ = oracle_restore(ck, sel["reuse_idx"], sel["reuse_cnt"])
    assert rc == oracle.OK
    for l in range(g.n_layers):
        for pool, orig, qmax in ((kp, ck.raw_kv[l][0], qmax_k), (vp, ck.raw_kv[l][1], qmax_v)):
            x = orig.numpy()[:ck.n_suffix_tokens].astype(np.float64)
            got = bf16_bits_to_f64(_dense(pool, ck, l))
            amax = np.abs(x.reshape(*x.shape[:-1], -1, g.group)).max(axis=-1, keepdims=True)
            step = np.repeat(amax / qmax, g.group, axis=-1).reshape(x.shape) * (1 + 2.0 ** -10)
            assert np.all(np.abs(got - x) <= 0.5 * step + bf16_ulp(x))
            # and the bound is tight enough to be a real check: errors do reach a good part of half a step
            assert np.max(np.abs(got - x) / (0.5 * step + 1e-30)) > 0.5


def test_bf16_blocks_are_copied_bit_for_bit_including_nan_and_negative_zero():
    ck = _ck((1.0, 0, 0, 0))
    pay = ck.payload.numpy().view(np.uint16)
    # plant special bit patterns into the first V element slots of block 0 of layer 0
    g = ck.geom
    v_off = (ck.layer_off[0] + int(ck.blk_off[0, 0]) + 2 * 16 * g.n_kv_heads * g.head_dim) // 2
    specials = np.array([0x8000, 0x7FC1, 0xFFFF, 0x7F80, 0x0001], dtype=np.uint16)
    pay[v_off:v_off + 5] = specials
    _, sel = oracle_select(ck)
    rc, kp, vp, _ = oracle_restore(ck, sel["reuse_idx"], sel["reuse_cnt"])
    assert np.array_equal(vp[0].reshape(-1)[:5], specials)
    want_k = ck.raw_kv[0][0].to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)[:ck.n_suffix_tokens]
    assert np.array_equal(_dense(kp, ck, 0), want_k)


def test_values_are_never_rotated():
    a = _ck((0.3, 0.4, 0.3, 0), delta=0, seed=22)
    b = _ck((0.3, 0.4, 0.3, 0), delta=777, seed=22)
    _, sel = oracle_select(a)
    _, ka, va, _ = oracle_restore(a, sel["reuse_idx"], sel["reuse_cnt"])
    _, kb, vb, _ = oracle_restore(b, sel["reuse_idx"], sel["reuse_cnt"])
    assert np.array_equal(va, vb) and not np.array_equal(ka, kb)


def test_permuted_table_is_a_bijection_onto_the_reused_pages():
    ck = pin.config_tiny()
    g = ck.geom
    _, sel = oracle_select(ck)
    rc, kp, vp, _ = oracle_restore(ck, sel["reuse_idx"], sel["reuse_cnt"])
    ident = pin.config_tiny(table="identity")
    rc, kd, vd, _ = oracle_restore(ident, sel["reuse_idx"], sel["reuse_cnt"])
    table = ck.block_table.numpy()
    for l in range(g.n_layers):
        F = sel["reuse_idx"][l, :sel["reuse_cnt"][l]]
        written = set(int(table[j]) for j in F)
        assert len(written) == len(F)
        for p in range(ck.n_pages):
            if p in written:
                j = int(np.nonzero(table == p)[0][0])
                assert np.array_equal(kp[l, p], kd[l, j]) and np.array_equal(vp[l, p], vd[l, j])
            else:       # pages of repaired blocks and unused pages keep the sentinel
                assert np.all(kp[l, p] == pin.SENTINEL) and np.all(vp[l, p] == pin.SENTINEL)


@pytest.mark.parametrize("shift,P", [(5, 16), (0, 32), (11, 32), (3, 8)])
def test_misaligned_destination_pages(shift, P):
    """Source blocks that straddle destination pages: token u = j*B + t + shift lands in slot u % P of
    logical page u // P.  Compared token by token with the aligned dense restore."""
    base = _ck((0.3, 0.4, 0.3, 0), seed=23, delta=55, n=150, dirty_tokens=40, top_k=2, scores="mass")
    _, sel = oracle_select(base)
    rc, kd, vd, _ = oracle_restore(base, sel["reuse_idx"], sel["reuse_cnt"])
    g2 = pin.Geometry(2, 2, 64, 64, pin.ROPE_HALF, 1e4, 16, P, 32)
    n_pages = 40
    ck = _ck((0.3, 0.4, 0.3, 0), seed=23, delta=55, n=150, dirty_tokens=40, top_k=2, geom=g2, dst_shift=shift,
             n_pages=n_pages, table="permutation")
    assert torch.equal(ck.payload, base.payload)
    rc, kp, vp, _ = oracle_restore(ck, sel["reuse_idx"], sel["reuse_cnt"])
    assert rc == oracle.OK
    table = ck.block_table.numpy()
    touched = np.zeros((2, n_pages, P), dtype=bool)
    for l in range(2):
        reused = set(sel["reuse_idx"][l, :sel["reuse_cnt"][l]])
        for s in range(150):
            if s // 16 not in reused:
                continue
            u = s + shift
            page, slot = int(table[u // P]), u % P
            touched[l, page, slot] = True
            assert np.array_equal(kp[l, page, slot], kd[l].reshape(-1, 2, 64)[s])
            assert np.array_equal(vp[l, page, slot], vd[l].reshape(-1, 2, 64)[s])
    assert np.all(kp[~touched] == pin.SENTINEL) and np.all(vp[~touched] == pin.SENTINEL)


def test_ragged_suffix_writes_only_valid_tokens():
    ck = _ck((0.3, 0.4, 0.3, 0), n=150, seed=24)        # last block holds 6 tokens
    _, sel = oracle_select(ck)
    rc, kp, vp, _ = oracle_restore(ck, sel["reuse_idx"], sel["reuse_cnt"])
    flat = kp[0].reshape(-1, 2, 64)
    assert not np.any(np.all(flat[:150] == pin.SENTINEL, axis=(1, 2)))
    assert np.all(flat[150:] == pin.SENTINEL)


def test_all_dirty_is_a_no_op_and_empty_suffix_is_ok():
    ck = _ck((0.3, 0.4, 0.3, 0), dirty_tokens=10 ** 6)
    _, sel = oracle_select(ck)
    assert list(sel["reuse_cnt"]) == [0, 0]
    rc, kp, vp, _ = oracle_restore(ck, sel["reuse_idx"], sel["reuse_cnt"])
    assert rc == oracle.OK and np.all(kp == pin.SENTINEL) and np.all(vp == pin.SENTINEL)


@pytest.mark.parametrize("what", ["page", "negative_page", "tag", "offset", "reuse_index", "table_short"])
def test_out_of_range_items_are_skipped_whole_and_reported(what):
    ck = _ck((0.3, 0.4, 0.3, 0), seed=25)
    _, sel = oracle_select(ck)
    rc, k_ok, v_ok, _ = oracle_restore(ck, sel["reuse_idx"], sel["reuse_cnt"])
    over = {}
    table = ck.block_table.numpy().copy()
    tags = ck.tags.numpy().copy()
    off = ck.blk_off.numpy().copy()
    ridx = sel["reuse_idx"].copy()
    bad_block = 3
    if what == "page":
        table[bad_block] = ck.n_pages
        over["block_table"] = table
    elif what == "negative_page":
        table[bad_block] = -1
        over["block_table"] = table
    elif what == "tag":
        tags[:, bad_block] = 9
        over["tags"] = tags
    elif what == "offset":
        off[:, bad_block] = max(ck.layer_bytes) - 16
        over["blk_off"] = off
    elif what == "reuse_index":
        ridx[:, bad_block] = ck.n_blocks
    elif what == "table_short":
        over["block_table"] = table[:-1]
        bad_block = ck.n_blocks - 1
    rc, kp, vp, _ = oracle_restore(ck, ridx, sel["reuse_cnt"], **over)
    assert rc == oracle.E_BOUNDS
    page_of_bad = int(ck.block_table[bad_block])
    for l in range(2):
        for p in range(ck.n_pages):
            if p == page_of_bad:
                assert np.all(kp[l, p] == pin.SENTINEL) and np.all(vp[l, p] == pin.SENTINEL)
            else:
                assert np.array_equal(kp[l, p], k_ok[l, p]) and np.array_equal(vp[l, p], v_ok[l, p])


def test_invalid_geometry_is_rejected():
    ck = _ck((1.0, 0, 0, 0))
    _, sel = oracle_select(ck)
    rc, *_ = oracle_restore(ck, sel["reuse_idx"], sel["reuse_cnt"], dst_shift=16)
    assert rc == oracle.E_INVALID


def test_thread_count_does_not_change_the_result():
    ck = pin.config_tiny()
    _, sel = oracle_select(ck)
    _, k1, v1, _ = oracle_restore(ck, sel["reuse_idx"], sel["reuse_cnt"], n_threads=1)
    _, k8, v8, _ = oracle_restore(ck, sel["reuse_idx"], sel["reuse_cnt"], n_threads=8)
    assert np.array_equal(k1, k8) and np.array_equal(v1, v8)
