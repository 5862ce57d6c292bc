"""Plumbing of the GPU parity tests: run a checkpoint through the C-ABI library and through the oracle."""
from __future__ import annotations

import numpy as np
import torch

import oracle
import patchkv_inputs as pin
from helpers import bf16_bits_to_f64, bf16_ulp, np_u16, oracle_restore, oracle_select

DEV = "cuda:0"


def new_context(**kw):
    from paper_2609_26219_b200 import build, binding as pk
    build.build()
    return pk.Context(device=0, **kw)


def staged(ck, **kw):
    from patchkv_inputs.staging import StagedCheckpoint
    return StagedCheckpoint(ck, DEV, **kw)


def gpu_pool(ck, n_pages=None):
    from patchkv_inputs.staging import device_pool
    return device_pool(ck, DEV, n_pages)


def check_select(st, sel, mass=None):
    """Bit-exact comparison of every selection output with the oracle's."""
    torch.cuda.synchronize()
    assert np.array_equal(st.repair_cnt.cpu().numpy(), sel["repair_cnt"])
    assert np.array_equal(st.reuse_cnt.cpu().numpy(), sel["reuse_cnt"])
    assert np.array_equal(st.repair_mask.cpu().numpy(), sel["mask"])
    assert np.array_equal(st.repair_idx.cpu().numpy(), sel["repair_idx"])
    assert np.array_equal(st.reuse_idx.cpu().numpy(), sel["reuse_idx"])
    if mass is not None:
        assert np.array_equal(st.mass_out.cpu().numpy().astype(np.uint64), mass)


def check_pools(k_gpu, v_gpu, k_ref, v_ref, geom, expect_exact_k=True):
    """V and placement bit-exact (every page, sentinel pages included).  K: channels outside the rotary dimension
    bit-exact; a rotated channel within 2 bf16 ulp of the reference at the scale of its rotary PAIR,
    abs(gpu - ref) <= 2 ulp(max(abs(ref), 2^-7 * pair)), and within 1e-2 absolute where the pair stays within 8.
    `pair` is max(abs a', abs b') / sqrt(2) of the reference outputs, which never exceeds the max(abs a, abs b) of the
    pair's inputs (a rotation keeps the norm), so the band is at least as tight as one built on the inputs.
    Returns the fraction of K halfwords that are bit-identical."""
    kg, vg = np_u16(k_gpu).reshape(k_ref.shape), np_u16(v_gpu).reshape(v_ref.shape)
    assert np.array_equal(vg, v_ref), "V / placement mismatch"
    same = kg == k_ref
    frac = float(same.mean())
    if not same.all():
        # a sentinel on one side only is a placement error, not a numeric one
        assert np.array_equal(kg == pin.SENTINEL, k_ref == pin.SENTINEL), "K placement mismatch"
        D, Dr = geom.head_dim, geom.rotary_dim
        assert same[..., Dr:].all(), "K channel outside the rotary dimension differs"
        c = np.arange(Dr)
        partner = np.where(c < Dr // 2, c + Dr // 2, c - Dr // 2) if geom.rope_style == pin.ROPE_HALF else c ^ 1
        g, r = bf16_bits_to_f64(kg[..., :Dr]), bf16_bits_to_f64(k_ref[..., :Dr])
        live = k_ref[..., :Dr] != pin.SENTINEL
        r_live = np.where(live, r, 0.0)
        pair = np.maximum(np.abs(r_live), np.abs(r_live[..., partner])) / np.sqrt(2.0)
        tol = 2 * bf16_ulp(np.maximum(np.abs(r_live), 2.0 ** -7 * pair))
        err = np.where(live, np.abs(g - r), 0.0)
        nan_ok = np.isnan(g) & np.isnan(r)
        err = np.where(nan_ok, 0.0, err)
        assert np.all(err <= tol), f"K beyond 2 bf16 ulp: max err {err.max()}"
        assert np.all(err[pair * np.sqrt(2.0) <= 8] <= 1e-2)
    if expect_exact_k:
        assert frac == 1.0, f"K not bit-exact: {frac}"
    return frac


def run_select_and_restore(ctx, ck, layers=None, host=False, oracle_threads=0, inv_freq=None):
    """select_repair + restore through the C ABI, the same through the oracle, compared in full on `layers`."""
    st = staged(ck, payload_on_host=host)
    mass, sel = oracle_select(ck)
    ctx.select_repair(st.select_args())
    check_select(st, sel, mass if ck.attn is not None else None)
    k, v, pool = gpu_pool(ck)
    inv_t = None if inv_freq is None else torch.from_numpy(np.ascontiguousarray(inv_freq, dtype=np.float32))
    if host:
        ctx.restore_from_host(st.geom(inv_t), pool, [st.host_session()])
    else:
        ctx.restore(st.geom(inv_t), pool, [st.session()])
    torch.cuda.synchronize()
    assert ctx.query_status() == 0
    layers = list(range(ck.geom.n_layers)) if layers is None else layers
    rc, k_ref, v_ref, _ = oracle_restore(ck, sel["reuse_idx"], sel["reuse_cnt"], layers=layers,
                                         n_threads=oracle_threads, inv_freq=inv_freq)
    assert rc == oracle.OK
    frac = check_pools(k[layers], v[layers], k_ref, v_ref, ck.geom)
    return st, sel, (k, v), frac
