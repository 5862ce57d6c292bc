"""The 70B-shaped stress workload at its full size: 80 layers, 8 sessions with a 64k-token suffix each, one shared
pool of 32768 pages, payloads in pinned host memory, restored by patchkv_restore_from_host one wave of 10 layers
at a time (the 80-layer pool and payload do not fit next to each other; the benchmark times the same waves).

Checked against the oracle: per session its first layer, its last layer and two seeded layers, compared in full
(the whole shared-pool layer, so all eight sessions' pages of that layer), and on every layer of every wave a scan
on the device that each page that is no reused block's destination still holds the sentinel, while every page that
is one no longer does."""
import numpy as np
import pytest
import torch

import oracle
import patchkv_inputs as pin
from gpu_common import DEV, check_pools, gpu_pool, new_context, staged
from helpers import np_u16, oracle_restore, oracle_select

pytestmark = pytest.mark.gpu

WAVE = pin.STRESS_WAVE_LAYERS
N_WAVES = pin.STRESS_LAYERS // WAVE


def sampled_layers():
    """Global layer indices compared in full: first and last, and two seeded layers per session."""
    rng = np.random.default_rng(1005)
    picks = {0, pin.STRESS_LAYERS - 1}
    for _ in range(8):
        picks.update(int(x) for x in rng.choice(np.arange(1, pin.STRESS_LAYERS - 1), size=2, replace=False))
    return sorted(picks)


@pytest.mark.parametrize("flags", [0, 2], ids=["staged", "zero_copy"])
def test_stress_full_size_sampled_layers_and_sentinel_scan(flags):
    picks = sampled_layers()
    fill = pin.SENTINEL - 0x10000
    ctx = new_context(flags=flags)
    try:
        waves = range(N_WAVES) if flags == 0 else [0, N_WAVES - 1]        # the zero-copy mode: first and last wave
        for w in waves:
            local = [l - w * WAVE for l in picks if w * WAVE <= l < (w + 1) * WAVE]
            sess = pin.stress_wave(w, device=DEV)
            sts = [staged(c, payload_on_host=True) for c in sess]
            for s in sts:
                ctx.select_repair(s.select_args())
            torch.cuda.synchronize()
            k, v, pool = gpu_pool(sess[0])
            rc, stats = ctx.restore_from_host(sts[0].geom(), pool, [s.host_session() for s in sts])
            torch.cuda.synchronize()
            assert ctx.query_status() == 0
            sels = [oracle_select(c)[1] for c in sess]
            assert stats.n_block_layers == sum(int(sel["reuse_cnt"].sum()) for sel in sels)
            for s, sel in zip(sts, sels):
                assert np.array_equal(s.reuse_idx.cpu().numpy(), sel["reuse_idx"])
                assert np.array_equal(s.reuse_cnt.cpu().numpy(), sel["reuse_cnt"])
            # ---- scan on the device, every layer of the wave: block j of a session lands in page table[j] (P = B)
            n_pages = sess[0].n_pages
            target = torch.zeros((WAVE, n_pages), dtype=torch.bool, device=DEV)
            for c, sel in zip(sess, sels):
                table = c.block_table.to(DEV).long()
                for l in range(WAVE):
                    F = torch.from_numpy(sel["reuse_idx"][l, :sel["reuse_cnt"][l]].astype(np.int64)).to(DEV)
                    target[l, table[F]] = True
            for t in (k, v):
                clean = (t.view(WAVE, n_pages, -1) == fill).all(dim=2)       # page still all sentinel
                assert bool((clean == ~target).all()), "a page outside the reuse set was written, or one inside it was not"
            # ---- sampled layers in full, against the oracle's restore of all eight sessions into one shared pool
            for l in local:
                k_ref = v_ref = None
                for c, sel in zip(sess, sels):
                    pools = None if k_ref is None else (k_ref, v_ref)
                    rc, k_ref, v_ref, _ = oracle_restore(c, sel["reuse_idx"], sel["reuse_cnt"], layers=[l], pools=pools)
                    assert rc == oracle.OK
                same_v = torch.equal(v[l].cpu(), torch.from_numpy(v_ref[0].view(np.int16)))
                same_k = torch.equal(k[l].cpu(), torch.from_numpy(k_ref[0].view(np.int16)))
                if not (same_v and same_k):
                    check_pools(k[l:l + 1], v[l:l + 1], k_ref, v_ref, sess[0].geom)
            del sts, k, v, pool, sess, target
            torch.cuda.empty_cache()
    finally:
        ctx.close()
