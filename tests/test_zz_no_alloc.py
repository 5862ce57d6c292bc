"""patchkv_select_repair_static, the selection entry point for callers that cannot allocate device memory
(an engine whose KV pool already owns all of HBM; a resume path that must not stall the device with an
allocation).  Collected last on purpose: a failure here cannot hide any other test behind `-x`.

The check: through the C ABI, its outputs equal those of patchkv_select_repair bit for bit, on two calls in a
row that reuse the library's fixed scratch array with different contents, and oversize problems are refused.
"""
import numpy as np
import pytest
import torch

import patchkv_inputs as pin

pytestmark = pytest.mark.gpu

DEV = "cuda:0"


def _both(ctx, ck):
    from paper_2609_26219_b200 import binding as pk
    from patchkv_inputs.staging import StagedCheckpoint
    ref = StagedCheckpoint(ck, DEV)
    new = StagedCheckpoint(ck, DEV)
    ctx.select_repair(ref.select_args())
    status = torch.zeros(1, dtype=torch.int32, device=DEV)
    assert pk.select_repair_static(new.select_args(), None, status) == pk.OK
    torch.cuda.synchronize()
    for name in ("repair_mask", "repair_idx", "repair_cnt", "reuse_idx", "reuse_cnt"):
        assert torch.equal(getattr(ref, name), getattr(new, name)), name
    if ck.attn is not None:
        assert torch.equal(ref.mass_out, new.mass_out)
    assert int(status.item()) == 0
    return new


def test_static_scratch_variant_matches_the_context_variant_twice_in_a_row():
    from paper_2609_26219_b200 import build, binding as pk
    build.build()
    torch.cuda.set_device(0)
    ctx = pk.Context(device=0)
    try:
        # first call: stored attention, per-layer sets; second call right after it: other data, a ragged suffix
        # and layer-shared ranking, so the array's leftovers from the first call would show
        a = _both(ctx, pin.config_tiny())
        assert int(a.reuse_cnt[0]) == 56
        _both(ctx, pin.config_tiny(seed=4242, n=1000, top_k=7, dirty_tokens=33, layer_mode=pin.LAYERS_SHARED))
        # stored block masses need no scratch at all unless layers are shared
        _both(ctx, pin.config_llama8b(n_layers=3))
    finally:
        ctx.close()


def test_static_scratch_variant_refuses_what_does_not_fit_and_reports_bad_input():
    from paper_2609_26219_b200 import build, binding as pk
    from patchkv_inputs.staging import StagedCheckpoint
    build.build()
    torch.cuda.set_device(0)
    ck = pin.config_tiny()
    st = StagedCheckpoint(ck, DEV)
    # claim a problem of L * NB = 2 * 200000 masses: more than the fixed array holds -> refused, nothing runs
    big = st.select_args(n_suffix_tokens=200000 * 16)
    assert pk.select_repair_static(big, None, None) == pk.E_TOO_LARGE
    torch.cuda.synchronize()
    assert int(st.repair_cnt[0]) == -7          # outputs untouched
    bad = st.select_args()
    bad.top_k = -1
    assert pk.select_repair_static(bad, None, None) == pk.E_INVALID
    # a negative attention entry is latched into the caller's status word
    st.attn[0, 0, 0, 5] = -1.0
    status = torch.zeros(1, dtype=torch.int32, device=DEV)
    assert pk.select_repair_static(st.select_args(), None, status) == pk.OK
    torch.cuda.synchronize()
    assert int(status.item()) == pk.E_BADINPUT
