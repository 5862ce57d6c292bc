"""The K acceptance band used by the GPU parity tests, checked on the CPU with made-up pools: one bf16 step on a
rotated channel is inside it, a larger error is not, and a channel outside the rotary dimension, a V element or a
placement difference is never tolerated."""
import numpy as np
import pytest
import torch

import patchkv_inputs as pin
from gpu_common import check_pools


def _pools(seed=0, shape=(1, 3, 4, 2, 32)):
    rng = np.random.default_rng(seed)
    k = (rng.standard_normal(shape).astype(np.float32).view(np.uint32) >> 16).astype(np.uint16)
    v = (rng.standard_normal(shape).astype(np.float32).view(np.uint32) >> 16).astype(np.uint16)
    k[0, 2] = pin.SENTINEL
    v[0, 2] = pin.SENTINEL
    return k, v


def _t(a):
    return torch.from_numpy(a.view(np.int16).copy())


@pytest.mark.parametrize("style", [pin.ROPE_HALF, pin.ROPE_INTERLEAVED])
def test_band(style):
    g = pin.Geometry(1, 2, 32, 16, style, 1e4, 4, 4, 8)
    k, v = _pools()
    assert check_pools(_t(k), _t(v), k, v, g) == 1.0
    one = k.copy()
    one[0, 0, 1, 1, 3] += 1                                   # one bf16 step on a rotated channel
    assert check_pools(_t(one), _t(v), k, v, g, expect_exact_k=False) < 1.0
    with pytest.raises(AssertionError):
        check_pools(_t(one), _t(v), k, v, g)                  # bit-exactness is still what the tests demand
    far = k.copy()
    far[0, 0, 1, 1, 3] += 5
    with pytest.raises(AssertionError):
        check_pools(_t(far), _t(v), k, v, g, expect_exact_k=False)
    plain = k.copy()
    plain[0, 0, 1, 1, 20] += 1                                # channel 20 >= rotary_dim 16: never rotated, must be exact
    with pytest.raises(AssertionError):
        check_pools(_t(plain), _t(v), k, v, g, expect_exact_k=False)
    vbad = v.copy()
    vbad[0, 1, 0, 0, 0] ^= 1
    with pytest.raises(AssertionError):
        check_pools(_t(k), _t(vbad), k, v, g, expect_exact_k=False)
    moved = k.copy()
    moved[0, 2, 0, 0, 0] = 0x3F80                             # a write into a page that must keep the sentinel
    with pytest.raises(AssertionError):
        check_pools(_t(moved), _t(v), k, v, g, expect_exact_k=False)


def test_band_scales_with_the_pair_not_the_row():
    """An element that is tiny next to its rotary partner may be off by the partner's scale (cancellation), but an
    element whose own pair is small gets no slack from a large value elsewhere in the head vector."""
    g = pin.Geometry(1, 1, 32, 32, pin.ROPE_HALF, 1e4, 1, 1, 8)
    k = np.full((1, 1, 1, 1, 32), 0x3000, dtype=np.uint16)    # 2^-31-ish small values everywhere
    k[..., 5] = 0x4280                                        # 64.0 at channel 5 ...
    k[..., 21] = 0x2000                                       # ... whose HALF partner (5 + 16) is tiny
    v = k.copy()
    ok = k.copy()
    ok[..., 21] = 0x3B00                                      # off by 2^-9: far beyond 2 ulp of itself, inside 2 ulp(2^-7 * 64 / sqrt 2)
    check_pools(_t(ok), _t(v), k, v, g, expect_exact_k=False)
    bad = k.copy()
    bad[..., 9] = 0x3B00                                      # the same error on a channel whose own pair is tiny
    with pytest.raises(AssertionError):
        check_pools(_t(bad), _t(v), k, v, g, expect_exact_k=False)
