"""Pins of the oracle's precision planner (Eqs. 13-14): closed forms, the limiting cases alpha = 0 and 1,
threshold ordering, and a float64 numpy statement within fp32 rounding."""
import numpy as np
import pytest

import oracle


def test_closed_forms_per_block():
    # block 0: one fragile token; block 1: uniform; block 2 (ragged): a single token
    attn = np.array([0.25, 0, 0, 0, 0.04, 0.04, 0.04, 0.04, 0.01], dtype=np.float32)
    resid = np.array([0.16, 0, 0, 0, 0.25, 0.25, 0.25, 0.25, 0.01], dtype=np.float32)
    rc, tags, risk = oracle.plan_precision(attn, resid, 4, 0.5, 0.05, 0.15, 0.2)
    assert rc == oracle.OK
    z0 = np.sqrt(np.float32(0.25) * np.float32(0.16))           # 0.2 ; mean 0.05
    assert abs(risk[0] - (0.5 * z0 + 0.5 * z0 / 4)) < 1e-7
    assert abs(risk[1] - 0.1) < 1e-7                            # max = mean = sqrt(0.01)
    assert abs(risk[2] - 0.01) < 1e-7
    assert list(tags) == [1, 1, 2]      # 0.125 and 0.1 in [tau_L, tau_H); 0.01 < tau_L with residual 0.01 <= eps4


def test_alpha_limits_and_thresholds():
    rng = np.random.default_rng(2)
    attn = rng.random(640).astype(np.float32) / 640
    resid = rng.random(640).astype(np.float32) * 0.3
    z = np.sqrt(attn.astype(np.float64) * resid.astype(np.float64)).reshape(40, 16)
    _, _, r_max = oracle.plan_precision(attn, resid, 16, 1.0, 0.0, 1.0, 1.0)
    _, _, r_mean = oracle.plan_precision(attn, resid, 16, 0.0, 0.0, 1.0, 1.0)
    assert np.allclose(r_max, z.max(axis=1), rtol=1e-6) and np.allclose(r_mean, z.mean(axis=1), rtol=1e-6)
    for alpha in (0.2, 0.7):
        _, tags, r = oracle.plan_precision(attn, resid, 16, alpha, 0.004, 0.008, 0.25)
        want = alpha * z.max(axis=1) + (1 - alpha) * z.mean(axis=1)
        assert np.allclose(r, want, rtol=1e-6)
        emax = resid.reshape(40, 16).max(axis=1)
        margin = np.minimum(np.abs(want - 0.004), np.abs(want - 0.008)) > 1e-7     # away from the thresholds
        exp = np.where(want >= 0.008, 0, np.where(want >= 0.004, 1, np.where(emax <= 0.25, 2, 1)))
        assert np.array_equal(tags[margin], exp[margin].astype(np.uint8))
        assert set(tags) <= {0, 1, 2}
    # raising the risk never lowers the precision tier: scale attention up
    _, t1, _ = oracle.plan_precision(attn, resid, 16, 0.5, 0.004, 0.008, 1.0)
    _, t2, _ = oracle.plan_precision(attn * 4, resid, 16, 0.5, 0.004, 0.008, 1.0)
    tier = {0: 2, 1: 1, 2: 0}
    assert all(tier[int(b)] >= tier[int(a)] for a, b in zip(t1, t2))


def test_low_bit_test_gates_the_four_bit_tier_and_bad_arguments():
    attn = np.full(32, 1e-4, dtype=np.float32)
    resid = np.full(32, 0.01, dtype=np.float32)
    resid[20] = 0.9                                  # one token with a large residual in block 1
    _, tags, _ = oracle.plan_precision(attn, resid, 16, 0.0, 0.5, 0.9, 0.1)
    assert list(tags) == [2, 1]
    assert oracle.plan_precision(attn, resid, 16, 1.5, 0.1, 0.2, 0.1)[0] == oracle.E_INVALID
    assert oracle.plan_precision(attn, resid, 16, 0.5, 0.3, 0.2, 0.1)[0] == oracle.E_INVALID
