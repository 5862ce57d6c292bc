"""Pins of the oracle's RoPE phase correction (Eq. 3): composition, identity, inverse, norm, sign."""
import numpy as np
import pytest

import oracle
import patchkv_inputs as pin
from helpers import bf16_bits_to_f64, bf16_ulp, oracle_restore, oracle_select


def rope_f64(x, pos, base, Dr, style):
    """Textbook RoPE in float64 on x [..., D]: x*cos + rotate(x)*sin with theta_i = base^(-2i/Dr)."""
    x = np.asarray(x, dtype=np.float64)
    i = np.arange(Dr // 2, dtype=np.float64)
    phi = pos * base ** (-2.0 * i / Dr)
    out = x.copy()
    if style == pin.ROPE_HALF:
        cos = np.concatenate([np.cos(phi), np.cos(phi)])
        sin = np.concatenate([np.sin(phi), np.sin(phi)])
        xr = x[..., :Dr]
        rot = np.concatenate([-xr[..., Dr // 2:], xr[..., :Dr // 2]], axis=-1)
    else:
        cos = np.repeat(np.cos(phi), 2)
        sin = np.repeat(np.sin(phi), 2)
        xr = x[..., :Dr]
        rot = np.stack([-xr[..., 1::2], xr[..., 0::2]], axis=-1).reshape(xr.shape)
    out[..., :Dr] = xr * cos + rot * sin
    return out


def pair_norm(x, Dr, style):
    """Norm of the rotary pair each channel belongs to (channels >= Dr: |x|)."""
    x = np.asarray(x, dtype=np.float64)
    out = np.abs(x).copy()
    if style == pin.ROPE_HALF:
        nrm = np.hypot(x[..., :Dr // 2], x[..., Dr // 2:Dr])
        out[..., :Dr // 2] = nrm
        out[..., Dr // 2:Dr] = nrm
    else:
        nrm = np.hypot(x[..., 0:Dr:2], x[..., 1:Dr:2])
        out[..., 0:Dr:2] = nrm
        out[..., 1:Dr:2] = nrm
    return out


def test_table_is_the_angle_addition_identity():
    # cos(d t) cos(p t) - sin(d t) sin(p t) = cos((p + d) t): the table at delta composes with position p
    for base, Dr, p, d in [(1e4, 64, 4096, 137), (5e5, 128, 20000, -2048), (1e6, 128, 31000, -3000)]:
        c, s = oracle.rope_table(Dr, base, d)
        theta = base ** (-2.0 * np.arange(Dr // 2) / Dr)
        lhs = c.astype(np.float64) * np.cos(p * theta) - s.astype(np.float64) * np.sin(p * theta)
        assert np.max(np.abs(lhs - np.cos((p + d) * theta))) < 2.0 ** -22
        assert np.max(np.abs(c.astype(np.float64) ** 2 + s.astype(np.float64) ** 2 - 1)) < 2.0 ** -22


def test_table_delta_zero_is_exact_identity_and_inv_freq_override():
    c, s = oracle.rope_table(64, 1e4, 0)
    assert np.all(c == 1.0) and np.all(s == 0.0)
    inv = (1e4 ** (-2.0 * np.arange(32) / 64)).astype(np.float32)
    c1, s1 = oracle.rope_table(64, 123.0, 77, inv_freq=inv)   # base ignored when inv_freq is given
    assert np.allclose(c1, np.cos(77 * inv.astype(np.float64)), atol=2 ** -23)
    assert np.allclose(s1, np.sin(77 * inv.astype(np.float64)), atol=2 ** -23)


def test_sign_convention_positive_delta_rotates_counter_clockwise():
    # theta_0 = 1: the pair (1, 0) moved by delta lands on (cos delta, sin delta)
    c, s = oracle.rope_table(4, 1e4, 1)
    a, b = oracle.rotate_pair_f32(1.0, 0.0, float(c[0]), float(s[0]))
    assert abs(a - np.cos(1.0)) < 1e-7 and abs(b - np.sin(1.0)) < 1e-7
    a, b = oracle.rotate_pair_f32(0.0, 1.0, float(c[0]), float(s[0]))
    assert abs(a + np.sin(1.0)) < 1e-7 and abs(b - np.cos(1.0)) < 1e-7


def test_rotate_pair_unit_table_is_identity_for_finite_values():
    rng = np.random.default_rng(3)
    for a, b in rng.standard_normal((100, 2)).astype(np.float32):
        assert oracle.rotate_pair_f32(float(a), float(b), 1.0, 0.0) == (float(a), float(b))


@pytest.mark.parametrize("style", [pin.ROPE_HALF, pin.ROPE_INTERLEAVED])
@pytest.mark.parametrize("D,Dr", [(64, 64), (128, 128), (64, 32)])
def test_composition_invariant_fp32(style, D, Dr):
    """A key stored at position p and moved by delta equals fresh RoPE at p + delta of the un-rotated key."""
    rng = np.random.default_rng(11)
    base, p, delta = 1e4, 4096, 137
    kt = rng.standard_normal((64, D))
    k_old = rope_f64(kt, p, base, Dr, style).astype(np.float32)
    c, s = oracle.rope_table(Dr, base, delta)
    got = oracle.rotate_head_f32(k_old, Dr, style, c, s).astype(np.float64)
    want = rope_f64(kt, p + delta, base, Dr, style)
    assert np.all(np.abs(got - want) <= 2.0 ** -20 * np.maximum(pair_norm(kt, Dr, style), 1e-30))
    # channels past the rotary dimension are untouched
    assert np.array_equal(got[:, Dr:], k_old[:, Dr:].astype(np.float64))


@pytest.mark.parametrize("style", [pin.ROPE_HALF, pin.ROPE_INTERLEAVED])
def test_matches_numpy_rotate_half_formulation(style):
    rng = np.random.default_rng(12)
    x = rng.standard_normal((32, 128)).astype(np.float32)
    for delta in (1, -1, 2048, -3000, 8192):
        c, s = oracle.rope_table(128, 5e5, delta)
        got = oracle.rotate_head_f32(x, 128, style, c, s).astype(np.float64)
        want = rope_f64(x, delta, 5e5, 128, style)
        assert np.all(np.abs(got - want) <= 2.0 ** -21 * pair_norm(x, 128, style))


def test_norm_is_preserved_per_pair():
    rng = np.random.default_rng(13)
    x = rng.standard_normal((64, 64)).astype(np.float32)
    c, s = oracle.rope_table(64, 1e4, -555)
    y = oracle.rotate_head_f32(x, 64, pin.ROPE_HALF, c, s)
    n_in = pair_norm(x, 64, pin.ROPE_HALF)
    n_out = pair_norm(y, 64, pin.ROPE_HALF)
    assert np.all(np.abs(n_out - n_in) <= 2.0 ** -21 * n_in)


def _bf16_checkpoint(style=pin.ROPE_HALF, D=64, Dr=64, delta=137):
    g = pin.Geometry(1, 2, D, Dr, style, 1e4, 16, 16, 32)
    return pin.make_checkpoint(name="bf16", seed=5, geom=g, n=128, delta=delta, tag_probs=(1.0, 0, 0, 0),
                               n_pages=8, table="identity", dirty_tokens=0, top_k=0, keep_kv=True)


@pytest.mark.parametrize("style", [pin.ROPE_HALF, pin.ROPE_INTERLEAVED])
def test_restore_composition_through_bf16_storage(style):
    """End to end through the restore routine: K stored in bf16 at position p, restored with delta, is within
    2 bf16 ulp (at the pair-norm scale) of fresh RoPE at p + delta."""
    ck = _bf16_checkpoint(style)
    g = ck.geom
    k_old = ck.raw_kv[0][0].numpy().astype(np.float64)          # treat the stored K as already rotated to p
    p = 4096
    kt = rope_f64(k_old, -p, g.rope_base, g.rotary_dim, style)   # the un-rotated key
    _, sel = oracle_select(ck)
    rc, kp, vp, _ = oracle_restore(ck, sel["reuse_idx"], sel["reuse_cnt"])
    assert rc == oracle.OK
    got = bf16_bits_to_f64(kp.reshape(128, g.n_kv_heads, g.head_dim))
    want = rope_f64(kt, p + ck.delta, g.rope_base, g.rotary_dim, style)
    assert np.all(np.abs(got - want) <= 2 * bf16_ulp(pair_norm(k_old, g.rotary_dim, style)))


def test_restore_delta_zero_copies_bf16_keys_and_matches_value_path():
    ck = _bf16_checkpoint(delta=0)
    _, sel = oracle_select(ck)
    rc, kp, vp, _ = oracle_restore(ck, sel["reuse_idx"], sel["reuse_cnt"])
    k_bits = ck.raw_kv[0][0].to(__import__("torch").bfloat16).view(__import__("torch").int16).numpy().view(np.uint16)
    assert np.array_equal(kp.reshape(k_bits.shape), k_bits)


@pytest.mark.parametrize("tag_probs", [(0, 1.0, 0, 0), (0, 0, 0, 1.0)])
def test_restore_delta_zero_quantised_key_equals_value_style_dequant(tag_probs):
    """With delta = 0 the K path is the V path: a checkpoint whose K and V sections hold the same data
    restores to identical K and V pages (int8 K vs int8 V; int4 K vs int4 V)."""
    g = pin.Geometry(1, 2, 64, 64, pin.ROPE_HALF, 1e4, 16, 16, 32)
    ck = pin.make_checkpoint(name="same", seed=6, geom=g, n=64, delta=0, tag_probs=tag_probs, n_pages=4,
                             table="identity", dirty_tokens=0, top_k=0)
    # overwrite every V section with its K section
    pay = ck.payload.numpy()
    tag = int(ck.tags[0, 0])
    half = pin.record_bytes(tag, g) // 2
    for j in range(ck.n_blocks):
        o = ck.layer_off[0] + int(ck.blk_off[0, j])
        pay[o + half:o + 2 * half] = pay[o:o + half]
    _, sel = oracle_select(ck)
    rc, kp, vp, _ = oracle_restore(ck, sel["reuse_idx"], sel["reuse_cnt"])
    assert rc == oracle.OK and np.array_equal(kp, vp)
    assert not np.any(kp == pin.SENTINEL)


def test_restore_then_inverse_delta_returns_the_input():
    ck = _bf16_checkpoint(delta=911)
    g = ck.geom
    _, sel = oracle_select(ck)
    rc, kp, vp, _ = oracle_restore(ck, sel["reuse_idx"], sel["reuse_cnt"])
    # feed the restored pages back as a bf16 checkpoint and undo the shift
    back = _bf16_checkpoint(delta=-911)
    pay = back.payload.numpy()
    rec = pin.record_bytes(pin.TAG_BF16, g)
    kblocks = kp.reshape(back.n_blocks, -1).view(np.uint8)
    for j in range(back.n_blocks):
        o = back.layer_off[0] + int(back.blk_off[0, j])
        pay[o:o + rec // 2] = kblocks[j]
    rc, kp2, _, _ = oracle_restore(back, sel["reuse_idx"], sel["reuse_cnt"])
    k0 = ck.raw_kv[0][0].numpy().astype(np.float64)
    got = bf16_bits_to_f64(kp2.reshape(k0.shape))
    assert np.all(np.abs(got - k0) <= 2 * bf16_ulp(pair_norm(k0, g.rotary_dim, g.rope_style)))


def test_fp32_recipe_is_close_to_the_double_evaluation():
    ck = pin.config_tiny()
    _, sel = oracle_select(ck)
    rc, kp, vp, stats = oracle_restore(ck, sel["reuse_idx"], sel["reuse_cnt"], want_stats=True)
    assert rc == oracle.OK
    max_abs, n_diff, n_tot = stats
    assert n_tot == 2 * 56 * 16 * 4 * 64
    assert n_diff / n_tot < 1e-3          # double rounding differs only at near-ties
