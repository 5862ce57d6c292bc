"""Pins of the oracle's repair-set selection (Eqs. 9-12 at block granularity): brute force, closed forms,
set identities, tie rule, exactness and order independence of the block mass."""
import itertools

import numpy as np
import pytest

import oracle
import patchkv_inputs as pin


def brute_select(mass_row, n, B, d_hat, k):
    """Independent statement: python sets, full sort with the (mass desc, index asc) key."""
    NB = -(-n // B)
    n_d = min(max(d_hat, 0), n)
    dirty = {j for j in range(NB) if j * B < n_d}
    cand = sorted((j for j in range(NB) if j not in dirty), key=lambda j: (-int(mass_row[j]), j))
    R = dirty | set(cand[:k])
    return sorted(R), sorted(set(range(NB)) - R)


@pytest.mark.parametrize("n,B", [(256, 16), (250, 16), (96, 32), (17, 16), (16, 16), (1, 16)])
def test_brute_force_all_k(n, B):
    rng = np.random.default_rng(n * 31 + B)
    NB = -(-n // B)
    mass = rng.integers(0, 50, size=(3, NB)).astype(np.uint64)   # small range: many ties
    for d_hat in (-1, 0, 1, B - 1, B, B + 1, n - 1, n, n + 5):
        for k in range(0, NB + 2):
            sel = oracle.select(mass, n, B, d_hat, k)
            assert sel["status"] == oracle.OK
            for l in range(3):
                R, F = brute_select(mass[l], n, B, d_hat, k)
                assert list(sel["repair_idx"][l, :sel["repair_cnt"][l]]) == R
                assert list(sel["reuse_idx"][l, :sel["reuse_cnt"][l]]) == F
                assert list(np.nonzero(sel["mask"][l])[0]) == R
                assert np.all(sel["repair_idx"][l, len(R):] == -1) and np.all(sel["reuse_idx"][l, len(F):] == -1)


def test_dirty_window_closed_form_and_set_identities():
    n, B, NB = 1000, 16, 63
    rng = np.random.default_rng(5)
    mass = rng.integers(0, 2 ** 40, size=(2, NB)).astype(np.uint64)
    for d_hat in (-1, 0, 1, 15, 16, 17, 999, 1000, 1005):
        n_dirty = -(-min(max(d_hat, 0), n) // B)
        for k in (0, 1, 5, 63, 100):
            sel = oracle.select(mass, n, B, d_hat, k)
            for l in range(2):
                R = set(sel["repair_idx"][l, :sel["repair_cnt"][l]])
                F = set(sel["reuse_idx"][l, :sel["reuse_cnt"][l]])
                assert R | F == set(range(NB)) and not (R & F)
                assert set(range(n_dirty)) <= R
                assert len(R) == n_dirty + min(k, NB - n_dirty)


def test_raising_k_only_adds_blocks():
    rng = np.random.default_rng(6)
    mass = rng.integers(0, 1000, size=(1, 64)).astype(np.uint64)
    prev = set()
    for k in range(0, 60):
        sel = oracle.select(mass, 1024, 16, 90, k)
        R = set(sel["repair_idx"][0, :sel["repair_cnt"][0]])
        assert prev <= R
        prev = R


def test_constant_mass_takes_lowest_index_candidates():
    mass = np.full((1, 64), 12345, dtype=np.uint64)
    sel = oracle.select(mass, 1024, 16, 90, 5)
    assert list(sel["repair_idx"][0, :11]) == list(range(6)) + [6, 7, 8, 9, 10]


def test_one_unit_difference_decides_the_order():
    mass = np.full((1, 8), 2 ** 39, dtype=np.uint64)
    mass[0, 6] += 1
    sel = oracle.select(mass, 128, 16, 0, 1)
    assert list(sel["repair_idx"][0, :1]) == [6]


def test_layers_shared_ranks_on_the_summed_mass():
    mass = np.array([[5, 0, 9, 1], [0, 8, 0, 1], [0, 2, 0, 1]], dtype=np.uint64)   # sums: 5, 10, 9, 3
    sel = oracle.select(mass, 64, 16, 0, 2, pin.LAYERS_SHARED)
    for l in range(3):
        assert list(sel["repair_idx"][l, :2]) == [1, 2]
    ind = oracle.select(mass, 64, 16, 0, 2, pin.LAYERS_INDEPENDENT)
    assert list(ind["repair_idx"][0, :2]) == [0, 2] and list(ind["repair_idx"][1, :2]) == [1, 3]


def test_block_mass_is_exact_and_matches_fractions():
    rng = np.random.default_rng(14)
    # values across the whole fp16 range, including subnormals and large numbers
    bits = rng.integers(0, 0x7C00, size=(2, 3, 4, 100)).astype(np.uint16)
    rc, mass = oracle.block_mass(bits, 16)
    assert rc == oracle.OK
    vals = bits.view(np.float16).astype(np.float64)           # every fp16 is exact in float64
    for l in range(2):
        for j in range(7):
            seg = vals[l, :, :, j * 16:(j + 1) * 16]
            units = sum(int(v * 2 ** 24) for v in seg.reshape(-1))   # exact python integers
            assert int(mass[l, j]) == units
    rc, m64 = oracle.block_mass(bits, 16, as_double=True)
    assert np.array_equal(m64.astype(np.uint64), mass)


def test_block_mass_partial_last_block_and_order_independence():
    ck = pin.config_tiny()
    a = ck.attn.numpy()[:, :, :, :1000]
    a = np.ascontiguousarray(a)
    rc, mass = oracle.block_mass(a, 16)
    assert mass.shape == (2, 63)
    ref = a.astype(np.float64)[:, :, :, 992:].sum(axis=(1, 2, 3)) * 2 ** 24
    assert np.array_equal(mass[:, 62], ref.astype(np.uint64))
    perm_h = np.random.default_rng(1).permutation(a.shape[1])
    perm_q = np.random.default_rng(2).permutation(a.shape[2])
    rc, mass2 = oracle.block_mass(np.ascontiguousarray(a[:, perm_h][:, :, perm_q]), 16)
    assert np.array_equal(mass, mass2)


def test_block_mass_softmax_rows_sum_to_queries_times_heads():
    """Row-softmaxed attention: the total mass of a layer is (close to) Hq * Q, a closed form."""
    ck = pin.config_tiny()
    rc, mass = oracle.block_mass(ck.attn.numpy(), 16)
    total = mass.sum(axis=1).astype(np.float64) / 2 ** 24
    assert np.all(np.abs(total - 8 * 16) < 0.05)


def test_block_mass_strided_view_and_bad_input():
    rng = np.random.default_rng(15)
    big = rng.integers(0, 0x3C00, size=(2, 4, 6, 64)).astype(np.uint16)
    view = big[:, ::2, 1:5, :]                      # non-contiguous heads / queries
    rc, m1 = oracle.block_mass(view, 16)
    rc, m2 = oracle.block_mass(np.ascontiguousarray(view), 16)
    assert np.array_equal(m1, m2)
    bad = big.copy()
    bad[0, 0, 0, 3] = 0xBC00      # -1.0
    bad[1, 1, 1, 40] = 0x7C00     # +inf
    bad[1, 1, 1, 41] = 0x7E00     # NaN
    bad[0, 0, 0, 4] = 0x8000      # -0 is fine
    rc, mb = oracle.block_mass(bad, 16)
    assert rc == oracle.E_BADINPUT
    clean = bad.copy()
    clean[0, 0, 0, 3] = 0
    clean[1, 1, 1, 40] = 0
    clean[1, 1, 1, 41] = 0
    clean[0, 0, 0, 4] = 0
    rc, mc = oracle.block_mass(clean, 16)
    assert rc == oracle.OK and np.array_equal(mb, mc)


def test_tiny_config_counts():
    ck = pin.config_tiny()
    rc, mass = oracle.block_mass(ck.attn.numpy(), 16)
    sel = oracle.select(mass, 1024, 16, ck.dirty_tokens, ck.top_k)
    assert list(sel["repair_cnt"]) == [8, 8] and list(sel["reuse_cnt"]) == [56, 56]
    assert list(sel["repair_idx"][0, :6]) == [0, 1, 2, 3, 4, 5]


# ---------------------------------------------------------------- Norm of Eq. 10 (reported score, not used for ranking)
def test_normalise_closed_forms():
    """Constant masses give exactly 1/NB; a single non-zero unit gives exactly 1; a zero row gives zeros;
    a mass of 1 against a total of 2^k gives exactly 2^-k."""
    for NB in (1, 3, 64, 1000):
        out = oracle.normalise(np.full((2, NB), 12345, dtype=np.uint64))
        assert np.all(out == np.float32(1.0 / NB))
    m = np.zeros((3, 10), dtype=np.uint64)
    m[0, 4] = 7
    m[2, 0] = 1
    m[2, 9] = (1 << 40) - 1
    out = oracle.normalise(m)
    assert out[0, 4] == 1.0 and out[0].sum() == 1.0
    assert np.all(out[1] == 0.0)
    assert out[2, 0] == np.float32(2.0 ** -40) and out[2, 9] == np.float32(1.0)


def test_normalise_sums_to_one_keeps_order_and_ignores_scale():
    rng = np.random.default_rng(11)
    m = rng.integers(0, 1 << 38, size=(4, 777)).astype(np.uint64)
    m[1, :100] = 0
    out = oracle.normalise(m)
    assert out.dtype == np.float32 and out.shape == m.shape
    assert np.all(np.abs(out.astype(np.float64).sum(axis=1) - 1.0) < 777 * 2.0 ** -25)
    for l in range(4):                                     # a larger mass never gets a smaller score
        order = np.argsort(m[l], kind="stable")
        assert np.all(np.diff(out[l][order]) >= 0)
    assert np.array_equal(oracle.normalise(m * np.uint64(8)), out)       # Norm is scale-free (powers of two: exactly)
    # the same quotient by a library routine
    want = (m.astype(np.float64) / m.sum(axis=1, dtype=np.uint64).astype(np.float64)[:, None]).astype(np.float32)
    assert np.array_equal(out, want)


def test_normalise_shared_mode_is_the_share_of_the_layer_summed_mass():
    rng = np.random.default_rng(12)
    m = rng.integers(0, 1 << 30, size=(5, 64)).astype(np.uint64)
    out = oracle.normalise(m, layer_mode=1)
    assert out.shape == (64,)
    summed = m.sum(axis=0, dtype=np.uint64)[None, :]
    assert np.array_equal(out, oracle.normalise(summed)[0])
    # ranking by the score agrees with ranking by the exact mass wherever the scores differ
    sel = oracle.select(m, 64 * 16, 16, 0, 8, 1)
    top = set(sel["repair_idx"][0, :8].tolist())
    assert min(out[j] for j in top) >= max(out[j] for j in range(64) if j not in top)
