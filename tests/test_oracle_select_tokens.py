"""Pins of the oracle's token-level selection (Eqs. 9-12 as the paper prints them: top-kappa TOKENS, then block
rounding): brute force with python sets, reductions to the block form, closure properties."""
import numpy as np
import pytest

import oracle
import patchkv_inputs as pin


def brute(mass_row, n, B, d_hat, kappa):
    nd = min(max(d_hat, 0), n)
    D = set(range(nd))
    cand = sorted((i for i in range(n) if i not in D), key=lambda i: (-int(mass_row[i]), i))
    H = set(cand[:kappa])
    R = sorted({i // B for i in D | H})
    NB = -(-n // B)
    return D | H, R, sorted(set(range(NB)) - set(R))


@pytest.mark.parametrize("n,B", [(200, 16), (193, 16), (64, 32), (17, 16), (5, 8)])
@pytest.mark.parametrize("mode", [pin.LAYERS_INDEPENDENT, pin.LAYERS_SHARED])
def test_brute_force(n, B, mode):
    rng = np.random.default_rng(n + B)
    mass = rng.integers(0, 30, size=(3, n)).astype(np.uint64)          # many ties
    ranked = mass if mode == pin.LAYERS_INDEPENDENT else np.tile(mass.sum(axis=0), (3, 1))
    for d_hat in (-3, 0, 1, B - 1, B, B + 1, n - 1, n, n + 9):
        for kappa in (0, 1, 2, 7, n // 3, n, n + 4):
            sel = oracle.select_tokens(mass, B, d_hat, kappa, mode)
            assert sel["status"] == oracle.OK
            for l in range(3):
                T, R, F = brute(ranked[l], n, B, d_hat, kappa)
                assert set(np.nonzero(sel["token_mask"][l])[0]) == T
                assert list(sel["repair_idx"][l, :sel["repair_cnt"][l]]) == R
                assert list(sel["reuse_idx"][l, :sel["reuse_cnt"][l]]) == F
                assert list(np.nonzero(sel["mask"][l])[0]) == R


def test_block_size_one_is_the_block_form():
    rng = np.random.default_rng(3)
    mass = rng.integers(0, 10 ** 6, size=(2, 300)).astype(np.uint64)
    tok = oracle.select_tokens(mass, 1, 40, 25, pin.LAYERS_INDEPENDENT)
    blk = oracle.select(mass, 300, 1, 40, 25, pin.LAYERS_INDEPENDENT)
    for key in ("mask", "repair_idx", "repair_cnt", "reuse_idx", "reuse_cnt"):
        assert np.array_equal(tok[key], blk[key])


def test_token_and_block_forms_can_differ_and_every_chosen_token_is_covered():
    # one heavy token in block 5, two medium tokens in block 2 whose SUM is larger: the block form takes block 2
    # first, the token form takes block 5 first
    n, B = 128, 16
    mass = np.ones((1, n), dtype=np.uint64)
    mass[0, 5 * B + 3] = 1000
    mass[0, 2 * B + 1] = 600
    mass[0, 2 * B + 9] = 600
    tok = oracle.select_tokens(mass, B, 0, 1, pin.LAYERS_INDEPENDENT)
    assert list(tok["repair_idx"][0, :tok["repair_cnt"][0]]) == [5]
    bm = mass.reshape(1, n // B, B).sum(axis=2)
    blk = oracle.select(bm, n, B, 0, 1, pin.LAYERS_INDEPENDENT)
    assert list(blk["repair_idx"][0, :blk["repair_cnt"][0]]) == [2]
    # closure: the blocks of R cover D u H, and kappa tokens mark at most kappa extra blocks
    rng = np.random.default_rng(4)
    mass = rng.integers(0, 10 ** 9, size=(2, 1000)).astype(np.uint64)
    sel = oracle.select_tokens(mass, 16, 90, 15, pin.LAYERS_SHARED)
    for l in range(2):
        R = set(sel["repair_idx"][l, :sel["repair_cnt"][l]])
        assert {i // 16 for i in np.nonzero(sel["token_mask"][l])[0]} == R
        assert 6 <= len(R) <= 6 + 15
        assert int(sel["token_mask"][l].sum()) == 90 + 15


def test_raising_kappa_only_adds_blocks_and_shared_mode_gives_every_layer_the_same_sets():
    rng = np.random.default_rng(5)
    mass = rng.integers(0, 50, size=(3, 400)).astype(np.uint64)
    prev = set()
    for kappa in range(0, 60, 3):
        sel = oracle.select_tokens(mass, 16, 33, kappa, pin.LAYERS_SHARED)
        R = set(sel["repair_idx"][0, :sel["repair_cnt"][0]])
        assert prev <= R
        prev = R
        assert np.array_equal(sel["mask"][0], sel["mask"][1]) and np.array_equal(sel["mask"][1], sel["mask"][2])
