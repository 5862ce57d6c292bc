"""GPU parity of patchkv_select_repair_tokens (token-level Top-kappa, then block rounding) against the oracle."""
import numpy as np
import pytest
import torch

import oracle
import patchkv_inputs as pin
from gpu_common import DEV, new_context, staged

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def ctx():
    c = new_context()
    yield c
    c.close()


def _outputs(L, NB):
    return dict(repair_mask=torch.full((L, NB), 9, dtype=torch.uint8, device=DEV),
                repair_idx=torch.full((L, NB), -7, dtype=torch.int32, device=DEV),
                repair_cnt=torch.full((L,), -7, dtype=torch.int32, device=DEV),
                reuse_idx=torch.full((L, NB), -7, dtype=torch.int32, device=DEV),
                reuse_cnt=torch.full((L,), -7, dtype=torch.int32, device=DEV))


def _check(out, sel):
    torch.cuda.synchronize()
    assert np.array_equal(out["repair_mask"].cpu().numpy(), sel["mask"])
    assert np.array_equal(out["repair_idx"].cpu().numpy(), sel["repair_idx"])
    assert np.array_equal(out["reuse_idx"].cpu().numpy(), sel["reuse_idx"])
    assert np.array_equal(out["repair_cnt"].cpu().numpy(), sel["repair_cnt"])
    assert np.array_equal(out["reuse_cnt"].cpu().numpy(), sel["reuse_cnt"])


@pytest.mark.parametrize("n,B,d_hat,kappa,mode", [(1024, 16, 90, 15, 1), (1000, 16, 90, 15, 0), (1024, 32, 64, 40, 1),
                                                 (777, 24, 0, 5, 1), (1024, 16, -4, 0, 1), (1024, 16, 5000, 3, 0),
                                                 (1024, 16, 10, 5000, 1), (9, 16, 0, 2, 0)])
def test_from_attention(ctx, n, B, d_hat, kappa, mode):
    from paper_2609_26219_b200 import binding as pk
    ck = pin.config_tiny(n=n, n_pages=512)
    attn = ck.attn.to(DEV)
    rc, tmass = oracle.block_mass(ck.attn.numpy(), 1)
    sel = oracle.select_tokens(tmass, B, d_hat, kappa, mode)
    NB = -(-n // B)
    out = _outputs(2, NB)
    mass_out = torch.zeros((2, n), dtype=torch.int64, device=DEV)
    a = pk.select_args(kind=pk.SCORE_ATTN_F16, n_layers=2, n_suffix_tokens=n, block_tokens=B, dirty_tokens=d_hat,
                       top_k=kappa, layer_mode=mode, attn=attn, mass_out=mass_out, **out)
    ctx.select_repair_tokens(a)
    _check(out, sel)
    assert np.array_equal(mass_out.cpu().numpy().astype(np.uint64), tmass)
    a2 = pk.select_args(kind=pk.SCORE_ATTN_F16, n_layers=2, n_suffix_tokens=n, block_tokens=B, dirty_tokens=d_hat,
                        top_k=kappa, layer_mode=mode, attn=attn, **_outputs(2, NB))
    out2 = _outputs(2, NB)
    a2 = pk.select_args(kind=pk.SCORE_ATTN_F16, n_layers=2, n_suffix_tokens=n, block_tokens=B, dirty_tokens=d_hat,
                        top_k=kappa, layer_mode=mode, attn=attn, **out2)
    ctx.select_repair_tokens(a2)          # masses kept in the workspace
    _check(out2, sel)
    assert ctx.query_status() == 0


def test_from_token_mass_long_suffix_with_ties(ctx):
    """64k-token suffix, 3 layers, 1.5 % of the tokens selected (the paper's operating point), many equal scores."""
    from paper_2609_26219_b200 import binding as pk
    rng = np.random.default_rng(8)
    n, B, L = 65536, 32, 3
    mass = rng.integers(0, 500, size=(L, n)).astype(np.int64)
    kappa = int(0.015 * n)
    for mode in (0, 1):
        sel = oracle.select_tokens(mass.astype(np.uint64), B, 64, kappa, mode)
        out = _outputs(L, n // B)
        a = pk.select_args(kind=pk.SCORE_TOKEN_MASS, n_layers=L, n_suffix_tokens=n, block_tokens=B, dirty_tokens=64,
                           top_k=kappa, layer_mode=mode, mass=torch.from_numpy(mass).to(DEV), **out)
        ctx.select_repair_tokens(a)
        _check(out, sel)


def test_token_form_and_block_form_differ_on_the_constructed_case(ctx):
    from paper_2609_26219_b200 import binding as pk
    n, B = 128, 16
    mass = np.ones((1, n), dtype=np.int64)
    mass[0, 5 * B + 3] = 1000
    mass[0, 2 * B + 1] = 600
    mass[0, 2 * B + 9] = 600
    out = _outputs(1, n // B)
    a = pk.select_args(kind=pk.SCORE_TOKEN_MASS, n_layers=1, n_suffix_tokens=n, block_tokens=B, dirty_tokens=0,
                       top_k=1, layer_mode=0, mass=torch.from_numpy(mass).to(DEV), **out)
    ctx.select_repair_tokens(a)
    torch.cuda.synchronize()
    assert out["repair_idx"][0, 0].item() == 5 and out["repair_cnt"][0].item() == 1
    bm = torch.from_numpy(mass.reshape(1, n // B, B).sum(axis=2)).to(DEV)
    out_b = _outputs(1, n // B)
    b = pk.select_args(kind=pk.SCORE_BLOCK_MASS, n_layers=1, n_suffix_tokens=n, block_tokens=B, dirty_tokens=0,
                       top_k=1, layer_mode=0, mass=bm, **out_b)
    ctx.select_repair(b)
    torch.cuda.synchronize()
    assert out_b["repair_idx"][0, 0].item() == 2
    bad = pk.select_args(kind=pk.SCORE_BLOCK_MASS, n_layers=1, n_suffix_tokens=n, block_tokens=B, dirty_tokens=0,
                         top_k=1, layer_mode=0, mass=bm, **out_b)
    assert ctx.select_repair_tokens(bad, check=False) == pk.E_INVALID


def test_strided_and_unaligned_attention(ctx):
    from paper_2609_26219_b200 import binding as pk
    ck = pin.config_tiny()
    rc, tmass = oracle.block_mass(ck.attn.numpy(), 1)
    sel = oracle.select_tokens(tmass, 16, 90, 15, 1)
    big = torch.zeros((2, 8, 16, 1024 + 3), dtype=torch.float16, device=DEV)
    big[..., 3:] = ck.attn.to(DEV)
    wide = torch.zeros((2, 16, 16, 1024), dtype=torch.float16, device=DEV)
    wide[:, ::2] = ck.attn.to(DEV)
    for view in (big[..., 3:], wide[:, ::2]):
        out = _outputs(2, 64)
        mass_out = torch.zeros((2, 1024), dtype=torch.int64, device=DEV)
        a = pk.select_args(kind=pk.SCORE_ATTN_F16, n_layers=2, n_suffix_tokens=1024, block_tokens=16, dirty_tokens=90,
                           top_k=15, layer_mode=1, attn=view, mass_out=mass_out, **out)
        ctx.select_repair_tokens(a)
        _check(out, sel)
        assert np.array_equal(mass_out.cpu().numpy().astype(np.uint64), tmass)


@pytest.mark.parametrize("Q", [70, 72])
def test_token_mass_over_the_whole_fp16_range_and_bad_entries(ctx, Q):
    """Q = 72 takes the kernel's regular row loop (batches of eight rows inside one head), Q = 70 the general one."""
    from paper_2609_26219_b200 import binding as pk
    rng = np.random.default_rng(5)
    bits = rng.integers(0, 0x7C00, size=(2, 3, Q, 512)).astype(np.uint16)
    bits[0, 0, 0, 3] = 0xBC00       # -1.0
    bits[1, 2, 5, 40] = 0x7E00      # NaN
    rc, tmass = oracle.block_mass(bits, 1)
    assert rc == oracle.E_BADINPUT
    sel = oracle.select_tokens(tmass, 16, 33, 20, 0)
    out = _outputs(2, 32)
    mass_out = torch.zeros((2, 512), dtype=torch.int64, device=DEV)
    a = pk.select_args(kind=pk.SCORE_ATTN_F16, n_layers=2, n_suffix_tokens=512, block_tokens=16, dirty_tokens=33,
                       top_k=20, layer_mode=0, attn=torch.from_numpy(bits.view(np.float16).copy()).to(DEV),
                       mass_out=mass_out, **out)
    ctx.select_repair_tokens(a)
    _check(out, sel)
    assert np.array_equal(mass_out.cpu().numpy().astype(np.uint64), tmass)
    assert ctx.query_status() == -7


def test_token_level_normalised_score(ctx):
    """score_out of the token form: one fp32 per token, request-level (layers summed) and per layer."""
    from paper_2609_26219_b200 import binding as pk
    ck = pin.config_tiny()
    rc, tmass = oracle.block_mass(ck.attn.numpy(), 1)
    for mode in (1, 0):
        want = oracle.normalise(tmass, mode)
        out = _outputs(2, 64)
        score = torch.full((2, 1024), -1.0, dtype=torch.float32, device=DEV)
        a = pk.select_args(kind=pk.SCORE_ATTN_F16, n_layers=2, n_suffix_tokens=1024, block_tokens=16, dirty_tokens=90,
                           top_k=15, layer_mode=mode, attn=ck.attn.to(DEV), score_out=score, **out)
        ctx.select_repair_tokens(a)
        _check(out, oracle.select_tokens(tmass, 16, 90, 15, mode))
        got = score.cpu().numpy()
        if mode == 1:
            assert np.array_equal(got[0].view(np.uint32), want.view(np.uint32)) and np.all(got[1] == -1.0)
        else:
            assert np.array_equal(got.view(np.uint32), want.view(np.uint32))
