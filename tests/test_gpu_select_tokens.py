"""GPU parity of patchkv_select_repair_tokens (token-level Top-kappa, then block rounding) against the oracle."""
import numpy as np
import pytest
import torch

import oracle
import patchkv_inputs as pin
from gpu_common import DEV, new_context, staged

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module", params=[0, 1], ids=["pipeline", "direct_loads"])
def ctx(request):
    """Both per-token mass kernels run every case: rows staged through shared memory by bulk copies (regular shapes),
    and plain 128-bit loads (the only one for irregular shapes; forced by the flag otherwise)."""
    c = new_context(flags=request.param)
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


@pytest.mark.parametrize("L,Hq,Q,n", [(4, 8, 64, 4104), (2, 3, 8, 2048), (3, 2, 16, 6152), (1, 1, 8, 8)])
def test_token_mass_over_several_column_tiles_and_pieces(ctx, L, Hq, Q, n):
    """Shapes of the staged kernel whose per-CTA pieces of the (layer, column tile, batch of rows) list cross tile and
    layer boundaries (768 batches over 296 CTAs in the first case), with a ragged last column tile of 8 tokens."""
    from paper_2609_26219_b200 import binding as pk
    rng = np.random.default_rng(L * 1000 + n)
    logits = rng.normal(size=(L, Hq, Q, n)).astype(np.float32) * 3.0
    e = np.exp(logits - logits.max(axis=-1, keepdims=True))
    attn = (e / e.sum(axis=-1, keepdims=True)).astype(np.float16)
    attn[0, 0, 0, 0] = np.float16(1.0)                   # one entry outside the exact-fp32 fast paths
    attn[L - 1, Hq - 1, Q - 1, n - 1] = np.float16(0.25)
    rc, tmass = oracle.block_mass(attn, 1)
    assert rc == oracle.OK
    B = 8
    NB = -(-n // B)
    for mode in (0, 1):
        sel = oracle.select_tokens(tmass, B, 16, max(1, n // 64), mode)
        out = _outputs(L, NB)
        mass_out = torch.zeros((L, n), dtype=torch.int64, device=DEV)
        a = pk.select_args(kind=pk.SCORE_ATTN_F16, n_layers=L, n_suffix_tokens=n, block_tokens=B, dirty_tokens=16,
                           top_k=max(1, n // 64), layer_mode=mode, attn=torch.from_numpy(attn).to(DEV), mass_out=mass_out, **out)
        ctx.select_repair_tokens(a)
        _check(out, sel)
        assert np.array_equal(mass_out.cpu().numpy().astype(np.uint64), tmass)
        out2 = _outputs(L, NB)                            # and without mass_out: shared mode adds every layer into one row
        a2 = pk.select_args(kind=pk.SCORE_ATTN_F16, n_layers=L, n_suffix_tokens=n, block_tokens=B, dirty_tokens=16,
                            top_k=max(1, n // 64), layer_mode=mode, attn=torch.from_numpy(attn).to(DEV), **out2)
        ctx.select_repair_tokens(a2)
        _check(out2, sel)
    assert ctx.query_status() == 0


def test_token_mass_pipeline_leaves_cleanly_when_a_wait_runs_out():
    """The staged per-token mass kernel with one `empty` arrival withheld: the producer's bounded wait runs out, the
    kernel drains its copies and returns, PATCHKV_E_TIMEOUT is latched, and the next call is correct."""
    from paper_2609_26219_b200 import binding as pk
    c = new_context()
    try:
        rng = np.random.default_rng(3)
        L, Hq, Q, n, B = 4, 32, 64, 4096, 16               # 2048 batches of rows: about seven per CTA, the ring has three stages
        attn = (rng.random(size=(L, Hq, Q, n), dtype=np.float32) * 1e-3).astype(np.float16)
        rc, tmass = oracle.block_mass(attn, 1)
        sel = oracle.select_tokens(tmass, B, 32, 20, 0)
        dev_attn = torch.from_numpy(attn).to(DEV)
        out = _outputs(L, n // B)
        a = pk.select_args(kind=pk.SCORE_ATTN_F16, n_layers=L, n_suffix_tokens=n, block_tokens=B, dirty_tokens=32,
                           top_k=20, layer_mode=0, attn=dev_attn, **out)
        c.selftest_stall_next_launch(0, 2000)
        c.select_repair_tokens(a)
        assert c.query_status() == pk.E_TIMEOUT
        out = _outputs(L, n // B)
        a = pk.select_args(kind=pk.SCORE_ATTN_F16, n_layers=L, n_suffix_tokens=n, block_tokens=B, dirty_tokens=32,
                           top_k=20, layer_mode=0, attn=dev_attn, **out)
        c.select_repair_tokens(a)
        _check(out, sel)
        assert c.query_status() == 0
    finally:
        c.close()


def test_token_form_at_scale_full_size_sampled_layers(ctx):
    """Stored attention [32][32][64][16384] fp16 (2 GiB): per-token masses and the lists of the token-level selection
    compared on sampled layers (per-layer ranking), and the request-level ranking against the oracle's on all layers'
    summed masses."""
    from paper_2609_26219_b200 import binding as pk
    ck = pin.config_select_scale(device=DEV, n_layers=32)
    L, n, B = 32, ck.n_suffix_tokens, 16
    NB = n // B
    kappa = int(0.015 * n)
    mass_out = torch.zeros((L, n), dtype=torch.int64, device=DEV)
    out = _outputs(L, NB)
    a = pk.select_args(kind=pk.SCORE_ATTN_F16, n_layers=L, n_suffix_tokens=n, block_tokens=B, dirty_tokens=ck.dirty_tokens,
                       top_k=kappa, layer_mode=0, attn=ck.attn, mass_out=mass_out, **out)
    ctx.select_repair_tokens(a)
    torch.cuda.synchronize()
    assert ctx.query_status() == 0
    for l in (0, 13, 31):
        rc, tmass = oracle.block_mass(ck.attn[l:l + 1].cpu().numpy(), 1)
        assert rc == oracle.OK
        assert np.array_equal(mass_out[l].cpu().numpy().astype(np.uint64), tmass[0])
        sel = oracle.select_tokens(tmass, B, ck.dirty_tokens, kappa, 0)
        assert np.array_equal(out["repair_idx"][l].cpu().numpy(), sel["repair_idx"][0])
        assert np.array_equal(out["reuse_idx"][l].cpu().numpy(), sel["reuse_idx"][0])
    # request-level: the masses just checked on three layers are summed over all 32 by the library itself
    out2 = _outputs(L, NB)
    a2 = pk.select_args(kind=pk.SCORE_ATTN_F16, n_layers=L, n_suffix_tokens=n, block_tokens=B, dirty_tokens=ck.dirty_tokens,
                        top_k=kappa, layer_mode=1, attn=ck.attn, **out2)
    ctx.select_repair_tokens(a2)
    torch.cuda.synchronize()
    sel = oracle.select_tokens(mass_out.cpu().numpy().astype(np.uint64), B, ck.dirty_tokens, kappa, 1)
    _check(out2, sel)
    assert ctx.query_status() == 0


@pytest.mark.parametrize("case", ["tiny_keys", "distinct", "band_600", "band_3000", "all_equal", "huge_keys"])
def test_many_candidates_every_way_through_the_ranking(ctx, case):
    """With 4096 candidates or more the first cut of the ranking is a histogram of coarse key codes made by several
    CTAs; what is left is ranked from a list (directly when short, by radix passes when longer) or, when thousands of
    keys share the deciding code, by the passes over all candidates.  Each case is built to take one of those ways, with
    duplicates around the threshold so that the order of equal keys matters."""
    from paper_2609_26219_b200 import binding as pk
    rng = np.random.default_rng(sum(map(ord, case)))
    n, B, L = 8192, 16, 2
    if case == "tiny_keys":                               # every key below 64: the code is the key
        mass = rng.integers(0, 64, size=(L, n))
        kappa = 700
    elif case == "distinct":                              # keys spread over twenty octaves: a handful per code
        mass = (2.0 ** rng.uniform(4, 24, size=(L, n))).astype(np.int64)
        kappa = 123
    elif case in ("band_600", "band_3000"):               # a band of keys that share one code holds the threshold
        band = 600 if case == "band_600" else 3000
        mass = rng.integers(0, 1 << 20, size=(L, n))
        pos = rng.permutation(n)[:band]
        mass[:, pos] = (1 << 30) + (rng.integers(0, 40, size=(L, band)) << 12)
        kappa = band // 2
    elif case == "all_equal":
        mass = np.full((L, n), 12345, dtype=np.int64)
        kappa = 1000
    else:                                                 # keys with the top bit of 64 set (one layer: no sum to overflow)
        L = 1
        mass = rng.integers(0, 1 << 62, size=(L, n)).astype(np.uint64)
        mass[:, ::3] |= np.uint64(1 << 63)
        kappa = 2000
    mass = np.ascontiguousarray(mass.astype(np.uint64))
    for mode in (0, 1):
        sel = oracle.select_tokens(mass, B, 100, kappa, mode)
        out = _outputs(L, n // B)
        a = pk.select_args(kind=pk.SCORE_TOKEN_MASS, n_layers=L, n_suffix_tokens=n, block_tokens=B, dirty_tokens=100,
                           top_k=kappa, layer_mode=mode, mass=torch.from_numpy(mass.view(np.int64)).to(DEV), **out)
        ctx.select_repair_tokens(a)
        _check(out, sel)
    assert ctx.query_status() == 0


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
