"""Pins of the oracle's number formats, quantised codes and record sizes (CPU only)."""
import os
from fractions import Fraction

import numpy as np
import pytest
import torch

import oracle

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def test_fp16_to_f32_all_patterns_match_numpy():
    h = np.arange(65536, dtype=np.uint16)
    got = oracle.fp16_to_f32_array(h)
    want = h.view(np.float16).astype(np.float32)
    nan = np.isnan(want)
    assert np.array_equal(np.isnan(got), nan)
    assert np.array_equal(got.view(np.uint32)[~nan], want.view(np.uint32)[~nan])


def test_bf16_rne_halfway_cases_and_neighbours():
    # every exact halfway point of the binade [1, 2): ties go to the even 7-bit mantissa
    for m in range(128):
        lo = 0x3F80 + m
        mid = np.array([(lo << 16) | 0x8000], dtype=np.uint32)
        want_tie = lo if (lo & 1) == 0 else lo + 1
        assert oracle.f32_to_bf16_array(mid.view(np.float32))[0] == want_tie
        below = (mid - 1).view(np.float32)
        above = (mid + 1).view(np.float32)
        assert oracle.f32_to_bf16_array(below)[0] == lo
        assert oracle.f32_to_bf16_array(above)[0] == lo + 1


def test_bf16_rne_special_values():
    f = oracle.f32_to_bf16
    assert f(0.0) == 0x0000 and f(-0.0) == 0x8000
    assert f(float("inf")) == 0x7F80 and f(float("-inf")) == 0xFF80
    maxf = np.array([0x7F7FFFFF], dtype=np.uint32).view(np.float32)   # max finite fp32 rounds up to inf
    assert oracle.f32_to_bf16_array(maxf)[0] == 0x7F80
    sub = np.array([0x00000001, 0x00008000, 0x00008001, 0x00018000], dtype=np.uint32).view(np.float32)
    assert list(oracle.f32_to_bf16_array(sub)) == [0x0000, 0x0000, 0x0001, 0x0002]
    nan = oracle.f32_to_bf16(float("nan"))
    assert (nan & 0x7F80) == 0x7F80 and (nan & 0x007F) != 0


def test_bf16_rne_matches_torch_on_random_bit_patterns():
    rng = np.random.default_rng(7)
    bits = rng.integers(0, 2 ** 32, size=1 << 24, dtype=np.uint64).astype(np.uint32)
    x = bits.view(np.float32)
    got = oracle.f32_to_bf16_array(x)
    want = torch.from_numpy(x.copy()).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)
    ok = ~np.isnan(x)
    assert np.array_equal(got[ok], want[ok])
    assert np.all((got[~ok] & 0x7F80) == 0x7F80) and np.all((got[~ok] & 0x7F) != 0)


def test_f32_to_fp16_matches_numpy():
    rng = np.random.default_rng(8)
    x = np.concatenate([
        rng.standard_normal(1 << 20).astype(np.float32) * np.float32(10.0) ** rng.integers(-9, 6, 1 << 20).astype(np.float32),
        np.array([0.0, -0.0, 65504.0, 65519.99, 65520.0, 65536.0, 1e9, 2.0 ** -24, 2.0 ** -25, 1.5 * 2.0 ** -25,
                  2.0 ** -14, (1 - 2.0 ** -11) * 2.0 ** -14, np.inf, -np.inf], dtype=np.float32)])
    # add every fp16 value and the midpoints between neighbours
    h = np.arange(0x7C00, dtype=np.uint16).view(np.float16).astype(np.float32)
    x = np.concatenate([x, h, (h[:-1] + h[1:]) / 2, -h]).astype(np.float32)
    got = oracle.f32_to_fp16_array(x)
    with np.errstate(over="ignore"):
        want = x.astype(np.float16).view(np.uint16)
    assert np.array_equal(got, want)


@pytest.mark.parametrize("qmax", [127, 7])
def test_dequantise_is_the_exact_rational_product(qmax):
    rng = np.random.default_rng(9)
    for _ in range(200):
        s_bits = int(rng.integers(1, 0x7C00))            # any positive finite fp16 scale
        q = rng.integers(-qmax - 1, qmax + 1, size=32).astype(np.int8)
        x = oracle.dequantise_group(q, s_bits)
        e, m = (s_bits >> 10) & 31, s_bits & 1023
        s_exact = Fraction(m, 2 ** 24) if e == 0 else Fraction(1024 + m, 2 ** 10) * Fraction(2) ** (e - 15)
        for qi, xi in zip(q, x):
            assert Fraction(float(xi)) == int(qi) * s_exact


@pytest.mark.parametrize("qmax", [127, 7])
def test_quantise_dequantise_round_trip_is_exact(qmax):
    """Codes with a +-qmax in the group and any positive fp16 scale survive dequantise -> quantise unchanged."""
    rng = np.random.default_rng(10)
    for _ in range(500):
        s_bits = int(rng.integers(1, 0x7C00))
        if oracle.fp16_to_f32(s_bits) * qmax >= 3.0e38:
            continue
        q = rng.integers(-qmax, qmax + 1, size=32).astype(np.int8)
        q[int(rng.integers(32))] = qmax if rng.integers(2) else -qmax
        x = oracle.dequantise_group(q, s_bits)
        q2, s2 = oracle.quantise_group(x, qmax)
        assert s2 == s_bits
        assert np.array_equal(q2, q)


def test_quantise_zero_group_gives_zero_scale_and_codes():
    q, s = oracle.quantise_group(np.zeros(32, dtype=np.float32), 127)
    assert s == 0 and not q.any()


def test_record_sizes_closed_forms():
    # 16-token blocks, group 32 (the benchmark geometry): sizes fixed by the layout description
    assert oracle.record_bytes(0, 16, 8, 128, 32) == 65536
    assert oracle.record_bytes(1, 16, 8, 128, 32) == 34816
    assert oracle.record_bytes(2, 16, 8, 128, 32) == 26624
    assert oracle.record_bytes(3, 16, 8, 128, 32) == 18432
    assert oracle.record_bytes(0, 16, 4, 64, 32) == 16384
    assert oracle.record_bytes(1, 16, 4, 64, 32) == 8704
    assert oracle.record_bytes(2, 16, 4, 64, 32) == 6656
    assert oracle.record_bytes(4, 16, 4, 64, 32) == 0 and oracle.record_bytes(-1, 16, 4, 64, 32) == 0


def test_record_sizes_reproduce_the_papers_payload_ratios():
    """One fp16 scale per 128-channel vector reproduces the printed INT8/FP16 and INT4/FP16 payload ratios
    to within the metadata residual (under half a percent of the FP16 payload)."""
    rows = {}
    for line in open(os.path.join(GOLDEN, "payload_mib.txt")):
        if line.strip() and not line.startswith("#"):
            name, mib, ms = line.split()
            rows[name] = float(mib)
    fp16 = oracle.record_bytes(0, 32, 8, 128, 128)
    int8 = oracle.record_bytes(1, 32, 8, 128, 128)
    int4 = oracle.record_bytes(3, 32, 8, 128, 128)
    assert abs(int8 / fp16 - rows["INT8"] / rows["FP16"]) < 0.005
    assert abs(int4 / fp16 - rows["INT4"] / rows["FP16"]) < 0.005
    # the mixed K8/V4 tier sits strictly between them
    assert int4 < oracle.record_bytes(2, 32, 8, 128, 128) < int8
