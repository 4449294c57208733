"""Pins for the checker's binary32 -> bfloat16 rounding (CPU only).

The rounding is pinned by what the format fixes, not by itself: hand-worked patterns, the identity on every
bfloat16 pattern, a library conversion, the half-spacing bound and monotonicity.
"""
import os

import numpy as np
import torch

import oracle

GOLDEN = os.path.join(os.path.dirname(os.path.abspath(__file__)), "golden", "bf16_rounding_cases.txt")


def _from_bits32(bits):
    return np.array(bits, dtype=np.uint32).view(np.float32)


def test_hand_worked_patterns():
    src, want = [], []
    with open(GOLDEN) as f:
        for line in f:
            if line.startswith("#") or not line.strip():
                continue
            a, b, _ = [t.strip() for t in line.split(";")]
            src.append(int(a, 16))
            want.append(int(b, 16))
    assert len(src) >= 20
    bits, values = oracle.round_bf16(_from_bits32(src))
    assert [int(b) for b in bits] == want
    # the widened values are the patterns placed in the upper half of a binary32
    assert np.array_equal(values.view(np.uint32), np.array(want, dtype=np.uint32) << 16)


def test_every_bfloat16_value_is_a_fixed_point():
    pats = np.arange(1 << 16, dtype=np.uint32)
    x = (pats << 16).view(np.float32)
    bits, values = oracle.round_bf16(x)
    nan = np.isnan(x)
    assert np.array_equal(bits[~nan], pats[~nan].astype(np.uint16))
    assert np.all(np.isnan(values[nan])) and np.all((bits[nan] & 0x7FC0) == 0x7FC0)
    assert np.array_equal(bits[nan] >> 15, (pats[nan] >> 15).astype(np.uint16))        # NaN keeps its sign


def test_against_a_library_conversion():
    rng = np.random.default_rng(7)
    # random patterns cover every exponent, subnormals and both signs; NaNs are compared as NaNs
    x = rng.integers(0, 1 << 32, size=1_000_000, dtype=np.uint64).astype(np.uint32).view(np.float32)
    # plus a dense sweep across ties: every pattern whose discarded half is 7FFF, 8000 or 8001
    top = rng.integers(0, 1 << 16, size=30_000, dtype=np.uint64).astype(np.uint32) << 16
    ties = np.concatenate([top | 0x7FFF, top | 0x8000, top | 0x8001]).view(np.float32)
    x = np.concatenate([x, ties])
    bits, values = oracle.round_bf16(x)
    lib = torch.from_numpy(x).to(torch.bfloat16)
    lib_bits = lib.view(torch.int16).numpy().view(np.uint16)
    ok = ~np.isnan(x)
    assert np.array_equal(bits[ok], lib_bits[ok])
    assert np.all(np.isnan(values[~ok])) and bool(torch.isnan(lib[torch.from_numpy(~ok)]).all())


def test_half_ulp_bound_and_monotonicity():
    rng = np.random.default_rng(11)
    x = np.sort((rng.standard_normal(200_000) * np.exp(rng.uniform(-20, 20, 200_000))).astype(np.float32))
    _, v = oracle.round_bf16(x)
    xd, vd = x.astype(np.float64), v.astype(np.float64)
    # normal range: 8 significant bits, spacing 2^(e-7) in [2^e, 2^(e+1)), so |r(x) - x| <= 2^(e-8) <= 2^-8 |x|,
    # and the bound is reached only at ties, never exceeded; on average the error is far smaller
    assert np.all(np.abs(vd - xd) <= 2.0 ** -8 * np.abs(xd))
    e = np.floor(np.log2(np.abs(xd)))
    assert np.all(np.abs(vd - xd) <= 2.0 ** (e - 8))
    assert np.all(np.diff(vd) >= 0)                                  # rounding never reorders values
    # the result has at most 8 significant bits: the low 16 bits of its binary32 pattern are zero
    assert np.all((v.view(np.uint32) & 0xFFFF) == 0)
    # idempotent
    _, v2 = oracle.round_bf16(v)
    assert np.array_equal(v2, v)


def test_a_planted_mistake_would_be_caught():
    """Truncation instead of rounding, and ties rounded up instead of to even, both fail the golden cases."""
    src = np.array([0x3F808001, 0x3F808000], dtype=np.uint32)
    bits, _ = oracle.round_bf16(src.view(np.float32))
    truncated = (src >> 16).astype(np.uint16)
    ties_up = ((src + 0x8000) >> 16).astype(np.uint16)
    assert not np.array_equal(bits, truncated) and not np.array_equal(bits, ties_up)
