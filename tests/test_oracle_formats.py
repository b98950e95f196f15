"""Pins for the oracle's number formats: the paper's printed value set and
maxima, torch's own float8 / bfloat16 conversions (a library routine the
oracle does not use), brute force, and structural invariants."""
import os

import numpy as np
import torch

from oracle import formats as F

GOLD = os.path.join(os.path.dirname(__file__), "golden")


def _read_numbers(name):
    with open(os.path.join(GOLD, name)) as fh:
        lines = [ln for ln in fh if not ln.startswith("#") and ln.strip()]
    return lines


def test_e2m1_table_is_the_papers_set():
    vals = [float(v) for v in _read_numbers("e2m1_magnitudes.txt")[0].split()]
    assert list(F.E2M1_MAGNITUDES) == vals
    # both signs: 16 codes, bit 3 is the sign
    dec = F.e2m1_decode(np.arange(16))
    assert list(dec[:8]) == vals and list(dec[8:]) == [-v for v in vals]


def test_e4m3_facts_from_paper():
    facts = dict(ln.split() for ln in _read_numbers("e4m3_facts.txt"))
    assert F.E4M3_EXP_BITS == int(facts["exp_bits"]) and F.E4M3_MAN_BITS == int(facts["man_bits"])
    assert 1 + F.E4M3_EXP_BITS + F.E4M3_MAN_BITS == int(facts["bits"])
    assert F.E4M3_MAX == float(facts["max"])
    assert F.e4m3_decode(0x7E) == 448.0
    assert np.isnan(F.e4m3_decode(0x7F)) and np.isnan(F.e4m3_decode(0xFF))


def test_e4m3_decode_matches_torch_float8():
    codes = np.arange(256, dtype=np.uint8)
    ours = F.e4m3_decode(codes)
    ref = torch.from_numpy(codes).view(torch.float8_e4m3fn).to(torch.float64).numpy()
    ok = ~np.isnan(ref)
    assert ok.sum() == 254
    assert np.array_equal(ours[ok], ref[ok])
    assert np.all(np.isnan(ours[~ok]))


def test_e4m3_encode_matches_torch_float8_in_range():
    rng = np.random.default_rng(0)
    mags = F.E4M3_MAGNITUDES
    mids = 0.5 * (mags[:-1] + mags[1:])
    vals = np.concatenate([
        mags, mids, np.nextafter(mids.astype(np.float32), np.float32(0)),
        np.nextafter(mids.astype(np.float32), np.float32(1e9)),
        rng.uniform(0, 448, 20000), np.exp(rng.uniform(np.log(1e-5), np.log(448), 20000)),
    ]).astype(np.float32)
    vals = np.concatenate([vals, -vals])
    ours = F.e4m3_encode(vals)
    ref = torch.from_numpy(vals).to(torch.float8_e4m3fn).view(torch.uint8).numpy()
    assert np.array_equal(ours, ref)


def test_e4m3_saturates_instead_of_nan():
    assert F.e4m3_encode(np.float32(448.0)) == 0x7E
    assert F.e4m3_encode(np.float32(464.0)) == 0x7E      # the would-be tie to 480
    assert F.e4m3_encode(np.float32(1e30)) == 0x7E
    assert F.e4m3_encode(np.float32(-1e30)) == 0xFE


def test_roundtrip_every_code():
    c4 = np.arange(16, dtype=np.uint8)
    assert np.array_equal(F.e2m1_encode(F.e2m1_decode(c4).astype(np.float32)), c4)
    c8 = np.array([c for c in range(256) if c & 0x7F != 0x7F], dtype=np.uint8)
    assert np.array_equal(F.e4m3_encode(F.e4m3_decode(c8).astype(np.float32)), c8)


def test_e2m1_ties_go_to_even_mantissa():
    # midpoint -> expected magnitude (the neighbour whose mantissa bit is 0)
    ties = {0.25: 0.0, 0.75: 1.0, 1.25: 1.0, 1.75: 2.0, 2.5: 2.0, 3.5: 4.0, 5.0: 4.0}
    for v, want in ties.items():
        for s in (1.0, -1.0):
            got = F.e2m1_decode(F.e2m1_encode(np.float32(s * v)))
            assert got == s * want or (want == 0 and got == 0), (v, got)
            below = np.nextafter(np.float32(v), np.float32(0))
            above = np.nextafter(np.float32(v), np.float32(100))
            lo = max(m for m in F.E2M1_MAGNITUDES if m < v)
            hi = min(m for m in F.E2M1_MAGNITUDES if m > v)
            assert abs(F.e2m1_decode(F.e2m1_encode(np.float32(s * below)))) == lo
            assert abs(F.e2m1_decode(F.e2m1_encode(np.float32(s * above)))) == hi
    assert F.e2m1_encode(np.float32(100.0)) == 7 and F.e2m1_encode(np.float32(-7.0)) == 15
    # the sign bit is copied even when the magnitude rounds to zero
    assert F.e2m1_encode(np.float32(-0.0)) == 8 and F.e2m1_encode(np.float32(-0.1)) == 8


def test_encode_is_brute_force_nearest_and_monotone():
    rng = np.random.default_rng(1)
    v = np.concatenate([rng.uniform(-7, 7, 4000), rng.normal(0, 1, 4000)]).astype(np.float32)
    got = F.e2m1_decode(F.e2m1_encode(v))
    table = np.concatenate([-F.E2M1_MAGNITUDES[::-1], F.E2M1_MAGNITUDES])
    for x, g in zip(v.astype(np.float64), got):
        assert abs(x - g) == np.min(np.abs(table - x))       # nearest (ties: equal distance)
    s = np.sort(v)
    assert np.all(np.diff(F.e2m1_decode(F.e2m1_encode(s))) >= 0)
    u = np.sort(np.exp(rng.uniform(np.log(1e-4), np.log(500), 5000))).astype(np.float32)
    d = F.e4m3_decode(F.e4m3_encode(u))
    assert np.all(np.diff(d) >= 0)
    t8 = F.E4M3_MAGNITUDES
    for x, g in zip(u.astype(np.float64)[::10], d[::10]):
        assert abs(x - g) == np.min(np.abs(t8 - x))


def test_bf16_round_matches_torch():
    rng = np.random.default_rng(2)
    x = np.concatenate([rng.normal(0, 1, 50000), rng.normal(0, 1e-3, 1000),
                        np.exp(rng.uniform(-60, 60, 5000))]).astype(np.float32)
    # exact ties: bf16 midpoints are float32 with low half 0x8000
    base = (rng.integers(0, 2 ** 12, 2000).astype(np.uint32) << 16) + np.uint32(0x3F000000)
    ties = (base | np.uint32(0x8000)).view(np.float32)
    x = np.concatenate([x, ties, -ties])
    ours = F.bf16_round(x)
    ref = torch.from_numpy(x).to(torch.bfloat16).to(torch.float32).numpy()
    assert np.array_equal(ours.view(np.uint32), ref.view(np.uint32))
    # float64 input that would double-round through float32
    y = np.float64(1.0) + 2.0 ** -8 + 2.0 ** -40          # just above a bf16 midpoint
    assert F.bf16_round(y) == np.float32(1.0 + 2.0 ** -7)
    y = np.float64(1.0) + 2.0 ** -8 - 2.0 ** -40
    assert F.bf16_round(y) == np.float32(1.0)
    assert np.array_equal(F.bf16_from_bits(F.bf16_bits(ours)), ours)


def test_nibble_packing_roundtrip():
    rng = np.random.default_rng(3)
    c = rng.integers(0, 16, (5, 32)).astype(np.uint8)
    p = F.pack_nibbles(c)
    assert p.shape == (5, 16)
    assert p[0, 0] == (c[0, 0] | (c[0, 1] << 4))
    assert np.array_equal(F.unpack_nibbles(p), c)
