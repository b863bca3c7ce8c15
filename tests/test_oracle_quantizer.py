"""Pins for the oracle's group quantiser (CPU only).

Nothing here re-types the oracle's formulas: expected values are derived by hand from
the paper's equations (Section "Asymmetric and Symmetric Quantization", Section "Hybrid
Quantization"), or are properties any correct implementation must have (nearest level,
error bound, exactness on representable grids, brute force over both modes).
"""
import itertools
import os

import numpy as np
import pytest

from oracle import innerq_oracle as O

f32 = np.float32


def h2bits(x):
    return int(np.array(x, dtype=np.float16).view(np.uint16))


def q(x, bits=2, mode=O.HYBRID, variant=O.FULLRANGE):
    return O.quantize_groups(np.array(x, dtype=f32), bits, mode, variant)


# ---------------------------------------------------------------- hand-derived vectors
def test_hand_vector_positive_ramp_prefers_asym():
    # G = {0.5, 1, 1.5, 2}, b = 2.  Asym: Z = 0.5, S = (2 - 0.5)/3 = 0.5, codes 0..3, exact.
    # Sym (3 levels -S, 0, S with S = 2): 0.25 -> 0, 0.5 -> 0 (half-to-even), 0.75 -> 1, 1 -> 1;
    # reconstruction {0, 0, 2, 2}, L1 error 0.5 + 1 + 0.5 + 0 = 2.  So M = 1.
    r = q([0.5, 1.0, 1.5, 2.0])
    assert bool(r["flag"]) is True
    assert r["code"].tolist() == [0, 1, 2, 3]
    assert int(r["scale_bits"]) == (h2bits(0.5) | 0x8000)       # M lives in the scale's sign bit
    assert int(r["zero_bits"]) == h2bits(0.5)
    assert r["err_asym"] == 0.0 and r["err_sym"] == pytest.approx(2.0)


def test_hand_vector_symmetric_group_prefers_sym():
    # G = {-1, 0, 0, 1}, b = 2.  Sym: S = 1, q = {-1, 0, 0, 1}, exact.  Offset-binary u = q + 2.
    # Asym: Z = -1, S = fp16(2/3) = 0x3955 = 0.66650390625; (x+1)/S = {0, 1.5004, 1.5004, 3.0007}
    # -> codes {0, 2, 2, 3}; error on the two zeros = |0 - (2*S - 1)| = 0.33301 each, on 1: 0.00049.
    r = q([-1.0, 0.0, 0.0, 1.0])
    assert bool(r["flag"]) is False
    assert r["code"].tolist() == [1, 2, 2, 3]
    assert int(r["scale_bits"]) == h2bits(1.0)
    assert int(r["zero_bits"]) == 0                              # Z = 0 when M = 0 (Figure "hybrid", third mux)
    assert r["err_sym"] == 0.0
    S = float(np.float16(2.0 / 3.0))
    assert S == 0.66650390625
    assert r["err_asym"] == pytest.approx(2 * abs(2 * S - 1) + abs(3 * S - 2))
    ra = q([-1.0, 0.0, 0.0, 1.0], mode=O.ASYM)
    assert ra["code"].tolist() == [0, 2, 2, 3] and int(ra["scale_bits"]) == (0x3955 | 0x8000)
    assert int(ra["zero_bits"]) == h2bits(-1.0)


def test_hand_vector_bits_change_the_choice():
    # {-3, -1, 1, 3}: at b = 2 asym is exact (Z = -3, S = 2) while sym (S = 3) maps +-1 to 0 -> M = 1.
    # At b = 3 sym has levels -3..3 with S = 1 and is exact; asym has S = fp16(6/7), inexact -> M = 0.
    r2 = q([-3.0, -1.0, 1.0, 3.0], bits=2)
    assert bool(r2["flag"]) and r2["code"].tolist() == [0, 1, 2, 3] and r2["err_sym"] == pytest.approx(2.0)
    r3 = q([-3.0, -1.0, 1.0, 3.0], bits=3)
    assert not bool(r3["flag"]) and r3["code"].tolist() == [1, 3, 5, 7]   # q + 4
    assert r3["err_sym"] == 0.0 and r3["err_asym"] > 0.0


def test_constant_and_zero_groups():
    # constant group: asym S = 0, Z = 1.5, codes 0, exact; sym S = 1.5, q = 1, exact; tie -> sym.
    r = q([1.5] * 4)
    assert not bool(r["flag"]) and r["code"].tolist() == [3, 3, 3, 3] and int(r["scale_bits"]) == h2bits(1.5)
    ra = q([1.5] * 4, mode=O.ASYM)
    assert ra["code"].tolist() == [0, 0, 0, 0] and int(ra["scale_bits"]) == 0x8000   # -0.0: flag on a zero scale
    assert int(ra["zero_bits"]) == h2bits(1.5)
    assert np.all(O.dequantize_groups(ra["code"], ra["scale_bits"], ra["zero_bits"], 2) == 1.5)
    rz = q([0.0] * 4)
    assert rz["code"].tolist() == [2, 2, 2, 2] and int(rz["scale_bits"]) == 0 and int(rz["zero_bits"]) == 0
    assert np.all(O.dequantize_groups(rz["code"], rz["scale_bits"], rz["zero_bits"], 2) == 0.0)


def test_paper_literal_symmetric_variant_clips():
    # S = max|G|/(2^b - 1) as printed: fp16(1/3) = 0.333251953125; -1/S = -3.0007 -> -3, clipped to the
    # signed 2-bit minimum -2; +1/S -> 3, clipped to +1.
    r = q([-1.0, 0.0, 0.0, 1.0], mode=O.SYM, variant=O.PAPER_LITERAL)
    assert float(np.array(r["scale_bits"], dtype=np.uint16).view(np.float16)) == 0.333251953125
    assert (r["code"].astype(int) - 2).tolist() == [-2, 0, 0, 1]


# ---------------------------------------------------------------- properties
def _rand_groups(seed, n, G, kind):
    g = np.random.default_rng(seed)
    x = g.standard_normal((n, G)).astype(f32)
    if kind == "shifted":
        x = x + g.uniform(-4, 4, size=(n, 1)).astype(f32)
    if kind == "fp16grid":
        x = x.astype(np.float16).astype(f32)
    if kind == "heavy":
        x = (x / np.sqrt(g.chisquare(4, size=(n, G)) / 4)).astype(f32)
    return x


@pytest.mark.parametrize("bits", [2, 3, 4])
@pytest.mark.parametrize("G", [32, 64, 128])
@pytest.mark.parametrize("kind", ["plain", "shifted", "fp16grid", "heavy"])
def test_asym_endpoints_bound_and_nearest_level(bits, G, kind):
    x = _rand_groups(bits * 100 + G, 200, G, kind)
    r = O.quantize_groups(x, bits, O.ASYM)
    L = 2 ** bits - 1
    s = (r["scale_bits"] & 0x7FFF).view(np.float16).astype(np.float64)
    Z = r["zero_bits"].view(np.float16).astype(np.float64)
    xh = O.dequantize_groups(r["code"], r["scale_bits"], r["zero_bits"], bits)
    assert np.all(r["scale_bits"] & 0x8000)
    # code(min) = 0, code(max) = L, dequant(min) = Z exactly
    imin, imax = x.argmin(1), x.argmax(1)
    rows = np.arange(len(x))
    assert np.all(r["code"][rows, imin] == 0) and np.all(r["code"][rows, imax] == L)
    assert np.all(xh[rows, imin] == Z)
    # Z and S are what the paper defines, up to fp16 rounding
    assert np.all(Z == x.min(1).astype(np.float16).astype(np.float64))
    assert np.allclose(s, (x.max(1).astype(np.float64) - x.min(1)) / L, rtol=2 ** -10, atol=2 ** -24)
    # |x - x^| <= S/2 (+ the fp16 rounding of Z and S themselves; the last level may sit
    # up to L * ulp(S)/2 below the maximum)
    slack = s[:, None] * 2 ** -9 * L + np.abs(Z)[:, None] * 2 ** -10 + 1e-7
    assert np.all(np.abs(x - xh) <= s[:, None] / 2 + slack)
    # brute force: no other level is closer (up to rounding ties)
    levels = s[:, None, None] * np.arange(L + 1)[None, None, :] + Z[:, None, None]
    best = np.abs(x[:, :, None].astype(np.float64) - levels).min(-1)
    assert np.all(np.abs(x - xh) <= best + s[:, None] * 1e-5 + 1e-9)


@pytest.mark.parametrize("bits", [2, 3, 4])
@pytest.mark.parametrize("kind", ["plain", "shifted", "heavy"])
def test_sym_fullrange_bound_zero_and_extremes(bits, kind):
    G = 32
    x = _rand_groups(7 + bits, 300, G, kind)
    x[:, 5] = 0.0
    r = O.quantize_groups(x, bits, O.SYM, O.FULLRANGE)
    den = 2 ** (bits - 1) - 1
    s = r["scale_bits"].view(np.float16).astype(np.float64)
    assert not np.any(r["scale_bits"] & 0x8000) and not np.any(r["zero_bits"])
    xh = O.dequantize_groups(r["code"], r["scale_bits"], r["zero_bits"], bits)
    qs = r["code"].astype(int) - 2 ** (bits - 1)
    assert qs.min() >= -den and qs.max() <= den
    assert np.all(xh[:, 5] == 0.0)                                  # zero is a level
    iam = np.abs(x).argmax(1)
    rows = np.arange(len(x))
    assert np.all(qs[rows, iam] == den * np.sign(x[rows, iam]))      # +-max|G| hits the end level
    assert np.allclose(s, np.abs(x).max(1).astype(np.float64) / den, rtol=2 ** -10)
    assert np.all(np.abs(x - xh) <= s[:, None] / 2 * (1 + 2 ** -9 * den * 2) + 1e-7)
    levels = s[:, None, None] * np.arange(-den, den + 1)[None, None, :]
    best = np.abs(x[:, :, None].astype(np.float64) - levels).min(-1)
    assert np.all(np.abs(x - xh) <= best + s[:, None] * 1e-5 + 1e-9)


@pytest.mark.parametrize("bits", [2, 3, 4])
def test_sym_paper_literal_bound_on_unclipped(bits):
    x = _rand_groups(11 + bits, 300, 32, "plain")
    r = O.quantize_groups(x, bits, O.SYM, O.PAPER_LITERAL)
    s = r["scale_bits"].view(np.float16).astype(np.float64)
    assert np.allclose(s, np.abs(x).max(1).astype(np.float64) / (2 ** bits - 1), rtol=2 ** -10)
    qs = r["code"].astype(int) - 2 ** (bits - 1)
    lo, hi = -(2 ** (bits - 1)), 2 ** (bits - 1) - 1
    assert qs.min() >= lo and qs.max() <= hi
    xh = O.dequantize_groups(r["code"], r["scale_bits"], r["zero_bits"], bits)
    inside = (qs > lo) & (qs < hi)
    assert np.all(np.abs(x - xh)[inside] <= (s[:, None] / 2 * (1 + 2 ** -8) + 1e-7).repeat(32, 1)[inside])
    assert np.any(~inside)          # the literal formula does clip the tails


@pytest.mark.parametrize("bits", [2, 3, 4])
def test_lossless_on_representable_grids(bits):
    # values already on z + s*u with power-of-two s: asym must reproduce them exactly;
    # values on s*q: sym (FULLRANGE) must reproduce them exactly, and hybrid has zero error.
    g = np.random.default_rng(3)
    L = 2 ** bits - 1
    u = g.integers(0, L + 1, size=(100, 32))
    u[:, 0], u[:, 1] = 0, L
    x = (0.25 * u - 1.75).astype(f32)
    r = O.quantize_groups(x, bits, O.ASYM)
    assert np.array_equal(r["code"], u.astype(np.uint8))
    assert np.all(O.dequantize_groups(r["code"], r["scale_bits"], r["zero_bits"], bits) == x)
    den = 2 ** (bits - 1) - 1
    qq = g.integers(-den, den + 1, size=(100, 32))
    qq[:, 0] = den
    xs = (0.5 * qq).astype(f32)
    rs = O.quantize_groups(xs, bits, O.SYM)
    assert np.all(O.dequantize_groups(rs["code"], rs["scale_bits"], rs["zero_bits"], bits) == xs)
    rh = O.quantize_groups(xs, bits, O.HYBRID)
    assert np.all(O.dequantize_groups(rh["code"], rh["scale_bits"], rh["zero_bits"], bits) == xs)


@pytest.mark.parametrize("bits", [2, 3, 4])
@pytest.mark.parametrize("variant", [O.FULLRANGE, O.PAPER_LITERAL])
def test_hybrid_is_the_better_of_the_two_modes(bits, variant):
    # Brute force: quantise every group in both pure modes, measure the L1 error of what the
    # decoder reconstructs, and require hybrid to equal the better one (tie -> symmetric).
    x = np.concatenate([_rand_groups(1, 300, 32, "plain"), _rand_groups(2, 300, 32, "shifted"),
                        np.abs(_rand_groups(3, 100, 32, "plain")),
                        np.sign(_rand_groups(4, 50, 32, "plain")) * f32(0.75),      # two-valued +-c groups
                        np.zeros((5, 32), dtype=f32)])                              # all-zero groups: a tie
    ra = O.quantize_groups(x, bits, O.ASYM, variant)
    rs = O.quantize_groups(x, bits, O.SYM, variant)
    rh = O.quantize_groups(x, bits, O.HYBRID, variant)
    ea = np.abs(x - O.dequantize_groups(ra["code"], ra["scale_bits"], ra["zero_bits"], bits)).sum(1)
    es = np.abs(x - O.dequantize_groups(rs["code"], rs["scale_bits"], rs["zero_bits"], bits)).sum(1)
    want_asym = ea < es
    clear = np.abs(ea - es) > 1e-9 * np.maximum(ea, es)
    flag = (rh["scale_bits"] & 0x8000) != 0
    assert np.array_equal(flag[clear], want_asym[clear])
    assert 0 < flag.sum() < len(flag)                 # both modes occur in this data
    for name in ("code", "scale_bits", "zero_bits"):
        assert np.array_equal(rh[name][flag], ra[name][flag])
        assert np.array_equal(rh[name][~flag], rs[name][~flag])
        # the candidate hybrid did not choose is the other pure mode's result, for every group
        assert np.array_equal(rh["alt_" + name][flag], rs[name][flag])
        assert np.array_equal(rh["alt_" + name][~flag], ra[name][~flag])
    assert not np.any(rh["zero_bits"][~flag])
    xh = O.dequantize_groups(rh["code"], rh["scale_bits"], rh["zero_bits"], bits)
    assert np.allclose(np.abs(x - xh).sum(1), np.minimum(ea, es), rtol=1e-12)


def test_exhaustive_tiny_groups_against_bruteforce_levels():
    # every group of 3 values from a small set, b = 2: the asym result must be the nearest level
    # of {Z + S*u}; the hybrid choice must be the smaller total error.
    vals = [-2.0, -0.75, 0.0, 0.5, 1.25, 3.0]
    for trip in itertools.product(vals, repeat=3):
        x = np.array(trip, dtype=f32)
        r = O.quantize_groups(x, 2, O.HYBRID)
        xh = O.dequantize_groups(r["code"], r["scale_bits"], r["zero_bits"], 2)
        mn, mx, am = float(x.min()), float(x.max()), float(np.abs(x).max())
        Sa, Za = float(np.float16((mx - mn) / 3)), float(np.float16(mn))
        la = [Za + Sa * u for u in range(4)]
        ls = [float(np.float16(am)) * k for k in (-1, 0, 1)]
        ea = sum(min(abs(v - l) for l in la) for v in trip)
        es = sum(min(abs(v - l) for l in ls) for v in trip)
        got = float(np.abs(x - xh).sum())
        assert got == pytest.approx(min(ea, es), abs=1e-6), trip
        if abs(ea - es) > 1e-6:
            assert bool(r["flag"]) == (ea < es), trip


def test_effective_bits_match_table_bits():
    # Table "bits": count what the oracle actually stores for G = 32, D = 128.
    path = os.path.join(os.path.dirname(__file__), "golden", "table_bits.txt")
    rows = [l.split() for l in open(path) if l.strip() and not l.startswith("#")]
    assert len(rows) == 4
    D, G, n = 128, 32, 64
    x = np.random.default_rng(0).standard_normal((n, D // G, G)).astype(f32)
    for name, kb, kz, vb, vz, eff in rows:
        total = 0.0
        for b, z in ((int(kb), int(kz)), (int(vb), int(vz))):
            r = O.quantize_groups(x, b, O.HYBRID if z else O.SYM)
            stored = r["code"].size * b + r["scale_bits"].size * 16 + (r["zero_bits"].size * 16 if z else 0)
            if not z:
                assert not np.any(r["zero_bits"])     # nothing to store
            total += stored / r["code"].size
        assert total / 2 == pytest.approx(float(eff)), name
