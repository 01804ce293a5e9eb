"""Pins for the BF16 CPU oracle (oracle/pd_oracle_bf16.c): every function is checked against something other
than itself -- the bfloat16 format via binary32 bit patterns and exact rationals, brute force in exact rational
arithmetic for the scale grid, numpy's binary32 addition for the merge, library GEMMs and the identities of Eq. 1,
and the pinned FP16 oracle on inputs that both formats hold exactly.  As for the FP16 oracle, planted mistakes are
compiled into copies of the C file and each must fail at least one pin.
"""
import os
import subprocess
import tempfile
from fractions import Fraction

import numpy as np
import pytest

from oracle import pd_oracle as orc16
from oracle import pd_oracle_bf16 as orc
from paper_2512_19720_b200 import synth

ROW, COL = orc.AXIS_ROW, orc.AXIS_COL


@pytest.fixture(scope="module", autouse=True)
def _built():
    orc.build()
    orc16.build()


# ---------------------------------------------------------------- independent helpers
def bf16_fraction(h):
    """bfloat16 decoded from the format definition, exactly (finite values only)."""
    s, e, m = h >> 15, (h >> 7) & 255, h & 127
    mag = Fraction(m) * Fraction(2) ** -133 if e == 0 else Fraction(m + 128) * Fraction(2) ** (e - 134)
    return -mag if s else mag


def half_fraction(h):
    s, e, m = h >> 15, (h >> 10) & 31, h & 1023
    mag = Fraction(m, 1 << 24) if e == 0 else Fraction(m + 1024) * Fraction(2) ** (e - 25)
    return -mag if s else mag


_POS_BF16 = [bf16_fraction(h) for h in range(0x7F80)]  # ascending, 0 .. max finite
_POS_HALF = [half_fraction(h) for h in range(0x7C00)]


def _nearest_even(grid, q, overflow_at, inf_code):
    if q >= overflow_at:
        return inf_code
    lo, hi = 0, len(grid) - 1
    while hi - lo > 1:
        mid = (lo + hi) // 2
        if grid[mid] <= q:
            lo = mid
        else:
            hi = mid
    dl, dh = q - grid[lo], grid[hi] - q
    if dl != dh:
        return lo if dl < dh else hi
    return lo if lo % 2 == 0 else hi


def rn_bf16(q):
    return _nearest_even(_POS_BF16, q, Fraction(511) * Fraction(2) ** 119, 0x7F80)


def rn_half(q):
    return _nearest_even(_POS_HALF, q, Fraction(65520), 0x7C00)


def f32_of_bits(b):
    return synth.bf16_bits_to_f32(np.asarray(b, dtype=np.uint16))


def small_case(d_out, d_in, seed, sigma=1e-3):
    w_b = synth.gen_base_bf16(d_out, d_in, seed)
    return w_b, synth.gen_finetuned_bf16(w_b, seed + 1000, sigma)


def wild_case(d_out, d_in, seed):
    """Magnitudes from subnormal to thousands, exact zeros, +-0, equal entries, pairs far apart."""
    rng = np.random.default_rng(seed)
    mag = rng.choice([1e-40, 1e-30, 1e-12, 3e-8, 6e-8, 1e-5, 1e-3, 0.02, 0.7, 1.0, 40.0], size=(d_out, d_in))
    w_b = synth.to_bf16_bits((rng.standard_normal((d_out, d_in)) * mag).astype(np.float32))
    mag2 = rng.choice([1e-40, 1e-20, 2e-8, 1e-6, 1e-3, 0.5], size=(d_out, d_in))
    w_f = synth.to_bf16_bits((f32_of_bits(w_b).astype(np.float64) + rng.standard_normal((d_out, d_in)) * mag2).astype(np.float32))
    w_f[0, 0] = w_b[0, 0]
    w_b[0, 1], w_f[0, 1] = 0x0000, 0x8000  # +0 vs -0
    w_b[0, 2], w_f[0, 2] = 0x3F80, 0x0001  # 1.0 vs the smallest subnormal: |dW| just below 1
    w_b[0, 3], w_f[0, 3] = 0x0001, 0x3F80
    return w_b, w_f


def units_fraction(a, b):
    """floor(|a - b| * 2^24) in exact rational arithmetic."""
    q = abs(a - b) * (1 << 24)
    return q.numerator // q.denominator


# ---------------------------------------------------------------- codec
def check_bf16_decode_all_patterns():
    bits = np.arange(65536, dtype=np.uint16)
    with np.errstate(invalid="ignore"):
        ref = f32_of_bits(bits).astype(np.float64)  # bfloat16 = the upper half of a binary32
    got = np.array([orc.bf16_to_double(int(b)) for b in bits])
    nan = np.isnan(ref)
    assert np.array_equal(np.isnan(got), nan)
    assert np.array_equal(got[~nan], ref[~nan])
    assert np.array_equal(np.signbit(got[~nan]), np.signbit(ref[~nan]))
    for h in (0x0001, 0x007F, 0x0080, 0x3F80, 0x7F7F, 0x8001, 0xC2F7):
        assert Fraction(orc.bf16_to_double(h)) == bf16_fraction(h)


def check_bf16_encode():
    rng = np.random.default_rng(7)
    grid = np.array([float(q) for q in _POS_BF16])  # every bfloat16 is exact in fp64
    mid = (grid[:-1] + grid[1:]) / 2                # exact in fp64
    vals = np.concatenate([grid, -grid, mid, -mid, np.nextafter(mid, np.inf), np.nextafter(mid, -np.inf),
                           np.array([3.3961775e38, 3.39e38, 3.4e38, np.inf, -np.inf, 0.0, -0.0, 2.0 ** -134,
                                     np.nextafter(2.0 ** -134, 1), 2.0 ** -135, 3 * 2.0 ** -134])])
    got = np.array([orc.double_to_bf16(float(v)) for v in vals], dtype=np.uint16)
    # grid points and everything strictly between midpoints: the binary32 bit trick agrees (it is exact there)
    with np.errstate(over="ignore"):
        ref = synth.to_bf16_bits(vals.astype(np.float32))
    exact32 = vals.astype(np.float32).astype(np.float64) == vals
    assert np.array_equal(got[exact32], ref[exact32])
    # exact rational rounding on samples across the whole range, midpoints included
    sample = np.concatenate([rng.uniform(0, 1, 300) * 2.0 ** rng.integers(-140, 128, 300), mid[::97], mid[:300]])
    for v in sample:
        assert orc.double_to_bf16(float(v)) == rn_bf16(Fraction(float(v))), v
        assert orc.double_to_bf16(-float(v)) == (rn_bf16(Fraction(float(v))) | 0x8000)


# ---------------------------------------------------------------- pack
def check_mask_is_the_exact_comparison():
    for case in (small_case(5, 64, 1), small_case(33, 96, 2), wild_case(8, 64, 3)):
        w_b, w_f = case
        fb, ff = f32_of_bits(w_b).astype(np.float64), f32_of_bits(w_f).astype(np.float64)
        mask, _, _ = orc.pack(w_f, w_b)
        assert mask.shape == (w_b.shape[0], w_b.shape[1] // 32)
        bits = (mask[:, :, None] >> np.arange(32, dtype=np.uint32)[None, None, :]) & 1
        assert np.array_equal(bits.reshape(w_b.shape).astype(bool), ff >= fb)
    # bit order and signed zeros: an asymmetric pattern
    w_b = np.zeros((3, 64), dtype=np.uint16)
    w_f = np.full((3, 64), 0xBF80, dtype=np.uint16)  # -1
    w_f[0, 5] = 0x3F80
    w_f[2, 40] = 0x3F80
    w_f[1, 0] = 0x8000  # -0 >= +0
    expect = np.zeros((3, 2), dtype=np.uint32)
    expect[0, 0], expect[2, 1], expect[1, 0] = 1 << 5, 1 << 8, 1
    assert np.array_equal(orc.pack(w_f, w_b)[0], expect)


def check_scales_bruteforce_rational():
    for w_b, w_f in (small_case(4, 32, 11), small_case(7, 64, 12, 3e-2), wild_case(6, 64, 13), wild_case(9, 32, 14)):
        d_out, d_in = w_b.shape
        fb = [[bf16_fraction(int(h)) for h in r] for r in w_b]
        ff = [[bf16_fraction(int(h)) for h in r] for r in w_f]
        _, v_row, v_col = orc.pack(w_f, w_b)
        for o in range(d_out):
            units = sum(units_fraction(ff[o][i], fb[o][i]) for i in range(d_in))
            assert int(v_row.view(np.uint16)[o]) == rn_half(Fraction(units, d_in) / (1 << 24)), o
        for i in range(d_in):
            units = sum(units_fraction(ff[o][i], fb[o][i]) for o in range(d_out))
            assert int(v_col.view(np.uint16)[i]) == rn_half(Fraction(units, d_out) / (1 << 24)), i


def check_scale_grid_cuts_down_and_never_rounds_up():
    # |dW| = 1 - 2^-133 is cut down to 2^24 - 1 units; |dW| = 1.5 * 2^-24 counts as one unit; below 2^-24: none,
    # also when it misses 2^-24 by the smallest subnormal only (a difference rounded to nearest would reach it)
    d_in = 32
    w_b = np.zeros((4, d_in), dtype=np.uint16)
    w_f = np.zeros((4, d_in), dtype=np.uint16)
    w_b[0, :], w_f[0, :] = 0x3F80, 0x0001
    w_f[1, :] = 0x33C0   # 1.5 * 2^-24
    w_f[2, :] = 0x3300   # 2^-25
    w_b[3, :], w_f[3, :] = 0x0001, 0x3380  # 2^-24 - 2^-133
    _, v_row, _ = orc.pack(w_f, w_b)
    assert int(v_row.view(np.uint16)[0]) == rn_half(Fraction((1 << 24) - 1, 1 << 24))
    assert float(v_row[1]) == 2.0 ** -24 and float(v_row[2]) == 0.0 and float(v_row[3]) == 0.0


def check_pack_agrees_with_the_fp16_oracle_on_common_values():
    # values with at most 8 significant bits in the binary16 normal range are exact in both formats
    rng = np.random.default_rng(17)
    d_out, d_in = 6, 64
    sig = rng.integers(128, 256, size=(2, d_out, d_in)) * np.where(rng.random((2, d_out, d_in)) < 0.5, -1.0, 1.0)
    vals = sig * 2.0 ** rng.integers(-17, -2, size=(2, d_out, d_in))
    b16, f16 = vals[0].astype(np.float16), vals[1].astype(np.float16)
    assert np.array_equal(b16.astype(np.float64), vals[0])
    bb, fb = synth.to_bf16_bits(vals[0].astype(np.float32)), synth.to_bf16_bits(vals[1].astype(np.float32))
    assert np.array_equal(f32_of_bits(bb).astype(np.float64), vals[0])
    m16, r16, c16 = orc16.pack(f16, b16)
    m, r, c = orc.pack(fb, bb)
    assert np.array_equal(m, m16)
    assert np.array_equal(r.view(np.uint16), r16.view(np.uint16)) and np.array_equal(c.view(np.uint16), c16.view(np.uint16))


# ---------------------------------------------------------------- reconstruct / merge
def check_reconstruct_identity_bruteforce():
    for axis in (ROW, COL):
        for (d_out, d_in, seed) in [(2, 32, 21), (8, 64, 22)]:
            w_b, w_f = small_case(d_out, d_in, seed)
            mask, v_row, v_col = orc.pack(w_f, w_b)
            v = v_row if axis == ROW else v_col
            wb64, v64 = f32_of_bits(w_b).astype(np.float64), v.astype(np.float64)
            b = np.where(f32_of_bits(w_f) >= f32_of_bits(w_b), 1.0, -1.0)
            ref = np.empty((d_out, d_in))
            for o in range(d_out):
                for i in range(d_in):
                    ref[o, i] = wb64[o, i] + (v64[o] if axis == ROW else v64[i]) * b[o, i]
            assert np.array_equal(orc.reconstruct(w_b, mask, v, axis), ref)


def check_merge_is_binary32_add_then_bf16():
    rng = np.random.default_rng(31)
    for axis in (ROW, COL):
        d_out, d_in = 9, 64
        w_b, _ = wild_case(d_out, d_in, 32 + axis)
        mask = rng.integers(0, 2 ** 32, size=(d_out, d_in // 32), dtype=np.uint64).astype(np.uint32)
        n = d_out if axis == ROW else d_in
        v = rng.integers(0, 0x5000, size=n).astype(np.uint16).view(np.float16)
        bits = ((mask[:, :, None] >> np.arange(32, dtype=np.uint32)[None, None, :]) & 1).reshape(d_out, d_in)
        sign = np.where(bits == 1, np.float32(1), np.float32(-1))
        vb = np.broadcast_to(v.astype(np.float32)[:, None] if axis == ROW else v.astype(np.float32)[None, :], (d_out, d_in))
        s32 = f32_of_bits(w_b) + sign * vb  # numpy's binary32 addition: one rounding
        got = orc.merge(w_b, mask, v, axis)
        for o in range(d_out):
            for i in range(d_in):
                q = Fraction(float(s32[o, i]))
                want = rn_bf16(abs(q)) | (0x8000 if np.signbit(s32[o, i]) else 0)
                assert int(got[o, i]) == want, (o, i)
    # v = 0 gives the base back, bit for bit (apart from the sign of zero)
    w_b, w_f = small_case(4, 32, 35)
    mask, _, _ = orc.pack(w_f, w_b)
    assert np.array_equal(orc.merge(w_b, mask, np.zeros(4, dtype=np.float16), ROW) & 0x7FFF, w_b & 0x7FFF)


# ---------------------------------------------------------------- linear
def check_linear_v0_is_library_gemm():
    w_b, w_f = small_case(24, 96, 41)
    mask, _, _ = orc.pack(w_f, w_b)
    x = synth.gen_x_bf16(5, 96, 42)
    ref = f32_of_bits(x).astype(np.float64) @ f32_of_bits(w_b).astype(np.float64).T
    for axis, n in ((ROW, 24), (COL, 96)):
        got = orc.linear(x, w_b, mask, np.zeros(n, dtype=np.float16), axis)
        assert np.allclose(got, ref, rtol=1e-12, atol=1e-12)


def check_linear_one_hot_gives_merged_columns():
    w_b, w_f = small_case(16, 64, 43)
    mask, v_row, v_col = orc.pack(w_f, w_b)
    cols = [0, 1, 31, 32, 63]
    x = np.zeros((len(cols), 64), dtype=np.uint16)
    x[np.arange(len(cols)), cols] = 0x3F80
    for axis, v in ((ROW, v_row), (COL, v_col)):
        y = orc.linear(x, w_b, mask, v, axis)
        merged = orc.merge(w_b, mask, v, axis)
        rounded = np.array([[orc.double_to_bf16(float(np.float32(t))) for t in r] for r in y], dtype=np.uint16)
        assert np.array_equal(rounded, merged[:, cols].T)


def check_linear_pm1_integer_sums_and_split():
    rng = np.random.default_rng(44)
    d_out, d_in, m = 12, 96, 4
    w_b0 = np.zeros((d_out, d_in), dtype=np.uint16)
    w_f = np.where(rng.random((d_out, d_in)) < 0.5, 0x3F80, 0xBF80).astype(np.uint16)
    mask, _, _ = orc.pack(w_f, w_b0)
    xi = rng.integers(-3, 4, size=(m, d_in)).astype(np.float32)
    x = synth.to_bf16_bits(xi)
    ref = xi.astype(np.float64) @ f32_of_bits(w_f).astype(np.float64).T
    for axis, n in ((ROW, d_out), (COL, d_in)):
        assert np.array_equal(orc.linear(x, w_b0, mask, np.ones(n, dtype=np.float16), axis), ref)
    # algebraic split of Eq. 1 as a second fp64 path, on a generic case
    w_b, w_f = small_case(d_out, d_in, 45)
    mask, v_row, v_col = orc.pack(w_f, w_b)
    xg = synth.gen_x_bf16(m, d_in, 46)
    x64, wb64 = f32_of_bits(xg).astype(np.float64), f32_of_bits(w_b).astype(np.float64)
    b = np.where(f32_of_bits(w_f) >= f32_of_bits(w_b), 1.0, -1.0)
    assert np.allclose(orc.linear(xg, w_b, mask, v_row, ROW), x64 @ wb64.T + (x64 @ b.T) * v_row.astype(np.float64)[None, :], rtol=1e-10, atol=1e-12)
    assert np.allclose(orc.linear(xg, w_b, mask, v_col, COL), x64 @ wb64.T + (x64 * v_col.astype(np.float64)[None, :]) @ b.T, rtol=1e-10, atol=1e-12)
    # constant v: row mode == col mode
    c = np.float16(0.0123)
    assert np.allclose(orc.linear(xg, w_b, mask, np.full(d_out, c), ROW), orc.linear(xg, w_b, mask, np.full(d_in, c), COL), rtol=1e-12, atol=1e-14)


def check_multivariant_identities():
    d_out, d_in, n_var, m = 10, 64, 3, 9
    w_b = synth.gen_base_bf16(d_out, d_in, 51)
    masks = np.empty((n_var, d_out, d_in // 32), dtype=np.uint32)
    vs = np.zeros((n_var, 64), dtype=np.float16)
    axes = np.array([0, 1, 0], dtype=np.uint8)
    for g in range(n_var):
        mk, vr, vc = orc.pack(synth.gen_finetuned_bf16(w_b, 1051 + g), w_b)
        masks[g] = mk
        vs[g, :(d_out if axes[g] == 0 else d_in)] = vr if axes[g] == 0 else vc
    x = synth.gen_x_bf16(m, d_in, 52)
    ids = np.array([0, 1, 2, -1, 2, 1, 0, 0, -1], dtype=np.int32)
    y, bad = orc.linear_multivariant(x, ids, w_b, masks, vs, axes)
    assert bad == 0
    for r in range(m):
        g = ids[r]
        if g < 0:
            ref = f32_of_bits(x[r:r + 1]).astype(np.float64) @ f32_of_bits(w_b).astype(np.float64).T
            assert np.allclose(y[r:r + 1], ref, rtol=1e-12, atol=1e-12)
        else:
            n = d_out if axes[g] == 0 else d_in
            assert np.array_equal(y[r:r + 1], orc.linear(x[r:r + 1], w_b, masks[g], vs[g, :n], int(axes[g])))
    perm = np.array([3, 1, 4, 0, 8, 2, 7, 5, 6])
    y2, _ = orc.linear_multivariant(x[perm], ids[perm], w_b, masks, vs, axes)
    assert np.array_equal(y2, y[perm])
    ids_bad = ids.copy()
    ids_bad[4] = 7
    assert orc.linear_multivariant(x, ids_bad, w_b, masks, vs, axes)[1] == 1


CHECKS = [v for k, v in sorted(globals().items()) if k.startswith("check_")]


@pytest.mark.parametrize("check", CHECKS, ids=[c.__name__ for c in CHECKS])
def test_pin(check):
    check()


# ---------------------------------------------------------------- mutation: the pins must bite
MUTATIONS = [
    ("sign_of_zero", "if (f >= b) mask", "if (f > b) mask"),
    ("bit_order", "(uint32_t)1 << (i % 32)", "(uint32_t)1 << (31 - i % 32)"),
    ("units_round_to_nearest", "    fesetround(FE_TOWARDZERO);\n    d = x - y;", "    d = x - y;"),
    ("units_rounded_not_cut", "return floor(fabs(d) * 16777216.0);", "return floor(fabs(d) * 16777216.0 + 0.5);"),
    ("row_mean_divisor", "sum_units / (double)d_in", "sum_units / (double)d_out"),
    ("col_mean_divisor", "col[i] / (double)d_out", "col[i] / (double)d_in"),
    ("axis_swapped", "half_to_double(v[axis == AXIS_ROW ? o : i]);\n    return", "half_to_double(v[axis == AXIS_ROW ? i % 1 : o % 1]);\n    return"),
    ("unpack_polarity", "& 1u) ? 1.0 : -1.0;", "& 1u) ? -1.0 : 1.0;"),
    ("merge_in_fp64", "volatile float sum32 = plus ? base + scale : base - scale;",
     "volatile double sum32 = plus ? (double)base + (double)scale : (double)base - (double)scale;"),
    ("merge_sign", "plus ? base + scale : base - scale", "plus ? base - scale : base + scale"),
    ("linear_dropped_delta", "+ scale * b;", "+ 0.0 * scale * b;"),
    ("linear_wrong_x_stride", "x[m * ldx + i]) * row[i]", "x[i]) * row[i]"),
    ("encode_ties_away", "return (fmod(fl, 2.0) == 0.0) ? fl : fl + 1.0;", "return fl + 1.0;"),
    ("decode_subnormal", "v = ldexp((double)m, -133);", "v = ldexp((double)m, -134);"),
    ("decode_fraction_bits", "v = ldexp((double)(m + 128), e - 134);", "v = ldexp((double)(m + 128), e - 135);"),
    ("multivariant_wrong_variant", "masks + (int64_t)g * mask_words", "masks + (int64_t)0 * mask_words"),
]


@pytest.mark.parametrize("name,old,new", MUTATIONS, ids=[m[0] for m in MUTATIONS])
def test_planted_mistake_is_caught(name, old, new):
    src = open(os.path.join(os.path.dirname(orc.__file__), "pd_oracle_bf16.c")).read()
    assert src.count(old) >= 1, f"mutation anchor for {name} not found"
    with tempfile.TemporaryDirectory() as tmp:
        c_path, so_path = os.path.join(tmp, "mut.c"), os.path.join(tmp, "mut.so")
        open(c_path, "w").write(src.replace(old, new))
        subprocess.check_call(["gcc", "-O1", "-std=c11", "-frounding-math", "-fopenmp", "-shared", "-fPIC", "-o", so_path, c_path, "-lm"])
        caught = []
        with orc.use_library(so_path):
            for check in CHECKS:
                try:
                    check()
                except (AssertionError, OverflowError, IndexError, ValueError):
                    caught.append(check.__name__)
        assert caught, f"no pin noticed the planted mistake '{name}'"
