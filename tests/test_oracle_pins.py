"""Pins for the CPU oracle: every oracle function is checked against something other
than itself -- the format definition via numpy's independent fp16 codec, brute force
in exact rational arithmetic, closed forms, library routines on special cases, and
identities that follow from Eq. 1 of the paper.

The checks live in plain functions taking no arguments so that the mutation test at the
bottom can re-run them against deliberately broken builds of the oracle and demand that
at least one of them fails for each planted mistake.
"""
import math
import os
import subprocess
import sys
import tempfile
from fractions import Fraction

import numpy as np
import pytest

from oracle import pd_oracle as orc
from paper_2512_19720_b200 import synth

ROW, COL = orc.AXIS_ROW, orc.AXIS_COL
GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


# ---------------------------------------------------------------- independent helpers
def half_bits_to_fraction(h):
    """binary16 decoded from the format definition, exactly (finite values only)."""
    s, e, m = h >> 15, (h >> 10) & 31, h & 1023
    mag = Fraction(m, 1 << 24) if e == 0 else Fraction(m + 1024) * Fraction(2) ** (e - 25)
    return -mag if s else mag


_POS = [half_bits_to_fraction(h) for h in range(0x7C00)]  # ascending, 0 .. 65504


def rn16_of_fraction(q):
    """Nearest binary16 to a non-negative rational, ties to even, by search over the grid."""
    assert q >= 0
    if q >= Fraction(65520):
        return 0x7C00
    lo, hi = 0, len(_POS) - 1
    while hi - lo > 1:
        mid = (lo + hi) // 2
        if _POS[mid] <= q:
            lo = mid
        else:
            hi = mid
    dl, dh = q - _POS[lo], _POS[hi] - q
    if dl < dh:
        return lo
    if dh < dl:
        return hi
    return lo if lo % 2 == 0 else hi


def f16_from_bits(bits):
    return np.array(bits, dtype=np.uint16).view(np.float16)


def small_case(d_out, d_in, seed, sigma=1e-3):
    w_b = synth.gen_base(d_out, d_in, seed)
    w_f = synth.gen_finetuned(w_b, seed + 1000, sigma)
    return w_b, w_f


def dense_sign(w_f, w_b):
    d = w_f.astype(np.float64) - w_b.astype(np.float64)
    return np.where(d >= 0, 1, -1).astype(np.int8), d


# ---------------------------------------------------------------- fp16 codec
def check_half_decode_all_patterns():
    bits = np.arange(65536, dtype=np.uint16)
    ref = bits.view(np.float16).astype(np.float64)
    got = np.array([orc.half_to_double(int(b)) for b in bits])
    nan = np.isnan(ref)
    assert np.array_equal(np.isnan(got), nan)
    assert np.array_equal(got[~nan], ref[~nan])
    assert np.array_equal(np.signbit(got[~nan]), np.signbit(ref[~nan]))


def check_half_encode():
    rng = np.random.default_rng(7)
    vals = []
    for e in range(-30, 18):
        vals.append(rng.uniform(-1, 1, 400) * 2.0 ** e)
    grid = np.arange(0x7C00, dtype=np.uint16).view(np.float16).astype(np.float64)
    mid = (grid[:-1] + grid[1:]) / 2  # exact in fp64
    vals += [grid, -grid, mid, -mid, np.nextafter(mid, np.inf), np.nextafter(mid, -np.inf),
             np.array([65519.99, 65520.0, 65520.01, 1e6, -1e6, np.inf, -np.inf, 0.0, -0.0,
                       2.0 ** -25, np.nextafter(2.0 ** -25, 1), 2.0 ** -26, 3 * 2.0 ** -25])]
    vals = np.concatenate(vals)
    with np.errstate(over="ignore"):
        ref = vals.astype(np.float16).view(np.uint16)
    got = np.array([orc.double_to_half(float(v)) for v in vals], dtype=np.uint16)
    assert np.array_equal(got, ref)
    # and against exact rational rounding on a sample (numpy itself is not the definition)
    for v in rng.uniform(0, 1, 300) * 2.0 ** rng.integers(-26, 16, 300):
        assert orc.double_to_half(float(v)) == rn16_of_fraction(Fraction(float(v)))


# ---------------------------------------------------------------- pack: mask
def parse_cols(spec):
    out = []
    spec = spec.strip()
    if spec == "-":
        return out
    for part in spec.split(","):
        if "-" in part:
            a, b = part.split("-")
            out += list(range(int(a), int(b) + 1))
        else:
            out.append(int(part))
    return out


def check_bit_layout_golden():
    n = 0
    for line in open(os.path.join(GOLDEN, "bit_layout_cases.txt")):
        if line.startswith("#") or not line.strip():
            continue
        d_in, pos, zero, words = [t.strip() for t in line.split("|")]
        d_in = int(d_in)
        w_b = np.full((1, d_in), 0.5, dtype=np.float16)
        w_f = np.full((1, d_in), 0.25, dtype=np.float16)  # dW < 0 by default
        w_f[0, parse_cols(pos)] = 1.0
        w_f[0, parse_cols(zero)] = 0.5
        mask, _, _ = orc.pack(w_f, w_b)
        expect = np.array([int(w, 16) for w in words.split(",")], dtype=np.uint32)
        assert np.array_equal(mask[0], expect), (line, mask)
        n += 1
    assert n >= 8


def check_unpack_inverts_pack():
    for (d_out, d_in, seed) in [(5, 64, 1), (33, 96, 2), (64, 256, 3)]:
        w_b, w_f = small_case(d_out, d_in, seed)
        w_f[1, 3] = w_b[1, 3]  # an exact zero delta
        b_ref, d = dense_sign(w_f, w_b)
        assert (d == 0).any()
        mask, _, _ = orc.pack(w_f, w_b)
        assert mask.shape == (d_out, d_in // 32) and mask.nbytes * 8 == d_out * d_in
        b = orc.unpack(mask, d_in)
        assert np.array_equal(b, b_ref)
        assert set(np.unique(b)) <= {-1, 1}
        pop = sum(bin(int(w)).count("1") for w in mask.ravel())
        assert pop == int((d >= 0).sum())


def check_signed_zero_and_asymmetric_rows():
    # row/column asymmetric pattern: catches a transposed mask
    d_out, d_in = 3, 64
    w_b = np.zeros((d_out, d_in), dtype=np.float16)
    w_f = np.full((d_out, d_in), -1.0, dtype=np.float16)
    w_f[0, 5] = 1.0
    w_f[2, 40] = 1.0
    w_f[1, 0] = -0.0  # -0 - 0 = -0 >= 0 is true
    mask, _, _ = orc.pack(w_f, w_b)
    expect = np.zeros((3, 2), dtype=np.uint32)
    expect[0, 0] = 1 << 5
    expect[2, 1] = 1 << 8
    expect[1, 0] = 1
    assert np.array_equal(mask, expect)


# ---------------------------------------------------------------- pack: scales
def check_v_init_bruteforce_rational():
    for (d_out, d_in, seed, sigma) in [(4, 32, 11, 1e-3), (7, 64, 12, 3e-2), (16, 96, 13, 1e-4)]:
        w_b, w_f = small_case(d_out, d_in, seed, sigma)
        fb = [[half_bits_to_fraction(int(h)) for h in r] for r in w_b.view(np.uint16)]
        ff = [[half_bits_to_fraction(int(h)) for h in r] for r in w_f.view(np.uint16)]
        _, v_row, v_col = orc.pack(w_f, w_b)
        for o in range(d_out):
            mean = sum(abs(ff[o][i] - fb[o][i]) for i in range(d_in)) / d_in
            assert int(v_row.view(np.uint16)[o]) == rn16_of_fraction(mean)
        for i in range(d_in):
            mean = sum(abs(ff[o][i] - fb[o][i]) for o in range(d_out)) / d_out
            assert int(v_col.view(np.uint16)[i]) == rn16_of_fraction(mean)


def check_v_init_dyadic():
    # |dW| = 2^-k patterns whose means are exactly representable; rows and columns differ
    d_out, d_in = 4, 32
    w_b = np.zeros((d_out, d_in), dtype=np.float16)
    w_f = np.zeros((d_out, d_in), dtype=np.float16)
    for o in range(d_out):
        for i in range(d_in):
            w_f[o, i] = (2.0 ** -(o + 1)) * (1 if (i % 2) else -1) * (2 if i < 16 else 1)
    _, v_row, v_col = orc.pack(w_f, w_b)
    for o in range(d_out):
        assert float(v_row[o]) == 1.5 * 2.0 ** -(o + 1)
    col_lo = sum(2.0 ** -(o + 1) for o in range(d_out)) / d_out
    assert np.all(v_col[:16].astype(np.float64) == np.float16(2 * col_lo))
    assert np.all(v_col[16:].astype(np.float64) == np.float16(col_lo))
    assert v_row.shape == (d_out,) and v_col.shape == (d_in,)


def check_v_init_gaussian_closed_form():
    d_out, d_in, seed = 256, 4096, 0
    w_b = synth.gen_base(d_out, d_in, seed)
    w_f = synth.gen_finetuned(w_b, seed + 1000)
    s_r = synth.gen_row_spread(d_out, seed + 1000)
    _, v_row, v_col = orc.pack(w_f, w_b)
    c = math.sqrt(2 / math.pi) * 1e-3
    rel = v_row.astype(np.float64) / (c * s_r) - 1
    assert np.max(np.abs(rel)) < 0.06, np.max(np.abs(rel))  # ~4.5 sigma of 0.756/sqrt(4096) + fp16 grid
    assert abs(np.mean(rel)) < 0.01
    relc = v_col.astype(np.float64) / (c * s_r.mean()) - 1
    assert np.max(np.abs(relc)) < 0.35 and abs(np.mean(relc)) < 0.01


# ---------------------------------------------------------------- reconstruct / merge
def check_reconstruct_identity_bruteforce():
    for axis in (ROW, COL):
        for (d_out, d_in, seed) in [(2, 32, 21), (8, 64, 22), (5, 96, 23)]:
            w_b, w_f = small_case(d_out, d_in, seed)
            mask, v_row, v_col = orc.pack(w_f, w_b)
            v = v_row if axis == ROW else v_col
            b, _ = dense_sign(w_f, w_b)
            wb64, v64 = w_b.astype(np.float64), v.astype(np.float64)
            ref = np.empty((d_out, d_in))
            for o in range(d_out):
                for i in range(d_in):
                    ref[o, i] = wb64[o, i] + (v64[o] if axis == ROW else v64[i]) * b[o, i]
            got = orc.reconstruct(w_b, mask, v, axis)
            assert np.array_equal(got, ref)
            # |W_hat - W_b| is the broadcast scale: rows constant (row axis) or columns constant (col axis)
            dev = np.abs(got - wb64)
            want = np.broadcast_to(v64[:, None] if axis == ROW else v64[None, :], dev.shape)
            assert np.allclose(dev, want, rtol=0, atol=1e-12)


def check_merge_matches_fp32_add_then_fp16():
    for axis in (ROW, COL):
        for (d_out, d_in, seed, sigma) in [(8, 64, 31, 1e-3), (16, 128, 32, 0.3)]:
            w_b, w_f = small_case(d_out, d_in, seed, sigma)
            mask, v_row, v_col = orc.pack(w_f, w_b)
            v = v_row if axis == ROW else v_col
            b, _ = dense_sign(w_f, w_b)
            vb = (v[:, None] if axis == ROW else v[None, :]).astype(np.float32) * b.astype(np.float32)
            ref = (w_b.astype(np.float32) + vb).astype(np.float16)  # numpy: IEEE fp32 add, RN16
            got = orc.merge(w_b, mask, v, axis)
            assert np.array_equal(got.view(np.uint16), ref.view(np.uint16))
    # v = 0 leaves the base untouched, bit for bit
    w_b, w_f = small_case(8, 64, 33)
    mask, _, _ = orc.pack(w_f, w_b)
    z = np.zeros(8, dtype=np.float16)
    assert np.array_equal(orc.merge(w_b, mask, z, ROW).view(np.uint16), w_b.view(np.uint16))
    assert np.array_equal(orc.reconstruct(w_b, mask, z, ROW), w_b.astype(np.float64))


def check_merge_equals_exact_rounding():
    # fp32 carries 24 >= 2*11 + 2 significant bits, so rounding the sum of two binary16 numbers to
    # fp32 first and to fp16 second can never differ from rounding the exact sum once (the classic
    # double-rounding bound for addition).  Hence merge must equal RN16 of the exact rational sum,
    # including across wide exponent gaps and at ties.
    rng = np.random.default_rng(34)
    wb_bits = rng.integers(0, 0x7800, size=(4, 32)).astype(np.uint16)  # magnitudes up to 32768
    wb_bits[0, :8] = [0x3C00, 0x3C01, 0x4000, 0x6800, 0x0001, 0x03FF, 0x0400, 0x3BFF]
    wb_bits ^= (rng.integers(0, 2, size=(4, 32)).astype(np.uint16) << 15)
    w_b = f16_from_bits(wb_bits)
    v_bits = np.array([0x1001, 0x0001, 0x3C00, 0x2C01], dtype=np.uint16)
    v = f16_from_bits(v_bits)
    mask = rng.integers(0, 2 ** 32, size=(4, 1), dtype=np.uint64).astype(np.uint32)
    got = orc.merge(w_b, mask, v, ROW).view(np.uint16)
    for o in range(4):
        for i in range(32):
            sgn = 1 if (int(mask[o, 0]) >> i) & 1 else -1
            exact = half_bits_to_fraction(int(wb_bits[o, i])) + sgn * half_bits_to_fraction(int(v_bits[o]))
            want = rn16_of_fraction(abs(exact))
            if exact < 0 or (exact == 0 and False):
                want |= 0x8000
            if exact == 0:
                assert int(got[o, i]) & 0x7FFF == 0
            else:
                assert int(got[o, i]) == want, (o, i, hex(int(got[o, i])), hex(want))


def check_pack_merge_round_trip():
    w_b, w_f = small_case(32, 128, 41)
    mask, v_row, _ = orc.pack(w_f, w_b)
    w_hat = orc.merge(w_b, mask, v_row, ROW)
    mask2, v2, _ = orc.pack(w_hat, w_b)
    moved = w_hat.view(np.uint16) != w_b.view(np.uint16)
    b1, b2 = orc.unpack(mask, 128), orc.unpack(mask2, 128)
    assert np.array_equal(b1[moved], b2[moved])
    assert np.allclose(v2.astype(np.float64), v_row.astype(np.float64), rtol=0.02)


# ---------------------------------------------------------------- linear
def check_linear_v0_is_library_gemm():
    w_b, w_f = small_case(48, 160, 51)
    mask, _, _ = orc.pack(w_f, w_b)
    x = synth.gen_x(5, 160, 52)
    ref = x.astype(np.float64) @ w_b.astype(np.float64).T
    for axis, n in ((ROW, 48), (COL, 160)):
        y = orc.linear(x, w_b, mask, np.zeros(n, dtype=np.float16), axis)
        assert y.shape == (5, 48)
        assert np.allclose(y, ref, rtol=1e-13, atol=1e-15)


def check_linear_one_hot_gives_columns():
    d_out, d_in = 24, 96
    w_b, w_f = small_case(d_out, d_in, 53)
    mask, v_row, v_col = orc.pack(w_f, w_b)
    x = np.zeros((d_in, d_in), dtype=np.float16)
    x[np.arange(d_in), np.arange(d_in)] = 1.0
    for axis, v in ((ROW, v_row), (COL, v_col)):
        y = orc.linear(x, w_b, mask, v, axis)  # y[i, o] = W_hat[o, i]
        assert np.array_equal(y.T, orc.reconstruct(w_b, mask, v, axis))
        y16 = y.astype(np.float32).astype(np.float16)
        assert np.array_equal(y16.T.view(np.uint16), orc.merge(w_b, mask, v, axis).view(np.uint16))


def check_linear_pm1_integer_sums():
    d_out, d_in, m = 6, 64, 3
    rng = np.random.default_rng(54)
    w_b0 = np.zeros((d_out, d_in), dtype=np.float16)
    w_f = rng.choice([-1.0, 1.0], size=(d_out, d_in)).astype(np.float16)
    mask, _, _ = orc.pack(w_f, w_b0)
    xi = rng.integers(-4, 5, size=(m, d_in))
    x = xi.astype(np.float16)
    ref = [[sum(int(xi[r, i]) * int(w_f[o, i]) for i in range(d_in)) for o in range(d_out)] for r in range(m)]
    for axis, n in ((ROW, d_out), (COL, d_in)):
        y = orc.linear(x, w_b0, mask, np.ones(n, dtype=np.float16), axis)
        assert np.array_equal(y, np.array(ref, dtype=np.float64))


def check_linear_row_col_agree_for_constant_v():
    w_b, w_f = small_case(40, 128, 55)
    mask, _, _ = orc.pack(w_f, w_b)
    x = synth.gen_x(4, 128, 56)
    c = np.float16(7.5e-4)
    y_r = orc.linear(x, w_b, mask, np.full(40, c, dtype=np.float16), ROW)
    y_c = orc.linear(x, w_b, mask, np.full(128, c, dtype=np.float16), COL)
    assert np.allclose(y_r, y_c, rtol=1e-12, atol=1e-15)


def check_linear_algebraic_split():
    d_out, d_in = 40, 128
    w_b, w_f = small_case(d_out, d_in, 57)
    mask, v_row, v_col = orc.pack(w_f, w_b)
    # distinct, non-constant scales so that a row/col mix-up shows
    v_row = (v_row.astype(np.float32) * np.linspace(0.5, 2, d_out)).astype(np.float16)
    v_col = (v_col.astype(np.float32) * np.linspace(2, 0.5, d_in)).astype(np.float16)
    x = synth.gen_x(4, d_in, 58)
    b, _ = dense_sign(w_f, w_b)
    x64, wb64, b64 = x.astype(np.float64), w_b.astype(np.float64), b.astype(np.float64)
    ref_row = x64 @ wb64.T + (x64 @ b64.T) * v_row.astype(np.float64)[None, :]
    ref_col = x64 @ wb64.T + (x64 * v_col.astype(np.float64)[None, :]) @ b64.T
    assert np.allclose(orc.linear(x, w_b, mask, v_row, ROW), ref_row, rtol=1e-11, atol=1e-14)
    assert np.allclose(orc.linear(x, w_b, mask, v_col, COL), ref_col, rtol=1e-11, atol=1e-14)
    assert not np.allclose(ref_row, ref_col, rtol=1e-4)
    # linearity in x
    y1 = orc.linear(x[:2], w_b, mask, v_row, ROW)
    y2 = orc.linear(x[2:], w_b, mask, v_row, ROW)
    xs = (x[:2].astype(np.float32) * 2).astype(np.float16)
    assert np.allclose(orc.linear(xs, w_b, mask, v_row, ROW), 2 * y1, rtol=1e-12)
    assert y1.shape == y2.shape


def check_linear_equals_dense_on_merged_up_to_fp16():
    # "inference identical to FP16 weights": the fused form and a dense product on the merged
    # fp16 weights differ only by the merge rounding (<= 2^-11 relative per weight)
    w_b, w_f = small_case(64, 256, 59)
    mask, v_row, _ = orc.pack(w_f, w_b)
    x = synth.gen_x(3, 256, 60)
    y = orc.linear(x, w_b, mask, v_row, ROW)
    y_m = x.astype(np.float64) @ orc.merge(w_b, mask, v_row, ROW).astype(np.float64).T
    assert np.max(np.abs(y - y_m)) / np.max(np.abs(y)) < 2e-3


# ---------------------------------------------------------------- multivariant
def _variants(d_out, d_in, n_var, seed):
    w_b = synth.gen_base(d_out, d_in, seed)
    masks = np.empty((n_var, d_out, d_in // 32), dtype=np.uint32)
    stride = max(d_out, d_in)
    vs = np.zeros((n_var, stride), dtype=np.float16)
    axes = np.zeros(n_var, dtype=np.uint8)
    for g in range(n_var):
        w_f = synth.gen_finetuned(w_b, seed + 1000 + g)
        m, vr, vc = orc.pack(w_f, w_b)
        masks[g] = m
        axes[g] = g % 2
        if axes[g] == ROW:
            vs[g, :d_out] = vr
        else:
            vs[g, :d_in] = vc
    return w_b, masks, vs, axes


def check_multivariant_identities():
    d_out, d_in, n_var, m = 24, 96, 3, 9
    w_b, masks, vs, axes = _variants(d_out, d_in, n_var, 61)
    x = synth.gen_x(m, d_in, 62)
    ids = np.array([0, 1, 2, -1, 2, 1, 0, -1, 1], dtype=np.int32)
    y, bad = orc.linear_multivariant(x, ids, w_b, masks, vs, axes)
    assert bad == 0
    for r in range(m):
        g = ids[r]
        if g < 0:
            ref = x[r:r + 1].astype(np.float64) @ w_b.astype(np.float64).T
        else:
            n = d_out if axes[g] == ROW else d_in
            ref = orc.linear(x[r:r + 1], w_b, masks[g], vs[g, :n].copy(), int(axes[g]))
        assert np.allclose(y[r], ref[0], rtol=1e-12, atol=1e-15)
    # permuting rows (and ids) permutes outputs
    perm = np.random.default_rng(63).permutation(m)
    y_p, _ = orc.linear_multivariant(x[perm].copy(), ids[perm].copy(), w_b, masks, vs, axes)
    assert np.array_equal(y_p, y[perm])
    # a single variant with all ids 0 is the plain fused linear
    y1, _ = orc.linear_multivariant(x, np.zeros(m, dtype=np.int32), w_b, masks[:1], vs[:1], axes[:1])
    assert np.allclose(y1, orc.linear(x, w_b, masks[0], vs[0, :d_out].copy(), ROW), rtol=1e-12)
    # invalid ids are counted
    _, bad = orc.linear_multivariant(x, np.array([0, 3, -2] + [0] * 6, dtype=np.int32), w_b, masks, vs, axes)
    assert bad == 2


def check_size_accounting():
    # one bit per entry: E/8 bytes of mask; with fp16 scales the delta of a d x d layer is
    # 16x smaller than its fp16 weights up to the 2*d bytes of v
    for (d_out, d_in) in [(64, 128), (128, 64)]:
        w_b, w_f = small_case(d_out, d_in, 71)
        mask, v_row, v_col = orc.pack(w_f, w_b)
        assert mask.nbytes == d_out * d_in // 8
        assert v_row.nbytes == 2 * d_out and v_col.nbytes == 2 * d_in
        assert w_b.nbytes / mask.nbytes == 16


CHECKS = [v for k, v in sorted(globals().items()) if k.startswith("check_")]


@pytest.mark.parametrize("check", CHECKS, ids=[c.__name__ for c in CHECKS])
def test_pin(check, oracle):
    check()


# ---------------------------------------------------------------- mutation: the pins must bite
MUTATIONS = [
    ("sign_of_zero", "if (dw >= 0.0) mask", "if (dw > 0.0) mask"),
    ("bit_order", "(uint32_t)1 << (i % 32)", "(uint32_t)1 << (31 - i % 32)"),
    ("delta_sign", "pdo_half_to_double(w_f[o * d_in + i]) - pdo_half_to_double(w_b[o * d_in + i]);\n            if",
     "pdo_half_to_double(w_b[o * d_in + i]) - pdo_half_to_double(w_f[o * d_in + i]);\n            if"),
    ("row_mean_divisor", "sum_abs / (double)d_in", "sum_abs / (double)d_out"),
    ("col_mean_divisor", "col[i] / (double)d_out", "col[i] / (double)d_in"),
    ("dropped_abs", "sum_abs += fabs(dw);", "sum_abs += dw;"),
    ("axis_swapped", "v[axis == AXIS_ROW ? o : i]", "v[axis == AXIS_ROW ? i % 1 : o % 1]"),
    ("unpack_polarity", "& 1u) ? 1.0 : -1.0;", "& 1u) ? -1.0 : 1.0;"),
    ("merge_rounds_down", "float sum32 = (float)exact;", "float sum32 = nextafterf((float)exact, 0.0f);"),
    ("linear_dropped_delta", "+ scale * b;", "+ 0.0 * scale * b;"),
    ("linear_wrong_x_stride", "x[m * ldx + i]) * row[i]", "x[i]) * row[i]"),
    ("encode_truncates", "if (diff > 0.5) return fl + 1.0;", "if (diff > 0.75) return fl + 1.0;"),
    ("encode_ties_away", "return (fmod(fl, 2.0) == 0.0) ? fl : fl + 1.0;", "return fl + 1.0;"),
    ("decode_subnormal", "v = ldexp((double)m, -24);", "v = ldexp((double)m, -25);"),
    ("multivariant_wrong_variant", "masks + (int64_t)g * mask_words", "masks + (int64_t)0 * mask_words"),
    ("multivariant_base_only", "(g < 0) ? pdo_half_to_double", "(g < -5) ? pdo_half_to_double"),
]


@pytest.mark.parametrize("name,old,new", MUTATIONS, ids=[m[0] for m in MUTATIONS])
def test_planted_mistake_is_caught(name, old, new, oracle):
    src = open(os.path.join(os.path.dirname(orc.__file__), "pd_oracle.c")).read()
    assert src.count(old) >= 1, f"mutation anchor for {name} not found"
    with tempfile.TemporaryDirectory() as tmp:
        c_path, so_path = os.path.join(tmp, "mut.c"), os.path.join(tmp, "mut.so")
        open(c_path, "w").write(src.replace(old, new))
        subprocess.check_call(["gcc", "-O1", "-std=c11", "-fopenmp", "-shared", "-fPIC", "-o", so_path, c_path, "-lm"])
        caught = []
        with orc.use_library(so_path):
            for check in CHECKS:
                try:
                    check()
                except (AssertionError, OverflowError, IndexError, ValueError):
                    caught.append(check.__name__)
        assert caught, f"no pin noticed the planted mistake '{name}'"
