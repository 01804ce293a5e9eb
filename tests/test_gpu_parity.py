"""GPU parity: the CUDA library (through its C ABI) against the CPU oracle, element by element,
on the same seeded inputs.  Pack and merge must be bit-exact; linear outputs must satisfy
max|y - y_ref| / max|y_ref| <= 5e-3 (fp16 products, fp32 accumulation, one fp16 rounding)."""
import numpy as np
import pytest
import torch

from oracle import pd_oracle as orc
from paper_2512_19720_b200 import synth

pytestmark = pytest.mark.gpu
ROW, COL = 0, 1
TOL = 5e-3


@pytest.fixture(scope="module")
def api():
    assert torch.cuda.is_available(), "GPU tests need a CUDA device"
    from paper_2512_19720_b200 import api as _api
    return _api


def dev(a):
    if a.dtype == np.uint32:
        a = a.view(np.int32)
    return torch.from_numpy(np.ascontiguousarray(a)).cuda()


def host(t):
    a = t.detach().cpu().numpy()
    return a.view(np.uint32) if a.dtype == np.int32 else a


def bits(a):
    return np.ascontiguousarray(a).view(np.uint16)


def rel_err(y, y_ref):
    return float(np.max(np.abs(y.astype(np.float64) - y_ref)) / np.max(np.abs(y_ref)))


class Layer:
    """One synthetic (W_b, W_f) pair with the oracle's pack results, on host and device."""

    def __init__(self, d_out, d_in, seed=0, ft_seed=None, sigma=1e-3):
        self.d_out, self.d_in = d_out, d_in
        self.w_b = synth.gen_base(d_out, d_in, seed)
        self.w_f = synth.gen_finetuned(self.w_b, 1000 + seed if ft_seed is None else ft_seed, sigma)
        self.mask, self.v_row, self.v_col = orc.pack(self.w_f, self.w_b)
        self.d_w_b, self.d_w_f = dev(self.w_b), dev(self.w_f)
        self.d_mask, self.d_v_row, self.d_v_col = dev(self.mask), dev(self.v_row), dev(self.v_col)

    def v(self, axis):
        return self.v_row if axis == ROW else self.v_col

    def d_v(self, axis):
        return self.d_v_row if axis == ROW else self.d_v_col


_layers = {}


def layer(d_out, d_in, seed=0):
    key = (d_out, d_in, seed)
    if key not in _layers:
        if len(_layers) > 3:
            _layers.clear()
            torch.cuda.empty_cache()
        _layers[key] = Layer(d_out, d_in, seed)
    return _layers[key]


# ------------------------------------------------------------------ pack
PACK_SHAPES = [(1024, 1024), (64, 32), (1, 32), (65, 96), (200, 1056), (130, 288), (4096, 4096), (4096, 11008)]


@pytest.mark.parametrize("d_out,d_in", PACK_SHAPES)
def test_pack_bit_exact(api, d_out, d_in):
    L = layer(d_out, d_in)
    guard = 64
    mask = torch.full((d_out * (d_in // 32) + 2 * guard,), 0x5A5A5A5A, dtype=torch.int32, device="cuda")
    v_row = torch.full((d_out + 2 * guard,), 123.0, dtype=torch.float16, device="cuda")
    v_col = torch.full((d_in + 2 * guard,), 123.0, dtype=torch.float16, device="cuda")
    m_view = mask[guard:-guard].view(d_out, d_in // 32)
    api.pd_pack_delta(L.d_w_f, L.d_w_b, mask=m_view, v_row=v_row[guard:-guard], v_col=v_col[guard:-guard])
    torch.cuda.synchronize()
    assert np.array_equal(host(m_view), L.mask)
    assert np.array_equal(bits(host(v_row[guard:-guard])), bits(L.v_row))
    assert np.array_equal(bits(host(v_col[guard:-guard])), bits(L.v_col))
    for buf, fill in ((mask, 0x5A5A5A5A), (v_row, 123.0), (v_col, 123.0)):  # canaries untouched
        assert bool((buf[:guard] == fill).all()) and bool((buf[-guard:] == fill).all())
    # one axis at a time gives the same answers, and a second run is bit-identical
    m2, vr2, none = api.pd_pack_delta(L.d_w_f, L.d_w_b, want_col=False)
    m3, none2, vc3 = api.pd_pack_delta(L.d_w_f, L.d_w_b, want_row=False)
    torch.cuda.synchronize()
    assert none is None and none2 is None
    assert np.array_equal(host(m2), L.mask) and np.array_equal(host(m3), L.mask)
    assert np.array_equal(bits(host(vr2)), bits(L.v_row)) and np.array_equal(bits(host(vc3)), bits(L.v_col))


def test_pack_large_magnitudes_take_the_exact_wide_path(api):
    # weights up to +-60000 and subnormals: the 64-bit fixed-point path must still be exact
    rng = np.random.default_rng(5)
    d_out, d_in = 96, 320
    w_b = (rng.standard_normal((d_out, d_in)) * rng.choice([1e-6, 1e-3, 0.3, 40.0, 9000.0], size=(d_out, d_in))).astype(np.float16)
    w_f = (w_b.astype(np.float64) + rng.standard_normal((d_out, d_in)) * rng.choice([1e-7, 1e-2, 5.0], size=(d_out, d_in))).astype(np.float16)
    w_f[3, 7] = w_b[3, 7]
    w_b[5, 9], w_f[5, 9] = np.float16(0.0), np.float16(-0.0)
    mask, v_row, v_col = orc.pack(w_f, w_b)
    m, vr, vc = api.pd_pack_delta(dev(w_f), dev(w_b))
    torch.cuda.synchronize()
    assert np.array_equal(host(m), mask)
    assert np.array_equal(bits(host(vr)), bits(v_row))
    assert np.array_equal(bits(host(vc)), bits(v_col))


# ------------------------------------------------------------------ merge
@pytest.mark.parametrize("axis", [ROW, COL])
@pytest.mark.parametrize("d_out,d_in", [(1024, 1024), (65, 96), (200, 1056), (4096, 4096), (11008, 4096)])
def test_merge_bit_exact(api, d_out, d_in, axis):
    L = layer(d_out, d_in)
    ref = orc.merge(L.w_b, L.mask, L.v(axis), axis)
    out = api.pd_merge(L.d_w_b, L.d_mask, L.d_v(axis), axis)
    torch.cuda.synchronize()
    assert np.array_equal(bits(host(out)), bits(ref))
    # in place over the base
    w = L.d_w_b.clone()
    api.pd_merge(w, L.d_mask, L.d_v(axis), axis, w_hat=w)
    torch.cuda.synchronize()
    assert np.array_equal(bits(host(w)), bits(ref))


def test_merge_wide_exponent_range(api):
    rng = np.random.default_rng(6)
    d_out, d_in = 64, 256
    w_b = rng.integers(0, 0x7800, size=(d_out, d_in)).astype(np.uint16)
    w_b ^= (rng.integers(0, 2, size=(d_out, d_in)).astype(np.uint16) << 15)
    w_b = w_b.view(np.float16)
    mask = rng.integers(0, 2 ** 32, size=(d_out, d_in // 32), dtype=np.uint64).astype(np.uint32)
    for axis, n in ((ROW, d_out), (COL, d_in)):
        v = rng.integers(0, 0x5000, size=n).astype(np.uint16).view(np.float16)
        ref = orc.merge(w_b, mask, v, axis)
        out = api.pd_merge(dev(w_b), dev(mask), dev(v), axis)
        torch.cuda.synchronize()
        assert np.array_equal(bits(host(out)), bits(ref))


def test_pack_merge_round_trip_on_device(api):
    L = layer(1024, 1024)
    w_hat = api.pd_merge(L.d_w_b, L.d_mask, L.d_v_row, ROW)
    m2, _, _ = api.pd_pack_delta(w_hat, L.d_w_b)
    torch.cuda.synchronize()
    moved = bits(host(w_hat)) != bits(L.w_b)
    b1, b2 = orc.unpack(L.mask, 1024), orc.unpack(host(m2), 1024)
    assert np.array_equal(b1[moved], b2[moved])


# ------------------------------------------------------------------ decode linear
def check_linear(api, L, m, axis, seed=2000, ldx_pad=0):
    x = synth.gen_x(m, L.d_in, seed)
    ref = orc.linear(x, L.w_b, L.mask, L.v(axis), axis)
    d_x = dev(x)
    if ldx_pad:
        buf = torch.zeros((m, L.d_in + ldx_pad), dtype=torch.float16, device="cuda")
        buf[:, :L.d_in] = d_x
        d_x = buf[:, :L.d_in]
    y = api.pd_linear(d_x, L.d_w_b, L.d_mask, L.d_v(axis), axis)
    y2 = api.pd_linear(d_x, L.d_w_b, L.d_mask, L.d_v(axis), axis)
    torch.cuda.synchronize()
    assert api.pd_device_status() == 0
    err = rel_err(host(y), ref)
    assert err <= TOL, (L.d_out, L.d_in, m, axis, err)
    assert torch.equal(y, y2), "two runs must be bit-identical"
    return err


@pytest.mark.parametrize("axis", [ROW, COL])
@pytest.mark.parametrize("m", [1, 16])
def test_linear_config1(api, m, axis):
    check_linear(api, layer(1024, 1024), m, axis)


@pytest.mark.parametrize("axis", [ROW, COL])
@pytest.mark.parametrize("d_out,d_in,m", [(200, 1152, 3), (130, 384, 8), (65, 128, 9), (129, 2304, 16), (8, 128, 1),
                                          (1000, 4224, 5), (64, 96, 7), (33, 1056, 16), (300, 32, 2)])
def test_linear_ragged_shapes(api, d_out, d_in, m, axis):
    check_linear(api, layer(d_out, d_in, seed=3), m, axis, ldx_pad=8 if m % 2 else 0)


@pytest.mark.parametrize("axis", [ROW, COL])
@pytest.mark.parametrize("d_out,d_in", [(4096, 4096), (11008, 4096), (4096, 11008)])
def test_linear_7b_decode(api, d_out, d_in, axis):
    L = layer(d_out, d_in)
    for m in (1, 4, 16):
        check_linear(api, L, m, axis)


def test_linear_sign_expansion_is_exact(api):
    # W_b = 0, v = 1, small integer x: y = x . B^T is an exact integer, any bit-order slip shows
    rng = np.random.default_rng(8)
    d_out, d_in, m = 136, 640, 16
    w_b = np.zeros((d_out, d_in), dtype=np.float16)
    w_f = rng.choice([-1.0, 1.0], size=(d_out, d_in)).astype(np.float16)
    mask, _, _ = orc.pack(w_f, w_b)
    x = rng.integers(-3, 4, size=(m, d_in)).astype(np.float16)
    ref = x.astype(np.float64) @ w_f.astype(np.float64).T
    for axis, n in ((ROW, d_out), (COL, d_in)):
        y = api.pd_linear(dev(x), dev(w_b), dev(mask), dev(np.ones(n, dtype=np.float16)), axis)
        torch.cuda.synchronize()
        assert np.array_equal(host(y).astype(np.float64), ref)


def test_linear_base_only_and_one_hot(api):
    L = layer(1024, 1024)
    x = synth.gen_x(4, 1024, 7)
    y = api.pd_linear(dev(x), L.d_w_b, None, None, ROW)
    torch.cuda.synchronize()
    ref = x.astype(np.float64) @ L.w_b.astype(np.float64).T
    assert rel_err(host(y), ref) <= TOL
    # one-hot rows pick out columns of the merged weights exactly (one product, one fp32 add, RN16)
    cols = [0, 1, 31, 32, 517, 1023]
    xo = np.zeros((len(cols), 1024), dtype=np.float16)
    xo[np.arange(len(cols)), cols] = 1.0
    for axis in (ROW, COL):
        y = api.pd_linear(dev(xo), L.d_w_b, L.d_mask, L.d_v(axis), axis)
        torch.cuda.synchronize()
        merged = orc.merge(L.w_b, L.mask, L.v(axis), axis)
        assert np.array_equal(bits(host(y)), bits(merged[:, cols].T))


@pytest.mark.parametrize("m", [17, 33, 40])
def test_linear_between_decode_and_prefill(api, m):
    check_linear(api, layer(1024, 1024), m, ROW)
    check_linear(api, layer(200, 1152, seed=3), m, COL)


def test_linear_host_buffers_side_stream_and_odd_output_pitch(api):
    # pd_linear_host: x from pinned host memory, y back to pinned host memory, on a non-default stream
    L = layer(1024, 1024)
    for m in (4, 40):
        x = synth.gen_x(m, 1024, 30 + m)
        ref = orc.linear(x, L.w_b, L.mask, L.v_col, COL)
        x_host = torch.from_numpy(x).pin_memory()
        y_host = torch.empty((m, 1024), dtype=torch.float16).pin_memory()
        x_dev = torch.empty((m, 1024), dtype=torch.float16, device="cuda")
        y_dev = torch.empty((m, 1024), dtype=torch.float16, device="cuda")
        side = torch.cuda.Stream()
        side.wait_stream(torch.cuda.current_stream())
        with torch.cuda.stream(side):
            api.pd_linear_host(x_host, x_dev, L.d_w_b, L.d_mask, L.d_v_col, COL, y_dev, y_host)
        side.synchronize()
        assert rel_err(y_host.numpy(), ref) <= TOL
        # an output view with an odd row pitch and a 2-byte-aligned base: the vector stores must not be used
        buf = torch.zeros((m, 1024 + 3), dtype=torch.float16, device="cuda")
        y_view = buf[:, 1:1025]
        api.pd_linear(dev(x), L.d_w_b, L.d_mask, L.d_v_col, COL, y=y_view)
        torch.cuda.synchronize()
        assert api.pd_device_status() == 0
        assert rel_err(host(y_view), ref) <= TOL
        assert bool((buf[:, 0] == 0).all()) and bool((buf[:, 1025:] == 0).all())


# ------------------------------------------------------------------ prefill linear (tensor-core path)
def check_prefill(api, L, m, axis, rows=None, seed=2000):
    x = synth.gen_x(m, L.d_in, seed)
    y = api.pd_linear(dev(x), L.d_w_b, L.d_mask, L.d_v(axis), axis)
    y2 = api.pd_linear(dev(x), L.d_w_b, L.d_mask, L.d_v(axis), axis)
    torch.cuda.synchronize()
    assert api.pd_device_status() == 0
    assert torch.equal(y, y2)
    yh = host(y)
    if rows is None:
        ref = orc.linear(x, L.w_b, L.mask, L.v(axis), axis)
        err = rel_err(yh, ref)
    else:
        ref = orc.linear(np.ascontiguousarray(x[rows]), L.w_b, L.mask, L.v(axis), axis)
        err = rel_err(yh[rows], ref)
        assert np.isfinite(yh.astype(np.float32)).all()
    assert err <= TOL, (L.d_out, L.d_in, m, axis, err)
    return err


@pytest.mark.parametrize("axis", [ROW, COL])
@pytest.mark.parametrize("d_out,d_in,m", [(1024, 1024, 256), (128, 64, 65), (200, 1152, 100), (130, 96, 257),
                                          (1000, 4224, 300), (64, 32, 70), (129, 2304, 513), (256, 512, 1024)])
def test_prefill_small_shapes(api, d_out, d_in, m, axis):
    check_prefill(api, layer(d_out, d_in, seed=3 if d_out != 1024 else 0), m, axis)


def test_prefill_base_only_and_exact_signs(api):
    L = layer(1024, 1024)
    x = synth.gen_x(300, 1024, 7)
    y = api.pd_linear(dev(x), L.d_w_b, None, None, ROW)
    torch.cuda.synchronize()
    assert rel_err(host(y), x.astype(np.float64) @ L.w_b.astype(np.float64).T) <= TOL
    # W_b = 0, v = 1: W_hat = B exactly, small-integer x gives exact integer outputs
    rng = np.random.default_rng(9)
    d_out, d_in, m = 200, 320, 130
    w_b = np.zeros((d_out, d_in), dtype=np.float16)
    w_f = rng.choice([-1.0, 1.0], size=(d_out, d_in)).astype(np.float16)
    mask, _, _ = orc.pack(w_f, w_b)
    xi = rng.integers(-3, 4, size=(m, d_in)).astype(np.float16)
    ref = xi.astype(np.float64) @ w_f.astype(np.float64).T
    for axis, n in ((ROW, d_out), (COL, d_in)):
        y = api.pd_linear(dev(xi), dev(w_b), dev(mask), dev(np.ones(n, dtype=np.float16)), axis)
        torch.cuda.synchronize()
        assert api.pd_device_status() == 0
        assert np.array_equal(host(y).astype(np.float64), ref)


@pytest.mark.parametrize("axis", [ROW, COL])
def test_prefill_7b_m256_full(api, axis):
    check_prefill(api, layer(4096, 4096), 256, axis)


@pytest.mark.parametrize("axis", [ROW, COL])
# every 7B shape at M = 256, 2048 and 8192 (4096 x 4096 at M = 256 is checked in full above); (4096, 4096, 512) takes
# 128-token tiles, (11008, 4096, 256) one 256-token tile per pair of CTAs, the others full 256-token tiles.
# Rows checked: m mod 128 in {0, 1, 127} plus 64 seeded random rows, every output column.
@pytest.mark.parametrize("d_out,d_in,m", [(4096, 4096, 2048), (11008, 4096, 2048), (4096, 11008, 2048), (4096, 4096, 8192),
                                          (11008, 4096, 8192), (4096, 11008, 8192), (4096, 4096, 512), (11008, 4096, 256),
                                          (4096, 11008, 256)])
def test_prefill_7b_sampled_rows(api, d_out, d_in, m, axis):
    check_prefill(api, layer(d_out, d_in), m, axis, rows=synth.sample_rows(m, n_random=64))


@pytest.mark.parametrize("axis", [ROW, COL])
@pytest.mark.parametrize("d_out,d_in,m", [(1152, 992, 4000), (1100, 1088, 3900), (256, 4096, 37000)])
def test_prefill_cta_pair_ragged_edges(api, d_out, d_in, m, axis):
    # sizes that take the 256-row x 256-token tiles of the two-CTA kernel with ragged edges: an odd number of
    # 128-row tiles (the second CTA of the last pair has no rows at all), rows and tokens that end inside a tile,
    # a last k step of 32 columns, and one row-tile pair walking many token tiles
    L = layer(d_out, d_in, seed=5)
    rows = np.unique(np.concatenate([synth.sample_rows(m, n_random=24), np.arange(m - 130, m), np.arange(120, 136)]))
    check_prefill(api, L, m, axis, rows=rows)


@pytest.mark.parametrize("axis", [ROW, COL])
@pytest.mark.parametrize("d_out,d_in,m", [(256, 160, 17), (257, 96, 33), (383, 992, 64), (385, 224, 65), (512, 64, 129),
                                          (300, 2080, 255), (640, 128, 257), (1100, 1088, 31)])
def test_linear_tensor_core_edge_sizes(api, d_out, d_in, m, axis):
    # the smallest layers that take the two-CTA tiles (256 rows and up), with row counts on both sides of a 128-row
    # tile, token counts on both sides of the 32-token MMA granule and of the 64/128/256-token tiles, one and two
    # k steps, an odd number of k steps (padded to even) and a last k step of 32 columns; checked on every output
    L = layer(d_out, d_in, seed=11)
    check_prefill(api, L, m, axis)
    x = synth.gen_x(m, d_in, 77)
    y = api.pd_linear(dev(x), L.d_w_b, None, None, ROW)  # base only through the same tiles
    torch.cuda.synchronize()
    assert api.pd_device_status() == 0
    assert rel_err(host(y), x.astype(np.float64) @ L.w_b.astype(np.float64).T) <= TOL


# ------------------------------------------------------------------ multi-variant
def make_variants(w_b, n_var, seed, mixed_axes=True, axis=ROW):
    d_out, d_in = w_b.shape
    masks = np.empty((n_var, d_out, d_in // 32), dtype=np.uint32)
    stride = (max(d_out, d_in) + 7) // 8 * 8  # each variant's scales must start 16-byte aligned
    vs = np.zeros((n_var, stride), dtype=np.float16)
    axes = np.zeros(n_var, dtype=np.uint8)
    for g in range(n_var):
        w_f = synth.gen_finetuned(w_b, 1000 + seed + g)
        m, vr, vc = orc.pack(w_f, w_b)
        masks[g] = m
        axes[g] = (g % 2) if mixed_axes else axis
        if axes[g] == ROW:
            vs[g, :d_out] = vr
        else:
            vs[g, :d_in] = vc
    return masks, vs, axes


@pytest.mark.parametrize("d_out,d_in,n_var,m", [(256, 512, 3, 20), (200, 1152, 4, 37), (130, 96, 2, 9), (1024, 1024, 16, 64)])
def test_multivariant_small(api, d_out, d_in, n_var, m):
    w_b = synth.gen_base(d_out, d_in, 11)
    masks, vs, axes = make_variants(w_b, n_var, 11)
    x = synth.gen_x(m, d_in, 12)
    ids = synth.gen_ids(m, n_var, 13)
    ids[1] = -1
    ids[m - 1] = -1
    ref, bad = orc.linear_multivariant(x, ids, w_b, masks, vs, axes)
    assert bad == 0
    args = (dev(x), dev(ids), dev(w_b), dev(masks), dev(vs), axes)
    y = api.pd_linear_multivariant(*args)
    y2 = api.pd_linear_multivariant(*args)
    torch.cuda.synchronize()
    assert api.pd_device_status() == 0
    assert rel_err(host(y), ref) <= TOL
    assert torch.equal(y, y2)
    # per-row check too: no row may borrow another variant's delta
    yh = host(y).astype(np.float64)
    for r in range(m):
        assert np.max(np.abs(yh[r] - ref[r])) / np.max(np.abs(ref[r])) <= 2 * TOL


# (384, 320, 2, 700) and (640, 992, 3, 1000): buckets of more than 256 rows are cut into several tiles of the two-CTA kernel
@pytest.mark.parametrize("d_out,d_in,n_var,m", [(256, 512, 5, 300), (200, 1152, 3, 150), (1024, 1024, 16, 2112), (130, 96, 2, 700),
                                                (384, 320, 2, 700), (640, 992, 3, 1000)])
def test_multivariant_prefill_sized(api, d_out, d_in, n_var, m):
    # more than 64 rows: rows are bucketed by variant and run through the grouped tensor-core kernel
    w_b = synth.gen_base(d_out, d_in, 21)
    masks, vs, axes = make_variants(w_b, n_var, 21)
    x = synth.gen_x(m, d_in, 22)
    ids = synth.gen_ids(m, n_var, 23)
    ids[::37] = -1
    ref, bad = orc.linear_multivariant(x, ids, w_b, masks, vs, axes)
    assert bad == 0
    args = (dev(x), dev(ids), dev(w_b), dev(masks), dev(vs), axes)
    y = api.pd_linear_multivariant(*args)
    y2 = api.pd_linear_multivariant(*args)
    torch.cuda.synchronize()
    assert api.pd_device_status() == 0
    yh = host(y).astype(np.float64)
    assert np.isfinite(yh).all()
    assert rel_err(host(y), ref) <= TOL
    assert torch.equal(y, y2)
    for r in range(0, m, 7):  # no row may borrow another variant's delta
        assert np.max(np.abs(yh[r] - ref[r])) / np.max(np.abs(ref[r])) <= 2 * TOL


def pack_variants(w_b, n_var, seed):
    """Masks and both scale vectors of n_var fine-tunes of w_b (the oracle's pack)."""
    d_out, d_in = w_b.shape
    masks = np.empty((n_var, d_out, d_in // 32), dtype=np.uint32)
    v_rows = np.empty((n_var, d_out), dtype=np.float16)
    v_cols = np.empty((n_var, d_in), dtype=np.float16)
    for g in range(n_var):
        masks[g], v_rows[g], v_cols[g] = orc.pack(synth.gen_finetuned(w_b, 1000 + seed + g), w_b)
    return masks, v_rows, v_cols


def scales_for(axes, v_rows, v_cols):
    n_var, d_out, d_in = len(axes), v_rows.shape[1], v_cols.shape[1]
    vs = np.zeros((n_var, (max(d_out, d_in) + 7) // 8 * 8), dtype=np.float16)
    for g in range(n_var):
        if axes[g] == ROW:
            vs[g, :d_out] = v_rows[g]
        else:
            vs[g, :d_in] = v_cols[g]
    return vs


def check_multivariant_rows(api, x, ids, w_b, masks, vs, axes, d_w_b, d_masks, rows, expect_status=0):
    y = api.pd_linear_multivariant(dev(x), dev(ids), d_w_b, d_masks, dev(vs), axes)
    y2 = api.pd_linear_multivariant(dev(x), dev(ids), d_w_b, d_masks, dev(vs), axes)
    torch.cuda.synchronize()
    assert api.pd_device_status() == expect_status
    assert torch.equal(y[rows], y2[rows]), "two runs must be bit-identical"
    ref, _ = orc.linear_multivariant(np.ascontiguousarray(x[rows]), np.ascontiguousarray(ids[rows]), w_b, masks, vs, axes)
    yh = host(y).astype(np.float64)
    assert np.isfinite(yh[rows]).all()
    assert rel_err(yh[rows], ref) <= TOL
    for i, r in enumerate(rows):  # row by row: no row may borrow another variant's delta
        assert np.max(np.abs(yh[r] - ref[i])) / np.max(np.abs(ref[i])) <= 2 * TOL


# the multi-variant serving batch at full size on every 7B shape: 16 variants over one base; 64 decode rows (own id
# each), 64 + 4 x 512 rows with an id per row, and the same with one id per 512-row sequence; uniform row axis
# (both per-row batches), uniform col axis (decode batch) and mixed axes (decode batch and per-sequence batch);
# oracle on all 64 decode rows / on m mod 128 in {0, 1, 127} plus 64 random rows
@pytest.mark.parametrize("d_out,d_in", [(4096, 4096), (11008, 4096), (4096, 11008)])
def test_multivariant_7b_shapes_16_variants(api, d_out, d_in):
    n_var = 16
    w_b = synth.gen_base(d_out, d_in, 31)
    masks, v_rows, v_cols = pack_variants(w_b, n_var, 31)
    d_w_b, d_masks = dev(w_b), dev(masks)
    batches = [(64, synth.gen_ids(64, n_var, 33)), (2112, synth.gen_ids(2112, n_var, 34)),
               (2112, synth.gen_ids_per_sequence(64, 4, 512, n_var, 35))]
    plan = (("row", [ROW] * n_var, batches[:2]), ("col", [COL] * n_var, batches[:1]),
            ("mixed", [g % 2 for g in range(n_var)], batches[::2]))
    for name, axes, todo in plan:
        axes = np.array(axes, dtype=np.uint8)
        vs = scales_for(axes, v_rows, v_cols)
        for m, ids in todo:
            x = synth.gen_x(m, d_in, 32 + m)
            rows = np.arange(m) if m <= 64 else synth.sample_rows(m, n_random=64)
            check_multivariant_rows(api, x, ids, w_b, masks, vs, axes, d_w_b, d_masks, rows)
    del d_w_b, d_masks
    torch.cuda.empty_cache()


# decode-sized batches through the one-pass kernel: few rows, few or many variants, ids of -1, mixed axes,
# more than eight rows of one variant, more items than one pass holds
@pytest.mark.parametrize("d_out,d_in", [(1024, 1024), (4096, 4096)])
def test_multivariant_decode_batches(api, d_out, d_in):
    w_b = synth.gen_base(d_out, d_in, 41)
    masks, v_rows, v_cols = pack_variants(w_b, 16, 41)
    d_w_b = dev(w_b)
    for m, n_var, seed in ((5, 4, 1), (16, 4, 2), (16, 16, 3), (5, 16, 4), (1, 16, 5), (40, 2, 6), (64, 16, 7)):
        axes = np.array([g % 2 for g in range(n_var)], dtype=np.uint8)
        vs = scales_for(axes, v_rows[:n_var], v_cols[:n_var])
        ids = synth.gen_ids(m, n_var, 50 + seed)
        if m >= 5:
            ids[1] = -1
            ids[m - 1] = -1
        x = synth.gen_x(m, d_in, 60 + seed)
        check_multivariant_rows(api, x, ids, w_b, masks[:n_var], vs, axes, d_w_b, dev(masks[:n_var]), np.arange(m))
    # 64 rows over 64 variants: 64 items, four passes
    if d_out == 1024:
        masks64 = np.concatenate([masks] * 4)
        axes = np.array([g % 2 for g in range(64)], dtype=np.uint8)
        vs = scales_for(axes, np.concatenate([v_rows] * 4), np.concatenate([v_cols] * 4))
        ids = np.arange(64, dtype=np.int32)[::-1].copy()
        x = synth.gen_x(64, d_in, 70)
        check_multivariant_rows(api, x, ids, w_b, masks64, vs, axes, d_w_b, dev(masks64), np.arange(64))


def test_multivariant_bad_id_is_latched(api):
    w_b = synth.gen_base(128, 128, 14)
    masks, vs, axes = make_variants(w_b, 2, 14)
    x = synth.gen_x(6, 128, 15)
    ids = np.array([0, 1, 5, 0, -1, 1], dtype=np.int32)
    y = api.pd_linear_multivariant(dev(x), dev(ids), dev(w_b), dev(masks), dev(vs), axes)
    assert api.pd_device_status() == 6  # PD_ERR_BAD_VARIANT
    assert api.pd_device_status() == 0  # cleared by the read
    ref, bad = orc.linear_multivariant(x, ids, w_b, masks, vs, axes)
    assert bad == 1
    keep = [0, 1, 3, 4, 5]
    assert rel_err(host(y)[keep], ref[keep]) <= TOL


@pytest.mark.parametrize("m", [40, 100])
def test_multivariant_bad_id_in_a_larger_batch(api, m):
    # one id out of range among m rows, on a private zero-filled workspace: m = 40 runs the one-pass decode kernel,
    # m = 100 the sorted tensor-core path (whose gather must skip the row that belongs to no bucket).  The call
    # latches PD_ERR_BAD_VARIANT and every other row is still right.
    d_out, d_in, n_var = 256, 512, 3
    w_b = synth.gen_base(d_out, d_in, 16)
    masks, vs, axes = make_variants(w_b, n_var, 16)
    x = synth.gen_x(m, d_in, 17)
    ids = synth.gen_ids(m, n_var, 18)
    ids[7] = n_var + 4
    ws = torch.zeros(api.workspace_bytes(api.OP_LINEAR_MULTIVARIANT, m, n_var, d_out, d_in), dtype=torch.uint8, device="cuda")
    y = api.pd_linear_multivariant(dev(x), dev(ids), dev(w_b), dev(masks), dev(vs), axes, workspace=ws)
    assert api.pd_device_status(workspace=ws) == 6  # PD_ERR_BAD_VARIANT
    assert api.pd_device_status(workspace=ws) == 0
    ref, bad = orc.linear_multivariant(x, ids, w_b, masks, vs, axes)
    assert bad == 1
    keep = [r for r in range(m) if r != 7]
    assert rel_err(host(y)[keep], ref[keep]) <= TOL


# ------------------------------------------------------------------ stream order, failure path
def test_linear_right_after_pack_and_merge_on_one_stream(api):
    # pd_pack_delta -> pd_linear and pd_merge -> pd_linear(w_hat, mask = NULL), queued back to back with no
    # synchronisation in between and with the intermediate buffers full of garbage beforehand: the decode kernel
    # may start early (programmatic dependent launch) but must not read the weights before they are written
    for d_out, d_in in ((4096, 4096), (1024, 1024)):
        L = layer(d_out, d_in)
        x = synth.gen_x(4, d_in, 80)
        d_x = dev(x)
        for axis in (ROW, COL):
            ref = orc.linear(x, L.w_b, L.mask, L.v(axis), axis)
            merged = orc.merge(L.w_b, L.mask, L.v(axis), axis)
            ref_dense = x.astype(np.float64) @ merged.astype(np.float64).T
            for rep in range(3):
                mask = torch.full((d_out, d_in // 32), 0x5A5A5A5A, dtype=torch.int32, device="cuda")
                v_row = torch.full((d_out,), 77.0, dtype=torch.float16, device="cuda")
                v_col = torch.full((d_in,), 77.0, dtype=torch.float16, device="cuda")
                w_hat = torch.full((d_out, d_in), 55.0, dtype=torch.float16, device="cuda")
                torch.cuda.synchronize()
                api.pd_pack_delta(L.d_w_f, L.d_w_b, mask=mask, v_row=v_row, v_col=v_col)
                y = api.pd_linear(d_x, L.d_w_b, mask, v_row if axis == ROW else v_col, axis)
                api.pd_merge(L.d_w_b, mask, v_row if axis == ROW else v_col, axis, w_hat=w_hat)
                y_dense = api.pd_linear(d_x, w_hat, None, None, ROW)
                torch.cuda.synchronize()
                assert api.pd_device_status() == 0
                assert rel_err(host(y), ref) <= TOL
                assert rel_err(host(y_dense), ref_dense) <= TOL
    # the resident-weights flag gives the same numbers when the weights really are resident
    L = layer(1024, 1024)
    x = synth.gen_x(16, 1024, 81)
    y0 = api.pd_linear(dev(x), L.d_w_b, L.d_mask, L.d_v_row, ROW)
    y1 = api.pd_linear(dev(x), L.d_w_b, L.d_mask, L.d_v_row, ROW, weights_resident=True)
    torch.cuda.synchronize()
    assert torch.equal(y0, y1)


def test_bounded_wait_runs_out_and_is_reported(api):
    # a wait that nothing satisfies gives up after its limit, latches PD_ERR_DEVICE_TIMEOUT and the kernel returns;
    # the context stays usable
    ws = torch.zeros(1024, dtype=torch.uint8, device="cuda")
    api.pd_selftest_bounded_wait(100000, workspace=ws)
    torch.cuda.synchronize()
    assert int(ws[4:8].view(torch.int32).item()) == 99  # the detail word names the wait that gave up
    assert api.pd_device_status(workspace=ws) == 7  # PD_ERR_DEVICE_TIMEOUT
    assert api.pd_device_status(workspace=ws) == 0  # reading it clears it
    L = layer(1024, 1024)
    check_linear(api, L, 4, ROW)


def test_native_library_is_the_one_in_tree(api):
    import os
    assert os.path.basename(api.LIB_PATH) == "libpd.so" and os.path.exists(api.LIB_PATH)
    before = api.launch_count()
    L = layer(1024, 1024)
    api.pd_merge(L.d_w_b, L.d_mask, L.d_v_row, ROW)
    torch.cuda.synchronize()
    assert api.launch_count() == before + 1
