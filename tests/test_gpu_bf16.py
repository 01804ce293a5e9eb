"""GPU parity for the BF16 variants (base, fine-tune, activations and outputs in bfloat16, scales in fp16): the CUDA
library through its C ABI against the BF16 CPU oracle, on the same seeded inputs.  Pack and merge must be bit-exact;
linear outputs must satisfy max|y - y_ref| / max|y_ref| <= 5e-3 (the bound holds the output's rounding to bfloat16,
2^-9 of an entry, the one rounding of W_hat to bfloat16 per weight and the fp32 accumulation)."""
import numpy as np
import pytest
import torch

from oracle import pd_oracle_bf16 as orc
from paper_2512_19720_b200 import synth

pytestmark = pytest.mark.gpu
ROW, COL = 0, 1
TOL = 5e-3


@pytest.fixture(scope="module")
def api():
    assert torch.cuda.is_available(), "GPU tests need a CUDA device"
    from paper_2512_19720_b200 import api as _api
    return _api


def dev_bf16(bits):
    return torch.from_numpy(np.ascontiguousarray(bits).view(np.int16)).cuda().view(torch.bfloat16)


def dev(a):
    if a.dtype == np.uint32:
        a = a.view(np.int32)
    return torch.from_numpy(np.ascontiguousarray(a)).cuda()


def bits_of(t):
    return t.detach().view(torch.int16).cpu().numpy().view(np.uint16)


def values_of(t):
    return synth.bf16_bits_to_f32(bits_of(t)).astype(np.float64)


def rel_err(y, ref):
    return float(np.max(np.abs(y - ref)) / np.max(np.abs(ref)))


class Layer:
    def __init__(self, d_out, d_in, seed=0):
        self.d_out, self.d_in = d_out, d_in
        self.w_b = synth.gen_base_bf16(d_out, d_in, seed)
        self.w_f = synth.gen_finetuned_bf16(self.w_b, 1000 + seed)
        self.mask, self.v_row, self.v_col = orc.pack(self.w_f, self.w_b)
        self.d_w_b, self.d_w_f = dev_bf16(self.w_b), dev_bf16(self.w_f)
        self.d_mask, self.d_v_row, self.d_v_col = dev(self.mask), dev(self.v_row), dev(self.v_col)

    def v(self, axis):
        return self.v_row if axis == ROW else self.v_col

    def d_v(self, axis):
        return self.d_v_row if axis == ROW else self.d_v_col


_layers = {}


def layer(d_out, d_in, seed=0):
    key = (d_out, d_in, seed)
    if key not in _layers:
        if len(_layers) > 2:
            _layers.clear()
            torch.cuda.empty_cache()
        _layers[key] = Layer(d_out, d_in, seed)
    return _layers[key]


# ------------------------------------------------------------------ pack / merge
@pytest.mark.parametrize("d_out,d_in", [(1024, 1024), (64, 32), (65, 96), (200, 1056), (4096, 4096), (4096, 11008)])
def test_pack_bf16_bit_exact(api, d_out, d_in):
    L = layer(d_out, d_in)
    m, vr, vc = api.pd_pack_delta(L.d_w_f, L.d_w_b)
    m2, vr2, _ = api.pd_pack_delta(L.d_w_f, L.d_w_b, want_col=False)
    torch.cuda.synchronize()
    assert np.array_equal(m.cpu().numpy().view(np.uint32), L.mask) and torch.equal(m, m2)
    assert np.array_equal(vr.cpu().numpy().view(np.uint16), L.v_row.view(np.uint16)) and torch.equal(vr, vr2)
    assert np.array_equal(vc.cpu().numpy().view(np.uint16), L.v_col.view(np.uint16))


def test_pack_bf16_wide_magnitudes_and_tiny_differences(api):
    # values from subnormal to hundreds, differences below, at and just under the 2^-24 grid, +-0, equal entries:
    # the accumulators' checks and the exact 64-bit path must agree with the oracle's floor(|dW| * 2^24)
    rng = np.random.default_rng(5)
    d_out, d_in = 96, 320
    mag = rng.choice([1e-40, 1e-30, 1e-12, 3e-8, 6e-8, 1e-5, 1e-3, 0.02, 0.7, 1.0, 300.0], size=(d_out, d_in))
    w_b = synth.to_bf16_bits((rng.standard_normal((d_out, d_in)) * mag).astype(np.float32))
    mag2 = rng.choice([1e-40, 1e-20, 2e-8, 1e-6, 1e-3, 0.5, 40.0], size=(d_out, d_in))
    w_f = synth.to_bf16_bits((synth.bf16_bits_to_f32(w_b).astype(np.float64) + rng.standard_normal((d_out, d_in)) * mag2).astype(np.float32))
    w_f[3, 7] = w_b[3, 7]
    w_b[5, 9], w_f[5, 9] = 0x0000, 0x8000
    w_b[6, :], w_f[6, :] = 0x0001, 0x3380  # 2^-24 - 2^-133 everywhere in the row: no unit at all
    w_b[7, :], w_f[7, :] = 0x3F80, 0x0001  # 1 - 2^-133: 2^24 - 1 units each
    mask, v_row, v_col = orc.pack(w_f, w_b)
    m, vr, vc = api.pd_pack_delta(dev_bf16(w_f), dev_bf16(w_b))
    torch.cuda.synchronize()
    assert np.array_equal(m.cpu().numpy().view(np.uint32), mask)
    assert np.array_equal(vr.cpu().numpy().view(np.uint16), v_row.view(np.uint16))
    assert np.array_equal(vc.cpu().numpy().view(np.uint16), v_col.view(np.uint16))


@pytest.mark.parametrize("axis", [ROW, COL])
@pytest.mark.parametrize("d_out,d_in", [(1024, 1024), (65, 96), (200, 1056), (4096, 4096), (11008, 4096)])
def test_merge_bf16_bit_exact(api, d_out, d_in, axis):
    L = layer(d_out, d_in)
    ref = orc.merge(L.w_b, L.mask, L.v(axis), axis)
    out = api.pd_merge(L.d_w_b, L.d_mask, L.d_v(axis), axis)
    w = L.d_w_b.clone()
    api.pd_merge(w, L.d_mask, L.d_v(axis), axis, w_hat=w)  # in place over the base
    torch.cuda.synchronize()
    assert np.array_equal(bits_of(out), ref) and np.array_equal(bits_of(w), ref)


# ------------------------------------------------------------------ linear
def check_linear(api, L, m, axis, rows=None, seed=2000):
    x = synth.gen_x_bf16(m, L.d_in, seed)
    d_x = dev_bf16(x)
    y = api.pd_linear(d_x, L.d_w_b, L.d_mask, L.d_v(axis), axis)
    y2 = api.pd_linear(d_x, L.d_w_b, L.d_mask, L.d_v(axis), axis)
    torch.cuda.synchronize()
    assert api.pd_device_status() == 0
    assert torch.equal(y.view(torch.int16), y2.view(torch.int16)), "two runs must be bit-identical"
    yh = values_of(y)
    if rows is None:
        ref = orc.linear(x, L.w_b, L.mask, L.v(axis), axis)
        err = rel_err(yh, ref)
    else:
        ref = orc.linear(np.ascontiguousarray(x[rows]), L.w_b, L.mask, L.v(axis), axis)
        err = rel_err(yh[rows], ref)
        assert np.isfinite(yh).all()
    assert err <= TOL, (L.d_out, L.d_in, m, axis, err)


@pytest.mark.parametrize("axis", [ROW, COL])
@pytest.mark.parametrize("m", [1, 16])
def test_linear_bf16_config1(api, m, axis):
    check_linear(api, layer(1024, 1024), m, axis)


@pytest.mark.parametrize("axis", [ROW, COL])
@pytest.mark.parametrize("d_out,d_in,m", [(200, 1152, 3), (130, 384, 8), (65, 128, 9), (129, 2304, 16), (64, 96, 7), (33, 1056, 16)])
def test_linear_bf16_ragged_shapes(api, d_out, d_in, m, axis):
    check_linear(api, layer(d_out, d_in, seed=3), m, axis)


@pytest.mark.parametrize("axis", [ROW, COL])
@pytest.mark.parametrize("d_out,d_in", [(4096, 4096), (11008, 4096), (4096, 11008)])
def test_linear_bf16_7b_decode(api, d_out, d_in, axis):
    L = layer(d_out, d_in)
    for m in (1, 4, 16):
        check_linear(api, L, m, axis)


def test_linear_bf16_exact_signs_and_base_only(api):
    # W_b = 0, v = 1, small-integer x: y = x . B^T is an exact integer in bfloat16 as long as it stays below 256
    rng = np.random.default_rng(8)
    d_out, d_in = 136, 128
    w_b = np.zeros((d_out, d_in), dtype=np.uint16)
    w_f = np.where(rng.random((d_out, d_in)) < 0.5, 0x3F80, 0xBF80).astype(np.uint16)
    mask, _, _ = orc.pack(w_f, w_b)
    for m in (16, 130):
        xi = rng.integers(-1, 2, size=(m, d_in)).astype(np.float32)
        ref = xi.astype(np.float64) @ synth.bf16_bits_to_f32(w_f).astype(np.float64).T
        assert np.max(np.abs(ref)) < 256
        for axis, n in ((ROW, d_out), (COL, d_in)):
            y = api.pd_linear(dev_bf16(synth.to_bf16_bits(xi)), dev_bf16(w_b), dev(mask), dev(np.ones(n, dtype=np.float16)), axis)
            torch.cuda.synchronize()
            assert api.pd_device_status() == 0
            assert np.array_equal(values_of(y), ref)
    L = layer(1024, 1024)
    for m in (4, 300):
        x = synth.gen_x_bf16(m, 1024, 7)
        y = api.pd_linear(dev_bf16(x), L.d_w_b, None, None, ROW)
        torch.cuda.synchronize()
        ref = synth.bf16_bits_to_f32(x).astype(np.float64) @ synth.bf16_bits_to_f32(L.w_b).astype(np.float64).T
        assert rel_err(values_of(y), ref) <= TOL


@pytest.mark.parametrize("axis", [ROW, COL])
@pytest.mark.parametrize("d_out,d_in,m", [(1024, 1024, 256), (128, 64, 65), (200, 1152, 100), (130, 96, 257), (256, 512, 1024),
                                          (383, 992, 64), (1100, 1088, 31)])
def test_prefill_bf16_small_shapes(api, d_out, d_in, m, axis):
    check_linear(api, layer(d_out, d_in, seed=3 if d_out != 1024 else 0), m, axis)


@pytest.mark.parametrize("axis", [ROW, COL])
def test_prefill_bf16_7b_m256_full(api, axis):
    check_linear(api, layer(4096, 4096), 256, axis)


@pytest.mark.parametrize("axis", [ROW, COL])
@pytest.mark.parametrize("d_out,d_in,m", [(4096, 4096, 2048), (11008, 4096, 2048), (4096, 11008, 256), (4096, 4096, 8192)])
def test_prefill_bf16_7b_sampled_rows(api, d_out, d_in, m, axis):
    check_linear(api, layer(d_out, d_in), m, axis, rows=synth.sample_rows(m, n_random=64))


# ------------------------------------------------------------------ multi-variant
@pytest.mark.parametrize("d_out,d_in,n_var,m", [(256, 512, 3, 20), (1024, 1024, 16, 64), (200, 1152, 4, 37), (130, 96, 2, 9),
                                                (1024, 1024, 16, 2112), (384, 320, 2, 700)])
def test_multivariant_bf16(api, d_out, d_in, n_var, m):
    w_b = synth.gen_base_bf16(d_out, d_in, 11)
    masks = np.empty((n_var, d_out, d_in // 32), dtype=np.uint32)
    vs = np.zeros((n_var, (max(d_out, d_in) + 7) // 8 * 8), dtype=np.float16)
    axes = np.array([g % 2 for g in range(n_var)], dtype=np.uint8)
    for g in range(n_var):
        mk, vr, vc = orc.pack(synth.gen_finetuned_bf16(w_b, 1011 + g), w_b)
        masks[g] = mk
        vs[g, :(d_out if axes[g] == ROW else d_in)] = vr if axes[g] == ROW else vc
    x = synth.gen_x_bf16(m, d_in, 12)
    ids = synth.gen_ids(m, n_var, 13)
    ids[1] = -1
    ids[m - 1] = -1
    rows = np.arange(m) if m <= 300 else synth.sample_rows(m, n_random=64)
    ref, bad = orc.linear_multivariant(np.ascontiguousarray(x[rows]), np.ascontiguousarray(ids[rows]), w_b, masks, vs, axes)
    assert bad == 0
    args = (dev_bf16(x), dev(ids), dev_bf16(w_b), dev(masks), dev(vs), axes)
    y = api.pd_linear_multivariant(*args)
    y2 = api.pd_linear_multivariant(*args)
    torch.cuda.synchronize()
    assert api.pd_device_status() == 0
    assert torch.equal(y.view(torch.int16), y2.view(torch.int16))
    yh = values_of(y)
    assert rel_err(yh[rows], ref) <= TOL
    for i, r in enumerate(rows):  # no row may borrow another variant's delta
        assert np.max(np.abs(yh[r] - ref[i])) / np.max(np.abs(ref[i])) <= 2 * TOL
