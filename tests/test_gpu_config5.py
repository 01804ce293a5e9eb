"""GPU parity at the 70B-block shapes (whole-model delta build + merge, 80 layers): for the first and the
last layer's seeds, pack -> merge -> decode GEMV at M = 1 on every distinct linear shape, against the CPU
oracle.  Pack and merge must be bit-exact; the fused GEMV and the dense GEMV on the merged weights must both
stay within 5e-3 of the oracle's fp64 result."""
import numpy as np
import pytest
import torch

from oracle import pd_oracle as orc
from paper_2512_19720_b200 import synth

pytestmark = pytest.mark.gpu
ROW, COL = 0, 1
TOL = 5e-3
# distinct shapes of a 70B block (q/o, k/v, gate/up, down); merge and both GEMVs run on both axes of every shape
SHAPES = [("q", 8192, 8192), ("k", 1024, 8192), ("gate", 28672, 8192), ("down", 8192, 28672)]


def dev(a):
    if a.dtype == np.uint32:
        a = a.view(np.int32)
    return torch.from_numpy(np.ascontiguousarray(a)).cuda()


def bits(t):
    a = t.detach().cpu().numpy()
    return a.view(np.uint16)


def rel_err(y, ref):
    return float(np.max(np.abs(y.astype(np.float64) - ref)) / np.max(np.abs(ref)))


@pytest.mark.parametrize("layer", [0, 79])
@pytest.mark.parametrize("name,d_out,d_in", SHAPES)
def test_build_merge_decode_70b_shapes(name, d_out, d_in, layer):
    assert torch.cuda.is_available(), "GPU tests need a CUDA device"
    from paper_2512_19720_b200 import api
    w_b = synth.gen_base(d_out, d_in, 100 + layer)
    w_f = synth.gen_finetuned(w_b, 1100 + layer)
    mask, v_row, v_col = orc.pack(w_f, w_b)
    d_w_b, d_w_f = dev(w_b), dev(w_f)
    del w_f

    g_mask, g_vr, g_vc = api.pd_pack_delta(d_w_f, d_w_b)
    torch.cuda.synchronize()
    del d_w_f
    assert np.array_equal(g_mask.cpu().numpy().view(np.uint32), mask)
    assert np.array_equal(bits(g_vr), v_row.view(np.uint16))
    assert np.array_equal(bits(g_vc), v_col.view(np.uint16))

    x = synth.gen_x(1, d_in, 2000 + layer)
    d_x = dev(x)
    for axis in (ROW, COL):
        v, g_v = (v_row, g_vr) if axis == ROW else (v_col, g_vc)
        w_hat = api.pd_merge(d_w_b, g_mask, g_v, axis)
        torch.cuda.synchronize()
        ref_hat = orc.merge(w_b, mask, v, axis)
        assert np.array_equal(bits(w_hat), ref_hat.view(np.uint16))
        del ref_hat
        ref = orc.linear(x, w_b, mask, v, axis)
        y_fused = api.pd_linear(d_x, d_w_b, g_mask, g_v, axis)
        y_dense = api.pd_linear(d_x, w_hat, None, None, ROW)  # the merged model: plain dense GEMV
        torch.cuda.synchronize()
        assert api.pd_device_status() == 0
        assert rel_err(y_fused.cpu().numpy(), ref) <= TOL
        assert rel_err(y_dense.cpu().numpy(), ref) <= TOL
        del w_hat
    del d_w_b, g_mask
    torch.cuda.empty_cache()
