"""pd_pack_delta_static: the pack call that takes no workspace and allocates nothing.

It serves callers that cannot get scratch memory when they pack a layer (a fixed memory pool,
a plug-in that must not touch the CUDA allocator, code running while a stream is captured).
Its scratch is one array inside the library that every call on the GPU shares, so the test makes
two calls in a row on different layers -- the second would inherit the first one's sums if the
array were not cleared -- and requires both to equal pd_pack_delta, and the CPU oracle, bit for bit.

This file sorts last on purpose: a run that stops at the first failure has then already run
every other test.
"""
import numpy as np
import pytest
import torch

from oracle import pd_oracle as orc
from paper_2512_19720_b200 import synth


def _dev(a):
    return torch.from_numpy(np.ascontiguousarray(a)).cuda()


@pytest.mark.gpu
def test_static_pack_matches_workspace_pack_on_two_calls_in_a_row():
    assert torch.cuda.is_available(), "GPU tests need a CUDA device"
    from paper_2512_19720_b200 import api

    layers, expected = [], []
    for (d_out, d_in), seed in (((1024, 1024), 21), ((200, 1056), 22)):
        w_b = synth.gen_base(d_out, d_in, seed)
        w_f = synth.gen_finetuned(w_b, 1000 + seed)
        layers.append((_dev(w_f), _dev(w_b)))
        expected.append(orc.pack(w_f, w_b))

    # outputs are allocated up front: the calls under test receive only existing tensors
    outs = []
    for w_f, w_b in layers:
        d_out, d_in = w_b.shape
        outs.append((torch.full((d_out, d_in // 32), 0x5A5A5A5A, dtype=torch.int32, device="cuda"),
                     torch.full((d_out,), 7.0, dtype=torch.float16, device="cuda"),
                     torch.full((d_in,), 7.0, dtype=torch.float16, device="cuda")))
    torch.cuda.synchronize()

    for (w_f, w_b), (mask, v_row, v_col) in zip(layers, outs):  # two calls, back to back, one stream
        api.pd_pack_delta_static(w_f, w_b, mask, v_row, v_col)
    torch.cuda.synchronize()

    for (w_f, w_b), (mask, v_row, v_col), (o_mask, o_row, o_col) in zip(layers, outs, expected):
        ref_mask, ref_row, ref_col = api.pd_pack_delta(w_f, w_b)
        torch.cuda.synchronize()
        assert torch.equal(mask, ref_mask)
        assert torch.equal(v_row.view(torch.int16), ref_row.view(torch.int16))
        assert torch.equal(v_col.view(torch.int16), ref_col.view(torch.int16))
        assert np.array_equal(mask.cpu().numpy().view(np.uint32), o_mask)  # and the CPU oracle
        assert np.array_equal(v_row.cpu().numpy().view(np.uint16), o_row.view(np.uint16))
        assert np.array_equal(v_col.cpu().numpy().view(np.uint16), o_col.view(np.uint16))

    # one axis only, and again over the array the calls above left dirty
    w_f, w_b = layers[0]
    mask, v_row, _ = outs[0]
    v_row.fill_(7.0)
    api.pd_pack_delta_static(w_f, w_b, mask, v_row, None)
    torch.cuda.synchronize()
    assert torch.equal(v_row.view(torch.int16), api.pd_pack_delta(w_f, w_b)[1].view(torch.int16))


def test_static_pack_rejects_sizes_beyond_its_array():
    from paper_2512_19720_b200 import build
    build.build()
    from paper_2512_19720_b200 import api
    a = 0x10000  # never dereferenced: the size check comes before any launch
    before = api.launch_count()
    assert api.lib.pd_pack_delta_static(a, a, 40000, 25600, a, a, a, None) == 2  # PD_ERR_UNSUPPORTED_SHAPE
    assert api.lib.pd_pack_delta_static(a, a, 65536, 32, a, a, a, None) == 2
    assert api.lib.pd_pack_delta_static(a, a, 64, 64, a, None, None, None) == 1  # PD_ERR_INVALID_ARG
    assert api.launch_count() == before
