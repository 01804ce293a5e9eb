"""Independent calls on several CUDA streams at once (the launch shape of the bench's *_par* sections): linears with
outputs of their own, packs and split-K prefills with a workspace per stream.  Every result must equal the one the
same call gives alone (bit for bit: the kernels add in a fixed order) and, on samples, the CPU oracle."""
import numpy as np
import pytest
import torch

from oracle import pd_oracle as orc
from paper_2512_19720_b200 import synth

pytestmark = pytest.mark.gpu
ROW, COL = 0, 1
N_STREAMS = 4


def dev(a):
    if a.dtype == np.uint32:
        a = a.view(np.int32)
    return torch.from_numpy(np.ascontiguousarray(a)).cuda()


def on_streams(streams, calls):
    cur = torch.cuda.current_stream()
    for s in streams:
        s.wait_stream(cur)
    for i, call in enumerate(calls):
        with torch.cuda.stream(streams[i % len(streams)]):
            call(i % len(streams))
    for s in streams:
        cur.wait_stream(s)
    torch.cuda.synchronize()


def test_linears_and_packs_on_four_streams_match_the_single_calls_and_the_oracle():
    assert torch.cuda.is_available(), "GPU tests need a CUDA device"
    from paper_2512_19720_b200 import api
    streams = [torch.cuda.Stream() for _ in range(N_STREAMS)]
    shapes = [(4096, 4096), (1024, 2048), (4096, 4096), (2048, 1024), (4096, 4096), (512, 4096)]
    layers = []
    for i, (d_out, d_in) in enumerate(shapes):
        w_b = synth.gen_base(d_out, d_in, 40 + i)
        w_f = synth.gen_finetuned(w_b, 1040 + i)
        layers.append(dict(d_out=d_out, d_in=d_in, w_b=w_b, w_f=w_f, d_w_b=dev(w_b), d_w_f=dev(w_f)))
    # ---- packs: a zeroed workspace per stream
    ws = [torch.zeros(api.workspace_bytes(api.OP_PACK, 0, 0, 4096, 4096), dtype=torch.uint8, device="cuda") for _ in range(N_STREAMS)]
    outs = [dict(mask=torch.empty((L["d_out"], L["d_in"] // 32), dtype=torch.int32, device="cuda"),
                 v_row=torch.empty(L["d_out"], dtype=torch.float16, device="cuda"),
                 v_col=torch.empty(L["d_in"], dtype=torch.float16, device="cuda")) for L in layers]
    for _ in range(2):  # twice: the workspaces must come back zeroed
        on_streams(streams, [lambda b, L=L, o=o: api.pd_pack_delta(L["d_w_f"], L["d_w_b"], mask=o["mask"], v_row=o["v_row"], v_col=o["v_col"],
                                                                   workspace=ws[b]) for L, o in zip(layers, outs)])
    for L, o in zip(layers, outs):
        mask, v_row, v_col = orc.pack(L["w_f"], L["w_b"])
        assert np.array_equal(o["mask"].cpu().numpy().view(np.uint32), mask)
        assert np.array_equal(o["v_row"].cpu().numpy().view(np.uint16), v_row.view(np.uint16))
        assert np.array_equal(o["v_col"].cpu().numpy().view(np.uint16), v_col.view(np.uint16))
        L.update(mask=mask, v=(v_row, v_col), d_mask=o["mask"], d_v=(o["v_row"], o["v_col"]))
    assert all(int(w.max()) == 0 for w in ws)
    # ---- decode linears (M = 4) and split-K prefills (M = 96), both axes, all at once
    for m, use_ws in ((4, False), (96, True)):
        xs = {d_in: synth.gen_x(m, d_in, 2400 + d_in + m) for d_in in {L["d_in"] for L in layers}}
        d_xs = {k: dev(v) for k, v in xs.items()}
        lin_ws = [torch.zeros(max(api.workspace_bytes(api.OP_LINEAR, m, 0, L["d_out"], L["d_in"]) for L in layers), dtype=torch.uint8,
                              device="cuda") for _ in range(N_STREAMS)]
        jobs = [(L, axis) for axis in (ROW, COL) for L in layers]
        ys = [torch.empty((m, L["d_out"]), dtype=torch.float16, device="cuda") for L, _ in jobs]
        on_streams(streams, [lambda b, L=L, axis=axis, y=y: api.pd_linear(d_xs[L["d_in"]], L["d_w_b"], L["d_mask"], L["d_v"][axis], axis, y=y,
                                                                           workspace=lin_ws[b] if use_ws else None,
                                                                           weights_resident=True) for (L, axis), y in zip(jobs, ys)])
        assert all(api.pd_device_status(workspace=w) == 0 for w in lin_ws)
        for j, ((L, axis), y) in enumerate(zip(jobs, ys)):
            alone = api.pd_linear(d_xs[L["d_in"]], L["d_w_b"], L["d_mask"], L["d_v"][axis], axis)
            torch.cuda.synchronize()
            assert torch.equal(y, alone), (m, j)
            if j % 4 == 0:  # a sample of the jobs against the oracle
                ref = orc.linear(xs[L["d_in"]], L["w_b"], L["mask"], L["v"][axis], axis)
                err = np.max(np.abs(y.cpu().numpy().astype(np.float64) - ref)) / np.max(np.abs(ref))
                assert err <= 5e-3, (m, j, err)
