"""Cold start of a variant (pd_load_merged): artifacts in pinned host memory are copied module by module while the
previous module is merged; every merged matrix must equal the CPU oracle's merge bit for bit."""
import numpy as np
import pytest
import torch

from oracle import pd_oracle as orc
from oracle import pd_oracle_bf16 as orc_bf
from paper_2512_19720_b200 import synth

ROW, COL = 0, 1


def _dev16(bits, bf16):
    t = torch.from_numpy(np.ascontiguousarray(bits).view(np.int16)).cuda()
    return t.view(torch.bfloat16 if bf16 else torch.float16)


@pytest.mark.gpu
@pytest.mark.parametrize("same_stream", [False, True])
def test_load_merged_matches_the_oracle_module_by_module(same_stream):
    assert torch.cuda.is_available(), "GPU tests need a CUDA device"
    from paper_2512_19720_b200 import api
    specs = [(512, 1024, ROW, False), (200, 1056, COL, False), (1024, 512, COL, True), (64, 32, ROW, True),
             (4096, 4096, ROW, False), (130, 288, COL, False), (1024, 1024, ROW, True)]
    modules, expected = [], []
    for i, (d_out, d_in, axis, bf16) in enumerate(specs):
        if bf16:
            w_b = synth.gen_base_bf16(d_out, d_in, 60 + i)
            mask, v_row, v_col = orc_bf.pack(synth.gen_finetuned_bf16(w_b, 1060 + i), w_b)
            ref = orc_bf.merge(w_b, mask, v_row if axis == ROW else v_col, axis)
        else:
            w_b16 = synth.gen_base(d_out, d_in, 60 + i)
            mask, v_row, v_col = orc.pack(synth.gen_finetuned(w_b16, 1060 + i), w_b16)
            ref = orc.merge(w_b16, mask, v_row if axis == ROW else v_col, axis).view(np.uint16)
            w_b = w_b16.view(np.uint16)
        v = v_row if axis == ROW else v_col
        art = api.make_artifact(torch.from_numpy(mask.view(np.int32)), torch.from_numpy(v))
        d_w_b = _dev16(w_b, bf16)
        w_hat = d_w_b if i % 3 == 0 else torch.full_like(d_w_b, 7.0)  # every third module is patched in place
        modules.append((d_w_b, w_hat, art, axis))
        expected.append(ref)
    need = 2 * max((api.artifact_bytes(s[0], s[1], s[2]) + 255) // 256 * 256 for s in specs)
    staging = torch.full((need,), 0xA5, dtype=torch.uint8, device="cuda")
    copy_stream = torch.cuda.current_stream() if same_stream else torch.cuda.Stream()
    torch.cuda.synchronize()
    before = api.launch_count()
    api.pd_load_merged(modules, staging, copy_stream)
    torch.cuda.synchronize()
    assert api.launch_count() == before + len(specs)
    for (w_b, w_hat, art, axis), ref in zip(modules, expected):
        assert np.array_equal(w_hat.view(torch.int16).cpu().numpy().view(np.uint16), ref)
    # a second load over freshly restored bases gives the same bits (the staging halves are reused in order)
    with pytest.raises(api.PdError) as e:
        api.pd_load_merged(modules, staging[:need // 2 - 256], copy_stream)
    assert e.value.code == 4  # PD_ERR_WORKSPACE: nothing was queued


def test_load_merged_rejects_bad_descriptors_on_the_host():
    from paper_2512_19720_b200 import build
    build.build()
    from paper_2512_19720_b200 import api
    A = 0x10000
    before = api.launch_count()
    one = (api.PdModule * 1)(api.PdModule(A, A, A, 64, 64, 0, 0))
    bad_axis = (api.PdModule * 1)(api.PdModule(A, A, A, 64, 64, 5, 0))
    bad_shape = (api.PdModule * 1)(api.PdModule(A, A, A, 64, 48, 0, 0))
    null_art = (api.PdModule * 1)(api.PdModule(A, A, None, 64, 64, 0, 0))
    assert api.lib.pd_load_merged(bad_axis, 1, A, 1 << 20, None, None) == 1
    assert api.lib.pd_load_merged(bad_shape, 1, A, 1 << 20, None, None) == 2
    assert api.lib.pd_load_merged(null_art, 1, A, 1 << 20, None, None) == 1
    assert api.lib.pd_load_merged(bad_axis, 0, A, 1 << 20, None, None) == 1
    assert api.lib.pd_load_merged(one, 1, A, 64, None, None) == 4
    assert api.artifact_bytes(4096, 4096, 0) == 4096 * 128 * 4 + 8192 and api.artifact_bytes(64, 48, 0) == 0
    assert api.launch_count() == before
