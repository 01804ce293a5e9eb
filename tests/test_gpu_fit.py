"""Scale fitting on the GPU (pd_transpose_mask, pd_fit_loss_grad, pd_fit_adamw_step, pd_fit_layer) against the fp64
CPU oracle, through the C ABI.  Tolerances: the tensor cores accumulate exact fp16 products in fp32 (relative error of
a length-d sum about 1e-6 sqrt(d) of its magnitude); the col axis multiplies with binary16 copies of the scales and
stores the residual as binary16 between its two passes (relative 2^-11 per element, independent between elements)."""
import numpy as np
import pytest
import torch

from oracle import pd_oracle as orc16
from oracle import pd_oracle_fit as orc
from paper_2512_19720_b200 import synth

ROW, COL, SCALAR = 0, 1, 2
SHAPES = [(256, 256, 200), (136, 96, 130), (384, 512, 300), (128, 1024, 64)]  # d_out, d_in, tokens


def make_case(d_out, d_in, m, seed, sigma=3e-3):
    w_b = synth.gen_base(d_out, d_in, seed)
    w_f = synth.gen_finetuned(w_b, seed + 1000, sigma)
    mask, v_row, v_col = orc16.pack(w_f, w_b)
    x = synth.gen_x(m, d_in, seed + 2000)
    y = synth.gen_teacher_outputs(x, w_f)
    return w_b, mask, v_row, v_col, x, y


def dev(a):
    if a.dtype == np.uint32:
        return torch.from_numpy(a.view(np.int32)).cuda()
    return torch.from_numpy(a).cuda()


def start(axis, v_row, v_col, factor):
    if axis == ROW:
        return v_row.astype(np.float32) * np.float32(factor)
    if axis == COL:
        return v_col.astype(np.float32) * np.float32(factor)
    return np.array([v_row.astype(np.float64).mean() * factor], dtype=np.float32)


@pytest.mark.gpu
@pytest.mark.parametrize("d_out,d_in", [(256, 256), (136, 96), (40, 2048), (1000, 64)])
def test_transpose_mask_is_the_bit_transpose(d_out, d_in):
    from paper_2512_19720_b200 import api
    rng = np.random.default_rng(d_out + d_in)
    mask = rng.integers(0, 2 ** 32, size=(d_out, d_in // 32), dtype=np.uint64).astype(np.uint32)
    got = api.pd_transpose_mask(dev(mask), d_out, d_in).cpu().numpy().view(np.uint32)
    bits = (mask[:, :, None] >> np.arange(32, dtype=np.uint32)) & 1          # [o][word][bit] -> column = 32 word + bit
    bits = bits.reshape(d_out, d_in).T                                       # [i][o]
    pad = (-d_out) % 32
    bits = np.pad(bits, ((0, 0), (0, pad))).reshape(d_in, -1, 32).astype(np.uint64)
    want = (bits << np.arange(32, dtype=np.uint64)).sum(axis=2).astype(np.uint32)
    assert np.array_equal(got, want)


@pytest.mark.gpu
@pytest.mark.parametrize("shape", SHAPES, ids=lambda s: "x".join(map(str, s)))
@pytest.mark.parametrize("axis", [ROW, COL, SCALAR])
def test_loss_and_gradient_match_the_oracle(shape, axis):
    from paper_2512_19720_b200 import api
    d_out, d_in, m = shape
    w_b, mask, v_row, v_col, x, y = make_case(d_out, d_in, m, 11 + d_out)
    v = start(axis, v_row, v_col, 0.6)  # away from the optimum: the gradient is well above the rounding noise
    d_mask = dev(mask)
    mask_t = api.pd_transpose_mask(d_mask, d_out, d_in)
    loss, grad = api.pd_fit_loss_grad(dev(x), dev(y), dev(w_b), d_mask, dev(v), axis, mask_t=mask_t)
    assert api.pd_device_status() == 0
    loss_o, grad_o = orc.loss_grad(x, y, w_b, mask, v.astype(np.float64), axis)
    assert abs(loss.item() - loss_o) <= 2e-3 * loss_o
    g = grad.cpu().numpy().astype(np.float64)
    scale = np.sqrt(np.mean(grad_o ** 2))
    assert np.all(np.abs(g - grad_o) <= 3e-3 * np.abs(grad_o) + 3e-3 * scale), float(np.max(np.abs(g - grad_o)) / scale)
    # loss only, and the same bits on a second call
    loss2, none = api.pd_fit_loss_grad(dev(x), dev(y), dev(w_b), d_mask, dev(v), axis, mask_t=mask_t, want_grad=False)
    assert none is None and loss2.item() == loss.item()
    _, grad2 = api.pd_fit_loss_grad(dev(x), dev(y), dev(w_b), d_mask, dev(v), axis, mask_t=mask_t)
    assert torch.equal(grad, grad2)


@pytest.mark.gpu
def test_gradient_vanishes_at_an_exact_fit():
    # targets produced by the compressed layer itself: the residual is the fp16 rounding of y, the gradient is noise
    from paper_2512_19720_b200 import api
    d_out, d_in, m = 256, 256, 192
    w_b, mask, v_row, v_col, x, _ = make_case(d_out, d_in, m, 5)
    signs = orc16.unpack(mask, d_in).astype(np.float64)
    w_hat = w_b.astype(np.float64) + v_row.astype(np.float64)[:, None] * signs
    y = (x.astype(np.float64) @ w_hat.T).astype(np.float16)
    v = v_row.astype(np.float32)
    loss, grad = api.pd_fit_loss_grad(dev(x), dev(y), dev(w_b), dev(mask), dev(v), ROW)
    loss_o, grad_o = orc.loss_grad(x, y, w_b, mask, v.astype(np.float64), ROW)
    assert loss.item() < 1e-6 and abs(loss.item() - loss_o) <= 1e-2 * loss_o + 1e-12
    assert np.max(np.abs(grad.cpu().numpy() - grad_o)) <= 1e-5


@pytest.mark.gpu
def test_adamw_steps_match_the_oracle():
    from paper_2512_19720_b200 import api
    rng = np.random.default_rng(3)
    n = 1000
    v0 = (rng.standard_normal(n) * 1e-3).astype(np.float32)
    for lr, wd in ((1e-4, 0.01), (3e-3, 0.1)):
        opt = api.adamw(lr=lr, weight_decay=wd)
        v, m1, m2 = dev(v0.copy()), torch.zeros(n, device="cuda"), torch.zeros(n, device="cuda")
        vo, m1o, m2o = v0.astype(np.float64), np.zeros(n), np.zeros(n)
        for t in range(1, 9):
            g = (rng.standard_normal(n) * 10.0 ** rng.integers(-6, 0)).astype(np.float32)
            api.pd_fit_adamw_step(v, m1, m2, dev(g), t, opt)
            orc.adamw_step(vo, m1o, m2o, g.astype(np.float64), t, lr, 0.9, 0.999, 1e-8, wd)
            assert np.allclose(v.cpu().numpy(), vo, rtol=2e-5, atol=lr * 2e-5), (lr, t)


@pytest.mark.gpu
@pytest.mark.parametrize("cosine", [False, True])
def test_fit_layer_matches_the_oracle(cosine):
    from paper_2512_19720_b200 import api
    d_out, d_in, m_tr, m_val, batch, epochs, lr = 256, 384, 330, 140, 128, 3, 1e-4
    w_b, mask, v_row, v_col, x, y = make_case(d_out, d_in, m_tr + m_val, 21)
    axis_o, v_o, (e_row, e_col), (vr_o, vc_o) = orc.fit_layer(x[:m_tr], y[:m_tr], x[m_tr:], y[m_tr:], w_b, mask, v_row, v_col,
                                                              epochs, batch, lr, cosine=cosine)
    d_x, d_y = dev(x), dev(y)
    v_out, axis_out, val_loss = api.pd_fit_layer(d_x[:m_tr], d_y[:m_tr], d_x[m_tr:], d_y[m_tr:], dev(w_b), dev(mask), dev(v_row),
                                                 dev(v_col), epochs, batch, api.adamw(lr=lr), cosine=cosine)
    assert api.pd_device_status() == 0
    e = val_loss.cpu().numpy().astype(np.float64)
    assert abs(e[0] - e_row) <= 2e-3 * e_row and abs(e[1] - e_col) <= 2e-3 * e_col
    if abs(e_row - e_col) > 5e-3 * max(e_row, e_col):  # the choice is only unique when the losses are apart
        assert int(axis_out.item()) == axis_o
    chosen = int(axis_out.item())
    want = vr_o if chosen == ROW else vc_o
    got = v_out.cpu().numpy().astype(np.float64)[:len(want)]
    steps = epochs * ((m_tr + batch - 1) // batch)
    # every AdamW step moves an entry by at most about lr; the two trajectories may differ by a small fraction of the
    # path walked, plus the final rounding to binary16
    assert np.max(np.abs(got - want)) <= 0.05 * lr * steps + 2.0 ** -11 * np.max(np.abs(want))
    assert np.max(np.abs(want - (v_row if chosen == ROW else v_col).astype(np.float64))) > 0.3 * lr * steps  # it did train


@pytest.mark.gpu
def test_fit_argument_errors():
    from paper_2512_19720_b200 import api
    w_b, mask, v_row, v_col, x, y = make_case(64, 64, 16, 2)
    d = [dev(a) for a in (x, y, w_b, mask)]
    with pytest.raises(api.PdError) as e:
        api.pd_fit_loss_grad(d[0], d[1], d[2], d[3], dev(v_col.astype(np.float32)), COL, mask_t=None)
    assert e.value.code == 1
    with pytest.raises(api.PdError) as e:
        api.pd_fit_loss_grad(d[0], d[1], d[2], d[3], dev(v_row.astype(np.float32)), ROW, workspace=torch.zeros(512, dtype=torch.uint8, device="cuda"))
    assert e.value.code == 4
    with pytest.raises(api.PdError) as e:
        api.pd_fit_loss_grad(d[0], d[1], d[2], d[3], dev(v_row.astype(np.float32)), 3)
    assert e.value.code == 1


@pytest.mark.gpu
@pytest.mark.parametrize("d_out,d_in", [(4096, 4096), (11008, 4096), (4096, 11008)])
def test_full_size_layers_on_sampled_rows(d_out, d_in):
    # 7B-shaped layers with 2048 calibration tokens.  The row gradient of output row o depends on that row only, so the
    # oracle evaluates a sample of rows (its loss over those rows is the mean of their squared residuals); the col
    # gradient needs every row and is checked on the first 32 tokens.
    from paper_2512_19720_b200 import api, synth_torch
    m = 2048
    dev0 = torch.device("cuda")
    w_b = synth_torch.gen_base(d_out, d_in, 7, dev0)
    w_f = synth_torch.gen_finetuned(w_b, 1007, 3e-3)
    mask, v_row, v_col = api.pd_pack_delta(w_f, w_b)
    x = synth_torch.gen_x(m, d_in, 2007, dev0)
    y = torch.empty(m, d_out, dtype=torch.float16, device=dev0)
    for r0 in range(0, d_out, 2048):  # teacher outputs in fp64 blocks, rounded once to fp16
        y[:, r0:r0 + 2048] = (x.double() @ w_f[r0:r0 + 2048].double().T).half()
    mask_t = api.pd_transpose_mask(mask, d_out, d_in)
    rows = np.sort(synth.sample_rows(d_out, 24, seed=d_out + d_in))
    h = lambda t: t.cpu().numpy()
    v32 = (v_row.float() * 0.6).contiguous()
    loss, grad = api.pd_fit_loss_grad(x, y, w_b, mask, v32, ROW)
    assert api.pd_device_status() == 0
    loss_o, grad_o = orc.loss_grad(h(x), h(y[:, rows].contiguous()), h(w_b[rows].contiguous()), h(mask[rows].contiguous()).view(np.uint32),
                                   h(v32[rows]).astype(np.float64), ROW)
    g = h(grad)[rows].astype(np.float64) * (d_out / len(rows))  # the oracle's n counts the sampled rows only
    assert np.all(np.abs(g - grad_o) <= 3e-3 * np.abs(grad_o) + 3e-3 * np.sqrt(np.mean(grad_o ** 2)))
    # whole-matrix properties: the scalar gradient is the sum of the row gradients at a constant vector, same loss
    c = torch.full((d_out,), float(v32.mean()), device=dev0)
    loss_r, grad_r = api.pd_fit_loss_grad(x, y, w_b, mask, c, ROW)
    loss_s, grad_s = api.pd_fit_loss_grad(x, y, w_b, mask, c[:1].contiguous(), SCALAR)
    assert loss_s.item() == loss_r.item()
    assert abs(grad_s.item() - grad_r.double().sum().item()) <= 1e-5 * grad_r.double().abs().sum().item()
    # col axis on 32 tokens against the oracle in full
    mc = 32
    vc32 = (v_col.float() * 0.6).contiguous()
    loss_c, grad_c = api.pd_fit_loss_grad(x[:mc], y[:mc], w_b, mask, vc32, COL, mask_t=mask_t)
    assert api.pd_device_status() == 0
    loss_co, grad_co = orc.loss_grad(h(x[:mc]), h(y[:mc]), h(w_b), h(mask).view(np.uint32), h(vc32).astype(np.float64), COL)
    assert abs(loss_c.item() - loss_co) <= 2e-3 * loss_co
    gc = h(grad_c).astype(np.float64)
    assert np.all(np.abs(gc - grad_co) <= 3e-3 * np.abs(grad_co) + 3e-3 * np.sqrt(np.mean(grad_co ** 2)))
