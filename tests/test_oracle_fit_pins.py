"""Pins for the scale-fitting CPU oracle (oracle/pd_oracle_fit.c): the loss against a library fp64 GEMM on the
reconstructed weights, the gradient against central differences of that loss (the loss is quadratic in v, so they
are exact up to rounding) and against torch's autograd on the same formula, closed forms on tiny cases, and the
optimiser step against torch.optim.AdamW.  Planted mistakes are compiled into copies and each must fail a pin."""
import os
import subprocess
import tempfile

import numpy as np
import pytest
import torch

from oracle import pd_oracle as orc16
from oracle import pd_oracle_fit as orc
from paper_2512_19720_b200 import synth

ROW, COL, SCALAR = orc.AXIS_ROW, orc.AXIS_COL, orc.AXIS_SCALAR


@pytest.fixture(scope="module", autouse=True)
def _built():
    orc.build()
    orc16.build()


def case(d_out, d_in, m, seed):
    w_b = synth.gen_base(d_out, d_in, seed)
    w_f = synth.gen_finetuned(w_b, seed + 1000, 3e-3)
    mask, v_row, v_col = orc16.pack(w_f, w_b)
    x = synth.gen_x(m, d_in, seed + 2000)
    y = (x.astype(np.float64) @ w_f.astype(np.float64).T).astype(np.float16)  # the teacher layer's outputs
    return w_b, w_f, mask, v_row, v_col, x, y


def signs(mask, d_in):
    return orc16.unpack(mask, d_in).astype(np.float64)


def start_vector(axis, v_row, v_col):
    if axis == ROW:
        return v_row.astype(np.float64)
    if axis == COL:
        return v_col.astype(np.float64)
    return np.array([float(v_row.astype(np.float64).mean())])


def dense_w_hat(w_b, b, v, axis):
    s = v[:, None] if axis == ROW else (v[None, :] if axis == COL else v[0])
    return w_b.astype(np.float64) + s * b


def check_loss_is_mse_of_a_library_gemm():
    w_b, _, mask, v_row, v_col, x, y = case(12, 64, 7, 1)
    b = signs(mask, 64)
    for axis in (ROW, COL, SCALAR):
        v = start_vector(axis, v_row, v_col) * 1.3
        ref = np.mean((x.astype(np.float64) @ dense_w_hat(w_b, b, v, axis).T - y.astype(np.float64)) ** 2)
        loss, _ = orc.loss_grad(x, y, w_b, mask, v, axis, want_grad=False)
        assert abs(loss - ref) <= 1e-12 * max(1.0, ref)


def check_gradient_is_the_central_difference_of_the_loss():
    w_b, _, mask, v_row, v_col, x, y = case(10, 96, 9, 2)
    for axis in (ROW, COL, SCALAR):
        v = start_vector(axis, v_row, v_col) * 0.7
        _, g = orc.loss_grad(x, y, w_b, mask, v, axis)
        h = 1e-3
        for k in range(0, len(v), max(1, len(v) // 7)):
            vp, vm = v.copy(), v.copy()
            vp[k] += h
            vm[k] -= h
            lp, _ = orc.loss_grad(x, y, w_b, mask, vp, axis, want_grad=False)
            lm, _ = orc.loss_grad(x, y, w_b, mask, vm, axis, want_grad=False)
            fd = (lp - lm) / (2 * h)
            assert abs(fd - g[k]) <= 1e-7 * max(1e-3, abs(g[k])), (axis, k, fd, g[k])


def check_gradient_matches_autograd():
    w_b, _, mask, v_row, v_col, x, y = case(16, 64, 11, 3)
    b = torch.from_numpy(signs(mask, 64))
    xt, yt, wt = (torch.from_numpy(a.astype(np.float64)) for a in (x, y, w_b))
    for axis in (ROW, COL, SCALAR):
        v = torch.from_numpy(start_vector(axis, v_row, v_col)).clone().requires_grad_(True)
        s = v[:, None] if axis == ROW else (v[None, :] if axis == COL else v[0])
        loss = torch.mean((xt @ (wt + s * b).T - yt) ** 2)
        loss.backward()
        l, g = orc.loss_grad(x, y, w_b, mask, v.detach().numpy(), axis)
        assert abs(l - loss.item()) <= 1e-12 * max(1.0, loss.item())
        assert np.allclose(g, v.grad.numpy(), rtol=1e-10, atol=1e-14)


def check_closed_forms():
    # one token, one row, all signs +1, W_b = 0: Y_hat = v * sum(x), L = (v*S - y)^2, dL/dv = 2 (v*S - y) S
    d_in = 32
    w_b = np.zeros((1, d_in), dtype=np.float16)
    mask = np.full((1, 1), 0xFFFFFFFF, dtype=np.uint32)
    x = np.arange(1, d_in + 1, dtype=np.float16).reshape(1, d_in) / 16
    y = np.array([[3.0]], dtype=np.float16)
    big_s = float(x.astype(np.float64).sum())
    v = np.array([0.25])
    for axis in (ROW, SCALAR):
        l, g = orc.loss_grad(x, y, w_b, mask, v, axis)
        assert abs(l - (0.25 * big_s - 3.0) ** 2) < 1e-12 and abs(g[0] - 2 * (0.25 * big_s - 3.0) * big_s) < 1e-10
    vc = np.full(d_in, 0.25)
    l, g = orc.loss_grad(x, y, w_b, mask, vc, COL)
    assert np.allclose(g, 2 * (0.25 * big_s - 3.0) * x.astype(np.float64)[0], rtol=1e-12)
    # the scalar gradient is the sum of the row gradients at a constant vector; a perfect fit has zero gradient
    w_b, w_f, mask, v_row, v_col, x, y = case(8, 64, 5, 4)
    c = 0.002
    _, gr = orc.loss_grad(x, y, w_b, mask, np.full(8, c), ROW)
    _, gs = orc.loss_grad(x, y, w_b, mask, np.array([c]), SCALAR)
    assert abs(gs[0] - gr.sum()) <= 1e-12 * max(1.0, abs(gs[0]))
    y_fit = None
    b = signs(mask, 64)
    v = v_row.astype(np.float64)
    y_exact = x.astype(np.float64) @ dense_w_hat(w_b, b, v, ROW).T
    y_fit = y_exact.astype(np.float16)
    l, g = orc.loss_grad(x, y_fit, w_b, mask, v, ROW)
    assert l < 1e-6 and np.max(np.abs(g)) < 1e-3


def check_adamw_matches_torch():
    rng = np.random.default_rng(5)
    n = 37
    v0 = rng.standard_normal(n) * 1e-3
    for (lr, wd) in ((1e-4, 0.01), (3e-3, 0.1), (1e-5, 0.0)):
        p = torch.nn.Parameter(torch.from_numpy(v0.copy()))
        opt = torch.optim.AdamW([p], lr=lr, betas=(0.9, 0.999), eps=1e-8, weight_decay=wd)
        v, m1, m2 = v0.copy(), np.zeros(n), np.zeros(n)
        for t in range(1, 8):
            g = rng.standard_normal(n) * 10.0 ** rng.integers(-6, 0)
            p.grad = torch.from_numpy(g.copy())
            opt.step()
            orc.adamw_step(v, m1, m2, g, t, lr, 0.9, 0.999, 1e-8, wd)
            assert np.allclose(v, p.detach().numpy(), rtol=1e-12, atol=1e-18), (lr, wd, t)


def check_descent_lowers_the_loss_and_selection_prefers_the_matching_axis():
    # a fine-tune whose delta magnitude varies along the rows only: after the same number of steps the row-axis
    # fit must reach a lower loss than the col-axis fit (the selection rule keeps the lower one)
    w_b, w_f, mask, v_row, v_col, x, y = case(24, 64, 48, 6)
    final = {}
    for axis in (ROW, COL):
        v = start_vector(axis, v_row, v_col)
        m1, m2 = np.zeros_like(v), np.zeros_like(v)
        l0, _ = orc.loss_grad(x, y, w_b, mask, v, axis, want_grad=False)
        for t in range(1, 41):
            _, g = orc.loss_grad(x, y, w_b, mask, v, axis)
            orc.adamw_step(v, m1, m2, g, t, 1e-4, 0.9, 0.999, 1e-8, 0.0)
        final[axis], _ = orc.loss_grad(x, y, w_b, mask, v, axis, want_grad=False)
        assert final[axis] < l0
    assert final[ROW] <= final[COL]


def check_training_loop_matches_a_torch_loop():
    # the loop of the training algorithm against autograd + torch.optim.AdamW + CosineAnnealingLR stepped per minibatch
    w_b, _, mask, v_row, v_col, x, y = case(12, 64, 40, 7)
    xv, yv = x[32:], y[32:]
    b = torch.from_numpy(signs(mask, 64))
    wt = torch.from_numpy(w_b.astype(np.float64))
    for axis, cosine in ((ROW, False), (COL, True)):
        v0 = start_vector(axis, v_row, v_col)
        v_o, val_o = orc.train(x[:32], y[:32], xv, yv, w_b, mask, v0, axis, epochs=3, batch=12, lr=1e-4, cosine=cosine)
        p = torch.nn.Parameter(torch.from_numpy(v0.copy()))
        opt = torch.optim.AdamW([p], lr=1e-4, betas=(0.9, 0.999), eps=1e-8, weight_decay=0.01)
        sched = torch.optim.lr_scheduler.CosineAnnealingLR(opt, T_max=9) if cosine else None

        def forward(xa):
            s = p[:, None] if axis == ROW else p[None, :]
            return torch.from_numpy(xa.astype(np.float64)) @ (wt + s * b).T

        for _ in range(3):
            for b0 in (0, 12, 24):
                opt.zero_grad()
                loss = torch.mean((forward(x[b0:min(b0 + 12, 32)]) - torch.from_numpy(y[b0:min(b0 + 12, 32)].astype(np.float64))) ** 2)
                loss.backward()
                opt.step()
                if sched:
                    sched.step()
        val_t = torch.mean((forward(xv) - torch.from_numpy(yv.astype(np.float64))) ** 2).item()
        assert np.allclose(v_o, p.detach().numpy(), rtol=1e-9, atol=1e-15), axis
        assert abs(val_o - val_t) <= 1e-10 * max(1.0, val_t)


def check_selection_keeps_the_lower_validation_loss():
    w_b, _, mask, v_row, v_col, x, y = case(16, 64, 40, 8)
    axis, v, (e_row, e_col), (vr, vc) = orc.fit_layer(x[:32], y[:32], x[32:], y[32:], w_b, mask, v_row, v_col, epochs=2, batch=16, lr=1e-4)
    assert axis == (ROW if e_row <= e_col else COL)
    assert np.array_equal(v, vr if axis == ROW else vc)
    for a, vec, e in ((ROW, vr, e_row), (COL, vc, e_col)):
        again, _ = orc.loss_grad(x[32:], y[32:], w_b, mask, vec, a, want_grad=False)
        assert abs(again - e) <= 1e-13 * e  # the OpenMP reduction adds the threads' partial sums in any order


CHECKS = [v for k, v in sorted(globals().items()) if k.startswith("check_")]


@pytest.mark.parametrize("check", CHECKS, ids=[c.__name__ for c in CHECKS])
def test_pin(check):
    check()


MUTATIONS = [
    ("loss_not_a_mean", "loss /= n;", "loss /= (double)M;"),
    ("grad_factor", "(2.0 / n) * r * d;", "(1.0 / n) * r * d;"),
    ("grad_sign_dropped", "double d = half_to_double(x[m * d_in + i]) * sign_of(mask, d_in, o, i);", "double d = half_to_double(x[m * d_in + i]);"),
    ("grad_axis_swapped", "grad[axis == AXIS_ROW ? o : (axis == AXIS_COL ? i : 0)]", "grad[axis == AXIS_ROW ? i % len : (axis == AXIS_COL ? o % len : 0)]"),
    ("residual_sign", "double r = acc - half_to_double(y[m * d_out + o]);", "double r = acc + half_to_double(y[m * d_out + o]);"),
    ("forward_drops_delta", "+ scale_of(v, axis, o, i) * sign_of(mask, d_in, o, i));", "+ 0.0 * scale_of(v, axis, o, i) * sign_of(mask, d_in, o, i));"),
    ("adamw_coupled_decay", "v[k] *= 1.0 - lr * wd;", "v[k] *= 1.0;"),
    ("adamw_no_bias_correction", "double c1 = 1.0 - pow(b1, (double)t), c2", "double c1 = 1.0, c2"),
    ("adamw_eps_inside_sqrt", "(sqrt(m2[k] / c2) + eps)", "sqrt(m2[k] / c2 + eps)"),
    ("adamw_second_moment", "(1.0 - b2) * g[k] * g[k];", "(1.0 - b2) * fabs(g[k]);"),
]


@pytest.mark.parametrize("name,old,new", MUTATIONS, ids=[m[0] for m in MUTATIONS])
def test_planted_mistake_is_caught(name, old, new):
    src = open(os.path.join(os.path.dirname(orc.__file__), "pd_oracle_fit.c")).read()
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
