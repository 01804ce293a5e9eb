"""Device-side version of the synthetic recipe in synth.py, for throughput runs where the
tensors are too large to draw on the host in reasonable time.  Same distributions, torch's
Philox streams instead of numpy's; like synth.py it holds none of the method's arithmetic."""
from __future__ import annotations

import torch


def _gen(device, seed):
    g = torch.Generator(device=device)
    g.manual_seed(int(seed))
    return g


def gen_base(d_out, d_in, seed, device):
    """W_b fp16 [d_out, d_in] ~ N(0, 0.02^2)."""
    g = _gen(device, seed * 7919 + 1)
    return (torch.randn((d_out, d_in), generator=g, device=device, dtype=torch.float32) * 0.02).half()


def gen_finetuned(w_b, seed, sigma=1e-3):
    """W_f = W_b + fp16(sigma * s_r[o] * z) rounded to the dtype of W_b (float16 or bfloat16), s_r ~ U(0.5, 2) per row."""
    d_out, d_in = w_b.shape
    g = _gen(w_b.device, seed * 7919 + 2)
    s_r = 0.5 + 1.5 * torch.rand(d_out, generator=g, device=w_b.device, dtype=torch.float32)
    w_f = torch.empty_like(w_b)
    rows = max(1, (1 << 26) // d_in)
    for r0 in range(0, d_out, rows):
        r1 = min(d_out, r0 + rows)
        z = torch.randn((r1 - r0, d_in), generator=g, device=w_b.device, dtype=torch.float32)
        dw16 = (z * (sigma * s_r[r0:r1])[:, None]).half()
        w_f[r0:r1] = (w_b[r0:r1].double() + dw16.double()).to(w_b.dtype)
    return w_f


def gen_x(m, d_in, seed, device):
    g = _gen(device, seed * 7919 + 3)
    return torch.randn((m, d_in), generator=g, device=device, dtype=torch.float32).half()


def gen_ids(m, n_variants, seed, device):
    g = _gen(device, seed * 7919 + 4)
    return torch.randint(0, n_variants, (m,), generator=g, device=device, dtype=torch.int32)
