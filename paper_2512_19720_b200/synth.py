"""Seeded synthetic inputs shared by the tests, the oracle checks and the benchmark.

This module only draws random tensors.  It holds none of the method's arithmetic
(no sign masks, no scales, no reconstruction): the CUDA path and the CPU oracle both
receive the bytes produced here and never exchange anything else.

Recipe (stands in for a real base/fine-tune checkpoint pair, which is not available
offline; only shapes and magnitudes are imitated):

    W_b[o,i]  = fp16( 0.02 * z1 )                         z1 ~ N(0,1)
    s_r[o]    = 0.5 + 1.5 * u[o]                          u  ~ U(0,1), one per output row
    dW16[o,i] = fp16( 1e-3 * s_r[o] * z2 )                z2 ~ N(0,1)
    W_f[o,i]  = fp16( float64(W_b) + float64(dW16) )      round-to-nearest-even
    x[m,i]    = fp16( z3 )                                z3 ~ N(0,1)
    ids[m]    ~ Uniform{0..V-1}

Every stream is a Philox counter-based generator keyed by (seed, tag), so a tensor
depends only on its own seed and shape, never on what was drawn before it.
"""
from __future__ import annotations

import numpy as np

TAG_BASE = 1
TAG_ROW_SCALE = 2
TAG_DELTA = 3
TAG_X = 4
TAG_IDS = 5

# Llama-7B-shaped decoder block linears (d_out, d_in): q, k, v, o, gate, up, down.
BLOCK_7B = [(4096, 4096)] * 4 + [(11008, 4096)] * 2 + [(4096, 11008)]
BLOCK_7B_NAMES = ["q", "k", "v", "o", "gate", "up", "down"]
# 70B-shaped block linears: q, k, v, o, gate, up, down.
BLOCK_70B = [(8192, 8192), (1024, 8192), (1024, 8192), (8192, 8192),
             (28672, 8192), (28672, 8192), (8192, 28672)]
BLOCK_70B_NAMES = ["q", "k", "v", "o", "gate", "up", "down"]


def _rng(seed: int, tag: int) -> np.random.Generator:
    return np.random.Generator(np.random.Philox(key=[int(seed) & 0xFFFFFFFFFFFFFFFF, int(tag)]))


def gen_base(d_out: int, d_in: int, seed: int = 0) -> np.ndarray:
    """Base weights W_b, fp16 [d_out, d_in], entries ~ N(0, 0.02^2)."""
    z = _rng(seed, TAG_BASE).standard_normal((d_out, d_in), dtype=np.float32)
    z *= np.float32(0.02)
    return z.astype(np.float16)


def gen_row_spread(d_out: int, seed: int) -> np.ndarray:
    """Per-row spread s_r ~ U(0.5, 2), float64 [d_out]."""
    return 0.5 + 1.5 * _rng(seed, TAG_ROW_SCALE).random(d_out)


def gen_finetuned(w_b: np.ndarray, seed: int, sigma: float = 1e-3) -> np.ndarray:
    """Fine-tuned weights W_f = fp16(W_b + dW16), dW16 = fp16(sigma * s_r[o] * z)."""
    d_out, d_in = w_b.shape
    s_r = gen_row_spread(d_out, seed).astype(np.float32)
    rng = _rng(seed, TAG_DELTA)
    w_f = np.empty_like(w_b)
    rows = max(1, (1 << 24) // d_in)
    for r0 in range(0, d_out, rows):
        r1 = min(d_out, r0 + rows)
        z = rng.standard_normal((r1 - r0, d_in), dtype=np.float32)
        z *= (np.float32(sigma) * s_r[r0:r1])[:, None]
        dw16 = z.astype(np.float16)
        w_f[r0:r1] = (w_b[r0:r1].astype(np.float64) + dw16.astype(np.float64)).astype(np.float16)
    return w_f


def to_bf16_bits(a: np.ndarray) -> np.ndarray:
    """float32 array -> bfloat16 bit patterns (uint16), round to nearest even (storage conversion only)."""
    u = np.ascontiguousarray(a, dtype=np.float32).view(np.uint32).astype(np.uint64)
    u = (u + 0x7FFF + ((u >> 16) & 1)) >> 16
    return u.astype(np.uint16)


def bf16_bits_to_f32(b: np.ndarray) -> np.ndarray:
    """bfloat16 bit patterns -> the float32 values they denote (exact)."""
    return (np.ascontiguousarray(b, dtype=np.uint16).astype(np.uint32) << 16).view(np.float32)


def gen_base_bf16(d_out: int, d_in: int, seed: int = 0) -> np.ndarray:
    """Base weights as bfloat16 bit patterns [d_out, d_in], entries ~ N(0, 0.02^2) (the draws of gen_base)."""
    z = _rng(seed, TAG_BASE).standard_normal((d_out, d_in), dtype=np.float32)
    z *= np.float32(0.02)
    return to_bf16_bits(z)


def gen_finetuned_bf16(w_b: np.ndarray, seed: int, sigma: float = 1e-3) -> np.ndarray:
    """Fine-tuned weights W_f = bf16(W_b + sigma * s_r[o] * z) as bfloat16 bit patterns."""
    d_out, d_in = w_b.shape
    s_r = gen_row_spread(d_out, seed).astype(np.float32)
    rng = _rng(seed, TAG_DELTA)
    w_f = np.empty_like(w_b)
    rows = max(1, (1 << 24) // d_in)
    for r0 in range(0, d_out, rows):
        r1 = min(d_out, r0 + rows)
        z = rng.standard_normal((r1 - r0, d_in), dtype=np.float32)
        z *= (np.float32(sigma) * s_r[r0:r1])[:, None]
        w_f[r0:r1] = to_bf16_bits((bf16_bits_to_f32(w_b[r0:r1]).astype(np.float64) + z.astype(np.float64)).astype(np.float32))
    return w_f


def gen_x_bf16(m: int, d_in: int, seed: int = 2000) -> np.ndarray:
    """Activations as bfloat16 bit patterns [M, d_in], entries ~ N(0,1)."""
    return to_bf16_bits(_rng(seed, TAG_X).standard_normal((m, d_in), dtype=np.float32))


def gen_x(m: int, d_in: int, seed: int = 2000) -> np.ndarray:
    """Activations x, fp16 [M, d_in], entries ~ N(0,1)."""
    return _rng(seed, TAG_X).standard_normal((m, d_in), dtype=np.float32).astype(np.float16)


def gen_ids(m: int, n_variants: int, seed: int = 3000) -> np.ndarray:
    """Variant id per token row, int32 [M], uniform over {0..V-1}."""
    return _rng(seed, TAG_IDS).integers(0, n_variants, size=m, dtype=np.int32)


def gen_ids_per_sequence(n_decode: int, n_seq: int, seq_len: int, n_variants: int,
                         seed: int = 3000) -> np.ndarray:
    """n_decode rows with one id each, then n_seq sequences of seq_len rows sharing an id."""
    rng = _rng(seed, TAG_IDS)
    head = rng.integers(0, n_variants, size=n_decode, dtype=np.int32)
    seq = rng.integers(0, n_variants, size=n_seq, dtype=np.int32)
    return np.concatenate([head, np.repeat(seq, seq_len)]).astype(np.int32)


def sample_rows(m: int, n_random: int = 64, seed: int = 4000) -> np.ndarray:
    """Fixed sample of token rows for large-M parity: m mod 128 in {0,1,127} plus seeded random rows."""
    base = [r for r in range(m) if (r % 128) in (0, 1, 127)]
    extra = _rng(seed, 99).integers(0, m, size=n_random).tolist()
    return np.array(sorted(set(base + extra)), dtype=np.int64)


def gen_teacher_outputs(x: np.ndarray, w_f: np.ndarray) -> np.ndarray:
    """Calibration targets of one layer: the fine-tuned layer's outputs for the inputs x, stored as float16
    (a dense layer's forward pass in fp64 -- input data for the scale fit, not part of the method)."""
    return (x.astype(np.float64) @ w_f.astype(np.float64).T).astype(np.float16)
