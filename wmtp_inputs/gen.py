"""Seeded synthetic tensors for draft-attention workloads.

This module only produces inputs: counter-based normal deviates (numpy's Philox
bit generator, keyed by (seed, tensor_id, chunk)), rounded to bf16 and returned
as raw ``uint16`` bit patterns.  It contains none of the attention or ring-buffer
arithmetic; both the CPU oracle and the CUDA path are fed the very same bits.

The paper's draft heads attend over a bf16 KV cache of 2 KV heads with head_dim
256 or 128 at roughly a million tokens of context (Section 5, "Setup"); the
cache contents do not influence the cost of the path, so N(0,1) values stand in
for real activations.
"""
from __future__ import annotations

import os
from concurrent.futures import ThreadPoolExecutor

import numpy as np

_CHUNK = 1 << 22  # elements per independently-keyed chunk (fixed: part of the recipe)


def f32_to_bf16_bits(x: np.ndarray) -> np.ndarray:
    """Round float32 to bf16 (round-to-nearest-even); returns uint16 bit patterns."""
    x = np.ascontiguousarray(x, dtype=np.float32)
    u = x.view(np.uint32)
    bias = ((u >> np.uint32(16)) & np.uint32(1)) + np.uint32(0x7FFF)
    r = (u + bias) >> np.uint32(16)
    return r.astype(np.uint16)


def bf16_bits_to_f32(b: np.ndarray) -> np.ndarray:
    """Exact widening of bf16 bit patterns (uint16) to float32."""
    b = np.ascontiguousarray(b, dtype=np.uint16)
    return (b.astype(np.uint32) << np.uint32(16)).view(np.float32)


def bf16_bits_to_f64(b: np.ndarray) -> np.ndarray:
    return bf16_bits_to_f32(b).astype(np.float64)


def _key(tensor_id) -> list[int]:
    if isinstance(tensor_id, (tuple, list)):
        return [int(t) for t in tensor_id]
    return [int(tensor_id)]


def _fill_chunk(out: np.ndarray, seed: int, tensor_id: int, chunk: int, lo: int, hi: int,
                scale: float, mean: float) -> None:
    ss = np.random.SeedSequence([int(seed), *_key(tensor_id), int(chunk)])
    g = np.random.Generator(np.random.Philox(ss))
    x = g.standard_normal(hi - lo, dtype=np.float32)
    if scale != 1.0:
        x *= np.float32(scale)
    if mean != 0.0:
        x += np.float32(mean)
    out[lo:hi] = f32_to_bf16_bits(x)


def normal_bf16(seed: int, tensor_id, shape, scale: float = 1.0, mean: float = 0.0,
                threads: int | None = None) -> np.ndarray:
    """N(mean, scale^2) deviates rounded to bf16, as a uint16 array of ``shape``.

    Element i of the flattened tensor belongs to chunk i // 2^22 and every chunk has its
    own Philox key, so the result does not depend on the number of worker threads.
    """
    n = int(np.prod(shape, dtype=np.int64))
    out = np.empty(n, dtype=np.uint16)
    nchunks = (n + _CHUNK - 1) // _CHUNK
    jobs = [(c, c * _CHUNK, min(n, (c + 1) * _CHUNK)) for c in range(nchunks)]
    if threads is None:
        threads = min(32, os.cpu_count() or 1)
    if nchunks <= 1 or threads <= 1:
        for c, lo, hi in jobs:
            _fill_chunk(out, seed, tensor_id, c, lo, hi, scale, mean)
    else:
        with ThreadPoolExecutor(max_workers=threads) as ex:
            list(ex.map(lambda j: _fill_chunk(out, seed, tensor_id, j[0], j[1], j[2], scale, mean), jobs))
    return out.reshape(shape)


def rng(seed: int, tensor_id) -> np.random.Generator:
    """A generator for small integer/structural draws (sequence lengths, page permutations)."""
    return np.random.Generator(np.random.Philox(np.random.SeedSequence([int(seed), *_key(tensor_id)])))


def e4m3_codes_trunc(bits: np.ndarray, unit: float) -> np.ndarray:
    """Synthetic fp8 store contents from bf16 draws: the draw, in units of ``unit``, cut toward zero onto
    the e4m3 code grid (3 mantissa bits, exponents 2^-6 .. 2^8, magnitudes capped at 448, anything below
    2^-6 cut to a multiple of 2^-9).  Pure field extraction from the fp32 bit pattern; this defines what
    the synthetic store contains and is not the store's quantiser."""
    t = (bf16_bits_to_f32(bits) / np.float32(unit)).astype(np.float32)
    u = t.view(np.uint32)
    sign = ((u >> 31) & 1).astype(np.uint8) << 7
    a = np.minimum(np.abs(t), np.float32(448.0))
    ua = a.view(np.uint32)
    expo = ((ua >> 23) & 0xFF).astype(np.int32) - 120          # e4m3 exponent field of a normal code
    mant = ((ua >> 20) & 7).astype(np.int32)
    normal = (expo << 3) | mant
    sub = np.floor(a * np.float32(512.0)).astype(np.int32)      # below 2^-6: multiples of 2^-9
    code = np.where(expo >= 1, normal, np.minimum(sub, 7))
    return (code.astype(np.uint8) | sign).reshape(bits.shape)
