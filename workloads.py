"""Seeded synthetic inputs for the transposable N:M mask search.

This module only *generates data*: it holds none of the method's arithmetic and
is the one module that both the CPU oracle's tests and the CUDA path's tests /
benchmarks may import.  Every tensor is produced on the host by
``numpy.random.Generator(PCG64(seed))``; bf16 tensors are returned as the raw
16-bit patterns (``numpy.uint16``), fp32 tensors as ``numpy.float32``.

The five named workloads follow the layer *shapes* and *value distributions* of
the vision and language models the paper trains (ResNet-50 and BERT-large,
Section 4.1); no dataset item or trained weight is used.
"""
from __future__ import annotations

import numpy as np

F32 = 0
BF16 = 1


def f32_to_bf16_bits(x: np.ndarray) -> np.ndarray:
    """Round fp32 values to bf16 (round-to-nearest-even) and return the uint16 patterns."""
    u = np.ascontiguousarray(x, dtype=np.float32).view(np.uint32)
    rounding = ((u >> np.uint32(16)) & np.uint32(1)) + np.uint32(0x7FFF)
    return ((u + rounding) >> np.uint32(16)).astype(np.uint16)


def bf16_bits_to_f32(b: np.ndarray) -> np.ndarray:
    """Widen uint16 bf16 patterns to the fp32 values they denote (exact)."""
    return (np.ascontiguousarray(b, dtype=np.uint16).astype(np.uint32) << np.uint32(16)).view(np.float32)


def _rng(seed: int) -> np.random.Generator:
    return np.random.Generator(np.random.PCG64(seed))


def normal_f32(rows: int, cols: int, sigma: float, seed: int) -> np.ndarray:
    return (_rng(seed).standard_normal((rows, cols), dtype=np.float32) * np.float32(sigma)).astype(np.float32)


def laplace_f32(rows: int, cols: int, b: float, seed: int) -> np.ndarray:
    return _rng(seed).laplace(0.0, b, size=(rows, cols)).astype(np.float32)


def normal_bf16(rows: int, cols: int, sigma: float, seed: int) -> np.ndarray:
    return f32_to_bf16_bits(normal_f32(rows, cols, sigma, seed))


def quantised_bf16(rows: int, cols: int, sigma: float, seed: int, chunk_rows: int = 1024) -> np.ndarray:
    """N(0, sigma) quantised to 256 levels k * 2^-11, k in [-128, 127] (all exact in bf16).

    Only 129 distinct magnitudes exist, so nearly every 4x4 block contains ties.
    Generated in row chunks so that the 12288 x 49152 case needs no fp64 temporary.
    """
    rng = _rng(seed)
    levels = (np.arange(-128, 128, dtype=np.float32) * np.float32(2.0 ** -11)).astype(np.float32)
    table = f32_to_bf16_bits(levels)
    assert np.array_equal(bf16_bits_to_f32(table), levels)
    out = np.empty((rows, cols), dtype=np.uint16)
    inv = np.float32(2.0 ** 11)
    for r0 in range(0, rows, chunk_rows):
        r1 = min(rows, r0 + chunk_rows)
        x = rng.standard_normal((r1 - r0, cols), dtype=np.float32)
        x *= np.float32(sigma) * inv
        k = np.clip(np.rint(x), -128, 127).astype(np.int16)
        out[r0:r1] = table[k + 128]
    return out


# ---------------------------------------------------------------------------
# The five named workloads
# ---------------------------------------------------------------------------

def config1():
    """One 256 x 256 fp32 matrix, N(0, 0.02), seed 0 (4096 4x4 blocks)."""
    return [normal_f32(256, 256, 0.02, 0)]


# (Cout, Cin*kh*kw, multiplicity) of ResNet-50's 53 convolutions and its classifier.
RESNET50_SHAPES = [
    (64, 147, 1), (64, 64, 1), (64, 256, 2), (64, 576, 3), (256, 64, 4),
    (128, 256, 1), (128, 512, 3), (128, 1152, 4), (512, 128, 4), (512, 256, 1),
    (256, 512, 1), (256, 1024, 5), (256, 2304, 6), (1024, 256, 6), (1024, 512, 1),
    (512, 1024, 1), (512, 2048, 2), (512, 4608, 3), (2048, 512, 3), (2048, 1024, 1),
    (1000, 2048, 1),
]


def resnet50_layer_shapes():
    out = []
    for r, c, k in RESNET50_SHAPES:
        out.extend([(r, c)] * k)
    return out


def config2():
    """54 fp32 matrices with ResNet-50's layer shapes, Kaiming-normal, columns zero-padded to a multiple of 4."""
    mats = []
    for idx, (r, c) in enumerate(resnet50_layer_shapes()):
        w = normal_f32(r, c, float(np.sqrt(2.0 / c)), 1000 + idx)
        pad = (-c) % 4
        if pad:
            w = np.concatenate([w, np.zeros((r, pad), dtype=np.float32)], axis=1)
        mats.append(np.ascontiguousarray(w))
    return mats


BERT_LARGE_SHAPES = [(3072, 1024), (1024, 1024), (4096, 1024), (1024, 4096)]


def bert_large_layer_shapes(layers: int = 24):
    return [s for _ in range(layers) for s in BERT_LARGE_SHAPES]


def config3(layers: int = 24):
    """24 x {QKV, attn-out, FFN-up, FFN-down} bf16 matrices, N(0, 0.02), seed 2000 + index."""
    return [normal_bf16(r, c, 0.02, 2000 + i) for i, (r, c) in enumerate(bert_large_layer_shapes(layers))]


def config3_perturbed(mats, step: int):
    """A later simulated training step: add a seeded N(0, 1e-3) perturbation on the host."""
    out = []
    for i, m in enumerate(mats):
        x = bf16_bits_to_f32(m)
        x = x + normal_f32(x.shape[0], x.shape[1], 1e-3, 3000 + 1000 * step + i)
        out.append(f32_to_bf16_bits(x))
    return out


def config4(n: int = 8192):
    """One n x n fp32 matrix, Laplace(0, 0.05), seed 4 (8x8 blocks for the 4:8 search)."""
    return [laplace_f32(n, n, 0.05, 4)]


def config5(rows: int = 12288, cols: int = 49152):
    """One rows x cols bf16 matrix, N(0, 0.02) quantised to 256 levels, seed 5."""
    return [quantised_bf16(rows, cols, 0.02, 5)]


def adversarial_blocks_f32(M: int) -> np.ndarray:
    """A stack of hand-made M x M fp32 blocks: all-equal, all-zero, one non-zero, permutation
    weights, few-level quantised values, huge exponent spread, subnormals, signed zeros."""
    rng = _rng(77 + M)
    blocks = []
    blocks.append(np.ones((M, M), np.float32))
    blocks.append(np.zeros((M, M), np.float32))
    one = np.zeros((M, M), np.float32); one[M // 2, 1] = -3.5
    blocks.append(one)
    blocks.append(np.eye(M, dtype=np.float32)[rng.permutation(M)] * np.float32(2.0))
    blocks.append(rng.integers(-2, 3, size=(M, M)).astype(np.float32))
    blocks.append(rng.integers(-1, 2, size=(M, M)).astype(np.float32) * np.float32(0.25))
    spread = np.ldexp(rng.standard_normal((M, M)), rng.integers(-120, 120, size=(M, M))).astype(np.float32)
    blocks.append(spread)
    sub = (rng.integers(0, 9, size=(M, M)).astype(np.uint32)).view(np.float32)  # subnormals and zeros
    blocks.append(sub.copy())
    mixed = spread.copy(); mixed[::2, ::2] = sub[::2, ::2]
    blocks.append(mixed)
    negz = np.zeros((M, M), np.float32); negz[0, :] = -0.0; negz[1, 1] = 1e-30
    blocks.append(negz)
    pad = rng.standard_normal((M, M)).astype(np.float32); pad[:, M - 1] = 0.0  # a zero-padded column
    blocks.append(pad)
    return np.stack(blocks)
