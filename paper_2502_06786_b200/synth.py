"""Seeded synthetic inputs shared by the tests, the benchmark and the CPU oracle.

This module holds data generation and the bf16 storage format only: no
quantisation, slicing, packing or matmul arithmetic lives here, so the CUDA
path and the CPU oracle stay independent while seeing identical inputs.

All tensors are produced on the host with NumPy's counter-based Philox
generator.  bf16 tensors are returned as ``uint16`` arrays holding the raw
bit patterns (round-to-nearest-even from fp32).

The real workloads of the paper (Gemma-2 2B / 9B and Mistral 7B FFN and
attention weights, Section 4) are not available offline; tensors with the
same layer shapes and the value distributions below stand in for them.
"""
from __future__ import annotations

import numpy as np

BASE_SEED = 0x250206786


def seed_for(config: int, tensor_index: int) -> int:
    """One Philox key per (workload, tensor)."""
    return BASE_SEED + 1000 * int(config) + int(tensor_index)


def _rng(seed: int) -> np.random.Generator:
    return np.random.Generator(np.random.Philox(int(seed)))


def f32_to_bf16_bits(a: np.ndarray) -> np.ndarray:
    """fp32 -> bf16 bit patterns, round to nearest even; NaN stays NaN."""
    a = np.ascontiguousarray(a, dtype=np.float32)
    u = a.view(np.uint32)
    lsb = (u >> np.uint32(16)) & np.uint32(1)
    r = (u + np.uint32(0x7FFF) + lsb) >> np.uint32(16)
    nan = np.isnan(a)
    if nan.any():
        r = np.where(nan, (u >> np.uint32(16)) | np.uint32(0x40), r)
    return r.astype(np.uint16)


def bf16_bits_to_f32(b: np.ndarray) -> np.ndarray:
    """bf16 bit patterns -> fp32 (exact)."""
    b = np.ascontiguousarray(b, dtype=np.uint16)
    return (b.astype(np.uint32) << np.uint32(16)).view(np.float32)


def normal_bf16(shape, std: float, seed: int) -> np.ndarray:
    """N(0, std^2) rounded to bf16."""
    g = _rng(seed)
    a = g.standard_normal(size=shape, dtype=np.float32)
    a *= np.float32(std)
    return f32_to_bf16_bits(a)


def student_t_bf16(shape, nu: float, std: float, seed: int) -> np.ndarray:
    """Student-t with ``nu`` degrees of freedom, rescaled to standard
    deviation ``std`` (needs nu > 2), rounded to bf16.  Heavy tails stand in
    for the outlier channels of trained FFN weights."""
    g = _rng(seed)
    z = g.standard_normal(size=shape, dtype=np.float32)
    chi = g.chisquare(nu, size=shape).astype(np.float32)
    t = z / np.sqrt(chi / np.float32(nu))
    t *= np.float32(std / np.sqrt(nu / (nu - 2.0)))
    return f32_to_bf16_bits(t)


def uniform_codes(shape, seed: int) -> np.ndarray:
    """uint8 codes uniform on [0, 255]."""
    return _rng(seed).integers(0, 256, size=shape, dtype=np.uint8)


def skewed_codes(shape, p_top: float, top_from: int, seed: int) -> np.ndarray:
    """uint8 codes with P(code >= top_from) = p_top and the rest uniform below
    ``top_from``.  Stands in for the right-shifted code histograms of trained
    models (Figure 1c), whose upper bucket is far fuller than plain min-max
    codes of Gaussian weights give."""
    g = _rng(seed)
    lo = g.integers(0, top_from, size=shape, dtype=np.uint8)
    hi = g.integers(top_from, 256, size=shape, dtype=np.uint8)
    pick = g.random(size=shape, dtype=np.float32) < np.float32(p_top)
    return np.where(pick, hi, lo).astype(np.uint8)


def small_int_bf16(shape, lo: int, hi: int, seed: int) -> np.ndarray:
    """Integers in [lo, hi] stored as bf16 (|v| <= 256 is exact in bf16)."""
    g = _rng(seed)
    v = g.integers(lo, hi + 1, size=shape).astype(np.float32)
    return f32_to_bf16_bits(v)


# --------------------------------------------------------------------------
# Layer shapes of the benchmark workloads: (name, N = output channels, K = input features)
# --------------------------------------------------------------------------

def gemma2_2b_mlp_layer():
    d, ff = 2304, 9216
    return [("gate", ff, d), ("up", ff, d), ("down", d, ff)]


def gemma2_9b_decoder_layer():
    d, ff = 3584, 14336
    return [("q", 16 * 256, d), ("k", 8 * 256, d), ("v", 8 * 256, d), ("o", d, 16 * 256),
            ("gate", ff, d), ("up", ff, d), ("down", d, ff)]


def gemma2_9b_mlp_layer():
    d, ff = 3584, 14336
    return [("gate", ff, d), ("up", ff, d), ("down", d, ff)]


WORKLOADS = {
    # id: (description, per-layer shapes, layers, weight distribution)
    1: dict(name="linear-1024", layer=[("w", 1024, 1024)], layers=1, dist="normal"),
    2: dict(name="gemma2-2b-mlp-decode", layer=gemma2_2b_mlp_layer(), layers=26, dist="normal"),
    3: dict(name="gemma2-9b-decode-stack", layer=gemma2_9b_decoder_layer(), layers=42, dist="normal"),
    4: dict(name="mistral-7b-cotrain-forward", layer=[("w", 14336, 4096)], layers=1, dist="normal"),
    5: dict(name="gemma2-9b-mlp-extra-precision", layer=gemma2_9b_mlp_layer(), layers=42, dist="student_t3"),
}


def stack_shapes(config: int, layers: int | None = None):
    """[(tensor_index, layer, name, N, K)] for a workload; ``layers`` truncates the stack."""
    w = WORKLOADS[config]
    nl = w["layers"] if layers is None else min(layers, w["layers"])
    out = []
    idx = 0
    for l in range(nl):
        for (nm, n, k) in w["layer"]:
            out.append((idx, l, nm, n, k))
            idx += 1
    return out


def weight_bf16(config: int, tensor_index: int, n: int, k: int) -> np.ndarray:
    """Weights of one matrix of a workload, bf16 bits [n, k], std 0.02."""
    dist = WORKLOADS[config]["dist"]
    seed = seed_for(config, tensor_index)
    if dist == "student_t3":
        return student_t_bf16((n, k), 3.0, 0.02, seed)
    return normal_bf16((n, k), 0.02, seed)


def activation_bf16(config: int, tensor_index: int, b: int, k: int) -> np.ndarray:
    """Activations x ~ N(0,1), bf16 bits [b, k]; seeds sit above the weight seeds."""
    return normal_bf16((b, k), 1.0, seed_for(config, 500 + tensor_index))
