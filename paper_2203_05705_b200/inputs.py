"""Seeded synthetic inputs shared by the tests, the benchmark and the CPU reference
implementation used by the tests.

This module holds none of the method's arithmetic: it only draws tensors with
the shapes and value distributions of the paper's MLP / LSTM workloads (Sec. 7).
It imports neither the CUDA binding nor that reference implementation.
"""
from __future__ import annotations

import math
import numpy as np

BASE_SEED = 20220305


def rng_for(config: int, tensor: int, extra: int = 0) -> np.random.Generator:
    return np.random.Generator(np.random.PCG64(BASE_SEED + 1000 * config + tensor + 100000 * extra))


def bf16_bits(x: np.ndarray) -> np.ndarray:
    """Round fp32 -> bf16 (round to nearest even); returns the uint16 bit patterns."""
    u = np.ascontiguousarray(x, dtype=np.float32).view(np.uint32)
    rounded = u + (np.uint32(0x7FFF) + ((u >> np.uint32(16)) & np.uint32(1)))
    return (rounded >> np.uint32(16)).astype(np.uint16)


def bf16_to_f32(bits: np.ndarray) -> np.ndarray:
    return (bits.astype(np.uint32) << np.uint32(16)).view(np.float32)


def bf16_round(x: np.ndarray) -> np.ndarray:
    """fp32 array holding values exactly representable in bf16."""
    return bf16_to_f32(bf16_bits(x)).reshape(np.shape(x))


# ---------------------------------------------------------------------------
# Workloads.  W is returned in the math orientation W[K x N] (Y = X W); the
# CUDA path stores it neuron-major, i.e. W.T made contiguous.
# ---------------------------------------------------------------------------
def config1():
    """Tiny fp32 MLP layer: X[64x784], W[784x256] ~ N(0, 0.05^2), dY[64x256] ~ N(0,1)."""
    X = rng_for(1, 0).normal(0.0, 0.05, size=(64, 784)).astype(np.float32)
    W = rng_for(1, 1).normal(0.0, 0.05, size=(784, 256)).astype(np.float32)
    dY = rng_for(1, 2).normal(0.0, 1.0, size=(64, 256)).astype(np.float32)
    return {"X": X, "W": W, "dY": dY, "p": 0.5, "n_dp": 8}


def config2_weights():
    """784-2048-2048-10 MLP, Kaiming-normal weights, values representable in bf16."""
    dims = [784, 2048, 2048, 10]
    Ws = []
    for l in range(3):
        fan_in = dims[l]
        w = rng_for(2, l).normal(0.0, math.sqrt(2.0 / fan_in), size=(dims[l], dims[l + 1]))
        Ws.append(bf16_round(w.astype(np.float32)))
    return Ws


def config2_step(step: int, batch: int = 128):
    """Inputs ~ U[0,1) and the loss gradient of one training step."""
    X = bf16_round(rng_for(2, 10, step).random(size=(batch, 784)).astype(np.float32))
    dZ3 = bf16_round((rng_for(2, 11, step).normal(size=(batch, 10)) / batch).astype(np.float32))
    return X, dZ3


def dense_layer(config: int, B: int, K: int, N: int, w_scale: float):
    """X[BxK], dY[BxN] ~ N(0,1) and W[KxN] ~ N(0,1)*w_scale, bf16-representable."""
    X = bf16_round(rng_for(config, 0).standard_normal(size=(B, K), dtype=np.float32))
    W = bf16_round(rng_for(config, 1).standard_normal(size=(K, N), dtype=np.float32) * np.float32(w_scale))
    dY = bf16_round(rng_for(config, 2).standard_normal(size=(B, N), dtype=np.float32))
    return {"X": X, "W": W, "dY": dY}


def config3(B: int = 1024, D: int = 4096):
    """Tile-based DropConnect layer: 4096x4096 weight, batch 1024, 64x64 tiles."""
    d = dense_layer(3, B, D, D, 1.0 / 64.0)
    d.update(ts=64, n_dp=16)
    return d


def config4(T: int = 35, B: int = 64, I: int = 1024, H: int = 1024, seq: int = 0):
    """LSTM layer: W[(I+H) x 4H] ~ U[-0.03, 0.03], x_t ~ N(0,1), dH_t ~ N(0,1)/64."""
    W = bf16_round(rng_for(4, 0).uniform(-0.03, 0.03, size=(I + H, 4 * H)).astype(np.float32))
    X = bf16_round(rng_for(4, 1, seq).standard_normal(size=(T, B, I), dtype=np.float32))
    dH = bf16_round((rng_for(4, 2, seq).standard_normal(size=(T, B, H), dtype=np.float32) / np.float32(64.0)))
    return {"W": W, "X": X, "dH": dH, "n_dp": 16}


def config5(B: int = 4096, D: int = 8192):
    """Large MLP layer: W 8192x8192 ~ N(0,1)/90, X and dY [4096x8192] ~ N(0,1)."""
    d = dense_layer(5, B, D, D, 1.0 / 90.0)
    d.update(ts=128, n_dp=16)
    return d
