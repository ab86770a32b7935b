"""Seeded synthetic inputs with the shapes and value distributions of BERT linears.

This module only draws random numbers and lists shapes.  It contains none of the
quantization arithmetic, so that the CPU oracle and the CUDA library can be fed
the very same arrays without sharing any of the method's code.

The tensors stand in for fine-tuned BERT weights and activations:

* activations ``X``  i.i.d. N(0, 1); two "outlier channels" (columns drawn from the seed)
  are multiplied by 20;
* weights ``W``      i.i.d. N(0, 0.02); each element independently, with probability 0.01,
  replaced by a Laplace(0, 0.1) draw;
* bias               i.i.d. N(0, 0.02).
"""
from __future__ import annotations

from dataclasses import dataclass

import numpy as np

BITS_CHOICES = (2, 3, 4, 8)

# Per-layer weight bit widths printed in the paper's appendix tables (encoder layers 1..12).
MP_PRESETS = {
    # "Bits setting for 2/3-bit Q-BERT MP"
    "2/3-MP SST-2":    (2, 2, 2, 3, 3, 3, 3, 3, 3, 2, 2, 2),
    "2/3-MP MNLI":     (2, 2, 2, 2, 3, 3, 3, 3, 2, 2, 2, 2),
    "2/3-MP CoNLL-03": (2, 3, 3, 3, 3, 2, 2, 2, 2, 2, 2, 2),
    "2/3-MP SQuAD":    (2, 2, 2, 3, 3, 3, 3, 3, 3, 2, 2, 2),
    # "Bits setting for 2/4-bit Q-BERT MP"
    "2/4-MP SST-2":    (2, 2, 4, 4, 4, 2, 4, 4, 4, 2, 2, 2),
    "2/4-MP MNLI":     (2, 2, 2, 4, 4, 4, 4, 4, 2, 2, 2, 2),
    "2/4-MP CoNLL-03": (2, 2, 2, 4, 4, 4, 4, 4, 2, 2, 2, 2),
    "2/4-MP SQuAD":    (2, 2, 2, 4, 4, 4, 4, 4, 2, 2, 2, 2),
}


@dataclass(frozen=True)
class LinearShape:
    name: str
    N: int       # output neurons (rows of W)
    K: int       # input features
    groups: int  # row groups of the weight matrix


def encoder_linears(hidden: int, ffn: int, groups: int = 128) -> tuple[LinearShape, ...]:
    """The four linears of one encoder layer, in execution order.

    The fused QKV matrix carries ``groups`` groups for each of its three attention matrices.
    """
    return (
        LinearShape("qkv", 3 * hidden, hidden, 3 * groups),
        LinearShape("attn_out", hidden, hidden, groups),
        LinearShape("ffn1", ffn, hidden, groups),
        LinearShape("ffn2", hidden, ffn, groups),
    )


BERT_BASE = encoder_linears(768, 3072)
BERT_LARGE = encoder_linears(1024, 4096)


def seed_for(config: int, layer: int = 0, matrix: int = 0) -> int:
    return 1000 * config + 10 * layer + matrix


def activations(M: int, K: int, seed: int, outlier_gain: float = 20.0) -> np.ndarray:
    rng = np.random.default_rng([seed, 1])
    x = rng.standard_normal((M, K), dtype=np.float32)
    cols = rng.choice(K, size=2, replace=False)
    x[:, cols] *= np.float32(outlier_gain)
    return x


def weights(N: int, K: int, seed: int, sigma: float = 0.02, p_outlier: float = 0.01,
            laplace_b: float = 0.1) -> np.ndarray:
    rng = np.random.default_rng([seed, 2])
    w = rng.standard_normal((N, K), dtype=np.float32) * np.float32(sigma)
    mask = rng.random((N, K), dtype=np.float32) < np.float32(p_outlier)
    w[mask] = rng.laplace(0.0, laplace_b, size=int(mask.sum())).astype(np.float32)
    return w


def bias(N: int, seed: int, sigma: float = 0.02) -> np.ndarray:
    rng = np.random.default_rng([seed, 3])
    return rng.standard_normal(N, dtype=np.float32) * np.float32(sigma)


def mixed_bits(layers: int, seed: int) -> tuple[int, ...]:
    """Per-layer bit widths: half of the layers (chosen by seed) get 2 bits, the others are
    drawn uniformly from {2, 3, 4, 8}."""
    rng = np.random.default_rng([seed, 4])
    bits = rng.choice(BITS_CHOICES, size=layers)
    two = rng.choice(layers, size=(layers + 1) // 2, replace=False)
    bits[two] = 2
    return tuple(int(b) for b in bits)


@dataclass(frozen=True)
class Workload:
    config: int
    name: str
    M: int
    layers: int
    linears: tuple[LinearShape, ...]
    bits: tuple[int, ...]  # one entry per layer


def workload(config: int) -> Workload:
    """The GEMM workloads (configs 0-3); config 4 is ``quantizer_sweep_shapes``."""
    if config == 0:
        return Workload(0, "bert-base query projection, M=1024, 4-bit, 12 groups", 1024, 1,
                        (LinearShape("query", 768, 768, 12),), (4,))
    if config == 1:
        return Workload(1, "bert-base encoder layer linears, M=4096, 3-bit, 128 groups", 4096, 1, BERT_BASE,
                        (3,))
    if config == 2:
        return Workload(2, "bert-base 12-layer linear stack, M=128, mixed precision, 128 groups", 128, 12,
                        BERT_BASE, mixed_bits(12, seed_for(2)))
    if config == 3:
        return Workload(3, "bert-large 24-layer linear stack, M=24576, 4-bit, 128 groups", 24576, 24,
                        BERT_LARGE, (4,) * 24)
    raise ValueError(f"no GEMM workload for config {config}")


def quantizer_sweep_shapes() -> list[tuple[int, int]]:
    """Config 4: a 109,117,440-parameter set of BERT-base-shaped matrices (rows, cols)."""
    shapes = [(s.N, s.K) for _ in range(12) for s in BERT_BASE]
    shapes.append((768, 30720))  # embedding-shaped, vocabulary padded, embedding dims as rows
    shapes.append((768, 768))    # pooler-shaped
    return shapes


QUANTIZER_SWEEP_ACT = (64 * 384, 4096)
