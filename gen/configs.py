"""Workload table: the five benchmark configurations as (layer name, N, K, had_block) shapes.

K = input channels, N = output rows, M = tokens.  had_block is the block size of the
block-diagonal Hadamard rotation applied to the activation before quantization: the full K
when K is a power of two, 128 otherwise.
"""
from dataclasses import dataclass
from typing import List, Tuple

BASE_SEED = 250215779


@dataclass(frozen=True)
class Layer:
    name: str
    N: int
    K: int
    had_block: int


@dataclass(frozen=True)
class Config:
    key: str
    title: str
    layers: Tuple[Layer, ...]
    Ms: Tuple[int, ...]
    codes: str  # "uniform" or "rotated_laplace"


def _hb(K: int) -> int:
    return K if (K & (K - 1)) == 0 else 128


def _L(name, N, K):
    return Layer(name, N, K, _hb(K))


CONFIGS: List[Config] = [
    Config("single_2048", "single W2A4 GEMV 2048x2048", (_L("gemv", 2048, 2048),), (1,), "uniform"),
    Config("llama32_1b", "LLaMA-3.2-1B-shaped decode layer",
           (_L("q", 2048, 2048), _L("k", 512, 2048), _L("v", 512, 2048), _L("o", 2048, 2048),
            _L("gate", 8192, 2048), _L("up", 8192, 2048), _L("down", 2048, 8192)), (1,), "rotated_laplace"),
    Config("llama2_7b", "LLaMA-2-7B-shaped decode layer",
           (_L("qkv", 12288, 4096), _L("o", 4096, 4096), _L("gate_up", 22016, 4096), _L("down", 4096, 11008)),
           (1,), "rotated_laplace"),
    Config("llama3_8b", "LLaMA-3-8B-shaped decode layer",
           (_L("qkv", 6144, 4096), _L("o", 4096, 4096), _L("gate_up", 28672, 4096), _L("down", 4096, 14336)),
           (1, 2, 4, 8, 16), "rotated_laplace"),
    Config("llama2_70b", "LLaMA-2-70B-sized decode layer",
           (_L("qkv", 10240, 8192), _L("o", 8192, 8192), _L("gate_up", 57344, 8192), _L("down", 8192, 28672)),
           (1, 8), "rotated_laplace"),
]

BY_KEY = {c.key: c for c in CONFIGS}


def gemv_bytes(M: int, N: int, K: int) -> int:
    """Algorithmic bytes of one GEMV call: packed codes + per-row LUT + packed activations + fp16 output."""
    return N * K // 4 + 8 * N + M * K // 2 + 2 * M * N


def gemv_grouped_bytes(M: int, N: int, K: int, G: int) -> int:
    """The same with one four-entry fp16 grid per group of G weights instead of one per row."""
    return N * K // 4 + 8 * N * (K // G) + M * K // 2 + 2 * M * N


def quant_bytes(M: int, K: int) -> int:
    """Algorithmic bytes of one activation-quantization call: fp16 in, nibbles + fp16 scale out."""
    return 2 * M * K + M * K // 2 + 2 * M


def gemv_w2a16_bytes(M: int, N: int, K: int) -> int:
    """Algorithmic bytes of one weight-only GEMV call: packed codes + per-row LUT + fp16 activations + fp16 output."""
    return N * K // 4 + 8 * N + 2 * M * K + 2 * M * N


def gemv_w3a4_bytes(M: int, N: int, K: int) -> int:
    """Algorithmic bytes of one W3A4 GEMV call: 3-bit codes + eight fp16 levels per row + int4 activations + fp16 output."""
    return 3 * N * K // 8 + 16 * N + M * K // 2 + 2 * M * N
