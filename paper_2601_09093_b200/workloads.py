"""Seeded synthetic inputs for the five benchmark configurations.

This module holds none of the method's arithmetic: it only draws numbers,
lengths and masks, and converts between float32 and bfloat16 bit patterns.
Both the CUDA tests/benchmark and the CPU oracle's tests take their inputs
from here, so that the two sides see the same bytes.

Generator: numpy's counter-based Philox keyed by (seed, tensor id); every
tensor has its own stream, so the order in which tensors are drawn does not
matter.  Normal variates for bf16 configurations are rounded to bf16
(round-to-nearest-even) here and handed out as uint16 bit patterns together
with their exact float32 values.

The shapes stand in for the paper's workloads (64 sampled traces per problem,
tens of thousands of tokens per trace, hidden size 4096/5120, scorer width
512, roughly one step boundary per 10^2 tokens); the paper's benchmark suites,
model weights and trained scorers are not reproduced.
"""
from __future__ import annotations

import dataclasses
import math

import numpy as np

# tensor ids (second half of the Philox key)
TID_Q, TID_K, TID_V, TID_KPRE, TID_VPRE, TID_LEN, TID_HID, TID_MASK = 1, 2, 3, 4, 5, 6, 7, 8
TID_W1, TID_W2, TID_B1, TID_PERM, TID_ANS, TID_KNEW, TID_VNEW, TID_VOCAB, TID_TOK = 9, 10, 11, 12, 13, 14, 15, 16, 17


@dataclasses.dataclass(frozen=True)
class Config:
    name: str
    n_traces: int
    num_layers: int
    num_q_heads: int
    num_kv_heads: int
    head_dim: int
    page_size: int
    dtype: str                 # "bf16" | "fp32"
    prefix_len: int
    suffix_lo: int
    suffix_hi: int
    suffix_dist: str           # "uniform" | "loguniform" | "grow"
    scorer_D: int
    scorer_m: int
    boundary_density: float
    shuffle_pages: bool = False
    keep_frac: float = 0.5
    threshold: float = 0.95
    num_blocks: int = 0        # 0: sized by the harness from the lengths
    seed: int = 1000

    @property
    def group(self):
        return self.num_q_heads // self.num_kv_heads

    @property
    def elem_bytes(self):
        return 2 if self.dtype == "bf16" else 4

    @property
    def bytes_per_token_layer(self):
        return self.num_kv_heads * self.head_dim * 2 * self.elem_bytes

    @property
    def bytes_per_token(self):
        return self.num_layers * self.bytes_per_token_layer


K = 1024
C0 = Config("C0-tiny", 8, 1, 4, 1, 64, 16, "fp32", 32, 32, 224, "uniform", 256, 64, 1.0,
            num_blocks=256, seed=1000)
C1 = Config("C1-qwen3-8b-1layer", 64, 1, 32, 8, 128, 16, "bf16", 512, 4 * K, 16 * K, "uniform",
            4096, 512, 1.0 / 64, seed=1001)
C2 = Config("C2-long-trace-36layer", 64, 36, 32, 8, 128, 16, "bf16", 512, 16 * K, 32 * K, "uniform",
            4096, 512, 1.0 / 64, shuffle_pages=True, seed=1002)
C3 = Config("C3-memory-saturated", 64, 36, 32, 8, 128, 16, "bf16", 512, 0, 0, "grow",
            4096, 512, 1.0 / 64, num_blocks=65536, seed=1003)
C4 = Config("C4-gqa8", 128, 1, 64, 8, 128, 16, "bf16", 1024, 1 * K, 24 * K, "loguniform",
            5120, 1024, 0.02, seed=1004)
CONFIGS = [C0, C1, C2, C3, C4]


def rng(seed: int, tensor_id: int, sub: int = 0) -> np.random.Generator:
    return np.random.Generator(np.random.Philox(key=[(seed << 20) ^ sub, tensor_id]))


# ---------------------------------------------------------------- bf16 bit utilities
def f32_to_bf16_bits(x: np.ndarray) -> np.ndarray:
    """Round float32 to bfloat16 (nearest even); returns uint16 bit patterns."""
    u = np.ascontiguousarray(x, dtype=np.float32).view(np.uint32)
    rounding = ((u >> 16) & 1) + np.uint32(0x7FFF)
    return ((u + rounding) >> 16).astype(np.uint16)


def bf16_bits_to_f32(b: np.ndarray) -> np.ndarray:
    return (np.ascontiguousarray(b, dtype=np.uint16).astype(np.uint32) << 16).view(np.float32)


def normal(seed, tensor_id, shape, dtype, std=1.0, sub=0):
    """N(0, std^2) values.  Returns (device_bits, exact_values_f32).

    For "bf16" device_bits is uint16 and exact_values is what those bits mean;
    for "fp32" both are the same float32 array.
    """
    x = rng(seed, tensor_id, sub).standard_normal(shape, dtype=np.float32)
    if std != 1.0:
        x = (x * np.float32(std)).astype(np.float32)
    if dtype == "bf16":
        bits = f32_to_bf16_bits(x)
        return bits, bf16_bits_to_f32(bits)
    return x, x


def suffix_lengths(cfg: Config, n=None) -> np.ndarray:
    """Per-trace suffix lengths (inclusive integer ranges; k = 1024)."""
    n = cfg.n_traces if n is None else n
    g = rng(cfg.seed, TID_LEN)
    if cfg.suffix_dist == "uniform":
        return g.integers(cfg.suffix_lo, cfg.suffix_hi + 1, size=n).astype(np.int64)
    if cfg.suffix_dist == "loguniform":
        u = g.uniform(math.log(cfg.suffix_lo), math.log(cfg.suffix_hi), size=n)
        return np.clip(np.rint(np.exp(u)), cfg.suffix_lo, cfg.suffix_hi).astype(np.int64)
    return np.zeros(n, dtype=np.int64)


def boundary_mask(cfg: Config, n_rows: int, sub: int = 0, density=None) -> np.ndarray:
    """Bernoulli(density) step-end flags, uint8."""
    p = cfg.boundary_density if density is None else density
    if p >= 1.0:
        return np.ones(n_rows, dtype=np.uint8)
    return (rng(cfg.seed, TID_MASK, sub).random(n_rows) < p).astype(np.uint8)


def scorer_weights(cfg: Config, std=0.05, bias_std=0.0):
    """W1 [m, D], b1 [m], w2 [m], b2 as (bits, exact) pairs; biases zero by default."""
    W1 = normal(cfg.seed, TID_W1, (cfg.scorer_m, cfg.scorer_D), cfg.dtype, std)
    w2 = normal(cfg.seed, TID_W2, (cfg.scorer_m,), cfg.dtype, std)
    if bias_std > 0:
        b1 = normal(cfg.seed, TID_B1, (cfg.scorer_m,), cfg.dtype, bias_std)
        b2 = float(rng(cfg.seed, TID_B1, 1).standard_normal() * bias_std)
    else:
        z = np.zeros(cfg.scorer_m, dtype=np.float32)
        b1 = (f32_to_bf16_bits(z), z) if cfg.dtype == "bf16" else (z, z)
        b2 = 0.0
    return W1, b1, w2, b2


def block_permutation(seed: int, num_blocks: int) -> np.ndarray:
    """A seeded permutation of block ids (for scattering pages across the pool)."""
    return rng(seed, TID_PERM).permutation(num_blocks).astype(np.int32)


def scaled(cfg: Config, **kw) -> Config:
    """A copy of cfg with some fields replaced (cut-down variants for tests)."""
    return dataclasses.replace(cfg, **kw)


def synthetic_vocab(seed: int, vocab_size: int, step_end_frac: float = 0.01):
    """A stand-in for a tokenizer's vocabulary: `vocab_size` byte strings of 1-8 bytes drawn from letters, digits,
    space, punctuation and the newline character; about `step_end_frac` of the entries get two newlines in a row
    planted somewhere (entries may also contain them by chance, or single and separated newlines, which do not
    count).  Entry 0 is empty.  Returns a list of bytes."""
    g = rng(seed, TID_VOCAB)
    alphabet = np.frombuffer(b"abcdefghijklmnopqrstuvwxyzABCDEFGHIJKLMNOPQRSTUVWXYZ0123456789 .,:;()=+-\n", dtype=np.uint8)
    out = [b""]
    for v in range(1, vocab_size):
        n = int(g.integers(1, 9))
        t = bytearray(alphabet[g.integers(0, len(alphabet), size=n)].tobytes())
        if g.random() < step_end_frac:
            at = int(g.integers(0, n + 1))
            t[at:at] = b"\n\n"
        out.append(bytes(t))
    return out


def token_ids(seed: int, n_rows: int, vocab_size: int, step_end_ids, density: float, sub: int = 0) -> np.ndarray:
    """Sampled-token stand-ins: row i is one of `step_end_ids` with probability `density`, else a uniformly drawn id
    (which may itself end a step).  int32."""
    g = rng(seed, TID_TOK, sub)
    ids = g.integers(0, vocab_size, size=n_rows).astype(np.int32)
    if len(step_end_ids) and density > 0:
        pick = g.random(n_rows) < density
        ids[pick] = np.asarray(step_end_ids, dtype=np.int32)[g.integers(0, len(step_end_ids), size=int(pick.sum()))]
    return ids
