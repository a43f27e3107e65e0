"""Seeded synthetic input generators shared by the tests, the benchmark and the oracle checks.

This module holds none of the method's arithmetic: it only draws random tensors (bf16 bit
patterns, uniforms, token ids) and names the workload shapes.  It imports neither the CUDA
binding nor the oracle, so either side can be fed from it.

All bf16 tensors are returned as ``numpy.uint16`` bit patterns (numpy has no bf16 dtype); the
float32 values they stand for are obtained with :func:`bf16_bits_to_f32`.
"""
from __future__ import annotations

import dataclasses

import numpy as np

BASE_SEED = 260830252


# --------------------------------------------------------------------------- bf16 bit patterns
def f32_to_bf16_bits(x: np.ndarray) -> np.ndarray:
    """Round float32 values to bf16 (round-to-nearest-even) and return the 16-bit patterns."""
    x = np.ascontiguousarray(x, dtype=np.float32)
    u = x.view(np.uint32).astype(np.uint64)
    lsb = (u >> 16) & 1
    u = u + 0x7FFF + lsb
    return ((u >> 16) & 0xFFFF).astype(np.uint16)


def bf16_bits_to_f32(bits: np.ndarray) -> np.ndarray:
    """Exact widening of bf16 bit patterns to float32."""
    b = np.ascontiguousarray(bits, dtype=np.uint16).astype(np.uint32) << 16
    return b.view(np.float32)


def normal_bf16(rng: np.random.Generator, shape, std: float = 1.0) -> np.ndarray:
    """i.i.d. N(0, std^2) rounded to bf16; returned as uint16 bit patterns."""
    return f32_to_bf16_bits((rng.standard_normal(shape, dtype=np.float32) * np.float32(std)))


def uniforms_24bit(rng: np.random.Generator, shape) -> np.ndarray:
    """Uniforms k * 2^-24, k in [0, 2^24): exactly representable in float32."""
    k = rng.integers(0, 1 << 24, size=shape, dtype=np.int64)
    return (k.astype(np.float64) * 2.0 ** -24).astype(np.float32)


def quantize_e4m3_pages(x: np.ndarray):
    """Quantises a float32 cache [n_pages, Hkv, 128, D] to e4m3 bytes with one scale per (page, KV head): scale =
    amax / 448 (rounded to fp16, the precision the library uses it in), byte = nearest e4m3 of x / scale.  How a
    serving stack quantises its cache is its own business; this is merely how the synthetic FP8 caches of the tests
    and the benchmark are made.  Returns (uint8 bytes, float32 scales [n_pages, Hkv])."""
    import torch
    x = np.ascontiguousarray(x, dtype=np.float32)
    amax = np.abs(x).max(axis=(2, 3))
    scale = np.maximum(amax / 448.0, 2.0 ** -14).astype(np.float16).astype(np.float32)
    q = torch.from_numpy(x / scale[:, :, None, None]).clamp_(-448.0, 448.0).to(torch.float8_e4m3fn)
    return q.view(torch.uint8).numpy().copy(), scale


def rng_for(config_id: int, layer: int = 0, stream: int = 0) -> np.random.Generator:
    """Seed recipe: base + 1000 * config + layer, with an extra stream index for independent draws."""
    return np.random.default_rng([BASE_SEED + 1000 * config_id + layer, stream])


# --------------------------------------------------------------------------- workload shapes
@dataclasses.dataclass(frozen=True)
class Workload:
    """Shapes of one benchmark configuration (draft memory, target cache, speculative step)."""

    name: str
    config_id: int
    # draft model attention geometry and memory
    d_layers: int
    d_q_heads: int
    d_kv_heads: int
    d_head_dim: int
    sink: int
    slots: int          # M: slots materialised so far
    window: int         # W
    slot_interval: int  # r
    # target model attention geometry
    t_layers: int
    t_q_heads: int
    t_kv_heads: int
    t_head_dim: int
    prefix: int         # P
    gamma: int
    batch: int = 1
    vocab: int = 32000
    rollback: int = 16

    @property
    def d_model(self) -> int:
        return self.d_q_heads * self.d_head_dim

    @property
    def draft_entries(self) -> int:
        return self.sink + self.slots + self.window

    def draft_kv_bytes_per_layer(self, entries: int | None = None) -> int:
        n = self.draft_entries if entries is None else entries
        return 2 * n * self.d_kv_heads * self.d_head_dim * 2 * self.batch

    def verify_kv_bytes_per_layer(self, rows: int | None = None) -> int:
        t = self.gamma if rows is None else rows
        return 2 * (self.prefix + t) * self.t_kv_heads * self.t_head_dim * 2 * self.batch


WORKLOADS = {
    # tiny single-layer case the oracle finishes in seconds
    "cfg1_tiny": Workload("cfg1_tiny", 1, 1, 8, 2, 64, 0, 64, 64, 16, 1, 8, 2, 128, 1024, 4),
    # 8B-shaped target / 1B-shaped draft at 8K
    "cfg2_8b_8k": Workload("cfg2_8b_8k", 2, 16, 32, 8, 64, 0, 1024, 1024, 8, 32, 32, 8, 128, 8192, 5),
    # same at 32K
    "cfg3_8b_32k": Workload("cfg3_8b_32k", 3, 16, 32, 8, 64, 0, 4096, 4096, 8, 32, 32, 8, 128, 32768, 5),
    # 70B-shaped target / 8B-shaped draft at 32K
    "cfg4_70b_32k": Workload("cfg4_70b_32k", 4, 32, 32, 8, 128, 0, 4096, 4096, 8, 80, 64, 8, 128, 32768, 6),
    # the paper's own constants (sink = window = 128, rollback 16) at 32K, r = 4 and 8
    "paper_r4_32k": Workload("paper_r4_32k", 6, 16, 32, 8, 64, 128, 8160, 128, 4, 32, 32, 8, 128, 32768, 5),
    "paper_r8_32k": Workload("paper_r8_32k", 7, 16, 32, 8, 64, 128, 4080, 128, 8, 32, 32, 8, 128, 32768, 5),
}


def sweep_workloads(prefixes=(4096, 8192, 16384, 32768), batches=(1, 4, 16), gammas=(2, 5, 8),
                    intervals=(20, 16, 10, 8, 5, 4)):
    """The cfg5 sweep grid on 8B-target / 1B-draft shapes: M = W = floor(P / r)."""
    out = []
    for p in prefixes:
        for b in batches:
            for g in gammas:
                for r in intervals:
                    m = p // r
                    out.append(Workload(f"cfg5_p{p}_b{b}_g{g}_r{r}", 5, 16, 32, 8, 64, 0, m, m, r,
                                        32, 32, 8, 128, p, g, batch=b))
    return out


# --------------------------------------------------------------------------- logits for accept/reject
def logits_pair(rng: np.random.Generator, batch: int, gamma: int, vocab: int,
                target_std: float = 4.0, noise_std: float = 1.0):
    """Target logits N(0, target_std^2) and draft logits = target + N(0, noise_std^2), both bf16 bits.

    Target: ``[batch, gamma + 1, vocab]``; draft: ``[batch, gamma, vocab]``.
    """
    tgt = rng.standard_normal((batch, gamma + 1, vocab), dtype=np.float32) * np.float32(target_std)
    drf = tgt[:, :gamma, :] + rng.standard_normal((batch, gamma, vocab), dtype=np.float32) * np.float32(noise_std)
    return f32_to_bf16_bits(tgt), f32_to_bf16_bits(drf)
