"""Seeded synthetic inputs for the Q4 KV-cache path: shapes, lengths, block tables, K/V/q values.

This module holds input generation only -- none of the method's arithmetic
(no quantizer, no attention).  Both the CUDA path's tests/bench and the CPU
oracle's tests draw from it so that they see identical bits.

Random numbers come from numpy's counter-based Philox generator keyed by
(seed, stream id).  Values are drawn as N(0,1) in float32 and rounded to
bfloat16 (round-to-nearest-even); tensors are handed out as uint16 bit
patterns so that no framework conversion can change them.

The five workload shapes follow the three models the paper evaluates
(Section 4 "Setup"; Section 3.6): Llama-3.1-8B (32 layers, 32/8 heads, d 128),
Gemma-3-12B (48 layers, 16/8 heads, d 256, 40 of 48 layers with a 1024 window),
DeepSeek-Coder-V2-Lite (27 layers, 16 heads, MLA), context lengths 1K-32K, and
the cross-phase injection scenario of Section 3.5.  They stand in for real
activations, which need model weights and a text corpus.
"""
from __future__ import annotations

import math
from dataclasses import dataclass, field

import numpy as np

BLOCK_TOKENS = 256
BASE_SEED = 20260304


def rng(seed: int, stream: int) -> np.random.Generator:
    return np.random.Generator(np.random.Philox(key=[int(seed) & (2**64 - 1), int(stream) & (2**64 - 1)]))


def f32_to_bf16_bits(x: np.ndarray) -> np.ndarray:
    """Round float32 to bfloat16 (nearest even); returns uint16 bit patterns."""
    u = np.ascontiguousarray(x, dtype=np.float32).view(np.uint32)
    r = ((u >> np.uint32(16)) & np.uint32(1)) + np.uint32(0x7FFF)
    return ((u + r) >> np.uint32(16)).astype(np.uint16)


def bf16_bits_to_f32(bits: np.ndarray) -> np.ndarray:
    return (np.asarray(bits, dtype=np.uint16).astype(np.uint32) << np.uint32(16)).view(np.float32)


def normal_bf16(seed: int, stream: int, shape) -> np.ndarray:
    """N(0,1) values rounded to bf16, as uint16 bit patterns."""
    g = rng(seed, stream)
    return f32_to_bf16_bits(g.standard_normal(size=shape, dtype=np.float32))


def outlier_channels(seed: int, stream: int, n_kv_heads: int, d: int, frac: float = 0.01) -> np.ndarray:
    """Indices (flat head*d + dim) of ceil(frac*Hkv*d) channels that get scaled up."""
    n = math.ceil(frac * n_kv_heads * d)
    g = rng(seed, stream)
    return np.sort(g.choice(n_kv_heads * d, size=n, replace=False))


def kv_bf16(seed: int, stream: int, n_tokens: int, n_kv_heads: int, d: int,
            outliers: np.ndarray | None = None, outlier_gain: float = 8.0) -> np.ndarray:
    """[n_tokens][Hkv][d] bf16 bit patterns; optional channels multiplied by a gain before rounding."""
    g = rng(seed, stream)
    x = g.standard_normal(size=(n_tokens, n_kv_heads * d), dtype=np.float32)
    if outliers is not None and len(outliers):
        x[:, outliers] *= np.float32(outlier_gain)
    return f32_to_bf16_bits(x).reshape(n_tokens, n_kv_heads, d)


def loguniform_lengths(seed: int, stream: int, n: int, lo: int, hi: int) -> np.ndarray:
    g = rng(seed, stream)
    u = g.uniform(math.log(lo), math.log(hi), size=n)
    return np.floor(np.exp(u)).astype(np.int32)


def block_tables(seed: int, stream: int, lens, n_blocks: int, max_blocks: int | None = None,
                 extra_tokens: int = 0) -> np.ndarray:
    """Per-agent block tables: a seeded permutation of the pool's block ids, dealt out in order.

    Each agent gets ceil((len+extra_tokens)/256) distinct physical blocks; unused entries are -1.
    """
    need = [-(-(int(n) + extra_tokens) // BLOCK_TOKENS) for n in lens]
    assert sum(need) <= n_blocks, "pool too small"
    mb = max(need) if max_blocks is None else max_blocks
    perm = rng(seed, stream).permutation(n_blocks).astype(np.int32)
    tab = np.full((len(lens), mb), -1, dtype=np.int32)
    k = 0
    for a, nb in enumerate(need):
        tab[a, :nb] = perm[k:k + nb]
        k += nb
    return tab


@dataclass
class Workload:
    """One benchmark/parity configuration (shapes only; values come from the generators above)."""
    name: str
    n_layers: int
    n_q_heads: int
    n_kv_heads: int
    d_qk: int
    d_v: int
    v_aliases_k: bool
    lens: list                      # cached tokens per agent before the step
    new_tokens: int                 # tokens appended per agent in the step
    window: int = 0                 # sliding window on window layers (0 = none)
    global_every: int = 0           # layer l is global iff (l+1) % global_every == 0 (0 = all global)
    softmax_scale: float = 0.0
    outlier_frac: float = 0.0
    seed: int = BASE_SEED
    kind: str = "decode"            # "decode" | "prefill"
    extra: dict = field(default_factory=dict)

    @property
    def n_agents(self):
        return len(self.lens)

    def layer_window(self, layer: int) -> int:
        if self.window == 0:
            return 0
        if self.global_every and (layer + 1) % self.global_every == 0:
            return 0
        return self.window

    def blocks_needed(self) -> int:
        return sum(-(-(n + self.new_tokens) // BLOCK_TOKENS) for n in self.lens)


def workload(index: int) -> Workload:
    """The five benchmark configurations, 0-based, and (index 5) the per-head MLA cache of Section 3.6 at the sizes of
    configuration 4: keys of 192 dims (3 groups), values of 128 (2 groups), 16 KV heads; (index 6) a chunked-prefill
    phase at d = 256; (index 7) a chunked-prefill phase on the per-head MLA cache."""
    seed = BASE_SEED + index
    if index == 0:
        return Workload("tiny_gqa_decode", 1, 8, 2, 128, 128, False, [1000, 700], 1,
                        softmax_scale=1.0 / math.sqrt(128), seed=seed)
    if index == 1:
        return Workload("llama31_8b_decode", 32, 32, 8, 128, 128, False, [4096] * 5, 1,
                        softmax_scale=1.0 / math.sqrt(128), outlier_frac=0.01, seed=seed)
    if index == 2:
        lens = [int(x) for x in loguniform_lengths(seed, 1, 10, 1024, 32768)]
        return Workload("gemma3_12b_ragged_decode", 48, 16, 8, 256, 256, False, lens, 1,
                        window=1024, global_every=6, softmax_scale=1.0 / math.sqrt(256), seed=seed)
    if index == 3:
        return Workload("dsv2lite_mla_decode", 27, 16, 1, 576, 512, True, [16384] * 4, 1,
                        softmax_scale=1.0 / math.sqrt(192), seed=seed)
    if index == 4:
        return Workload("llama31_8b_chunked_prefill", 32, 32, 8, 128, 128, False, [8192] * 8, 1024,
                        softmax_scale=1.0 / math.sqrt(128), seed=seed, kind="prefill")
    if index == 5:
        return Workload("dsv2lite_perhead_mla_decode", 27, 16, 16, 192, 128, False, [16384] * 4, 1,
                        softmax_scale=1.0 / math.sqrt(192), seed=seed)
    if index == 6:
        # a d = 256 phase (Gemma-3-12B's head shape, global layers)
        return Workload("gemma3_12b_shaped_global_prefill", 8, 16, 8, 256, 256, False, [4096] * 8, 512,
                        softmax_scale=1.0 / math.sqrt(256), seed=seed, kind="prefill")
    if index == 7:
        # a phase on the per-head MLA cache (d_qk 192 / d_v 128, 16 KV heads, one query head each)
        return Workload("dsv2lite_perhead_mla_prefill", 8, 16, 16, 192, 128, False, [4096] * 8, 512,
                        softmax_scale=1.0 / math.sqrt(192), seed=seed, kind="prefill")
    raise IndexError(index)
