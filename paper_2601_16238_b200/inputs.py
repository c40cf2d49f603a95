"""Seeded synthetic inputs shared by the tests, the benchmark and the oracle checks.

This module holds no attention arithmetic: it draws i.i.d. N(0,1) values from a
host-side Philox generator in fp32, rounds them once to bfloat16
(round-to-nearest-even) and hands out the bit patterns as ``uint16`` arrays.
The CPU oracle and the GPU library both consume exactly these bits.

The named workloads mirror the shapes the paper reports or trains on: the
kernel-microbenchmark rows "Attention (fwd)/(bwd)" (shape tuple
(B, Hq, Hkv, S, D), bf16, causal) and the attention shapes of its miniGPT and
ViT training checks.  Data sets are replaced by N(0,1) values.
"""
from __future__ import annotations

from dataclasses import dataclass, replace

import numpy as np


@dataclass(frozen=True)
class AttnConfig:
    name: str
    index: int          # seed family: tensors use seeds 1000*index + {1,2,3,4}
    B: int
    Hq: int
    Hkv: int
    Sq: int
    Sk: int
    D: int
    causal: bool        # False / True (top-left aligned); the int 2 selects the bottom-right aligned mask
    backward: bool

    @property
    def scale(self) -> float:
        """1/sqrt(D) rounded to fp32 (the value passed through the C ABI)."""
        return float(np.float32(1.0) / np.sqrt(np.float32(self.D)))

    def fwd_flops(self) -> float:
        """4*B*Hq*Sq*Sk*D, halved when causal (the benchmark's flop convention).  For the bottom-right
        aligned mask with Sq != Sk the factor is the visible share of the Sq x Sk rectangle in the same
        continuous approximation (1/2 when square): 1 - Sq/(2 Sk), or Sk/(2 Sq) when Sk < Sq."""
        f = 4.0 * self.B * self.Hq * self.Sq * self.Sk * self.D
        if int(self.causal) == 2:
            return f * (1.0 - self.Sq / (2.0 * self.Sk) if self.Sk >= self.Sq else self.Sk / (2.0 * self.Sq))
        return f * 0.5 if self.causal else f

    def bwd_flops(self) -> float:
        return 2.5 * self.fwd_flops()

    def with_(self, **kw) -> "AttnConfig":
        return replace(self, **kw)


def _c4(s: int, causal: bool) -> AttnConfig:
    tag = "c" if causal else "nc"
    return AttnConfig(f"sdpa_s{s}_{tag}", 4, 4, 16, 16, s, s, 128, causal, False)


CONFIGS = {
    "tiny": AttnConfig("tiny", 1, 1, 2, 2, 128, 128, 64, False, True),
    "minigpt": AttnConfig("minigpt", 2, 8, 8, 8, 256, 256, 64, True, True),
    "vit": AttnConfig("vit", 3, 128, 6, 6, 65, 65, 64, False, True),
    **{c.name: c for c in (_c4(s, causal) for s in (1024, 2048, 4096, 8192)
                           for causal in (False, True))},
    "gqa_long": AttnConfig("gqa_long", 5, 1, 32, 8, 16384, 16384, 128, True, True),
    # a long D=64 shape (not a graded config): the exponential unit, not the tensor core, bounds it
    "d64_s4096_nc": AttnConfig("d64_s4096_nc", 7, 4, 16, 16, 4096, 4096, 64, False, True),
    # a long D=256 shape (not a graded config): the forward with 256 columns, the backward's kernels for 128 < D <= 256
    "d256_s4096_nc": AttnConfig("d256_s4096_nc", 8, 4, 8, 8, 4096, 4096, 256, False, True),
    # low-occupancy shapes for the split-KV forward: one decoded token against a long cache, and a prefill chunk at the
    # end of a long context (bottom-right aligned mask); forward only
    "decode_32k": AttnConfig("decode_32k", 12, 4, 32, 8, 1, 32768, 128, 2, False),
    "prefill_chunk": AttnConfig("prefill_chunk", 13, 1, 32, 8, 512, 16384, 128, 2, False),
    # the shape of the paper's own attention rows (context, not a graded config)
    "paper_shape": AttnConfig("paper_shape", 6, 32, 10, 10, 2048, 2048, 128, True, True),
}


def f32_to_bf16_bits(x: np.ndarray) -> np.ndarray:
    """Round fp32 to bfloat16 (nearest even) and return the uint16 bit patterns."""
    u = np.ascontiguousarray(x, dtype=np.float32).view(np.uint32)
    rounded = u + np.uint32(0x7FFF) + ((u >> np.uint32(16)) & np.uint32(1))
    return (rounded >> np.uint32(16)).astype(np.uint16)


def normal_bf16(shape, seed: int) -> np.ndarray:
    """i.i.d. N(0,1) in fp32 from Philox(key=seed), rounded to bf16 bits (uint16)."""
    gen = np.random.Generator(np.random.Philox(key=int(seed)))
    n = int(np.prod(shape))
    out = np.empty(n, dtype=np.uint16)
    chunk = 1 << 24
    for s in range(0, n, chunk):
        e = min(n, s + chunk)
        out[s:e] = f32_to_bf16_bits(gen.standard_normal(e - s, dtype=np.float32))
    return out.reshape(shape)


def normal_f16(shape, seed: int) -> np.ndarray:
    """i.i.d. N(0,1) in fp32 from Philox(key=seed), rounded to IEEE half bits (uint16)."""
    gen = np.random.Generator(np.random.Philox(key=int(seed)))
    return gen.standard_normal(int(np.prod(shape)), dtype=np.float32).astype(np.float16).view(np.uint16).reshape(shape)


def make_inputs(cfg: AttnConfig, with_do: bool = True, seed_offset: int = 0):
    """Q, K, V (and dO) bit patterns for ``cfg``; layout [B, H, S, D], D innermost."""
    base = 1000 * cfg.index + seed_offset
    q = normal_bf16((cfg.B, cfg.Hq, cfg.Sq, cfg.D), base + 1)
    k = normal_bf16((cfg.B, cfg.Hkv, cfg.Sk, cfg.D), base + 2)
    v = normal_bf16((cfg.B, cfg.Hkv, cfg.Sk, cfg.D), base + 3)
    if not with_do:
        return q, k, v
    d_o = normal_bf16((cfg.B, cfg.Hq, cfg.Sq, cfg.D), base + 4)
    return q, k, v, d_o


# --------------------------------------------------------------------------------------------
# Packed (variable-length) workloads: documents of different lengths concatenated without padding,
# the batch shape of a NanoChat-style training step (the paper's attention rows use "batch 32,
# sequence length 2048"; real batches of that size are packed from documents).
# --------------------------------------------------------------------------------------------
@dataclass(frozen=True)
class VarlenConfig:
    name: str
    index: int
    Hq: int
    Hkv: int
    D: int
    causal: bool
    total: int          # tokens in the packed batch (self-attention: same for q and k)
    min_len: int
    max_len: int

    @property
    def scale(self) -> float:
        return float(np.float32(1.0) / np.sqrt(np.float32(self.D)))

    def lengths(self):
        """Seeded document lengths, uniform in [min_len, max_len], the last one cut to fill `total` exactly."""
        gen = np.random.Generator(np.random.Philox(key=1000 * self.index))
        out, left = [], self.total
        while left > 0:
            n = int(min(left, gen.integers(self.min_len, self.max_len + 1)))
            out.append(n)
            left -= n
        return out

    def cu_seqlens(self) -> np.ndarray:
        return np.concatenate([[0], np.cumsum(self.lengths())]).astype(np.int32)

    def fwd_flops(self) -> float:
        f = sum(4.0 * self.Hq * n * n * self.D for n in self.lengths())
        return f * 0.5 if self.causal else f

    def bwd_flops(self) -> float:
        return 2.5 * self.fwd_flops()


VARLEN_CONFIGS = {
    # 32 x 2048 tokens of the paper's head shape (Hq = Hkv = 10, D = 128, causal), packed from documents of 64..2048 tokens
    "packed_docs": VarlenConfig("packed_docs", 8, 10, 10, 128, True, 32 * 2048, 64, 2048),
    "packed_docs_small": VarlenConfig("packed_docs_small", 9, 4, 2, 64, True, 2048, 1, 300),
}


def make_varlen_inputs(cfg: VarlenConfig, with_do: bool = True):
    """q, k, v (and dO) bit patterns, packed [total, H, D], plus cu_seqlens (int32)."""
    base = 1000 * cfg.index
    q = normal_bf16((cfg.total, cfg.Hq, cfg.D), base + 1)
    k = normal_bf16((cfg.total, cfg.Hkv, cfg.D), base + 2)
    v = normal_bf16((cfg.total, cfg.Hkv, cfg.D), base + 3)
    cu = cfg.cu_seqlens()
    if not with_do:
        return q, k, v, cu
    return q, k, v, normal_bf16((cfg.total, cfg.Hq, cfg.D), base + 4), cu
