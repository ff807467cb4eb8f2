"""Seeded synthetic inputs for Bi-Level Routing Attention (BRA) workloads.

This module serves both the CPU oracle's tests and the CUDA path's tests and
benchmark.  It holds none of the method's arithmetic: only shapes, random
draws and storage-format conversion (fp32 -> bf16 bit patterns).

The shapes are the BiFormer-T stage shapes at 224x224 input (56/28/14 feature
maps with C = 64/128/256, heads of 32 channels, S = 7, topk = 1/4/16: paper
Section 3.4 and Table 1), a 512x512 dense-prediction map at stride 4 with
S = 8, and a tiny fp32 correctness case.  Values are i.i.d. N(0, 1) for Q, K,
V and dO and N(0, 0.02^2) for the LCE depthwise weights; they stand in for the
feature maps of ImageNet / ADE20K images, which are not available here.
"""
from __future__ import annotations

from dataclasses import dataclass, asdict

import numpy as np


@dataclass(frozen=True)
class BraConfig:
    """Problem statement in the paper's notation (Algorithm 1: H, W, C, S, k)."""

    name: str
    B: int
    H: int
    W: int
    C: int
    heads: int
    S: int
    topk: int
    dtype: str  # "f32" or "bf16"
    backward: bool = False

    @property
    def d(self) -> int:
        return self.C // self.heads

    @property
    def R(self) -> int:
        return self.S * self.S

    @property
    def n_r(self) -> int:
        return (self.H // self.S) * (self.W // self.S)

    @property
    def N(self) -> int:
        return self.H * self.W

    @property
    def keys_per_query(self) -> int:
        return self.topk * self.n_r

    def asdict(self):
        return asdict(self)


# 1-based numbering, in the order the benchmark definition lists them.
CONFIGS = {
    1: BraConfig("tiny-fp32", 1, 16, 16, 32, 1, 4, 2, "f32", backward=True),
    2: BraConfig("biformer-t-stage1", 64, 56, 56, 64, 2, 7, 1, "bf16"),
    3: BraConfig("biformer-t-stage3", 64, 14, 14, 256, 8, 7, 16, "bf16"),
    4: BraConfig("dense-pred-512", 2, 128, 128, 64, 2, 8, 4, "bf16"),
    5: BraConfig("biformer-t-stage2-train", 64, 28, 28, 128, 4, 7, 4, "bf16", backward=True),
    # not one of the benchmark's five: the plain-ViT adaptation of Appendix D (DeiT-B width: 12 heads of 64
    # channels, 32 x 32 map, S = 8, k = 12: 192 keys per query); the batch size is ours
    6: BraConfig("vit-adaptation", 16, 32, 32, 768, 12, 8, 12, "bf16"),
}


def with_batch(cfg: BraConfig, B: int) -> BraConfig:
    """Same shape with another batch size (bounded samples, sharding)."""
    d = cfg.asdict()
    d["B"] = int(B)
    return BraConfig(**d)


def bf16_bits(x32: np.ndarray) -> np.ndarray:
    """fp32 -> bf16 bit patterns (uint16), round to nearest even."""
    u = np.ascontiguousarray(x32, dtype=np.float32).view(np.uint32)
    bias = np.uint32(0x7FFF) + ((u >> np.uint32(16)) & np.uint32(1))
    return ((u + bias) >> np.uint32(16)).astype(np.uint16)


def bf16_bits_to_f32(bits: np.ndarray) -> np.ndarray:
    """bf16 bit patterns (uint16) -> the fp32 values they denote (exact)."""
    return (bits.astype(np.uint32) << np.uint32(16)).view(np.float32)


def round_to_dtype(x32: np.ndarray, dtype: str) -> np.ndarray:
    """fp32 array holding exactly the values the storage dtype can represent."""
    if dtype == "bf16":
        return bf16_bits_to_f32(bf16_bits(x32))
    if dtype == "f32":
        return np.ascontiguousarray(x32, dtype=np.float32)
    raise ValueError(f"unknown dtype {dtype!r}")


def make_inputs(cfg: BraConfig, seed: int, clustered: bool = False, with_do: bool = False):
    """Draw Q, K, V [B,H,W,C], LCE weights w [C,5,5] (and dO) for one problem.

    Each tensor has its own PCG64 stream (seed, seed+1, ...) so that a tensor
    does not change when another is added.  Returned arrays are fp32 holding
    values exactly representable in ``cfg.dtype``; ``w`` is always fp32.

    ``clustered=True`` adds to Q and K a per-region offset drawn from four
    cluster centres, so that a few key regions are routed to by most query
    regions (semantic grouping); it exercises fan-in in the backward pass.
    """
    shape = (cfg.B, cfg.H, cfg.W, cfg.C)
    out = {}
    for i, name in enumerate(("Q", "K", "V")):
        rng = np.random.Generator(np.random.PCG64(seed + i))
        out[name] = rng.standard_normal(shape, dtype=np.float32)
    rng = np.random.Generator(np.random.PCG64(seed + 3))
    out["w"] = (0.02 * rng.standard_normal((cfg.C, 5, 5), dtype=np.float32)).astype(np.float32)
    if with_do:
        rng = np.random.Generator(np.random.PCG64(seed + 4))
        out["dO"] = rng.standard_normal(shape, dtype=np.float32)
    if clustered:
        rng = np.random.Generator(np.random.PCG64(seed + 5))
        centres = rng.standard_normal((4, cfg.C), dtype=np.float32)
        hs, ws = cfg.H // cfg.S, cfg.W // cfg.S
        which_q = rng.integers(0, 4, size=(cfg.B, cfg.S, cfg.S))
        which_k = rng.integers(0, 4, size=(cfg.B, cfg.S, cfg.S))
        off_q = np.repeat(np.repeat(centres[which_q], hs, axis=1), ws, axis=2)
        off_k = np.repeat(np.repeat(centres[which_k], hs, axis=1), ws, axis=2)
        out["Q"] = out["Q"] + off_q
        out["K"] = out["K"] + off_k
    for name in ("Q", "K", "V", "dO"):
        if name in out:
            out[name] = round_to_dtype(out[name], cfg.dtype)
    return out
