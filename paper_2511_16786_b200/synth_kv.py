"""Seeded synthetic KV caches shaped like the paper's MLLM prefill workloads.

This module only makes inputs.  It holds none of the compression method's
arithmetic and is the one piece of code that both the CUDA path's callers and
the CPU oracle's tests may use.  The real workloads (prefill KV caches of
Qwen2.5-VL / LLaVA-OneVision on multi-image, high-resolution and video
benchmarks) need model weights and datasets; these tensors stand in for them
with the structure the paper reports: energy concentrated at low token-axis
frequencies (Fig. 1), a sparse set of rows far from that smooth trend
(Fig. 2), and layers that differ in how much outlier energy they carry
(Fig. 4).

Recipe for one (layer, sequence) of length N, every KV head h and channel c:

    X[i, h, c] = sum_{m < M} a[m, h, c] * cos(pi * m * (2 i + 1) / (2 N))
                 + 0.1 * n[i, h, c],            a, n ~ N(0, 1)

(un-normalised cosines, so the smooth part carries most of the energy), then a
set of round(f * N) token rows, drawn without replacement per head and shared
by K and V, is replaced by 5 * N(0, 1), and the result is cast to the storage
dtype.  K and V use independent draws of a and n.
"""
from __future__ import annotations

import math
import zlib
from dataclasses import dataclass, field

import torch

_DTYPES = {"f32": torch.float32, "f16": torch.float16, "bf16": torch.bfloat16}


@dataclass(frozen=True)
class KVConfig:
    name: str
    num_layers: int
    num_heads: int
    head_dim: int
    seqlens: tuple            # one entry per sequence of the packed batch
    dtype: str                # "f32" | "f16" | "bf16"
    num_low: int              # M: number of low-frequency cosine components
    outlier: tuple            # ("fixed", f) | ("per_layer", lo, hi) | ("per_seq", lo, hi)
    rho: float                # overall retention ratio
    gamma: float = 0.2        # low-pass cutoff factor
    min_keep: int = 1
    seed: int = 0
    note: str = field(default="", compare=False)

    @property
    def torch_dtype(self):
        return _DTYPES[self.dtype]

    @property
    def total_tokens(self) -> int:
        return int(sum(self.seqlens))

    @property
    def cu_seqlens(self) -> list:
        cu = [0]
        for n in self.seqlens:
            cu.append(cu[-1] + int(n))
        return cu


def _ragged_lengths(seed: int, batch: int, lo: int, hi: int) -> tuple:
    g = torch.Generator(device="cpu")
    g.manual_seed(1000003 * seed + 7919 * batch + lo + hi)
    return tuple(int(x) for x in torch.randint(lo, hi + 1, (batch,), generator=g))


def paper_configs() -> dict:
    """The five workload shapes the build is measured and checked on."""
    return {
        "cfg1": KVConfig("cfg1", 1, 4, 128, (1024,), "f32", 8, ("fixed", 0.02), 0.2,
                         note="single layer, 4 KV heads, N=1024, fp32"),
        "cfg2": KVConfig("cfg2", 28, 4, 128, (8192,), "bf16", 8, ("per_layer", 0.005, 0.05), 0.2,
                         note="Qwen2.5-VL-7B-shaped prefill, N=8192, bf16"),
        "cfg3": KVConfig("cfg3", 28, 4, 128, (32768,), "bf16", 16, ("fixed", 0.01), 0.1,
                         note="long multi-image context, N=32768, bf16"),
        "cfg4": KVConfig("cfg4", 32, 32, 128, (16384,), "f16", 8, ("fixed", 0.02), 0.2,
                         note="MHA LLaVA-7B-shaped, N=16384, fp16"),
        "cfg5": KVConfig("cfg5", 28, 4, 128, _ragged_lengths(0, 8, 4096, 65536), "bf16", 8,
                         ("per_seq", 0.005, 0.05), 0.2,
                         note="8 ragged video-style sequences, packed varlen, bf16"),
    }


def _stream(cfg: KVConfig, device, *key) -> torch.Generator:
    g = torch.Generator(device=device)
    h = zlib.crc32(repr((cfg.name, cfg.seed) + tuple(key)).encode())
    g.manual_seed(h + (cfg.seed << 32))
    return g


def outlier_fraction(cfg: KVConfig, layer: int, seq: int) -> float:
    kind = cfg.outlier[0]
    if kind == "fixed":
        return float(cfg.outlier[1])
    lo, hi = cfg.outlier[1], cfg.outlier[2]
    g = _stream(cfg, "cpu", "frac", layer if kind == "per_layer" else -1,
                seq if kind == "per_seq" else -1)
    return float(lo + (hi - lo) * torch.rand((), generator=g, dtype=torch.float64))


def make_layer(cfg: KVConfig, layer: int, device="cpu"):
    """K, V of one layer: [T, H, d] tensors of cfg.torch_dtype on `device`,
    the sequences of the batch packed along the token axis."""
    device = torch.device(device)
    H, d, M = cfg.num_heads, cfg.head_dim, cfg.num_low
    T = cfg.total_tokens
    K = torch.empty((T, H, d), dtype=cfg.torch_dtype, device=device)
    V = torch.empty((T, H, d), dtype=cfg.torch_dtype, device=device)
    cu = cfg.cu_seqlens
    for b, N in enumerate(cfg.seqlens):
        if N == 0:
            continue
        g = _stream(cfg, device, "kv", layer, b)
        i = torch.arange(N, device=device, dtype=torch.float64)
        m = torch.arange(M, device=device, dtype=torch.float64)
        basis = torch.cos(math.pi * (2.0 * i[:, None] + 1.0) * m[None, :] / (2.0 * N)).to(torch.float32)
        f = outlier_fraction(cfg, layer, b)
        n_out = int(round(f * N))
        rows = None
        if n_out > 0:
            rows = torch.stack([torch.randperm(N, generator=g, device=device)[:n_out]
                                for _ in range(H)])          # [H, n_out]
        for dst in (K, V):
            a = torch.randn((M, H * d), generator=g, device=device, dtype=torch.float32)
            x = basis @ a
            x.add_(torch.randn((N, H * d), generator=g, device=device, dtype=torch.float32), alpha=0.1)
            x = x.view(N, H, d)
            if rows is not None:
                repl = 5.0 * torch.randn((H, n_out, d), generator=g, device=device, dtype=torch.float32)
                for h in range(H):
                    x[rows[h], h, :] = repl[h]
            dst[cu[b]:cu[b + 1]] = x.to(cfg.torch_dtype)
    return K, V


def scaled(cfg: KVConfig, name: str, **changes) -> KVConfig:
    """A copy of cfg with some fields replaced (smaller test-sized variants)."""
    base = {f: getattr(cfg, f) for f in cfg.__dataclass_fields__}
    base.update(changes)
    base["name"] = name
    return KVConfig(**base)
