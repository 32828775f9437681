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
dtype.  K and V use independent draws of a and n.  Every draw comes from a
counter-based generator written in exactly defined tensor operations (see
_normal), so a configuration, layer and seed name the same bytes on the CPU and
on a GPU; the normal draws are sums of twelve uniforms.
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


# ---------------------------------------------------------------------------
# Counter-based draws that give the same bytes on every device.  Only operations whose
# results are fixed by their definition are used on tensors: wrapping 64-bit integer
# arithmetic, exact integer-to-float conversion, and single correctly rounded float64
# multiplies, adds and subtractions (one torch call each, so nothing is fused).  No
# library random generator, no transcendental function and no matrix product touches a
# tensor; the few sines and cosines needed are Python floats computed on the host.
# ---------------------------------------------------------------------------
def _signed64(x: int) -> int:
    x &= (1 << 64) - 1
    return x - (1 << 64) if x >= (1 << 63) else x


_M1, _M2, _GOLD = _signed64(0xBF58476D1CE4E5B9), _signed64(0x94D049BB133111EB), _signed64(0x9E3779B97F4A7C15)


def _key(cfg: KVConfig, *key) -> int:
    h = zlib.crc32(repr((cfg.name, cfg.seed) + tuple(key)).encode())
    return _signed64(h * 0x9E3779B97F4A7C15 + cfg.seed * 0xD1B54A32D192ED03 + 0x632BE59BD9B4E019)


def _mix(x: torch.Tensor) -> torch.Tensor:
    """The splitmix64 finaliser on an int64 tensor (logical shifts, wrapping products)."""
    x = x ^ ((x >> 30) & 0x3FFFFFFFF)
    x = x * _M1
    x = x ^ ((x >> 27) & 0x1FFFFFFFFF)
    x = x * _M2
    return x ^ ((x >> 31) & 0x1FFFFFFFF)


def _normal(key: int, count: int, device) -> torch.Tensor:
    """count draws, float64: the sum of twelve independent 16-bit uniforms, centred and scaled to unit
    variance (Irwin-Hall; within 6 standard deviations, kurtosis 2.9)."""
    idx = torch.arange(count, dtype=torch.int64, device=device) * 3
    total = torch.zeros(count, dtype=torch.int64, device=device)
    for r in range(3):
        h = _mix((idx + r) * _GOLD + key)
        for sh in (0, 16, 32, 48):
            total += (h >> sh) & 0xFFFF
    return (total - 6 * 65535).to(torch.float64) * (1.0 / 65536.0)


def _cos_basis(N: int, M: int, device) -> list:
    """[cos(pi * m * (2 i + 1) / (2 N)) for m < M] as float64 vectors over i: e^{j theta_i} by products of
    host-computed rotations chosen by the bits of i, then the three-term recurrence in m."""
    i = torch.arange(N, dtype=torch.int64, device=device)
    t0 = math.pi / (2.0 * N)
    zr = torch.full((N,), math.cos(t0), dtype=torch.float64, device=device)
    zi = torch.full((N,), math.sin(t0), dtype=torch.float64, device=device)
    k = 0
    while (1 << k) < N:
        ang = (math.pi / N) * (1 << k)
        rr, ri = math.cos(ang), math.sin(ang)
        on = ((i >> k) & 1).bool()
        nr = zr * rr - zi * ri
        ni = zr * ri + zi * rr
        zr = torch.where(on, nr, zr)
        zi = torch.where(on, ni, zi)
        k += 1
    out = [torch.ones(N, dtype=torch.float64, device=device)]
    if M > 1:
        out.append(zr)
    two_c = zr * 2.0
    for m in range(2, M):
        out.append(two_c * out[m - 1] - out[m - 2])
    return out[:M]


def outlier_fraction(cfg: KVConfig, layer: int, seq: int) -> float:
    kind = cfg.outlier[0]
    if kind == "fixed":
        return float(cfg.outlier[1])
    lo, hi = cfg.outlier[1], cfg.outlier[2]
    g = _stream(cfg, "cpu", "frac", layer if kind == "per_layer" else -1,
                seq if kind == "per_seq" else -1)
    return float(lo + (hi - lo) * torch.rand((), generator=g, dtype=torch.float64))


def make_layer(cfg: KVConfig, layer: int, device="cpu"):
    """K, V of one layer: [T, H, d] tensors of cfg.torch_dtype on `device`, the sequences of the batch
    packed along the token axis.  The same configuration, layer and seed give the same bytes on every
    device."""
    device = torch.device(device)
    H, d, M = cfg.num_heads, cfg.head_dim, cfg.num_low
    T = cfg.total_tokens
    K = torch.empty((T, H, d), dtype=cfg.torch_dtype, device=device)
    V = torch.empty((T, H, d), dtype=cfg.torch_dtype, device=device)
    cu = cfg.cu_seqlens
    for b, N in enumerate(cfg.seqlens):
        if N == 0:
            continue
        basis = _cos_basis(N, M, device)
        f = outlier_fraction(cfg, layer, b)
        n_out = int(round(f * N))
        rows = None
        if n_out > 0:          # n_out distinct tokens per head: the smallest of N hashed keys
            pos = torch.arange(N, dtype=torch.int64, device=device)
            rows = [torch.sort(_mix(pos * _GOLD + _key(cfg, "rows", layer, b, h)), stable=True).indices[:n_out]
                    for h in range(H)]
        for which, dst in (("k", K), ("v", V)):
            a = _normal(_key(cfg, "coef", which, layer, b), M * H * d, device).view(M, H * d)
            x = _normal(_key(cfg, "noise", which, layer, b), N * H * d, device).view(N, H * d) * 0.1
            for m in range(M):
                x = x + basis[m][:, None] * a[m][None, :]
            x = x.view(N, H, d)
            if rows is not None:
                repl = (_normal(_key(cfg, "outl", which, layer, b), H * n_out * d, device) * 5.0).view(H, n_out, d)
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
