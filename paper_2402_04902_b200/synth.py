"""Seeded synthetic inputs for the L4Q linear layer.

This module only draws numbers and lays them out; it holds none of the
layer's arithmetic (no merge, quantization, matmul or gradient).  Both the
CPU oracle's tests and the CUDA path's tests/benchmarks take their inputs
from here so that they see identical bits.

Generator: a counter-based hash (splitmix64 finaliser) of
(seed, stream id, element index) -> 64 random bits -> uniform in (0, 1) ->
Box-Muller for normals.  No state, so any slice of any tensor can be
regenerated independently and results do not depend on a library version.

The value recipe follows the workload description of the benchmark configs:
W0 ~ N(0, 0.02^2) with optionally 0.1 % of entries scaled x20 (outliers),
A ~ U(-1/sqrt(d_in), 1/sqrt(d_in)) (Kaiming-uniform with a = sqrt(5), the
LoRA default named in Sec. 4.1), B ~ N(0, 1e-3^2), X and dY ~ N(0, 1);
s = (max - min) / (2^bits - 1) and b = min of each weight group of W0
(min/max asymmetric initialisation, App. B), on the unsigned grid.
"""
from __future__ import annotations

import os
from concurrent.futures import ThreadPoolExecutor
from dataclasses import dataclass, replace

import numpy as np

_U64 = np.uint64
_GOLDEN = _U64(0x9E3779B97F4A7C15)
_CHUNK = 1 << 20


@dataclass(frozen=True)
class LayerConfig:
    """One L4Q linear layer workload."""

    name: str
    tokens: int
    d_in: int
    d_out: int
    rank: int
    alpha: float
    bits: int
    group_size: int
    io_dtype: str = "bf16"        # "bf16" or "f32": dtype of X, dY, W0, Y, dX
    outliers: bool = True         # 0.1 % of W0 entries scaled x20
    signed_grid: bool = False

    def with_(self, **kw) -> "LayerConfig":
        return replace(self, **kw)


def _mix(z: np.ndarray) -> np.ndarray:
    z = (z ^ (z >> _U64(30))) * _U64(0xBF58476D1CE4E5B9)
    z = (z ^ (z >> _U64(27))) * _U64(0x94D049BB133111EB)
    return z ^ (z >> _U64(31))


def _bits64(seed: int, stream: int, lane: int, start: int, count: int) -> np.ndarray:
    """64 random bits for element indices [start, start+count) of one stream/lane."""
    with np.errstate(over="ignore"):
        key = _mix(_U64(seed) * _GOLDEN + _U64(stream) * _U64(0xD1342543DE82EF95) + _U64(lane))
        idx = np.arange(start, start + count, dtype=np.uint64)
        return _mix((idx + _U64(1)) * _GOLDEN ^ key)


def _unit(bits: np.ndarray) -> np.ndarray:
    """Top 53 bits -> uniform double strictly inside (0, 1)."""
    return ((bits >> _U64(11)).astype(np.float64) + 0.5) * (1.0 / 9007199254740992.0)


def _chunked(fill, n: int) -> np.ndarray:
    """Run ``fill(out, start, count)`` over chunks of [0, n); chunks are independent
    (counter-based generator), so they are spread over a few host threads."""
    out = np.empty(n, dtype=np.float64)
    starts = list(range(0, n, _CHUNK))
    if len(starts) <= 1:
        for s0 in starts:
            fill(out, s0, min(_CHUNK, n - s0))
        return out
    with ThreadPoolExecutor(max_workers=min(16, os.cpu_count() or 1)) as pool:
        list(pool.map(lambda s0: fill(out, s0, min(_CHUNK, n - s0)), starts))
    return out


def uniform01(seed: int, stream: int, n: int, lane: int = 0) -> np.ndarray:
    def fill(out, s0, c):
        out[s0:s0 + c] = _unit(_bits64(seed, stream, lane, s0, c))
    return _chunked(fill, n)


def normal(seed: int, stream: int, n: int) -> np.ndarray:
    """Standard normals by Box-Muller (one normal per index; two uniforms each)."""
    def fill(out, s0, c):
        u1 = _unit(_bits64(seed, stream, 0, s0, c))
        u2 = _unit(_bits64(seed, stream, 1, s0, c))
        out[s0:s0 + c] = np.sqrt(-2.0 * np.log(u1)) * np.cos(2.0 * np.pi * u2)
    return _chunked(fill, n)


def f32_to_bf16_bits(x: np.ndarray) -> np.ndarray:
    """float32 -> bfloat16 bit pattern (uint16), round to nearest even."""
    u = np.ascontiguousarray(x, dtype=np.float32).view(np.uint32)
    r = (u + np.uint32(0x7FFF) + ((u >> np.uint32(16)) & np.uint32(1))) >> np.uint32(16)
    return r.astype(np.uint16)


def bf16_bits_to_f32(h: np.ndarray) -> np.ndarray:
    """bfloat16 bit pattern (uint16) -> float32 (exact)."""
    return (np.ascontiguousarray(h, dtype=np.uint16).astype(np.uint32) << np.uint32(16)).view(np.float32)


# stream ids of the tensors of one layer
_S_W0, _S_OUT, _S_A, _S_B, _S_X, _S_DY = 1, 2, 3, 4, 5, 6


def _narrow(x64: np.ndarray, io_dtype: str) -> np.ndarray:
    """Round to the layer's I/O dtype and return the values as float32."""
    x32 = x64.astype(np.float32)
    if io_dtype == "bf16":
        return bf16_bits_to_f32(f32_to_bf16_bits(x32))
    return x32


def group_minmax_init(W0: np.ndarray, bits: int, group_size: int, signed_grid: bool = False):
    """Asymmetric min/max initialisation of (s, b) per group of W0 (float32).

    Unsigned grid: s = (max-min)/(2^bits-1), b = min.  Signed grid (App. B,
    "Asymm"): same s, b = min - s*Q_N.  s is floored at 1e-8.
    """
    o, i = W0.shape
    Wg = W0.astype(np.float32).reshape(o, i // group_size, group_size)
    lo = Wg.min(axis=2)
    hi = Wg.max(axis=2)
    s = np.maximum((hi - lo) / np.float32((1 << bits) - 1), np.float32(1e-8)).astype(np.float32)
    b = lo.astype(np.float32)
    if signed_grid:
        b = (lo - s * np.float32(-(1 << (bits - 1)))).astype(np.float32)
    return s, b


def make_layer_acts(cfg: LayerConfig, seed: int = 0, layer_id: int = 0) -> dict:
    """X and dY of one layer only (same streams as :func:`make_layer_inputs`)."""
    o, i, M = cfg.d_out, cfg.d_in, cfg.tokens
    base = 16 * layer_id
    return {"X": _narrow(normal(seed, base + _S_X, M * i), cfg.io_dtype).reshape(M, i),
            "dY": _narrow(normal(seed, base + _S_DY, M * o), cfg.io_dtype).reshape(M, o)}


def make_layer_inputs(cfg: LayerConfig, seed: int = 0, layer_id: int = 0,
                      zero_B: bool = False, need_acts: bool = True) -> dict:
    """All tensors of one layer, as float32 numpy arrays holding values that
    are exactly representable in the layer's I/O dtype (bf16 tensors are
    returned as float32 carrying bf16 values; see :func:`f32_to_bf16_bits`)."""
    o, i, r, M = cfg.d_out, cfg.d_in, cfg.rank, cfg.tokens
    base = 16 * layer_id
    W0 = 0.02 * normal(seed, base + _S_W0, o * i)
    if cfg.outliers:
        pick = uniform01(seed, base + _S_OUT, o * i) < 1e-3
        W0[pick] *= 20.0
    W0 = _narrow(W0, cfg.io_dtype).reshape(o, i)
    bound = 1.0 / np.sqrt(float(i))
    A = ((2.0 * uniform01(seed, base + _S_A, r * i) - 1.0) * bound).astype(np.float32).reshape(r, i)
    if zero_B:
        B = np.zeros((o, r), dtype=np.float32)
    else:
        B = (1e-3 * normal(seed, base + _S_B, o * r)).astype(np.float32).reshape(o, r)
    s, b = group_minmax_init(W0, cfg.bits, cfg.group_size, cfg.signed_grid)
    out = {"W0": W0, "A": A, "B": B, "s": s, "b": b}
    if need_acts:
        out.update(make_layer_acts(cfg, seed, layer_id))
    return out


# ---------------------------------------------------------------------------
# The benchmark configurations (shapes of the LLaMA-7B / Mistral-7B linears)
# ---------------------------------------------------------------------------

CONFIG1 = LayerConfig("cfg1_256x256_f32", tokens=128, d_in=256, d_out=256, rank=8, alpha=16.0,
                      bits=4, group_size=64, io_dtype="f32", outliers=False)
CONFIG2 = LayerConfig("cfg2_attn_4096x4096", tokens=4096, d_in=4096, d_out=4096, rank=16, alpha=32.0,
                      bits=4, group_size=128)
CONFIG3A = LayerConfig("cfg3a_mlp_up_4096x11008", tokens=8192, d_in=4096, d_out=11008, rank=16,
                       alpha=32.0, bits=4, group_size=128)
CONFIG3B = LayerConfig("cfg3b_mlp_down_11008x4096", tokens=8192, d_in=11008, d_out=4096, rank=16,
                       alpha=32.0, bits=4, group_size=128)
CONFIG4A = CONFIG3A.with_(name="cfg4a_mlp_up_3bit_r64", rank=64, bits=3, group_size=64)
CONFIG4B = CONFIG3B.with_(name="cfg4b_mlp_down_3bit_r64", rank=64, bits=3, group_size=64)


def mistral_block_layers(tokens: int = 8192) -> list[LayerConfig]:
    """The seven L4Q linears of one Mistral-7B-shaped decoder block (config 5)."""
    def L(name, i, o):
        return LayerConfig("cfg5_" + name, tokens=tokens, d_in=i, d_out=o, rank=16, alpha=32.0,
                           bits=4, group_size=128)
    return [L("q", 4096, 4096), L("k", 4096, 1024), L("v", 4096, 1024), L("o", 4096, 4096),
            L("gate", 4096, 14336), L("up", 4096, 14336), L("down", 14336, 4096)]
