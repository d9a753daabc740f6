"""Seeded synthetic inputs for the MoE decode layer: shapes, streams, bf16 packing.

This module only *makes inputs*. It holds none of the method's arithmetic (no
routing, scoring, selection or expert math) so that the CPU oracle and the CUDA
path can both be fed from it without sharing any of their own code.

Every tensor is a pure function of ``(seed, config name, layer, tensor name,
element index)``: element ``i`` of a stream is ``table[mix64(key, i) >> 48]``
where ``table`` holds the 65536 mid-point quantiles of a normal distribution.
The generator is integer arithmetic plus one table lookup, so the numpy (host)
and torch (device) implementations below are bit-identical, any slice of any
tensor can be regenerated on its own (one expert of one layer, say), and a
58 GB stack can be produced directly in device memory.

Recipe (standing in for the paper's checkpoints, which cannot be loaded here):
hidden states are N(0,1) draws scaled to unit RMS per token and rounded to
bf16; router, expert and predictor matrices are N(0, 0.02) rounded to bf16; the
predictor intercept is N(0, 0.02) in fp32; the router bias is
``-1.1 * ln(rank_e)`` for a seeded random ranking of the experts, so that the
softmax of the bias alone is the Zipf(1.1) distribution over experts.
"""

from __future__ import annotations

import hashlib
from dataclasses import dataclass, field
from functools import lru_cache

import numpy as np

_GAMMA = 0x9E3779B97F4A7C15
_M1 = 0xBF58476D1CE4E5B9
_M2 = 0x94D049BB133111EB
_MASK64 = (1 << 64) - 1
TABLE_BITS = 16
TABLE_SIZE = 1 << TABLE_BITS


@dataclass(frozen=True)
class LayerConfig:
    """Shape of one MoE decode workload. ``budgets`` are expert budgets M."""

    name: str
    d: int          # d_model
    E: int          # routed experts (the paper's N)
    K: int          # router top-K
    I: int          # SwiGLU intermediate size
    T: int          # decode tokens in the batch
    budgets: tuple
    layers: int = 1
    batches: tuple = field(default_factory=tuple)  # stack sweep only
    router_norm: int = 0   # 0: router weights renormalised over the top-K; 1: plain softmax over all experts

    @property
    def expert_bytes(self) -> int:
        return 3 * self.d * self.I * 2


CONFIGS = {
    "tiny": LayerConfig("tiny", d=256, E=16, K=4, I=128, T=8, budgets=(6,)),
    "mid": LayerConfig("mid", d=2048, E=64, K=8, I=1024, T=32, budgets=(8, 16, 24, 64)),
    "qwen3": LayerConfig("qwen3", d=2048, E=128, K=8, I=768, T=64, budgets=(16, 32, 64, 128)),
    "qwen3_stack": LayerConfig("qwen3_stack", d=2048, E=128, K=8, I=768, T=64, budgets=(16, 32, 64),
                               layers=48, batches=(1, 8, 32, 64, 128, 256)),
    "mixtral": LayerConfig("mixtral", d=4096, E=8, K=2, I=14336, T=128, budgets=(2, 4, 6, 8)),
    # The paper's two other models, routed experts only (their always-on shared experts are outside the selection,
    # Sec. 3.1). The paper gives expert counts and top-K; widths are those of the public model configurations
    # (hidden 2048, expert intermediate 1408 for both); neither renormalises the top-K router weights.
    "dsv2lite": LayerConfig("dsv2lite", d=2048, E=64, K=6, I=1408, T=64, budgets=(8, 16, 24, 32, 64), router_norm=1),
    "qwen15moe": LayerConfig("qwen15moe", d=2048, E=60, K=4, I=1408, T=64, budgets=(8, 16, 24, 32, 60), router_norm=1),
}
CONFIG_ORDER = ("tiny", "mid", "qwen3", "qwen3_stack", "mixtral")


# --------------------------------------------------------------------------- bf16 packing

def f32_to_bf16_bits(x: np.ndarray) -> np.ndarray:
    """Round fp32 to bf16 (nearest even) and return the 16-bit patterns."""
    b = np.ascontiguousarray(x, dtype=np.float32).view(np.uint32)
    r = b + (np.uint32(0x7FFF) + ((b >> np.uint32(16)) & np.uint32(1)))
    return (r >> np.uint32(16)).astype(np.uint16)


def bf16_bits_to_f32(bits: np.ndarray) -> np.ndarray:
    """Exact widening of bf16 bit patterns to fp32."""
    return (np.ascontiguousarray(bits, dtype=np.uint16).astype(np.uint32) << np.uint32(16)).view(np.float32)


def bf16_bits_to_f64(bits: np.ndarray) -> np.ndarray:
    return bf16_bits_to_f32(bits).astype(np.float64)


# --------------------------------------------------------------------------- counter-based streams

def stream_key(seed: int, config: str, layer: int, tensor: str) -> int:
    """64-bit key of one tensor's stream."""
    h = hashlib.blake2b(f"{seed}/{config}/{layer}/{tensor}".encode(), digest_size=8)
    return int.from_bytes(h.digest(), "little")


def mix64_np(key: int, start: int, count: int) -> np.ndarray:
    """splitmix64 output for counters start .. start+count-1 (uint64)."""
    with np.errstate(over="ignore"):
        ctr = np.arange(start + 1, start + 1 + count, dtype=np.uint64)
        z = ctr * np.uint64(_GAMMA) + np.uint64(key)
        z = (z ^ (z >> np.uint64(30))) * np.uint64(_M1)
        z = (z ^ (z >> np.uint64(27))) * np.uint64(_M2)
        z = z ^ (z >> np.uint64(31))
    return z


def _s64(c: int) -> int:
    c &= _MASK64
    return c - (1 << 64) if c >= (1 << 63) else c


def mix64_torch(key: int, start: int, count: int, device):
    """Same stream as :func:`mix64_np`, computed with wrapping int64 torch ops."""
    import torch

    def lsr(z, s):
        return (z >> s) & ((1 << (64 - s)) - 1)

    ctr = torch.arange(start + 1, start + 1 + count, dtype=torch.int64, device=device)
    z = ctr * _s64(_GAMMA) + _s64(key)
    z = (z ^ lsr(z, 30)) * _s64(_M1)
    z = (z ^ lsr(z, 27)) * _s64(_M2)
    z = z ^ lsr(z, 31)
    return z


@lru_cache(maxsize=1)
def normal_quantiles() -> np.ndarray:
    """fp64 mid-point quantiles of N(0,1): q[i] = Phi^-1((i + 1/2) / 65536)."""
    from scipy.special import ndtri

    p = (np.arange(TABLE_SIZE, dtype=np.float64) + 0.5) / TABLE_SIZE
    return ndtri(p)


@lru_cache(maxsize=8)
def _bf16_table(sigma: float) -> np.ndarray:
    return f32_to_bf16_bits((normal_quantiles() * sigma).astype(np.float32))


def _index_np(key: int, start: int, count: int) -> np.ndarray:
    """Table indices (top 16 bits of the stream), computed in place on one temporary."""
    with np.errstate(over="ignore"):
        z = np.arange(start + 1, start + 1 + count, dtype=np.uint64)
        z *= np.uint64(_GAMMA)
        z += np.uint64(key)
        t = z >> np.uint64(30)
        z ^= t
        z *= np.uint64(_M1)
        np.right_shift(z, np.uint64(27), out=t)
        z ^= t
        z *= np.uint64(_M2)
        np.right_shift(z, np.uint64(31), out=t)
        z ^= t
        z >>= np.uint64(64 - TABLE_BITS)
    return z


def normal_f64(key: int, start: int, count: int) -> np.ndarray:
    """N(0,1) draws in fp64 (65536-level table)."""
    return normal_quantiles()[_index_np(key, start, count)]


def normal_bf16_bits(key: int, start: int, count: int, sigma: float, chunk: int = 1 << 18,
                     threads: int | None = None) -> np.ndarray:
    """N(0, sigma) draws rounded to bf16, as uint16 bit patterns (host; chunks run on a thread pool)."""
    table = _bf16_table(float(sigma))
    out = np.empty(count, dtype=np.uint16)

    def work(off):
        n = min(chunk, count - off)
        out[off:off + n] = table[_index_np(key, start + off, n)]

    offsets = range(0, count, chunk)
    if count <= chunk:
        for off in offsets:
            work(off)
    else:
        from concurrent.futures import ThreadPoolExecutor
        import os
        with ThreadPoolExecutor(threads or min(16, os.cpu_count() or 1)) as ex:
            list(ex.map(work, offsets))
    return out


def normal_bf16_device(key: int, start: int, count: int, sigma: float, device, chunk: int = 1 << 26):
    """Same values as :func:`normal_bf16_bits`, produced in device memory as a bf16 tensor."""
    import torch

    table = torch.from_numpy(_bf16_table(float(sigma)).view(np.int16).copy()).to(device)
    out = torch.empty(count, dtype=torch.int16, device=device)
    for off in range(0, count, chunk):
        n = min(chunk, count - off)
        z = mix64_torch(key, start + off, n, device)
        idx = (z >> (64 - TABLE_BITS)) & (TABLE_SIZE - 1)
        out[off:off + n] = table[idx]
    return out.view(torch.bfloat16)


# --------------------------------------------------------------------------- tensors of one layer

WEIGHT_SIGMA = 0.02
ZIPF_EXPONENT = 1.1

_EXPERT_TENSORS = ("w_gate", "w_up", "w_down")


def expert_tensor_shape(cfg: LayerConfig, tensor: str):
    if tensor in ("w_gate", "w_up"):
        return (cfg.E, cfg.I, cfg.d)
    if tensor == "w_down":
        return (cfg.E, cfg.d, cfg.I)
    raise KeyError(tensor)


def hidden_bits(cfg: LayerConfig, T: int | None = None, seed: int = 0, layer: int = 0,
                stream: str = "hidden") -> np.ndarray:
    """[T, d] bf16 bits: N(0,1) rows scaled to unit RMS, then rounded to bf16."""
    T = cfg.T if T is None else T
    z = normal_f64(stream_key(seed, cfg.name, layer, stream), 0, T * cfg.d).reshape(T, cfg.d)
    z = z / np.sqrt(np.mean(z * z, axis=1, keepdims=True))
    return f32_to_bf16_bits(z.astype(np.float32)).reshape(T, cfg.d)


def router_bias(cfg: LayerConfig, seed: int = 0, layer: int = 0, scale: float = 1.0) -> np.ndarray:
    """[E] fp32: -1.1 ln(rank) over a seeded random ranking of the experts."""
    h = mix64_np(stream_key(seed, cfg.name, layer, "router_rank"), 0, cfg.E)
    order = np.argsort(h, kind="stable")
    rank = np.empty(cfg.E, dtype=np.float64)
    rank[order] = np.arange(1, cfg.E + 1, dtype=np.float64)
    return (-ZIPF_EXPONENT * scale * np.log(rank)).astype(np.float32)


def small_tensors(cfg: LayerConfig, seed: int = 0, layer: int = 0) -> dict:
    """Router and predictor parameters of one layer (host arrays).

    router_w, pred_A: [E, d] bf16 bits; router_bias, pred_b: [E] fp32.
    """
    E, d = cfg.E, cfg.d
    key = lambda name: stream_key(seed, cfg.name, layer, name)
    return {
        "router_w": normal_bf16_bits(key("router_w"), 0, E * d, WEIGHT_SIGMA).reshape(E, d),
        "router_bias": router_bias(cfg, seed, layer),
        "pred_A": normal_bf16_bits(key("pred_A"), 0, E * d, WEIGHT_SIGMA).reshape(E, d),
        "pred_b": (normal_f64(key("pred_b"), 0, E) * WEIGHT_SIGMA).astype(np.float32),
    }


def expert_weights_host(cfg: LayerConfig, expert: int, seed: int = 0, layer: int = 0) -> dict:
    """bf16 bits of one expert: w_gate [I,d], w_up [I,d], w_down [d,I]."""
    out = {}
    for name in _EXPERT_TENSORS:
        shp = expert_tensor_shape(cfg, name)[1:]
        n = shp[0] * shp[1]
        out[name] = normal_bf16_bits(stream_key(seed, cfg.name, layer, name), expert * n, n,
                                     WEIGHT_SIGMA).reshape(shp)
    return out


def expert_weights_host_all(cfg: LayerConfig, seed: int = 0, layer: int = 0) -> dict:
    """bf16 bits of all experts of a layer: w_gate/w_up [E,I,d], w_down [E,d,I]."""
    out = {}
    for name in _EXPERT_TENSORS:
        shp = expert_tensor_shape(cfg, name)
        out[name] = normal_bf16_bits(stream_key(seed, cfg.name, layer, name), 0, int(np.prod(shp)),
                                     WEIGHT_SIGMA).reshape(shp)
    return out


def expert_weights_device(cfg: LayerConfig, device, seed: int = 0, layer: int = 0) -> dict:
    """All experts of a layer as bf16 torch tensors generated in device memory."""
    out = {}
    for name in _EXPERT_TENSORS:
        shp = expert_tensor_shape(cfg, name)
        out[name] = normal_bf16_device(stream_key(seed, cfg.name, layer, name), 0, int(np.prod(shp)),
                                       WEIGHT_SIGMA, device).view(shp)
    return out


def plant_energy_direction(cfg: LayerConfig, w_gate_bits: np.ndarray, alpha: float, seed: int = 0) -> np.ndarray:
    """Extra test workload: add alpha * 1 v_u^T (v_u a seeded unit vector) to each expert's gate
    matrix so that its output energy depends on the direction of the token. Returns bf16 bits."""
    E, I, d = w_gate_bits.shape
    v = normal_f64(stream_key(seed, cfg.name, 0, "planted_v"), 0, E * d).reshape(E, d)
    v /= np.linalg.norm(v, axis=1, keepdims=True)
    w = bf16_bits_to_f32(w_gate_bits).reshape(E, I, d) + (alpha * v[:, None, :]).astype(np.float32)
    return f32_to_bf16_bits(w).reshape(E, I, d)
