"""Seeded synthetic inputs for the MatKV attention path.

This module serves both the CPU oracle's tests and the CUDA path's tests and
benchmark.  It holds NO attention arithmetic: only a counter-based generator of
bf16 bit patterns, the workload shapes, and the chunk-id selection recipes.

Generator (integer-only, so a host and a device implementation give identical
bytes): element ``idx`` of stream ``stream`` under ``seed`` is

    acc = sum over k in {0,1,2} of the four 16-bit fields of
          mix64(seed * C1 + stream * C2 + 3 * idx + k)
    x   = (acc - 393210) * 2**(shift - 16)

i.e. a centred sum of twelve uniform 16-bit integers (variance 1 at shift 0,
|x| < 6), rounded to bf16 with round-to-nearest-even.  ``mix64`` is the
splitmix64 finaliser.  Workload shapes follow the paper's RAG settings
(1,024-token chunks, 2-10 chunks per request, ~20-token query suffixes, batch
1-32, skewed chunk reuse); the values themselves are noise standing in for
real model K/V, which would need model weights and the paper's datasets.
"""
from __future__ import annotations

from dataclasses import dataclass, field
from typing import List

import numpy as np

_C1 = np.uint64(0x9E3779B97F4A7C15)
_C2 = np.uint64(0xD1B54A32D192ED03)
_M1 = np.uint64(0xBF58476D1CE4E5B9)
_M2 = np.uint64(0x94D049BB133111EB)
_CENTER = 393210  # 12 * 65535 / 2


def mix64(x: np.ndarray) -> np.ndarray:
    """splitmix64 finaliser on uint64 arrays (wrapping arithmetic)."""
    x = x.astype(np.uint64, copy=True)
    with np.errstate(over="ignore"):
        x ^= x >> np.uint64(30)
        x *= _M1
        x ^= x >> np.uint64(27)
        x *= _M2
        x ^= x >> np.uint64(31)
    return x


def _acc(seed: int, stream: int, start: int, n: int) -> np.ndarray:
    idx = np.arange(start, start + n, dtype=np.uint64)
    with np.errstate(over="ignore"):
        base = np.uint64(seed) * _C1 + np.uint64(stream) * _C2 + idx * np.uint64(3)
    acc = np.zeros(n, dtype=np.int64)
    m16 = np.uint64(0xFFFF)
    for k in range(3):
        with np.errstate(over="ignore"):
            h = mix64(base + np.uint64(k))
        acc += (h & m16).astype(np.int64)
        acc += ((h >> np.uint64(16)) & m16).astype(np.int64)
        acc += ((h >> np.uint64(32)) & m16).astype(np.int64)
        acc += (h >> np.uint64(48)).astype(np.int64)
    return acc


def f32_to_bf16_bits(x: np.ndarray) -> np.ndarray:
    """Round fp32 values to bf16 bit patterns, nearest-even (finite inputs)."""
    u = np.ascontiguousarray(x, dtype=np.float32).view(np.uint32)
    r = u + np.uint32(0x7FFF) + ((u >> np.uint32(16)) & np.uint32(1))
    return (r >> np.uint32(16)).astype(np.uint16)


def bf16_bits_to_f64(b: np.ndarray) -> np.ndarray:
    """Widen bf16 bit patterns exactly to float64."""
    u = np.ascontiguousarray(b, dtype=np.uint16).astype(np.uint32) << np.uint32(16)
    return u.view(np.float32).astype(np.float64)


def normal_bf16(seed: int, stream: int, n: int, shift: int = 0, start: int = 0) -> np.ndarray:
    """``n`` bf16 bit patterns (uint16) of the generator, elements start..start+n."""
    out = np.empty(n, dtype=np.uint16)
    step = 1 << 22
    for o in range(0, n, step):
        m = min(step, n - o)
        acc = _acc(seed, stream, start + o, m)
        x = (acc - _CENTER).astype(np.float32) * np.float32(2.0 ** (shift - 16))
        out[o:o + m] = f32_to_bf16_bits(x)
    return out


def uniform01(seed: int, stream: int, n: int) -> np.ndarray:
    """``n`` doubles in [0,1) from the same counter-based hash (workload structure only)."""
    idx = np.arange(n, dtype=np.uint64)
    with np.errstate(over="ignore"):
        h = mix64(np.uint64(seed) * _C1 + np.uint64(stream) * _C2 + idx)
    return (h >> np.uint64(11)).astype(np.float64) * (1.0 / (1 << 53))


# stream ids: one per tensor kind so that tensors never share counters
STREAM_CHUNK = 1 << 20      # + chunk index
STREAM_Q_PREFILL = 1
STREAM_K_PREFILL = 2
STREAM_V_PREFILL = 3
STREAM_Q_DECODE = 4
STREAM_K_DECODE = 5
STREAM_V_DECODE = 6
STREAM_PICK = 7


@dataclass
class Workload:
    """Shape of one synthetic RAG attention workload (notation of the scope table)."""
    name: str
    n_layers: int
    n_q_heads: int
    n_kv_heads: int
    head_dim: int
    batch: int
    chunk_tokens: int
    chunks_per_req: int
    pool_chunks: int          # number of distinct materialised chunks
    suffix: int               # S
    decode_steps: int         # T
    seed: int
    pick: str = "own"         # own | zipf | uniform
    n_batches: int = 1
    extra: dict = field(default_factory=dict)

    @property
    def group(self) -> int:
        return self.n_q_heads // self.n_kv_heads

    @property
    def beta(self) -> int:
        """KV bytes per token per layer: K and V, all KV heads, bf16."""
        return 2 * self.n_kv_heads * self.head_dim * 2

    @property
    def chunk_elems(self) -> int:
        return self.n_layers * 2 * self.n_kv_heads * self.chunk_tokens * self.head_dim

    @property
    def chunk_bytes(self) -> int:
        return self.chunk_elems * 2

    def chunk_ids(self, batch_index: int = 0) -> List[List[int]]:
        """Ordered chunk-id list per request of one batch."""
        B, n, P = self.batch, self.chunks_per_req, self.pool_chunks
        if self.pick == "own":
            return [[(r * n + i) % P for i in range(n)] for r in range(B)]
        u = uniform01(self.seed, STREAM_PICK + 64 * batch_index, B * n * 64)
        if self.pick == "zipf":
            w = np.arange(1, P + 1, dtype=np.float64) ** (-float(self.extra.get("zipf_s", 1.1)))
            cdf = np.cumsum(w) / np.sum(w)
        else:
            cdf = np.arange(1, P + 1, dtype=np.float64) / P
        out, k = [], 0
        for _ in range(B):
            ids: List[int] = []
            while len(ids) < n:
                c = int(np.searchsorted(cdf, u[k], side="right"))
                k += 1
                c = min(c, P - 1)
                if c not in ids:        # distinct ids per request (top-K retrieval)
                    ids.append(c)
            out.append(ids)
        return out


def workload(name: str) -> Workload:
    """The five benchmark configurations (BASELINE configs 1-5, 0-based names cfg1..cfg5)."""
    if name == "cfg1":
        return Workload(name, 1, 8, 2, 64, 1, 128, 2, 2, 16, 8, seed=0)
    if name == "cfg2":
        return Workload(name, 32, 32, 8, 128, 1, 1024, 5, 5, 64, 128, seed=1)
    if name == "cfg3":
        return Workload(name, 32, 32, 8, 128, 16, 1024, 10, 256, 32, 256, seed=2, pick="zipf",
                        extra={"zipf_s": 1.1})
    if name == "cfg4":
        return Workload(name, 80, 64, 8, 128, 4, 2048, 32, 128, 128, 64, seed=3)
    if name == "cfg5":
        return Workload(name, 32, 32, 8, 128, 8, 1024, 10, 296, 32, 128, seed=4, pick="uniform",
                        n_batches=64)
    raise KeyError(name)


def chunk_blob(w: Workload, chunk_index: int, n_tokens: int | None = None, shift: int = 0) -> np.ndarray:
    """One materialised chunk, layout [L][2 (K,V)][Hkv][n_tokens][D], as uint16 bf16 bits."""
    t = w.chunk_tokens if n_tokens is None else n_tokens
    n = w.n_layers * 2 * w.n_kv_heads * t * w.head_dim
    return normal_bf16(w.seed, STREAM_CHUNK + chunk_index, n, shift).reshape(
        w.n_layers, 2, w.n_kv_heads, t, w.head_dim)


def chunk_blob_layers(w: Workload, chunk_index: int, n_layers: int) -> np.ndarray:
    """The first `n_layers` layers of one materialised chunk, [n_layers][2][Hkv][chunk_tokens][D] (a prefix of
    the chunk's counter stream, so it equals chunk_blob(...)[:n_layers] without generating the rest)."""
    n = n_layers * 2 * w.n_kv_heads * w.chunk_tokens * w.head_dim
    return normal_bf16(w.seed, STREAM_CHUNK + chunk_index, n).reshape(n_layers, 2, w.n_kv_heads, w.chunk_tokens, w.head_dim)


def prefill_inputs(w: Workload, layer: int, q_shift: int = 0):
    """(q [B,S,Hq,D], k_new [B,S,Hkv,D], v_new [B,S,Hkv,D]) bf16 bits for one layer."""
    B, S, Hq, Hkv, D = w.batch, w.suffix, w.n_q_heads, w.n_kv_heads, w.head_dim
    nq, nk = B * S * Hq * D, B * S * Hkv * D
    q = normal_bf16(w.seed, STREAM_Q_PREFILL, nq, q_shift, start=layer * nq).reshape(B, S, Hq, D)
    k = normal_bf16(w.seed, STREAM_K_PREFILL, nk, 0, start=layer * nk).reshape(B, S, Hkv, D)
    v = normal_bf16(w.seed, STREAM_V_PREFILL, nk, 0, start=layer * nk).reshape(B, S, Hkv, D)
    return q, k, v


def decode_inputs(w: Workload, step: int, q_shift: int = 0):
    """(q [L,B,Hq,D], k_new [L,B,Hkv,D], v_new [L,B,Hkv,D]) bf16 bits for one decode step."""
    L, B, Hq, Hkv, D = w.n_layers, w.batch, w.n_q_heads, w.n_kv_heads, w.head_dim
    nq, nk = L * B * Hq * D, L * B * Hkv * D
    q = normal_bf16(w.seed, STREAM_Q_DECODE, nq, q_shift, start=step * nq).reshape(L, B, Hq, D)
    k = normal_bf16(w.seed, STREAM_K_DECODE, nk, 0, start=step * nk).reshape(L, B, Hkv, D)
    v = normal_bf16(w.seed, STREAM_V_DECODE, nk, 0, start=step * nk).reshape(L, B, Hkv, D)
    return q, k, v
