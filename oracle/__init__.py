"""CPU oracle of the MatKV attention path -- TEST INFRASTRUCTURE, not product code.

Thin ctypes access to ``matkv_oracle.c`` (plain fp64 C) plus the bookkeeping of
one request's tail (query-suffix and generated tokens).  Only ``tests/``, the
smoke check and the benchmark's CPU-baseline / reference legs may import this
package; the CUDA library and its Python binding never do, and nothing here
imports them.

Semantics (paper, Section III-B and Section IV): the materialised chunks sit
before the query, all of their tokens are visible, their K is used verbatim
(each chunk was computed with its tokens at positions 0..len-1), and the query
suffix and generated tokens form an ordinary causal continuation.

Pins: see ``tests/test_oracle_pins.py`` (three evaluators against each other,
textbook causal attention through a library routine, closed forms, planted
needles, permutation and duplication invariants, rotary shift invariance).
Parity unpinned: the position base of the query tokens in rotary mode against
the authors' own code, which is not available; it is a parameter here and is
inert in every timed configuration.
"""
from __future__ import annotations

import ctypes as C
import os
import subprocess
from typing import List, Sequence

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "matkv_oracle.c")
_SO = os.path.join(_HERE, "libmatkv_oracle.so")
_lib = None


def build(force: bool = False) -> str:
    """Compile the oracle with gcc (no CUDA involved)."""
    if force or not os.path.exists(_SO) or os.path.getmtime(_SO) < os.path.getmtime(_SRC):
        subprocess.check_call(["gcc", "-O2", "-std=c11", "-fPIC", "-shared", "-o", _SO, _SRC, "-lm"])
    return _SO


class _Shape(C.Structure):
    _fields_ = [("n_layers", C.c_int32), ("n_q_heads", C.c_int32), ("n_kv_heads", C.c_int32),
                ("head_dim", C.c_int32), ("scale", C.c_double)]


def _load():
    global _lib
    if _lib is None:
        lib = C.CDLL(build())
        pp = C.POINTER(C.c_void_p)
        for name in ("matkv_oracle_attend_walk", "matkv_oracle_attend_brute", "matkv_oracle_attend_merge"):
            f = getattr(lib, name)
            f.restype = C.c_int
            f.argtypes = [C.POINTER(_Shape), C.c_int32, C.c_int32, pp, C.c_void_p, C.c_void_p, C.c_void_p,
                          C.c_int32, C.c_int32, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p]
        lib.matkv_oracle_lse_merge.restype = None
        lib.matkv_oracle_lse_merge.argtypes = [C.c_int32, C.c_int32, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p]
        lib.matkv_oracle_rope.restype = None
        lib.matkv_oracle_rope.argtypes = [C.c_int32, C.c_int32, C.c_double, C.c_void_p, C.c_void_p, C.c_void_p]
        lib.matkv_oracle_e4m3_value.restype = C.c_double
        lib.matkv_oracle_e4m3_value.argtypes = [C.c_uint8]
        lib.matkv_oracle_e4m3_encode.restype = C.c_uint8
        lib.matkv_oracle_e4m3_encode.argtypes = [C.c_double]
        lib.matkv_oracle_fp8_block_exponent.restype = C.c_int32
        lib.matkv_oracle_fp8_block_exponent.argtypes = [C.c_double]
        for name in ("matkv_oracle_fp8_quantize_blob", "matkv_oracle_fp8_dequantize_blob"):
            f = getattr(lib, name)
            f.restype = None
            f.argtypes = [C.POINTER(_Shape), C.c_int32, C.c_void_p, C.c_void_p, C.c_void_p]
        _lib = lib
    return _lib


def _u16(a) -> np.ndarray:
    a = np.ascontiguousarray(a)
    assert a.dtype == np.uint16, a.dtype
    return a


class Shape:
    def __init__(self, n_layers: int, n_q_heads: int, n_kv_heads: int, head_dim: int, scale: float | None = None):
        assert n_q_heads % n_kv_heads == 0
        self.n_layers, self.n_q_heads, self.n_kv_heads, self.head_dim = n_layers, n_q_heads, n_kv_heads, head_dim
        self.scale = float(scale) if scale else 1.0 / float(np.sqrt(head_dim))

    def c(self) -> _Shape:
        return _Shape(self.n_layers, self.n_q_heads, self.n_kv_heads, self.head_dim, self.scale)


def attend(shape: Shape, layer: int, chunks: Sequence[np.ndarray], tail_k: np.ndarray, tail_v: np.ndarray,
           q: np.ndarray, visible: Sequence[int], evaluator: str = "walk"):
    """Attention of query rows ``q`` [n_q, Hq, D] over ``chunks`` (blobs [L,2,Hkv,len,D]) and
    the first ``visible[i]`` rows of the tail ([Hkv, cap, D] for this request and layer).
    Returns (o [n_q,Hq,D] float64, lse [n_q,Hq] float64)."""
    lib = _load()
    Hq, Hkv, D = shape.n_q_heads, shape.n_kv_heads, shape.head_dim
    q = _u16(q)
    n_q = q.shape[0]
    assert q.shape == (n_q, Hq, D)
    chunks = [_u16(c) for c in chunks]
    for c in chunks:
        assert c.shape[0] == shape.n_layers and c.shape[1] == 2 and c.shape[2] == Hkv and c.shape[4] == D, c.shape
    tail_k, tail_v = _u16(tail_k), _u16(tail_v)
    cap = tail_k.shape[1]
    assert tail_k.shape == (Hkv, cap, D) and tail_v.shape == (Hkv, cap, D)
    vis = np.ascontiguousarray(visible, dtype=np.int32)
    assert vis.shape == (n_q,)
    n_seg = len(chunks)
    ptrs = (C.c_void_p * max(n_seg, 1))(*[c.ctypes.data for c in chunks])
    lens = np.ascontiguousarray([c.shape[3] for c in chunks], dtype=np.int32)
    o = np.empty((n_q, Hq, D), dtype=np.float64)
    lse = np.empty((n_q, Hq), dtype=np.float64)
    fn = {"walk": lib.matkv_oracle_attend_walk, "brute": lib.matkv_oracle_attend_brute,
          "merge": lib.matkv_oracle_attend_merge}[evaluator]
    sh = shape.c()
    rc = fn(C.byref(sh), layer, n_seg, ptrs, lens.ctypes.data, tail_k.ctypes.data, tail_v.ctypes.data, cap,
            n_q, q.ctypes.data, vis.ctypes.data, o.ctypes.data, lse.ctypes.data)
    if rc != 0:
        raise RuntimeError(f"oracle evaluator {evaluator} failed: {rc}")
    return o, lse


def lse_merge(o_parts: np.ndarray, lse_parts: np.ndarray):
    """Merge partial attentions: o_parts [n, D], lse_parts [n] -> (o [D], lse)."""
    lib = _load()
    o_parts = np.ascontiguousarray(o_parts, dtype=np.float64)
    lse_parts = np.ascontiguousarray(lse_parts, dtype=np.float64)
    n, D = o_parts.shape
    o = np.empty(D, dtype=np.float64)
    lse = np.empty(1, dtype=np.float64)
    lib.matkv_oracle_lse_merge(n, D, o_parts.ctypes.data, lse_parts.ctypes.data, o.ctypes.data, lse.ctypes.data)
    return o, float(lse[0])


def rope(x: np.ndarray, pos: Sequence[int], theta: float) -> np.ndarray:
    """Rotate bf16 vectors x [n, D] at integer positions pos [n] (rotate-half pairing)."""
    lib = _load()
    x = _u16(x)
    n, D = x.shape
    p = np.ascontiguousarray(pos, dtype=np.int64)
    assert p.shape == (n,)
    out = np.empty_like(x)
    lib.matkv_oracle_rope(n, D, float(theta), p.ctypes.data, x.ctypes.data, out.ctypes.data)
    return out


def e4m3_value(code: int) -> float:
    return float(_load().matkv_oracle_e4m3_value(int(code)))


def e4m3_encode(x: float) -> int:
    return int(_load().matkv_oracle_e4m3_encode(float(x)))


def fp8_block_exponent(amax: float) -> int:
    return int(_load().matkv_oracle_fp8_block_exponent(float(amax)))


def fp8_quantize_blob(shape: "Shape", blob: np.ndarray):
    """bf16 chunk blob [L, 2, Hkv, len, D] -> (e4m3 codes, same shape, uint8; exponents [L, 2, Hkv, ceil(len/64)] int8)."""
    blob = _u16(blob)
    L, two, Hkv, n, D = blob.shape
    assert (L, two, Hkv, D) == (shape.n_layers, 2, shape.n_kv_heads, shape.head_dim)
    codes = np.empty(blob.shape, dtype=np.uint8)
    exps = np.empty((L, 2, Hkv, (n + 63) // 64), dtype=np.int8)
    sh = shape.c()
    _load().matkv_oracle_fp8_quantize_blob(C.byref(sh), n, blob.ctypes.data, codes.ctypes.data, exps.ctypes.data)
    return codes, exps


def fp8_dequantize_blob(shape: "Shape", codes: np.ndarray, exps: np.ndarray) -> np.ndarray:
    """The bf16 blob a compressed chunk stands for (exact: every value(code) * 2^e is a bf16 number)."""
    codes = np.ascontiguousarray(codes, dtype=np.uint8)
    exps = np.ascontiguousarray(exps, dtype=np.int8)
    out = np.empty(codes.shape, dtype=np.uint16)
    sh = shape.c()
    _load().matkv_oracle_fp8_dequantize_blob(C.byref(sh), codes.shape[3], codes.ctypes.data, exps.ctypes.data, out.ctypes.data)
    return out


class Request:
    """One request: an ordered list of materialised chunks and a tail that grows with the
    query suffix (prefill) and the generated tokens (decode)."""

    def __init__(self, shape: Shape, chunks: List[np.ndarray], tail_cap: int, rope_theta: float = 0.0,
                 pos_base: int | None = None):
        self.shape, self.chunks, self.cap = shape, [_u16(c) for c in chunks], tail_cap
        L, Hkv, D = shape.n_layers, shape.n_kv_heads, shape.head_dim
        self.tail_k = np.zeros((L, Hkv, tail_cap, D), dtype=np.uint16)
        self.tail_v = np.zeros((L, Hkv, tail_cap, D), dtype=np.uint16)
        self.tail_len = 0
        self.theta = rope_theta
        # the query continues after the chunks: its first token sits at sum of chunk lengths
        self.pos_base = sum(c.shape[3] for c in self.chunks) if pos_base is None else pos_base

    def _rot(self, x: np.ndarray, first_pos: int) -> np.ndarray:
        """x [n, H, D]: rotate row i of every head at position first_pos + i."""
        if self.theta == 0.0:
            return _u16(x)
        n, H, D = x.shape
        pos = np.repeat(np.arange(first_pos, first_pos + n, dtype=np.int64), H)
        return rope(_u16(x).reshape(n * H, D), pos, self.theta).reshape(n, H, D)

    def attend_new(self, layer: int, q: np.ndarray, k_new: np.ndarray, v_new: np.ndarray, evaluator: str = "walk"):
        """Append n new tokens (k_new, v_new [n,Hkv,D]) at tail[tail_len..) of ``layer`` and attend
        with q [n,Hq,D]: row i sees all chunks and tail[0 .. tail_len+i].  n = S for the query
        sub-prefill, n = 1 for a decode step.  ``tail_len`` moves only through advance()."""
        n = q.shape[0]
        t0 = self.tail_len
        assert t0 + n <= self.cap
        p0 = self.pos_base + t0
        qr, kr = self._rot(q, p0), self._rot(k_new, p0)
        self.tail_k[layer, :, t0:t0 + n, :] = np.transpose(kr, (1, 0, 2))
        self.tail_v[layer, :, t0:t0 + n, :] = np.transpose(_u16(v_new), (1, 0, 2))
        vis = [t0 + i + 1 for i in range(n)]
        return attend(self.shape, layer, self.chunks, self.tail_k[layer], self.tail_v[layer], qr, vis, evaluator)

    def append_only(self, layer: int, k_new: np.ndarray, v_new: np.ndarray) -> None:
        """Write n new tokens at tail[tail_len..) of ``layer`` without attending (bookkeeping only)."""
        n = k_new.shape[0]
        t0 = self.tail_len
        assert t0 + n <= self.cap
        kr = self._rot(k_new, self.pos_base + t0)
        self.tail_k[layer, :, t0:t0 + n, :] = np.transpose(kr, (1, 0, 2))
        self.tail_v[layer, :, t0:t0 + n, :] = np.transpose(_u16(v_new), (1, 0, 2))

    def advance(self, n: int) -> None:
        self.tail_len += n
