"""ctypes binding of libmatkv.so: the same names as the C ABI, argument marshalling only.

Every step of the attention path runs inside the library's CUDA kernels.  There is no
fallback: if the shared library is missing or an entry point fails, an exception is raised.
Device buffers are passed as integer addresses (``tensor.data_ptr()``), streams as
``torch.cuda.Stream.cuda_stream`` integers (0 = legacy default stream).
"""
from __future__ import annotations

import ctypes as C
import os
from typing import Optional, Sequence

HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(HERE, "libmatkv.so")

OK, E_INVALID_ARG, E_UNKNOWN_CHUNK, E_NOT_STAGED, E_NOT_READY = 0, -1, -2, -3, -4
E_CAPACITY, E_ALIGNMENT, E_CUDA, E_TIMEOUT, E_BOUNDS, E_IO = -5, -6, -7, -8, -9, -10
OPT_DECODE_CTAS, OPT_PREFILL_IMPL, OPT_PREFILL_CTAS, OPT_STAGE_CTAS, OPT_DECODE_ADVANCES_TAIL = 1, 2, 3, 4, 5
OPT_DECODE_IMPL, OPT_SHARE_TILES, OPT_FP8_RESIDENT, OPT_IO_TIMEOUT_MS, OPT_IO_TEST_DELAY_MS, OPT_CLUSTER_DECODE, OPT_CLUSTER_MAX = 6, 7, 8, 9, 10, 11, 12

EXPORTS = [
    "matkv_create", "matkv_destroy", "matkv_last_error", "matkv_set_option", "matkv_workspace_bytes",
    "matkv_set_workspace", "matkv_status", "matkv_register_chunk", "matkv_unregister_chunk",
    "matkv_stage_chunks_async", "matkv_stage_query", "matkv_stage_wait", "matkv_build_chunk_table",
    "matkv_table_free", "matkv_table_advance", "matkv_table_set_tail_len", "matkv_attend_prefill",
    "matkv_attend_decode", "matkv_attend_decode_all_layers", "matkv_lse_combine", "matkv_gather_debug",
    "matkv_probe_read", "matkv_attend_decode_static", "matkv_selftest_wait_timeout",
    "matkv_register_chunk_file", "matkv_set_bounce_buffer", "matkv_export_tail_as_chunk",
    "matkv_attend_prefill_all_layers", "matkv_table_sharing", "matkv_table_workspace_bytes",
    "matkv_fp8_blob_bytes", "matkv_fp8_resident_bytes", "matkv_quantize_chunk_fp8", "matkv_register_chunk_fp8", "matkv_register_chunk_file_fp8",
    "matkv_table_set_pos_base", "matkv_stage_pending",
]


class MatkvError(RuntimeError):
    def __init__(self, code: int, msg: str):
        super().__init__(f"matkv error {code}: {msg}")
        self.code = code


class matkv_config(C.Structure):
    _fields_ = [("n_layers", C.c_int32), ("n_q_heads", C.c_int32), ("n_kv_heads", C.c_int32),
                ("head_dim", C.c_int32), ("max_batch", C.c_int32), ("max_chunks_per_req", C.c_int32),
                ("max_tail_tokens", C.c_int32), ("softmax_scale", C.c_float), ("rope_theta", C.c_float),
                ("pos_mode", C.c_int32), ("device", C.c_int32)]


_lib = None


def lib() -> C.CDLL:
    """The loaded shared library; raises if it has not been built."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise ImportError(f"{LIB_PATH} is missing: build it with `python -m paper_2512_22195_b200.build` "
                              "(there is no non-CUDA fallback)")
        L = C.CDLL(LIB_PATH)
        vp, i32, i64, u64 = C.c_void_p, C.c_int32, C.c_int64, C.c_uint64
        sig = {
            "matkv_create": (C.c_int, [C.POINTER(matkv_config), C.POINTER(vp)]),
            "matkv_destroy": (C.c_int, [vp]),
            "matkv_last_error": (C.c_char_p, []),
            "matkv_set_option": (C.c_int, [vp, i32, i64]),
            "matkv_workspace_bytes": (C.c_size_t, [vp]),
            "matkv_set_workspace": (C.c_int, [vp, vp, C.c_size_t]),
            "matkv_status": (C.c_int, [vp, C.POINTER(i32), i32]),
            "matkv_register_chunk": (C.c_int, [vp, u64, i32, vp, vp]),
            "matkv_unregister_chunk": (C.c_int, [vp, u64]),
            "matkv_stage_chunks_async": (C.c_int, [vp, C.POINTER(u64), i32, vp, C.c_size_t, i32, vp, C.POINTER(u64)]),
            "matkv_stage_query": (C.c_int, [vp, u64]),
            "matkv_stage_wait": (C.c_int, [vp, u64]),
            "matkv_build_chunk_table": (C.c_int, [vp, i32, C.POINTER(i32), C.POINTER(u64), vp, vp, vp, C.POINTER(vp)]),
            "matkv_table_free": (C.c_int, [vp, vp]),
            "matkv_table_advance": (C.c_int, [vp, i32, vp]),
            "matkv_table_set_tail_len": (C.c_int, [vp, i32, vp]),
            "matkv_table_set_pos_base": (C.c_int, [vp, C.POINTER(i32), vp]),
            "matkv_stage_pending": (C.c_int, [vp, C.POINTER(i32)]),
            "matkv_attend_prefill": (C.c_int, [vp, vp, i32, i32, vp, vp, vp, vp, vp, vp]),
            "matkv_attend_decode": (C.c_int, [vp, vp, i32, vp, vp, vp, vp, vp, vp]),
            "matkv_attend_decode_all_layers": (C.c_int, [vp, vp, vp, vp, vp, vp, vp, vp]),
            "matkv_lse_combine": (C.c_int, [vp, i32, i32, i32, vp, vp, vp, vp, vp]),
            "matkv_gather_debug": (C.c_int, [vp, vp, i32, i32, vp, vp, i64, C.POINTER(i64), vp]),
            "matkv_probe_read": (C.c_int, [vp, vp, C.c_size_t, vp]),
            "matkv_attend_decode_static": (C.c_int, [vp, vp, i32, vp, vp, vp, vp, vp, vp]),
            "matkv_selftest_wait_timeout": (C.c_int, [vp, C.c_double, vp]),
            "matkv_register_chunk_file": (C.c_int, [vp, u64, i32, C.c_char_p, u64]),
            "matkv_set_bounce_buffer": (C.c_int, [vp, vp, C.c_size_t, C.c_size_t, i32]),
            "matkv_export_tail_as_chunk": (C.c_int, [vp, vp, i32, i32, vp, vp, vp]),
            "matkv_attend_prefill_all_layers": (C.c_int, [vp, vp, i32, vp, vp, vp, vp, vp, vp]),
            "matkv_table_sharing": (C.c_int, [vp, C.POINTER(i64), C.POINTER(i64)]),
            "matkv_table_workspace_bytes": (C.c_size_t, [vp, i32]),
            "matkv_fp8_blob_bytes": (C.c_size_t, [vp, i32]),
            "matkv_fp8_resident_bytes": (C.c_size_t, [vp, i32]),
            "matkv_quantize_chunk_fp8": (C.c_int, [vp, vp, i32, vp, vp]),
            "matkv_register_chunk_fp8": (C.c_int, [vp, u64, i32, vp]),
            "matkv_register_chunk_file_fp8": (C.c_int, [vp, u64, i32, C.c_char_p, u64]),
        }
        for name, (res, args) in sig.items():
            f = getattr(L, name)
            f.restype, f.argtypes = res, args
        _lib = L
    return _lib


def _check(rc: int) -> None:
    if rc != 0:
        raise MatkvError(rc, lib().matkv_last_error().decode("utf-8", "replace"))


def matkv_last_error() -> str:
    return lib().matkv_last_error().decode("utf-8", "replace")


def matkv_create(n_layers: int, n_q_heads: int, n_kv_heads: int, head_dim: int, max_batch: int,
                 max_chunks_per_req: int, max_tail_tokens: int, softmax_scale: float = 0.0,
                 rope_theta: float = 0.0, pos_mode: int = 0, device: int = -1) -> int:
    cfg = matkv_config(n_layers, n_q_heads, n_kv_heads, head_dim, max_batch, max_chunks_per_req,
                       max_tail_tokens, softmax_scale, rope_theta, pos_mode, device)
    out = C.c_void_p()
    _check(lib().matkv_create(C.byref(cfg), C.byref(out)))
    return out.value


def matkv_destroy(ctx: int) -> None:
    _check(lib().matkv_destroy(ctx))


def matkv_set_option(ctx: int, option: int, value: int) -> None:
    _check(lib().matkv_set_option(ctx, option, value))


def matkv_workspace_bytes(ctx: int) -> int:
    return int(lib().matkv_workspace_bytes(ctx))


def matkv_set_workspace(ctx: int, dev_ptr: int, nbytes: int) -> None:
    _check(lib().matkv_set_workspace(ctx, dev_ptr, nbytes))


def matkv_status(ctx: int, clear: bool = False) -> int:
    st = C.c_int32(0)
    _check(lib().matkv_status(ctx, C.byref(st), 1 if clear else 0))
    return st.value


def matkv_register_chunk(ctx: int, chunk_id: int, n_tokens: int, host_ptr: Optional[int], dev_ptr: Optional[int]) -> None:
    _check(lib().matkv_register_chunk(ctx, chunk_id, n_tokens, host_ptr or None, dev_ptr or None))


def matkv_unregister_chunk(ctx: int, chunk_id: int) -> None:
    _check(lib().matkv_unregister_chunk(ctx, chunk_id))


def matkv_stage_chunks_async(ctx: int, chunk_ids: Sequence[int], dev_slots: int, slot_bytes: int, n_slots: int,
                             copy_stream: int = 0) -> int:
    n = len(chunk_ids)
    arr = (C.c_uint64 * max(n, 1))(*chunk_ids)
    ticket = C.c_uint64(0)
    _check(lib().matkv_stage_chunks_async(ctx, arr, n, dev_slots, slot_bytes, n_slots, copy_stream or None,
                                          C.byref(ticket)))
    return ticket.value


def matkv_stage_query(ctx: int, ticket: int) -> bool:
    rc = lib().matkv_stage_query(ctx, ticket)
    if rc == E_NOT_READY:
        return False
    _check(rc)
    return True


def matkv_stage_wait(ctx: int, ticket: int) -> None:
    _check(lib().matkv_stage_wait(ctx, ticket))


def matkv_build_chunk_table(ctx: int, chunk_ids_per_req: Sequence[Sequence[int]], tail_k: int, tail_v: int,
                            stream: int = 0) -> int:
    B = len(chunk_ids_per_req)
    counts = (C.c_int32 * max(B, 1))(*[len(r) for r in chunk_ids_per_req])
    flat = [c for r in chunk_ids_per_req for c in r]
    ids = (C.c_uint64 * max(len(flat), 1))(*flat)
    out = C.c_void_p()
    _check(lib().matkv_build_chunk_table(ctx, B, counts, ids, tail_k, tail_v, stream or None, C.byref(out)))
    return out.value


def matkv_table_free(table: int, stream: int = 0) -> None:
    _check(lib().matkv_table_free(table, stream or None))


def matkv_table_advance(table: int, n_tokens: int, stream: int = 0) -> None:
    _check(lib().matkv_table_advance(table, n_tokens, stream or None))


def matkv_table_set_tail_len(table: int, tail_len: int, stream: int = 0) -> None:
    _check(lib().matkv_table_set_tail_len(table, tail_len, stream or None))


def matkv_attend_prefill(ctx: int, table: int, layer: int, S: int, q: int, k_new: int, v_new: int, out: int,
                         lse_out: Optional[int] = None, stream: int = 0) -> None:
    _check(lib().matkv_attend_prefill(ctx, table, layer, S, q, k_new, v_new, out, lse_out or None, stream or None))


def matkv_attend_decode(ctx: int, table: int, layer: int, q: int, k_new: int, v_new: int, out: int,
                        lse_out: Optional[int] = None, stream: int = 0) -> None:
    _check(lib().matkv_attend_decode(ctx, table, layer, q, k_new, v_new, out, lse_out or None, stream or None))


def matkv_attend_decode_all_layers(ctx: int, table: int, q: int, k_new: int, v_new: int, out: int,
                                   lse_out: Optional[int] = None, stream: int = 0) -> None:
    _check(lib().matkv_attend_decode_all_layers(ctx, table, q, k_new, v_new, out, lse_out or None, stream or None))


def matkv_lse_combine(ctx: int, n_rows: int, n_parts: int, D: int, o_parts: int, lse_parts: int, out: int,
                      lse_out: Optional[int] = None, stream: int = 0) -> None:
    _check(lib().matkv_lse_combine(ctx, n_rows, n_parts, D, o_parts, lse_parts, out, lse_out or None, stream or None))


def matkv_gather_debug(ctx: int, table: int, layer: int, req: int, k_out: int, v_out: int, capacity_rows: int,
                       stream: int = 0) -> int:
    rows = C.c_int64(0)
    _check(lib().matkv_gather_debug(ctx, table, layer, req, k_out, v_out, capacity_rows, C.byref(rows), stream or None))
    return rows.value


def matkv_probe_read(ctx: int, dev_ptr: int, nbytes: int, stream: int = 0) -> None:
    _check(lib().matkv_probe_read(ctx, dev_ptr, nbytes, stream or None))


def matkv_attend_decode_static(ctx: int, table: int, layer: int, q: int, k_new: int, v_new: int, out: int,
                               lse_out: Optional[int] = None, stream: int = 0) -> None:
    """matkv_attend_decode for callers that may not allocate or lend a workspace: the split-KV scratch is
    an array built into the library (batch x n_kv_heads <= 256).  First call per device: outside any
    stream capture.  Calls must not overlap on the GPU (they share the array)."""
    _check(lib().matkv_attend_decode_static(ctx, table, layer, q, k_new, v_new, out, lse_out or None, stream or None))


def matkv_selftest_wait_timeout(ctx: int, seconds: float = 0.2, stream: int = 0) -> None:
    _check(lib().matkv_selftest_wait_timeout(ctx, seconds, stream or None))


def matkv_register_chunk_file(ctx: int, chunk_id: int, n_tokens: int, path: str, file_offset: int = 0) -> None:
    _check(lib().matkv_register_chunk_file(ctx, chunk_id, n_tokens, path.encode(), file_offset))


def matkv_set_bounce_buffer(ctx: int, pinned_host_ptr: int, nbytes: int, slab_bytes: int, n_io_threads: int = 4) -> None:
    _check(lib().matkv_set_bounce_buffer(ctx, pinned_host_ptr, nbytes, slab_bytes, n_io_threads))


def matkv_export_tail_as_chunk(ctx: int, table: int, req: int, n_tokens: int, dev_blob: int, host_blob: Optional[int] = None,
                               stream: int = 0) -> None:
    _check(lib().matkv_export_tail_as_chunk(ctx, table, req, n_tokens, dev_blob, host_blob or None, stream or None))


def matkv_attend_prefill_all_layers(ctx: int, table: int, S: int, q: int, k_new: int, v_new: int, out: int,
                                    lse_out: Optional[int] = None, stream: int = 0) -> None:
    _check(lib().matkv_attend_prefill_all_layers(ctx, table, S, q, k_new, v_new, out, lse_out or None, stream or None))


def matkv_table_sharing(table: int):
    """(chunk tiles the table's requests list, chunk tiles the chunk-major decode reads) per layer and KV head."""
    a, b = C.c_int64(0), C.c_int64(0)
    _check(lib().matkv_table_sharing(table, C.byref(a), C.byref(b)))
    return a.value, b.value


def matkv_table_workspace_bytes(table: int, n_layers_launch: int) -> int:
    return int(lib().matkv_table_workspace_bytes(table, n_layers_launch))


def matkv_fp8_blob_bytes(ctx: int, n_tokens: int) -> int:
    return int(lib().matkv_fp8_blob_bytes(ctx, n_tokens))


def matkv_fp8_resident_bytes(ctx: int, n_tokens: int) -> int:
    return int(lib().matkv_fp8_resident_bytes(ctx, n_tokens))


def matkv_quantize_chunk_fp8(ctx: int, dev_blob: int, n_tokens: int, dev_blob_fp8: int, stream: int = 0) -> None:
    _check(lib().matkv_quantize_chunk_fp8(ctx, dev_blob, n_tokens, dev_blob_fp8, stream or None))


def matkv_register_chunk_fp8(ctx: int, chunk_id: int, n_tokens: int, host_blob_fp8: int) -> None:
    _check(lib().matkv_register_chunk_fp8(ctx, chunk_id, n_tokens, host_blob_fp8))


def matkv_register_chunk_file_fp8(ctx: int, chunk_id: int, n_tokens: int, path: str, file_offset: int = 0) -> None:
    _check(lib().matkv_register_chunk_file_fp8(ctx, chunk_id, n_tokens, path.encode(), file_offset))


def matkv_table_set_pos_base(table: int, pos_base: Sequence[int], stream: int = 0) -> None:
    """pos_mode 2: position of the first tail token of every request (one value per request of the table)."""
    arr = (C.c_int32 * max(len(pos_base), 1))(*pos_base)
    _check(lib().matkv_table_set_pos_base(table, arr, stream or None))


def matkv_stage_pending(ctx: int) -> int:
    """Staging calls not yet seen complete."""
    n = C.c_int32(0)
    _check(lib().matkv_stage_pending(ctx, C.byref(n)))
    return n.value
