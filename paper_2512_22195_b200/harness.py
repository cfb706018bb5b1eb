"""Device-memory and stream plumbing around the C-ABI binding (torch is used for nothing else).

``Session`` owns the context, the workspace, the tails and the chunk buffers as torch tensors and
forwards every call to the library; no attention arithmetic happens in Python.
"""
from __future__ import annotations

from typing import Dict, List, Optional, Sequence

import numpy as np
import torch

from . import binding as mk


def bits_to_dev(a: np.ndarray, device="cuda") -> torch.Tensor:
    """uint16 bf16 bit patterns -> CUDA bf16 tensor with the same bytes."""
    a = np.ascontiguousarray(a)
    assert a.dtype == np.uint16
    return torch.from_numpy(a.view(np.int16)).to(device).view(torch.bfloat16)


def dev_to_bits(t: torch.Tensor) -> np.ndarray:
    """CUDA/CPU bf16 tensor -> uint16 bit patterns (numpy)."""
    return t.detach().contiguous().view(torch.int16).cpu().numpy().view(np.uint16)


class Session:
    def __init__(self, n_layers: int, n_q_heads: int, n_kv_heads: int, head_dim: int, max_batch: int,
                 max_chunks_per_req: int, max_tail_tokens: int, softmax_scale: float = 0.0, rope_theta: float = 0.0,
                 pos_mode: int = 0, device: int = 0):
        self.L, self.Hq, self.Hkv, self.D = n_layers, n_q_heads, n_kv_heads, head_dim
        self.max_batch, self.max_tail = max_batch, max_tail_tokens
        self.dev = torch.device("cuda", device)
        torch.cuda.set_device(self.dev)
        self.ctx = mk.matkv_create(n_layers, n_q_heads, n_kv_heads, head_dim, max_batch, max_chunks_per_req,
                                   max_tail_tokens, softmax_scale, rope_theta, pos_mode, device)
        nbytes = mk.matkv_workspace_bytes(self.ctx)
        self.workspace = torch.empty(nbytes, dtype=torch.uint8, device=self.dev)
        mk.matkv_set_workspace(self.ctx, self.workspace.data_ptr(), nbytes)
        shape = (max_batch, n_layers, n_kv_heads, max_tail_tokens, head_dim)
        self.tail_k = torch.zeros(shape, dtype=torch.bfloat16, device=self.dev)
        self.tail_v = torch.zeros(shape, dtype=torch.bfloat16, device=self.dev)
        self.chunks: Dict[int, torch.Tensor] = {}
        self.host_chunks: Dict[int, torch.Tensor] = {}
        self.table: Optional[int] = None
        self.batch = 0

    # -- chunks -------------------------------------------------------------------------------
    def register_device_chunk(self, chunk_id: int, blob) -> torch.Tensor:
        """blob: numpy uint16 [L,2,Hkv,n,D] or a CUDA bf16 tensor of that shape (kept alive here)."""
        t = bits_to_dev(blob, self.dev) if isinstance(blob, np.ndarray) else blob
        assert t.shape[0] == self.L and t.shape[1] == 2 and t.shape[2] == self.Hkv and t.shape[4] == self.D
        mk.matkv_register_chunk(self.ctx, chunk_id, t.shape[3], None, t.data_ptr())
        self.chunks[chunk_id] = t
        return t

    def register_host_chunk(self, chunk_id: int, blob) -> torch.Tensor:
        """blob: numpy uint16 or CPU bf16 tensor; copied into pinned host memory kept alive here."""
        src = torch.from_numpy(np.ascontiguousarray(blob).view(np.int16)).view(torch.bfloat16) \
            if isinstance(blob, np.ndarray) else blob
        t = torch.empty(src.shape, dtype=torch.bfloat16, pin_memory=True)
        t.copy_(src)
        mk.matkv_register_chunk(self.ctx, chunk_id, t.shape[3], t.data_ptr(), None)
        self.host_chunks[chunk_id] = t
        return t

    def stage(self, chunk_ids: Sequence[int], slots: torch.Tensor, slot_bytes: int, copy_stream: torch.cuda.Stream) -> int:
        n_slots = slots.numel() * slots.element_size() // slot_bytes
        return mk.matkv_stage_chunks_async(self.ctx, list(chunk_ids), slots.data_ptr(), slot_bytes, n_slots,
                                           copy_stream.cuda_stream)

    # -- table ----------------------------------------------------------------------------------
    def build_table(self, ids_per_req: Sequence[Sequence[int]], stream: int = 0) -> int:
        if self.table is not None:
            mk.matkv_table_free(self.table, stream)
        self.batch = len(ids_per_req)
        self.table = mk.matkv_build_chunk_table(self.ctx, ids_per_req, self.tail_k.data_ptr(), self.tail_v.data_ptr(),
                                                stream)
        # room for the chunk-major decode's partials (all layers in one launch) when this table needs more
        need = mk.matkv_table_workspace_bytes(self.table, self.L)
        if need > self.workspace.numel():
            self.workspace = torch.empty(need, dtype=torch.uint8, device=self.dev)
            mk.matkv_set_workspace(self.ctx, self.workspace.data_ptr(), need)
        return self.table

    def advance(self, n: int, stream: int = 0) -> None:
        mk.matkv_table_advance(self.table, n, stream)

    # -- attention --------------------------------------------------------------------------------
    def prefill(self, layer: int, q: torch.Tensor, k_new: torch.Tensor, v_new: torch.Tensor, want_lse=True, stream: int = 0):
        B, S = q.shape[0], q.shape[1]
        out = torch.empty_like(q)
        lse = torch.empty((B, S, self.Hq), dtype=torch.float32, device=self.dev) if want_lse else None
        mk.matkv_attend_prefill(self.ctx, self.table, layer, S, q.data_ptr(), k_new.data_ptr(), v_new.data_ptr(),
                                out.data_ptr(), lse.data_ptr() if want_lse else None, stream)
        return out, lse

    def prefill_all_layers(self, q: torch.Tensor, k_new: torch.Tensor, v_new: torch.Tensor, want_lse=True, stream: int = 0):
        L, B, S = q.shape[0], q.shape[1], q.shape[2]
        out = torch.empty_like(q)
        lse = torch.empty((L, B, S, self.Hq), dtype=torch.float32, device=self.dev) if want_lse else None
        mk.matkv_attend_prefill_all_layers(self.ctx, self.table, S, q.data_ptr(), k_new.data_ptr(), v_new.data_ptr(),
                                           out.data_ptr(), lse.data_ptr() if want_lse else None, stream)
        return out, lse

    def decode(self, layer: int, q: torch.Tensor, k_new: torch.Tensor, v_new: torch.Tensor, want_lse=True, stream: int = 0):
        out = torch.empty_like(q)
        lse = torch.empty((q.shape[0], self.Hq), dtype=torch.float32, device=self.dev) if want_lse else None
        mk.matkv_attend_decode(self.ctx, self.table, layer, q.data_ptr(), k_new.data_ptr(), v_new.data_ptr(),
                               out.data_ptr(), lse.data_ptr() if want_lse else None, stream)
        return out, lse

    def decode_all_layers(self, q: torch.Tensor, k_new: torch.Tensor, v_new: torch.Tensor, want_lse=True, stream: int = 0):
        out = torch.empty_like(q)
        lse = torch.empty((self.L, q.shape[1], self.Hq), dtype=torch.float32, device=self.dev) if want_lse else None
        mk.matkv_attend_decode_all_layers(self.ctx, self.table, q.data_ptr(), k_new.data_ptr(), v_new.data_ptr(),
                                          out.data_ptr(), lse.data_ptr() if want_lse else None, stream)
        return out, lse

    def gather(self, layer: int, req: int, rows: int):
        k = torch.empty((self.Hkv, rows, self.D), dtype=torch.bfloat16, device=self.dev)
        v = torch.empty_like(k)
        n = mk.matkv_gather_debug(self.ctx, self.table, layer, req, k.data_ptr(), v.data_ptr(), rows)
        assert n == rows, (n, rows)
        return k, v

    def status(self, clear: bool = False) -> int:
        return mk.matkv_status(self.ctx, clear)

    def close(self) -> None:
        if self.ctx:
            torch.cuda.synchronize(self.dev)
            mk.matkv_destroy(self.ctx)
            self.ctx, self.table = 0, None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass
