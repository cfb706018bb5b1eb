"""Pipelined serving of sequential request batches (the paper's overlap of the next batch's KV load with the
current batch's decode, Section III-C), as a sequence of C-ABI calls on two CUDA streams.

Batch n's chunks are staged from the host (pinned memory or chunk files) into slot region n mod R on the copy
stream; its table is built on the compute stream, which makes that stream wait for the copies; batch n+1 is
staged right after table n has been built, so its copies run under batch n's sub-prefill and decode.  Freeing
table n (done when table n+1 is built) marks the end of its region's use, and a later staging call into that
region waits for that mark on the copy stream.  Nothing here blocks the host and nothing is computed in Python.
"""
from __future__ import annotations

from typing import Callable, Optional, Sequence

import torch

from . import binding as mk
from .harness import Session


class PipelinedBatches:
    def __init__(self, sess: Session, n_slots: int, slot_bytes: int, stream: torch.cuda.Stream, copy: torch.cuda.Stream,
                 n_regions: int = 2):
        self.sess, self.slot_bytes, self.stream, self.copy = sess, slot_bytes, stream, copy
        self.slots = [torch.empty(n_slots * slot_bytes, dtype=torch.uint8, device=sess.dev) for _ in range(n_regions)]

    def stage(self, n: int, needed: Sequence[int]) -> int:
        """Batch n's distinct chunk ids into region n mod R, on the copy stream; returns the staging ticket."""
        return self.sess.stage(needed, self.slots[n % len(self.slots)], self.slot_bytes, self.copy)

    def compute(self, n: int, ids: Sequence[Sequence[int]], S: int, T: int, q_pf, k_pf, v_pf, o_pf, q_dc, k_dc, v_dc, o_dc,
                stage_next: Optional[Sequence[int]] = None, after_decode: Optional[Callable[[int], None]] = None) -> int:
        """Table, sub-prefill of all layers and T decode steps (all layers per launch) of batch n on the compute stream.
        q_pf [L,B,S,Hq,D] ... o_dc [T,L,B,Hq,D] are device tensors.  `stage_next`: the next batch's chunk ids, staged as
        soon as this batch's table exists.  `after_decode(table)` runs before the table can be freed."""
        sess, sp, ctx = self.sess, self.stream.cuda_stream, self.sess.ctx
        table = sess.build_table(ids, sp)      # frees the previous table on the stream: its region may be overwritten after that
        if stage_next is not None:
            self.stage(n + 1, stage_next)
        mk.matkv_attend_prefill_all_layers(ctx, table, S, q_pf.data_ptr(), k_pf.data_ptr(), v_pf.data_ptr(), o_pf.data_ptr(), None, sp)
        mk.matkv_table_advance(table, S, sp)
        qd_t, kd_t = q_dc[0].numel() * 2, k_dc[0].numel() * 2
        for t in range(T):
            mk.matkv_attend_decode_all_layers(ctx, table, q_dc.data_ptr() + t * qd_t, k_dc.data_ptr() + t * kd_t,
                                              v_dc.data_ptr() + t * kd_t, o_dc.data_ptr() + t * qd_t, None, sp)
            mk.matkv_table_advance(table, 1, sp)
        if after_decode is not None:
            after_decode(table)
        return table
