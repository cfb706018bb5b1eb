#!/usr/bin/env python
"""Benchmark of the attention path over materialised KV chunks (one JSON line on stdout).

A "step" is one pass of the whole hot path for one request batch: build the chunk table, run the
query sub-prefill for every layer, then T decode steps over every layer (split-KV partials merged
by log-sum-exp inside the same launches).  `value` is decode tokens per second of that whole step
with every input already resident in HBM; `e2e` repeats it through the same C-ABI calls starting
from HOST buffers (chunk blobs staged from pinned host memory, q/k/v copied in per step, outputs
copied back).  The numbers are attention-path only (no model weights, no MLP).

With no --workload the headline configuration runs: config 4 (Llama-3-70B head shape, 80 layers, batch 4, 32 x 2,048-token
chunks per request = 64K tokens of context and 86 GB of KV in HBM), the largest configuration that fits one GPU; the lines
of configurations 2, 3 and 5 (each from a child process of its own once the headline has released the GPU's memory) are
attached under `other_workloads`.  --gpus N without a torchrun environment starts N ranks itself (independent replicas:
the only cross-rank traffic is the barrier and the max over ranks of the measured time).

  python bench.py [--gpus N] [--steps K] [--warmup W] [--workload cfg4] [--decode-launch all_layers|per_layer]
  python bench.py --impl reference ...      # the CPU oracle as it stands, on the host cores
"""
from __future__ import annotations

import argparse
import json
import os
import subprocess
import sys
import threading
import time
from concurrent.futures import ThreadPoolExecutor

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

import matkv_inputs as mi  # noqa: E402

NOMINAL_HBM_GBS = 8000.0
FALLBACK_HBM_GBS = 6650.0
FALLBACK_BF16_TFLOPS = 1590.0
HEADLINE = "cfg4"
# DRAM bytes (read + write) of ONE all-layers decode launch, from one ncu capture of the kernels as they are built now:
# (workload, launch mode) -> (bytes of the captured launch, layers of the captured case).  A capture of the full launch
# is used as it is; a capture of a few-layer case (the full workload is too large to capture) is scaled by the layer
# count, traffic being proportional to it.  None: not captured for this build, `traffic` is then null.
NCU_TRAFFIC = {("cfg2", "all_layers"): (688_347_008 + 1_927_168, 32),      # k_attend_stream<128,4>: all 32 layers captured
               ("cfg4", "all_layers"): (2_153_027_840 + 2_343_680, 2),       # k_attend_stream<128,8>: a 2-layer case (2.15 GB), scaled x 40
               ("cfg3", "all_layers"): (619_040_000 + 2_553_856, 2)}         # k_attend_shared<128,4>: a 2-layer case (0.7 GB), scaled x 16


def log(*a):
    print(*a, file=sys.stderr, flush=True)


def measured_peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        with open(p) as f:
            return json.load(f), "measured"
    return {"hbm_gbs": FALLBACK_HBM_GBS}, "fallback"


# ---- clocks ------------------------------------------------------------------------------------
class ClockSampler:
    Q = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
         "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.rows, self.proc = [], None
        try:
            self.proc = subprocess.Popen(["nvidia-smi", f"--id={index}", f"--query-gpu={self.Q}",
                                          "--format=csv,noheader,nounits", "-lms", "100"],
                                         stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.th = threading.Thread(target=self._read, daemon=True)
            self.th.start()
        except Exception:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.rows.append((time.time(), line.strip()))

    def stop(self, t0: float, t1: float):
        if not self.proc:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        time.sleep(0.15)
        self.proc.terminate()
        sm, mx, reasons = [], None, set()
        for ts, line in self.rows:
            f = [x.strip() for x in line.split(",")]
            if len(f) < 7 or not (t0 - 0.05 <= ts <= t1 + 0.15):
                continue
            try:
                sm.append(float(f[0]))
                mx = float(f[1])
            except ValueError:
                continue
            for name, v in zip(("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"), f[3:7]):
                if v.lower().startswith("active"):
                    reasons.add(name)
        return {"sm_mhz": float(np.median(sm)) if sm else None, "sm_max_mhz": mx, "reasons": sorted(reasons),
                "samples": len(sm)}


# ---- the CPU oracle legs -------------------------------------------------------------------------
class OracleState:
    """Host copies of one batch and the oracle's requests (used by cpu_baseline and --impl reference).
    `layers` selects a subset of the model's layers (the work is exactly linear in layers); the chunk
    blobs handed in hold only those layers, in that order."""

    def __init__(self, w: mi.Workload, host_chunks, ids, layers=None):
        import oracle
        self.oracle, self.w = oracle, w
        self.layers = list(range(w.n_layers)) if layers is None else list(layers)
        self.sh = oracle.Shape(len(self.layers), w.n_q_heads, w.n_kv_heads, w.head_dim)
        cap = w.suffix + w.decode_steps
        self.reqs = [oracle.Request(self.sh, [host_chunks[c] for c in row], cap) for row in ids]
        self.cores = os.cpu_count() or 1
        # the tail as it stands after the sub-prefill: appended without attending (bookkeeping only)
        for li, layer in enumerate(self.layers):
            _, k, v = mi.prefill_inputs(w, layer)
            for r, rq in enumerate(self.reqs):
                rq.append_only(li, k[r], v[r])
        for rq in self.reqs:
            rq.advance(w.suffix)

    def decode_steps(self, first_step: int, n_steps: int):
        """Time n_steps decode steps (the selected layers, all requests) on all host cores; returns seconds."""
        w = self.w
        t0 = time.perf_counter()
        with ThreadPoolExecutor(max_workers=self.cores) as ex:
            for s in range(first_step, first_step + n_steps):
                q, k, v = mi.decode_inputs(w, s)
                jobs = [(li, layer, r) for li, layer in enumerate(self.layers) for r in range(w.batch)]
                list(ex.map(lambda j: self.reqs[j[2]].attend_new(j[0], q[j[1], j[2]][None], k[j[1], j[2]][None],
                                                                 v[j[1], j[2]][None]), jobs))
                for rq in self.reqs:
                    rq.advance(1)
        return time.perf_counter() - t0

    def rewind(self, n_steps: int):
        for rq in self.reqs:
            rq.tail_len -= n_steps


def host_chunks_numpy(w: mi.Workload, needed):
    return {c: mi.chunk_blob(w, c) for c in needed}


def run_reference(args):
    """The reference arm: the CPU oracle, as it stands, on this machine's host cores."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    import oracle
    oracle.build()
    w = mi.workload(args.workload)
    ids = w.chunk_ids(0)
    needed = sorted({c for row in ids for c in row})
    log(f"[reference] generating {len(needed)} chunks on the host ...")
    # larger workloads: a few layers per step, enough (layer, request) units to keep every host thread busy (stated in `sample`)
    cores = os.cpu_count() or 1
    n_l = w.n_layers if w.name in ("cfg1", "cfg2") else max(1, min(w.n_layers, 4, -(-cores // w.batch)))
    with ThreadPoolExecutor(max_workers=cores) as ex:       # the generator is numpy: it releases the interpreter lock
        blobs = dict(zip(needed, ex.map(lambda c: mi.chunk_blob_layers(w, c, n_l), needed)))
    st = OracleState(w, blobs, ids, layers=list(range(n_l)))
    per_step = 1  # each bench step = one decode step of the workload over the sampled layers and all requests
    for _ in range(args.warmup):
        st.decode_steps(0, per_step)
        st.rewind(per_step)
    t = 0.0
    for _ in range(args.steps):
        t += st.decode_steps(0, per_step)
        st.rewind(per_step)
    tok_s = args.steps * per_step * w.batch / (t * w.n_layers / n_l)
    n_req = [len(row) * w.chunk_tokens for row in ids]
    config = workload_config(w, "all_layers", kv_bytes_of_decode(w, n_req) / w.decode_steps)
    sample = (f"decode step 0 of {w.name} ({n_l} of {w.n_layers} layers, batch {w.batch}), repeated per bench step"
              + ("" if n_l == w.n_layers else ", extrapolated linearly to all layers"))
    print(json.dumps({
        "impl": "reference", "metric": "decode_tokens_per_s", "value": tok_s, "unit": "tokens/s", "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1e3 * t / args.steps, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": config,
        "cpu_baseline": {"value": tok_s, "unit": "tokens/s", "cores": min(st.cores, n_l * w.batch), "kind": "oracle", "sample": sample},
        "e2e": {"value": tok_s, "unit": "tokens/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
    }), flush=True)


# ---- pipelined serving (config 5): staging of batch n+1 under the compute of batch n ------------------
def run_pipeline(args):
    """Sequential request batches whose chunks live in a pinned host pool.  Three passes over the same
    batches: staging alone, serial (stage, wait, compute), pipelined (batch n+1 staged on a side stream
    while batch n is prefilled and decoded).  Overlap efficiency = (t_serial - t_pipelined) / t_stage."""
    import torch
    import paper_2512_22195_b200 as mk
    import matkv_inputs.device as gen
    from paper_2512_22195_b200.harness import Session

    dev = torch.device("cuda", int(os.environ.get("LOCAL_RANK", "0")))
    torch.cuda.set_device(dev)
    w = mi.workload(args.workload)
    if args.layers:
        w.n_layers = args.layers
    if args.decode_steps:
        w.decode_steps = args.decode_steps
    if args.pool_chunks:
        w.pool_chunks = args.pool_chunks
    n_batches = args.batches or w.n_batches
    L, B, S, T, Hq, Hkv, D = w.n_layers, w.batch, w.suffix, w.decode_steps, w.n_q_heads, w.n_kv_heads, w.head_dim
    batches = [w.chunk_ids(i) for i in range(n_batches)]
    needed = [sorted({c for row in ids for c in row}) for ids in batches]
    n_slots = max(len(x) for x in needed)
    slot_bytes = w.chunk_bytes
    log(f"[pipeline] pinned pool: {w.pool_chunks} chunks x {slot_bytes / 1e6:.0f} MB = {w.pool_chunks * slot_bytes / 1e9:.1f} GB; "
        f"{n_batches} batches of {B} x {w.chunks_per_req} chunks; 2 x {n_slots} device slots")
    sess = Session(L, Hq, Hkv, D, B, w.chunks_per_req, S + T, device=dev.index)
    if args.stage_ctas < 0:
        args.stage_ctas = 16
    if args.stage_ctas:
        mk.matkv_set_option(sess.ctx, mk.OPT_STAGE_CTAS, args.stage_ctas)
    if args.decode_ctas:
        mk.matkv_set_option(sess.ctx, mk.OPT_DECODE_CTAS, args.decode_ctas)
    tmp = torch.empty((L, 2, Hkv, w.chunk_tokens, D), dtype=torch.bfloat16, device=dev)
    host_pool = ring = None
    fp8 = args.kv_store == "fp8"
    stored_bytes = mk.matkv_fp8_blob_bytes(sess.ctx, w.chunk_tokens) if fp8 else slot_bytes   # bytes of a chunk where it is kept
    tmp8 = torch.empty(stored_bytes, dtype=torch.uint8, device=dev) if fp8 else None

    def chunk_to(dst_u8, c):
        """Chunk c's stored form (generated on the device, compressed there if asked) into a pinned uint8 buffer."""
        gen.fill_bf16(tmp, w.seed, mi.STREAM_CHUNK + c)
        if fp8:
            mk.matkv_quantize_chunk_fp8(sess.ctx, tmp.data_ptr(), w.chunk_tokens, tmp8.data_ptr())
            dst_u8.copy_(tmp8)
        else:
            dst_u8.copy_(tmp.view(torch.uint8).reshape(-1))

    if args.store_dir:
        # the materialised-KV store: one raw-bytes file per chunk id
        os.makedirs(args.store_dir, exist_ok=True)
        bounce = torch.empty(stored_bytes, dtype=torch.uint8, pin_memory=True)
        t_w = time.perf_counter()
        for c in range(w.pool_chunks):
            path = os.path.join(args.store_dir, f"{c}.kv8" if fp8 else f"{c}.kv")
            if not (os.path.exists(path) and os.path.getsize(path) == stored_bytes):
                chunk_to(bounce, c)
                torch.cuda.synchronize()
                with open(path, "wb") as f:
                    f.write(memoryview(bounce.numpy()))
            if fp8:
                mk.matkv_register_chunk_file_fp8(sess.ctx, c, w.chunk_tokens, path, 0)
            else:
                mk.matkv_register_chunk_file(sess.ctx, c, w.chunk_tokens, path, 0)
        os.sync()
        log(f"[pipeline] store written/checked in {time.perf_counter() - t_w:.1f} s")
        n_slabs = 8
        slab = (stored_bytes + 4095) // 4096 * 4096
        ring = torch.empty(n_slabs * slab + 4096, dtype=torch.uint8, pin_memory=True)
        ring_base = (ring.data_ptr() + 4095) // 4096 * 4096
        mk.matkv_set_bounce_buffer(sess.ctx, ring_base, n_slabs * slab, slab, args.io_threads)
    else:
        host_pool = torch.empty((w.pool_chunks, stored_bytes), dtype=torch.uint8, pin_memory=True)
        for c in range(w.pool_chunks):
            chunk_to(host_pool[c], c)
            if fp8:
                mk.matkv_register_chunk_fp8(sess.ctx, c, w.chunk_tokens, host_pool[c].data_ptr())
            else:
                mk.matkv_register_chunk(sess.ctx, c, w.chunk_tokens, host_pool[c].data_ptr(), None)
    torch.cuda.synchronize()
    del tmp8
    del tmp
    q_pf = torch.empty((L, B, S, Hq, D), dtype=torch.bfloat16, device=dev)
    k_pf = torch.empty((L, B, S, Hkv, D), dtype=torch.bfloat16, device=dev)
    v_pf = torch.empty_like(k_pf)
    q_dc = torch.empty((T, L, B, Hq, D), dtype=torch.bfloat16, device=dev)
    k_dc = torch.empty((T, L, B, Hkv, D), dtype=torch.bfloat16, device=dev)
    v_dc = torch.empty_like(k_dc)
    for t_, st in ((q_pf, mi.STREAM_Q_PREFILL), (k_pf, mi.STREAM_K_PREFILL), (v_pf, mi.STREAM_V_PREFILL),
                   (q_dc, mi.STREAM_Q_DECODE), (k_dc, mi.STREAM_K_DECODE), (v_dc, mi.STREAM_V_DECODE)):
        gen.fill_bf16(t_, w.seed, st)
    o_pf, o_dc = torch.empty_like(q_pf), torch.empty_like(q_dc)
    ho_dc = torch.empty(o_dc.shape, dtype=torch.bfloat16, pin_memory=True)
    stream, copy = torch.cuda.Stream(device=dev), torch.cuda.Stream(device=dev)
    ctx = sess.ctx
    from paper_2512_22195_b200.pipeline import PipelinedBatches
    pipe = PipelinedBatches(sess, n_slots, slot_bytes, stream, copy)     # two slot regions; the tests run this same class
    torch.cuda.synchronize()

    def stage(n):
        return pipe.stage(n, needed[n])

    def compute(n, stage_next=None):
        pipe.compute(n, batches[n], S, T, q_pf, k_pf, v_pf, o_pf, q_dc, k_dc, v_dc, o_dc, stage_next=stage_next)
        with torch.cuda.stream(stream):
            ho_dc.copy_(o_dc, non_blocking=True)

    def wall(fn):
        torch.cuda.synchronize()
        t0 = time.perf_counter()
        fn()
        torch.cuda.synchronize()
        return time.perf_counter() - t0

    def only_stage():
        for n in range(n_batches):
            stage(n)

    def serial():
        for n in range(n_batches):
            tk = stage(n)
            mk.matkv_stage_wait(ctx, tk)
            compute(n)
            torch.cuda.synchronize()

    def pipelined():
        stage(0)
        for n in range(n_batches):   # table n is built (its slots resolved), then batch n+1 goes to the other region
            compute(n, stage_next=needed[n + 1] if n + 1 < n_batches else None)

    # warm-up: two batches through the whole path
    stage(0); compute(0); stage(1); compute(1)
    torch.cuda.synchronize()
    sampler = ClockSampler(dev.index)
    t_stage = wall(only_stage)
    t_serial = wall(serial)
    t0 = time.time()
    t_pipe = wall(pipelined)
    t1 = time.time()
    clocks = sampler.stop(t0, t1)
    if sess.status() != 0:
        raise RuntimeError("device status non-zero after the pipeline")
    # bytes one pass really copies: a chunk that already sits in the target slot region is not copied again
    occ, n_copied = [set(), set()], 0
    for n in range(n_batches):
        new = set(needed[n]) - occ[n % 2]
        n_copied += len(new)
        occ[n % 2] = set(needed[n])
        occ[(n + 1) % 2] -= new
    staged_bytes = n_copied * stored_bytes          # bytes that crossed the link (or left storage)
    tokens = n_batches * B * T
    kv_bytes = sum((len(row) * w.chunk_tokens + S + t + 1) * w.beta for ids in batches for row in ids for t in range(T)) * L
    t_compute = t_serial - t_stage
    print(json.dumps({
        "metric": "decode_tokens_per_s", "value": tokens / t_pipe, "unit": "tokens/s", "n_gpus": 1, "steps": n_batches,
        "warmup": 2, "ms_per_step": 1e3 * t_pipe / n_batches, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "bf16 in, fp32 softmax/accumulate", "data": "synthetic",
        "config": {"workload": w.name, "layers": L, "batch": B, "chunks_per_request": w.chunks_per_req, "suffix": S,
                   "decode_steps": T, "pool_chunks": w.pool_chunks, "pinned_pool_gb": w.pool_chunks * stored_bytes / 1e9,
                   "kv_store": ("e4m3 codes + power-of-two scale per 64-token block, expanded to bf16 while staged (lossy store: "
                                "a workload of its own)" if fp8 else "bf16"),
                   "batches": n_batches, "timing": "host wall clock around synchronised passes (copy and compute streams)",
                   "chunk_pool": (f"files in {args.store_dir} read with O_DIRECT by {args.io_threads} threads through a pinned ring of 8 slabs"
                                  if args.store_dir else "pinned host memory"),
                   "staging": f"copy kernel, {args.stage_ctas} CTAs" if args.stage_ctas else "copy engine"},
        "clocks": clocks,
        "pipeline": {"t_stage_s": t_stage, "t_serial_s": t_serial, "t_pipelined_s": t_pipe,
                     ("storage_to_hbm_gbs_staging_alone" if args.store_dir else "h2d_gbs_staging_alone"): staged_bytes / t_stage / 1e9,
                     "staged_bytes": staged_bytes, "bf16_bytes_delivered_to_hbm": n_copied * slot_bytes,
                     "load_s_per_request_staging_alone": t_stage / (n_batches * B),
                     "overlap_efficiency": (t_serial - t_pipe) / t_stage if t_stage > 0 else None,
                     "requests_per_s": n_batches * B / t_pipe, "compute_s_estimate": t_compute,
                     "decode_kv_gbs_pipelined_lower_bound": kv_bytes / t_pipe / 1e9},
        "e2e": {"value": tokens / t_pipe, "unit": "tokens/s", "h2d_bytes_per_step": staged_bytes / n_batches,
                "d2h_bytes_per_step": ho_dc.numel() * 2},
    }), flush=True)
    sess.close()


# ---- materialisation side (store_KV): chunks prefilled alone and written out ----------------------------
def run_materialise(args):
    """The paper's store_KV on this path's terms: every chunk is attended alone, causally, from position 0 (synthetic
    q/k/v stand in for the model's projections), its K,V are laid out as a chunk blob, optionally compressed, and copied
    to pinned host memory on a side stream while the next chunk is computed."""
    import torch
    import paper_2512_22195_b200 as mk
    import matkv_inputs.device as gen
    from paper_2512_22195_b200.harness import Session
    dev = torch.device("cuda", int(os.environ.get("LOCAL_RANK", "0")))
    torch.cuda.set_device(dev)
    w = mi.workload("cfg2")
    if args.layers:
        w.n_layers = args.layers
    L, Hq, Hkv, D, n = w.n_layers, w.n_q_heads, w.n_kv_heads, w.head_dim, w.chunk_tokens
    n_chunks = args.batches or 16
    fp8 = args.kv_store == "fp8"
    sess = Session(L, Hq, Hkv, D, 1, 1, n, device=dev.index)
    q = torch.empty((L, 1, n, Hq, D), dtype=torch.bfloat16, device=dev)
    k = torch.empty((L, 1, n, Hkv, D), dtype=torch.bfloat16, device=dev)
    v = torch.empty_like(k)
    for t_, st in ((q, mi.STREAM_Q_PREFILL), (k, mi.STREAM_K_PREFILL), (v, mi.STREAM_V_PREFILL)):
        gen.fill_bf16(t_, w.seed, st)
    out = torch.empty_like(q)
    stored = mk.matkv_fp8_blob_bytes(sess.ctx, n) if fp8 else w.chunk_bytes
    blobs = [torch.empty(w.chunk_bytes, dtype=torch.uint8, device=dev) for _ in range(2)]
    blobs8 = [torch.empty(stored, dtype=torch.uint8, device=dev) for _ in range(2)] if fp8 else None
    host = torch.empty((n_chunks, stored), dtype=torch.uint8, pin_memory=True)
    stream, side = torch.cuda.Stream(device=dev), torch.cuda.Stream(device=dev)
    sp = stream.cuda_stream
    done = [torch.cuda.Event() for _ in range(2)]
    copied = [torch.cuda.Event() for _ in range(2)]

    def one(c):
        i = c % 2
        table = sess.build_table([[]], sp)
        mk.matkv_attend_prefill_all_layers(sess.ctx, table, n, q.data_ptr(), k.data_ptr(), v.data_ptr(), out.data_ptr(), None, sp)
        mk.matkv_table_advance(table, n, sp)
        if c >= 2:
            stream.wait_event(copied[i])                  # the blob buffer's previous contents have left
        mk.matkv_export_tail_as_chunk(sess.ctx, table, 0, n, blobs[i].data_ptr(), None, sp)
        src = blobs[i]
        if fp8:
            mk.matkv_quantize_chunk_fp8(sess.ctx, blobs[i].data_ptr(), n, blobs8[i].data_ptr(), sp)
            src = blobs8[i]
        done[i].record(stream)
        side.wait_event(done[i])
        with torch.cuda.stream(side):
            host[c].copy_(src, non_blocking=True)
            copied[i].record(side)

    with torch.cuda.stream(stream):
        for c in range(2):
            one(c)
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(stream)
        for c in range(n_chunks):
            one(c)
        stream.wait_stream(side)
        e1.record(stream)
        torch.cuda.synchronize()
    ms = e0.elapsed_time(e1)
    if sess.status() != 0:
        raise RuntimeError("device status non-zero")
    flops = 4.0 * Hq * D * L * (n * (n + 1) / 2) * n_chunks
    print(json.dumps({
        "metric": "materialised_tokens_per_s", "value": n_chunks * n / (ms * 1e-3), "unit": "tokens/s", "n_gpus": 1, "steps": n_chunks,
        "warmup": 2, "ms_per_step": ms / n_chunks, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "bf16 in, fp32 softmax/accumulate", "data": "synthetic",
        "config": {"workload": "materialise", "layers": L, "q_heads": Hq, "kv_heads": Hkv, "head_dim": D, "chunk_tokens": n,
                   "chunks": n_chunks, "stored_as": "e4m3 codes + block exponents" if fp8 else "bf16 blob",
                   "note": "attention and write-out only: the model's projections and MLPs are outside this path"},
        "phases": {"causal_attention_tflops": flops / (ms * 1e-3) / 1e12, "bytes_to_host_per_chunk": stored,
                   "d2h_gbs": stored * n_chunks / (ms * 1e-3) / 1e9, "chunks_per_s": n_chunks / (ms * 1e-3)},
    }), flush=True)
    sess.close()


# ---- the CUDA arm ----------------------------------------------------------------------------------
def parse_args(argv=None):
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=10)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="matkv", choices=["matkv", "reference"])
    ap.add_argument("--workload", default=HEADLINE, help="cfg1 .. cfg5 or materialise; default: the headline configuration "
                    "(the largest that fits one GPU), with the other configurations' lines attached")
    ap.add_argument("--decode-launch", default="all_layers", choices=["all_layers", "per_layer", "per_layer_graph"])
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--decode-ctas", type=int, default=0)
    ap.add_argument("--no-other-mode", action="store_true", help="skip the extra passes in the other decode launch modes")
    ap.add_argument("--no-other-workloads", action="store_true", help="headline run: do not attach the other configurations' lines")
    ap.add_argument("--batches", type=int, default=0, help="pipelined serving: number of sequential batches")
    ap.add_argument("--pool-chunks", type=int, default=0, help="pipelined serving: chunks in the pinned host pool")
    ap.add_argument("--store-dir", default="", help="pipelined serving: keep the chunk pool as files in this directory "
                    "(storage tier: reader threads -> pinned bounce ring -> device) instead of in pinned host memory")
    ap.add_argument("--io-threads", type=int, default=8)
    ap.add_argument("--stage-ctas", type=int, default=-1, help="stage host chunks with a copy kernel of this many CTAs; 0 = copy "
                    "engine; -1 = auto: 16 CTAs in the pipelined-serving mode, 8 in the single-batch end-to-end leg (a decode that "
                    "saturates HBM starves the copy engine: 38 GB/s against 45 with the copy kernel; more than 10 copy CTAs "
                    "slow the short decode launches of that leg down more than they add)")
    ap.add_argument("--kv-store", default="bf16", choices=["bf16", "fp8"],
                    help="pipelined serving: keep the host / file chunk pool as plain bf16 blobs or compressed (e4m3 codes with a "
                    "power-of-two scale per 64-token block, expanded to bf16 while staged; a lossy store, so a separate workload)")
    ap.add_argument("--copy-streams", type=int, default=0, help="end-to-end leg: copy streams the chunk staging of a step is split over "
                    "(0 = auto: one with the copy kernel, two with the copy engine)")
    ap.add_argument("--kv-hbm", default="bf16", choices=["bf16", "fp8"],
                    help="fp8: the chunks sit in HBM as e4m3 codes (MATKV_OPT_FP8_RESIDENT) and the streaming kernel converts them "
                    "in registers; a lossy KV format, so a workload of its own (forces --no-e2e)")
    ap.add_argument("--prefill-impl", type=int, default=0, choices=[0, 1, 2, 3],
                    help="sub-prefill kernel: 0 auto, 1 streaming kernel, 2 tensor-core kernel, 3 the same with two row blocks per CTA")
    ap.add_argument("--decode-impl", type=int, default=0, choices=[0, 1, 2],
                    help="decode kernel: 0 auto (chunk-major when the batch's requests share chunks), 1 request-major, 2 chunk-major")
    ap.add_argument("--share-tiles", type=int, default=0, help="chunk-major decode: 64-token tiles per work item (0 = the library's default)")
    ap.add_argument("--layers", type=int, default=0, help="override the workload's layer count (small profiling cases)")
    ap.add_argument("--decode-steps", type=int, default=0, help="override the workload's decode steps (small profiling cases)")
    return ap.parse_args(argv)


def _spawned_rank(rank, args):
    """One rank of a run that bench.py started itself (--gpus N without a torchrun environment)."""
    result = run_cuda_arm(args)
    if result is not None:
        print(json.dumps(result), flush=True)


def main(argv=None):
    args = parse_args(argv)
    if args.impl == "reference":
        return run_reference(args)
    import __graft_entry__ as ge
    ge.build()                      # no-op when the in-tree libraries are up to date
    if args.workload == "materialise":
        return run_materialise(args)
    if args.workload == "cfg5":
        return run_pipeline(args)
    if args.gpus > 1 and "WORLD_SIZE" not in os.environ:
        # not under torchrun: start the N ranks here (one process per GPU; independent replicas)
        import torch
        from paper_2512_22195_b200 import replicas
        if torch.cuda.device_count() < args.gpus:
            raise SystemExit(f"--gpus {args.gpus}: this machine shows {torch.cuda.device_count()} CUDA device(s)")
        replicas.launch(args.gpus, _spawned_rank, args)
        return
    result = run_cuda_arm(args)
    if result is None:
        return
    headline_alone = (args.workload == HEADLINE and int(os.environ.get("WORLD_SIZE", "1")) == 1 and not args.no_other_workloads
                      and not (args.layers or args.decode_steps or args.pool_chunks) and args.kv_hbm == "bf16")
    if headline_alone:
        import gc
        import torch
        gc.collect()
        torch.cuda.empty_cache()    # the headline's 86 GB of chunks are released: the child processes need the memory
        result["other_workloads"] = run_other_workloads(args)
    print(json.dumps(result), flush=True)


def workload_config(w: mi.Workload, decode_launch: str, kv_bytes_per_step: float):
    """The `config` object of a line: the same for the CUDA arm and the reference arm of a workload."""
    return {"workload": w.name, "layers": w.n_layers, "q_heads": w.n_q_heads, "kv_heads": w.n_kv_heads, "head_dim": w.head_dim,
            "batch": w.batch, "chunks_per_request": w.chunks_per_req, "chunk_tokens": w.chunk_tokens, "suffix": w.suffix,
            "decode_steps": w.decode_steps, "decode_launch": decode_launch,
            "prefill_launch": "all_layers" if decode_launch == "all_layers" else "per_layer",
            "l2": f"inputs larger than L2 (KV per decode step = {kv_bytes_per_step / 1e6:.0f} MB vs 126 MB L2)",
            "multi_gpu": "independent replicas per rank"}


def kv_bytes_of_decode(w: mi.Workload, n_req, n_steps=None):
    """Algorithmic KV bytes of `n_steps` decode steps (default: all): every visible K and V element once."""
    T = w.decode_steps if n_steps is None else n_steps
    return sum((n + w.suffix + t + 1) * w.beta for n in n_req for t in range(T)) * w.n_layers


def run_other_workloads(args):
    """The other configurations' lines, each from a child process (the GPU's memory is free again by now)."""
    out = {}
    steps = str(max(3, min(args.steps, 5)))
    cases = {"cfg2": ["--workload", "cfg2", "--steps", str(args.steps), "--warmup", str(args.warmup)],
             "cfg3": ["--workload", "cfg3", "--steps", steps, "--warmup", "3", "--no-e2e"],
             # the pipelined-serving mode on a reduced pool and batch count (stated in its config): 40 GB cannot be pinned
             # and walked three times within this run's time
             "cfg5": ["--workload", "cfg5", "--batches", "10", "--pool-chunks", "128"]}
    for name, extra in cases.items():
        t0 = time.time()
        try:
            r = subprocess.run([sys.executable, os.path.abspath(__file__), "--gpus", "1", "--no-cpu-baseline", "--no-other-workloads"] + extra,
                               capture_output=True, text=True, timeout=600)
            lines = [ln for ln in r.stdout.splitlines() if ln.startswith("{")]
            out[name] = json.loads(lines[-1]) if (r.returncode == 0 and lines) else {"failed": f"rc {r.returncode}", "stderr_tail": r.stderr[-400:]}
        except Exception as e:  # noqa: BLE001  (a failed side line must not lose the headline)
            out[name] = {"failed": repr(e)}
        out[name]["wall_s"] = round(time.time() - t0, 1)
        log(f"[other workloads] {name}: {out[name].get('value', out[name].get('failed'))} in {out[name]['wall_s']} s")
    return out


def run_cuda_arm(args):
    args.warmup = max(args.warmup, 3)

    import torch
    import torch.distributed as dist
    import paper_2512_22195_b200 as mk
    import matkv_inputs.device as gen
    from paper_2512_22195_b200 import replicas
    from paper_2512_22195_b200.harness import Session

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if world != args.gpus:
        log(f"[bench] --gpus {args.gpus} but WORLD_SIZE {world}: the process group decides, n_gpus = {world}")
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    replicas.init_from_env("nccl", dev)

    w = mi.workload(args.workload)
    if args.layers:
        w.n_layers = args.layers
        w.name += f"-L{args.layers}"
    if args.decode_steps:
        w.decode_steps = args.decode_steps
        w.name += f"-T{args.decode_steps}"
    if args.pool_chunks:
        w.pool_chunks = args.pool_chunks
        w.name += f"-P{args.pool_chunks}"
    L, B, S, T, Hq, Hkv, D = w.n_layers, w.batch, w.suffix, w.decode_steps, w.n_q_heads, w.n_kv_heads, w.head_dim
    ids = w.chunk_ids(0)
    needed = sorted({c for row in ids for c in row})
    sess = Session(L, Hq, Hkv, D, B, w.chunks_per_req, S + T, device=local)
    if args.decode_ctas:
        mk.matkv_set_option(sess.ctx, mk.OPT_DECODE_CTAS, args.decode_ctas)
    if args.decode_impl:
        mk.matkv_set_option(sess.ctx, mk.OPT_DECODE_IMPL, args.decode_impl)
    if args.prefill_impl:
        mk.matkv_set_option(sess.ctx, mk.OPT_PREFILL_IMPL, args.prefill_impl)
    if args.share_tiles:
        mk.matkv_set_option(sess.ctx, mk.OPT_SHARE_TILES, args.share_tiles)
    fused_advance = args.decode_launch == "all_layers"
    if fused_advance:   # the all-layers decode launch moves the tail itself: no separate counter kernel per step
        mk.matkv_set_option(sess.ctx, mk.OPT_DECODE_ADVANCES_TAIL, 1)
    # every rank works on its own replica of the batch (independent requests: no data-path collective)
    chunks = {}
    pool = torch.empty((len(needed), L, 2, Hkv, w.chunk_tokens, D), dtype=torch.bfloat16, device=dev)
    fp8_hbm = args.kv_hbm == "fp8"
    if fp8_hbm:
        # compress every chunk (device quantiser), park the codes in pinned host memory, stage them ONCE into device slots
        # in the compressed-resident form; the timed steps then only build tables over the staged chunks
        args.no_e2e = True
        w.name += "-fp8hbm"
        mk.matkv_set_option(sess.ctx, mk.OPT_FP8_RESIDENT, 1)
        stored = mk.matkv_fp8_blob_bytes(sess.ctx, w.chunk_tokens)
        host8 = torch.empty((len(needed), stored), dtype=torch.uint8, pin_memory=True)
        tmp8 = torch.empty(stored, dtype=torch.uint8, device=dev)
        for i, c in enumerate(needed):
            gen.fill_bf16(pool[i], w.seed, mi.STREAM_CHUNK + c)
            chunks[c] = pool[i]
            mk.matkv_quantize_chunk_fp8(sess.ctx, pool[i].data_ptr(), w.chunk_tokens, tmp8.data_ptr())
            host8[i].copy_(tmp8)
            mk.matkv_register_chunk_fp8(sess.ctx, c, w.chunk_tokens, host8[i].data_ptr())
        slot8 = mk.matkv_fp8_resident_bytes(sess.ctx, w.chunk_tokens)   # the resident form: codes plus 16-byte exponent records
        slots8 = torch.empty(len(needed) * slot8, dtype=torch.uint8, device=dev)
        cs8 = torch.cuda.Stream(device=dev)
        mk.matkv_stage_wait(sess.ctx, sess.stage(needed, slots8, slot8, cs8))
    else:
        for i, c in enumerate(needed):
            gen.fill_bf16(pool[i], w.seed, mi.STREAM_CHUNK + c)
            chunks[c] = pool[i]
            sess.register_device_chunk(c, pool[i])
    q_pf = torch.empty((L, B, S, Hq, D), dtype=torch.bfloat16, device=dev)
    k_pf = torch.empty((L, B, S, Hkv, D), dtype=torch.bfloat16, device=dev)
    v_pf = torch.empty_like(k_pf)
    gen.fill_bf16(q_pf, w.seed, mi.STREAM_Q_PREFILL)
    gen.fill_bf16(k_pf, w.seed, mi.STREAM_K_PREFILL)
    gen.fill_bf16(v_pf, w.seed, mi.STREAM_V_PREFILL)
    q_dc = torch.empty((T, L, B, Hq, D), dtype=torch.bfloat16, device=dev)
    k_dc = torch.empty((T, L, B, Hkv, D), dtype=torch.bfloat16, device=dev)
    v_dc = torch.empty_like(k_dc)
    gen.fill_bf16(q_dc, w.seed, mi.STREAM_Q_DECODE)
    gen.fill_bf16(k_dc, w.seed, mi.STREAM_K_DECODE)
    gen.fill_bf16(v_dc, w.seed, mi.STREAM_V_DECODE)
    o_pf = torch.empty_like(q_pf)
    o_dc = torch.empty_like(q_dc)
    torch.cuda.synchronize()

    stream = torch.cuda.Stream(device=dev)
    sp = stream.cuda_stream
    ctx = sess.ctx
    qs_l, ks_l = q_pf[0].numel() * 2, k_pf[0].numel() * 2
    qd_t, kd_t = q_dc[0].numel() * 2, k_dc[0].numel() * 2
    qd_l, kd_l = q_dc[0, 0].numel() * 2, k_dc[0, 0].numel() * 2
    g_q, g_k, g_v, g_o = torch.empty_like(q_dc[0]), torch.empty_like(k_dc[0]), torch.empty_like(v_dc[0]), torch.empty_like(q_dc[0])
    launches = {"n": 0}
    ev_d0 = [torch.cuda.Event(enable_timing=True) for _ in range(args.steps)]
    ev_d1 = [torch.cuda.Event(enable_timing=True) for _ in range(args.steps)]
    ev_p0 = [torch.cuda.Event(enable_timing=True) for _ in range(args.steps)]
    ev_g0 = [torch.cuda.Event(enable_timing=True) for _ in range(args.steps)]   # graph mode: replays start here
    table_us = []   # host time of matkv_build_chunk_table per timed step

    def one_step(q_pf_p, k_pf_p, v_pf_p, q_dc_p, k_dc_p, v_dc_p, timed_index=None, mode=args.decode_launch):
        """All pointers are device addresses; nothing here but C-ABI calls."""
        t_h = time.perf_counter()
        table = sess.build_table(ids, sp)
        if timed_index is not None:
            table_us.append((time.perf_counter() - t_h) * 1e6)
            ev_p0[timed_index].record(stream)
        if mode == "all_layers":
            mk.matkv_attend_prefill_all_layers(ctx, table, S, q_pf_p, k_pf_p, v_pf_p, o_pf.data_ptr(), None, sp)
        else:
            for layer in range(L):
                mk.matkv_attend_prefill(ctx, table, layer, S, q_pf_p + layer * qs_l, k_pf_p + layer * ks_l, v_pf_p + layer * ks_l,
                                        o_pf.data_ptr() + layer * qs_l, None, sp)
        mk.matkv_table_advance(table, S, sp)
        if timed_index is not None:
            ev_d0[timed_index].record(stream)
        n = (1 if mode == "all_layers" else L) + 1
        if mode == "per_layer_graph":
            # one decode step (L per-layer launches + the tail counter) captured once per table and replayed
            # T times; each step's q/k/v are copied into fixed buffers first (a graph replays fixed addresses)
            g_q.copy_(q_dc[0]); g_k.copy_(k_dc[0]); g_v.copy_(v_dc[0])
            graph = torch.cuda.CUDAGraph()
            with torch.cuda.graph(graph, stream=stream):
                for layer in range(L):
                    mk.matkv_attend_decode(ctx, table, layer, g_q.data_ptr() + layer * qd_l, g_k.data_ptr() + layer * kd_l,
                                           g_v.data_ptr() + layer * kd_l, g_o.data_ptr() + layer * qd_l, None, sp)
                mk.matkv_table_advance(table, 1, sp)
            mk.matkv_table_set_tail_len(table, S, sp)       # the capture ran nothing but moved the host-side mirror
            # The decode window of this mode starts here: capture and instantiation (torch synchronises, collects
            # garbage and empties its cache around a capture: milliseconds of host time that vary from call to call)
            # belong to the step, not to the replayed launches a serving loop would reuse for many steps.
            if timed_index is not None:
                ev_g0[timed_index].record(stream)
            for t in range(T):
                g_q.copy_(q_dc[t], non_blocking=True); g_k.copy_(k_dc[t], non_blocking=True); g_v.copy_(v_dc[t], non_blocking=True)
                graph.replay()
                o_dc[t].copy_(g_o, non_blocking=True)
            n += T * (L + 1)
            if timed_index is not None:
                ev_d1[timed_index].record(stream)
            return n
        for t in range(T):
            if mode == "all_layers":
                mk.matkv_attend_decode_all_layers(ctx, table, q_dc_p + t * qd_t, k_dc_p + t * kd_t, v_dc_p + t * kd_t,
                                                  o_dc.data_ptr() + t * qd_t, None, sp)
                n += 1
                if fused_advance:
                    continue
                n += 1
            else:
                for layer in range(L):
                    mk.matkv_attend_decode(ctx, table, layer, q_dc_p + t * qd_t + layer * qd_l, k_dc_p + t * kd_t + layer * kd_l,
                                           v_dc_p + t * kd_t + layer * kd_l, o_dc.data_ptr() + t * qd_t + layer * qd_l, None, sp)
                n += L + 1
            mk.matkv_table_advance(table, 1, sp)
        if timed_index is not None:
            ev_d1[timed_index].record(stream)
        return n

    def barrier():
        torch.cuda.synchronize()
        replicas.barrier()
        torch.cuda.synchronize()

    def timed_region(fn, steps):
        """K steps bracketed by barrier + synchronize; returns device milliseconds (max over ranks)."""
        barrier()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        t0 = time.time()
        e0.record(stream)
        n = 0
        for i in range(steps):
            n += fn(i)
        e1.record(stream)
        barrier()
        t1 = time.time()
        ms = replicas.max_over_ranks(e0.elapsed_time(e1), dev)
        return ms, n, t0, t1

    dev_ptrs = (q_pf.data_ptr(), k_pf.data_ptr(), v_pf.data_ptr(), q_dc.data_ptr(), k_dc.data_ptr(), v_dc.data_ptr())
    with torch.cuda.stream(stream):
        for _ in range(args.warmup):
            one_step(*dev_ptrs)
        sampler = ClockSampler(local) if rank == 0 else None
        ms, n_launch, t0, t1 = timed_region(lambda i: one_step(*dev_ptrs, timed_index=i), args.steps)
        clocks = sampler.stop(t0, t1) if sampler else None
        st = sess.status()
        if st != 0:
            raise RuntimeError(f"device status {st} after the timed region")
        ev_dec = ev_g0 if args.decode_launch == "per_layer_graph" else ev_d0
        dec_ms = sum(a.elapsed_time(b) for a, b in zip(ev_dec, ev_d1))
        pre_ms = sum(a.elapsed_time(b) for a, b in zip(ev_p0, ev_d0))
        step_ms = sorted(a.elapsed_time(b) for a, b in zip(ev_p0, ev_d1))      # every timed step on its own (table upload excluded)
        dec_step_ms = sorted(a.elapsed_time(b) for a, b in zip(ev_dec, ev_d1))
        table_us_main = sorted(table_us)
        # the other launch granularities, for the record (same work): one launch per layer is what a model calls, replayed from
        # a CUDA graph or launched one by one
        others = [m for m in ("all_layers", "per_layer_graph", "per_layer") if m != args.decode_launch]
        other_dec_ms = {}
        if not args.no_other_mode:
            for other in others:
                k_o = min(args.steps, 3)
                for _ in range(2):   # the first graph capture of a process pays one-off costs
                    one_step(*dev_ptrs, mode=other)
                timed_region(lambda i: one_step(*dev_ptrs, timed_index=i, mode=other), k_o)
                ev_dec_o = ev_g0 if other == "per_layer_graph" else ev_d0
                other_dec_ms[other] = sum(a.elapsed_time(b) for a, b in zip(ev_dec_o[:k_o], ev_d1[:k_o])) / k_o

    # read-only streaming probe over the same chunk memory (plain 16-byte loads), same run
    probe_gbs = None
    with torch.cuda.stream(stream):
        pe0, pe1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        for _ in range(2):
            mk.matkv_probe_read(ctx, pool.data_ptr(), pool.numel() * 2, sp)
        pe0.record(stream)
        for _ in range(5):
            mk.matkv_probe_read(ctx, pool.data_ptr(), pool.numel() * 2, sp)
        pe1.record(stream)
        torch.cuda.synchronize()
        probe_gbs = 5 * pool.numel() * 2 / (pe0.elapsed_time(pe1) * 1e-3) / 1e9

    # algorithmic KV bytes of the decode loop of one step: every visible K and V element once
    n_req = [sum(chunks[c].shape[3] for c in row) for row in ids]
    kv_bytes_decode = sum((n + S + t + 1) * w.beta for n in n_req for t in range(T)) * L
    kv_bytes_prefill = sum((n + S) * w.beta for n in n_req) * L
    if fp8_hbm:   # chunk tokens cost half the bytes plus a 16-byte exponent record per 64-token block and KV head; the tail stays bf16
        beta8 = w.beta // 2 + Hkv * 16 / 64.0
        kv_bytes_decode = sum(n * beta8 + (S + t + 1) * w.beta for n in n_req for t in range(T)) * L
        kv_bytes_prefill = sum(n * beta8 + S * w.beta for n in n_req) * L
    # algorithmic flops of the sub-prefill: 4 * Hq * D per (query token, visible key), the causal part of the suffix block once
    prefill_flops = 4.0 * Hq * D * L * sum(S * n + S * (S + 1) / 2 for n in n_req)
    tokens = B * T * world
    value = tokens * args.steps / (ms * 1e-3)
    decode_launches = T * (1 if args.decode_launch == "all_layers" else L)
    avg_launch_ms = dec_ms / (args.steps * decode_launches)
    achieved = kv_bytes_decode / decode_launches / (avg_launch_ms * 1e-3) / 1e9
    peaks, peak_kind = measured_peaks()
    peak = float(peaks["hbm_gbs"])
    # chunk tiles the batch lists against the tiles the decode kernel in use reads (chunk-major stacking)
    tiles_logical, tiles_read = mk.matkv_table_sharing(sess.table)
    chunk_major = args.decode_impl == 2 or (args.decode_impl == 0 and tiles_logical * 4 >= tiles_read * 5)
    logical_gbs = achieved
    if chunk_major:
        # the chunk-major kernel reads a chunk once per 16 / G requests that list it: its algorithmic bytes are the
        # tiles it reads (64 tokens x K and V x all KV heads) plus every request's tail
        tile_bytes = 64 * w.beta
        read_bytes_decode = sum(tiles_read * tile_bytes + sum(S + t + 1 for _ in range(B)) * w.beta for t in range(T)) * L
        achieved = read_bytes_decode / decode_launches / (avg_launch_ms * 1e-3) / 1e9
    tflops_peak_sus = float(peaks.get("bf16_tflops_sustained", FALLBACK_BF16_TFLOPS))
    tflops_peak_burst = float(peaks.get("bf16_tflops", FALLBACK_BF16_TFLOPS))
    prefill_tflops = prefill_flops * args.steps / (pre_ms * 1e-3) / 1e12
    cap = NCU_TRAFFIC.get((args.workload, args.decode_launch)) if not (args.layers or args.decode_steps or fp8_hbm) else None
    traffic = cap[0] * (L / cap[1]) if cap else None
    kv_launch_mean = kv_bytes_decode / T          # KV bytes of one decode step (all layers), mean over the steps

    def per_layer_phase(ms_per_step_decode):
        us = ms_per_step_decode * 1e3 / (T * L)
        return {"us_per_layer_launch": us, "kv_gbs": kv_launch_mean / L / (us * 1e-6) / 1e9,
                "frac_of_hbm_peak": kv_launch_mean / L / (us * 1e-6) / 1e9 / peak,
                "decode_only_tokens_per_s": B * T / (ms_per_step_decode * 1e-3)}

    modes = {args.decode_launch: dec_ms / args.steps}
    modes.update(other_dec_ms)
    result = {
        "metric": "decode_tokens_per_s", "value": value, "unit": "tokens/s", "n_gpus": world, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": ms / args.steps, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "bf16 in, fp32 softmax/accumulate" + (", chunk KV as e4m3 codes in HBM (fp16 MMAs)" if fp8_hbm else ""), "data": "synthetic",
        "config": workload_config(w, args.decode_launch, kv_bytes_decode / T),
        "gpu_launches": n_launch,
        "clocks": clocks,
        "roofline": {"bound": "hbm", "kernel": "k_attend_shared (chunk-major decode)" if chunk_major else "k_attend_stream (decode)",
                     "chunk_tiles_listed_vs_read": [tiles_logical, tiles_read if chunk_major else tiles_logical],
                     "achieved": achieved, "peak": peak,
                     "unit": "GB/s", "frac": achieved / peak, "peak_kind": f"of {peak_kind}",
                     "frac_of_nominal_8TBs": achieved / NOMINAL_HBM_GBS,
                     "read_probe_gbs_same_run": probe_gbs,
                     "traffic": traffic,
                     "traffic_source": (None if not cap else "one ncu capture of this kernel build" + ("" if cap[1] == L else
                                        f" on a {cap[1]}-layer case, scaled by the layer count")),
                     "algorithmic_bytes_per_launch": (read_bytes_decode if chunk_major else kv_bytes_decode) / decode_launches,
                     "logical_kv_gbs": logical_gbs,
                     "avg_launch_us": avg_launch_ms * 1e3},
        # the sub-prefill tiles: a dense contraction on the tensor cores (tcgen05), timed inside the step
        "roofline_prefill": {"bound": "tensor", "kernel": "k_prefill_tc (sub-prefill)", "achieved": prefill_tflops, "unit": "TFLOP/s",
                             "peak": tflops_peak_sus, "frac": prefill_tflops / tflops_peak_sus,
                             "peak_kind": f"of {peak_kind} (bf16 sustained: the kernel runs inside a long step)",
                             "frac_of_burst_peak": prefill_tflops / tflops_peak_burst,
                             "flops_per_step": prefill_flops, "intensity_flop_per_byte": S * (Hq // Hkv)},
        "repeats": {"steps": args.steps, "step_ms_min": step_ms[0], "step_ms_median": step_ms[len(step_ms) // 2],
                    "decode_ms_min": dec_step_ms[0], "decode_ms_median": dec_step_ms[len(dec_step_ms) // 2],
                    "tokens_per_s_best_step": B * T * world / (step_ms[0] * 1e-3),
                    "table_build_host_us_median": table_us_main[len(table_us_main) // 2]},
        "phases": {"prefill_ms_per_step": pre_ms / args.steps, "decode_ms_per_step": dec_ms / args.steps,
                   "prefill_tflops": prefill_tflops,
                   "decode_only_tokens_per_s": B * T * args.steps / (dec_ms * 1e-3),
                   "decode_kv_gbs": kv_bytes_decode * args.steps / (dec_ms * 1e-3) / 1e9,
                   "prefill_kv_gbs": kv_bytes_prefill * args.steps / (pre_ms * 1e-3) / 1e9,
                   # one launch per layer is what a model's forward pass calls: per-launch time and KV GB/s, replayed from a
                   # CUDA graph and launched one by one
                   "per_layer_graph": per_layer_phase(modes["per_layer_graph"]) if "per_layer_graph" in modes else None,
                   "per_layer": per_layer_phase(modes["per_layer"]) if "per_layer" in modes else None,
                   "all_layers_decode_ms_per_step": modes.get("all_layers")},
    }

    # ---- end to end: the same step through the same calls, from host buffers --------------------
    # A workload whose chunks do not fit ~24 GB of pinned host memory (and three device slot regions of that size) runs this
    # leg on a subset of its layers, stated in the result: copies and compute are both exactly linear in the layer count, so
    # the step time scales by L / layers-in-the-subset.
    e2e_bytes = len(needed) * w.chunk_bytes
    Le = L
    if e2e_bytes > 24e9:
        Le = max(d for d in range(1, L + 1) if L % d == 0 and e2e_bytes * d / L <= 24e9)
    e2e_scale = L / Le
    if not args.no_e2e:
        copy = torch.cuda.Stream(device=dev)
        host = {c: torch.empty((Le,) + tuple(chunks[c].shape[1:]), dtype=torch.bfloat16, pin_memory=True) for c in needed}
        for c in needed:
            host[c].copy_(chunks[c][:Le])
        # the query-side tensors of the subset's layers (dense copies: the calls take dense [layers of the context] tensors)
        eq_pf, ek_pf, ev_pf = (x[:Le].contiguous() for x in (q_pf, k_pf, v_pf))
        eq_dc, ek_dc, ev_dc = (x[:, :Le].contiguous() for x in (q_dc, k_dc, v_dc))
        hq_pf, hk_pf, hv_pf = (x.cpu().pin_memory() for x in (eq_pf, ek_pf, ev_pf))
        hq_dc, hk_dc, hv_dc = (x.cpu().pin_memory() for x in (eq_dc, ek_dc, ev_dc))
        ho_pf = torch.empty(eq_pf.shape, dtype=torch.bfloat16, pin_memory=True)
        ho_dc = torch.empty(eq_dc.shape, dtype=torch.bfloat16, pin_memory=True)
        qs_l, ks_l = eq_pf[0].numel() * 2, ek_pf[0].numel() * 2
        qd_t, kd_t = eq_dc[0].numel() * 2, ek_dc[0].numel() * 2
        qd_l, kd_l = eq_dc[0, 0].numel() * 2, ek_dc[0, 0].numel() * 2
        torch.cuda.synchronize()
        sess2 = Session(Le, Hq, Hkv, D, B, w.chunks_per_req, S + T, device=local)
        # staging: 8 copy CTAs beside short decode launches (config 2: 45 GB/s against 38 with the copy engine); the copy engine
        # on two streams when a step moves tens of gigabytes under long launches (config 4: 54.7 GB/s against 41 with 16 - 32 copy CTAs)
        e2e_stage_ctas = args.stage_ctas if args.stage_ctas >= 0 else (8 if e2e_bytes < 4e9 else 0)
        if e2e_stage_ctas > 0:
            mk.matkv_set_option(sess2.ctx, mk.OPT_STAGE_CTAS, e2e_stage_ctas)
        if args.decode_impl:
            mk.matkv_set_option(sess2.ctx, mk.OPT_DECODE_IMPL, args.decode_impl)
        for c in needed:
            mk.matkv_register_chunk(sess2.ctx, c, w.chunk_tokens, host[c].data_ptr(), None)
        slot_bytes = w.chunk_bytes // L * Le
        # the chunks of a step are split over N_COPY copy streams, each with slot regions of its own: several copies in
        # flight keep the link busier while the decode saturates HBM
        n_copy = max(1, min(args.copy_streams if args.copy_streams > 0 else (1 if e2e_stage_ctas > 0 else 2), len(needed)))
        parts = [needed[k::n_copy] for k in range(n_copy)]
        copies = [copy] + [torch.cuda.Stream(device=dev) for _ in range(n_copy - 1)]
        # Three regions of chunk slots and of query-side buffers: the copies of step i+2 start as soon as step i-1 has
        # finished with its region, so the link never waits for the compute (with two regions the copies of step i+1
        # could only start when step i's compute did, and a step took as long as its copies plus the hand-over).
        NB = 3
        slots = [[torch.empty(len(parts[k]) * slot_bytes, dtype=torch.uint8, device=dev) for k in range(n_copy)] for _ in range(NB)]
        d_in = [tuple(torch.empty_like(x) for x in (eq_pf, ek_pf, ev_pf, eq_dc, ek_dc, ev_dc)) for _ in range(NB)]
        d_out = [(torch.empty_like(eq_pf), torch.empty_like(eq_dc)) for _ in range(NB)]
        h_in = (hq_pf, hk_pf, hv_pf, hq_dc, hk_dc, hv_dc)
        h2d = len(needed) * slot_bytes + sum(x.numel() * 2 for x in h_in)
        d2h = (ho_pf.numel() + ho_dc.numel()) * 2
        ctx2 = sess2.ctx
        out_stream = torch.cuda.Stream(device=dev)
        in_ready = [torch.cuda.Event() for _ in range(NB)]
        comp_done = [torch.cuda.Event() for _ in range(NB)]
        out_done = [torch.cuda.Event() for _ in range(NB)]
        load_done = [torch.cuda.Event() for _ in range(n_copy)]
        state = {"loaded": -1, "table": None}

        def load(i):
            """Everything step i needs from the host: its query-side inputs (small, first) on the first copy stream, its
            chunks into slot region i % NB over all copy streams.  No copy starts before step i - NB, the last user of
            the region, has finished."""
            r = i % NB
            if i >= NB:
                for cs in copies:
                    cs.wait_event(comp_done[r])
            with torch.cuda.stream(copy):
                for dst, src in zip(d_in[r], h_in):
                    dst.copy_(src, non_blocking=True)
                in_ready[r].record(copy)
            for k in range(n_copy):
                sess2.stage(parts[k], slots[r][k], slot_bytes, copies[k])
                load_done[k].record(copies[k])
            state["loaded"] = i

        def drain_copies():
            """The compute stream waits for every copy issued so far.  Called right before the timed region and at its
            end: the region then holds exactly as many whole loads as steps (the loads it starts with in flight are
            finished first, the ones it issues ahead for later steps are finished inside it)."""
            for k in range(n_copy):
                stream.wait_event(load_done[k])

        def e2e_step(i, last=False):
            # step i's table was built at the end of step i-1 (or before the first step), AFTER load(i) and BEFORE
            # load(i+1): a table points at the places its chunks were staged to most recently
            table = state["table"]
            r = i % NB
            dq_pf, dk_pf, dv_pf, dq_dc, dk_dc, dv_dc = d_in[r]
            eo_pf, eo_dc = d_out[r]
            stream.wait_event(in_ready[r])
            if i >= NB:
                stream.wait_event(out_done[r])             # step i-NB's outputs have left these buffers
            if args.decode_launch == "all_layers":
                mk.matkv_attend_prefill_all_layers(ctx2, table, S, dq_pf.data_ptr(), dk_pf.data_ptr(), dv_pf.data_ptr(), eo_pf.data_ptr(), None, sp)
            else:
                for layer in range(Le):
                    mk.matkv_attend_prefill(ctx2, table, layer, S, dq_pf.data_ptr() + layer * qs_l, dk_pf.data_ptr() + layer * ks_l,
                                            dv_pf.data_ptr() + layer * ks_l, eo_pf.data_ptr() + layer * qs_l, None, sp)
            mk.matkv_table_advance(table, S, sp)
            for t in range(T):
                if args.decode_launch == "all_layers":
                    mk.matkv_attend_decode_all_layers(ctx2, table, dq_dc.data_ptr() + t * qd_t, dk_dc.data_ptr() + t * kd_t,
                                                      dv_dc.data_ptr() + t * kd_t, eo_dc.data_ptr() + t * qd_t, None, sp)
                    if fused_advance:
                        continue
                else:
                    for layer in range(Le):
                        mk.matkv_attend_decode(ctx2, table, layer, dq_dc.data_ptr() + t * qd_t + layer * qd_l,
                                               dk_dc.data_ptr() + t * kd_t + layer * kd_l, dv_dc.data_ptr() + t * kd_t + layer * kd_l,
                                               eo_dc.data_ptr() + t * qd_t + layer * qd_l, None, sp)
                mk.matkv_table_advance(table, 1, sp)
            comp_done[r].record(stream)
            out_stream.wait_event(comp_done[r])
            with torch.cuda.stream(out_stream):            # the step's results go back to the host
                ho_pf.copy_(eo_pf, non_blocking=True)
                ho_dc.copy_(eo_dc, non_blocking=True)
                out_done[r].record(out_stream)
            # the next step's table (its build makes the compute stream wait for that step's chunk copies, issued one
            # step ago), then the copies of the step after it
            state["table"] = sess2.build_table(ids, sp)
            load(i + 2)
            if last:
                stream.wait_event(out_done[r])             # the timed region ends when the last result is on the host
                drain_copies()                             # and when every copy it issued has landed
            return 0

        if fused_advance:
            mk.matkv_set_option(ctx2, mk.OPT_DECODE_ADVANCES_TAIL, 1)
        with torch.cuda.stream(stream):
            load(0)
            state["table"] = sess2.build_table(ids, sp)
            load(1)
            w_e2e = max(3, min(args.warmup, 5))
            for i in range(w_e2e):
                e2e_step(i)
            drain_copies()
            k_e2e = min(args.steps, 5)
            ms_e, _, _, _ = timed_region(lambda i: e2e_step(i + w_e2e, last=(i == k_e2e - 1)), k_e2e)
        if sess2.status() != 0:
            raise RuntimeError("device status non-zero after the end-to-end region")
        result["e2e"] = {"value": tokens * k_e2e / (ms_e * 1e-3 * e2e_scale), "unit": "tokens/s", "h2d_bytes_per_step": h2d * e2e_scale,
                         "d2h_bytes_per_step": d2h * e2e_scale, "ms_per_step": ms_e / k_e2e * e2e_scale, "steps": k_e2e, "warmup": w_e2e,
                         "subset": (None if Le == L else f"layers 0..{Le - 1} of {L}: the chunks of all {L} layers ({e2e_bytes / 1e9:.0f} GB) fit neither the "
                                    f"pinned host pool nor three device slot regions; measured {ms_e / k_e2e:.1f} ms per step with "
                                    f"{h2d / 1e9:.1f} GB copied in, scaled by {e2e_scale:g} (copies and compute are linear in layers)"),
                         "overlap": "the chunks and query-side inputs of the next two steps copied in (three slot regions), and the previous "
                                    "step's outputs copied out, on side streams under this step's prefill and decode",
                         "staging": (f"copy kernel, {e2e_stage_ctas} CTAs" if e2e_stage_ctas > 0 else "copy engine") + f", {n_copy} copy streams",
                         "h2d_gbs_if_copy_bound": h2d * k_e2e / (ms_e * 1e-3) / 1e9}
        sess2.close()
        del host, slots

    # ---- the oracle on this machine's host cores, bounded sample (rank 0, N = 1 only) ------------------
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        import oracle
        oracle.build()
        from paper_2512_22195_b200.harness import dev_to_bits
        # calibrate on one layer, then take as many layers and steps as fit ~12 s (work is linear in both)
        probe = OracleState(w, {c: dev_to_bits(chunks[c][0:1]) for c in needed}, ids, layers=[0])
        t_one = max(probe.decode_steps(0, 1), 1e-3)
        n_l = int(max(1, min(L, 40.0 / t_one)))     # about 40 seconds of oracle work in all
        n_l = int(max(1, min(n_l, 4e9 // (len(needed) * (w.chunk_bytes // L)))))   # and at most ~4 GB of chunk layers on the host
        n_s = int(max(1, min(T - 1, round(40.0 / (t_one * n_l)))))
        st_o = OracleState(w, {c: dev_to_bits(chunks[c][0:n_l]) for c in needed}, ids, layers=list(range(n_l)))
        t_s = st_o.decode_steps(0, n_s)
        per_step_full = t_s / n_s * (L / n_l)
        how = "" if n_l == L else f", extrapolated linearly from layers 0..{n_l - 1} to all {L}"
        result["cpu_baseline"] = {"value": B / per_step_full, "unit": "tokens/s", "cores": min(st_o.cores, n_l * B), "kind": "oracle",
                                  "sample": f"decode steps 0..{n_s - 1} of {T} of {w.name} ({n_l} of {L} layers, batch {B}), "
                                            f"{t_s:.1f} s on {st_o.cores} threads{how}",
                                  "kv_gbs": sum((n + S + t + 1) * w.beta for n in n_req for t in range(n_s)) * n_l / t_s / 1e9}
    sess.close()
    if world > 1:
        dist.destroy_process_group()
    return result if rank == 0 else None


if __name__ == "__main__":
    main()
