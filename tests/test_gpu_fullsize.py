"""Parity at the benchmark's full size and launch configuration (config 2: 32 layers, Llama-3-8B head
shape, 5 x 1,024-token chunks, 64-token suffix through the tile kernel, 128 decode steps with all layers
in one launch; config 3: batch 16, 10 of 256 chunks per request by Zipf rank, chunk-major decode; config 4: the 70B head
shape with 64K tokens of context per request), on
sampled outputs the oracle computes one by one."""
import numpy as np
import pytest
import torch

import matkv_inputs as mi
import oracle
from _util import check

pytestmark = pytest.mark.gpu


def test_cfg2_full_size_sampled_units():
    import matkv_inputs.device as gen
    from paper_2512_22195_b200.harness import Session, dev_to_bits
    w = mi.workload("cfg2")
    L, B, S, T, Hq, Hkv, D = w.n_layers, w.batch, w.suffix, w.decode_steps, w.n_q_heads, w.n_kv_heads, w.head_dim
    ids = w.chunk_ids(0)
    needed = sorted({c for row in ids for c in row})
    sess = Session(L, Hq, Hkv, D, B, w.chunks_per_req, S + T)
    pool = torch.empty((len(needed), L, 2, Hkv, w.chunk_tokens, D), dtype=torch.bfloat16, device="cuda")
    for i, c in enumerate(needed):
        gen.fill_bf16(pool[i], w.seed, mi.STREAM_CHUNK + c)
        sess.register_device_chunk(c, pool[i])
    q_pf = torch.empty((L, B, S, Hq, D), dtype=torch.bfloat16, device="cuda")
    k_pf = torch.empty((L, B, S, Hkv, D), dtype=torch.bfloat16, device="cuda")
    v_pf = torch.empty_like(k_pf)
    q_dc = torch.empty((T, L, B, Hq, D), dtype=torch.bfloat16, device="cuda")
    k_dc = torch.empty((T, L, B, Hkv, D), dtype=torch.bfloat16, device="cuda")
    v_dc = torch.empty_like(k_dc)
    for t_, st in ((q_pf, mi.STREAM_Q_PREFILL), (k_pf, mi.STREAM_K_PREFILL), (v_pf, mi.STREAM_V_PREFILL),
                   (q_dc, mi.STREAM_Q_DECODE), (k_dc, mi.STREAM_K_DECODE), (v_dc, mi.STREAM_V_DECODE)):
        gen.fill_bf16(t_, w.seed, st)
    sess.build_table(ids)
    pf_out, pf_lse = sess.prefill_all_layers(q_pf, k_pf, v_pf)       # one launch for all layers, as the bench does
    pf = [(pf_out[layer], pf_lse[layer]) for layer in range(L)]
    sess.advance(S)
    dc = []
    for t in range(T):
        dc.append(sess.decode_all_layers(q_dc[t], k_dc[t], v_dc[t]))
        sess.advance(1)
    assert sess.status() == 0

    sh1 = oracle.Shape(1, Hq, Hkv, D)                     # the oracle sees one layer's slabs at a time

    def layer_request(layer, n_decode):
        blobs = [dev_to_bits(pool[needed.index(c)][layer:layer + 1]) for c in ids[0]]
        rq = oracle.Request(sh1, blobs, S + T)
        _, k, v = mi.prefill_inputs(w, layer)
        rq.append_only(0, k[0], v[0])
        rq.advance(S)
        for s_ in range(n_decode):
            _, k, v = mi.decode_inputs(w, s_)
            rq.append_only(0, k[layer, 0][None], v[layer, 0][None])
            rq.advance(1)
        return rq

    # sub-prefill: layers 0 and 31, suffix rows 0, 31, 63
    for layer in (0, L - 1):
        rq = layer_request(layer, 0)
        q, _, _ = mi.prefill_inputs(w, layer)
        rows = [0, S // 2 - 1, S - 1]
        o_ref, l_ref = oracle.attend(sh1, 0, rq.chunks, rq.tail_k[0], rq.tail_v[0], q[0][rows], [r + 1 for r in rows])
        out, lse = pf[layer]
        check(dev_to_bits(out)[0][rows], o_ref, lse.cpu().numpy()[0][rows], l_ref, f"full-size prefill layer {layer}")
    # decode: sampled (step, layer) pairs, every head
    for step, layer in ((0, 0), (0, L - 1), (63, 17), (T - 1, 0), (T - 1, L - 1)):
        rq = layer_request(layer, step)
        q, k, v = mi.decode_inputs(w, step)
        o_ref, l_ref = rq.attend_new(0, q[layer, 0][None], k[layer, 0][None], v[layer, 0][None])
        out, lse = dc[step]
        check(dev_to_bits(out)[layer, 0], o_ref[0], lse.cpu().numpy()[layer, 0], l_ref[0], f"full-size decode step {step} layer {layer}")
    # the inputs the GPU consumed are the generator's bytes (the oracle regenerated them on the host)
    assert np.array_equal(dev_to_bits(q_dc[5]), mi.decode_inputs(w, 5)[0])
    sess.close()


def test_cfg3_full_size_chunk_major_sampled_units():
    """Config 3 at full size: 16 requests x 10 chunks drawn by Zipf rank from 256 (73 distinct), 32 layers,
    32-token suffix, 256 decode steps, every step one all-layers launch of the chunk-major kernel that also
    advances the tail; sampled (step, layer, request) outputs against the oracle."""
    import matkv_inputs.device as gen
    import paper_2512_22195_b200 as mk
    from paper_2512_22195_b200.harness import Session, dev_to_bits
    w = mi.workload("cfg3")
    L, B, S, T, Hq, Hkv, D = w.n_layers, w.batch, w.suffix, w.decode_steps, w.n_q_heads, w.n_kv_heads, w.head_dim
    ids = w.chunk_ids(0)
    needed = sorted({c for row in ids for c in row})
    sess = Session(L, Hq, Hkv, D, B, w.chunks_per_req, S + T)
    mk.matkv_set_option(sess.ctx, mk.OPT_DECODE_IMPL, 2)
    mk.matkv_set_option(sess.ctx, mk.OPT_DECODE_ADVANCES_TAIL, 1)
    pool = torch.empty((len(needed), L, 2, Hkv, w.chunk_tokens, D), dtype=torch.bfloat16, device="cuda")
    for i, c in enumerate(needed):
        gen.fill_bf16(pool[i], w.seed, mi.STREAM_CHUNK + c)
        sess.register_device_chunk(c, pool[i])
    q_pf = torch.empty((L, B, S, Hq, D), dtype=torch.bfloat16, device="cuda")
    k_pf = torch.empty((L, B, S, Hkv, D), dtype=torch.bfloat16, device="cuda")
    v_pf = torch.empty_like(k_pf)
    q_dc = torch.empty((T, L, B, Hq, D), dtype=torch.bfloat16, device="cuda")
    k_dc = torch.empty((T, L, B, Hkv, D), dtype=torch.bfloat16, device="cuda")
    v_dc = torch.empty_like(k_dc)
    for t_, st in ((q_pf, mi.STREAM_Q_PREFILL), (k_pf, mi.STREAM_K_PREFILL), (v_pf, mi.STREAM_V_PREFILL),
                   (q_dc, mi.STREAM_Q_DECODE), (k_dc, mi.STREAM_K_DECODE), (v_dc, mi.STREAM_V_DECODE)):
        gen.fill_bf16(t_, w.seed, st)
    table = sess.build_table(ids)
    listed, read = mk.matkv_table_sharing(table)
    assert listed == B * w.chunks_per_req * (w.chunk_tokens // 64) and read < listed * 0.6   # stacking nearly halves the reads
    sess.prefill_all_layers(q_pf, k_pf, v_pf)
    sess.advance(S)
    samples = {0: [(0, 0), (L - 1, 3)], 100: [(17, 9)], T - 1: [(0, B - 1), (L - 1, 0)]}   # step -> (layer, request)
    got = {}
    for t in range(T):
        out, lse = sess.decode_all_layers(q_dc[t], k_dc[t], v_dc[t])
        if t in samples:
            got[t] = (dev_to_bits(out), lse.cpu().numpy())
    assert sess.status() == 0
    sh1 = oracle.Shape(1, Hq, Hkv, D)
    for step, pairs in samples.items():
        q, k, v = mi.decode_inputs(w, step)
        for layer, r in pairs:
            blobs = [dev_to_bits(pool[needed.index(c)][layer:layer + 1]) for c in ids[r]]
            rq = oracle.Request(sh1, blobs, S + T)
            _, kp, vp = mi.prefill_inputs(w, layer)
            rq.append_only(0, kp[r], vp[r])
            rq.advance(S)
            for s_ in range(step):
                _, kk, vv = mi.decode_inputs(w, s_)
                rq.append_only(0, kk[layer, r][None], vv[layer, r][None])
                rq.advance(1)
            o_ref, l_ref = rq.attend_new(0, q[layer, r][None], k[layer, r][None], v[layer, r][None])
            check(got[step][0][layer, r], o_ref[0], got[step][1][layer, r], l_ref[0],
                  f"full-size chunk-major decode step {step} layer {layer} request {r}")
    sess.close()


def test_cfg4_full_size_sampled_units():
    """Config 4 at full size (Llama-3-70B head shape: 64 query heads on 8 KV heads, 80 layers, 4 requests x 32 chunks of
    2,048 tokens = 86 GB of chunks in HBM, 128-token suffix: 1,024 query rows per KV head through the tile kernel with
    two row blocks per CTA, all 80 layers in one launch of 10,240 CTAs; 64 decode steps, all layers per launch);
    sampled outputs against the oracle."""
    import matkv_inputs.device as gen
    from paper_2512_22195_b200.harness import Session, dev_to_bits
    w = mi.workload("cfg4")
    L, B, S, T, Hq, Hkv, D = w.n_layers, w.batch, w.suffix, w.decode_steps, w.n_q_heads, w.n_kv_heads, w.head_dim
    free, _ = torch.cuda.mem_get_info()
    if free < 100e9:
        pytest.skip("needs 100 GB of free device memory")
    ids = w.chunk_ids(0)
    needed = sorted({c for row in ids for c in row})
    sess = Session(L, Hq, Hkv, D, B, w.chunks_per_req, S + T)
    pool = torch.empty((len(needed), L, 2, Hkv, w.chunk_tokens, D), dtype=torch.bfloat16, device="cuda")
    for i, c in enumerate(needed):
        gen.fill_bf16(pool[i], w.seed, mi.STREAM_CHUNK + c)
        sess.register_device_chunk(c, pool[i])
    q_pf = torch.empty((L, B, S, Hq, D), dtype=torch.bfloat16, device="cuda")
    k_pf = torch.empty((L, B, S, Hkv, D), dtype=torch.bfloat16, device="cuda")
    v_pf = torch.empty_like(k_pf)
    q_dc = torch.empty((T, L, B, Hq, D), dtype=torch.bfloat16, device="cuda")
    k_dc = torch.empty((T, L, B, Hkv, D), dtype=torch.bfloat16, device="cuda")
    v_dc = torch.empty_like(k_dc)
    for t_, st in ((q_pf, mi.STREAM_Q_PREFILL), (k_pf, mi.STREAM_K_PREFILL), (v_pf, mi.STREAM_V_PREFILL),
                   (q_dc, mi.STREAM_Q_DECODE), (k_dc, mi.STREAM_K_DECODE), (v_dc, mi.STREAM_V_DECODE)):
        gen.fill_bf16(t_, w.seed, st)
    sess.build_table(ids)
    pf_out, pf_lse = sess.prefill_all_layers(q_pf, k_pf, v_pf)
    sess.advance(S)
    samples = {0: [(0, 0)], 31: [(40, 2)], T - 1: [(L - 1, 3)]}          # decode step -> (layer, request)
    got = {}
    for t in range(T):
        out, lse = sess.decode_all_layers(q_dc[t], k_dc[t], v_dc[t])
        if t in samples:
            got[t] = (dev_to_bits(out), lse.cpu().numpy())
        sess.advance(1)
    assert sess.status() == 0
    sh1 = oracle.Shape(1, Hq, Hkv, D)

    def layer_request(layer, r, n_decode):
        blobs = [dev_to_bits(pool[needed.index(c)][layer:layer + 1]) for c in ids[r]]
        rq = oracle.Request(sh1, blobs, S + T)
        _, k, v = mi.prefill_inputs(w, layer)
        rq.append_only(0, k[r], v[r])
        rq.advance(S)
        for s_ in range(n_decode):
            _, k, v = mi.decode_inputs(w, s_)
            rq.append_only(0, k[layer, r][None], v[layer, r][None])
            rq.advance(1)
        return rq

    # sub-prefill: first, middle and last suffix token of a request in the first and the last layer (every head)
    for layer, r in ((0, 0), (L - 1, B - 1)):
        rq = layer_request(layer, r, 0)
        q, _, _ = mi.prefill_inputs(w, layer)
        rows = [0, S // 2 - 1, S - 1]
        o_ref, l_ref = oracle.attend(sh1, 0, rq.chunks, rq.tail_k[0], rq.tail_v[0], q[r][rows], [x + 1 for x in rows])
        check(dev_to_bits(pf_out[layer])[r][rows], o_ref, pf_lse[layer].cpu().numpy()[r][rows], l_ref,
              f"config 4 full-size prefill layer {layer} request {r}")
    for step, pairs in samples.items():
        q, k, v = mi.decode_inputs(w, step)
        for layer, r in pairs:
            rq = layer_request(layer, r, step)
            o_ref, l_ref = rq.attend_new(0, q[layer, r][None], k[layer, r][None], v[layer, r][None])
            check(got[step][0][layer, r], o_ref[0], got[step][1][layer, r], l_ref[0],
                  f"config 4 full-size decode step {step} layer {layer} request {r}")
    sess.close()


def test_cfg5_pipelined_serving_sampled_units():
    """Config 5 at its own configuration, through the class the benchmark runs: Llama-3-8B head shape, batches of
    8 requests x 10 distinct 1,024-token chunks drawn from a pinned host pool, every batch staged by the copy kernel
    (16 CTAs) on a side stream into one of two slot regions WHILE the previous batch is prefilled and decoded (32-token
    suffix, 128 decode steps, all layers per launch), the previous table freed in between, no host wait anywhere.
    Reduced, and said so: 8 of the 32 layers and a pool of 100 chunks instead of 296 (so that batches also meet
    chunks that still sit in their region from two batches ago).  Checked: one request's whole gather per batch bit
    for bit against the host pool, and sampled (batch, step, layer, request) outputs against the oracle."""
    import matkv_inputs.device as gen
    import paper_2512_22195_b200 as mk
    from paper_2512_22195_b200.harness import Session, dev_to_bits
    from paper_2512_22195_b200.pipeline import PipelinedBatches
    w = mi.workload("cfg5")
    w.n_layers, w.pool_chunks = 8, 100
    n_batches = 4
    L, B, S, T, Hq, Hkv, D, n = w.n_layers, w.batch, w.suffix, w.decode_steps, w.n_q_heads, w.n_kv_heads, w.head_dim, w.chunk_tokens
    batches = [w.chunk_ids(i) for i in range(n_batches)]
    needed = [sorted({c for row in ids for c in row}) for ids in batches]
    assert all(len(set(row)) == w.chunks_per_req for ids in batches for row in ids)
    sess = Session(L, Hq, Hkv, D, B, w.chunks_per_req, S + T)
    mk.matkv_set_option(sess.ctx, mk.OPT_STAGE_CTAS, 16)
    host_pool = torch.empty((w.pool_chunks, L, 2, Hkv, n, D), dtype=torch.bfloat16, pin_memory=True)
    tmp = torch.empty((L, 2, Hkv, n, D), dtype=torch.bfloat16, device="cuda")
    for c in range(w.pool_chunks):
        gen.fill_bf16(tmp, w.seed, mi.STREAM_CHUNK + c)
        host_pool[c].copy_(tmp)
        mk.matkv_register_chunk(sess.ctx, c, n, host_pool[c].data_ptr(), None)
    torch.cuda.synchronize()
    q_pf = torch.empty((L, B, S, Hq, D), dtype=torch.bfloat16, device="cuda")
    k_pf = torch.empty((L, B, S, Hkv, D), dtype=torch.bfloat16, device="cuda")
    v_pf = torch.empty_like(k_pf)
    q_dc = torch.empty((T, L, B, Hq, D), dtype=torch.bfloat16, device="cuda")
    k_dc = torch.empty((T, L, B, Hkv, D), dtype=torch.bfloat16, device="cuda")
    v_dc = torch.empty_like(k_dc)
    for t_, st in ((q_pf, mi.STREAM_Q_PREFILL), (k_pf, mi.STREAM_K_PREFILL), (v_pf, mi.STREAM_V_PREFILL),
                   (q_dc, mi.STREAM_Q_DECODE), (k_dc, mi.STREAM_K_DECODE), (v_dc, mi.STREAM_V_DECODE)):
        gen.fill_bf16(t_, w.seed, st)
    o_pf = [torch.empty_like(q_pf) for _ in range(n_batches)]
    o_dc = [torch.empty_like(q_dc) for _ in range(n_batches)]
    stream, copy = torch.cuda.Stream(), torch.cuda.Stream()
    pipe = PipelinedBatches(sess, max(len(x) for x in needed), w.chunk_bytes, stream, copy)
    g_layer, g_req = L - 1, [0, 3, 7, 5]
    rows = w.chunks_per_req * n + S + T
    gathered = [(torch.empty((Hkv, rows, D), dtype=torch.bfloat16, device="cuda"), torch.empty((Hkv, rows, D), dtype=torch.bfloat16, device="cuda"))
                for _ in range(n_batches)]
    torch.cuda.synchronize()
    pipe.stage(0, needed[0])
    for b in range(n_batches):
        def after(table, b=b):
            got = mk.matkv_gather_debug(sess.ctx, table, g_layer, g_req[b], gathered[b][0].data_ptr(), gathered[b][1].data_ptr(), rows,
                                        stream.cuda_stream)
            assert got == rows
        pipe.compute(b, batches[b], S, T, q_pf, k_pf, v_pf, o_pf[b], q_dc, k_dc, v_dc, o_dc[b],
                     stage_next=needed[b + 1] if b + 1 < n_batches else None, after_decode=after)
    torch.cuda.synchronize()
    assert sess.status() == 0
    assert mk.matkv_stage_pending(sess.ctx) == 0
    pool_bits = host_pool.view(torch.int16).numpy().view(np.uint16)      # [pool, L, 2, Hkv, n, D]
    # the staged bytes: the whole chunk part of one request's gather per batch
    for b in range(n_batches):
        row = batches[b][g_req[b]]
        k_bits, v_bits = dev_to_bits(gathered[b][0]), dev_to_bits(gathered[b][1])
        assert np.array_equal(k_bits[:, :w.chunks_per_req * n], np.concatenate([pool_bits[c, g_layer, 0] for c in row], axis=1)), f"batch {b}"
        assert np.array_equal(v_bits[:, :w.chunks_per_req * n], np.concatenate([pool_bits[c, g_layer, 1] for c in row], axis=1)), f"batch {b}"
    sh1 = oracle.Shape(1, Hq, Hkv, D)

    def layer_request(b, layer, r, n_decode):
        rq = oracle.Request(sh1, [pool_bits[c, layer:layer + 1] for c in batches[b][r]], S + T)
        _, k, v = mi.prefill_inputs(w, layer)
        rq.append_only(0, k[r], v[r])
        rq.advance(S)
        for s_ in range(n_decode):
            _, k, v = mi.decode_inputs(w, s_)
            rq.append_only(0, k[layer, r][None], v[layer, r][None])
            rq.advance(1)
        return rq

    # sub-prefill: first and last suffix token of one request per batch
    for b, layer, r in ((0, 0, 1), (1, 5, 6), (2, L - 1, 0), (3, 2, 4)):
        rq = layer_request(b, layer, r, 0)
        q, _, _ = mi.prefill_inputs(w, layer)
        rws = [0, S - 1]
        o_ref, l_ref = oracle.attend(sh1, 0, rq.chunks, rq.tail_k[0], rq.tail_v[0], q[r][rws], [x + 1 for x in rws])
        check(dev_to_bits(o_pf[b][layer])[r][rws], o_ref, None, None, f"pipelined batch {b} prefill layer {layer} request {r}")
    # decode: (batch, step, layer, request)
    for b, step, layer, r in ((0, 0, 0, 0), (0, T - 1, L - 1, 7), (1, 64, 3, 2), (2, 5, 1, 5), (2, T - 1, 0, 0), (3, 0, L - 1, 3), (3, 100, 4, 6)):
        rq = layer_request(b, layer, r, step)
        q, k, v = mi.decode_inputs(w, step)
        o_ref, _ = rq.attend_new(0, q[layer, r][None], k[layer, r][None], v[layer, r][None])
        check(dev_to_bits(o_dc[b][step])[layer, r], o_ref[0], None, None, f"pipelined batch {b} decode step {step} layer {layer} request {r}")
    sess.close()
