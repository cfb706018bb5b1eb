"""GPU tests of the chunk table, the bit-exact gather, staging and the host-side error paths."""
import numpy as np
import pytest
import torch

from _util import rand_bits

pytestmark = pytest.mark.gpu


def _mk():
    import paper_2512_22195_b200 as mk
    from paper_2512_22195_b200.harness import Session, bits_to_dev, dev_to_bits
    return mk, Session, bits_to_dev, dev_to_bits


def test_p8_gather_is_bit_exact_with_shared_and_ragged_chunks():
    mk, Session, to_dev, to_bits = _mk()
    L, Hq, Hkv, D = 2, 4, 2, 64
    sess = Session(L, Hq, Hkv, D, 3, 5, 16)
    lens = [1, 7, 127, 129, 300]
    blobs = [rand_bits(41, i, (L, 2, Hkv, n, D)) for i, n in enumerate(lens)]
    for i, b in enumerate(blobs):
        sess.register_device_chunk(i, b)
    ids = [[4, 0, 2], [2, 2, 1, 3], []]
    sess.build_table(ids)
    # put something in the tails too
    tk, tv = rand_bits(41, 90, (3, L, Hkv, 16, D)), rand_bits(41, 91, (3, L, Hkv, 16, D))
    sess.tail_k.copy_(to_dev(tk)); sess.tail_v.copy_(to_dev(tv))
    mk.matkv_table_set_tail_len(sess.table, 5)
    for r, row in enumerate(ids):
        for layer in range(L):
            rows = sum(lens[c] for c in row) + 5
            k, v = sess.gather(layer, r, rows)
            want_k = np.concatenate([blobs[c][layer, 0] for c in row] + [tk[r, layer, :, :5]], axis=1)
            want_v = np.concatenate([blobs[c][layer, 1] for c in row] + [tv[r, layer, :, :5]], axis=1)
            assert np.array_equal(to_bits(k), want_k) and np.array_equal(to_bits(v), want_v)
    assert sess.status() == 0
    sess.close()


def test_staging_then_gather_bit_exact_and_overlap_bookkeeping():
    mk, Session, to_dev, to_bits = _mk()
    L, Hq, Hkv, D, n = 2, 4, 2, 64, 96
    sess = Session(L, Hq, Hkv, D, 2, 3, 8)
    blobs = [rand_bits(42, i, (L, 2, Hkv, n, D)) for i in range(5)]
    for i, b in enumerate(blobs):
        sess.register_host_chunk(i, b)
    slot_bytes = blobs[0].nbytes
    assert slot_bytes % 256 == 0
    slots_a = torch.empty(3 * slot_bytes, dtype=torch.uint8, device="cuda")
    slots_b = torch.empty(3 * slot_bytes, dtype=torch.uint8, device="cuda")
    copy = torch.cuda.Stream()
    # not staged yet -> the table cannot be built
    with pytest.raises(mk.MatkvError) as e:
        sess.build_table([[0, 1], [1]])
    assert e.value.code == mk.E_NOT_STAGED
    t1 = sess.stage([0, 1, 1, 0], slots_a, slot_bytes, copy)           # duplicates are copied once
    sess.build_table([[0, 1], [1]])                                    # stream waits for the copies, host does not
    k, v = sess.gather(1, 0, 2 * n)
    assert np.array_equal(to_bits(k), np.concatenate([blobs[0][1, 0], blobs[1][1, 0]], axis=1))
    # next batch goes to the other region while the first table is alive
    t2 = sess.stage([2, 3, 4], slots_b, slot_bytes, copy)
    mk.matkv_stage_wait(sess.ctx, t2)
    assert mk.matkv_stage_query(sess.ctx, t1) and mk.matkv_stage_query(sess.ctx, t2)
    sess.build_table([[4, 2], [3]])
    k, v = sess.gather(0, 0, 2 * n)
    assert np.array_equal(to_bits(v), np.concatenate([blobs[4][0, 1], blobs[2][0, 1]], axis=1))
    # re-staging into region A evicts chunk 0 but keeps chunk 1 in place (no new copy needed)
    sess.stage([1, 2], slots_a, slot_bytes, copy)
    with pytest.raises(mk.MatkvError) as e:
        mk.matkv_build_chunk_table(sess.ctx, [[0]], sess.tail_k.data_ptr(), sess.tail_v.data_ptr())
    assert e.value.code == mk.E_NOT_STAGED
    sess.build_table([[1, 2], [2]])
    k, v = sess.gather(1, 1, n)
    assert np.array_equal(to_bits(k), blobs[2][1, 0])
    # too many distinct chunks for the region
    with pytest.raises(mk.MatkvError) as e:
        sess.stage([0, 1, 2, 3], slots_a, slot_bytes, copy)
    assert e.value.code == mk.E_CAPACITY
    sess.close()


def test_staging_with_the_copy_kernel_is_bit_exact():
    mk, Session, to_dev, to_bits = _mk()
    L, Hq, Hkv, D = 2, 4, 2, 128
    sess = Session(L, Hq, Hkv, D, 1, 3, 8)
    mk.matkv_set_option(sess.ctx, mk.OPT_STAGE_CTAS, 4)
    lens = [1000, 33, 257]
    blobs = [rand_bits(45, i, (L, 2, Hkv, n, D)) for i, n in enumerate(lens)]
    for i, b in enumerate(blobs):
        sess.register_host_chunk(i, b)
    slot_bytes = (max(b.nbytes for b in blobs) + 255) // 256 * 256
    slots = torch.empty(3 * slot_bytes, dtype=torch.uint8, device="cuda")
    copy = torch.cuda.Stream()
    tk = sess.stage([2, 0, 1], slots, slot_bytes, copy)
    sess.build_table([[0, 1, 2]])
    k, v = sess.gather(1, 0, sum(lens))
    assert np.array_equal(to_bits(k), np.concatenate([b[1, 0] for b in blobs], axis=1))
    assert np.array_equal(to_bits(v), np.concatenate([b[1, 1] for b in blobs], axis=1))
    mk.matkv_stage_wait(sess.ctx, tk)
    with pytest.raises(mk.MatkvError):
        mk.matkv_set_option(sess.ctx, mk.OPT_STAGE_CTAS, 1000)
    sess.close()


def test_host_side_error_paths():
    mk, Session, to_dev, to_bits = _mk()
    with pytest.raises(mk.MatkvError):
        mk.matkv_create(1, 8, 3, 64, 1, 1, 8)             # heads do not divide
    with pytest.raises(mk.MatkvError):
        mk.matkv_create(1, 8, 2, 96, 1, 1, 8)             # unsupported head_dim
    sess = Session(1, 8, 2, 64, 2, 2, 4)
    blob = rand_bits(43, 0, (1, 2, 2, 8, 64))
    sess.register_device_chunk(7, blob)
    with pytest.raises(mk.MatkvError) as e:
        mk.matkv_register_chunk(sess.ctx, 7, 8, None, sess.chunks[7].data_ptr())     # duplicate id
    assert e.value.code == mk.E_INVALID_ARG
    with pytest.raises(mk.MatkvError) as e:
        mk.matkv_register_chunk(sess.ctx, 8, 8, None, sess.chunks[7].data_ptr() + 2)  # misaligned
    assert e.value.code == mk.E_ALIGNMENT
    with pytest.raises(mk.MatkvError) as e:
        sess.build_table([[99]])
    assert e.value.code == mk.E_UNKNOWN_CHUNK
    with pytest.raises(mk.MatkvError) as e:
        sess.build_table([[7, 7, 7]])                                             # more than max_chunks_per_req
    assert e.value.code == mk.E_CAPACITY
    with pytest.raises(mk.MatkvError) as e:
        sess.build_table([[7], [7], [7]])                                         # batch > max_batch
    assert e.value.code == mk.E_CAPACITY
    sess.build_table([[7], []])
    q = to_dev(rand_bits(43, 1, (2, 5, 8, 64)))
    kv = to_dev(rand_bits(43, 2, (2, 5, 2, 64)))
    with pytest.raises(mk.MatkvError) as e:
        sess.prefill(0, q, kv, kv)                                               # 5 tokens > tail capacity 4
    assert e.value.code == mk.E_CAPACITY
    with pytest.raises(mk.MatkvError) as e:
        sess.decode(3, q[:, 0], kv[:, 0], kv[:, 0])                              # layer out of range
    assert e.value.code == mk.E_INVALID_ARG
    mk.matkv_table_set_tail_len(sess.table, 4)
    with pytest.raises(mk.MatkvError) as e:
        sess.decode(0, q[:, 0], kv[:, 0], kv[:, 0])                              # tail full
    assert e.value.code == mk.E_CAPACITY
    mk.matkv_unregister_chunk(sess.ctx, 7)
    with pytest.raises(mk.MatkvError) as e:
        mk.matkv_unregister_chunk(sess.ctx, 7)
    assert e.value.code == mk.E_UNKNOWN_CHUNK
    assert sess.status() == 0
    sess.close()


def test_device_generator_matches_host_generator():
    import matkv_inputs as mi
    import matkv_inputs.device as gen
    _, _, _, to_bits = _mk()
    t = torch.empty(100003, dtype=torch.bfloat16, device="cuda")
    gen.fill_bf16(t, seed=5, stream=77, shift=0, start=12345)
    assert np.array_equal(to_bits(t), mi.normal_bf16(5, 77, 100003, 0, start=12345))
    gen.fill_bf16(t, seed=5, stream=78, shift=3, start=0)
    assert np.array_equal(to_bits(t), mi.normal_bf16(5, 78, 100003, 3))


def test_bounded_wait_runs_out_and_reports_without_losing_the_context():
    """Failure detection without a fault: a wait that nothing satisfies gives up after its limit and the
    status word says so; the context keeps working afterwards."""
    import time
    mk, Session, to_dev, to_bits = _mk()
    sess = Session(1, 8, 2, 64, 1, 1, 4)
    assert sess.status() == 0
    t0 = time.perf_counter()
    mk.matkv_selftest_wait_timeout(sess.ctx, 0.25)
    st = sess.status(clear=True)                      # synchronises
    dt = time.perf_counter() - t0
    assert st == mk.E_TIMEOUT
    assert 0.1 < dt < 3.0, dt
    assert sess.status() == 0
    # the same context still computes
    sess.register_device_chunk(0, rand_bits(44, 0, (1, 2, 2, 40, 64)))
    sess.build_table([[0]])
    q, kv = to_dev(rand_bits(44, 1, (1, 8, 64))), to_dev(rand_bits(44, 2, (1, 2, 64)))
    out, _ = sess.decode(0, q, kv, kv)
    assert torch.isfinite(out.float()).all() and sess.status() == 0
    with pytest.raises(mk.MatkvError):
        mk.matkv_selftest_wait_timeout(sess.ctx, 30.0)
    sess.close()


def test_storage_tier_files_through_the_bounce_ring(tmp_path):
    """Chunks stored as raw-bytes files (one per chunk id): reader threads -> pinned ring -> device slots.
    More chunks than ring slabs, an odd-sized chunk (buffered read path), then gather bit-exact and decode."""
    import oracle
    from _util import check
    mk, Session, to_dev, to_bits = _mk()
    L, Hq, Hkv, D = 2, 8, 2, 64
    lens = [64, 7, 128, 33, 64, 96, 1]
    sess = Session(L, Hq, Hkv, D, 2, 4, 8)
    blobs = [rand_bits(61, i, (L, 2, Hkv, n, D)) for i, n in enumerate(lens)]
    for i, b in enumerate(blobs):
        path = tmp_path / f"{i}.kv"
        with open(path, "wb") as f:
            f.write(b"\0" * (4096 if i == 2 else 0))          # chunk 2 sits at an offset inside its file
            f.write(b.tobytes())
        mk.matkv_register_chunk_file(sess.ctx, i, lens[i], str(path), 4096 if i == 2 else 0)
    slot_bytes = max(b.nbytes for b in blobs)
    slot_bytes = (slot_bytes + 4095) // 4096 * 4096
    slots = torch.empty(len(lens) * slot_bytes, dtype=torch.uint8, device="cuda")
    copy = torch.cuda.Stream()
    with pytest.raises(mk.MatkvError):                         # no bounce buffer yet
        sess.stage([0], slots, slot_bytes, copy)
    ring = torch.empty(3 * slot_bytes + 4096, dtype=torch.uint8, pin_memory=True)
    base = (ring.data_ptr() + 4095) // 4096 * 4096
    mk.matkv_set_bounce_buffer(sess.ctx, base, 3 * slot_bytes, slot_bytes, 2)     # 3 slabs, 7 chunks: the ring wraps
    tk = sess.stage(list(range(len(lens))), slots, slot_bytes, copy)
    ids = [[0, 1, 2, 3], [6, 5, 4, 2]]
    sess.build_table(ids)                                       # the compute stream waits for the copies
    for r, row in enumerate(ids):
        rows = sum(lens[c] for c in row)
        k, v = sess.gather(1, r, rows)
        assert np.array_equal(to_bits(k), np.concatenate([blobs[c][1, 0] for c in row], axis=1))
        assert np.array_equal(to_bits(v), np.concatenate([blobs[c][1, 1] for c in row], axis=1))
    mk.matkv_stage_wait(sess.ctx, tk)
    assert mk.matkv_stage_query(sess.ctx, tk)
    sh = oracle.Shape(L, Hq, Hkv, D)
    q, k, v = rand_bits(61, 100, (2, Hq, D)), rand_bits(61, 101, (2, Hkv, D)), rand_bits(61, 102, (2, Hkv, D))
    out, lse = sess.decode(0, to_dev(q), to_dev(k), to_dev(v))
    for r, row in enumerate(ids):
        o_ref, l_ref = oracle.Request(sh, [blobs[c] for c in row], 8).attend_new(0, q[r][None], k[r][None], v[r][None])
        check(to_bits(out)[r], o_ref[0], lse.cpu().numpy()[r], l_ref[0], f"file-backed decode req {r}")
    # error paths: missing file, file shorter than the chunk
    with pytest.raises(mk.MatkvError) as e:
        mk.matkv_register_chunk_file(sess.ctx, 100, 8, str(tmp_path / "nope.kv"))
    assert e.value.code == mk.E_IO
    with pytest.raises(mk.MatkvError) as e:
        mk.matkv_register_chunk_file(sess.ctx, 101, 4096, str(tmp_path / "1.kv"))
    assert e.value.code == mk.E_IO
    assert sess.status() == 0
    sess.close()


def test_materialise_then_reuse_round_trip():
    """store_KV in kernel terms: a chunk's tokens are sub-prefilled alone (empty chunk list, causal, from
    position 0), the tail is exported as a chunk blob, and that blob serves later requests.  The exported
    bytes equal the K,V that went in, the causal outputs match the oracle, and a request that reuses the
    blob gets the same answer as one that was given the original K,V as a chunk."""
    import oracle
    from _util import check
    mk, Session, to_dev, to_bits = _mk()
    L, Hq, Hkv, D, n = 2, 8, 2, 128, 150
    sess = Session(L, Hq, Hkv, D, 1, 2, n)
    sh = oracle.Shape(L, Hq, Hkv, D)
    q = rand_bits(71, 1, (L, 1, n, Hq, D))
    k = rand_bits(71, 2, (L, 1, n, Hkv, D))
    v = rand_bits(71, 3, (L, 1, n, Hkv, D))
    sess.build_table([[]])
    ref = oracle.Request(sh, [], n)
    for layer in range(L):
        out, lse = sess.prefill(layer, to_dev(q[layer]), to_dev(k[layer]), to_dev(v[layer]))
        o_ref, l_ref = ref.attend_new(layer, q[layer, 0], k[layer, 0], v[layer, 0])     # plain causal attention from position 0
        check(to_bits(out)[0], o_ref, lse.cpu().numpy()[0], l_ref, f"materialisation layer {layer}")
    sess.advance(n)
    blob_dev = torch.empty((L, 2, Hkv, n, D), dtype=torch.bfloat16, device="cuda")
    blob_host = torch.empty((L, 2, Hkv, n, D), dtype=torch.bfloat16, pin_memory=True)
    mk.matkv_export_tail_as_chunk(sess.ctx, sess.table, 0, n, blob_dev.data_ptr(), blob_host.data_ptr())
    torch.cuda.synchronize()
    want = np.stack([np.stack([k[layer, 0].transpose(1, 0, 2), v[layer, 0].transpose(1, 0, 2)]) for layer in range(L)])
    assert np.array_equal(to_bits(blob_dev), want) and np.array_equal(to_bits(blob_host), want)
    with pytest.raises(mk.MatkvError) as e:
        mk.matkv_export_tail_as_chunk(sess.ctx, sess.table, 0, n + 1, blob_dev.data_ptr())
    assert e.value.code == mk.E_CAPACITY
    # reuse: the exported blob as a materialised chunk of a new request
    sess2 = Session(L, Hq, Hkv, D, 1, 2, 8)
    sess2.register_device_chunk(5, blob_dev)
    sess2.build_table([[5]])
    q1, k1, v1 = rand_bits(71, 4, (1, Hq, D)), rand_bits(71, 5, (1, Hkv, D)), rand_bits(71, 6, (1, Hkv, D))
    out, lse = sess2.decode(1, to_dev(q1), to_dev(k1), to_dev(v1))
    o_ref, l_ref = oracle.Request(sh, [want], 8).attend_new(1, q1, k1, v1)
    check(to_bits(out)[0], o_ref[0], lse.cpu().numpy()[0], l_ref[0], "decode over the re-used chunk")
    assert sess.status() == 0 and sess2.status() == 0
    sess.close(); sess2.close()


def test_context_and_table_churn_leaves_no_device_memory_behind():
    """A serving process creates and frees tables for every batch and contexts now and then: 150 contexts, ten tables
    each (both decode kernels' tables), a sub-prefill and two decode steps per table; the device's free memory at
    the end is what it was after the first cycle (torch's caching allocator keeps the harness's own tensors, so what
    would show here is memory the library itself allocated and lost)."""
    mk, Session, bits_to_dev, dev_to_bits = _mk()
    L, Hq, Hkv, D, B = 2, 8, 2, 128, 3
    blobs = [bits_to_dev(rand_bits(91, i, (L, 2, Hkv, n, D))) for i, n in enumerate([130, 64, 200])]
    q = bits_to_dev(rand_bits(91, 10, (B, 5, Hq, D)))
    k = bits_to_dev(rand_bits(91, 11, (B, 5, Hkv, D)))
    q1, k1 = q[:, :1].contiguous(), k[:, :1].contiguous()

    def cycle(i):
        sess = Session(L, Hq, Hkv, D, B, 3, 16)
        if i % 2:
            mk.matkv_set_option(sess.ctx, mk.OPT_DECODE_IMPL, 2)
        for c, b in enumerate(blobs):
            sess.register_device_chunk(c, b)
        for t in range(10):
            sess.build_table([[0, 1, 2], [t % 3], [2, 0]])
            for layer in range(L):
                sess.prefill(layer, q, k, k, want_lse=False)
            sess.advance(5)
            for _ in range(2):
                for layer in range(L):
                    sess.decode(layer, q1[:, 0], k1[:, 0], k1[:, 0])
                sess.advance(1)
        assert sess.status() == 0
        sess.close()

    cycle(0)
    cycle(1)
    torch.cuda.synchronize()
    free0, _ = torch.cuda.mem_get_info()
    for i in range(150):
        cycle(i)
    torch.cuda.synchronize()
    free1, _ = torch.cuda.mem_get_info()
    assert free0 - free1 < 8 << 20, f"{(free0 - free1) / 2**20:.1f} MiB of device memory did not come back"


def test_two_host_threads_with_a_context_each():
    """Contexts are independent: two host threads, each with a context, tables and launches of its own, run at the
    same time (the binding releases the interpreter lock inside the library); every output of both is compared with
    the oracle.  (Calls on ONE context from several threads must be serialised by the caller.)"""
    import threading
    from test_gpu_parity import run_requests
    errors = []

    def worker(seed, impl):
        try:
            for rep in range(3):
                run_requests(2, 8, 2, 128, [[130, 64], [200]], 40, 3, seed=seed + rep, prefill_impl=impl, all_layers=bool(rep & 1))
                run_requests(1, 8, 4, 64, [[0, 1], [1]], 3, 2, seed=seed + 10 + rep, pool=[70, 33], decode_impl=2)
        except BaseException as e:   # noqa: BLE001 - reported by the main thread
            errors.append(e)

    threads = [threading.Thread(target=worker, args=(700, 2)), threading.Thread(target=worker, args=(800, 0))]
    for t in threads:
        t.start()
    for t in threads:
        t.join()
    assert not errors, errors


def test_attend_after_graph_replays_needs_the_tail_length_set_again():
    """A captured decode step advances the device-side tail counter every time it is replayed, but the host-side copy
    only when it was captured.  An attend call outside a capture splits its work by the host-side copy and checks it
    against the device counter: after replays it reports MATKV_E_BOUNDS in the device status unless the tail length
    has been set again; after matkv_table_set_tail_len the same call is right (compared with the oracle)."""
    import oracle
    from _util import check
    mk, Session, bits_to_dev, dev_to_bits = _mk()
    L, Hq, Hkv, D, B = 1, 8, 2, 128, 1
    blob = rand_bits(95, 0, (L, 2, Hkv, 150, D))
    sess = Session(L, Hq, Hkv, D, B, 1, 16)
    mk.matkv_set_option(sess.ctx, mk.OPT_CLUSTER_DECODE, 0)     # the streaming kernel (the cluster kernel never splits by the host's copy)
    sess.register_device_chunk(0, bits_to_dev(blob))
    sess.build_table([[0]])
    qs = [rand_bits(95, 10 + i, (B, Hq, D)) for i in range(4)]
    ks = [rand_bits(95, 20 + i, (B, Hkv, D)) for i in range(4)]
    g_q, g_k = bits_to_dev(qs[0]).clone(), bits_to_dev(ks[0]).clone()
    g_o = torch.empty_like(g_q)
    stream = torch.cuda.Stream()
    sp = stream.cuda_stream
    with torch.cuda.stream(stream):
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph, stream=stream):
            mk.matkv_attend_decode(sess.ctx, sess.table, 0, g_q.data_ptr(), g_k.data_ptr(), g_k.data_ptr(), g_o.data_ptr(), None, sp)
            mk.matkv_table_advance(sess.table, 1, sp)
        mk.matkv_table_set_tail_len(sess.table, 0, sp)          # the capture moved the host-side copy only
        for i in range(3):                                      # three replayed steps: the device counter is at 3
            g_q.copy_(bits_to_dev(qs[i])); g_k.copy_(bits_to_dev(ks[i]))
            graph.replay()
        q3, k3 = bits_to_dev(qs[3]), bits_to_dev(ks[3])
        out = torch.empty_like(q3)
        mk.matkv_attend_decode(sess.ctx, sess.table, 0, q3.data_ptr(), k3.data_ptr(), k3.data_ptr(), out.data_ptr(), None, sp)
        stream.synchronize()
        assert sess.status(clear=True) == mk.E_BOUNDS
        mk.matkv_table_set_tail_len(sess.table, 3, sp)
        lse = torch.empty((B, Hq), dtype=torch.float32, device="cuda")
        mk.matkv_attend_decode(sess.ctx, sess.table, 0, q3.data_ptr(), k3.data_ptr(), k3.data_ptr(), out.data_ptr(), lse.data_ptr(), sp)
        stream.synchronize()
    assert sess.status() == 0
    req = oracle.Request(oracle.Shape(L, Hq, Hkv, D), [blob], 16)
    for i in range(3):
        req.append_only(0, ks[i][0][None], ks[i][0][None])
        req.advance(1)
    o_ref, l_ref = req.attend_new(0, qs[3][0][None], ks[3][0][None], ks[3][0][None])
    check(dev_to_bits(out)[0], o_ref[0], lse.cpu().numpy()[0], l_ref[0], "decode after replays, tail length set again")
    sess.close()


def test_pageable_host_blob_is_staged_by_the_copy_engine_even_with_the_copy_kernel_on():
    """The copy kernel reads host blobs over the link, which only page-locked memory allows.  A pageable blob
    (an ordinary numpy array) must therefore never reach it: it is staged by the copy engine instead."""
    mk, Session, to_dev, to_bits = _mk()
    L, Hq, Hkv, D, n = 1, 4, 2, 64, 200
    sess = Session(L, Hq, Hkv, D, 1, 2, 4)
    mk.matkv_set_option(sess.ctx, mk.OPT_STAGE_CTAS, 4)
    pageable = np.ascontiguousarray(rand_bits(46, 0, (L, 2, Hkv, n, D)))       # ordinary host memory
    assert pageable.ctypes.data % 16 == 0
    mk.matkv_register_chunk(sess.ctx, 0, n, pageable.ctypes.data, None)
    pinned = sess.register_host_chunk(1, rand_bits(46, 1, (L, 2, Hkv, n, D)))  # this one goes through the copy kernel
    slot_bytes = pageable.nbytes
    slots = torch.zeros(2 * slot_bytes, dtype=torch.uint8, device="cuda")
    tk = sess.stage([0, 1], slots, slot_bytes, torch.cuda.Stream())
    mk.matkv_stage_wait(sess.ctx, tk)
    sess.build_table([[0, 1]])
    k, v = sess.gather(0, 0, 2 * n)
    assert np.array_equal(to_bits(k)[:, :n], pageable[0, 0]) and np.array_equal(to_bits(v)[:, :n], pageable[0, 1])
    assert np.array_equal(to_bits(k)[:, n:], to_bits(pinned)[0, 0])
    assert sess.status() == 0
    sess.close()


def test_staging_tickets_are_retired_so_a_long_serving_loop_stays_bounded():
    """Every staging call creates an event; a server stages a batch per step for ever.  Finished calls must give
    their events back (seen complete by a query, a wait or simply by the next staging call), and a retired ticket
    keeps answering."""
    mk, Session, to_dev, to_bits = _mk()
    L, Hq, Hkv, D, n = 1, 4, 2, 64, 64
    sess = Session(L, Hq, Hkv, D, 1, 2, 4)
    blobs = [rand_bits(47, i, (L, 2, Hkv, n, D)) for i in range(4)]
    for i, b in enumerate(blobs):
        sess.register_host_chunk(i, b)
    slot_bytes = blobs[0].nbytes
    regions = [torch.empty(2 * slot_bytes, dtype=torch.uint8, device="cuda") for _ in range(2)]
    copy = torch.cuda.Stream()
    tickets = []
    for step in range(300):
        pair = [(2 * step) % 4, (2 * step + 1) % 4]
        tickets.append(sess.stage(pair, regions[step % 2], slot_bytes, copy))
        sess.build_table([pair])                               # never queries or waits for a ticket
        if step % 50 == 49:
            torch.cuda.synchronize()
            assert mk.matkv_stage_pending(sess.ctx) == 0       # everything finished has been retired
    assert mk.matkv_stage_pending(sess.ctx) <= 2
    k, v = sess.gather(0, 0, 2 * n)                            # the last table still reads the right bytes
    assert np.array_equal(to_bits(k), np.concatenate([blobs[2][0, 0], blobs[3][0, 0]], axis=1))
    for tk in (tickets[0], tickets[150], tickets[-1]):
        mk.matkv_stage_wait(sess.ctx, tk)                      # retired tickets answer as finished
        assert mk.matkv_stage_query(sess.ctx, tk)
    with pytest.raises(mk.MatkvError):
        mk.matkv_stage_query(sess.ctx, tickets[-1] + 1000)     # a number never handed out
    assert sess.status() == 0
    sess.close()


def test_storage_read_failures_reach_the_attention_path(tmp_path):
    """Failures injected on the host, no GPU fault anywhere: (1) a chunk file truncated after registration makes the
    read come back short; (2) reads delayed beyond the time limit make the copy stream give up on them.  Either way
    the wait reports MATKV_E_IO, a table over such a chunk is refused, and the device status word reads MATKV_E_IO
    for work queued behind the staging call without any host wait; the context stays usable afterwards."""
    import os
    mk, Session, to_dev, to_bits = _mk()
    L, Hq, Hkv, D, n = 1, 4, 2, 64, 64
    blobs = [rand_bits(48, i, (L, 2, Hkv, n, D)) for i in range(3)]
    slot_bytes = (blobs[0].nbytes + 4095) // 4096 * 4096

    def fresh():
        sess = Session(L, Hq, Hkv, D, 1, 3, 4)
        for i, b in enumerate(blobs):
            with open(tmp_path / f"{i}.kv", "wb") as f:
                f.write(b.tobytes())
            mk.matkv_register_chunk_file(sess.ctx, i, n, str(tmp_path / f"{i}.kv"))
        ring = torch.empty(2 * slot_bytes + 4096, dtype=torch.uint8, pin_memory=True)
        base = (ring.data_ptr() + 4095) // 4096 * 4096
        mk.matkv_set_bounce_buffer(sess.ctx, base, 2 * slot_bytes, slot_bytes, 2)
        slots = torch.zeros(3 * slot_bytes, dtype=torch.uint8, device="cuda")
        return sess, ring, slots

    # (1) short file
    sess, ring, slots = fresh()
    os.truncate(tmp_path / "1.kv", blobs[1].nbytes // 2)
    copy = torch.cuda.Stream()
    tk = sess.stage([0, 1, 2], slots, slot_bytes, copy)
    try:                                                        # usually too early for the host to know of the failure
        table = mk.matkv_build_chunk_table(sess.ctx, [[0, 1, 2]], sess.tail_k.data_ptr(), sess.tail_v.data_ptr())
    except mk.MatkvError as e:
        assert e.code == mk.E_IO
        table = None
    torch.cuda.synchronize()
    assert sess.status(clear=True) == mk.E_IO                   # flagged behind the copies, no host wait needed
    if table:
        mk.matkv_table_free(table)
    with pytest.raises(mk.MatkvError) as e:
        mk.matkv_stage_wait(sess.ctx, tk)
    assert e.value.code == mk.E_IO
    with pytest.raises(mk.MatkvError) as e:
        mk.matkv_stage_query(sess.ctx, tk)                      # the retired ticket remembers
    assert e.value.code == mk.E_IO
    with pytest.raises(mk.MatkvError) as e:
        sess.build_table([[0, 1, 2]])                           # now the failure is known: refused
    assert e.value.code == mk.E_IO
    sess.close()
    del ring

    # (2) reads that take longer than the stream is willing to wait
    sess, ring, slots = fresh()
    mk.matkv_set_option(sess.ctx, mk.OPT_IO_TIMEOUT_MS, 50)
    mk.matkv_set_option(sess.ctx, mk.OPT_IO_TEST_DELAY_MS, 400)
    tk = sess.stage([0], slots, slot_bytes, copy)
    with pytest.raises(mk.MatkvError) as e:
        mk.matkv_stage_wait(sess.ctx, tk)
    assert e.value.code == mk.E_IO
    assert sess.status(clear=True) == mk.E_IO
    # the late read returns, the slab is free again, and the same context stages the chunk properly
    mk.matkv_set_option(sess.ctx, mk.OPT_IO_TEST_DELAY_MS, 0)
    mk.matkv_set_option(sess.ctx, mk.OPT_IO_TIMEOUT_MS, 30000)
    slots2 = torch.zeros(3 * slot_bytes, dtype=torch.uint8, device="cuda")
    tk = sess.stage([0, 2], slots2, slot_bytes, copy)
    mk.matkv_stage_wait(sess.ctx, tk)
    sess.build_table([[2, 0]])
    k, v = sess.gather(0, 0, 2 * n)
    assert np.array_equal(to_bits(k), np.concatenate([blobs[2][0, 0], blobs[0][0, 0]], axis=1))
    assert sess.status() == 0                                   # a staging call that went well does not inherit the earlier failure
    sess.close()
    del ring


def test_p9_rotary_position_base_given_by_the_caller():
    """pos_mode 2: the position of every request's first tail token is whatever the caller says."""
    import oracle
    from _util import check
    mk, Session, to_dev, to_bits = _mk()
    L, Hq, Hkv, D, S = 1, 8, 2, 128, 6
    theta = 500000.0
    sess = Session(L, Hq, Hkv, D, 2, 2, S + 2, rope_theta=theta, pos_mode=2)
    blobs = [rand_bits(54, i, (L, 2, Hkv, n, D)) for i, n in enumerate([100, 30])]
    for i, b in enumerate(blobs):
        sess.register_device_chunk(i, b)
    ids = [[0, 1], [1]]
    bases = [7, 4096]
    sess.build_table(ids)
    mk.matkv_table_set_pos_base(sess.table, bases)
    sh = oracle.Shape(L, Hq, Hkv, D)
    reqs = [oracle.Request(sh, [blobs[c] for c in row], S + 2, rope_theta=theta, pos_base=bases[r]) for r, row in enumerate(ids)]
    q, k, v = rand_bits(54, 10, (2, S, Hq, D)), rand_bits(54, 11, (2, S, Hkv, D)), rand_bits(54, 12, (2, S, Hkv, D))
    out, lse = sess.prefill(0, to_dev(q), to_dev(k), to_dev(v))
    for r in range(2):
        o_ref, l_ref = reqs[r].attend_new(0, q[r], k[r], v[r])
        check(to_bits(out)[r], o_ref, lse.cpu().numpy()[r], l_ref, f"caller-given base, prefill request {r}")
        reqs[r].advance(S)
    sess.advance(S)
    q, k, v = rand_bits(54, 20, (2, Hq, D)), rand_bits(54, 21, (2, Hkv, D)), rand_bits(54, 22, (2, Hkv, D))
    out, lse = sess.decode(0, to_dev(q), to_dev(k), to_dev(v))
    for r in range(2):
        o_ref, l_ref = reqs[r].attend_new(0, q[r][None], k[r][None], v[r][None])
        check(to_bits(out)[r], o_ref[0], lse.cpu().numpy()[r], l_ref[0], f"caller-given base, decode request {r}")
    tk = to_bits(sess.tail_k)
    for r in range(2):                                          # the rotated keys in the tail match bit for bit
        assert np.array_equal(tk[r, :, :, :S + 1], reqs[r].tail_k[:, :, :S + 1])
    # a context in another mode refuses the call
    other = Session(L, Hq, Hkv, D, 1, 1, 4, rope_theta=theta)
    other.register_device_chunk(0, blobs[0])
    other.build_table([[0]])
    with pytest.raises(mk.MatkvError):
        mk.matkv_table_set_pos_base(other.table, [5])
    other.close()
    assert sess.status() == 0
    sess.close()
