"""GPU parity: the CUDA path, called through the C ABI, against the CPU oracle element by element."""
import math

import numpy as np
import pytest
import torch

import matkv_inputs as mi
import oracle
from _util import check, rand_bits

pytestmark = pytest.mark.gpu


def _session(L, Hq, Hkv, D, B, max_chunks, max_tail, **kw):
    from paper_2512_22195_b200.harness import Session
    return Session(L, Hq, Hkv, D, B, max_chunks, max_tail, **kw)


def _dev(a):
    from paper_2512_22195_b200.harness import bits_to_dev
    return bits_to_dev(a)


def _bits(t):
    from paper_2512_22195_b200.harness import dev_to_bits
    return dev_to_bits(t)


def run_requests(L, Hq, Hkv, D, lens_per_req, S, T, seed, ctas=0, all_layers=False, q_shift=0, cap=None,
                 prefill_impl=0, prefill_ctas=0, rope_theta=0.0, pos_mode=0, fused_advance=False, pool=None,
                 decode_impl=0, share_tiles=0, cluster=None):
    """Prefill S tokens then T decode steps for a batch; compare every output with the oracle.
    lens_per_req: chunk lengths per request (every chunk its own), or, with `pool` (a list of chunk lengths),
    indices into the pool per request, so that requests can list the same chunk."""
    import paper_2512_22195_b200 as mk
    B = len(lens_per_req)
    cap = cap or (S + T)
    sess = _session(L, Hq, Hkv, D, B, max(1, max(len(x) for x in lens_per_req)), cap, rope_theta=rope_theta, pos_mode=pos_mode)
    if decode_impl:
        mk.matkv_set_option(sess.ctx, mk.OPT_DECODE_IMPL, decode_impl)
    if cluster is not None:
        mk.matkv_set_option(sess.ctx, mk.OPT_CLUSTER_DECODE, cluster)
    if share_tiles:
        mk.matkv_set_option(sess.ctx, mk.OPT_SHARE_TILES, share_tiles)
    if ctas:
        mk.matkv_set_option(sess.ctx, mk.OPT_DECODE_CTAS, ctas)
    if prefill_impl:
        mk.matkv_set_option(sess.ctx, mk.OPT_PREFILL_IMPL, prefill_impl)
    if prefill_ctas:
        mk.matkv_set_option(sess.ctx, mk.OPT_PREFILL_CTAS, prefill_ctas)
    if fused_advance:
        mk.matkv_set_option(sess.ctx, mk.OPT_DECODE_ADVANCES_TAIL, 1)
    sh = oracle.Shape(L, Hq, Hkv, D)
    blobs, ids, cid = {}, [], 0
    if pool is not None:
        for cid, n in enumerate(pool):
            blobs[cid] = rand_bits(seed, 1000 + cid, (L, 2, Hkv, n, D))
            sess.register_device_chunk(cid, blobs[cid])
        ids = [list(row) for row in lens_per_req]
    else:
        for r, lens in enumerate(lens_per_req):
            row = []
            for n in lens:
                blobs[cid] = rand_bits(seed, 1000 + cid, (L, 2, Hkv, n, D))
                sess.register_device_chunk(cid, blobs[cid])
                row.append(cid)
                cid += 1
            ids.append(row)
    sess.build_table(ids)
    def pos_base(row):
        lens = [blobs[c].shape[3] for c in row]
        return None if pos_mode == 0 else max(lens, default=0)
    reqs = [oracle.Request(sh, [blobs[c] for c in row], cap, rope_theta=rope_theta, pos_base=pos_base(row)) for row in ids]
    worst = [0.0, 0.0, 0.0]

    def upd(m):
        for i in range(3):
            worst[i] = max(worst[i], m[i])

    if S > 0:
        qs = [rand_bits(seed, 10 + layer, (B, S, Hq, D), q_shift) for layer in range(L)]
        ks = [rand_bits(seed, 40 + layer, (B, S, Hkv, D)) for layer in range(L)]
        vs = [rand_bits(seed, 70 + layer, (B, S, Hkv, D)) for layer in range(L)]
        if all_layers:      # one launch for the sub-prefill of every layer
            out_all, lse_all = sess.prefill_all_layers(_dev(np.stack(qs)), _dev(np.stack(ks)), _dev(np.stack(vs)))
            ob_all, lb_all = _bits(out_all), lse_all.cpu().numpy()
        for layer in range(L):
            q, k, v = qs[layer], ks[layer], vs[layer]
            if all_layers:
                ob, lb = ob_all[layer], lb_all[layer]
            else:
                out, lse = sess.prefill(layer, _dev(q), _dev(k), _dev(v))
                ob, lb = _bits(out), lse.cpu().numpy()
            for r in range(B):
                o_ref, l_ref = reqs[r].attend_new(layer, q[r], k[r], v[r])
                upd(check(ob[r], o_ref, lb[r], l_ref, f"prefill layer {layer} req {r}"))
        sess.advance(S)
        for r in reqs:
            r.advance(S)
    for t in range(T):
        q = rand_bits(seed, 2000 + t, (L, B, Hq, D), q_shift)
        k = rand_bits(seed, 3000 + t, (L, B, Hkv, D))
        v = rand_bits(seed, 4000 + t, (L, B, Hkv, D))
        qd, kd, vd = _dev(q), _dev(k), _dev(v)
        if all_layers:
            out, lse = sess.decode_all_layers(qd, kd, vd)
            ob, lb = _bits(out), lse.cpu().numpy()
        else:
            outs = [sess.decode(layer, qd[layer], kd[layer], vd[layer]) for layer in range(L)]
            ob = np.stack([_bits(o) for o, _ in outs])
            lb = np.stack([l.cpu().numpy() for _, l in outs])
        for layer in range(L):
            for r in range(B):
                o_ref, l_ref = reqs[r].attend_new(layer, q[layer, r][None], k[layer, r][None], v[layer, r][None])
                upd(check(ob[layer, r], o_ref[0], lb[layer, r], l_ref[0], f"decode step {t} layer {layer} req {r}"))
        if not (fused_advance and all_layers):
            sess.advance(1)
        for r in reqs:
            r.advance(1)
    # the tails the kernels wrote must equal the oracle's bookkeeping bit for bit
    tk, tv = _bits(sess.tail_k), _bits(sess.tail_v)
    for r in range(B):
        n = reqs[r].tail_len
        assert np.array_equal(tk[r, :, :, :n], reqs[r].tail_k[:, :, :n]) and np.array_equal(tv[r, :, :, :n], reqs[r].tail_v[:, :, :n])
    assert sess.status() == 0
    sess.close()
    return worst


def test_cfg1_full():
    """Config 1: 1 layer, 8 q heads / 2 kv heads, D=64, 2 chunks x 128, 16-token suffix, 8 decode steps."""
    w = mi.workload("cfg1")
    run_requests(w.n_layers, w.n_q_heads, w.n_kv_heads, w.head_dim, [[128, 128]], w.suffix, w.decode_steps, seed=0)


@pytest.mark.parametrize("Hq,Hkv,D", [(8, 2, 64), (4, 4, 128), (8, 4, 128), (32, 8, 128), (64, 8, 128), (8, 1, 64), (2, 2, 64)])
def test_head_shapes(Hq, Hkv, D):
    run_requests(2, Hq, Hkv, D, [[40, 7], [129]], 5, 3, seed=21)


@pytest.mark.parametrize("lens", [[[1]], [[7, 127, 129, 1000]], [[]], [[33], [], [1, 1, 1]], [[64, 64], [32]]])
def test_ragged_chunks_and_empty_lists(lens):
    run_requests(1, 8, 2, 64, lens, 3, 4, seed=22)


def test_tail_crosses_tile_boundaries():
    run_requests(1, 4, 2, 128, [[50]], 30, 40, seed=23)           # tail grows through 32 and 64


def test_all_layers_launch_matches_oracle():
    run_requests(3, 8, 2, 128, [[200, 31], [97]], 4, 3, seed=24, all_layers=True)


@pytest.mark.parametrize("S,impl", [(40, 2), (70, 3), (5, 1)])
def test_all_layers_prefill_launch(S, impl):
    run_requests(3, 32, 8, 128, [[200, 31], [97]], S, 2, seed=27, all_layers=True, prefill_impl=impl)


@pytest.mark.parametrize("ctas", [0, 3, 1000])
def test_decode_launch_that_advances_the_tail_itself(ctas):
    run_requests(2, 8, 2, 128, [[200, 31], [97], []], 3, 5, seed=28, all_layers=True, fused_advance=True, ctas=ctas)


def test_decode_launch_that_advances_the_tail_itself_single_layer_model():
    """With one layer the all-layers launch is a one-layer launch: it must still advance the tail (such a launch stays
    with the streaming kernel, whose last CTA moves the counter)."""
    run_requests(1, 8, 2, 128, [[200, 31], [97]], 3, 5, seed=30, all_layers=True, fused_advance=True)


@pytest.mark.parametrize("decode_impl,L,lens", [(1, 2, [[130, 64], [200], [64]]), (1, 32, [[1024, 1024, 512]]), (2, 2, [[130, 64], [200], [64]])])
def test_back_to_back_decode_launches_across_a_tail_tile_boundary(decode_impl, L, lens):
    """Twelve decode steps issued back to back WITHOUT a host synchronisation in between, every launch advancing the
    tail itself, while the tail grows from 58 to 70 tokens (a second tail tile appears at 64): each launch is split
    by the host's copy of the tail length and starts under its predecessor's tail (its producer already fetching
    chunk tiles), and each step's appended row must be there for the next.  All outputs are compared afterwards."""
    import paper_2512_22195_b200 as mk
    Hq, Hkv, D, S, T, seed = 8, 2, 128, 58, 12, 29
    B = len(lens)
    sess = _session(L, Hq, Hkv, D, B, max(len(x) for x in lens), S + T)
    mk.matkv_set_option(sess.ctx, mk.OPT_DECODE_IMPL, decode_impl)
    mk.matkv_set_option(sess.ctx, mk.OPT_DECODE_ADVANCES_TAIL, 1)
    sh = oracle.Shape(L, Hq, Hkv, D)
    reqs, ids, cid = [], [], 0
    for row in lens:
        blobs, mine = [], []
        for n in row:
            bl = rand_bits(seed, 100 + cid, (L, 2, Hkv, n, D))
            sess.register_device_chunk(cid, _dev(bl))
            blobs.append(bl); mine.append(cid); cid += 1
        reqs.append(oracle.Request(sh, blobs, S + T)); ids.append(mine)
    sess.build_table(ids)
    q = rand_bits(seed, 1, (L, B, S, Hq, D)); k = rand_bits(seed, 2, (L, B, S, Hkv, D)); v = rand_bits(seed, 3, (L, B, S, Hkv, D))
    sess.prefill_all_layers(_dev(q), _dev(k), _dev(v), want_lse=False)
    for layer in range(L):
        for r in range(B):
            reqs[r].append_only(layer, k[layer, r], v[layer, r])
    sess.advance(S)
    for r in reqs:
        r.advance(S)
    qs = [rand_bits(seed, 2000 + t, (L, B, Hq, D)) for t in range(T)]
    ks = [rand_bits(seed, 3000 + t, (L, B, Hkv, D)) for t in range(T)]
    vs = [rand_bits(seed, 4000 + t, (L, B, Hkv, D)) for t in range(T)]
    dq, dk, dv = [_dev(x) for x in qs], [_dev(x) for x in ks], [_dev(x) for x in vs]
    torch.cuda.synchronize()
    outs = [sess.decode_all_layers(dq[t], dk[t], dv[t]) for t in range(T)]      # nothing in between: the launches queue up
    torch.cuda.synchronize()
    assert sess.status() == 0
    sample_layers = sorted({0, L // 2, L - 1})
    for t in range(T):
        ob, lb = _bits(outs[t][0]), outs[t][1].cpu().numpy()
        for layer in range(L):
            for r in range(B):
                if layer in sample_layers:
                    o_ref, l_ref = reqs[r].attend_new(layer, qs[t][layer, r][None], ks[t][layer, r][None], vs[t][layer, r][None])
                    check(ob[layer, r], o_ref[0], lb[layer, r], l_ref[0], f"step {t} layer {layer} request {r}")
                else:
                    reqs[r].append_only(layer, ks[t][layer, r][None], vs[t][layer, r][None])
        for r in reqs:
            r.advance(1)
    tk, tv = _bits(sess.tail_k), _bits(sess.tail_v)
    for r in range(B):
        n = reqs[r].tail_len
        assert n == S + T
        assert np.array_equal(tk[r, :, :, :n], reqs[r].tail_k[:, :, :n]) and np.array_equal(tv[r, :, :, :n], reqs[r].tail_v[:, :, :n])
    sess.close()


# ---- per-layer decode of small batches as thread-block clusters ----------------------------------------
@pytest.mark.parametrize("Hq,Hkv,D,lens", [
    (32, 8, 128, [[1024, 1024, 512]]),                 # 8 units: clusters of 16 CTAs (42 tiles per unit)
    (8, 2, 128, [[300, 77], [129]]),                   # 4 units, unequal requests
    (64, 8, 128, [[200, 64]]),                         # G = 8: clusters of 8 at most (landing zone rows)
    (8, 2, 64, [[128, 128]]),                          # D = 64
    (4, 4, 128, [[65, 1, 64], [], [7]]),               # G = 1; a request without chunks; shares without any tile
    (16, 2, 128, [[33]]),                              # fewer tiles than a full cluster
    (8, 8, 64, [[500], [40, 40], [64], [1]]),          # 32 units: clusters of up to 9
    (8, 8, 64, [[70, 3]] * 33),                        # 264 units: one CTA each, both CTA places of every SM taken
    (16, 4, 128, [[130], [64, 64], []] * 7),           # 84 units in clusters of 3, ragged requests, some without chunks
])
def test_cluster_decode_matches_the_oracle(Hq, Hkv, D, lens):
    """decode_impl 1 + cluster 2 forces the cluster kernel wherever the launch fits it; the tail grows through a tile
    boundary (suffix of 60 tokens, 8 steps); sharper queries (scaled by 2) in a second pass."""
    run_requests(2, Hq, Hkv, D, lens, 60, 8, seed=81, decode_impl=1, cluster=2)
    run_requests(1, Hq, Hkv, D, lens, 3, 2, seed=82, decode_impl=1, cluster=2, q_shift=1)


def test_cluster_decode_replayed_from_a_graph_while_the_tail_grows():
    """One decode step (a launch per layer, then the tail counter) captured when the tail holds 60 tokens and replayed
    twelve times: the shares were balanced for one tail tile, the tail grows into a second one, and every replayed
    launch must still see exactly its tail (the kernel places tail tiles by the device's counter) and start its chunk
    loads under its predecessor's tail.  Every step against the oracle; the tails bit for bit."""
    import paper_2512_22195_b200 as mk
    L, Hq, Hkv, D, S, T, seed = 3, 32, 8, 128, 60, 12, 83
    lens = [1024, 300]
    sess = _session(L, Hq, Hkv, D, 1, 2, S + T)
    blobs = [rand_bits(seed, 100 + i, (L, 2, Hkv, n, D)) for i, n in enumerate(lens)]
    for i, b in enumerate(blobs):
        sess.register_device_chunk(i, b)
    sess.build_table([[0, 1]])
    req = oracle.Request(oracle.Shape(L, Hq, Hkv, D), blobs, S + T)
    q, k, v = rand_bits(seed, 1, (L, 1, S, Hq, D)), rand_bits(seed, 2, (L, 1, S, Hkv, D)), rand_bits(seed, 3, (L, 1, S, Hkv, D))
    sess.prefill_all_layers(_dev(q), _dev(k), _dev(v), want_lse=False)
    for layer in range(L):
        req.append_only(layer, k[layer, 0], v[layer, 0])
    sess.advance(S)
    req.advance(S)
    qs = [rand_bits(seed, 2000 + t, (L, 1, Hq, D)) for t in range(T)]
    ks = [rand_bits(seed, 3000 + t, (L, 1, Hkv, D)) for t in range(T)]
    vs = [rand_bits(seed, 4000 + t, (L, 1, Hkv, D)) for t in range(T)]
    g_q, g_k, g_v = _dev(qs[0]).clone(), _dev(ks[0]).clone(), _dev(vs[0]).clone()
    g_o = torch.empty_like(g_q)
    g_l = torch.empty((L, 1, Hq), dtype=torch.float32, device="cuda")
    stream = torch.cuda.Stream()
    sp = stream.cuda_stream
    outs = []
    with torch.cuda.stream(stream):
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph, stream=stream):
            for layer in range(L):
                mk.matkv_attend_decode(sess.ctx, sess.table, layer, g_q[layer].data_ptr(), g_k[layer].data_ptr(), g_v[layer].data_ptr(),
                                       g_o[layer].data_ptr(), g_l[layer].data_ptr(), sp)
            mk.matkv_table_advance(sess.table, 1, sp)
        mk.matkv_table_set_tail_len(sess.table, S, sp)          # the capture ran nothing but moved the host-side mirror
        for t in range(T):
            g_q.copy_(_dev(qs[t])); g_k.copy_(_dev(ks[t])); g_v.copy_(_dev(vs[t]))
            graph.replay()
            outs.append((g_o.clone(), g_l.clone()))
        stream.synchronize()
    assert sess.status() == 0
    for t in range(T):
        ob, lb = _bits(outs[t][0]), outs[t][1].cpu().numpy()
        for layer in range(L):
            o_ref, l_ref = req.attend_new(layer, qs[t][layer, 0][None], ks[t][layer, 0][None], vs[t][layer, 0][None])
            check(ob[layer, 0], o_ref[0], lb[layer, 0], l_ref[0], f"replayed step {t} layer {layer}")
        req.advance(1)
    tk, tv = _bits(sess.tail_k), _bits(sess.tail_v)
    assert np.array_equal(tk[0, :, :, :S + T], req.tail_k[:, :, :S + T]) and np.array_equal(tv[0, :, :, :S + T], req.tail_v[:, :, :S + T])
    sess.close()


def test_cluster_decode_long_replay_never_reads_a_tile_before_it_has_landed():
    """The benchmark's per-layer mode at the Llama-3-8B head shape: 5 x 1,024-token chunks, a decode step of 8
    per-layer launches captured once and replayed 128 times while the tail grows from 64 to 192 tokens (one, two, then
    three tail tiles against shares balanced for one).  The two groups of consumer warps of a CTA reach a ring stage at
    different times, so a stage's fill number has to be checked before its barrier phase: thousands of back-to-back
    launches must leave the status word clean (a consumer that ran ahead would end in a bounded wait running out), and
    sampled steps must match the oracle."""
    import paper_2512_22195_b200 as mk
    L, Hq, Hkv, D, S, T, seed = 8, 32, 8, 128, 64, 128, 84
    sess = _session(L, Hq, Hkv, D, 1, 5, S + T)
    blobs = [rand_bits(seed, 100 + i, (L, 2, Hkv, 1024, D)) for i in range(5)]
    for i, b in enumerate(blobs):
        sess.register_device_chunk(i, b)
    sess.build_table([list(range(5))])
    req = oracle.Request(oracle.Shape(L, Hq, Hkv, D), blobs, S + T)
    q, k, v = rand_bits(seed, 1, (L, 1, S, Hq, D)), rand_bits(seed, 2, (L, 1, S, Hkv, D)), rand_bits(seed, 3, (L, 1, S, Hkv, D))
    sess.prefill_all_layers(_dev(q), _dev(k), _dev(v), want_lse=False)
    for layer in range(L):
        req.append_only(layer, k[layer, 0], v[layer, 0])
    sess.advance(S)
    req.advance(S)
    qs = rand_bits(seed, 2000, (T, L, 1, Hq, D))
    ks = rand_bits(seed, 3000, (T, L, 1, Hkv, D))
    vs = rand_bits(seed, 4000, (T, L, 1, Hkv, D))
    dq, dk, dv = _dev(qs), _dev(ks), _dev(vs)
    g_q, g_k, g_v = dq[0].clone(), dk[0].clone(), dv[0].clone()
    g_o = torch.empty_like(g_q)
    outs = torch.empty_like(dq)
    stream = torch.cuda.Stream()
    sp = stream.cuda_stream
    with torch.cuda.stream(stream):
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph, stream=stream):
            for layer in range(L):
                mk.matkv_attend_decode(sess.ctx, sess.table, layer, g_q[layer].data_ptr(), g_k[layer].data_ptr(), g_v[layer].data_ptr(),
                                       g_o[layer].data_ptr(), None, sp)
            mk.matkv_table_advance(sess.table, 1, sp)
        mk.matkv_table_set_tail_len(sess.table, S, sp)
        for t in range(T):
            g_q.copy_(dq[t], non_blocking=True); g_k.copy_(dk[t], non_blocking=True); g_v.copy_(dv[t], non_blocking=True)
            graph.replay()
            outs[t].copy_(g_o, non_blocking=True)
        stream.synchronize()
    assert sess.status() == 0
    ob = _bits(outs)
    for t in range(T):
        for layer in range(L):
            if t in (0, 1, 63, 64, 127) and layer in (0, L - 1):
                o_ref, _ = req.attend_new(layer, qs[t, layer, 0][None], ks[t, layer, 0][None], vs[t, layer, 0][None])
                check(ob[t, layer, 0], o_ref[0], None, None, f"replayed step {t} layer {layer}")
            else:
                req.append_only(layer, ks[t, layer, 0][None], vs[t, layer, 0][None])
        req.advance(1)
    tk = _bits(sess.tail_k)
    assert np.array_equal(tk[0, :, :, :S + T], req.tail_k[:, :, :S + T])
    sess.close()


def test_peaky_queries():
    run_requests(1, 8, 2, 128, [[300, 300]], 8, 4, seed=25, q_shift=3)   # q scaled by 8: sharp softmax


@pytest.mark.parametrize("ctas", [1, 2, 3, 7, 0])
def test_p7_split_count_invariance(ctas):
    run_requests(2, 8, 2, 128, [[500, 77, 260]], 2, 3, seed=26, ctas=ctas)


def test_p7_combine_kernel_alone():
    import paper_2512_22195_b200 as mk
    sess = _session(1, 8, 2, 64, 1, 1, 8)
    rng = np.random.default_rng(3)
    for n_rows, P, D in [(5, 1, 64), (9, 7, 128), (3, 40, 128), (2, 33, 32)]:
        o_parts = rng.normal(size=(n_rows, P, D)).astype(np.float32)
        lse_parts = (rng.normal(size=(n_rows, P)) * 4).astype(np.float32)
        lse_parts[0, 0] = -np.inf
        if P > 1:
            lse_parts[1, :] = -np.inf
            lse_parts[1, 1] = 0.5
        op, lp = torch.from_numpy(o_parts).cuda(), torch.from_numpy(lse_parts).cuda()
        out = torch.empty((n_rows, D), dtype=torch.bfloat16, device="cuda")
        lse = torch.empty(n_rows, dtype=torch.float32, device="cuda")
        mk.matkv_lse_combine(sess.ctx, n_rows, P, D, op.data_ptr(), lp.data_ptr(), out.data_ptr(), lse.data_ptr())
        ob, lb = _bits(out), lse.cpu().numpy()
        for r in range(n_rows):
            o_ref, l_ref = oracle.lse_merge(o_parts[r].astype(np.float64), lse_parts[r].astype(np.float64))
            if np.isneginf(l_ref):
                assert np.all(ob[r] == 0) and np.isneginf(lb[r])
                continue
            o = mi.bf16_bits_to_f64(ob[r])
            assert np.max(np.abs(o - o_ref)) <= 2 ** -8 * max(1.0, np.max(np.abs(o_ref))) and abs(lb[r] - l_ref) <= 1e-4
    sess.close()


def test_p4_needle_on_gpu():
    """A planted dominant key at every segment edge, tile edge and the causal edge of the tail."""
    L, Hq, Hkv, D = 1, 4, 2, 128
    lens = [33, 64, 1, 95]
    sess = _session(L, Hq, Hkv, D, 1, 4, 40)
    seed, g, h = 31, 1, 3
    q = rand_bits(seed, 1, (1, Hq, D))
    qv = mi.bf16_bits_to_f64(q[0, h])
    needle = mi.f32_to_bf16_bits((qv * 16.0).astype(np.float32))
    blobs = [rand_bits(seed, 10 + i, (L, 2, Hkv, n, D)) for i, n in enumerate(lens)]
    spots = [(c, t) for c, n in enumerate(lens) for t in sorted({0, n - 1, min(31, n - 1), min(32, n - 1)})]
    k_new, v_new = rand_bits(seed, 2, (1, Hkv, D)), rand_bits(seed, 3, (1, Hkv, D))
    for trial, (c, t) in enumerate(spots):
        bl = [b.copy() for b in blobs]
        bl[c][0, 0, g, t] = needle
        for i, b in enumerate(bl):
            sess.register_device_chunk(100 * trial + i, b)
        sess.build_table([[100 * trial + i for i in range(4)]])
        out, _ = sess.decode(0, _dev(q), _dev(k_new), _dev(v_new))
        o = mi.bf16_bits_to_f64(_bits(out))[0, h]
        want = mi.bf16_bits_to_f64(bl[c][0, 1, g, t])
        assert np.max(np.abs(o - want)) <= 2 ** -7 * np.max(np.abs(want)) + 1e-6, (c, t)
    # needle as the new token itself (tail[v-1]) is visible (clean chunks: no other needle around)
    for i, b in enumerate(blobs):
        sess.register_device_chunk(9000 + i, b)
    sess.build_table([[9000 + i for i in range(4)]])
    kn = k_new.copy()
    kn[0, g] = needle
    out, _ = sess.decode(0, _dev(q), _dev(kn), _dev(v_new))
    o = mi.bf16_bits_to_f64(_bits(out))[0, h]
    want = mi.bf16_bits_to_f64(v_new[0, g])
    assert np.max(np.abs(o - want)) <= 2 ** -7 * np.max(np.abs(want)) + 1e-6
    # a needle sitting in the tail one past the visible range must not be seen
    sess.tail_k[0, 0, g, 1] = _dev(needle)
    out2, _ = sess.decode(0, _dev(q), _dev(k_new), _dev(v_new))
    sess.tail_k[0, 0, g, 1] = 0
    out3, _ = sess.decode(0, _dev(q), _dev(k_new), _dev(v_new))
    assert np.array_equal(_bits(out2), _bits(out3))
    sess.close()


def test_p5_p6_order_and_duplicates_on_gpu():
    L, Hq, Hkv, D = 1, 8, 2, 64
    sess = _session(L, Hq, Hkv, D, 3, 4, 8)
    seed = 32
    blobs = [rand_bits(seed, 10 + i, (L, 2, Hkv, n, D)) for i, n in enumerate([70, 33, 128])]
    for i, b in enumerate(blobs):
        sess.register_device_chunk(i, b)
    q = rand_bits(seed, 1, (3, Hq, D))
    q[1], q[2] = q[0], q[0]
    kn = np.repeat(rand_bits(seed, 2, (1, Hkv, D)), 3, axis=0)
    vn = np.repeat(rand_bits(seed, 3, (1, Hkv, D)), 3, axis=0)
    sess.build_table([[0, 1, 2], [2, 0, 1], [1, 2, 0]])
    out, lse = sess.decode(0, _dev(q), _dev(kn), _dev(vn))
    o, l = mi.bf16_bits_to_f64(_bits(out)), lse.cpu().numpy()
    assert np.max(np.abs(o[0] - o[1])) <= 2 ** -7 and np.max(np.abs(o[0] - o[2])) <= 2 ** -7
    assert np.max(np.abs(l[0] - l[1])) <= 1e-4 and np.max(np.abs(l[0] - l[2])) <= 1e-4
    # [A, A] against [A]: same o, lse larger by ln 2 -- compare through the oracle (the new token is also seen)
    sh = oracle.Shape(L, Hq, Hkv, D)
    sess.build_table([[0, 0], [0], []])
    out, lse = sess.decode(0, _dev(q), _dev(kn), _dev(vn))
    ob, lb = _bits(out), lse.cpu().numpy()
    for r, ch in enumerate([[blobs[0], blobs[0]], [blobs[0]], []]):
        o_ref, l_ref = oracle.Request(sh, ch, 8).attend_new(0, q[r][None], kn[r][None], vn[r][None])
        check(ob[r], o_ref[0], lb[r], l_ref[0], f"dup case {r}")
    sess.close()


@pytest.mark.parametrize("Hq,Hkv,D,lens,S", [
    (8, 2, 64, [[128, 128]], 16),                 # config 1 shape: 64 query rows per KV head
    (32, 8, 128, [[300, 77], [129]], 40),         # ragged chunks, two requests, 160 rows -> two row blocks
    (64, 8, 128, [[200]], 20),                    # G = 8
    (4, 4, 128, [[65, 1, 64]], 70),               # G = 1, suffix longer than one tile (causal across two new tiles)
    (8, 2, 128, [[]], 33),                        # no chunks at all: plain causal attention over the suffix
    (8, 4, 64, [[31], [], [500, 3]], 130),        # D = 64, three new tiles, an empty request in the batch
    (8, 2, 128, [[64]], 1),                       # a single suffix token through the tile kernel
])
def test_prefill_tensor_core_kernel(Hq, Hkv, D, lens, S):
    run_requests(2, Hq, Hkv, D, lens, S, 3, seed=41, prefill_impl=2)


@pytest.mark.parametrize("Hq,Hkv,D,lens,S,splits", [
    (32, 8, 128, [[300, 77], [129]], 40, 0),      # 160 rows: second block partly empty
    (64, 8, 128, [[200, 64]], 70, 3),             # G = 8, 560 rows: three CTAs of two blocks, KV splits
    (8, 2, 64, [[100]], 130, 2),                  # D = 64, 520 rows, three new-token tiles
    (16, 1, 128, [[64], []], 17, 1),              # G = 16 is not supported -> use G = 8 below
])
def test_prefill_tensor_core_two_row_blocks(Hq, Hkv, D, lens, S, splits):
    if Hq // Hkv > 8:
        Hq = 8 * Hkv
    run_requests(1, Hq, Hkv, D, lens, S, 2, seed=45, prefill_impl=3, prefill_ctas=splits)


@pytest.mark.parametrize("impl", [2, 3])
def test_prefill_tensor_core_peaky_queries_rescale_in_tmem(impl):
    """q scaled by 8: the running maximum jumps by far more than 2^8 between tiles, so the O rows are
    rescaled in tensor memory several times per row."""
    run_requests(1, 32, 8, 128, [[500, 300, 64]], 40, 2, seed=46, prefill_impl=impl, q_shift=3)
    run_requests(1, 8, 2, 64, [[129, 64]], 70, 1, seed=47, prefill_impl=impl, q_shift=3, prefill_ctas=1)


@pytest.mark.parametrize("splits", [1, 2, 5])
def test_prefill_tensor_core_split_invariance(splits):
    run_requests(1, 32, 8, 128, [[700, 260, 64]], 24, 2, seed=42, prefill_impl=2, prefill_ctas=splits)


def test_prefill_streaming_kernel_long_suffix():
    run_requests(1, 8, 2, 128, [[100, 30]], 37, 2, seed=43, prefill_impl=1)   # forced onto the streaming kernel


@pytest.mark.parametrize("Hq,Hkv,S,ctas,all_layers", [(8, 2, 70, 1000, False), (8, 2, 130, 1000, True), (8, 1, 70, 37, False),
                                                       (4, 4, 200, 1000, False), (8, 2, 70, 0, False)])
def test_prefill_streaming_kernel_suffix_of_several_new_token_tiles(Hq, Hkv, S, ctas, all_layers):
    """A suffix longer than one tile on the streaming kernel: every token block lists all ceil(S / 64) new-token tiles,
    and a block of early tokens sees nothing in the later ones.  With one CTA per tile such a tile is a CTA's whole
    share of the unit: an empty part (zero weight, lse = -inf) that the merge must ignore, never 0 / 0."""
    run_requests(2, Hq, Hkv, 128, [[100, 30], []], S, 2, seed=48, prefill_impl=1, ctas=ctas, all_layers=all_layers)


def test_prefill_appends_after_existing_tail():
    """Two prefill calls in a row (chunked sub-prefill): the second sees the first's tokens in the tail."""
    import paper_2512_22195_b200 as mk
    L, Hq, Hkv, D = 1, 8, 2, 128
    for impl in (1, 2):
        sess = _session(L, Hq, Hkv, D, 1, 2, 80)
        mk.matkv_set_option(sess.ctx, mk.OPT_PREFILL_IMPL, impl)
        blobs = [rand_bits(44, i, (L, 2, Hkv, n, D)) for i, n in enumerate([90, 70])]
        for i, b in enumerate(blobs):
            sess.register_device_chunk(i, b)
        sess.build_table([[0, 1]])
        req = oracle.Request(oracle.Shape(L, Hq, Hkv, D), blobs, 80)
        for part, S in enumerate([40, 24]):
            q, k, v = rand_bits(44, 10 + part, (1, S, Hq, D)), rand_bits(44, 20 + part, (1, S, Hkv, D)), rand_bits(44, 30 + part, (1, S, Hkv, D))
            out, lse = sess.prefill(0, _dev(q), _dev(k), _dev(v))
            o_ref, l_ref = req.attend_new(0, q[0], k[0], v[0])
            check(_bits(out)[0], o_ref, lse.cpu().numpy()[0], l_ref, f"impl {impl} part {part}")
            sess.advance(S)
            req.advance(S)
        assert sess.status() == 0
        sess.close()


@pytest.mark.parametrize("S,impl", [(5, 0), (40, 2)])
def test_p9_rotary_mode_positions(S, impl):
    """q and k_new are rotated at position (sum of chunk lengths) + tail index; stored chunk K is used as it is.
    The tails must match the oracle's bit for bit (rotation in fp64, rounded once to bf16, on both sides)."""
    run_requests(2, 8, 2, 128, [[300, 77], [129]], S, 3, seed=51, rope_theta=500000.0, prefill_impl=impl)
    run_requests(1, 8, 2, 64, [[64, 200]], S, 2, seed=52, rope_theta=10000.0, prefill_impl=impl, all_layers=True)


def test_p9_rotary_position_base_is_a_parameter():
    run_requests(1, 4, 2, 128, [[100, 30]], 6, 2, seed=53, rope_theta=500000.0, pos_mode=1)   # base = longest chunk


def test_cfg2_shape_two_layers_sampled_steps():
    """Llama-3-8B head shape, 5 x 1,024-token chunks, 64-token suffix, 128 decode steps, 2 layers;
    all steps run on the GPU, the oracle checks the prefill of layer 1 rows {0, 31, 63} and decode
    steps {0, 1, 63, 127} (every layer, every head)."""
    L, Hq, Hkv, D, S, T = 2, 32, 8, 128, 64, 128
    seed = 1
    sess = _session(L, Hq, Hkv, D, 1, 5, S + T)
    sh = oracle.Shape(L, Hq, Hkv, D)
    blobs = [rand_bits(seed, 1000 + i, (L, 2, Hkv, 1024, D)) for i in range(5)]
    for i, b in enumerate(blobs):
        sess.register_device_chunk(i, b)
    sess.build_table([list(range(5))])
    req = oracle.Request(sh, blobs, S + T)
    for layer in range(L):
        q, k, v = rand_bits(seed, 10 + layer, (1, S, Hq, D)), rand_bits(seed, 40 + layer, (1, S, Hkv, D)), rand_bits(seed, 70 + layer, (1, S, Hkv, D))
        out, lse = sess.prefill(layer, _dev(q), _dev(k), _dev(v))
        req.append_only(layer, k[0], v[0])
        if layer == 1:
            rows = [0, 31, 63]
            o_ref, l_ref = oracle.attend(sh, layer, blobs, req.tail_k[layer], req.tail_v[layer], q[0][rows], [r + 1 for r in rows])
            check(_bits(out)[0][rows], o_ref, lse.cpu().numpy()[0][rows], l_ref, "cfg2 prefill")
    sess.advance(S)
    req.advance(S)
    for t in range(T):
        q, k, v = rand_bits(seed, 2000 + t, (L, 1, Hq, D)), rand_bits(seed, 3000 + t, (L, 1, Hkv, D)), rand_bits(seed, 4000 + t, (L, 1, Hkv, D))
        out, lse = sess.decode_all_layers(_dev(q), _dev(k), _dev(v))
        for layer in range(L):
            req.append_only(layer, k[layer], v[layer])
        if t in (0, 1, 63, 127):
            ob, lb = _bits(out), lse.cpu().numpy()
            for layer in range(L):
                o_ref, l_ref = oracle.attend(sh, layer, blobs, req.tail_k[layer], req.tail_v[layer], q[layer], [req.tail_len + 1])
                check(ob[layer], o_ref, lb[layer], l_ref, f"cfg2 decode step {t} layer {layer}")
        sess.advance(1)
        req.advance(1)
    assert sess.status() == 0
    sess.close()


# ---- chunk-major decode (requests that list the same chunks) ----------------------------------------
@pytest.mark.parametrize("Hq,Hkv,D", [(8, 2, 128), (32, 8, 128), (16, 2, 128), (4, 4, 64), (4, 2, 64), (8, 2, 64)])
def test_chunk_major_decode_shared_chunks(Hq, Hkv, D):
    """Seven requests over a pool of five chunks (ragged lengths, one listed by six requests, one request
    listing a chunk twice, one without chunks): the chunk-major kernel against the oracle."""
    pool = [200, 64, 33, 129, 1]
    ids = [[0, 1], [0, 2, 3], [1, 0], [0], [3, 0, 3], [], [4, 0, 2]]
    run_requests(2, Hq, Hkv, D, ids, 3, 4, seed=61, pool=pool, decode_impl=2)


def test_chunk_major_decode_all_layers_fused_advance_and_small_items():
    """One launch for all layers with the tail advanced by the launch itself; items of two tiles, so long
    chunks are cut into several items (several partials per chunk and request); few CTAs and many."""
    pool = [300, 130, 70]
    ids = [[0, 1, 2], [2, 0], [0], [1, 0], [0, 2]]
    for ctas in (3, 0):
        run_requests(3, 8, 2, 128, ids, 2, 5, seed=62, pool=pool, decode_impl=2, share_tiles=2, all_layers=True,
                     fused_advance=True, ctas=ctas)


def test_chunk_major_decode_tail_grows_over_tiles():
    """A tail that grows through 64 tokens under the chunk-major kernel (the tail item spans tiles)."""
    run_requests(1, 4, 2, 128, [[0], [0]], 60, 10, seed=63, pool=[50], decode_impl=2)


def test_auto_choice_matches_sharing():
    """The automatic choice takes the chunk-major kernel only when stacking saves chunk reads."""
    import paper_2512_22195_b200 as mk
    sess = _session(1, 8, 2, 128, 4, 2, 8)
    for cid, n in enumerate([128, 128, 64]):
        sess.register_device_chunk(cid, rand_bits(5, cid, (1, 2, 2, n, 128)))
    t = sess.build_table([[0, 1], [0, 1], [0, 2], [0]])
    logical, read = mk.matkv_table_sharing(t)
    assert (logical, read) == (4 + 4 + 3 + 2, 2 + 2 + 1)   # 13 tiles listed; chunks 0, 1, 2 read once each
    t = sess.build_table([[0], [1], [2]])
    assert mk.matkv_table_sharing(t) == (5, 5)
    assert mk.matkv_table_workspace_bytes(t, 1) >= mk.matkv_workspace_bytes(sess.ctx)
    sess.close()


def test_chunk_major_decode_many_parts_and_rotary_mode():
    """More than 32 partials per request (one-tile items of a 2,200-token chunk: the general merge path), and the
    chunk-major kernel behind the rotary pre-rotation (q and k_new rotated at each request's own position)."""
    pool = [2200, 130]
    run_requests(1, 8, 2, 128, [[0, 1], [0], [1, 0]], 2, 2, seed=64, pool=pool, decode_impl=2, share_tiles=1)
    run_requests(2, 8, 2, 64, [[0, 1], [1], [1, 0]], 3, 3, seed=65, pool=[70, 33], decode_impl=2, rope_theta=10000.0)
    run_requests(2, 8, 2, 64, [[0, 1], [1], [1, 0]], 3, 3, seed=66, pool=[70, 33], decode_impl=2, rope_theta=500000.0, pos_mode=1)


@pytest.mark.parametrize("case", range(24))
def test_random_tables_against_the_oracle(case):
    """Seeded random workloads: head shapes, ragged chunk lengths, shared and repeated chunks, empty lists, suffix
    and decode lengths, launch granularity, grid size and kernel choice are all drawn; every output is compared."""
    rng = np.random.default_rng(1000 + case)
    Hkv = int(rng.choice([1, 2, 4, 8]))
    G = int(rng.choice([1, 2, 4, 8]))
    D = int(rng.choice([64, 128]))
    L = int(rng.integers(1, 4))
    n_pool = int(rng.integers(1, 6))
    pool = [int(rng.choice([1, 7, 33, 64, 65, 127, 128, 200, 300, 513])) for _ in range(n_pool)]
    B = int(rng.integers(1, 6))
    ids = []
    for _ in range(B):
        k = int(rng.integers(0, 4))
        ids.append([int(rng.integers(0, n_pool)) for _ in range(k)])       # repeats inside a request are allowed
    S = int(rng.choice([1, 3, 9, 17, 40]))
    T = int(rng.integers(1, 5))
    kw = dict(
        ctas=int(rng.choice([0, 0, 1, 5, 37])),
        all_layers=bool(rng.integers(0, 2)),
        decode_impl=int(rng.choice([0, 1, 2])),
        share_tiles=int(rng.choice([0, 1, 3])),
        prefill_impl=int(rng.choice([0, 1, 2, 3])),
    )
    kw["fused_advance"] = kw["all_layers"] and bool(rng.integers(0, 2))
    run_requests(L, Hkv * G, Hkv, D, ids, S, T, seed=500 + case, pool=pool, **kw)
