"""Planted needles on the GPU: one key made dominant for one query row must pull that row's output onto the
value stored beside it, wherever the key sits -- first and last token of every 64-token tile of every chunk (so
every tile, every KV-split boundary and every item cut is crossed), the tail's first and last token, the row's
own new token -- and a key one past the causal edge must not be seen at all.  Random-data parity alone leaves a
dropped tile at long context close to the tolerance; a needle makes it exact.  Run through the tensor-core
sub-prefill (one and two row blocks per CTA, one and several KV splits), the chunk-major decode (items of one
and three tiles), the request-major decode with one CTA per tile and the cluster decode."""
import numpy as np
import pytest
import torch

import matkv_inputs as mi
from _util import rand_bits

pytestmark = pytest.mark.gpu

L, HQ, HKV, D = 1, 8, 2, 128
G = HQ // HKV


def _mk():
    import paper_2512_22195_b200 as mk
    from paper_2512_22195_b200.harness import Session, bits_to_dev, dev_to_bits
    return mk, Session, bits_to_dev, dev_to_bits


def _needle_for(q_row_bits):
    """A key 16 times the query row: its logit is ~180 above every other key's."""
    return mi.f32_to_bf16_bits((mi.bf16_bits_to_f64(q_row_bits) * 16.0).astype(np.float32))


def _close_to(o_bits, want_bits, what):
    o, want = mi.bf16_bits_to_f64(o_bits), mi.bf16_bits_to_f64(want_bits)
    assert np.max(np.abs(o - want)) <= 2 ** -7 * np.max(np.abs(want)) + 1e-6, what


def _tile_edges(n):
    """first and last valid token of every 64-token tile of a chunk of n tokens"""
    out = set()
    for t0 in range(0, n, 64):
        out.add(t0)
        out.add(min(n, t0 + 64) - 1)
    return sorted(out)


@pytest.mark.parametrize("impl,splits", [(2, 1), (2, 3), (3, 1), (3, 4)])
def test_needles_through_the_tensor_core_prefill(impl, splits):
    mk, Session, to_dev, to_bits = _mk()
    lens = [130, 64, 1, 200]                     # 3 + 1 + 1 + 4 chunk tiles; the last tiles are ragged
    PRE, S = 5, 70                               # 5 tokens already in the tail, then a 70-token suffix (two new-token tiles)
    seed = 91
    sess = Session(L, HQ, HKV, D, 1, len(lens), PRE + S)
    mk.matkv_set_option(sess.ctx, mk.OPT_PREFILL_IMPL, impl)
    mk.matkv_set_option(sess.ctx, mk.OPT_PREFILL_CTAS, splits)
    blobs = [rand_bits(seed, 10 + i, (L, 2, HKV, n, D)) for i, n in enumerate(lens)]
    dev_chunks = [sess.register_device_chunk(i, b) for i, b in enumerate(blobs)]
    q_pre, k_pre, v_pre = rand_bits(seed, 1, (1, PRE, HQ, D)), rand_bits(seed, 2, (1, PRE, HKV, D)), rand_bits(seed, 3, (1, PRE, HKV, D))
    q, k_new, v_new = rand_bits(seed, 4, (1, S, HQ, D)), rand_bits(seed, 5, (1, S, HKV, D)), rand_bits(seed, 6, (1, S, HKV, D))
    dq_pre, dq = to_dev(q_pre), to_dev(q)

    def run(k_pre_b, k_new_b):
        sess.build_table([list(range(len(lens)))])
        sess.prefill(0, dq_pre, to_dev(k_pre_b), to_dev(v_pre), want_lse=False)
        sess.advance(PRE)
        out, _ = sess.prefill(0, dq, to_dev(k_new_b), to_dev(v_new))
        torch.cuda.synchronize()
        return to_bits(out)[0]

    clean = run(k_pre, k_new)
    rows = [(0, 0), (31, 5), (32, 2), (63, 7), (64, 1), (69, 6), (17, 3), (45, 4)]   # (suffix token, query head): both row blocks, every head
    trial = 0
    # chunk tokens: every tile edge of every chunk
    for c, n in enumerate(lens):
        for t in _tile_edges(n):
            i, h = rows[trial % len(rows)]
            trial += 1
            g = h // G
            keep = dev_chunks[c][0, 0, g, t].clone()
            dev_chunks[c][0, 0, g, t] = to_dev(_needle_for(q[0, i, h]))
            torch.cuda.synchronize()
            got = run(k_pre, k_new)
            dev_chunks[c][0, 0, g, t] = keep
            _close_to(got[i, h], blobs[c][0, 1, g, t], f"needle at chunk {c} token {t}, row ({i}, {h})")
    # the tail's first and last token
    for t in (0, PRE - 1):
        i, h = rows[trial % len(rows)]
        trial += 1
        kp = k_pre.copy()
        kp[0, t, h // G] = _needle_for(q[0, i, h])
        _close_to(run(kp, k_new)[i, h], v_pre[0, t, h // G], f"needle at tail token {t}")
    # the call's new tokens: the first one (seen by every row), the row's own token, the edges of the new-token tiles
    for i, h, t in [(40, 3, 0), (40, 3, 40), (63, 0, 63), (64, 5, 63), (64, 5, 64), (69, 2, 64), (69, 7, 69), (0, 4, 0)]:
        kn = k_new.copy()
        kn[0, t, h // G] = _needle_for(q[0, i, h])
        _close_to(run(k_pre, kn)[i, h], v_new[0, t, h // G], f"needle at new token {t}, row ({i}, {h})")
    # one past the causal edge: rows of tokens <= i must not change by a bit
    for i, h in [(0, 1), (39, 6), (62, 0), (63, 3), (68, 5)]:
        kn = k_new.copy()
        kn[0, i + 1, h // G] = _needle_for(q[0, i, h])
        got = run(k_pre, kn)
        assert np.array_equal(got[:i + 1], clean[:i + 1]), f"a key at new token {i + 1} leaked into rows of tokens <= {i}"
    assert sess.status() == 0
    sess.close()


@pytest.mark.parametrize("decode_impl,share_tiles,ctas,cluster", [(2, 1, 0, 0), (2, 3, 0, 0), (2, 3, 5, 0), (1, 0, 1000, 0), (1, 0, 0, 0),
                                                                  (1, 0, 0, 2)])
def test_needles_through_the_decode_kernels(decode_impl, share_tiles, ctas, cluster):
    mk, Session, to_dev, to_bits = _mk()
    pool = [200, 64, 33, 129]
    ids = [[0, 1], [0, 2, 3], [1, 0], [0], [3, 0]]       # chunk 0 is listed by five requests: two stacked groups at G = 4
    B, PRE = len(ids), 3
    seed = 92
    sess = Session(L, HQ, HKV, D, B, 3, PRE + 3)
    mk.matkv_set_option(sess.ctx, mk.OPT_DECODE_IMPL, decode_impl)
    mk.matkv_set_option(sess.ctx, mk.OPT_CLUSTER_DECODE, cluster)     # 2: the cluster kernel (clusters of 8 CTAs per request and KV head)
    if share_tiles:
        mk.matkv_set_option(sess.ctx, mk.OPT_SHARE_TILES, share_tiles)
    if ctas:
        mk.matkv_set_option(sess.ctx, mk.OPT_DECODE_CTAS, ctas)
    blobs = [rand_bits(seed, 10 + i, (L, 2, HKV, n, D)) for i, n in enumerate(pool)]
    dev_chunks = [sess.register_device_chunk(i, b) for i, b in enumerate(blobs)]
    q_pre, k_pre, v_pre = rand_bits(seed, 1, (B, PRE, HQ, D)), rand_bits(seed, 2, (B, PRE, HKV, D)), rand_bits(seed, 3, (B, PRE, HKV, D))
    q, k_new, v_new = rand_bits(seed, 4, (B, HQ, D)), rand_bits(seed, 5, (B, HKV, D)), rand_bits(seed, 6, (B, HKV, D))
    dq_pre, dq = to_dev(q_pre), to_dev(q)

    def run(k_pre_b, k_new_b):
        sess.build_table(ids)
        sess.prefill(0, dq_pre, to_dev(k_pre_b), to_dev(v_pre), want_lse=False)
        sess.advance(PRE)
        out, _ = sess.decode(0, dq, to_dev(k_new_b), to_dev(v_new))
        torch.cuda.synchronize()
        return to_bits(out)

    clean = run(k_pre, k_new)
    trial = 0
    for c, n in enumerate(pool):
        users = [r for r, row in enumerate(ids) if c in row]
        for t in _tile_edges(n):
            r, h = users[trial % len(users)], trial % HQ
            trial += 1
            g = h // G
            keep = dev_chunks[c][0, 0, g, t].clone()
            dev_chunks[c][0, 0, g, t] = to_dev(_needle_for(q[r, h]))
            torch.cuda.synchronize()
            got = run(k_pre, k_new)
            dev_chunks[c][0, 0, g, t] = keep
            _close_to(got[r, h], blobs[c][0, 1, g, t], f"needle at chunk {c} token {t}, request {r} head {h}")
    for r, h, t in [(0, 1, 0), (3, 6, PRE - 1), (4, 3, 1)]:          # the tail (suffix tokens appended by the sub-prefill)
        kp = k_pre.copy()
        kp[r, t, h // G] = _needle_for(q[r, h])
        _close_to(run(kp, k_new)[r, h], v_pre[r, t, h // G], f"needle at tail token {t} of request {r}")
    for r, h in [(1, 0), (2, 7)]:                                    # the step's own new token
        kn = k_new.copy()
        kn[r, h // G] = _needle_for(q[r, h])
        _close_to(run(k_pre, kn)[r, h], v_new[r, h // G], f"needle as the new token of request {r}")
    # a key sitting in the tail one past the new token must not be seen
    sess.build_table(ids)
    sess.prefill(0, dq_pre, to_dev(k_pre), to_dev(v_pre), want_lse=False)
    sess.advance(PRE)
    sess.tail_k[2, 0, 1, PRE + 1] = to_dev(_needle_for(q[2, 5]))
    out, _ = sess.decode(0, dq, to_dev(k_new), to_dev(v_new))
    torch.cuda.synchronize()
    sess.tail_k[2, 0, 1, PRE + 1] = 0
    if decode_impl == 1:     # a static split: the same bits run after run
        assert np.array_equal(to_bits(out), clean), "a key past the causal edge of the tail was seen"
    else:                    # items are drawn dynamically, so the summation order may differ between two runs
        a, b = mi.bf16_bits_to_f64(to_bits(out)), mi.bf16_bits_to_f64(clean)
        assert np.max(np.abs(a - b)) <= 2 ** -7 * np.max(np.abs(b)), "a key past the causal edge of the tail was seen"
    assert sess.status() == 0
    sess.close()
