"""GPU checks of the compressed chunk store: the quantiser kernel against the oracle's codec bit for bit, the
expanding staging copy bit for bit, and attention over staged compressed chunks against the oracle."""
import os

import numpy as np
import pytest
import torch

import matkv_inputs as mi
import oracle
from _util import check, rand_bits

pytestmark = pytest.mark.gpu


def _fp8_blob_np(sess, mk, codes, exps):
    """The compressed blob's bytes as the C ABI lays them out."""
    n = codes.shape[3]
    total = mk.matkv_fp8_blob_bytes(sess.ctx, n)
    raw = np.zeros(total, dtype=np.uint8)
    raw[:codes.size] = codes.reshape(-1)
    off = (codes.size + 255) // 256 * 256
    raw[off:off + exps.size] = exps.reshape(-1).view(np.uint8)
    return raw


@pytest.mark.parametrize("n,shift", [(1, 0), (63, 0), (64, 2), (65, -6), (200, 0), (1024, 0)])
def test_quantiser_kernel_matches_the_oracle_codec_bit_for_bit(n, shift):
    import paper_2512_22195_b200 as mk
    from paper_2512_22195_b200.harness import Session, bits_to_dev
    L, Hq, Hkv, D = 2, 8, 2, 128
    sess = Session(L, Hq, Hkv, D, 1, 1, 8)
    sh = oracle.Shape(L, Hq, Hkv, D)
    blob = rand_bits(71, n, (L, 2, Hkv, n, D), shift)
    blob[1, 0, 1, : min(n, 64)] = 0                       # an all-zero block
    blob[0, 1, 0, 0, 0] = 0x8000                          # a negative zero
    if n >= 2:
        blob[0, 0, 0, 1, :4] = [0x3f80, 0xbf80, 0x0001, 0x7f7f]   # 1, -1, the smallest subnormal, the largest finite bf16
    codes, exps = oracle.fp8_quantize_blob(sh, blob)
    d_blob = bits_to_dev(blob)
    out = torch.zeros(mk.matkv_fp8_blob_bytes(sess.ctx, n), dtype=torch.uint8, device="cuda")
    mk.matkv_quantize_chunk_fp8(sess.ctx, d_blob.data_ptr(), n, out.data_ptr())
    torch.cuda.synchronize()
    assert np.array_equal(out.cpu().numpy(), _fp8_blob_np(sess, mk, codes, exps))
    sess.close()


def test_staged_compressed_chunks_expand_exactly_and_attend_like_the_oracle():
    """Compressed chunks in pinned host memory -> staging (expanding copy kernel) -> the table's gather is bit-exact
    with the oracle's dequantised blob; sub-prefill and decode over them match the oracle on those values."""
    import paper_2512_22195_b200 as mk
    from paper_2512_22195_b200.harness import Session, bits_to_dev, dev_to_bits
    L, Hq, Hkv, D = 2, 8, 2, 128
    lens = [200, 64, 33]
    S, T = 5, 3
    sess = Session(L, Hq, Hkv, D, 2, 3, S + T)
    sh = oracle.Shape(L, Hq, Hkv, D)
    deq, keep = {}, []
    for cid, n in enumerate(lens):
        blob = rand_bits(72, cid, (L, 2, Hkv, n, D), cid - 2)       # different block exponents per chunk, at most unit scale
        codes, exps = oracle.fp8_quantize_blob(sh, blob)
        deq[cid] = oracle.fp8_dequantize_blob(sh, codes, exps)
        host = torch.from_numpy(_fp8_blob_np(sess, mk, codes, exps)).pin_memory()
        keep.append(host)
        mk.matkv_register_chunk_fp8(sess.ctx, cid, n, host.data_ptr())
    slot_bytes = (L * 2 * Hkv * max(lens) * D * 2 + 255) // 256 * 256
    slots = torch.zeros(3 * slot_bytes, dtype=torch.uint8, device="cuda")
    copy = torch.cuda.Stream()
    sess.stage([0, 1, 2], slots, slot_bytes, copy)
    ids = [[0, 1, 2], [2, 0]]
    sess.build_table(ids)
    # the staged copies are the dequantised blobs, bit for bit
    for r, row in enumerate(ids):
        rows = sum(lens[c] for c in row)
        for layer in range(L):
            k, v = sess.gather(layer, r, rows)
            ref_k = np.concatenate([deq[c][layer, 0] for c in row], axis=1)
            ref_v = np.concatenate([deq[c][layer, 1] for c in row], axis=1)
            assert np.array_equal(dev_to_bits(k), ref_k) and np.array_equal(dev_to_bits(v), ref_v)
    reqs = [oracle.Request(sh, [deq[c] for c in row], S + T) for row in ids]
    B = len(ids)
    for layer in range(L):
        q, k, v = (rand_bits(72, 100 + 3 * layer + i, (B, S, Hq if i == 0 else Hkv, D)) for i in range(3))
        out, lse = sess.prefill(layer, bits_to_dev(q), bits_to_dev(k), bits_to_dev(v))
        for r in range(B):
            o_ref, l_ref = reqs[r].attend_new(layer, q[r], k[r], v[r])
            check(dev_to_bits(out)[r], o_ref, lse.cpu().numpy()[r], l_ref, f"prefill over compressed chunks, layer {layer} request {r}")
    sess.advance(S)
    for rq in reqs:
        rq.advance(S)
    for t in range(T):
        q, k, v = (rand_bits(72, 200 + 3 * t + i, (L, B, Hq if i == 0 else Hkv, D)) for i in range(3))
        out, lse = sess.decode_all_layers(bits_to_dev(q), bits_to_dev(k), bits_to_dev(v))
        for layer in range(L):
            for r in range(B):
                o_ref, l_ref = reqs[r].attend_new(layer, q[layer, r][None], k[layer, r][None], v[layer, r][None])
                check(dev_to_bits(out)[layer, r], o_ref[0], lse.cpu().numpy()[layer, r], l_ref[0], f"decode over compressed chunks, step {t}")
        sess.advance(1)
        for rq in reqs:
            rq.advance(1)
    assert sess.status() == 0
    sess.close()


def test_compressed_chunk_files_through_the_bounce_ring(tmp_path):
    """The storage tier with compressed files: reader threads -> pinned ring -> expanding copy -> slots."""
    import paper_2512_22195_b200 as mk
    from paper_2512_22195_b200.harness import Session, bits_to_dev, dev_to_bits
    L, Hq, Hkv, D = 1, 4, 2, 64
    n = 150
    sess = Session(L, Hq, Hkv, D, 1, 2, 4)
    sh = oracle.Shape(L, Hq, Hkv, D)
    deq = {}
    for cid in range(2):
        blob = rand_bits(73, cid, (L, 2, Hkv, n, D))
        codes, exps = oracle.fp8_quantize_blob(sh, blob)
        deq[cid] = oracle.fp8_dequantize_blob(sh, codes, exps)
        path = os.path.join(tmp_path, f"{cid}.kv8")
        _fp8_blob_np(sess, mk, codes, exps).tofile(path)
        mk.matkv_register_chunk_file_fp8(sess.ctx, cid, n, path)
    slab = (mk.matkv_fp8_blob_bytes(sess.ctx, n) + 4095) // 4096 * 4096
    ring = torch.empty(2 * slab + 4096, dtype=torch.uint8).pin_memory()
    base = (ring.data_ptr() + 4095) // 4096 * 4096
    mk.matkv_set_bounce_buffer(sess.ctx, base, 2 * slab, slab, 2)
    slot_bytes = (L * 2 * Hkv * n * D * 2 + 255) // 256 * 256
    slots = torch.zeros(2 * slot_bytes, dtype=torch.uint8, device="cuda")
    sess.stage([0, 1], slots, slot_bytes, torch.cuda.Stream())
    sess.build_table([[1, 0]])
    k, v = sess.gather(0, 0, 2 * n)
    assert np.array_equal(dev_to_bits(k), np.concatenate([deq[1][0, 0], deq[0][0, 0]], axis=1))
    assert np.array_equal(dev_to_bits(v), np.concatenate([deq[1][0, 1], deq[0][0, 1]], axis=1))
    sess.close()
    del ring


@pytest.mark.parametrize("Hq,Hkv", [(8, 2), (32, 8), (16, 2), (4, 4), (4, 2)])
def test_compressed_resident_chunks_attend_like_the_oracle(Hq, Hkv):
    """Compressed chunks kept compressed in HBM (MATKV_OPT_FP8_RESIDENT): the streaming kernel reads the codes and
    converts in registers.  Ragged lengths, different block exponents, one ordinary bf16 chunk in the same table,
    sub-prefill (several token blocks) and decode with a tail that crosses a tile; against the oracle on the values
    the codes stand for."""
    import paper_2512_22195_b200 as mk
    from paper_2512_22195_b200.harness import Session, bits_to_dev, dev_to_bits
    L, D = 2, 128
    lens = [200, 64, 33, 1, 130]
    S, T = 5, 4
    sess = Session(L, Hq, Hkv, D, 3, 4, 70 + S + T)
    mk.matkv_set_option(sess.ctx, mk.OPT_FP8_RESIDENT, 1)
    sh = oracle.Shape(L, Hq, Hkv, D)
    vals, keep = {}, []
    for cid, n in enumerate(lens[:4]):
        blob = rand_bits(74, cid, (L, 2, Hkv, n, D), cid - 3)       # scales 1/8 .. 1: different block exponents
        codes, exps = oracle.fp8_quantize_blob(sh, blob)
        vals[cid] = oracle.fp8_dequantize_blob(sh, codes, exps)
        host = torch.from_numpy(_fp8_blob_np(sess, mk, codes, exps)).pin_memory()
        keep.append(host)
        mk.matkv_register_chunk_fp8(sess.ctx, cid, n, host.data_ptr())
    vals[4] = rand_bits(74, 4, (L, 2, Hkv, lens[4], D))               # a plain bf16 chunk, device-resident
    sess.register_device_chunk(4, vals[4])
    slot_bytes = (L * 2 * Hkv * max(lens) * D * 2 + 255) // 256 * 256
    slots = torch.zeros(4 * slot_bytes, dtype=torch.uint8, device="cuda")
    sess.stage([0, 1, 2, 3], slots, slot_bytes, torch.cuda.Stream())
    ids = [[0, 4, 2], [3, 1, 0, 2], [4]]
    sess.build_table(ids)
    B = len(ids)
    reqs = [oracle.Request(sh, [vals[c] for c in row], 70 + S + T) for row in ids]
    # a tail of 62 tokens first (plain appends), so that the decode steps cross the 64-token tile boundary
    pre = 62
    for layer in range(L):
        q, k, v = (rand_bits(74, 50 + 3 * layer + i, (B, pre, Hq if i == 0 else Hkv, D)) for i in range(3))
        sess.prefill(layer, bits_to_dev(q), bits_to_dev(k), bits_to_dev(v))
        for r in range(B):
            reqs[r].append_only(layer, k[r], v[r])
    sess.advance(pre)
    for rq in reqs:
        rq.advance(pre)
    for layer in range(L):
        q, k, v = (rand_bits(74, 100 + 3 * layer + i, (B, S, Hq if i == 0 else Hkv, D)) for i in range(3))
        out, lse = sess.prefill(layer, bits_to_dev(q), bits_to_dev(k), bits_to_dev(v))
        for r in range(B):
            o_ref, l_ref = reqs[r].attend_new(layer, q[r], k[r], v[r])
            check(dev_to_bits(out)[r], o_ref, lse.cpu().numpy()[r], l_ref, f"prefill over resident codes, layer {layer} request {r}")
    sess.advance(S)
    for rq in reqs:
        rq.advance(S)
    for t in range(T):
        q, k, v = (rand_bits(74, 200 + 3 * t + i, (L, B, Hq if i == 0 else Hkv, D)) for i in range(3))
        if t % 2:
            out, lse = sess.decode_all_layers(bits_to_dev(q), bits_to_dev(k), bits_to_dev(v))
            ob, lb = dev_to_bits(out), lse.cpu().numpy()
        else:
            outs = [sess.decode(layer, bits_to_dev(q[layer]), bits_to_dev(k[layer]), bits_to_dev(v[layer])) for layer in range(L)]
            ob = np.stack([dev_to_bits(o) for o, _ in outs])
            lb = np.stack([l.cpu().numpy() for _, l in outs])
        for layer in range(L):
            for r in range(B):
                o_ref, l_ref = reqs[r].attend_new(layer, q[layer, r][None], k[layer, r][None], v[layer, r][None])
                check(ob[layer, r], o_ref[0], lb[layer, r], l_ref[0], f"decode over resident codes, step {t} layer {layer} request {r}")
        sess.advance(1)
        for rq in reqs:
            rq.advance(1)
    assert sess.status() == 0
    sess.close()


@pytest.mark.parametrize("impl,ctas,splits", [(1, 0, 0), (1, 1000, 0), (2, 0, 0), (2, 0, 1), (2, 0, 3)])
def test_compressed_resident_chunks_suffix_of_two_new_token_tiles(impl, ctas, splits):
    """A 70-token suffix over compressed-resident chunks, on the streaming kernel (two tiles of new tokens per token
    block; with one CTA per tile the second tile is an empty part for the blocks of early tokens) and on the tensor-core
    tile kernel, whose converter warps expand the code tiles to bf16 operand tiles in shared memory (one and several KV
    splits: 280 query rows per KV head in three row blocks)."""
    import paper_2512_22195_b200 as mk
    from paper_2512_22195_b200.harness import Session, bits_to_dev, dev_to_bits
    L, Hq, Hkv, D, S = 1, 8, 2, 128, 70
    lens = [130, 64, 33, 500]
    sess = Session(L, Hq, Hkv, D, 1, 4, S + 2)
    mk.matkv_set_option(sess.ctx, mk.OPT_FP8_RESIDENT, 1)
    mk.matkv_set_option(sess.ctx, mk.OPT_PREFILL_IMPL, impl)
    if ctas:
        mk.matkv_set_option(sess.ctx, mk.OPT_DECODE_CTAS, ctas)
    if splits:
        mk.matkv_set_option(sess.ctx, mk.OPT_PREFILL_CTAS, splits)
    sh = oracle.Shape(L, Hq, Hkv, D)
    vals, keep = [], []
    for cid, n in enumerate(lens):
        codes, exps = oracle.fp8_quantize_blob(sh, rand_bits(75, cid, (L, 2, Hkv, n, D), cid - 3))   # scales 1/8 .. 1: different block exponents
        vals.append(oracle.fp8_dequantize_blob(sh, codes, exps))
        host = torch.from_numpy(_fp8_blob_np(sess, mk, codes, exps)).pin_memory()
        keep.append(host)
        mk.matkv_register_chunk_fp8(sess.ctx, cid, n, host.data_ptr())
    slot_bytes = (L * 2 * Hkv * max(lens) * D * 2 + 255) // 256 * 256
    slots = torch.zeros(4 * slot_bytes, dtype=torch.uint8, device="cuda")
    sess.stage([0, 1, 2, 3], slots, slot_bytes, torch.cuda.Stream())
    sess.build_table([[0, 1, 2, 3]])
    rq = oracle.Request(sh, vals, S + 2)
    q, k, v = (rand_bits(75, 10 + i, (1, S, Hq if i == 0 else Hkv, D)) for i in range(3))
    out, lse = sess.prefill(0, bits_to_dev(q), bits_to_dev(k), bits_to_dev(v))
    o_ref, l_ref = rq.attend_new(0, q[0], k[0], v[0])
    check(dev_to_bits(out)[0], o_ref, lse.cpu().numpy()[0], l_ref, "70-token suffix over resident codes")
    assert sess.status() == 0
    sess.close()
