"""The allocation-free decode entry point against the CPU oracle and the ordinary entry point (collected last on purpose).

`matkv_attend_decode_static` serves callers that may neither allocate device memory nor lend a
workspace (a server whose KV pool owns all of HBM, a plug-in under a host that forbids allocation
after start-up): its split-KV scratch is an array built into the library.  It must give what
the oracle computes and what `matkv_attend_decode` gives, on consecutive calls that reuse that one array,
and must refuse calls larger than the array with a clear error.
"""
import numpy as np
import pytest
import torch

import matkv_inputs as mi
import oracle
from _util import MAX_ABS, MEAN_ABS, check, rand_bits

pytestmark = pytest.mark.gpu


def test_static_scratch_decode_matches_workspace_decode_twice():
    import paper_2512_22195_b200 as mk
    from paper_2512_22195_b200.harness import Session, bits_to_dev, dev_to_bits
    L, Hq, Hkv, D, B = 2, 32, 8, 128, 2
    sess = Session(L, Hq, Hkv, D, B, 3, 8)
    lens = [700, 130, 64]
    blobs = [rand_bits(77, i, (L, 2, Hkv, n, D)) for i, n in enumerate(lens)]
    for i, b in enumerate(blobs):
        sess.register_device_chunk(i, b)
    ids = [[0, 1, 2], [2, 0]]
    sess.build_table(ids)
    reqs = [oracle.Request(oracle.Shape(L, Hq, Hkv, D), [blobs[c] for c in row], 8) for row in ids]
    for step in range(2):                                   # two calls in a row share the built-in array
        for layer in range(L):
            qb, kb, vb = (rand_bits(77, s0 + 10 * step + layer, (B, Hq if s0 == 100 else Hkv, D)) for s0 in (100, 200, 300))
            q, k, v = bits_to_dev(qb), bits_to_dev(kb), bits_to_dev(vb)
            ref, ref_lse = sess.decode(layer, q, k, v)
            out = torch.zeros_like(q)
            lse = torch.zeros((B, Hq), dtype=torch.float32, device="cuda")
            mk.matkv_attend_decode_static(sess.ctx, sess.table, layer, q.data_ptr(), k.data_ptr(), v.data_ptr(),
                                          out.data_ptr(), lse.data_ptr())
            for r in range(B):                              # first against the oracle, like every other kernel
                o_ref, l_ref = reqs[r].attend_new(layer, qb[r][None], kb[r][None], vb[r][None])
                check(dev_to_bits(out)[r], o_ref[0], lse.cpu().numpy()[r], l_ref[0], f"static decode step {step} layer {layer} request {r}")
            a, b = mi.bf16_bits_to_f64(dev_to_bits(out)), mi.bf16_bits_to_f64(dev_to_bits(ref))
            assert np.all(np.isfinite(a))
            assert np.max(np.abs(a - b)) <= MAX_ABS and np.mean(np.abs(a - b)) <= MEAN_ABS
            assert np.max(np.abs(lse.cpu().numpy() - ref_lse.cpu().numpy())) <= 1e-3
            assert np.linalg.norm(b) > 0
        sess.advance(1)
        for rq in reqs:
            rq.advance(1)
    assert sess.status() == 0
    sess.close()


def test_static_scratch_decode_rejects_calls_beyond_its_array():
    import paper_2512_22195_b200 as mk
    from paper_2512_22195_b200.harness import Session, bits_to_dev
    L, Hq, Hkv, D, B = 1, 8, 8, 64, 33                      # 33 x 8 = 264 units > 256
    sess = Session(L, Hq, Hkv, D, B, 1, 2)
    sess.register_device_chunk(0, rand_bits(78, 0, (L, 2, Hkv, 16, D)))
    sess.build_table([[0]] * B)
    q = bits_to_dev(rand_bits(78, 1, (B, Hq, D)))
    kv = bits_to_dev(rand_bits(78, 2, (B, Hkv, D)))
    out = torch.empty_like(q)
    with pytest.raises(mk.MatkvError) as e:
        mk.matkv_attend_decode_static(sess.ctx, sess.table, 0, q.data_ptr(), kv.data_ptr(), kv.data_ptr(), out.data_ptr())
    assert e.value.code == mk.E_CAPACITY and "256" in str(e.value)
    sess.decode(0, q, kv, kv)                                # the ordinary entry point still takes it
    assert sess.status() == 0
    sess.close()
