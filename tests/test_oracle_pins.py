"""Pins for the CPU oracle: each one ties it to something other than itself.

No test here touches the CUDA library.  What fixes the expected values:
  * a library routine (torch scaled_dot_product_attention, fp64, CPU) on the special case
    that reduces to textbook causal attention;
  * closed forms (uniform weights, constant V, two-key softmax, shifts of V);
  * invariants stated by the method (chunks are position-independent and used verbatim:
    permuting the chunk list changes nothing; listing a chunk twice adds ln 2 to lse);
  * planted needles that make one known token dominate;
  * the three separately written evaluators against each other (concatenation == LSE merge).
"""
import json
import math
import os

import numpy as np
import pytest
import torch

import matkv_inputs as mi
import oracle

GOLD = os.path.join(os.path.dirname(__file__), "golden")


def bits(x):
    return mi.f32_to_bf16_bits(np.asarray(x, dtype=np.float32))


def rand_bits(seed, stream, shape, shift=0):
    return mi.normal_bf16(seed, stream, int(np.prod(shape)), shift).reshape(shape)


def make_case(seed, L, Hq, Hkv, D, lens, S, cap=None):
    sh = oracle.Shape(L, Hq, Hkv, D)
    chunks = [rand_bits(seed, 100 + i, (L, 2, Hkv, n, D)) for i, n in enumerate(lens)]
    cap = cap or (S + 4)
    tail_k = rand_bits(seed, 50, (Hkv, cap, D))
    tail_v = rand_bits(seed, 51, (Hkv, cap, D))
    q = rand_bits(seed, 52, (S, Hq, D))
    return sh, chunks, tail_k, tail_v, q


# ---- P1: the three evaluators agree (concat == per-chunk + LSE merge == brute force) -------
@pytest.mark.parametrize("Hq,Hkv,D", [(1, 1, 8), (2, 1, 64), (8, 2, 64), (8, 8, 128), (4, 2, 128)])
@pytest.mark.parametrize("lens", [[], [1], [7, 40], [3, 1, 17, 5]])
@pytest.mark.parametrize("S", [1, 5, 16])
def test_p1_three_evaluators_agree(Hq, Hkv, D, lens, S):
    L = 2
    sh, chunks, tk, tv, q = make_case(11 + S, L, Hq, Hkv, D, lens, S, cap=S + 3)
    for layer in range(L):
        for t0 in (0, 3):                       # T in {0, 3}: rows see t0 + i + 1 tail tokens
            vis = [t0 + i + 1 for i in range(S)]
            o1, l1 = oracle.attend(sh, layer, chunks, tk, tv, q, vis, "walk")
            o2, l2 = oracle.attend(sh, layer, chunks, tk, tv, q, vis, "brute")
            o3, l3 = oracle.attend(sh, layer, chunks, tk, tv, q, vis, "merge")
            assert np.max(np.abs(o1 - o2)) <= 1e-12 and np.max(np.abs(l1 - l2)) <= 1e-12
            assert np.max(np.abs(o1 - o3)) <= 1e-12 and np.max(np.abs(l1 - l3)) <= 1e-12


# ---- P2: one chunk + suffix == last S rows of textbook causal attention (library routine) ---
@pytest.mark.parametrize("Hq,Hkv,D,ell,S", [(8, 2, 64, 37, 9), (4, 4, 128, 16, 16), (8, 1, 32, 1, 5), (6, 3, 64, 129, 1)])
def test_p2_single_chunk_is_causal_attention(Hq, Hkv, D, ell, S):
    L, layer = 2, 1
    sh = oracle.Shape(L, Hq, Hkv, D)
    G = Hq // Hkv
    chunk = rand_bits(3, 7, (L, 2, Hkv, ell, D))
    q = rand_bits(3, 8, (S, Hq, D))
    kn = rand_bits(3, 9, (S, Hkv, D))
    vn = rand_bits(3, 10, (S, Hkv, D))
    req = oracle.Request(sh, [chunk], tail_cap=S + 2)
    o, lse = req.attend_new(layer, q, kn, vn)
    # textbook: one sequence of ell + S tokens, square causal mask, query heads grouped contiguously
    K = np.concatenate([mi.bf16_bits_to_f64(chunk[layer, 0]), mi.bf16_bits_to_f64(kn).transpose(1, 0, 2)], axis=1)
    V = np.concatenate([mi.bf16_bits_to_f64(chunk[layer, 1]), mi.bf16_bits_to_f64(vn).transpose(1, 0, 2)], axis=1)
    Qfull = np.zeros((Hq, ell + S, D))
    Qfull[:, ell:, :] = mi.bf16_bits_to_f64(q).transpose(1, 0, 2)
    Kt = torch.from_numpy(K).repeat_interleave(G, dim=0)
    Vt = torch.from_numpy(V).repeat_interleave(G, dim=0)
    ref = torch.nn.functional.scaled_dot_product_attention(
        torch.from_numpy(Qfull)[None], Kt[None], Vt[None], is_causal=True)[0, :, ell:, :].numpy()
    assert np.max(np.abs(o - ref.transpose(1, 0, 2))) <= 1e-12
    # lse from the same library's logsumexp over the causal scores
    sc = torch.einsum("hqd,hkd->hqk", torch.from_numpy(Qfull), Kt) / math.sqrt(D)
    msk = torch.ones(ell + S, ell + S, dtype=torch.bool).tril()
    ref_lse = torch.logsumexp(sc.masked_fill(~msk, -math.inf), dim=-1)[:, ell:].numpy()
    assert np.max(np.abs(lse - ref_lse.T)) <= 1e-12


# ---- P3: closed forms ------------------------------------------------------------------------
def test_p3_zero_query_gives_mean_and_log_n():
    sh, chunks, tk, tv, q = make_case(5, 1, 4, 2, 64, [9, 30], 3, cap=8)
    q[:] = 0
    for t0 in (0, 4):
        vis = [t0 + i + 1 for i in range(3)]
        o, lse = oracle.attend(sh, 0, chunks, tk, tv, q, vis)
        for i, v in enumerate(vis):
            n = 39 + v
            assert np.allclose(lse[i], math.log(n), atol=1e-13)        # off-by-one in v shows here
            for h in range(4):
                g = h // 2
                Vs = np.concatenate([mi.bf16_bits_to_f64(c[0, 1, g]) for c in chunks] + [mi.bf16_bits_to_f64(tv[g, :v])])
                assert np.allclose(o[i, h], Vs.mean(axis=0), atol=1e-13)


def test_p3_constant_v_and_shift_of_v():
    sh, chunks, tk, tv, q = make_case(6, 1, 4, 1, 32, [5, 12], 4, cap=6)
    vis = [1, 2, 3, 4]
    o0, l0 = oracle.attend(sh, 0, chunks, tk, tv, q, vis)
    # V <- V + c (c = 2, exact in bf16 only if V's low bits allow: use V = small integers instead)
    ints = lambda a: bits(np.round(np.clip(mi.bf16_bits_to_f64(a), -3, 3)))
    c2 = [c.copy() for c in chunks]
    for c in c2:
        c[:, 1] = ints(c[:, 1])
    tv2 = ints(tv)
    oa, la = oracle.attend(sh, 0, c2, tk, tv2, q, vis)
    c3 = [c.copy() for c in c2]
    for c in c3:
        c[:, 1] = bits(mi.bf16_bits_to_f64(c[:, 1]) + 2.0)
    tv3 = bits(mi.bf16_bits_to_f64(tv2) + 2.0)
    ob, lb = oracle.attend(sh, 0, c3, tk, tv3, q, vis)
    assert np.allclose(ob, oa + 2.0, atol=1e-12) and np.allclose(lb, la, atol=1e-13) and np.allclose(la, l0, atol=1e-13)
    # every V row equal to one vector v  =>  o = v for every row and head
    vrow = rand_bits(6, 77, (32,))
    c4 = [c.copy() for c in chunks]
    for c in c4:
        c[:, 1] = vrow
    tv4 = np.broadcast_to(vrow, tv.shape).copy()
    oc, _ = oracle.attend(sh, 0, c4, tk, tv4, q, vis)
    assert np.allclose(oc, mi.bf16_bits_to_f64(vrow)[None, None, :], atol=1e-13)


def test_p3_equal_keys_give_uniform_weights():
    sh, chunks, tk, tv, q = make_case(8, 1, 2, 2, 16, [6], 2, cap=4)
    krow = rand_bits(8, 78, (16,))
    chunks[0][:, 0] = krow
    tk[:] = krow
    vis = [1, 2]
    o, lse = oracle.attend(sh, 0, chunks, tk, tv, q, vis)
    for i, v in enumerate(vis):
        for h in range(2):
            Vs = np.concatenate([mi.bf16_bits_to_f64(chunks[0][0, 1, h]), mi.bf16_bits_to_f64(tv[h, :v])])
            assert np.allclose(o[i, h], Vs.mean(axis=0), atol=1e-13)
            s = 0.25 * float(mi.bf16_bits_to_f64(q[i, h]) @ mi.bf16_bits_to_f64(krow))
            assert abs(lse[i, h] - (s + math.log(6 + v))) <= 1e-12


def test_p3_two_key_softmax_golden():
    """Hand-derived case stored as text: q=(1,0), keys (0,0),(1,0), scale 1, values e_1, e_2."""
    with open(os.path.join(GOLD, "two_key_softmax.json")) as f:
        g = json.load(f)
    sh = oracle.Shape(1, 1, 1, 2, scale=g["scale"])
    chunk = np.zeros((1, 2, 1, 2, 2), dtype=np.uint16)
    chunk[0, 0, 0] = bits(g["K"])
    chunk[0, 1, 0] = bits(g["V"])
    empty = np.zeros((1, 1, 2), dtype=np.uint16)
    for ev in ("walk", "brute", "merge"):
        o, lse = oracle.attend(sh, 0, [chunk], empty, empty, bits(g["q"]).reshape(1, 1, 2), [0], ev)
        assert np.allclose(o[0, 0], g["o"], atol=1e-15) and abs(lse[0, 0] - g["lse"]) <= 1e-15
    # the stored numbers are the closed form 1/(1+e), e/(1+e), ln(1+e)
    assert abs(g["o"][1] - math.e / (1 + math.e)) < 1e-15 and abs(g["lse"] - math.log1p(math.e)) < 1e-15


def test_p3_scale_enters_once():
    """Doubling the scale equals doubling q (power of two: exact in bf16)."""
    sh, chunks, tk, tv, q = make_case(9, 1, 2, 1, 16, [10], 2, cap=3)
    q2 = bits(mi.bf16_bits_to_f64(q) * 2.0)
    sh2 = oracle.Shape(1, 2, 1, 16, scale=2.0 * sh.scale)
    oa, la = oracle.attend(sh2, 0, chunks, tk, tv, q, [1, 2])
    ob, lb = oracle.attend(sh, 0, chunks, tk, tv, q2, [1, 2])
    assert np.max(np.abs(oa - ob)) <= 1e-14 and np.max(np.abs(la - lb)) <= 1e-13
    assert abs(sh.scale - 0.25) < 1e-15            # default 1/sqrt(D)


# ---- P4: planted needle -----------------------------------------------------------------------
def test_p4_needle_reaches_every_segment_and_causal_edge():
    L, Hq, Hkv, D, S = 2, 4, 2, 64, 3
    lens = [5, 64, 1, 33]
    sh, chunks, tk, tv, q = make_case(12, L, Hq, Hkv, D, lens, S, cap=S + 2)
    layer, i, h, g = 1, 1, 2, 1
    vis = [2, 3, 4]                                 # row 1 sees tail[0..3)
    qv = mi.bf16_bits_to_f64(q[i, h])
    needle = bits(qv * 64.0)                        # score = 64 |q|^2 / 8, dwarfs N(0,1)-sized scores
    spots = [(c, t) for c, n in enumerate(lens) for t in (0, n - 1)] + [("tail", 0), ("tail", 2)]
    for where, t in spots:
        cs = [c.copy() for c in chunks]
        tk2 = tk.copy()
        if where == "tail":
            tk2[g, t] = needle
            want = mi.bf16_bits_to_f64(tv[g, t])
        else:
            cs[where][layer, 0, g, t] = needle
            want = mi.bf16_bits_to_f64(cs[where][layer, 1, g, t])
        o, _ = oracle.attend(sh, layer, cs, tk2, tv, q, vis)
        assert np.max(np.abs(o[i, h] - want)) < 1e-6, (where, t)
    # a needle at tail[v] (first invisible row) must change nothing
    o0, l0 = oracle.attend(sh, layer, chunks, tk, tv, q, vis)
    tk2 = tk.copy()
    tk2[g, 3] = needle
    o1, l1 = oracle.attend(sh, layer, chunks, tk2, tv, q, vis)
    assert np.array_equal(o0[i], o1[i]) and np.array_equal(l0[i], l1[i])
    # ... and a needle in the other layer or other KV head is not seen by this head
    cs = [c.copy() for c in chunks]
    cs[1][0, 0, g, 7] = needle
    cs[1][layer, 0, 0, 7] = needle
    o2, _ = oracle.attend(sh, layer, cs, tk, tv, q, vis)
    assert np.array_equal(o0[i, h], o2[i, h])


# ---- P5 / P6: chunk order and duplication -------------------------------------------------------
def test_p5_permuting_the_chunk_list_changes_nothing():
    sh, chunks, tk, tv, q = make_case(13, 1, 8, 2, 64, [20, 3, 41, 8], 4, cap=6)
    vis = [1, 2, 3, 4]
    o0, l0 = oracle.attend(sh, 0, chunks, tk, tv, q, vis)
    for perm in ([3, 2, 1, 0], [1, 3, 0, 2]):
        o1, l1 = oracle.attend(sh, 0, [chunks[p] for p in perm], tk, tv, q, vis)
        assert np.max(np.abs(o0 - o1)) <= 1e-12 and np.max(np.abs(l0 - l1)) <= 1e-12


def test_p6_duplicate_chunk_adds_ln2_to_lse():
    sh, chunks, tk, tv, q = make_case(14, 1, 4, 4, 32, [25], 2, cap=2)
    o1, l1 = oracle.attend(sh, 0, chunks, tk, tv, q, [0, 0])
    o2, l2 = oracle.attend(sh, 0, chunks * 2, tk, tv, q, [0, 0])
    assert np.max(np.abs(o1 - o2)) <= 1e-13 and np.max(np.abs(l2 - l1 - math.log(2))) <= 1e-13


def test_empty_visible_set():
    sh, _, tk, tv, q = make_case(15, 1, 2, 1, 16, [], 2, cap=2)
    o, lse = oracle.attend(sh, 0, [], tk, tv, q, [0, 1])
    assert np.all(o[0] == 0) and np.all(np.isneginf(lse[0]))
    assert np.allclose(o[1, 0], mi.bf16_bits_to_f64(tv[0, 0]))       # one visible token: o = its V


def test_lse_merge_against_direct_softmax():
    rng = np.random.default_rng(0)
    o_parts = rng.normal(size=(5, 8))
    lse_parts = rng.normal(size=5) * 3
    lse_parts[2] = -np.inf
    o, lse = oracle.lse_merge(o_parts, lse_parts)
    w = np.exp(lse_parts - np.logaddexp.reduce(lse_parts))
    assert abs(lse - np.logaddexp.reduce(lse_parts)) < 1e-13 and np.allclose(o, w @ o_parts, atol=1e-13)


# ---- P9: rotary mode -------------------------------------------------------------------------
def test_p9_rope_identity_norm_and_relative_shift():
    D, theta = 64, 500000.0
    x = rand_bits(16, 1, (6, D))
    assert np.array_equal(oracle.rope(x, [0] * 6, theta), x)            # R_0 = identity
    # compare in fp64 through the rotation's defining property, using high-precision inputs:
    # bf16 rounding of the outputs limits agreement to ~2^-8 relative per element.
    a, b = x[:1], x[1:2]
    def score(pa, pb):
        ra = mi.bf16_bits_to_f64(oracle.rope(a, [pa], theta))[0]
        rb = mi.bf16_bits_to_f64(oracle.rope(b, [pb], theta))[0]
        return float(ra @ rb)
    base = score(7, 3)
    for delta in (1, 50, 1000):
        assert abs(score(7 + delta, 3 + delta) - base) < 0.25           # depends on p - j only
    assert abs(score(7, 3) - score(3, 7)) > 1e-3                        # but not on |p - j| alone
    # rotation preserves the norm (up to bf16 rounding)
    n0 = np.linalg.norm(mi.bf16_bits_to_f64(x), axis=1)
    n1 = np.linalg.norm(mi.bf16_bits_to_f64(oracle.rope(x, [5, 9, 100, 4096, 70000, 1], theta)), axis=1)
    assert np.allclose(n0, n1, rtol=4e-3)
    # first pair (d=0) rotates by exactly pos radians: check against cos/sin directly
    e = np.zeros((1, D), dtype=np.float32)
    e[0, 0] = 1.0
    r = mi.bf16_bits_to_f64(oracle.rope(bits(e), [2], theta))[0]
    assert abs(r[0] - math.cos(2.0)) < 4e-3 and abs(r[D // 2] - math.sin(2.0)) < 4e-3
    # last pair rotates by pos * theta^(-(D-2)/D)
    e[:] = 0
    e[0, D // 2 - 1] = 1.0
    r = mi.bf16_bits_to_f64(oracle.rope(bits(e), [100000], theta))[0]
    ang = 100000 * theta ** (-(D - 2) / D)
    assert abs(r[D // 2 - 1] - math.cos(ang)) < 4e-3 and abs(r[D - 1] - math.sin(ang)) < 4e-3


def test_request_position_base_and_tail_growth():
    """Query tokens continue after the chunks: first suffix token at position sum(len)."""
    sh = oracle.Shape(1, 2, 1, 16)
    chunks = [rand_bits(17, 1, (1, 2, 1, 9, 16)), rand_bits(17, 2, (1, 2, 1, 4, 16))]
    req = oracle.Request(sh, chunks, tail_cap=6, rope_theta=500000.0)
    assert req.pos_base == 13
    q, k, v = rand_bits(17, 3, (2, 2, 16)), rand_bits(17, 4, (2, 1, 16)), rand_bits(17, 5, (2, 1, 16))
    req.attend_new(0, q, k, v)
    assert np.array_equal(req.tail_k[0, 0, :2], oracle.rope(k[:, 0], [13, 14], 500000.0))
    assert np.array_equal(req.tail_v[0, 0, :2], v[:, 0])                 # V is never rotated
    req.advance(2)
    q1, k1, v1 = q[:1], k[:1], v[:1]
    o, lse = req.attend_new(0, q1, k1, v1)
    assert np.array_equal(req.tail_k[0, 0, 2], oracle.rope(k1[:, 0], [15], 500000.0)[0])
    # decode row sees 13 chunk tokens + 3 tail tokens: with q = 0 lse = ln 16
    req2 = oracle.Request(sh, chunks, tail_cap=6)
    req2.attend_new(0, q, k, v); req2.advance(2)
    _, l0 = req2.attend_new(0, np.zeros_like(q1), k1, v1)
    assert np.allclose(l0, math.log(16), atol=1e-13)


def test_generator_statistics_and_determinism():
    a = mi.normal_bf16(0, 1, 1 << 16)
    b = mi.normal_bf16(0, 1, 1 << 15, start=1 << 15)
    assert np.array_equal(a[1 << 15:], b)                                 # counter-based
    x = mi.bf16_bits_to_f64(a)
    assert abs(x.mean()) < 0.02 and abs(x.std() - 1.0) < 0.02 and np.max(np.abs(x)) < 6.0
    assert not np.array_equal(a, mi.normal_bf16(1, 1, 1 << 16))
    y = mi.bf16_bits_to_f64(mi.normal_bf16(0, 1, 1024, shift=3))
    assert np.array_equal(y, 8.0 * x[:1024])
