// Chunk-major decode: the decode step (one new token per request) for batches whose requests list the
// same chunks.  The paper observes that retrieval is skewed: a small share of the chunks takes most of
// the hits (Section III-B / V: re-use of materialised KVs across requests).  A request-major kernel
// reads a chunk once per request that lists it; here the work item is a CHUNK (up to `n_tiles` tiles of
// it, one KV head, one layer) and the query rows of every request that lists it are stacked into the 16
// rows of the MMA tile (16 / G requests), so the chunk's K and V rows cross HBM once for all of them.
// Items with more requests than fit are repeated for the next 16 / G requests right after (the second
// read hits L2).  Every (item, request) pair leaves one normalised partial (o, lse); each request's
// tail (its suffix and generated tokens plus the step's new token, appended on the way) is one more
// item; the last partial of a (layer, request, KV head) to arrive merges them all by log-sum-exp
// (atomic ticket, nobody waits).
//
// Scheduling: one persistent CTA per SM; the producer thread of a CTA draws the next item from a
// global counter (items are ordered layer, KV head, chunk, so neighbours in time read neighbouring
// data), feeds the same TMA ring as the request-major kernel and tells the consumer warps which item
// the tiles belong to through a small queue in shared memory.  All waits are bounded.
#include <algorithm>

#include "stream_common.cuh"

namespace matkv {

constexpr int kItemQ = 16;  // depth of the producer -> consumers item queue (the ring holds fewer tiles than that)

struct SharedParams {
    const DevReq *reqs;
    const CUtensorMap *tmaps;   // [n_seg_total] chunk maps, then tail K, tail V
    const DevItem *items;
    int32_t n_seg_total, n_items, parts_total;
    const int32_t *tail_len;
    __nv_bfloat16 *tail_k, *tail_v;
    const __nv_bfloat16 *q;
    __nv_bfloat16 *out;
    float *lse_out;
    int64_t q_sl, q_sb, lse_sl, lse_sb;
    int32_t layer0, n_layers_launch, n_layers_total, B, Hkv, max_tail;
    float scale_log2;
    int32_t *counters;          // [layers of the launch][Hkv][B] arrival counters, zero between launches
    float *part_lse, *part_o;   // [layers][Hkv][parts_total][G] (x D)
    int32_t *status;
    int32_t advance;
    int32_t *done_count;        // CTAs that have finished (reset by the last one)
    int32_t *work;              // next item to hand out (reset by the last CTA)
};

template <int D, int G>
struct SharedCfg {
    static constexpr int R = kShareRows / G;               // requests stacked in one item
    static constexpr int NBOX = D / 64;
    static constexpr int BOX_BYTES = kTile * 128;
    static constexpr int STAGE_BYTES = 2 * NBOX * BOX_BYTES;
    static constexpr int KS = D / 16;
    // merge area: one 64-column half of O per warp and row, then m, l, rounded l per warp and row
    static constexpr int MERGE_BYTES = (kCW * kShareRows * (64 + 3) * 4 + 15) / 16 * 16;
    static constexpr int FIXED_BYTES = MERGE_BYTES + 1024 + 1024;
    static constexpr int NSTAGE_MAX = (kMaxDynSmem - FIXED_BYTES) / STAGE_BYTES;
    static constexpr int NSTAGE = NSTAGE_MAX > 12 ? 12 : NSTAGE_MAX;
    static constexpr int SMEM_BYTES = NSTAGE * STAGE_BYTES + FIXED_BYTES;
    static_assert(kShareRows % G == 0, "unsupported group size");
    static_assert(D % 64 == 0 && NSTAGE >= 3 && NSTAGE < kItemQ, "unsupported head_dim");
};

// What an item id stands for.  Ids run over (layer of the launch, KV head, item of the table), the table's
// chunk items first and then one tail item per request.
struct ItemPos {
    int32_t l_rel, g, k;
    int32_t n_tiles;            // tiles of the item (a tail item: the tail's tiles and one tile for the new token)
    int32_t tail_tiles, t0, b;  // tail items only (b < 0 for a chunk item)
    int32_t tmap, len, tile0;   // chunk items only
};

struct CurItem {
    ItemPos u;
    int32_t n_req, id;
};

__device__ __forceinline__ int32_t shared_t0(const SharedParams &p, int b) {
    int32_t t0 = p.tail_len[b];
    if (t0 < 0 || t0 + 1 > p.max_tail) {
        atomicCAS(p.status, 0, MATKV_E_CAPACITY);
        t0 = max(0, min(t0, p.max_tail - 1));
    }
    return t0;
}

__device__ __forceinline__ void locate_item(const SharedParams &p, int32_t id, ItemPos &u) {
    const int32_t per_head = p.n_items + p.B;
    const int32_t lg = id / per_head;
    u.k = id % per_head;
    u.l_rel = lg / p.Hkv;
    u.g = lg % p.Hkv;
    if (u.k < p.n_items) {
        const int4 h = *(const int4 *)(p.items + u.k);  // tmap, len, tile0, n_tiles
        u.tmap = h.x; u.len = h.y; u.tile0 = h.z; u.n_tiles = h.w;
        u.b = -1; u.t0 = 0; u.tail_tiles = 0;
    } else {
        u.b = u.k - p.n_items;
        u.t0 = shared_t0(p, u.b);
        u.tail_tiles = ceil_div(u.t0, kTile);
        u.n_tiles = u.tail_tiles + 1;
        u.tmap = 0; u.len = 0; u.tile0 = 0;
    }
}

template <int D, int G>
__global__ void __launch_bounds__(kThreads, 1)
k_attend_shared(const __grid_constant__ SharedParams p, const __grid_constant__ CUtensorMap kn_map, const __grid_constant__ CUtensorMap vn_map) {
    using C = SharedCfg<D, G>;
    extern __shared__ unsigned char smem_raw[];
    unsigned char *smem = (unsigned char *)(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
    unsigned char *ring = smem;
    float *merge_o = (float *)(smem + C::NSTAGE * C::STAGE_BYTES);  // [warp][row][64]
    float *merge_m = merge_o + kCW * kShareRows * 64;               // [warp][row]  (log2 units, scaled)
    float *merge_l = merge_m + kCW * kShareRows;
    float *merge_r = merge_l + kCW * kShareRows;
    unsigned char *misc = smem + C::NSTAGE * C::STAGE_BYTES + C::MERGE_BYTES;
    uint64_t *bars = (uint64_t *)misc;                                            // full[NSTAGE], empty[NSTAGE]
    volatile uint32_t *tags = (volatile uint32_t *)(misc + 2 * 12 * 8);           // per stage: rows | kTagNew | fill << 16
    volatile unsigned long long *item_q = (volatile unsigned long long *)(misc + 2 * 12 * 8 + 12 * 4 + 8);  // (k + 1) << 32 | id
    volatile int *flags = (volatile int *)(misc + 2 * 12 * 8 + 12 * 4 + 8 + kItemQ * 8);  // [0] abort, [1..] last-arriver per stacked request
    int64_t *row_slot = (int64_t *)(misc + 2 * 12 * 8 + 12 * 4 + 8 + kItemQ * 8 + (2 + kShareRows) * 4);  // [R] partial slot per stacked request
    int32_t *row_req = (int32_t *)(row_slot + kShareRows);   // [R] request
    int32_t *row_np = row_req + kShareRows;                  // [R] parts of that request
    volatile CurItem *curv = (volatile CurItem *)(row_np + kShareRows);
    CurItem *cur = const_cast<CurItem *>(curv);

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    if (tid == 0) {
        for (int s = 0; s < C::NSTAGE; ++s) {
            mbar_init(smem_u32(bars + s), 1);
            mbar_init(smem_u32(bars + C::NSTAGE + s), kItems);
            tags[s] = 0xffff0000u;
        }
        for (int s = 0; s < kItemQ; ++s) item_q[s] = 0ull;
        for (int s = 0; s < 2 + kShareRows; ++s) flags[s] = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    __syncthreads();
    const int32_t n_ids = p.n_layers_launch * p.Hkv * (p.n_items + p.B);
    const uint32_t ring_u32 = smem_u32(ring), full_u32 = smem_u32(bars), empty_u32 = smem_u32(bars + C::NSTAGE);

    if (warp == kCW) {
        // ================= producer: draws items and feeds the ring =================
        if (lane != 0) return;
        uint32_t seq = 0, kq = 0;
        bool ok = true;
        while (ok) {
            const int32_t id = atomicAdd(p.work, 1);
            if (id >= n_ids) {
                item_q[kq % kItemQ] = ((unsigned long long)(kq + 1) << 32) | 0xffffffffull;
                break;
            }
            item_q[kq % kItemQ] = ((unsigned long long)(kq + 1) << 32) | (uint32_t)id;
            ++kq;
            ItemPos u;
            locate_item(p, id, u);
            const int layer = p.layer0 + u.l_rel;
            for (int t = 0; t < u.n_tiles; ++t, ++seq) {
                const uint32_t stage = seq % C::NSTAGE, use = seq / C::NSTAGE;
                if (use > 0 && !mbar_wait(empty_u32 + stage * 8, (use - 1) & 1, flags)) {
                    ok = false;
                    break;
                }
                const uint32_t bar = full_u32 + stage * 8, dst = ring_u32 + stage * C::STAGE_BYTES;
                if (u.b >= 0 && t == u.tail_tiles) {  // the step's new token, from k_new / v_new [layer][request][head][D]
                    const int32_t z = u.l_rel * p.B + u.b;
                    tags[stage] = 1u | kTagNew | (use << 16);
                    mbar_expect_tx(bar, C::STAGE_BYTES);
#pragma unroll
                    for (int bx = 0; bx < C::NBOX; ++bx) {
                        tma_load_3d(dst + bx * C::BOX_BYTES, &kn_map, bx * 64, u.g, z, bar);
                        tma_load_3d(dst + (C::NBOX + bx) * C::BOX_BYTES, &vn_map, bx * 64, u.g, z, bar);
                    }
                    continue;
                }
                const CUtensorMap *mk, *mv;
                int32_t yk, yv, rows;
                if (u.b < 0) {
                    const int r0 = (u.tile0 + t) * kTile;
                    mk = mv = p.tmaps + u.tmap;
                    yk = ((layer * 2) * p.Hkv + u.g) * u.len + r0;
                    yv = ((layer * 2 + 1) * p.Hkv + u.g) * u.len + r0;
                    rows = min(kTile, u.len - r0);
                } else {
                    const int r0 = t * kTile;
                    mk = p.tmaps + p.n_seg_total;
                    mv = mk + 1;
                    yk = yv = ((u.b * p.n_layers_total + layer) * p.Hkv + u.g) * p.max_tail + r0;
                    rows = min(kTile, u.t0 - r0);
                }
                tags[stage] = (uint32_t)rows | (use << 16);
                mbar_expect_tx(bar, C::STAGE_BYTES);
#pragma unroll
                for (int bx = 0; bx < C::NBOX; ++bx) {
                    tma_load_2d(dst + bx * C::BOX_BYTES, mk, bx * 64, yk, bar);
                    tma_load_2d(dst + (C::NBOX + bx) * C::BOX_BYTES, mv, bx * 64, yv, bar);
                }
            }
        }
        if (!ok) {
            // gave up: tell the consumers there is nothing more, then wait (bounded) for the copies in flight
            atomicCAS(p.status, 0, MATKV_E_TIMEOUT);
            item_q[kq % kItemQ] = ((unsigned long long)(kq + 1) << 32) | 0xffffffffull;
            const uint32_t lo = seq > (uint32_t)C::NSTAGE ? seq - C::NSTAGE : 0;
            for (uint32_t s2 = lo; s2 < seq; ++s2) {
                const long long t0 = clock64();
                while (!mbar_try_wait(full_u32 + (s2 % C::NSTAGE) * 8, (s2 / C::NSTAGE) & 1) && clock64() - t0 < kWaitCycles) {}
            }
        }
        return;
    }

    // ================= consumers =================
    const int qr = lane >> 2, qc = lane & 3;   // mma rows qr and qr + 8, column pair qc
    const int mi = lane >> 3, ri = lane & 7;   // ldmatrix addressing

    uint32_t qa[C::KS][4];   // A fragments of Q: rows qr / qr+8, k columns 0-7 / 8-15 of every k-step
    float o[2 * C::KS][4];   // O accumulators: [8-column block of d][row qr: c0, c1; row qr+8: c2, c3]
    float m_run[2], l_run[2], l_rnd[2];

    int64_t j_base = 0;      // CTA-local index of the item's first tile
    for (uint32_t kq = 0;; ++kq) {
        // ---- which item: warp 0 reads the queue (bounded wait) and lays the item out for everybody ----
        if (warp == 0) {
            int32_t id = -1;
            if (lane == 0) {
                unsigned long long v = item_q[kq % kItemQ];
                if ((uint32_t)(v >> 32) != kq + 1) {
                    const long long t0 = clock64();
                    while (true) {
                        v = item_q[kq % kItemQ];
                        if ((uint32_t)(v >> 32) == kq + 1 || *flags) break;
                        if (clock64() - t0 > kWaitCycles) {
                            *flags = 1;
                            break;
                        }
                    }
                }
                if ((uint32_t)(v >> 32) == kq + 1) id = (int32_t)(uint32_t)v;
            }
            id = __shfl_sync(0xffffffffu, id, 0);
            if (id >= 0) {
                ItemPos w;
                locate_item(p, id, w);
                const int lgw = w.l_rel * p.Hkv + w.g;
                int nr = 1;
                if (w.b < 0) {
                    nr = p.items[w.k].n_req;
                    if (lane < nr) {
                        const int b = p.items[w.k].req[lane];
                        const DevReq rq = p.reqs[b];
                        row_req[lane] = b;
                        row_np[lane] = rq.n_parts;
                        row_slot[lane] = (int64_t)lgw * p.parts_total + rq.part_base + p.items[w.k].part[lane];
                    }
                } else if (lane == 0) {
                    const DevReq rq = p.reqs[w.b];
                    row_req[0] = w.b;
                    row_np[0] = rq.n_parts;
                    row_slot[0] = (int64_t)lgw * p.parts_total + rq.part_base + rq.n_parts - 1;
                }
                if (lane == 0) {
                    cur->u = w;
                    cur->n_req = nr;
                }
            }
            if (lane == 0) cur->id = id;
        }
        consumer_bar();
        if (cur->id < 0) break;
        const ItemPos u = cur->u;
        const int n_req = cur->n_req;
        const int layer = p.layer0 + u.l_rel;
        const int lg = u.l_rel * p.Hkv + u.g;
        const int n_rows = n_req * G;
        // ---- per-item setup: the stacked requests' query rows ----
#pragma unroll
        for (int hh = 0; hh < 2; ++hh) {
            const int r = qr + 8 * hh;
            const bool real = r < n_rows;
            const __nv_bfloat16 *qrow =
                p.q + (int64_t)u.l_rel * p.q_sl + (int64_t)(real ? row_req[r / G] : 0) * p.q_sb + (int64_t)(u.g * G + r % G) * D;
#pragma unroll
            for (int ks = 0; ks < C::KS; ++ks) {
                qa[ks][hh] = real ? *(const uint32_t *)(qrow + ks * 16 + 2 * qc) : 0u;
                qa[ks][2 + hh] = real ? *(const uint32_t *)(qrow + ks * 16 + 8 + 2 * qc) : 0u;
            }
            m_run[hh] = -CUDART_INF_F;
            l_run[hh] = 0.f;
            l_rnd[hh] = 0.f;
        }
#pragma unroll
        for (int nb = 0; nb < 2 * C::KS; ++nb) o[nb][0] = o[nb][1] = o[nb][2] = o[nb][3] = 0.f;

        // ---- this warp's 16-token pieces of the item ----
        const int64_t hj_begin = j_base * kItems, hj_end = (j_base + u.n_tiles) * kItems;
        int64_t hj = hj_begin + (int)((warp - hj_begin % kCW + kCW) % kCW);
        for (; hj < hj_end; hj += kCW) {
            const uint32_t j = (uint32_t)(hj / kItems);
            const int r0 = (int)(hj % kItems) * kItemRows;
            const uint32_t stage = j % C::NSTAGE, use = j / C::NSTAGE;
            const uint32_t tag = stage_wait(tags + stage, use, full_u32 + stage * 8, use & 1, flags);
            const uint32_t stage_u32 = ring_u32 + stage * C::STAGE_BYTES;
            const int vis = (int)(tag & 0x7f) - r0;   // valid tokens of this piece (may be <= 0)
            if (vis > 0) {
                // ---------- S = Q K^T for 16 tokens ----------
                float s0[4] = {0.f, 0.f, 0.f, 0.f}, s1[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
                for (int ks = 0; ks < C::KS; ++ks) {
                    const int c = (ks * 2 + (mi & 1)) & 7;
                    uint32_t kb[4];
                    ldsm_x4(stage_u32 + (ks / 4) * C::BOX_BYTES + swz(r0 + (mi >> 1) * 8 + ri, c), kb);
                    mma_bf16(s0, qa[ks][0], qa[ks][1], qa[ks][2], qa[ks][3], kb[0], kb[1]);
                    mma_bf16(s1, qa[ks][0], qa[ks][1], qa[ks][2], qa[ks][3], kb[2], kb[3]);
                }
                // ---------- online softmax: rows qr (c0, c1) and qr + 8 (c2, c3); tokens 2qc, 2qc+1, 8+2qc, 9+2qc ----------
                uint32_t pa[4];
                float alpha[2];
#pragma unroll
                for (int hh = 0; hh < 2; ++hh) {
                    const float x0 = 2 * qc < vis ? s0[2 * hh] * p.scale_log2 : -CUDART_INF_F;
                    const float x1 = 2 * qc + 1 < vis ? s0[2 * hh + 1] * p.scale_log2 : -CUDART_INF_F;
                    const float x2 = 8 + 2 * qc < vis ? s1[2 * hh] * p.scale_log2 : -CUDART_INF_F;
                    const float x3 = 9 + 2 * qc < vis ? s1[2 * hh + 1] * p.scale_log2 : -CUDART_INF_F;
                    float tmax = fmaxf(fmaxf(x0, x1), fmaxf(x2, x3));
                    tmax = fmaxf(tmax, __shfl_xor_sync(0xffffffffu, tmax, 1));
                    tmax = fmaxf(tmax, __shfl_xor_sync(0xffffffffu, tmax, 2));
                    const float m_new = fmaxf(m_run[hh], tmax);   // finite: token 0 of the piece is visible to every row
                    alpha[hh] = fast_exp2(m_run[hh] - m_new);
                    const float p0 = fast_exp2(x0 - m_new), p1 = fast_exp2(x1 - m_new);
                    const float p2 = fast_exp2(x2 - m_new), p3 = fast_exp2(x3 - m_new);
                    pa[hh] = pack_bf16(p0, p1);
                    pa[2 + hh] = pack_bf16(p2, p3);
                    l_run[hh] = l_run[hh] * alpha[hh] + ((p0 + p1) + (p2 + p3));
                    l_rnd[hh] = l_rnd[hh] * alpha[hh] + ((bf_lo(pa[hh]) + bf_hi(pa[hh])) + (bf_lo(pa[2 + hh]) + bf_hi(pa[2 + hh])));
                    m_run[hh] = m_new;
                }
                if (__any_sync(0xffffffffu, alpha[0] != 1.0f || alpha[1] != 1.0f)) {
#pragma unroll
                    for (int nb = 0; nb < 2 * C::KS; ++nb) {
                        o[nb][0] *= alpha[0];
                        o[nb][1] *= alpha[0];
                        o[nb][2] *= alpha[1];
                        o[nb][3] *= alpha[1];
                    }
                }
                // ---------- O += P V ----------
                const uint32_t v_u32 = stage_u32 + C::NBOX * C::BOX_BYTES;
#pragma unroll
                for (int dp = 0; dp < C::KS; ++dp) {
                    const int c = (dp * 2 + (mi >> 1)) & 7;
                    uint32_t vb[4];
                    ldsm_x4_trans(v_u32 + (dp / 4) * C::BOX_BYTES + swz(r0 + (mi & 1) * 8 + ri, c), vb);
                    mma_bf16(o[2 * dp], pa[0], pa[1], pa[2], pa[3], vb[0], vb[1]);
                    mma_bf16(o[2 * dp + 1], pa[0], pa[1], pa[2], pa[3], vb[2], vb[3]);
                }
                // ---------- the new token goes to the request's tail for later steps ----------
                if ((tag & kTagNew) && r0 == 0 && u.t0 < p.max_tail) {
                    constexpr int CPR = D / 8;  // 16-byte chunks per row; lanes 0..CPR-1 move K, the next CPR lanes move V
                    const unsigned char *ring_stage = ring + stage * C::STAGE_BYTES;
                    const int64_t off = ((((int64_t)u.b * p.n_layers_total + layer) * p.Hkv + u.g) * p.max_tail + u.t0) * D;
                    const int ch = lane % CPR, kv = lane / CPR;
                    if (kv < 2) {
                        const uint4 val = *(const uint4 *)(ring_stage + kv * C::NBOX * C::BOX_BYTES + (ch / 8) * C::BOX_BYTES + swz(0, ch % 8));
                        *(uint4 *)((kv ? p.tail_v : p.tail_k) + off + ch * 8) = val;
                    }
                }
            }
            __syncwarp();
            if (lane == 0) mbar_arrive(empty_u32 + stage * 8);
        }

        // ---- end of the item: merge the warps' states, one 64-column half of O at a time ----
        {
#pragma unroll
            for (int hh = 0; hh < 2; ++hh) {
                float l_tot = l_run[hh], r_tot = l_rnd[hh];
                l_tot += __shfl_xor_sync(0xffffffffu, l_tot, 1);
                l_tot += __shfl_xor_sync(0xffffffffu, l_tot, 2);
                r_tot += __shfl_xor_sync(0xffffffffu, r_tot, 1);
                r_tot += __shfl_xor_sync(0xffffffffu, r_tot, 2);
                if (qc == 0) {
                    merge_m[warp * kShareRows + qr + 8 * hh] = m_run[hh];
                    merge_l[warp * kShareRows + qr + 8 * hh] = l_tot;
                    merge_r[warp * kShareRows + qr + 8 * hh] = r_tot;
                }
            }
        }
#pragma unroll
        for (int half = 0; half < D / 64; ++half) {
            if (half) consumer_bar();  // the previous half has been read
#pragma unroll
            for (int nb = 0; nb < 8; ++nb) {
                *(float2 *)(merge_o + (warp * kShareRows + qr) * 64 + nb * 8 + 2 * qc) = make_float2(o[half * 8 + nb][0], o[half * 8 + nb][1]);
                *(float2 *)(merge_o + (warp * kShareRows + qr + 8) * 64 + nb * 8 + 2 * qc) = make_float2(o[half * 8 + nb][2], o[half * 8 + nb][3]);
            }
            consumer_bar();
            for (int idx = tid; idx < n_rows * 64; idx += kCW * 32) {
                const int r = idx >> 6, d = half * 64 + (idx & 63);
                float M = -CUDART_INF_F;
#pragma unroll
                for (int w = 0; w < kCW; ++w) M = fmaxf(M, merge_m[w * kShareRows + r]);
                float acc = 0.f, L = 0.f, Lr = 0.f;
#pragma unroll
                for (int w = 0; w < kCW; ++w) {
                    const float mw = merge_m[w * kShareRows + r];
                    const float sw = mw == -CUDART_INF_F ? 0.f : fast_exp2(mw - M);
                    acc = fmaf(sw, merge_o[(w * kShareRows + r) * 64 + (idx & 63)], acc);
                    L = fmaf(sw, merge_l[w * kShareRows + r], L);
                    Lr = fmaf(sw, merge_r[w * kShareRows + r], Lr);
                }
                const float ov = acc / Lr;
                const int j = r / G, h = r % G;
                if (row_np[j] == 1) {  // a request without chunks: its tail item is the whole answer
                    p.out[(int64_t)u.l_rel * p.q_sl + (int64_t)row_req[j] * p.q_sb + (int64_t)(u.g * G + h) * D + d] = __float2bfloat16(ov);
                    if (p.lse_out && d == 0)
                        p.lse_out[(int64_t)u.l_rel * p.lse_sl + (int64_t)row_req[j] * p.lse_sb + u.g * G + h] = (M + log2f(L)) * kLn2;
                } else {
                    p.part_o[(row_slot[j] * G + h) * D + d] = ov;
                    if (d == 0) p.part_lse[row_slot[j] * G + h] = (M + log2f(L)) * kLn2;
                }
            }
        }
        // ---- arrival tickets: the last partial of a (layer, request, KV head) merges them all ----
        __threadfence();
        consumer_bar();
        if (tid < n_req) {
            int last = 0;
            if (row_np[tid] > 1) {
                int32_t *cnt = p.counters + (int64_t)lg * p.B + row_req[tid];
                last = atomicAdd(cnt, 1) == row_np[tid] - 1;
                if (last) *cnt = 0;  // ready for the next launch
            }
            flags[2 + tid] = last;
        }
        consumer_bar();
        for (int pr = warp; pr < n_rows; pr += kCW) {
            const int j = pr / G, h = pr % G;
            if (!flags[2 + j]) continue;
            __threadfence();
            const DevReq rq = p.reqs[row_req[j]];
            const int64_t first = (int64_t)lg * p.parts_total + rq.part_base;
            combine_warp(p.part_o + (first * G + h) * D, (int64_t)G * D, p.part_lse + first * G + h, G, rq.n_parts, D,
                         p.out + (int64_t)u.l_rel * p.q_sl + (int64_t)row_req[j] * p.q_sb + (int64_t)(u.g * G + h) * D,
                         p.lse_out ? p.lse_out + (int64_t)u.l_rel * p.lse_sl + (int64_t)row_req[j] * p.lse_sb + u.g * G + h : nullptr);
        }
        consumer_bar();  // merge area, row tables and flags are free again
        j_base += u.n_tiles;
    }
    if (flags[0] && tid == 0) atomicCAS(p.status, 0, MATKV_E_TIMEOUT);
    // the last CTA of the launch to get here re-arms the work counter and, if asked, moves every tail length
    if (tid == 0) {
        __threadfence();
        if (atomicAdd(p.done_count, 1) == (int)gridDim.x - 1) {
            if (p.advance > 0)
                for (int b = 0; b < p.B; ++b) {
                    int32_t v = p.tail_len[b] + p.advance;
                    if (v > p.max_tail) {
                        v = p.max_tail;
                        atomicCAS(p.status, 0, MATKV_E_CAPACITY);
                    }
                    const_cast<int32_t *>(p.tail_len)[b] = v;
                }
            *p.work = 0;
            *p.done_count = 0;
        }
    }
}

template <int D, int G>
static int launch_shared_t(const SharedParams &p, const CUtensorMap &kn_map, const CUtensorMap &vn_map, int grid, cudaStream_t stream) {
    using C = SharedCfg<D, G>;
    static bool configured = false;
    if (!configured) {
        MATKV_CUDA(cudaFuncSetAttribute(k_attend_shared<D, G>, cudaFuncAttributeMaxDynamicSharedMemorySize, C::SMEM_BYTES));
        configured = true;
    }
    k_attend_shared<D, G><<<grid, kThreads, C::SMEM_BYTES, stream>>>(p, kn_map, vn_map);
    MATKV_CUDA(cudaGetLastError());
    return MATKV_OK;
}

static size_t align256(size_t x) { return (x + 255) / 256 * 256; }

size_t shared_region_bytes(const matkv_config &c, const matkv_table *t, int n_layers_launch) {
    const int G = c.n_q_heads / c.n_kv_heads;
    const size_t rows = (size_t)n_layers_launch * c.n_kv_heads * (size_t)t->parts_total * G;
    return align256(rows * sizeof(float)) + align256(rows * c.head_dim * sizeof(float));
}

int launch_attend_shared(matkv_ctx *ctx, matkv_table *t, const AttendArgs &a, void *region, size_t region_bytes, cudaStream_t stream) {
    const matkv_config &c = ctx->cfg;
    const int G = c.n_q_heads / c.n_kv_heads;
    if (a.S != 1) return fail(MATKV_E_INVALID_ARG, "the chunk-major kernel handles decode steps only");
    if (region_bytes < shared_region_bytes(c, t, a.n_layers_launch))
        return fail(MATKV_E_CAPACITY, "chunk-major decode needs %zu bytes of scratch, %zu given", shared_region_bytes(c, t, a.n_layers_launch),
                    region_bytes);
    WorkspaceView ws;
    workspace_bytes_for(c, &ws, ctx->workspace);
    if ((int64_t)a.n_layers_launch * c.n_kv_heads * t->batch > ws.n_counter_slots)
        return fail(MATKV_E_CAPACITY, "launch exceeds the workspace's arrival counters");
    SharedParams p;
    p.reqs = t->d_reqs;
    p.tmaps = t->d_tmaps;
    p.items = t->d_items;
    p.n_seg_total = t->n_seg_total;
    p.n_items = t->n_items;
    p.parts_total = t->parts_total;
    p.tail_len = t->d_tail_len;
    p.tail_k = t->tail_k;
    p.tail_v = t->tail_v;
    p.q = a.q; p.out = a.out; p.lse_out = a.lse_out;
    p.q_sl = a.q_sl; p.q_sb = a.q_sb; p.lse_sl = a.lse_sl; p.lse_sb = a.lse_sb;
    p.layer0 = a.layer0; p.n_layers_launch = a.n_layers_launch; p.n_layers_total = c.n_layers;
    p.B = t->batch; p.Hkv = c.n_kv_heads; p.max_tail = c.max_tail_tokens;
    p.scale_log2 = ctx->scale * kLog2e;
    p.counters = ws.counters;
    const size_t rows = (size_t)a.n_layers_launch * c.n_kv_heads * (size_t)t->parts_total * G;
    p.part_lse = (float *)region;
    p.part_o = (float *)((char *)region + align256(rows * sizeof(float)));
    p.status = ctx->d_status;
    p.advance = a.advance;
    p.done_count = ctx->d_status + 2;
    p.work = ctx->d_status + 3;
    CUtensorMap kn_map, vn_map;
    {
        const uint64_t n_tok = (uint64_t)a.n_layers_launch * t->batch;
        int rc = encode_new_rows_map(&kn_map, a.k_new, c.head_dim, c.n_kv_heads, n_tok);
        if (!rc) rc = encode_new_rows_map(&vn_map, a.v_new, c.head_dim, c.n_kv_heads, n_tok);
        if (rc) return rc;
    }
    const int64_t n_ids = (int64_t)a.n_layers_launch * c.n_kv_heads * (t->n_items + t->batch);
    if (n_ids > 0x7fff0000ll) return fail(MATKV_E_CAPACITY, "launch of %lld items", (long long)n_ids);
    int64_t grid = ctx->opt_decode_ctas > 0 ? ctx->opt_decode_ctas : ctx->n_sm;
    grid = std::max<int64_t>(1, std::min<int64_t>(grid, n_ids));
#define MATKV_CASE(DD, GG) \
    if (c.head_dim == DD && G == GG) return launch_shared_t<DD, GG>(p, kn_map, vn_map, (int)grid, stream);
    MATKV_CASE(128, 1) MATKV_CASE(128, 2) MATKV_CASE(128, 4) MATKV_CASE(128, 8)
    MATKV_CASE(64, 1) MATKV_CASE(64, 2) MATKV_CASE(64, 4) MATKV_CASE(64, 8)
#undef MATKV_CASE
    return fail(MATKV_E_INVALID_ARG, "unsupported head_dim %d / group %d", c.head_dim, G);
}

}  // namespace matkv
