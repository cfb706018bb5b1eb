// Chunk-major decode: the decode step (one new token per request) for batches whose requests list the
// same chunks.  The paper observes that retrieval is skewed: a small share of the chunks takes most of
// the hits (Section II-C, the access-skew figure: most chunks are retrieved by several queries).  A request-major kernel
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
// data), looks it up, feeds the same TMA ring as the request-major kernel and hands the consumer warps the
// item's description through a small queue in shared memory.  All waits are bounded.
#include <algorithm>

#include "stream_common.cuh"

namespace matkv {

constexpr int kPend = 96;   // (item, stacked request) pairs whose arrival tickets are drawn together
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
    // merge area: one 64-column half of O per warp and row, then m, l, rounded l per warp and row, the rows' maxima
    static constexpr int MERGE_BYTES = ((kCW * kShareRows * (64 + 3) + kShareRows) * 4 + 15) / 16 * 16;
    static constexpr int MISC_BYTES = 3840;                // barriers, tags, flags, the item queue
    static constexpr int FIXED_BYTES = MERGE_BYTES + MISC_BYTES + 1024;  // + slack for the 1024-byte alignment of the ring
    static constexpr int NSTAGE_MAX = (kMaxDynSmem - FIXED_BYTES) / STAGE_BYTES;
    static constexpr int NSTAGE_CAP = 192 * 1024 / STAGE_BYTES;
    static constexpr int NSTAGE = NSTAGE_MAX > NSTAGE_CAP ? NSTAGE_CAP : NSTAGE_MAX;
    static constexpr int SMEM_BYTES = NSTAGE * STAGE_BYTES + FIXED_BYTES;
    static_assert(kShareRows % G == 0, "unsupported group size");
    // the producer runs at most NSTAGE + 1 items ahead of the consumers: the queue must be deeper than that
    static_assert(D % 64 == 0 && NSTAGE >= 3 && NSTAGE + 3 <= kItemQ, "unsupported head_dim");
};

// One entry of the producer -> consumers item queue: everything the consumers need to know about an item,
// looked up by the producer while it is ahead.  Item ids run over (layer of the launch, KV head, item of the
// table); the table's chunk items come first, then one tail item per request.
struct QEntry {
    uint32_t seq1;              // number of the item in this CTA's sequence, plus one; written last
    int32_t id;                 // < 0: no more items
    int32_t l_rel, g;
    int32_t n_tiles;            // tiles of the item (a tail item: the tail's tiles and one tile for the new token)
    int32_t n_req;              // requests stacked in the item
    int32_t b, t0;              // tail items: request and tail length (b < 0 for a chunk item)
    int32_t tmap, len, tile0;   // chunk items: descriptor, chunk tokens, first tile
    int32_t last_read;          // nothing reads these tiles again in this launch: load them with the evict-first L2 policy
    int32_t part[kShareRows];   // partial slot of (item, stacked request) inside one (layer, KV head)
    int16_t req[kShareRows];    // stacked requests
    int16_t np[kShareRows];     // partials each of them collects
};
static_assert(sizeof(QEntry) == 48 + 64 + 64, "queue entry layout");

__device__ __forceinline__ int32_t shared_t0(const SharedParams &p, int b) {
    int32_t t0 = p.tail_len[b];
    if (t0 < 0 || t0 + 1 > p.max_tail) {
        atomicCAS(p.status, 0, MATKV_E_CAPACITY);
        t0 = max(0, min(t0, p.max_tail - 1));
    }
    return t0;
}

// Producer side: looks item `id` up and fills a queue entry (everything but seq1).
__device__ __forceinline__ void locate_item(const SharedParams &p, int32_t id, volatile QEntry *e) {
    const int32_t per_head = p.n_items + p.B;
    const int32_t lg = id / per_head, k = id % per_head;
    e->id = id;
    e->l_rel = lg / p.Hkv;
    e->g = lg % p.Hkv;
    if (k < p.n_items) {
        const int4 *it = (const int4 *)(p.items + k);
        const int4 h0 = it[0], h1 = it[1];  // tmap, len, tile0, n_tiles; n_req
        e->tmap = h0.x; e->len = h0.y; e->tile0 = h0.z; e->n_tiles = h0.w;
        e->n_req = h1.x;
        e->last_read = h1.y;
        e->b = -1; e->t0 = 0;
        int4 rq[4], pt[4], np[4];
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            rq[i] = it[2 + i];
            pt[i] = it[6 + i];
            np[i] = it[10 + i];
        }
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            e->req[4 * i] = (int16_t)rq[i].x; e->req[4 * i + 1] = (int16_t)rq[i].y;
            e->req[4 * i + 2] = (int16_t)rq[i].z; e->req[4 * i + 3] = (int16_t)rq[i].w;
            e->part[4 * i] = pt[i].x; e->part[4 * i + 1] = pt[i].y; e->part[4 * i + 2] = pt[i].z; e->part[4 * i + 3] = pt[i].w;
            e->np[4 * i] = (int16_t)np[i].x; e->np[4 * i + 1] = (int16_t)np[i].y;
            e->np[4 * i + 2] = (int16_t)np[i].z; e->np[4 * i + 3] = (int16_t)np[i].w;
        }
    } else {
        const int b = k - p.n_items;
        const DevReq rq = p.reqs[b];
        const int32_t t0 = shared_t0(p, b);
        e->b = b; e->t0 = t0;
        e->n_tiles = ceil_div(t0, kTile) + 1;
        e->n_req = 1;
        e->last_read = 1;
        e->tmap = 0; e->len = 0; e->tile0 = 0;
        e->req[0] = (int16_t)b;
        e->part[0] = rq.part_base + rq.n_parts - 1;
        e->np[0] = (int16_t)rq.n_parts;
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
    float *row_max = merge_r + kCW * kShareRows;                    // [row] overall running maximum of the item
    unsigned char *misc = smem + C::NSTAGE * C::STAGE_BYTES + C::MERGE_BYTES;
    uint64_t *bars = (uint64_t *)misc;                                   // full[NSTAGE], empty[NSTAGE]
    volatile uint32_t *tags = (volatile uint32_t *)(misc + 2 * 12 * 8);  // per stage: rows | kTagNew | fill << 16
    volatile QEntry *item_q = (volatile QEntry *)(misc + 256);           // [kItemQ]
    volatile int *flags = (volatile int *)(misc + 256 + kItemQ * sizeof(QEntry));  // [0] abort, [1] end of items
    int32_t *pend_idx = (int32_t *)(misc + 256 + kItemQ * sizeof(QEntry) + 8);   // [kPend] arrival counter of a pending pair
    int16_t *pend_np = (int16_t *)(pend_idx + kPend);                             // [kPend] partials its row collects
    uint8_t *pend_last = (uint8_t *)(pend_np + kPend);                            // [kPend] this CTA delivered the last one
    static_assert(256 + kItemQ * sizeof(QEntry) + 8 + kPend * 7 <= C::MISC_BYTES, "misc area");

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    if (tid == 0) {
        for (int s = 0; s < C::NSTAGE; ++s) {
            mbar_init(smem_u32(bars + s), 1);
            mbar_init(smem_u32(bars + C::NSTAGE + s), kItems);
            tags[s] = 0xffff0000u;
        }
        for (int s = 0; s < kItemQ; ++s) item_q[s].seq1 = 0u;
        flags[0] = flags[1] = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    __syncthreads();
    const int32_t n_ids = p.n_layers_launch * p.Hkv * (p.n_items + p.B);
    const uint32_t ring_u32 = smem_u32(ring), full_u32 = smem_u32(bars), empty_u32 = smem_u32(bars + C::NSTAGE);

    if (warp == kCW) {
        // ================= producer: draws items, looks them up and feeds the ring =================
        if (lane != 0) return;
        // entry kq of the queue is filled and published while the tiles of item kq - 1 are being issued: a pause
        // of the producer (an atomic round trip, then dependent loads) would drain the ring, which is no deeper
        // than the memory latency
        auto publish = [&](uint32_t kq, int32_t id) {
            volatile QEntry *e = item_q + kq % kItemQ;
            if (id < n_ids) locate_item(p, id, e);
            else e->id = -1;
            __threadfence_block();
            e->seq1 = kq + 1;
        };
        const uint64_t pol_stream = l2_policy_evict_first(), pol_keep = l2_policy_evict_normal();
        uint32_t seq = 0, kq = 0;
        bool ok = true;
        int32_t id = atomicAdd(p.work, 1);
        publish(0, id);
        while (ok && id < n_ids) {
            volatile QEntry *e = item_q + kq % kItemQ;
            const int32_t l_rel = e->l_rel, g = e->g, n_tiles = e->n_tiles, b = e->b, t0 = e->t0;
            const int32_t tmap = e->tmap, len = e->len, tile0 = e->tile0;
            const uint64_t pol = e->last_read ? pol_stream : pol_keep;
            const int32_t tail_tiles = n_tiles - 1;  // tail items only
            const int32_t id_next = atomicAdd(p.work, 1);
            bool next_published = false;
            const int layer = p.layer0 + l_rel;
            for (int t = 0; t < n_tiles; ++t, ++seq) {
                if (t == n_tiles / 2) {
                    publish(kq + 1, id_next);
                    next_published = true;
                }
                const uint32_t stage = seq % C::NSTAGE, use = seq / C::NSTAGE;
                if (use > 0 && !mbar_wait(empty_u32 + stage * 8, (use - 1) & 1, flags)) {
                    ok = false;
                    break;
                }
                const uint32_t bar = full_u32 + stage * 8, dst = ring_u32 + stage * C::STAGE_BYTES;
                if (b >= 0 && t == tail_tiles) {  // the step's new token, from k_new / v_new [layer][request][head][D]
                    const int32_t z = l_rel * p.B + b;
                    tags[stage] = 1u | kTagNew | (use << 16);
                    mbar_expect_tx(bar, C::STAGE_BYTES);
#pragma unroll
                    for (int bx = 0; bx < C::NBOX; ++bx) {
                        tma_load_3d(dst + bx * C::BOX_BYTES, &kn_map, bx * 64, g, z, bar);
                        tma_load_3d(dst + (C::NBOX + bx) * C::BOX_BYTES, &vn_map, bx * 64, g, z, bar);
                    }
                    continue;
                }
                const CUtensorMap *mk, *mv;
                int32_t yk, yv, rows;
                if (b < 0) {
                    const int r0 = (tile0 + t) * kTile;
                    mk = mv = p.tmaps + tmap;
                    yk = ((layer * 2) * p.Hkv + g) * len + r0;
                    yv = ((layer * 2 + 1) * p.Hkv + g) * len + r0;
                    rows = min(kTile, len - r0);
                } else {
                    const int r0 = t * kTile;
                    mk = p.tmaps + p.n_seg_total;
                    mv = mk + 1;
                    yk = yv = ((b * p.n_layers_total + layer) * p.Hkv + g) * p.max_tail + r0;
                    rows = min(kTile, t0 - r0);
                }
                tags[stage] = (uint32_t)rows | (use << 16);  // published only after the stage's previous fill was released
                mbar_expect_tx(bar, C::STAGE_BYTES);
#pragma unroll
                for (int bx = 0; bx < C::NBOX; ++bx) {
                    tma_load_2d_hint(dst + bx * C::BOX_BYTES, mk, bx * 64, yk, bar, pol);
                    tma_load_2d_hint(dst + (C::NBOX + bx) * C::BOX_BYTES, mv, bx * 64, yv, bar, pol);
                }
            }
            if (!ok && !next_published) publish(kq + 1, n_ids);  // gave up: the consumers must not wait for another item
            ++kq;
            id = id_next;
        }
        if (!ok) {
            // wait (bounded) for the copies in flight so that none lands after the CTA has gone
            atomicCAS(p.status, 0, MATKV_E_TIMEOUT);
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
    const int tq = qr;                         // transposed items: accumulator rows (tokens, then dimensions) tq and tq + 8
    const int mi = lane >> 3, ri = lane & 7;   // ldmatrix addressing

    uint32_t qa[C::KS][4];   // A fragments of Q: rows qr / qr+8, k columns 0-7 / 8-15 of every k-step
    float o[2 * C::KS][4];   // O accumulators: [8-column block of d][row qr: c0, c1; row qr+8: c2, c3]
    float m_run[2], l_run[2];
    float lr[4];             // row sums of the bf16-rounded numerators (an MMA against ones): O is normalised by them

    // thread 0 waits (bounded) for entry k of the queue; flags[1] tells everybody whether it holds an item
    auto await_entry = [&](uint32_t k) {
        volatile QEntry *e = item_q + k % kItemQ;
        bool got = e->seq1 == k + 1;
        if (!got) {
            const long long t0 = clock64();
            while (true) {
                got = e->seq1 == k + 1;
                if (got || flags[0]) break;
                if (clock64() - t0 > kWaitCycles) {
                    flags[0] = 1;
                    break;
                }
            }
        }
        flags[1] = (got && e->id >= 0) ? 0 : 1;
    };
    // the query rows of the requests stacked in an item, as A fragments
    auto load_q = [&](const volatile QEntry *e) {
        const int n_rows = e->n_req * G;
        const int64_t base = (int64_t)e->l_rel * p.q_sl + (int64_t)e->g * G * D;
        if (n_rows <= 8) {
            // transposed item (see the piece loop): Q^T as the B operand, column tq = query row tq
            const bool real = tq < n_rows;
            const __nv_bfloat16 *qrow = p.q + base + (int64_t)(real ? e->req[tq / G] : 0) * p.q_sb + (tq % G) * D;
#pragma unroll
            for (int ks = 0; ks < C::KS; ++ks) {
                qa[ks][0] = real ? *(const uint32_t *)(qrow + ks * 16 + 2 * qc) : 0u;
                qa[ks][1] = real ? *(const uint32_t *)(qrow + ks * 16 + 8 + 2 * qc) : 0u;
            }
            return;
        }
#pragma unroll
        for (int hh = 0; hh < 2; ++hh) {
            const int r = qr + 8 * hh;
            const bool real = r < n_rows;
            const __nv_bfloat16 *qrow = p.q + base + (int64_t)(real ? e->req[r / G] : 0) * p.q_sb + (r % G) * D;
#pragma unroll
            for (int ks = 0; ks < C::KS; ++ks) {
                qa[ks][hh] = real ? *(const uint32_t *)(qrow + ks * 16 + 2 * qc) : 0u;
                qa[ks][2 + hh] = real ? *(const uint32_t *)(qrow + ks * 16 + 8 + 2 * qc) : 0u;
            }
        }
    };
    // Arrival tickets are settled in batches.  A ticket must follow a device-wide fence, and a fence costs
    // microseconds while the SM has a ring full of copies in flight: one per item would stall the consumers
    // as long as a fifth of the item's stream time.  So every (item, stacked request) pair that has left a
    // partial is only noted in shared memory, and once the list is nearly full (and after the last item) all
    // its tickets are drawn behind one fence per thread; the last partial of a (layer, request, KV head) to be
    // ticketed merges that row's partials.
    int n_pend = 0;  // the same in every consumer thread
    auto flush = [&]() {
        consumer_bar();  // the partials of every listed pair have been written
        for (int i = tid; i < n_pend; i += kCW * 32) {
            int last = 0;
            if (pend_np[i] > 1) {
                __threadfence();
                int32_t *cnt = p.counters + pend_idx[i];
                last = atomicAdd(cnt, 1) == pend_np[i] - 1;
                if (last) *cnt = 0;  // ready for the next launch
            }
            pend_last[i] = (uint8_t)last;
        }
        consumer_bar();
        for (int pr = warp; pr < n_pend * G; pr += kCW) {
            const int i = pr / G, h = pr % G;
            if (!pend_last[i]) continue;
            __threadfence();
            const int lg = pend_idx[i] / p.B, b = pend_idx[i] % p.B;
            const int l_rel = lg / p.Hkv, g = lg % p.Hkv;
            const int64_t first = (int64_t)lg * p.parts_total + p.reqs[b].part_base;
            combine_warp(p.part_o + (first * G + h) * D, (int64_t)G * D, p.part_lse + first * G + h, G, pend_np[i], D,
                         p.out + (int64_t)l_rel * p.q_sl + (int64_t)b * p.q_sb + (int64_t)(g * G + h) * D,
                         p.lse_out ? p.lse_out + (int64_t)l_rel * p.lse_sl + (int64_t)b * p.lse_sb + g * G + h : nullptr);
        }
        n_pend = 0;  // the list is rewritten only after the next item's first barrier, which every warp reaches after this
    };

    if (tid == 0) await_entry(0);
    consumer_bar();
    bool have = flags[1] == 0;
    if (have) load_q(item_q);
    int64_t j_base = 0;      // CTA-local index of the item's first tile
    uint32_t k = 0;
    for (; have; ++k) {
        const volatile QEntry *e = item_q + k % kItemQ;
        const int l_rel = e->l_rel, g = e->g, n_tiles = e->n_tiles, n_req = e->n_req, b_tail = e->b, t0 = e->t0;
        const int layer = p.layer0 + l_rel;
        const int lg = l_rel * p.Hkv + g;
        const int n_rows = n_req * G;
        const bool tr = n_rows <= 8;   // the transposed form (see the piece loop)
#pragma unroll
        for (int hh = 0; hh < 2; ++hh) {
            m_run[hh] = -CUDART_INF_F;
            l_run[hh] = 0.f;
        }
        lr[0] = lr[1] = lr[2] = lr[3] = 0.f;
#pragma unroll
        for (int nb = 0; nb < 2 * C::KS; ++nb) o[nb][0] = o[nb][1] = o[nb][2] = o[nb][3] = 0.f;

        // ---- this warp's 16-token pieces of the item ----
        const int64_t hj_begin = j_base * kItems, hj_end = (j_base + n_tiles) * kItems;
        int64_t hj = hj_begin + (int)((warp - hj_begin % kCW + kCW) % kCW);
        for (; hj < hj_end; hj += kCW) {
            const uint32_t j = (uint32_t)(hj / kItems);
            const int r0 = (int)(hj % kItems) * kItemRows;
            const uint32_t stage = j % C::NSTAGE, use = j / C::NSTAGE;
            const uint32_t tag = stage_wait(tags + stage, use, full_u32 + stage * 8, use & 1, flags);
            const uint32_t stage_u32 = ring_u32 + stage * C::STAGE_BYTES;
            const int vis = (int)(tag & 0x7f) - r0;   // valid tokens of this piece (may be <= 0)
            if (vis > 0 && tr) {
                // ---------- an item of at most 8 query rows: the products transposed, S^T = K Q^T and O^T += V^T P^T (tokens,
                // then head dimensions, on the 16-row axis of the MMA, the query rows on its 8-column axis): half the MMAs of
                // the stacked form, whose rows 8..15 would be padding here.  o[0 .. KS-1], m_run, l_run, lr[0 .. 1] hold the state. ----------
                float sa[4] = {0.f, 0.f, 0.f, 0.f}, sb[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
                for (int ks = 0; ks < C::KS; ++ks) {
                    // A = K rows, fragments a0..a3: (tokens 0-7, d-chunk 2ks), (tokens 8-15, 2ks), (tokens 0-7, 2ks+1), (tokens 8-15, 2ks+1)
                    uint32_t ka[4];
                    ldsm_x4(stage_u32 + (ks / 4) * C::BOX_BYTES + swz(r0 + (mi & 1) * 8 + ri, (ks * 2 + (mi >> 1)) & 7), ka);
                    if (ks & 1) mma_bf16(sb, ka[0], ka[1], ka[2], ka[3], qa[ks][0], qa[ks][1]);
                    else mma_bf16(sa, ka[0], ka[1], ka[2], ka[3], qa[ks][0], qa[ks][1]);
                }
                // this thread: tokens tq (x0, x1) and tq + 8 (x2, x3) against query rows 2 qc (x0, x2) and 2 qc + 1 (x1, x3)
                const float x0 = tq < vis ? (sa[0] + sb[0]) * p.scale_log2 : -CUDART_INF_F;
                const float x1 = tq < vis ? (sa[1] + sb[1]) * p.scale_log2 : -CUDART_INF_F;
                const float x2 = tq + 8 < vis ? (sa[2] + sb[2]) * p.scale_log2 : -CUDART_INF_F;
                const float x3 = tq + 8 < vis ? (sa[3] + sb[3]) * p.scale_log2 : -CUDART_INF_F;
                float mx0 = fmaxf(x0, x2), mx1 = fmaxf(x1, x3);
#pragma unroll
                for (int off = 4; off < 32; off <<= 1) {   // over the eight token pairs of the piece (lanes with the same qc)
                    mx0 = fmaxf(mx0, __shfl_xor_sync(0xffffffffu, mx0, off));
                    mx1 = fmaxf(mx1, __shfl_xor_sync(0xffffffffu, mx1, off));
                }
                const float mn0 = fmaxf(m_run[0], mx0), mn1 = fmaxf(m_run[1], mx1);   // finite: token 0 of the piece is valid
                const float al0 = fast_exp2(m_run[0] - mn0), al1 = fast_exp2(m_run[1] - mn1);
                const float p0 = fast_exp2(x0 - mn0), p1 = fast_exp2(x1 - mn1), p2 = fast_exp2(x2 - mn0), p3 = fast_exp2(x3 - mn1);
                const uint32_t w0 = pack_bf16(p0, p1), w1 = pack_bf16(p2, p3);   // (token tq | tq + 8; rows 2 qc, 2 qc + 1)
                l_run[0] = l_run[0] * al0 + (p0 + p2);
                l_run[1] = l_run[1] * al1 + (p1 + p3);
                lr[0] = lr[0] * al0 + (bf_lo(w0) + bf_lo(w1));   // this thread's share of the rounded numerators' sums
                lr[1] = lr[1] * al1 + (bf_hi(w0) + bf_hi(w1));
                m_run[0] = mn0;
                m_run[1] = mn1;
                if (__any_sync(0xffffffffu, al0 != 1.0f || al1 != 1.0f)) {
#pragma unroll
                    for (int mt = 0; mt < C::KS; ++mt) {
                        o[mt][0] *= al0; o[mt][1] *= al1; o[mt][2] *= al0; o[mt][3] *= al1;
                    }
                }
                uint32_t pb0, pb1;   // P^T as the B operand: the 8 x 8 blocks (tokens x rows) transposed across the warp
                asm volatile("movmatrix.sync.aligned.m8n8.trans.b16 %0, %1;" : "=r"(pb0) : "r"(w0));
                asm volatile("movmatrix.sync.aligned.m8n8.trans.b16 %0, %1;" : "=r"(pb1) : "r"(w1));
                const uint32_t v_u32 = stage_u32 + C::NBOX * C::BOX_BYTES;
#pragma unroll
                for (int mt = 0; mt < C::KS; ++mt) {
                    // A = V^T: (d-chunk 2mt, tokens 0-7), (2mt+1, tokens 0-7), (2mt, tokens 8-15), (2mt+1, tokens 8-15), transposed on the way
                    uint32_t va[4];
                    ldsm_x4_trans(v_u32 + (mt / 4) * C::BOX_BYTES + swz(r0 + (mi >> 1) * 8 + ri, (mt * 2 + (mi & 1)) & 7), va);
                    mma_bf16(o[mt], va[0], va[1], va[2], va[3], pb0, pb1);
                }
            } else if (vis > 0) {
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
                    lr[0] *= alpha[0];
                    lr[2] *= alpha[1];
                }
                mma_bf16(lr, pa[0], pa[1], pa[2], pa[3], 0x3f803f80u, 0x3f803f80u);  // P times a column of ones
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
            }
            if (vis > 0) {
                // ---------- the new token goes to the request's tail for later steps ----------
                if ((tag & kTagNew) && r0 == 0 && t0 < p.max_tail) {
                    constexpr int CPR = D / 8;  // 16-byte chunks per row; lanes 0..CPR-1 move K, the next CPR lanes move V
                    const unsigned char *ring_stage = ring + stage * C::STAGE_BYTES;
                    const int64_t off = ((((int64_t)b_tail * p.n_layers_total + layer) * p.Hkv + g) * p.max_tail + t0) * D;
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

        // ---- end of the item ----
        // The global round trips of an item boundary are off the critical path: the next item's description was
        // prepared by the producer, its query rows are fetched while this item's partials are being reduced, and
        // the arrival tickets wait for the next batched flush.
        if (tid == 0) await_entry(k + 1);
        // The seven warps' states are merged through shared memory.  First the running maxima: once every thread
        // knows its rows' overall maximum it scales its own accumulators while it writes them, so that the reduction
        // itself is a plain sum (no exponentials, no per-warp weights).
        // (stacked items: this thread's rows are qr and qr + 8, a row's tokens sit in the four lanes of a quad; transposed
        // items: rows 2 qc and 2 qc + 1, a row's tokens sit in the eight lanes that share qc)
        if (tr ? tq == 0 : qc == 0) {
            merge_m[warp * kShareRows + (tr ? 2 * qc : qr)] = m_run[0];
            merge_m[warp * kShareRows + (tr ? 2 * qc + 1 : qr + 8)] = m_run[1];
        }
        consumer_bar();
        float sw[2];
#pragma unroll
        for (int hh = 0; hh < 2; ++hh) {
            const int r = tr ? 2 * qc + hh : qr + 8 * hh;
            float M = merge_m[r];
#pragma unroll
            for (int w = 1; w < kCW; ++w) M = fmaxf(M, merge_m[w * kShareRows + r]);
            sw[hh] = m_run[hh] == -CUDART_INF_F ? 0.f : fast_exp2(m_run[hh] - M);   // a warp without pieces of this item: weight 0
            float l_tot = l_run[hh], r_tot = tr ? lr[hh] : lr[2 * hh];
            if (tr) {
#pragma unroll
                for (int off = 4; off < 32; off <<= 1) {
                    l_tot += __shfl_xor_sync(0xffffffffu, l_tot, off);
                    r_tot += __shfl_xor_sync(0xffffffffu, r_tot, off);
                }
            } else {
                l_tot += __shfl_xor_sync(0xffffffffu, l_tot, 1);
                l_tot += __shfl_xor_sync(0xffffffffu, l_tot, 2);
            }
            if (tr ? tq == 0 : qc == 0) {
                merge_l[warp * kShareRows + r] = l_tot * sw[hh];
                merge_r[warp * kShareRows + r] = r_tot * sw[hh];
                if (warp == 0) row_max[r] = M;
            }
        }
        bool have_next = false;
#pragma unroll
        for (int half = 0; half < D / 64; ++half) {
            if (half) consumer_bar();  // the previous half has been read
            if (tr) {   // O^T accumulators: [16-dimension block][(d = tq, row 2 qc), (tq, 2 qc + 1), (tq + 8, 2 qc), (tq + 8, 2 qc + 1)]
#pragma unroll
                for (int m4 = 0; m4 < 4; ++m4) {
#pragma unroll
                    for (int hh = 0; hh < 2; ++hh) {
                        float *row = merge_o + (warp * kShareRows + 2 * qc + hh) * 64 + m4 * 16 + tq;
                        row[0] = o[half * 4 + m4][hh] * sw[hh];
                        row[8] = o[half * 4 + m4][2 + hh] * sw[hh];
                    }
                }
            } else {
#pragma unroll
                for (int nb = 0; nb < 8; ++nb) {
                    *(float2 *)(merge_o + (warp * kShareRows + qr) * 64 + nb * 8 + 2 * qc) =
                        make_float2(o[half * 8 + nb][0] * sw[0], o[half * 8 + nb][1] * sw[0]);
                    *(float2 *)(merge_o + (warp * kShareRows + qr + 8) * 64 + nb * 8 + 2 * qc) =
                        make_float2(o[half * 8 + nb][2] * sw[1], o[half * 8 + nb][3] * sw[1]);
                }
            }
            consumer_bar();
            if (half == 0) {
                if (tid < n_req) {  // note the item's (request, KV head, layer) rows for the next ticket flush
                    pend_idx[n_pend + tid] = lg * p.B + e->req[tid];
                    pend_np[n_pend + tid] = e->np[tid];
                }
                have_next = flags[1] == 0;
                if (have_next) load_q(item_q + (k + 1) % kItemQ);
            }
            // one (row, four columns) unit per thread and pass: plain sums over the warps
            for (int idx = tid; idx < n_rows * 16; idx += kCW * 32) {
                const int r = idx >> 4, c4 = idx & 15;
                float4 acc = *(const float4 *)(merge_o + r * 64 + 4 * c4);
                float Lr = merge_r[r];
#pragma unroll
                for (int w = 1; w < kCW; ++w) {
                    const float4 v = *(const float4 *)(merge_o + (w * kShareRows + r) * 64 + 4 * c4);
                    acc.x += v.x; acc.y += v.y; acc.z += v.z; acc.w += v.w;
                    Lr += merge_r[w * kShareRows + r];
                }
                const float inv = 1.f / Lr;
                acc.x *= inv; acc.y *= inv; acc.z *= inv; acc.w *= inv;
                const int j = r / G, h = r % G, d = half * 64 + 4 * c4;
                const int b = e->req[j];
                float lse = 0.f;
                if (d == 0) {
                    float L = merge_l[r];
#pragma unroll
                    for (int w = 1; w < kCW; ++w) L += merge_l[w * kShareRows + r];
                    lse = (row_max[r] + log2f(L)) * kLn2;
                }
                if (e->np[j] == 1) {  // a request without chunks: its tail item is the whole answer
                    *(uint2 *)(p.out + (int64_t)l_rel * p.q_sl + (int64_t)b * p.q_sb + (int64_t)(g * G + h) * D + d) =
                        make_uint2(pack_bf16(acc.x, acc.y), pack_bf16(acc.z, acc.w));
                    if (p.lse_out && d == 0) p.lse_out[(int64_t)l_rel * p.lse_sl + (int64_t)b * p.lse_sb + g * G + h] = lse;
                } else {
                    const int64_t row = ((int64_t)lg * p.parts_total + e->part[j]) * G + h;
                    *(float4 *)(p.part_o + row * D + d) = acc;
                    if (d == 0) p.part_lse[row] = lse;
                }
            }
        }
        n_pend += n_req;
        j_base += n_tiles;
        have = have_next;
        if (n_pend + kShareRows > kPend || !have) flush();
        else consumer_bar();  // the merge area is free again
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
    static PerDeviceOnce configured;
    int once_dev;
    if (configured.need(&once_dev)) {
        MATKV_CUDA(cudaFuncSetAttribute(k_attend_shared<D, G>, cudaFuncAttributeMaxDynamicSharedMemorySize, C::SMEM_BYTES));
        configured.mark(once_dev);
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
    // by default one CTA per SM, less the SMs left to the staging copy kernel when that is in use (the launch is
    // bound by HBM with ~130 CTAs already; a copy CTA sharing an SM with a decode CTA makes that SM the straggler)
    int64_t grid = ctx->opt_decode_ctas > 0 ? ctx->opt_decode_ctas : std::max<int64_t>(ctx->n_sm - ctx->opt_stage_ctas, ctx->n_sm / 2);
    grid = std::max<int64_t>(1, std::min<int64_t>(grid, n_ids));
#define MATKV_CASE(DD, GG) \
    if (c.head_dim == DD && G == GG) return launch_shared_t<DD, GG>(p, kn_map, vn_map, (int)grid, stream);
    MATKV_CASE(128, 1) MATKV_CASE(128, 2) MATKV_CASE(128, 4) MATKV_CASE(128, 8)
    MATKV_CASE(64, 1) MATKV_CASE(64, 2) MATKV_CASE(64, 4) MATKV_CASE(64, 8)
#undef MATKV_CASE
    return fail(MATKV_E_INVALID_ARG, "unsupported head_dim %d / group %d", c.head_dim, G);
}

}  // namespace matkv
