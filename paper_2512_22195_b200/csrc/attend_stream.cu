// K1: chunk-table streaming attention (decode, and small query suffixes) + K2: log-sum-exp combine.
//
// One persistent CTA per SM.  The work of a launch is the flat list of KV tiles (kTile tokens of one
// "unit" = (layer, request, block of suffix tokens, KV head)); CTA c owns the contiguous range
// [c*W/n, (c+1)*W/n) of that list, so every SM streams the same number of bytes whatever the shape.
// Inside a CTA one producer thread walks its range and moves each tile's K rows and V rows from the
// scattered chunk blobs (or the tail) into a shared-memory ring with TMA tensor copies (128-byte
// swizzle, mbarrier complete_tx).  Seven consumer warps take 16-token pieces of the tiles round-robin;
// each keeps the unit's query rows (up to 8: the G heads of the KV group for up to 8/G suffix tokens)
// as mma A fragments and runs an independent online softmax: S = Q K^T and O += P V are warp-level
// m16n8k16 bf16 MMAs fed by ldmatrix from the swizzled tiles, so the instruction stream per KV byte is
// short enough for the kernel to stay HBM-bound at any G (a plain-FMA inner product measured
// issue-bound: 42% issue utilisation with 8 resident warps and 48% of DRAM peak).  fp32 scores,
// exp2-based softmax, fp32 accumulators; P is rounded to bf16 for the second MMA.
// The new tokens of the call (not yet in the tail) come through the same ring from k_new / v_new (a
// per-call TMA descriptor) with a causal mask, and the warp that handles them appends them to the tail.  At the end of a unit the warps' states are merged through shared memory;
// a unit that spans several CTAs leaves one partial (normalised o, lse) per CTA in the workspace and
// the last CTA to arrive (atomic ticket, no waiting) merges them by log-sum-exp.
#include <algorithm>

#include "stream_common.cuh"

namespace matkv {

struct StreamParams {
    const DevReq *reqs;
    const CUtensorMap *tmaps;   // [n_seg_total] chunk maps, then tail K, tail V
    const CUtensorMap *tmaps8;  // [n_seg_total][2] maps of compressed-resident chunks (K codes, transposed V codes), or null
    const DevSeg *segs;         // [n_seg_total]
    int32_t n_seg_total;
    const int32_t *tail_len;
    __nv_bfloat16 *tail_k, *tail_v;
    const __nv_bfloat16 *q, *k_new, *v_new;
    __nv_bfloat16 *out;
    float *lse_out;
    int64_t q_sl, q_sb, q_ss, kn_sl, kn_sb, kn_ss, lse_sl, lse_sb, lse_ss;
    int32_t layer0, n_layers_launch, n_layers_total, B, S, Hkv, max_tail;
    float scale_log2;
    int32_t *counters;
    float *part_lse, *part_o;
    int64_t n_part_slots, n_counter_slots;
    int32_t *status;
    int32_t advance;      // > 0: the last CTA to finish adds this to every request's tail length
    int32_t *done_count;  // CTAs of the launch that have finished (reset by the last one)
    int32_t stream_hint;  // 1: no chunk of the table is listed twice, load chunk tiles with the evict-first L2 policy
    // >= 0: every request's tail length as the host knows it.  The work split is then computed from it, BEFORE the
    // kernel waits for its predecessor on the stream, and the producer pulls its first chunk tiles (immutable data)
    // into the ring under the predecessor's tail; the device counter is compared with it after the wait
    // (MATKV_E_BOUNDS in the status word if they differ).  -1: read the device counter (after the wait).
    int32_t tail_hint;
};

// ---- the flat work list ----------------------------------------------------------------------------

struct UnitPos {
    int32_t l_rel, b, blk, g;  // layer (relative to layer0), request, block of suffix tokens, KV head
    int32_t tile;              // first tile of this CTA's share inside the unit
    int32_t rt;                // tiles in the unit: chunk tiles, tail tiles, ceil(S / kTile) tiles of new tokens
    int32_t chunk_tiles, tail_tiles, t0, seg_begin;
    int64_t flat_begin;        // flat index of the unit's first tile
};

struct CtaRange {
    int64_t begin, end, W;
    UnitPos first;
};

__device__ __forceinline__ int32_t clamp_t0(const StreamParams &p, int b) {
    int32_t t0 = p.tail_hint >= 0 ? p.tail_hint : p.tail_len[b];
    if (t0 < 0 || t0 + p.S > p.max_tail) {
        atomicCAS(p.status, 0, MATKV_E_CAPACITY);
        t0 = max(0, min(t0, p.max_tail - p.S));
    }
    return t0;
}

__device__ __forceinline__ void load_req(const StreamParams &p, UnitPos &u) {
    const DevReq rq = p.reqs[u.b];
    u.t0 = clamp_t0(p, u.b);
    u.chunk_tiles = rq.chunk_tiles;
    u.seg_begin = rq.seg_begin;
    u.tail_tiles = ceil_div(u.t0, kTile);
    u.rt = u.chunk_tiles + u.tail_tiles + ceil_div(p.S, kTile);
}

// advance to the next unit in (layer, request, token block, head) order
__device__ __forceinline__ void next_unit(const StreamParams &p, UnitPos &u, int n_blk) {
    u.flat_begin += u.rt;
    u.tile = 0;
    if (++u.g < p.Hkv) return;
    u.g = 0;
    if (++u.blk < n_blk) return;
    u.blk = 0;
    if (++u.b >= p.B) {
        u.b = 0;
        ++u.l_rel;
    }
    if (u.l_rel < p.n_layers_launch) load_req(p, u);
}

__device__ void locate_range(const StreamParams &p, CtaRange &r, int n_blk) {
    int64_t w_layer = 0;
    for (int b = 0; b < p.B; ++b) {
        const int rt = p.reqs[b].chunk_tiles + ceil_div(clamp_t0(p, b), kTile) + ceil_div(p.S, kTile);
        w_layer += (int64_t)p.Hkv * n_blk * rt;
    }
    r.W = w_layer * p.n_layers_launch;
    const int64_t n = gridDim.x, c = blockIdx.x;
    r.begin = c * r.W / n;
    r.end = (c + 1) * r.W / n;
    UnitPos &u = r.first;
    u = UnitPos{};
    if (r.begin >= r.end) return;
    const int64_t f = r.begin;
    u.l_rel = (int32_t)(f / w_layer);
    int64_t rem = f % w_layer;
    int b = 0;
    for (; b < p.B; ++b) {
        const int rt = p.reqs[b].chunk_tiles + ceil_div(clamp_t0(p, b), kTile) + ceil_div(p.S, kTile);
        const int64_t blk = (int64_t)p.Hkv * n_blk * rt;
        if (rem < blk) break;
        rem -= blk;
    }
    u.b = b;
    load_req(p, u);
    u.blk = (int32_t)(rem / ((int64_t)p.Hkv * u.rt));
    rem -= (int64_t)u.blk * p.Hkv * u.rt;
    u.g = (int32_t)(rem / u.rt);
    u.tile = (int32_t)(rem % u.rt);
    u.flat_begin = f - u.tile;
}

// CTA that owns flat tile f when W tiles are split over n CTAs as [c*W/n, (c+1)*W/n)
__device__ __forceinline__ int cta_of(int64_t f, int64_t W, int64_t n) { return (int)(((f + 1) * n - 1) / W); }

__global__ void k_lse_combine(int n_rows, int P, int D, const float *__restrict__ o_parts,
                              const float *__restrict__ lse_parts, __nv_bfloat16 *__restrict__ out, float *lse_out) {
    const int row = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
    if (row >= n_rows) return;
    combine_warp(o_parts + (int64_t)row * P * D, D, lse_parts + (int64_t)row * P, 1, P, D, out + (int64_t)row * D,
                 lse_out ? lse_out + row : nullptr);
}

// ---- K1 -------------------------------------------------------------------------------------------
template <int D, int G, bool F8 = false>
struct StreamCfg {
    static constexpr int TPU = kUnitRows / G;              // suffix tokens per unit
    static constexpr int NBOX = D / 64;                    // 64-column TMA boxes per row
    static constexpr int BOX_BYTES = kTile * 128;          // one box: kTile rows x 128 bytes (swizzled)
    static constexpr int STAGE_BYTES = 2 * NBOX * BOX_BYTES;  // K boxes then V boxes
    static constexpr int KS = D / 16;                      // k-steps of S = Q K^T; also n-block pairs of O += P V
    static constexpr int MERGE_BYTES = (kCW * kUnitRows * (D + 3) * 4 + 15) / 16 * 16;
    static constexpr int FIXED_BYTES = MERGE_BYTES + 1024 + 1024;  // + misc + slack for 1024-byte alignment of the ring
    static constexpr int NSTAGE_MAX = (kMaxDynSmem - FIXED_BYTES) / STAGE_BYTES;
    // Measured on B200 (chunk tiles loaded with the evict-first L2 policy): a ring of 128 KB is faster than one
    // that fills shared memory.  Config 2, all-layers launch: 107.7 us with 4 stages of 32 KB, 107.9 with 5,
    // 111.1 with 6; config 4: 11.63 / 11.84 / 12.50 ms.  More copies in flight than the memory latency needs
    // only lengthen the queues in front of DRAM.
    // (a tile of codes fills only half of its 32 KB stage: the compressed variant keeps six stages in flight)
    static constexpr int NSTAGE_CAP = (F8 ? 192 : 128) * 1024 / STAGE_BYTES;
    static constexpr int NSTAGE = NSTAGE_MAX > NSTAGE_CAP ? NSTAGE_CAP : NSTAGE_MAX;
    static constexpr int SMEM_BYTES = NSTAGE * STAGE_BYTES + FIXED_BYTES;
    static_assert(G >= 1 && G <= kUnitRows && kUnitRows % G == 0, "unsupported group size");
    static_assert(D % 64 == 0 && NSTAGE >= 3, "unsupported head_dim");
};


template <int D, int G, bool F8>
__global__ void __launch_bounds__(kThreads, 1)
k_attend_stream(const __grid_constant__ StreamParams p, const __grid_constant__ CUtensorMap kn_map, const __grid_constant__ CUtensorMap vn_map) {
    using C = StreamCfg<D, G, F8>;
    static_assert(!F8 || D == 128, "compressed-resident chunks: head_dim 128 only");
    extern __shared__ unsigned char smem_raw[];
    // the swizzle pattern repeats every 1024 bytes: align the ring to it
    unsigned char *smem = (unsigned char *)(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
    unsigned char *ring = smem;
    float *merge_o = (float *)(smem + C::NSTAGE * C::STAGE_BYTES);  // [warp][row][D]
    float *merge_m = merge_o + kCW * kUnitRows * D;                 // [warp][row]  (log2 units, scaled)
    float *merge_l = merge_m + kCW * kUnitRows;                     // [warp][row]
    float *merge_r = merge_l + kCW * kUnitRows;                     // [warp][row]  sum of the rounded numerators
    unsigned char *misc = smem + C::NSTAGE * C::STAGE_BYTES + C::MERGE_BYTES;
    uint64_t *bars = (uint64_t *)misc;                              // full[NSTAGE], empty[NSTAGE]
    // per stage tag: valid rows | kTagNew | (number of the stage's current fill) << 16
    volatile uint32_t *tags = (volatile uint32_t *)(misc + 2 * 12 * 8);
    CtaRange *range = (CtaRange *)(misc + 2 * 12 * 8 + 12 * 4 + 8);
    volatile int *flags = (volatile int *)(misc + 2 * 12 * 8 + 12 * 4 + 8 + sizeof(CtaRange) + 8);  // [0] abort, [1] last arriver

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int n_blk = ceil_div(p.S, C::TPU);
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");   // the next launch may be set up under this one
    if (tid == 0) {
        for (int s = 0; s < C::NSTAGE; ++s) {
            mbar_init(smem_u32(bars + s), 1);
            mbar_init(smem_u32(bars + C::NSTAGE + s), kItems);
            tags[s] = 0xffff0000u;
        }
        flags[0] = 0;
        flags[1] = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    // short launches are chains of latencies: the range lookup (dependent loads of the table) runs in another warp beside
    // the barrier set-up.  Everything from here on may read what the previous kernel on the stream wrote (tail lengths,
    // tail rows, the call's q / k / v, the workspace): wait for it to have completed.
    // With the host's tail length at hand the split is located first and only the threads that touch such data wait
    // (the producer thread goes ahead with chunk tiles, see there).
    const bool early = p.tail_hint >= 0;
    if (!early && tid != 0) asm volatile("griddepcontrol.wait;" ::: "memory");
    if (tid == 32) locate_range(p, *range, n_blk);
    if (!early && tid == 0) asm volatile("griddepcontrol.wait;" ::: "memory");
    __syncthreads();
    if (early && !(warp == kCW && lane == 0)) {
        asm volatile("griddepcontrol.wait;" ::: "memory");
        if (blockIdx.x == 0)   // the host's tail length must be the device's: a launch split by a stale value is void
            for (int b = tid; b < p.B; b += kThreads)
                if (p.tail_len[b] != p.tail_hint) atomicCAS(p.status, 0, MATKV_E_BOUNDS);
    }
    const int64_t f_begin = range->begin, f_end = range->end, W = range->W;
    // the fused tail advance: the last CTA of the launch to get here moves every request's tail length
    auto finish_cta = [&]() {
        if (p.advance <= 0) return;
        __threadfence();
        if (atomicAdd(p.done_count, 1) == (int)gridDim.x - 1) {
            for (int b = 0; b < p.B; ++b) {
                int32_t v = p.tail_len[b] + p.advance;
                if (v > p.max_tail) {
                    v = p.max_tail;
                    atomicCAS(p.status, 0, MATKV_E_CAPACITY);
                }
                const_cast<int32_t *>(p.tail_len)[b] = v;
            }
            *p.done_count = 0;
        }
    };
    if (f_begin >= f_end) {
        if (tid == 0) finish_cta();
        return;
    }
    const uint32_t ring_u32 = smem_u32(ring), full_u32 = smem_u32(bars), empty_u32 = smem_u32(bars + C::NSTAGE);

    if (warp == kCW) {
        // ================= producer: one thread walks the table and feeds the ring =================
        if (lane != 0) return;
        // chunk rows are read once per launch unless requests share chunks: keep them out of L2's way then
        const uint64_t pol = p.stream_hint ? l2_policy_evict_first() : l2_policy_evict_normal();
        UnitPos u = range->first;
        int seg = -1, tiles_before = 0, seg_tiles = 0, seg_len = 0, seg_fmt = 0;  // cursor over the request's segments
        const unsigned char *seg_base = nullptr;
        int64_t f = f_begin;
        uint32_t seq = 0;
        bool ok = true;
        bool waited = !early;   // chunk tiles are immutable: they may be fetched before the predecessor kernel is done
        while (f < f_end && ok) {
            const int t_end = (int)min((int64_t)u.rt, f_end - u.flat_begin);
            const int layer = p.layer0 + u.l_rel;
            for (int t = u.tile; t < t_end; ++t, ++f, ++seq) {
                if (!waited && t >= u.chunk_tiles) {   // tail rows and the call's new tokens: written by earlier kernels
                    asm volatile("griddepcontrol.wait;" ::: "memory");
                    waited = true;
                }
                const uint32_t stage = seq % C::NSTAGE, use = seq / C::NSTAGE;
                if (use > 0 && !mbar_wait(empty_u32 + stage * 8, (use - 1) & 1, flags)) {
                    ok = false;
                    break;
                }
                const uint32_t bar = full_u32 + stage * 8, dst = ring_u32 + stage * C::STAGE_BYTES;
                if (t >= u.chunk_tiles + u.tail_tiles) {  // the call's new tokens, from k_new / v_new [layer][request][token][head][D]
                    const int nt = t - u.chunk_tiles - u.tail_tiles;
                    const int32_t z = (u.l_rel * p.B + u.b) * p.S + nt * kTile;
                    tags[stage] = (uint32_t)min(kTile, p.S - nt * kTile) | ((uint32_t)nt << 8) | kTagNew | (use << 16);
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
                if (t < u.chunk_tiles) {
                    while (seg < 0 || t >= tiles_before + seg_tiles) {
                        tiles_before += seg_tiles;
                        ++seg;
                        const DevSeg sg = p.segs[u.seg_begin + seg];
                        seg_len = sg.len;
                        seg_fmt = sg.fmt;
                        seg_base = (const unsigned char *)sg.base;
                        seg_tiles = ceil_div(seg_len, kTile);
                    }
                    const int r0 = (t - tiles_before) * kTile;
                    if constexpr (F8) {
                        if (seg_fmt == 1) {
                            // codes of one 64-token block: K rows (8 KB), V transposed (8 KB), the block's exponent record (16 bytes)
                            const int64_t blk = ((int64_t)layer * p.Hkv + u.g) * seg_tiles + (t - tiles_before);
                            const int64_t region = ((int64_t)p.n_layers_total * p.Hkv * seg_tiles * kTile * D + 255) / 256 * 256;
                            const CUtensorMap *m8 = p.tmaps8 + 2 * (u.seg_begin + seg);
                            tags[stage] = (uint32_t)min(kTile, seg_len - r0) | kTagF8 | (use << 16);
                            mbar_expect_tx(bar, 2 * kTile * D + 16);
                            tma_load_2d_hint(dst, m8, 0, (int32_t)(blk * kTile), bar, pol);
                            tma_load_2d_hint(dst + kTile * D, m8 + 1, 0, (int32_t)(blk * D), bar, pol);
                            bulk_load(dst + 2 * kTile * D, seg_base + 2 * region + blk * 16, 16, bar);
                            continue;
                        }
                    }
                    mk = mv = p.tmaps + u.seg_begin + seg;
                    yk = ((layer * 2) * p.Hkv + u.g) * seg_len + r0;
                    yv = ((layer * 2 + 1) * p.Hkv + u.g) * seg_len + r0;
                    rows = min(kTile, seg_len - r0);
                } else {
                    const int r0 = (t - u.chunk_tiles) * kTile;
                    mk = p.tmaps + p.n_seg_total;
                    mv = mk + 1;
                    yk = yv = ((u.b * p.n_layers_total + layer) * p.Hkv + u.g) * p.max_tail + r0;
                    rows = min(kTile, u.t0 - r0);
                }
                tags[stage] = (uint32_t)rows | (use << 16);  // published only after the stage's previous fill was released
                mbar_expect_tx(bar, C::STAGE_BYTES);
#pragma unroll
                for (int bx = 0; bx < C::NBOX; ++bx) {
                    tma_load_2d_hint(dst + bx * C::BOX_BYTES, mk, bx * 64, yk, bar, pol);
                    tma_load_2d_hint(dst + (C::NBOX + bx) * C::BOX_BYTES, mv, bx * 64, yv, bar, pol);
                }
            }
            if (f < f_end && ok) {
                next_unit(p, u, n_blk);
                seg = -1; tiles_before = 0; seg_tiles = 0;
            }
        }
        if (!ok) {
            // gave up: wait (bounded) for the copies already issued so none lands after the CTA has gone
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
    // mma fragment coordinates of this thread: query row `qr` (rows 8..15 of the 16-row tile are padding),
    // column pair `qc` (two adjacent columns 2*qc, 2*qc+1 of every 8-column block)
    const int qr = lane >> 2, qc = lane & 3;
    // ldmatrix row addressing: matrix mi = lane / 8 of the x4 group, row ri = lane % 8 inside it
    const int mi = lane >> 3, ri = lane & 7;

    uint32_t qa[C::KS][2];   // A fragments of Q for the real rows: [k-step][cols 0-7 | cols 8-15]
    // compressed tiles: the same rows as fp16 (scaled by 2^-eq so that any bf16 row fits), with the 16 dimensions of a
    // k-step assigned to the fragment's k slots the way four consecutive codes fall out of ldmatrix (slots 2qc, 2qc+1
    // <- dimensions 4qc, 4qc+1; slots 2qc+8, 2qc+9 <- 4qc+2, 4qc+3); q_scale = softmax scale * 2^eq undoes the scaling
    uint32_t qh[F8 ? C::KS : 1][2];
    float q_scale = 0.f;
    int ev_cur = 0;          // compressed V: exponent the O accumulators are currently expressed in
    bool ev_set = false;
    float o[2 * C::KS][4];   // O accumulators: [8-column block of d][c0, c1 real row; c2, c3 padding rows]
    // running max (scaled, log2 units), this thread's share of the sum of the numerators (for the log-sum-exp)
    // and of the sum of their bf16 roundings (what the tensor core multiplies with V: O is normalised by it,
    // so that a dominant token's rounding error cancels)
    float m_run = -CUDART_INF_F, l_run = 0.f, l_rnd = 0.f;

    UnitPos u = range->first;
    int64_t f_unit = f_begin;   // flat index of this CTA's first tile inside the current unit
    int64_t j_base = 0;         // CTA-local index of that tile
    while (f_unit < f_end) {
        const int t_begin = u.tile;
        const int t_end = (int)min((int64_t)u.rt, f_end - u.flat_begin);
        const int layer = p.layer0 + u.l_rel;
        const int tok0 = u.blk * C::TPU;                    // first suffix token of the unit
        const int n_tok = min(C::TPU, p.S - tok0);
        const int n_rows = n_tok * G;                       // real query rows: row = token * G + head
        const int64_t q_base = (int64_t)u.l_rel * p.q_sl + (int64_t)u.b * p.q_sb + (int64_t)tok0 * p.q_ss + (int64_t)u.g * G * D;
        // ---- per-unit setup ----
        {
            const bool real = qr < n_rows;
            const __nv_bfloat16 *qrow = p.q + q_base + (int64_t)(qr / G) * p.q_ss + (qr % G) * D;
#pragma unroll
            for (int ks = 0; ks < C::KS; ++ks) {
                qa[ks][0] = real ? *(const uint32_t *)(qrow + ks * 16 + 2 * qc) : 0u;
                qa[ks][1] = real ? *(const uint32_t *)(qrow + ks * 16 + 8 + 2 * qc) : 0u;
            }
            if constexpr (F8) {
                uint2 raw[C::KS];
                uint32_t amax = 0;   // largest |q| of the row, as bf16 bits (they order like the values)
#pragma unroll
                for (int ks = 0; ks < C::KS; ++ks) {
                    raw[ks] = real ? *(const uint2 *)(qrow + ks * 16 + 4 * qc) : make_uint2(0u, 0u);
                    amax = max(amax, max(max(raw[ks].x & 0x7fffu, (raw[ks].x >> 16) & 0x7fffu), max(raw[ks].y & 0x7fffu, (raw[ks].y >> 16) & 0x7fffu)));
                }
                amax = max(amax, __shfl_xor_sync(0xffffffffu, amax, 1));
                amax = max(amax, __shfl_xor_sync(0xffffffffu, amax, 2));
                const int eq = amax >= 0x80u ? min((int)(amax >> 7) - 127, 126) : -126;  // |q| * 2^-eq < 2 (< 4 for the largest binade)
                const float down = __uint_as_float((uint32_t)(127 - eq) << 23);        // 2^-eq (eq in [-126, 127])
                q_scale = p.scale_log2 * __uint_as_float((uint32_t)(127 + max(eq, -126)) << 23);
#pragma unroll
                for (int ks = 0; ks < C::KS; ++ks) {
                    qh[ks][0] = pack_f16(bf_lo(raw[ks].x) * down, bf_hi(raw[ks].x) * down);
                    qh[ks][1] = pack_f16(bf_lo(raw[ks].y) * down, bf_hi(raw[ks].y) * down);
                }
                ev_set = false;
            }
#pragma unroll
            for (int nb = 0; nb < 2 * C::KS; ++nb) o[nb][0] = o[nb][1] = o[nb][2] = o[nb][3] = 0.f;
            m_run = -CUDART_INF_F;
            l_run = 0.f;
            l_rnd = 0.f;
        }
        // ---- this warp's work items of the unit ----
        // CTA-local tile j = j_base + (t - t_begin) splits into kItems work items hj = j*kItems + piece;
        // warp w takes hj == w (mod kCW)
        const int64_t hj_begin = j_base * kItems, hj_end = (j_base + (t_end - t_begin)) * kItems;
        int64_t hj = hj_begin + (int)((warp - hj_begin % kCW + kCW) % kCW);
        for (; hj < hj_end; hj += kCW) {
            const uint32_t j = (uint32_t)(hj / kItems);
            const int piece = (int)(hj % kItems);
            const int r0 = piece * kItemRows;
            const uint32_t stage = j % C::NSTAGE, use = j / C::NSTAGE;
            const uint32_t tag = stage_wait(tags + stage, use, full_u32 + stage * 8, use & 1, flags);
            const uint32_t stage_u32 = ring_u32 + stage * C::STAGE_BYTES;

            int rows = (int)(tag & 0x7f) - r0;        // valid rows of this work item (may be <= 0)
            // new tokens: column c of the item is token new0 + c of the call; this thread's query row
            // (suffix token tok0 + qr / G) sees the tokens up to and including itself
            const bool is_new = (tag & kTagNew) != 0;
            const int new0 = (int)((tag >> 8) & 0x7f) * kTile + r0;
            int vis = rows;                           // columns this thread's row may see
            if (is_new) {
                vis = min(rows, tok0 + qr / G - new0 + 1);
                rows = min(rows, tok0 + n_tok - new0);  // nothing past the unit's last token is visible to any row
            }
            if (rows > 0) {
                // ---------- S = Q K^T for 16 tokens (two 8-token blocks) ----------
                float s0[4] = {0.f, 0.f, 0.f, 0.f}, s1[4] = {0.f, 0.f, 0.f, 0.f};
                const bool is_f8 = F8 && (tag & kTagF8) != 0;
                // token of the piece behind each of this thread's four score columns (s0[0], s0[1], s1[0], s1[1])
                int c0 = 2 * qc, c1 = 2 * qc + 1, c2 = 8 + 2 * qc, c3 = 9 + 2 * qc;
                float xs = p.scale_log2;
                if (is_f8) {
                    if constexpr (F8) {
                        // A K row is 128 codes: one 16-byte chunk per k-step.  The two 8-token MMA blocks take tokens
                        // {0,1,4,5,8,9,12,13} and {2,3,6,7,10,11,14,15} of the piece, so that a thread's score columns are
                        // tokens 4qc .. 4qc+3: the four consecutive codes it later gets from a row of transposed V.
                        const int set = mi >> 1, tr = r0 + (ri >> 1) * 4 + (ri & 1) + 2 * set;
#pragma unroll
                        for (int kp = 0; kp < C::KS / 2; ++kp) {
                            uint32_t kb[4], b0, b1;
                            ldsm_x4(stage_u32 + tr * 128 + (((2 * kp + (mi & 1)) ^ (tr & 7)) << 4), kb);
                            cvt_e4m3x4_f16(kb[0], b0, b1);
                            mma_f16(s0, qh[2 * kp][0], 0u, qh[2 * kp][1], 0u, b0, b1);
                            cvt_e4m3x4_f16(kb[1], b0, b1);
                            mma_f16(s0, qh[2 * kp + 1][0], 0u, qh[2 * kp + 1][1], 0u, b0, b1);
                            cvt_e4m3x4_f16(kb[2], b0, b1);
                            mma_f16(s1, qh[2 * kp][0], 0u, qh[2 * kp][1], 0u, b0, b1);
                            cvt_e4m3x4_f16(kb[3], b0, b1);
                            mma_f16(s1, qh[2 * kp + 1][0], 0u, qh[2 * kp + 1][1], 0u, b0, b1);
                        }
                        c0 = 4 * qc; c1 = 4 * qc + 1; c2 = 4 * qc + 2; c3 = 4 * qc + 3;
                        const int ek = (int)*(const signed char *)(ring + stage * C::STAGE_BYTES + 2 * kTile * D);
                        xs = q_scale * __uint_as_float((uint32_t)(127 + max(ek, -126)) << 23);
                    }
                } else {
#pragma unroll
                    for (int ks = 0; ks < C::KS; ++ks) {
                        // matrices: (tokens 0-7, d-chunk 2ks), (tokens 0-7, 2ks+1), (tokens 8-15, 2ks), (tokens 8-15, 2ks+1)
                        const int c = (ks * 2 + (mi & 1)) & 7;
                        uint32_t kb[4];
                        ldsm_x4(stage_u32 + (ks / 4) * C::BOX_BYTES + swz(r0 + (mi >> 1) * 8 + ri, c), kb);
                        mma_bf16(s0, qa[ks][0], 0u, qa[ks][1], 0u, kb[0], kb[1]);
                        mma_bf16(s1, qa[ks][0], 0u, qa[ks][1], 0u, kb[2], kb[3]);
                    }
                }
                // ---------- online softmax (this thread: row qr, tokens 2qc, 2qc+1, 8+2qc, 9+2qc) ----------
                const float x0 = c0 < vis ? s0[0] * xs : -CUDART_INF_F;
                const float x1 = c1 < vis ? s0[1] * xs : -CUDART_INF_F;
                const float x2 = c2 < vis ? s1[0] * xs : -CUDART_INF_F;
                const float x3 = c3 < vis ? s1[1] * xs : -CUDART_INF_F;
                float tmax = fmaxf(fmaxf(x0, x1), fmaxf(x2, x3));
                tmax = fmaxf(tmax, __shfl_xor_sync(0xffffffffu, tmax, 1));
                tmax = fmaxf(tmax, __shfl_xor_sync(0xffffffffu, tmax, 2));
                const float m_new = fmaxf(m_run, tmax);
                // a row that has seen nothing yet (causal edge of the new tokens) keeps an empty state
                const float m_use = m_new == -CUDART_INF_F ? 0.f : m_new;
                const float alpha = m_new == -CUDART_INF_F ? 1.f : fast_exp2(m_run - m_new);
                const float p0 = fast_exp2(x0 - m_use), p1 = fast_exp2(x1 - m_use);
                const float p2 = fast_exp2(x2 - m_use), p3 = fast_exp2(x3 - m_use);
                // P as the second MMA's operand: bf16, or fp16 against a tile of codes
                const uint32_t pa0 = is_f8 ? pack_f16(p0, p1) : pack_bf16(p0, p1), pa2 = is_f8 ? pack_f16(p2, p3) : pack_bf16(p2, p3);
                l_run = l_run * alpha + ((p0 + p1) + (p2 + p3));
                l_rnd = l_rnd * alpha + (is_f8 ? ((f16_lo(pa0) + f16_hi(pa0)) + (f16_lo(pa2) + f16_hi(pa2)))
                                               : ((bf_lo(pa0) + bf_hi(pa0)) + (bf_lo(pa2) + bf_hi(pa2))));
                m_run = m_new;
                if (__any_sync(0xffffffffu, alpha != 1.0f)) {
#pragma unroll
                    for (int nb = 0; nb < 2 * C::KS; ++nb) {
                        o[nb][0] *= alpha;
                        o[nb][1] *= alpha;
                    }
                }
                // ---------- O += P V ----------
                if constexpr (F8) {
                    // the accumulators are kept in units of 2^ev of the V block last seen (0 for bf16 tiles); a change of
                    // exponent rescales them (a power of two: exact), like a change of the running maximum does
                    const int ev = is_f8 ? (int)*(const signed char *)(ring + stage * C::STAGE_BYTES + 2 * kTile * D + 1) : 0;
                    if (!ev_set) {
                        ev_cur = ev;
                        ev_set = true;
                    } else if (ev != ev_cur) {
                        const float f = exp2f((float)max(-126, min(126, ev_cur - ev)));
#pragma unroll
                        for (int nb = 0; nb < 2 * C::KS; ++nb) {
                            o[nb][0] *= f;
                            o[nb][1] *= f;
                        }
                        ev_cur = ev;
                    }
                }
                if (is_f8) {
                    if constexpr (F8) {
                        // V codes of the block, transposed: row d holds its 64 tokens; this piece is 16-byte chunk r0 / 16 of it
                        const uint32_t v8 = stage_u32 + kTile * D;
#pragma unroll
                        for (int q4 = 0; q4 < D / 32; ++q4) {
                            const int d = 32 * q4 + 8 * mi + ri;
                            uint32_t vb[4], b0, b1;
                            ldsm_x4(v8 + d * 64 + (((r0 >> 4) ^ ((d >> 1) & 3)) << 4), vb);
#pragma unroll
                            for (int m2 = 0; m2 < 4; ++m2) {
                                cvt_e4m3x4_f16(vb[m2], b0, b1);
                                mma_f16(o[4 * q4 + m2], pa0, 0u, pa2, 0u, b0, b1);
                            }
                        }
                    }
                } else {
                const uint32_t v_u32 = stage_u32 + C::NBOX * C::BOX_BYTES;
#pragma unroll
                for (int dp = 0; dp < C::KS; ++dp) {
                    // matrices: (tokens 0-7, d-chunk 2dp), (tokens 8-15, 2dp), (tokens 0-7, 2dp+1), (tokens 8-15, 2dp+1)
                    const int c = (dp * 2 + (mi >> 1)) & 7;
                    uint32_t vb[4];
                    ldsm_x4_trans(v_u32 + (dp / 4) * C::BOX_BYTES + swz(r0 + (mi & 1) * 8 + ri, c), vb);
                    mma_bf16(o[2 * dp], pa0, 0u, pa2, 0u, vb[0], vb[1]);
                    mma_bf16(o[2 * dp + 1], pa0, 0u, pa2, 0u, vb[2], vb[3]);
                }
                }
                // ---------- the unit's own new tokens go to the tail for later calls ----------
                // (not when the launch was split by a stale tail length: it is void and must leave the tail alone)
                if (is_new && !(early && p.tail_len[u.b] != p.tail_hint)) {
                    constexpr int CPR = D / 8;  // 16-byte chunks per row; lanes 0..CPR-1 move K, the next CPR lanes move V
                    const unsigned char *ring_stage = ring + stage * C::STAGE_BYTES;
                    for (int r = max(0, tok0 - new0); r < rows; ++r) {
                        const int tok = new0 + r;  // token of the call, tok0 <= tok < tok0 + n_tok
                        if (u.t0 + tok >= p.max_tail) break;
                        const int64_t off = ((((int64_t)u.b * p.n_layers_total + layer) * p.Hkv + u.g) * p.max_tail + u.t0 + tok) * D;
                        const int ch = lane % CPR, kv = lane / CPR;
                        if (kv < 2) {
                            const uint4 val = *(const uint4 *)(ring_stage + kv * C::NBOX * C::BOX_BYTES + (ch / 8) * C::BOX_BYTES +
                                                               swz(r0 + r, ch % 8));
                            *(uint4 *)((kv ? p.tail_v : p.tail_k) + off + ch * 8) = val;
                        }
                    }
                }
            }
            __syncwarp();
            if (lane == 0) mbar_arrive(empty_u32 + stage * 8);
        }

        // ---- end of this CTA's share of the unit: merge the warps' states ----
        {
            float l_tot = l_run, r_tot = l_rnd;
            l_tot += __shfl_xor_sync(0xffffffffu, l_tot, 1);
            l_tot += __shfl_xor_sync(0xffffffffu, l_tot, 2);
            r_tot += __shfl_xor_sync(0xffffffffu, r_tot, 1);
            r_tot += __shfl_xor_sync(0xffffffffu, r_tot, 2);
            float ev_f = 1.f;
            if constexpr (F8) ev_f = ev_set ? exp2f((float)max(-126, min(126, ev_cur))) : 1.f;   // back to plain units
#pragma unroll
            for (int nb = 0; nb < 2 * C::KS; ++nb)
                *(float2 *)(merge_o + (warp * kUnitRows + qr) * D + nb * 8 + 2 * qc) = make_float2(o[nb][0] * ev_f, o[nb][1] * ev_f);
            if (qc == 0) {
                merge_m[warp * kUnitRows + qr] = m_run;
                merge_l[warp * kUnitRows + qr] = l_tot;
                merge_r[warp * kUnitRows + qr] = r_tot;
            }
        }
        consumer_bar();
        const int64_t unit_index = (((int64_t)u.l_rel * p.B + u.b) * n_blk + u.blk) * p.Hkv + u.g;
        const int c_first = cta_of(u.flat_begin, W, gridDim.x);
        const int c_last = cta_of(u.flat_begin + u.rt - 1, W, gridDim.x);
        const int n_parts = c_last - c_first + 1;
        const int64_t lse_base = (int64_t)u.l_rel * p.lse_sl + (int64_t)u.b * p.lse_sb + (int64_t)tok0 * p.lse_ss + (int64_t)u.g * G;
        const int64_t slot = unit_index + blockIdx.x;
        const bool slot_ok = slot < p.n_part_slots && unit_index < p.n_counter_slots;
        if (n_parts > 1 && !slot_ok && tid == 0) atomicCAS(p.status, 0, MATKV_E_BOUNDS);
        for (int idx = tid; idx < n_rows * D; idx += kCW * 32) {
            const int r = idx / D, d = idx % D;
            float M = -CUDART_INF_F;
#pragma unroll
            for (int w = 0; w < kCW; ++w) M = fmaxf(M, merge_m[w * kUnitRows + r]);
            float acc = 0.f, L = 0.f, Lr = 0.f;
#pragma unroll
            for (int w = 0; w < kCW; ++w) {
                const float mw = merge_m[w * kUnitRows + r];
                const float sw = mw == -CUDART_INF_F ? 0.f : fast_exp2(mw - M);
                acc = fmaf(sw, merge_o[(w * kUnitRows + r) * D + d], acc);
                L = fmaf(sw, merge_l[w * kUnitRows + r], L);
                Lr = fmaf(sw, merge_r[w * kUnitRows + r], Lr);
            }
            // a share that holds only tiles no row can see (new-token tiles past the block's last token) is an empty
            // part: zero output, lse = -inf, never 0 / 0
            const float ov = Lr > 0.f ? acc / Lr : 0.f;
            const float lse = L > 0.f ? (M + log2f(L)) * kLn2 : -CUDART_INF_F;
            if (n_parts == 1) {
                p.out[q_base + (int64_t)(r / G) * p.q_ss + (r % G) * D + d] = __float2bfloat16(ov);
                if (p.lse_out && d == 0) p.lse_out[lse_base + (int64_t)(r / G) * p.lse_ss + (r % G)] = lse;
            } else if (slot_ok) {
                p.part_o[(slot * kUnitRows + r) * D + d] = ov;
                if (d == 0) p.part_lse[slot * kUnitRows + r] = lse;
            }
        }
        if (n_parts > 1 && slot_ok) {
            __threadfence();
            consumer_bar();
            if (tid == 0) {
                const int old = atomicAdd(p.counters + unit_index, 1);
                const int last = (old == n_parts - 1);
                if (last) p.counters[unit_index] = 0;  // ready for the next launch
                flags[1] = last;
            }
            consumer_bar();
            if (flags[1]) {
                __threadfence();
                const int64_t first_slot = unit_index + c_first;
                for (int r = warp; r < n_rows; r += kCW)
                    combine_warp(p.part_o + (first_slot * kUnitRows + r) * D, (int64_t)kUnitRows * D,
                                 p.part_lse + first_slot * kUnitRows + r, kUnitRows, n_parts, D,
                                 p.out + q_base + (int64_t)(r / G) * p.q_ss + (r % G) * D,
                                 p.lse_out ? p.lse_out + lse_base + (int64_t)(r / G) * p.lse_ss + (r % G) : nullptr);
            }
        }
        consumer_bar();  // merge area and flags are free again

        j_base += t_end - t_begin;
        f_unit = u.flat_begin + t_end;
        if (f_unit < f_end) next_unit(p, u, n_blk);
    }
    if (flags[0] && tid == 0) atomicCAS(p.status, 0, MATKV_E_TIMEOUT);
    if (tid == 0) finish_cta();   // after the last consumer barrier: every tile of this CTA has been consumed
}

// ---- launchers --------------------------------------------------------------------------------------
template <int D, int G, bool F8 = false>
static int launch_stream_t(const StreamParams &p, const CUtensorMap &kn_map, const CUtensorMap &vn_map, int grid, cudaStream_t stream) {
    using C = StreamCfg<D, G, F8>;
    static PerDeviceOnce configured;
    int once_dev;
    if (configured.need(&once_dev)) {
        MATKV_CUDA(cudaFuncSetAttribute(k_attend_stream<D, G, F8>, cudaFuncAttributeMaxDynamicSharedMemorySize, C::SMEM_BYTES));
        configured.mark(once_dev);
    }
    // Programmatic dependent launch: when the kernel before this one on the stream lets its dependents go early (this
    // kernel does, first thing), the launch itself and this kernel's barrier set-up run under that kernel's tail; the
    // kernel waits for the predecessor's completion (griddepcontrol.wait) before it reads anything a predecessor may
    // have written.  With any other predecessor the attribute changes nothing.
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)grid);
    cfg.blockDim = dim3((unsigned)kThreads);
    cfg.dynamicSmemBytes = C::SMEM_BYTES;
    cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    MATKV_CUDA(cudaLaunchKernelEx(&cfg, k_attend_stream<D, G, F8>, p, kn_map, vn_map));
    return MATKV_OK;
}

int launch_attend_stream(matkv_ctx *ctx, matkv_table *t, const AttendArgs &a, cudaStream_t stream) {
    const matkv_config &c = ctx->cfg;
    WorkspaceView ws;
    workspace_bytes_for(c, &ws, ctx->workspace);
    const int G = c.n_q_heads / c.n_kv_heads;
    const int n_blk = ceil_div(a.S, kUnitRows / G);
    StreamParams p;
    p.reqs = t->d_reqs;
    p.tmaps = t->d_tmaps;
    p.tmaps8 = t->d_tmaps8;
    p.segs = t->d_segs;
    p.n_seg_total = t->n_seg_total;
    p.tail_len = t->d_tail_len;
    p.tail_k = t->tail_k;
    p.tail_v = t->tail_v;
    p.q = a.q; p.k_new = a.k_new; p.v_new = a.v_new; p.out = a.out; p.lse_out = a.lse_out;
    p.q_sl = a.q_sl; p.q_sb = a.q_sb; p.q_ss = a.q_ss;
    p.kn_sl = a.kn_sl; p.kn_sb = a.kn_sb; p.kn_ss = a.kn_ss;
    p.lse_sl = a.lse_sl; p.lse_sb = a.lse_sb; p.lse_ss = a.lse_ss;
    p.layer0 = a.layer0; p.n_layers_launch = a.n_layers_launch; p.n_layers_total = c.n_layers;
    p.B = t->batch; p.S = a.S; p.Hkv = c.n_kv_heads; p.max_tail = c.max_tail_tokens;
    p.scale_log2 = ctx->scale * kLog2e;
    p.counters = ws.counters; p.part_lse = ws.part_lse; p.part_o = ws.part_o;
    p.n_part_slots = ws.n_part_slots; p.n_counter_slots = ws.n_counter_slots;
    p.status = ctx->d_status;
    p.advance = a.advance;
    p.done_count = ctx->d_status + 2;
    p.stream_hint = t->distinct_chunk_tiles == t->total_chunk_tiles && n_blk == 1;  // several token blocks re-read the tiles
    {   // the host's mirror of the tail length is exact unless the stream is being captured (replays do not move it)
        cudaStreamCaptureStatus cap = cudaStreamCaptureStatusNone;
        p.tail_hint = (cudaStreamIsCapturing(stream, &cap) == cudaSuccess && cap == cudaStreamCaptureStatusNone) ? t->tail_len_host : -1;
    }
    const int64_t n_units = (int64_t)a.n_layers_launch * t->batch * n_blk * c.n_kv_heads;
    if (n_units > ws.n_counter_slots)
        return fail(MATKV_E_CAPACITY, "launch of %lld units exceeds the workspace's %lld", (long long)n_units,
                    (long long)ws.n_counter_slots);
    // tiles in the launch as far as the host knows (the device recomputes it from its own tail length)
    int64_t W = 0;
    for (int b = 0; b < t->batch; ++b)
        W += (int64_t)c.n_kv_heads * n_blk * (t->h_reqs[b].chunk_tiles + ceil_div(t->tail_len_host, kTile) + ceil_div(a.S, kTile));
    W *= a.n_layers_launch;
    // the call's new tokens are fetched through their own descriptor: k_new / v_new [layers][B][S][Hkv][D]
    CUtensorMap kn_map, vn_map;
    {
        const uint64_t n_tok = (uint64_t)a.n_layers_launch * t->batch * a.S;
        int rc = encode_new_rows_map(&kn_map, a.k_new, c.head_dim, c.n_kv_heads, n_tok);
        if (!rc) rc = encode_new_rows_map(&vn_map, a.v_new, c.head_dim, c.n_kv_heads, n_tok);
        if (rc) return rc;
    }
    // by default one CTA per SM, less the SMs left to the staging copy kernel when that is in use (the launch is
    // bound by HBM with ~130 CTAs already; a copy CTA sharing an SM with a decode CTA makes that SM the straggler)
    int64_t grid = ctx->opt_decode_ctas > 0 ? ctx->opt_decode_ctas : std::max<int64_t>(ctx->n_sm - ctx->opt_stage_ctas, ctx->n_sm / 2);
    // A short launch (a few tiles per CTA: one layer of a small batch) is a chain of latencies, not a stream: every unit
    // gets the same number of CTAs, 16 at most (the last arriver then merges its unit's partials in one round trip and
    // equal units are never cut inside a CTA), and the SMs left over are where the next launch starts early.
    // Measured, config 2 with one launch per layer (8 units of 84 tiles): 13.4 us with 148 CTAs, 12.0 with 144,
    // 11.6 with 128 or 120; long launches stream best with every SM (config 4: 12.0 ms with 148, 12.4 with 128).
    if (ctx->opt_decode_ctas <= 0 && W < 32 * grid && n_units <= grid) grid = n_units * std::min<int64_t>(16, grid / n_units);
    grid = std::max<int64_t>(1, std::min<int64_t>(grid, W));
    if (t->has_fp8) {   // tables with compressed-resident chunks: the variant that also reads tiles of codes
#define MATKV_CASE8(GG) \
        if (c.head_dim == 128 && G == GG) return launch_stream_t<128, GG, true>(p, kn_map, vn_map, (int)grid, stream);
        MATKV_CASE8(1) MATKV_CASE8(2) MATKV_CASE8(4) MATKV_CASE8(8)
#undef MATKV_CASE8
        return fail(MATKV_E_INVALID_ARG, "compressed-resident chunks: unsupported head_dim %d / group %d", c.head_dim, G);
    }
#define MATKV_CASE(DD, GG) \
    if (c.head_dim == DD && G == GG) return launch_stream_t<DD, GG>(p, kn_map, vn_map, (int)grid, stream);
    MATKV_CASE(128, 1) MATKV_CASE(128, 2) MATKV_CASE(128, 4) MATKV_CASE(128, 8)
    MATKV_CASE(64, 1) MATKV_CASE(64, 2) MATKV_CASE(64, 4) MATKV_CASE(64, 8)
#undef MATKV_CASE
    return fail(MATKV_E_INVALID_ARG, "unsupported head_dim %d / group %d", c.head_dim, G);
}

// ---- decode with built-in scratch (no allocation anywhere on this path) ----------------------------
// The split-KV partials and arrival counters of this one entry point live in a file-scope device
// array instead of the caller's workspace.  Every GPU that loads the library carries the array until
// the process exits, so it is kept small: it bounds the call at kStaticUnits (request, KV head) pairs
// and kStaticCtas CTAs.
constexpr int kStaticUnits = 256;
constexpr int kStaticCtas = 256;
constexpr int kStaticParts = kStaticUnits + kStaticCtas;
constexpr size_t kStaticCounterBytes = sizeof(int32_t) * kStaticUnits;                    //      1,024
constexpr size_t kStaticLseBytes = sizeof(float) * kStaticParts * kUnitRows;              //     16,384
constexpr size_t kStaticOBytes = sizeof(float) * (size_t)kStaticParts * kUnitRows * 128;  //  2,097,152
constexpr size_t kStaticBytes = kStaticCounterBytes + kStaticLseBytes + kStaticOBytes;    //  2,114,560 in all
static __device__ __align__(256) unsigned char g_static_scratch[kStaticBytes];
// Device address of g_static_scratch per device ordinal.  In host code the array's name is only a
// stand-in for the symbol, never an address a kernel may use: the address comes from
// cudaGetSymbolAddress, asked once per device with that device current.
static void *g_static_scratch_addr[64] = {};

}  // namespace matkv

extern "C" int matkv_attend_decode_static(matkv_ctx *ctx, matkv_table *t, int32_t layer, const void *q, const void *k_new,
                                          const void *v_new, void *out, float *lse_out, void *stream) {
    using namespace matkv;
    if (!ctx || !t || !q || !k_new || !v_new || !out) return fail(MATKV_E_INVALID_ARG, "matkv_attend_decode_static: null argument");
    if (t->ctx != ctx) return fail(MATKV_E_INVALID_ARG, "matkv_attend_decode_static: table belongs to another context");
    const matkv_config &c = ctx->cfg;
    if (layer < 0 || layer >= c.n_layers) return fail(MATKV_E_INVALID_ARG, "matkv_attend_decode_static: layer %d", layer);
    if (((uintptr_t)q | (uintptr_t)k_new | (uintptr_t)v_new | (uintptr_t)out) % 16)
        return fail(MATKV_E_ALIGNMENT, "matkv_attend_decode_static: q, k_new, v_new and out must be 16-byte aligned");
    if (c.rope_theta != 0.f) return fail(MATKV_E_INVALID_ARG, "matkv_attend_decode_static: rotary mode is not available");
    if (t->has_fp8) return fail(MATKV_E_INVALID_ARG, "matkv_attend_decode_static: the table holds compressed-resident chunks");
    if (t->tail_len_host + 1 > c.max_tail_tokens)
        return fail(MATKV_E_CAPACITY, "matkv_attend_decode_static: tail holds %d tokens, one more exceeds max_tail_tokens %d",
                    t->tail_len_host, c.max_tail_tokens);
    const int64_t n_units = (int64_t)t->batch * c.n_kv_heads;
    if (n_units > kStaticUnits)
        return fail(MATKV_E_CAPACITY,
                    "matkv_attend_decode_static: batch %d x %d KV heads = %lld units, the built-in scratch holds %d; "
                    "use matkv_attend_decode with a caller workspace",
                    t->batch, c.n_kv_heads, (long long)n_units, kStaticUnits);
    if (ctx->device < 0 || ctx->device >= 64) return fail(MATKV_E_CAPACITY, "matkv_attend_decode_static: device ordinal %d", ctx->device);
    int prev = -1;
    MATKV_CUDA(cudaGetDevice(&prev));
    if (prev != ctx->device) MATKV_CUDA(cudaSetDevice(ctx->device));
    int rc = MATKV_OK;
    do {
        void *&base = g_static_scratch_addr[ctx->device];
        if (!base) {  // first call on this device: resolve the symbol (not inside a stream capture)
            void *ptr = nullptr;
            cudaError_t e = cudaGetSymbolAddress(&ptr, g_static_scratch);
            if (e != cudaSuccess || !ptr) {
                rc = cuda_fail(e, "cudaGetSymbolAddress(g_static_scratch)");
                break;
            }
            base = ptr;
        }
        cudaStream_t st = (cudaStream_t)stream;
        // the array keeps the last call's contents: the arrival counters must start at zero
        cudaError_t e = cudaMemsetAsync(base, 0, kStaticCounterBytes, st);
        if (e != cudaSuccess) {
            rc = cuda_fail(e, "cudaMemsetAsync(counters)");
            break;
        }
        StreamParams p;
        p.reqs = t->d_reqs;
        p.tmaps = t->d_tmaps;
        p.tmaps8 = nullptr;
        p.segs = t->d_segs;
        p.n_seg_total = t->n_seg_total;
        p.tail_len = t->d_tail_len;
        p.tail_k = t->tail_k;
        p.tail_v = t->tail_v;
        p.q = (const __nv_bfloat16 *)q; p.k_new = (const __nv_bfloat16 *)k_new; p.v_new = (const __nv_bfloat16 *)v_new;
        p.out = (__nv_bfloat16 *)out; p.lse_out = lse_out;
        p.q_sl = 0; p.q_sb = (int64_t)c.n_q_heads * c.head_dim; p.q_ss = 0;
        p.kn_sl = 0; p.kn_sb = (int64_t)c.n_kv_heads * c.head_dim; p.kn_ss = 0;
        p.lse_sl = 0; p.lse_sb = c.n_q_heads; p.lse_ss = 0;
        p.layer0 = layer; p.n_layers_launch = 1; p.n_layers_total = c.n_layers;
        p.B = t->batch; p.S = 1; p.Hkv = c.n_kv_heads; p.max_tail = c.max_tail_tokens;
        p.scale_log2 = ctx->scale * kLog2e;
        p.counters = (int32_t *)base;
        p.part_lse = (float *)((char *)base + kStaticCounterBytes);
        p.part_o = (float *)((char *)base + kStaticCounterBytes + kStaticLseBytes);
        p.n_part_slots = kStaticParts; p.n_counter_slots = kStaticUnits;
        p.status = ctx->d_status;
        p.advance = 0;
        p.done_count = ctx->d_status + 2;
        p.stream_hint = t->distinct_chunk_tiles == t->total_chunk_tiles;
        p.tail_hint = -1;
        CUtensorMap kn_map, vn_map;
        rc = encode_new_rows_map(&kn_map, k_new, c.head_dim, c.n_kv_heads, (uint64_t)t->batch);
        if (!rc) rc = encode_new_rows_map(&vn_map, v_new, c.head_dim, c.n_kv_heads, (uint64_t)t->batch);
        if (rc) break;
        int64_t W = 0;
        for (int b = 0; b < t->batch; ++b)
            W += (int64_t)c.n_kv_heads * (t->h_reqs[b].chunk_tiles + ceil_div(t->tail_len_host, kTile) + 1);
        int64_t grid = std::min<int64_t>(std::min<int64_t>(ctx->n_sm, kStaticCtas), W);
        if (grid < 1) grid = 1;
        const int G = c.n_q_heads / c.n_kv_heads;
        rc = fail(MATKV_E_INVALID_ARG, "unsupported head_dim %d / group %d", c.head_dim, G);
#define MATKV_CASE(DD, GG) \
        if (c.head_dim == DD && G == GG) rc = launch_stream_t<DD, GG>(p, kn_map, vn_map, (int)grid, st);
        MATKV_CASE(128, 1) MATKV_CASE(128, 2) MATKV_CASE(128, 4) MATKV_CASE(128, 8)
        MATKV_CASE(64, 1) MATKV_CASE(64, 2) MATKV_CASE(64, 4) MATKV_CASE(64, 8)
#undef MATKV_CASE
    } while (0);
    if (prev != ctx->device) cudaSetDevice(prev);
    return rc;
}

namespace matkv {

// Self-test of the bounded wait: one thread waits on a barrier that nothing ever signals.  The wait must
// give up after its limit, report MATKV_E_TIMEOUT through the status word and return normally.
__global__ void k_wait_selftest(int32_t *status, long long limit_cycles) {
    __shared__ uint64_t bar;
    __shared__ int abort_flag;
    if (threadIdx.x == 0) {
        mbar_init(smem_u32(&bar), 1);
        abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        const long long t0 = clock64();
        bool done = false;
        while (!done && clock64() - t0 <= limit_cycles) done = mbar_try_wait(smem_u32(&bar), 0);
        if (!done) atomicCAS(status, 0, MATKV_E_TIMEOUT);
    }
}

int launch_wait_selftest(matkv_ctx *ctx, double seconds, cudaStream_t stream) {
    int khz = 0;
    MATKV_CUDA(cudaDeviceGetAttribute(&khz, cudaDevAttrClockRate, ctx->device));
    k_wait_selftest<<<1, 32, 0, stream>>>(ctx->d_status, (long long)(seconds * 1e3 * khz));
    MATKV_CUDA(cudaGetLastError());
    return MATKV_OK;
}

int launch_lse_combine(matkv_ctx *, int32_t n_rows, int32_t n_parts, int32_t D, const float *o_parts, const float *lse_parts,
                       void *out, float *lse_out, cudaStream_t stream) {
    const int warps = 4;
    k_lse_combine<<<(n_rows + warps - 1) / warps, warps * 32, 0, stream>>>(n_rows, n_parts, D, o_parts, lse_parts,
                                                                         (__nv_bfloat16 *)out, lse_out);
    MATKV_CUDA(cudaGetLastError());
    return MATKV_OK;
}

}  // namespace matkv
