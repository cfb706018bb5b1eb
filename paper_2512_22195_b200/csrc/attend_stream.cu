// K1: chunk-table streaming attention (decode, and small query suffixes) + K2: log-sum-exp combine.
//
// One persistent CTA per SM.  The work of a launch is the flat list of KV tiles (kTile tokens of one
// (layer, request, suffix token, KV head) "unit"); CTA c owns the contiguous range
// [c*W/n, (c+1)*W/n) of that list, so every SM streams the same number of bytes whatever the shape.
// Inside a CTA one producer thread walks its range and moves each tile's K rows and V rows from the
// scattered chunk blobs (or the tail, or the new tokens) into a shared-memory ring with bulk
// asynchronous copies (cp.async.bulk + mbarrier complete_tx); the consumer warps take the tiles round-robin and run an independent online softmax for the G query heads that share the KV head
// (fp32, exp2-based).  At the end of a unit the warps' states are merged through shared memory; a
// unit that spans several CTAs leaves one partial (normalised o, lse) per CTA in the workspace and
// the last CTA to arrive (atomic ticket, no waiting) merges them by log-sum-exp.
#include <cuda_runtime.h>
#include <cuda_bf16.h>
#include <math_constants.h>

#include <algorithm>

#include "matkv_internal.h"

namespace matkv {

// Consumer warps per CTA (+1 producer warp).  Registers are allocated to warps in fours, so a CTA is
// 8 warps x 255 registers or 16 warps x 128 registers; the thin variant hides more latency and is used
// whenever q and o of the G heads fit its register budget.
// Copies are issued per 64-token tile (large copies keep the copy engine's per-copy cost low); a warp
// works on a quarter (thin variant) or half (fat variant) of a tile so that the slots being consumed
// leave room in the ring for tiles in flight.
template <int G> constexpr bool thin_variant() { return G == 2 || G == 4; }
template <int G> constexpr int consumer_warps() { return thin_variant<G>() ? 15 : 7; }
constexpr int kMaxDynSmem = 232448;            // 227 KB opt-in limit per CTA on sm_100
constexpr long long kWaitCycles = 2000000000LL;  // bounded waits give up after about a second
constexpr float kLog2e = 1.4426950408889634f;
constexpr float kLn2 = 0.6931471805599453f;

struct StreamParams {
    const DevSeg *segs;
    const DevReq *reqs;
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
};

// ---- PTX helpers ---------------------------------------------------------------------------------
__device__ __forceinline__ uint32_t smem_u32(const void *p) { return (uint32_t)__cvta_generic_to_shared(p); }
__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count));
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
    asm volatile("{\n .reg .b64 st;\n mbarrier.arrive.shared::cta.b64 st, [%0];\n}" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
    asm volatile("{\n .reg .b64 st;\n mbarrier.arrive.expect_tx.shared::cta.b64 st, [%0], %1;\n}" ::"r"(bar), "r"(bytes)
                 : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity) {
    uint32_t ok;
    asm volatile(
        "{\n .reg .pred p;\n mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n selp.u32 %0, 1, 0, p;\n}"
        : "=r"(ok)
        : "r"(bar), "r"(parity)
        : "memory");
    return ok != 0;
}
// Bounded wait: returns false (and raises the CTA's abort flag) after about a second.
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile int *abort_flag) {
    if (mbar_try_wait(bar, parity)) return true;
    const long long t0 = clock64();
    while (true) {
        if (mbar_try_wait(bar, parity)) return true;
        if (*abort_flag) return false;
        if (clock64() - t0 > kWaitCycles) {
            *abort_flag = 1;
            return false;
        }
    }
}
// A consumer's wait for fill number `want` of a ring slot.  Warps take work items round-robin, so a
// warp can reach a slot whose PREVIOUS fill is still in flight, and the one-bit phase of an mbarrier
// cannot tell "fill n-1 incomplete" from "fill n complete".  The producer therefore publishes the fill
// number of a slot (upper half of the slot's tag word) before it issues the copy, which it does only
// after the slot's previous fill was consumed and released; once the consumer sees its number there,
// the parity test is unambiguous.  Returns the tag word, or 0 after the bounded wait ran out.
__device__ __forceinline__ uint32_t slot_wait(const volatile uint32_t *tag, uint32_t want, uint32_t bar, uint32_t parity,
                                              volatile int *abort_flag) {
    uint32_t w = *tag;
    if ((w >> 16) == (want & 0xffffu) && mbar_try_wait(bar, parity)) return w;
    const long long t0 = clock64();
    while (true) {
        w = *tag;
        if ((w >> 16) == (want & 0xffffu) && mbar_try_wait(bar, parity)) return w;
        if (*abort_flag) return 0;
        if (clock64() - t0 > kWaitCycles) {
            *abort_flag = 1;
            return 0;
        }
    }
}
__device__ __forceinline__ void bulk_g2s(uint32_t dst, const void *src, uint32_t bytes, uint32_t bar) {
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(dst),
                 "l"(src), "r"(bytes), "r"(bar)
                 : "memory");
}
template <int CW> __device__ __forceinline__ void consumer_bar() { asm volatile("bar.sync 1, %0;" ::"n"(CW * 32) : "memory"); }
__device__ __forceinline__ float fast_exp2(float x) {
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}
__device__ __forceinline__ float bf_lo(uint32_t w) { return __uint_as_float(w << 16); }
__device__ __forceinline__ float bf_hi(uint32_t w) { return __uint_as_float(w & 0xffff0000u); }

// ---- the flat work list ----------------------------------------------------------------------------
__host__ __device__ __forceinline__ int ceil_div(int a, int b) { return (a + b - 1) / b; }
// sum over i in [0, S) of ceil((i + 1) / kTile)
__host__ __device__ __forceinline__ int64_t new_tiles_sum(int S) {
    const int64_t full = S / kTile, rem = S % kTile;
    return (int64_t)kTile * full * (full + 1) / 2 + rem * (full + 1);
}

struct UnitPos {
    int32_t l_rel, b, i, g;  // layer (relative to layer0), request, suffix token, KV head
    int32_t tile;            // first tile of this CTA's share inside the unit
    int32_t rt;              // tiles in the unit
    int32_t chunk_tiles, tail_tiles, t0, seg_begin;
    int64_t flat_begin;      // flat index of the unit's first tile
};

struct CtaRange {
    int64_t begin, end, W;
    UnitPos first;
};

__device__ __forceinline__ int32_t clamp_t0(const StreamParams &p, int b) {
    int32_t t0 = p.tail_len[b];
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
}
__device__ __forceinline__ void set_rt(UnitPos &u) { u.rt = u.chunk_tiles + u.tail_tiles + ceil_div(u.i + 1, kTile); }

// advance to the next unit in (layer, request, token, head) order
__device__ __forceinline__ void next_unit(const StreamParams &p, UnitPos &u) {
    u.flat_begin += u.rt;
    u.tile = 0;
    if (++u.g < p.Hkv) return;
    u.g = 0;
    if (++u.i < p.S) {
        set_rt(u);
        return;
    }
    u.i = 0;
    if (++u.b >= p.B) {
        u.b = 0;
        ++u.l_rel;
    }
    if (u.l_rel < p.n_layers_launch) load_req(p, u);
    set_rt(u);
}

__device__ void locate_range(const StreamParams &p, CtaRange &r) {
    int64_t w_layer = 0;
    for (int b = 0; b < p.B; ++b) {
        const int base = p.reqs[b].chunk_tiles + ceil_div(clamp_t0(p, b), kTile);
        w_layer += (int64_t)p.Hkv * ((int64_t)p.S * base + new_tiles_sum(p.S));
    }
    r.W = w_layer * p.n_layers_launch;
    const int64_t n = gridDim.x, c = blockIdx.x;
    r.begin = c * r.W / n;
    r.end = (c + 1) * r.W / n;
    UnitPos &u = r.first;
    u = UnitPos{};
    if (r.begin >= r.end) return;
    int64_t f = r.begin;
    u.l_rel = (int32_t)(f / w_layer);
    int64_t rem = f % w_layer;
    int b = 0;
    for (; b < p.B; ++b) {
        const int base = p.reqs[b].chunk_tiles + ceil_div(clamp_t0(p, b), kTile);
        const int64_t blk = (int64_t)p.Hkv * ((int64_t)p.S * base + new_tiles_sum(p.S));
        if (rem < blk) break;
        rem -= blk;
    }
    u.b = b;
    load_req(p, u);
    int i = 0;
    for (; i < p.S; ++i) {
        const int64_t blk = (int64_t)p.Hkv * (u.chunk_tiles + u.tail_tiles + ceil_div(i + 1, kTile));
        if (rem < blk) break;
        rem -= blk;
    }
    u.i = i;
    set_rt(u);
    u.g = (int32_t)(rem / u.rt);
    u.tile = (int32_t)(rem % u.rt);
    u.flat_begin = f - u.tile;
}

// CTA that owns flat tile f when W tiles are split over n CTAs as [c*W/n, (c+1)*W/n)
__device__ __forceinline__ int cta_of(int64_t f, int64_t W, int64_t n) { return (int)(((f + 1) * n - 1) / W); }

// Where a unit's tile lives.
struct TileSrc {
    const __nv_bfloat16 *k, *v;  // first row
    int64_t row_stride;          // elements between rows
    int32_t rows;
    int32_t new_first;           // >= 0: tile holds new tokens new_first .. new_first+rows-1; else -1
};

// The producer's cursor over a request's segments.  Tile indices only grow inside a unit, so the
// current segment stays in registers and global memory is touched once per segment, not per tile.
struct SegCursor {
    int32_t seg, tiles_before, seg_tiles;
    DevSeg sg;
    __device__ __forceinline__ void reset() { seg = -1; tiles_before = 0; seg_tiles = 0; }
};

template <int D>
__device__ __forceinline__ TileSrc tile_source(const StreamParams &p, const UnitPos &u, int tile, SegCursor &cur) {
    TileSrc s;
    const int layer = p.layer0 + u.l_rel;
    if (tile < u.chunk_tiles) {
        while (cur.seg < 0 || tile >= cur.tiles_before + cur.seg_tiles) {
            cur.tiles_before += cur.seg_tiles;
            ++cur.seg;
            cur.sg = p.segs[u.seg_begin + cur.seg];
            cur.seg_tiles = ceil_div(cur.sg.len, kTile);
        }
        const int r0 = (tile - cur.tiles_before) * kTile;
        const int64_t kslab = ((int64_t)layer * 2 * p.Hkv + u.g) * cur.sg.len;
        const int64_t vslab = (((int64_t)layer * 2 + 1) * p.Hkv + u.g) * cur.sg.len;
        s.k = cur.sg.base + (kslab + r0) * D;
        s.v = cur.sg.base + (vslab + r0) * D;
        s.row_stride = D;
        s.rows = min(kTile, cur.sg.len - r0);
        s.new_first = -1;
    } else if (tile < u.chunk_tiles + u.tail_tiles) {
        const int r0 = (tile - u.chunk_tiles) * kTile;
        const int64_t off = ((((int64_t)u.b * p.n_layers_total + layer) * p.Hkv + u.g) * p.max_tail + r0) * D;
        s.k = p.tail_k + off;
        s.v = p.tail_v + off;
        s.row_stride = D;
        s.rows = min(kTile, u.t0 - r0);
        s.new_first = -1;
    } else {
        const int r0 = (tile - u.chunk_tiles - u.tail_tiles) * kTile;
        const int64_t off = (int64_t)u.l_rel * p.kn_sl + (int64_t)u.b * p.kn_sb + (int64_t)r0 * p.kn_ss + (int64_t)u.g * D;
        s.k = p.k_new + off;
        s.v = p.v_new + off;
        s.row_stride = p.kn_ss;
        s.rows = min(kTile, u.i + 1 - r0);
        s.new_first = r0;
    }
    return s;
}

// ---- K2 core: merge P partial attentions of one row with one warp -----------------------------------
// o_parts: part p at o_parts + p*o_stride (D floats, normalised inside the part); lse natural log.
__device__ void combine_warp(const float *o_parts, int64_t o_stride, const float *lse_parts, int64_t lse_stride, int P,
                             int D, __nv_bfloat16 *out, float *lse_out) {
    const int lane = threadIdx.x & 31;
    float m = -CUDART_INF_F;
    for (int p = lane; p < P; p += 32) m = fmaxf(m, __ldcg(lse_parts + p * lse_stride));
#pragma unroll
    for (int off = 16; off; off >>= 1) m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, off));
    if (m == -CUDART_INF_F) {  // no part saw any key
        for (int d = lane; d < D; d += 32) out[d] = __float2bfloat16(0.f);
        if (lse_out && lane == 0) *lse_out = -CUDART_INF_F;
        return;
    }
    float z = 0.f;
    for (int p = lane; p < P; p += 32) z += exp2f((__ldcg(lse_parts + p * lse_stride) - m) * kLog2e);
#pragma unroll
    for (int off = 16; off; off >>= 1) z += __shfl_xor_sync(0xffffffffu, z, off);
    const float lse = m + logf(z);
    for (int d = lane; d < D; d += 32) {
        float acc = 0.f;
        for (int p = 0; p < P; ++p) {
            const float w = exp2f((__ldcg(lse_parts + p * lse_stride) - lse) * kLog2e);
            acc = fmaf(w, __ldcg(o_parts + p * o_stride + d), acc);
        }
        out[d] = __float2bfloat16(acc);
    }
    if (lse_out && lane == 0) *lse_out = lse;
}

__global__ void k_lse_combine(int n_rows, int P, int D, const float *__restrict__ o_parts,
                              const float *__restrict__ lse_parts, __nv_bfloat16 *__restrict__ out, float *lse_out) {
    const int row = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
    if (row >= n_rows) return;
    combine_warp(o_parts + (int64_t)row * P * D, D, lse_parts + (int64_t)row * P, 1, P, D, out + (int64_t)row * D,
                 lse_out ? lse_out + row : nullptr);
}

// ---- K1 -------------------------------------------------------------------------------------------
// packed fp32 pairs: sm_100 issues two FMAs per instruction on a 64-bit register pair
__device__ __forceinline__ float2 ffma2(float2 a, float2 b, float2 c) {
    unsigned long long d;
    asm("fma.rn.f32x2 %0, %1, %2, %3;"
        : "=l"(d)
        : "l"(*reinterpret_cast<unsigned long long *>(&a)), "l"(*reinterpret_cast<unsigned long long *>(&b)),
          "l"(*reinterpret_cast<unsigned long long *>(&c)));
    return *reinterpret_cast<float2 *>(&d);
}
__device__ __forceinline__ float2 fmul2(float2 a, float2 b) {
    unsigned long long d;
    asm("mul.rn.f32x2 %0, %1, %2;"
        : "=l"(d)
        : "l"(*reinterpret_cast<unsigned long long *>(&a)), "l"(*reinterpret_cast<unsigned long long *>(&b)));
    return *reinterpret_cast<float2 *>(&d);
}
__device__ __forceinline__ float2 bf2(uint32_t w) { return make_float2(bf_lo(w), bf_hi(w)); }

template <int D, int G>
struct StreamCfg {
    static constexpr int CW = consumer_warps<G>();             // consumer warps
    static constexpr int THREADS = (CW + 1) * 32;
    static constexpr int SPLIT = thin_variant<G>() ? 4 : 2;    // warps that share one tile
    static constexpr int HROWS = kTile / SPLIT;                // rows of a tile one warp handles
    static constexpr int LPR = (D == 128 && (SPLIT == 2 || G == 8)) ? 16 : 8;  // lanes that share one K/V row
    static constexpr int DPL = D / LPR;                        // dims per lane
    static constexpr int NV = DPL / 8;                         // 16-byte vectors per lane per row
    static constexpr int NPAIR = DPL / 2;                      // fp32 pairs per lane per row
    static constexpr int RG = 32 / LPR;                        // row groups per warp
    static constexpr int RPG = HROWS / RG;                     // rows per group per work item
    static constexpr int SUBR = (RPG < 32 / G) ? RPG : 32 / G; // rows per group per reduce batch
    static constexpr int NSUB = RPG / SUBR;
    static constexpr int NP = G * SUBR;                        // partial dot products per lane per batch
    static constexpr int NF = NP / LPR;                        // scores per lane after the reduce-scatter
    static constexpr int LPH = LPR / G;                        // lanes of a group that end up with the same head
    static constexpr int SLOT_BYTES = kTile * D * 2;
    static constexpr int MERGE_BYTES = (CW * G * (D + 2) * 4 + 15) / 16 * 16;
    static constexpr int PS_STRIDE = (HROWS * G * 2 + G + 3) / 4 * 4;  // floats per warp: p pairs [row][head], alpha[head]
    static constexpr int PS_BYTES = CW * PS_STRIDE * 4;
    static constexpr int FIXED_BYTES = MERGE_BYTES + PS_BYTES + 1024;
    static constexpr int NSLOT_MAX = (kMaxDynSmem - FIXED_BYTES) / SLOT_BYTES;
    static constexpr int NSLOT = NSLOT_MAX > 24 ? 24 : NSLOT_MAX;
    static constexpr int SMEM_BYTES = NSLOT * SLOT_BYTES + FIXED_BYTES;
    static_assert(DPL % 8 == 0 && NF >= 1 && SUBR % NF == 0 && LPH >= 1, "unsupported head_dim / group size");
    static_assert(NSLOT >= 4, "ring too small");
};

template <int D, int G>
__global__ void __launch_bounds__((consumer_warps<G>() + 1) * 32, 1) k_attend_stream(const StreamParams p) {
    using C = StreamCfg<D, G>;
    extern __shared__ __align__(128) unsigned char smem[];
    unsigned char *ring = smem;
    float *merge_o = (float *)(smem + C::NSLOT * C::SLOT_BYTES);         // [warp][G][D]
    float *merge_m = merge_o + C::CW * G * D;                   // [warp][G]
    float *merge_l = merge_m + C::CW * G;                       // [warp][G]
    float *ps_all = (float *)(smem + C::NSLOT * C::SLOT_BYTES + C::MERGE_BYTES);  // [warp][PS_STRIDE]
    unsigned char *misc = smem + C::NSLOT * C::SLOT_BYTES + C::MERGE_BYTES + C::PS_BYTES;
    uint64_t *bars = (uint64_t *)misc;                                   // full[NSLOT], empty[NSLOT]
    // per slot tag: rows | (the unit's own new row + 1) << 8 | (number of the slot's current fill) << 16
    volatile uint32_t *tags = (volatile uint32_t *)(misc + 2 * 24 * 8);
    CtaRange *range = (CtaRange *)(misc + 2 * 24 * 8 + 2 * 24 * 4);
    volatile int *flags = (volatile int *)(misc + 2 * 24 * 8 + 2 * 24 * 4 + sizeof(CtaRange) + 8);  // [0] abort, [1] last arriver

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    if (tid == 0) {
        for (int s = 0; s < C::NSLOT; ++s) {
            mbar_init(smem_u32(bars + s), 1);
            mbar_init(smem_u32(bars + C::NSLOT + s), C::SPLIT);
            tags[s] = 0xffff0000u;
        }
        flags[0] = 0;
        flags[1] = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
        locate_range(p, *range);
    }
    __syncthreads();
    const int64_t f_begin = range->begin, f_end = range->end, W = range->W;
    if (f_begin >= f_end) return;
    const uint32_t ring_u32 = smem_u32(ring), full_u32 = smem_u32(bars), empty_u32 = smem_u32(bars + C::NSLOT);

    if (warp == C::CW) {
        // ================= producer: one thread walks the table and feeds the ring =================
        if (lane != 0) return;
        UnitPos u = range->first;
        SegCursor cur;
        cur.reset();
        int64_t f = f_begin;
        uint32_t seq = 0;
        bool ok = true;
        while (f < f_end && ok) {
            const int t_end = (int)min((int64_t)u.rt, f_end - u.flat_begin);
            for (int t = u.tile; t < t_end && ok; ++t, ++f) {
                const TileSrc s = tile_source<D>(p, u, t, cur);
                uint32_t m = (uint32_t)s.rows;
                if (s.new_first >= 0 && u.i >= s.new_first && u.i < s.new_first + s.rows) m |= (uint32_t)(u.i - s.new_first + 1) << 8;
#pragma unroll
                for (int kv = 0; kv < 2; ++kv, ++seq) {
                    const uint32_t slot = seq % C::NSLOT, use = seq / C::NSLOT;
                    if (use > 0 && !mbar_wait(empty_u32 + slot * 8, (use - 1) & 1, flags)) {
                        ok = false;
                        break;
                    }
                    const __nv_bfloat16 *src = kv ? s.v : s.k;
                    const uint32_t dst = ring_u32 + slot * C::SLOT_BYTES, bar = full_u32 + slot * 8;
                    tags[slot] = m | (use << 16);  // published only after the slot's previous fill was consumed and released
                    mbar_expect_tx(bar, (uint32_t)s.rows * D * 2);
                    if (s.row_stride == D) {
                        bulk_g2s(dst, src, (uint32_t)s.rows * D * 2, bar);
                    } else {
                        for (int r = 0; r < s.rows; ++r) bulk_g2s(dst + r * D * 2, src + (int64_t)r * s.row_stride, D * 2, bar);
                    }
                }
            }
            if (f < f_end && ok) {
                next_unit(p, u);
                cur.reset();
            }
        }
        if (!ok) {
            // gave up: wait (bounded) for the copies already issued so none lands after the CTA has gone
            atomicCAS(p.status, 0, MATKV_E_TIMEOUT);
            const uint32_t lo = seq > (uint32_t)C::NSLOT ? seq - C::NSLOT : 0;
            for (uint32_t s2 = lo; s2 < seq; ++s2) {
                const long long t0 = clock64();
                while (!mbar_try_wait(full_u32 + (s2 % C::NSLOT) * 8, (s2 / C::NSLOT) & 1) && clock64() - t0 < kWaitCycles) {}
            }
        }
        return;
    }

    // ================= consumers =================
    const int grp = lane / C::LPR, jl = lane % C::LPR;
    const int my_h = jl / C::LPH;  // head whose scores this lane holds after the reduce-scatter
    float *ps = ps_all + warp * C::PS_STRIDE;     // this warp's (p, p)[row][head], then alpha[head]
    float *alpha_s = ps + C::HROWS * G * 2;

    float2 qf[G][C::NPAIR];
    float2 of[G][C::NPAIR];
    float m_run = -CUDART_INF_F, l_run = 0.f;

    UnitPos u = range->first;
    int64_t f_unit = f_begin;   // flat index of this CTA's first tile inside the current unit
    int64_t j_base = 0;         // CTA-local index of that tile
    while (f_unit < f_end) {
        const int t_begin = u.tile;
        const int t_end = (int)min((int64_t)u.rt, f_end - u.flat_begin);
        const int layer = p.layer0 + u.l_rel;
        // ---- per-unit setup: query (pre-scaled by scale*log2 e), cleared state ----
        {
            const __nv_bfloat16 *qb = p.q + (int64_t)u.l_rel * p.q_sl + (int64_t)u.b * p.q_sb + (int64_t)u.i * p.q_ss +
                                      (int64_t)u.g * G * D;
            const float2 sc2 = make_float2(p.scale_log2, p.scale_log2);
#pragma unroll
            for (int h = 0; h < G; ++h)
#pragma unroll
                for (int v = 0; v < C::NV; ++v) {
                    const uint4 w = *(const uint4 *)(qb + h * D + (v * C::LPR + jl) * 8);
                    qf[h][v * 4 + 0] = fmul2(bf2(w.x), sc2);
                    qf[h][v * 4 + 1] = fmul2(bf2(w.y), sc2);
                    qf[h][v * 4 + 2] = fmul2(bf2(w.z), sc2);
                    qf[h][v * 4 + 3] = fmul2(bf2(w.w), sc2);
                }
#pragma unroll
            for (int h = 0; h < G; ++h)
#pragma unroll
                for (int d = 0; d < C::NPAIR; ++d) of[h][d] = make_float2(0.f, 0.f);
            m_run = -CUDART_INF_F;
            l_run = 0.f;
        }
        // ---- this warp's work items of the unit ----
        // CTA-local tile j = j_base + (t - t_begin) splits into SPLIT work items hj = j*SPLIT + half;
        // warp w takes hj == w (mod CW)
        const int64_t hj_begin = j_base * C::SPLIT, hj_end = (j_base + (t_end - t_begin)) * C::SPLIT;
        int64_t hj = hj_begin + (int)((warp - hj_begin % C::CW + C::CW) % C::CW);
        for (; hj < hj_end; hj += C::CW) {
            const int64_t j = hj / C::SPLIT;
            const int row0 = (int)(hj % C::SPLIT) * C::HROWS;
            const uint32_t seq_k = (uint32_t)(2 * j), seq_v = seq_k + 1;
            const uint32_t slot_k = seq_k % C::NSLOT, slot_v = seq_v % C::NSLOT;
            const unsigned char *ks = ring + slot_k * C::SLOT_BYTES + row0 * (D * 2);
            const unsigned char *vs = ring + slot_v * C::SLOT_BYTES + row0 * (D * 2);

            // ---------- scores ----------
            const uint32_t mt = slot_wait(tags + slot_k, seq_k / C::NSLOT, full_u32 + slot_k * 8, (seq_k / C::NSLOT) & 1, flags);
            const int rows = (int)(mt & 0xff) - row0;   // valid rows of this work item (may be <= 0)
            int own_row = (int)((mt >> 8) & 0xff) - 1 - row0;  // the unit's own new token, if it sits in this work item
            if (own_row >= C::HROWS) own_row = -1;
            if (rows <= 0) {                            // the tile ends before this half: just release the slots
                slot_wait(tags + slot_v, seq_v / C::NSLOT, full_u32 + slot_v * 8, (seq_v / C::NSLOT) & 1, flags);
                __syncwarp();
                if (lane == 0) {
                    mbar_arrive(empty_u32 + slot_k * 8);
                    mbar_arrive(empty_u32 + slot_v * 8);
                }
                continue;
            }
            float sc[C::NSUB][C::NF];
#pragma unroll
            for (int sub = 0; sub < C::NSUB; ++sub) {
                float part[C::NP];
#pragma unroll
                for (int r = 0; r < C::SUBR; ++r) {
                    const int row = (sub * C::SUBR + r) * C::RG + grp;
                    float2 kf[C::NPAIR];
#pragma unroll
                    for (int v = 0; v < C::NV; ++v) {
                        const uint4 w = *(const uint4 *)(ks + row * (D * 2) + (v * C::LPR + jl) * 16);
                        kf[v * 4 + 0] = bf2(w.x); kf[v * 4 + 1] = bf2(w.y);
                        kf[v * 4 + 2] = bf2(w.z); kf[v * 4 + 3] = bf2(w.w);
                    }
#pragma unroll
                    for (int h = 0; h < G; ++h) {
                        float2 a = make_float2(0.f, 0.f);
#pragma unroll
                        for (int d = 0; d < C::NPAIR; ++d) a = ffma2(qf[h][d], kf[d], a);
                        part[h * C::SUBR + r] = a.x + a.y;
                    }
                }
                // reduce-scatter over the LPR lanes of the row group: afterwards this lane holds the
                // complete dot products number base + 0..NF-1, base = its lane bits read as an index
                int n = C::NP;
#pragma unroll
                for (int off = C::LPR / 2; off >= 1; off >>= 1) {
                    n >>= 1;
                    const bool upper = (jl & off) != 0;
#pragma unroll
                    for (int k = 0; k < n; ++k) {
                        const float send = upper ? part[k] : part[k + n];
                        const float keep = upper ? part[k + n] : part[k];
                        part[k] = keep + __shfl_xor_sync(0xffffffffu, send, off);
                    }
                }
#pragma unroll
                for (int k = 0; k < C::NF; ++k) {
                    const int r = (jl % C::LPH) * C::NF + k;  // row of the batch (head index = my_h)
                    const int row = (sub * C::SUBR + r) * C::RG + grp;
                    sc[sub][k] = row < rows ? part[k] : -CUDART_INF_F;
                }
            }
            // the new token's K row goes to the tail for later steps (this unit's own token only)
            if (own_row >= 0 && u.t0 + u.i < p.max_tail) {
                const int64_t off = ((((int64_t)u.b * p.n_layers_total + layer) * p.Hkv + u.g) * p.max_tail + u.t0 + u.i) * D;
                if (lane < D / 8) *(uint4 *)(p.tail_k + off + lane * 8) = *(const uint4 *)(ks + own_row * (D * 2) + lane * 16);
            }
            __syncwarp();
            if (lane == 0) mbar_arrive(empty_u32 + slot_k * 8);

            // ---------- online softmax over the tile ----------
            float tmax = -CUDART_INF_F;
#pragma unroll
            for (int sub = 0; sub < C::NSUB; ++sub)
#pragma unroll
                for (int k = 0; k < C::NF; ++k) tmax = fmaxf(tmax, sc[sub][k]);
#pragma unroll
            for (int off = 1; off < C::LPH; off <<= 1) tmax = fmaxf(tmax, __shfl_xor_sync(0xffffffffu, tmax, off));
#pragma unroll
            for (int off = C::LPR; off < 32; off <<= 1) tmax = fmaxf(tmax, __shfl_xor_sync(0xffffffffu, tmax, off));
            const float m_new = fmaxf(m_run, tmax);  // finite: the work item has at least one valid row
            const float alpha = fast_exp2(m_run - m_new);
            float psum = 0.f;
#pragma unroll
            for (int sub = 0; sub < C::NSUB; ++sub)
#pragma unroll
                for (int k = 0; k < C::NF; ++k) {
                    const float pv = fast_exp2(sc[sub][k] - m_new);
                    psum += pv;
                    const int r = (jl % C::LPH) * C::NF + k;
                    const int row = (sub * C::SUBR + r) * C::RG + grp;
                    *(float2 *)(ps + (row * G + my_h) * 2) = make_float2(pv, pv);
                }
            l_run = l_run * alpha + psum;
            m_run = m_new;
            alpha_s[my_h] = alpha;
            const bool rescale = __any_sync(0xffffffffu, alpha != 1.0f);
            __syncwarp();

            // ---------- weighted sum of V ----------
            if (rescale) {
#pragma unroll
                for (int h = 0; h < G; ++h) {
                    const float a = alpha_s[h];
                    const float2 a2 = make_float2(a, a);
#pragma unroll
                    for (int d = 0; d < C::NPAIR; ++d) of[h][d] = fmul2(of[h][d], a2);
                }
            }
            slot_wait(tags + slot_v, seq_v / C::NSLOT, full_u32 + slot_v * 8, (seq_v / C::NSLOT) & 1, flags);
#pragma unroll
            for (int r = 0; r < C::RPG; ++r) {
                const int row = r * C::RG + grp;
                if (row < rows) {
                    float2 vf[C::NPAIR];
#pragma unroll
                    for (int v = 0; v < C::NV; ++v) {
                        const uint4 w = *(const uint4 *)(vs + row * (D * 2) + (v * C::LPR + jl) * 16);
                        vf[v * 4 + 0] = bf2(w.x); vf[v * 4 + 1] = bf2(w.y);
                        vf[v * 4 + 2] = bf2(w.z); vf[v * 4 + 3] = bf2(w.w);
                    }
                    float2 pr[G];
                    if constexpr (G % 2 == 0) {
#pragma unroll
                        for (int h2 = 0; h2 < G / 2; ++h2) {
                            const float4 t4 = *(const float4 *)(ps + (row * G + h2 * 2) * 2);
                            pr[h2 * 2 + 0] = make_float2(t4.x, t4.y);
                            pr[h2 * 2 + 1] = make_float2(t4.z, t4.w);
                        }
                    } else {
                        pr[0] = *(const float2 *)(ps + row * 2);
                    }
#pragma unroll
                    for (int h = 0; h < G; ++h)
#pragma unroll
                        for (int d = 0; d < C::NPAIR; ++d) of[h][d] = ffma2(pr[h], vf[d], of[h][d]);
                }
            }
            if (own_row >= 0 && u.t0 + u.i < p.max_tail) {
                const int64_t off = ((((int64_t)u.b * p.n_layers_total + layer) * p.Hkv + u.g) * p.max_tail + u.t0 + u.i) * D;
                if (lane < D / 8) *(uint4 *)(p.tail_v + off + lane * 8) = *(const uint4 *)(vs + own_row * (D * 2) + lane * 16);
            }
            __syncwarp();
            if (lane == 0) mbar_arrive(empty_u32 + slot_v * 8);
        }

        // ---- end of this CTA's share of the unit: merge the warps' states ----
        {
            float l_tot = l_run;
#pragma unroll
            for (int off = 1; off < C::LPH; off <<= 1) l_tot += __shfl_xor_sync(0xffffffffu, l_tot, off);
#pragma unroll
            for (int off = C::LPR; off < 32; off <<= 1) l_tot += __shfl_xor_sync(0xffffffffu, l_tot, off);
#pragma unroll
            for (int h = 0; h < G; ++h)
#pragma unroll
                for (int d = 0; d < C::NPAIR; ++d) {
                    float2 x = of[h][d];
#pragma unroll
                    for (int off = C::LPR; off < 32; off <<= 1) {
                        x.x += __shfl_xor_sync(0xffffffffu, x.x, off);
                        x.y += __shfl_xor_sync(0xffffffffu, x.y, off);
                    }
                    of[h][d] = x;
                }
            if (grp == 0) {
#pragma unroll
                for (int h = 0; h < G; ++h)
#pragma unroll
                    for (int v = 0; v < C::NV; ++v)
#pragma unroll
                        for (int e = 0; e < 4; ++e)
                            *(float2 *)(merge_o + (warp * G + h) * D + (v * C::LPR + jl) * 8 + 2 * e) = of[h][v * 4 + e];
                if (jl % C::LPH == 0) {
                    merge_m[warp * G + my_h] = m_run;
                    merge_l[warp * G + my_h] = l_tot;
                }
            }
        }
        consumer_bar<C::CW>();
        const int64_t unit_index = (((int64_t)u.l_rel * p.B + u.b) * p.S + u.i) * p.Hkv + u.g;
        const int c_first = cta_of(u.flat_begin, W, gridDim.x);
        const int c_last = cta_of(u.flat_begin + u.rt - 1, W, gridDim.x);
        const int n_parts = c_last - c_first + 1;
        const int64_t io_off = (int64_t)u.l_rel * p.q_sl + (int64_t)u.b * p.q_sb + (int64_t)u.i * p.q_ss + (int64_t)u.g * G * D;
        const int64_t lse_off = (int64_t)u.l_rel * p.lse_sl + (int64_t)u.b * p.lse_sb + (int64_t)u.i * p.lse_ss + (int64_t)u.g * G;
        const int64_t slot = unit_index + blockIdx.x;
        const bool slot_ok = slot < p.n_part_slots && unit_index < p.n_counter_slots;
        if (n_parts > 1 && !slot_ok && tid == 0) atomicCAS(p.status, 0, MATKV_E_BOUNDS);
        for (int idx = tid; idx < G * D; idx += C::CW * 32) {
            const int h = idx / D, d = idx % D;
            float M = -CUDART_INF_F;
#pragma unroll
            for (int w = 0; w < C::CW; ++w) M = fmaxf(M, merge_m[w * G + h]);
            float acc = 0.f, L = 0.f;
#pragma unroll
            for (int w = 0; w < C::CW; ++w) {
                const float sw = fast_exp2(merge_m[w * G + h] - M);
                acc = fmaf(sw, merge_o[(w * G + h) * D + d], acc);
                L = fmaf(sw, merge_l[w * G + h], L);
            }
            const float o = acc / L;
            const float lse = (M + log2f(L)) * kLn2;
            if (n_parts == 1) {
                p.out[io_off + h * D + d] = __float2bfloat16(o);
                if (p.lse_out && d == 0) p.lse_out[lse_off + h] = lse;
            } else if (slot_ok) {
                p.part_o[(slot * G + h) * D + d] = o;
                if (d == 0) p.part_lse[slot * G + h] = lse;
            }
        }
        if (n_parts > 1 && slot_ok) {
            __threadfence();
            consumer_bar<C::CW>();
            if (tid == 0) {
                const int old = atomicAdd(p.counters + unit_index, 1);
                const int last = (old == n_parts - 1);
                if (last) p.counters[unit_index] = 0;  // ready for the next launch
                flags[1] = last;
            }
            consumer_bar<C::CW>();
            if (flags[1]) {
                __threadfence();
                const int64_t first_slot = unit_index + c_first;
                for (int h = warp; h < G; h += C::CW)
                    combine_warp(p.part_o + (first_slot * G + h) * D, (int64_t)G * D, p.part_lse + first_slot * G + h, G,
                                 n_parts, D, p.out + io_off + h * D, p.lse_out ? p.lse_out + lse_off + h : nullptr);
            }
        }
        consumer_bar<C::CW>();  // merge area and flags are free again

        j_base += t_end - t_begin;
        f_unit = u.flat_begin + t_end;
        if (f_unit < f_end) next_unit(p, u);
    }
    if (flags[0] && tid == 0) atomicCAS(p.status, 0, MATKV_E_TIMEOUT);
}

// ---- launchers --------------------------------------------------------------------------------------
template <int D, int G>
static int launch_stream_t(const StreamParams &p, int grid, cudaStream_t stream) {
    using C = StreamCfg<D, G>;
    static bool configured = false;
    if (!configured) {
        MATKV_CUDA(cudaFuncSetAttribute(k_attend_stream<D, G>, cudaFuncAttributeMaxDynamicSharedMemorySize, C::SMEM_BYTES));
        configured = true;
    }
    k_attend_stream<D, G><<<grid, C::THREADS, C::SMEM_BYTES, stream>>>(p);
    MATKV_CUDA(cudaGetLastError());
    return MATKV_OK;
}

int launch_attend_stream(matkv_ctx *ctx, matkv_table *t, const AttendArgs &a, cudaStream_t stream) {
    const matkv_config &c = ctx->cfg;
    WorkspaceView ws;
    workspace_bytes_for(c, &ws, ctx->workspace);
    StreamParams p;
    p.segs = t->d_segs;
    p.reqs = t->d_reqs;
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
    const int64_t n_units = (int64_t)a.n_layers_launch * t->batch * a.S * c.n_kv_heads;
    if (n_units > ws.n_counter_slots)
        return fail(MATKV_E_CAPACITY, "launch of %lld units exceeds the workspace's %lld", (long long)n_units,
                    (long long)ws.n_counter_slots);
    // tiles in the launch as far as the host knows (the device recomputes it from its own tail length)
    int64_t W = 0;
    for (int b = 0; b < t->batch; ++b) {
        const int base = t->h_reqs[b].chunk_tiles + ceil_div(t->tail_len_host, kTile);
        W += (int64_t)c.n_kv_heads * ((int64_t)a.S * base + new_tiles_sum(a.S));
    }
    W *= a.n_layers_launch;
    int64_t grid = ctx->opt_decode_ctas > 0 ? ctx->opt_decode_ctas : ctx->n_sm;
    grid = std::max<int64_t>(1, std::min<int64_t>(grid, W));
    const int G = c.n_q_heads / c.n_kv_heads;
#define MATKV_CASE(DD, GG) \
    if (c.head_dim == DD && G == GG) return launch_stream_t<DD, GG>(p, (int)grid, stream);
    MATKV_CASE(128, 1) MATKV_CASE(128, 2) MATKV_CASE(128, 4) MATKV_CASE(128, 8)
    MATKV_CASE(64, 1) MATKV_CASE(64, 2) MATKV_CASE(64, 4) MATKV_CASE(64, 8)
#undef MATKV_CASE
    return fail(MATKV_E_INVALID_ARG, "unsupported head_dim %d / group %d", c.head_dim, G);
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
