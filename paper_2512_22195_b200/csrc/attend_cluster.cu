// K1c: the decode step of ONE layer for small batches, as thread-block clusters.
//
// One layer of a small batch is a few megabytes of K,V (21.5 MB for one request over five 1,024-token chunks at the
// Llama-3-8B head shape): 3.3 us of HBM streaming, so the launch is a chain of latencies, not a stream, and every
// link of the chain is shortened here:
//   - a unit (request, KV head) is served by a CLUSTER of CS CTAs; the unit's KV tiles are cut into CS contiguous
//     shares by a rule that needs nothing but launch parameters (the request's chunk tile count and a nominal tail
//     tile count for balance), so a CTA knows its first chunk tile at once: no dependent walk of the table;
//   - the table carries a directory with one 16-byte record per chunk tile (descriptor, first row, chunk length, valid
//     rows): the producer thread reads its records with independent loads and issues the TMA copies of its first
//     chunk tiles BEFORE the kernel waits for its predecessor on the stream (chunk rows are immutable), i.e. under
//     the previous layer's tail, also when the launch is replayed from a CUDA graph;
//   - tail tiles and the step's new token follow the wait; their placement uses the device's tail length, so a
//     replayed launch stays correct while the tail grows (only the balance drifts);
//   - eight consumer warps: four take one 16-token piece each of the even tiles, four of the odd tiles.  The products
//     are formed transposed, S^T = K Q^T and O^T += V^T P^T (m16n8k16 bf16 MMAs: tokens, then head dimensions, on
//     the 16-row axis, the unit's up to 8 query rows on the 8-column axis), so no tensor-core row is padding, the
//     accumulators take 32 registers and a piece costs 16 MMAs; P^T reaches the second product's operand layout
//     through movmatrix (an 8 x 8 transpose across the warp); fp32 online softmax per query row; the warps' states
//     are merged through shared memory at the end;
//   - the CTAs' partials (o, lse) are exchanged through distributed shared memory as a reduce-scatter: CTA i of the
//     cluster owns the output column groups (of four) i, i + CS, ..., every CTA stores those groups of its partial straight into CTA i's
//     shared memory (st.shared::cluster) and each storing thread announces its unit on an mbarrier there (remote arrive,
//     release at cluster scope); every CTA then merges its own slice over the CS parts by log-sum-exp and writes those columns of the
//     output.  No global partials, no device-wide fence, no atomic ticket, no workspace, and the landing zone of a
//     CTA is a few kilobytes.
// A CTA needs ~100 KB of shared memory (a ring of three 32 KB tiles) and few registers, so two launches' CTAs fit an SM
// side by side: with programmatic dependent launch the next layer's CTAs start and pull their first three chunk
// tiles while this layer's CTAs are still exchanging and merging.
// All waits are bounded; a CTA that gave up still announces itself, so that nobody waits for it.
#include <stdio.h>

#include <algorithm>

#include "stream_common.cuh"

namespace matkv {

constexpr int kClMaxReq = 64;      // requests per launch the parameter block has room for
constexpr int kClWarps = 8;        // consumer warps: warp w takes tokens [16 (w & 3), 16 (w & 3) + 16) of the tiles of parity w >> 2
constexpr int kClThreads = (kClWarps + 1) * 32;
constexpr int kClStages = 3;
constexpr int kClMaxCs = 16;       // largest cluster (non-portable size; the launcher asks the occupancy API before using it)

struct ClusterParams {
    const int4 *tile_dir;       // one record per chunk tile of every request: {descriptor index, first row, chunk tokens, valid rows}
    const CUtensorMap *tmaps;   // [n_seg_total] chunk maps, then tail K, tail V
    int32_t n_seg_total;
    const int32_t *tail_len;
    __nv_bfloat16 *tail_k, *tail_v;
    const __nv_bfloat16 *q;
    __nv_bfloat16 *out;
    float *lse_out;
    int64_t q_sb, lse_sb;
    int32_t layer, n_layers_total, B, Hkv, max_tail;
    int32_t cs;                 // cluster size = CTAs per unit
    int32_t tt_nom;             // nominal tail tile count the shares are balanced for (the host's view at launch time)
    float scale_log2;
    int32_t *status;
    int32_t stream_hint;        // 1: no chunk is listed twice, load chunk tiles with the evict-first L2 policy
    int32_t chunk_tiles[kClMaxReq];
    int32_t dir_begin[kClMaxReq];
};

// the wait for the predecessor kernel on the stream (a profiling build can leave it out to see the launch without its dependency)
#ifdef MATKV_EXP_NODEP
#define CL_GDC_WAIT()
#else
#define CL_GDC_WAIT() asm volatile("griddepcontrol.wait;" ::: "memory")
#endif

#ifdef MATKV_STAMPS
// Timeline stamps of a profiling build (never compiled into the library proper): [layer][CTA][point], nanoseconds.
__device__ unsigned long long g_cl_stamps[64][160][16];
__device__ long long g_cl_clk[64][160][16];   // the same points in SM clock cycles (finer than the global timer)
__device__ __forceinline__ void cl_stamp(int layer, int point) {
#ifdef MATKV_STAMPS_CLOCK_ONLY   // reading the global timer costs hundreds of cycles: leave it out when phases are measured in cycles
    if (layer < 64 && blockIdx.x < 160) g_cl_clk[layer][blockIdx.x][point] = clock64();
#else
    unsigned long long t;
    asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
    if (layer < 64 && blockIdx.x < 160) {
        g_cl_stamps[layer][blockIdx.x][point] = t;
        g_cl_clk[layer][blockIdx.x][point] = clock64();
    }
#endif
}
#define CL_STAMP(point) cl_stamp(p.layer, point)
// per-tile stamps: [layer][CTA][kind: 0 issued, 1 seen landed, 2 consumed][tile]
__device__ unsigned long long g_cl_tiles[64][160][3][8];
__device__ __forceinline__ void cl_tile_stamp(int layer, int kind, int tile) {
#ifdef MATKV_STAMPS_CLOCK_ONLY
    return;
#endif
    unsigned long long t;
    asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
    if (layer < 64 && blockIdx.x < 160 && tile < 8) g_cl_tiles[layer][blockIdx.x][kind][tile] = t;
}
#define CL_TILE(kind, tile) cl_tile_stamp(p.layer, kind, tile)
#else
#define CL_STAMP(point)
#define CL_TILE(kind, tile)
#endif

// ---- cluster / distributed shared memory helpers ---------------------------------------------------
__device__ __forceinline__ uint32_t cluster_ctarank() {
    uint32_t r;
    asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
    return r;
}
__device__ __forceinline__ void cluster_arrive_release() { asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory"); }
__device__ __forceinline__ void cluster_wait_acquire() { asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory"); }
// address of `local` (a shared::cta address of this CTA) in the shared memory of CTA `rank` of the cluster
__device__ __forceinline__ uint32_t map_to_rank(uint32_t local, uint32_t rank) {
    uint32_t a;
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(a) : "r"(local), "r"(rank));
    return a;
}
__device__ __forceinline__ void st_cluster_f4(uint32_t addr, float4 v) {
    asm volatile("st.shared::cluster.v4.f32 [%0], {%1, %2, %3, %4};" ::"r"(addr), "f"(v.x), "f"(v.y), "f"(v.z), "f"(v.w) : "memory");
}
__device__ __forceinline__ void st_cluster_f1(uint32_t addr, float v) {
    asm volatile("st.shared::cluster.f32 [%0], %1;" ::"r"(addr), "f"(v) : "memory");
}
__device__ __forceinline__ void mbar_arrive_remote_release(uint32_t cluster_addr) {
    asm volatile("mbarrier.arrive.release.cluster.shared::cluster.b64 _, [%0];" ::"r"(cluster_addr) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait_acquire_cluster(uint32_t bar, uint32_t parity) {
    uint32_t ok;
    asm volatile(
        "{\n .reg .pred p;\n mbarrier.try_wait.parity.acquire.cluster.shared::cta.b64 p, [%1], %2;\n selp.u32 %0, 1, 0, p;\n}"
        : "=r"(ok)
        : "r"(bar), "r"(parity)
        : "memory");
    return ok != 0;
}

// The share of CTA `rank` of a unit: chunk tiles [c0, c0 + n_chunk), tail tiles [j0, j0 + n_tail) and, for the last
// CTA, the tile of the step's new token.  The cut follows the nominal list (chunk tiles, tt_nom tail tiles, the new
// token), so the chunk part depends on launch parameters only; tail tiles beyond the nominal count go to the last CTA.
struct ClShare {
    int32_t c0, n_chunk, j0, n_tail, has_new;
};
__device__ __forceinline__ ClShare cl_share(int32_t ct, int32_t tt_nom, int32_t cs, int32_t rank, int32_t tt_real) {
    const int32_t total = ct + tt_nom + 1;
    const int32_t lo = rank * total / cs, hi = (rank + 1) * total / cs;   // (a request lists at most 2^20 chunk tiles here)
    ClShare s;
    s.c0 = min(lo, ct);
    s.n_chunk = min(hi, ct) - s.c0;
    const bool last = rank == cs - 1;
    const int32_t a = max(lo, ct) - ct;                       // nominal slots [a, b): slot < tt_nom is tail tile `slot`
    const int32_t b = last ? max(tt_nom, tt_real) : max(hi, ct) - ct;
    s.j0 = min(a, tt_real);
    s.n_tail = max(0, min(b, tt_real) - s.j0);
    s.has_new = last ? 1 : 0;
    return s;
}

template <int D, int G>
struct ClusterCfg {
    static constexpr int NBOX = D / 64;
    static constexpr int BOX_BYTES = kTile * 128;
    static constexpr int STAGE_BYTES = 2 * NBOX * BOX_BYTES;      // K boxes then V boxes of one 64-token tile
    static constexpr int KS = D / 16;
    static constexpr int RING_BYTES = kClStages * STAGE_BYTES;
    // the warps' states at the end of the CTA's share sit in the ring (all of its tiles have been consumed by then)
    static constexpr int MROW = D + 4;                            // padded row of the merge area (bank spread)
    static constexpr int MERGE_BYTES = kClWarps * kUnitRows * (MROW + 3) * 4;
    // landing zone: this CTA's column groups of every CTA's partial ([part][row][ceil(D / 4 / CS)] groups of four floats: at
    // most rows x (D / 4 + CS) groups whatever CS is), then every CTA's lse per row
    static constexpr int LAND_O_FLOATS = kUnitRows * (D / 4 + kClMaxCs) * 4;
    static constexpr int LAND_BYTES = (LAND_O_FLOATS + kClMaxCs * kUnitRows) * 4;
    static constexpr int MISC_BYTES = 256;
    static constexpr int SMEM_BYTES = 1024 + RING_BYTES + LAND_BYTES + MISC_BYTES;
    static_assert(MERGE_BYTES <= RING_BYTES, "merge area must fit the ring");
    static_assert(G >= 1 && G <= kUnitRows, "unsupported group size");
};

template <int D, int G>
__global__ void __launch_bounds__(kClThreads, 2)
k_decode_cluster(const __grid_constant__ ClusterParams p, const __grid_constant__ CUtensorMap kn_map, const __grid_constant__ CUtensorMap vn_map) {
    using C = ClusterCfg<D, G>;
    extern __shared__ unsigned char smem_raw[];
    unsigned char *smem = (unsigned char *)(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);   // the same offset in every CTA of the cluster
    unsigned char *ring = smem;
    float *land_o = (float *)(smem + C::RING_BYTES);                // [part][row][ceil(D / 4 / cs)][4]: this CTA's column groups of every partial
    float *land_lse = land_o + C::LAND_O_FLOATS;                    // [part][row]
    unsigned char *misc = smem + C::RING_BYTES + C::LAND_BYTES;
    uint64_t *bars = (uint64_t *)misc;                              // full[stages], empty[stages], landing
    volatile uint32_t *tags = (volatile uint32_t *)(misc + 64);     // per stage: valid rows | kTagNew | (number of the stage's current fill) << 16
    volatile int *flags = (volatile int *)(misc + 96);              // [0] abort
    float *merge_o = (float *)ring;                                 // [warp][row][MROW]   (after the last tile)
    float *merge_m = merge_o + kClWarps * kUnitRows * C::MROW;      // [warp][row]
    float *merge_l = merge_m + kClWarps * kUnitRows;
    float *merge_r = merge_l + kClWarps * kUnitRows;

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");   // the next launch may be set up beside this one
    const int cs = p.cs;
    const int rank = cs > 1 ? (int)cluster_ctarank() : 0;
    const int unit = blockIdx.x / cs;
    const int b = unit / p.Hkv, g = unit % p.Hkv;
    const uint32_t full_u32 = smem_u32(bars), empty_u32 = smem_u32(bars + kClStages), land_u32 = smem_u32(bars + 2 * kClStages);
    const uint32_t ring_u32 = smem_u32(ring);
    if (tid == 0) {
        CL_STAMP(0);
        for (int s = 0; s < kClStages; ++s) {
            mbar_init(full_u32 + s * 8, 1);
            mbar_init(empty_u32 + s * 8, 4);   // the four warps that share a tile
            tags[s] = 0xffff0000u;
        }
        // the landing barrier counts one arrival per (row, column group) unit this CTA owns from every CTA of the cluster
        // (its own included): every thread that stores a unit announces it itself, no CTA-wide step in between
        mbar_init(land_u32, cs > 1 ? cs * G * ((D / 4 - rank + cs - 1) / cs) : 1);
        flags[0] = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    __syncthreads();
    // every CTA of the cluster has to be running, its barriers initialised, before anybody writes into a neighbour's shared
    // memory: arrive now, wait only right before the first remote access (a few microseconds from here)
    if (cs > 1) cluster_arrive_release();

    const int32_t ct = p.chunk_tiles[b];
    const int n_rows = G;   // one new token per request: the G heads of the KV group

    if (warp == kClWarps) {
        // ================= producer =================
        if (lane == 0) {
            const uint64_t pol = p.stream_hint ? l2_policy_evict_first() : l2_policy_evict_normal();
            // chunk part of the share: known from the launch parameters alone
            const ClShare s0 = cl_share(ct, p.tt_nom, cs, rank, 0);
            const int4 *dir = p.tile_dir + p.dir_begin[b] + s0.c0;
            int4 ahead[4];
#pragma unroll
            for (int i = 0; i < 4; ++i) ahead[i] = i < s0.n_chunk ? __ldg(dir + i) : make_int4(0, 0, 0, 0);
            uint32_t seq = 0;
            bool ok = true;
            // a stage's tag carries the number of its fill: the two groups of consumer warps reach a stage at different
            // times, and the one-bit phase of an mbarrier cannot tell "the previous fill has not landed yet" from "this
            // fill has landed" (see stage_wait)
            uint32_t fill = 0;
            auto acquire = [&](uint32_t &stage, uint32_t &bar, uint32_t &dst) {
                stage = seq % kClStages;
                const uint32_t use = seq / kClStages;
                fill = use << 16;
                if (use > 0 && !mbar_wait(empty_u32 + stage * 8, (use - 1) & 1, flags)) return false;
                bar = full_u32 + stage * 8;
                dst = ring_u32 + stage * C::STAGE_BYTES;
                return true;
            };
            for (int j = 0; j < s0.n_chunk && ok; ++j, ++seq) {
                const int4 e = ahead[j & 3];
                if (j + 4 < s0.n_chunk) ahead[j & 3] = __ldg(dir + j + 4);
                uint32_t stage, bar, dst;
                if (!(ok = acquire(stage, bar, dst))) break;
                const CUtensorMap *m = p.tmaps + e.x;   // e: descriptor index, first row inside the chunk, chunk tokens, valid rows
                const int32_t yk = ((p.layer * 2) * p.Hkv + g) * e.z + e.y, yv = ((p.layer * 2 + 1) * p.Hkv + g) * e.z + e.y;
                tags[stage] = (uint32_t)e.w | fill;
                mbar_expect_tx(bar, C::STAGE_BYTES);
#pragma unroll
                for (int bx = 0; bx < C::NBOX; ++bx) {
                    tma_load_2d_hint(dst + bx * C::BOX_BYTES, m, bx * 64, yk, bar, pol);
                    tma_load_2d_hint(dst + (C::NBOX + bx) * C::BOX_BYTES, m, bx * 64, yv, bar, pol);
                }
                if (j == 0) CL_STAMP(1);
                CL_TILE(0, j);
            }
            // tail rows and the step's new token were written by earlier kernels on the stream
            CL_GDC_WAIT();
            CL_STAMP(2);
            if (ok) {
                int32_t t0 = p.tail_len[b];
                if (t0 < 0 || t0 + 1 > p.max_tail) t0 = max(0, min(t0, p.max_tail - 1));   // reported by the consumers
                const ClShare s = cl_share(ct, p.tt_nom, cs, rank, ceil_div(t0, kTile));
                const CUtensorMap *mk = p.tmaps + p.n_seg_total, *mv = mk + 1;
                const uint64_t pol_n = l2_policy_evict_normal();
                for (int j = 0; j < s.n_tail && ok; ++j, ++seq) {
                    uint32_t stage, bar, dst;
                    if (!(ok = acquire(stage, bar, dst))) break;
                    const int r0 = (s.j0 + j) * kTile;
                    const int32_t y = ((b * p.n_layers_total + p.layer) * p.Hkv + g) * p.max_tail + r0;
                    tags[stage] = (uint32_t)min(kTile, t0 - r0) | fill;
                    mbar_expect_tx(bar, C::STAGE_BYTES);
#pragma unroll
                    for (int bx = 0; bx < C::NBOX; ++bx) {
                        tma_load_2d_hint(dst + bx * C::BOX_BYTES, mk, bx * 64, y, bar, pol_n);
                        tma_load_2d_hint(dst + (C::NBOX + bx) * C::BOX_BYTES, mv, bx * 64, y, bar, pol_n);
                    }
                    CL_TILE(0, (int)seq);
                }
                if (s.has_new && ok) {
                    uint32_t stage, bar, dst;
                    if ((ok = acquire(stage, bar, dst))) {
                        tags[stage] = 1u | kTagNew | fill;
                        mbar_expect_tx(bar, C::STAGE_BYTES);
#pragma unroll
                        for (int bx = 0; bx < C::NBOX; ++bx) {
                            tma_load_3d(dst + bx * C::BOX_BYTES, &kn_map, bx * 64, g, b, bar);
                            tma_load_3d(dst + (C::NBOX + bx) * C::BOX_BYTES, &vn_map, bx * 64, g, b, bar);
                        }
                        CL_TILE(0, (int)seq);
                        ++seq;
                    }
                }
            }
            if (!ok) {
                // gave up: wait (bounded) for the copies already issued so that none lands after the CTA has gone
                atomicCAS(p.status, 0, MATKV_E_TIMEOUT);
                const uint32_t lo = seq > (uint32_t)kClStages ? seq - kClStages : 0;
                for (uint32_t s2 = lo; s2 < seq; ++s2) {
                    const long long t0c = clock64();
                    while (!mbar_try_wait(full_u32 + (s2 % kClStages) * 8, (s2 / kClStages) & 1) && clock64() - t0c < kWaitCycles) {}
                }
            }
        }
        __syncwarp();
        if (cs > 1) cluster_wait_acquire();   // completes this warp's part of the start-up barrier
        return;
    }

    // ================= consumers =================
    // Fragment coordinates (m16n8k16): as the B operand / accumulator column, this thread's query rows are 2 qc and
    // 2 qc + 1 (accumulator) or tq (B operand of S^T); as accumulator rows it has tokens (or dimensions) tq and tq + 8.
    const int tq = lane >> 2, qc = lane & 3;
    const int mi = lane >> 3, ri = lane & 7;   // ldmatrix addressing
    // Everything that does not depend on the predecessor kernel comes before the wait for it: what follows the wait is
    // the launch's critical path.  The chunk part of the share is known from the launch parameters; how many tail tiles
    // follow depends on the device's tail length, which is requested right after the wait and first looked at when the
    // chunk tiles are done (a dependent load less in front of the first tile).
    int n_mine = cl_share(ct, p.tt_nom, cs, rank, 0).n_chunk;
    bool tail_known = false;
    int32_t t0 = 0;
    const bool real = tq < n_rows;
    const __nv_bfloat16 *qrow = p.q + (int64_t)b * p.q_sb + (int64_t)(g * G + (real ? tq : 0)) * D + 2 * qc;
    const int32_t *tail_len_b = p.tail_len + b;
    CL_GDC_WAIT();   // q, the tail length and the tail rows come from earlier kernels
    if (tid == 0) CL_STAMP(3);
    const int32_t t0_dev = *tail_len_b;

    // Q^T as the B operand of S^T = K Q^T: column n = tq is query row tq, k = the 16 dimensions of a k-step
    uint32_t qb[C::KS][2];
    {
#pragma unroll
        for (int ks = 0; ks < C::KS; ++ks) {
            qb[ks][0] = real ? *(const uint32_t *)(qrow + ks * 16) : 0u;
            qb[ks][1] = real ? *(const uint32_t *)(qrow + ks * 16 + 8) : 0u;
        }
    }
    // O^T accumulators: [16-dimension block][c0: (d = tq, row 2 qc), c1: (tq, 2 qc + 1), c2: (tq + 8, 2 qc), c3: (tq + 8, 2 qc + 1)]
    float o[C::KS][4];
#pragma unroll
    for (int mt = 0; mt < C::KS; ++mt) o[mt][0] = o[mt][1] = o[mt][2] = o[mt][3] = 0.f;
    // per query row (2 qc, 2 qc + 1): running maximum (the same in the lanes that share qc), and THIS thread's share of
    // the sum of the numerators and of their bf16 roundings (its tokens tq and tq + 8 of every piece)
    float m_run[2] = {-CUDART_INF_F, -CUDART_INF_F}, l_run[2] = {0.f, 0.f}, l_rnd[2] = {0.f, 0.f};
    const int r0 = (warp & 3) * kItemRows;   // this warp's 16 tokens of its tiles

    for (int j = warp >> 2;; j += 2) {
        if (j >= n_mine) {
            if (tail_known) break;
            tail_known = true;
            t0 = t0_dev;
            if (t0 < 0 || t0 + 1 > p.max_tail) {
                if (tid == 0) atomicCAS(p.status, 0, MATKV_E_CAPACITY);
                t0 = max(0, min(t0, p.max_tail - 1));
            }
            const ClShare sh = cl_share(ct, p.tt_nom, cs, rank, ceil_div(t0, kTile));
            n_mine = sh.n_chunk + sh.n_tail + sh.has_new;
            if (j >= n_mine) break;
        }
        const uint32_t stage = j % kClStages, use = j / kClStages;
        // (after a bounded wait ran out the loop goes on without computing: every lane of the warp takes the same path)
        const uint32_t tag = __shfl_sync(0xffffffffu, stage_wait(tags + stage, use, full_u32 + stage * 8, use & 1, flags), 0);   // 0: gave up
        if (tid == 0 && j == 0) CL_STAMP(4);
        if (lane == 0 && (warp & 3) == 0) CL_TILE(1, j);
        const uint32_t stage_u32 = ring_u32 + stage * C::STAGE_BYTES;
        const int rows = (int)(tag & 0x7f) - r0;   // valid tokens of this warp's piece (may be <= 0)
        if (rows > 0) {
            // ---------- S^T = K Q^T: 16 tokens x 8 query rows, two accumulation chains ----------
            float sa[4] = {0.f, 0.f, 0.f, 0.f}, sb[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
            for (int ks = 0; ks < C::KS; ++ks) {
                // A = K rows, fragments a0..a3: (tokens 0-7, d-chunk 2ks), (tokens 8-15, 2ks), (tokens 0-7, 2ks+1), (tokens 8-15, 2ks+1)
                uint32_t ka[4];
                ldsm_x4(stage_u32 + (ks / 4) * C::BOX_BYTES + swz(r0 + (mi & 1) * 8 + ri, (ks * 2 + (mi >> 1)) & 7), ka);
                if (ks & 1) mma_bf16(sb, ka[0], ka[1], ka[2], ka[3], qb[ks][0], qb[ks][1]);
                else mma_bf16(sa, ka[0], ka[1], ka[2], ka[3], qb[ks][0], qb[ks][1]);
            }
            // this thread: tokens tq (x0, x1) and tq + 8 (x2, x3) against query rows 2 qc (x0, x2) and 2 qc + 1 (x1, x3)
            const float x0 = tq < rows ? (sa[0] + sb[0]) * p.scale_log2 : -CUDART_INF_F;
            const float x1 = tq < rows ? (sa[1] + sb[1]) * p.scale_log2 : -CUDART_INF_F;
            const float x2 = tq + 8 < rows ? (sa[2] + sb[2]) * p.scale_log2 : -CUDART_INF_F;
            const float x3 = tq + 8 < rows ? (sa[3] + sb[3]) * p.scale_log2 : -CUDART_INF_F;
            float mx0 = fmaxf(x0, x2), mx1 = fmaxf(x1, x3);
#pragma unroll
            for (int off = 4; off < 32; off <<= 1) {   // over the eight token pairs of the piece (lanes with the same qc)
                mx0 = fmaxf(mx0, __shfl_xor_sync(0xffffffffu, mx0, off));
                mx1 = fmaxf(mx1, __shfl_xor_sync(0xffffffffu, mx1, off));
            }
            const float mn0 = fmaxf(m_run[0], mx0), mn1 = fmaxf(m_run[1], mx1);   // finite: token 0 of the piece is valid
            const float al0 = fast_exp2(m_run[0] - mn0), al1 = fast_exp2(m_run[1] - mn1);   // 0 for the first piece
            const float p0 = fast_exp2(x0 - mn0), p1 = fast_exp2(x1 - mn1), p2 = fast_exp2(x2 - mn0), p3 = fast_exp2(x3 - mn1);
            const uint32_t w0 = pack_bf16(p0, p1), w1 = pack_bf16(p2, p3);   // (token tq | tq + 8; rows 2 qc, 2 qc + 1)
            l_run[0] = l_run[0] * al0 + (p0 + p2);
            l_run[1] = l_run[1] * al1 + (p1 + p3);
            l_rnd[0] = l_rnd[0] * al0 + (bf_lo(w0) + bf_lo(w1));
            l_rnd[1] = l_rnd[1] * al1 + (bf_hi(w0) + bf_hi(w1));
            m_run[0] = mn0;
            m_run[1] = mn1;
            if (__any_sync(0xffffffffu, al0 != 1.0f || al1 != 1.0f)) {
#pragma unroll
                for (int mt = 0; mt < C::KS; ++mt) {
                    o[mt][0] *= al0; o[mt][1] *= al1; o[mt][2] *= al0; o[mt][3] *= al1;
                }
            }
            // P^T as the B operand of O^T += V^T P^T: the 8 x 8 blocks (tokens x rows) transposed across the warp
            uint32_t pb0, pb1;
            asm volatile("movmatrix.sync.aligned.m8n8.trans.b16 %0, %1;" : "=r"(pb0) : "r"(w0));
            asm volatile("movmatrix.sync.aligned.m8n8.trans.b16 %0, %1;" : "=r"(pb1) : "r"(w1));
            // ---------- O^T += V^T P^T: 16 dimensions x 8 query rows per block ----------
            const uint32_t v_u32 = stage_u32 + C::NBOX * C::BOX_BYTES;
#pragma unroll
            for (int mt = 0; mt < C::KS; ++mt) {
                // A = V^T: matrices (d-chunk 2mt, tokens 0-7), (2mt+1, tokens 0-7), (2mt, tokens 8-15), (2mt+1, tokens 8-15), transposed on the way
                uint32_t va[4];
                ldsm_x4_trans(v_u32 + (mt / 4) * C::BOX_BYTES + swz(r0 + (mi >> 1) * 8 + ri, (mt * 2 + (mi & 1)) & 7), va);
                mma_bf16(o[mt], va[0], va[1], va[2], va[3], pb0, pb1);
            }
            // the step's new token goes to the tail for later steps (it is row 0 of its tile: the warp of piece 0 has it)
            if ((tag & kTagNew) && t0 < p.max_tail) {
                constexpr int CPR = D / 8;   // 16-byte chunks per row; lanes 0..CPR-1 move K, the next CPR lanes move V
                const unsigned char *ring_stage = ring + stage * C::STAGE_BYTES;
                const int64_t off = ((((int64_t)b * p.n_layers_total + p.layer) * p.Hkv + g) * p.max_tail + t0) * D;
                const int ch = lane % CPR, kv = lane / CPR;
                if (kv < 2) {
                    const uint4 val = *(const uint4 *)(ring_stage + kv * C::NBOX * C::BOX_BYTES + (ch / 8) * C::BOX_BYTES + swz(0, ch % 8));
                    *(uint4 *)((kv ? p.tail_v : p.tail_k) + off + ch * 8) = val;
                }
            }
        }
        __syncwarp();
        if (lane == 0) mbar_arrive(empty_u32 + stage * 8);
        if (lane == 0 && (warp & 3) == 0) CL_TILE(2, j);
    }

    // ---- the warps' states are merged through shared memory (the ring is free: every tile has been consumed) ----
    if (tid == 0) CL_STAMP(5);
    asm volatile("bar.sync 1, %0;" ::"n"(kClWarps * 32) : "memory");
    if (tid == 0) CL_STAMP(6);
    {
#pragma unroll
        for (int h = 0; h < 2; ++h) {   // the row sums over the lanes that share qc
#pragma unroll
            for (int off = 4; off < 32; off <<= 1) {
                l_run[h] += __shfl_xor_sync(0xffffffffu, l_run[h], off);
                l_rnd[h] += __shfl_xor_sync(0xffffffffu, l_rnd[h], off);
            }
        }
#pragma unroll
        for (int h = 0; h < 2; ++h) {
            const int r = 2 * qc + h;
            if (r < n_rows) {   // columns past the unit's G heads are padding of the MMA tile
                float *row = merge_o + (warp * kUnitRows + r) * C::MROW;
#pragma unroll
                for (int mt = 0; mt < C::KS; ++mt) {
                    row[mt * 16 + tq] = o[mt][h];
                    row[mt * 16 + 8 + tq] = o[mt][2 + h];
                }
                if (tq == 0) {
                    merge_m[warp * kUnitRows + r] = m_run[h];
                    merge_l[warp * kUnitRows + r] = l_run[h];
                    merge_r[warp * kUnitRows + r] = l_rnd[h];
                }
            }
        }
    }
    asm volatile("bar.sync 1, %0;" ::"n"(kClWarps * 32) : "memory");
    const bool aborted = flags[0] != 0;
    if (aborted && tid == 0) atomicCAS(p.status, 0, MATKV_E_TIMEOUT);
    if (tid == 0) CL_STAMP(10);
    if (cs > 1) cluster_wait_acquire();
   // the start-up barrier: every neighbour's landing zone and barrier exist from here on
    if (tid == 0) CL_STAMP(11);
    // one (row, group of four columns) unit per thread and pass; column group q belongs to CTA q mod cs of the cluster (any
    // cluster size works), which keeps it as group q / cs of its landing zone
    const int ngm = ceil_div(D / 4, cs);   // groups a CTA owns at most
    const uint32_t land_o_u32 = smem_u32(land_o), land_lse_u32 = smem_u32(land_lse);
    for (int idx = tid; idx < n_rows * (D / 4); idx += kClWarps * 32) {
        const int r = idx / (D / 4), d = (idx % (D / 4)) * 4;
        float M = -CUDART_INF_F;
#pragma unroll
        for (int w = 0; w < kClWarps; ++w) M = fmaxf(M, merge_m[w * kUnitRows + r]);
        float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
        float L = 0.f, Lr = 0.f;
#pragma unroll
        for (int w = 0; w < kClWarps; ++w) {
            const float mw = merge_m[w * kUnitRows + r];
            const float wgt = mw == -CUDART_INF_F ? 0.f : fast_exp2(mw - M);
            const float4 v = *(const float4 *)(merge_o + (w * kUnitRows + r) * C::MROW + d);
            acc.x = fmaf(wgt, v.x, acc.x); acc.y = fmaf(wgt, v.y, acc.y); acc.z = fmaf(wgt, v.z, acc.z); acc.w = fmaf(wgt, v.w, acc.w);
            L = fmaf(wgt, merge_l[w * kUnitRows + r], L);
            Lr = fmaf(wgt, merge_r[w * kUnitRows + r], Lr);
        }
        const float inv = Lr > 0.f ? 1.f / Lr : 0.f;   // a share without tiles is an empty part
        acc.x *= inv; acc.y *= inv; acc.z *= inv; acc.w *= inv;
        const float lse = L > 0.f ? (M + log2f(L)) * kLn2 : -CUDART_INF_F;
        if (cs == 1) {
            *(uint2 *)(p.out + (int64_t)b * p.q_sb + (int64_t)(g * G + r) * D + d) = make_uint2(pack_bf16(acc.x, acc.y), pack_bf16(acc.z, acc.w));
            if (p.lse_out && d == 0) p.lse_out[(int64_t)b * p.lse_sb + g * G + r] = lse;
            continue;
        }
        // these four columns belong to CTA `dst`: into part `rank` of its landing zone (its own groups stay local)
        const int dst = (d / 4) % cs;
        const uint32_t off = (uint32_t)(((rank * n_rows + r) * ngm + (d / 4) / cs) * 16);
        // (the unit's row lse travels with it: the owner gets it once per unit of that row, always the same value).  Then the
        // unit is announced on the owner's landing barrier, after a timeout too (nobody must wait for this CTA): the release
        // orders this thread's stores before the arrival, which is all the owner's acquire needs.
        if (!aborted) {
            st_cluster_f4(map_to_rank(land_o_u32, dst) + off, acc);   // (the own rank maps to this CTA's own memory)
            st_cluster_f1(map_to_rank(land_lse_u32, dst) + (uint32_t)((rank * n_rows + r) * 4), lse);
        }
        mbar_arrive_remote_release(map_to_rank(land_u32, dst));
    }
    if (cs == 1) return;
    if (tid == 0) CL_STAMP(7);
    // ---- this CTA's columns: merge over the CS parts by log-sum-exp ----
    // every thread that takes part in the merge waits for all parts itself (bounded)
    const int ng = (D / 4 - rank + cs - 1) / cs;   // column groups this CTA owns: rank, rank + cs, ...
    const int n_items = n_rows * ng;               // (row, group of four columns) units; TP threads share one: each takes every
    const int tp = cs >= 4 ? 4 : 2;                // TP-th part, then the TP partial sums meet by shuffle (few threads, short chains)
    if (tid < 32 * ceil_div(n_items * tp, 32)) {   // whole warps, for the shuffles
        bool got = mbar_try_wait_acquire_cluster(land_u32, 0);
        const long long tw = clock64();
        while (!got) {
            got = mbar_try_wait_acquire_cluster(land_u32, 0);
            if (!got && clock64() - tw > 2 * kWaitCycles) break;
        }
        if (tid == 0) CL_STAMP(8);
        got = __all_sync(0xffffffffu, got);
        if (!got) {
            if (tid == 0) atomicCAS(p.status, 0, MATKV_E_TIMEOUT);
        } else {
            const int item = tid / tp, sub = tid % tp;
            const bool valid = item < n_items;
            const int r = valid ? item / ng : 0, li = valid ? item % ng : 0;
            // the row's maximum over all parts (independent loads), then this thread's parts with their weights exp(lse_part - max)
            float M = -CUDART_INF_F;
#pragma unroll
            for (int c = 0; c < kClMaxCs; ++c)
                if (c < cs) M = fmaxf(M, land_lse[c * n_rows + r]);
            if (tid == 0) CL_STAMP(12);
            float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
            float Z = 0.f;
#pragma unroll
            for (int k = 0; k < kClMaxCs / 2; ++k) {
                const int c = sub + k * tp;
                if (c < cs) {
                    const float lc = land_lse[c * n_rows + r];
                    if (lc != -CUDART_INF_F) {   // an empty part carries no weight, whatever its row holds
                        const float wgt = fast_exp2((lc - M) * kLog2e);
                        const float4 v = *(const float4 *)(land_o + ((c * n_rows + r) * ngm + li) * 4);
                        acc.x = fmaf(wgt, v.x, acc.x); acc.y = fmaf(wgt, v.y, acc.y); acc.z = fmaf(wgt, v.z, acc.z); acc.w = fmaf(wgt, v.w, acc.w);
                        Z += wgt;
                    }
                }
            }
            for (int off = 1; off < tp; off <<= 1) {
                acc.x += __shfl_xor_sync(0xffffffffu, acc.x, off); acc.y += __shfl_xor_sync(0xffffffffu, acc.y, off);
                acc.z += __shfl_xor_sync(0xffffffffu, acc.z, off); acc.w += __shfl_xor_sync(0xffffffffu, acc.w, off);
                Z += __shfl_xor_sync(0xffffffffu, Z, off);
            }
            if (tid == 0) CL_STAMP(13);
            if (valid && sub == 0) {
                const float inv = Z > 0.f ? __frcp_rn(Z) : 0.f;
                const int d = (li * cs + rank) * 4;
                *(uint2 *)(p.out + (int64_t)b * p.q_sb + (int64_t)(g * G + r) * D + d) =
                    make_uint2(pack_bf16(acc.x * inv, acc.y * inv), pack_bf16(acc.z * inv, acc.w * inv));
                if (li == 0 && rank == 0 && p.lse_out) p.lse_out[(int64_t)b * p.lse_sb + g * G + r] = Z > 0.f ? M + logf(Z) : -CUDART_INF_F;
            }
        }
    }
    if (tid == 0) CL_STAMP(9);
}

// ---- launcher ---------------------------------------------------------------------------------------
// How many clusters of `cs` CTAs of this kernel the device can hold at once (asked once per size and device; -1: cannot say).
template <int D, int G>
static int max_active_clusters(int cs) {
    using C = ClusterCfg<D, G>;
    static std::atomic<int> cache[64][kClMaxCs + 1] = {};
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return -1;
    int known = cache[dev][cs].load(std::memory_order_acquire);
    if (known == 0) {
        cudaLaunchConfig_t cfg = {};
        cfg.gridDim = dim3((unsigned)cs);
        cfg.blockDim = dim3((unsigned)kClThreads);
        cfg.dynamicSmemBytes = C::SMEM_BYTES;
        cudaLaunchAttribute attr[1];
        attr[0].id = cudaLaunchAttributeClusterDimension;
        attr[0].val.clusterDim.x = (unsigned)cs;
        attr[0].val.clusterDim.y = 1;
        attr[0].val.clusterDim.z = 1;
        cfg.attrs = attr;
        cfg.numAttrs = 1;
        int n = 0;
        if (cudaOccupancyMaxActiveClusters(&n, k_decode_cluster<D, G>, &cfg) != cudaSuccess) {
            cudaGetLastError();
            n = -1;
        }
        known = n > 0 ? n : -1;
        cache[dev][cs].store(known, std::memory_order_release);
#ifdef MATKV_STAMPS
        fprintf(stderr, "[cluster decode] cluster size %d: %d clusters can be active at once, %d bytes of shared memory per CTA\n", cs, n, C::SMEM_BYTES);
#endif
    }
    return known;
}

// Picks the cluster size (the largest up to cs_max whose clusters can all be resident at once and whose CTAs stay within
// `cta_limit`), and launches; *fits = false when no size will do.
template <int D, int G>
static int launch_cluster_t(ClusterParams p, const CUtensorMap &kn_map, const CUtensorMap &vn_map, int n_units, int cs_max, int64_t cta_limit,
                            int64_t cta_limit_pairs, cudaStream_t stream, bool *fits) {
    using C = ClusterCfg<D, G>;
    static PerDeviceOnce configured;
    int once_dev;
    if (configured.need(&once_dev)) {
        MATKV_CUDA(cudaFuncSetAttribute(k_decode_cluster<D, G>, cudaFuncAttributeMaxDynamicSharedMemorySize, C::SMEM_BYTES));
        MATKV_CUDA(cudaFuncSetAttribute(k_decode_cluster<D, G>, cudaFuncAttributeNonPortableClusterSizeAllowed, 1));
        configured.mark(once_dev);
    }
    int cs = 0;
    for (int c = cs_max; c >= 1; --c) {
        if ((int64_t)n_units * c > (c <= 2 ? cta_limit_pairs : cta_limit)) continue;
        if (max_active_clusters<D, G>(c) >= n_units) {
            cs = c;
            break;
        }
    }
    *fits = cs > 0;
    if (!cs) return MATKV_OK;
    p.cs = cs;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)(n_units * cs));
    cfg.blockDim = dim3((unsigned)kClThreads);
    cfg.dynamicSmemBytes = C::SMEM_BYTES;
    cfg.stream = stream;
    cudaLaunchAttribute attr[2];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    attr[1].id = cudaLaunchAttributeClusterDimension;
    attr[1].val.clusterDim.x = (unsigned)cs;
    attr[1].val.clusterDim.y = 1;
    attr[1].val.clusterDim.z = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 2;
    MATKV_CUDA(cudaLaunchKernelEx(&cfg, k_decode_cluster<D, G>, p, kn_map, vn_map));
    return MATKV_OK;
}

// Decode step of one layer through the cluster kernel when the launch is short enough to be a chain of latencies.
// *taken = false: the launch does not fit this kernel (the caller uses the streaming kernel).
int launch_decode_cluster(matkv_ctx *ctx, matkv_table *t, const AttendArgs &a, cudaStream_t stream, bool *taken) {
    *taken = false;
    const matkv_config &c = ctx->cfg;
    const int G = c.n_q_heads / c.n_kv_heads;
    // (a launch that is to advance the tail itself stays with the streaming kernel, whose last CTA does that)
    if (a.S != 1 || a.n_layers_launch != 1 || a.advance != 0 || t->has_fp8 || t->batch > kClMaxReq || !t->d_tile_dir || ctx->opt_decode_ctas > 0) return MATKV_OK;
    const int n_units = t->batch * c.n_kv_heads;
    const int64_t grid_max = std::max<int64_t>(ctx->n_sm - ctx->opt_stage_ctas, ctx->n_sm / 2);
    // Two CTAs of this kernel fit an SM.  A launch may take both places of every SM (it then cannot start beside its
    // predecessor, but all the SMs' shared memory is prefetching for it); measured, launches of more than 0.9 x 2 x SMs CTAs in
    // clusters of three or more do not become resident in one wave (B = 7 in clusters of 5, 280 CTAs: 36 us against 25.6 in
    // clusters of 4), pairs and single CTAs do up to the full 2 x SMs.
    const int64_t cta_limit = 2 * grid_max * 9 / 10, cta_limit_pairs = 2 * grid_max;
    if (n_units > cta_limit_pairs) return MATKV_OK;
    const int tt_nom = ceil_div(t->tail_len_host, kTile);
    int64_t W = 0, min_tiles = 1 << 30;
    for (int b = 0; b < t->batch; ++b) {
        const int64_t tiles = t->h_reqs[b].chunk_tiles + tt_nom + 1;
        W += (int64_t)c.n_kv_heads * tiles;
        min_tiles = std::min(min_tiles, tiles);
    }
    // cluster size: as many CTAs per unit as the SMs allow (any size up to 16, not only powers of two)
    int cs_max = (int)std::max<int64_t>(1, std::min<int64_t>(std::min<int64_t>(kClMaxCs, cta_limit_pairs / n_units), std::min<int64_t>(min_tiles, c.head_dim / 4)));
    if (ctx->opt_cluster_max > 0) cs_max = std::min<int>(cs_max, (int)ctx->opt_cluster_max);
    // Measured against the streaming kernel (8B and 70B head shapes, 5 / 10 / 40 chunks of 1,024 tokens per request, B = 1 .. 32,
    // launches replayed from a graph; us per layer, this kernel / streaming): 5 chunks: B = 1 9.4 / 12.0, B = 2 12.3 / 15.6,
    // B = 4 17.1 / 21.6, B = 8 28.4 / 35.6, B = 12 43.2 / 49.1, B = 16 52.9 / 59.6, B = 24 82 / 87, B = 32 102 / 110;
    // 10 chunks: B = 4 28.6 / 35.4, B = 16 101 / 107, B = 32 198 / 202; 40 chunks, G = 8: B = 2 59 / 65, B = 8 194 / 202.
    // It loses only where it cannot put enough CTAs to work: a launch with much work on few CTAs stays with the streaming
    // kernel, whose flat split uses every SM (B = 1 over 40 chunks in clusters of 8: 49.7 against 43.7).
    if ((int64_t)n_units * cs_max * 10 < grid_max * 6 && W >= 32 * grid_max) return MATKV_OK;
    ClusterParams p;
    p.tile_dir = t->d_tile_dir;
    p.tmaps = t->d_tmaps;
    p.n_seg_total = t->n_seg_total;
    p.tail_len = t->d_tail_len;
    p.tail_k = t->tail_k;
    p.tail_v = t->tail_v;
    p.q = a.q; p.out = a.out; p.lse_out = a.lse_out;
    p.q_sb = a.q_sb; p.lse_sb = a.lse_sb;
    p.layer = a.layer0; p.n_layers_total = c.n_layers; p.B = t->batch; p.Hkv = c.n_kv_heads; p.max_tail = c.max_tail_tokens;
    p.cs = 0;   // (chosen by the launcher)
    p.tt_nom = tt_nom;
    p.scale_log2 = ctx->scale * kLog2e;
    p.status = ctx->d_status;
    p.stream_hint = t->distinct_chunk_tiles == t->total_chunk_tiles;
    for (int b = 0; b < kClMaxReq; ++b) {
        p.chunk_tiles[b] = b < t->batch ? t->h_reqs[b].chunk_tiles : 0;
        p.dir_begin[b] = b < t->batch ? t->h_dir_begin[b] : 0;
    }
    CUtensorMap kn_map, vn_map;
    int rc = encode_new_rows_map(&kn_map, a.k_new, c.head_dim, c.n_kv_heads, (uint64_t)t->batch);
    if (!rc) rc = encode_new_rows_map(&vn_map, a.v_new, c.head_dim, c.n_kv_heads, (uint64_t)t->batch);
    if (rc) return rc;
    rc = fail(MATKV_E_INVALID_ARG, "unsupported head_dim %d / group %d", c.head_dim, G);
#define MATKV_CASE(DD, GG) \
    if (c.head_dim == DD && G == GG) rc = launch_cluster_t<DD, GG>(p, kn_map, vn_map, n_units, cs_max, cta_limit, cta_limit_pairs, stream, taken);
    MATKV_CASE(128, 1) MATKV_CASE(128, 2) MATKV_CASE(128, 4) MATKV_CASE(128, 8)
    MATKV_CASE(64, 1) MATKV_CASE(64, 2) MATKV_CASE(64, 4) MATKV_CASE(64, 8)
#undef MATKV_CASE
    return rc;
}

}  // namespace matkv

#ifdef MATKV_STAMPS
extern "C" int matkv_debug_cluster_stamps(unsigned long long *host_out) {
    return (int)cudaMemcpyFromSymbol(host_out, matkv::g_cl_stamps, sizeof(matkv::g_cl_stamps));
}
extern "C" int matkv_debug_cluster_clk(long long *host_out) {
    return (int)cudaMemcpyFromSymbol(host_out, matkv::g_cl_clk, sizeof(matkv::g_cl_clk));
}
extern "C" int matkv_debug_cluster_tiles(unsigned long long *host_out) {
    return (int)cudaMemcpyFromSymbol(host_out, matkv::g_cl_tiles, sizeof(matkv::g_cl_tiles));
}
#endif
