// K3: query sub-prefill over the chunk table on the 5th-generation tensor cores (tcgen05 + TMEM).
//
// One CTA = (request, KV head, NBLK blocks of 128 query rows, KV split).  A query row is (suffix token,
// head of the KV group), row = token * G + head, so the G heads that share a KV head and up to
// NBLK*128/G suffix tokens share every K/V tile that is fetched.  Per 64-token KV tile and row block:
//     S  = Q K^T      tcgen05.mma  M=128, N=64,  K=D   (both operands K-major, 128-byte swizzle)  -> TMEM
//     P  = softmax numerators of S (one thread per row: tcgen05.ld, fp32, exp2-based) -> bf16 pairs written back
//          into S's own TMEM columns (tcgen05.st): the second MMA takes P as its A operand from tensor memory
//     O += P V        tcgen05.mma  M=128, N=D,   K=64  (V is MN-major straight from its [token][d] tile),
//                     accumulated in TMEM across the tiles
// The exponent's reference maximum of a row only moves when the running maximum has grown by more than
// 2^8 (lazy rescale): then the row's thread multiplies its O row in TMEM (tcgen05.ld / tcgen05.st) and
// its running sum by the same factor, so numerators stay below 2^8 and O, l stay consistent.
// Warp roles: warp 0 producer (TMA tensor copies of chunk / tail tiles through the table's descriptors,
// of the call's new tokens through a per-call descriptor; appends the new tokens to the tail), warp 1
// issues the MMAs and owns the TMEM allocation, then four softmax warps per row block.  S is
// double-buffered in TMEM so that the tensor core works on tile j+1 while the softmax threads work on
// tile j; with two row blocks two softmax warps share each SM sub-partition.  Every wait is bounded and
// reports through the status word; TMEM is always released.
//
// Compressed-resident chunks (template parameter F8; head_dim 128, one row block per CTA): the producer brings a tile's
// e4m3 codes (K rows, V transposed per 64-token block, the block's two exponents) into a staging ring, and four
// converter warps expand them to bf16 in the operand ring: K as before, V^T [d][token] as a K-major B operand of
// O += P V (so the transposed store needs no transposing).  Every code stands for a bf16 number, so the expansion is
// exact and the tiles the tensor core sees are the ones the expanding staging copy would have written to HBM.
#include <cuda_runtime.h>
#include <cuda_bf16.h>
#include <cuda_fp16.h>
#include <math_constants.h>

#include <algorithm>

#include "matkv_internal.h"

namespace matkv {

namespace k3 {

constexpr int kRowsPerCta = 128;
constexpr long long kWaitCycles = 2000000000LL;
constexpr float kLog2e = 1.4426950408889634f;
constexpr float kLn2 = 0.6931471805599453f;

struct Params {
    const DevReq *reqs;
    const DevSeg *segs;
    const CUtensorMap *tmaps;
    const CUtensorMap *tmaps8;  // [n_seg_total][2] maps of compressed-resident chunks (K codes, transposed V codes), or null
    int32_t n_seg_total;
    const int32_t *tail_len;
    __nv_bfloat16 *tail_k, *tail_v;
    const __nv_bfloat16 *q, *k_new, *v_new;
    __nv_bfloat16 *out;
    float *lse_out;
    int64_t q_sl, q_sb, q_ss, kn_sl, kn_sb, kn_ss;  // element strides: layer, request, suffix token
    int32_t layer0, n_layers_launch, n_layers_total, B, S, Hq, Hkv, max_tail, n_rb, n_split;
    float scale_log2;
    float *part_o, *part_lse;  // [row][split][D], [row][split]; row = ((layer*B + b)*S + i)*Hq + head
    int32_t *status;
};

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
// Bounded wait; false once the CTA's abort flag is up or after about a second (which raises it).
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
__device__ __forceinline__ void tma_load_2d(uint32_t dst, const CUtensorMap *map, int32_t x, int32_t y, uint32_t bar) {
    asm volatile(
        "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];" ::"r"(dst),
        "l"(map), "r"(x), "r"(y), "r"(bar)
        : "memory");
}
__device__ __forceinline__ void tma_load_3d(uint32_t dst, const CUtensorMap *map, int32_t x, int32_t y, int32_t z, uint32_t bar) {
    asm volatile(
        "cp.async.bulk.tensor.3d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3, %4}], [%5];" ::"r"(dst),
        "l"(map), "r"(x), "r"(y), "r"(z), "r"(bar)
        : "memory");
}
// untiled bulk copy global -> shared with mbarrier completion (both addresses 16-byte aligned, size a multiple of 16)
__device__ __forceinline__ void bulk_load(uint32_t dst, const void *src, uint32_t bytes, uint32_t bar) {
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(dst), "l"(src), "r"(bytes),
                 "r"(bar)
                 : "memory");
}
__device__ __forceinline__ void fence_async_smem() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
__device__ __forceinline__ float fast_exp2(float x) {
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}

// Shared-memory matrix descriptor of a 128-byte-swizzled tile whose rows are 128 bytes (64 bf16).
//   K-major operand  (rows = M or N index, the 128 bytes run along K): SBO = 1024 (next group of 8 rows),
//                     LBO unused; a 16-element K slice is a 32-byte step of the start address.
//   MN-major operand (rows = K index, the 128 bytes run along M or N): SBO = 1024 (next 8 K rows),
//                     LBO = distance to the next 64-wide block along N.
// bits: [0,14) address >> 4, [16,30) LBO >> 4, [32,46) SBO >> 4, [46,48) version 1, [61,64) layout 2 = SWIZZLE_128B.
// (desc_lo below builds bits 0..31; the MMA helpers append the constant bits 32..63.)
// Instruction descriptor, kind::f16: fp32 accumulate, bf16 x bf16, A K-major, B K- or MN-major, M x N.
__host__ __device__ constexpr uint32_t instr_desc(int M, int N, bool b_mn_major) {
    return (1u << 4) | (1u << 7) | (1u << 10) | ((b_mn_major ? 1u : 0u) << 16) | ((uint32_t)(N >> 3) << 17) |
           ((uint32_t)(M >> 4) << 24);
}
// D (TMEM) = or += A (smem) B (smem).  The descriptors are given as low words (address and LBO, see desc_lo): the high
// word (SBO 1024, version 1, 128-byte swizzle) is the same for every operand here, so the low word advances by a plain
// 32-bit add and the issuing thread spends a handful of instructions per MMA instead of rebuilding 64-bit descriptors.
__device__ __forceinline__ void umma2(uint32_t d_tmem, uint32_t a_lo, uint32_t b_lo, uint32_t idesc, uint32_t accumulate) {
    constexpr uint32_t kHi = (1024u >> 4) | (1u << 14) | (2u << 29);   // bits 32.. of the descriptor
    asm volatile(
        "{\n .reg .pred p;\n .reg .b64 da, db;\n setp.ne.b32 p, %4, 0;\n mov.b64 da, {%1, %5};\n mov.b64 db, {%2, %5};\n"
        " tcgen05.mma.cta_group::1.kind::f16 [%0], da, db, %3, p;\n}" ::"r"(d_tmem),
        "r"(a_lo), "r"(b_lo), "r"(idesc), "r"(accumulate), "r"(kHi)
        : "memory");
}
// A operand taken from tensor memory (lane = row, 32-bit columns hold consecutive pairs of bf16 along K): the softmax
// threads leave P where S was, so the second MMA reads only V from shared memory.  Shared-memory bandwidth is what
// bounds this kernel: an M 128 x N 64 x K 16 MMA reads 6 KB of operands in the 32 cycles it computes.
__device__ __forceinline__ void umma_ta(uint32_t d_tmem, uint32_t a_tmem, uint32_t b_lo, uint32_t idesc, uint32_t accumulate) {
    constexpr uint32_t kHi = (1024u >> 4) | (1u << 14) | (2u << 29);
    asm volatile(
        "{\n .reg .pred p;\n .reg .b64 db;\n setp.ne.b32 p, %4, 0;\n mov.b64 db, {%2, %5};\n"
        " tcgen05.mma.cta_group::1.kind::f16 [%0], [%1], db, %3, p;\n}" ::"r"(d_tmem),
        "r"(a_tmem), "r"(b_lo), "r"(idesc), "r"(accumulate), "r"(kHi)
        : "memory");
}
// 32 consecutive 32-bit columns of this thread's TMEM lane (warp-collective), then wait for the store
__device__ __forceinline__ void tmem_st32(uint32_t taddr, const uint32_t (&r)[32]) {
    asm volatile(
        "tcgen05.st.sync.aligned.32x32b.x32.b32 [%0], {%1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, %16, "
        "%17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31, %32};" ::"r"(taddr),
        "r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7]), "r"(r[8]), "r"(r[9]), "r"(r[10]),
        "r"(r[11]), "r"(r[12]), "r"(r[13]), "r"(r[14]), "r"(r[15]), "r"(r[16]), "r"(r[17]), "r"(r[18]), "r"(r[19]), "r"(r[20]),
        "r"(r[21]), "r"(r[22]), "r"(r[23]), "r"(r[24]), "r"(r[25]), "r"(r[26]), "r"(r[27]), "r"(r[28]), "r"(r[29]), "r"(r[30]),
        "r"(r[31])
        : "memory");
    asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory");
}
// low word of a descriptor: address >> 4 in bits [0,14), LBO >> 4 in bits [16,30)
__device__ __forceinline__ uint32_t desc_lo(uint32_t addr, uint32_t lbo_bytes) {
    return ((addr & 0x3FFFFu) >> 4) | (((lbo_bytes >> 4) & 0x3FFFu) << 16);
}
__device__ __forceinline__ void umma_commit(uint32_t bar) {
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
// 32 consecutive 32-bit columns of this thread's TMEM lane: the load is only issued; tmem_ld_wait() completes it
__device__ __forceinline__ void tmem_ld32_issue(uint32_t taddr, uint32_t (&r)[32]) {
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x32.b32 {%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, %16, "
        "%17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]),
          "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]), "=r"(r[16]),
          "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]), "=r"(r[24]),
          "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
        : "r"(taddr));
}
__device__ __forceinline__ void tmem_ld_wait() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }
// 32 consecutive fp32 columns of this thread's TMEM lane
__device__ __forceinline__ void tmem_ld32(uint32_t taddr, float (&v)[32]) {
    uint32_t r[32];
    tmem_ld32_issue(taddr, r);
    tmem_ld_wait();
#pragma unroll
    for (int i = 0; i < 32; ++i) v[i] = __uint_as_float(r[i]);
}
__device__ __forceinline__ float2 fadd2(float2 a, float2 b) {  // two fp32 adds in one instruction (sm_100)
    unsigned long long d;
    asm("add.rn.f32x2 %0, %1, %2;"
        : "=l"(d)
        : "l"(*reinterpret_cast<unsigned long long *>(&a)), "l"(*reinterpret_cast<unsigned long long *>(&b)));
    return *reinterpret_cast<float2 *>(&d);
}
__device__ __forceinline__ float2 ffma2(float2 a, float2 b, float2 c) {  // two fp32 FMAs in one instruction (sm_100)
    unsigned long long d;
    asm("fma.rn.f32x2 %0, %1, %2, %3;"
        : "=l"(d)
        : "l"(*reinterpret_cast<unsigned long long *>(&a)), "l"(*reinterpret_cast<unsigned long long *>(&b)),
          "l"(*reinterpret_cast<unsigned long long *>(&c)));
    return *reinterpret_cast<float2 *>(&d);
}
// multiply 32 consecutive fp32 columns of this thread's TMEM lane by `f` (load, scale, store back)
__device__ __forceinline__ void tmem_scale32(uint32_t taddr, float f) {
    float v[32];
    tmem_ld32(taddr, v);
    uint32_t r[32];
#pragma unroll
    for (int i = 0; i < 32; ++i) r[i] = __float_as_uint(v[i] * f);
    asm volatile(
        "tcgen05.st.sync.aligned.32x32b.x32.b32 [%0], {%1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, %16, "
        "%17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31, %32};" ::"r"(taddr),
        "r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7]), "r"(r[8]), "r"(r[9]), "r"(r[10]),
        "r"(r[11]), "r"(r[12]), "r"(r[13]), "r"(r[14]), "r"(r[15]), "r"(r[16]), "r"(r[17]), "r"(r[18]), "r"(r[19]), "r"(r[20]),
        "r"(r[21]), "r"(r[22]), "r"(r[23]), "r"(r[24]), "r"(r[25]), "r"(r[26]), "r"(r[27]), "r"(r[28]), "r"(r[29]), "r"(r[30]),
        "r"(r[31])
        : "memory");
    asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi) {
    __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
    return *reinterpret_cast<uint32_t *>(&v);
}
// 16 e4m3 codes (one 16-byte chunk) times a power of two -> 16 bf16 (two chunks); exact: every code x 2^e is a bf16 number
__device__ __forceinline__ void expand16(const uint4 w, const float scale, uint4 &lo, uint4 &hi) {
    const uint32_t in[4] = {w.x, w.y, w.z, w.w};
    uint32_t out[8];
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        uint32_t h0, h1;   // codes 0,1 and 2,3 of the word as fp16 pairs (exact)
        asm("{\n .reg .b16 a, b;\n mov.b32 {a, b}, %2;\n cvt.rn.f16x2.e4m3x2 %0, a;\n cvt.rn.f16x2.e4m3x2 %1, b;\n}" : "=r"(h0), "=r"(h1) : "r"(in[i]));
        const float2 f0 = __half22float2(*reinterpret_cast<const __half2 *>(&h0)), f1 = __half22float2(*reinterpret_cast<const __half2 *>(&h1));
        out[2 * i] = pack_bf16(f0.x * scale, f0.y * scale);
        out[2 * i + 1] = pack_bf16(f1.x * scale, f1.y * scale);
    }
    lo = make_uint4(out[0], out[1], out[2], out[3]);
    hi = make_uint4(out[4], out[5], out[6], out[7]);
}
// true in exactly one lane of the (converged) warp
__device__ __forceinline__ bool elect_one() {
    uint32_t pred;
    asm volatile("{\n .reg .pred p;\n elect.sync _|p, 0xffffffff;\n selp.b32 %0, 1, 0, p;\n}" : "=r"(pred));
    return pred != 0;
}
__host__ __device__ __forceinline__ int cdiv(int a, int b) { return (a + b - 1) / b; }

// tile t of a unit: kind 0 = chunk, 1 = tail, 2 = new tokens
struct Tile {
    int kind, seg, r0, rows, seg_len;
    int fmt;   // chunk tiles: 0 = bf16 blob, 1 = compressed-resident codes
};

template <int D, int NBLK, bool F8 = false>
struct Cfg {
    static constexpr int NBOX = D / 64;
    static constexpr int BOX_BYTES = kTile * 128;        // 64 rows x 128 bytes
    static constexpr int KV_BYTES = NBOX * BOX_BYTES;    // K (or V) of one tile
    static constexpr int STAGE_BYTES = 2 * KV_BYTES;
    static constexpr int QBLK_BYTES = NBOX * kRowsPerCta * 128;   // Q of one row block
    static constexpr int STAGES = F8 ? 3 : 4;
    // staging ring of code tiles (compressed-resident chunks): K codes, V codes, then the block's exponent record
    static constexpr int CODE_STAGES = F8 ? 3 : 0;
    static constexpr int CODE_BYTES = kTile * D;                  // codes of K (or of V) of one tile
    static constexpr int CODE_STAGE_BYTES = 2 * CODE_BYTES + 1024;   // (+ the 16-byte record; keeps the 1024-byte alignment)
    static constexpr int CONV_WARPS = F8 ? 4 : 0;
    // producer warp, MMA warp of row block 0, 4 softmax warps per block, (last) the MMA warp of row block 1; then the converter warps
    static constexpr int THREADS = (2 + 4 * NBLK + (NBLK - 1) + CONV_WARPS) * 32;
    static constexpr int SMEM_BYTES = 1024 + NBLK * QBLK_BYTES + STAGES * STAGE_BYTES + CODE_STAGES * CODE_STAGE_BYTES + 512;
    // TMEM columns of row block b: S[2] at b*256 + {0, 64}; O at b*256 + 128 (D columns)
    static constexpr int COL_BLK = 256, COL_O = 128;
    static constexpr int TMEM_COLS = NBLK == 2 ? 512 : 256;
    static_assert(SMEM_BYTES <= 232448, "shared memory budget");
    static_assert(!F8 || (NBLK == 1 && D == 128), "compressed-resident chunks: head_dim 128, one row block per CTA");
};

// barrier slots (8 bytes each)
constexpr int kBarFull = 0, kBarEmpty = 4, kBarSFull = 8 /* [blk][2] */, kBarPReady = 12 /* [blk][2] */,
              kBarODone = 16 /* [blk][2] */, kBarQReady = 20, kBarCodeFull = 21 /* [3] */, kBarCodeEmpty = 24 /* [3] */, kBarCount = 27;

template <int D, int G, int NBLK, bool F8 = false>
__global__ void __launch_bounds__(Cfg<D, NBLK, F8>::THREADS, 1)
k_prefill_tc(const __grid_constant__ Params p, const __grid_constant__ CUtensorMap kn_map, const __grid_constant__ CUtensorMap vn_map) {
    using C = Cfg<D, NBLK, F8>;
    constexpr int kStages = C::STAGES;
    extern __shared__ unsigned char smem_raw[];
    unsigned char *smem = (unsigned char *)(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
    unsigned char *q_s = smem;                                   // [NBLK][NBOX boxes][128 rows][128 B]
    unsigned char *kv_s = q_s + NBLK * C::QBLK_BYTES;            // kStages x (K boxes, V boxes)
    unsigned char *code_s = kv_s + kStages * C::STAGE_BYTES;     // CODE_STAGES x (K codes, V codes, exponent record)
    uint64_t *bars = (uint64_t *)(code_s + C::CODE_STAGES * C::CODE_STAGE_BYTES);
    uint32_t *tmem_slot = (uint32_t *)(bars + kBarCount);
    volatile int *abort_flag = (volatile int *)(tmem_slot + 2);
    volatile int *v_kmajor = abort_flag + 1;                     // [kStages] 1: the stage's V is stored [d][token] (expanded codes)

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    // which unit
    int c = blockIdx.x;
    const int sp = c % p.n_split; c /= p.n_split;
    const int rb = c % p.n_rb; c /= p.n_rb;                      // index of this CTA's group of NBLK row blocks
    const int g = c % p.Hkv; c /= p.Hkv;
    const int b = c % p.B;
    const int l_rel = c / p.B;                                   // layer of the launch
    const int layer = p.layer0 + l_rel;
    const DevReq rq = p.reqs[b];
    int t0 = p.tail_len[b];
    if (t0 < 0 || t0 + p.S > p.max_tail) {
        if (tid == 0) atomicCAS(p.status, 0, MATKV_E_CAPACITY);
        t0 = max(0, min(t0, p.max_tail - p.S));
    }
    const int R = p.S * G;                       // query rows of the (request, KV head)
    const int row0 = rb * NBLK * kRowsPerCta;
    // new-token tiles past this CTA's last suffix token are invisible to all of its rows (causal): not visited at all,
    // which halves the work of a long causal sub-prefill (a chunk materialised alone: S = its length, no chunks)
    const int tok_last = min(p.S - 1, (row0 + NBLK * kRowsPerCta - 1) / G);
    const int tail_tiles = cdiv(t0, kTile), new_tiles = tok_last / kTile + 1;
    const int T = rq.chunk_tiles + tail_tiles + new_tiles;
    const int t_begin = (int)((int64_t)sp * T / p.n_split), t_end = (int)((int64_t)(sp + 1) * T / p.n_split);
    const int n_tiles = t_end - t_begin;

    const uint32_t bar0 = smem_u32(bars);
    const uint32_t full_kv = bar0 + kBarFull * 8, empty_kv = bar0 + kBarEmpty * 8, s_full = bar0 + kBarSFull * 8,
                   p_ready = bar0 + kBarPReady * 8, o_done = bar0 + kBarODone * 8, q_ready = bar0 + kBarQReady * 8;
    if (tid == 0) {
        for (int s = 0; s < 4; ++s) {
            mbar_init(full_kv + s * 8, 1);
            mbar_init(empty_kv + s * 8, NBLK);   // one commit per row block's MMA warp
            mbar_init(s_full + s * 8, 1);
            mbar_init(p_ready + s * 8, 128);
        }
        for (int s = 0; s < 4; ++s) mbar_init(o_done + s * 8, 1);
        for (int s = 0; s < 3; ++s) {
            mbar_init(bar0 + (kBarCodeFull + s) * 8, 1);
            mbar_init(bar0 + (kBarCodeEmpty + s) * 8, 1);
        }
        for (int s = 0; s < kStages; ++s) v_kmajor[s] = 0;
        mbar_init(q_ready, 128 * NBLK);
        *abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        fence_async_smem();
    }
    if (warp == 1) {  // TMEM (one CTA per SM)
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(tmem_slot)),
                     "r"((uint32_t)C::TMEM_COLS)
                     : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = *tmem_slot;

    // tile lookup shared by the producer and the softmax threads
    auto tile_at = [&](int t, int &seg, int &tiles_before, int &seg_tiles, int &seg_len, int &seg_fmt) {
        Tile ti;
        ti.fmt = 0;
        if (t < rq.chunk_tiles) {
            while (seg < 0 || t >= tiles_before + seg_tiles) {
                tiles_before += seg_tiles;
                ++seg;
                const DevSeg sg = p.segs[rq.seg_begin + seg];
                seg_len = sg.len;
                seg_fmt = F8 ? sg.fmt : 0;
                seg_tiles = cdiv(seg_len, kTile);
            }
            ti.kind = 0; ti.seg = seg; ti.seg_len = seg_len; ti.fmt = seg_fmt;
            ti.r0 = (t - tiles_before) * kTile;
            ti.rows = min(kTile, seg_len - ti.r0);
        } else if (t < rq.chunk_tiles + tail_tiles) {
            ti.kind = 1; ti.seg = 0; ti.seg_len = 0;
            ti.r0 = (t - rq.chunk_tiles) * kTile;
            ti.rows = min(kTile, t0 - ti.r0);
        } else {
            ti.kind = 2; ti.seg = 0; ti.seg_len = 0;
            ti.r0 = (t - rq.chunk_tiles - tail_tiles) * kTile;
            ti.rows = min(kTile, p.S - ti.r0);
        }
        return ti;
    };

    if (warp == 0) {
        // ===================== producer =====================
        // appends this CTA's share of the new tokens to the tail for later calls: the suffix tokens of its own query rows,
        // divided among the KV splits (a long suffix copied by the CTAs of row group 0 alone kept their SMs for hundreds
        // of microseconds)
        auto append_share = [&]() {
            constexpr int CPR = D / 8;
            const int tok_a = row0 / G, tok_b = min(p.S, (row0 + NBLK * kRowsPerCta) / G), n_own = max(0, tok_b - tok_a);
            const int a0 = tok_a + (int)((int64_t)sp * n_own / p.n_split), a1 = tok_a + (int)((int64_t)(sp + 1) * n_own / p.n_split);
#pragma unroll 8
            for (int idx = a0 * CPR + lane; idx < a1 * CPR; idx += 32) {
                const int tok = idx / CPR, ch = idx % CPR;
                if (t0 + tok < p.max_tail) {
                    const int64_t src = (int64_t)l_rel * p.kn_sl + (int64_t)b * p.kn_sb + (int64_t)tok * p.kn_ss + (int64_t)g * D + ch * 8;
                    const int64_t dsto = ((((int64_t)b * p.n_layers_total + layer) * p.Hkv + g) * p.max_tail + t0 + tok) * D + ch * 8;
                    *(uint4 *)(p.tail_k + dsto) = *(const uint4 *)(p.k_new + src);
                    *(uint4 *)(p.tail_v + dsto) = *(const uint4 *)(p.v_new + src);
                }
            }
        };
        int seg = -1, tiles_before = 0, seg_tiles = 0, seg_len = 0, seg_fmt = 0;
        int n_code = 0;   // code tiles issued so far (their staging ring has a sequence of its own)
        bool ok = true;
        for (int j = 0; j < n_tiles && ok; ++j) {
            const int st = j % kStages, use = j / kStages;
            const Tile ti = tile_at(t_begin + j, seg, tiles_before, seg_tiles, seg_len, seg_fmt);
            if constexpr (F8) {
                if (ti.kind == 0 && ti.fmt == 1) {
                    // a tile of codes goes to the staging ring; the converter warps expand it into operand stage `st`
                    // (they wait for that stage to be free themselves)
                    const int cst = n_code % C::CODE_STAGES, cuse = n_code / C::CODE_STAGES;
                    ++n_code;
                    if (cuse > 0) ok = mbar_wait(bar0 + (kBarCodeEmpty + cst) * 8, (cuse - 1) & 1, abort_flag);
                    ok = __all_sync(0xffffffffu, ok);
                    if (!ok) break;
                    if (lane == 0) {
                        const DevSeg sg = p.segs[rq.seg_begin + ti.seg];
                        const int st_tiles = cdiv(ti.seg_len, kTile);
                        const int64_t blk = ((int64_t)layer * p.Hkv + g) * st_tiles + ti.r0 / kTile;
                        const int64_t region = ((int64_t)p.n_layers_total * p.Hkv * st_tiles * kTile * D + 255) / 256 * 256;
                        const CUtensorMap *m8 = p.tmaps8 + 2 * (rq.seg_begin + ti.seg);
                        const uint32_t cdst = smem_u32(code_s + cst * C::CODE_STAGE_BYTES), cbar = bar0 + (kBarCodeFull + cst) * 8;
                        mbar_expect_tx(cbar, 2 * C::CODE_BYTES + 16);
                        tma_load_2d(cdst, m8, 0, (int32_t)(blk * kTile), cbar);
                        tma_load_2d(cdst + C::CODE_BYTES, m8 + 1, 0, (int32_t)(blk * D), cbar);
                        bulk_load(cdst + 2 * C::CODE_BYTES, (const unsigned char *)sg.base + 2 * region + blk * 16, 16, cbar);
                    }
                    continue;
                }
            }
            if (use > 0) ok = mbar_wait(empty_kv + st * 8, (use - 1) & 1, abort_flag);
            ok = __all_sync(0xffffffffu, ok);
            if (!ok) break;
            const uint32_t dst = smem_u32(kv_s + st * C::STAGE_BYTES), bar = full_kv + st * 8;
            if (lane == 0) {
                if constexpr (F8) v_kmajor[st] = 0;   // (ordered before the consumers' look by the barrier's release / acquire)
                mbar_expect_tx(bar, C::STAGE_BYTES);
                if (ti.kind < 2) {
                    const CUtensorMap *mk, *mv;
                    int32_t yk, yv;
                    if (ti.kind == 0) {
                        mk = mv = p.tmaps + rq.seg_begin + ti.seg;
                        yk = ((layer * 2) * p.Hkv + g) * ti.seg_len + ti.r0;
                        yv = ((layer * 2 + 1) * p.Hkv + g) * ti.seg_len + ti.r0;
                    } else {
                        mk = p.tmaps + p.n_seg_total;
                        mv = mk + 1;
                        yk = yv = ((b * p.n_layers_total + layer) * p.Hkv + g) * p.max_tail + ti.r0;
                    }
#pragma unroll
                    for (int bx = 0; bx < C::NBOX; ++bx) {
                        tma_load_2d(dst + bx * C::BOX_BYTES, mk, bx * 64, yk, bar);
                        tma_load_2d(dst + C::KV_BYTES + bx * C::BOX_BYTES, mv, bx * 64, yv, bar);
                    }
                } else {
                    // the call's new tokens, straight from k_new / v_new [B*S][Hkv][D] (rows past S are masked)
#pragma unroll
                    for (int bx = 0; bx < C::NBOX; ++bx) {
                        tma_load_3d(dst + bx * C::BOX_BYTES, &kn_map, bx * 64, g, (l_rel * p.B + b) * p.S + ti.r0, bar);
                        tma_load_3d(dst + C::KV_BYTES + bx * C::BOX_BYTES, &vn_map, bx * 64, g, (l_rel * p.B + b) * p.S + ti.r0, bar);
                    }
                }
            }
        }
        // Only later calls read the tail (this one takes the new tokens from k_new / v_new): the copy waits until every
        // tile load of the CTA has been issued.  Issued between two tile loads it held the second one back by its whole
        // duration (measured: 30 us per CTA on a 1,024-token suffix).
        append_share();
    } else if (warp == 1 || (NBLK == 2 && warp == 2 + 4 * NBLK)) {
        // ===================== MMA issuers: one warp per row block =====================
        // The whole warp walks the loop (waits and descriptor arithmetic on warp-uniform values); one elected lane
        // issues the MMAs and their commits.  With a single lane behind a divergent branch every tcgen05.mma cost
        // the issuing thread 65 to 85 cycles; this way it is about 45.
        // Each row block has an issuing warp of its own, so the blocks are independent pipelines that share only the
        // K/V ring (a stage is free when both warps' P V of its tile have run) and the tensor pipe itself: with one
        // warp issuing for both in a fixed order, each block's S = Q K^T waited for the other block's softmax.
        {
            const int blk = warp == 1 ? 0 : 1;
            constexpr uint32_t idesc_qk = instr_desc(kRowsPerCta, kTile, false);
            constexpr uint32_t idesc_pv = instr_desc(kRowsPerCta, D, true), idesc_pv_k = instr_desc(kRowsPerCta, D, false);
            const uint32_t q_lo = desc_lo(smem_u32(q_s) + blk * C::QBLK_BYTES, 0), kv_u32 = smem_u32(kv_s);
            const uint32_t tm = tmem + blk * C::COL_BLK;
            bool ok = __all_sync(0xffffffffu, mbar_wait(q_ready, 0, abort_flag));
            auto do_pv = [&](int t) {  // O += P(t) V(t), then this block's share of freeing the K/V stage
                const int bf = t & 1, st = t % kStages;
                if (!__all_sync(0xffffffffu, mbar_wait(p_ready + (blk * 2 + bf) * 8, (t >> 1) & 1, abort_flag))) return false;
                tc_fence_after();
                // V as stored, [token][d] (MN-major: 16 tokens = 16 rows of 128 bytes per step), or, expanded from codes,
                // V^T [d][token] (K-major like K: 16 tokens = 32 bytes per step)
                const bool vk = F8 && v_kmajor[st] != 0;
                const uint32_t v_lo = desc_lo(kv_u32 + st * C::STAGE_BYTES + C::KV_BYTES, vk ? 0 : C::BOX_BYTES);
                const uint32_t v_step = vk ? (32 >> 4) : (2048 >> 4), idesc_v = vk ? idesc_pv_k : idesc_pv;
                if (elect_one()) {
#pragma unroll
                    for (int ks = 0; ks < kTile / 16; ++ks)  // 16 tokens per MMA: P advances 8 TMEM columns (in S's place)
                        umma_ta(tm + C::COL_O, tm + bf * kTile + ks * 8, v_lo + ks * v_step, idesc_v, (t > 0 || ks > 0) ? 1u : 0u);
                    umma_commit(o_done + (blk * 2 + bf) * 8);
                    umma_commit(empty_kv + st * 8);
                }
                __syncwarp();
                return true;
            };
            for (int j = 0; j < n_tiles && ok; ++j) {
                const int st = j % kStages;
                ok = __all_sync(0xffffffffu, mbar_wait(full_kv + st * 8, (j / kStages) & 1, abort_flag));
                if (!ok) break;
                tc_fence_after();
                const uint32_t k_lo = desc_lo(kv_u32 + st * C::STAGE_BYTES, 0);
                if (elect_one()) {
#pragma unroll
                    for (int ks = 0; ks < D / 16; ++ks)  // 16 dims per MMA; 4 such slices per 64-wide box
                        umma2(tm + (j & 1) * kTile, q_lo + (((ks / 4) * (kRowsPerCta * 128) + (ks % 4) * 32) >> 4),
                              k_lo + (((ks / 4) * C::BOX_BYTES + (ks % 4) * 32) >> 4), idesc_qk, ks > 0);
                    umma_commit(s_full + (blk * 2 + (j & 1)) * 8);
                }
                __syncwarp();
                if (j >= 1) ok = do_pv(j - 1);
            }
            if (ok && n_tiles > 0) do_pv(n_tiles - 1);
        }
    } else if (F8 && warp >= 2 + 4 * NBLK + (NBLK - 1)) {
        // ===================== converter warps: tiles of codes -> bf16 operand tiles =====================
        if constexpr (F8) {
            const int ct = tid - (2 + 4 * NBLK + (NBLK - 1)) * 32;   // 0..127
            int seg = -1, tiles_before = 0, seg_tiles = 0, seg_len = 0, seg_fmt = 0, n_code = 0;
            bool ok = true;
            for (int j = 0; j < n_tiles && ok; ++j) {
                const Tile ti = tile_at(t_begin + j, seg, tiles_before, seg_tiles, seg_len, seg_fmt);
                if (!(ti.kind == 0 && ti.fmt == 1)) continue;
                const int st = j % kStages, use = j / kStages;
                const int cst = n_code % C::CODE_STAGES, cuse = n_code / C::CODE_STAGES;
                ++n_code;
                ok = mbar_wait(bar0 + (kBarCodeFull + cst) * 8, cuse & 1, abort_flag);
                if (ok && use > 0) ok = mbar_wait(empty_kv + st * 8, (use - 1) & 1, abort_flag);
                ok = __all_sync(0xffffffffu, ok);
                if (!ok) break;
                const unsigned char *cs_ = code_s + cst * C::CODE_STAGE_BYTES;
                unsigned char *ks_ = kv_s + st * C::STAGE_BYTES;
                const int ek = (int)*(const signed char *)(cs_ + 2 * C::CODE_BYTES), ev = (int)*(const signed char *)(cs_ + 2 * C::CODE_BYTES + 1);
                const float sk = __uint_as_float(ek > -127 ? (uint32_t)(ek + 127) << 23 : 0x00400000u);   // 2^e (2^-127 is a subnormal float)
                const float sv = __uint_as_float(ev > -127 ? (uint32_t)(ev + 127) << 23 : 0x00400000u);
#pragma unroll
                for (int i = 0; i < kTile * D / 16 / 128; ++i) {
                    // K: row t of 128 codes (128-byte swizzle); 16 codes = dimensions 16c .. 16c+15 -> two 16-byte chunks of bf16
                    const int q = ct + 128 * i, t = q >> 3, c = q & 7;
                    const uint4 w = *(const uint4 *)(cs_ + t * 128 + ((c ^ (t & 7)) << 4));
                    uint4 lo, hi;
                    expand16(w, sk, lo, hi);
                    unsigned char *row = ks_ + (c >> 2) * C::BOX_BYTES + t * 128;
                    *(uint4 *)(row + ((((2 * c) & 7) ^ (t & 7)) << 4)) = lo;
                    *(uint4 *)(row + ((((2 * c + 1) & 7) ^ (t & 7)) << 4)) = hi;
                }
#pragma unroll
                for (int i = 0; i < kTile * D / 16 / 128; ++i) {
                    // V^T: row d of 64 codes (64-byte swizzle); 16 codes = tokens 16c .. 16c+15 -> two chunks of the [d][token] tile
                    const int q = ct + 128 * i, d = q >> 2, c = q & 3;
                    const uint4 w = *(const uint4 *)(cs_ + C::CODE_BYTES + d * 64 + ((c ^ ((d >> 1) & 3)) << 4));
                    uint4 lo, hi;
                    expand16(w, sv, lo, hi);
                    unsigned char *row = ks_ + C::KV_BYTES + d * 128;
                    *(uint4 *)(row + (((2 * c) ^ (d & 7)) << 4)) = lo;
                    *(uint4 *)(row + (((2 * c + 1) ^ (d & 7)) << 4)) = hi;
                }
                fence_async_smem();                                   // the tensor core reads these tiles through the async proxy
                asm volatile("bar.sync 2, 128;" ::: "memory");        // the four converter warps
                if (ct == 0) {
                    v_kmajor[st] = 1;
                    mbar_arrive(full_kv + st * 8);                    // the operand stage holds tile j
                    mbar_arrive(bar0 + (kBarCodeEmpty + cst) * 8);    // the code stage may be refilled
                }
            }
        }
    } else {
        // ===================== softmax threads: one query row each =====================
        const int blk = (warp - 2) >> 2;                      // row block of this warp
        const int r = (warp & 3) * 32 + lane;                 // TMEM lane = row inside the block
        const int grow = row0 + blk * kRowsPerCta + r;        // row inside the (request, KV head)
        const bool real = grow < R;
        const int tok = grow / G, hd = grow % G;              // suffix token and head of the group
        const uint32_t lane_base = tmem + blk * C::COL_BLK + ((uint32_t)((warp & 3) * 32) << 16);
        // Q row -> swizzled smem (zeros for rows past R)
        {
            const __nv_bfloat16 *qrow = p.q + (int64_t)l_rel * p.q_sl + (int64_t)b * p.q_sb + (int64_t)tok * p.q_ss + (int64_t)(g * G + hd) * D;
            unsigned char *qb = q_s + blk * C::QBLK_BYTES;
#pragma unroll
            for (int ch = 0; ch < D / 8; ++ch) {
                const uint4 v = real ? *(const uint4 *)(qrow + ch * 8) : make_uint4(0, 0, 0, 0);
                *(uint4 *)(qb + (ch / 8) * (kRowsPerCta * 128) + r * 128 + (((ch % 8) ^ (r & 7)) << 4)) = v;
            }
            fence_async_smem();
            mbar_arrive(q_ready);
        }
        // m_ref: the maximum the exponents refer to (log2 units, scaled); it trails the true running maximum by
        // at most 8, so numerators stay below 2^8.  l_run: sum of the numerators relative to m_ref.
        // l_rnd: the same sum over the bf16-rounded numerators the tensor core really multiplies with V; O is
        // normalised by it (a dominant token's rounding error then cancels), the log-sum-exp uses l_run.
        float m_ref = -CUDART_INF_F, l_run = 0.f, l_rnd = 0.f;
        int seg = -1, tiles_before = 0, seg_tiles = 0, seg_len = 0, seg_fmt = 0;
        bool ok = true;
        int plain_end = 0;   // tiles before it (of the unit) are full chunk tiles: every column visible, nothing to look up
        for (int j = 0; j < n_tiles && ok; ++j) {
            // visible columns: all valid rows of a chunk / tail tile; causal inside the new tokens
            int n_vis = kTile;
            if (t_begin + j >= plain_end) {
                const Tile ti = tile_at(t_begin + j, seg, tiles_before, seg_tiles, seg_len, seg_fmt);
                n_vis = ti.rows;
                if (ti.kind == 2) n_vis = min(ti.rows, tok - ti.r0 + 1);
                if (ti.kind == 0) plain_end = tiles_before + seg_len / kTile;
            }
            const int bf = j & 1;
            ok = mbar_wait(s_full + (blk * 2 + bf) * 8, (j >> 1) & 1, abort_flag);
            ok = __all_sync(0xffffffffu, ok);   // the TMEM loads below are warp-collective
            if (!ok) break;
            tc_fence_after();
            float s[kTile];
            // the row's 64 scores from tensor memory (warp-collective), masked: ragged or causal tiles (a full tile skips that).
            // Scores stay raw (unscaled): the scale is folded into the exponent's FMA below.
            auto load_scores = [&]() {
                uint32_t r0[32], r1[32];   // both halves in flight before the one wait
                tmem_ld32_issue(lane_base + bf * kTile, r0);
                tmem_ld32_issue(lane_base + bf * kTile + 32, r1);
                tmem_ld_wait();
#pragma unroll
                for (int i = 0; i < 32; ++i) {
                    s[i] = __uint_as_float(r0[i]);
                    s[32 + i] = __uint_as_float(r1[i]);
                }
                if (n_vis < kTile) {
#pragma unroll
                    for (int i = 0; i < kTile; ++i) s[i] = i < n_vis ? s[i] : -CUDART_INF_F;
                }
            };
            load_scores();
            // The row's numerators against the CURRENT reference maximum: P as bf16 pairs (they go where S was: the first 32
            // columns of the buffer), their sum and the sum of their roundings.
            uint32_t pw[kTile / 2];
            float psum, prnd;
            auto numerators = [&]() {
                const float m_neg = m_ref == -CUDART_INF_F ? 0.f : -m_ref;
                const float2 sc2 = make_float2(p.scale_log2, p.scale_log2), mn2 = make_float2(m_neg, m_neg);
                float2 psum2 = make_float2(0.f, 0.f), prnd2 = make_float2(0.f, 0.f);  // packed fp32 pairs: half the adds
#pragma unroll
                for (int ch = 0; ch < kTile / 8; ++ch) {
                    float e[8];
#pragma unroll
                    for (int i = 0; i < 4; ++i) {   // scale and offset as packed pairs: half the FMAs
                        const float2 x = ffma2(make_float2(s[ch * 8 + 2 * i], s[ch * 8 + 2 * i + 1]), sc2, mn2);
                        e[2 * i] = fast_exp2(x.x);
                        e[2 * i + 1] = fast_exp2(x.y);
                    }
                    const uint32_t pk[4] = {pack_bf16(e[0], e[1]), pack_bf16(e[2], e[3]), pack_bf16(e[4], e[5]), pack_bf16(e[6], e[7])};
#pragma unroll
                    for (int i = 0; i < 4; ++i) {
                        psum2 = fadd2(psum2, make_float2(e[2 * i], e[2 * i + 1]));
                        prnd2 = fadd2(prnd2, make_float2(__uint_as_float(pk[i] << 16), __uint_as_float(pk[i] & 0xffff0000u)));
                    }
                    pw[ch * 4] = pk[0]; pw[ch * 4 + 1] = pk[1]; pw[ch * 4 + 2] = pk[2]; pw[ch * 4 + 3] = pk[3];
                }
                psum = psum2.x + psum2.y;
                prnd = prnd2.x + prnd2.y;
            };
            // Lazy rescale, decided optimistically.  The reference only has to move when some numerator would exceed 2^8,
            // and after the first tiles that is rare: the numerators are formed against the reference as it stands, and
            // only a row sum of 2^8 or more (no numerator can be that large otherwise; an overflow to infinity lands here
            // too), or a row that has no reference yet, makes the warp look for the row maximum at all.  The 64-way
            // maximum, which cost a quarter of the row pass, is off the common path.
            numerators();
            const bool look = m_ref == -CUDART_INF_F ? n_vis > 0 : !(psum < 256.0f);
            if (__any_sync(0xffffffffu, look)) {     // tcgen05.ld / st are warp-collective: decide per warp
                load_scores();   // again (P has not been stored over them yet): the common path need not keep 64 scores alive
                float tmax = -CUDART_INF_F;
                if (look) {   // eight independent chains, then a tree: a single chain of 64 dependent maxima costs 250 cycles of latency
                    float mx[8];
#pragma unroll
                    for (int i = 0; i < 8; ++i) mx[i] = s[i];
#pragma unroll
                    for (int i = 8; i < kTile; ++i) mx[i & 7] = fmaxf(mx[i & 7], s[i]);
                    tmax = fmaxf(fmaxf(fmaxf(mx[0], mx[1]), fmaxf(mx[2], mx[3])), fmaxf(fmaxf(mx[4], mx[5]), fmaxf(mx[6], mx[7])));
                    tmax *= p.scale_log2;   // the scale is positive: the maximum commutes with it
                }
                // move the reference only when the maximum has grown by more than 2^8
                const bool grow_ref = look && tmax > m_ref + 8.0f;   // also true for the first visible column (m_ref = -inf)
                // o_done has one barrier per parity of the tile index, like S: a waiter is never more than one use of a
                // barrier behind (the P V of tile j+1 cannot be issued before this thread has delivered P of tile j+1), so
                // tiles whose completion nobody needs to see are simply not waited for.
                if (__any_sync(0xffffffffu, grow_ref)) {
                    const float alpha = grow_ref ? (m_ref == -CUDART_INF_F ? 0.f : fast_exp2(m_ref - tmax)) : 1.f;
                    if (j > 0) {
                        // O of tiles 0..j-1 must be complete before it is scaled
                        ok = mbar_wait(o_done + (blk * 2 + ((j - 1) & 1)) * 8, ((j - 1) >> 1) & 1, abort_flag);
                        ok = __all_sync(0xffffffffu, ok);
                        if (!ok) break;
                        tc_fence_after();
#pragma unroll
                        for (int c0 = 0; c0 < D; c0 += 32) tmem_scale32(lane_base + C::COL_O + c0, alpha);
                        tc_fence_before();
                    }
                    if (grow_ref) {
                        l_run *= alpha;
                        l_rnd *= alpha;
                        m_ref = tmax;
                    }
                }
                // again, against the reference as it is now (every lane: the lanes whose reference stayed get the same values,
                // and nothing of the first pass has to be kept alive across this rare path)
                numerators();
            }
            tmem_st32(lane_base + bf * kTile, pw);
            l_run += psum;
            l_rnd += prnd;
            tc_fence_before();
            mbar_arrive(p_ready + (blk * 2 + bf) * 8);
        }
        // epilogue: O is complete once the last P V has run
        if (ok && n_tiles > 0) {
            ok = mbar_wait(o_done + (blk * 2 + ((n_tiles - 1) & 1)) * 8, ((n_tiles - 1) >> 1) & 1, abort_flag);
            ok = __all_sync(0xffffffffu, ok);
        }
        if (ok) {
            tc_fence_after();
            const float inv = l_rnd > 0.f ? 1.f / l_rnd : 0.f;
            const float lse = l_run > 0.f ? (m_ref + log2f(l_run)) * kLn2 : -CUDART_INF_F;
            const int64_t orow = (((int64_t)l_rel * p.B + b) * p.S + tok) * p.Hq + g * G + hd;
#pragma unroll
            for (int c0 = 0; c0 < D; c0 += 32) {
                float v[32];
                tmem_ld32(lane_base + C::COL_O + c0, v);   // warp-collective: every lane loads, real rows store
                if (real) {
                    if (p.n_split == 1) {
                        __nv_bfloat16 *dst = p.out + (int64_t)l_rel * p.q_sl + (int64_t)b * p.q_sb + (int64_t)tok * p.q_ss + (int64_t)(g * G + hd) * D + c0;
#pragma unroll
                        for (int ch = 0; ch < 4; ++ch)
                            *(uint4 *)(dst + ch * 8) = make_uint4(
                                pack_bf16(v[ch * 8] * inv, v[ch * 8 + 1] * inv), pack_bf16(v[ch * 8 + 2] * inv, v[ch * 8 + 3] * inv),
                                pack_bf16(v[ch * 8 + 4] * inv, v[ch * 8 + 5] * inv), pack_bf16(v[ch * 8 + 6] * inv, v[ch * 8 + 7] * inv));
                    } else {
                        float *dst = p.part_o + (orow * p.n_split + sp) * D + c0;
#pragma unroll
                        for (int ch = 0; ch < 8; ++ch)
                            *(float4 *)(dst + ch * 4) = make_float4(v[ch * 4] * inv, v[ch * 4 + 1] * inv, v[ch * 4 + 2] * inv, v[ch * 4 + 3] * inv);
                    }
                }
            }
            if (real) {
                if (p.n_split == 1) {
                    if (p.lse_out) p.lse_out[orow] = lse;
                } else {
                    p.part_lse[orow * p.n_split + sp] = lse;
                }
            }
        }
    }
    // ---- teardown: every thread gets here, TMEM is always given back ----
    tc_fence_before();
    __syncthreads();
    if (warp == 1) {
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"((uint32_t)C::TMEM_COLS) : "memory");
    }
    if (tid == 0 && *abort_flag) atomicCAS(p.status, 0, MATKV_E_TIMEOUT);
}

}  // namespace k3

template <int D, int G, int NBLK, bool F8 = false>
static int launch_k3(const k3::Params &p, const CUtensorMap &kn_map, const CUtensorMap &vn_map, int grid, cudaStream_t stream) {
    using C = k3::Cfg<D, NBLK, F8>;
    static PerDeviceOnce configured;
    int once_dev;
    if (configured.need(&once_dev)) {
        MATKV_CUDA(cudaFuncSetAttribute(k3::k_prefill_tc<D, G, NBLK, F8>, cudaFuncAttributeMaxDynamicSharedMemorySize, C::SMEM_BYTES));
        configured.mark(once_dev);
    }
    k3::k_prefill_tc<D, G, NBLK, F8><<<grid, C::THREADS, C::SMEM_BYTES, stream>>>(p, kn_map, vn_map);
    MATKV_CUDA(cudaGetLastError());
    return MATKV_OK;
}

int launch_prefill_tc(matkv_ctx *ctx, matkv_table *t, const AttendArgs &a, cudaStream_t stream) {
    const matkv_config &c = ctx->cfg;
    const int G = c.n_q_heads / c.n_kv_heads, D = c.head_dim;
    k3::Params p;
    p.reqs = t->d_reqs; p.segs = t->d_segs; p.tmaps = t->d_tmaps; p.tmaps8 = t->d_tmaps8; p.n_seg_total = t->n_seg_total;
    p.tail_len = t->d_tail_len; p.tail_k = t->tail_k; p.tail_v = t->tail_v;
    p.q = a.q; p.k_new = a.k_new; p.v_new = a.v_new; p.out = a.out; p.lse_out = a.lse_out;
    p.q_sl = a.q_sl; p.q_sb = a.q_sb; p.q_ss = a.q_ss; p.kn_sl = a.kn_sl; p.kn_sb = a.kn_sb; p.kn_ss = a.kn_ss;
    p.layer0 = a.layer0; p.n_layers_launch = a.n_layers_launch; p.n_layers_total = c.n_layers; p.B = t->batch; p.S = a.S; p.Hq = c.n_q_heads; p.Hkv = c.n_kv_heads;
    p.max_tail = c.max_tail_tokens;
    // two row blocks per CTA when the (request, KV head) has more than 128 query rows and there are still
    // enough CTAs to fill most of the SMs (otherwise one block per CTA and more KV splits)
    const int R = a.S * G;
    const bool fill = (int64_t)a.n_layers_launch * t->batch * c.n_kv_heads * ((R + 255) / 256) * 10 >= 6 * (int64_t)ctx->n_sm;
    // (tables with compressed-resident chunks: one row block per CTA, the converter warps take the other block's place)
    const int nblk = (!t->has_fp8 && R > k3::kRowsPerCta && (fill || ctx->opt_prefill_impl == 3)) ? 2 : 1;
    p.n_rb = (a.S * G + nblk * k3::kRowsPerCta - 1) / (nblk * k3::kRowsPerCta);
    p.scale_log2 = ctx->scale * k3::kLog2e;
    p.status = ctx->d_status;
    // KV splits: fill the SMs, never more splits than the shortest request has tiles, and only as many
    // as the workspace can hold partials for
    const int64_t combos = (int64_t)a.n_layers_launch * t->batch * c.n_kv_heads * p.n_rb;
    int min_tiles = 1 << 30;
    for (int b = 0; b < t->batch; ++b)
        min_tiles = std::min(min_tiles, t->h_reqs[b].chunk_tiles + k3::cdiv(t->tail_len_host, kTile) + 1);   // the first row block sees one tile of new tokens
    int64_t ns = ctx->opt_prefill_ctas > 0 ? ctx->opt_prefill_ctas : std::max<int64_t>(1, ctx->n_sm / combos);
    ns = std::min<int64_t>(ns, std::max(1, min_tiles));
    // the partials live in the workspace's partial regions (its head holds the streaming kernel's counters)
    WorkspaceView ws;
    workspace_bytes_for(c, &ws, ctx->workspace);
    const int64_t rows = (int64_t)a.n_layers_launch * t->batch * a.S * c.n_q_heads;
    ns = std::min<int64_t>(ns, std::max<int64_t>(1, ws.n_part_slots * kUnitRows / rows));
    ns = std::min<int64_t>(ns, 64);
    p.n_split = (int)ns;
    p.part_lse = ws.part_lse;
    p.part_o = ws.part_o;
    const int64_t grid = combos * p.n_split;
    CUtensorMap kn_map, vn_map;
    {
        const uint64_t n_tok = (uint64_t)a.n_layers_launch * t->batch * a.S;
        int rc2 = encode_new_rows_map(&kn_map, a.k_new, D, c.n_kv_heads, n_tok);
        if (!rc2) rc2 = encode_new_rows_map(&vn_map, a.v_new, D, c.n_kv_heads, n_tok);
        if (rc2) return rc2;
    }
    int rc = fail(MATKV_E_INVALID_ARG, "tensor-core prefill: unsupported head_dim %d / group %d", D, G);
    if (t->has_fp8) {
#define MATKV_CASE8(GG) \
        if (D == 128 && G == GG) rc = launch_k3<128, GG, 1, true>(p, kn_map, vn_map, (int)grid, stream);
        MATKV_CASE8(1) MATKV_CASE8(2) MATKV_CASE8(4) MATKV_CASE8(8)
#undef MATKV_CASE8
        if (rc) return rc;
        if (p.n_split > 1)
            return launch_lse_combine(ctx, (int32_t)rows, p.n_split, D, p.part_o, p.part_lse, a.out, a.lse_out, stream);
        return MATKV_OK;
    }
#define MATKV_CASE(DD, GG) \
    if (D == DD && G == GG) rc = nblk == 2 ? launch_k3<DD, GG, 2>(p, kn_map, vn_map, (int)grid, stream) : launch_k3<DD, GG, 1>(p, kn_map, vn_map, (int)grid, stream);
    MATKV_CASE(128, 1) MATKV_CASE(128, 2) MATKV_CASE(128, 4) MATKV_CASE(128, 8)
    MATKV_CASE(64, 1) MATKV_CASE(64, 2) MATKV_CASE(64, 4) MATKV_CASE(64, 8)
#undef MATKV_CASE
    if (rc) return rc;
    if (p.n_split > 1)
        return launch_lse_combine(ctx, (int32_t)rows, p.n_split, D, p.part_o, p.part_lse, a.out, a.lse_out, stream);
    return MATKV_OK;
}

}  // namespace matkv
