// Pieces shared by the streaming attention kernels: constants, PTX wrappers (mbarrier, TMA, ldmatrix, mma),
// the bounded waits, the swizzle address helper and the one-warp log-sum-exp merge.
#pragma once
#include <cuda_runtime.h>
#include <cuda_bf16.h>
#include <math_constants.h>

#include "matkv_internal.h"

namespace matkv {

constexpr int kCW = 7;                          // consumer warps (+1 producer warp)
constexpr int kThreads = (kCW + 1) * 32;
constexpr int kItemRows = 16;                   // tokens per consumer work item
constexpr int kItems = kTile / kItemRows;       // work items per tile
constexpr int kMaxDynSmem = 232448;             // 227 KB opt-in limit per CTA on sm_100
constexpr long long kWaitCycles = 2000000000LL; // bounded waits give up after about a second
constexpr float kLog2e = 1.4426950408889634f;
constexpr float kLn2 = 0.6931471805599453f;
constexpr uint32_t kTagF8 = 0x0080u;            // tile tag: a tile of e4m3 codes (compressed-resident chunk)
constexpr uint32_t kTagNew = 0x8000u;           // tile tag: a tile of the call's new tokens (bits 8..14: its index)

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
// A consumer's wait for fill number `want` of a ring stage.  Warps take work items round-robin, so a
// warp can reach a stage whose PREVIOUS fill is still in flight, and the one-bit phase of an mbarrier
// cannot tell "fill n-1 incomplete" from "fill n complete".  The producer therefore publishes the fill
// number of a stage (upper half of the stage's tag word) before it issues the copies, which it does
// only after the stage's previous fill was consumed and released; once the consumer sees its number
// there, the parity test is unambiguous.  Returns the tag word, or 0 after the bounded wait ran out.
__device__ __forceinline__ uint32_t stage_wait(const volatile uint32_t *tag, uint32_t want, uint32_t bar, uint32_t parity,
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
// TMA: one 64-column x kTile-row box of a [rows][D] bf16 tensor, starting at column x (a multiple of
// 64: 128 bytes, so the 16-byte rule on the innermost coordinate holds) and row y.
__device__ __forceinline__ void tma_load_2d(uint32_t dst, const CUtensorMap *map, int32_t x, int32_t y, uint32_t bar) {
    asm volatile(
        "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];" ::"r"(dst),
        "l"(map), "r"(x), "r"(y), "r"(bar)
        : "memory");
}
// the same with an L2 eviction policy (from createpolicy)
__device__ __forceinline__ void tma_load_2d_hint(uint32_t dst, const CUtensorMap *map, int32_t x, int32_t y, uint32_t bar, uint64_t policy) {
    asm volatile(
        "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes.L2::cache_hint [%0], [%1, {%2, %3}], [%4], %5;" ::"r"(dst),
        "l"(map), "r"(x), "r"(y), "r"(bar), "l"(policy)
        : "memory");
}
__device__ __forceinline__ uint64_t l2_policy_evict_first() {
    uint64_t pol;
    asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(pol));
    return pol;
}
__device__ __forceinline__ uint64_t l2_policy_evict_normal() {
    uint64_t pol;
    asm volatile("createpolicy.fractional.L2::evict_normal.b64 %0, 1.0;" : "=l"(pol));
    return pol;
}
__device__ __forceinline__ void tma_load_3d(uint32_t dst, const CUtensorMap *map, int32_t x, int32_t y, int32_t z, uint32_t bar) {
    asm volatile(
        "cp.async.bulk.tensor.3d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3, %4}], [%5];" ::"r"(dst),
        "l"(map), "r"(x), "r"(y), "r"(z), "r"(bar)
        : "memory");
}
__device__ __forceinline__ void consumer_bar() { asm volatile("bar.sync 1, %0;" ::"n"(kCW * 32) : "memory"); }
__device__ __forceinline__ float fast_exp2(float x) {
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}
__device__ __forceinline__ void ldsm_x4(uint32_t addr, uint32_t (&r)[4]) {
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0, %1, %2, %3}, [%4];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3])
                 : "r"(addr));
}
__device__ __forceinline__ void ldsm_x4_trans(uint32_t addr, uint32_t (&r)[4]) {
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0, %1, %2, %3}, [%4];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3])
                 : "r"(addr));
}
// D (16x8, fp32) += A (16x16, bf16, row) * B (16x8, bf16, col)
__device__ __forceinline__ void mma_bf16(float (&d)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3, uint32_t b0,
                                         uint32_t b1) {
    asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0, %1, %2, %3}, {%4, %5, %6, %7}, {%8, %9}, {%0, %1, %2, %3};"
                 : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
                 : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}
// the same with fp16 operands (the compressed-chunk path: e4m3 codes convert to fp16 with one instruction per pair)
__device__ __forceinline__ void mma_f16(float (&d)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3, uint32_t b0,
                                        uint32_t b1) {
    asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.f16.f16.f32 {%0, %1, %2, %3}, {%4, %5, %6, %7}, {%8, %9}, {%0, %1, %2, %3};"
                 : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
                 : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}
// four e4m3 codes (one 32-bit word) -> two fp16 pairs: codes 0,1 and codes 2,3 (exact)
__device__ __forceinline__ void cvt_e4m3x4_f16(uint32_t w, uint32_t &lo, uint32_t &hi) {
    asm("{\n .reg .b16 a, b;\n mov.b32 {a, b}, %2;\n cvt.rn.f16x2.e4m3x2 %0, a;\n cvt.rn.f16x2.e4m3x2 %1, b;\n}" : "=r"(lo), "=r"(hi) : "r"(w));
}
__device__ __forceinline__ uint32_t pack_f16(float lo, float hi) {
    uint32_t r;
    asm("cvt.rn.f16x2.f32 %0, %2, %1;" : "=r"(r) : "f"(lo), "f"(hi));   // the first source lands in the upper half
    return r;
}
__device__ __forceinline__ float f16_lo(uint32_t w) {
    float f;
    asm("{\n .reg .b16 a, b;\n mov.b32 {a, b}, %1;\n cvt.f32.f16 %0, a;\n}" : "=f"(f) : "r"(w));
    return f;
}
__device__ __forceinline__ float f16_hi(uint32_t w) {
    float f;
    asm("{\n .reg .b16 a, b;\n mov.b32 {a, b}, %1;\n cvt.f32.f16 %0, b;\n}" : "=f"(f) : "r"(w));
    return f;
}
// untiled bulk copy global -> shared with mbarrier completion (both addresses 16-byte aligned, size a multiple of 16)
__device__ __forceinline__ void bulk_load(uint32_t dst, const void *src, uint32_t bytes, uint32_t bar) {
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(dst), "l"(src), "r"(bytes),
                 "r"(bar)
                 : "memory");
}
__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi) {
    __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
    return *reinterpret_cast<uint32_t *>(&v);
}
__device__ __forceinline__ float bf_lo(uint32_t w) { return __uint_as_float(w << 16); }
__device__ __forceinline__ float bf_hi(uint32_t w) { return __uint_as_float(w & 0xffff0000u); }

__host__ __device__ __forceinline__ int ceil_div(int a, int b) { return (a + b - 1) / b; }

// ---- K2 core: merge P partial attentions of one row with one warp -----------------------------------
// o_parts: part p at o_parts + p*o_stride (D floats, normalised inside the part); lse natural log.
static __device__ void combine_warp(const float *o_parts, int64_t o_stride, const float *lse_parts, int64_t lse_stride, int P,
                             int D, __nv_bfloat16 *out, float *lse_out) {
    const int lane = threadIdx.x & 31;
    const int dpl = D >> 5;  // every lane owns D/32 consecutive dims
    if (P <= 32 && dpl == 4) {
        // common case (at most 32 parts, D = 128): the first 16 parts' rows and one part's lse per lane are requested
        // together (one round trip to L2 for up to 16 parts, two beyond); the weights travel by shuffle
        float4 v[16];
#pragma unroll
        for (int i = 0; i < 16; ++i)
            v[i] = i < P ? __ldcg((const float4 *)(o_parts + i * o_stride + lane * 4)) : make_float4(0.f, 0.f, 0.f, 0.f);
        const float lse_l = lane < P ? __ldcg(lse_parts + lane * lse_stride) : -CUDART_INF_F;
        float m = lse_l;
#pragma unroll
        for (int off = 16; off; off >>= 1) m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, off));
        if (m == -CUDART_INF_F) {  // no part saw any key
            *(uint2 *)(out + lane * 4) = make_uint2(0u, 0u);
            if (lse_out && lane == 0) *lse_out = -CUDART_INF_F;
            return;
        }
        float w_l = lse_l == -CUDART_INF_F ? 0.f : exp2f((lse_l - m) * kLog2e);
        float z = w_l;
#pragma unroll
        for (int off = 16; off; off >>= 1) z += __shfl_xor_sync(0xffffffffu, z, off);
        w_l /= z;
        float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
        for (int p0 = 0; p0 < P; p0 += 16) {
            if (p0) {
#pragma unroll
                for (int i = 0; i < 16; ++i)
                    v[i] = p0 + i < P ? __ldcg((const float4 *)(o_parts + (p0 + i) * o_stride + lane * 4)) : make_float4(0.f, 0.f, 0.f, 0.f);
            }
#pragma unroll
            for (int i = 0; i < 16; ++i) {
                const float w = __shfl_sync(0xffffffffu, w_l, (p0 + i) & 31);
                if (w == 0.f) continue;   // an empty part carries no weight, whatever its row holds
                acc.x = fmaf(w, v[i].x, acc.x); acc.y = fmaf(w, v[i].y, acc.y);
                acc.z = fmaf(w, v[i].z, acc.z); acc.w = fmaf(w, v[i].w, acc.w);
            }
        }
        __nv_bfloat162 lo = __floats2bfloat162_rn(acc.x, acc.y), hi = __floats2bfloat162_rn(acc.z, acc.w);
        *(uint2 *)(out + lane * 4) = make_uint2(*reinterpret_cast<uint32_t *>(&lo), *reinterpret_cast<uint32_t *>(&hi));
        if (lse_out && lane == 0) *lse_out = m + logf(z);
        return;
    }
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
    // the weights of 32 parts at a time sit one per lane and are broadcast by shuffle, so the loads of the
    // parts' rows are independent and stay in flight together
    float acc[8] = {0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f};
    for (int p0 = 0; p0 < P; p0 += 32) {
        const float w_mine = p0 + lane < P ? exp2f((__ldcg(lse_parts + (p0 + lane) * lse_stride) - lse) * kLog2e) : 0.f;
        const int np = min(32, P - p0);
#pragma unroll 4
        for (int pp = 0; pp < np; ++pp) {
            const float w = __shfl_sync(0xffffffffu, w_mine, pp);
            if (w == 0.f) continue;   // an empty part carries no weight, whatever its row holds
            const float *row = o_parts + (p0 + pp) * o_stride + lane * dpl;
            if (dpl == 4) {
                const float4 v = __ldcg((const float4 *)row);
                acc[0] = fmaf(w, v.x, acc[0]); acc[1] = fmaf(w, v.y, acc[1]);
                acc[2] = fmaf(w, v.z, acc[2]); acc[3] = fmaf(w, v.w, acc[3]);
            } else if (dpl == 2) {
                const float2 v = __ldcg((const float2 *)row);
                acc[0] = fmaf(w, v.x, acc[0]); acc[1] = fmaf(w, v.y, acc[1]);
            } else {
                for (int i = 0; i < dpl; ++i) acc[i] = fmaf(w, __ldcg(row + i), acc[i]);
            }
        }
    }
    for (int i = 0; i < dpl; ++i) out[lane * dpl + i] = __float2bfloat16(acc[i]);
    if (lse_out && lane == 0) *lse_out = lse;
}

// byte offset of 16-byte chunk c of row r inside one 128-byte-swizzled box
__device__ __forceinline__ uint32_t swz(int r, int c) { return (uint32_t)(r * 128 + ((c ^ (r & 7)) << 4)); }

}  // namespace matkv
