// Compressed chunk store: a materialised chunk kept on the host (or in a file) as e4m3 codes with one
// power-of-two scale per block of 64 tokens of a (layer, K or V, KV head) slab, expanded to the ordinary
// bf16 chunk blob while it is staged into HBM.  The paper names KV compression as the lever on the storage
// cost of materialised KVs (its discussion of total cost of ownership) and loading as the cost that
// replaces prefill; this halves the bytes on storage and on the host-to-device link.  Attention itself
// still reads bf16 from HBM: every value a code stands for, value(code) * 2^e, is a bf16 number, so the
// expansion is exact and the attention kernels are unchanged.
//
// Blob layout: codes [L][2][Hkv][n_tokens][D] (one byte each), then, at the next multiple of 256 bytes,
// exponents [L][2][Hkv][ceil(n_tokens / 64)] (int8).
#include <cuda_fp8.h>
#include <cuda_runtime.h>

#include <algorithm>

#include "matkv_internal.h"

namespace matkv {

static size_t up256(size_t x) { return (x + 255) / 256 * 256; }

size_t fp8_codes_bytes(const matkv_config &c, int32_t n_tokens) {
    return (size_t)c.n_layers * 2 * c.n_kv_heads * (size_t)n_tokens * c.head_dim;
}
size_t fp8_blob_bytes(const matkv_config &c, int32_t n_tokens) {
    return up256(fp8_codes_bytes(c, n_tokens)) + up256((size_t)c.n_layers * 2 * c.n_kv_heads * ((n_tokens + 63) / 64));
}

// ---- quantiser: one CTA per (slab, 64-token block) -------------------------------------------------------
// e = the smallest integer with amax * 2^-e <= 448 = 1.75 * 2^8 (0 for an all-zero block, clamped to
// [-127, 127]), read off the bf16 bits of amax; code = e4m3 nearest to x * 2^-e, ties to even, and a zero
// carries no sign.  Inputs must be finite.
__global__ void __launch_bounds__(256) k_quantize_fp8(const uint16_t *__restrict__ blob, uint8_t *__restrict__ codes,
                                                      int8_t *__restrict__ exps, int32_t n_tokens, int32_t D, int32_t nb) {
    __shared__ uint32_t s_max[8];
    __shared__ int s_e;
    const int64_t slab = blockIdx.y;
    const int b = blockIdx.x;
    const int t0 = b * 64, nt = min(64, n_tokens - t0);
    const int64_t off = (slab * n_tokens + t0) * D;
    const int n_el = nt * D;
    uint32_t m = 0;
    for (int i = threadIdx.x; i < n_el; i += blockDim.x) m = max(m, (uint32_t)(blob[off + i] & 0x7fffu));  // |x| orders like its bits
#pragma unroll
    for (int o = 16; o; o >>= 1) m = max(m, __shfl_xor_sync(0xffffffffu, m, o));
    if ((threadIdx.x & 31) == 0) s_max[threadIdx.x >> 5] = m;
    __syncthreads();
    if (threadIdx.x == 0) {
        uint32_t a = 0;
        for (int w = 0; w < (int)(blockDim.x >> 5); ++w) a = max(a, s_max[w]);
        int e = 0;
        if (a != 0) {
            const int E = (int)(a >> 7), frac = (int)(a & 0x7f);
            e = E == 0 ? -127 : (E - 127) - 8 + (frac > 0x60 ? 1 : 0);  // amax = (1 + frac/128) * 2^(E-127); 1.75 = 1 + 0x60/128
            e = max(-127, min(127, e));
        }
        s_e = e;
        exps[slab * nb + b] = (int8_t)e;
    }
    __syncthreads();
    const int e = s_e;
    for (int i = threadIdx.x; i < n_el; i += blockDim.x) {
        const float x = __uint_as_float((uint32_t)blob[off + i] << 16);
        uint8_t c = (uint8_t)__nv_cvt_float_to_fp8(ldexpf(x, -e), __NV_SATFINITE, __NV_E4M3);  // exact scaling, then round to nearest even
        if ((c & 0x7f) == 0) c = 0;
        codes[off + i] = c;
    }
}

// ---- expanding copy: compressed blob (pinned host memory or device memory) -> bf16 blob in HBM -----------
// A few small CTAs, like the plain staging copy kernel: they sit beside the decode CTAs and keep the loads
// over the link in flight.  The exponents (a few KB) are first brought into shared memory by every CTA.
__global__ void __launch_bounds__(128) k_stage_expand_fp8(const uint4 *__restrict__ codes, const int8_t *__restrict__ exps,
                                                          uint4 *__restrict__ out, int64_t n_vec, int32_t vec_per_slab,
                                                          int32_t vec_per_block, int32_t nb, int32_t n_exps) {
    extern __shared__ __align__(16) int8_t s_exps[];
    // 16 bytes per load: the exponent area is padded to a multiple of 256 bytes, and every load crosses the link
    for (int i = threadIdx.x; i < (n_exps + 15) / 16; i += blockDim.x) ((uint4 *)s_exps)[i] = __ldcs((const uint4 *)exps + i);
    __syncthreads();
    const int64_t stride = (int64_t)gridDim.x * blockDim.x;
    for (int64_t i0 = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i0 < n_vec; i0 += 8 * stride) {
        uint4 v[8];   // eight 16-byte loads in flight per thread: the link's latency is microseconds
#pragma unroll
        for (int k = 0; k < 8; ++k)
            if (i0 + k * stride < n_vec) v[k] = __ldcs(codes + i0 + k * stride);
#pragma unroll
        for (int k = 0; k < 8; ++k) {
            const int64_t i = i0 + k * stride;   // 16 codes: never across a block, a block is a multiple of 16 codes
            if (i >= n_vec) break;
            const int64_t slab = i / vec_per_slab;
            const int blk = (int)((i % vec_per_slab) / vec_per_block);
            const int e = s_exps[slab * nb + blk];
            const float scale = __uint_as_float(e > -127 ? (uint32_t)(e + 127) << 23 : 0x00400000u);  // 2^e (2^-127 is a subnormal float)
            const uint32_t w[4] = {v[k].x, v[k].y, v[k].z, v[k].w};
            uint32_t o[8];
#pragma unroll
            for (int j = 0; j < 4; ++j) {
#pragma unroll
                for (int h = 0; h < 2; ++h) {
                    const uint32_t c0 = (w[j] >> (16 * h)) & 0xffu, c1 = (w[j] >> (16 * h + 8)) & 0xffu;
                    // the code's 7 magnitude bits sit where a float keeps its low exponent bits and top mantissa bits:
                    // that float is value(code) * 2^-120, subnormal codes included
                    const float f0 = __uint_as_float(((c0 & 0x80u) << 24) | ((c0 & 0x7fu) << 20)) * 0x1p120f * scale;
                    const float f1 = __uint_as_float(((c1 & 0x80u) << 24) | ((c1 & 0x7fu) << 20)) * 0x1p120f * scale;
                    __nv_bfloat162 p = __floats2bfloat162_rn(f0, f1);
                    o[2 * j + h] = *reinterpret_cast<uint32_t *>(&p);
                }
            }
            out[2 * i] = make_uint4(o[0], o[1], o[2], o[3]);
            out[2 * i + 1] = make_uint4(o[4], o[5], o[6], o[7]);
        }
    }
}


// ---- the HBM-resident compressed form (read by the streaming attention kernel without expansion) -----------
// nb = ceil(n_tokens / 64) blocks per (layer, KV head); three regions, each starting at a multiple of 256 bytes:
//   K codes   [L][Hkv][nb * 64][D]      token rows of D bytes (rows past n_tokens are zero)
//   V codes   [L][Hkv][nb][D][64]       per block transposed: row d holds the block's 64 tokens (the P V product wants
//                                       consecutive tokens of one dimension side by side)
//   exponents [L][Hkv][nb] x 16 bytes   byte 0 = K block exponent, byte 1 = V block exponent (a 16-byte record so that
//                                       one bulk copy brings it in beside the tile)
size_t fp8_resident_bytes(const matkv_config &c, int32_t n_tokens) {
    const size_t nb = (size_t)(n_tokens + 63) / 64, slabs = (size_t)c.n_layers * c.n_kv_heads;
    return 2 * up256(slabs * nb * 64 * c.head_dim) + up256(slabs * nb * 16);
}

// one CTA per (layer, KV head, block): store form -> resident form
__global__ void __launch_bounds__(256) k_relayout_fp8(const uint8_t *__restrict__ codes, const int8_t *__restrict__ exps,
                                                      uint8_t *__restrict__ k_out, uint8_t *__restrict__ v_out, uint8_t *__restrict__ e_out,
                                                      int32_t n_tokens, int32_t D, int32_t Hkv, int32_t nb) {
    __shared__ __align__(16) uint8_t tile[64 * 129];   // V block, rows padded to 129 bytes for the transposed read
    const int b = blockIdx.x, lh = blockIdx.y;          // block, layer * Hkv + head
    const int l = lh / Hkv, h = lh % Hkv;
    const int t0 = b * 64, nt = min(64, n_tokens - t0);
    const int64_t k_slab = ((int64_t)(l * 2) * Hkv + h), v_slab = ((int64_t)(l * 2 + 1) * Hkv + h);
    // K rows: straight copy, 16 bytes at a time (D is a multiple of 16), zero rows past the end
    const uint4 *ksrc = (const uint4 *)(codes + (k_slab * n_tokens + t0) * D);
    uint4 *kdst = (uint4 *)(k_out + (((int64_t)lh * nb + b) * 64) * D);
    const int vec_row = D / 16;
    for (int i = threadIdx.x; i < 64 * vec_row; i += blockDim.x)
        kdst[i] = i / vec_row < nt ? __ldcs(ksrc + i) : make_uint4(0u, 0u, 0u, 0u);
    // V block through shared memory, transposed on the way out
    const uint4 *vsrc = (const uint4 *)(codes + (v_slab * n_tokens + t0) * D);
    for (int i = threadIdx.x; i < 64 * vec_row; i += blockDim.x) {
        const int t = i / vec_row, c = i % vec_row;
        const uint4 v = t < nt ? __ldcs(vsrc + i) : make_uint4(0u, 0u, 0u, 0u);
        const uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
        for (int j = 0; j < 16; ++j) tile[t * 129 + c * 16 + j] = (uint8_t)(w[j >> 2] >> (8 * (j & 3)));
    }
    __syncthreads();
    uint8_t *vdst = v_out + (((int64_t)lh * nb + b) * D) * 64;
    for (int i = threadIdx.x; i < D * 16; i += blockDim.x) {   // 4 tokens (one 32-bit word) of one dimension per step
        const int d = i / 16, tq = (i % 16) * 4;
        const uint32_t w = (uint32_t)tile[tq * 129 + d] | ((uint32_t)tile[(tq + 1) * 129 + d] << 8) |
                           ((uint32_t)tile[(tq + 2) * 129 + d] << 16) | ((uint32_t)tile[(tq + 3) * 129 + d] << 24);
        *(uint32_t *)(vdst + d * 64 + tq) = w;
    }
    if (threadIdx.x < 4) {
        uint32_t w = 0;
        if (threadIdx.x == 0)
            w = (uint32_t)(uint8_t)exps[k_slab * nb + b] | ((uint32_t)(uint8_t)exps[v_slab * nb + b] << 8);
        ((uint32_t *)(e_out + ((int64_t)lh * nb + b) * 16))[threadIdx.x] = w;
    }
}

int launch_stage_relayout_fp8(matkv_ctx *ctx, const void *src_fp8, void *dev_dst, int32_t n_tokens, cudaStream_t stream) {
    const matkv_config &c = ctx->cfg;
    if (c.head_dim != 128) return fail(MATKV_E_INVALID_ARG, "compressed-resident chunks need head_dim 128");
    const int nb = (n_tokens + 63) / 64;
    const int64_t lh = (int64_t)c.n_layers * c.n_kv_heads;
    if (lh > 65535) return fail(MATKV_E_CAPACITY, "too many (layer, head) slabs for one re-layout launch");
    const uint8_t *codes = (const uint8_t *)src_fp8;
    const int8_t *exps = (const int8_t *)(codes + up256(fp8_codes_bytes(c, n_tokens)));
    const size_t region = up256((size_t)lh * nb * 64 * c.head_dim);
    uint8_t *k_out = (uint8_t *)dev_dst, *v_out = k_out + region, *e_out = v_out + region;
    k_relayout_fp8<<<dim3(nb, (unsigned)lh), 256, 0, stream>>>(codes, exps, k_out, v_out, e_out, n_tokens, c.head_dim, c.n_kv_heads, nb);
    MATKV_CUDA(cudaGetLastError());
    return MATKV_OK;
}

int launch_quantize_fp8(matkv_ctx *ctx, const void *dev_blob, int32_t n_tokens, void *dev_fp8, cudaStream_t stream) {
    const matkv_config &c = ctx->cfg;
    const int nb = (n_tokens + 63) / 64;
    const int64_t n_slab = (int64_t)c.n_layers * 2 * c.n_kv_heads;
    if (n_slab > 65535) return fail(MATKV_E_CAPACITY, "too many (layer, head) slabs for one quantiser launch");
    uint8_t *codes = (uint8_t *)dev_fp8;
    int8_t *exps = (int8_t *)(codes + up256(fp8_codes_bytes(c, n_tokens)));
    k_quantize_fp8<<<dim3(nb, (unsigned)n_slab), 256, 0, stream>>>((const uint16_t *)dev_blob, codes, exps, n_tokens, c.head_dim, nb);
    MATKV_CUDA(cudaGetLastError());
    return MATKV_OK;
}

int launch_stage_expand_fp8(matkv_ctx *ctx, const void *src_fp8, void *dev_dst, int32_t n_tokens, int n_ctas, cudaStream_t stream) {
    const matkv_config &c = ctx->cfg;
    const int nb = (n_tokens + 63) / 64;
    const int64_t n_slab = (int64_t)c.n_layers * 2 * c.n_kv_heads;
    const int64_t n_exps = n_slab * nb;
    if (n_exps > 200 * 1024) return fail(MATKV_E_CAPACITY, "%lld block exponents do not fit the expanding copy's shared memory", (long long)n_exps);
    const uint8_t *codes = (const uint8_t *)src_fp8;
    const int8_t *exps = (const int8_t *)(codes + up256(fp8_codes_bytes(c, n_tokens)));
    const int64_t n_vec = (int64_t)(fp8_codes_bytes(c, n_tokens) / 16);
    const int32_t vec_per_slab = (int32_t)((int64_t)n_tokens * c.head_dim / 16);
    const int32_t vec_per_block = 64 * c.head_dim / 16;
    static PerDeviceOnce configured;
    int once_dev;
    if (configured.need(&once_dev)) {
        MATKV_CUDA(cudaFuncSetAttribute(k_stage_expand_fp8, cudaFuncAttributeMaxDynamicSharedMemorySize, 200 * 1024));
        configured.mark(once_dev);
    }
    k_stage_expand_fp8<<<n_ctas, 128, (size_t)((n_exps + 15) / 16 * 16), stream>>>((const uint4 *)codes, exps, (uint4 *)dev_dst, n_vec, vec_per_slab,
                                                                                 vec_per_block, nb, (int32_t)n_exps);
    MATKV_CUDA(cudaGetLastError());
    return MATKV_OK;
}

}  // namespace matkv
