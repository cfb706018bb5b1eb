// Rotary mode: rotate the call's q and k_new at their positions before attention.
//
// The stored chunk K is never touched (each chunk was materialised alone, already rotated for
// positions 0..len-1).  Only the tokens that arrive with a call are rotated: token i of request b sits
// at position pos_base_b + tail_len_b + i, where pos_base_b is the request's position base from the
// table (by default the sum of its chunk lengths: the query continues after the documents).
// Rotate-half pairing (d, d + D/2), angle = position * theta^(-2d/D).  The angle and its sine and
// cosine are evaluated in fp64 and the result is rounded once to bf16, which is what a model would
// have handed to the attention path; the volume is tiny (a few thousand vectors per call).
#include "matkv_internal.h"

namespace matkv {

__global__ void k_rope(const __nv_bfloat16 *__restrict__ src, __nv_bfloat16 *__restrict__ dst, const DevReq *__restrict__ reqs,
                       const int32_t *__restrict__ tail_len, int32_t n_layers, int32_t B, int32_t S, int32_t H, int32_t D,
                       int64_t s_l, int64_t s_b, int64_t s_s, double theta) {
    // one thread per (layer, request, token, head, pair)
    const int half = D / 2;
    const int64_t n = (int64_t)n_layers * B * S * H * half;
    for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < n; i += (int64_t)gridDim.x * blockDim.x) {
        int64_t r = i;
        const int d = (int)(r % half); r /= half;
        const int h = (int)(r % H); r /= H;
        const int tok = (int)(r % S); r /= S;
        const int b = (int)(r % B); r /= B;
        const int l = (int)r;
        const int64_t off = l * s_l + b * s_b + tok * s_s + (int64_t)h * D + d;
        const double pos = (double)(reqs[b].pos_base + tail_len[b] + tok);
        const double ang = pos * pow(theta, -2.0 * (double)d / (double)D);
        double sn, cs;
        sincos(ang, &sn, &cs);
        const double x = (double)__bfloat162float(src[off]), y = (double)__bfloat162float(src[off + half]);
        dst[off] = __float2bfloat16_rn(__double2float_rn(x * cs - y * sn));
        dst[off + half] = __float2bfloat16_rn(__double2float_rn(y * cs + x * sn));
    }
}

// Rotates a.q and a.k_new into the context's scratch (behind the split-KV workspace) and points the
// arguments at the rotated copies.  v_new is never rotated.
int launch_rope(matkv_ctx *ctx, matkv_table *t, AttendArgs &a, cudaStream_t stream) {
    const matkv_config &c = ctx->cfg;
    const size_t base = workspace_bytes_for(c, nullptr, nullptr) - rope_scratch_bytes(c);
    const int64_t nq = (int64_t)a.n_layers_launch * t->batch * a.S * c.n_q_heads * c.head_dim;
    const int64_t nk = (int64_t)a.n_layers_launch * t->batch * a.S * c.n_kv_heads * c.head_dim;
    if ((size_t)(nq + nk) * sizeof(__nv_bfloat16) > rope_scratch_bytes(c))
        return fail(MATKV_E_CAPACITY, "rotary scratch too small for this call");
    // the scratch holds dense copies, so the strides are the dense ones of the call's shape
    __nv_bfloat16 *q_rot = (__nv_bfloat16 *)((char *)ctx->workspace + base);
    __nv_bfloat16 *k_rot = q_rot + nq;
    const int threads = 256;
    auto blocks = [&](int64_t n) { return (int)std::min<int64_t>((n / 2 + threads - 1) / threads, 4 * (int64_t)ctx->n_sm); };
    k_rope<<<blocks(nq), threads, 0, stream>>>(a.q, q_rot, t->d_reqs, t->d_tail_len, a.n_layers_launch, t->batch, a.S,
                                             c.n_q_heads, c.head_dim, a.q_sl, a.q_sb, a.q_ss, (double)c.rope_theta);
    k_rope<<<blocks(nk), threads, 0, stream>>>(a.k_new, k_rot, t->d_reqs, t->d_tail_len, a.n_layers_launch, t->batch, a.S,
                                             c.n_kv_heads, c.head_dim, a.kn_sl, a.kn_sb, a.kn_ss, (double)c.rope_theta);
    MATKV_CUDA(cudaGetLastError());
    a.q = q_rot;
    a.k_new = k_rot;
    return MATKV_OK;
}

}  // namespace matkv
