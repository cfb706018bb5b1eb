// Host side of the C ABI: context, chunk registry, staging, chunk table, status.
// No attention arithmetic lives here; the kernels and their launchers are in the other files.
#include <stdarg.h>
#include <stdio.h>
#include <string.h>

#include <algorithm>
#include <cmath>

#include "matkv_internal.h"

namespace matkv {

static thread_local char g_err[512] = "";

int fail(int code, const char *fmt, ...) {
    va_list ap;
    va_start(ap, fmt);
    vsnprintf(g_err, sizeof g_err, fmt, ap);
    va_end(ap);
    return code;
}

int cuda_fail(cudaError_t e, const char *what) {
    return fail(MATKV_E_CUDA, "CUDA error %d (%s) in %s", (int)e, cudaGetErrorString(e), what);
}

static size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

typedef CUresult (*EncodeFn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *, const cuuint64_t *,
                             const cuuint32_t *, const cuuint32_t *, CUtensorMapInterleave, CUtensorMapSwizzle,
                             CUtensorMapL2promotion, CUtensorMapFloatOOBfill);
static EncodeFn tensor_map_encoder() {
    static EncodeFn fn = nullptr;
    if (!fn) {
        void *p = nullptr;
        cudaDriverEntryPointQueryResult q;
        cudaError_t e = cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q);
        if (e == cudaSuccess && q == cudaDriverEntryPointSuccess) fn = (EncodeFn)p;
    }
    return fn;
}

int encode_rows_map(CUtensorMap *out, const void *base, int D, uint64_t rows) {
    EncodeFn fn = tensor_map_encoder();
    if (!fn) return fail(MATKV_E_CUDA, "cuTensorMapEncodeTiled is not available from this driver");
    const cuuint64_t gdim[2] = {(cuuint64_t)D, (cuuint64_t)rows};
    const cuuint64_t gstride[1] = {(cuuint64_t)D * 2};
    const cuuint32_t box[2] = {64, (cuuint32_t)kTile};
    const cuuint32_t estride[2] = {1, 1};
    CUresult r = fn(out, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void *>(base), gdim, gstride, box, estride,
                    CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                    CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) return fail(MATKV_E_CUDA, "cuTensorMapEncodeTiled failed with %d", (int)r);
    return MATKV_OK;
}

// Tensor maps of a compressed-resident chunk (head_dim 128): [0] K codes as rows of 128 bytes, box 64 rows, 128-byte
// swizzle; [1] V codes, per block transposed, as rows of 64 bytes (one dimension's 64 tokens), box 128 rows, 64-byte swizzle.
int encode_fp8_maps(CUtensorMap *out2, const void *dev_resident, const matkv_config &c, int32_t n_tokens) {
    EncodeFn fn = tensor_map_encoder();
    if (!fn) return fail(MATKV_E_CUDA, "cuTensorMapEncodeTiled is not available from this driver");
    const uint64_t nb = (uint64_t)(n_tokens + 63) / 64, lh = (uint64_t)c.n_layers * c.n_kv_heads;
    const size_t region = align_up((size_t)(lh * nb * 64 * c.head_dim), 256);
    const cuuint32_t estride[2] = {1, 1};
    {
        const cuuint64_t gdim[2] = {(cuuint64_t)c.head_dim, (cuuint64_t)(lh * nb * 64)};
        const cuuint64_t gstride[1] = {(cuuint64_t)c.head_dim};
        const cuuint32_t box[2] = {128, 64};
        CUresult r = fn(&out2[0], CU_TENSOR_MAP_DATA_TYPE_UINT8, 2, const_cast<void *>(dev_resident), gdim, gstride, box, estride,
                        CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                        CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
        if (r != CUDA_SUCCESS) return fail(MATKV_E_CUDA, "cuTensorMapEncodeTiled (K codes) failed with %d", (int)r);
    }
    {
        const cuuint64_t gdim[2] = {64, (cuuint64_t)(lh * nb * c.head_dim)};
        const cuuint64_t gstride[1] = {64};
        const cuuint32_t box[2] = {64, 128};
        CUresult r = fn(&out2[1], CU_TENSOR_MAP_DATA_TYPE_UINT8, 2, (char *)const_cast<void *>(dev_resident) + region, gdim, gstride, box,
                        estride, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_64B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                        CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
        if (r != CUDA_SUCCESS) return fail(MATKV_E_CUDA, "cuTensorMapEncodeTiled (V codes) failed with %d", (int)r);
    }
    return MATKV_OK;
}

int encode_new_rows_map(CUtensorMap *out, const void *base, int D, int Hkv, uint64_t n_tok) {
    EncodeFn fn = tensor_map_encoder();
    if (!fn) return fail(MATKV_E_CUDA, "cuTensorMapEncodeTiled is not available from this driver");
    const cuuint64_t gdim[3] = {(cuuint64_t)D, (cuuint64_t)Hkv, (cuuint64_t)n_tok};
    const cuuint64_t gstride[2] = {(cuuint64_t)D * 2, (cuuint64_t)Hkv * D * 2};
    const cuuint32_t box[3] = {64, 1, (cuuint32_t)kTile};
    const cuuint32_t estride[3] = {1, 1, 1};
    CUresult r = fn(out, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void *>(base), gdim, gstride, box, estride,
                    CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                    CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) return fail(MATKV_E_CUDA, "cuTensorMapEncodeTiled (new rows) failed with %d", (int)r);
    return MATKV_OK;
}

size_t rope_scratch_bytes(const matkv_config &c) {
    if (c.rope_theta == 0.f) return 0;
    const size_t per_tok = (size_t)(c.n_q_heads + c.n_kv_heads) * c.head_dim * sizeof(__nv_bfloat16);
    // the largest call: every layer, up to max_tail tokens per request
    return align_up((size_t)c.n_layers * c.max_batch * c.max_tail_tokens * per_tok, 256);
}

size_t workspace_bytes_for(const matkv_config &c, WorkspaceView *v, void *base) {
    const int64_t G = kUnitRows;
    const int64_t units_decode = (int64_t)c.n_layers * c.max_batch * c.n_kv_heads;
    const int64_t units_prefill = (int64_t)c.max_batch * c.max_tail_tokens * c.n_kv_heads;
    const int64_t n_units = std::max(units_decode, units_prefill);
    const int64_t n_parts = n_units + kMaxGridCtas;
    size_t off = 0;
    const size_t counters_off = off;
    off = align_up(off + sizeof(int32_t) * (size_t)n_units, 256);
    const size_t lse_off = off;
    off = align_up(off + sizeof(float) * (size_t)(n_parts * G), 256);
    const size_t o_off = off;
    off = align_up(off + sizeof(float) * (size_t)(n_parts * G * c.head_dim), 256);
    if (v) {
        char *b = (char *)base;
        v->counters = (int32_t *)(b + counters_off);
        v->part_lse = (float *)(b + lse_off);
        v->part_o = (float *)(b + o_off);
        v->n_counter_slots = n_units;
        v->n_part_slots = n_parts;
    }
    off += rope_scratch_bytes(c);  // rotary mode: the rotated q / k_new of one call sit behind the partials
    return off;
}

static void reap_graveyard(matkv_ctx *ctx, bool force);

}  // namespace matkv

using namespace matkv;

// table images (pinned upload buffer + device copy) are recycled: allocating them per batch costs
// milliseconds (cudaMallocHost and cudaMalloc synchronise).  A freed table's image waits in the context's
// graveyard until the stream work that may still read it has finished, then moves to the context's pool.
static void matkv::reap_graveyard(matkv_ctx *ctx, bool force) {
    auto &v = ctx->image_graves;
    for (size_t i = 0; i < v.size();) {
        bool done = force;
        if (force) cudaEventSynchronize(v[i].ev);
        else done = (cudaEventQuery(v[i].ev) == cudaSuccess);
        if (done) {
            if (force) {
                cudaFreeHost(v[i].h_pinned);
                cudaFree(v[i].d_image);
            } else {
                ctx->image_pool.push_back(PooledImage{v[i].h_pinned, v[i].d_image, v[i].bytes});
            }
            cudaEventDestroy(v[i].ev);
            v[i] = v.back();
            v.pop_back();
        } else {
            ++i;
        }
    }
    if (force) {
        for (auto &im : ctx->image_pool) {
            cudaFreeHost(im.h_pinned);
            cudaFree(im.d_image);
        }
        ctx->image_pool.clear();
    }
}

// A staging call that has been seen complete gives its event back: the chunks it staged no longer need to wait for
// it, so they drop their reference, the event is destroyed and the ticket leaves the map (a failed one leaves its
// number behind).  Called from the query / wait functions and, for every finished ticket, from the next staging call.
static void retire_ticket(matkv_ctx *ctx, std::unordered_map<uint64_t, Ticket>::iterator it) {
    Ticket &tk = it->second;
    for (uint64_t id : tk.chunk_ids) {
        auto c = ctx->chunks.find(id);
        if (c != ctx->chunks.end() && c->second.ticket == it->first) c->second.ready = nullptr;
    }
    if (tk.io_failed && tk.io_failed->host.load(std::memory_order_acquire)) {
        if (ctx->failed_tickets.size() >= 1024) ctx->failed_tickets.erase(ctx->failed_tickets.begin());
        ctx->failed_tickets.push_back(it->first);
    }
    cudaEventDestroy(tk.done);
    ctx->tickets.erase(it);
}

static void retire_finished_tickets(matkv_ctx *ctx) {
    for (auto it = ctx->tickets.begin(); it != ctx->tickets.end();) {
        auto cur = it++;
        if (cudaEventQuery(cur->second.done) == cudaSuccess) retire_ticket(ctx, cur);
        else cudaGetLastError();
    }
}

static size_t blob_bytes(const matkv_config &c, int32_t n_tokens) {
    return (size_t)c.n_layers * 2 * c.n_kv_heads * (size_t)n_tokens * c.head_dim * sizeof(__nv_bfloat16);
}

extern "C" {

const char *matkv_last_error(void) { return g_err; }

int matkv_create(const matkv_config *cfg, matkv_ctx **out) {
    if (!cfg || !out) return fail(MATKV_E_INVALID_ARG, "matkv_create: null argument");
    *out = nullptr;
    if (cfg->n_layers < 1 || cfg->n_q_heads < 1 || cfg->n_kv_heads < 1 || cfg->n_q_heads % cfg->n_kv_heads)
        return fail(MATKV_E_INVALID_ARG, "matkv_create: bad layer/head counts");
    const int G = cfg->n_q_heads / cfg->n_kv_heads;
    if (cfg->head_dim != 64 && cfg->head_dim != 128)
        return fail(MATKV_E_INVALID_ARG, "matkv_create: head_dim must be 64 or 128");
    if (G != 1 && G != 2 && G != 4 && G != 8)
        return fail(MATKV_E_INVALID_ARG, "matkv_create: query heads per KV head must be 1, 2, 4 or 8");
    if (cfg->max_batch < 1 || cfg->max_batch > 1024 || cfg->max_chunks_per_req < 0 || cfg->max_tail_tokens < 1)
        return fail(MATKV_E_INVALID_ARG, "matkv_create: bad capacity");
    if ((int64_t)cfg->max_batch * cfg->n_layers * cfg->n_kv_heads * cfg->max_tail_tokens >= (int64_t)1 << 31)
        return fail(MATKV_E_CAPACITY, "matkv_create: max_batch x layers x KV heads x max_tail_tokens must stay below 2^31 rows");
    if (cfg->softmax_scale < 0.f || cfg->rope_theta < 0.f || cfg->pos_mode < 0 || cfg->pos_mode > 2)
        return fail(MATKV_E_INVALID_ARG, "matkv_create: bad scale / rotary settings");
    int dev = cfg->device;
    if (dev < 0) MATKV_CUDA(cudaGetDevice(&dev));
    DeviceGuard guard(dev);
    cudaDeviceProp prop;
    MATKV_CUDA(cudaGetDeviceProperties(&prop, dev));
    if (prop.major != 10)
        return fail(MATKV_E_CUDA, "matkv_create: device %d is sm_%d%d; this library is built for sm_100a only", dev,
                    prop.major, prop.minor);
    matkv_ctx *ctx = new matkv_ctx();
    ctx->cfg = *cfg;
    ctx->device = dev;
    ctx->cfg.device = dev;
    ctx->scale = cfg->softmax_scale > 0.f ? cfg->softmax_scale : 1.0f / std::sqrt((float)cfg->head_dim);
    ctx->n_sm = prop.multiProcessorCount;
    cudaError_t e = cudaMalloc(&ctx->d_status, 4 * sizeof(int32_t));  // [0] status, [1] probe sink
    if (e == cudaSuccess) e = cudaMemset(ctx->d_status, 0, 4 * sizeof(int32_t));
    if (e != cudaSuccess) {
        delete ctx;
        return cuda_fail(e, "status word");
    }
    *out = ctx;
    return MATKV_OK;
}

int matkv_destroy(matkv_ctx *ctx) {
    if (!ctx) return MATKV_OK;
    DeviceGuard guard(ctx->device);
    cudaDeviceSynchronize();          // pending copies and their host callbacks finish first
    io_engine_destroy(ctx);
    for (auto &kv : ctx->chunks) close_chunk_file(kv.second.file_fd);
    for (matkv_table *t : std::vector<matkv_table *>(ctx->tables)) {
        cudaFreeHost(t->h_pinned);
        cudaFree(t->d_image);
        delete t;
    }
    ctx->tables.clear();
    reap_graveyard(ctx, true);
    for (auto &kv : ctx->tickets) cudaEventDestroy(kv.second.done);
    for (auto &kv : ctx->regions) {
        if (kv.second->last_use) cudaEventDestroy(kv.second->last_use);
        delete kv.second;
    }
    cudaFree(ctx->d_status);
    delete ctx;
    return MATKV_OK;
}

int matkv_set_option(matkv_ctx *ctx, int32_t option, int64_t value) {
    if (!ctx) return fail(MATKV_E_INVALID_ARG, "matkv_set_option: null context");
    switch (option) {
        case MATKV_OPT_DECODE_CTAS:
            if (value < 0 || value > kMaxGridCtas) return fail(MATKV_E_INVALID_ARG, "decode CTAs must be 0..%d", kMaxGridCtas);
            ctx->opt_decode_ctas = value;
            return MATKV_OK;
        case MATKV_OPT_PREFILL_IMPL:
            if (value < 0 || value > 3) return fail(MATKV_E_INVALID_ARG, "prefill impl must be 0..3");
            ctx->opt_prefill_impl = value;
            return MATKV_OK;
        case MATKV_OPT_DECODE_ADVANCES_TAIL:
            if (value < 0 || value > 1) return fail(MATKV_E_INVALID_ARG, "decode-advances-tail must be 0 or 1");
            ctx->opt_fused_advance = value;
            return MATKV_OK;
        case MATKV_OPT_STAGE_CTAS:
            if (value < 0 || value > 148) return fail(MATKV_E_INVALID_ARG, "staging CTAs must be 0..148");
            ctx->opt_stage_ctas = value;
            return MATKV_OK;
        case MATKV_OPT_DECODE_IMPL:
            if (value < 0 || value > 2) return fail(MATKV_E_INVALID_ARG, "decode impl must be 0..2");
            ctx->opt_decode_impl = value;
            return MATKV_OK;
        case MATKV_OPT_FP8_RESIDENT:
            if (value < 0 || value > 1) return fail(MATKV_E_INVALID_ARG, "fp8-resident must be 0 or 1");
            ctx->opt_fp8_resident = value;
            return MATKV_OK;
        case MATKV_OPT_SHARE_TILES:
            if (value < 1 || value > 1024) return fail(MATKV_E_INVALID_ARG, "tiles per chunk-major item must be 1..1024");
            ctx->opt_share_tiles = value;
            return MATKV_OK;
        case MATKV_OPT_IO_TIMEOUT_MS:
            if (value < 1 || value > 3600000) return fail(MATKV_E_INVALID_ARG, "storage read time limit must be 1..3600000 ms");
            ctx->opt_io_timeout_ms = value;
            io_engine_configure(ctx);
            return MATKV_OK;
        case MATKV_OPT_IO_TEST_DELAY_MS:
            if (value < 0 || value > 60000) return fail(MATKV_E_INVALID_ARG, "injected read delay must be 0..60000 ms");
            ctx->opt_io_test_delay_ms = value;
            io_engine_configure(ctx);
            return MATKV_OK;
        case MATKV_OPT_CLUSTER_DECODE:
            if (value < 0 || value > 2) return fail(MATKV_E_INVALID_ARG, "cluster decode must be 0, 1 or 2");
            ctx->opt_cluster_decode = value;
            return MATKV_OK;
        case MATKV_OPT_CLUSTER_MAX:
            if (value < 0 || value > 16) return fail(MATKV_E_INVALID_ARG, "largest cluster must be 0 (automatic) .. 16");
            ctx->opt_cluster_max = value;
            return MATKV_OK;
        case MATKV_OPT_PREFILL_CTAS:
            if (value < 0 || value > 64) return fail(MATKV_E_INVALID_ARG, "prefill CTAs per head must be 0..64");
            ctx->opt_prefill_ctas = value;
            return MATKV_OK;
    }
    return fail(MATKV_E_INVALID_ARG, "matkv_set_option: unknown option %d", option);
}

size_t matkv_workspace_bytes(const matkv_ctx *ctx) {
    if (!ctx) return 0;
    return workspace_bytes_for(ctx->cfg, nullptr, nullptr);
}

int matkv_set_workspace(matkv_ctx *ctx, void *dev, size_t bytes) {
    if (!ctx || !dev) return fail(MATKV_E_INVALID_ARG, "matkv_set_workspace: null argument");
    if ((uintptr_t)dev % 256) return fail(MATKV_E_ALIGNMENT, "workspace must be 256-byte aligned");
    WorkspaceView v;
    const size_t need = workspace_bytes_for(ctx->cfg, &v, dev);
    if (bytes < need) return fail(MATKV_E_CAPACITY, "workspace of %zu bytes is smaller than the %zu needed", bytes, need);
    DeviceGuard guard(ctx->device);
    MATKV_CUDA(cudaDeviceSynchronize());
    MATKV_CUDA(cudaMemset(v.counters, 0, sizeof(int32_t) * (size_t)v.n_counter_slots));
    ctx->workspace = dev;
    ctx->workspace_bytes = bytes;
    return MATKV_OK;
}

int matkv_status(matkv_ctx *ctx, int32_t *dev_status_out, int32_t clear) {
    if (!ctx || !dev_status_out) return fail(MATKV_E_INVALID_ARG, "matkv_status: null argument");
    DeviceGuard guard(ctx->device);
    MATKV_CUDA(cudaDeviceSynchronize());
    MATKV_CUDA(cudaMemcpy(dev_status_out, ctx->d_status, sizeof(int32_t), cudaMemcpyDeviceToHost));
    if (clear) MATKV_CUDA(cudaMemset(ctx->d_status, 0, sizeof(int32_t)));
    return MATKV_OK;
}

// ---- a1 --------------------------------------------------------------------------------------
int matkv_register_chunk(matkv_ctx *ctx, uint64_t chunk_id, int32_t n_tokens, const void *host_blob, void *dev_blob) {
    if (!ctx) return fail(MATKV_E_INVALID_ARG, "matkv_register_chunk: null context");
    if (n_tokens < 1) return fail(MATKV_E_INVALID_ARG, "chunk %llu: n_tokens must be >= 1", (unsigned long long)chunk_id);
    if ((int64_t)ctx->cfg.n_layers * 2 * ctx->cfg.n_kv_heads * n_tokens >= (int64_t)1 << 31)
        return fail(MATKV_E_CAPACITY, "chunk %llu: layers x 2 x KV heads x tokens must stay below 2^31 rows", (unsigned long long)chunk_id);
    if (!host_blob && !dev_blob) return fail(MATKV_E_INVALID_ARG, "chunk %llu: no blob given", (unsigned long long)chunk_id);
    if (dev_blob && (uintptr_t)dev_blob % 256)
        return fail(MATKV_E_ALIGNMENT, "chunk %llu: device blob must be 256-byte aligned", (unsigned long long)chunk_id);
    if (host_blob && (uintptr_t)host_blob % 16)
        return fail(MATKV_E_ALIGNMENT, "chunk %llu: host blob must be 16-byte aligned", (unsigned long long)chunk_id);
    if (ctx->chunks.count(chunk_id))
        return fail(MATKV_E_INVALID_ARG, "chunk %llu is already registered", (unsigned long long)chunk_id);
    Chunk c;
    c.n_tokens = n_tokens;
    c.host_blob = host_blob;
    c.dev_blob = dev_blob;
    if (host_blob) {
        // the staging copy kernel reads a host blob over the link: only page-locked (or managed) memory allows that;
        // a pageable blob is staged by the copy engine whatever MATKV_OPT_STAGE_CTAS says
        DeviceGuard guard(ctx->device);
        cudaPointerAttributes at;
        if (cudaPointerGetAttributes(&at, host_blob) == cudaSuccess)
            c.host_device_readable = at.type == cudaMemoryTypeHost || at.type == cudaMemoryTypeManaged || at.type == cudaMemoryTypeDevice;
        else
            cudaGetLastError();
    }
    if (dev_blob) {
        int rc = encode_rows_map(&c.tmap, dev_blob, ctx->cfg.head_dim, (uint64_t)ctx->cfg.n_layers * 2 * ctx->cfg.n_kv_heads * n_tokens);
        if (rc) return rc;
    }
    ctx->chunks.emplace(chunk_id, c);
    return MATKV_OK;
}

int matkv_register_chunk_file(matkv_ctx *ctx, uint64_t chunk_id, int32_t n_tokens, const char *path, uint64_t file_offset) {
    if (!ctx || !path) return fail(MATKV_E_INVALID_ARG, "matkv_register_chunk_file: null argument");
    if (n_tokens < 1) return fail(MATKV_E_INVALID_ARG, "chunk %llu: n_tokens must be >= 1", (unsigned long long)chunk_id);
    if ((int64_t)ctx->cfg.n_layers * 2 * ctx->cfg.n_kv_heads * n_tokens >= (int64_t)1 << 31)
        return fail(MATKV_E_CAPACITY, "chunk %llu: layers x 2 x KV heads x tokens must stay below 2^31 rows", (unsigned long long)chunk_id);
    if (ctx->chunks.count(chunk_id))
        return fail(MATKV_E_INVALID_ARG, "chunk %llu is already registered", (unsigned long long)chunk_id);
    Chunk c;
    c.n_tokens = n_tokens;
    c.file_offset = file_offset;
    int rc = open_chunk_file(path, file_offset, blob_bytes(ctx->cfg, n_tokens), &c.file_fd);
    if (rc) return rc;
    ctx->chunks.emplace(chunk_id, c);
    return MATKV_OK;
}

// ---- compressed chunk store -------------------------------------------------------------------
size_t matkv_fp8_blob_bytes(const matkv_ctx *ctx, int32_t n_tokens) {
    if (!ctx || n_tokens < 1) return 0;
    return fp8_blob_bytes(ctx->cfg, n_tokens);
}

size_t matkv_fp8_resident_bytes(const matkv_ctx *ctx, int32_t n_tokens) {
    if (!ctx || n_tokens < 1) return 0;
    return fp8_resident_bytes(ctx->cfg, n_tokens);
}

int matkv_quantize_chunk_fp8(matkv_ctx *ctx, const void *dev_blob, int32_t n_tokens, void *dev_blob_fp8, void *stream) {
    if (!ctx || !dev_blob || !dev_blob_fp8) return fail(MATKV_E_INVALID_ARG, "matkv_quantize_chunk_fp8: null argument");
    if (n_tokens < 1) return fail(MATKV_E_INVALID_ARG, "matkv_quantize_chunk_fp8: n_tokens must be >= 1");
    if ((uintptr_t)dev_blob % 16 || (uintptr_t)dev_blob_fp8 % 256)
        return fail(MATKV_E_ALIGNMENT, "matkv_quantize_chunk_fp8: the bf16 blob must be 16-byte, the fp8 blob 256-byte aligned");
    DeviceGuard guard(ctx->device);
    return launch_quantize_fp8(ctx, dev_blob, n_tokens, dev_blob_fp8, (cudaStream_t)stream);
}

int matkv_register_chunk_fp8(matkv_ctx *ctx, uint64_t chunk_id, int32_t n_tokens, const void *host_blob_fp8) {
    if (!ctx || !host_blob_fp8) return fail(MATKV_E_INVALID_ARG, "matkv_register_chunk_fp8: null argument");
    if (n_tokens < 1) return fail(MATKV_E_INVALID_ARG, "chunk %llu: n_tokens must be >= 1", (unsigned long long)chunk_id);
    if ((int64_t)ctx->cfg.n_layers * 2 * ctx->cfg.n_kv_heads * n_tokens >= (int64_t)1 << 31)
        return fail(MATKV_E_CAPACITY, "chunk %llu: layers x 2 x KV heads x tokens must stay below 2^31 rows", (unsigned long long)chunk_id);
    if ((uintptr_t)host_blob_fp8 % 256)
        return fail(MATKV_E_ALIGNMENT, "chunk %llu: the compressed blob must be 256-byte aligned", (unsigned long long)chunk_id);
    if (ctx->chunks.count(chunk_id))
        return fail(MATKV_E_INVALID_ARG, "chunk %llu is already registered", (unsigned long long)chunk_id);
    {   // the expanding copy kernel reads the blob over the link: it must be page-locked, device-accessible memory
        DeviceGuard guard(ctx->device);
        cudaPointerAttributes at;
        cudaError_t e = cudaPointerGetAttributes(&at, host_blob_fp8);
        if (e != cudaSuccess || (at.type != cudaMemoryTypeHost && at.type != cudaMemoryTypeManaged && at.type != cudaMemoryTypeDevice)) {
            cudaGetLastError();
            return fail(MATKV_E_INVALID_ARG, "chunk %llu: the compressed blob must be pinned (page-locked) host memory", (unsigned long long)chunk_id);
        }
    }
    Chunk c;
    c.n_tokens = n_tokens;
    c.host_blob = host_blob_fp8;
    c.host_device_readable = true;
    c.fp8 = true;
    ctx->chunks.emplace(chunk_id, c);
    return MATKV_OK;
}

int matkv_register_chunk_file_fp8(matkv_ctx *ctx, uint64_t chunk_id, int32_t n_tokens, const char *path, uint64_t file_offset) {
    if (!ctx || !path) return fail(MATKV_E_INVALID_ARG, "matkv_register_chunk_file_fp8: null argument");
    if (n_tokens < 1) return fail(MATKV_E_INVALID_ARG, "chunk %llu: n_tokens must be >= 1", (unsigned long long)chunk_id);
    if ((int64_t)ctx->cfg.n_layers * 2 * ctx->cfg.n_kv_heads * n_tokens >= (int64_t)1 << 31)
        return fail(MATKV_E_CAPACITY, "chunk %llu: layers x 2 x KV heads x tokens must stay below 2^31 rows", (unsigned long long)chunk_id);
    if (ctx->chunks.count(chunk_id))
        return fail(MATKV_E_INVALID_ARG, "chunk %llu is already registered", (unsigned long long)chunk_id);
    Chunk c;
    c.n_tokens = n_tokens;
    c.file_offset = file_offset;
    c.fp8 = true;
    int rc = open_chunk_file(path, file_offset, fp8_blob_bytes(ctx->cfg, n_tokens), &c.file_fd);
    if (rc) return rc;
    ctx->chunks.emplace(chunk_id, c);
    return MATKV_OK;
}

int matkv_set_bounce_buffer(matkv_ctx *ctx, void *pinned_host, size_t bytes, size_t slab_bytes, int32_t n_io_threads) {
    if (!ctx || !pinned_host) return fail(MATKV_E_INVALID_ARG, "matkv_set_bounce_buffer: null argument");
    if ((uintptr_t)pinned_host % 4096 || slab_bytes == 0 || slab_bytes % 4096)
        return fail(MATKV_E_ALIGNMENT, "bounce buffer and slab size must be multiples of 4096 bytes");
    if (bytes / slab_bytes < 2) return fail(MATKV_E_CAPACITY, "bounce buffer must hold at least two slabs");
    if (n_io_threads < 1 || n_io_threads > 64) return fail(MATKV_E_INVALID_ARG, "reader threads must be 1..64");
    if (ctx->io) {
        DeviceGuard guard(ctx->device);
        MATKV_CUDA(cudaDeviceSynchronize());
        io_engine_destroy(ctx);
    }
    return io_engine_create(ctx, pinned_host, bytes, slab_bytes, n_io_threads);
}

int matkv_unregister_chunk(matkv_ctx *ctx, uint64_t chunk_id) {
    if (!ctx) return fail(MATKV_E_INVALID_ARG, "matkv_unregister_chunk: null context");
    auto it = ctx->chunks.find(chunk_id);
    if (it == ctx->chunks.end()) return fail(MATKV_E_UNKNOWN_CHUNK, "chunk %llu is not registered", (unsigned long long)chunk_id);
    Chunk &c = it->second;
    if (c.region && c.slot >= 0) c.region->used[c.slot] = 0;
    close_chunk_file(c.file_fd);
    ctx->chunks.erase(it);
    return MATKV_OK;
}


// ---- a2 --------------------------------------------------------------------------------------
int matkv_stage_chunks_async(matkv_ctx *ctx, const uint64_t *ids, int32_t n, void *dev_slots, size_t slot_bytes,
                             int32_t n_slots, void *copy_stream, uint64_t *ticket_out) {
    if (!ctx || (!ids && n > 0) || !dev_slots || !ticket_out)
        return fail(MATKV_E_INVALID_ARG, "matkv_stage_chunks_async: null argument");
    if (n < 0 || n_slots < 1 || slot_bytes == 0) return fail(MATKV_E_INVALID_ARG, "matkv_stage_chunks_async: bad sizes");
    if ((uintptr_t)dev_slots % 256 || slot_bytes % 256)
        return fail(MATKV_E_ALIGNMENT, "slot base and slot size must be multiples of 256 bytes");
    DeviceGuard guard(ctx->device);
    cudaStream_t cs = (cudaStream_t)copy_stream;
    reap_graveyard(ctx, false);

    // distinct ids that need a copy into this region
    std::vector<uint64_t> want;
    for (int32_t i = 0; i < n; ++i) {
        auto it = ctx->chunks.find(ids[i]);
        if (it == ctx->chunks.end())
            return fail(MATKV_E_UNKNOWN_CHUNK, "chunk %llu is not registered", (unsigned long long)ids[i]);
        const Chunk &c = it->second;
        if (c.dev_blob) continue;  // resident: nothing to do
        if (!c.host_blob && c.file_fd < 0)
            return fail(MATKV_E_INVALID_ARG, "chunk %llu has no host blob or file to stage", (unsigned long long)ids[i]);
        const size_t stored = c.fp8 ? fp8_blob_bytes(ctx->cfg, c.n_tokens) : blob_bytes(ctx->cfg, c.n_tokens);
        if (c.file_fd >= 0 && !c.host_blob && stored > io_engine_slab_bytes(ctx))
            return fail(ctx->io ? MATKV_E_CAPACITY : MATKV_E_INVALID_ARG,
                        "chunk %llu lives in a file: set a bounce buffer with slabs of at least %zu bytes first",
                        (unsigned long long)ids[i], stored);
        const bool keep8 = c.fp8 && ctx->opt_fp8_resident;   // stays compressed in HBM
        if (keep8 && ctx->cfg.head_dim != 128)
            return fail(MATKV_E_INVALID_ARG, "compressed-resident chunks need head_dim 128");
        const size_t in_slot = keep8 ? fp8_resident_bytes(ctx->cfg, c.n_tokens) : blob_bytes(ctx->cfg, c.n_tokens);
        if (in_slot > slot_bytes)
            return fail(MATKV_E_CAPACITY, "chunk %llu (%zu bytes) does not fit a slot of %zu bytes",
                        (unsigned long long)ids[i], in_slot, slot_bytes);
        if (std::find(want.begin(), want.end(), ids[i]) == want.end()) want.push_back(ids[i]);
    }
    if ((int64_t)want.size() > n_slots)
        return fail(MATKV_E_CAPACITY, "%zu distinct chunks do not fit %d slots", want.size(), n_slots);

    Region *&rp = ctx->regions[dev_slots];
    if (!rp) {
        rp = new Region();
        rp->base = dev_slots;
    }
    Region *r = rp;
    if (r->slot_bytes != slot_bytes || r->n_slots != n_slots) {
        // geometry changed: drop every occupant
        for (size_t s = 0; s < r->occupant.size(); ++s)
            if (r->used[s]) {
                auto it = ctx->chunks.find(r->occupant[s]);
                if (it != ctx->chunks.end() && it->second.region == r) {
                    it->second.staged = nullptr;
                    it->second.region = nullptr;
                    it->second.slot = -1;
                }
            }
        r->slot_bytes = slot_bytes;
        r->n_slots = n_slots;
        r->occupant.assign(n_slots, 0);
        r->used.assign(n_slots, 0);
    }
    // keep occupants that are wanted again, evict the rest
    for (int32_t s = 0; s < n_slots; ++s) {
        if (!r->used[s]) continue;
        const uint64_t id = r->occupant[s];
        if (std::find(want.begin(), want.end(), id) != want.end()) continue;
        auto it = ctx->chunks.find(id);
        if (it != ctx->chunks.end() && it->second.region == r && it->second.slot == s) {
            it->second.staged = nullptr;
            it->second.region = nullptr;
            it->second.slot = -1;
        }
        r->used[s] = 0;
    }
    // the region's previous readers must be done before anything is overwritten
    if (r->has_last_use) MATKV_CUDA(cudaStreamWaitEvent(cs, r->last_use, 0));

    retire_finished_tickets(ctx);   // staging calls already seen complete give their events back: the map stays bounded
    Ticket tk;
    MATKV_CUDA(cudaEventCreateWithFlags(&tk.done, cudaEventDisableTiming));
    tk.io_failed = std::make_shared<FailFlag>();
    const uint64_t ticket = ctx->next_ticket++;
    io_engine_bind_fail_word(ctx, ticket, tk.io_failed.get());
    int32_t next_free = 0;
    int rc_fail = MATKV_OK;   // a failure part-way: the chunks already touched keep a valid event, then the error is returned
    bool any_file = false;
    for (uint64_t id : want) {
        Chunk &c = ctx->chunks[id];
        if (c.region == r && c.slot >= 0 && r->used[c.slot] && r->occupant[c.slot] == id) continue;  // already here
        while (next_free < n_slots && r->used[next_free]) ++next_free;
        if (next_free >= n_slots) {
            rc_fail = fail(MATKV_E_CAPACITY, "no free slot left in the region");
            break;
        }
        void *dst = (char *)dev_slots + (size_t)next_free * slot_bytes;
        const bool keep8 = c.fp8 && ctx->opt_fp8_resident;
        int rc = MATKV_OK;
        if (c.host_blob && c.fp8) {
            // compressed chunk: expanded to bf16 on its way in, or re-laid out into the resident compressed form (always
            // by an SM kernel that reads the host blob over the link: it must be device-accessible pinned memory)
            rc = keep8 ? launch_stage_relayout_fp8(ctx, c.host_blob, dst, c.n_tokens, cs)
                       : launch_stage_expand_fp8(ctx, c.host_blob, dst, c.n_tokens, ctx->opt_stage_ctas > 0 ? (int)ctx->opt_stage_ctas : 16, cs);
        } else if (c.host_blob && ctx->opt_stage_ctas > 0 && c.host_device_readable) {
            // SM-driven copy (checked at registration: the blob is page-locked memory the device can read)
            rc = launch_stage_copy(ctx, c.host_blob, dst, blob_bytes(ctx->cfg, c.n_tokens), (int)ctx->opt_stage_ctas, cs);
        } else if (c.host_blob) {
            cudaError_t e = cudaMemcpyAsync(dst, c.host_blob, blob_bytes(ctx->cfg, c.n_tokens), cudaMemcpyHostToDevice, cs);
            if (e != cudaSuccess) rc = cuda_fail(e, "staging copy");
        } else {  // storage tier: read into the bounce ring, then copy, all in the copy stream's order
            any_file = true;
            rc = io_engine_stage(ctx, c.file_fd, c.file_offset, c.fp8 ? fp8_blob_bytes(ctx->cfg, c.n_tokens) : blob_bytes(ctx->cfg, c.n_tokens),
                                 dst, cs, tk.io_failed, c.fp8 ? c.n_tokens : 0, keep8);
        }
        if (rc == MATKV_OK)
            rc = keep8 ? encode_fp8_maps(c.tmap8, dst, ctx->cfg, c.n_tokens)
                       : encode_rows_map(&c.tmap, dst, ctx->cfg.head_dim, (uint64_t)ctx->cfg.n_layers * 2 * ctx->cfg.n_kv_heads * c.n_tokens);
        if (rc) {
            // this chunk has no usable device copy (whatever was enqueued for it lands in a slot nobody points at)
            if (c.region && c.slot >= 0) c.region->used[c.slot] = 0;
            c.staged = nullptr;
            c.region = nullptr;
            c.slot = -1;
            c.ready = nullptr;
            rc_fail = rc;
            break;
        }
        if (c.region && c.slot >= 0) c.region->used[c.slot] = 0;  // moves from another region (or another slot)
        c.resident_fp8 = keep8;
        r->used[next_free] = 1;
        r->occupant[next_free] = id;
        c.staged = dst;
        c.region = r;
        c.slot = next_free;
        c.ready = tk.done;
        c.ticket = ticket;
        c.io_failed = tk.io_failed;
        tk.chunk_ids.push_back(id);
    }
    if (any_file) io_engine_flag_status(ctx, tk.io_failed, cs);   // a read failure of this call shows in the status word once the stream gets here
    cudaError_t e_rec = cudaEventRecord(tk.done, cs);
    ctx->tickets.emplace(ticket, tk);
    *ticket_out = ticket;
    if (rc_fail) return rc_fail;
    if (e_rec != cudaSuccess) return cuda_fail(e_rec, "cudaEventRecord(staging ticket)");
    return MATKV_OK;
}

// A ticket is live until its copies have been seen complete; retired tickets answer MATKV_OK (or MATKV_E_IO when a
// storage read of theirs failed).
static int retired_ticket_result(matkv_ctx *ctx, uint64_t ticket) {
    if (ticket == 0 || ticket >= ctx->next_ticket) return fail(MATKV_E_INVALID_ARG, "unknown staging ticket %llu", (unsigned long long)ticket);
    if (std::find(ctx->failed_tickets.begin(), ctx->failed_tickets.end(), ticket) != ctx->failed_tickets.end()) {
        const char *msg = "";
        io_engine_errors(ctx, &msg);
        return fail(MATKV_E_IO, "staging ticket %llu: reading from storage failed: %s", (unsigned long long)ticket, msg);
    }
    return MATKV_OK;
}

int matkv_stage_query(matkv_ctx *ctx, uint64_t ticket) {
    if (!ctx) return fail(MATKV_E_INVALID_ARG, "matkv_stage_query: null context");
    auto it = ctx->tickets.find(ticket);
    if (it == ctx->tickets.end()) return retired_ticket_result(ctx, ticket);
    DeviceGuard guard(ctx->device);
    cudaError_t e = cudaEventQuery(it->second.done);
    if (e == cudaErrorNotReady) return fail(MATKV_E_NOT_READY, "staging ticket %llu still copying", (unsigned long long)ticket);
    if (e != cudaSuccess) return cuda_fail(e, "cudaEventQuery");
    retire_ticket(ctx, it);
    return retired_ticket_result(ctx, ticket);
}

int matkv_stage_wait(matkv_ctx *ctx, uint64_t ticket) {
    if (!ctx) return fail(MATKV_E_INVALID_ARG, "matkv_stage_wait: null context");
    auto it = ctx->tickets.find(ticket);
    if (it == ctx->tickets.end()) return retired_ticket_result(ctx, ticket);
    DeviceGuard guard(ctx->device);
    MATKV_CUDA(cudaEventSynchronize(it->second.done));
    retire_ticket(ctx, it);
    return retired_ticket_result(ctx, ticket);
}

// ---- a3 --------------------------------------------------------------------------------------
int matkv_build_chunk_table(matkv_ctx *ctx, int32_t batch, const int32_t *n_chunks_per_req, const uint64_t *ids,
                            void *tail_k, void *tail_v, void *stream, matkv_table **out) {
    if (!ctx || !n_chunks_per_req || !tail_k || !tail_v || !out)
        return fail(MATKV_E_INVALID_ARG, "matkv_build_chunk_table: null argument");
    *out = nullptr;
    if (batch < 1 || batch > ctx->cfg.max_batch)
        return fail(MATKV_E_CAPACITY, "batch %d outside 1..%d", batch, ctx->cfg.max_batch);
    if ((uintptr_t)tail_k % 256 || (uintptr_t)tail_v % 256) return fail(MATKV_E_ALIGNMENT, "tails must be 256-byte aligned");
    int64_t total = 0;
    for (int32_t r = 0; r < batch; ++r) {
        if (n_chunks_per_req[r] < 0 || n_chunks_per_req[r] > ctx->cfg.max_chunks_per_req)
            return fail(MATKV_E_CAPACITY, "request %d lists %d chunks (max %d)", r, n_chunks_per_req[r],
                        ctx->cfg.max_chunks_per_req);
        total += n_chunks_per_req[r];
    }
    if (total > 0 && !ids) return fail(MATKV_E_INVALID_ARG, "matkv_build_chunk_table: null id list");
    DeviceGuard guard(ctx->device);
    cudaStream_t st = (cudaStream_t)stream;
    reap_graveyard(ctx, false);

    matkv_table *t = new matkv_table();
    t->ctx = ctx;
    t->batch = batch;
    t->tail_k = (__nv_bfloat16 *)tail_k;
    t->tail_v = (__nv_bfloat16 *)tail_v;
    std::vector<cudaEvent_t> waits;
    std::vector<const CUtensorMap *> seg_maps, seg_maps8;
    int64_t k = 0;
    for (int32_t r = 0; r < batch; ++r) {
        DevReq rq;
        memset(&rq, 0, sizeof rq);
        rq.seg_begin = (int32_t)t->h_segs.size();
        rq.n_seg = n_chunks_per_req[r];
        int32_t longest = 0;
        for (int32_t i = 0; i < rq.n_seg; ++i, ++k) {
            auto it = ctx->chunks.find(ids[k]);
            if (it == ctx->chunks.end()) {
                delete t;
                return fail(MATKV_E_UNKNOWN_CHUNK, "request %d: chunk %llu is not registered", r, (unsigned long long)ids[k]);
            }
            const Chunk &c = it->second;
            const void *dev = c.dev_blob ? c.dev_blob : c.staged;
            if (!dev) {
                delete t;
                return fail(MATKV_E_NOT_STAGED, "request %d: chunk %llu has no device copy (stage it first)", r,
                            (unsigned long long)ids[k]);
            }
            if (!c.dev_blob && c.io_failed && c.io_failed->host.load(std::memory_order_acquire)) {
                delete t;
                const char *msg = "";
                io_engine_errors(ctx, &msg);
                return fail(MATKV_E_IO, "request %d: chunk %llu was staged by a call whose storage reads failed: %s", r,
                            (unsigned long long)ids[k], msg);
            }
            if (!c.dev_blob) {
                if (c.ready && std::find(waits.begin(), waits.end(), c.ready) == waits.end()) waits.push_back(c.ready);
                if (std::find(t->regions.begin(), t->regions.end(), c.region) == t->regions.end())
                    t->regions.push_back(c.region);
            }
            DevSeg sg;
            sg.base = (const __nv_bfloat16 *)dev;
            sg.len = c.n_tokens;
            sg.start = rq.n_chunk_tokens;
            sg.fmt = (!c.dev_blob && c.resident_fp8) ? 1 : 0;
            sg.pad = 0;
            if (sg.fmt) t->has_fp8 = true;
            t->h_segs.push_back(sg);
            seg_maps.push_back(&c.tmap);
            seg_maps8.push_back(c.tmap8);
            rq.n_chunk_tokens += c.n_tokens;
            rq.chunk_tiles += (c.n_tokens + kTile - 1) / kTile;
            longest = std::max(longest, c.n_tokens);
        }
        rq.pos_base = ctx->cfg.pos_mode == 1 ? longest : rq.n_chunk_tokens;   // mode 2: the caller may replace it (matkv_table_set_pos_base)
        t->max_chunk_tiles = std::max(t->max_chunk_tiles, rq.chunk_tiles);
        t->total_chunk_tiles += rq.chunk_tiles;
        t->h_reqs.push_back(rq);
    }
    t->n_seg_total = (int32_t)t->h_segs.size();

    // chunk-major decode: requests that list the same device copy of a chunk are stacked, 16 / G per item,
    // so that the chunk's rows are read once for all of them; a long chunk is cut into items of at most
    // opt_share_tiles tiles.  Every (item, request) pair produces one partial, the request's tail one more.
    std::vector<DevItem> items;
    {
        const int G = ctx->cfg.n_q_heads / ctx->cfg.n_kv_heads;
        const int R = (G >= 1 && G <= kShareRows && kShareRows % G == 0) ? kShareRows / G : 0;
        const int T = (int)ctx->opt_share_tiles;
        std::map<std::pair<const void *, int32_t>, std::vector<std::pair<int32_t, int32_t>>> members;  // -> (request, segment)
        std::vector<int32_t> part_off(t->h_segs.size(), 0);
        int32_t part_base = 0;
        for (int32_t r = 0; r < batch; ++r) {
            DevReq &rq = t->h_reqs[r];
            int32_t n = 0;
            for (int32_t i = 0; i < rq.n_seg; ++i) {
                const int32_t si = rq.seg_begin + i;
                const DevSeg &sg = t->h_segs[si];
                members[{(const void *)sg.base, sg.len}].push_back({r, si});
                part_off[si] = n;
                n += ((sg.len + kTile - 1) / kTile + T - 1) / T;
            }
            rq.n_parts = n + 1;
            rq.part_base = part_base;
            part_base += rq.n_parts;
        }
        t->parts_total = part_base;
        for (auto &kv : members) t->distinct_chunk_tiles += (kv.first.second + kTile - 1) / kTile;
        bool fits = true;  // the kernel's item queue keeps request indices and part counts in 16 bits
        for (int32_t r = 0; r < batch; ++r) fits = fits && t->h_reqs[r].n_parts <= 32767;
        if (R > 0 && fits && !t->has_fp8) {   // the chunk-major kernel reads bf16 chunks only
            for (auto &kv : members) {
                const int32_t len = kv.first.second, tiles = (len + kTile - 1) / kTile;
                const auto &m = kv.second;
                for (int32_t tile0 = 0, sub = 0; tile0 < tiles; tile0 += T, ++sub)
                    for (size_t j0 = 0; j0 < m.size(); j0 += R) {
                        DevItem it;
                        memset(&it, 0, sizeof it);
                        it.tmap = m[j0].second;
                        it.len = len;
                        it.tile0 = tile0;
                        it.n_tiles = std::min(T, tiles - tile0);
                        it.n_req = (int32_t)std::min<size_t>(R, m.size() - j0);
                        it.last_read = j0 + R >= m.size();
                        for (int32_t j = 0; j < it.n_req; ++j) {
                            const DevReq &rq = t->h_reqs[m[j0 + j].first];
                            it.req[j] = m[j0 + j].first;
                            it.part[j] = rq.part_base + part_off[m[j0 + j].second] + sub;
                            it.np[j] = rq.n_parts;
                        }
                        t->item_tiles += it.n_tiles;
                        items.push_back(it);
                    }
            }
            t->n_items = (int32_t)items.size();
            t->share_ok = true;
        }
    }

    const size_t segs_bytes = align_up(sizeof(DevSeg) * std::max<size_t>(t->h_segs.size(), 1), 256);
    const size_t reqs_bytes = align_up(sizeof(DevReq) * (size_t)batch, 256);
    const size_t tl_bytes = align_up(sizeof(int32_t) * (size_t)batch, 256);
    const size_t maps_bytes = align_up(sizeof(CUtensorMap) * (seg_maps.size() + 2), 256);
    const size_t items_bytes = align_up(sizeof(DevItem) * std::max<size_t>(items.size(), 1), 256);
    const size_t maps8_bytes = t->has_fp8 ? align_up(sizeof(CUtensorMap) * 2 * seg_maps8.size(), 256) : 0;
    // tile directory for the cluster decode kernel: a CTA finds any chunk tile of a request with one load
    std::vector<int4> tile_dir;
    if (!t->has_fp8 && t->total_chunk_tiles <= (int64_t)1 << 20) {
        for (int32_t r = 0; r < batch; ++r) {
            const DevReq &rq = t->h_reqs[r];
            t->h_dir_begin.push_back((int32_t)tile_dir.size());
            for (int32_t i = 0; i < rq.n_seg; ++i) {
                const int32_t len = t->h_segs[rq.seg_begin + i].len;
                for (int32_t r0 = 0; r0 < len; r0 += kTile) tile_dir.push_back(make_int4(rq.seg_begin + i, r0, len, std::min(kTile, len - r0)));
            }
        }
    }
    const size_t dir_bytes = align_up(sizeof(int4) * std::max<size_t>(tile_dir.size(), 1), 256);
    t->image_bytes = segs_bytes + reqs_bytes + tl_bytes + maps_bytes + items_bytes + maps8_bytes + dir_bytes;
    CUtensorMap tail_maps[2];
    {
        const uint64_t tail_rows = (uint64_t)batch * ctx->cfg.n_layers * ctx->cfg.n_kv_heads * ctx->cfg.max_tail_tokens;
        int rc = encode_rows_map(&tail_maps[0], tail_k, ctx->cfg.head_dim, tail_rows);
        if (!rc) rc = encode_rows_map(&tail_maps[1], tail_v, ctx->cfg.head_dim, tail_rows);
        if (rc) {
            delete t;
            return rc;
        }
    }
    cudaError_t e = cudaSuccess;
    {
        auto &pool = ctx->image_pool;
        for (size_t i = 0; i < pool.size(); ++i)
            if (pool[i].bytes >= t->image_bytes) {
                t->h_pinned = pool[i].h_pinned;
                t->d_image = pool[i].d_image;
                t->image_alloc = pool[i].bytes;
                pool[i] = pool.back();
                pool.pop_back();
                break;
            }
    }
    if (!t->h_pinned) {
        t->image_alloc = std::max<size_t>(t->image_bytes, 64 * 1024);
        e = cudaMallocHost(&t->h_pinned, t->image_alloc);
        if (e == cudaSuccess) e = cudaMalloc(&t->d_image, t->image_alloc);
    }
    if (e != cudaSuccess) {
        cudaFreeHost(t->h_pinned);
        delete t;
        return cuda_fail(e, "table allocation");
    }
    memset(t->h_pinned, 0, t->image_bytes);
    if (!t->h_segs.empty()) memcpy(t->h_pinned, t->h_segs.data(), sizeof(DevSeg) * t->h_segs.size());
    memcpy((char *)t->h_pinned + segs_bytes, t->h_reqs.data(), sizeof(DevReq) * (size_t)batch);
    t->d_segs = (DevSeg *)t->d_image;
    t->d_reqs = (DevReq *)((char *)t->d_image + segs_bytes);
    t->d_tail_len = (int32_t *)((char *)t->d_image + segs_bytes + reqs_bytes);
    t->d_tmaps = (CUtensorMap *)((char *)t->d_image + segs_bytes + reqs_bytes + tl_bytes);
    t->d_items = (DevItem *)((char *)t->d_image + segs_bytes + reqs_bytes + tl_bytes + maps_bytes);
    if (!items.empty())
        memcpy((char *)t->h_pinned + segs_bytes + reqs_bytes + tl_bytes + maps_bytes, items.data(), sizeof(DevItem) * items.size());
    if (t->has_fp8) {
        const size_t off8 = segs_bytes + reqs_bytes + tl_bytes + maps_bytes + items_bytes;
        t->d_tmaps8 = (CUtensorMap *)((char *)t->d_image + off8);
        CUtensorMap *h8 = (CUtensorMap *)((char *)t->h_pinned + off8);
        for (size_t i = 0; i < seg_maps8.size(); ++i) memcpy(h8 + 2 * i, seg_maps8[i], 2 * sizeof(CUtensorMap));
    }
    if (!t->h_dir_begin.empty()) {
        const size_t offd = segs_bytes + reqs_bytes + tl_bytes + maps_bytes + items_bytes + maps8_bytes;
        t->d_tile_dir = (int4 *)((char *)t->d_image + offd);
        if (!tile_dir.empty()) memcpy((char *)t->h_pinned + offd, tile_dir.data(), sizeof(int4) * tile_dir.size());
    }
    {
        CUtensorMap *hm = (CUtensorMap *)((char *)t->h_pinned + segs_bytes + reqs_bytes + tl_bytes);
        for (size_t i = 0; i < seg_maps.size(); ++i) memcpy(hm + i, seg_maps[i], sizeof(CUtensorMap));
        memcpy(hm + seg_maps.size(), tail_maps, sizeof(tail_maps));
    }
    for (cudaEvent_t ev : waits) {
        e = cudaStreamWaitEvent(st, ev, 0);  // the stream waits for the copies; the host does not
        if (e != cudaSuccess) break;
    }
    if (e == cudaSuccess) e = cudaMemcpyAsync(t->d_image, t->h_pinned, t->image_bytes, cudaMemcpyHostToDevice, st);
    if (e != cudaSuccess) {
        cudaFreeHost(t->h_pinned);
        cudaFree(t->d_image);
        delete t;
        return cuda_fail(e, "table upload");
    }
    ctx->tables.push_back(t);
    *out = t;
    return MATKV_OK;
}

int matkv_table_free(matkv_table *t, void *stream) {
    if (!t) return MATKV_OK;
    matkv_ctx *ctx = t->ctx;
    DeviceGuard guard(ctx->device);
    cudaStream_t st = (cudaStream_t)stream;
    for (Region *r : t->regions) {
        if (!r->last_use) MATKV_CUDA(cudaEventCreateWithFlags(&r->last_use, cudaEventDisableTiming));
        MATKV_CUDA(cudaEventRecord(r->last_use, st));
        r->has_last_use = true;
    }
    Grave g;
    MATKV_CUDA(cudaEventCreateWithFlags(&g.ev, cudaEventDisableTiming));
    MATKV_CUDA(cudaEventRecord(g.ev, st));
    g.h_pinned = t->h_pinned;
    g.d_image = t->d_image;
    g.bytes = t->image_alloc;
    ctx->image_graves.push_back(g);
    ctx->tables.erase(std::remove(ctx->tables.begin(), ctx->tables.end(), t), ctx->tables.end());
    delete t;
    reap_graveyard(ctx, false);
    return MATKV_OK;
}

int matkv_table_advance(matkv_table *t, int32_t n_tokens, void *stream) {
    if (!t) return fail(MATKV_E_INVALID_ARG, "matkv_table_advance: null table");
    if (n_tokens < 0) return fail(MATKV_E_INVALID_ARG, "matkv_table_advance: negative count");
    if (t->tail_len_host + n_tokens > t->ctx->cfg.max_tail_tokens)
        return fail(MATKV_E_CAPACITY, "tail would hold %d tokens (max %d)", t->tail_len_host + n_tokens,
                    t->ctx->cfg.max_tail_tokens);
    DeviceGuard guard(t->ctx->device);
    int rc = launch_add_tail_len(t, n_tokens, 0, false, (cudaStream_t)stream);
    if (rc == MATKV_OK) t->tail_len_host += n_tokens;
    return rc;
}

int matkv_table_set_tail_len(matkv_table *t, int32_t tail_len, void *stream) {
    if (!t) return fail(MATKV_E_INVALID_ARG, "matkv_table_set_tail_len: null table");
    if (tail_len < 0 || tail_len > t->ctx->cfg.max_tail_tokens)
        return fail(MATKV_E_CAPACITY, "tail length %d outside 0..%d", tail_len, t->ctx->cfg.max_tail_tokens);
    DeviceGuard guard(t->ctx->device);
    int rc = launch_add_tail_len(t, 0, tail_len, true, (cudaStream_t)stream);
    if (rc == MATKV_OK) t->tail_len_host = tail_len;
    return rc;
}

int matkv_table_set_pos_base(matkv_table *t, const int32_t *pos_base, void *stream) {
    if (!t || !pos_base) return fail(MATKV_E_INVALID_ARG, "matkv_table_set_pos_base: null argument");
    matkv_ctx *ctx = t->ctx;
    if (ctx->cfg.pos_mode != 2) return fail(MATKV_E_INVALID_ARG, "matkv_table_set_pos_base: the context was not created with pos_mode 2");
    for (int32_t r = 0; r < t->batch; ++r)
        if (pos_base[r] < 0 || (int64_t)pos_base[r] + ctx->cfg.max_tail_tokens >= (int64_t)1 << 30)
            return fail(MATKV_E_INVALID_ARG, "matkv_table_set_pos_base: base %d of request %d out of range", pos_base[r], r);
    DeviceGuard guard(ctx->device);
    // the request records sit in the table's pinned upload image right behind the segments; the copy is ordered
    // behind the table's own upload on the same stream
    DevReq *h_reqs = (DevReq *)((char *)t->h_pinned + ((char *)t->d_reqs - (char *)t->d_image));
    for (int32_t r = 0; r < t->batch; ++r) {
        t->h_reqs[r].pos_base = pos_base[r];
        h_reqs[r].pos_base = pos_base[r];
    }
    MATKV_CUDA(cudaMemcpyAsync(t->d_reqs, h_reqs, sizeof(DevReq) * (size_t)t->batch, cudaMemcpyHostToDevice, (cudaStream_t)stream));
    return MATKV_OK;
}

int matkv_stage_pending(matkv_ctx *ctx, int32_t *n_out) {
    if (!ctx || !n_out) return fail(MATKV_E_INVALID_ARG, "matkv_stage_pending: null argument");
    DeviceGuard guard(ctx->device);
    retire_finished_tickets(ctx);
    *n_out = (int32_t)ctx->tickets.size();
    return MATKV_OK;
}

// ---- a4 / a5 / a6 argument checks, then the launchers -----------------------------------------
static int check_attend(matkv_ctx *ctx, matkv_table *t, const void *q, const void *kn, const void *vn, void *out,
                        int32_t n_new, const char *who) {
    if (!ctx || !t || !q || !kn || !vn || !out) return fail(MATKV_E_INVALID_ARG, "%s: null argument", who);
    if (t->ctx != ctx) return fail(MATKV_E_INVALID_ARG, "%s: table belongs to another context", who);
    if (((uintptr_t)q | (uintptr_t)kn | (uintptr_t)vn | (uintptr_t)out) % 16)
        return fail(MATKV_E_ALIGNMENT, "%s: q, k_new, v_new and out must be 16-byte aligned", who);
    if (!ctx->workspace) return fail(MATKV_E_INVALID_ARG, "%s: no workspace set (matkv_set_workspace)", who);
    if (t->tail_len_host + n_new > ctx->cfg.max_tail_tokens)
        return fail(MATKV_E_CAPACITY, "%s: tail holds %d tokens, %d more exceed max_tail_tokens %d", who, t->tail_len_host,
                    n_new, ctx->cfg.max_tail_tokens);
    return MATKV_OK;
}

// Where the chunk-major decode may keep its partials: the part of the configured workspace behind the
// arrival counters (in front of the rotary scratch) if that is large enough, else whatever the caller's
// workspace holds beyond the configured size.
static bool shared_region(matkv_ctx *ctx, const matkv_table *t, int n_layers_launch, void **region, size_t *bytes) {
    WorkspaceView v;
    const size_t cfg_bytes = workspace_bytes_for(ctx->cfg, &v, ctx->workspace);
    const size_t need = shared_region_bytes(ctx->cfg, t, n_layers_launch);
    const size_t a_off = (size_t)((char *)v.part_lse - (char *)ctx->workspace);
    const size_t a_bytes = cfg_bytes - rope_scratch_bytes(ctx->cfg) - a_off;
    if (need <= a_bytes) {
        *region = (char *)ctx->workspace + a_off;
        *bytes = a_bytes;
        return true;
    }
    const size_t b_off = align_up(cfg_bytes, 256);
    if (ctx->workspace_bytes >= b_off + need) {
        *region = (char *)ctx->workspace + b_off;
        *bytes = ctx->workspace_bytes - b_off;
        return true;
    }
    return false;
}

// a5: picks the request-major or the chunk-major kernel for a decode launch
static int launch_decode(matkv_ctx *ctx, matkv_table *t, const AttendArgs &a, cudaStream_t stream) {
    const int64_t impl = ctx->opt_decode_impl;
    // automatic choice: chunk-major when stacking saves at least a fifth of the chunk reads
    if (t->has_fp8 && impl == 2) return fail(MATKV_E_INVALID_ARG, "the chunk-major decode does not read compressed-resident chunks");
    bool shared = !t->has_fp8 && (impl == 2 || (impl == 0 && t->share_ok && t->n_items > 0 && t->total_chunk_tiles * 4 >= t->item_tiles * 5));
    void *region = nullptr;
    size_t region_bytes = 0;
    if (shared) {
        if (!t->share_ok) return fail(MATKV_E_INVALID_ARG, "chunk-major decode does not support this head grouping");
        if (!shared_region(ctx, t, a.n_layers_launch, &region, &region_bytes)) {
            if (impl == 2)
                return fail(MATKV_E_CAPACITY, "chunk-major decode needs a workspace of %zu bytes (matkv_table_workspace_bytes), %zu given",
                            matkv_table_workspace_bytes(t, a.n_layers_launch), ctx->workspace_bytes);
            shared = false;
        }
    }
    if (shared) return launch_attend_shared(ctx, t, a, region, region_bytes, stream);
    if (impl != 1 || ctx->opt_cluster_decode == 2) {   // (an explicit request for the request-major kernel means the streaming kernel)
        if (ctx->opt_cluster_decode != 0) {
            bool taken = false;
            int rc = launch_decode_cluster(ctx, t, a, stream, &taken);
            if (rc || taken) return rc;
        }
    }
    return launch_attend_stream(ctx, t, a, stream);
}

size_t matkv_table_workspace_bytes(const matkv_table *t, int32_t n_layers_launch) {
    if (!t || n_layers_launch < 1) return 0;
    const matkv_config &c = t->ctx->cfg;
    WorkspaceView v;
    const size_t cfg_bytes = workspace_bytes_for(c, &v, nullptr);
    const size_t need = shared_region_bytes(c, t, n_layers_launch);
    const size_t a_off = (size_t)((char *)v.part_lse - (char *)nullptr);
    if (need <= cfg_bytes - rope_scratch_bytes(c) - a_off) return cfg_bytes;
    return align_up(cfg_bytes, 256) + need;
}

int matkv_table_sharing(const matkv_table *t, int64_t *logical_tiles_out, int64_t *read_tiles_out) {
    if (!t) return fail(MATKV_E_INVALID_ARG, "matkv_table_sharing: null table");
    if (logical_tiles_out) *logical_tiles_out = t->total_chunk_tiles;
    if (read_tiles_out) *read_tiles_out = t->share_ok ? t->item_tiles : t->total_chunk_tiles;
    return MATKV_OK;
}

int matkv_attend_decode(matkv_ctx *ctx, matkv_table *t, int32_t layer, const void *q, const void *kn, const void *vn,
                        void *out, float *lse_out, void *stream) {
    int rc = check_attend(ctx, t, q, kn, vn, out, 1, "matkv_attend_decode");
    if (rc) return rc;
    if (layer < 0 || layer >= ctx->cfg.n_layers) return fail(MATKV_E_INVALID_ARG, "matkv_attend_decode: layer %d", layer);
    DeviceGuard guard(ctx->device);
    const matkv_config &c = ctx->cfg;
    AttendArgs a;
    a.layer0 = layer;
    a.n_layers_launch = 1;
    a.S = 1;
    a.q = (const __nv_bfloat16 *)q;
    a.k_new = (const __nv_bfloat16 *)kn;
    a.v_new = (const __nv_bfloat16 *)vn;
    a.out = (__nv_bfloat16 *)out;
    a.lse_out = lse_out;
    a.q_sl = 0; a.q_sb = (int64_t)c.n_q_heads * c.head_dim; a.q_ss = 0;
    a.kn_sl = 0; a.kn_sb = (int64_t)c.n_kv_heads * c.head_dim; a.kn_ss = 0;
    a.lse_sl = 0; a.lse_sb = c.n_q_heads; a.lse_ss = 0;
    if (c.rope_theta != 0.f) {
        rc = launch_rope(ctx, t, a, (cudaStream_t)stream);
        if (rc) return rc;
    }
    return launch_decode(ctx, t, a, (cudaStream_t)stream);
}

int matkv_attend_decode_all_layers(matkv_ctx *ctx, matkv_table *t, const void *q, const void *kn, const void *vn,
                                   void *out, float *lse_out, void *stream) {
    int rc = check_attend(ctx, t, q, kn, vn, out, 1, "matkv_attend_decode_all_layers");
    if (rc) return rc;
    DeviceGuard guard(ctx->device);
    const matkv_config &c = ctx->cfg;
    AttendArgs a;
    a.layer0 = 0;
    a.n_layers_launch = c.n_layers;
    a.S = 1;
    a.q = (const __nv_bfloat16 *)q;
    a.k_new = (const __nv_bfloat16 *)kn;
    a.v_new = (const __nv_bfloat16 *)vn;
    a.out = (__nv_bfloat16 *)out;
    a.lse_out = lse_out;
    a.q_sb = (int64_t)c.n_q_heads * c.head_dim; a.q_sl = a.q_sb * t->batch; a.q_ss = 0;
    a.kn_sb = (int64_t)c.n_kv_heads * c.head_dim; a.kn_sl = a.kn_sb * t->batch; a.kn_ss = 0;
    a.lse_sb = c.n_q_heads; a.lse_sl = a.lse_sb * t->batch; a.lse_ss = 0;
    if (c.rope_theta != 0.f) {
        rc = launch_rope(ctx, t, a, (cudaStream_t)stream);
        if (rc) return rc;
    }
    a.advance = ctx->opt_fused_advance ? 1 : 0;   // the launch itself moves the tail by one token when it is done
    rc = launch_decode(ctx, t, a, (cudaStream_t)stream);
    if (rc == MATKV_OK && a.advance) t->tail_len_host += 1;
    return rc;
}

int matkv_attend_prefill(matkv_ctx *ctx, matkv_table *t, int32_t layer, int32_t S, const void *q, const void *kn,
                         const void *vn, void *out, float *lse_out, void *stream) {
    if (S < 1) return fail(MATKV_E_INVALID_ARG, "matkv_attend_prefill: S must be >= 1");
    int rc = check_attend(ctx, t, q, kn, vn, out, S, "matkv_attend_prefill");
    if (rc) return rc;
    if (layer < 0 || layer >= ctx->cfg.n_layers) return fail(MATKV_E_INVALID_ARG, "matkv_attend_prefill: layer %d", layer);
    DeviceGuard guard(ctx->device);
    const matkv_config &c = ctx->cfg;
    AttendArgs a;
    a.layer0 = layer;
    a.n_layers_launch = 1;
    a.S = S;
    a.q = (const __nv_bfloat16 *)q;
    a.k_new = (const __nv_bfloat16 *)kn;
    a.v_new = (const __nv_bfloat16 *)vn;
    a.out = (__nv_bfloat16 *)out;
    a.lse_out = lse_out;
    a.q_ss = (int64_t)c.n_q_heads * c.head_dim; a.q_sb = a.q_ss * S; a.q_sl = 0;
    a.kn_ss = (int64_t)c.n_kv_heads * c.head_dim; a.kn_sb = a.kn_ss * S; a.kn_sl = 0;
    a.lse_ss = c.n_q_heads; a.lse_sb = a.lse_ss * S; a.lse_sl = 0;
    if (c.rope_theta != 0.f) {
        rc = launch_rope(ctx, t, a, (cudaStream_t)stream);
        if (rc) return rc;
    }
    // long suffixes go to the tcgen05 tile kernel, short ones stay on the streaming kernel
    const int G = c.n_q_heads / c.n_kv_heads;
    // (compressed-resident chunks exist for head_dim 128 only; the tile kernel expands their codes in shared memory)
    const bool tensor_core = ctx->opt_prefill_impl >= 2 || (ctx->opt_prefill_impl == 0 && S * G >= 64);
    if (tensor_core) return launch_prefill_tc(ctx, t, a, (cudaStream_t)stream);
    return launch_attend_stream(ctx, t, a, (cudaStream_t)stream);
}

int matkv_attend_prefill_all_layers(matkv_ctx *ctx, matkv_table *t, int32_t S, const void *q, const void *kn, const void *vn,
                                    void *out, float *lse_out, void *stream) {
    if (S < 1) return fail(MATKV_E_INVALID_ARG, "matkv_attend_prefill_all_layers: S must be >= 1");
    int rc = check_attend(ctx, t, q, kn, vn, out, S, "matkv_attend_prefill_all_layers");
    if (rc) return rc;
    DeviceGuard guard(ctx->device);
    const matkv_config &c = ctx->cfg;
    AttendArgs a;
    a.layer0 = 0;
    a.n_layers_launch = c.n_layers;
    a.S = S;
    a.q = (const __nv_bfloat16 *)q;
    a.k_new = (const __nv_bfloat16 *)kn;
    a.v_new = (const __nv_bfloat16 *)vn;
    a.out = (__nv_bfloat16 *)out;
    a.lse_out = lse_out;
    a.q_ss = (int64_t)c.n_q_heads * c.head_dim; a.q_sb = a.q_ss * S; a.q_sl = a.q_sb * t->batch;
    a.kn_ss = (int64_t)c.n_kv_heads * c.head_dim; a.kn_sb = a.kn_ss * S; a.kn_sl = a.kn_sb * t->batch;
    a.lse_ss = c.n_q_heads; a.lse_sb = a.lse_ss * S; a.lse_sl = a.lse_sb * t->batch;
    if (c.rope_theta != 0.f) {
        rc = launch_rope(ctx, t, a, (cudaStream_t)stream);
        if (rc) return rc;
    }
    const int G = c.n_q_heads / c.n_kv_heads;
    // (compressed-resident chunks exist for head_dim 128 only; the tile kernel expands their codes in shared memory)
    const bool tensor_core = ctx->opt_prefill_impl >= 2 || (ctx->opt_prefill_impl == 0 && S * G >= 64);
    if (tensor_core) return launch_prefill_tc(ctx, t, a, (cudaStream_t)stream);
    // short suffixes run on the streaming kernel; when its units do not fit the workspace's counters in one
    // launch, the layers are launched one by one (same result)
    WorkspaceView ws;
    workspace_bytes_for(c, &ws, ctx->workspace);
    const int64_t n_blk = (S + kUnitRows / G - 1) / (kUnitRows / G);
    if ((int64_t)c.n_layers * t->batch * n_blk * c.n_kv_heads <= ws.n_counter_slots)
        return launch_attend_stream(ctx, t, a, (cudaStream_t)stream);
    for (int32_t layer = 0; layer < c.n_layers; ++layer) {
        AttendArgs one = a;
        one.layer0 = layer;
        one.n_layers_launch = 1;
        one.q = a.q + layer * a.q_sl; one.k_new = a.k_new + layer * a.kn_sl; one.v_new = a.v_new + layer * a.kn_sl;
        one.out = a.out + layer * a.q_sl;
        one.lse_out = a.lse_out ? a.lse_out + layer * a.lse_sl : nullptr;
        rc = launch_attend_stream(ctx, t, one, (cudaStream_t)stream);
        if (rc) return rc;
    }
    return MATKV_OK;
}

int matkv_lse_combine(matkv_ctx *ctx, int32_t n_rows, int32_t n_parts, int32_t D, const float *o_parts,
                      const float *lse_parts, void *out, float *lse_out, void *stream) {
    if (!ctx || !o_parts || !lse_parts || !out) return fail(MATKV_E_INVALID_ARG, "matkv_lse_combine: null argument");
    if (n_rows < 0 || n_parts < 1 || D < 32 || D > 256 || D % 32)
        return fail(MATKV_E_INVALID_ARG, "matkv_lse_combine: bad sizes (D must be a multiple of 32, at most 256)");
    if (n_rows == 0) return MATKV_OK;
    DeviceGuard guard(ctx->device);
    return launch_lse_combine(ctx, n_rows, n_parts, D, o_parts, lse_parts, out, lse_out, (cudaStream_t)stream);
}

int matkv_export_tail_as_chunk(matkv_ctx *ctx, matkv_table *t, int32_t req, int32_t n_tokens, void *dev_blob, void *host_blob,
                               void *stream) {
    if (!ctx || !t || !dev_blob) return fail(MATKV_E_INVALID_ARG, "matkv_export_tail_as_chunk: null argument");
    if (t->ctx != ctx) return fail(MATKV_E_INVALID_ARG, "matkv_export_tail_as_chunk: table belongs to another context");
    if (req < 0 || req >= t->batch) return fail(MATKV_E_INVALID_ARG, "matkv_export_tail_as_chunk: request %d out of range", req);
    if (n_tokens < 1 || n_tokens > t->tail_len_host)
        return fail(MATKV_E_CAPACITY, "matkv_export_tail_as_chunk: %d tokens asked, the tail holds %d", n_tokens, t->tail_len_host);
    if ((uintptr_t)dev_blob % 256) return fail(MATKV_E_ALIGNMENT, "matkv_export_tail_as_chunk: device blob must be 256-byte aligned");
    DeviceGuard guard(ctx->device);
    int rc = launch_export_tail(ctx, t, req, n_tokens, dev_blob, (cudaStream_t)stream);
    if (rc) return rc;
    if (host_blob)  // the paper's GPU -> CPU bounce buffer hop of store_KV, asynchronous on the stream
        MATKV_CUDA(cudaMemcpyAsync(host_blob, dev_blob, blob_bytes(ctx->cfg, n_tokens), cudaMemcpyDeviceToHost, (cudaStream_t)stream));
    return MATKV_OK;
}

int matkv_selftest_wait_timeout(matkv_ctx *ctx, double seconds, void *stream) {
    if (!ctx) return fail(MATKV_E_INVALID_ARG, "matkv_selftest_wait_timeout: null context");
    if (!(seconds > 0.0) || seconds > 2.0) return fail(MATKV_E_INVALID_ARG, "matkv_selftest_wait_timeout: limit must be in (0, 2] seconds");
    DeviceGuard guard(ctx->device);
    return launch_wait_selftest(ctx, seconds, (cudaStream_t)stream);
}

int matkv_probe_read(matkv_ctx *ctx, const void *dev, size_t bytes, void *stream) {
    if (!ctx || !dev) return fail(MATKV_E_INVALID_ARG, "matkv_probe_read: null argument");
    if ((uintptr_t)dev % 16 || bytes < 16) return fail(MATKV_E_ALIGNMENT, "matkv_probe_read: buffer must be 16-byte aligned and non-empty");
    DeviceGuard guard(ctx->device);
    return launch_read_probe(ctx, dev, bytes, (cudaStream_t)stream);
}

int matkv_gather_debug(matkv_ctx *ctx, matkv_table *t, int32_t layer, int32_t req, void *k_out, void *v_out,
                       int64_t capacity_rows, int64_t *rows_out, void *stream) {
    if (!ctx || !t || !k_out || !v_out) return fail(MATKV_E_INVALID_ARG, "matkv_gather_debug: null argument");
    if (t->ctx != ctx) return fail(MATKV_E_INVALID_ARG, "matkv_gather_debug: table belongs to another context");
    if (layer < 0 || layer >= ctx->cfg.n_layers || req < 0 || req >= t->batch)
        return fail(MATKV_E_INVALID_ARG, "matkv_gather_debug: layer %d / request %d out of range", layer, req);
    const int64_t rows = (int64_t)t->h_reqs[req].n_chunk_tokens + t->tail_len_host;
    if (rows_out) *rows_out = rows;
    if (rows > capacity_rows) return fail(MATKV_E_CAPACITY, "gather needs %lld rows, buffers hold %lld", (long long)rows,
                                          (long long)capacity_rows);
    if (((uintptr_t)k_out | (uintptr_t)v_out) % 16) return fail(MATKV_E_ALIGNMENT, "gather outputs must be 16-byte aligned");
    if (rows == 0) return MATKV_OK;
    if (t && t->has_fp8) return fail(MATKV_E_INVALID_ARG, "matkv_gather_debug: the table holds compressed-resident chunks");
    DeviceGuard guard(ctx->device);
    return launch_gather(ctx, t, layer, req, k_out, v_out, rows, (cudaStream_t)stream);
}

}  // extern "C"
