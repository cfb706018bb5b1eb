// Internal declarations shared by the host-side C ABI and the kernels' launchers.
#pragma once
#include <atomic>
#include <cuda.h>  // CUtensorMap (types only; the encoder is fetched through the runtime, libcuda is not linked)
#include <cuda_runtime.h>
#include <cuda_bf16.h>
#include <stdint.h>

#include <map>
#include <memory>
#include <string>
#include <unordered_map>
#include <vector>

#include "../../include/matkv.h"

namespace matkv {

constexpr int kTile = 64;          // KV tokens per streaming tile (one ring slot holds K or V of one tile)
constexpr int kMaxGridCtas = 1024; // upper bound on the streaming kernel's grid (workspace is sized for it)

// ---- device-side table --------------------------------------------------------------------
// One segment = one materialised chunk as seen by one request (device address of its blob).
struct DevSeg {
    const __nv_bfloat16 *base;  // blob [L][2][Hkv][len][D]
    int32_t len;                // tokens
    int32_t start;              // tokens before this segment in the request's logical order
    int32_t fmt;                // 0: bf16 blob; 1: compressed, HBM-resident form (see fp8_store.cu)
    int32_t pad;
};
struct DevReq {
    int32_t seg_begin;       // index of the request's first segment in the segment array
    int32_t n_seg;
    int32_t n_chunk_tokens;  // sum of len
    int32_t chunk_tiles;     // sum of ceil(len / kTile)
    int32_t pos_base;        // rotary mode: position of tail token 0
    int32_t n_parts;         // chunk-major decode: partial results the request collects (its items, then its tail)
    int32_t part_base;       // chunk-major decode: first partial slot of the request inside one (layer, KV head)
    int32_t pad;
};
// One work item of the chunk-major decode: up to `n_tiles` tiles of one chunk, read once for every
// request stacked in the item (16 / G of them at most: their G query heads fill the 16 MMA rows).
constexpr int kShareRows = 16;
struct DevItem {
    int32_t tmap;      // index of the chunk's descriptor
    int32_t len;       // chunk tokens
    int32_t tile0;     // first tile of the item inside the chunk
    int32_t n_tiles;
    int32_t n_req;     // requests stacked in the item
    int32_t last_read; // 1: no later item reads these tiles again (the chunk's last group of requests)
    int32_t pad[2];
    int32_t req[kShareRows];   // request per stacked slot
    int32_t part[kShareRows];  // partial slot of (this item, that request) inside one (layer, KV head)
    int32_t np[kShareRows];    // partials that request collects in all (its n_parts)
};

// ---- host-side objects --------------------------------------------------------------------
struct Region;    // staged slot region
struct IoEngine;  // reader threads + pinned bounce ring for file-backed chunks

// Failure of a staging call's storage reads: the host's flag, and a page-locked word of the reader engine that a
// one-thread kernel behind the call's copies looks at (one word per call in flight, so that a later call that went
// well does not inherit an earlier call's failure).
struct FailFlag {
    std::atomic<int> host{0};
    volatile int *word = nullptr;
};

struct Chunk {
    int32_t n_tokens = 0;
    const void *host_blob = nullptr;
    bool host_device_readable = false;  // host_blob is page-locked (or managed) memory a kernel may read over the link
    int file_fd = -1;              // >= 0: the blob lives in a file, at file_offset
    uint64_t file_offset = 0;
    void *dev_blob = nullptr;      // caller-resident device copy
    bool fp8 = false;              // host_blob / the file holds the compressed form (e4m3 codes + block exponents)
    bool resident_fp8 = false;     // the staged device copy is the compressed, HBM-resident form
    alignas(64) CUtensorMap tmap8[2];  // resident form: K codes [rows][D] (128-byte swizzle), V codes transposed per block [rows][64] (64-byte swizzle)
    void *staged = nullptr;        // device copy inside a slot region (or nullptr)
    Region *region = nullptr;
    int32_t slot = -1;
    cudaEvent_t ready = nullptr;   // event of the staging call that (last) copied it; borrowed from the ticket, null once
                                   // that call has been seen complete (the ticket is retired then and its event destroyed)
    uint64_t ticket = 0;
    std::shared_ptr<FailFlag> io_failed;  // set by the storage tier when a read of that staging call failed
    alignas(64) CUtensorMap tmap;  // 2-D view [rows][D] of the current device copy, 64 x kTile boxes, 128-byte swizzle
};

struct Region {
    void *base = nullptr;
    size_t slot_bytes = 0;
    int32_t n_slots = 0;
    std::vector<uint64_t> occupant;  // chunk id per slot
    std::vector<uint8_t> used;
    cudaEvent_t last_use = nullptr;  // recorded by matkv_table_free
    bool has_last_use = false;
};

struct Grave {        // a freed table's image, until the stream work that may still read it is done
    cudaEvent_t ev;
    void *h_pinned;
    void *d_image;
    size_t bytes;
};
struct PooledImage {  // a table image (pinned upload buffer + device copy) ready for reuse
    void *h_pinned;
    void *d_image;
    size_t bytes;
};

struct Ticket {
    cudaEvent_t done = nullptr;
    std::vector<uint64_t> chunk_ids;              // chunks whose `ready` borrows the event
    std::shared_ptr<FailFlag> io_failed;  // shared with the storage tier's read jobs of this call
};

}  // namespace matkv

struct matkv_ctx {
    matkv_config cfg;
    int device = 0;
    float scale = 0.f;
    int n_sm = 0;
    int32_t *d_status = nullptr;
    void *workspace = nullptr;
    size_t workspace_bytes = 0;
    int64_t opt_decode_ctas = 0, opt_prefill_impl = 0, opt_prefill_ctas = 0, opt_stage_ctas = 0, opt_fused_advance = 0;
    int64_t opt_decode_impl = 0, opt_share_tiles = 16, opt_fp8_resident = 0;
    std::unordered_map<uint64_t, matkv::Chunk> chunks;
    std::map<void *, matkv::Region *> regions;
    std::unordered_map<uint64_t, matkv::Ticket> tickets;   // staging calls not yet seen complete
    std::vector<uint64_t> failed_tickets;                  // retired tickets whose storage reads failed
    uint64_t next_ticket = 1;
    int64_t opt_io_timeout_ms = 30000, opt_io_test_delay_ms = 0;
    int64_t opt_cluster_decode = 1, opt_cluster_max = 0;
    std::vector<matkv_table *> tables;
    matkv::IoEngine *io = nullptr;
    std::vector<matkv::PooledImage> image_pool;
    std::vector<matkv::Grave> image_graves;
};

struct matkv_table {
    matkv_ctx *ctx = nullptr;
    int32_t batch = 0;
    int32_t n_seg_total = 0;
    std::vector<matkv::DevSeg> h_segs;
    std::vector<matkv::DevReq> h_reqs;
    int32_t tail_len_host = 0;   // host mirror (not moved by graph replays)
    int32_t max_chunk_tiles = 0;
    int64_t total_chunk_tiles = 0;
    int64_t distinct_chunk_tiles = 0;  // tiles of the distinct device copies the requests list
    void *h_pinned = nullptr;    // pinned upload image
    void *d_image = nullptr;     // device image: segs | reqs | tail_len[B]
    size_t image_bytes = 0, image_alloc = 0;
    matkv::DevSeg *d_segs = nullptr;
    matkv::DevReq *d_reqs = nullptr;
    int32_t *d_tail_len = nullptr;
    CUtensorMap *d_tmaps = nullptr;  // one per segment, then the K tail and the V tail
    CUtensorMap *d_tmaps8 = nullptr; // two per segment (K codes, transposed V codes) when the table has compressed-resident chunks
    bool has_fp8 = false;            // some segment is compressed-resident: only the streaming kernel reads those
    int4 *d_tile_dir = nullptr;      // one record per chunk tile of every request, in the request's order:
                                     // {descriptor index, first row inside the chunk, chunk tokens, valid rows}
    std::vector<int32_t> h_dir_begin;  // first record of each request
    matkv::DevItem *d_items = nullptr;  // chunk-major decode: the chunk items of one (layer, KV head)
    bool share_ok = false;              // the head grouping fits the chunk-major kernel
    int32_t n_items = 0;                // chunk items (the requests' tail items follow implicitly)
    int32_t parts_total = 0;            // partial slots of one (layer, KV head): sum of the requests' n_parts
    int64_t item_tiles = 0;             // tiles the chunk items read per (layer, KV head); total_chunk_tiles is the logical count
    __nv_bfloat16 *tail_k = nullptr, *tail_v = nullptr;
    std::vector<matkv::Region *> regions;  // staged regions this table reads
};

namespace matkv {

// makes `dev` the current device for the scope (and restores the previous one)
struct DeviceGuard {
    int prev = -1;
    bool switched = false;
    explicit DeviceGuard(int dev) {
        if (cudaGetDevice(&prev) == cudaSuccess && prev != dev) switched = (cudaSetDevice(dev) == cudaSuccess);
    }
    ~DeviceGuard() {
        if (switched) cudaSetDevice(prev);
    }
};

int fail(int code, const char *fmt, ...);   // records the thread-local message, returns code
int cuda_fail(cudaError_t e, const char *what);
#define MATKV_CUDA(x)                                              \
    do {                                                           \
        cudaError_t e__ = (x);                                     \
        if (e__ != cudaSuccess) return ::matkv::cuda_fail(e__, #x); \
    } while (0)

// The opt-in shared-memory size of a kernel is a per-device attribute: launchers keep one flag per device ordinal.
struct PerDeviceOnce {
    std::atomic<bool> done[64] = {};
    // true until done() has been called on the current device.  Two host threads (two contexts) may both see true
    // and both run the one-time step, which is harmless for what it guards (setting a kernel attribute); neither
    // launches before the step has been done.
    bool need(int *dev_out) {
        int dev = 0;
        if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) dev = -1;
        *dev_out = dev;
        return dev < 0 || !done[dev].load(std::memory_order_acquire);
    }
    void mark(int dev) {
        if (dev >= 0) done[dev].store(true, std::memory_order_release);
    }
};

constexpr int kUnitRows = 8;  // query rows (suffix tokens x heads of one KV group) one streaming unit carries

// 2-D tensor map over `rows` rows of D bf16 starting at `base` (box 64 x kTile, 128-byte swizzle, zero fill)
int encode_rows_map(CUtensorMap *out, const void *base, int D, uint64_t rows);
// 3-D tensor map over new-token rows [n_tok][Hkv][D]: box 64 columns x 1 head x kTile tokens, 128-byte swizzle
int encode_new_rows_map(CUtensorMap *out, const void *base, int D, int Hkv, uint64_t n_tok);

// Workspace layout: [counters: int32 x n_counter_slots][lse parts: fp32][o parts: fp32]
struct WorkspaceView {
    int32_t *counters;
    float *part_lse;   // [n_part_slots][kUnitRows]
    float *part_o;     // [n_part_slots][kUnitRows][D]
    int64_t n_counter_slots, n_part_slots;
};
size_t workspace_bytes_for(const matkv_config &c, WorkspaceView *view_from_base, void *base);
size_t rope_scratch_bytes(const matkv_config &c);  // rotated q / k_new of one call (0 unless rotary mode)

// ---- launchers (defined next to their kernels) ----------------------------------------------
struct AttendArgs {
    // which units
    int32_t layer0, n_layers_launch, S;
    // inputs / outputs (bf16 device) and their element strides per (layer, request, suffix token)
    const __nv_bfloat16 *q, *k_new, *v_new;
    __nv_bfloat16 *out;
    float *lse_out;
    int64_t q_sl, q_sb, q_ss;     // q / out strides: layer, request, token (elements)
    int64_t kn_sl, kn_sb, kn_ss;  // k_new / v_new strides
    int64_t lse_sl, lse_sb, lse_ss;
    int32_t advance = 0;          // streaming kernel only: tokens the launch adds to the tail lengths when it is done
};
int launch_attend_stream(matkv_ctx *ctx, matkv_table *t, const AttendArgs &a, cudaStream_t stream);
// decode step of one layer of a small batch as thread-block clusters; *taken = false when the launch does not fit it
int launch_decode_cluster(matkv_ctx *ctx, matkv_table *t, const AttendArgs &a, cudaStream_t stream, bool *taken);
// chunk-major decode (S = 1): region = scratch for the partials, region_bytes its size
int launch_attend_shared(matkv_ctx *ctx, matkv_table *t, const AttendArgs &a, void *region, size_t region_bytes, cudaStream_t stream);
size_t shared_region_bytes(const matkv_config &c, const matkv_table *t, int n_layers_launch);
int launch_rope(matkv_ctx *ctx, matkv_table *t, AttendArgs &a, cudaStream_t stream);
int launch_prefill_tc(matkv_ctx *ctx, matkv_table *t, const AttendArgs &a, cudaStream_t stream);
int launch_lse_combine(matkv_ctx *ctx, int32_t n_rows, int32_t n_parts, int32_t D, const float *o_parts,
                       const float *lse_parts, void *out, float *lse_out, cudaStream_t stream);
int launch_gather(matkv_ctx *ctx, matkv_table *t, int32_t layer, int32_t req, void *k_out, void *v_out,
                  int64_t rows, cudaStream_t stream);
int io_engine_create(matkv_ctx *ctx, void *pinned, size_t bytes, size_t slab_bytes, int n_threads);
void io_engine_destroy(matkv_ctx *ctx);
void io_engine_configure(matkv_ctx *ctx);   // takes the read time limit (and the injected read delay) over from the context's options
size_t io_engine_slab_bytes(const matkv_ctx *ctx);
int io_engine_errors(matkv_ctx *ctx, const char **msg);
// fp8_tokens > 0: the file holds a compressed chunk of that many tokens; on its way from the slab to dst it is expanded to
// bf16 (fp8_resident false) or re-laid out into the HBM-resident compressed form (true)
int io_engine_stage(matkv_ctx *ctx, int fd, uint64_t offset, size_t bytes, void *dst, cudaStream_t copy_stream,
                    const std::shared_ptr<FailFlag> &failed, int32_t fp8_tokens = 0, bool fp8_resident = false);
// one tiny launch on the copy stream that turns a failed read of the calls so far into MATKV_E_IO in the status word
int io_engine_flag_status(matkv_ctx *ctx, const std::shared_ptr<FailFlag> &failed, cudaStream_t copy_stream);
// gives a staging call its page-locked failure word (cleared); no-op without a reader engine
void io_engine_bind_fail_word(matkv_ctx *ctx, uint64_t ticket, FailFlag *flag);
size_t fp8_codes_bytes(const matkv_config &c, int32_t n_tokens);
size_t fp8_blob_bytes(const matkv_config &c, int32_t n_tokens);
int launch_quantize_fp8(matkv_ctx *ctx, const void *dev_blob, int32_t n_tokens, void *dev_fp8, cudaStream_t stream);
size_t fp8_resident_bytes(const matkv_config &c, int32_t n_tokens);
int launch_stage_relayout_fp8(matkv_ctx *ctx, const void *src_fp8, void *dev_dst, int32_t n_tokens, cudaStream_t stream);
int encode_fp8_maps(CUtensorMap *out2, const void *dev_resident, const matkv_config &c, int32_t n_tokens);
int launch_stage_expand_fp8(matkv_ctx *ctx, const void *src_fp8, void *dev_dst, int32_t n_tokens, int n_ctas, cudaStream_t stream);
int open_chunk_file(const char *path, uint64_t offset, size_t bytes, int *fd_out);
void close_chunk_file(int fd);
int launch_wait_selftest(matkv_ctx *ctx, double seconds, cudaStream_t stream);
int launch_stage_copy(matkv_ctx *ctx, const void *host_src, void *dev_dst, size_t bytes, int n_ctas, cudaStream_t stream);
int launch_export_tail(matkv_ctx *ctx, matkv_table *t, int32_t req, int32_t n_tokens, void *dev_blob, cudaStream_t stream);
int launch_read_probe(matkv_ctx *ctx, const void *dev, size_t bytes, cudaStream_t stream);
int launch_add_tail_len(matkv_table *t, int32_t delta, int32_t set_value, bool set, cudaStream_t stream);

}  // namespace matkv
