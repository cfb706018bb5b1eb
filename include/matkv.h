/*
 * matkv.h -- C ABI of the B200 (sm_100a) attention path that remains on the GPU
 * in MatKV-style retrieval-augmented inference.
 *
 * Method (paper, Section III-B and Section IV): the K,V tensors of every
 * document chunk are computed once, each chunk alone with its tokens at
 * positions 0..len-1, stored under a chunk id, and at request time loaded
 * instead of recomputed and placed BEFORE the query.  Only the query suffix
 * (the "sub-prefill" after loading) and the generated tokens attend to them.
 * This library computes that attention directly over the scattered chunk
 * buffers: no concatenated copy is ever made.
 *
 * Conventions
 *   - every function returns MATKV_OK (0) or a negative MATKV_E_* code and never
 *     throws; matkv_last_error() gives a thread-local text for the last failure;
 *   - "device" pointers are CUDA device memory of the context's GPU, "host"
 *     pointers are ordinary or pinned host memory, as stated per argument;
 *   - streams are cudaStream_t passed as void* (NULL = the legacy default stream);
 *   - all attend / stage / table calls are asynchronous on the given stream and
 *     validate their arguments on the host before anything is launched;
 *   - the library allocates only small tables; chunk blobs, slots, tails,
 *     workspace, queries and outputs are owned by the caller and BORROWED;
 *   - problems only the device can see (a bounds check, a bounded wait that ran
 *     out) are written to a device status word, read with matkv_status();
 *   - one context serves one stream of attend calls at a time (they share the
 *     workspace); calls from several host threads on one context must be
 *     serialised by the caller.
 *
 * Data layouts (bf16 = 2-byte bfloat16, fp32 accumulation everywhere)
 *   chunk blob   [n_layers][2 (K, then V)][n_kv_heads][n_tokens][head_dim] bf16,
 *                contiguous, base 256-byte aligned.  K is stored as the model
 *                produced it (already rotated for positions 0..n_tokens-1) and is
 *                never modified or re-rotated.
 *   tail         [batch][n_layers][n_kv_heads][max_tail_tokens][head_dim] bf16, one
 *                buffer for K and one for V: the K,V of the query suffix and of the
 *                generated tokens.  Must not hold NaN/Inf bit patterns (zero it once).
 *   grouped-query attention: query head h reads KV head floor(h / G), G = Hq / Hkv.
 */
#ifndef MATKV_H
#define MATKV_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define MATKV_OK               0
#define MATKV_E_INVALID_ARG   (-1)
#define MATKV_E_UNKNOWN_CHUNK (-2)
#define MATKV_E_NOT_STAGED    (-3)  /* chunk has no device copy (never staged or evicted)   */
#define MATKV_E_NOT_READY     (-4)  /* an asynchronous copy has not finished yet             */
#define MATKV_E_CAPACITY      (-5)  /* too many chunks / slots / tail tokens / batch          */
#define MATKV_E_ALIGNMENT     (-6)
#define MATKV_E_CUDA          (-7)
#define MATKV_E_TIMEOUT       (-8)  /* device status: a bounded wait inside a kernel ran out */
#define MATKV_E_BOUNDS        (-9)  /* device status: a table-derived index was out of range */
#define MATKV_E_IO            (-10) /* a chunk file could not be opened or read                */

typedef struct matkv_ctx matkv_ctx;     /* opaque; owned by the library            */
typedef struct matkv_table matkv_table; /* opaque; one per in-flight request batch */

typedef struct {
    int32_t n_layers, n_q_heads, n_kv_heads;
    int32_t head_dim;            /* 64 or 128                                               */
    int32_t max_batch;           /* requests per table, 1..1024                             */
    int32_t max_chunks_per_req;  /* upper bound on a request's chunk list                   */
    int32_t max_tail_tokens;     /* capacity of each request's tail (suffix + generated)    */
    float softmax_scale;         /* 0 => 1/sqrt(head_dim)                                   */
    float rope_theta;            /* 0 => q and k_new arrive already rotated (default)       */
    int32_t pos_mode;            /* rotary mode only: position of the first tail token.
                                    0 = sum of the request's chunk lengths (the query continues
                                    after the documents, each of which starts at position 0);
                                    1 = longest chunk length; 2 = given per request with
                                    matkv_table_set_pos_base (until then as mode 0).  The paper
                                    fixes the documents' positions (each starts at the first input
                                    position, Section III-B) and is silent on the query's, hence a
                                    parameter.  Inert when rope_theta == 0.                      */
    int32_t device;              /* CUDA device ordinal, -1 = current device                */
} matkv_config;

/* options for matkv_set_option */
#define MATKV_OPT_DECODE_CTAS   1  /* number of CTAs the streaming kernel splits the KV over; 0 = auto: one per SM,
                                      less MATKV_OPT_STAGE_CTAS when the staging copy kernel is in use */
#define MATKV_OPT_PREFILL_IMPL  2  /* 0 = auto (tensor-core tiles when the suffix is large enough),
                                      1 = force the streaming kernel, 2 = force the tensor-core kernel,
                                      3 = tensor-core kernel with two 128-row blocks per CTA whenever a
                                          (request, KV head) has more than 128 query rows */
#define MATKV_OPT_STAGE_CTAS    4  /* 0 = stage host blobs with the copy engine (cudaMemcpyAsync); n > 0 = with a copy
                                      kernel of n small CTAs that runs beside the decode CTAs (the host blobs must
                                      then be pinned, device-accessible memory) */
#define MATKV_OPT_DECODE_ADVANCES_TAIL 5  /* 1 = matkv_attend_decode_all_layers adds one token to every request's tail
                                             length itself when the launch is done (its last CTA does it), so the caller
                                             omits matkv_table_advance between decode steps; 0 (default) = it does not */
#define MATKV_OPT_DECODE_IMPL   6  /* decode kernel: 0 = auto (chunk-major when the batch's requests share chunks and the
                                      workspace has room for its partials), 1 = request-major always, 2 = chunk-major
                                      always (MATKV_E_CAPACITY when the workspace is too small) */
#define MATKV_OPT_SHARE_TILES   7  /* chunk-major decode: 64-token tiles per work item (default 16); read when a table is built */
#define MATKV_OPT_FP8_RESIDENT  8  /* staging of compressed chunks (matkv_register_chunk_fp8 / _file_fp8): 0 (default) = expand
                                      to the bf16 blob in HBM; 1 = keep them compressed in HBM too (head_dim 128 only): the
                                      streaming kernel then reads the codes and converts in registers, halving the HBM bytes of
                                      decode; the tensor-core sub-prefill expands their code tiles to bf16 in shared memory (one row
                                      block per CTA); the chunk-major decode, the cluster decode (such launches take the streaming
                                      kernel), the allocation-free decode and matkv_gather_debug do not read tables that hold them */
#define MATKV_OPT_PREFILL_CTAS  3  /* CTAs per (request, KV head) the tensor-core prefill splits the KV over; 0 = auto */
#define MATKV_OPT_CLUSTER_DECODE 11 /* matkv_attend_decode (one layer per launch): 1 (default) = served by thread-block clusters, one
                                      cluster of up to 16 CTAs per (request, KV head), two CTAs per SM, whose CTAs merge their partials
                                      through distributed shared memory (no workspace traffic) and fetch their first chunk tiles under
                                      the previous kernel's tail; measured 5 - 25 % faster than the streaming kernel for launches of
                                      1 to 64 requests; 0 = always the streaming kernel; 2 = clusters even when MATKV_OPT_DECODE_IMPL
                                      is 1.  Launches it cannot spread over enough CTAs, tables with compressed-resident chunks and
                                      all-layers launches use the streaming kernel.  A captured (graph) launch balances its shares for
                                      the tail length at capture time and stays exact as the tail grows; re-capture now and then in a
                                      long generation to keep the balance */
#define MATKV_OPT_CLUSTER_MAX 12   /* largest cluster (CTAs per request and KV head) the cluster decode may use; 0 (default) = automatic */
#define MATKV_OPT_IO_TIMEOUT_MS 9  /* storage tier: how long the copy stream waits for one chunk's read before the staging call
                                      is marked failed (MATKV_E_IO) and the stream moves on; default 30,000 ms */
#define MATKV_OPT_IO_TEST_DELAY_MS 10 /* failure injection on the host, for tests: every storage read sleeps this long first
                                         (0 = off); with a time limit below it the reads "hang" without any GPU fault */

/* ---- context -------------------------------------------------------------------------- */
/* Creates a context on cfg->device.  Allocates the device status word and nothing large.   */
int matkv_create(const matkv_config *cfg, matkv_ctx **out);
/* Destroys the context and every table built from it.  Borrowed buffers are not touched.   */
int matkv_destroy(matkv_ctx *ctx);
const char *matkv_last_error(void);
int matkv_set_option(matkv_ctx *ctx, int32_t option, int64_t value);

/* Scratch memory for the split-KV partial results (fp32 o and log-sum-exp per part) and the
 * per-unit arrival counters.  matkv_workspace_bytes() is the size needed for the largest
 * launch the configuration allows; matkv_set_workspace() borrows `dev` (256-byte aligned
 * device memory) and clears its counter region with a synchronous memset.                  */
size_t matkv_workspace_bytes(const matkv_ctx *ctx);
int matkv_set_workspace(matkv_ctx *ctx, void *dev, size_t bytes);

/* Reads the device status word (synchronises the context's device first): 0 or MATKV_E_*.
 * `clear` != 0 resets it.                                                                  */
int matkv_status(matkv_ctx *ctx, int32_t *dev_status_out, int32_t clear);

/* ---- a1: chunk registry (the paper's "file named chunk_id"; Section IV, store_KV) ------- */
/* Records where the materialised K,V of `chunk_id` live.  host_blob: pinned (or pageable)
 * host memory or NULL (a pageable blob is always staged by the copy engine, whatever
 * MATKV_OPT_STAGE_CTAS says: only page-locked memory can be read by the copy kernel); dev_blob: device memory or NULL; at least one non-NULL.  Both are
 * borrowed until matkv_unregister_chunk / matkv_destroy.  Re-registering an id is an error.
 * A chunk is immutable (the method's premise): the device copy a table points at must not be
 * written while the table is in use, not even by earlier work on the same stream, because an
 * attend launch may fetch chunk rows before the kernel queued before it has finished.        */
int matkv_register_chunk(matkv_ctx *ctx, uint64_t chunk_id, int32_t n_tokens, const void *host_blob,
                         void *dev_blob);
/* The same for a chunk whose blob is stored in a file, `blob bytes` long at file_offset: the paper's
 * materialised-KV store keeps one raw-bytes file per chunk id on flash (Section IV, store_KV /
 * load_KV).  The file is opened now (O_DIRECT when offset and size are multiples of 4096 and the file
 * system allows it) and stays open until unregister / destroy.  Such a chunk is staged through the
 * bounce buffer set with matkv_set_bounce_buffer.                                                    */
int matkv_register_chunk_file(matkv_ctx *ctx, uint64_t chunk_id, int32_t n_tokens, const char *path, uint64_t file_offset);
/* Lends the library a pinned host ring for file-backed chunks (the paper's CPU bounce buffer between
 * SSD and GPU, Section IV): `bytes` of page-locked host memory, 4096-byte aligned, cut into slabs of
 * slab_bytes (>= the largest file-backed chunk, a multiple of 4096, at least two slabs), and starts
 * n_io_threads reader threads.  Storage reads, host-to-device copies and GPU work then overlap.      */
int matkv_set_bounce_buffer(matkv_ctx *ctx, void *pinned_host, size_t bytes, size_t slab_bytes, int32_t n_io_threads);
/* ---- compressed chunk store (the paper names KV compression as the lever on the storage cost of
 *      materialised KVs, in its discussion of total cost of ownership, without fixing a format) ----------
 * Format taken here: e4m3 codes (1-4-3 bits, bias 7, largest finite 448) with one power-of-two scale 2^e per
 * block of 64 consecutive tokens of a (layer, K or V, KV head) slab; a code stands for value(code) * 2^e,
 * always a bf16 number.  e = the smallest integer with amax * 2^-e <= 448 (0 for an all-zero block, clamped
 * to [-127, 127]); code = nearest e4m3 to x * 2^-e, ties to even, zero unsigned.  Inputs must be finite.
 * Compressed blob: codes [n_layers][2][n_kv_heads][n_tokens][head_dim] (bytes), then, at the next multiple
 * of 256 bytes, exponents [n_layers][2][n_kv_heads][ceil(n_tokens / 64)] (int8).  It halves the bytes on
 * storage and on the host-to-device link; staging expands it to the ordinary bf16 chunk blob in HBM (exactly),
 * so tables and attention calls do not change.
 *   matkv_fp8_blob_bytes     size of the compressed blob of an n_tokens chunk (a multiple of 256).
 *   matkv_quantize_chunk_fp8 bf16 chunk blob (device) -> compressed blob (device, 256-byte aligned), on `stream`;
 *                            the materialisation side: copy the result to the host or a file afterwards.
 *   matkv_register_chunk_fp8 like matkv_register_chunk for a compressed blob in PINNED host memory (256-byte
 *                            aligned; the expanding copy kernel reads it over the link, MATKV_OPT_STAGE_CTAS
 *                            CTAs, 16 when that option is 0).  Slots are sized for the bf16 blob.
 *   matkv_register_chunk_file_fp8  the same for a compressed blob stored in a file (see
 *                            matkv_register_chunk_file); it passes through the pinned bounce ring.             */
size_t matkv_fp8_blob_bytes(const matkv_ctx *ctx, int32_t n_tokens);
/* device slot bytes a compressed chunk needs when it stays compressed in HBM (MATKV_OPT_FP8_RESIDENT = 1) */
size_t matkv_fp8_resident_bytes(const matkv_ctx *ctx, int32_t n_tokens);
int matkv_quantize_chunk_fp8(matkv_ctx *ctx, const void *dev_blob, int32_t n_tokens, void *dev_blob_fp8, void *stream);
int matkv_register_chunk_fp8(matkv_ctx *ctx, uint64_t chunk_id, int32_t n_tokens, const void *host_blob_fp8);
int matkv_register_chunk_file_fp8(matkv_ctx *ctx, uint64_t chunk_id, int32_t n_tokens, const char *path, uint64_t file_offset);

/* The paper's delete(O) (Section IV): forgets the chunk.  Tables built earlier keep the
 * device address they resolved; the caller keeps that memory alive until they are freed.    */
int matkv_unregister_chunk(matkv_ctx *ctx, uint64_t chunk_id);

/* ---- a2: staging (the paper's load_KV, CPU bounce buffer -> GPU; Section IV, and the
 *      overlap of the next batch's load with the current decode, Section III-C) ------------ */
/* Copies the listed chunks' host blobs into `dev_slots` (n_slots slots of slot_bytes each,
 * device memory, 256-byte aligned, borrowed) with one asynchronous copy per chunk on
 * `copy_stream`, and records an event per call.  Duplicates in the list, chunks registered
 * with a dev_blob, and chunks already sitting in this same slot region are not copied again;
 * every other previous occupant of the region is evicted.  Before overwriting, copy_stream is
 * made to wait for the last table that used the region (see matkv_table_free).  *ticket_out
 * identifies the call for matkv_stage_query / matkv_stage_wait.  Never blocks the host.       */
int matkv_stage_chunks_async(matkv_ctx *ctx, const uint64_t *chunk_ids, int32_t n, void *dev_slots,
                             size_t slot_bytes, int32_t n_slots, void *copy_stream, uint64_t *ticket_out);
/* MATKV_OK when the ticket's copies have finished, MATKV_E_NOT_READY otherwise (no blocking). */
int matkv_stage_query(matkv_ctx *ctx, uint64_t ticket);
/* Blocks the calling host thread until the ticket's copies have finished.                     */
int matkv_stage_wait(matkv_ctx *ctx, uint64_t ticket);
/* Both return MATKV_E_IO when a storage read of that call failed or did not return within the
 * time limit (the slots of its chunks then hold garbage): a later matkv_build_chunk_table over
 * such a chunk is refused with MATKV_E_IO once the failure is known, and the device status
 * word reads MATKV_E_IO as soon as the copy stream has passed the call, so that attention
 * launched behind it without any host wait is flagged too.  A ticket that has been seen
 * complete (by these calls, or by a later staging call) is retired: its event is destroyed
 * and it keeps answering MATKV_OK / MATKV_E_IO.
 * matkv_stage_pending: number of staging calls not yet seen complete.                         */
int matkv_stage_pending(matkv_ctx *ctx, int32_t *n_out);

/* ---- a3: chunk table (replaces the concatenation of put_KV, Section IV) ------------------ */
/* chunk_ids_flat is the concatenation of each request's ORDERED id list (documents before
 * the query, Section III-B); n_chunks_per_req[r] may be 0 and ids may repeat.  tail_k / tail_v:
 * device tails (layout above, batch = `batch`), borrowed, written by the attend calls.
 * Resolves every id to its device copy (MATKV_E_NOT_STAGED if it has none), makes `stream`
 * wait for the staging copies it depends on (never the host), uploads the table on `stream`
 * and sets every request's tail length to 0.                                                 */
int matkv_build_chunk_table(matkv_ctx *ctx, int32_t batch, const int32_t *n_chunks_per_req,
                            const uint64_t *chunk_ids_flat, void *tail_k, void *tail_v, void *stream,
                            matkv_table **out);
/* Marks, on `stream`, the end of the table's use of staged slot regions (so that a later
 * matkv_stage_chunks_async into them waits for it) and frees the table stream-ordered.        */
int matkv_table_free(matkv_table *table, void *stream);
/* Adds n_tokens to every request's tail length (device-side counter, so a captured decode
 * loop can replay it).  Attend calls never move it: all layers of one step see one length.
 * The library also keeps a host-side copy of the length, moved by these two calls (and by a
 * decode launch that advances the tail itself) when they are made, not when a captured graph
 * is replayed.  Attend calls outside stream capture split their work by the host-side copy
 * (they can then start before the previous kernel on the stream has finished) and compare it
 * with the device counter: after replaying a captured loop, call matkv_table_set_tail_len
 * before the next attend call outside a capture, or that launch reports MATKV_E_BOUNDS in
 * the device status and its output is void (a launch served by the cluster kernel, see
 * MATKV_OPT_CLUSTER_DECODE, uses the host-side copy for balance only and is right anyway). */
int matkv_table_advance(matkv_table *table, int32_t n_tokens, void *stream);
int matkv_table_set_tail_len(matkv_table *table, int32_t tail_len, void *stream);
/* pos_mode 2 only: sets, on `stream`, the position of the first tail token of every request
 * (pos_base: host array of `batch` non-negative values, read before the call returns).  Tail
 * token i of request r is then rotated at pos_base[r] + i.  Call it before the first attend
 * call of the table.                                                                          */
int matkv_table_set_pos_base(matkv_table *table, const int32_t *pos_base, void *stream);

/* ---- a4: query sub-prefill (Section V-A "Prefill time": from the end of loading to the
 *      first token; the query is prefilled on top of the loaded KVs) ----------------------- */
/* q [B][S][Hq][D], k_new / v_new [B][S][Hkv][D], out [B][S][Hq][D] bf16 device; lse_out NULL
 * or [B][S][Hq] fp32 device (natural log).  Writes k_new / v_new to tail[t0 .. t0+S) of
 * `layer` (t0 = current tail length) and lets suffix token i attend to every chunk token and
 * to tail[0 .. t0+i].  In rotary mode q and k_new are rotated at position base + t0 + i first. */
int matkv_attend_prefill(matkv_ctx *ctx, matkv_table *table, int32_t layer, int32_t S, const void *q,
                         const void *k_new, const void *v_new, void *out, float *lse_out, void *stream);

/* The same for every layer in ONE launch: q [L][B][S][Hq][D], k_new / v_new [L][B][S][Hkv][D], out
 * [L][B][S][Hq][D], lse_out NULL or [L][B][S][Hq].  Like matkv_attend_decode_all_layers, only usable
 * when all layers' inputs exist up front (an attention-only benchmark).                              */
int matkv_attend_prefill_all_layers(matkv_ctx *ctx, matkv_table *table, int32_t S, const void *q, const void *k_new,
                                    const void *v_new, void *out, float *lse_out, void *stream);

/* ---- a5 + a6: decode step (Section V-A "Decode time"; memory-bound streaming over the
 *      loaded KVs) with split-KV partials merged by log-sum-exp ---------------------------- */
/* One new token per request.  q [B][Hq][D], k_new / v_new [B][Hkv][D], out [B][Hq][D] bf16
 * device; lse_out NULL or [B][Hq] fp32.  Writes k_new / v_new to tail[t0] of `layer` and
 * attends to every chunk token and to tail[0 .. t0].                                         */
int matkv_attend_decode(matkv_ctx *ctx, matkv_table *table, int32_t layer, const void *q, const void *k_new,
                        const void *v_new, void *out, float *lse_out, void *stream);
/* The same for every layer in ONE launch: q [L][B][Hq][D], k_new / v_new [L][B][Hkv][D],
 * out [L][B][Hq][D], lse_out NULL or [L][B][Hq].  Only usable when all layers' queries exist
 * up front (an attention-only benchmark; a real model produces layer l+1's q from layer l).  */
int matkv_attend_decode_all_layers(matkv_ctx *ctx, matkv_table *table, const void *q, const void *k_new,
                                   const void *v_new, void *out, float *lse_out, void *stream);

/* The decode step of one layer (same arguments, same result as matkv_attend_decode) for callers that
 * must not allocate device memory and have none to lend as a workspace: for example a serving process
 * that has handed all of HBM to its own KV pool, where a cudaMalloc would fail or stall every stream
 * while the driver synchronises, or a plug-in running under a host that forbids allocation after
 * start-up.  The paper has no counterpart; this is a packaging variant of a5 + a6.
 *   - The split-KV partials and arrival counters live in an array built into the library
 *     (2,114,560 bytes of device memory per GPU that loads it, held until the process exits) instead
 *     of the workspace given to matkv_set_workspace, which this call neither needs nor touches.
 *   - Limits: batch x n_kv_heads <= 256 and head_dim <= 128; larger calls return MATKV_E_CAPACITY.  Two kinds of
 *     call are refused with MATKV_E_INVALID_ARG: a context in rotary mode (rope_theta != 0: the rotated q / k_new
 *     would need scratch of their own) and a table that holds compressed-resident chunks.
 *   - Nothing is allocated or freed: no cudaMalloc / cudaFree and no allocating library routine.  The
 *     first call on a device looks up the array's device address (cudaGetSymbolAddress); make that
 *     first call outside any stream capture.
 *   - All calls share the one array and it keeps the previous call's contents; each call clears its
 *     arrival counters on `stream` before the kernel.  Two calls that overlap on the GPU (different
 *     streams, or different contexts on one device) race on it: serialise them.                      */
int matkv_attend_decode_static(matkv_ctx *ctx, matkv_table *table, int32_t layer, const void *q, const void *k_new,
                               const void *v_new, void *out, float *lse_out, void *stream);

/* Chunk-major decode for batches whose requests share chunks (the paper's skewed retrieval: a few
 * materialised chunks take most of the hits, Section II-C).  matkv_attend_decode and
 * matkv_attend_decode_all_layers then read a chunk listed by several requests of the table ONCE per
 * layer and KV head: the requests' query heads are stacked into one tensor-core tile (16 / G requests;
 * more requests repeat the read right away, where it hits L2), every (chunk, request) pair leaves a
 * partial result and the last one merges the request's partials by log-sum-exp.  Same results as the
 * request-major kernel up to summation order.  Two chunks are "the same" when they resolve to the same
 * device copy and length.
 *   matkv_table_sharing: chunk tiles (64 tokens) the table's requests list per layer and KV head, and
 *     the tiles the chunk-major kernel reads for them (either pointer may be NULL).
 *   matkv_table_workspace_bytes: size the workspace given to matkv_set_workspace must have for
 *     chunk-major launches of n_layers_launch layers on this table (never less than
 *     matkv_workspace_bytes); with a smaller workspace the automatic choice stays request-major.      */
int matkv_table_sharing(const matkv_table *table, int64_t *logical_tiles_out, int64_t *read_tiles_out);
size_t matkv_table_workspace_bytes(const matkv_table *table, int32_t n_layers_launch);

/* a6 alone: merges n_parts partial attentions per row.  o_parts [n_rows][n_parts][D] fp32
 * (each normalised within its part), lse_parts [n_rows][n_parts] fp32 natural log (-inf =
 * empty part), out [n_rows][D] bf16, lse_out NULL or [n_rows] fp32; all device.              */
int matkv_lse_combine(matkv_ctx *ctx, int32_t n_rows, int32_t n_parts, int32_t D, const float *o_parts,
                      const float *lse_parts, void *out, float *lse_out, void *stream);

/* ---- materialisation side (the paper's store_KV, Section IV: a chunk is prefilled alone, starting at
 *      the first input position, and its K,V are moved GPU -> CPU bounce buffer -> storage) ------------- */
/* After a causal sub-prefill of a chunk's own tokens over an EMPTY chunk list (matkv_attend_prefill for
 * every layer, then matkv_table_advance), the request's tail holds exactly the chunk's K,V.  This call
 * lays the first n_tokens of the tail of request `req` out as a chunk blob [L][2][Hkv][n_tokens][D] in
 * dev_blob (device, 256-byte aligned, bit-exact copy) and, when host_blob is not NULL, copies the blob
 * on to host memory (pinned for a truly asynchronous copy) on the same stream.  The blob can then be
 * written to a file and registered like any other chunk.                                               */
int matkv_export_tail_as_chunk(matkv_ctx *ctx, matkv_table *table, int32_t req, int32_t n_tokens, void *dev_blob,
                               void *host_blob, void *stream);

/* ---- debugging aid: the concatenation the table stands for ------------------------------- */
/* Copies, for (layer, request), the K and V rows the table addresses into contiguous
 * k_out / v_out [Hkv][n_chunk_tokens + tail_len][D] bf16 device buffers (bit-exact gather).
 * rows_out (host, may be NULL) receives n_chunk_tokens + tail_len as known to the host.      */
int matkv_gather_debug(matkv_ctx *ctx, matkv_table *table, int32_t layer, int32_t req, void *k_out,
                       void *v_out, int64_t capacity_rows, int64_t *rows_out, void *stream);

/* ---- measurement aid: read-only streaming probe ------------------------------------------- */
/* Reads `bytes` of device memory once with plain 16-byte loads (nothing is written): the HBM read
 * ceiling a decode launch is compared with.  No counterpart in the paper.  Asynchronous on `stream`. */
int matkv_probe_read(matkv_ctx *ctx, const void *dev, size_t bytes, void *stream);

/* ---- failure-detection self-test ------------------------------------------------------------ */
/* Launches one thread that waits, with the kernels' bounded-wait logic, on a barrier nothing ever
 * signals.  After `seconds` (0 < seconds <= 2) of SM clock the wait gives up, the kernel returns
 * normally and the device status word reads MATKV_E_TIMEOUT (see matkv_status): the context stays
 * usable.  No counterpart in the paper; it shows how a lost copy or a lost peer would surface.       */
int matkv_selftest_wait_timeout(matkv_ctx *ctx, double seconds, void *stream);

#ifdef __cplusplus
}
#endif
#endif /* MATKV_H */
