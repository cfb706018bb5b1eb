// Storage tier of the staging path: chunk blobs that live in files (the paper's materialised-KV store:
// one raw-bytes file per chunk id on flash) are read by a small pool of host threads into a pinned
// bounce ring lent by the caller, and copied from there to the device slots on the copy stream.
// Stream order does the sequencing: for every chunk the copy stream gets a host callback that waits
// for the chunk's read, the host-to-device copy out of the ring slab, and a callback that hands the
// slab back to the readers.  So storage reads, PCIe copies and the GPU's attention kernels overlap
// (three stages), and the staging call itself never blocks its caller.
// Failures stay on the host side of the link and are reported, never waited on for ever: a read that fails
// (or a file that turned out short) marks its staging call as failed; the callback's wait for a read has a
// limit, after which the call is marked failed too and the stream moves on; either way the status word
// reads MATKV_E_IO once the stream has passed the call, and table builds over such chunks are refused.
#include <errno.h>
#include <fcntl.h>
#include <string.h>
#include <unistd.h>

#include <chrono>
#include <condition_variable>
#include <deque>
#include <mutex>
#include <thread>

#include "matkv_internal.h"

namespace matkv {

constexpr int kFailWords = 256;   // staging calls whose failure words are live at once

struct IoJob {
    int fd;
    uint64_t offset;
    size_t bytes;
    int slab;
    uint64_t use;  // how many times the slab was used before this job
    std::shared_ptr<FailFlag> failed;  // the staging call's failure flag
};

struct IoEngine {
    char *base = nullptr;
    size_t slab_bytes = 0;
    int n_slabs = 0;
    uint64_t next_seq = 0;  // chunks handed to the engine so far (slab = seq % n_slabs)
    std::mutex m;
    std::condition_variable cv;
    std::deque<IoJob> queue;
    std::vector<uint64_t> reads_done, releases_done;  // per slab
    std::vector<std::thread> threads;
    bool stop = false;
    int errors = 0;
    char last_error[256] = "";
    int *h_flag = nullptr;   // kFailWords page-locked words the device can read, one per staging call in flight (ticket mod kFailWords)
    std::atomic<int64_t> timeout_ms{30000}, test_delay_ms{0};
};

// raises the device status word when the host has seen a read fail (launched behind a staging call's copies)
__global__ void k_io_flag(const volatile int *host_flag, int32_t *status) {
    if (*host_flag) atomicCAS(status, 0, MATKV_E_IO);
}

static void note_failure(IoEngine *e, const std::shared_ptr<FailFlag> &failed, const char *msg) {  // e->m held
    ++e->errors;
    snprintf(e->last_error, sizeof e->last_error, "%s", msg);
    if (failed) {
        failed->host.store(1, std::memory_order_release);
        if (failed->word) *failed->word = 1;
    }
}

static void io_worker(IoEngine *e) {
    for (;;) {
        IoJob job;
        {
            std::unique_lock<std::mutex> lk(e->m);
            e->cv.wait(lk, [&] { return e->stop || !e->queue.empty(); });
            if (e->queue.empty()) return;  // stop requested and nothing left
            job = e->queue.front();
            e->queue.pop_front();
            // the slab must have been handed back by the copy that used it last, and the read that filled it last must
            // have returned (a read the stream gave up waiting for may still be writing into the slab)
            auto slab_free = [&] { return e->releases_done[job.slab] == job.use && e->reads_done[job.slab] == job.use; };
            e->cv.wait(lk, [&] { return e->stop || slab_free(); });
            if (e->stop && !slab_free()) return;
        }
        if (const int64_t d = e->test_delay_ms.load()) std::this_thread::sleep_for(std::chrono::milliseconds(d));  // failure injection
        char *dst = e->base + (size_t)job.slab * e->slab_bytes;
        size_t done = 0;
        int err = 0;
        while (done < job.bytes) {
            const size_t want = std::min<size_t>(job.bytes - done, (size_t)16 << 20);
            const ssize_t got = pread(job.fd, dst + done, want, (off_t)(job.offset + done));
            if (got < 0) {
                if (errno == EINTR) continue;
                err = errno;
                break;
            }
            if (got == 0) {
                err = EIO;  // file shorter than the chunk
                break;
            }
            done += (size_t)got;
        }
        {
            std::lock_guard<std::mutex> lk(e->m);
            if (err) {
                char msg[256];
                snprintf(msg, sizeof msg, "read of %zu bytes at offset %llu failed: %s", job.bytes, (unsigned long long)job.offset,
                         strerror(err));
                note_failure(e, job.failed, msg);
            }
            e->reads_done[job.slab] = job.use + 1;
        }
        e->cv.notify_all();
    }
}

struct IoCallback {
    IoEngine *e;
    int slab;
    uint64_t use;
    std::shared_ptr<FailFlag> failed;
};

// Runs in stream order before the copy out of the slab.  The wait has a limit: a read that does not return
// (a hung network file system) must not stall every later operation of the copy stream for ever.  When the
// limit runs out the staging call is marked failed and the stream moves on (the copy then moves whatever the
// slab holds; the failure flag is what tells the caller not to use it).
static void CUDART_CB cb_wait_read(void *p) {
    IoCallback *c = (IoCallback *)p;
    {
        std::unique_lock<std::mutex> lk(c->e->m);
        const bool done = c->e->cv.wait_for(lk, std::chrono::milliseconds(std::max<int64_t>(1, c->e->timeout_ms.load())),
                                            [&] { return c->e->reads_done[c->slab] >= c->use + 1; });
        if (!done) note_failure(c->e, c->failed, "a storage read did not return within the time limit");
    }
    delete c;
}

static void CUDART_CB cb_release_slab(void *p) {  // runs in stream order after the copy out of the slab
    IoCallback *c = (IoCallback *)p;
    {
        std::lock_guard<std::mutex> lk(c->e->m);
        c->e->releases_done[c->slab] = c->use + 1;
    }
    c->e->cv.notify_all();
    delete c;
}

int io_engine_create(matkv_ctx *ctx, void *pinned, size_t bytes, size_t slab_bytes, int n_threads) {
    IoEngine *e = new IoEngine();
    e->base = (char *)pinned;
    e->slab_bytes = slab_bytes;
    e->n_slabs = (int)(bytes / slab_bytes);
    e->reads_done.assign(e->n_slabs, 0);
    e->releases_done.assign(e->n_slabs, 0);
    e->timeout_ms = ctx->opt_io_timeout_ms;
    e->test_delay_ms = ctx->opt_io_test_delay_ms;
    {
        DeviceGuard guard(ctx->device);
        cudaError_t err = cudaHostAlloc((void **)&e->h_flag, kFailWords * sizeof(int), cudaHostAllocMapped | cudaHostAllocPortable);
        if (err != cudaSuccess) {
            delete e;
            return cuda_fail(err, "cudaHostAlloc(read-failure flag)");
        }
        memset(e->h_flag, 0, kFailWords * sizeof(int));
    }
    for (int i = 0; i < n_threads; ++i) e->threads.emplace_back(io_worker, e);
    ctx->io = e;
    return MATKV_OK;
}

void io_engine_destroy(matkv_ctx *ctx) {
    IoEngine *e = ctx->io;
    if (!e) return;
    {
        std::lock_guard<std::mutex> lk(e->m);
        e->stop = true;
    }
    e->cv.notify_all();
    for (auto &t : e->threads) t.join();
    if (e->h_flag) cudaFreeHost(e->h_flag);
    delete e;
    ctx->io = nullptr;
}

void io_engine_configure(matkv_ctx *ctx) {
    if (!ctx->io) return;
    ctx->io->timeout_ms = ctx->opt_io_timeout_ms;
    ctx->io->test_delay_ms = ctx->opt_io_test_delay_ms;
}

void io_engine_bind_fail_word(matkv_ctx *ctx, uint64_t ticket, FailFlag *flag) {
    if (!ctx->io || !ctx->io->h_flag) return;
    flag->word = ctx->io->h_flag + ticket % kFailWords;
    *flag->word = 0;
}

int io_engine_flag_status(matkv_ctx *ctx, const std::shared_ptr<FailFlag> &failed, cudaStream_t copy_stream) {
    if (!ctx->io || !failed || !failed->word) return MATKV_OK;
    k_io_flag<<<1, 1, 0, copy_stream>>>(failed->word, ctx->d_status);
    MATKV_CUDA(cudaGetLastError());
    return MATKV_OK;
}

size_t io_engine_slab_bytes(const matkv_ctx *ctx) { return ctx->io ? ctx->io->slab_bytes : 0; }

int io_engine_errors(matkv_ctx *ctx, const char **msg) {
    if (!ctx->io) return 0;
    std::lock_guard<std::mutex> lk(ctx->io->m);
    if (msg) *msg = ctx->io->last_error;
    return ctx->io->errors;
}

// Hands a slab back on the host after an enqueue failed half-way: waits (with the read limit) for the slab's read to
// return, so that the next read into the slab cannot overlap it, then marks the slab released.
static void release_on_host(IoEngine *e, int slab, uint64_t use) {
    {
        std::unique_lock<std::mutex> lk(e->m);
        e->cv.wait_for(lk, std::chrono::milliseconds(std::max<int64_t>(1, e->timeout_ms.load())), [&] { return e->reads_done[slab] >= use + 1; });
        e->releases_done[slab] = use + 1;
    }
    e->cv.notify_all();
}

// Enqueues: read (worker threads) -> [copy stream] wait for the read, copy slab -> dst, release the slab.
int io_engine_stage(matkv_ctx *ctx, int fd, uint64_t offset, size_t bytes, void *dst, cudaStream_t copy_stream,
                    const std::shared_ptr<FailFlag> &failed, int32_t fp8_tokens, bool fp8_resident) {
    IoEngine *e = ctx->io;
    if (!e) return fail(MATKV_E_INVALID_ARG, "file-backed chunk: no bounce buffer set (matkv_set_bounce_buffer)");
    if (bytes > e->slab_bytes)
        return fail(MATKV_E_CAPACITY, "file-backed chunk of %zu bytes exceeds the bounce slab of %zu bytes", bytes, e->slab_bytes);
    IoJob job;
    {
        std::lock_guard<std::mutex> lk(e->m);
        const uint64_t seq = e->next_seq++;
        job.slab = (int)(seq % (uint64_t)e->n_slabs);
        job.use = seq / (uint64_t)e->n_slabs;
        job.fd = fd;
        job.offset = offset;
        job.bytes = bytes;
        job.failed = failed;
        e->queue.push_back(job);
    }
    e->cv.notify_all();
    // from here on the slab is owed a release: by the stream's second callback, or on the host when enqueueing fails
    IoCallback *cb = new IoCallback{e, job.slab, job.use, failed};
    cudaError_t err = cudaLaunchHostFunc(copy_stream, cb_wait_read, cb);
    if (err != cudaSuccess) {
        delete cb;
        release_on_host(e, job.slab, job.use);
        return cuda_fail(err, "cudaLaunchHostFunc(wait for the read)");
    }
    int rc = MATKV_OK;
    if (fp8_tokens > 0) {  // compressed chunk: the expanding copy reads the slab over the link (it must be device-accessible pinned memory)
        rc = fp8_resident ? launch_stage_relayout_fp8(ctx, e->base + (size_t)job.slab * e->slab_bytes, dst, fp8_tokens, copy_stream)
                          : launch_stage_expand_fp8(ctx, e->base + (size_t)job.slab * e->slab_bytes, dst, fp8_tokens,
                                                    ctx->opt_stage_ctas > 0 ? (int)ctx->opt_stage_ctas : 16, copy_stream);
    } else {
        err = cudaMemcpyAsync(dst, e->base + (size_t)job.slab * e->slab_bytes, bytes, cudaMemcpyHostToDevice, copy_stream);
        if (err != cudaSuccess) rc = cuda_fail(err, "copy out of the bounce slab");
    }
    cb = new IoCallback{e, job.slab, job.use, failed};
    err = cudaLaunchHostFunc(copy_stream, cb_release_slab, cb);
    if (err != cudaSuccess) {
        delete cb;
        release_on_host(e, job.slab, job.use);
        if (rc == MATKV_OK) rc = cuda_fail(err, "cudaLaunchHostFunc(release of the slab)");
    }
    return rc;
}

int open_chunk_file(const char *path, uint64_t offset, size_t bytes, int *fd_out) {
    int fd = -1;
    if (offset % 4096 == 0 && bytes % 4096 == 0) fd = open(path, O_RDONLY | O_DIRECT);  // bypass the page cache when possible
    if (fd < 0) fd = open(path, O_RDONLY);
    if (fd < 0) return fail(MATKV_E_IO, "cannot open chunk file %s: %s", path, strerror(errno));
    const off_t end = lseek(fd, 0, SEEK_END);
    if (end < 0 || (uint64_t)end < offset + bytes) {
        close(fd);
        return fail(MATKV_E_IO, "chunk file %s holds %lld bytes, the chunk needs %llu at offset %llu", path, (long long)end,
                    (unsigned long long)bytes, (unsigned long long)offset);
    }
    *fd_out = fd;
    return MATKV_OK;
}

void close_chunk_file(int fd) {
    if (fd >= 0) close(fd);
}

}  // namespace matkv
