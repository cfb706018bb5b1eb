// Storage tier of the staging path: chunk blobs that live in files (the paper's materialised-KV store:
// one raw-bytes file per chunk id on flash) are read by a small pool of host threads into a pinned
// bounce ring lent by the caller, and copied from there to the device slots on the copy stream.
// Stream order does the sequencing: for every chunk the copy stream gets a host callback that waits
// for the chunk's read, the host-to-device copy out of the ring slab, and a callback that hands the
// slab back to the readers.  So storage reads, PCIe copies and the GPU's attention kernels overlap
// (three stages), and the staging call itself never blocks its caller.
#include <errno.h>
#include <fcntl.h>
#include <string.h>
#include <unistd.h>

#include <condition_variable>
#include <deque>
#include <mutex>
#include <thread>

#include "matkv_internal.h"

namespace matkv {

struct IoJob {
    int fd;
    uint64_t offset;
    size_t bytes;
    int slab;
    uint64_t use;  // how many times the slab was used before this job
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
};

static void io_worker(IoEngine *e) {
    for (;;) {
        IoJob job;
        {
            std::unique_lock<std::mutex> lk(e->m);
            e->cv.wait(lk, [&] { return e->stop || !e->queue.empty(); });
            if (e->queue.empty()) return;  // stop requested and nothing left
            job = e->queue.front();
            e->queue.pop_front();
            // the slab must have been handed back by the copy that used it last
            e->cv.wait(lk, [&] { return e->stop || e->releases_done[job.slab] == job.use; });
            if (e->stop && e->releases_done[job.slab] != job.use) return;
        }
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
                ++e->errors;
                snprintf(e->last_error, sizeof e->last_error, "read of %zu bytes at offset %llu failed: %s", job.bytes,
                         (unsigned long long)job.offset, strerror(err));
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
};

static void CUDART_CB cb_wait_read(void *p) {  // runs in stream order before the copy out of the slab
    IoCallback *c = (IoCallback *)p;
    {
        std::unique_lock<std::mutex> lk(c->e->m);
        c->e->cv.wait(lk, [&] { return c->e->reads_done[c->slab] >= c->use + 1; });
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
    delete e;
    ctx->io = nullptr;
}

size_t io_engine_slab_bytes(const matkv_ctx *ctx) { return ctx->io ? ctx->io->slab_bytes : 0; }

int io_engine_errors(matkv_ctx *ctx, const char **msg) {
    if (!ctx->io) return 0;
    std::lock_guard<std::mutex> lk(ctx->io->m);
    if (msg) *msg = ctx->io->last_error;
    return ctx->io->errors;
}

// Enqueues: read (worker threads) -> [copy stream] wait for the read, copy slab -> dst, release the slab.
int io_engine_stage(matkv_ctx *ctx, int fd, uint64_t offset, size_t bytes, void *dst, cudaStream_t copy_stream, int32_t fp8_tokens, bool fp8_resident) {
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
        e->queue.push_back(job);
    }
    e->cv.notify_all();
    MATKV_CUDA(cudaLaunchHostFunc(copy_stream, cb_wait_read, new IoCallback{e, job.slab, job.use}));
    if (fp8_tokens > 0) {  // compressed chunk: the expanding copy reads the slab over the link (it must be device-accessible pinned memory)
        int rc = fp8_resident ? launch_stage_relayout_fp8(ctx, e->base + (size_t)job.slab * e->slab_bytes, dst, fp8_tokens, copy_stream)
                              : launch_stage_expand_fp8(ctx, e->base + (size_t)job.slab * e->slab_bytes, dst, fp8_tokens,
                                                        ctx->opt_stage_ctas > 0 ? (int)ctx->opt_stage_ctas : 16, copy_stream);
        if (rc) return rc;
    } else {
        MATKV_CUDA(cudaMemcpyAsync(dst, e->base + (size_t)job.slab * e->slab_bytes, bytes, cudaMemcpyHostToDevice, copy_stream));
    }
    MATKV_CUDA(cudaLaunchHostFunc(copy_stream, cb_release_slab, new IoCallback{e, job.slab, job.use}));
    return MATKV_OK;
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
