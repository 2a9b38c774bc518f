// Host memory behind the copy engines.  Staged plans move the host-side bytes of a call between
// pinned host memory and rings of device staging buffers with cudaMemcpyAsync on internal
// streams and run the kernel device to device, segment by segment, chained by events; streamed
// weight plans put a file in front of that pipeline (reader threads -> pinned ring).
#include <cuda_runtime.h>
#include <fcntl.h>
#include <pthread.h>
#include <unistd.h>

#include <algorithm>
#include <atomic>
#include <cerrno>
#include <condition_variable>
#include <cstring>
#include <mutex>
#include <thread>
#include <vector>

#include "exec.h"

namespace tc {

// ---- staged host path: copy engines <-> device staging ring <-> kernel ----------------------
// One ring per direction (0: device -> host, 1: host -> device), so that an offload and a
// reload running concurrently on two streams do not wait on each other's buffers.
struct StageRing {
    char *buf[kStageBuffers] = {};
    cudaEvent_t ready[kStageBuffers] = {}, freed[kStageBuffers] = {};
    bool freed_recorded[kStageBuffers] = {};
    cudaStream_t copy = nullptr;
    cudaEvent_t entry = nullptr;  // orders the ring's copy stream behind the caller's stream
    uint64_t next = 0;
};
// Pinned host buffers that file chunks are read into (tc_weights_materialize_file).
constexpr int kHostBuffers = 3;
struct HostRing {
    char *buf[kHostBuffers] = {};
    cudaEvent_t freed[kHostBuffers] = {};  // the copy engine has finished reading the buffer
    bool used[kHostBuffers] = {};
    uint64_t next = 0;
};
struct StageArena {
    StageRing ring[2];
    HostRing host;
    int refs = 0;
};
static StageArena g_stage[kMaxDevices];
// Locks are per device and per ring, plus one per device for file streaming: staged calls on
// different GPUs of one process, or in the two directions of one GPU, do not queue behind one
// another on the host.  Whoever needs both rings (allocation, trimming) takes ring 0 first.
struct DeviceLocks {
    pthread_mutex_t ring[2] = {PTHREAD_MUTEX_INITIALIZER, PTHREAD_MUTEX_INITIALIZER}, file = PTHREAD_MUTEX_INITIALIZER;
    void lock_both() { pthread_mutex_lock(&ring[0]); pthread_mutex_lock(&ring[1]); }
    void unlock_both() { pthread_mutex_unlock(&ring[1]); pthread_mutex_unlock(&ring[0]); }
};
static DeviceLocks g_locks[kMaxDevices];

static void stage_free(StageArena &a)
{
    for (StageRing &r : a.ring) {
        for (int b = 0; b < kStageBuffers; b++) {
            if (r.buf[b]) cudaFree(r.buf[b]);
            if (r.ready[b]) cudaEventDestroy(r.ready[b]);
            if (r.freed[b]) cudaEventDestroy(r.freed[b]);
        }
        if (r.copy) cudaStreamDestroy(r.copy);
        if (r.entry) cudaEventDestroy(r.entry);
    }
    for (int b = 0; b < kHostBuffers; b++) {
        if (a.host.buf[b]) cudaFreeHost(a.host.buf[b]);
        if (a.host.freed[b]) cudaEventDestroy(a.host.freed[b]);
    }
    a = StageArena();
}

int stage_acquire(int device, int64_t *bytes)
{
    if (device < 0 || device >= kMaxDevices) return fail(TC_ERR_INVALID_ARG, "device ordinal %d is not supported", device);
    g_locks[device].lock_both();
    StageArena &a = g_stage[device];
    int rc = TC_OK;
    if (a.refs == 0) {
        a.refs = 1;  // the library's own reference: keeps the rings alive between plans
        cudaError_t e = cudaSuccess;
        for (StageRing &r : a.ring) {
            if (e == cudaSuccess) e = cudaEventCreateWithFlags(&r.entry, cudaEventDisableTiming);
            if (e == cudaSuccess) e = cudaStreamCreateWithFlags(&r.copy, cudaStreamNonBlocking);
            for (int b = 0; b < kStageBuffers && e == cudaSuccess; b++) {
                e = cudaMalloc(&r.buf[b], kStageBytes);
                if (e == cudaSuccess) e = cudaEventCreateWithFlags(&r.ready[b], cudaEventDisableTiming);
                if (e == cudaSuccess) e = cudaEventCreateWithFlags(&r.freed[b], cudaEventDisableTiming);
            }
        }
        if (e != cudaSuccess) {
            rc = e == cudaErrorMemoryAllocation ? fail(TC_ERR_OOM, "device allocation of the staging rings failed") : cuda_fail(e, "creating the staging rings");
            stage_free(a);  // also resets refs to 0
        }
    }
    if (rc == TC_OK) {
        a.refs++;
        *bytes = 2 * kStageBytes * kStageBuffers;
    }
    g_locks[device].unlock_both();
    return rc;
}

// The rings are kept once allocated (like the plan-storage cache): a caller that creates one
// staged plan per scheduler step must not pay six cudaMalloc / cudaFree pairs per step.
void stage_release(int device)
{
    if (device < 0 || device >= kMaxDevices) return;
    g_locks[device].lock_both();
    StageArena &a = g_stage[device];
    if (a.refs > 1) a.refs--;  // the last reference is never dropped: the rings stay until exit
    g_locks[device].unlock_both();
}

#define TC_TRY(call, what)                                   \
    do {                                                     \
        cudaError_t e_ = (call);                             \
        if (e_ != cudaSuccess) { rc = cuda_fail(e_, what); goto out; } \
    } while (0)

// to the host:   device -> staging (kernel, caller's stream) -> host (copy engine).
// to the device: host -> staging (copy engine) -> device (kernel, caller's stream).
// The host side is table entry 0 of the call (the packed buffer, or the paged host pool).
// Every segment's kernel sees the staging buffer through a base pointer shifted by the
// segment's packed offset (0 for paged pools), so the descriptors are used unchanged.
int execute_staged(const tc_plan *plan, const Group &g, const void *const *src, void *const *dst, uint32_t ptr_align, cudaStream_t s,
                   unsigned long long *sums)
{
    StageArena &a = g_stage[plan->device];
    const bool to_device = g.host_is_src;
    StageRing &r = a.ring[to_device ? 1 : 0];
    int rc = TC_OK;
    pthread_mutex_t *mu = &g_locks[plan->device].ring[to_device ? 1 : 0];
    pthread_mutex_lock(mu);
    TC_TRY(cudaEventRecord(r.entry, s), "cudaEventRecord");
    TC_TRY(cudaStreamWaitEvent(r.copy, r.entry, 0), "cudaStreamWaitEvent");
    for (const Segment &seg : g.segments) {
        const int b = static_cast<int>(r.next++ % kStageBuffers);
        char *shifted = r.buf[b] - seg.shift;
        const uint32_t pa = std::min<uint32_t>(ptr_align, __builtin_ctzll(reinterpret_cast<uintptr_t>(shifted) | 16));
        if (to_device) {
            const char *host = static_cast<const char *>(src[0]);
            if (r.freed_recorded[b]) TC_TRY(cudaStreamWaitEvent(r.copy, r.freed[b], 0), "cudaStreamWaitEvent");
            for (uint32_t c = seg.copy0; c < seg.copy0 + seg.ncopy; c++)
                TC_TRY(cudaMemcpyAsync(r.buf[b] + g.copies[c].stage_off, host + g.copies[c].host_off, static_cast<size_t>(g.copies[c].bytes), cudaMemcpyHostToDevice, r.copy), "cudaMemcpyAsync(host to staging)");
            TC_TRY(cudaEventRecord(r.ready[b], r.copy), "cudaEventRecord");
            TC_TRY(cudaStreamWaitEvent(s, r.ready[b], 0), "cudaStreamWaitEvent");
            const void *stage_src[1] = {shifted};
            if ((rc = launch_any(plan, g, stage_src, dst, pa, s, &seg, sums)) != TC_OK) goto out;
            TC_TRY(cudaEventRecord(r.freed[b], s), "cudaEventRecord");
        } else {
            char *host = static_cast<char *>(dst[0]);
            if (r.freed_recorded[b]) TC_TRY(cudaStreamWaitEvent(s, r.freed[b], 0), "cudaStreamWaitEvent");
            void *stage_dst[1] = {shifted};
            if ((rc = launch_any(plan, g, src, stage_dst, pa, s, &seg)) != TC_OK) goto out;
            TC_TRY(cudaEventRecord(r.ready[b], s), "cudaEventRecord");
            TC_TRY(cudaStreamWaitEvent(r.copy, r.ready[b], 0), "cudaStreamWaitEvent");
            for (uint32_t c = seg.copy0; c < seg.copy0 + seg.ncopy; c++)
                TC_TRY(cudaMemcpyAsync(host + g.copies[c].host_off, r.buf[b] + g.copies[c].stage_off, static_cast<size_t>(g.copies[c].bytes), cudaMemcpyDeviceToHost, r.copy), "cudaMemcpyAsync(staging to host)");
            TC_TRY(cudaEventRecord(r.freed[b], r.copy), "cudaEventRecord");
        }
        r.freed_recorded[b] = true;
    }
    if (!to_device)  // the caller's stream completes only when the last copies to the host have landed
        for (int b = 0; b < kStageBuffers; b++)
            if (r.freed_recorded[b]) TC_TRY(cudaStreamWaitEvent(s, r.freed[b], 0), "cudaStreamWaitEvent");
out:
    pthread_mutex_unlock(mu);
    return rc;
}

// ---- cold path: file -> pinned host ring -> staging ring -> kernel ---------------------------

// Reader threads of one tc_weights_materialize_file call.  Every chunk of the plan is a job of
// 1 MiB pieces; the caller opens jobs in order as pinned buffers become free, the readers take
// pieces of the oldest open job from a shared counter and move on to the next open job without
// waiting for one another, so the file is read continuously across chunk boundaries (buffered
// reads of a cached or striped file scale with the number of readers).
struct ReadJob {
    int64_t off = 0, len = 0, n_pieces = 0;
    char *dst = nullptr;
    std::atomic<int64_t> next{0}, done{0};
};
struct ReaderPool {
    static constexpr int64_t kPiece = 1ll << 20;
    int fd;
    std::vector<ReadJob> jobs;
    size_t opened = 0;  // jobs [0, opened) may be read (guarded by mu)
    bool quit = false;
    std::atomic<int> err{0};  // 0, an errno, or -1 at end of file
    std::mutex mu;
    std::condition_variable cv;
    std::vector<std::thread> threads;

    ReaderPool(int fd_, size_t n_jobs) : fd(fd_), jobs(n_jobs) {}

    void start()
    {
        const unsigned hw = std::thread::hardware_concurrency();
        const int n = static_cast<int>(std::min<unsigned>(8, hw > 2 ? hw - 2 : 1));
        try {
            for (int i = 0; i < n; i++) threads.emplace_back([this] { run(); });
        } catch (...) {
            // fewer readers than wished for; with none at all the caller reads (see wait)
        }
    }
    void open(size_t j, int64_t off, int64_t len, char *dst)
    {
        ReadJob &job = jobs[j];
        job.off = off;
        job.len = len;
        job.dst = dst;
        job.n_pieces = (len + kPiece - 1) / kPiece;
        std::lock_guard<std::mutex> lk(mu);
        opened = j + 1;
        cv.notify_all();
    }
    bool read_piece(ReadJob &job)
    {
        const int64_t k = job.next.fetch_add(1, std::memory_order_relaxed);
        if (k >= job.n_pieces) return false;
        int64_t lo = job.off + k * kPiece;
        const int64_t hi = std::min(job.off + job.len, lo + kPiece);
        while (lo < hi && !err.load(std::memory_order_relaxed)) {
            const ssize_t got = pread(fd, job.dst + (lo - job.off), static_cast<size_t>(hi - lo), static_cast<off_t>(lo));
            if (got < 0) {
                if (errno == EINTR) continue;
                err = errno ? errno : EIO;
            } else if (got == 0) {
                err = -1;
            } else {
                lo += got;
            }
        }
        if (job.done.fetch_add(1, std::memory_order_acq_rel) + 1 == job.n_pieces) {
            std::lock_guard<std::mutex> lk(mu);
            cv.notify_all();
        }
        return true;
    }
    void run()
    {
        size_t j = 0;
        while (j < jobs.size()) {
            {
                std::unique_lock<std::mutex> lk(mu);
                cv.wait(lk, [&] { return quit || opened > j; });
                if (quit) return;
            }
            while (read_piece(jobs[j])) {}
            j++;
        }
    }
    // Block until job j has been read completely (or a read failed).  Returns err.
    int wait(size_t j)
    {
        ReadJob &job = jobs[j];
        if (threads.empty())
            while (read_piece(job)) {}
        std::unique_lock<std::mutex> lk(mu);
        cv.wait(lk, [&] { return job.done.load(std::memory_order_acquire) >= job.n_pieces; });
        return err.load();
    }
    ~ReaderPool()
    {
        {
            std::lock_guard<std::mutex> lk(mu);
            quit = true;
            err = err.load() ? err.load() : ECANCELED;  // readers in the middle of a job stop at the next piece
            cv.notify_all();
        }
        for (std::thread &t : threads) t.join();
    }
};

static int host_ring_acquire(HostRing &h)
{
    if (h.buf[0]) return TC_OK;
    for (int b = 0; b < kHostBuffers; b++) {
        cudaError_t e = cudaHostAlloc(reinterpret_cast<void **>(&h.buf[b]), kStageBytes, cudaHostAllocDefault);
        if (e == cudaSuccess) e = cudaEventCreateWithFlags(&h.freed[b], cudaEventDisableTiming);
        if (e != cudaSuccess) {
            for (int k = 0; k <= b; k++) {
                if (h.buf[k]) cudaFreeHost(h.buf[k]);
                if (h.freed[k]) cudaEventDestroy(h.freed[k]);
            }
            h = HostRing();
            return e == cudaErrorMemoryAllocation ? fail(TC_ERR_OOM, "pinned allocation of the file staging buffers failed") : cuda_fail(e, "creating the file staging buffers");
        }
    }
    return TC_OK;
}

// The caller's thread is the conductor: it opens chunk i + 2 for the readers as soon as the copy
// engine has drained that chunk's pinned buffer, waits until chunk i has been read, and enqueues
// copy, kernel and events for it exactly as execute_staged does.  Reading (where the call
// spends its time) thus runs two chunks ahead of the transfers.  The ring lock is taken per
// chunk, not per call, so staged KV traffic of other threads keeps flowing while a checkpoint
// streams in.
int execute_streamed(const tc_plan *plan, const Group &g, int fd, int64_t file_off, void *const *dst, uint32_t ptr_align, cudaStream_t s,
                     unsigned long long *sums)
{
    StageArena &a = g_stage[plan->device];
    StageRing &r = a.ring[1];
    HostRing &h = a.host;
    const size_t n = g.segments.size();
    int rc = TC_OK;
    pthread_mutex_t *mu = &g_locks[plan->device].ring[1], *file_mu = &g_locks[plan->device].file;
    pthread_mutex_lock(file_mu);  // one file stream per device at a time (they share the pinned buffers)
    pthread_mutex_lock(mu);
    rc = host_ring_acquire(h);
    pthread_mutex_unlock(mu);
    if (rc != TC_OK) {
        pthread_mutex_unlock(file_mu);
        return rc;
    }
    {
        ReaderPool pool(fd, n);
        const uint64_t first = h.next;
        h.next += n;
        auto host_buf = [&](size_t i) { return static_cast<int>((first + i) % kHostBuffers); };
        auto open = [&](size_t i) -> int {
            const int hb = host_buf(i);
            if (h.used[hb]) {
                cudaError_t e = cudaEventSynchronize(h.freed[hb]);
                if (e != cudaSuccess) return cuda_fail(e, "cudaEventSynchronize");
            }
            const StageCopy &c = g.copies[g.segments[i].copy0];
            posix_fadvise(fd, static_cast<off_t>(file_off + c.host_off), static_cast<off_t>(c.bytes), POSIX_FADV_WILLNEED);
            pool.open(i, file_off + c.host_off, c.bytes, h.buf[hb]);
            return TC_OK;
        };
        pool.start();
        for (size_t i = 0; i < n && i < kHostBuffers - 1 && rc == TC_OK; i++) rc = open(i);
        for (size_t i = 0; i < n && rc == TC_OK; i++) {
            if (i + kHostBuffers - 1 < n && (rc = open(i + kHostBuffers - 1)) != TC_OK) break;
            const Segment &seg = g.segments[i];
            const StageCopy &c = g.copies[seg.copy0];
            const int err = pool.wait(i);
            if (err) {
                rc = err < 0 ? fail(TC_ERR_IO, "the file ends inside blob bytes [%lld, %lld)", (long long)c.host_off, (long long)(c.host_off + c.bytes))
                             : fail(TC_ERR_IO, "reading blob bytes [%lld, %lld): %s", (long long)c.host_off, (long long)(c.host_off + c.bytes), strerror(err));
                break;
            }
            const int hb = host_buf(i);
            pthread_mutex_lock(mu);
            {
                const int b = static_cast<int>(r.next++ % kStageBuffers);
                char *shifted = r.buf[b] - seg.shift;
                const uint32_t pa = std::min<uint32_t>(ptr_align, __builtin_ctzll(reinterpret_cast<uintptr_t>(shifted) | 16));
                const void *stage_src[1] = {shifted};
                if (r.freed_recorded[b]) TC_TRY(cudaStreamWaitEvent(r.copy, r.freed[b], 0), "cudaStreamWaitEvent");
                TC_TRY(cudaMemcpyAsync(r.buf[b] + c.stage_off, h.buf[hb], static_cast<size_t>(c.bytes), cudaMemcpyHostToDevice, r.copy), "cudaMemcpyAsync(host to staging)");
                TC_TRY(cudaEventRecord(h.freed[hb], r.copy), "cudaEventRecord");
                h.used[hb] = true;
                TC_TRY(cudaEventRecord(r.ready[b], r.copy), "cudaEventRecord");
                TC_TRY(cudaStreamWaitEvent(s, r.ready[b], 0), "cudaStreamWaitEvent");
                if ((rc = launch_any(plan, g, stage_src, dst, pa, s, &seg, sums)) != TC_OK) goto out;
                TC_TRY(cudaEventRecord(r.freed[b], s), "cudaEventRecord");
                r.freed_recorded[b] = true;
            }
        out:
            pthread_mutex_unlock(mu);
        }
    }  // the pool's destructor stops and joins the readers
    pthread_mutex_unlock(file_mu);
    return rc;
}
#undef TC_TRY

void stage_trim()
{
    for (int device = 0; device < kMaxDevices; device++) {
        g_locks[device].lock_both();
        StageArena &a = g_stage[device];
        if (a.refs == 1) {  // only the library's own reference is left
            for (StageRing &r : a.ring)
                if (r.copy) cudaStreamSynchronize(r.copy);
            stage_free(a);
        }
        g_locks[device].unlock_both();
    }
}

}  // namespace tc
