// Plan lifecycle (device storage, upload), the checks every execute call makes, and the
// extern "C" entry points.  The kernels live in copy_kernel.cuh / launch.cu, the host-memory
// paths in staging.cu.
//
// Host memory: pointers to mapped pinned memory work in every call (the kernel loads / stores
// over the host link).  Staged plans instead move the host-side bytes with the copy engines
// through device staging rings and run the kernel device to device (see staging.cu).
#include <cuda_runtime.h>
#include <pthread.h>

#include <algorithm>
#include <cstdio>
#include <cstring>
#include <new>
#include <vector>

#include "exec.h"

namespace tc {

int cuda_fail(cudaError_t e, const char *what)
{
    return fail(TC_ERR_CUDA, "%s: %s", what, cudaGetErrorString(e));
}

// Device storage of plans comes from a small per-device cache of power-of-two blocks, so that
// a caller that creates and destroys one plan per scheduler step pays cudaMalloc / cudaFree
// (both of which may synchronise the device) only until the cache has warmed up.
namespace {
struct CachedBlock {
    void *ptr;
    size_t bytes;
    int device;
};
std::vector<CachedBlock> g_block_cache;
size_t g_block_cache_bytes = 0;
constexpr size_t kBlockCacheLimit = 256u << 20;
pthread_mutex_t g_block_mu = PTHREAD_MUTEX_INITIALIZER;

size_t block_size_for(size_t nb)
{
    size_t s = 64u << 10;
    while (s < nb) s <<= 1;
    return s;
}

cudaError_t block_alloc(int device, size_t nb, void **out, size_t *got)
{
    const size_t want = block_size_for(nb);
    pthread_mutex_lock(&g_block_mu);
    for (size_t i = 0; i < g_block_cache.size(); i++)
        if (g_block_cache[i].device == device && g_block_cache[i].bytes == want) {
            *out = g_block_cache[i].ptr;
            *got = want;
            g_block_cache_bytes -= want;
            g_block_cache.erase(g_block_cache.begin() + i);
            pthread_mutex_unlock(&g_block_mu);
            return cudaSuccess;
        }
    pthread_mutex_unlock(&g_block_mu);
    *got = want;
    return cudaMalloc(out, want);
}

// Plans are uploaded on a stream of the library's own, one per device, and the upload is waited
// for: a copy from pageable host memory may return once the bytes sit in the driver's staging
// buffer, before they have reached the device, and a kernel the caller then launches on a
// non-blocking stream would not wait for it (it would read whatever plan used the block before).
cudaStream_t g_upload_stream[kMaxDevices] = {};

cudaError_t upload_stream_for(int device, cudaStream_t *out)
{
    if (device < 0 || device >= kMaxDevices) {  // no private stream: the legacy stream, waited for as well
        *out = cudaStreamLegacy;
        return cudaSuccess;
    }
    cudaError_t e = cudaSuccess;
    pthread_mutex_lock(&g_block_mu);
    if (!g_upload_stream[device]) e = cudaStreamCreateWithFlags(&g_upload_stream[device], cudaStreamNonBlocking);
    *out = g_upload_stream[device];
    pthread_mutex_unlock(&g_block_mu);
    return e;
}

void block_free(int device, void *ptr, size_t bytes)
{
    if (!ptr) return;
    pthread_mutex_lock(&g_block_mu);
    if (g_block_cache_bytes + bytes <= kBlockCacheLimit) {
        g_block_cache.push_back(CachedBlock{ptr, bytes, device});
        g_block_cache_bytes += bytes;
        ptr = nullptr;
    }
    pthread_mutex_unlock(&g_block_mu);
    if (ptr) cudaFree(ptr);
}
}  // namespace

static void free_plan_storage(tc_plan *plan)
{
    for (auto &pair : plan->trace_ev)
        for (void *&ev : pair) {
            if (ev) cudaEventDestroy(static_cast<cudaEvent_t>(ev));
            ev = nullptr;
        }
    block_free(plan->device, plan->d_storage, plan->d_storage_bytes);
    plan->d_storage = nullptr;
    for (int k = 0; k < 2; k++) plan->group[k].d_descs = nullptr, plan->group[k].d_tile_desc = nullptr, plan->group[k].d_extents = nullptr;
}

// One allocation and one copy per plan: [g0 descriptors | g0 tiles | g1 descriptors | g1 tiles],
// every part 256-byte aligned.
static int upload_plan(tc_plan *plan)
{
    auto pad = [](size_t n) { return (n + 255) & ~size_t(255); };
    size_t off[4], ext_off[2], total = 0;
    for (int k = 0; k < 2; k++) {
        off[2 * k] = total;
        total += pad(plan->group[k].descs.size() * sizeof(Desc));
        off[2 * k + 1] = total;
        total += pad(plan->group[k].tile_desc.size() * sizeof(uint32_t));
        ext_off[k] = total;
        total += pad(plan->group[k].extents.size() * sizeof(int64_t));
    }
    if (total == 0) return TC_OK;
    std::vector<unsigned char> image(total);
    for (int k = 0; k < 2; k++) {
        const Group &g = plan->group[k];
        if (!g.descs.empty()) memcpy(image.data() + off[2 * k], g.descs.data(), g.descs.size() * sizeof(Desc));
        if (!g.tile_desc.empty()) memcpy(image.data() + off[2 * k + 1], g.tile_desc.data(), g.tile_desc.size() * sizeof(uint32_t));
        if (!g.extents.empty()) memcpy(image.data() + ext_off[k], g.extents.data(), g.extents.size() * sizeof(int64_t));
    }
    cudaError_t e = block_alloc(plan->device, total, &plan->d_storage, &plan->d_storage_bytes);
    if (e != cudaSuccess) {
        plan->d_storage = nullptr;
        return e == cudaErrorMemoryAllocation ? fail(TC_ERR_OOM, "device allocation of %zu plan bytes failed", total) : cuda_fail(e, "cudaMalloc");
    }
    cudaStream_t up;
    if ((e = upload_stream_for(plan->device, &up)) != cudaSuccess) return cuda_fail(e, "cudaStreamCreate(plan upload)");
    if ((e = cudaMemcpyAsync(plan->d_storage, image.data(), total, cudaMemcpyHostToDevice, up)) != cudaSuccess) return cuda_fail(e, "cudaMemcpyAsync(plan)");
    if ((e = cudaStreamSynchronize(up)) != cudaSuccess) return cuda_fail(e, "cudaStreamSynchronize(plan upload)");
    plan->device_bytes += static_cast<int64_t>(plan->d_storage_bytes);
    char *base = static_cast<char *>(plan->d_storage);
    for (int k = 0; k < 2; k++) {
        Group &g = plan->group[k];
        if (!g.descs.empty()) g.d_descs = reinterpret_cast<Desc *>(base + off[2 * k]);
        if (!g.tile_desc.empty()) g.d_tile_desc = reinterpret_cast<uint32_t *>(base + off[2 * k + 1]);
        if (!g.extents.empty()) g.d_extents = reinterpret_cast<int64_t *>(base + ext_off[k]);
    }
    return TC_OK;
}

// A table entry must be memory the device can address: device memory, managed memory, or host
// memory that is pinned and mapped.  Plain pageable host memory would make the kernel fault, so
// it is refused here, on the host.  Every entry is checked (a fraction of a microsecond each):
// one unchecked pageable pointer would be a GPU fault.
static int check_addressable(const void *const *table, size_t n, const char *what, bool *host_memory)
{
    for (size_t i = 0; i < n; i++) {
        cudaPointerAttributes attr;
        cudaError_t e = cudaPointerGetAttributes(&attr, table[i]);
        if (e != cudaSuccess) {
            cudaGetLastError();
            return fail(TC_ERR_INVALID_ARG, "%s table entry %zu (%p) is not a valid address for this device", what, i, table[i]);
        }
        if (attr.type == cudaMemoryTypeUnregistered)
            return fail(TC_ERR_INVALID_ARG, "%s table entry %zu (%p) is pageable host memory: pin it (cudaHostAlloc / cudaHostRegister) or use device memory", what, i, table[i]);
        if (attr.type == cudaMemoryTypeHost) *host_memory = true;
    }
    return TC_OK;
}

int execute(const tc_plan *plan, int gi, const void *const *src, size_t n_src, void *const *dst, size_t n_dst, void *stream,
            unsigned long long *sums, const FileSource *file)
{
    clear_error();
    if (!plan) return fail(TC_ERR_INVALID_ARG, "plan is NULL");
    if (plan->flags & TC_PLAN_HOST_ONLY) return fail(TC_ERR_INVALID_ARG, "a TC_PLAN_HOST_ONLY plan cannot be executed");
    const Group &g = plan->group[gi];
    if (n_src != g.n_src || n_dst != g.n_dst)
        return fail(TC_ERR_INVALID_ARG, "tables of %zu source and %zu destination pointers given, the plan needs %zu and %zu", n_src, n_dst, g.n_src, g.n_dst);
    if ((n_src && !src && !file) || (n_dst && !dst)) return fail(TC_ERR_INVALID_ARG, "pointer table is NULL");
    if (file && g.n_tiles && g.segments.empty()) return fail(TC_ERR_KIND, "the plan was not cut into chunks: create it with TC_PLAN_STREAM");
    if (plan->deadline_ns && now_ns() > plan->deadline_ns) return fail(TC_ERR_DEADLINE, "deadline passed before the call; nothing launched");
    int current = -1;
    if (cudaGetDevice(&current) != cudaSuccess || current != plan->device)
        return fail(TC_ERR_INVALID_ARG, "the plan lives on device %d but device %d is current", plan->device, current);
    if (sums) {
        cudaError_t e = cudaMemsetAsync(sums, 0, static_cast<size_t>(plan->n_sums) * sizeof(unsigned long long), static_cast<cudaStream_t>(stream));
        if (e != cudaSuccess) return cuda_fail(e, "zeroing the checksum accumulators");
    }
    if (g.n_tiles == 0) return TC_OK;
    uint32_t ptr_align = 4;
    for (size_t i = 0; i < n_src && !file; i++) {
        if (!src[i]) return fail(TC_ERR_INVALID_ARG, "source table entry %zu is NULL", i);
        ptr_align = std::min<uint32_t>(ptr_align, __builtin_ctzll(reinterpret_cast<uintptr_t>(src[i]) | 16));
    }
    for (size_t i = 0; i < n_dst; i++) {
        if (!dst[i]) return fail(TC_ERR_INVALID_ARG, "destination table entry %zu is NULL", i);
        ptr_align = std::min<uint32_t>(ptr_align, __builtin_ctzll(reinterpret_cast<uintptr_t>(dst[i]) | 16));
    }
    int rc;
    bool host_src = false, host_dst = false;  // some table entry is pinned host memory: the kernel works over the host link
    if (!file && (rc = check_addressable(src, n_src, "source", &host_src)) != TC_OK) return rc;
    if ((rc = check_addressable(const_cast<const void *const *>(dst), n_dst, "destination", &host_dst)) != TC_OK) return rc;
    const int host_memory = (host_src ? kHostSrc : 0) | (host_dst ? kHostDst : 0);
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    const bool trace = plan->trace_ev[gi][0] != nullptr;
    if (trace) {
        cudaError_t e = cudaEventRecord(static_cast<cudaEvent_t>(plan->trace_ev[gi][0]), s);
        if (e != cudaSuccess) return cuda_fail(e, "cudaEventRecord(trace)");
    }
    if (g.d_extents && (rc = launch_bounds_check(g, 0, s)) != TC_OK) return rc;  // TC_PLAN_DEBUG_BOUNDS
    if (file) rc = execute_streamed(plan, g, file->fd, file->offset, dst, ptr_align, s, sums);
    else if (!g.segments.empty()) rc = execute_staged(plan, g, src, dst, ptr_align, s, sums);
    else rc = launch_any(plan, g, src, dst, ptr_align, s, nullptr, sums, host_memory);
    if (trace && rc == TC_OK) {
        cudaError_t e = cudaEventRecord(static_cast<cudaEvent_t>(plan->trace_ev[gi][1]), s);
        if (e != cudaSuccess) return cuda_fail(e, "cudaEventRecord(trace)");
        plan->traced_once[gi] = true;
    }
    return rc;
}

}  // namespace tc

using namespace tc;

extern "C" int tc_plan_create(const tc_plan_spec_t *spec, tc_plan_t **out)
{
    clear_error();
    if (out) *out = nullptr;
    if (!spec || !out) return fail(TC_ERR_INVALID_ARG, "spec and out are required");
    if (spec->struct_size != sizeof(tc_plan_spec_t))
        return fail(TC_ERR_INVALID_ARG, "spec.struct_size %u != %zu: header and library disagree", spec->struct_size, sizeof(tc_plan_spec_t));
    if (spec->deadline_ns && now_ns() > spec->deadline_ns) return fail(TC_ERR_DEADLINE, "deadline passed before the call");
    tc_plan *plan = new (std::nothrow) tc_plan();
    if (!plan) return fail(TC_ERR_OOM, "host allocation failed");
    plan->kind = spec->kind;
    plan->flags = spec->flags;
    plan->trace_id = spec->trace_id;
    plan->deadline_ns = spec->deadline_ns;
    plan->tuning = spec->tuning;
    int rc;
    try {
        rc = build_plan(spec, plan);
    } catch (const std::bad_alloc &) {
        rc = fail(TC_ERR_OOM, "host allocation failed while lowering the plan");
    }
    if (rc == TC_OK && !(spec->flags & TC_PLAN_HOST_ONLY)) {
        cudaError_t e = cudaGetDevice(&plan->device);
        if (e == cudaSuccess) e = cudaDeviceGetAttribute(&plan->sm_count, cudaDevAttrMultiProcessorCount, plan->device);
        if (e != cudaSuccess) rc = cuda_fail(e, "querying the current device");
        if (rc == TC_OK && (!plan->group[0].segments.empty() || !plan->group[1].segments.empty())) {
            int64_t arena = 0;
            if ((rc = stage_acquire(plan->device, &arena)) == TC_OK) {
                plan->staged = true;
                plan->device_bytes += arena;
            }
        }
        if (rc == TC_OK) rc = upload_plan(plan);
        if (rc == TC_OK && (spec->flags & TC_PLAN_TRACE))
            for (auto &pair : plan->trace_ev)
                for (void *&ev : pair) {
                    cudaEvent_t made = nullptr;
                    cudaError_t e2 = cudaEventCreate(&made);
                    if (e2 != cudaSuccess && rc == TC_OK) rc = cuda_fail(e2, "cudaEventCreate(trace)");
                    ev = made;
                }
        for (int k = 0; k < 2 && rc == TC_OK; k++)
            if (plan->group[k].n_tiles) resident_ctas_for(plan->group[k].n_src + plan->group[k].n_dst, plan->group[k].resident_ctas);
    }
    if (rc != TC_OK) {
        free_plan_storage(plan);
        if (plan->staged) stage_release(plan->device);
        delete plan;
        return rc;
    }
    *out = plan;
    return TC_OK;
}

extern "C" int tc_plan_destroy(tc_plan_t *plan)
{
    if (!plan) return TC_OK;
    free_plan_storage(plan);
    if (plan->staged) stage_release(plan->device);
    delete plan;
    return TC_OK;
}

extern "C" int tc_kv_pack(const tc_plan_t *plan, const void *const *src_bases, size_t n_src, void *const *dst_bases, size_t n_dst, void *stream)
{
    if (plan && plan->kind != TC_KV_PACK && plan->kind != TC_KV_MIGRATE && plan->kind != TC_KV_MIXED) {
        clear_error();
        return fail(TC_ERR_KIND, "tc_kv_pack needs a PACK, MIGRATE or MIXED plan (kind %d given)", plan->kind);
    }
    return execute(plan, 0, src_bases, n_src, dst_bases, n_dst, stream);
}

extern "C" int tc_kv_unpack(const tc_plan_t *plan, const void *const *src_bases, size_t n_src, void *const *dst_bases, size_t n_dst, void *stream)
{
    if (plan && plan->kind != TC_KV_UNPACK && plan->kind != TC_KV_MIXED) {
        clear_error();
        return fail(TC_ERR_KIND, "tc_kv_unpack needs an UNPACK or MIXED plan (kind %d given)", plan->kind);
    }
    return execute(plan, 1, src_bases, n_src, dst_bases, n_dst, stream);
}

extern "C" int tc_weights_materialize(const tc_plan_t *plan, const void *blob, void *const *dst_ptrs, size_t n_dst, void *stream)
{
    if (plan && plan->kind != TC_WEIGHTS) {
        clear_error();
        return fail(TC_ERR_KIND, "tc_weights_materialize needs a WEIGHTS plan (kind %d given)", plan->kind);
    }
    const void *src[1] = {blob};
    return execute(plan, 0, src, 1, dst_ptrs, n_dst, stream);
}

extern "C" int tc_weights_materialize_checksum(const tc_plan_t *plan, const void *blob, void *const *dst_ptrs, size_t n_dst, uint64_t *checksums, void *stream)
{
    clear_error();
    if (plan && (plan->kind != TC_WEIGHTS || !plan->checksummed))
        return fail(TC_ERR_KIND, "tc_weights_materialize_checksum needs a WEIGHTS plan created with TC_PLAN_CHECKSUM");
    if (!checksums) return fail(TC_ERR_INVALID_ARG, "checksums is NULL");
    const void *src[1] = {blob};
    return execute(plan, 0, src, 1, dst_ptrs, n_dst, stream, reinterpret_cast<unsigned long long *>(checksums));
}

extern "C" int tc_weights_materialize_file(const tc_plan_t *plan, int fd, int64_t file_offset, void *const *dst_ptrs, size_t n_dst, uint64_t *checksums,
                                           void *stream)
{
    clear_error();
    if (plan && (plan->kind != TC_WEIGHTS || !(plan->flags & TC_PLAN_STREAM)))
        return fail(TC_ERR_KIND, "tc_weights_materialize_file needs a WEIGHTS plan created with TC_PLAN_STREAM");
    if (plan && checksums && !plan->checksummed) return fail(TC_ERR_KIND, "checksums need a plan created with TC_PLAN_CHECKSUM");
    if (fd < 0 || file_offset < 0) return fail(TC_ERR_INVALID_ARG, "fd %d / file_offset %lld: both must be >= 0", fd, (long long)file_offset);
    const FileSource file{fd, file_offset};
    return execute(plan, 0, nullptr, 1, dst_ptrs, n_dst, stream, reinterpret_cast<unsigned long long *>(checksums), &file);
}

extern "C" int tc_trim(void)
{
    clear_error();
    pthread_mutex_lock(&g_block_mu);
    for (const CachedBlock &b : g_block_cache) cudaFree(b.ptr);
    g_block_cache.clear();
    g_block_cache_bytes = 0;
    pthread_mutex_unlock(&g_block_mu);
    stage_trim();
    return TC_OK;
}

extern "C" int tc_device_status(uint32_t *flags)
{
    clear_error();
    if (!flags) return fail(TC_ERR_INVALID_ARG, "flags is NULL");
    unsigned int v = 0;
    const int rc = read_device_status(&v);
    *flags = v;
    return rc;
}

extern "C" int tc_plan_check_device(const tc_plan_t *plan, int64_t shrink, void *stream)
{
    clear_error();
    if (!plan) return fail(TC_ERR_INVALID_ARG, "plan is NULL");
    if (!(plan->flags & TC_PLAN_DEBUG_BOUNDS) || (plan->flags & TC_PLAN_HOST_ONLY))
        return fail(TC_ERR_KIND, "tc_plan_check_device needs an executable plan created with TC_PLAN_DEBUG_BOUNDS");
    if (shrink < 0) return fail(TC_ERR_INVALID_ARG, "shrink %lld < 0", (long long)shrink);
    int current = -1;
    if (cudaGetDevice(&current) != cudaSuccess || current != plan->device)
        return fail(TC_ERR_INVALID_ARG, "the plan lives on device %d but device %d is current", plan->device, current);
    for (int k = 0; k < 2; k++) {
        const Group &g = plan->group[k];
        if (g.descs.empty()) continue;
        const int rc = launch_bounds_check(g, shrink, static_cast<cudaStream_t>(stream));
        if (rc != TC_OK) return rc;
    }
    return TC_OK;
}

extern "C" int tc_selftest_wait_timeout(void *stream)
{
    clear_error();
    return launch_wait_timeout_probe(static_cast<cudaStream_t>(stream));
}

extern "C" int tc_plan_stats(const tc_plan_t *plan, tc_plan_stats_t *out)
{
    clear_error();
    if (!plan || !out) return fail(TC_ERR_INVALID_ARG, "plan and out are required");
    memset(out, 0, sizeof *out);
    out->trace_id = plan->trace_id;
    out->kind = plan->kind;
    out->executable = !(plan->flags & TC_PLAN_HOST_ONLY);
    for (int k = 0; k < 2; k++) {
        const Group &g = plan->group[k];
        out->n_descriptors[k] = static_cast<int64_t>(g.descs.size());
        out->n_tiles[k] = static_cast<int64_t>(g.n_tiles);
        out->payload_bytes[k] = g.payload;
        out->vec_bytes[k] = 1 << g.log2_align;
        out->path[k] = g.n_tiles ? (g.segments.empty() ? 1 : 3) : 0;
        if (!g.segments.empty()) out->launches_per_execute = static_cast<int32_t>(g.segments.size());
        out->grid[k] = g.n_tiles ? static_cast<int32_t>(grid_for(plan, g, mode_for(plan, g, 4))) : 0;
        if (plan->trace_ev[k][0]) {
            float ms = 0.f;
            out->last_device_us[k] = -1.0;
            if (plan->traced_once[k] && cudaEventElapsedTime(&ms, static_cast<cudaEvent_t>(plan->trace_ev[k][0]), static_cast<cudaEvent_t>(plan->trace_ev[k][1])) == cudaSuccess)
                out->last_device_us[k] = 1e3 * ms;
            else
                cudaGetLastError();  // cudaErrorNotReady is the expected answer while the run is in flight
        }
    }
    out->packed_bytes_required = plan->packed_required;
    out->device_bytes = plan->device_bytes;
    if (out->launches_per_execute == 0) out->launches_per_execute = 1;
    return TC_OK;
}

extern "C" int tc_plan_descriptors(const tc_plan_t *plan, int group, tc_descriptor_t *out, size_t cap, size_t *n_out)
{
    clear_error();
    if (!plan || group < 0 || group > 1) return fail(TC_ERR_INVALID_ARG, "plan is required and group must be 0 or 1");
    const Group &g = plan->group[group];
    if (n_out) *n_out = g.descs.size();
    if (!out) return TC_OK;
    for (size_t i = 0; i < g.descs.size() && i < cap; i++) {
        const Desc &d = g.descs[i];
        tc_descriptor_t &o = out[i];
        o.src_off = d.src_off; o.dst_off = d.dst_off; o.src_outer = d.src_outer; o.dst_outer = d.dst_outer;
        o.src_s0 = d.src_s0; o.src_s1 = d.src_s1; o.dst_s0 = d.dst_s0; o.dst_s1 = d.dst_s1;
        o.src_slot = d.src_slot; o.dst_slot = d.dst_slot - static_cast<uint32_t>(g.n_src);
        o.src_slot_step = d.src_slot_step; o.dst_slot_step = d.dst_slot_step;
        o.run_bytes = d.run; o.n0 = d.n0; o.rows = d.rows; o.n_outer = d.n_outer;
        o.rows_per_tile = d.rows_per_tile; o.tiles_per_outer = d.tiles_per_outer; o.tile0 = d.tile0; o.planes_per_tile = g.ppt;
    }
    return TC_OK;
}

extern "C" int tc_plan_segments(const tc_plan_t *plan, int group, tc_segment_t *out, size_t cap, size_t *n_out)
{
    clear_error();
    if (!plan || group < 0 || group > 1) return fail(TC_ERR_INVALID_ARG, "plan is required and group must be 0 or 1");
    const Group &g = plan->group[group];
    if (n_out) *n_out = g.segments.size();
    if (!out) return TC_OK;
    for (size_t i = 0; i < g.segments.size() && i < cap; i++) {
        const Segment &seg = g.segments[i];
        tc_segment_t &o = out[i];
        o.host_off = seg.ncopy ? g.copies[seg.copy0].host_off : 0;
        o.bytes = 0;
        for (uint32_t c = seg.copy0; c < seg.copy0 + seg.ncopy; c++) o.bytes += g.copies[c].bytes;
        o.tile0 = seg.nd ? 0 : seg.d0;
        o.n_tiles = seg.nd ? 0 : seg.no;
        o.desc0 = seg.nd ? seg.d0 : 0;
        o.n_descs = seg.nd;
        o.outer0 = seg.nd ? seg.o0 : 0;
        o.n_outer = seg.nd ? seg.no : 0;
    }
    return TC_OK;
}
