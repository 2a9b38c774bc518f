// tc_kv_pack_noalloc: tc_kv_pack for callers that must not allocate device memory.
#include <cuda_runtime.h>
#include <pthread.h>

#include <new>

#include "exec.h"

using namespace tc;

// ------------------------------------------------------------------------------ no-allocation variant
// Scratch for tc_kv_pack_noalloc: descriptors (and the tile list of non-uniform groups) of one
// call.  It lives in the library image, so no call ever allocates device memory for it.  In
// host code the array's name is only a stand-in for the symbol; the device address is looked
// up once per device with cudaGetSymbolAddress and that address is what the kernel is given.
static __device__ __align__(256) unsigned char g_noalloc_scratch[TC_NOALLOC_SCRATCH_BYTES];

namespace {
struct NoallocDevice {
    void *scratch = nullptr;  // device address of g_noalloc_scratch on this device
    int sm_count = 0;
};
NoallocDevice g_noalloc_dev[kMaxDevices];
pthread_mutex_t g_noalloc_mu = PTHREAD_MUTEX_INITIALIZER;

// Once per device, with that device current: resolve the scratch symbol's device address.
int noalloc_setup(int device, NoallocDevice *out)
{
    pthread_mutex_lock(&g_noalloc_mu);
    NoallocDevice &d = g_noalloc_dev[device];
    int rc = TC_OK;
    if (!d.scratch) {
        void *ptr = nullptr;
        cudaError_t e = cudaGetSymbolAddress(&ptr, g_noalloc_scratch);
        if (e == cudaSuccess) e = cudaDeviceGetAttribute(&d.sm_count, cudaDevAttrMultiProcessorCount, device);
        if (e != cudaSuccess) rc = cuda_fail(e, "resolving the scratch area of tc_kv_pack_noalloc");
        else d.scratch = ptr;
    }
    *out = d;
    pthread_mutex_unlock(&g_noalloc_mu);
    return rc;
}
}  // namespace

extern "C" int tc_kv_pack_noalloc(const tc_plan_spec_t *spec, const void *const *src_bases, size_t n_src,
                                  void *const *dst_bases, size_t n_dst, void *stream)
{
    clear_error();
    if (!spec) return fail(TC_ERR_INVALID_ARG, "spec is required");
    if (spec->struct_size != sizeof(tc_plan_spec_t))
        return fail(TC_ERR_INVALID_ARG, "spec.struct_size %u != %zu: header and library disagree", spec->struct_size, sizeof(tc_plan_spec_t));
    if (spec->kind != TC_KV_PACK && spec->kind != TC_KV_MIGRATE && spec->kind != TC_KV_MIXED)
        return fail(TC_ERR_KIND, "tc_kv_pack_noalloc needs a PACK, MIGRATE or MIXED spec (kind %d given)", spec->kind);
    if (spec->deadline_ns && now_ns() > spec->deadline_ns) return fail(TC_ERR_DEADLINE, "deadline passed before the call");
    if (spec->flags & TC_PLAN_STAGED) return fail(TC_ERR_INVALID_ARG, "tc_kv_pack_noalloc does not stage: the staging ring is allocated device memory");
    if (spec->flags & TC_PLAN_HOST_ONLY) return fail(TC_ERR_INVALID_ARG, "TC_PLAN_HOST_ONLY asks for a plan that is not executed; tc_kv_pack_noalloc always executes");
    if (spec->flags & TC_PLAN_DEBUG_BOUNDS) return fail(TC_ERR_INVALID_ARG, "TC_PLAN_DEBUG_BOUNDS keeps slot extents in allocated device memory; tc_kv_pack_noalloc allocates none");
    tc_plan plan;  // lives on the host for the duration of this call only
    plan.kind = spec->kind;
    plan.flags = spec->flags;
    plan.trace_id = spec->trace_id;
    plan.deadline_ns = spec->deadline_ns;
    plan.tuning = spec->tuning;
    int rc;
    try {
        rc = build_plan(spec, &plan);
    } catch (const std::bad_alloc &) {
        rc = fail(TC_ERR_OOM, "host allocation failed while lowering the plan");
    }
    if (rc != TC_OK) return rc;
    Group &g = plan.group[0];
    // The device is resolved before anything else: execute() checks it, also for a request that
    // moves nothing (R = 0, or every T_r = 0), which is a legal no-op returning TC_OK.
    cudaError_t e = cudaGetDevice(&plan.device);
    if (e != cudaSuccess) return cuda_fail(e, "querying the current device");
    if (plan.device < 0 || plan.device >= kMaxDevices) return fail(TC_ERR_INVALID_ARG, "device ordinal %d is not supported", plan.device);
    if (g.n_tiles == 0) return execute(&plan, 0, src_bases, n_src, dst_bases, n_dst, stream);
    const size_t desc_bytes = g.descs.size() * sizeof(Desc);
    const size_t tile_bytes = g.tile_desc.size() * sizeof(uint32_t);
    if (desc_bytes + tile_bytes > TC_NOALLOC_SCRATCH_BYTES)
        return fail(TC_ERR_TOO_LARGE, "the call needs %zu bytes of descriptors and tiles; tc_kv_pack_noalloc holds at most %u: split the request or use tc_plan_create",
                    desc_bytes + tile_bytes, TC_NOALLOC_SCRATCH_BYTES);
    NoallocDevice dev;
    if ((rc = noalloc_setup(plan.device, &dev)) != TC_OK) return rc;
    plan.sm_count = dev.sm_count;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    unsigned char *base = static_cast<unsigned char *>(dev.scratch);
    if ((e = cudaMemcpyAsync(base, g.descs.data(), desc_bytes, cudaMemcpyHostToDevice, s)) != cudaSuccess) return cuda_fail(e, "copying descriptors into the scratch area");
    g.d_descs = reinterpret_cast<Desc *>(base);
    if (tile_bytes) {
        if ((e = cudaMemcpyAsync(base + desc_bytes, g.tile_desc.data(), tile_bytes, cudaMemcpyHostToDevice, s)) != cudaSuccess) return cuda_fail(e, "copying tiles into the scratch area");
        g.d_tile_desc = reinterpret_cast<uint32_t *>(base + desc_bytes);
    }
    resident_ctas_for(g.n_src + g.n_dst, g.resident_ctas);
    rc = execute(&plan, 0, src_bases, n_src, dst_bases, n_dst, stream);
    g.d_descs = nullptr;  // the scratch area is not the plan's to free
    g.d_tile_desc = nullptr;
    return rc;
}
