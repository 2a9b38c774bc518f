// Host side of the executor: which build of the kernel a group needs, how large its grid is,
// and the launch itself.
#include <cuda_runtime.h>
#include <pthread.h>

#include <algorithm>

#include "copy_kernel.cuh"
#include "exec.h"

namespace tc {

// Which executor build a group needs, given the alignment shared by the call's base pointers.
int mode_for(const tc_plan *plan, const Group &g, uint32_t ptr_align, bool checksums)
{
    if (g.log2_align < 4 || ptr_align < 4) return kModeAny;
    if (plan->tuning.copy_path == 1 && g.ppt == 1 && !checksums) return kModeAny;  // staged through shared memory on request
    return g.single_run_tiles ? kModeRun : kModeRows;
}

template <int NPTR, int MODE>
static int resident_ctas()
{
    int n = 0;
    const size_t smem = MODE == kModeAny ? kRealignSmem : 0;
    if (smem) cudaFuncSetAttribute(tc_copy_kernel<NPTR, MODE>, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(smem));
    if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&n, tc_copy_kernel<NPTR, MODE>, Shape<MODE>::threads, smem) != cudaSuccess || n < 1) n = 1;
    return n;
}

template <int NPTR>
static void resident_ctas_all(int out[3])
{
    out[kModeRun] = resident_ctas<NPTR, kModeRun>();
    out[kModeRows] = resident_ctas<NPTR, kModeRows>();
    out[kModeAny] = resident_ctas<NPTR, kModeAny>();
}

static pthread_mutex_t g_occupancy_mu = PTHREAD_MUTEX_INITIALIZER;

void resident_ctas_for(size_t n_ptrs, int out[3])
{
    // queried once per table size class (the answer depends on the kernel, not on the plan)
    static int cache[3][3];
    static bool have[3];
    const int cls = n_ptrs <= 8 ? 0 : n_ptrs <= 400 ? 1 : 2;
    pthread_mutex_lock(&g_occupancy_mu);
    if (!have[cls]) {
        if (cls == 0) resident_ctas_all<8>(cache[cls]);
        else if (cls == 1) resident_ctas_all<400>(cache[cls]);
        else resident_ctas_all<TC_MAX_TABLE_SLOTS>(cache[cls]);
        have[cls] = true;
    }
    for (int m = 0; m < 3; m++) out[m] = cache[cls][m];
    pthread_mutex_unlock(&g_occupancy_mu);
}

// Tile rows per descriptor: planes, or groups of ppt planes.
static uint32_t outer_groups(const Group &g) { return (g.descs[0].n_outer + g.ppt - 1) / g.ppt; }

uint32_t grid_for(const tc_plan *plan, const Group &g, int mode, const Segment *win, int over_host_link)
{
    // Default: one CTA per tile.  The hardware block scheduler then balances the tiles over the
    // SMs and de-phases the CTAs' load and store bursts, which measured faster than a
    // persistent grid-stride grid.  tuning.ctas_per_sm / max_ctas select a persistent grid
    // (few CTAs suit transfers over the host link).
    uint64_t grid = std::min<uint64_t>(g.n_tiles, 0x7fffffffull);
    if (win) grid = win->nd ? static_cast<uint64_t>((win->no + g.ppt - 1) / g.ppt) * win->nd * (g.tiles_per_desc / outer_groups(g)) : win->no;
    if (plan->tuning.ctas_per_sm > 0) {
        int per_sm = g.resident_ctas[mode] > 0 ? g.resident_ctas[mode] : 1;
        per_sm = std::min(per_sm, plan->tuning.ctas_per_sm);
        grid = std::min<uint64_t>(grid, static_cast<uint64_t>(plan->sm_count > 0 ? plan->sm_count : 148) * per_sm);
    }
    if (plan->tuning.max_ctas > 0) grid = std::min<uint64_t>(grid, plan->tuning.max_ctas);
    // Over the host link (a table entry is pinned host memory) a persistent grid of one CTA per SM
    // is the default: with both directions of the link busy, 64 to 148 CTAs moved 72 GB/s where one
    // CTA per tile (tens of thousands of short-lived CTAs) moved 42 to 53 and 16 CTAs 60; one
    // direction alone does not care (51-52 GB/s either way).
    else if (over_host_link && plan->tuning.ctas_per_sm <= 0)
        grid = std::min<uint64_t>(grid, plan->sm_count > 0 ? plan->sm_count : 148);
    return static_cast<uint32_t>(grid);
}

template <int NPTR>
static int launch(const tc_plan *plan, const Group &g, const void *const *src, void *const *dst, uint32_t ptr_align, cudaStream_t stream,
                  const Segment *win, unsigned long long *sums, int over_host_link)
{
    // Uniform groups with planes (KV) are walked plane-major by default: all blocks of plane 0,
    // then plane 1, ...  Together with descriptors sorted by destination offset, every plane
    // pass writes ascending addresses (and pack / unpack stream through the packed buffer),
    // which measured 3-5 % faster than walking the planes of one block after another.
    Segment whole{0, static_cast<uint32_t>(g.descs.size()), 0, g.descs.empty() ? 0 : g.descs[0].n_outer, 0, 0, 0};
    // A paged host pool (pinned memory in which the planes of a block lie back to back: one page
    // per block) is walked block after block instead, so that a page is read or written in one
    // go; HBM locality is beside the point at the host link's speed (prefix-reload burst: 262-266
    // against 268-271 ms per step).  A contiguous packed host buffer keeps the plane-major walk,
    // which streams through it (offload by kernel stores: 80-81 against 78 GB/s).
    bool paged_host = false;
    if (over_host_link && !g.descs.empty()) {
        // the first, the middle and the last descriptor have one and the same plane stride and it is
        // the size of their largest plane (a block with a ragged tail has fewer rows than its page
        // has room for; the requests of a packed buffer differ in their plane strides)
        bool src_paged = (over_host_link & kHostSrc) != 0, dst_paged = (over_host_link & kHostDst) != 0;
        int64_t plane = 0;
        for (size_t i : {size_t(0), g.descs.size() / 2, g.descs.size() - 1}) plane = std::max<int64_t>(plane, static_cast<int64_t>(g.descs[i].rows) * g.descs[i].run);
        for (size_t i : {size_t(0), g.descs.size() / 2, g.descs.size() - 1}) {
            src_paged = src_paged && g.descs[i].src_outer == plane;
            dst_paged = dst_paged && g.descs[i].dst_outer == plane;
        }
        paged_host = src_paged || dst_paged;
    }
    const bool plane_major = plan->tuning.tile_order == 2 || (plan->tuning.tile_order == 0 && !paged_host);
    if (!win && g.tiles_per_desc && !g.descs.empty() && g.descs[0].n_outer > 1 && plane_major) win = &whole;
    const int mode = mode_for(plan, g, ptr_align, sums != nullptr);
    if (sums && mode == kModeAny) return fail(TC_ERR_INVALID_ARG, "checksums need 16-byte aligned base pointers");
    const uint32_t grid = grid_for(plan, g, mode, win, over_host_link);
    Params<NPTR> prm;
    prm.descs = g.d_descs;
    prm.tile_desc = g.d_tile_desc;
    prm.n_tiles = static_cast<uint32_t>(g.n_tiles);
    prm.n_descs = static_cast<uint32_t>(g.descs.size());
    prm.win_span = prm.win_d0 = prm.win_o0 = prm.win_tpo = prm.win_o_end = prm.tile_base = 0;
    prm.ppt = g.ppt;
    prm.log2_unit = g.log2_unit;
    if (win && win->nd == 0) {  // a range of global tile ids
        prm.tile_base = win->d0;
        prm.n_tiles = win->d0 + win->no;
    } else if (win) {
        prm.win_tpo = g.tiles_per_desc / outer_groups(g);
        prm.win_span = win->nd * prm.win_tpo;
        prm.win_d0 = win->d0;
        prm.win_o0 = win->o0;
        prm.win_o_end = win->o0 + win->no;
        prm.n_tiles = (win->no + g.ppt - 1) / g.ppt * prm.win_span;
    }
    prm.tiles_per_desc = g.tiles_per_desc;
    prm.div_tpd = g.div_tpd;
    prm.tpo = g.tiles_per_desc ? g.tiles_per_desc / outer_groups(g) : 1;
    prm.div_tpo = make_fastdiv(prm.tpo);
    prm.log2_ptr_align = ptr_align;
    prm.stage_bytes = 0;
    prm.stage_always = plan->tuning.copy_path == 1;
    prm.debug_bounds = g.d_extents != nullptr;
    prm.sums = sums;
    for (size_t i = 0; i < g.n_src; i++) prm.ptr[i] = const_cast<char *>(static_cast<const char *>(src[i]));
    for (size_t i = 0; i < g.n_dst; i++) prm.ptr[g.n_src + i] = static_cast<char *>(dst[i]);
    for (size_t i = g.n_src + g.n_dst; i < NPTR; i++) prm.ptr[i] = nullptr;
    // the realigning path stages rows in more dynamic shared memory than a kernel gets by
    // default; the opt-in is per device and costs nothing to repeat
    auto with_stage = [&](auto kernel) {
        prm.stage_bytes = std::max<uint32_t>(g.realign_smem, 1024);
        return cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(kRealignSmem));
    };
    if (g.ppt > 1) {
        // multi-plane tiles: KV groups only (two pools of at most L*2 pointers each)
        if (NPTR == TC_MAX_TABLE_SLOTS || sums) return fail(TC_ERR_INVALID_ARG, "internal: multi-plane tiles with a large table or checksums");
        if constexpr (NPTR != TC_MAX_TABLE_SLOTS) {
            bool step = false;  // some pool has one pointer per plane
            for (const Desc &d : g.descs) step = step || d.src_slot_step || d.dst_slot_step;
            if (step) {
                switch (mode) {
                case kModeRun: tc_copy_kernel<NPTR, kModeRun, false, 2><<<grid, Shape<kModeRun>::threads, 0, stream>>>(prm); break;
                case kModeRows: tc_copy_kernel<NPTR, kModeRows, false, 2><<<grid, Shape<kModeRows>::threads, 0, stream>>>(prm); break;
                default:
                    if (cudaError_t ea = with_stage(tc_copy_kernel<NPTR, kModeAny, false, 2>); ea != cudaSuccess) return cuda_fail(ea, "cudaFuncSetAttribute(dynamic shared memory)");
                    tc_copy_kernel<NPTR, kModeAny, false, 2><<<grid, Shape<kModeAny>::threads, prm.stage_bytes, stream>>>(prm);
                    break;
                }
            } else {
                switch (mode) {
                case kModeRun: tc_copy_kernel<NPTR, kModeRun, false, 1><<<grid, Shape<kModeRun>::threads, 0, stream>>>(prm); break;
                case kModeRows: tc_copy_kernel<NPTR, kModeRows, false, 1><<<grid, Shape<kModeRows>::threads, 0, stream>>>(prm); break;
                default:
                    if (cudaError_t ea = with_stage(tc_copy_kernel<NPTR, kModeAny, false, 1>); ea != cudaSuccess) return cuda_fail(ea, "cudaFuncSetAttribute(dynamic shared memory)");
                    tc_copy_kernel<NPTR, kModeAny, false, 1><<<grid, Shape<kModeAny>::threads, prm.stage_bytes, stream>>>(prm);
                    break;
                }
            }
        }
    } else if (sums) {
        if (mode == kModeRun) tc_copy_kernel<NPTR, kModeRun, true><<<grid, Shape<kModeRun>::threads, 0, stream>>>(prm);
        else tc_copy_kernel<NPTR, kModeRows, true><<<grid, Shape<kModeRows>::threads, 0, stream>>>(prm);
    } else
    switch (mode) {
    case kModeRun: tc_copy_kernel<NPTR, kModeRun><<<grid, Shape<kModeRun>::threads, 0, stream>>>(prm); break;
    case kModeRows: tc_copy_kernel<NPTR, kModeRows><<<grid, Shape<kModeRows>::threads, 0, stream>>>(prm); break;
    default:
        if (cudaError_t ea = with_stage(tc_copy_kernel<NPTR, kModeAny>); ea != cudaSuccess) return cuda_fail(ea, "cudaFuncSetAttribute(dynamic shared memory)");
        tc_copy_kernel<NPTR, kModeAny><<<grid, Shape<kModeAny>::threads, prm.stage_bytes, stream>>>(prm);
        break;
    }
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) return cuda_fail(e, "kernel launch");
    return TC_OK;
}

int read_device_status(unsigned int *out)
{
    unsigned int zero = 0;
    // a diagnostic: every stream's earlier work first, non-blocking streams included (a copy on
    // the legacy stream alone would not wait for those)
    cudaError_t e = cudaDeviceSynchronize();
    if (e == cudaSuccess) e = cudaMemcpyFromSymbol(out, g_device_status, sizeof *out);
    if (e == cudaSuccess && *out) e = cudaMemcpyToSymbol(g_device_status, &zero, sizeof zero);
    return e == cudaSuccess ? TC_OK : cuda_fail(e, "reading the device status word");
}

int launch_bounds_check(const Group &g, int64_t shrink, cudaStream_t s)
{
    const uint32_t n = static_cast<uint32_t>(g.descs.size());
    if (n == 0 || !g.d_extents) return TC_OK;
    tc_bounds_check_kernel<<<(n + 255) / 256, 256, 0, s>>>(g.d_descs, n, reinterpret_cast<const long long *>(g.d_extents), shrink);
    cudaError_t e = cudaGetLastError();
    return e == cudaSuccess ? TC_OK : cuda_fail(e, "kernel launch");
}

int launch_wait_timeout_probe(cudaStream_t s)
{
    tc_wait_timeout_probe<<<1, 32, 0, s>>>(256);
    cudaError_t e = cudaGetLastError();
    return e == cudaSuccess ? TC_OK : cuda_fail(e, "kernel launch");
}

int launch_any(const tc_plan *plan, const Group &g, const void *const *src, void *const *dst, uint32_t ptr_align, cudaStream_t s, const Segment *win,
               unsigned long long *sums, int over_host_link)
{
    const size_t n = g.n_src + g.n_dst;
    if (n <= 8) return launch<8>(plan, g, src, dst, ptr_align, s, win, sums, over_host_link);
    if (n <= 400) return launch<400>(plan, g, src, dst, ptr_align, s, win, sums, over_host_link);
    return launch<TC_MAX_TABLE_SLOTS>(plan, g, src, dst, ptr_align, s, win, sums, over_host_link);
}

}  // namespace tc
