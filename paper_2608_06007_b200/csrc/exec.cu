// Plan lifecycle and the copy-executor kernels (sm_100a).
//
// One launch executes one group of a plan (a staged plan: one launch per segment).  By default
// the grid has one CTA per tile - a tile is one plane of one descriptor and a row range of it,
// about tile_bytes (32 KiB) of payload - and the hardware block scheduler spreads the tiles over
// the SMs; KV groups walk their tiles plane-major over descriptors sorted by destination offset,
// so every plane pass writes ascending addresses.  tuning.ctas_per_sm / max_ctas turn the same
// kernel into a persistent grid-stride loop.  Inside a tile every thread moves 16-byte vectors
// (narrower when the geometry or a base pointer is less aligned): a batch of independent
// streaming loads first, then the stores, so that many requests per thread are in flight.
// Consecutive lanes touch consecutive vectors of a run, so every warp access is one or more
// whole, aligned lines on both the read and the write side.  Base pointers travel in the
// kernel parameters; nothing is allocated or copied per execute call.
//
// Host memory: pointers to mapped pinned memory work in every call (the kernel loads / stores
// over the host link).  Staged plans instead move the host-side bytes with the copy engines
// through device staging rings and run the kernel device to device (see execute_staged).
#include <cuda_runtime.h>
#include <fcntl.h>
#include <pthread.h>
#include <unistd.h>

#include <algorithm>
#include <atomic>
#include <cerrno>
#include <condition_variable>
#include <mutex>
#include <cstdio>
#include <cstring>
#include <new>
#include <thread>
#include <vector>

#include "plan.h"

namespace tc {

// Three builds of the executor, chosen per group on the host, so that the common cases do not
// pay registers for the rare ones:
//   kModeRun   every tile is one 16-byte-aligned contiguous run (same-layout KV blocks, whole
//              tensors, dim-0 slabs): no row decoding
//   kModeRows  every access is 16-byte aligned, tiles hold strided rows (layout transforms,
//              dim-1 slices)
//   kModeAny   some descriptor or base pointer is less aligned: width picked per tile
enum { kModeRun = 0, kModeRows = 1, kModeAny = 2 };

// CTA shape per build: threads x vectors in flight per thread (one pass covers a 32 KiB tile)
// and the residency the register budget is held to.
template <int MODE> struct Shape;
template <> struct Shape<kModeRun> { static constexpr int threads = 256, unroll = 8, min_ctas = 3; };
template <> struct Shape<kModeRows> { static constexpr int threads = 256, unroll = 8, min_ctas = 3; };
template <> struct Shape<kModeAny> { static constexpr int threads = 256, unroll = 4, min_ctas = 2; };

template <int NPTR>
struct Params {
    const Desc *descs;
    const uint32_t *tile_desc;  // null for uniform groups
    uint32_t n_tiles;
    uint32_t tiles_per_desc;    // > 0 for uniform groups
    FastDiv div_tpd;
    uint32_t tpo;               // uniform groups: tiles per plane of one descriptor
    FastDiv div_tpo;
    uint32_t log2_ptr_align;    // alignment shared by every base pointer (capped at 4)
    // launch window (win_span == 0: the whole group).  Tile ids then walk plane-major over
    // descriptors [win_d0, ...) x planes [win_o0, ...): win_span = descriptors x win_tpo.
    uint32_t win_span, win_d0, win_o0, win_tpo;
    uint32_t tile_base;         // first global tile id of this launch (tile-range segments)
    unsigned long long *sums;   // checksum accumulators (checked builds only)
    char *ptr[NPTR];            // src table then dst table
};

// Integrity checksum: position-weighted sum of the source's 4-byte words,
//   sum of x_u * key(u) mod 2^64,  key(u) = ((u * 0x9E3779B1) << 1 | 1) mod 2^32,
// u = word index relative to the tensor's first byte.  key(u + 1) = key(u) + 2 * 0x9E3779B1.
__device__ __forceinline__ unsigned long long csum_vec(uint4 v, unsigned long long byte_pos)
{
    constexpr uint32_t kStep = 0x9E3779B1u << 1;
    uint32_t k = ((static_cast<uint32_t>(byte_pos >> 2) * 0x9E3779B1u) << 1) | 1u;
    unsigned long long t = static_cast<unsigned long long>(v.x) * k;
    k += kStep;
    t += static_cast<unsigned long long>(v.y) * k;
    k += kStep;
    t += static_cast<unsigned long long>(v.z) * k;
    k += kStep;
    t += static_cast<unsigned long long>(v.w) * k;
    return t;
}
template <typename V> __device__ __forceinline__ unsigned long long csum_of(V, unsigned long long) { return 0; }
template <> __device__ __forceinline__ unsigned long long csum_of<uint4>(uint4 v, unsigned long long p) { return csum_vec(v, p); }

__device__ __forceinline__ uint32_t fastdiv(uint32_t n, FastDiv f) { return (__umulhi(n, f.mul) + n) >> f.shift; }

template <typename V> __device__ __forceinline__ V ld_stream(const char *p);
template <typename V> __device__ __forceinline__ void st_stream(char *p, V v);

template <> __device__ __forceinline__ uint4 ld_stream<uint4>(const char *p) { return __ldcs(reinterpret_cast<const uint4 *>(p)); }
template <> __device__ __forceinline__ void st_stream<uint4>(char *p, uint4 v) { __stcs(reinterpret_cast<uint4 *>(p), v); }
#define TC_NARROW(V)                                                                                  \
    template <> __device__ __forceinline__ V ld_stream<V>(const char *p) { return *reinterpret_cast<const V *>(p); } \
    template <> __device__ __forceinline__ void st_stream<V>(char *p, V v) { *reinterpret_cast<V *>(p) = v; }
TC_NARROW(uint2)
TC_NARROW(uint32_t)
TC_NARROW(uint16_t)
TC_NARROW(uint8_t)
#undef TC_NARROW

template <int LOGV> struct VecOf;
template <> struct VecOf<4> { using type = uint4; };
template <> struct VecOf<3> { using type = uint2; };
template <> struct VecOf<2> { using type = uint32_t; };
template <> struct VecOf<1> { using type = uint16_t; };
template <> struct VecOf<0> { using type = uint8_t; };

// Add the CTA's partial checksums to the accumulator: warp shuffles, then one atomic per CTA
// (many CTAs feed the same tensor's accumulator; same-address atomics are the scarce resource).
template <int kThreads>
__device__ __forceinline__ void csum_flush(unsigned long long *sum, unsigned long long acc)
{
    __shared__ unsigned long long warp_sums[kThreads / 32];
#pragma unroll
    for (int k = 16; k > 0; k >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, k);
    if ((threadIdx.x & 31) == 0) warp_sums[threadIdx.x >> 5] = acc;
    __syncthreads();
    if (threadIdx.x < 32) {
        acc = threadIdx.x < kThreads / 32 ? warp_sums[threadIdx.x] : 0;
#pragma unroll
        for (int k = 16; k > 0; k >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, k);
        if (threadIdx.x == 0) atomicAdd(sum, acc);
    }
    __syncthreads();
}

// Copy rows [row0, row0 + nrows) of one outer index of descriptor d; src / dst point at row 0.
// A thread's vectors are kThreads vectors apart, so a warp always covers 32 consecutive
// vectors of the tile's row space: whole aligned segments on both sides.
// CHECK: also add the checksum terms of the bytes read to acc; pos0 is the tensor-relative
// byte position of src.
template <int LOGV, int U, int kThreads, bool CHECK = false>
__device__ __forceinline__ void copy_rows(const Desc &d, const char *src, char *dst, uint32_t row0, uint32_t nrows,
                                          unsigned long long pos0 = 0, unsigned long long *acc = nullptr)
{
    using V = typename VecOf<LOGV>::type;
    const uint32_t nbytes = nrows * d.run;  // <= 1 MiB
    const uint32_t run = d.run, n0 = d.n0;
    const FastDiv div_run = d.div_run, div_n0 = d.div_n0;
    const uint32_t ss0 = d.src_s0, ss1 = d.src_s1, ds0 = d.dst_s0, ds1 = d.dst_s1;
#pragma unroll 1
    for (uint32_t base = threadIdx.x << LOGV; base < nbytes; base += (kThreads * U) << LOGV) {
        V val[U];
        uint32_t doff[U], soff[CHECK ? U : 1];
#pragma unroll
        for (int u = 0; u < U; u++) {
            const uint32_t byte = base + ((u * kThreads) << LOGV);
            if (byte < nbytes) {
                uint32_t r = fastdiv(byte, div_run);
                const uint32_t col = byte - r * run;
                r += row0;
                const uint32_t i1 = fastdiv(r, div_n0);
                const uint32_t i0 = r - i1 * n0;
                doff[u] = i1 * ds1 + i0 * ds0 + col;
                const uint32_t so = i1 * ss1 + i0 * ss0 + col;
                if (CHECK) soff[u] = so;
                val[u] = ld_stream<V>(src + so);
            }
        }
#pragma unroll
        for (int u = 0; u < U; u++) {
            const uint32_t byte = base + ((u * kThreads) << LOGV);
            if (byte < nbytes) {
                st_stream<V>(dst + doff[u], val[u]);
                if (CHECK) *acc += csum_of<V>(val[u], pos0 + soff[u]);
            }
        }
    }
}

// One contiguous run of 16-byte vectors: no row decoding at all.
template <int U, int kThreads, bool CHECK = false>
__device__ __forceinline__ void copy_run16(const char *src, char *dst, uint32_t nbytes, unsigned long long pos0 = 0, unsigned long long *acc = nullptr)
{
#pragma unroll 1
    for (uint32_t base = threadIdx.x << 4; base < nbytes; base += (kThreads * U) << 4) {
        uint4 val[U];
#pragma unroll
        for (int u = 0; u < U; u++)
            if (base + ((u * kThreads) << 4) < nbytes) val[u] = ld_stream<uint4>(src + base + ((u * kThreads) << 4));
#pragma unroll
        for (int u = 0; u < U; u++)
            if (base + ((u * kThreads) << 4) < nbytes) {
                st_stream<uint4>(dst + base + ((u * kThreads) << 4), val[u]);
                if (CHECK) *acc += csum_vec(val[u], pos0 + base + ((u * kThreads) << 4));
            }
    }
}

template <int NPTR, int MODE, bool CHECK = false>
__global__ void __launch_bounds__(Shape<MODE>::threads, Shape<MODE>::min_ctas) tc_copy_kernel(const __grid_constant__ Params<NPTR> prm)
{
    constexpr int kThreads = Shape<MODE>::threads, kUnroll = Shape<MODE>::unroll;
    __shared__ Desc sdesc[2];
    int buf = 0;
    for (uint32_t tile = blockIdx.x + prm.tile_base; tile < prm.n_tiles; tile += gridDim.x, buf ^= 1) {
        // tile id -> descriptor, plane o, part.  For uniform and windowed launches this needs
        // launch constants only, so it overlaps the descriptor fetch instead of waiting for it.
        uint32_t di, o = 0, part = 0;
        if (prm.win_span) {
            const uint32_t ow = tile / prm.win_span, rem = tile - ow * prm.win_span;
            const uint32_t dw = rem / prm.win_tpo;
            di = prm.win_d0 + dw;
            o = prm.win_o0 + ow;
            part = rem - dw * prm.win_tpo;
        } else if (prm.tiles_per_desc) {
            di = fastdiv(tile, prm.div_tpd);
            const uint32_t t = tile - di * prm.tiles_per_desc;
            o = fastdiv(t, prm.div_tpo);
            part = t - o * prm.tpo;
        } else {
            di = __ldg(prm.tile_desc + tile);
        }
        if (threadIdx.x < sizeof(Desc) / 16)
            reinterpret_cast<uint4 *>(&sdesc[buf])[threadIdx.x] = __ldg(reinterpret_cast<const uint4 *>(prm.descs + di) + threadIdx.x);
        __syncthreads();
        const Desc &d = sdesc[buf];
        if (!prm.tiles_per_desc && !prm.win_span) {
            const uint32_t t = tile - d.tile0;
            o = fastdiv(t, d.div_tpo);
            part = t - o * d.tiles_per_outer;
        }
        const uint32_t row0 = part * d.rows_per_tile;
        if (row0 >= d.rows) continue;  // padding tile of a uniform group
        const uint32_t nrows = min(d.rows_per_tile, d.rows - row0);
        const char *src = prm.ptr[d.src_slot + o * d.src_slot_step] + d.src_off + o * d.src_outer;
        char *dst = prm.ptr[d.dst_slot + o * d.dst_slot_step] + d.dst_off + o * d.dst_outer;
        if (MODE == kModeRun) {
            uint32_t so = 0, dof = 0;
            if (row0) {  // a long run that was cut into rows
                const uint32_t i1 = fastdiv(row0, d.div_n0), i0 = row0 - i1 * d.n0;
                so = i1 * d.src_s1 + i0 * d.src_s0;
                dof = i1 * d.dst_s1 + i0 * d.dst_s0;
            }
            if (CHECK) {
                unsigned long long acc = 0;
                copy_run16<kUnroll, kThreads, true>(src + so, dst + dof, d.run, static_cast<unsigned long long>(d.src_off + o * d.src_outer - d.csum_base) + so, &acc);
                csum_flush<kThreads>(prm.sums + d.tag, acc);
            } else {
                copy_run16<kUnroll, kThreads>(src + so, dst + dof, d.run);
            }
        } else if (MODE == kModeRows) {
            if (CHECK) {
                unsigned long long acc = 0;
                copy_rows<4, kUnroll, kThreads, true>(d, src, dst, row0, nrows, static_cast<unsigned long long>(d.src_off + o * d.src_outer - d.csum_base), &acc);
                csum_flush<kThreads>(prm.sums + d.tag, acc);
            } else {
                copy_rows<4, kUnroll, kThreads>(d, src, dst, row0, nrows);
            }
        } else {
            switch (min(d.log2_align, prm.log2_ptr_align)) {
            case 4: copy_rows<4, kUnroll, kThreads>(d, src, dst, row0, nrows); break;
            case 3: copy_rows<3, kUnroll, kThreads>(d, src, dst, row0, nrows); break;
            case 2: copy_rows<2, kUnroll, kThreads>(d, src, dst, row0, nrows); break;
            case 1: copy_rows<1, kUnroll, kThreads>(d, src, dst, row0, nrows); break;
            default: copy_rows<0, kUnroll, kThreads>(d, src, dst, row0, nrows); break;
            }
        }
    }
}

// ------------------------------------------------------------------------------ host side
static int cuda_fail(cudaError_t e, const char *what)
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
    block_free(plan->device, plan->d_storage, plan->d_storage_bytes);
    plan->d_storage = nullptr;
    for (int k = 0; k < 2; k++) plan->group[k].d_descs = nullptr, plan->group[k].d_tile_desc = nullptr;
}

// One allocation and one copy per plan: [g0 descriptors | g0 tiles | g1 descriptors | g1 tiles],
// every part 256-byte aligned.
static int upload_plan(tc_plan *plan)
{
    auto pad = [](size_t n) { return (n + 255) & ~size_t(255); };
    size_t off[4], total = 0;
    for (int k = 0; k < 2; k++) {
        off[2 * k] = total;
        total += pad(plan->group[k].descs.size() * sizeof(Desc));
        off[2 * k + 1] = total;
        total += pad(plan->group[k].tile_desc.size() * sizeof(uint32_t));
    }
    if (total == 0) return TC_OK;
    std::vector<unsigned char> image(total);
    for (int k = 0; k < 2; k++) {
        const Group &g = plan->group[k];
        if (!g.descs.empty()) memcpy(image.data() + off[2 * k], g.descs.data(), g.descs.size() * sizeof(Desc));
        if (!g.tile_desc.empty()) memcpy(image.data() + off[2 * k + 1], g.tile_desc.data(), g.tile_desc.size() * sizeof(uint32_t));
    }
    cudaError_t e = block_alloc(plan->device, total, &plan->d_storage, &plan->d_storage_bytes);
    if (e != cudaSuccess) {
        plan->d_storage = nullptr;
        return e == cudaErrorMemoryAllocation ? fail(TC_ERR_OOM, "device allocation of %zu plan bytes failed", total) : cuda_fail(e, "cudaMalloc");
    }
    if ((e = cudaMemcpy(plan->d_storage, image.data(), total, cudaMemcpyHostToDevice)) != cudaSuccess) return cuda_fail(e, "cudaMemcpy(plan)");
    plan->device_bytes += static_cast<int64_t>(plan->d_storage_bytes);
    char *base = static_cast<char *>(plan->d_storage);
    for (int k = 0; k < 2; k++) {
        Group &g = plan->group[k];
        if (!g.descs.empty()) g.d_descs = reinterpret_cast<Desc *>(base + off[2 * k]);
        if (!g.tile_desc.empty()) g.d_tile_desc = reinterpret_cast<uint32_t *>(base + off[2 * k + 1]);
    }
    return TC_OK;
}

// Which executor build a group needs, given the alignment shared by the call's base pointers.
static int mode_for(const Group &g, uint32_t ptr_align)
{
    if (g.log2_align < 4 || ptr_align < 4) return kModeAny;
    return g.single_run_tiles ? kModeRun : kModeRows;
}

template <int NPTR, int MODE>
static int resident_ctas()
{
    int n = 0;
    if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&n, tc_copy_kernel<NPTR, MODE>, Shape<MODE>::threads, 0) != cudaSuccess || n < 1) n = 1;
    return n;
}

template <int NPTR>
static void resident_ctas_all(int out[3])
{
    out[kModeRun] = resident_ctas<NPTR, kModeRun>();
    out[kModeRows] = resident_ctas<NPTR, kModeRows>();
    out[kModeAny] = resident_ctas<NPTR, kModeAny>();
}

static void resident_ctas_for(size_t n_ptrs, int out[3])
{
    // queried once per table size class (the answer depends on the kernel, not on the plan)
    static int cache[3][3];
    static bool have[3];
    const int cls = n_ptrs <= 8 ? 0 : n_ptrs <= 400 ? 1 : 2;
    pthread_mutex_lock(&g_block_mu);
    if (!have[cls]) {
        if (cls == 0) resident_ctas_all<8>(cache[cls]);
        else if (cls == 1) resident_ctas_all<400>(cache[cls]);
        else resident_ctas_all<TC_MAX_TABLE_SLOTS>(cache[cls]);
        have[cls] = true;
    }
    for (int m = 0; m < 3; m++) out[m] = cache[cls][m];
    pthread_mutex_unlock(&g_block_mu);
}

static uint32_t grid_for(const tc_plan *plan, const Group &g, int mode, const Segment *win = nullptr)
{
    // Default: one CTA per tile.  The hardware block scheduler then balances the tiles over the
    // SMs and de-phases the CTAs' load and store bursts, which measured faster than a
    // persistent grid-stride grid.  tuning.ctas_per_sm / max_ctas select a persistent grid
    // (few CTAs suit transfers over the host link).
    uint64_t grid = std::min<uint64_t>(g.n_tiles, 0x7fffffffull);
    if (win) grid = win->nd ? static_cast<uint64_t>(win->no) * win->nd * (g.tiles_per_desc / g.descs[0].n_outer) : win->no;
    if (plan->tuning.ctas_per_sm > 0) {
        int per_sm = g.resident_ctas[mode] > 0 ? g.resident_ctas[mode] : 1;
        per_sm = std::min(per_sm, plan->tuning.ctas_per_sm);
        grid = std::min<uint64_t>(grid, static_cast<uint64_t>(plan->sm_count > 0 ? plan->sm_count : 148) * per_sm);
    }
    if (plan->tuning.max_ctas > 0) grid = std::min<uint64_t>(grid, plan->tuning.max_ctas);
    return static_cast<uint32_t>(grid);
}

template <int NPTR>
static int launch(const tc_plan *plan, const Group &g, const void *const *src, void *const *dst, uint32_t ptr_align, cudaStream_t stream,
                  const Segment *win = nullptr, unsigned long long *sums = nullptr)
{
    // Uniform groups with planes (KV) are walked plane-major by default: all blocks of plane 0,
    // then plane 1, ...  Together with descriptors sorted by destination offset, every plane
    // pass writes ascending addresses (and pack / unpack stream through the packed buffer),
    // which measured 3-5 % faster than walking the planes of one block after another.
    Segment whole{0, static_cast<uint32_t>(g.descs.size()), 0, g.descs.empty() ? 0 : g.descs[0].n_outer, 0, 0, 0};
    if (!win && g.tiles_per_desc && !g.descs.empty() && g.descs[0].n_outer > 1 && plan->tuning.tile_order != 1) win = &whole;
    const int mode = mode_for(g, ptr_align);
    if (sums && mode == kModeAny) return fail(TC_ERR_INVALID_ARG, "checksums need 16-byte aligned base pointers");
    const uint32_t grid = grid_for(plan, g, mode, win);
    Params<NPTR> prm;
    prm.descs = g.d_descs;
    prm.tile_desc = g.d_tile_desc;
    prm.n_tiles = static_cast<uint32_t>(g.n_tiles);
    prm.win_span = prm.win_d0 = prm.win_o0 = prm.win_tpo = prm.tile_base = 0;
    if (win && win->nd == 0) {  // a range of global tile ids
        prm.tile_base = win->d0;
        prm.n_tiles = win->d0 + win->no;
    } else if (win) {
        prm.win_tpo = g.tiles_per_desc / g.descs[0].n_outer;
        prm.win_span = win->nd * prm.win_tpo;
        prm.win_d0 = win->d0;
        prm.win_o0 = win->o0;
        prm.n_tiles = win->no * prm.win_span;
    }
    prm.tiles_per_desc = g.tiles_per_desc;
    prm.div_tpd = g.div_tpd;
    prm.tpo = g.tiles_per_desc ? g.tiles_per_desc / g.descs[0].n_outer : 1;
    prm.div_tpo = make_fastdiv(prm.tpo);
    prm.log2_ptr_align = ptr_align;
    prm.sums = sums;
    for (size_t i = 0; i < g.n_src; i++) prm.ptr[i] = const_cast<char *>(static_cast<const char *>(src[i]));
    for (size_t i = 0; i < g.n_dst; i++) prm.ptr[g.n_src + i] = static_cast<char *>(dst[i]);
    for (size_t i = g.n_src + g.n_dst; i < NPTR; i++) prm.ptr[i] = nullptr;
    if (sums) {
        if (mode == kModeRun) tc_copy_kernel<NPTR, kModeRun, true><<<grid, Shape<kModeRun>::threads, 0, stream>>>(prm);
        else tc_copy_kernel<NPTR, kModeRows, true><<<grid, Shape<kModeRows>::threads, 0, stream>>>(prm);
    } else
    switch (mode) {
    case kModeRun: tc_copy_kernel<NPTR, kModeRun><<<grid, Shape<kModeRun>::threads, 0, stream>>>(prm); break;
    case kModeRows: tc_copy_kernel<NPTR, kModeRows><<<grid, Shape<kModeRows>::threads, 0, stream>>>(prm); break;
    default: tc_copy_kernel<NPTR, kModeAny><<<grid, Shape<kModeAny>::threads, 0, stream>>>(prm); break;
    }
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) return cuda_fail(e, "kernel launch");
    return TC_OK;
}

static int launch_any(const tc_plan *plan, const Group &g, const void *const *src, void *const *dst, uint32_t ptr_align, cudaStream_t s, const Segment *win,
                      unsigned long long *sums = nullptr)
{
    const size_t n = g.n_src + g.n_dst;
    if (n <= 8) return launch<8>(plan, g, src, dst, ptr_align, s, win, sums);
    if (n <= 400) return launch<400>(plan, g, src, dst, ptr_align, s, win, sums);
    return launch<TC_MAX_TABLE_SLOTS>(plan, g, src, dst, ptr_align, s, win, sums);
}

// ---- staged host path: copy engines <-> device staging ring <-> kernel ----------------------
constexpr int kMaxDevices = 64;
// One ring per direction (0: device -> host, 1: host -> device), so that an offload and a
// reload running concurrently on two streams do not wait on each other's buffers.
struct StageRing {
    char *buf[kStageBuffers] = {};
    cudaEvent_t ready[kStageBuffers] = {}, freed[kStageBuffers] = {};
    bool freed_recorded[kStageBuffers] = {};
    cudaStream_t copy = nullptr;
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
    cudaEvent_t entry = nullptr;
    int refs = 0;
};
static StageArena g_stage[kMaxDevices];
static pthread_mutex_t g_stage_mu = PTHREAD_MUTEX_INITIALIZER;

static void stage_free(StageArena &a)
{
    for (StageRing &r : a.ring) {
        for (int b = 0; b < kStageBuffers; b++) {
            if (r.buf[b]) cudaFree(r.buf[b]);
            if (r.ready[b]) cudaEventDestroy(r.ready[b]);
            if (r.freed[b]) cudaEventDestroy(r.freed[b]);
        }
        if (r.copy) cudaStreamDestroy(r.copy);
    }
    for (int b = 0; b < kHostBuffers; b++) {
        if (a.host.buf[b]) cudaFreeHost(a.host.buf[b]);
        if (a.host.freed[b]) cudaEventDestroy(a.host.freed[b]);
    }
    if (a.entry) cudaEventDestroy(a.entry);
    a = StageArena();
}

static int stage_acquire(int device, int64_t *bytes)
{
    if (device < 0 || device >= kMaxDevices) return fail(TC_ERR_INVALID_ARG, "device ordinal %d is not supported", device);
    pthread_mutex_lock(&g_stage_mu);
    StageArena &a = g_stage[device];
    int rc = TC_OK;
    if (a.refs == 0) {
        a.refs = 1;  // the library's own reference: keeps the rings alive between plans
        cudaError_t e = cudaEventCreateWithFlags(&a.entry, cudaEventDisableTiming);
        for (StageRing &r : a.ring) {
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
    pthread_mutex_unlock(&g_stage_mu);
    return rc;
}

// The rings are kept once allocated (like the plan-storage cache): a caller that creates one
// staged plan per scheduler step must not pay six cudaMalloc / cudaFree pairs per step.
static void stage_release(int device)
{
    if (device < 0 || device >= kMaxDevices) return;
    pthread_mutex_lock(&g_stage_mu);
    StageArena &a = g_stage[device];
    if (a.refs > 1) a.refs--;  // the last reference is never dropped: the rings stay until exit
    pthread_mutex_unlock(&g_stage_mu);
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
static int execute_staged(const tc_plan *plan, int gi, const Group &g, const void *const *src, void *const *dst, uint32_t ptr_align, cudaStream_t s,
                          unsigned long long *sums = nullptr)
{
    StageArena &a = g_stage[plan->device];
    const bool to_device = g.host_is_src;
    StageRing &r = a.ring[to_device ? 1 : 0];
    int rc = TC_OK;
    (void)gi;
    pthread_mutex_lock(&g_stage_mu);
    TC_TRY(cudaEventRecord(a.entry, s), "cudaEventRecord");
    TC_TRY(cudaStreamWaitEvent(r.copy, a.entry, 0), "cudaStreamWaitEvent");
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
    pthread_mutex_unlock(&g_stage_mu);
    return rc;
}

// ---- cold path: file -> pinned host ring -> staging ring -> kernel ---------------------------
static pthread_mutex_t g_file_mu = PTHREAD_MUTEX_INITIALIZER;  // one file stream per process at a time

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
static int execute_streamed(const tc_plan *plan, const Group &g, int fd, int64_t file_off, void *const *dst, uint32_t ptr_align, cudaStream_t s,
                            unsigned long long *sums)
{
    StageArena &a = g_stage[plan->device];
    StageRing &r = a.ring[1];
    HostRing &h = a.host;
    const size_t n = g.segments.size();
    int rc = TC_OK;
    pthread_mutex_lock(&g_file_mu);
    pthread_mutex_lock(&g_stage_mu);
    rc = host_ring_acquire(h);
    pthread_mutex_unlock(&g_stage_mu);
    if (rc != TC_OK) {
        pthread_mutex_unlock(&g_file_mu);
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
            pthread_mutex_lock(&g_stage_mu);
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
            pthread_mutex_unlock(&g_stage_mu);
        }
    }  // the pool's destructor stops and joins the readers
    pthread_mutex_unlock(&g_file_mu);
    return rc;
}
#undef TC_TRY

// A table entry must be memory the device can address: device memory, managed memory, or host
// memory that is pinned and mapped.  Plain pageable host memory would make the kernel fault, so
// it is refused here, on the host.  Large tables are spot-checked (first, last and evenly spaced
// entries) to keep the call cheap.
static int check_addressable(const void *const *table, size_t n, const char *what)
{
    const size_t step = n <= 32 ? 1 : n / 32;
    for (size_t i = 0; i < n; i = (i + step < n || i == n - 1) ? i + step : n - 1) {
        cudaPointerAttributes attr;
        cudaError_t e = cudaPointerGetAttributes(&attr, table[i]);
        if (e != cudaSuccess) {
            cudaGetLastError();
            return fail(TC_ERR_INVALID_ARG, "%s table entry %zu (%p) is not a valid address for this device", what, i, table[i]);
        }
        if (attr.type == cudaMemoryTypeUnregistered)
            return fail(TC_ERR_INVALID_ARG, "%s table entry %zu (%p) is pageable host memory: pin it (cudaHostAlloc / cudaHostRegister) or use device memory", what, i, table[i]);
    }
    return TC_OK;
}

struct FileSource {
    int fd;
    int64_t offset;
};

static int execute(const tc_plan *plan, int gi, const void *const *src, size_t n_src, void *const *dst, size_t n_dst, void *stream,
                   unsigned long long *sums = nullptr, const FileSource *file = nullptr)
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
    if (!file && (rc = check_addressable(src, n_src, "source")) != TC_OK) return rc;
    if ((rc = check_addressable(const_cast<const void *const *>(dst), n_dst, "destination")) != TC_OK) return rc;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    if (file) return execute_streamed(plan, g, file->fd, file->offset, dst, ptr_align, s, sums);
    if (!g.segments.empty()) return execute_staged(plan, gi, g, src, dst, ptr_align, s, sums);
    return launch_any(plan, g, src, dst, ptr_align, s, nullptr, sums);
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
    pthread_mutex_lock(&g_stage_mu);
    for (StageArena &a : g_stage)
        if (a.refs == 1) {  // only the library's own reference is left
            for (StageRing &r : a.ring)
                if (r.copy) cudaStreamSynchronize(r.copy);
            stage_free(a);
        }
    pthread_mutex_unlock(&g_stage_mu);
    return TC_OK;
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
        out->grid[k] = g.n_tiles ? static_cast<int32_t>(grid_for(plan, g, mode_for(g, 4))) : 0;
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
        o.rows_per_tile = d.rows_per_tile; o.tiles_per_outer = d.tiles_per_outer; o.tile0 = d.tile0; o.reserved = 0;
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
    tc_plan plan;  // lives on the host for the duration of this call only
    plan.kind = spec->kind;
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
    if (g.n_tiles == 0) return execute(&plan, 0, src_bases, n_src, dst_bases, n_dst, stream);
    const size_t desc_bytes = g.descs.size() * sizeof(Desc);
    const size_t tile_bytes = g.tile_desc.size() * sizeof(uint32_t);
    if (desc_bytes + tile_bytes > TC_NOALLOC_SCRATCH_BYTES)
        return fail(TC_ERR_TOO_LARGE, "the call needs %zu bytes of descriptors and tiles; tc_kv_pack_noalloc holds at most %u: split the request or use tc_plan_create",
                    desc_bytes + tile_bytes, TC_NOALLOC_SCRATCH_BYTES);
    cudaError_t e = cudaGetDevice(&plan.device);
    if (e != cudaSuccess) return cuda_fail(e, "querying the current device");
    if (plan.device < 0 || plan.device >= kMaxDevices) return fail(TC_ERR_INVALID_ARG, "device ordinal %d is not supported", plan.device);
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
