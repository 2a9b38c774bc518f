// The copy-executor kernels (sm_100a).
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
#pragma once

#include <cuda_runtime.h>

#include "exec.h"  // kModeRun / kModeRows / kModeAny
#include "plan.h"

namespace tc {

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
    uint32_t n_descs;           // descriptors of the group (bounds the look-ahead prefetch)
    uint32_t tiles_per_desc;    // > 0 for uniform groups
    FastDiv div_tpd;
    uint32_t tpo;               // uniform groups: tiles per plane of one descriptor
    FastDiv div_tpo;
    uint32_t log2_ptr_align;    // alignment shared by every base pointer (capped at 4)
    // launch window (win_span == 0: the whole group).  Tile ids then walk plane-major over
    // descriptors [win_d0, ...) x planes [win_o0, ...): win_span = descriptors x win_tpo.
    uint32_t win_span, win_d0, win_o0, win_tpo;
    uint32_t win_o_end;         // first plane past the window
    uint32_t ppt, log2_unit;    // multi-plane tiles (MULTI builds): planes per tile, log2 of the padded plane
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

// Metadata look-ahead distances: about two waves of resident CTAs (148 SMs x 3), and for
// listed groups, where the descriptor of a later tile is not known without a load, a fixed
// number of descriptors.
constexpr uint32_t kLookAheadTiles = 1024, kLookAheadDescs = 16;
__device__ __forceinline__ void prefetch_l2(const void *p) { asm volatile("prefetch.global.L2 [%0];" ::"l"(p)); }

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

// A tile of n_units consecutive planes of one descriptor (small planes, see Group::ppt).  The
// tile's byte space gives every plane 2^log2_unit bytes, of which the first rows * run are real.
// Plane k of the tile starts at table[slot + (o + k) * slot_step] + off + (o + k) * outer on
// each side: a byte stride for single-pointer pools, another table entry for pools with one
// pointer per plane (a warp never straddles planes - they own at least 512 bytes of the byte
// space - so that lookup has one index per warp).  ROWS: decode rows inside a plane, else
// every plane is one run.  STEP: some pool of the group has one pointer per plane; without it
// both base pointers are read once per tile.
template <int LOGV, int U, int kThreads, bool ROWS, bool STEP, int NPTR>
__device__ __forceinline__ void copy_multi(const Desc &d, const Params<NPTR> &prm, uint32_t o, uint32_t n_units)
{
    using V = typename VecOf<LOGV>::type;
    const uint32_t log2_unit = prm.log2_unit;
    const uint32_t unit_bytes = d.rows * d.run, mask = (1u << log2_unit) - 1;
    const uint32_t nbytes = n_units << log2_unit;
    const uint32_t run = d.run, n0 = d.n0;
    const FastDiv div_run = d.div_run, div_n0 = d.div_n0;
    const uint32_t ss0 = d.src_s0, ss1 = d.src_s1, ds0 = d.dst_s0, ds1 = d.dst_s1;
    const long long src_outer = d.src_outer, dst_outer = d.dst_outer, src_off = d.src_off, dst_off = d.dst_off;
    const uint32_t sslot = d.src_slot, dslot = d.dst_slot, sstep = d.src_slot_step, dstep = d.dst_slot_step;
    const char *src_base = STEP ? nullptr : prm.ptr[sslot] + src_off;
    char *dst_base = STEP ? nullptr : prm.ptr[dslot] + dst_off;
#pragma unroll 1
    for (uint32_t base = threadIdx.x << LOGV; base < nbytes; base += (kThreads * U) << LOGV) {
        V val[U];
        uint32_t doff[U];
#pragma unroll
        for (int u = 0; u < U; u++) {
            const uint32_t byte = base + ((u * kThreads) << LOGV);
            const uint32_t k = o + (byte >> log2_unit), w = byte & mask;
            if (byte < nbytes && w < unit_bytes) {
                uint32_t so = w;
                doff[u] = w;
                if (ROWS) {
                    const uint32_t r = fastdiv(w, div_run);
                    const uint32_t col = w - r * run;
                    const uint32_t i1 = fastdiv(r, div_n0);
                    const uint32_t i0 = r - i1 * n0;
                    doff[u] = i1 * ds1 + i0 * ds0 + col;
                    so = i1 * ss1 + i0 * ss0 + col;
                }
                val[u] = ld_stream<V>((STEP ? prm.ptr[sslot + k * sstep] + src_off : src_base) + k * src_outer + so);
            }
        }
#pragma unroll
        for (int u = 0; u < U; u++) {
            const uint32_t byte = base + ((u * kThreads) << LOGV);
            const uint32_t k = o + (byte >> log2_unit), w = byte & mask;
            if (byte < nbytes && w < unit_bytes) st_stream<V>((STEP ? prm.ptr[dslot + k * dstep] + dst_off : dst_base) + k * dst_outer + doff[u], val[u]);
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

// MULTI: 0 one plane per tile; 1 several planes per tile, planes a byte stride apart; 2 the
// same with a pool that has one pointer per plane.
template <int NPTR, int MODE, bool CHECK = false, int MULTI = 0>
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
            o = prm.win_o0 + (MULTI ? ow * prm.ppt : ow);
            part = rem - dw * prm.win_tpo;
        } else if (prm.tiles_per_desc) {
            di = fastdiv(tile, prm.div_tpd);
            const uint32_t t = tile - di * prm.tiles_per_desc;
            o = fastdiv(t, prm.div_tpo);
            part = t - o * prm.tpo;
            if (MULTI) o *= prm.ppt;
        } else {
            di = __ldg(prm.tile_desc + tile);
        }
        if (threadIdx.x < sizeof(Desc) / 16)
            reinterpret_cast<uint4 *>(&sdesc[buf])[threadIdx.x] = __ldg(reinterpret_cast<const uint4 *>(prm.descs + di) + threadIdx.x);
        // Look-ahead: pull the metadata of tiles a few waves ahead into L2.  Consecutive tiles
        // start almost together, so without this every tile of a short descriptor waits on the
        // same DRAM miss (and, in listed groups, on the tile-list line before it).
        if (threadIdx.x == kThreads - 1) {
            const uint32_t ahead = tile + kLookAheadTiles;
            uint32_t da;
            if (prm.win_span) {
                const uint32_t rem = ahead % prm.win_span;
                da = prm.win_d0 + rem / prm.win_tpo;
            } else if (prm.tiles_per_desc) {
                da = fastdiv(ahead, prm.div_tpd);
            } else {
                if (ahead < prm.n_tiles) prefetch_l2(prm.tile_desc + ahead);
                da = di + kLookAheadDescs;
            }
            if (da < prm.n_descs) prefetch_l2(prm.descs + da);
        }
        __syncthreads();
        const Desc &d = sdesc[buf];
        if (!prm.tiles_per_desc && !prm.win_span) {
            const uint32_t t = tile - d.tile0;
            o = fastdiv(t, d.div_tpo);
            part = t - o * d.tiles_per_outer;
        }
        if (MULTI) {  // several whole planes of one descriptor (uniform groups, one part per plane)
            const uint32_t o_end = prm.win_span ? prm.win_o_end : d.n_outer;
            if (o >= o_end) continue;
            const uint32_t n_units = min(prm.ppt, o_end - o);
            if (MODE == kModeRun) {
                copy_multi<4, kUnroll, kThreads, false, MULTI == 2>(d, prm, o, n_units);
            } else if (MODE == kModeRows) {
                copy_multi<4, kUnroll, kThreads, true, MULTI == 2>(d, prm, o, n_units);
            } else {
                switch (min(d.log2_align, prm.log2_ptr_align)) {
                case 4: copy_multi<4, kUnroll, kThreads, true, MULTI == 2>(d, prm, o, n_units); break;
                case 3: copy_multi<3, 2 * kUnroll, kThreads, true, MULTI == 2>(d, prm, o, n_units); break;
                case 2: copy_multi<2, 2 * kUnroll, kThreads, true, MULTI == 2>(d, prm, o, n_units); break;
                case 1: copy_multi<1, 2 * kUnroll, kThreads, true, MULTI == 2>(d, prm, o, n_units); break;
                default: copy_multi<0, 2 * kUnroll, kThreads, true, MULTI == 2>(d, prm, o, n_units); break;
                }
            }
            continue;
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
            // narrower vectors cost fewer registers each, so more of them can be in flight
            case 3: copy_rows<3, 2 * kUnroll, kThreads>(d, src, dst, row0, nrows); break;
            case 2: copy_rows<2, 2 * kUnroll, kThreads>(d, src, dst, row0, nrows); break;
            case 1: copy_rows<1, 2 * kUnroll, kThreads>(d, src, dst, row0, nrows); break;
            default: copy_rows<0, 2 * kUnroll, kThreads>(d, src, dst, row0, nrows); break;
            }
        }
    }
}

}  // namespace tc
