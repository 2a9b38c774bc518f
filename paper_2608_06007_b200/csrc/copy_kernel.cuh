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
template <> struct Shape<kModeAny> { static constexpr int threads = 256, unroll = 4, min_ctas = 6; };

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
    uint32_t stage_bytes;       // dynamic shared memory of the launch (realigning path)
    uint32_t stage_always;      // take the shared-memory path for aligned tiles too (tuning.copy_path)
    uint32_t debug_bounds;      // the plan's bounds checker ran just before: copy nothing if it raised its flag
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

// Rows of a few bytes each (an element-granular scatter) at less than 16-byte alignment: vectors
// as wide as the alignment allows, several in flight per thread.  Out of line, so that the four
// widths do not weigh on the register allocation of the kernel's main paths.
template <int U, int kThreads>
__device__ __noinline__ void copy_rows_narrow(const Desc &d, const char *src, char *dst, uint32_t row0, uint32_t nrows, uint32_t align)
{
    switch (align) {
    case 3: copy_rows<3, U, kThreads>(d, src, dst, row0, nrows); break;
    case 2: copy_rows<2, 2 * U, kThreads>(d, src, dst, row0, nrows); break;
    case 1: copy_rows<1, 2 * U, kThreads>(d, src, dst, row0, nrows); break;
    default: copy_rows<0, 2 * U, kThreads>(d, src, dst, row0, nrows); break;
    }
}

// ---- realigning path: rows whose source and destination are not both 16-byte aligned ---------
// Alignment should cost a row its head and its tail, not the width of every access.  The CTA
// first brings the 16-byte aligned source chunks that cover its rows into shared memory - one
// bulk asynchronous copy (cp.async.bulk, completion on an mbarrier) per row, issued by one
// thread, so loading costs neither registers nor instructions per byte - then walks the 16-byte
// aligned DESTINATION chunks of every row: two aligned shared-memory loads and a funnel shift
// give a chunk's 16 bytes whatever the difference between the two alignments is, and the chunk
// leaves with one aligned 16-byte store.  Only the first and last chunk of a row can be
// partial; they are stored in naturally aligned pieces of 8, 4, 2 and 1 bytes.  The source side
// reads whole aligned 16-byte chunks, so up to 15 bytes before a row's first byte and after
// its last one are read (never a chunk without a byte of the row, hence never another page);
// nothing outside the row is ever written.
// Tiles whose rows differ in alignment (a row pitch that is not a multiple of 16) load the same
// way and work out every chunk's own alignments at run time.
// The wait for the bulk copies is bounded: if it ever ran out, the CTA would record
// kStatusBulkWaitTimeout in the device status word, wait once more for its copies, and return
// without storing (the host reads the word with tc_device_status).
// Bytes [sh, sh + 16) of the 32 bytes a | b.
__device__ __forceinline__ uint4 shift_bytes(uint4 a, uint4 b, uint32_t sh)
{
    const bool w2 = sh & 8, w1 = sh & 4;
    uint32_t b0 = w2 ? a.z : a.x, b1 = w2 ? a.w : a.y, b2 = w2 ? b.x : a.z, b3 = w2 ? b.y : a.w, b4 = w2 ? b.z : b.x, b5 = w2 ? b.w : b.y;
    const uint32_t c0 = w1 ? b1 : b0, c1 = w1 ? b2 : b1, c2 = w1 ? b3 : b2, c3 = w1 ? b4 : b3, c4 = w1 ? b5 : b4;
    const uint32_t bits = (sh & 3) * 8;
    return make_uint4(__funnelshift_r(c0, c1, bits), __funnelshift_r(c1, c2, bits), __funnelshift_r(c2, c3, bits), __funnelshift_r(c3, c4, bits));
}

// Store bytes [lo, hi) of the 16-byte chunk v at the 16-byte aligned address p, in naturally
// aligned pieces: ascending sizes up to the first boundary that fits, then descending sizes.
__device__ __forceinline__ void store_partial(char *p, uint4 v, uint32_t lo, uint32_t hi)
{
    auto word = [&](uint32_t k) { const uint32_t i = k >> 2; return (i & 2) ? ((i & 1) ? v.w : v.z) : ((i & 1) ? v.y : v.x); };
    auto put = [&](uint32_t k, uint32_t size) {
        if (size == 8) *reinterpret_cast<uint2 *>(p + k) = k ? make_uint2(v.z, v.w) : make_uint2(v.x, v.y);
        else if (size == 4) *reinterpret_cast<uint32_t *>(p + k) = word(k);
        else if (size == 2) *reinterpret_cast<uint16_t *>(p + k) = static_cast<uint16_t>(word(k) >> ((k & 2) * 8));
        else *reinterpret_cast<uint8_t *>(p + k) = static_cast<uint8_t>(word(k) >> ((k & 3) * 8));
    };
    uint32_t k = lo;
#pragma unroll
    for (uint32_t size = 1; size <= 8; size <<= 1)
        if ((k & size) && k + size <= hi) { put(k, size); k += size; }
#pragma unroll
    for (uint32_t size = 8; size >= 1; size >>= 1)
        if (k + size <= hi) { put(k, size); k += size; }
}

// Bytes [4 * WS + bits / 8, ... + 16) of the 32 bytes a | b, word shift known at compile time.
template <int WS>
__device__ __forceinline__ uint4 shift_words(uint4 a, uint4 b, uint32_t bits)
{
    const uint32_t w[8] = {a.x, a.y, a.z, a.w, b.x, b.y, b.z, b.w};
    return make_uint4(__funnelshift_r(w[WS], w[WS + 1], bits), __funnelshift_r(w[WS + 1], w[WS + 2], bits),
                      __funnelshift_r(w[WS + 2], w[WS + 3], bits), __funnelshift_r(w[WS + 3], w[WS + 4], bits));
}

// Sticky error flags set by kernels (read and cleared by tc_device_status).
enum : unsigned int { kStatusBulkWaitTimeout = 1u, kStatusOutOfBounds = 2u };
__device__ unsigned int g_device_status = 0;

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count)
{
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes)
{
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
// One potentially blocking test of a phase: the hardware may park the thread for up to about
// `hint_ns` while the phase is incomplete, so a waiting thread does not compete for issue slots.
__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity, uint32_t hint_ns)
{
    uint32_t done;
    asm volatile("{\n\t.reg .pred p;\n\tmbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2, %3;\n\tselp.u32 %0, 1, 0, p;\n\t}"
                 : "=r"(done) : "r"(bar), "r"(parity), "r"(hint_ns) : "memory");
    return done != 0;
}
// Bounded wait for a phase of the barrier: false if it did not complete within the limit
// (a bulk copy takes microseconds; the limit is of the order of a second).
__device__ __forceinline__ bool mbar_wait_bounded(uint32_t bar, uint32_t parity, uint32_t limit = 1u << 20)
{
    for (uint32_t spin = 0; spin < limit; spin++) {
        if (mbar_try_wait(bar, parity, 1000)) return true;
        if (spin > 64) __nanosleep(1000);  // long past any normal completion: back off
    }
    return false;
}
// Self-test of the bounded wait: a barrier that nothing ever arrives at.  The wait runs out after
// `limit` tries (milliseconds), the thread records the flag exactly as the copy kernel would, and
// the kernel returns normally; no copy is in flight, so there is nothing else to wait for.
__global__ void tc_wait_timeout_probe(uint32_t limit)
{
    __shared__ __align__(8) unsigned long long probe_bar;
    if (threadIdx.x != 0) return;
    const uint32_t bar = static_cast<uint32_t>(__cvta_generic_to_shared(&probe_bar));
    mbar_init(bar, 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    if (!mbar_wait_bounded(bar, 0, limit)) atomicOr(&g_device_status, kStatusBulkWaitTimeout);
}

// global -> shared bulk copy of `bytes` (a multiple of 16; both addresses 16-byte aligned) that
// reports to the barrier.  The source is this GPU's memory, a peer's or mapped host memory; the
// copy lands in the issuing CTA's own shared memory only.
__device__ __forceinline__ void bulk_load(uint32_t smem_dst, const void *gsrc, uint32_t bytes, uint32_t bar)
{
    asm volatile("cp.async.bulk.shared::cta.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                 ::"r"(smem_dst), "l"(gsrc), "r"(bytes), "r"(bar) : "memory");
}

// Geometry of one pass of the realigning path when every row of the tile has the same source
// and the same destination alignment (all strides multiples of 16, the common case: a shifted
// base pointer, a blob with a lead pad).  Chunk u = rr * units + c of the pass (row rr, chunk c
// of the row's destination) finds its bytes in shared memory at data + 16 * u + delta,
// delta = s_lo - d_lo.
struct RealignPass {
    const char *src;  // row 0 of the tile, plus the column offset
    char *dst;
    uint32_t row_base, n_rows;  // rows [row_base, row_base + n_rows) of the descriptor
    uint32_t units, len;        // chunks per row in the unit space, bytes of the row (piece) that move
    uint32_t s_lo, d_lo;        // source / destination address modulo 16
};

// Bytes one row of the pass brings in: the aligned source chunks that hold the row's bytes.
__device__ __forceinline__ uint32_t realign_row_bytes(const RealignPass &p) { return ((p.s_lo + p.len + 15) >> 4) << 4; }

// One bulk copy per row.  EXPECT: also announce the pass's bytes to the barrier (a caller that
// loads several passes' worth at once announces their sum itself).
template <int kThreads, bool EXPECT = true>
__device__ __forceinline__ void realign_load(const Desc &d, const RealignPass &p, uint32_t data_addr, uint32_t bar)
{
    const uint32_t n0 = d.n0, ss0 = d.src_s0, ss1 = d.src_s1;
    const FastDiv div_n0 = d.div_n0;
    const uint32_t row_bytes = realign_row_bytes(p);
    const char *base = p.src - p.s_lo;
    if (EXPECT && threadIdx.x == 0) mbar_expect_tx(bar, p.n_rows * row_bytes);
    for (uint32_t rr = threadIdx.x; rr < p.n_rows; rr += kThreads) {
        const uint32_t r = p.row_base + rr, i1 = fastdiv(r, div_n0), i0 = r - i1 * n0;
        bulk_load(data_addr + 16 * rr * p.units, base + (i1 * ss1 + i0 * ss0), row_bytes, bar);
    }
}

__device__ __forceinline__ uint4 lds128(uint32_t addr)
{
    uint4 v;
    asm volatile("ld.shared.v4.u32 {%0, %1, %2, %3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "r"(addr));
    return v;
}

// A pass over several planes of one descriptor (multi-plane tiles): row rr of the pass is row
// rr % rows of plane rr / rows, and plane j's destination (its address rounded down to 16) is
// dst[j], an array in shared memory.  All planes of such a pass share one alignment.
struct PlaneSet {
    uint32_t rows, magic;            // rows per plane; ceil(2^32 / rows) for the division (rows > 1)
    const unsigned long long *dst;   // per plane: destination of row 0, chunk 0
};

// Destination of chunk 0 of row rr of the pass, and the row's index inside its descriptor.
template <bool PLANES>
__device__ __forceinline__ char *realign_row(const Desc &d, const RealignPass &p, const PlaneSet *ps, uint32_t rr, uint32_t &r)
{
    char *base;
    if (PLANES) {
        const uint32_t j = ps->rows > 1 ? __umulhi(rr, ps->magic) : rr;
        r = rr - j * ps->rows;
        base = reinterpret_cast<char *>(ps->dst[j]);
    } else {
        r = p.row_base + rr;
        base = p.dst - p.d_lo;
    }
    const uint32_t i1 = fastdiv(r, d.div_n0), i0 = r - i1 * d.n0;
    return base + (i1 * d.dst_s1 + i0 * d.dst_s0);
}

// Whole destination chunks [c_begin, c_end) of every row of the pass.  data_addr: shared-memory
// address of the staged rows.  Two thread mappings keep the loop body short:
//   long rows   all threads walk the chunks of one row, kThreads at a time; the row is decoded
//               once, outside the loop;
//   short rows  (fewer chunks than threads) the CTA splits into groups of `units` threads; a
//               thread keeps its chunk index and steps through the rows, one group apart.
template <int WS, int kThreads, bool PLANES = false>
__device__ __forceinline__ void realign_store_full(const Desc &d, const RealignPass &p, uint32_t data_addr, uint32_t c_begin, uint32_t c_end,
                                                   const PlaneSet *ps = nullptr)
{
    const uint32_t units = p.units;
    const FastDiv div_units{d.units_mul, d.units_shift};
    const int delta = static_cast<int>(p.s_lo) - static_cast<int>(p.d_lo);
    const uint32_t bits = (static_cast<uint32_t>(delta) & 3) * 8;
    const uint32_t shifted = data_addr + 16 * (delta >> 4);  // delta >> 4 is 0 or -1
    uint32_t r;
    if (units >= kThreads) {
        for (uint32_t rr = 0; rr < p.n_rows; rr++) {
            // a thread's chunks are threadIdx.x + k * kThreads whatever c_begin is, so that a warp's
            // 512 bytes keep to whole 128-byte lines of the destination
            uint32_t c = threadIdx.x < c_begin ? threadIdx.x + kThreads : threadIdx.x;
            uint32_t at = shifted + 16 * (rr * units + c);
            char *out = realign_row<PLANES>(d, p, ps, rr, r) + 16 * static_cast<size_t>(c);
#pragma unroll 2
            for (; c < c_end; c += kThreads, at += 16 * kThreads, out += 16 * kThreads)
                st_stream<uint4>(out, shift_words<WS>(lds128(at), lds128(at + 16), bits));
        }
    } else {
        const uint32_t groups = fastdiv(kThreads, div_units);  // >= 1
        const uint32_t g = fastdiv(threadIdx.x, div_units), c = threadIdx.x - g * units;
        if (g >= groups || c < c_begin || c >= c_end) return;
        uint32_t at = shifted + 16 * (g * units + c);
#pragma unroll 2
        for (uint32_t rr = g; rr < p.n_rows; rr += groups, at += 16 * groups * units)
            st_stream<uint4>(realign_row<PLANES>(d, p, ps, rr, r) + 16 * c, shift_words<WS>(lds128(at), lds128(at + 16), bits));
    }
}

// Bytes [0, t) of a and bytes [t, 16) of b.
__device__ __forceinline__ uint4 merge_bytes(uint4 a, uint4 b, uint32_t t)
{
    auto pick = [&](uint32_t x, uint32_t y, uint32_t w) {
        const int n = static_cast<int>(t) - static_cast<int>(4 * w);  // bytes of this word that come from a
        const uint32_t mask = n >= 4 ? 0xffffffffu : n <= 0 ? 0u : (1u << (8 * n)) - 1;
        return (x & mask) | (y & ~mask);
    };
    return make_uint4(pick(a.x, b.x, 0), pick(a.y, b.y, 1), pick(a.z, b.z, 2), pick(a.w, b.w, 3));
}

// The partial chunks of every row of the pass: a head of bytes [d_lo, 16) of chunk 0 and / or
// a tail of bytes [0, t) of chunk c_last (or the bytes [d_lo, end) of a row that lies inside
// its first chunk).  One thread per row.  Where the next row of the destination starts exactly
// where this one ends (rows `adj` apart in the descriptor's row order, adjacent in memory), its
// head and this row's tail fill one chunk between them: that chunk is assembled from both rows
// and stored whole, instead of as up to eight small pieces.

template <int WS, int kThreads, bool PLANES = false>
__device__ __forceinline__ void realign_store_edges(const Desc &d, const RealignPass &p, uint32_t data_addr, uint32_t c_last, uint32_t end,
                                                    const PlaneSet *ps = nullptr)
{
    const uint32_t n0 = d.n0, ds0 = d.dst_s0, ds1 = d.dst_s1, units = p.units;
    const int delta = static_cast<int>(p.s_lo) - static_cast<int>(p.d_lo);
    const uint32_t bits = (static_cast<uint32_t>(delta) & 3) * 8;
    const uint32_t shifted = data_addr + 16 * (delta >> 4);
    const bool one_chunk = c_last == 0;
    const uint32_t t = end & 15;  // bytes of the tail
    // rows adjacent in the destination: the whole row moves (no column pieces) and its length
    // keeps the alignment, so that a tail of t bytes meets a head that starts at byte t = d_lo
    uint32_t adj = 0;
    if (!one_chunk && t && p.len == d.run && (d.run & 15) == 0) adj = (n0 > 1 && ds0 == d.run) ? 1 : (ds1 == d.run ? n0 : 0);
    // rows of the descriptor that the pass holds of the row's plane: [first, first + count)
    const uint32_t first = PLANES ? 0 : p.row_base, count = PLANES ? ps->rows : p.n_rows;
    for (uint32_t rr = threadIdx.x; rr < p.n_rows; rr += kThreads) {
        uint32_t r;
        char *out = realign_row<PLANES>(d, p, ps, rr, r);
        const uint32_t i0 = r - fastdiv(r, d.div_n0) * n0;
        const uint32_t row_at = shifted + 16 * rr * units;
        const bool has_next = adj && (adj == 1 ? i0 + 1 < n0 : r + n0 < d.rows) && r + adj < first + count;
        const bool has_prev = adj && (adj == 1 ? i0 >= 1 : r >= n0) && r >= first + adj;
        if ((p.d_lo || one_chunk) && !has_prev)
            store_partial(out, shift_words<WS>(lds128(row_at), lds128(row_at + 16), bits), p.d_lo, one_chunk ? end : 16);
        if (!one_chunk && t) {
            const uint32_t at = row_at + 16 * c_last;
            const uint4 tail = shift_words<WS>(lds128(at), lds128(at + 16), bits);
            if (has_next) {
                const uint32_t next_at = row_at + 16 * adj * units;
                st_stream<uint4>(out + 16 * c_last, merge_bytes(tail, shift_words<WS>(lds128(next_at), lds128(next_at + 16), bits), t));
            } else {
                store_partial(out + 16 * c_last, tail, 0, t);
            }
        }
    }
}

// Long rows (few per tile, down to one 32 KiB run): one thread per BYTE of the heads and tails,
// all at once.  A single thread walking the pieces of a head and a tail at the end of the tile
// is a latency the whole CTA waits for (a misaligned destination cost long rows 4-6 % that way).
// Short rows have too many ends for byte stores (128 rows of 256 bytes: half the speed) and
// keep the per-row loop of realign_store_edges.
constexpr uint32_t kByteEdgeMinRow = 1024;
template <int kThreads>
__device__ __forceinline__ void realign_store_edge_bytes(const Desc &d, const RealignPass &p, uint32_t data_addr, uint32_t c_last, uint32_t end)
{
    const bool one_chunk = c_last == 0;
    const uint32_t t = end & 15, units = p.units;
    for (uint32_t item = threadIdx.x; item < p.n_rows * 32; item += kThreads) {
        const uint32_t rr = item >> 5, k = item & 31;
        // k < 16: byte k of the row's first chunk; else byte k - 16 of its last chunk
        const bool is_tail = k >= 16;
        const bool valid = is_tail ? (!one_chunk && k - 16 < t) : (k >= p.d_lo && k < min(end, 16u) && (p.d_lo || one_chunk));
        if (!valid) continue;
        uint32_t r;
        char *out = realign_row<false>(d, p, nullptr, rr, r);
        const uint32_t byte = is_tail ? 16 * c_last + (k - 16) : k;  // position in the row's chunk space
        uint32_t v;
        asm volatile("ld.shared.u8 %0, [%1];" : "=r"(v) : "r"(data_addr + 16 * rr * units + p.s_lo + byte - p.d_lo));
        out[byte] = static_cast<char>(v);
    }
}

template <int WS, int kThreads, bool PLANES = false>
__device__ __forceinline__ void realign_store_all(const Desc &d, const RealignPass &p, uint32_t data, const PlaneSet *ps = nullptr)
{
    // chunk c of a row's destination covers row bytes [16c - d_lo, 16c - d_lo + 16)
    const uint32_t end = p.d_lo + p.len;  // first byte past the row, counted from the row's first chunk
    const uint32_t c_first = p.d_lo ? 1 : 0, c_last = end >> 4;  // whole chunks: [c_first, c_last)
    if (c_last > c_first) realign_store_full<WS, kThreads, PLANES>(d, p, data, c_first, c_last, ps);
    if (p.d_lo || (end & 15)) {
        if (!PLANES && p.len >= kByteEdgeMinRow) realign_store_edge_bytes<kThreads>(d, p, data, c_last, end);
        else realign_store_edges<WS, kThreads, PLANES>(d, p, data, c_last, end, ps);
    }
}

// Wait for the bulk copies of the current phase.  One thread waits (bounded) and tells the
// others, so that the CTA stays together; false: the copies did not arrive in time, the status
// word says so, and the caller returns from the kernel.
__device__ __forceinline__ bool realign_wait(uint32_t bar, uint32_t &phase, uint32_t *wait_ok)
{
    if (threadIdx.x == 0) {
        bool ok = mbar_wait_bounded(bar, phase);
        if (!ok) {
            atomicOr(&g_device_status, kStatusBulkWaitTimeout);
            ok = mbar_wait_bounded(bar, phase);  // the copies still target this CTA's memory
            *wait_ok = 0;
        }
    }
    __syncthreads();
    if (!*wait_ok) return false;
    mbar_try_wait(bar, phase, 0);  // completed: every thread observes the phase itself
    phase ^= 1;
    return true;
}

template <int kThreads, bool PLANES = false>
__device__ __forceinline__ void realign_store_dispatch(const Desc &d, const RealignPass &p, uint32_t data_addr, const PlaneSet *ps = nullptr)
{
    switch (((p.s_lo - p.d_lo) & 15) >> 2) {
    case 0: realign_store_all<0, kThreads, PLANES>(d, p, data_addr, ps); break;
    case 1: realign_store_all<1, kThreads, PLANES>(d, p, data_addr, ps); break;
    case 2: realign_store_all<2, kThreads, PLANES>(d, p, data_addr, ps); break;
    default: realign_store_all<3, kThreads, PLANES>(d, p, data_addr, ps); break;
    }
}

// The same for tiles whose rows differ in alignment (a row pitch that is not a multiple of 16):
// one bulk copy per row as well - every row announces its own byte count, the sum reaches the
// barrier through a shared-memory counter - and every chunk works out its own row's alignments.
// Out of line: a rare geometry.  False: the copies did not arrive in time (see realign_wait).
template <int kThreads>
__device__ __noinline__ bool realign_pass_mixed(const Desc &d, const char *src, char *dst, uint32_t row_base, uint32_t n_rows, uint32_t len, char *data,
                                                uint32_t bar, uint32_t phase, uint32_t *wait_ok, uint32_t *tx_total)
{
    const uint32_t n0 = d.n0, ss0 = d.src_s0, ss1 = d.src_s1, ds0 = d.dst_s0, ds1 = d.dst_s1;
    const FastDiv div_n0 = d.div_n0, div_units{d.units_mul, d.units_shift};
    const uint32_t units = (min(d.run, kRealignColumn) + 30) >> 4;
    const uint32_t data_addr = static_cast<uint32_t>(__cvta_generic_to_shared(data));
    const uint32_t total = n_rows * units;
    if (threadIdx.x == 0) *tx_total = 0;
    __syncthreads();
    uint32_t mine = 0;
    for (uint32_t rr = threadIdx.x; rr < n_rows; rr += kThreads) {
        const uint32_t r = row_base + rr, i1 = fastdiv(r, div_n0), i0 = r - i1 * n0;
        const char *s = src + (i1 * ss1 + i0 * ss0);
        const uint32_t s_lo = static_cast<uint32_t>(reinterpret_cast<uintptr_t>(s)) & 15;
        const uint32_t bytes = ((s_lo + len + 15) >> 4) << 4;
        bulk_load(data_addr + 16 * rr * units, s - s_lo, bytes, bar);
        mine += bytes;
    }
    if (mine) atomicAdd(tx_total, mine);
    __syncthreads();
    // the copies may complete before their bytes are announced (the count runs negative for a
    // moment); the phase cannot end before the one arrival that comes with the announcement
    if (threadIdx.x == 0) mbar_expect_tx(bar, *tx_total);
    if (!realign_wait(bar, phase, wait_ok)) return false;  // the caller flips its own copy of the phase
    // whole chunks first, in one loop without the partial-store code; a chunk knows from its row's
    // destination alignment whether it is whole
    for (uint32_t u = threadIdx.x; u < total; u += kThreads) {
        const uint32_t rr = fastdiv(u, div_units), c = u - rr * units;
        const uint32_t r = row_base + rr, i1 = fastdiv(r, div_n0), i0 = r - i1 * n0;
        char *dp = dst + (i1 * ds1 + i0 * ds0);
        const uint32_t d_lo = static_cast<uint32_t>(reinterpret_cast<uintptr_t>(dp)) & 15;
        const int first = static_cast<int>(16 * c) - static_cast<int>(d_lo);  // row byte at the chunk's byte 0
        if (first < 0 || first + 16 > static_cast<int>(len)) continue;
        const uint32_t s_lo = static_cast<uint32_t>(reinterpret_cast<uintptr_t>(src + (i1 * ss1 + i0 * ss0))) & 15;
        const uint32_t q = s_lo + first;  // the row's byte b sits at 16 * rr * units + s_lo + b
        const uint32_t at = data_addr + 16 * (rr * units) + 16 * (q >> 4);
        st_stream<uint4>(dp + first, shift_bytes(lds128(at), lds128(at + 16), q & 15));
    }
    // then the partial first and last chunk of every row: one thread per (row, end).  (Storing
    // the chunk that two destination-adjacent rows share once, as the same-alignment path does,
    // measured no faster here.)
    for (uint32_t item = threadIdx.x; item < 2 * n_rows; item += kThreads) {
        const uint32_t rr = item >> 1;
        const uint32_t r = row_base + rr, i1 = fastdiv(r, div_n0), i0 = r - i1 * n0;
        char *dp = dst + (i1 * ds1 + i0 * ds0);
        const uint32_t d_lo = static_cast<uint32_t>(reinterpret_cast<uintptr_t>(dp)) & 15;
        const uint32_t end = d_lo + len;  // first byte past the row, counted from its first chunk
        uint32_t c, lo, hi;
        if (item & 1) {  // tail: chunk end / 16, unless the row ends on a boundary or lies in one chunk
            c = end >> 4;
            lo = 0;
            hi = end & 15;
            if (c == 0 || hi == 0) continue;
        } else {         // head: chunk 0, unless it is whole
            c = 0;
            lo = d_lo;
            hi = min(end, 16u);
            if (lo == 0 && hi == 16) continue;
        }
        const uint32_t s_lo = static_cast<uint32_t>(reinterpret_cast<uintptr_t>(src + (i1 * ss1 + i0 * ss0))) & 15;
        const int q = static_cast<int>(s_lo) + static_cast<int>(16 * c) - static_cast<int>(d_lo);  // >= -15
        const uint32_t at = data_addr + 16 * (rr * units) + 16 * (q >> 4);
        store_partial(dp - d_lo + 16 * c, shift_bytes(lds128(at), lds128(at + 16), static_cast<uint32_t>(q) & 15), lo, hi);
    }
    return true;
}

// Rows that are ADJACENT IN THE DESTINATION (tokens of one head in a head-major buffer, heads of
// one token in a token-major block, the rows of a dim-1 weight slice) are staged in destination
// order, back to back, so that a group of them is one long row for the store loop: one row
// decode per group, heads and tails only at the ends of a group.  With a misaligned source a row
// occupies [s_lo, s_lo + run) of its run + 16 covering bytes, and the next row's data begins in
// the chunk that holds this row's last s_lo bytes: the whole chunks of a row arrive by bulk copy,
// the chunk two rows share is put together by one thread from the two aligned source chunks.
// Geometry of the tile in the descriptor's row order k -> (i1, i0) = (k / n0, k % n0):
//   across  rows a step of n0 apart are adjacent (dst_s1 == run): the tile must hold whole
//           i1-columns, group g = i0, position i1; the groups are dst_s0 apart, and when that
//           equals a group's length the whole tile is one group;
//   along   rows one apart are adjacent (dst_s0 == run), the tile lies inside one i1 or the i1
//           are adjacent too: one group, position = row.
// Rows of at least kJoinMinRun bytes in groups of at least kThreads chunks only.  Short rows (the
// 256-byte head rows of a KV block) measured slower this way than in their own slots (pack / unpack
// with the source misaligned 5.9 / 5.6 against 6.3 / 6.4 TB/s: one more bulk copy and one merge
// per row, and a store loop entered once per group, cost more instructions than the per-row
// loop's heads and tails); rows of 1 KiB and more gain 3-4 % with a misaligned destination.
// Returns 1 done, 0 not this geometry (nothing touched), -1 the bulk copies did not arrive.
template <int WS, int kThreads>
__device__ __forceinline__ void realign_store_joined(char *dst0, uint32_t vstride, uint32_t groups, uint32_t units, uint32_t len, uint32_t s_lo, uint32_t d_lo,
                                                     uint32_t data_addr)
{
    const uint32_t end = d_lo + len, c_first = d_lo ? 1 : 0, c_last = end >> 4, t = end & 15;
    const int delta = static_cast<int>(s_lo) - static_cast<int>(d_lo);
    const uint32_t bits = (static_cast<uint32_t>(delta) & 3) * 8;
    const uint32_t shifted = data_addr + 16 * (delta >> 4);
    for (uint32_t g = 0; g < groups; g++) {
        uint32_t c = threadIdx.x < c_first ? threadIdx.x + kThreads : threadIdx.x;
        uint32_t at = shifted + 16 * (g * units + c);
        char *out = dst0 + static_cast<size_t>(g) * vstride + 16 * static_cast<size_t>(c);
#pragma unroll 2
        for (; c < c_last; c += kThreads, at += 16 * kThreads, out += 16 * kThreads)
            st_stream<uint4>(out, shift_words<WS>(lds128(at), lds128(at + 16), bits));
    }
    if (d_lo || t) {  // one thread per byte of the groups' heads and tails
        for (uint32_t item = threadIdx.x; item < groups * 32; item += kThreads) {
            const uint32_t g = item >> 5, k = item & 31;
            const bool is_tail = k >= 16;
            if (is_tail ? k - 16 >= t : (k < d_lo || !d_lo)) continue;
            const uint32_t byte = is_tail ? 16 * c_last + (k - 16) : k;
            uint32_t v;
            asm volatile("ld.shared.u8 %0, [%1];" : "=r"(v) : "r"(data_addr + 16 * g * units + s_lo + byte - d_lo));
            dst0[static_cast<size_t>(g) * vstride + byte] = static_cast<char>(v);
        }
    }
}

template <int kThreads>
__device__ __forceinline__ int realign_tile_joined(const Desc &d, const char *src, char *dst, uint32_t row0, uint32_t nrows, uint32_t data_addr, uint32_t stage_bytes,
                                                   uint32_t bar, uint32_t &phase, uint32_t *wait_ok)
{
    const uint32_t run = d.run, n0 = d.n0;
    if ((run & 15) || run < kJoinMinRun || run > kRealignColumn || nrows < 2) return 0;
    const uint32_t j1 = fastdiv(row0, d.div_n0), j0 = row0 - j1 * n0;  // the tile's first row
    bool across = false;
    uint32_t groups = 1, glen = nrows, vstride = 0, cols = 0;  // cols: i1-columns of the tile
    if (d.dst_s1 == run) {
        cols = fastdiv(nrows, d.div_n0);
        if (j0 || cols * n0 != nrows) return 0;
        across = true;
        if (n0 > 1 && d.dst_s0 != cols * run) groups = n0, glen = cols, vstride = d.dst_s0;
    } else if (n0 > 1 && d.dst_s0 == run) {
        if (j0 + nrows > n0 && d.dst_s1 != n0 * run) return 0;
    } else {
        return 0;
    }
    const uint32_t len = glen * run, units = (len + 30) >> 4;
    const uint32_t side = data_addr + groups * (units << 4) + 16;  // 16 bytes per row: the chunk that holds its last bytes
    if (glen < 2 || units < kThreads || groups * (units << 4) + 48 + 16 * (nrows + 1) > stage_bytes) return 0;
    const char *s0 = src + (j1 * d.src_s1 + j0 * d.src_s0);
    char *d0 = dst + (j1 * d.dst_s1 + j0 * d.dst_s0);
    const uint32_t s_lo = static_cast<uint32_t>(reinterpret_cast<uintptr_t>(s0)) & 15;
    const uint32_t d_lo = static_cast<uint32_t>(reinterpret_cast<uintptr_t>(d0)) & 15;
    if (threadIdx.x == 0) mbar_expect_tx(bar, nrows * (s_lo ? run + 16 : run));
    // row rr of the tile -> group g, position pos in it, place q among all staged rows
    auto place = [&](uint32_t rr, uint32_t &i1, uint32_t &i0, uint32_t &g, uint32_t &pos) {
        const uint32_t r = row0 + rr;
        i1 = fastdiv(r, d.div_n0);
        i0 = r - i1 * n0;
        g = 0;
        pos = rr;
        if (across) {
            if (groups > 1) g = i0, pos = i1 - j1;
            else pos = i0 * cols + (i1 - j1);
        }
    };
    for (uint32_t rr = threadIdx.x; rr < nrows; rr += kThreads) {
        uint32_t i1, i0, g, pos;
        place(rr, i1, i0, g, pos);
        const char *row = src + (i1 * d.src_s1 + i0 * d.src_s0) - s_lo;  // its first aligned chunk
        const uint32_t at = data_addr + 16 * g * units + pos * run;
        if (!s_lo || pos + 1 == glen) {
            bulk_load(at, row, s_lo ? run + 16 : run, bar);
        } else {
            // the chunk with the row's last s_lo bytes would land on the next row's first chunk
            bulk_load(at, row, run, bar);
            bulk_load(side + 16 * (g * glen + pos + 1), row + run, 16, bar);
        }
    }
    if (!realign_wait(bar, phase, wait_ok)) return -1;
    if (s_lo) {
        for (uint32_t rr = threadIdx.x; rr < nrows; rr += kThreads) {
            uint32_t i1, i0, g, pos;
            place(rr, i1, i0, g, pos);
            if (pos == 0) continue;
            const uint32_t at = data_addr + 16 * g * units + pos * run;
            const uint4 v = merge_bytes(lds128(side + 16 * (g * glen + pos)), lds128(at), s_lo);
            asm volatile("st.shared.v4.u32 [%0], {%1, %2, %3, %4};" ::"r"(at), "r"(v.x), "r"(v.y), "r"(v.z), "r"(v.w) : "memory");
        }
        __syncthreads();
    }
    char *out0 = d0 - d_lo;
    switch (((s_lo - d_lo) & 15) >> 2) {
    case 0: realign_store_joined<0, kThreads>(out0, vstride, groups, units, len, s_lo, d_lo, data_addr); break;
    case 1: realign_store_joined<1, kThreads>(out0, vstride, groups, units, len, s_lo, d_lo, data_addr); break;
    case 2: realign_store_joined<2, kThreads>(out0, vstride, groups, units, len, s_lo, d_lo, data_addr); break;
    default: realign_store_joined<3, kThreads>(out0, vstride, groups, units, len, s_lo, d_lo, data_addr); break;
    }
    // the next tile's bulk copies overwrite chunks this one wrote with ordinary stores
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    __syncthreads();
    return 1;
}

// SHORT rows that follow one another in the destination a step of n0 apart (dst_s1 == run: the
// tokens of a head in a head-major buffer, the heads of a token in a token-major block), through
// a MISALIGNED destination.  Stored row by row, every row boundary is two half-written 32-byte
// sectors - the chunk two rows share goes out apart from the chunk next to it - and partial
// sectors are what the memory system charges for.  Here the rows keep their own slots, each
// slot is completed after the wait with the first chunk of the row that follows it in the
// destination (copied from that row's slot, merged with the row's own last bytes when the source
// is misaligned too), and the store loop walks the DESTINATION: thread t takes the aligned chunks t, t + kThreads, ...
// of a destination run and finds each in its row's slot, so that a warp's store is 512 contiguous,
// sector-aligned bytes whatever rows they come from.  Only the two ends of a run are partial.
// Needs: whole i1-columns in the tile, chunks per row a power of two, and, where all rows of
// the tile form one run, a power-of-two column count.  Returns 1 done, 0 not this geometry
// (nothing touched), -1 the bulk copies did not arrive.
template <int WS, int kThreads>
__device__ __forceinline__ void realign_store_dest_order(char *out0, uint32_t vstride, uint32_t groups, uint32_t total, uint32_t lcpr, uint32_t pmask, uint32_t pshift,
                                                         uint32_t n0, uint32_t pitch, uint32_t extra, uint32_t s_lo, uint32_t d_lo, uint32_t data_addr)
{
    // row rr (column k1 = p & pmask of the tile) keeps its chunks from 16 * (rr * pitch + k1 * extra) on
    const int delta = static_cast<int>(s_lo) - static_cast<int>(d_lo);
    const uint32_t bits = (static_cast<uint32_t>(delta) & 3) * 8;
    const uint32_t shifted = data_addr + 16 * (delta >> 4);
    const uint32_t cmask = (1u << lcpr) - 1;
    const uint32_t off = d_lo ? 1 : 0;  // through a misaligned destination a run's first chunk is partial
    auto chunk_of = [&](uint32_t p, uint32_t c) { return ((p & pmask) * n0 + (p >> pshift)) * pitch + (p & pmask) * extra + c; };
    if (total <= kThreads) {
        // short runs (a head's 16 tokens): a thread keeps its chunk and steps through the runs;
        // where a run has fewer chunks than the CTA has threads (128-byte rows), gpar runs go side by side
        uint32_t m = threadIdx.x, g0 = 0, gpar = 1;
        if (total < kThreads && (total & (total - 1)) == 0) {
            const uint32_t lt = 31 - __clz(total);
            gpar = kThreads >> lt;
            g0 = m >> lt;
            m &= total - 1;
        }
        if (m >= off && m < total) {
            uint32_t at = shifted + 16 * (chunk_of((m - off) >> lcpr, ((m - off) & cmask) + off) + g0 * pitch);
            char *out = out0 + 16 * static_cast<size_t>(m) + static_cast<size_t>(g0) * vstride;
            const size_t ostep = static_cast<size_t>(gpar) * vstride;
#pragma unroll 4
            for (uint32_t g = g0; g < groups; g += gpar, at += 16 * pitch * gpar, out += ostep)
                st_stream<uint4>(out, shift_words<WS>(lds128(at), lds128(at + 16), bits));
        }
    } else if (const uint32_t rpi = kThreads >> lcpr, rr_inc = pshift == 31 ? rpi * n0 : ((rpi & pmask) == 0 ? rpi >> pshift : 0); rr_inc) {
        // longer runs whose rows advance by a constant from one sweep of the CTA over the run to the next
        // (rpi rows per sweep): the chunk is decoded once, the loop only adds
        const uint32_t m0 = threadIdx.x >= off ? threadIdx.x : kThreads;  // a partial chunk 0: thread 0 starts a sweep later
        const uint32_t at0 = shifted + 16 * chunk_of((m0 - off) >> lcpr, ((m0 - off) & cmask) + off);
        const uint32_t step = 16 * (pitch * rr_inc + (pshift == 31 ? extra * rpi : 0));
        for (uint32_t g = 0; g < groups; g++) {
            uint32_t at = at0 + 16 * g * pitch;
            char *out = out0 + static_cast<size_t>(g) * vstride + 16 * static_cast<size_t>(m0);
#pragma unroll 2
            for (uint32_t m = m0; m < total; m += kThreads, at += step, out += 16 * kThreads)
                st_stream<uint4>(out, shift_words<WS>(lds128(at), lds128(at + 16), bits));
        }
    } else {
        for (uint32_t g = 0; g < groups; g++) {
            char *out = out0 + static_cast<size_t>(g) * vstride;
#pragma unroll 2
            for (uint32_t m = threadIdx.x; m < total; m += kThreads) {
                if (m < off) continue;
                const uint32_t at = shifted + 16 * (chunk_of((m - off) >> lcpr, ((m - off) & cmask) + off) + g * pitch);
                st_stream<uint4>(out + 16 * static_cast<size_t>(m), shift_words<WS>(lds128(at), lds128(at + 16), bits));
            }
        }
    }
    // the first 16 - d_lo and the last d_lo bytes of every run, a thread per byte
    const uint32_t last_p = (total >> lcpr) - 1;
    for (uint32_t item = threadIdx.x; item < (d_lo ? groups * 16 : 0); item += kThreads) {
        const uint32_t g = item >> 4, k = item & 15;
        const bool tail = k < d_lo;  // k < d_lo: byte k of the run's last chunk; else byte k of its first
        const uint32_t row_byte = tail ? (16u << lcpr) - d_lo + k : k - d_lo;
        uint32_t v;
        asm volatile("ld.shared.u8 %0, [%1];" : "=r"(v) : "r"(data_addr + 16 * (chunk_of(tail ? last_p : 0, 0) + g * pitch) + s_lo + row_byte));
        out0[static_cast<size_t>(g) * vstride + (tail ? 16 * static_cast<size_t>(total) + k : k)] = static_cast<char>(v);
    }
}

template <int kThreads>
__device__ __forceinline__ int realign_tile_dest_order(const Desc &d, const char *src, char *dst, uint32_t row0, uint32_t nrows, uint32_t data_addr, uint32_t stage_bytes,
                                                       uint32_t bar, uint32_t &phase, uint32_t *wait_ok)
{
    const uint32_t run = d.run, n0 = d.n0, cpr = run >> 4;
    if ((run & 15) || (cpr & (cpr - 1)) || run >= kJoinMinRun || d.dst_s1 != run || (n0 > 1 && d.dst_s0 == run)) return 0;
    const uint32_t j1 = fastdiv(row0, d.div_n0), cols = fastdiv(nrows, d.div_n0);
    if (row0 != j1 * n0 || cols * n0 != nrows || cols < 2) return 0;
    const char *s0 = src + j1 * d.src_s1;
    char *d0 = dst + j1 * d.dst_s1;
    const uint32_t s_lo = static_cast<uint32_t>(reinterpret_cast<uintptr_t>(s0)) & 15;
    const uint32_t d_lo = static_cast<uint32_t>(reinterpret_cast<uintptr_t>(d0)) & 15;
    // An aligned destination is taken this way only where the misaligned source is contiguous
    // along i0 (a packed buffer's tokens): a column of n0 rows then arrives as ONE bulk copy, its
    // rows at the source's own pitch, instead of n0 overlapping ones (with a slot per row the walk
    // measured no faster than the per-row loop, and 1.5 % slower for unpack).
    const bool pieces = d_lo == 0 && d.src_s0 == run;  // (both sides aligned: tuning.copy_path = 1, or an aligned tile of a misaligned call)
    if (d_lo == 0 && !pieces) return 0;
    // chunks per slot: the row's own, and what the chunk it shares with the next row needs of that
    // row - its first aligned chunk, and its second one too when s_lo > d_lo
    const uint32_t units = pieces ? cpr : cpr + (s_lo > d_lo ? 2 : 1);
    if ((pieces ? cols * (n0 * cpr + 1) * 16 : nrows * (units << 4)) + 32 > stage_bytes) return 0;
    // one run per i0, dst_s0 apart - or, where those runs are adjacent too, one run in all
    const bool one_run = n0 == 1 || d.dst_s0 == cols * run;
    if (one_run && n0 > 1 && (cols & (cols - 1))) return 0;
    const uint32_t lcpr = 31 - __clz(cpr);
    const uint32_t groups = one_run ? 1 : n0, glen = one_run ? nrows : cols;
    const uint32_t pmask = one_run && n0 > 1 ? cols - 1 : 0xffffffffu, pshift = one_run && n0 > 1 ? 31 - __clz(cols) : 31;
    const char *base = s0 - s_lo;
    if (pieces) {
        const uint32_t piece_bytes = n0 * run + (s_lo ? 16 : 0);  // never a chunk without a byte of the column
        if (threadIdx.x == 0) mbar_expect_tx(bar, cols * piece_bytes);
        for (uint32_t k1 = threadIdx.x; k1 < cols; k1 += kThreads) bulk_load(data_addr + 16 * k1 * (n0 * cpr + 1), base + k1 * d.src_s1, piece_bytes, bar);
    } else {
        if (threadIdx.x == 0) mbar_expect_tx(bar, nrows * (s_lo ? run + 16 : run));
        for (uint32_t rr = threadIdx.x; rr < nrows; rr += kThreads) {
            const uint32_t k1 = fastdiv(rr, d.div_n0), i0 = rr - k1 * n0;  // the tile starts on an i1 boundary
            bulk_load(data_addr + 16 * rr * units, base + (k1 * d.src_s1 + i0 * d.src_s0), s_lo ? run + 16 : run, bar);
        }
    }
    if (!realign_wait(bar, phase, wait_ok)) return -1;
    // complete every slot with the first chunk of the row after it in the destination (the next
    // column of the same i0, or, in a single run, the first column of the next i0): from that
    // row's own slot - a second copy from global memory per row, bulk or not, cost more than it saved
    for (uint32_t rr = threadIdx.x; rr < (d_lo ? nrows : 0); rr += kThreads) {
        const uint32_t k1 = fastdiv(rr, d.div_n0), i0 = rr - k1 * n0;
        uint32_t next;
        if (k1 + 1 < cols) next = rr + n0;
        else if (one_run && i0 + 1 < n0) next = i0 + 1;
        else continue;
        const uint32_t at = data_addr + 16 * (rr * units + cpr);
        uint4 v = lds128(data_addr + 16 * next * units);
        if (s_lo) v = merge_bytes(lds128(at), v, s_lo);
        asm volatile("st.shared.v4.u32 [%0], {%1, %2, %3, %4};" ::"r"(at), "r"(v.x), "r"(v.y), "r"(v.z), "r"(v.w) : "memory");
        if (s_lo > d_lo) {
            v = lds128(data_addr + 16 * (next * units + 1));
            asm volatile("st.shared.v4.u32 [%0], {%1, %2, %3, %4};" ::"r"(at + 16), "r"(v.x), "r"(v.y), "r"(v.z), "r"(v.w) : "memory");
        }
    }
    if (d_lo) __syncthreads();
    char *out0 = d0 - d_lo;
    const uint32_t total = glen * cpr;
    switch (((s_lo - d_lo) & 15) >> 2) {
    case 0: realign_store_dest_order<0, kThreads>(out0, d.dst_s0, groups, total, lcpr, pmask, pshift, n0, units, pieces ? 1 : 0, s_lo, d_lo, data_addr); break;
    case 1: realign_store_dest_order<1, kThreads>(out0, d.dst_s0, groups, total, lcpr, pmask, pshift, n0, units, pieces ? 1 : 0, s_lo, d_lo, data_addr); break;
    case 2: realign_store_dest_order<2, kThreads>(out0, d.dst_s0, groups, total, lcpr, pmask, pshift, n0, units, pieces ? 1 : 0, s_lo, d_lo, data_addr); break;
    default: realign_store_dest_order<3, kThreads>(out0, d.dst_s0, groups, total, lcpr, pmask, pshift, n0, units, pieces ? 1 : 0, s_lo, d_lo, data_addr); break;
    }
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");  // ordinary stores into the slots, bulk copies next
    __syncthreads();
    return 1;
}

// Rows [row0, row0 + nrows) of one outer index of descriptor d, any alignment; src / dst point
// at row 0.  `stage` is the shared-memory staging area (16-byte aligned, stage_bytes long, of
// which the first and last 16 are padding that neighbouring-chunk loads may touch): a pass
// stages as many whole rows as fit, row rr in the `units` chunks from 16 * rr * units on,
// starting at the row's first aligned source chunk.  A row longer than kRealignColumn is taken
// in column pieces.  bar / phase: the CTA's mbarrier and the parity of its next phase.
// Returns false if a bulk copy did not arrive in time (the caller returns from the kernel).
template <int kThreads>
__device__ __forceinline__ bool copy_rows_realign(const Desc &d, const char *src, char *dst, uint32_t row0, uint32_t nrows, char *stage, uint32_t stage_bytes,
                                                  uint32_t bar, uint32_t &phase, uint32_t *wait_ok)
{
    const uint32_t run = d.run;
    const uint32_t column = min(run, kRealignColumn);
    const uint32_t units = (column + 30) >> 4;  // 16-byte chunks a row piece can touch, on either side
    const uint32_t rows_per_pass = (stage_bytes - 32) / (units << 4);  // >= 1: the launch sizes the area for it
    char *data = stage + 16;
    const uint32_t data_addr = static_cast<uint32_t>(__cvta_generic_to_shared(data));
    const bool same_alignment = ((d.src_s0 | d.src_s1 | d.dst_s0 | d.dst_s1) & 15) == 0;
    if (same_alignment) {
        const int joined = realign_tile_joined<kThreads>(d, src, dst, row0, nrows, data_addr, stage_bytes, bar, phase, wait_ok);
        if (joined) return joined > 0;
        const int walked = realign_tile_dest_order<kThreads>(d, src, dst, row0, nrows, data_addr, stage_bytes, bar, phase, wait_ok);
        if (walked) return walked > 0;
    }
    for (uint32_t col0 = 0; col0 < run; col0 += column) {
        const uint32_t len = min(column, run - col0);
        for (uint32_t r0 = 0; r0 < nrows; r0 += rows_per_pass) {
            const uint32_t n_rows = min(rows_per_pass, nrows - r0);
            if (same_alignment) {
                RealignPass p;
                p.src = src + col0;
                p.dst = dst + col0;
                p.row_base = row0 + r0;
                p.n_rows = n_rows;
                p.units = units;
                p.len = len;
                p.s_lo = static_cast<uint32_t>(reinterpret_cast<uintptr_t>(p.src)) & 15;
                p.d_lo = static_cast<uint32_t>(reinterpret_cast<uintptr_t>(p.dst)) & 15;
                realign_load<kThreads>(d, p, data_addr, bar);
                // one thread waits (bounded) and tells the others, so that the CTA stays together
                if (threadIdx.x == 0) {
                    bool ok = mbar_wait_bounded(bar, phase);
                    if (!ok) {
                        atomicOr(&g_device_status, kStatusBulkWaitTimeout);
                        ok = mbar_wait_bounded(bar, phase);  // the copies still target this CTA's memory
                        *wait_ok = 0;
                    }
                }
                __syncthreads();
                if (!*wait_ok) return false;
                mbar_try_wait(bar, phase, 0);  // completed: every thread observes the phase itself
                phase ^= 1;
                switch (((p.s_lo - p.d_lo) & 15) >> 2) {
                case 0: realign_store_all<0, kThreads>(d, p, data_addr); break;
                case 1: realign_store_all<1, kThreads>(d, p, data_addr); break;
                case 2: realign_store_all<2, kThreads>(d, p, data_addr); break;
                default: realign_store_all<3, kThreads>(d, p, data_addr); break;
                }
            } else {
                if (!realign_pass_mixed<kThreads>(d, src + col0, dst + col0, row0 + r0, n_rows, len, data, bar, phase, wait_ok, wait_ok + 1)) return false;
                phase ^= 1;
            }
            __syncthreads();
        }
    }
    return true;
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

// A multi-plane tile (planes o .. o + n_units of descriptor d) on the realigning path: the rows
// of all its planes are staged in one pass - plane j in its own region of the staging area, one
// bulk copy per row - and stored plane by plane; planes may differ in alignment (a pointer per
// plane).  False: not applicable to this tile (rows of a few bytes, rows that differ in alignment,
// a staging area too small), the caller takes the narrow-vector loop; `alive` false: give up.
template <int kThreads, bool STEP, int NPTR>
__device__ __forceinline__ bool copy_multi_realign(const Desc &d, const Params<NPTR> &prm, uint32_t o, uint32_t n_units, char *stage,
                                                   uint32_t bar, uint32_t &phase, uint32_t *wait_ok, bool &alive)
{
    const uint32_t units = (d.run + 30) >> 4, plane_stage = d.rows * units * 16;
    if (d.run < kRealignMinRun || d.run > kRealignColumn || ((d.src_s0 | d.src_s1 | d.dst_s0 | d.dst_s1) & 15) || n_units * plane_stage + 32 > prm.stage_bytes)
        return false;
    const uint32_t data_addr = static_cast<uint32_t>(__cvta_generic_to_shared(stage + 16));
    // Planes a byte stride apart whose misaligned source is contiguous along i0 and whose
    // destination is aligned (a packed buffer at an odd offset unpacked into a pool): every column
    // of n0 rows of every plane arrives as one bulk copy and each plane's destination is walked
    // (see realign_tile_dest_order)
    if (!STEP && ((d.src_outer | d.dst_outer) & 15) == 0) {
        const uint32_t run = d.run, n0 = d.n0, cpr = run >> 4, rows = d.rows, cols = fastdiv(rows, d.div_n0);
        const char *src0 = prm.ptr[d.src_slot] + d.src_off + static_cast<long long>(o) * d.src_outer;
        char *dst0 = prm.ptr[d.dst_slot] + d.dst_off + static_cast<long long>(o) * d.dst_outer;
        const uint32_t s_lo = static_cast<uint32_t>(reinterpret_cast<uintptr_t>(src0)) & 15;
        const bool one_run = n0 == 1 || d.dst_s0 == cols * run;
        const uint32_t piece_stage = cols * (n0 * cpr + 1) * 16;
        if (s_lo && (reinterpret_cast<uintptr_t>(dst0) & 15) == 0 && d.src_s0 == run && (run & 15) == 0 && (cpr & (cpr - 1)) == 0 && run < kJoinMinRun &&
            d.dst_s1 == run && !(n0 > 1 && d.dst_s0 == run) && cols >= 2 && cols * n0 == rows && !(one_run && n0 > 1 && (cols & (cols - 1))) &&
            n_units * piece_stage + 32 <= prm.stage_bytes) {
            if (threadIdx.x == 0) mbar_expect_tx(bar, n_units * cols * (n0 * run + 16));
            for (uint32_t item = threadIdx.x; item < n_units * cols; item += kThreads) {
                const uint32_t j = item / cols, k1 = item - j * cols;
                bulk_load(data_addr + j * piece_stage + 16 * k1 * (n0 * cpr + 1), src0 - s_lo + static_cast<long long>(j) * d.src_outer + k1 * d.src_s1, n0 * run + 16, bar);
            }
            if (!realign_wait(bar, phase, wait_ok)) {
                alive = false;
                return true;
            }
            const uint32_t lcpr = 31 - __clz(cpr), groups = one_run ? 1 : n0, total = (one_run ? rows : cols) * cpr;
            const uint32_t pmask = one_run && n0 > 1 ? cols - 1 : 0xffffffffu, pshift = one_run && n0 > 1 ? 31 - __clz(cols) : 31;
            for (uint32_t j = 0; j < n_units; j++) {
                char *out0 = dst0 + static_cast<long long>(j) * d.dst_outer;
                const uint32_t at_j = data_addr + j * piece_stage;
                switch ((s_lo & 15) >> 2) {
                case 0: realign_store_dest_order<0, kThreads>(out0, d.dst_s0, groups, total, lcpr, pmask, pshift, n0, cpr, 1, s_lo, 0, at_j); break;
                case 1: realign_store_dest_order<1, kThreads>(out0, d.dst_s0, groups, total, lcpr, pmask, pshift, n0, cpr, 1, s_lo, 0, at_j); break;
                case 2: realign_store_dest_order<2, kThreads>(out0, d.dst_s0, groups, total, lcpr, pmask, pshift, n0, cpr, 1, s_lo, 0, at_j); break;
                default: realign_store_dest_order<3, kThreads>(out0, d.dst_s0, groups, total, lcpr, pmask, pshift, n0, cpr, 1, s_lo, 0, at_j); break;
                }
            }
            __syncthreads();
            return true;
        }
    }
    auto plane = [&](uint32_t j) {
        const uint32_t k = o + j;
        RealignPass p;
        p.src = prm.ptr[d.src_slot + (STEP ? k * d.src_slot_step : 0)] + d.src_off + k * d.src_outer;
        p.dst = prm.ptr[d.dst_slot + (STEP ? k * d.dst_slot_step : 0)] + d.dst_off + k * d.dst_outer;
        p.row_base = 0;
        p.n_rows = d.rows;
        p.units = units;
        p.len = d.run;
        p.s_lo = static_cast<uint32_t>(reinterpret_cast<uintptr_t>(p.src)) & 15;
        p.d_lo = static_cast<uint32_t>(reinterpret_cast<uintptr_t>(p.dst)) & 15;
        return p;
    };
    // per plane: where its destination starts (rounded down to 16), and whether every plane has
    // the alignment of plane 0 on both sides, so that one pass of the store loops can serve all
    __shared__ unsigned long long plane_dst[64];
    __shared__ uint32_t same_alignment;
    uint32_t *same = &same_alignment;
    if (threadIdx.x == 0) {
        uint32_t bytes = 0, ok = 1;
        const RealignPass p0 = plane(0);
        for (uint32_t j = 0; j < n_units; j++) {
            const RealignPass pj = plane(j);
            bytes += d.rows * realign_row_bytes(pj);
            plane_dst[j] = reinterpret_cast<unsigned long long>(pj.dst - pj.d_lo);
            ok &= pj.s_lo == p0.s_lo && pj.d_lo == p0.d_lo;
        }
        same_alignment = ok;
        mbar_expect_tx(bar, bytes);
    }
    if (d.rows >= kThreads) {
        for (uint32_t j = 0; j < n_units; j++) realign_load<kThreads, false>(d, plane(j), data_addr + j * plane_stage, bar);
    } else {  // few rows per plane: one thread per row of the tile, whatever its plane
        const uint32_t magic = d.rows > 1 ? 0xffffffffu / d.rows + 1 : 0;
        for (uint32_t rr = threadIdx.x; rr < n_units * d.rows; rr += kThreads) {
            const uint32_t j = d.rows > 1 ? __umulhi(rr, magic) : rr, r = rr - j * d.rows;
            const RealignPass pj = plane(j);
            const uint32_t i1 = fastdiv(r, d.div_n0), i0 = r - i1 * d.n0;
            bulk_load(data_addr + 16 * rr * units, pj.src - pj.s_lo + (i1 * d.src_s1 + i0 * d.src_s0), realign_row_bytes(pj), bar);
        }
    }
    if (!realign_wait(bar, phase, wait_ok)) {
        alive = false;
        return true;
    }
    // planes of short rows that follow one another in the destination, through a misaligned
    // destination: complete the slots and walk each plane's destination (realign_tile_dest_order)
    const uint32_t cpr = d.run >> 4, cols = fastdiv(d.rows, d.div_n0);
    const RealignPass first = plane(0);
    if (*same && first.d_lo && first.s_lo <= first.d_lo && (d.run & 15) == 0 && (cpr & (cpr - 1)) == 0 && d.run < kJoinMinRun && d.dst_s1 == d.run &&
        !(d.n0 > 1 && d.dst_s0 == d.run) && cols >= 2 && cols * d.n0 == d.rows) {
        const bool one_run = d.n0 == 1 || d.dst_s0 == cols * d.run;
        if (!(one_run && d.n0 > 1 && (cols & (cols - 1)))) {
            const uint32_t s_lo = first.s_lo, d_lo = first.d_lo, n0 = d.n0, rows = d.rows;
            const uint32_t magic = 0xffffffffu / rows + 1;  // rows >= 2
            for (uint32_t rr = threadIdx.x; rr < n_units * rows; rr += kThreads) {
                const uint32_t j = __umulhi(rr, magic), r = rr - j * rows;
                const uint32_t k1 = fastdiv(r, d.div_n0), i0 = r - k1 * n0;
                uint32_t next;
                if (k1 + 1 < cols) next = rr + n0;
                else if (one_run && i0 + 1 < n0) next = j * rows + i0 + 1;
                else continue;
                const uint32_t at = data_addr + 16 * (rr * units + cpr);
                uint4 v = lds128(data_addr + 16 * next * units);
                if (s_lo) v = merge_bytes(lds128(at), v, s_lo);
                asm volatile("st.shared.v4.u32 [%0], {%1, %2, %3, %4};" ::"r"(at), "r"(v.x), "r"(v.y), "r"(v.z), "r"(v.w) : "memory");
            }
            __syncthreads();
            const uint32_t lcpr = 31 - __clz(cpr), groups = one_run ? 1 : n0, total = (one_run ? rows : cols) * cpr;
            const uint32_t pmask = one_run && n0 > 1 ? cols - 1 : 0xffffffffu, pshift = one_run && n0 > 1 ? 31 - __clz(cols) : 31;
            for (uint32_t j = 0; j < n_units; j++) {
                char *out0 = reinterpret_cast<char *>(plane_dst[j]);
                const uint32_t at_j = data_addr + j * plane_stage;
                switch (((s_lo - d_lo) & 15) >> 2) {
                case 0: realign_store_dest_order<0, kThreads>(out0, d.dst_s0, groups, total, lcpr, pmask, pshift, n0, units, 0, s_lo, d_lo, at_j); break;
                case 1: realign_store_dest_order<1, kThreads>(out0, d.dst_s0, groups, total, lcpr, pmask, pshift, n0, units, 0, s_lo, d_lo, at_j); break;
                case 2: realign_store_dest_order<2, kThreads>(out0, d.dst_s0, groups, total, lcpr, pmask, pshift, n0, units, 0, s_lo, d_lo, at_j); break;
                default: realign_store_dest_order<3, kThreads>(out0, d.dst_s0, groups, total, lcpr, pmask, pshift, n0, units, 0, s_lo, d_lo, at_j); break;
                }
            }
            asm volatile("fence.proxy.async.shared::cta;" ::: "memory");  // ordinary stores into the slots, bulk copies next
            __syncthreads();
            return true;
        }
    }
    if (*same) {  // one pass of the store loops over the rows of all planes
        RealignPass all = plane(0);
        all.n_rows = n_units * d.rows;
        PlaneSet ps;
        ps.rows = d.rows;
        ps.magic = d.rows > 1 ? 0xffffffffu / d.rows + 1 : 0;
        ps.dst = plane_dst;
        realign_store_dispatch<kThreads, true>(d, all, data_addr, &ps);
    } else {
        for (uint32_t j = 0; j < n_units; j++) realign_store_dispatch<kThreads>(d, plane(j), data_addr + j * plane_stage);
    }
    __syncthreads();
    return true;
}

// The narrow-vector loops of a multi-plane tile, out of line like copy_rows_narrow.
template <int U, int kThreads, bool STEP, int NPTR>
__device__ __noinline__ void copy_multi_narrow(const Desc &d, const Params<NPTR> &prm, uint32_t o, uint32_t n_units, uint32_t align)
{
    switch (align) {
    case 3: copy_multi<3, U, kThreads, true, STEP>(d, prm, o, n_units); break;
    case 2: copy_multi<2, U, kThreads, true, STEP>(d, prm, o, n_units); break;
    case 1: copy_multi<1, U, kThreads, true, STEP>(d, prm, o, n_units); break;
    default: copy_multi<0, U, kThreads, true, STEP>(d, prm, o, n_units); break;
    }
}

// Debugging aid (TC_PLAN_DEBUG_BOUNDS): one thread per (descriptor, outer index) works out the
// first and last byte the descriptor touches on each side and holds them against the declared
// extent of the table slot (less `shrink`, for the self-test).  A violation sets a flag; nothing
// traps, nothing is dereferenced.
__global__ void tc_bounds_check_kernel(const Desc *descs, uint32_t n_descs, const long long *extents, long long shrink)
{
    const uint32_t i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= n_descs) return;
    const Desc d = descs[i];
    bool bad = d.n0 == 0 || d.rows == 0 || d.run == 0;
    if (!bad) {
        // strides are unsigned: the farthest row is the last one, or the last of the row before
        const uint32_t last = d.rows - 1, i1 = last / d.n0, i0 = last - i1 * d.n0;
        long long s_far = static_cast<long long>(i1) * d.src_s1 + static_cast<long long>(i0) * d.src_s0;
        long long d_far = static_cast<long long>(i1) * d.dst_s1 + static_cast<long long>(i0) * d.dst_s0;
        if (i1) {
            s_far = max(s_far, static_cast<long long>(i1 - 1) * d.src_s1 + static_cast<long long>(d.n0 - 1) * d.src_s0);
            d_far = max(d_far, static_cast<long long>(i1 - 1) * d.dst_s1 + static_cast<long long>(d.n0 - 1) * d.dst_s0);
        }
        for (uint32_t o = 0; o < d.n_outer && !bad; o++) {
            const long long s_lo = d.src_off + static_cast<long long>(o) * d.src_outer, d_lo = d.dst_off + static_cast<long long>(o) * d.dst_outer;
            const long long s_ext = extents[d.src_slot + o * d.src_slot_step] - shrink, d_ext = extents[d.dst_slot + o * d.dst_slot_step] - shrink;
            bad = s_lo < 0 || d_lo < 0 || s_lo + s_far + d.run > s_ext || d_lo + d_far + d.run > d_ext;
        }
    }
    if (bad) atomicOr(&g_device_status, kStatusOutOfBounds);
}

// MULTI: 0 one plane per tile; 1 several planes per tile, planes a byte stride apart; 2 the
// same with a pool that has one pointer per plane.
template <int NPTR, int MODE, bool CHECK = false, int MULTI = 0>
__global__ void __launch_bounds__(Shape<MODE>::threads, Shape<MODE>::min_ctas) tc_copy_kernel(const __grid_constant__ Params<NPTR> prm)
{
    constexpr int kThreads = Shape<MODE>::threads, kUnroll = Shape<MODE>::unroll;
    __shared__ Desc sdesc[2];
    extern __shared__ __align__(16) char stage[];  // the realigning path's staging area (kModeAny only)
    __shared__ __align__(8) unsigned long long stage_bar;  // its mbarrier
    __shared__ uint32_t stage_ok[2];  // [0] the bulk copies arrived, [1] byte counter of the mixed-alignment path
    uint32_t bar = 0, phase = 0;
    if (MODE == kModeAny) {
        bar = static_cast<uint32_t>(__cvta_generic_to_shared(&stage_bar));
        if (threadIdx.x == 0) {
            mbar_init(bar, 1);
            stage_ok[0] = 1;
            asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        }
        // made visible to the CTA by the __syncthreads that follows the descriptor fetch below
    }
    // a debug-checked plan whose checker has raised its flag copies nothing
    if (prm.debug_bounds && (*static_cast<volatile unsigned int *>(&g_device_status) & kStatusOutOfBounds)) return;
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
                const uint32_t align = min(static_cast<uint32_t>(d.log2_align), prm.log2_ptr_align);
                bool alive = true;
                if (align == 4) copy_multi<4, kUnroll, kThreads, true, MULTI == 2>(d, prm, o, n_units);
                else if (!copy_multi_realign<kThreads, MULTI == 2>(d, prm, o, n_units, stage, bar, phase, stage_ok, alive))
                    copy_multi_narrow<2 * kUnroll, kThreads, MULTI == 2>(d, prm, o, n_units, align);
                if (!alive) return;
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
            const uint32_t align = min(static_cast<uint32_t>(d.log2_align), prm.log2_ptr_align);
            if (align == 4 && (!prm.stage_always || d.run < kRealignMinRun)) {
                copy_rows<4, kUnroll, kThreads>(d, src, dst, row0, nrows);
            } else if (d.run >= kRealignMinRun) {
                if (!copy_rows_realign<kThreads>(d, src, dst, row0, nrows, stage, prm.stage_bytes, bar, phase, stage_ok)) return;
            } else {
                copy_rows_narrow<kUnroll, kThreads>(d, src, dst, row0, nrows, align);
            }
        }
    }
}

}  // namespace tc
