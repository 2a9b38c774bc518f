// Internal plan representation shared by the host-side plan builder and the kernels.
// Nothing here is part of the public ABI (see include/tensorcast.h).
#pragma once

#include <cstdint>
#include <string>
#include <vector>

#include "tensorcast.h"

namespace tc {

// Exact unsigned division by a runtime constant for dividends below 2^31:
//   n / d == (umulhi(n, mul) + n) >> shift
struct FastDiv {
    uint32_t mul, shift;
};

inline FastDiv make_fastdiv(uint32_t d)
{
    uint32_t s = 0;
    while ((1ull << s) < d) s++;
    uint64_t m = ((1ull << 32) * ((1ull << s) - d)) / d + 1;
    return FastDiv{static_cast<uint32_t>(m), s};
}

inline uint32_t fastdiv_host(uint32_t n, FastDiv f)
{
    return static_cast<uint32_t>((((static_cast<uint64_t>(n) * f.mul) >> 32) + n) >> f.shift);
}

// One lowered copy descriptor as the kernels read it (128 bytes, 16-byte aligned).
// A box of n_outer x rows runs of `run` contiguous bytes; row k of outer index o starts at
//   table[src_slot + o*src_slot_step] + src_off + o*src_outer + (k / n0)*src_s1 + (k % n0)*src_s0
// and likewise for dst (dst_slot already includes the offset of the dst table inside the
// combined pointer table).  The builder guarantees that the row offsets of one descriptor,
// (k / n0)*s1 + (k % n0)*s0 + run, stay below 2^31 on both sides, so the kernels decode rows in
// 32-bit arithmetic.  Tiles: outer index o, row range [p*rows_per_tile, ...).
struct alignas(16) Desc {
    int64_t src_off, dst_off, src_outer, dst_outer;
    uint32_t src_s0, src_s1, dst_s0, dst_s1;
    uint16_t src_slot, dst_slot, src_slot_step, dst_slot_step;
    FastDiv div_run;  // byte index inside a tile -> row
    uint32_t run, n0, rows, n_outer;
    uint32_t rows_per_tile, tiles_per_outer, tile0;
    uint16_t log2_align;
    uint16_t units_shift; // with units_mul: FastDiv by the 16-byte units per row of the realigning
                          // path, (min(run, kRealignColumn) + 30) / 16 (see copy_kernel.cuh)
    FastDiv div_n0, div_tpo;
    uint32_t tag;        // checksummed plans: which accumulator (tensor index) this box feeds
    uint32_t units_mul;
    int64_t csum_base;   // checksummed plans: src byte offset of the tensor's first byte
};
static_assert(sizeof(Desc) == 128, "Desc must stay 128 bytes");

// A launch window: descriptors [d0, d0+nd) x planes [o0, o0+no), walked plane-major.
// A segment of a staged plan is a window whose packed-side bytes are one contiguous range.
struct Segment {
    uint32_t d0, nd, o0, no; // window of descriptors x planes; nd == 0: a range of global tile
                             // ids instead, [d0, d0 + no) (non-uniform groups, e.g. weights)
    int64_t shift;           // the kernel sees the staging buffer at (buffer - shift)
    uint32_t copy0, ncopy;   // its copies between host memory and the staging buffer
};

// One copy-engine transfer of a staged plan.
struct StageCopy {
    int64_t stage_off, host_off, bytes;
};

// Bookkeeping of one request while a KV group is lowered (staged plans cut segments from it).
struct RequestSpan {
    uint32_t d0, d1;      // its descriptors
    int64_t off, plane_bytes;
};

struct Group {
    std::vector<Desc> descs;
    std::vector<uint32_t> tile_desc;  // tile -> descriptor, only for non-uniform groups
    std::vector<RequestSpan> requests; // KV groups with a packed side
    std::vector<Segment> segments;    // staged plans only
    std::vector<StageCopy> copies;    // staged plans only
    std::vector<int64_t> extents;     // TC_PLAN_DEBUG_BOUNDS: byte extent of every table slot (src slots, then dst slots)
    bool stage_whole_host_pool = false; // staged MIXED group: the host side is a paged pool
    bool host_is_src = false;          // staged groups: direction (host -> device when true)
    uint32_t tiles_per_desc = 0;      // > 0: every descriptor owns exactly this many tile ids
    // Planes per tile.  When one plane of a block is much smaller than a tile (few KV heads:
    // 4-16 KiB), a tile takes ppt consecutive planes of its descriptor, each padded to
    // 2^log2_unit bytes of the tile's byte space.  1: a tile is (part of) one plane.
    uint32_t ppt = 1, log2_unit = 0;
    FastDiv div_tpd{0, 0};
    uint64_t n_tiles = 0;
    int64_t payload = 0;
    uint32_t log2_align = 4;
    uint32_t realign_smem = 0;        // staging bytes one CTA of the realigning path needs for this group's largest tile
    size_t n_src = 0, n_dst = 0;      // table lengths the execute call must be given
    bool single_run_tiles = true;     // every tile is one contiguous run
    int resident_ctas[3] = {0, 0, 0}; // CTAs one SM holds, per executor build
    // device copies (null for host-only plans and empty groups)
    Desc *d_descs = nullptr;
    uint32_t *d_tile_desc = nullptr;
    int64_t *d_extents = nullptr;
};

}  // namespace tc

struct tc_plan {
    int32_t kind = 0;
    uint32_t flags = 0;
    uint64_t trace_id = 0;
    int64_t deadline_ns = 0;
    tc_tuning_t tuning{};
    int device = -1;
    int sm_count = 0;
    int64_t packed_required = 0;
    int64_t device_bytes = 0;
    void *d_storage = nullptr;  // one device block holding both groups' descriptors and tiles
    size_t d_storage_bytes = 0;
    bool checksummed = false;  // built with TC_PLAN_CHECKSUM
    int64_t n_sums = 0;        // accumulators a checksummed execution fills
    bool staged = false;  // holds a reference on the device's staging ring
    void *trace_ev[2][2] = {{nullptr, nullptr}, {nullptr, nullptr}};  // TC_PLAN_TRACE: cudaEvent_t begin / end per group
    mutable bool traced_once[2] = {false, false};
    tc::Group group[2];
};

namespace tc {

// plan_build.cpp: validate `spec` and lower it into plan->group[*] (host vectors only).
int build_plan(const tc_plan_spec_t *spec, tc_plan *plan);

// error reporting shared by both translation units
int fail(int status, const char *fmt, ...);
void clear_error();
int64_t now_ns();

constexpr uint32_t kDefaultTileBytes = 32768;
constexpr int64_t kStageBytes = 64ll << 20;  // one staging buffer
constexpr int kStageBuffers = 3;
constexpr uint32_t kMaxTileBytes = 1u << 20;
// Realigning path (misaligned geometry or pointers): shared memory one CTA stages a tile's rows
// in, and the longest piece of a row it stages in one pass.
constexpr uint32_t kRealignSmem = 52u << 10;
constexpr uint32_t kRealignColumn = kRealignSmem - 64;
constexpr uint32_t kRealignMinRun = 32;  // shorter rows take the narrow-vector loop instead
constexpr uint32_t kJoinMinRun = 1024;   // rows at least this long are staged back to back where the destination has them so

}  // namespace tc
