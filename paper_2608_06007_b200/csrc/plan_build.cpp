// Host-side plan builder: validates a tc_plan_spec_t and lowers it to copy descriptors and
// tiles.  Pure host code (no CUDA call), so it can be exercised on a machine without a GPU.
//
// Lowering model.  Every operation of the library (publish, hydrate, migrate, tensor_dict,
// view, transform_into; Table 2 of the paper) is a set of strided boxes of bytes.  A box is
// given as a contiguous run plus a list of (extent, src stride, dst stride) dimensions; it is
// normalised (unit dims dropped, contiguous dims folded into the run, adjacent dims merged,
// over-long runs cut into tile-sized rows) and emitted as one or more Desc records with at
// most two strided dimensions, which is what the kernels decode.
#include <algorithm>
#include <cstdarg>
#include <cstdio>
#include <cstring>
#include <ctime>
#include <numeric>

#include "plan.h"

namespace tc {

// ------------------------------------------------------------------------------ errors
static thread_local std::string g_error;

int fail(int status, const char *fmt, ...)
{
    char buf[512];
    va_list ap;
    va_start(ap, fmt);
    vsnprintf(buf, sizeof buf, fmt, ap);
    va_end(ap);
    g_error = buf;
    return status;
}

void clear_error() { g_error.clear(); }

int64_t now_ns()
{
    timespec ts;
    clock_gettime(CLOCK_MONOTONIC, &ts);
    return static_cast<int64_t>(ts.tv_sec) * 1000000000ll + ts.tv_nsec;
}

const char *last_error() { return g_error.c_str(); }

// ------------------------------------------------------------------------------ boxes
struct Dim {
    int64_t ext, s, d;  // extent, source byte stride, destination byte stride
};

struct Box {
    int64_t run;              // contiguous bytes of the innermost run
    std::vector<Dim> dims;    // any order
    int64_t src_off, dst_off;
    uint32_t src_slot, dst_slot;
    // the table-stepping outer dimension (KV planes); n_outer == 1 when unused
    uint32_t n_outer = 1, src_slot_step = 0, dst_slot_step = 0;
    int64_t src_outer = 0, dst_outer = 0;
    uint32_t tag = 0;         // checksum accumulator
    int64_t csum_base = 0;    // source offset that checksum positions are relative to
};

static uint32_t ctz_cap(int64_t v, uint32_t cap = 4)
{
    if (v == 0) return cap;
    uint64_t u = static_cast<uint64_t>(v < 0 ? -v : v);
    uint32_t n = 0;
    while (n < cap && !(u & 1)) { u >>= 1; n++; }
    return n;
}

static void emit_desc(Group &g, const Box &b, int64_t run, const Dim *inner, const Dim *outer,
                      int64_t src_off, int64_t dst_off, uint32_t tile_bytes)
{
    Desc d{};
    d.src_off = src_off;
    d.dst_off = dst_off;
    d.src_outer = b.src_outer;
    d.dst_outer = b.dst_outer;
    d.n0 = inner ? static_cast<uint32_t>(inner->ext) : 1;
    d.src_s0 = inner ? static_cast<uint32_t>(inner->s) : 0;
    d.dst_s0 = inner ? static_cast<uint32_t>(inner->d) : 0;
    uint32_t n1 = outer ? static_cast<uint32_t>(outer->ext) : 1;
    d.src_s1 = outer ? static_cast<uint32_t>(outer->s) : 0;
    d.dst_s1 = outer ? static_cast<uint32_t>(outer->d) : 0;
    d.rows = d.n0 * n1;
    d.src_slot = static_cast<uint16_t>(b.src_slot);
    d.dst_slot = static_cast<uint16_t>(b.dst_slot);
    d.src_slot_step = static_cast<uint16_t>(b.src_slot_step);
    d.dst_slot_step = static_cast<uint16_t>(b.dst_slot_step);
    d.run = static_cast<uint32_t>(run);
    d.n_outer = b.n_outer;
    // Parts per outer index.  Normally the fewest parts that each fit tile_bytes (one pass of
    // the CTA), rows spread evenly.  When that would leave the parts small on average - 36 or
    // 40 KiB of rows would become two parts of 18 or 20 KiB - the nearest count is taken instead
    // and a part may reach 1.5 x tile_bytes: one tile of 36 KiB measured 6 % faster than two.
    const uint64_t bytes = static_cast<uint64_t>(d.rows) * d.run;
    const uint32_t fit = std::max<uint32_t>(1, tile_bytes / d.run);  // rows that fit one pass
    uint32_t parts = (d.rows + fit - 1) / fit;
    if (bytes * 4 < static_cast<uint64_t>(parts) * tile_bytes * 3)
        parts = static_cast<uint32_t>(std::min<uint64_t>(d.rows, std::max<uint64_t>(1, (bytes + tile_bytes / 2) / tile_bytes)));
    d.rows_per_tile = (d.rows + parts - 1) / parts;
    d.tiles_per_outer = (d.rows + d.rows_per_tile - 1) / d.rows_per_tile;
    d.div_run = make_fastdiv(d.run);
    d.div_n0 = make_fastdiv(d.n0);
    d.div_tpo = make_fastdiv(d.tiles_per_outer);
    uint32_t a = std::min({ctz_cap(run), ctz_cap(src_off), ctz_cap(dst_off)});
    if (d.n0 > 1) a = std::min({a, ctz_cap(d.src_s0), ctz_cap(d.dst_s0)});
    if (n1 > 1) a = std::min({a, ctz_cap(d.src_s1), ctz_cap(d.dst_s1)});
    if (d.n_outer > 1) a = std::min({a, ctz_cap(d.src_outer), ctz_cap(d.dst_outer)});
    d.log2_align = static_cast<uint16_t>(a);
    const FastDiv units = make_fastdiv((std::min<uint32_t>(d.run, kRealignColumn) + 30) >> 4);
    d.units_mul = units.mul;
    d.units_shift = static_cast<uint16_t>(units.shift);
    d.tag = b.tag;
    d.csum_base = b.csum_base;
    g.log2_align = std::min(g.log2_align, a);
    if (d.rows_per_tile > 1) g.single_run_tiles = false;
    g.payload += static_cast<int64_t>(d.run) * d.rows * d.n_outer;
    g.descs.push_back(d);
}

// Normalise a box and append its descriptors to the group.
static void lower_box(Group &g, Box b, uint32_t tile_bytes)
{
    if (b.run <= 0 || b.n_outer == 0) return;
    for (const Dim &d : b.dims)
        if (d.ext <= 0) return;  // empty box
    // 1. drop unit dims
    b.dims.erase(std::remove_if(b.dims.begin(), b.dims.end(), [](const Dim &d) { return d.ext == 1; }),
                 b.dims.end());
    // 2. fold dims that continue the run on both sides into the run
    for (bool again = true; again;) {
        again = false;
        for (size_t i = 0; i < b.dims.size(); i++)
            if (b.dims[i].s == b.run && b.dims[i].d == b.run) {
                b.run *= b.dims[i].ext;
                b.dims.erase(b.dims.begin() + i);
                again = true;
                break;
            }
    }
    // 3. merge pairs of dims that are one dimension in disguise on both sides
    for (bool again = true; again;) {
        again = false;
        for (size_t i = 0; i < b.dims.size() && !again; i++)
            for (size_t j = 0; j < b.dims.size() && !again; j++)
                if (i != j && b.dims[j].s == b.dims[i].s * b.dims[i].ext &&
                    b.dims[j].d == b.dims[i].d * b.dims[i].ext) {
                    b.dims[i].ext *= b.dims[j].ext;
                    b.dims.erase(b.dims.begin() + j);
                    again = true;
                }
    }
    // 4. a run much longer than a tile becomes rows of about tile_bytes plus a remainder box.
    //    Runs of up to 1.5 tiles stay whole (see emit_desc); multiples of tile_bytes are cut
    //    exactly; anything else into the fewest equal pieces that fit a tile (512-byte granules).
    if (b.run > static_cast<int64_t>(tile_bytes) * 3 / 2) {
        int64_t piece = tile_bytes;
        if (b.run % tile_bytes) {
            const int64_t n = (b.run + tile_bytes - 1) / tile_bytes;
            piece = ((b.run + n - 1) / n + 511) & ~int64_t(511);  // <= tile_bytes, a multiple of 512
        }
        int64_t full = b.run / piece, rem = b.run % piece;
        if (rem) {
            Box tail = b;
            tail.run = rem;
            tail.src_off += full * piece;
            tail.dst_off += full * piece;
            lower_box(g, tail, tile_bytes);
        }
        b.run = piece;
        b.dims.push_back(Dim{full, piece, piece});
        b.dims.erase(std::remove_if(b.dims.begin(), b.dims.end(), [](const Dim &d) { return d.ext == 1; }),
                     b.dims.end());
    }
    // 5. innermost = smallest source stride, so that a tile reads as densely as it can (its
    //    writes all land in L2 within microseconds and merge there; measured 1-1.5 % faster for
    //    the layout transforms than walking the rows in destination order)
    std::sort(b.dims.begin(), b.dims.end(), [](const Dim &x, const Dim &y) {
        return std::llabs(x.s) != std::llabs(y.s) ? std::llabs(x.s) < std::llabs(y.s) : std::llabs(x.d) < std::llabs(y.d);
    });
    // 6. one descriptor addresses its rows with 32-bit offsets: cut every dimension so that
    //    its own span stays below 2^30 bytes (and its extent below 2^20 rows)
    for (size_t i = 0; i < b.dims.size(); i++) {
        const int64_t stride = std::max<int64_t>(std::max(b.dims[i].s, b.dims[i].d), 1);
        const int64_t cap = std::max<int64_t>(1, std::min<int64_t>(1 << 20, ((1ll << 30) - b.run) / stride));
        if (b.dims[i].ext <= cap || cap <= 1) continue;
        // ext = q*cap + r: the r-tail becomes its own box, q*cap becomes two dims (cap, q)
        const int64_t q = b.dims[i].ext / cap, r = b.dims[i].ext % cap;
        if (r) {
            Box tail = b;
            tail.dims[i].ext = r;
            tail.src_off += q * cap * b.dims[i].s;
            tail.dst_off += q * cap * b.dims[i].d;
            lower_box(g, tail, tile_bytes);
        }
        Dim hi{q, b.dims[i].s * cap, b.dims[i].d * cap};
        b.dims[i].ext = cap;
        b.dims.push_back(hi);  // strides of 2^30 or more: always unrolled on the host below
    }
    // 7. at most two strided dims per descriptor, each of span < 2^30; the rest is unrolled here
    auto span = [](const Dim &d) { return (d.ext - 1) * std::max(d.s, d.d); };
    const int64_t span_cap = (1ll << 30) - b.run;
    std::stable_partition(b.dims.begin(), b.dims.end(), [&](const Dim &d) { return span(d) < span_cap && d.ext <= (1 << 20); });
    size_t keep = 0;
    while (keep < 2 && keep < b.dims.size() && span(b.dims[keep]) < span_cap && b.dims[keep].ext <= (1 << 20)) keep++;
    if (keep == 2 && b.dims[0].ext * b.dims[1].ext >= (1ll << 31)) keep = 1;
    std::vector<int64_t> idx(b.dims.size(), 0);
    for (;;) {
        int64_t so = b.src_off, dof = b.dst_off;
        for (size_t i = keep; i < b.dims.size(); i++) {
            so += idx[i] * b.dims[i].s;
            dof += idx[i] * b.dims[i].d;
        }
        emit_desc(g, b, b.run, keep >= 1 ? &b.dims[0] : nullptr, keep >= 2 ? &b.dims[1] : nullptr, so, dof,
                  tile_bytes);
        size_t i = keep;
        for (; i < b.dims.size(); i++) {
            if (++idx[i] < b.dims[i].ext) break;
            idx[i] = 0;
        }
        if (i >= b.dims.size()) break;
    }
}

// Assign tile ids.  A group whose descriptors all own (nearly) the same number of tiles is
// "uniform": tile -> descriptor is a division and short descriptors simply own a few empty
// tile ids.  Otherwise an explicit tile -> descriptor array is built.
static int finish_group(Group &g, uint32_t tile_bytes)
{
    if (g.descs.empty()) return TC_OK;
    // Small planes: let a tile span several planes of its descriptor (see Group::ppt).  Needs one
    // part per plane and a pointer table of at most 400 entries (the kernel classes built for it).
    g.ppt = 1;
    g.log2_unit = 0;
    {
        bool can = g.n_src + g.n_dst <= 400;
        uint32_t max_unit = 0, min_outer = ~0u;
        for (const Desc &d : g.descs) {
            if (d.n_outer < 2 || d.tiles_per_outer != 1) can = false;
            max_unit = std::max(max_unit, d.rows * d.run);
            min_outer = std::min(min_outer, d.n_outer);
        }
        if (can && 2ull * max_unit <= tile_bytes) {
            uint32_t lg = 9;  // units of at least 512 bytes
            while ((1u << lg) < max_unit) lg++;
            const uint32_t ppt = std::min({tile_bytes >> lg, min_outer, 64u});
            if (ppt > 1) {
                g.ppt = ppt;
                g.log2_unit = lg;
            }
        }
    }
    // Realigning path: one pass should hold a whole tile (every row in a slot of `units` 16-byte
    // chunks, all planes of a multi-plane tile, 32 bytes of padding), up to the size at which long
    // rows go in column pieces.
    auto realign_need = [&](uint32_t ppt) {
        uint64_t most = 0;
        for (const Desc &d : g.descs) {
            const uint64_t units = (std::min<uint32_t>(d.run, kRealignColumn) + 30) >> 4;
            const uint64_t rows = std::min<uint64_t>(d.rows_per_tile, d.rows);
            most = std::max<uint64_t>(most, rows * units * 16 * ppt + 32);
            // short rows a step of n0 apart in the destination: room for one more chunk per slot
            if (ppt == 1 && (d.run & 15) == 0 && d.run < kJoinMinRun && d.dst_s1 == d.run)
                most = std::max<uint64_t>(most, rows * (units + 1) * 16 + 32);
            // rows adjacent in the destination are staged back to back, one group per destination
            // run (16 bytes of slack each), plus one 16-byte side chunk per row
            if (ppt == 1 && (d.run & 15) == 0 && d.run >= kJoinMinRun && d.run <= kRealignColumn && (d.dst_s1 == d.run || d.dst_s0 == d.run))
                most = std::max<uint64_t>(most, rows * d.run + 16 * std::min<uint64_t>(d.n0, rows) + 16 * (rows + 1) + 64);
        }
        return static_cast<uint32_t>(std::min<uint64_t>(most, kRealignSmem));
    };
    g.realign_smem = realign_need(g.ppt);
    auto outer_groups = [&](const Desc &d) { return (d.n_outer + g.ppt - 1) / g.ppt; };
    uint64_t total = 0, max_t = 0;
    for (const Desc &d : g.descs) {
        uint64_t t = static_cast<uint64_t>(outer_groups(d)) * d.tiles_per_outer;
        total += t;
        max_t = std::max(max_t, t);
    }
    uint64_t padded = max_t * g.descs.size();
    bool same_shape = true;
    for (const Desc &d : g.descs)
        if (d.n_outer != g.descs[0].n_outer) same_shape = false;
    if (same_shape && padded < (1ull << 31) && total * 10 >= padded * 8) {
        // uniform: every descriptor is given max tiles_per_outer; extra parts are empty
        uint32_t tpo = static_cast<uint32_t>(max_t / outer_groups(g.descs[0]));
        for (size_t i = 0; i < g.descs.size(); i++) {
            Desc &d = g.descs[i];
            d.tiles_per_outer = tpo;
            d.div_tpo = make_fastdiv(tpo);
            d.tile0 = static_cast<uint32_t>(i * max_t);
        }
        g.tiles_per_desc = static_cast<uint32_t>(max_t);
        g.div_tpd = make_fastdiv(g.tiles_per_desc);
        g.n_tiles = padded;
        return TC_OK;
    }
    g.ppt = 1;  // listed groups keep one plane per tile
    g.log2_unit = 0;
    g.realign_smem = realign_need(1);
    total = 0;
    for (const Desc &d : g.descs) total += static_cast<uint64_t>(d.n_outer) * d.tiles_per_outer;
    if (total >= (1ull << 31)) return fail(TC_ERR_INVALID_ARG, "plan has %llu tiles (limit 2^31)", (unsigned long long)total);
    g.tile_desc.resize(total);
    uint64_t t0 = 0;
    for (size_t i = 0; i < g.descs.size(); i++) {
        Desc &d = g.descs[i];
        uint64_t t = static_cast<uint64_t>(d.n_outer) * d.tiles_per_outer;
        d.tile0 = static_cast<uint32_t>(t0);
        std::fill(g.tile_desc.begin() + t0, g.tile_desc.begin() + t0 + t, static_cast<uint32_t>(i));
        t0 += t;
    }
    g.tiles_per_desc = 0;
    g.n_tiles = total;
    return TC_OK;
}

// ------------------------------------------------------------------------------ KV
struct PoolView {
    const tc_kv_pool_t *p;
    int64_t chunk;         // B*H*D*E
    int64_t block_stride;  // resolved
    int64_t plane_stride;  // 0 when the pool has L*2 slots
    uint32_t slot_step;    // 1 when the pool has L*2 slots
    int64_t slot_need;     // minimum extent of a slot
};

static int check_pool(const tc_kv_spec_t &kv, const tc_kv_pool_t &p, const char *name, PoolView *out)
{
    const int64_t planes = kv.L * 2, chunk = kv.B * kv.H * kv.D * kv.E;
    if (p.layout != TC_NHD && p.layout != TC_HND) return fail(TC_ERR_INVALID_ARG, "%s.layout %d is not a tc_layout", name, p.layout);
    if (p.num_blocks < 0) return fail(TC_ERR_SHAPE, "%s.num_blocks %lld < 0", name, (long long)p.num_blocks);
    if (p.n_slots != 1 && p.n_slots != planes)
        return fail(TC_ERR_INVALID_ARG, "%s.n_slots %lld must be 1 or L*2 = %lld", name, (long long)p.n_slots, (long long)planes);
    int64_t bs = p.block_stride ? p.block_stride : chunk;
    if (bs < chunk) return fail(TC_ERR_OVERLAP, "%s.block_stride %lld < block bytes %lld: blocks overlap", name, (long long)bs, (long long)chunk);
    out->p = &p;
    out->chunk = chunk;
    out->block_stride = bs;
    const int64_t nb = std::max<int64_t>(p.num_blocks, 1);
    if (p.n_slots == 1) {
        int64_t ps = p.plane_stride;
        // plane-major (each plane holds all its blocks) or page-first (each block holds all planes)
        bool plane_major = ps >= (nb - 1) * bs + chunk;
        bool page_first = ps >= chunk && bs >= (planes - 1) * ps + chunk;
        if (planes > 1 && !plane_major && !page_first)
            return fail(TC_ERR_OVERLAP, "%s: plane_stride %lld and block_stride %lld make planes overlap", name, (long long)ps, (long long)bs);
        out->plane_stride = planes > 1 ? ps : 0;
        out->slot_step = 0;
        out->slot_need = (planes - 1) * out->plane_stride + (nb - 1) * bs + chunk;
    } else {
        out->plane_stride = 0;
        out->slot_step = 1;
        out->slot_need = (nb - 1) * bs + chunk;
    }
    if (p.slot_bytes && p.slot_bytes < out->slot_need && p.num_blocks > 0)
        return fail(TC_ERR_BOUNDS, "%s.slot_bytes %lld < %lld needed for %lld blocks", name, (long long)p.slot_bytes, (long long)out->slot_need, (long long)p.num_blocks);
    return TC_OK;
}

static int check_group(const tc_kv_spec_t &kv, const tc_kv_group_t &g, const char *name, bool need_src,
                       const tc_kv_pool_t *src_pool, bool need_dst, const tc_kv_pool_t *dst_pool)
{
    if (g.R < 0) return fail(TC_ERR_SHAPE, "%s.R %lld < 0", name, (long long)g.R);
    if (g.R == 0) return TC_OK;
    if (!g.T || !g.bt_off) return fail(TC_ERR_INVALID_ARG, "%s: T and bt_off are required when R > 0", name);
    if (g.bt_off[0] != 0) return fail(TC_ERR_INVALID_ARG, "%s.bt_off[0] must be 0", name);
    for (int64_t r = 0; r < g.R; r++) {
        if (g.T[r] < 0) return fail(TC_ERR_SHAPE, "%s.T[%lld] = %lld < 0", name, (long long)r, (long long)g.T[r]);
        int64_t n = (g.T[r] + kv.B - 1) / kv.B;
        if (g.bt_off[r + 1] - g.bt_off[r] != n)
            return fail(TC_ERR_INVALID_ARG, "%s: request %lld has %lld tokens = %lld blocks but its table holds %lld", name,
                        (long long)r, (long long)g.T[r], (long long)n, (long long)(g.bt_off[r + 1] - g.bt_off[r]));
    }
    const int64_t nblk = g.bt_off[g.R];
    if (nblk > 0 && need_src && !g.bt_src) return fail(TC_ERR_INVALID_ARG, "%s.bt_src is required", name);
    if (nblk > 0 && need_dst && !g.bt_dst) return fail(TC_ERR_INVALID_ARG, "%s.bt_dst is required", name);
    if (need_src)
        for (int64_t j = 0; j < nblk; j++)
            if (g.bt_src[j] < 0 || g.bt_src[j] >= src_pool->num_blocks)
                return fail(TC_ERR_BOUNDS, "%s.bt_src[%lld] = %d outside [0, %lld)", name, (long long)j, g.bt_src[j], (long long)src_pool->num_blocks);
    if (need_dst) {
        std::vector<uint8_t> seen(static_cast<size_t>(dst_pool->num_blocks), 0);
        for (int64_t j = 0; j < nblk; j++) {
            int32_t b = g.bt_dst[j];
            if (b < 0 || b >= dst_pool->num_blocks)
                return fail(TC_ERR_BOUNDS, "%s.bt_dst[%lld] = %d outside [0, %lld)", name, (long long)j, b, (long long)dst_pool->num_blocks);
            if (seen[b]) return fail(TC_ERR_OVERLAP, "%s.bt_dst names block %d twice: its bytes would be written twice", name, b);
            seen[b] = 1;
        }
    }
    return TC_OK;
}

// strides of (slot n, head h) rows of D*E bytes inside one block / one packed request plane
static void pool_strides(const tc_kv_spec_t &kv, int32_t layout, int64_t *sn, int64_t *sh)
{
    const int64_t row = kv.D * kv.E;
    if (layout == TC_NHD) { *sn = kv.H * row; *sh = row; }
    else                  { *sn = row;        *sh = kv.B * row; }
}

// same for the packed buffer, which holds hs heads of a request of Tr tokens
static void packed_strides(const tc_kv_spec_t &kv, int32_t layout, int64_t Tr, int64_t hs, int64_t *sn, int64_t *sh)
{
    const int64_t row = kv.D * kv.E;
    if (layout == TC_NHD) { *sn = hs * row; *sh = row; }
    else                  { *sn = row;      *sh = Tr * row; }
}

static int64_t planes_of(const tc_kv_spec_t &kv) { return kv.L * 2; }

// Staged MIXED group: descriptor k (one per block, in table order) uses ring slot k % slots;
// a segment is the run of descriptors that fills one staging buffer.
static void stage_pages(Group &g, const int32_t *host_blocks, int64_t n_blocks, int64_t slots, int64_t page, int64_t host_block_stride)
{
    if (static_cast<int64_t>(g.descs.size()) != n_blocks) {  // a block lowered to several descriptors: stay zero copy
        g.stage_whole_host_pool = false;
        return;
    }
    for (int64_t k0 = 0; k0 < n_blocks; k0 += slots) {
        const int64_t n = std::min(slots, n_blocks - k0);
        g.segments.push_back(Segment{static_cast<uint32_t>(k0), static_cast<uint32_t>(n), 0, static_cast<uint32_t>(g.descs[0].n_outer), 0,
                                     static_cast<uint32_t>(g.copies.size()), static_cast<uint32_t>(n)});
        for (int64_t k = k0; k < k0 + n; k++) g.copies.push_back(StageCopy{(k - k0) * page, host_blocks[k] * host_block_stride, page});
    }
}

// Lower one group.  src_pool / dst_pool null = that side is the packed buffer.
static void lower_kv_group(Group &g, const tc_kv_spec_t &kv, const tc_kv_group_t &grp, const PoolView *src_pool,
                           const PoolView *dst_pool, int32_t packed_layout, uint32_t tile_bytes)
{
    const int64_t row = kv.D * kv.E, planes = kv.L * 2;
    const bool has_packed = !src_pool || !dst_pool;
    // the packed side may hold a head slice and may be ordered layer-major
    const int64_t h0 = has_packed ? kv.head_begin : 0;
    const int64_t hs = has_packed && kv.head_count ? kv.head_count : kv.H - h0;
    const bool layer_major = has_packed && kv.packed_order == TC_LAYER_MAJOR;
    int64_t total_tokens = 0;
    for (int64_t r = 0; r < grp.R; r++) total_tokens += grp.T[r];
    int64_t off_r = 0;
    g.descs.reserve(grp.R ? static_cast<size_t>(grp.bt_off[grp.R]) : 0);
    for (int64_t r = 0; r < grp.R; r++) {
        const int64_t Tr = grp.T[r];
        const int64_t plane_bytes = Tr * hs * row;  // one (l,c) plane of this request, packed
        const int64_t packed_outer = layer_major ? total_tokens * hs * row : plane_bytes;
        const uint32_t first_desc = static_cast<uint32_t>(g.descs.size());
        for (int64_t j = 0; j * kv.B < Tr; j++) {
            const int64_t nvalid = std::min(kv.B, Tr - j * kv.B);
            const int64_t jj = grp.bt_off[r] + j;
            Box b;
            b.run = row;
            b.n_outer = static_cast<uint32_t>(planes);
            int64_t ssn, ssh, dsn, dsh;
            if (src_pool) {
                pool_strides(kv, src_pool->p->layout, &ssn, &ssh);
                b.src_off = grp.bt_src[jj] * src_pool->block_stride + h0 * ssh;
                b.src_outer = src_pool->plane_stride;
                b.src_slot_step = src_pool->slot_step;
            } else {
                packed_strides(kv, packed_layout, Tr, hs, &ssn, &ssh);
                b.src_off = off_r + j * kv.B * ssn;
                b.src_outer = packed_outer;
            }
            if (dst_pool) {
                pool_strides(kv, dst_pool->p->layout, &dsn, &dsh);
                b.dst_off = grp.bt_dst[jj] * dst_pool->block_stride + h0 * dsh;
                b.dst_outer = dst_pool->plane_stride;
                b.dst_slot_step = dst_pool->slot_step;
            } else {
                packed_strides(kv, packed_layout, Tr, hs, &dsn, &dsh);
                b.dst_off = off_r + j * kv.B * dsn;
                b.dst_outer = packed_outer;
            }
            b.src_slot = 0;
            b.dst_slot = 0;
            b.dims = {Dim{hs, ssh, dsh}, Dim{nvalid, ssn, dsn}};
            lower_box(g, b, tile_bytes);
        }
        if (has_packed)  // staged plans cut segments from the requests' contiguous regions
            g.requests.push_back(RequestSpan{first_desc, static_cast<uint32_t>(g.descs.size()), off_r, plane_bytes});
        off_r += layer_major ? plane_bytes : planes * plane_bytes;
    }
}

// Cut a staged group into segments: windows of descriptors x planes whose packed-side bytes
// are one contiguous range of at most kStageBytes.  Runs of small consecutive requests share
// a segment; a request larger than a staging buffer is cut at plane boundaries.
//
// Layer-major packed buffers: plane (l,c) of ALL requests is contiguous (stride P = one plane of
// every request), and q.off is the request's offset inside a plane.  A segment is a run of whole
// planes when P fits a staging buffer several times, else a run of requests inside one plane;
// segments come out in buffer order, plane 0 first, so a consumer of the host buffer (or of the
// pool, on reload) sees the layers complete one after the other.
static int build_segments(Group &g, int64_t planes, bool layer_major)
{
    if (!g.tiles_per_desc) return TC_OK;  // non-uniform group: stays on the zero-copy path
    for (const Desc &d : g.descs)
        if (d.n_outer != planes) return TC_OK;
    if (layer_major) {
        int64_t P = 0;
        for (const RequestSpan &q : g.requests) {
            if (q.plane_bytes > kStageBytes)
                return fail(TC_ERR_TOO_LARGE, "a staged plan needs every (layer, K|V) plane of a request to fit a %lld-byte staging buffer; one has %lld bytes", (long long)kStageBytes, (long long)q.plane_bytes);
            P += q.plane_bytes;
        }
        if (P == 0) return TC_OK;
        const uint32_t nd_all = static_cast<uint32_t>(g.descs.size());
        if (P <= kStageBytes) {
            const int64_t per = kStageBytes / P;
            for (int64_t o0 = 0; o0 < planes; o0 += per) {
                const int64_t no = std::min(per, planes - o0);
                g.segments.push_back(Segment{0, nd_all, static_cast<uint32_t>(o0), static_cast<uint32_t>(no), o0 * P, static_cast<uint32_t>(g.copies.size()), 1});
                g.copies.push_back(StageCopy{0, o0 * P, no * P});
            }
            return TC_OK;
        }
        for (int64_t o = 0; o < planes; o++) {
            size_t i = 0;
            while (i < g.requests.size()) {
                int64_t sum = 0;
                size_t j = i;
                while (j < g.requests.size() && sum + g.requests[j].plane_bytes <= kStageBytes) sum += g.requests[j++].plane_bytes;
                const RequestSpan &q = g.requests[i];
                if (sum > 0) {
                    g.segments.push_back(Segment{q.d0, g.requests[j - 1].d1 - q.d0, static_cast<uint32_t>(o), 1, o * P + q.off, static_cast<uint32_t>(g.copies.size()), 1});
                    g.copies.push_back(StageCopy{0, o * P + q.off, sum});
                }
                i = j;
            }
        }
        return TC_OK;
    }
    size_t i = 0;
    while (i < g.requests.size()) {
        const RequestSpan &q = g.requests[i];
        const int64_t total = planes * q.plane_bytes;
        if (total == 0) { i++; continue; }
        if (total <= kStageBytes) {
            int64_t sum = 0;
            size_t j = i;
            while (j < g.requests.size() && sum + planes * g.requests[j].plane_bytes <= kStageBytes) sum += planes * g.requests[j++].plane_bytes;
            g.segments.push_back(Segment{q.d0, g.requests[j - 1].d1 - q.d0, 0, static_cast<uint32_t>(planes), q.off, static_cast<uint32_t>(g.copies.size()), 1});
            g.copies.push_back(StageCopy{0, q.off, sum});
            i = j;
        } else {
            if (q.plane_bytes > kStageBytes)
                return fail(TC_ERR_TOO_LARGE, "a staged plan needs every (layer, K|V) plane of a request to fit a %lld-byte staging buffer; one has %lld bytes", (long long)kStageBytes, (long long)q.plane_bytes);
            const int64_t per = kStageBytes / q.plane_bytes;
            for (int64_t o0 = 0; o0 < planes; o0 += per) {
                const int64_t no = std::min(per, planes - o0);
                g.segments.push_back(Segment{q.d0, q.d1 - q.d0, static_cast<uint32_t>(o0), static_cast<uint32_t>(no), q.off + o0 * q.plane_bytes, static_cast<uint32_t>(g.copies.size()), 1});
                g.copies.push_back(StageCopy{0, q.off + o0 * q.plane_bytes, no * q.plane_bytes});
            }
            i++;
        }
    }
    return TC_OK;
}

static int build_kv(const tc_plan_spec_t *spec, tc_plan *plan, uint32_t tile_bytes)
{
    const tc_kv_spec_t &kv = spec->kv;
    if (kv.L < 1 || kv.B < 1 || kv.H < 1 || kv.D < 1) return fail(TC_ERR_SHAPE, "L, B, H, D must be >= 1");
    if (kv.E != 1 && kv.E != 2 && kv.E != 4 && kv.E != 8) return fail(TC_ERR_SHAPE, "E = %lld must be 1, 2, 4 or 8", (long long)kv.E);
    if (kv.L * 2 > TC_MAX_TABLE_SLOTS / 2) return fail(TC_ERR_INVALID_ARG, "L*2 = %lld exceeds the table limit", (long long)(kv.L * 2));
    const int kind = spec->kind;
    const bool src_is_pool = kind != TC_KV_UNPACK, dst_is_pool = kind != TC_KV_PACK;
    PoolView sp{}, dp{};
    int rc;
    if (src_is_pool && (rc = check_pool(kv, kv.src_pool, "src_pool", &sp))) return rc;
    if (dst_is_pool && (rc = check_pool(kv, kv.dst_pool, "dst_pool", &dp))) return rc;
    if ((rc = check_group(kv, kv.group, "group", src_is_pool, &kv.src_pool, dst_is_pool, &kv.dst_pool))) return rc;
    if (kv.head_begin < 0 || kv.head_count < 0 || kv.head_begin + kv.head_count > kv.H || kv.head_begin >= kv.H)
        return fail(TC_ERR_BOUNDS, "head slice [%lld, +%lld) lies outside the %lld heads", (long long)kv.head_begin, (long long)kv.head_count, (long long)kv.H);
    if (kv.packed_order != TC_REQUEST_MAJOR && kv.packed_order != TC_LAYER_MAJOR)
        return fail(TC_ERR_INVALID_ARG, "packed_order %d is not a tc_packed_order", kv.packed_order);
    if ((kind == TC_KV_MIGRATE || kind == TC_KV_MIXED) && (kv.head_begin || kv.head_count || kv.packed_order))
        return fail(TC_ERR_INVALID_ARG, "head slices and packed_order apply to plans with a packed buffer (PACK, UNPACK)");
    if (kind == TC_KV_PACK || kind == TC_KV_UNPACK) {
        if (kv.packed_layout != TC_NHD && kv.packed_layout != TC_HND)
            return fail(TC_ERR_INVALID_ARG, "packed_layout %d is not a tc_layout", kv.packed_layout);
        const int64_t hs = kv.head_count ? kv.head_count : kv.H - kv.head_begin;
        int64_t need = 0;
        for (int64_t r = 0; r < kv.group.R; r++) need += kv.L * 2 * kv.group.T[r] * hs * kv.D * kv.E;
        plan->packed_required = need;
        if (kv.packed_bytes && kv.packed_bytes < need)
            return fail(TC_ERR_BOUNDS, "packed_bytes %lld < %lld required", (long long)kv.packed_bytes, (long long)need);
    }
    Group &g0 = plan->group[0], &g1 = plan->group[1];
    if (kind == TC_KV_PACK) {
        lower_kv_group(g0, kv, kv.group, &sp, nullptr, kv.packed_layout, tile_bytes);
        g0.n_src = kv.src_pool.n_slots;
        g0.n_dst = 1;
    } else if (kind == TC_KV_UNPACK) {
        lower_kv_group(g1, kv, kv.group, nullptr, &dp, kv.packed_layout, tile_bytes);
        g1.n_src = 1;
        g1.n_dst = kv.dst_pool.n_slots;
    } else if (kind == TC_KV_MIGRATE) {
        if (spec->flags & TC_PLAN_SAME_POOL) {
            const tc_kv_pool_t &a = kv.src_pool, &b = kv.dst_pool;
            if (a.layout != b.layout || a.num_blocks != b.num_blocks || a.n_slots != b.n_slots || sp.block_stride != dp.block_stride || sp.plane_stride != dp.plane_stride)
                return fail(TC_ERR_INVALID_ARG, "TC_PLAN_SAME_POOL: src_pool and dst_pool must describe the same pool");
            const int64_t n = kv.group.R ? kv.group.bt_off[kv.group.R] : 0;
            std::vector<uint8_t> read(static_cast<size_t>(a.num_blocks), 0);
            for (int64_t j = 0; j < n; j++) read[kv.group.bt_src[j]] = 1;
            for (int64_t j = 0; j < n; j++)
                if (read[kv.group.bt_dst[j]])
                    return fail(TC_ERR_OVERLAP, "TC_PLAN_SAME_POOL: block %d is both read and written", kv.group.bt_dst[j]);
        }
        lower_kv_group(g0, kv, kv.group, &sp, &dp, 0, tile_bytes);
        g0.n_src = kv.src_pool.n_slots;
        g0.n_dst = kv.dst_pool.n_slots;
    } else {  // MIXED: offload src_pool -> dst_pool, reload dst_pool -> src_pool
        if ((rc = check_group(kv, kv.reload, "reload", true, &kv.dst_pool, true, &kv.src_pool))) return rc;
        const int64_t n_off = kv.group.R ? kv.group.bt_off[kv.group.R] : 0;
        const int64_t n_rel = kv.reload.R ? kv.reload.bt_off[kv.reload.R] : 0;
        // the two groups may run concurrently: neither may write what the other reads or writes
        std::vector<uint8_t> host_used(static_cast<size_t>(kv.dst_pool.num_blocks), 0), dev_used(static_cast<size_t>(kv.src_pool.num_blocks), 0);
        for (int64_t j = 0; j < n_off; j++) { host_used[kv.group.bt_dst[j]] = 1; dev_used[kv.group.bt_src[j]] = 1; }
        for (int64_t j = 0; j < n_rel; j++) {
            if (host_used[kv.reload.bt_src[j]])
                return fail(TC_ERR_OVERLAP, "block %d of dst_pool is written by the offload group and read by the reload group", kv.reload.bt_src[j]);
            if (dev_used[kv.reload.bt_dst[j]])
                return fail(TC_ERR_OVERLAP, "block %d of src_pool is read by the offload group and written by the reload group", kv.reload.bt_dst[j]);
        }
        // Staged variant: the host pool's pages travel through the device staging ring with the
        // copy engines, one transfer per 2 MiB-like page, and the kernels run device to device
        // against a virtual pool of ring slots.  It needs whole pages on the host side: a
        // page-first pool in one allocation and groups made of full blocks only.
        const int64_t page = planes_of(kv) * dp.chunk;
        auto whole_blocks = [&](const tc_kv_group_t &g) {
            for (int64_t r = 0; r < g.R; r++)
                if (g.T[r] % kv.B) return false;
            return true;
        };
        const bool can_stage = (spec->flags & TC_PLAN_STAGED) && kv.dst_pool.n_slots == 1 && dp.plane_stride == dp.chunk &&
                               page <= kStageBytes && whole_blocks(kv.group) && whole_blocks(kv.reload);
        if (can_stage) {
            const int64_t slots = kStageBytes / page;
            PoolView ring = dp;       // same page layout, block id = slot in the ring buffer
            ring.block_stride = page;
            std::vector<int32_t> virt(static_cast<size_t>(std::max(n_off, n_rel)));
            for (size_t k = 0; k < virt.size(); k++) virt[k] = static_cast<int32_t>(k % slots);
            tc_kv_group_t off_v = kv.group, rel_v = kv.reload;
            off_v.bt_dst = virt.data();
            rel_v.bt_src = virt.data();
            if (spec->flags & TC_PLAN_OFFLOAD_ZERO_COPY) {  // only the reload travels through the ring
                lower_kv_group(g0, kv, kv.group, &sp, &dp, 0, tile_bytes);
            } else {
                lower_kv_group(g0, kv, off_v, &sp, &ring, 0, tile_bytes);
                g0.stage_whole_host_pool = true;
                stage_pages(g0, kv.group.bt_dst, n_off, slots, page, dp.block_stride);
            }
            lower_kv_group(g1, kv, rel_v, &ring, &sp, 0, tile_bytes);
            g1.stage_whole_host_pool = true;
            stage_pages(g1, kv.reload.bt_src, n_rel, slots, page, dp.block_stride);
        } else {
            lower_kv_group(g0, kv, kv.group, &sp, &dp, 0, tile_bytes);
            lower_kv_group(g1, kv, kv.reload, &dp, &sp, 0, tile_bytes);
        }
        g0.n_src = kv.src_pool.n_slots;
        g0.n_dst = kv.dst_pool.n_slots;
        g1.n_src = kv.dst_pool.n_slots;
        g1.n_dst = kv.src_pool.n_slots;
    }
    if (spec->flags & TC_PLAN_DEBUG_BOUNDS) {
        // what every table slot is declared to hold: the device-side checker holds the uploaded
        // descriptors against these numbers
        auto pool_extent = [](const tc_kv_pool_t &p, const PoolView &v) { return p.slot_bytes ? p.slot_bytes : v.slot_need; };
        const int64_t packed = kv.packed_bytes ? kv.packed_bytes : plan->packed_required;
        auto fill = [&](Group &g, bool src_pool_side, bool dst_pool_side, const tc_kv_pool_t &spool, const PoolView &sv, const tc_kv_pool_t &dpool, const PoolView &dv) {
            g.extents.assign(g.n_src, src_pool_side ? pool_extent(spool, sv) : packed);
            g.extents.insert(g.extents.end(), g.n_dst, dst_pool_side ? pool_extent(dpool, dv) : packed);
        };
        if (kind == TC_KV_PACK) fill(g0, true, false, kv.src_pool, sp, kv.dst_pool, dp);
        else if (kind == TC_KV_UNPACK) fill(g1, false, true, kv.src_pool, sp, kv.dst_pool, dp);
        else {
            fill(g0, true, true, kv.src_pool, sp, kv.dst_pool, dp);
            if (kind == TC_KV_MIXED) fill(g1, true, true, kv.dst_pool, dp, kv.src_pool, sp);
        }
    }
    return TC_OK;
}

// ------------------------------------------------------------------------------ weights
struct Span {
    int64_t lo, hi;
    int64_t tensor;
};

static int build_weights(const tc_plan_spec_t *spec, tc_plan *plan, uint32_t tile_bytes)
{
    const tc_weights_spec_t &w = spec->weights;
    if (w.n_tensors < 0) return fail(TC_ERR_SHAPE, "n_tensors %lld < 0", (long long)w.n_tensors);
    if (w.n_tensors > 0 && !w.index) return fail(TC_ERR_INVALID_ARG, "index is required");
    if (w.world < 1 || w.rank < 0 || w.rank >= w.world)
        return fail(TC_ERR_INVALID_ARG, "rank %d / world %d is not a valid tensor-parallel position", w.rank, w.world);
    const int64_t n_dst = w.n_dst ? w.n_dst : w.n_tensors;
    if (n_dst + 1 > TC_MAX_TABLE_SLOTS) return fail(TC_ERR_INVALID_ARG, "%lld destination slots exceed the table limit %d", (long long)n_dst, TC_MAX_TABLE_SLOTS - 1);
    Group &g = plan->group[0];
    g.n_src = 1;
    g.n_dst = static_cast<size_t>(n_dst);
    std::vector<std::vector<Span>> spans(static_cast<size_t>(n_dst));
    std::vector<uint8_t> verify_rows(static_cast<size_t>(n_dst), 0);  // slots that need the exact check
    std::vector<Box> boxes;
    boxes.reserve(static_cast<size_t>(w.n_tensors));
    for (int64_t i = 0; i < w.n_tensors; i++) {
        const tc_index_entry_t &t = w.index[i];
        if (t.ndim < 1 || t.ndim > 4) return fail(TC_ERR_SHAPE, "tensor %lld: ndim %u outside 1..4", (long long)i, t.ndim);
        if (t.elem_bytes != 1 && t.elem_bytes != 2 && t.elem_bytes != 4 && t.elem_bytes != 8)
            return fail(TC_ERR_SHAPE, "tensor %lld: elem_bytes %u", (long long)i, t.elem_bytes);
        int64_t shp[4] = {1, 1, 1, 1}, count = 1;
        for (uint32_t m = 0; m < 4; m++) {
            if (m < t.ndim) shp[m] = static_cast<int64_t>(t.shape[m]);
            else if (t.shape[m] > 1) return fail(TC_ERR_SHAPE, "tensor %lld: shape[%u] = %llu beyond ndim", (long long)i, m, (unsigned long long)t.shape[m]);
            if (shp[m] < 0 || (shp[m] && count > (1ll << 62) / std::max<int64_t>(shp[m], 1)))
                return fail(TC_ERR_SHAPE, "tensor %lld: extent overflow", (long long)i);
            count *= shp[m];
        }
        if (static_cast<int64_t>(t.nbytes) != count * t.elem_bytes)
            return fail(TC_ERR_SHAPE, "tensor %lld: nbytes %llu != elem_bytes * prod(shape) = %lld", (long long)i, (unsigned long long)t.nbytes, (long long)(count * t.elem_bytes));
        if (static_cast<int64_t>(t.byte_off) < 0 || static_cast<int64_t>(t.byte_off + t.nbytes) > w.blob_bytes)
            return fail(TC_ERR_BOUNDS, "tensor %lld: bytes [%llu, %llu) lie outside the blob of %lld", (long long)i, (unsigned long long)t.byte_off, (unsigned long long)(t.byte_off + t.nbytes), (long long)w.blob_bytes);
        tc_weight_rule_t rule{};
        rule.split_dim = -1;
        rule.dst_slot = -1;
        if (w.rules) rule = w.rules[i];
        int64_t ext[4] = {shp[0], shp[1], shp[2], shp[3]}, shift = 0;
        int64_t sstr[4];
        sstr[3] = t.elem_bytes;
        for (int m = 2; m >= 0; m--) sstr[m] = sstr[m + 1] * shp[m + 1];
        if (rule.split_dim >= 0) {
            if (rule.split_dim >= static_cast<int32_t>(t.ndim)) return fail(TC_ERR_SHAPE, "tensor %lld: split_dim %d >= ndim %u", (long long)i, rule.split_dim, t.ndim);
            if (shp[rule.split_dim] % w.world) return fail(TC_ERR_SHAPE, "tensor %lld: dim %d of extent %lld is not divisible by world %d", (long long)i, rule.split_dim, (long long)shp[rule.split_dim], w.world);
            ext[rule.split_dim] = shp[rule.split_dim] / w.world;
            shift = w.rank * ext[rule.split_dim] * sstr[rule.split_dim];
        } else if (rule.split_dim != -1) {
            return fail(TC_ERR_INVALID_ARG, "tensor %lld: split_dim %d", (long long)i, rule.split_dim);
        }
        int64_t dstr[4];
        bool tight = !(rule.dst_stride[0] | rule.dst_stride[1] | rule.dst_stride[2] | rule.dst_stride[3]);
        if (tight) {
            dstr[3] = t.elem_bytes;
            for (int m = 2; m >= 0; m--) dstr[m] = dstr[m + 1] * ext[m + 1];
        } else {
            for (int m = 0; m < 4; m++) {
                dstr[m] = rule.dst_stride[m];
                if (ext[m] > 1 && dstr[m] <= 0) return fail(TC_ERR_INVALID_ARG, "tensor %lld: dst_stride[%d] = %lld must be positive", (long long)i, m, (long long)dstr[m]);
            }
        }
        const int64_t slot = rule.dst_slot < 0 ? i : rule.dst_slot;
        if (slot >= n_dst) return fail(TC_ERR_INVALID_ARG, "tensor %lld: dst_slot %lld >= n_dst %lld", (long long)i, (long long)slot, (long long)n_dst);
        if (rule.dst_off < 0) return fail(TC_ERR_BOUNDS, "tensor %lld: dst_off %lld < 0", (long long)i, (long long)rule.dst_off);
        int64_t n_el = ext[0] * ext[1] * ext[2] * ext[3];
        if (n_el == 0) continue;
        int64_t hi = rule.dst_off + t.elem_bytes;
        for (int m = 0; m < 4; m++) hi += (ext[m] - 1) * dstr[m];
        const int64_t slot_extent = w.dst_bytes ? w.dst_bytes[slot] : (tight && rule.dst_off == 0 ? n_el * t.elem_bytes : -1);
        if (slot_extent < 0) return fail(TC_ERR_INVALID_ARG, "tensor %lld: dst_bytes is required when a rule sets dst_off or dst_stride", (long long)i);
        if (hi > slot_extent) return fail(TC_ERR_BOUNDS, "tensor %lld: writes up to byte %lld of a %lld-byte destination", (long long)i, (long long)hi, (long long)slot_extent);
        spans[static_cast<size_t>(slot)].push_back(Span{rule.dst_off, hi, i});
        if (!tight) {
            // A tensor may also overlap ITSELF: rows or elements closer together than they are
            // long.  Sufficient for disjointness: taken by ascending stride, every dimension
            // steps over the whole extent of the dimensions inside it.  Strides that do not nest
            // this way (interleavings) are decided by the exact check below.
            std::pair<int64_t, int64_t> by_stride[4];
            int nd = 0;
            for (int m = 0; m < 4; m++)
                if (ext[m] > 1) by_stride[nd++] = {dstr[m], ext[m]};
            std::sort(by_stride, by_stride + nd);
            int64_t inner = t.elem_bytes;
            for (int k = 0; k < nd; k++) {
                if (by_stride[k].first < inner) verify_rows[static_cast<size_t>(slot)] = 1;
                inner += (by_stride[k].second - 1) * by_stride[k].first;
            }
        }
        Box b;
        b.run = t.elem_bytes;
        b.tag = static_cast<uint32_t>(i);
        b.csum_base = static_cast<int64_t>(t.byte_off);
        b.src_off = static_cast<int64_t>(t.byte_off) + shift;
        b.dst_off = rule.dst_off;
        b.src_slot = 0;
        b.dst_slot = static_cast<uint32_t>(slot);
        for (int m = 3; m >= 0; m--) b.dims.push_back(Dim{ext[m], sstr[m], dstr[m]});
        boxes.push_back(std::move(b));
    }
    // exactly-once writes: bounding spans of one slot may not intersect and no tensor may overlap
    // itself.  (Interleaved strided destinations, whose bounding spans intersect or whose strides
    // do not nest, are checked row by row below.)
    for (size_t s = 0; s < spans.size(); s++) {
        auto &v = spans[s];
        std::sort(v.begin(), v.end(), [](const Span &a, const Span &b) { return a.lo < b.lo; });
        bool clash = verify_rows[s] != 0;
        for (size_t k = 1; k < v.size(); k++)
            if (v[k].lo < v[k - 1].hi) clash = true;
        if (!clash) continue;
        // exact check over the rows of every box that targets this slot
        Group tmp;
        for (const Box &b : boxes)
            if (b.dst_slot == s) lower_box(tmp, b, kMaxTileBytes);
        std::vector<std::pair<int64_t, int64_t>> rows;
        uint64_t total_rows = 0;
        for (const Desc &d : tmp.descs) total_rows += d.rows;
        if (total_rows > (64ull << 20)) return fail(TC_ERR_OVERLAP, "destination slot %zu: overlapping windows too fine to verify", s);
        rows.reserve(total_rows);
        for (const Desc &d : tmp.descs)
            for (uint32_t k = 0; k < d.rows; k++) {
                int64_t a = d.dst_off + static_cast<int64_t>(k / d.n0) * d.dst_s1 + static_cast<int64_t>(k % d.n0) * d.dst_s0;
                rows.emplace_back(a, a + d.run);
            }
        std::sort(rows.begin(), rows.end());
        for (size_t k = 1; k < rows.size(); k++)
            if (rows[k].first < rows[k - 1].second)
                return fail(TC_ERR_OVERLAP, "destination slot %zu: byte %lld would be written twice", s, (long long)rows[k].first);
    }
    for (const Box &b : boxes) lower_box(g, b, tile_bytes);
    g.host_is_src = true;
    if (spec->flags & TC_PLAN_DEBUG_BOUNDS) {
        g.extents.assign(1, w.blob_bytes);
        g.extents.resize(1 + static_cast<size_t>(n_dst), 0);
        for (size_t slot = 0; slot < spans.size(); slot++)
            for (const Span &sp_ : spans[slot])
                g.extents[1 + slot] = w.dst_bytes ? w.dst_bytes[slot] : std::max(g.extents[1 + slot], sp_.hi);
    }
    if (spec->flags & TC_PLAN_CHECKSUM) {
        // checksums are sums over aligned 4-byte words of each tensor: every run must be made of
        // whole words and every access must be 16-byte aligned
        if (g.log2_align < 4) return fail(TC_ERR_INVALID_ARG, "TC_PLAN_CHECKSUM needs 16-byte aligned offsets, strides and runs");
        for (int64_t i = 0; i < w.n_tensors; i++)
            if (w.index[i].byte_off % 4) return fail(TC_ERR_INVALID_ARG, "TC_PLAN_CHECKSUM: tensor %lld starts at byte %llu, not a multiple of 4", (long long)i, (unsigned long long)w.index[i].byte_off);
        plan->checksummed = true;
        plan->n_sums = w.n_tensors;
    }
    return TC_OK;
}

// Byte range of the blob that tile (outer o, part p) of descriptor d reads: [*lo, *hi).
static void tile_cover(const Desc &d, uint32_t o, uint32_t p, int64_t *lo, int64_t *hi)
{
    const uint32_t row0 = p * d.rows_per_tile, last = std::min(d.rows, row0 + d.rows_per_tile) - 1;
    const uint32_t i1a = row0 / d.n0, i0a = row0 % d.n0, i1b = last / d.n0, i0b = last % d.n0;
    auto at = [&](uint32_t i1, uint32_t i0) { return static_cast<int64_t>(i1) * d.src_s1 + static_cast<int64_t>(i0) * d.src_s0; };
    int64_t first = at(i1a, i0a), end = at(i1b, i0b);
    if (i1a != i1b) {  // the tile wraps over the inner index: its extremes may sit at the wrap
        first = std::min(first, at(i1a + 1, 0));
        end = std::max(end, at(i1b - 1, d.n0 - 1));
    }
    const int64_t base = d.src_off + static_cast<int64_t>(o) * d.src_outer;
    *lo = base + first;
    *hi = base + end + d.run;
}

// Weights: cut the tile sequence into segments whose blob bytes form one range of at most one
// staging buffer.  Plain staging (blob in pinned memory) takes only tensors read in contiguous
// pieces, back to back; anything else leaves the whole group zero copy (the kernel then fetches
// exactly the bytes it needs over the link).  Streaming (`covering`) takes every descriptor: a
// strided slice travels as the byte range that covers it, as a loader reading whole rows from
// storage would, and tiles whose ranges are close (gap no longer than the tile's own range)
// share a segment.  Segment starts are rounded down to 4 KiB: file reads start on page
// boundaries and every byte keeps its alignment modulo 16 inside the staging buffer.
static int build_segments_blob(Group &g, bool covering)
{
    if (g.descs.empty()) return TC_OK;
    if (!covering)
        for (const Desc &d : g.descs) {
            const bool rows_contiguous = d.rows == 1 || (d.src_s0 == d.run && (d.rows == d.n0 || d.src_s1 == d.n0 * d.run));
            if (d.n_outer != 1 || !rows_contiguous || d.src_slot != 0) return TC_OK;
        }
    int64_t seg_lo = -1, seg_hi = -1;
    uint32_t seg_t0 = 0, seg_t1 = 0;
    auto flush = [&]() {
        if (seg_lo < 0) return;
        g.segments.push_back(Segment{seg_t0, 0, 0, seg_t1 - seg_t0, seg_lo, static_cast<uint32_t>(g.copies.size()), 1});
        g.copies.push_back(StageCopy{0, seg_lo, seg_hi - seg_lo});
        seg_lo = -1;
    };
    for (const Desc &d : g.descs)
        for (uint32_t o = 0; o < d.n_outer; o++)
            for (uint32_t p = 0; p < d.tiles_per_outer; p++) {
                if (p * d.rows_per_tile >= d.rows) continue;  // padding part of a uniform group: empty
                const uint32_t t = d.tile0 + o * d.tiles_per_outer + p;
                int64_t lo, hi;
                tile_cover(d, o, p, &lo, &hi);
                const int64_t gap_ok = covering ? hi - lo : 0;
                const bool joins = seg_lo >= 0 && lo >= seg_lo && lo - seg_hi <= gap_ok && (covering || lo == seg_hi);
                if (!joins || std::max(hi, seg_hi) - seg_lo > kStageBytes) flush();
                if (seg_lo < 0) {
                    seg_lo = covering ? lo & ~int64_t(4095) : lo;
                    seg_hi = hi;
                    seg_t0 = t;
                    if (hi - seg_lo > kStageBytes) {
                        g.segments.clear();
                        g.copies.clear();
                        return fail(TC_ERR_TOO_LARGE, "a tile of the plan reads a blob range of %lld bytes, more than one %lld-byte staging buffer: the slice is too sparse to stream", (long long)(hi - seg_lo), (long long)kStageBytes);
                    }
                }
                seg_hi = std::max(seg_hi, hi);
                seg_t1 = t + 1;
            }
    flush();
    return TC_OK;
}

// ------------------------------------------------------------------------------ entry
int build_plan(const tc_plan_spec_t *spec, tc_plan *plan)
{
    // Checksummed plans default to tiles of twice the size: every tile ends with a block-wide
    // reduction of the checksum, and at 64 KiB that tail is hidden (measured: 6.77 TB/s against
    // 6.53 TB/s with 32 KiB tiles; a plain run of the same plan gives up 1.5 %).
    const uint32_t default_tile = (spec->flags & TC_PLAN_CHECKSUM) ? 2 * kDefaultTileBytes : kDefaultTileBytes;
    uint32_t tile_bytes = spec->tuning.tile_bytes > 0 ? static_cast<uint32_t>(spec->tuning.tile_bytes) : default_tile;
    if (tile_bytes < 512 || tile_bytes > kMaxTileBytes || (tile_bytes & (tile_bytes - 1)))
        return fail(TC_ERR_INVALID_ARG, "tuning.tile_bytes %u must be a power of two in [512, %u]", tile_bytes, kMaxTileBytes);
    if (spec->tuning.tile_order < 0 || spec->tuning.tile_order > 2)
        return fail(TC_ERR_INVALID_ARG, "tuning.tile_order %d must be 0 (auto), 1 (descriptor order) or 2 (plane-major)", spec->tuning.tile_order);
    if (spec->tuning.copy_path != 0 && spec->tuning.copy_path != 1)
        return fail(TC_ERR_INVALID_ARG, "tuning.copy_path %d must be 0 (auto) or 1 (through shared memory)", spec->tuning.copy_path);
    int rc;
    switch (spec->kind) {
    case TC_KV_PACK:
    case TC_KV_UNPACK:
    case TC_KV_MIGRATE:
    case TC_KV_MIXED:
        rc = build_kv(spec, plan, tile_bytes);
        break;
    case TC_WEIGHTS:
        rc = build_weights(spec, plan, tile_bytes);
        break;
    default:
        return fail(TC_ERR_INVALID_ARG, "kind %d is not a tc_kind", spec->kind);
    }
    if (rc) return rc;
    for (int k = 0; k < 2; k++) {
        Group &g = plan->group[k];
        // destination slots follow the source slots in the combined pointer table
        for (Desc &d : g.descs) d.dst_slot = static_cast<uint16_t>(d.dst_slot + g.n_src);
        // KV groups that are not staged: ascending destination offsets (descriptors are
        // independent, so their order is free; staged groups keep request order, which their
        // segments are cut from)
        const bool kv_kind = spec->kind != TC_WEIGHTS;
        if (kv_kind && !(spec->flags & TC_PLAN_STAGED) && spec->tuning.tile_order != 1 &&
            !std::is_sorted(g.descs.begin(), g.descs.end(), [](const Desc &a, const Desc &b) { return a.dst_off < b.dst_off; })) {
            // sort 12-byte keys, then move every 128-byte descriptor once
            std::vector<std::pair<int64_t, uint32_t>> key(g.descs.size());
            for (size_t i = 0; i < key.size(); i++) key[i] = {g.descs[i].dst_off, static_cast<uint32_t>(i)};
            std::sort(key.begin(), key.end());  // ties keep their order: the index is the second key
            std::vector<Desc> sorted(g.descs.size());
            for (size_t i = 0; i < key.size(); i++) sorted[i] = g.descs[key[i].second];
            g.descs.swap(sorted);
        }
        if ((rc = finish_group(g, tile_bytes))) return rc;
    }
    if ((spec->flags & TC_PLAN_SAME_POOL) && spec->kind != TC_KV_MIGRATE)
        return fail(TC_ERR_KIND, "TC_PLAN_SAME_POOL applies to TC_KV_MIGRATE plans only");
    if ((spec->flags & TC_PLAN_CHECKSUM) && spec->kind != TC_WEIGHTS)
        return fail(TC_ERR_KIND, "TC_PLAN_CHECKSUM applies to TC_WEIGHTS plans only");
    plan->group[1].host_is_src = true;  // UNPACK / reload read the host side
    if ((spec->flags & TC_PLAN_OFFLOAD_ZERO_COPY) && (spec->kind != TC_KV_MIXED || !(spec->flags & TC_PLAN_STAGED)))
        return fail(TC_ERR_KIND, "TC_PLAN_OFFLOAD_ZERO_COPY applies to staged TC_KV_MIXED plans only");
    if ((spec->flags & TC_PLAN_DEBUG_BOUNDS) && (spec->flags & (TC_PLAN_STAGED | TC_PLAN_STREAM)))
        return fail(TC_ERR_INVALID_ARG, "TC_PLAN_DEBUG_BOUNDS checks plans that run directly, not staged or streamed ones");
    if ((spec->flags & TC_PLAN_STREAM) && spec->kind != TC_WEIGHTS)
        return fail(TC_ERR_KIND, "TC_PLAN_STREAM applies to TC_WEIGHTS plans only");
    if (spec->flags & (TC_PLAN_STAGED | TC_PLAN_STREAM)) {
        if (spec->kind == TC_KV_MIGRATE)
            return fail(TC_ERR_KIND, "TC_PLAN_STAGED does not apply to TC_KV_MIGRATE plans (no host side)");
        if (spec->kind == TC_WEIGHTS) {
            if ((rc = build_segments_blob(plan->group[0], (spec->flags & TC_PLAN_STREAM) != 0))) return rc;
        } else if (spec->kind == TC_KV_MIXED) {
            // segments were cut while lowering; a group that could not be staged must drop them
            for (int k = 0; k < 2; k++) {
                Group &g = plan->group[k];
                if (!g.stage_whole_host_pool || !g.tiles_per_desc) {
                    if (g.stage_whole_host_pool && !g.descs.empty()) return fail(TC_ERR_INVALID_ARG, "staged MIXED group is not uniform");
                    g.segments.clear();
                    g.copies.clear();
                }
            }
        } else {
            Group &g = plan->group[spec->kind == TC_KV_PACK ? 0 : 1];
            if ((rc = build_segments(g, spec->kv.L * 2, spec->kv.packed_order == TC_LAYER_MAJOR))) return rc;
        }
    }
    return TC_OK;
}

}  // namespace tc

extern "C" const char *tc_last_error(void) { return tc::last_error(); }

extern "C" const char *tc_strerror(int status)
{
    switch (status) {
    case TC_OK: return "TC_OK";
    case TC_ERR_INVALID_ARG: return "TC_ERR_INVALID_ARG";
    case TC_ERR_SHAPE: return "TC_ERR_SHAPE";
    case TC_ERR_BOUNDS: return "TC_ERR_BOUNDS";
    case TC_ERR_OVERLAP: return "TC_ERR_OVERLAP";
    case TC_ERR_KIND: return "TC_ERR_KIND";
    case TC_ERR_OOM: return "TC_ERR_OOM";
    case TC_ERR_CUDA: return "TC_ERR_CUDA";
    case TC_ERR_DEADLINE: return "TC_ERR_DEADLINE";
    case TC_ERR_TOO_LARGE: return "TC_ERR_TOO_LARGE";
    case TC_ERR_IO: return "TC_ERR_IO";
    default: return "TC_ERR_UNKNOWN";
    }
}
