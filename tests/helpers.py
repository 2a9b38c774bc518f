"""Shared test helpers: a numpy interpreter of lowered descriptors (test-only: it lets the CPU
suite check the plan builder against the oracle without a GPU) and small case builders."""
import numpy as np

import oracle
import paper_2608_06007_b200 as tc
import workloads as wl


def run_descriptors(descs, src_tables, dst_tables, dst_counts=None):
    """Execute tc_descriptor_t records on flat uint8 numpy buffers, byte-run by byte-run."""
    for d in descs:
        for o in range(d.n_outer):
            s = src_tables[d.src_slot + o * d.src_slot_step]
            t = dst_tables[d.dst_slot + o * d.dst_slot_step]
            for k in range(d.rows):
                i1, i0 = divmod(k, d.n0)
                a = d.src_off + o * d.src_outer + i1 * d.src_s1 + i0 * d.src_s0
                b = d.dst_off + o * d.dst_outer + i1 * d.dst_s1 + i0 * d.dst_s0
                # no sanitizer runs on the GPU pool, so every lowered access is bounds-checked here
                assert 0 <= a and a + d.run_bytes <= s.size, "descriptor reads outside its source slot"
                assert 0 <= b and b + d.run_bytes <= t.size, "descriptor writes outside its destination slot"
                t[b:b + d.run_bytes] = s[a:a + d.run_bytes]
                if dst_counts is not None:
                    dst_counts[d.dst_slot + o * d.dst_slot_step][b:b + d.run_bytes] += 1


def run_window(descs, seg, src_tables, dst_tables, dst_counts=None, src_shift=0, dst_shift=0):
    """Execute the window of descriptors x planes of one staged KV segment; the staged side's
    addresses are taken relative to the segment's first host byte (src_shift or dst_shift)."""
    for d in descs[seg.desc0:seg.desc0 + seg.n_descs]:
        for o in range(seg.outer0, seg.outer0 + seg.n_outer):
            assert o < d.n_outer
            s = src_tables[d.src_slot + o * d.src_slot_step]
            t = dst_tables[d.dst_slot + o * d.dst_slot_step]
            for k in range(d.rows):
                i1, i0 = divmod(k, d.n0)
                a = d.src_off + o * d.src_outer + i1 * d.src_s1 + i0 * d.src_s0 - src_shift
                b = d.dst_off + o * d.dst_outer + i1 * d.dst_s1 + i0 * d.dst_s0 - dst_shift
                assert 0 <= a and a + d.run_bytes <= s.size, "window reads outside its source"
                assert 0 <= b and b + d.run_bytes <= t.size, "window writes outside its destination"
                t[b:b + d.run_bytes] = s[a:a + d.run_bytes]
                if dst_counts is not None:
                    dst_counts[d.dst_slot + o * d.dst_slot_step][b:b + d.run_bytes] += 1


def run_tile_range(descs, tile0, n_tiles, src_tables, dst_tables, dst_counts=None, src_shift=0):
    """Execute only the tiles [tile0, tile0 + n_tiles) of the descriptors, as one launch of a
    staged / streamed segment does; source addresses are taken relative to `src_shift` (the
    segment's first host byte sits at the start of the staging buffer)."""
    for d in descs:
        for o in range(d.n_outer):
            s = src_tables[d.src_slot + o * d.src_slot_step]
            t = dst_tables[d.dst_slot + o * d.dst_slot_step]
            for p in range(d.tiles_per_outer):
                if not tile0 <= d.tile0 + o * d.tiles_per_outer + p < tile0 + n_tiles:
                    continue
                for k in range(p * d.rows_per_tile, min(d.rows, (p + 1) * d.rows_per_tile)):
                    i1, i0 = divmod(k, d.n0)
                    a = d.src_off + o * d.src_outer + i1 * d.src_s1 + i0 * d.src_s0 - src_shift
                    b = d.dst_off + o * d.dst_outer + i1 * d.dst_s1 + i0 * d.dst_s0
                    assert 0 <= a and a + d.run_bytes <= s.size, "tile reads outside its segment's staged bytes"
                    assert 0 <= b and b + d.run_bytes <= t.size, "tile writes outside its destination slot"
                    t[b:b + d.run_bytes] = s[a:a + d.run_bytes]
                    if dst_counts is not None:
                        dst_counts[d.dst_slot + o * d.dst_slot_step][b:b + d.run_bytes] += 1


def run_multiplane_tiles(descs, n_tiles, src_tables, dst_tables, dst_counts=None, threads=256, vec=16):
    """Walk a uniform group whose tiles take several planes of a descriptor (planes_per_tile > 1)
    tile id by tile id, with the index arithmetic of the kernel's multi-plane path: tile ->
    (descriptor, first plane); inside the tile every plane owns 2^log2_unit bytes of a byte space
    that `threads` lanes cross `vec` bytes at a time; byte -> (plane, row, column).  Every access is
    bounds-checked; lanes past a plane's real bytes or past the descriptor's last plane stay idle."""
    ppt = descs[0].planes_per_tile
    assert ppt > 1
    unit_max = max(d.rows * d.run_bytes for d in descs)
    log2_unit = 9
    while (1 << log2_unit) < unit_max:
        log2_unit += 1
    mask = (1 << log2_unit) - 1
    groups = -(-descs[0].n_outer // ppt)
    tiles_per_desc = groups * descs[0].tiles_per_outer
    assert n_tiles == tiles_per_desc * len(descs) and all(d.tiles_per_outer == 1 for d in descs)
    for tile in range(n_tiles):
        di, t = divmod(tile, tiles_per_desc)
        d = descs[di]
        assert d.tile0 == di * tiles_per_desc
        o = t * ppt
        if o >= d.n_outer:
            continue
        n_units = min(ppt, d.n_outer - o)
        unit_bytes = d.rows * d.run_bytes
        for byte in range(0, n_units << log2_unit, vec):          # lane order does not matter on the CPU
            k, w = o + (byte >> log2_unit), byte & mask
            if w >= unit_bytes:
                continue
            assert w + vec <= unit_bytes, "a vector straddles the end of a plane"
            r, col = divmod(w, d.run_bytes)
            i1, i0 = divmod(r, d.n0)
            a = d.src_off + k * d.src_outer + i1 * d.src_s1 + i0 * d.src_s0 + col
            b = d.dst_off + k * d.dst_outer + i1 * d.dst_s1 + i0 * d.dst_s0 + col
            s_ = src_tables[d.src_slot + k * d.src_slot_step]
            t_ = dst_tables[d.dst_slot + k * d.dst_slot_step]
            assert 0 <= a and a + vec <= s_.size, "multi-plane tile reads outside its source slot"
            assert 0 <= b and b + vec <= t_.size, "multi-plane tile writes outside its destination slot"
            t_[b:b + vec] = s_[a:a + vec]
            if dst_counts is not None:
                dst_counts[d.dst_slot + k * d.dst_slot_step][b:b + vec] += 1


class _Mem:
    """A flat buffer placed at a virtual address, so that a model can reason about alignment.
    Reads of whole aligned 16-byte chunks may reach up to 15 bytes outside the buffer (the
    kernel's realigning path does that, staying inside chunks that hold a byte it needs); those
    bytes read as 0xCC.  Writes outside the buffer are errors."""

    def __init__(self, arr, va):
        self.a, self.va = arr, va

    def read16(self, addr):
        assert addr % 16 == 0
        lo = addr - self.va
        out = np.full(16, 0xCC, dtype=np.uint8)
        a, b = max(lo, 0), min(lo + 16, self.a.size)
        assert a < b, "an aligned chunk with no byte of the buffer was read"
        out[a - lo:b - lo] = self.a[a:b]
        return out

    def write(self, addr, data, cnt=None):
        lo = addr - self.va
        assert 0 <= lo and lo + len(data) <= self.a.size, "write outside the destination"
        self.a[lo:lo + len(data)] = data
        if cnt is not None:
            cnt[lo:lo + len(data)] += 1


JOIN_MIN_RUN = 1024


def run_realign_tile_joined(d, o, part, src, dst, cnt, smem_bytes=52 << 10, threads=256):
    """The realigning path's back-to-back staging of rows that are adjacent in the destination
    (rows of at least JOIN_MIN_RUN bytes), replayed like run_realign_tile.  Returns False,
    touching nothing, for a tile the kernel would not take this way.  Per row one bulk load of
    its whole chunks to its place in its group, one of the chunk that holds its last s_lo bytes
    to a side array (unless it is the last of its group), then a merge of that side chunk into
    the next row's first chunk; the groups are then stored as long rows: whole chunks, heads and
    tails byte by byte."""
    run, n0 = d.run_bytes, d.n0
    row0 = part * d.rows_per_tile
    nrows = min(d.rows_per_tile, d.rows - row0)
    if run % 16 or run < JOIN_MIN_RUN or run > smem_bytes - 64 or nrows < 2:
        return False
    j1, j0 = divmod(row0, n0)
    across, groups, glen, vstride, cols = False, 1, nrows, 0, 0
    if d.dst_s1 == run:
        cols = nrows // n0
        if j0 or cols * n0 != nrows:
            return False
        across = True
        if n0 > 1 and d.dst_s0 != cols * run:
            groups, glen, vstride = n0, cols, d.dst_s0
    elif n0 > 1 and d.dst_s0 == run:
        if j0 + nrows > n0 and d.dst_s1 != n0 * run:
            return False
    else:
        return False
    length = glen * run
    units = (length + 30) >> 4
    data = 16
    side = data + groups * (units << 4) + 16
    if glen < 2 or units < threads or groups * (units << 4) + 48 + 16 * (nrows + 1) > smem_bytes:
        return False
    src0 = src.va + d.src_off + o * d.src_outer
    dst0 = dst.va + d.dst_off + o * d.dst_outer
    s_first = src0 + j1 * d.src_s1 + j0 * d.src_s0
    d_first = dst0 + j1 * d.dst_s1 + j0 * d.dst_s0
    s_lo, d_lo = s_first % 16, d_first % 16
    stage = np.full(smem_bytes, 0xDD, dtype=np.uint8)
    loaded = np.zeros(smem_bytes, dtype=bool)

    def place(rr):
        i1, i0 = divmod(row0 + rr, n0)
        g, pos = 0, rr
        if across:
            g, pos = (i0, i1 - j1) if groups > 1 else (0, i0 * cols + (i1 - j1))
        return i1, i0, g, pos

    def bulk(at, gaddr, nbytes):
        assert at % 16 == 0 and gaddr % 16 == 0 and nbytes % 16 == 0 and nbytes > 0 and at + nbytes <= smem_bytes
        for c in range(nbytes // 16):
            assert not loaded[at + 16 * c], "two bulk copies land on one staged chunk"
            stage[at + 16 * c:at + 16 * c + 16] = src.read16(gaddr + 16 * c)
            loaded[at + 16 * c:at + 16 * c + 16] = True

    announced = nrows * (run + 16 if s_lo else run)
    arrived = 0
    for rr in range(nrows):
        i1, i0, g, pos = place(rr)
        row = src0 + i1 * d.src_s1 + i0 * d.src_s0 - s_lo
        at = data + 16 * g * units + pos * run
        if not s_lo or pos + 1 == glen:
            n = run + 16 if s_lo else run
            bulk(at, row, n)
            arrived += n
        else:
            bulk(at, row, run)
            bulk(side + 16 * (g * glen + pos + 1), row + run, 16)
            arrived += run + 16
    assert arrived == announced, "the barrier's byte count"
    if s_lo:
        for rr in range(nrows):
            _, _, g, pos = place(rr)
            if pos == 0:
                continue
            at = data + 16 * g * units + pos * run
            sd = side + 16 * (g * glen + pos)
            assert loaded[sd:sd + 16].all() and loaded[at:at + 16].all()
            stage[at:at + s_lo] = stage[sd:sd + s_lo]
    delta = s_lo - d_lo
    sh, shifted = delta % 16, data + 16 * (delta >> 4)
    end = d_lo + length
    c_first, c_last, t = (1 if d_lo else 0), end >> 4, end & 15
    out0 = d_first - d_lo
    for g in range(groups):
        for c in range(c_first, c_last):
            at = shifted + 16 * (g * units + c)
            assert 0 <= at and at + 32 <= smem_bytes, "staging read outside the area"
            assert loaded[at + sh:at + sh + 16].all(), "a staged byte that was never loaded is consumed"
            dst.write(out0 + g * vstride + 16 * c, stage[at + sh:at + sh + 16].copy(), cnt)
        for k in range(32):
            is_tail = k >= 16
            if (k - 16 >= t) if is_tail else (k < d_lo or not d_lo):
                continue
            byte = 16 * c_last + (k - 16) if is_tail else k
            at = data + 16 * g * units + s_lo + byte - d_lo
            assert loaded[at], "a staged byte that was never loaded is consumed"
            dst.write(out0 + g * vstride + byte, stage[at:at + 1], cnt)
    return True


def run_realign_tile_dest_order(d, o, part, src, dst, cnt, smem_bytes=52 << 10, threads=256):
    """The realigning path for SHORT rows that follow one another in the destination a step of n0
    apart, replayed like run_realign_tile.  Returns False, touching nothing, for a tile the kernel
    would not take this way.  Through a misaligned destination every row is loaded into a slot of
    its own; after the wait each slot is completed with the first chunk (two when s_lo > d_lo) of
    the row that follows it in the destination, taken from that row's slot; the stores then walk
    the aligned chunks of every destination run, finding each in its row's slot; the first
    16 - d_lo and last d_lo bytes of a run go out byte by byte.  With an aligned destination and a
    misaligned source that is contiguous along i0, a column of n0 rows arrives as one bulk copy,
    its rows at the source's own pitch, and the same walk stores them."""
    run, n0 = d.run_bytes, d.n0
    row0 = part * d.rows_per_tile
    nrows = min(d.rows_per_tile, d.rows - row0)
    cpr = run >> 4
    if run % 16 or cpr & (cpr - 1) or run >= JOIN_MIN_RUN or d.dst_s1 != run or (n0 > 1 and d.dst_s0 == run):
        return False
    j1, cols = row0 // n0, nrows // n0
    if row0 != j1 * n0 or cols * n0 != nrows or cols < 2:
        return False
    src0 = src.va + d.src_off + o * d.src_outer + j1 * d.src_s1
    dst0 = dst.va + d.dst_off + o * d.dst_outer + j1 * d.dst_s1
    s_lo, d_lo = src0 % 16, dst0 % 16
    pieces = d_lo == 0 and d.src_s0 == run
    if d_lo == 0 and not pieces:
        return False
    pitch = cpr if pieces else cpr + (2 if s_lo > d_lo else 1)
    extra = 1 if pieces else 0
    if (cols * (n0 * cpr + 1) * 16 if pieces else nrows * (pitch << 4)) + 32 > smem_bytes:
        return False
    one_run = n0 == 1 or d.dst_s0 == cols * run
    if one_run and n0 > 1 and cols & (cols - 1):
        return False
    groups, glen = (1, nrows) if one_run else (n0, cols)
    data = 16
    stage = np.full(smem_bytes, 0xDD, dtype=np.uint8)
    loaded = np.zeros(smem_bytes, dtype=bool)

    def bulk(at, g, nbytes):
        assert at % 16 == 0 and g % 16 == 0 and nbytes % 16 == 0 and at + nbytes <= smem_bytes
        for c in range(nbytes // 16):
            assert not loaded[at + 16 * c], "two bulk copies land on one staged chunk"
            stage[at + 16 * c:at + 16 * c + 16] = src.read16(g + 16 * c)
            loaded[at + 16 * c:at + 16 * c + 16] = True

    def slot(rr):                                             # chunk index of row rr's first chunk
        return rr * pitch + (rr // n0) * extra

    if pieces:
        for k1 in range(cols):                                # one bulk copy per column of n0 rows
            bulk(data + 16 * k1 * (n0 * cpr + 1), src0 - s_lo + k1 * d.src_s1, n0 * run + (16 if s_lo else 0))
    else:
        for rr in range(nrows):                               # one bulk copy per row
            k1, i0 = divmod(rr, n0)
            bulk(data + 16 * slot(rr), src0 - s_lo + k1 * d.src_s1 + i0 * d.src_s0, run + 16 if s_lo else run)
    if d_lo:
        snap, snap_loaded = stage.copy(), loaded.copy()       # the fill reads what the copies brought
        for rr in range(nrows):
            k1, i0 = divmod(rr, n0)
            if k1 + 1 < cols:
                nxt = rr + n0
            elif one_run and i0 + 1 < n0:
                nxt = i0 + 1
            else:
                continue
            at, na = data + 16 * (slot(rr) + cpr), data + 16 * slot(nxt)
            assert snap_loaded[na + s_lo:na + 16].all() and (not s_lo or snap_loaded[at:at + s_lo].all())
            stage[at + s_lo:at + 16] = snap[na + s_lo:na + 16]
            loaded[at + s_lo:at + 16] = True
            if s_lo > d_lo:
                assert snap_loaded[na + 16:na + 32].all()
                stage[at + 16:at + 32] = snap[na + 16:na + 32]
                loaded[at + 16:at + 32] = True
    delta = s_lo - d_lo
    sh, shifted = delta % 16, data + 16 * (delta >> 4)
    total = glen * cpr
    off = 1 if d_lo else 0
    out0 = dst0 - d_lo

    def row_of(p, g):
        if one_run and n0 > 1:
            return (p & (cols - 1)) * n0 + (p // cols) + g
        return p * n0 + g

    for g in range(groups):
        out = out0 + g * d.dst_s0
        for m in range(off, total):
            p, c = divmod(m - off, cpr)
            c += off
            at = shifted + 16 * (slot(row_of(p, g)) + c)
            assert 0 <= at and at + 32 <= smem_bytes, "staging read outside the area"
            assert loaded[at + sh:at + sh + 16].all(), "a staged byte that was never loaded is consumed"
            dst.write(out + 16 * m, stage[at + sh:at + sh + 16].copy(), cnt)
        for k in range(16 if d_lo else 0):
            tail = k < d_lo
            p = glen - 1 if tail else 0
            row_byte = run - d_lo + k if tail else k - d_lo
            at = data + 16 * slot(row_of(p, g)) + s_lo + row_byte
            assert loaded[at], "a staged byte that was never loaded is consumed"
            dst.write(out + (16 * total + k if tail else k), stage[at:at + 1], cnt)
    return True


def run_realign_tile(d, o, part, src, dst, cnt, smem_bytes=52 << 10, threads=256):
    """The realigning path of the kernel (rows whose source and destination are not both
    16-byte aligned, all strides multiples of 16), replayed for tile (outer o, part) of
    descriptor d on _Mem buffers: per pass, one aligned bulk load per row into a staging array,
    then aligned 16-byte destination chunks assembled from two staged chunks, partial first /
    last chunks in aligned pieces, and the chunk that two destination-adjacent rows share
    stored once.  Same quantities and formulas as the CUDA code; every staged byte that is
    consumed must have been loaded, every destination byte is counted."""
    assert all(x % 16 == 0 for x in (d.src_s0, d.src_s1, d.dst_s0, d.dst_s1))
    if run_realign_tile_joined(d, o, part, src, dst, cnt, smem_bytes, threads):
        return "joined"
    if run_realign_tile_dest_order(d, o, part, src, dst, cnt, smem_bytes, threads):
        return "destination order"
    column_max = smem_bytes - 64
    row0 = part * d.rows_per_tile
    nrows = min(d.rows_per_tile, d.rows - row0)
    run = d.run_bytes
    column = min(run, column_max)
    units = (column + 30) >> 4
    rows_per_pass = (smem_bytes - 32) // (units << 4)
    assert rows_per_pass >= 1
    src0 = src.va + d.src_off + o * d.src_outer
    dst0 = dst.va + d.dst_off + o * d.dst_outer
    rowoff = lambda r, s0, s1: (r // d.n0) * s1 + (r % d.n0) * s0
    for col0 in range(0, run, column):
        length = min(column, run - col0)
        for r0 in range(0, nrows, rows_per_pass):
            n_rows = min(rows_per_pass, nrows - r0)
            row_base = row0 + r0
            s_lo, d_lo = (src0 + col0) % 16, (dst0 + col0) % 16
            stage = np.full(smem_bytes, 0xDD, dtype=np.uint8)
            loaded = np.zeros(smem_bytes, dtype=bool)
            data = 16
            row_bytes = ((s_lo + length + 15) >> 4) << 4
            for rr in range(n_rows):                          # one bulk copy per row
                g = src0 + col0 - s_lo + rowoff(row_base + rr, d.src_s0, d.src_s1)
                at = data + 16 * rr * units
                assert at + row_bytes <= smem_bytes - 16
                for c in range(row_bytes // 16):
                    stage[at + 16 * c:at + 16 * c + 16] = src.read16(g + 16 * c)
                    loaded[at + 16 * c:at + 16 * c + 16] = True
            delta = s_lo - d_lo
            sh, shifted = delta % 16, data + 16 * (delta >> 4)
            end = d_lo + length
            c_first, c_last = (1 if d_lo else 0), end >> 4

            def chunk(u, lo, hi):
                at = shifted + 16 * u + sh
                assert 0 <= shifted + 16 * u and shifted + 16 * u + 32 <= smem_bytes, "staging read outside the area"
                assert loaded[at + lo:at + hi].all(), "a staged byte that was never loaded is consumed"
                return stage[at:at + 16].copy()

            def out_addr(rr, c):
                return dst0 + col0 - d_lo + rowoff(row_base + rr, d.dst_s0, d.dst_s1) + 16 * c

            for rr in range(n_rows):                          # whole chunks (either thread mapping covers exactly these)
                for c in range(c_first, c_last):
                    dst.write(out_addr(rr, c), chunk(rr * units + c, 0, 16), cnt)
            one_chunk, t = c_last == 0, end & 15
            if not (d_lo or t):
                continue
            if length >= 1024:                                # long rows: heads and tails byte by byte, a thread each
                for rr in range(n_rows):
                    for k in range(32):
                        is_tail = k >= 16
                        valid = (not one_chunk and k - 16 < t) if is_tail else (d_lo <= k < min(end, 16) and bool(d_lo or one_chunk))
                        if not valid:
                            continue
                        byte = 16 * c_last + (k - 16) if is_tail else k
                        at = data + 16 * rr * units + s_lo + byte - d_lo
                        assert loaded[at], "a staged byte that was never loaded is consumed"
                        dst.write(out_addr(rr, 0) + byte, stage[at:at + 1], cnt)
                continue
            adj = 0
            if not one_chunk and t and length == run and run % 16 == 0:
                adj = 1 if (d.n0 > 1 and d.dst_s0 == run) else (d.n0 if d.dst_s1 == run else 0)
            for rr in range(n_rows):                          # partial chunks, one thread per row
                r = row_base + rr
                i0 = r % d.n0
                has_next = bool(adj) and (i0 + 1 < d.n0 if adj == 1 else r + d.n0 < d.rows) and rr + adj < n_rows
                has_prev = bool(adj) and (i0 >= 1 if adj == 1 else r >= d.n0) and rr >= adj
                if (d_lo or one_chunk) and not has_prev:
                    hi = end if one_chunk else 16
                    dst.write(out_addr(rr, 0) + d_lo, chunk(rr * units, d_lo, hi)[d_lo:hi], cnt)
                if not one_chunk and t:
                    tail = chunk(rr * units + c_last, 0, t)
                    if has_next:
                        head = chunk((rr + adj) * units, t, 16)
                        dst.write(out_addr(rr, c_last), np.concatenate([tail[:t], head[t:]]), cnt)
                    else:
                        dst.write(out_addr(rr, c_last), tail[:t], cnt)


def run_realign_tile_mixed(d, o, part, src, dst, cnt, smem_bytes=52 << 10):
    """The realigning path for rows that differ in alignment (a row pitch that is not a multiple
    of 16), replayed like run_realign_tile: one aligned bulk load per row, then every whole
    destination chunk from its own row's two alignments, then each row's partial first and last
    chunk."""
    column_max = smem_bytes - 64
    row0 = part * d.rows_per_tile
    nrows = min(d.rows_per_tile, d.rows - row0)
    run = d.run_bytes
    column = min(run, column_max)
    units = (column + 30) >> 4
    rows_per_pass = (smem_bytes - 32) // (units << 4)
    src0 = src.va + d.src_off + o * d.src_outer
    dst0 = dst.va + d.dst_off + o * d.dst_outer
    rowoff = lambda r, s0, s1: (r // d.n0) * s1 + (r % d.n0) * s0
    data = 16
    for col0 in range(0, run, column):
        length = min(column, run - col0)
        for r0 in range(0, nrows, rows_per_pass):
            n_rows = min(rows_per_pass, nrows - r0)
            stage = np.full(smem_bytes, 0xDD, dtype=np.uint8)
            loaded = np.zeros(smem_bytes, dtype=bool)
            for rr in range(n_rows):
                s = src0 + col0 + rowoff(row0 + r0 + rr, d.src_s0, d.src_s1)
                s_lo = s % 16
                nbytes = ((s_lo + length + 15) >> 4) << 4
                at = data + 16 * rr * units
                assert nbytes <= units * 16 and at + nbytes <= smem_bytes - 16
                for c in range(nbytes // 16):
                    stage[at + 16 * c:at + 16 * c + 16] = src.read16(s - s_lo + 16 * c)
                    loaded[at + 16 * c:at + 16 * c + 16] = True

            def chunk(rr, q, lo, hi):                         # 16 bytes that start q bytes into row rr's staged chunks
                at = data + 16 * rr * units + q
                assert data - 16 <= at - (q % 16) and at - (q % 16) + 32 <= smem_bytes, "staging read outside the area"
                assert loaded[at + lo:at + hi].all(), "a staged byte that was never loaded is consumed"
                return stage[at:at + 16].copy()

            for rr in range(n_rows):
                s = src0 + col0 + rowoff(row0 + r0 + rr, d.src_s0, d.src_s1)
                dp = dst0 + col0 + rowoff(row0 + r0 + rr, d.dst_s0, d.dst_s1)
                s_lo, d_lo = s % 16, dp % 16
                end = d_lo + length
                for c in range(units):                        # whole chunks
                    first = 16 * c - d_lo
                    if first < 0 or first + 16 > length:
                        continue
                    dst.write(dp + first, chunk(rr, s_lo + first, 0, 16), cnt)
                if not (d_lo == 0 and min(end, 16) == 16):    # head
                    hi = min(end, 16)
                    dst.write(dp, chunk(rr, s_lo - d_lo, d_lo, hi)[d_lo:hi], cnt)
                c, t = end >> 4, end & 15                     # tail
                if c and t:
                    dst.write(dp - d_lo + 16 * c, chunk(rr, s_lo + 16 * c - d_lo, 0, t)[:t], cnt)


def planes_of(pool, n_planes):
    per = pool.size // n_planes
    return [pool[i * per:(i + 1) * per] for i in range(n_planes)]


def kv_case(rng, L=2, NB=12, B=4, H=3, D=8, E=2, T=(8, 4, 12), pad_blocks=0):
    shape = (L, B, H, D, E)
    chunk = B * H * D * E
    stride = chunk + pad_blocks
    pool = rng.integers(0, 256, L * 2 * NB * stride, dtype=np.uint8)
    T = np.array(T, dtype=np.int64)
    off = np.concatenate([[0], np.cumsum((T + B - 1) // B)]).astype(np.int64)
    bt = rng.permutation(NB)[:off[-1]].astype(np.int32)
    return shape, NB, stride, pool, T, off, bt


def small_checkpoint(**kw):
    return wl.llama_checkpoint(hidden=64, layers=2, q_heads=8, kv_heads=4, head_dim=8, mlp=96,
                               vocab=160, **kw)


def ck_spec(ck, **kw):
    nbytes = [ck.nbytes(i) for i in range(ck.N)]
    kw.setdefault("blob_bytes", ck.nbytes_total)
    return tc.weights_spec(ck.byte_off, nbytes, ck.E, ck.ndim, ck.shapes, **kw)


def ipc_pack_child(q_in, q_out):
    """Runs in a spawned process: receives a pool another process allocated (torch maps it through
    CUDA IPC), packs from it with this process's own plan and returns the packed bytes."""
    try:
        import torch
        pool_t, shape, pool_args, T, off, bt, packed_l, n = q_in.get()
        pl = tc.pool(*pool_args[0], **pool_args[1])
        plan = tc.tc_plan_create(tc.kv_spec(tc.TC_KV_PACK, shape, src_pool=pl, packed_layout=packed_l, T=T, bt_off=off, bt_src=bt))
        out = torch.zeros(n, dtype=torch.uint8, device="cuda")
        tc.tc_kv_pack(plan, [pool_t], [out])
        torch.cuda.synchronize()
        q_out.put(("ok", out.cpu().numpy()))
        plan.destroy()
        del pool_t
    except Exception as e:  # noqa: BLE001
        q_out.put(("error", repr(e)))
