"""GPU parity: the CUDA path, called through the C ABI, against the CPU oracle, byte for byte.
Everything is copy and indexing, so the bar is exact equality of whole buffers (including
sentinel-filled destinations and red zones around them)."""
import itertools
import os
import time

import numpy as np
import pytest
import torch

import oracle
import paper_2608_06007_b200 as tc
import workloads as wl
from helpers import ck_spec, kv_case, planes_of, small_checkpoint

pytestmark = pytest.mark.gpu
LAYOUTS = [tc.TC_NHD, tc.TC_HND]
RED = 256  # red-zone bytes on both sides of every destination


def dev(a: np.ndarray) -> torch.Tensor:
    return torch.from_numpy(a).cuda()


class Guarded:
    """A device destination of n bytes with sentinel-filled red zones on both sides."""

    def __init__(self, n, fill=0xA5, init=None, shift=0):
        self.n, self.fill, self.shift = n, fill, shift
        self.buf = torch.full((n + 2 * RED + shift,), 0x3C, dtype=torch.uint8, device="cuda")
        self.view = self.buf[RED + shift:RED + shift + n]
        if init is not None:
            self.view.copy_(dev(init))
        else:
            self.view.fill_(fill)

    def ptr(self, off=0):
        return self.view.data_ptr() + off

    def result(self):
        torch.cuda.synchronize()
        host = self.buf.cpu().numpy()
        assert (host[:RED + self.shift] == 0x3C).all() and (host[RED + self.shift + self.n:] == 0x3C).all(), "red zone written"
        return host[RED + self.shift:RED + self.shift + self.n]


def pool_tables(g: Guarded, n_planes, slots):
    per = g.n // n_planes
    return [g.ptr(p * per) for p in range(n_planes)] if slots == "planes" else [g.ptr()]


# --------------------------------------------------------------------------- config 1
@pytest.mark.parametrize("packed_l", LAYOUTS)
def test_config1_pack_then_unpack(packed_l):
    shape, NB, src, dst = wl.config1()
    s = shape.tuple
    pool = np.zeros(2 * NB * shape.chunk_bytes, dtype=np.uint8)
    wl.fill_np(pool, wl.SEED_BASE + 1)
    planes = planes_of(pool, 2)
    want = np.zeros(oracle.packed_nbytes(s, src.T), dtype=np.uint8)
    oracle.kv_pack(s, oracle.NHD, shape.chunk_bytes, planes, src.T, src.bt_off, src.bt, packed_l, want)
    d_pool = dev(pool)
    pl = tc.pool(tc.TC_NHD, NB, 1, plane_stride=NB * shape.chunk_bytes, slot_bytes=pool.size)
    plan = tc.tc_plan_create(tc.kv_spec(tc.TC_KV_PACK, s, src_pool=pl, packed_layout=packed_l, T=src.T, bt_off=src.bt_off, bt_src=src.bt))
    out = Guarded(want.size)
    tc.tc_kv_pack(plan, [d_pool], [out.ptr()])
    got = out.result()
    assert got.size == 1400832 and np.array_equal(got, want)
    # unpack into a fresh pool filled with the 0xA5A5 sentinel, through an independent table
    want_pool = np.full_like(pool, 0xA5)
    oracle.kv_unpack(s, oracle.NHD, shape.chunk_bytes, planes_of(want_pool, 2), dst.T, dst.bt_off, dst.bt, packed_l, want)
    plan2 = tc.tc_plan_create(tc.kv_spec(tc.TC_KV_UNPACK, s, dst_pool=pl, packed_layout=packed_l, T=dst.T, bt_off=dst.bt_off, bt_dst=dst.bt))
    fresh = Guarded(pool.size)
    tc.tc_kv_unpack(plan2, [out.ptr()], [fresh.ptr()])
    assert np.array_equal(fresh.result(), want_pool)
    # idempotent re-execution of both plans gives the same bytes
    tc.tc_kv_pack(plan, [d_pool], [out.ptr()])
    tc.tc_kv_unpack(plan2, [out.ptr()], [fresh.ptr()])
    assert np.array_equal(out.result(), want) and np.array_equal(fresh.result(), want_pool)
    assert plan.stats().launches_per_execute == 1


# --------------------------------------------------------------------------- layouts, tails, tiles
@pytest.mark.parametrize("pool_l,packed_l", list(itertools.product(LAYOUTS, LAYOUTS)))
@pytest.mark.parametrize("slots", ["planes", "one"])
@pytest.mark.parametrize("tile", [0, 2048])
def test_pack_unpack_all_layouts(pool_l, packed_l, slots, tile):
    rng = np.random.default_rng(21)
    # 2 KiB token rows, blocks of 16: several tiles per block with tile=2048, ragged tails
    shape, NB, stride, pool, T, off, bt = kv_case(rng, L=3, NB=40, B=16, H=4, D=64, E=2, T=(37, 0, 100, 5, 16, 200), pad_blocks=0)
    L = shape[0]
    tune = dict(tile_bytes=tile) if tile else None
    want = np.zeros(oracle.packed_nbytes(shape, T), dtype=np.uint8)
    oracle.kv_pack(shape, pool_l, stride, planes_of(pool, L * 2), T, off, bt, packed_l, want)
    d_pool = Guarded(pool.size, init=pool)
    if slots == "planes":
        pl = tc.pool(pool_l, NB, L * 2, block_stride=stride, slot_bytes=pool.size // (L * 2))
    else:
        pl = tc.pool(pool_l, NB, 1, plane_stride=pool.size // (L * 2), block_stride=stride, slot_bytes=pool.size)
    plan = tc.tc_plan_create(tc.kv_spec(tc.TC_KV_PACK, shape, src_pool=pl, packed_layout=packed_l, T=T, bt_off=off, bt_src=bt, tuning=tune))
    out = Guarded(want.size)
    tc.tc_kv_pack(plan, pool_tables(d_pool, L * 2, slots), [out.ptr()])
    assert np.array_equal(out.result(), want)
    assert np.array_equal(d_pool.result(), pool)          # sources are never written
    bt2 = rng.permutation(NB)[:off[-1]].astype(np.int32)
    want_pool = np.full_like(pool, 0xA5)
    oracle.kv_unpack(shape, pool_l, stride, planes_of(want_pool, L * 2), T, off, bt2, packed_l, want)
    plan2 = tc.tc_plan_create(tc.kv_spec(tc.TC_KV_UNPACK, shape, dst_pool=pl, packed_layout=packed_l, T=T, bt_off=off, bt_dst=bt2, tuning=tune))
    fresh = Guarded(pool.size)
    tc.tc_kv_unpack(plan2, [out.ptr()], pool_tables(fresh, L * 2, slots))
    assert np.array_equal(fresh.result(), want_pool)


@pytest.mark.parametrize("H,L", [(1, 5), (2, 3), (4, 6)])
@pytest.mark.parametrize("pool_l,packed_l", list(itertools.product(LAYOUTS, LAYOUTS)))
def test_few_kv_heads_several_planes_per_tile(H, L, pool_l, packed_l):
    """Planes of 4-16 KiB (1, 2, 4 KV heads): a tile moves several planes of one block.  L is
    chosen so that the last tile row of every block is only partly filled; ragged last blocks,
    an empty request, block strides with padding, a pointer shifted by 8 bytes (narrow-vector
    build), and staged windows whose plane ranges are not multiples of the planes per tile."""
    rng = np.random.default_rng(40 + H)
    shape, NB, stride, pool, T, off, bt = kv_case(rng, L=L, NB=70, B=16, H=H, D=128, E=2, T=(300, 16, 0, 37, 5, 512), pad_blocks=256)
    want = np.zeros(oracle.packed_nbytes(shape, T), dtype=np.uint8)
    oracle.kv_pack(shape, pool_l, stride, planes_of(pool, L * 2), T, off, bt, packed_l, want, threads=8)
    pl = tc.pool(pool_l, NB, 1, plane_stride=NB * stride, block_stride=stride)
    plan = tc.tc_plan_create(tc.kv_spec(tc.TC_KV_PACK, shape, src_pool=pl, packed_layout=packed_l, T=T, bt_off=off, bt_src=bt))
    assert plan.descriptors(0)[0].planes_per_tile == min(8 // H, 2 * L)
    d_pool = Guarded(pool.size, init=pool)
    out = Guarded(want.size)
    tc.tc_kv_pack(plan, [d_pool.ptr()], [out.ptr()])
    assert np.array_equal(out.result(), want)
    shifted = Guarded(want.size, shift=8)                      # 8-byte aligned destination: the narrow-vector build
    tc.tc_kv_pack(plan, [d_pool.ptr()], [shifted.ptr()])
    assert np.array_equal(shifted.result(), want)
    bt2 = rng.permutation(NB)[:off[-1]].astype(np.int32)
    want_pool = np.full_like(pool, 0xA5)
    oracle.kv_unpack(shape, pool_l, stride, planes_of(want_pool, L * 2), T, off, bt2, packed_l, want, threads=8)
    plan2 = tc.tc_plan_create(tc.kv_spec(tc.TC_KV_UNPACK, shape, dst_pool=pl, packed_layout=packed_l, T=T, bt_off=off, bt_dst=bt2))
    fresh = Guarded(pool.size)
    tc.tc_kv_unpack(plan2, [out.ptr()], [fresh.ptr()])
    assert np.array_equal(fresh.result(), want_pool)
    want_mig = np.full_like(pool, 0xA5)
    oracle.kv_migrate(shape, pool_l, stride, planes_of(pool, L * 2), pool_l, stride, planes_of(want_mig, L * 2), T, off, bt, bt2, threads=8)
    mig = tc.tc_plan_create(tc.kv_spec(tc.TC_KV_MIGRATE, shape, src_pool=pl, dst_pool=pl, T=T, bt_off=off, bt_src=bt, bt_dst=bt2, tuning=dict(tile_order=1)))
    moved = Guarded(pool.size)
    tc.tc_kv_pack(mig, [d_pool.ptr()], [moved.ptr()])
    assert np.array_equal(moved.result(), want_mig)
    # the same pools addressed through one pointer per plane
    per_plane = tc.pool(pool_l, NB, L * 2, block_stride=stride, slot_bytes=pool.size // (L * 2))
    pp = tc.tc_plan_create(tc.kv_spec(tc.TC_KV_PACK, shape, src_pool=per_plane, packed_layout=packed_l, T=T, bt_off=off, bt_src=bt))
    assert pp.descriptors(0)[0].planes_per_tile == min(8 // H, 2 * L)
    out2 = Guarded(want.size)
    tc.tc_kv_pack(pp, pool_tables(d_pool, L * 2, "planes"), [out2.ptr()])
    assert np.array_equal(out2.result(), want)
    mp = tc.tc_plan_create(tc.kv_spec(tc.TC_KV_MIGRATE, shape, src_pool=per_plane, dst_pool=pl, T=T, bt_off=off, bt_src=bt, bt_dst=bt2))
    moved2 = Guarded(pool.size)
    tc.tc_kv_pack(mp, pool_tables(d_pool, L * 2, "planes"), [moved2.ptr()])
    assert np.array_equal(moved2.result(), want_mig)
    up2 = tc.tc_plan_create(tc.kv_spec(tc.TC_KV_UNPACK, shape, dst_pool=per_plane, packed_layout=packed_l, T=T, bt_off=off, bt_dst=bt2))
    fresh2 = Guarded(pool.size)
    tc.tc_kv_unpack(up2, [out.ptr()], pool_tables(fresh2, L * 2, "planes"))
    assert np.array_equal(fresh2.result(), want_pool)
    # staged: the copy-engine path launches windows of planes
    host = torch.full((want.size,), 0x77, dtype=torch.uint8).pin_memory()
    sp = tc.tc_plan_create(tc.kv_spec(tc.TC_KV_PACK, shape, src_pool=pl, packed_layout=packed_l, T=T, bt_off=off, bt_src=bt, flags=tc.TC_PLAN_STAGED))
    su = tc.tc_plan_create(tc.kv_spec(tc.TC_KV_UNPACK, shape, dst_pool=pl, packed_layout=packed_l, T=T, bt_off=off, bt_dst=bt2, flags=tc.TC_PLAN_STAGED))
    refill = Guarded(pool.size)
    tc.tc_kv_pack(sp, [d_pool.ptr()], [host])
    tc.tc_kv_unpack(su, [host], [refill.ptr()])
    torch.cuda.synchronize()
    assert np.array_equal(host.numpy(), want)
    assert np.array_equal(refill.result(), want_pool)


def test_staged_windows_cut_inside_a_tile_row_of_planes():
    """Two KV heads, six planes, four planes per tile; one request of 184 MB is staged in windows
    of two planes (30.7 MB each), so every window starts and ends inside a tile row."""
    rng = np.random.default_rng(47)
    shape, NB, stride, pool, T, off, bt = kv_case(rng, L=3, NB=3800, B=16, H=2, D=128, E=2, T=(60000, 100))
    L = shape[0]
    want = np.zeros(oracle.packed_nbytes(shape, T), dtype=np.uint8)
    oracle.kv_pack(shape, oracle.NHD, stride, planes_of(pool, L * 2), T, off, bt, oracle.HND, want, threads=8)
    pl = tc.pool(tc.TC_NHD, NB, 1, plane_stride=NB * stride)
    sp = tc.tc_plan_create(tc.kv_spec(tc.TC_KV_PACK, shape, src_pool=pl, packed_layout=tc.TC_HND, T=T, bt_off=off, bt_src=bt, flags=tc.TC_PLAN_STAGED))
    assert sp.descriptors(0)[0].planes_per_tile == 4
    segs = sp.segments(0)
    assert [(sg.outer0, sg.n_outer) for sg in segs[:3]] == [(0, 2), (2, 2), (4, 2)]
    d_pool = dev(pool)
    host = torch.full((want.size,), 0x77, dtype=torch.uint8).pin_memory()
    tc.tc_kv_pack(sp, [d_pool], [host])
    torch.cuda.synchronize()
    assert np.array_equal(host.numpy(), want)
    bt2 = rng.permutation(NB)[:off[-1]].astype(np.int32)
    want_pool = np.full_like(pool, 0xA5)
    oracle.kv_unpack(shape, oracle.NHD, stride, planes_of(want_pool, L * 2), T, off, bt2, oracle.HND, want, threads=8)
    su = tc.tc_plan_create(tc.kv_spec(tc.TC_KV_UNPACK, shape, dst_pool=pl, packed_layout=tc.TC_HND, T=T, bt_off=off, bt_dst=bt2, flags=tc.TC_PLAN_STAGED))
    fresh = Guarded(pool.size)
    tc.tc_kv_unpack(su, [host], [fresh.ptr()])
    assert np.array_equal(fresh.result(), want_pool)


@pytest.mark.parametrize("tune", [dict(tile_order=1), dict(tile_order=2), dict(ctas_per_sm=2), dict(max_ctas=7), dict(tile_bytes=65536), dict(tile_bytes=1024, ctas_per_sm=1, tile_order=1)])
def test_tuning_knobs_change_the_schedule_not_the_bytes(tune):
    rng = np.random.default_rng(29)
    shape, NB, stride, pool, T, off, bt = kv_case(rng, L=3, NB=90, B=32, H=8, D=128, E=2, T=(700, 33, 0, 64, 1200))
    L = shape[0]
    bt2 = rng.permutation(NB)[:off[-1]].astype(np.int32)
    pl = tc.pool(tc.TC_NHD, NB, 1, plane_stride=NB * stride)
    d_pool = dev(pool)
    want = np.zeros(oracle.packed_nbytes(shape, T), dtype=np.uint8)
    oracle.kv_pack(shape, oracle.NHD, stride, planes_of(pool, L * 2), T, off, bt, oracle.HND, want, threads=8)
    out = Guarded(want.size)
    plan = tc.tc_plan_create(tc.kv_spec(tc.TC_KV_PACK, shape, src_pool=pl, packed_layout=tc.TC_HND, T=T, bt_off=off, bt_src=bt, tuning=tune))
    tc.tc_kv_pack(plan, [d_pool], [out.ptr()])
    assert np.array_equal(out.result(), want)
    want_pool = np.full_like(pool, 0xA5)
    oracle.kv_migrate(shape, oracle.NHD, stride, planes_of(pool, L * 2), oracle.NHD, stride, planes_of(want_pool, L * 2), T, off, bt, bt2, threads=8)
    mig = tc.tc_plan_create(tc.kv_spec(tc.TC_KV_MIGRATE, shape, src_pool=pl, dst_pool=pl, T=T, bt_off=off, bt_src=bt, bt_dst=bt2, tuning=tune))
    fresh = Guarded(pool.size)
    tc.tc_kv_pack(mig, [d_pool], [fresh.ptr()])
    assert np.array_equal(fresh.result(), want_pool)
    if "max_ctas" in tune:
        assert plan.stats().grid[0] == 7


@pytest.mark.parametrize("E,D,shift", [(1, 7, 0), (2, 5, 0), (4, 3, 0), (8, 3, 0), (2, 64, 2), (2, 64, 4), (2, 64, 8), (1, 33, 1)])
def test_odd_shapes_and_misaligned_pointers_fall_back_to_narrow_vectors(E, D, shift):
    rng = np.random.default_rng(22)
    shape, NB, stride, pool, T, off, bt = kv_case(rng, L=2, NB=20, B=4, H=3, D=D, E=E, T=(9, 1, 0, 16, 7), pad_blocks=E * 3)
    L = shape[0]
    for pool_l, packed_l in itertools.product(LAYOUTS, LAYOUTS):
        want = np.zeros(oracle.packed_nbytes(shape, T), dtype=np.uint8)
        oracle.kv_pack(shape, pool_l, stride, planes_of(pool, L * 2), T, off, bt, packed_l, want)
        d_pool = Guarded(pool.size, init=pool, shift=shift)
        pl = tc.pool(pool_l, NB, L * 2, block_stride=stride)
        plan = tc.tc_plan_create(tc.kv_spec(tc.TC_KV_PACK, shape, src_pool=pl, packed_layout=packed_l, T=T, bt_off=off, bt_src=bt))
        out = Guarded(want.size, shift=shift)
        tc.tc_kv_pack(plan, pool_tables(d_pool, L * 2, "planes"), [out.ptr()])
        assert np.array_equal(out.result(), want)
        want_pool = np.full_like(pool, 0xA5)
        oracle.kv_unpack(shape, pool_l, stride, planes_of(want_pool, L * 2), T, off, bt, packed_l, want)
        plan2 = tc.tc_plan_create(tc.kv_spec(tc.TC_KV_UNPACK, shape, dst_pool=pl, packed_layout=packed_l, T=T, bt_off=off, bt_dst=bt))
        fresh = Guarded(pool.size, shift=shift)
        tc.tc_kv_unpack(plan2, [out.ptr()], pool_tables(fresh, L * 2, "planes"))
        assert np.array_equal(fresh.result(), want_pool)


# --------------------------------------------------------------------------- migrate, mixed, pinned host
@pytest.mark.parametrize("src_l,dst_l", list(itertools.product(LAYOUTS, LAYOUTS)))
def test_migrate_pool_to_pool(src_l, dst_l):
    rng = np.random.default_rng(23)
    shape, NB, stride, pool, T, off, bt = kv_case(rng, L=4, NB=48, B=32, H=2, D=128, E=2, T=(512, 33, 1, 300, 64))
    L, B, H, D, E = shape
    NB2 = NB + 5
    bt2 = rng.permutation(NB2)[:off[-1]].astype(np.int32)
    want = np.full(L * 2 * NB2 * stride, 0xA5, dtype=np.uint8)
    oracle.kv_migrate(shape, src_l, stride, planes_of(pool, L * 2), dst_l, stride, planes_of(want, L * 2), T, off, bt, bt2, threads=4)
    sp = tc.pool(src_l, NB, 1, plane_stride=NB * stride)
    dp = tc.pool(dst_l, NB2, 1, plane_stride=NB2 * stride)
    plan = tc.tc_plan_create(tc.kv_spec(tc.TC_KV_MIGRATE, shape, src_pool=sp, dst_pool=dp, T=T, bt_off=off, bt_src=bt, bt_dst=bt2))
    out = Guarded(want.size)
    tc.tc_kv_pack(plan, [dev(pool)], [out.ptr()])
    assert np.array_equal(out.result(), want)


@pytest.mark.parametrize("order", [tc.TC_REQUEST_MAJOR, tc.TC_LAYER_MAJOR])
@pytest.mark.parametrize("packed_l", LAYOUTS)
def test_head_slice_view_and_layer_major_order(order, packed_l):
    """A tensor-parallel consumer's view: 2 of 8 KV heads of every request, optionally with the
    packed buffer ordered layer-major; unpacking writes those heads only."""
    rng = np.random.default_rng(27)
    shape, NB, stride, pool, T, off, bt = kv_case(rng, L=3, NB=120, B=16, H=8, D=128, E=2, T=(300, 16, 45, 0, 700))
    L = shape[0]
    h0, hs = 4, 2
    kw = dict(order=order, head_begin=h0, head_count=hs)
    want = np.zeros(oracle.packed_nbytes(shape, T, hs), dtype=np.uint8)
    oracle.kv_pack(shape, oracle.NHD, stride, planes_of(pool, L * 2), T, off, bt, packed_l, want, threads=4, **kw)
    pl = tc.pool(tc.TC_NHD, NB, 1, plane_stride=NB * stride)
    lib_kw = dict(packed_layout=packed_l, packed_order=order, head_begin=h0, head_count=hs, T=T, bt_off=off)
    plan = tc.tc_plan_create(tc.kv_spec(tc.TC_KV_PACK, shape, src_pool=pl, bt_src=bt, **lib_kw))
    out = Guarded(want.size)
    tc.tc_kv_pack(plan, [dev(pool)], [out.ptr()])
    assert np.array_equal(out.result(), want)
    bt2 = rng.permutation(NB)[:off[-1]].astype(np.int32)
    want_pool = np.full_like(pool, 0xA5)
    oracle.kv_unpack(shape, oracle.NHD, stride, planes_of(want_pool, L * 2), T, off, bt2, packed_l, want, threads=4, **kw)
    plan2 = tc.tc_plan_create(tc.kv_spec(tc.TC_KV_UNPACK, shape, dst_pool=pl, bt_dst=bt2, **lib_kw))
    fresh = Guarded(pool.size)
    tc.tc_kv_unpack(plan2, [out.ptr()], [fresh.ptr()])
    assert np.array_equal(fresh.result(), want_pool)


def test_same_pool_compaction_in_place():
    rng = np.random.default_rng(26)
    shape, NB, stride, pool, T, off, bt = kv_case(rng, L=3, NB=200, B=16, H=8, D=128, E=2, T=(300, 16, 45, 700))
    L = shape[0]
    n = int(off[-1])
    bt = (rng.permutation(NB - n)[:n] + n).astype(np.int32)
    dst = np.arange(n, dtype=np.int32)
    want = pool.copy()
    oracle.kv_migrate(shape, oracle.NHD, stride, planes_of(pool, L * 2), oracle.NHD, stride, planes_of(want, L * 2), T, off, bt, dst, threads=4)
    pl = tc.pool(tc.TC_NHD, NB, 1, plane_stride=NB * stride)
    plan = tc.tc_plan_create(tc.kv_spec(tc.TC_KV_MIGRATE, shape, src_pool=pl, dst_pool=pl, T=T, bt_off=off, bt_src=bt, bt_dst=dst, flags=tc.TC_PLAN_SAME_POOL))
    buf = Guarded(pool.size, init=pool)
    tc.tc_kv_pack(plan, [buf.ptr()], [buf.ptr()])
    assert np.array_equal(buf.result(), want)


@pytest.mark.parametrize("flags", [0, tc.TC_PLAN_STAGED, tc.TC_PLAN_STAGED | tc.TC_PLAN_OFFLOAD_ZERO_COPY])
def test_mixed_plan_offload_and_reload_through_pinned_host_pool(flags):
    """Device NHD pool <-> pinned page-first HND host pool, both directions of one plan on two
    streams; the kernels store into / load from host memory directly."""
    shape = wl.KVShape(L=2, B=16, H=8, D=128, E=2)
    s = shape.tuple
    NBd, NBh = 96, 160
    step = next(wl.config5(NB_dev=NBd, NB_host=NBh, sessions=12, steps=1, shape=shape, p=0.4, max_prefix=6, max_new=3))
    chunk = shape.chunk_bytes
    devp = np.zeros(4 * NBd * chunk, dtype=np.uint8)
    hostp = np.zeros(NBh * 4 * chunk, dtype=np.uint8)
    wl.fill_np(devp, 1)
    wl.fill_np(hostp, 2)
    want_dev, want_host = devp.copy(), hostp.copy()
    hp = lambda a: [a[p * chunk:] for p in range(4)]
    oracle.kv_migrate(s, oracle.NHD, chunk, planes_of(devp, 4), oracle.HND, 4 * chunk, hp(want_host), step.offload_T, step.offload_off, step.offload_dev, step.offload_host)
    oracle.kv_migrate(s, oracle.HND, 4 * chunk, hp(hostp), oracle.NHD, chunk, planes_of(want_dev, 4), step.reload_T, step.reload_off, step.reload_host, step.reload_dev)
    d_dev = dev(devp)
    h_host = torch.from_numpy(hostp.copy()).pin_memory()
    spec = tc.kv_spec(tc.TC_KV_MIXED, s, src_pool=tc.pool(tc.TC_NHD, NBd, 1, plane_stride=NBd * chunk, slot_bytes=devp.size),
                      dst_pool=tc.pool(tc.TC_HND, NBh, 1, plane_stride=chunk, block_stride=4 * chunk, slot_bytes=hostp.size),
                      T=step.offload_T, bt_off=step.offload_off, bt_src=step.offload_dev, bt_dst=step.offload_host,
                      reload=dict(T=step.reload_T, bt_off=step.reload_off, bt_src=step.reload_host, bt_dst=step.reload_dev), flags=flags)
    plan = tc.tc_plan_create(spec)
    assert plan.stats().path[0] == (3 if flags == tc.TC_PLAN_STAGED else 1) and plan.stats().path[1] == (3 if flags else 1)
    s1, s2 = torch.cuda.Stream(), torch.cuda.Stream()
    torch.cuda.synchronize()
    tc.tc_kv_pack(plan, [d_dev], [h_host], stream=s1)
    tc.tc_kv_unpack(plan, [h_host], [d_dev], stream=s2)
    torch.cuda.synchronize()
    assert np.array_equal(d_dev.cpu().numpy(), want_dev)
    assert np.array_equal(h_host.numpy(), want_host)


def test_pack_to_pinned_host_hnd_and_reload():
    rng = np.random.default_rng(24)
    shape, NB, stride, pool, T, off, bt = kv_case(rng, L=2, NB=64, B=16, H=8, D=128, E=2, T=(700, 16, 45, 130))
    L = shape[0]
    want = np.zeros(oracle.packed_nbytes(shape, T), dtype=np.uint8)
    oracle.kv_pack(shape, oracle.NHD, stride, planes_of(pool, L * 2), T, off, bt, oracle.HND, want, threads=4)
    pl = tc.pool(tc.TC_NHD, NB, 1, plane_stride=NB * stride)
    host = torch.zeros(want.size, dtype=torch.uint8).pin_memory()
    plan = tc.tc_plan_create(tc.kv_spec(tc.TC_KV_PACK, shape, src_pool=pl, packed_layout=tc.TC_HND, T=T, bt_off=off, bt_src=bt, tuning=dict(max_ctas=32)))
    assert plan.stats().grid[0] <= 32
    tc.tc_kv_pack(plan, [dev(pool)], [host])
    torch.cuda.synchronize()
    assert np.array_equal(host.numpy(), want)
    bt2 = rng.permutation(NB)[:off[-1]].astype(np.int32)
    want_pool = np.full_like(pool, 0xA5)
    oracle.kv_unpack(shape, oracle.NHD, stride, planes_of(want_pool, L * 2), T, off, bt2, oracle.HND, want, threads=4)
    plan2 = tc.tc_plan_create(tc.kv_spec(tc.TC_KV_UNPACK, shape, dst_pool=pl, packed_layout=tc.TC_HND, T=T, bt_off=off, bt_dst=bt2))
    fresh = Guarded(pool.size)
    tc.tc_kv_unpack(plan2, [host], [fresh.ptr()])
    assert np.array_equal(fresh.result(), want_pool)


def test_zero_copy_offload_and_reload_through_a_misaligned_pinned_buffer():
    """The packed buffer is a view at an odd offset of a pinned host allocation: the realigning
    path then stores to and bulk-loads from host memory over the link."""
    rng = np.random.default_rng(26)
    shape, NB, stride, pool, T, off, bt = kv_case(rng, L=2, NB=64, B=16, H=8, D=128, E=2, T=(300, 16, 45))
    L = shape[0]
    want = np.zeros(oracle.packed_nbytes(shape, T), dtype=np.uint8)
    oracle.kv_pack(shape, oracle.NHD, stride, planes_of(pool, L * 2), T, off, bt, oracle.HND, want)
    pl = tc.pool(tc.TC_NHD, NB, 1, plane_stride=NB * stride)
    raw = torch.full((want.size + 64,), 0x3C, dtype=torch.uint8).pin_memory()
    for shift in (2, 9):
        raw.fill_(0x3C)
        host = raw[shift:shift + want.size]
        plan = tc.tc_plan_create(tc.kv_spec(tc.TC_KV_PACK, shape, src_pool=pl, packed_layout=tc.TC_HND, T=T, bt_off=off, bt_src=bt))
        tc.tc_kv_pack(plan, [dev(pool)], [host.data_ptr()])
        torch.cuda.synchronize()
        assert np.array_equal(host.numpy(), want)
        assert bool((raw[:shift] == 0x3C).all()) and bool((raw[shift + want.size:] == 0x3C).all())
        bt2 = rng.permutation(NB)[:off[-1]].astype(np.int32)
        want_pool = np.full_like(pool, 0xA5)
        oracle.kv_unpack(shape, oracle.NHD, stride, planes_of(want_pool, L * 2), T, off, bt2, oracle.HND, want)
        plan2 = tc.tc_plan_create(tc.kv_spec(tc.TC_KV_UNPACK, shape, dst_pool=pl, packed_layout=tc.TC_HND, T=T, bt_off=off, bt_dst=bt2))
        fresh = Guarded(pool.size)
        tc.tc_kv_unpack(plan2, [host.data_ptr()], [fresh.ptr()])
        assert np.array_equal(fresh.result(), want_pool)
    assert tc.tc_device_status() == 0


@pytest.mark.parametrize("packed_l", LAYOUTS)
@pytest.mark.parametrize("order", [tc.TC_REQUEST_MAJOR, tc.TC_LAYER_MAJOR])
def test_staged_offload_and_reload_through_the_copy_engines(packed_l, order):
    """TC_PLAN_STAGED: packed buffer in pinned host memory, moved by the copy engines through
    the device staging ring; one request is larger than a staging buffer (cut at planes), the
    small ones share a segment.  Run twice to reuse ring buffers across calls."""
    rng = np.random.default_rng(25)
    shape, NB, stride, pool, T, off, bt = kv_case(rng, L=4, NB=400, B=16, H=8, D=128, E=2, T=(5000, 37, 0, 100, 700))
    L = shape[0]
    want = np.zeros(oracle.packed_nbytes(shape, T), dtype=np.uint8)
    oracle.kv_pack(shape, oracle.NHD, stride, planes_of(pool, L * 2), T, off, bt, packed_l, want, order=order, threads=8)
    pl = tc.pool(tc.TC_NHD, NB, 1, plane_stride=NB * stride)
    d_pool = dev(pool)
    plan = tc.tc_plan_create(tc.kv_spec(tc.TC_KV_PACK, shape, src_pool=pl, packed_layout=packed_l, packed_order=order, T=T, bt_off=off, bt_src=bt, flags=tc.TC_PLAN_STAGED))
    assert plan.stats().path[0] == 3 and plan.stats().launches_per_execute == (3 if order == tc.TC_REQUEST_MAJOR else 2)
    bt2 = rng.permutation(NB)[:off[-1]].astype(np.int32)
    want_pool = np.full_like(pool, 0xA5)
    oracle.kv_unpack(shape, oracle.NHD, stride, planes_of(want_pool, L * 2), T, off, bt2, packed_l, want, order=order, threads=8)
    plan2 = tc.tc_plan_create(tc.kv_spec(tc.TC_KV_UNPACK, shape, dst_pool=pl, packed_layout=packed_l, packed_order=order, T=T, bt_off=off, bt_dst=bt2, flags=tc.TC_PLAN_STAGED))
    stream = torch.cuda.Stream()
    for _ in range(2):
        host = torch.full((want.size + 4096,), 0x77, dtype=torch.uint8).pin_memory()
        fresh = Guarded(pool.size)
        torch.cuda.synchronize()
        tc.tc_kv_pack(plan, [d_pool], [host], stream.cuda_stream)
        tc.tc_kv_unpack(plan2, [host], [fresh.ptr()], stream.cuda_stream)   # ordered after the pack on the same stream
        stream.synchronize()
        assert np.array_equal(host.numpy()[:want.size], want)
        assert (host.numpy()[want.size:] == 0x77).all()
        assert np.array_equal(fresh.result(), want_pool)
    plan.destroy()
    plan2.destroy()


# --------------------------------------------------------------------------- weights
@pytest.mark.parametrize("variant", ["tight", "permuted_misaligned"])
def test_weights_full_and_every_shard(variant):
    ck = small_checkpoint() if variant == "tight" else small_checkpoint(order_seed=3, lead_pad=2)
    blob = np.zeros(ck.nbytes_total + (ck.nbytes_total & 1), dtype=np.uint8)
    wl.fill_np(blob, 5, "normal")
    blob = blob[:ck.nbytes_total]
    d_blob = dev(blob)
    for world in (1, 4):
        for rank in range(world):
            split = ck.split_dim if world > 1 else np.full(ck.N, -1)
            sizes = [ck.nbytes(i) // (world if split[i] >= 0 else 1) for i in range(ck.N)]
            want = [np.zeros(n, dtype=np.uint8) for n in sizes]
            oracle.weights(ck.byte_off, ck.E, ck.shapes, split, rank, world, blob, want)
            plan = tc.tc_plan_create(ck_spec(ck, split_dim=split, rank=rank, world=world, tuning=dict(tile_bytes=4096)))
            outs = [Guarded(n, fill=0xEE) for n in sizes]
            tc.tc_weights_materialize(plan, d_blob, [o.ptr() for o in outs])
            for i in range(ck.N):
                assert np.array_equal(outs[i].result(), want[i]), (ck.names[i], world, rank)


def test_tp_resharding_8_to_2_and_2_to_8_on_the_gpu():
    """A checkpoint saved as W shard blobs, loaded at another TP degree.  8 -> 2: rank r' of 2
    gathers four source shards into one buffer (dst_off / dst_stride windows, one plan per source
    blob).  2 -> 8: rank r' of 8 takes a quarter of one source shard.  The expected bytes are the
    oracle's direct shard of the FULL tensor at the new degree."""
    rng = np.random.default_rng(8)
    shp, E = (512, 768), 2                                 # rows of 1536 B; eighths are 192 B pieces
    full = rng.integers(0, 256, shp[0] * shp[1] * E, dtype=np.uint8)
    for dim in (0, 1):
        def shard(rank, world):
            out = np.zeros(full.size // world, dtype=np.uint8)
            oracle.weights([0], [E], [[shp[0], shp[1], 1, 1]], [dim], rank, world, full, [out])
            return out
        sshape = lambda world: [shp[0] // world if dim == 0 else shp[0], shp[1] // world if dim == 1 else shp[1], 1, 1]
        for r2 in range(2):                                # 8 -> 2
            want = shard(r2, 2)
            got = Guarded(want.size, fill=0xEE)
            d2, s8 = sshape(2), sshape(8)
            keep = []
            for k in range(4):
                src_blob = shard(4 * r2 + k, 8)
                off = k * src_blob.size if dim == 0 else k * s8[1] * E
                spec = tc.weights_spec([0], [src_blob.size], [E], [2], [s8], blob_bytes=src_blob.size, dst_slot=[0], dst_off=[off],
                                       dst_stride=[[d2[1] * E, E, E, E]], n_dst=1, dst_bytes=[want.size], tuning=dict(tile_bytes=4096))
                plan = tc.tc_plan_create(spec)
                d_src = dev(src_blob)
                tc.tc_weights_materialize(plan, d_src, [got.ptr()])
                keep.append((plan, d_src))
            assert np.array_equal(got.result(), want), (dim, r2)
        for r8 in range(8):                                # 2 -> 8
            src_blob = shard(r8 // 4, 2)
            want = shard(r8, 8)
            got = Guarded(want.size, fill=0xEE)
            plan = tc.tc_plan_create(tc.weights_spec([0], [src_blob.size], [E], [2], [sshape(2)], split_dim=[dim], rank=r8 % 4, world=4,
                                                     blob_bytes=src_blob.size, tuning=dict(tile_bytes=4096)))
            tc.tc_weights_materialize(plan, dev(src_blob), [got.ptr()])
            assert np.array_equal(got.result(), want), (dim, r8)


def test_weights_from_a_pinned_blob_zero_copy_and_staged():
    ck = wl.llama_checkpoint(hidden=512, layers=3, q_heads=8, kv_heads=4, head_dim=64, mlp=2048, vocab=70000)   # 190 MB: several staging buffers
    blob = np.zeros(ck.nbytes_total, dtype=np.uint8)
    wl.fill_np(blob, 9, "normal")
    h_blob = torch.from_numpy(blob).pin_memory()
    nbytes = [ck.nbytes(i) for i in range(ck.N)]
    want = [np.zeros(n, dtype=np.uint8) for n in nbytes]
    oracle.weights(ck.byte_off, ck.E, ck.shapes, np.full(ck.N, -1), 0, 1, blob, want, threads=8)
    want_sums = oracle.weights_checksum(ck.byte_off, ck.E, ck.shapes, np.full(ck.N, -1), 0, 1, blob)
    for flags in (0, tc.TC_PLAN_STAGED, tc.TC_PLAN_STAGED | tc.TC_PLAN_CHECKSUM):
        plan = tc.tc_plan_create(tc.weights_spec(ck.byte_off, nbytes, ck.E, ck.ndim, ck.shapes, blob_bytes=ck.nbytes_total, flags=flags))
        st = plan.stats()
        assert st.path[0] == (3 if flags & tc.TC_PLAN_STAGED else 1)
        if flags & tc.TC_PLAN_STAGED:
            assert st.launches_per_execute >= 3
        outs = [Guarded(n, fill=0xEE) for n in nbytes]
        if flags & tc.TC_PLAN_CHECKSUM:
            sums = torch.zeros(ck.N, dtype=torch.int64, device="cuda")
            tc.tc_weights_materialize_checksum(plan, h_blob, [o.ptr() for o in outs], sums)
            torch.cuda.synchronize()
            assert np.array_equal(sums.cpu().numpy().view(np.uint64), want_sums)
        else:
            tc.tc_weights_materialize(plan, h_blob, [o.ptr() for o in outs])
        for i in range(ck.N):
            assert np.array_equal(outs[i].result(), want[i]), (ck.names[i], flags)
    # a shard reads strided slices: it stays on the zero-copy path even when staging is asked for
    plan = tc.tc_plan_create(tc.weights_spec(ck.byte_off, nbytes, ck.E, ck.ndim, ck.shapes, split_dim=ck.split_dim, rank=1, world=4,
                                             blob_bytes=ck.nbytes_total, flags=tc.TC_PLAN_STAGED))
    assert plan.stats().path[0] == 1
    sizes = [n // (4 if ck.split_dim[i] >= 0 else 1) for i, n in enumerate(nbytes)]
    want = [np.zeros(n, dtype=np.uint8) for n in sizes]
    oracle.weights(ck.byte_off, ck.E, ck.shapes, ck.split_dim, 1, 4, blob, want, threads=8)
    outs = [Guarded(n, fill=0xEE) for n in sizes]
    tc.tc_weights_materialize(plan, h_blob, [o.ptr() for o in outs])
    for i in range(ck.N):
        assert np.array_equal(outs[i].result(), want[i]), ck.names[i]


def test_moe_checkpoint_many_tensors_and_expert_stacking():
    """A MoE-shaped checkpoint: (a) 1 500+ tensors, one destination each - the pointer table of
    the launch grows to thousands of slots; (b) transform_into with expert stacking: the gate and
    up matrices of all experts of a layer land in one fused [experts, 2*moe_mlp/W, hidden] buffer
    as rank r's shard, the down matrices in one [experts, hidden, moe_mlp/W] buffer (strided)."""
    ck = wl.moe_checkpoint(hidden=64, layers=4, experts=128, moe_mlp=32)
    assert ck.N > 1500
    blob = np.zeros(ck.nbytes_total, dtype=np.uint8)
    wl.fill_np(blob, 11, "normal")
    d_blob = dev(blob)
    nbytes = [ck.nbytes(i) for i in range(ck.N)]
    W, rank = 2, 1
    sizes = [n // (W if ck.split_dim[i] >= 0 else 1) for i, n in enumerate(nbytes)]
    want = [np.zeros(n, dtype=np.uint8) for n in sizes]
    oracle.weights(ck.byte_off, ck.E, ck.shapes, ck.split_dim, rank, W, blob, want)
    plan = tc.tc_plan_create(tc.weights_spec(ck.byte_off, nbytes, ck.E, ck.ndim, ck.shapes, split_dim=ck.split_dim, rank=rank, world=W, blob_bytes=ck.nbytes_total))
    arena = Guarded(sum(sizes), fill=0xEE)
    offs = np.concatenate([[0], np.cumsum(sizes)])
    tc.tc_weights_materialize(plan, d_blob, [arena.ptr(int(o)) for o in offs[:-1]])
    got = arena.result()
    for i in range(ck.N):
        assert np.array_equal(got[offs[i]:offs[i + 1]], want[i]), ck.names[i]
    # (b) expert stacking for layer 2
    experts, mlp, hidden, E = 128, 32, 64, 2
    ids, slot, doff, dstride = [], [], [], []
    gu_row = hidden * E                     # one row of a gate/up shard
    gu_exp = 2 * (mlp // W) * gu_row        # one expert of the fused gate_up buffer
    dn_exp = hidden * (mlp // W) * E        # one expert of the stacked down buffer
    for e in range(experts):
        for k, nm in enumerate(("gate_proj", "up_proj")):
            ids.append(ck.names.index(f"layers.2.experts.{e}.{nm}"))
            slot.append(0)
            doff.append(e * gu_exp + k * (mlp // W) * gu_row)
            dstride.append([gu_row, E, E, E])
        ids.append(ck.names.index(f"layers.2.experts.{e}.down_proj"))
        slot.append(1)
        doff.append(e * dn_exp)
        dstride.append([(mlp // W) * E, E, E, E])
    ids = np.array(ids)
    nb = [nbytes[i] for i in ids]
    spec = tc.weights_spec(ck.byte_off[ids], nb, ck.E[ids], ck.ndim[ids], ck.shapes[ids], split_dim=ck.split_dim[ids], rank=rank, world=W,
                           blob_bytes=ck.nbytes_total, dst_slot=slot, dst_off=doff, dst_stride=dstride, n_dst=2, dst_bytes=[experts * gu_exp, experts * dn_exp])
    gate_up, down = Guarded(experts * gu_exp), Guarded(experts * dn_exp)
    tc.tc_weights_materialize(tc.tc_plan_create(spec), d_blob, [gate_up.ptr(), down.ptr()])
    want_gu, want_dn = np.full(experts * gu_exp, 0xA5, dtype=np.uint8), np.full(experts * dn_exp, 0xA5, dtype=np.uint8)
    oracle.weights(ck.byte_off[ids], ck.E[ids], ck.shapes[ids], ck.split_dim[ids], rank, W, blob,
                   [want_gu if s_ == 0 else want_dn for s_ in slot], dst_off=doff, dst_stride=dstride)
    assert np.array_equal(gate_up.result(), want_gu) and np.array_equal(down.result(), want_dn)
    assert not (want_gu == 0xA5).all()


def test_weights_streamed_from_a_file(tmp_path):
    """Cold path: the blob sits in a file behind a header; chunks travel file -> pinned ring ->
    staging ring -> kernel.  Full checkpoint (with fused checksums) and a shard whose strided
    slices stream as covering ranges."""
    ck = wl.llama_checkpoint(hidden=512, layers=3, q_heads=8, kv_heads=4, head_dim=64, mlp=2048, vocab=70000)   # 190 MB: several chunks
    blob = np.zeros(ck.nbytes_total, dtype=np.uint8)
    wl.fill_np(blob, 9, "normal")
    header = 4099                                             # the blob need not start on any boundary of the file
    path = tmp_path / "checkpoint.bin"
    with open(path, "wb") as f:
        f.write(bytes(header))
        f.write(blob.tobytes())
    nbytes = [ck.nbytes(i) for i in range(ck.N)]
    fd = os.open(path, os.O_RDONLY)
    try:
        for world, rank in ((1, 0), (4, 1), (4, 3)):
            split = ck.split_dim if world > 1 else np.full(ck.N, -1)
            sizes = [n // (world if split[i] >= 0 else 1) for i, n in enumerate(nbytes)]
            want = [np.zeros(n, dtype=np.uint8) for n in sizes]
            oracle.weights(ck.byte_off, ck.E, ck.shapes, split, rank, world, blob, want, threads=8)
            want_sums = oracle.weights_checksum(ck.byte_off, ck.E, ck.shapes, split, rank, world, blob)
            plan = tc.tc_plan_create(tc.weights_spec(ck.byte_off, nbytes, ck.E, ck.ndim, ck.shapes, split_dim=split, rank=rank, world=world,
                                                     blob_bytes=ck.nbytes_total, flags=tc.TC_PLAN_STREAM | tc.TC_PLAN_CHECKSUM))
            st = plan.stats()
            assert st.path[0] == 3 and st.launches_per_execute >= 3
            sums = torch.full((ck.N,), -1, dtype=torch.int64, device="cuda")
            for rep in range(2):                               # the second pass reuses every ring buffer
                outs = [Guarded(n, fill=0xEE) for n in sizes]
                tc.tc_weights_materialize_file(plan, fd, header, [o.ptr() for o in outs], checksums=sums if rep else None)
                for i in range(ck.N):
                    assert np.array_equal(outs[i].result(), want[i]), (ck.names[i], world, rank, rep)
            assert np.array_equal(sums.cpu().numpy().view(np.uint64), want_sums)
            # the same chunked plan also takes the blob from pinned memory
            h_blob = torch.from_numpy(blob).pin_memory()
            outs = [Guarded(n, fill=0xEE) for n in sizes]
            tc.tc_weights_materialize(plan, h_blob, [o.ptr() for o in outs])
            for i in range(ck.N):
                assert np.array_equal(outs[i].result(), want[i]), (ck.names[i], world, rank, "pinned")
        # the file ends early: reported, nothing hangs, the context stays usable
        with pytest.raises(tc.TensorCastError) as e:
            tc.tc_weights_materialize_file(plan, fd, header + (100 << 20), [o.ptr() for o in outs])
        assert e.value.status == tc.TC_ERR_IO and "ends" in str(e.value)
        torch.cuda.synchronize()
        plain = tc.tc_plan_create(tc.weights_spec(ck.byte_off, nbytes, ck.E, ck.ndim, ck.shapes, blob_bytes=ck.nbytes_total, flags=tc.TC_PLAN_STAGED))
        full = [Guarded(n, fill=0xEE) for n in nbytes]
        with pytest.raises(tc.TensorCastError) as e:
            tc.tc_weights_materialize_file(plain, fd, header, [o.ptr() for o in full])
        assert e.value.status == tc.TC_ERR_KIND
        with pytest.raises(tc.TensorCastError) as e:
            tc.tc_weights_materialize_file(plan, -1, 0, [o.ptr() for o in outs])
        assert e.value.status == tc.TC_ERR_INVALID_ARG
    finally:
        os.close(fd)


def test_weights_transform_into_fused_and_strided_targets():
    ck = small_checkpoint()
    blob = np.zeros(ck.nbytes_total, dtype=np.uint8)
    wl.fill_np(blob, 6, "normal")
    ids = [ck.names.index(f"layers.1.{n}_proj") for n in "qkv"]
    sizes = [ck.nbytes(i) for i in ids]
    offs = np.concatenate([[0], np.cumsum(sizes)])
    spec = tc.weights_spec(ck.byte_off[ids], sizes, ck.E[ids], ck.ndim[ids], ck.shapes[ids], blob_bytes=blob.size,
                           dst_slot=[0, 0, 0], dst_off=offs[:3], n_dst=1, dst_bytes=[offs[-1]])
    fused = Guarded(int(offs[-1]))
    tc.tc_weights_materialize(tc.tc_plan_create(spec), dev(blob), [fused.ptr()])
    want = np.zeros(offs[-1], dtype=np.uint8)
    oracle.weights(ck.byte_off[ids], ck.E[ids], ck.shapes[ids], [-1] * 3, 0, 1, blob, [want] * 3, dst_off=offs[:3])
    assert np.array_equal(fused.result(), want)
    # middle-dim split into a strided window of a larger target
    rng = np.random.default_rng(4)
    full = rng.integers(0, 2 ** 32, (4, 6, 5), dtype=np.uint32)
    blob2 = np.concatenate([np.zeros(4, dtype=np.uint8), full.reshape(-1).view(np.uint8)])
    spec = tc.weights_spec([4], [full.nbytes], [4], [3], [[4, 6, 5, 1]], split_dim=[1], rank=2, world=3, blob_bytes=blob2.size,
                           dst_slot=[0], dst_off=[12], dst_stride=[[64, 32, 4, 4]], n_dst=1, dst_bytes=[256])
    target = Guarded(256, fill=0)
    tc.tc_weights_materialize(tc.tc_plan_create(spec), dev(blob2), [target.ptr()])
    want2 = np.zeros(256, dtype=np.uint8)
    oracle.weights([4], [4], [[4, 6, 5, 1]], [1], 2, 3, blob2, [want2], dst_off=[12], dst_stride=[[64, 32, 4, 4]])
    assert np.array_equal(target.result(), want2)


def test_weights_checksum_fused_with_the_copy():
    ck = wl.llama_checkpoint(hidden=256, layers=2, q_heads=8, kv_heads=4, head_dim=32, mlp=512, vocab=1024)
    blob = np.zeros(ck.nbytes_total, dtype=np.uint8)
    wl.fill_np(blob, 8, "normal")
    d_blob = dev(blob)
    nbytes = [ck.nbytes(i) for i in range(ck.N)]
    for world, ranks in ((1, [0]), (4, [0, 3])):
        for rank in ranks:
            split = ck.split_dim if world > 1 else np.full(ck.N, -1)
            sizes = [n // (world if split[i] >= 0 else 1) for i, n in enumerate(nbytes)]
            want = [np.zeros(n, dtype=np.uint8) for n in sizes]
            oracle.weights(ck.byte_off, ck.E, ck.shapes, split, rank, world, blob, want)
            want_sums = oracle.weights_checksum(ck.byte_off, ck.E, ck.shapes, split, rank, world, blob)
            plan = tc.tc_plan_create(tc.weights_spec(ck.byte_off, nbytes, ck.E, ck.ndim, ck.shapes, split_dim=split, rank=rank, world=world,
                                                     blob_bytes=ck.nbytes_total, flags=tc.TC_PLAN_CHECKSUM, tuning=dict(tile_bytes=4096)))
            outs = [Guarded(n, fill=0xEE) for n in sizes]
            sums = torch.full((ck.N,), -1, dtype=torch.int64, device="cuda")
            for _ in range(2):                                     # accumulators are zeroed by every call
                tc.tc_weights_materialize_checksum(plan, d_blob, [o.ptr() for o in outs], sums)
            torch.cuda.synchronize()
            assert np.array_equal(sums.cpu().numpy().view(np.uint64), want_sums)
            for i in range(ck.N):
                assert np.array_equal(outs[i].result(), want[i]), ck.names[i]
            tc.tc_weights_materialize(plan, d_blob, [o.ptr() for o in outs])   # the plan still runs unchecked
    # a corrupted blob is detected
    bad = blob.copy()
    assert ck.split_dim[1] < 0                                 # a replicated norm: every rank reads all of it
    bad[ck.byte_off[1] + 100] ^= 0x10
    tc.tc_weights_materialize_checksum(plan, dev(bad), [o.ptr() for o in outs], sums)
    torch.cuda.synchronize()
    got = sums.cpu().numpy().view(np.uint64)
    assert (got != want_sums).sum() == 1 and got[1] != want_sums[1]
    plain = tc.tc_plan_create(tc.weights_spec(ck.byte_off, nbytes, ck.E, ck.ndim, ck.shapes, blob_bytes=ck.nbytes_total))
    with pytest.raises(tc.TensorCastError) as e:
        tc.tc_weights_materialize_checksum(plain, d_blob, [o.ptr() for o in outs], sums)
    assert e.value.status == tc.TC_ERR_KIND


def test_a_wait_that_cannot_complete_ends_with_a_status_word_not_a_hang():
    """The realigning build waits for its bulk copies with a bound.  The self-test waits on a
    barrier nothing arrives at: the wait runs out, the kernel returns normally, the status word
    carries the flag once, and the device keeps working."""
    assert tc.tc_device_status() == 0
    tc.tc_selftest_wait_timeout()
    torch.cuda.synchronize()
    assert tc.tc_device_status() == tc.TC_DEVICE_BULK_WAIT_TIMEOUT
    assert tc.tc_device_status() == 0                       # reading cleared it
    x = torch.arange(1024, device="cuda")
    assert int(x.sum().item()) == 1023 * 512                # the context is alive and well


def test_debug_plans_check_their_descriptors_on_the_device_and_skip_the_copy_when_out_of_bounds():
    """TC_PLAN_DEBUG_BOUNDS: a small kernel holds the uploaded descriptors against the slot extents
    before each execution.  A valid plan passes (and copies the right bytes); with every slot
    pretended one byte smaller a plan that fills its packed buffer to the last byte must raise
    TC_DEVICE_OUT_OF_BOUNDS, and while the flag stands the copy kernel copies nothing.  Nothing
    traps and the context stays usable."""
    rng = np.random.default_rng(31)
    shape, NB, stride, pool, T, off, bt = kv_case(rng, L=2, NB=40, B=16, H=8, D=64, E=2, T=(100, 16, 7, 333))
    L = shape[0]
    pl = tc.pool(tc.TC_NHD, NB, 1, plane_stride=NB * stride, slot_bytes=pool.size)
    d_pool = dev(pool)
    want = np.zeros(oracle.packed_nbytes(shape, T), dtype=np.uint8)
    oracle.kv_pack(shape, oracle.NHD, stride, planes_of(pool, L * 2), T, off, bt, oracle.HND, want)
    plan = tc.tc_plan_create(tc.kv_spec(tc.TC_KV_PACK, shape, src_pool=pl, packed_layout=tc.TC_HND, T=T, bt_off=off, bt_src=bt,
                                        packed_bytes=want.size, flags=tc.TC_PLAN_DEBUG_BOUNDS))
    assert tc.tc_device_status() == 0
    packed = Guarded(want.size)
    tc.tc_kv_pack(plan, [d_pool], [packed.ptr()])
    assert np.array_equal(packed.result(), want)
    assert tc.tc_device_status() == 0
    tc.tc_plan_check_device(plan, 0)
    torch.cuda.synchronize()
    assert tc.tc_device_status() == 0
    tc.tc_plan_check_device(plan, 1)                          # every slot one byte smaller
    untouched = Guarded(want.size, fill=0xEE)
    tc.tc_kv_pack(plan, [d_pool], [untouched.ptr()])          # the flag stands: nothing is copied
    assert (untouched.result() == 0xEE).all()
    assert tc.tc_device_status() == tc.TC_DEVICE_OUT_OF_BOUNDS
    assert tc.tc_device_status() == 0                         # reading cleared it
    tc.tc_kv_pack(plan, [d_pool], [untouched.ptr()])
    assert np.array_equal(untouched.result(), want)
    # unpack (group 1), migrate and weights plans pass their own check too
    bt2 = rng.permutation(NB)[:off[-1]].astype(np.int32)
    for spec in (tc.kv_spec(tc.TC_KV_UNPACK, shape, dst_pool=pl, packed_layout=tc.TC_HND, T=T, bt_off=off, bt_dst=bt2, flags=tc.TC_PLAN_DEBUG_BOUNDS),
                 tc.kv_spec(tc.TC_KV_MIGRATE, shape, src_pool=pl, dst_pool=pl, T=T, bt_off=off, bt_src=bt, bt_dst=bt2, flags=tc.TC_PLAN_DEBUG_BOUNDS)):
        p2 = tc.tc_plan_create(spec)
        tc.tc_plan_check_device(p2, 0)
        assert tc.tc_device_status() == 0
        tc.tc_plan_check_device(p2, pool.size)                # no slot left at all
        assert tc.tc_device_status() == tc.TC_DEVICE_OUT_OF_BOUNDS
    # a mixed plan carries extents for both of its groups (offload: pool -> host pool, reload: back)
    hpool = tc.pool(tc.TC_HND, 24, 1, plane_stride=stride, block_stride=L * 2 * stride, slot_bytes=24 * L * 2 * stride)
    n_off = int(off[1])
    mixed = tc.tc_plan_create(tc.kv_spec(tc.TC_KV_MIXED, shape, src_pool=pl, dst_pool=hpool, T=T[:1], bt_off=off[:2], bt_src=bt[:n_off],
                                         bt_dst=np.arange(n_off, dtype=np.int32),
                                         reload=dict(T=T[1:2], bt_off=off[1:3] - off[1], bt_src=np.array([23], dtype=np.int32), bt_dst=bt2[:1]),
                                         flags=tc.TC_PLAN_DEBUG_BOUNDS))
    tc.tc_plan_check_device(mixed, 0)
    assert tc.tc_device_status() == 0
    tc.tc_plan_check_device(mixed, 1)                         # host block 23 ends on the host pool's last byte
    assert tc.tc_device_status() == tc.TC_DEVICE_OUT_OF_BOUNDS
    ck = small_checkpoint()
    blob = np.zeros(ck.nbytes_total, dtype=np.uint8)
    wl.fill_np(blob, 5, "normal")
    sizes = [ck.nbytes(i) // (4 if ck.split_dim[i] >= 0 else 1) for i in range(ck.N)]
    want_w = [np.zeros(n, dtype=np.uint8) for n in sizes]
    oracle.weights(ck.byte_off, ck.E, ck.shapes, ck.split_dim, 2, 4, blob, want_w)
    outs = [Guarded(n, fill=0xEE) for n in sizes]
    wplan = tc.tc_plan_create(ck_spec(ck, split_dim=ck.split_dim, rank=2, world=4, flags=tc.TC_PLAN_DEBUG_BOUNDS))
    tc.tc_weights_materialize(wplan, dev(blob), [o.ptr() for o in outs])
    for i in range(ck.N):
        assert np.array_equal(outs[i].result(), want_w[i]), ck.names[i]
    assert tc.tc_device_status() == 0
    tc.tc_plan_check_device(wplan, 1)
    assert tc.tc_device_status() == tc.TC_DEVICE_OUT_OF_BOUNDS
    with pytest.raises(tc.TensorCastError) as e:              # only plans made for it carry the extents
        tc.tc_plan_check_device(tc.tc_plan_create(ck_spec(ck)), 0)
    assert e.value.status == tc.TC_ERR_KIND
    x = torch.arange(1024, device="cuda")
    assert int(x.sum().item()) == 1023 * 512


def test_traced_plan_reports_the_device_time_of_its_last_execution():
    shape = wl.KVShape(L=4, B=16, H=8, D=128, E=2)
    NB = 512
    T = np.array([NB * shape.B], dtype=np.int64)
    off = np.array([0, NB], dtype=np.int64)
    bt = np.random.default_rng(5).permutation(NB).astype(np.int32)
    pool = torch.zeros(NB * shape.block_bytes, dtype=torch.uint8, device="cuda")
    out = torch.zeros(NB * shape.block_bytes, dtype=torch.uint8, device="cuda")
    pl = tc.pool(tc.TC_NHD, NB, 1, plane_stride=NB * shape.chunk_bytes, slot_bytes=pool.numel())
    plan = tc.tc_plan_create(tc.kv_spec(tc.TC_KV_PACK, shape.tuple, src_pool=pl, packed_layout=tc.TC_HND, T=T, bt_off=off, bt_src=bt,
                                        flags=tc.TC_PLAN_TRACE, trace_id=77))
    assert plan.stats().last_device_us[0] == -1.0            # not run yet
    stream = torch.cuda.Stream()
    a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    a.record(stream)
    tc.tc_kv_pack(plan, [pool], [out], stream.cuda_stream)
    b.record(stream)
    stream.synchronize()
    st = plan.stats()
    outer_us = 1e3 * a.elapsed_time(b)
    assert st.trace_id == 77 and st.last_device_us[0] <= outer_us + 1.0
    assert st.last_device_us[0] > 2 * pool.numel() / 8e12 * 1e6   # 128 MiB read and written cannot beat 8 TB/s
    untraced = tc.tc_plan_create(tc.kv_spec(tc.TC_KV_PACK, shape.tuple, src_pool=pl, packed_layout=tc.TC_HND, T=T, bt_off=off, bt_src=bt))
    assert untraced.stats().last_device_us[0] == 0.0


# --------------------------------------------------------------------------- another GPU's memory
@pytest.mark.skipif(torch.cuda.is_available() and torch.cuda.device_count() < 2, reason="needs two GPUs with peer access")
def test_pack_and_migrate_from_a_pool_on_another_gpu():
    """Cross-GPU migration: the source pool lives on device 1, the plan and the destination on
    device 0.  A table entry is then a peer pointer; every CTA moves its own tile with plain loads
    over NVLink (no bulk copy is involved: the geometry is aligned, so the register
    path runs).  Compared with the oracle like any other pack / migrate."""
    if not torch.cuda.can_device_access_peer(0, 1):
        pytest.skip("devices 0 and 1 have no peer access")
    rng = np.random.default_rng(91)
    shape, NB, stride, pool, T, off, bt = kv_case(rng, L=2, NB=48, B=16, H=8, D=128, E=2, T=(100, 16, 7, 333))
    L = shape[0]
    bt2 = rng.permutation(NB)[:off[-1]].astype(np.int32)
    remote = torch.from_numpy(pool).to("cuda:1")           # the other engine's pool
    torch.cuda.synchronize(1)
    torch.cuda.set_device(0)
    x = torch.empty(16, dtype=torch.uint8, device="cuda:0")
    x.copy_(remote[:16])                                   # torch enables peer access between the two devices here
    torch.cuda.synchronize(0)
    pl = tc.pool(tc.TC_NHD, NB, 1, plane_stride=NB * stride, slot_bytes=pool.size)
    for packed_l in LAYOUTS:
        want = np.zeros(oracle.packed_nbytes(shape, T), dtype=np.uint8)
        oracle.kv_pack(shape, oracle.NHD, stride, planes_of(pool, L * 2), T, off, bt, packed_l, want)
        packed = Guarded(want.size)
        plan = tc.tc_plan_create(tc.kv_spec(tc.TC_KV_PACK, shape, src_pool=pl, packed_layout=packed_l, T=T, bt_off=off, bt_src=bt))
        tc.tc_kv_pack(plan, [remote.data_ptr()], [packed.ptr()])
        assert np.array_equal(packed.result(), want), packed_l
    for dst_l in LAYOUTS:
        pl2 = tc.pool(dst_l, NB, 1, plane_stride=NB * stride, slot_bytes=pool.size)
        want_pool = np.full_like(pool, 0xA5)
        oracle.kv_migrate(shape, oracle.NHD, stride, planes_of(pool, L * 2), dst_l, stride, planes_of(want_pool, L * 2), T, off, bt, bt2)
        fresh = Guarded(pool.size)
        plan = tc.tc_plan_create(tc.kv_spec(tc.TC_KV_MIGRATE, shape, src_pool=pl, dst_pool=pl2, T=T, bt_off=off, bt_src=bt, bt_dst=bt2))
        tc.tc_kv_pack(plan, [remote.data_ptr()], [fresh.ptr()])
        assert np.array_equal(fresh.result(), want_pool), dst_l


# --------------------------------------------------------------------------- misaligned rows
@pytest.mark.parametrize("cols,pitch,tile", [(100, 116, 0), (256, 256 + 16, 0), (33, 64, 1024), (5000, 5003, 0), (40000, 40000 + 7, 0), (70000, 70001, 65536)])
def test_rows_at_every_source_and_destination_alignment(cols, pitch, tile):
    """Rows of `cols` bytes whose source starts at blob offset ... + a and whose destination
    starts at b inside its own slot, for a and b over all residues modulo 16 (a sample of the
    256 pairs for the long rows).  Every slot is a guarded buffer, so a head or tail byte that
    lands outside its row shows up either in the red zones or in the sentinel bytes between the
    rows; pitch is not a multiple of 16 in most cases, so the rows of one tensor differ in
    alignment as well."""
    rng = np.random.default_rng(cols)
    rows = 5 if cols < 1000 else 2
    pairs = [(a, b) for a in range(16) for b in range(16)]
    if cols >= 1000:
        pairs = [pairs[i] for i in rng.permutation(256)[:40]] + [(0, 1), (1, 0), (15, 15), (8, 0), (3, 3)]
    src_off, pos = [], 0
    for a, b in pairs:
        pos = (pos + 15) // 16 * 16 + a
        src_off.append(pos)
        pos += rows * cols
    blob = rng.integers(0, 256, pos + 16, dtype=np.uint8)
    N = len(pairs)
    slot_bytes = [b + (rows - 1) * pitch + cols for a, b in pairs]
    kw = dict(dst_off=[b for a, b in pairs], dst_stride=[[pitch, 1, 1, 1]] * N)
    shapes = [[rows, cols, 1, 1]] * N
    spec = tc.weights_spec(src_off, [rows * cols] * N, [1] * N, [2] * N, shapes, blob_bytes=blob.size, dst_slot=list(range(N)),
                           n_dst=N, dst_bytes=slot_bytes, tuning=dict(tile_bytes=tile) if tile else None, **kw)
    plan = tc.tc_plan_create(spec)
    assert plan.stats().vec_bytes[0] == 1
    want = [np.full(n, 0xEE, dtype=np.uint8) for n in slot_bytes]
    oracle.weights(src_off, [1] * N, shapes, [-1] * N, 0, 1, blob, want, **kw)
    d_blob = dev(blob)
    for shift in (0, 1):                                      # destination buffers 16-byte aligned, then odd
        outs = [Guarded(n, fill=0xEE, shift=shift) for n in slot_bytes]
        tc.tc_weights_materialize(plan, d_blob, [o.ptr() for o in outs])
        for k in range(N):
            assert np.array_equal(outs[k].result(), want[k]), (pairs[k], shift)


@pytest.mark.parametrize("a,b", [(0, 1), (2, 0), (15, 15), (8, 4), (3, 9), (0, 0)])
def test_dim1_weight_slices_with_long_rows_through_misaligned_pointers(a, b):
    """Row-parallel shards of [rows, cols] matrices: strided source rows of 1-3.5 KiB that are
    adjacent in the destination, the blob starting a bytes and the outputs b bytes off a 16-byte
    boundary.  Such rows are staged back to back and stored as one long destination run."""
    rng = np.random.default_rng(60 + a + b)
    shapes = [[96, 4096, 1, 1], [40, 7168, 1, 1], [33, 2048, 1, 1], [5, 8192, 1, 1]]
    nbytes = [2 * r * c for r, c, _, _ in shapes]
    byte_off = np.concatenate([[0], np.cumsum(nbytes)[:-1]]).tolist()
    total = int(sum(nbytes))
    blob = rng.integers(0, 256, total, dtype=np.uint8)
    raw = torch.zeros(total + 16, dtype=torch.uint8, device="cuda")
    raw[a:a + total].copy_(dev(blob))
    for world, rank in ((4, 1), (8, 7), (2, 0)):
        want = [np.zeros(n // world, dtype=np.uint8) for n in nbytes]
        oracle.weights(byte_off, [2] * 4, shapes, [1] * 4, rank, world, blob, want)
        plan = tc.tc_plan_create(tc.weights_spec(byte_off, nbytes, [2] * 4, [2] * 4, shapes, split_dim=[1] * 4, rank=rank, world=world, blob_bytes=total))
        outs = [Guarded(n // world, fill=0xEE, shift=b) for n in nbytes]
        tc.tc_weights_materialize(plan, raw[a:].data_ptr(), [o.ptr() for o in outs])
        for i in range(4):
            assert np.array_equal(outs[i].result(), want[i]), (i, world, rank)
    assert tc.tc_device_status() == 0


@pytest.mark.parametrize("H,D,E,slots", [(8, 128, 2, "one"), (8, 64, 2, "one"), (8, 32, 2, "planes"), (8, 512, 2, "one"), (2, 512, 2, "one"), (4, 256, 4, "one"), (16, 64, 2, "one"), (32, 32, 2, "one")])
@pytest.mark.parametrize("shift_pool,shift_packed", [(0, 2), (2, 0), (6, 6), (1, 9), (8, 4)])
def test_kv_pack_unpack_migrate_through_misaligned_pointers(shift_pool, shift_packed, H, D, E, slots):
    """Aligned geometry, misaligned base pointers: the pool and / or the packed buffer start at
    an odd address (a view into a larger allocation).  Rows of D * E bytes (NHD <-> HND) and whole
    planes (same layout) both take the realigning path; with D = 64 and 32 a plane is small enough
    for tiles of two and four planes, in a pool with one pointer or a pointer per plane; rows of
    1 KiB are staged back to back where the destination has them adjacent (a head's tokens, a
    token's heads); with 16 and 32 heads of 128- and 64-byte rows a destination run has fewer chunks
    than the CTA has threads and several runs go side by side."""
    rng = np.random.default_rng(77)
    shape, NB, stride, pool, T, off, bt = kv_case(rng, L=2, NB=40, B=16, H=H, D=D, E=E, T=(100, 16, 7, 333))
    L, B, H, D, E = shape
    planes = planes_of(pool, L * 2)
    bt2 = rng.permutation(NB)[:off[-1]].astype(np.int32)
    n_slots = L * 2 if slots == "planes" else 1
    pl = tc.pool(tc.TC_NHD, NB, n_slots, plane_stride=0 if slots == "planes" else NB * stride, slot_bytes=pool.size // n_slots)
    raw = torch.zeros(pool.size + 16, dtype=torch.uint8, device="cuda")
    d_pool = raw[shift_pool:shift_pool + pool.size]
    d_pool.copy_(dev(pool))
    per = pool.size // (L * 2)
    table = lambda base: [base + p * per for p in range(L * 2)] if slots == "planes" else [base]
    for packed_l in LAYOUTS:
        want = np.zeros(oracle.packed_nbytes(shape, T), dtype=np.uint8)
        oracle.kv_pack(shape, oracle.NHD, stride, planes, T, off, bt, packed_l, want)
        packed = Guarded(want.size, shift=shift_packed)
        plan = tc.tc_plan_create(tc.kv_spec(tc.TC_KV_PACK, shape, src_pool=pl, packed_layout=packed_l, T=T, bt_off=off, bt_src=bt))
        tc.tc_kv_pack(plan, table(d_pool.data_ptr()), [packed.ptr()])
        assert np.array_equal(packed.result(), want), packed_l
        want_pool = np.full_like(pool, 0xA5)
        oracle.kv_unpack(shape, oracle.NHD, stride, planes_of(want_pool, L * 2), T, off, bt2, packed_l, want)
        fresh = Guarded(pool.size, shift=shift_pool)
        plan2 = tc.tc_plan_create(tc.kv_spec(tc.TC_KV_UNPACK, shape, dst_pool=pl, packed_layout=packed_l, T=T, bt_off=off, bt_dst=bt2))
        tc.tc_kv_unpack(plan2, [packed.ptr()], table(fresh.ptr()))
        assert np.array_equal(fresh.result(), want_pool), packed_l
    for dst_l in LAYOUTS:
        pl2 = tc.pool(dst_l, NB, n_slots, plane_stride=0 if slots == "planes" else NB * stride, slot_bytes=pool.size // n_slots)
        want_pool = np.full_like(pool, 0xA5)
        oracle.kv_migrate(shape, oracle.NHD, stride, planes, dst_l, stride, planes_of(want_pool, L * 2), T, off, bt, bt2)
        fresh = Guarded(pool.size, shift=shift_packed)
        plan3 = tc.tc_plan_create(tc.kv_spec(tc.TC_KV_MIGRATE, shape, src_pool=pl, dst_pool=pl2, T=T, bt_off=off, bt_src=bt, bt_dst=bt2))
        tc.tc_kv_pack(plan3, table(d_pool.data_ptr()), table(fresh.ptr()))
        assert np.array_equal(fresh.result(), want_pool), dst_l
    assert tc.tc_device_status() == 0


def test_shared_memory_copy_path_on_aligned_geometry():
    """tuning.copy_path = 1 sends aligned geometry through the shared-memory path too (it exists
    to compare the two paths); the bytes must not depend on the path."""
    rng = np.random.default_rng(78)
    shape, NB, stride, pool, T, off, bt = kv_case(rng, L=2, NB=40, B=16, H=8, D=64, E=2, T=(100, 16, 7, 333))
    L, B, H, D, E = shape
    bt2 = rng.permutation(NB)[:off[-1]].astype(np.int32)
    pl = tc.pool(tc.TC_NHD, NB, 1, plane_stride=NB * stride, slot_bytes=pool.size)
    d_pool = dev(pool)
    smem = dict(copy_path=1)
    want = np.zeros(oracle.packed_nbytes(shape, T), dtype=np.uint8)
    oracle.kv_pack(shape, oracle.NHD, stride, planes_of(pool, L * 2), T, off, bt, oracle.HND, want)
    packed = Guarded(want.size)
    tc.tc_kv_pack(tc.tc_plan_create(tc.kv_spec(tc.TC_KV_PACK, shape, src_pool=pl, packed_layout=tc.TC_HND, T=T, bt_off=off, bt_src=bt, tuning=smem)),
                  [d_pool], [packed.ptr()])
    assert np.array_equal(packed.result(), want)
    want_pool = np.full_like(pool, 0xA5)
    oracle.kv_migrate(shape, oracle.NHD, stride, planes_of(pool, L * 2), oracle.NHD, stride, planes_of(want_pool, L * 2), T, off, bt, bt2)
    fresh = Guarded(pool.size)
    tc.tc_kv_pack(tc.tc_plan_create(tc.kv_spec(tc.TC_KV_MIGRATE, shape, src_pool=pl, dst_pool=pl, T=T, bt_off=off, bt_src=bt, bt_dst=bt2, tuning=smem)),
                  [d_pool], [fresh.ptr()])
    assert np.array_equal(fresh.result(), want_pool)
    ck = small_checkpoint()
    blob = np.zeros(ck.nbytes_total, dtype=np.uint8)
    wl.fill_np(blob, 5, "normal")
    sizes = [ck.nbytes(i) // (4 if ck.split_dim[i] >= 0 else 1) for i in range(ck.N)]
    want_w = [np.zeros(n, dtype=np.uint8) for n in sizes]
    oracle.weights(ck.byte_off, ck.E, ck.shapes, ck.split_dim, 2, 4, blob, want_w)
    outs = [Guarded(n, fill=0xEE) for n in sizes]
    tc.tc_weights_materialize(tc.tc_plan_create(ck_spec(ck, split_dim=ck.split_dim, rank=2, world=4, tuning=smem)), dev(blob), [o.ptr() for o in outs])
    for i in range(ck.N):
        assert np.array_equal(outs[i].result(), want_w[i]), ck.names[i]
    with pytest.raises(tc.TensorCastError) as e:
        tc.tc_plan_create(ck_spec(ck, tuning=dict(copy_path=7)))
    assert e.value.status == tc.TC_ERR_INVALID_ARG
    assert tc.tc_device_status() == 0


# --------------------------------------------------------------------------- random geometries
@pytest.mark.parametrize("seed", range(24))
def test_random_geometries_on_the_device(seed):
    rng = np.random.default_rng(1000 + seed)
    L, B, H = int(rng.integers(1, 4)), int(rng.choice([1, 2, 4, 16, 32])), int(rng.integers(1, 9))
    D, E = int(rng.choice([3, 8, 16, 64, 128])), int(rng.choice([1, 2, 4, 8]))
    R = int(rng.integers(1, 7))
    T = [int(rng.choice([0, 1, B, B + 1, 3 * B - 1, 9 * B, 17 * B + B // 2])) for _ in range(R)]
    pad = int(rng.choice([0, 0, E, 32]))
    shift = int(rng.choice([0, 0, 0, E, 16]))
    tile = int(rng.choice([0, 0, 1024, 8192]))
    pool_l, other_l = int(rng.integers(0, 2)), int(rng.integers(0, 2))
    slots = str(rng.choice(["planes", "one"]))             # one pointer per plane, or one pointer and a plane stride
    shape = (L, B, H, D, E)
    T = np.array(T, dtype=np.int64)
    off = np.concatenate([[0], np.cumsum((T + B - 1) // B)]).astype(np.int64)
    NB = int(off[-1]) + 2
    stride = B * H * D * E + pad
    pool = rng.integers(0, 256, L * 2 * NB * stride, dtype=np.uint8)
    bt = rng.permutation(NB)[:off[-1]].astype(np.int32)
    bt2 = rng.permutation(NB)[:off[-1]].astype(np.int32)
    tune = dict(tile_bytes=tile) if tile else None
    def mkpool(layout):
        if slots == "planes":
            return tc.pool(layout, NB, L * 2, block_stride=stride, slot_bytes=NB * stride)
        return tc.pool(layout, NB, 1, plane_stride=NB * stride, block_stride=stride, slot_bytes=L * 2 * NB * stride)
    pl = mkpool(pool_l)
    want = np.zeros(oracle.packed_nbytes(shape, T), dtype=np.uint8)
    oracle.kv_pack(shape, pool_l, stride, planes_of(pool, L * 2), T, off, bt, other_l, want)
    d_pool = Guarded(pool.size, init=pool, shift=shift)
    out = Guarded(max(want.size, 1), shift=shift)
    plan = tc.tc_plan_create(tc.kv_spec(tc.TC_KV_PACK, shape, src_pool=pl, packed_layout=other_l, T=T, bt_off=off, bt_src=bt, tuning=tune))
    tc.tc_kv_pack(plan, pool_tables(d_pool, L * 2, slots), [out.ptr()])
    assert np.array_equal(out.result()[:want.size], want)
    want_pool = np.full_like(pool, 0xA5)
    oracle.kv_migrate(shape, pool_l, stride, planes_of(pool, L * 2), other_l, stride, planes_of(want_pool, L * 2), T, off, bt, bt2)
    pl2 = mkpool(other_l)
    mig = tc.tc_plan_create(tc.kv_spec(tc.TC_KV_MIGRATE, shape, src_pool=pl, dst_pool=pl2, T=T, bt_off=off, bt_src=bt, bt_dst=bt2, tuning=tune))
    fresh = Guarded(pool.size, shift=shift)
    tc.tc_kv_pack(mig, pool_tables(d_pool, L * 2, slots), pool_tables(fresh, L * 2, slots))
    assert np.array_equal(fresh.result(), want_pool)


@pytest.mark.parametrize("seed", range(32))
def test_random_misaligned_geometries_on_the_device(seed):
    """Random shapes, every buffer at its own random address modulo 16, rows of D * E bytes that
    are or are not multiples of 16 (same alignment in every row, or a different one per row), block
    strides with odd padding: pack, unpack and migrate against the oracle, destinations guarded."""
    rng = np.random.default_rng(2000 + seed)
    L, B, H = int(rng.integers(1, 4)), int(rng.choice([1, 4, 16, 32])), int(rng.integers(1, 9))
    D, E = int(rng.choice([16, 20, 33, 64, 100, 128, 192])), int(rng.choice([1, 2, 4]))
    R = int(rng.integers(1, 6))
    T = np.array([int(rng.choice([0, 1, B, B + 1, 3 * B - 1, 9 * B, 12 * B + B // 2])) for _ in range(R)], dtype=np.int64)
    pad = int(rng.choice([0, 0, E, 16, 48]))
    s_pool, s_out, s_dst = (int(x) for x in rng.integers(0, 16, 3))
    tile = int(rng.choice([0, 0, 2048, 8192]))
    pool_l, other_l = int(rng.integers(0, 2)), int(rng.integers(0, 2))
    slots = str(rng.choice(["planes", "one"]))
    shape = (L, B, H, D, E)
    off = np.concatenate([[0], np.cumsum((T + B - 1) // B)]).astype(np.int64)
    NB = int(off[-1]) + 2
    stride = B * H * D * E + pad
    pool = rng.integers(0, 256, L * 2 * NB * stride, dtype=np.uint8)
    bt = rng.permutation(NB)[:off[-1]].astype(np.int32)
    bt2 = rng.permutation(NB)[:off[-1]].astype(np.int32)
    tune = dict(tile_bytes=tile) if tile else None
    def mkpool(layout):
        if slots == "planes":
            return tc.pool(layout, NB, L * 2, block_stride=stride, slot_bytes=NB * stride)
        return tc.pool(layout, NB, 1, plane_stride=NB * stride, block_stride=stride, slot_bytes=L * 2 * NB * stride)
    pl, pl2 = mkpool(pool_l), mkpool(other_l)
    want = np.zeros(oracle.packed_nbytes(shape, T), dtype=np.uint8)
    oracle.kv_pack(shape, pool_l, stride, planes_of(pool, L * 2), T, off, bt, other_l, want)
    d_pool = Guarded(pool.size, init=pool, shift=s_pool)
    out = Guarded(max(want.size, 1), shift=s_out)
    plan = tc.tc_plan_create(tc.kv_spec(tc.TC_KV_PACK, shape, src_pool=pl, packed_layout=other_l, T=T, bt_off=off, bt_src=bt, tuning=tune))
    tc.tc_kv_pack(plan, pool_tables(d_pool, L * 2, slots), [out.ptr()])
    assert np.array_equal(out.result()[:want.size], want)
    want_pool = np.full_like(pool, 0xA5)
    oracle.kv_unpack(shape, pool_l, stride, planes_of(want_pool, L * 2), T, off, bt2, other_l, want)
    fresh = Guarded(pool.size, shift=s_dst)
    plan2 = tc.tc_plan_create(tc.kv_spec(tc.TC_KV_UNPACK, shape, dst_pool=pl, packed_layout=other_l, T=T, bt_off=off, bt_dst=bt2, tuning=tune))
    tc.tc_kv_unpack(plan2, [out.ptr()], pool_tables(fresh, L * 2, slots))
    assert np.array_equal(fresh.result(), want_pool)
    want_pool = np.full_like(pool, 0xA5)
    oracle.kv_migrate(shape, pool_l, stride, planes_of(pool, L * 2), other_l, stride, planes_of(want_pool, L * 2), T, off, bt, bt2)
    mig = tc.tc_plan_create(tc.kv_spec(tc.TC_KV_MIGRATE, shape, src_pool=pl, dst_pool=pl2, T=T, bt_off=off, bt_src=bt, bt_dst=bt2, tuning=tune))
    fresh = Guarded(pool.size, shift=s_dst)
    tc.tc_kv_pack(mig, pool_tables(d_pool, L * 2, slots), pool_tables(fresh, L * 2, slots))
    assert np.array_equal(fresh.result(), want_pool)
    assert tc.tc_device_status() == 0


@pytest.mark.parametrize("shift", [0, 2])
def test_execute_calls_can_be_captured_in_a_cuda_graph_and_replayed(shift):
    """Launch-bound use (config 1 moves 1.4 MB): pack + unpack captured once, replayed many
    times; every replay reproduces the oracle's bytes (re-execution is idempotent).  With the
    packed buffer at a misaligned address the captured kernels are the realigning build."""
    shape, NB, src, dst = wl.config1()
    s = shape.tuple
    pool = np.zeros(2 * NB * shape.chunk_bytes, dtype=np.uint8)
    wl.fill_np(pool, wl.SEED_BASE + 1)
    want = np.zeros(oracle.packed_nbytes(s, src.T), dtype=np.uint8)
    oracle.kv_pack(s, oracle.NHD, shape.chunk_bytes, planes_of(pool, 2), src.T, src.bt_off, src.bt, oracle.HND, want)
    want_pool = np.full_like(pool, 0xA5)
    oracle.kv_unpack(s, oracle.NHD, shape.chunk_bytes, planes_of(want_pool, 2), dst.T, dst.bt_off, dst.bt, oracle.HND, want)
    pl = tc.pool(tc.TC_NHD, NB, 1, plane_stride=NB * shape.chunk_bytes, slot_bytes=pool.size)
    pack = tc.tc_plan_create(tc.kv_spec(tc.TC_KV_PACK, s, src_pool=pl, packed_layout=tc.TC_HND, T=src.T, bt_off=src.bt_off, bt_src=src.bt))
    unpack = tc.tc_plan_create(tc.kv_spec(tc.TC_KV_UNPACK, s, dst_pool=pl, packed_layout=tc.TC_HND, T=dst.T, bt_off=dst.bt_off, bt_dst=dst.bt))
    d_pool, fresh = dev(pool), Guarded(pool.size)
    packed = torch.zeros(want.size + 16, dtype=torch.uint8, device="cuda")[shift:shift + want.size]
    side = torch.cuda.Stream()
    graph = torch.cuda.CUDAGraph()
    torch.cuda.synchronize()
    with torch.cuda.graph(graph, stream=side):
        tc.tc_kv_pack(pack, [d_pool], [packed], side.cuda_stream)
        tc.tc_kv_unpack(unpack, [packed], [fresh.ptr()], side.cuda_stream)
    for _ in range(3):
        packed.zero_()
        fresh.view.fill_(0xA5)
        graph.replay()
        torch.cuda.synchronize()
        assert np.array_equal(packed.cpu().numpy(), want)
        assert np.array_equal(fresh.result(), want_pool)


def test_a_plan_can_run_on_a_non_blocking_stream_the_moment_it_is_created():
    """Plans of 2 000 descriptors (a 256 KB upload) created, executed at once on a non-blocking
    stream and destroyed, two geometries taking turns so that each inherits the other's storage
    block: the upload must have landed when tc_plan_create returns, whatever stream runs next."""
    rng = np.random.default_rng(41)
    shape, NB, stride, pool, _, _, _ = kv_case(rng, L=1, NB=2400, B=4, H=1, D=8, E=2, T=(4,))
    d_pool = dev(pool)
    pl = tc.pool(tc.TC_NHD, NB, 1, plane_stride=NB * stride, slot_bytes=pool.size)
    cases = []
    for k in range(2):
        T = np.full(2000, 4 - k, dtype=np.int64)               # one block per request; full or ragged
        off = np.arange(2001, dtype=np.int64)
        bt = rng.permutation(NB)[:2000].astype(np.int32)
        want = np.zeros(oracle.packed_nbytes(shape, T), dtype=np.uint8)
        oracle.kv_pack(shape, oracle.NHD, stride, planes_of(pool, 2), T, off, bt, oracle.NHD, want, threads=4)
        cases.append((T, off, bt, torch.from_numpy(want).cuda(), torch.zeros(want.size, dtype=torch.uint8, device="cuda")))
    stream = torch.cuda.Stream()
    torch.cuda.synchronize()
    for it in range(60):
        T, off, bt, want, out = cases[it % 2]
        plan = tc.tc_plan_create(tc.kv_spec(tc.TC_KV_PACK, shape, src_pool=pl, packed_layout=tc.TC_NHD, T=T, bt_off=off, bt_src=bt))
        tc.tc_kv_pack(plan, [d_pool], [out], stream.cuda_stream)
        stream.synchronize()
        assert torch.equal(out, want), it
        out.zero_()
        torch.cuda.synchronize()
        plan.destroy()


def test_concurrent_threads_create_execute_destroy():
    """Calls on distinct plans are thread safe (plan-storage cache, staging rings, per-thread error
    text): four threads each create, run on their own stream and destroy plans in a loop."""
    import threading
    rng = np.random.default_rng(28)
    shape, NB, stride, pool, T, off, bt = kv_case(rng, L=2, NB=64, B=16, H=8, D=128, E=2, T=(100, 37, 16, 5, 200))
    L = shape[0]
    d_pool = dev(pool)
    pl = tc.pool(tc.TC_NHD, NB, 1, plane_stride=NB * stride)
    wants = {}
    for lay in LAYOUTS:
        w = np.zeros(oracle.packed_nbytes(shape, T), dtype=np.uint8)
        oracle.kv_pack(shape, oracle.NHD, stride, planes_of(pool, L * 2), T, off, bt, lay, w, threads=4)
        wants[lay] = w
    errors = []

    def worker(k):
        try:
            stream = torch.cuda.Stream()
            lay = LAYOUTS[k % 2]
            out = torch.zeros(wants[lay].size, dtype=torch.uint8, device="cuda")
            host = torch.zeros(wants[lay].size, dtype=torch.uint8).pin_memory()
            torch.cuda.synchronize()                         # `out` was zeroed on the default stream
            for it in range(25):
                flags = tc.TC_PLAN_STAGED if (it + k) % 3 == 0 else 0
                plan = tc.tc_plan_create(tc.kv_spec(tc.TC_KV_PACK, shape, src_pool=pl, packed_layout=lay, T=T, bt_off=off, bt_src=bt, flags=flags))
                target = host if flags else out
                tc.tc_kv_pack(plan, [d_pool], [target], stream.cuda_stream)
                stream.synchronize()
                got = target.cpu().numpy() if not flags else host.numpy().copy()
                if not np.array_equal(got, wants[lay]):
                    errors.append((k, it, "mismatch"))
                try:
                    tc.tc_kv_unpack(plan, [target], [d_pool])      # wrong kind: error text is per thread
                except tc.TensorCastError as e:
                    if e.status != tc.TC_ERR_KIND or "tc_kv_unpack" not in str(e):
                        errors.append((k, it, str(e)))
                plan.destroy()
        except Exception as e:  # noqa: BLE001
            errors.append((k, repr(e)))

    threads = [threading.Thread(target=worker, args=(k,)) for k in range(4)]
    for t in threads:
        t.start()
    for t in threads:
        t.join()
    assert not errors, errors[:3]


def test_file_stream_and_staged_reload_share_the_staging_ring(tmp_path):
    """A checkpoint streams in from a file while another thread reloads KV through the same
    host-to-device staging ring: the ring is locked per chunk, so the two interleave."""
    import threading
    ck = wl.llama_checkpoint(hidden=512, layers=3, q_heads=8, kv_heads=4, head_dim=64, mlp=2048, vocab=70000)
    blob = np.zeros(ck.nbytes_total, dtype=np.uint8)
    wl.fill_np(blob, 11, "normal")
    path = tmp_path / "blob.bin"
    blob.tofile(path)
    nbytes = [ck.nbytes(i) for i in range(ck.N)]
    wplan = tc.tc_plan_create(tc.weights_spec(ck.byte_off, nbytes, ck.E, ck.ndim, ck.shapes, blob_bytes=ck.nbytes_total, flags=tc.TC_PLAN_STREAM))
    rng = np.random.default_rng(29)
    shape, NB, stride, pool, T, off, bt = kv_case(rng, L=4, NB=400, B=16, H=8, D=128, E=2, T=(5000, 37, 0, 100, 700))
    L = shape[0]
    packed = np.zeros(oracle.packed_nbytes(shape, T), dtype=np.uint8)
    wl.fill_np(packed[:packed.size & ~1], 12)
    want_pool = np.full_like(pool, 0xA5)
    oracle.kv_unpack(shape, oracle.NHD, stride, planes_of(want_pool, L * 2), T, off, bt, oracle.HND, packed, threads=8)
    pl = tc.pool(tc.TC_NHD, NB, 1, plane_stride=NB * stride)
    uplan = tc.tc_plan_create(tc.kv_spec(tc.TC_KV_UNPACK, shape, dst_pool=pl, packed_layout=tc.TC_HND, T=T, bt_off=off, bt_dst=bt, flags=tc.TC_PLAN_STAGED))
    h_packed = torch.from_numpy(packed).pin_memory()
    errors = []

    def loader():
        try:
            fd = os.open(path, os.O_RDONLY)
            stream = torch.cuda.Stream()
            out = torch.empty(ck.nbytes_total, dtype=torch.uint8, device="cuda")
            ptrs = [out.data_ptr() + int(o) for o in np.concatenate([[0], np.cumsum(nbytes)])[:-1]]
            for it in range(4):
                out.fill_(0xEE)
                torch.cuda.current_stream().synchronize()
                tc.tc_weights_materialize_file(wplan, fd, 0, ptrs, stream=stream.cuda_stream)
                stream.synchronize()
                if not np.array_equal(out.cpu().numpy(), blob):   # tight canonical order: the outputs concatenate to the blob
                    errors.append(("loader", it))
            os.close(fd)
        except Exception as e:  # noqa: BLE001
            errors.append(("loader", repr(e)))

    def reloader():
        try:
            stream = torch.cuda.Stream()
            for it in range(12):
                fresh = Guarded(pool.size)
                torch.cuda.current_stream().synchronize()
                tc.tc_kv_unpack(uplan, [h_packed], [fresh.ptr()], stream.cuda_stream)
                stream.synchronize()
                if not np.array_equal(fresh.result(), want_pool):
                    errors.append(("reloader", it))
        except Exception as e:  # noqa: BLE001
            errors.append(("reloader", repr(e)))

    threads = [threading.Thread(target=loader), threading.Thread(target=reloader)]
    for t in threads:
        t.start()
    for t in threads:
        t.join()
    assert not errors, errors[:3]


def test_pool_of_another_process_through_cuda_ipc():
    """Same-host sharing: a KV pool allocated by this process is opened by a second process
    through CUDA IPC and used there as the source table of its own plan (data buffers are
    caller-leased plain pointers, so nothing in the library is special-cased for this)."""
    import torch.multiprocessing as mp
    from helpers import ipc_pack_child
    rng = np.random.default_rng(33)
    shape, NB, stride, pool, T, off, bt = kv_case(rng, L=2, NB=40, B=16, H=8, D=128, E=2, T=(100, 37, 16, 5, 200))
    L = shape[0]
    want = np.zeros(oracle.packed_nbytes(shape, T), dtype=np.uint8)
    oracle.kv_pack(shape, oracle.NHD, stride, planes_of(pool, L * 2), T, off, bt, oracle.HND, want, threads=4)
    d_pool = dev(pool)
    torch.cuda.synchronize()
    ctx = mp.get_context("spawn")
    q_in, q_out = ctx.Queue(), ctx.Queue()
    child = ctx.Process(target=ipc_pack_child, args=(q_in, q_out))
    child.start()
    try:
        q_in.put((d_pool, shape, ((tc.TC_NHD, NB, 1), dict(plane_stride=NB * stride)), T, off, bt, tc.TC_HND, want.size))
        status, got = q_out.get(timeout=300)
    finally:
        child.join(timeout=60)
        if child.is_alive():
            child.kill()
    assert status == "ok", got
    assert np.array_equal(got, want)


# --------------------------------------------------------------------------- lifecycle on the device
def test_empty_plan_wrong_tables_and_deadline_launch_nothing():
    shape, NB, src, dst = wl.config1()
    s = shape.tuple
    pl = tc.pool(tc.TC_NHD, NB, 2)
    empty = tc.tc_plan_create(tc.kv_spec(tc.TC_KV_PACK, s, src_pool=pl))
    buf = torch.zeros(64, dtype=torch.uint8, device="cuda")
    tc.tc_kv_pack(empty, [buf, buf], [buf])                # no-op, returns TC_OK
    plan = tc.tc_plan_create(tc.kv_spec(tc.TC_KV_PACK, s, src_pool=pl, T=src.T, bt_off=src.bt_off, bt_src=src.bt))
    with pytest.raises(tc.TensorCastError) as e:
        tc.tc_kv_pack(plan, [buf], [buf])                  # the pool has two table slots
    assert e.value.status == tc.TC_ERR_INVALID_ARG
    with pytest.raises(tc.TensorCastError) as e:
        tc.tc_kv_pack(plan, [buf, 0], [buf])               # NULL table entry
    assert e.value.status == tc.TC_ERR_INVALID_ARG
    pageable = np.zeros(1400832, dtype=np.uint8)           # ordinary host memory: the kernel could not address it
    pool_ok = torch.zeros(2 * NB * shape.chunk_bytes, dtype=torch.uint8, device="cuda")
    with pytest.raises(tc.TensorCastError) as e:
        tc.tc_kv_pack(plan, [pool_ok, pool_ok[NB * shape.chunk_bytes:]], [pageable])
    assert e.value.status == tc.TC_ERR_INVALID_ARG and "pageable" in str(e.value)
    soon = time.clock_gettime_ns(time.CLOCK_MONOTONIC) + 50_000_000
    late = tc.tc_plan_create(tc.kv_spec(tc.TC_KV_PACK, s, src_pool=pl, T=src.T, bt_off=src.bt_off, bt_src=src.bt, deadline_ns=soon))
    time.sleep(0.1)
    out = Guarded(1400832)
    pool = torch.zeros(2 * NB * shape.chunk_bytes, dtype=torch.uint8, device="cuda")
    with pytest.raises(tc.TensorCastError) as e:
        tc.tc_kv_pack(late, [pool, pool[NB * shape.chunk_bytes:]], [out.ptr()])
    assert e.value.status == tc.TC_ERR_DEADLINE
    assert (out.result() == 0xA5).all()                     # nothing was launched
    assert plan.stats().device_bytes > 0 and plan.stats().executable
    # the caches can be dropped at any time; the library allocates again on demand
    free0 = torch.cuda.mem_get_info()[0]
    staged = tc.tc_plan_create(tc.kv_spec(tc.TC_KV_PACK, s, src_pool=pl, T=src.T, bt_off=src.bt_off, bt_src=src.bt, flags=tc.TC_PLAN_STAGED))
    staged.destroy()
    plan.destroy()
    late.destroy()
    empty.destroy()
    tc.tc_trim()
    assert torch.cuda.mem_get_info()[0] >= free0
    again = tc.tc_plan_create(tc.kv_spec(tc.TC_KV_PACK, s, src_pool=pl, T=src.T, bt_off=src.bt_off, bt_src=src.bt, flags=tc.TC_PLAN_STAGED))
    host = torch.zeros(1400832, dtype=torch.uint8).pin_memory()
    tc.tc_kv_pack(again, [pool_ok, pool_ok[NB * shape.chunk_bytes:]], [host])
    torch.cuda.synchronize()
    assert not host.numpy().any()                         # an all-zero pool packs to zeros
