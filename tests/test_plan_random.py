"""Randomised checks of the plan builder on the CPU: hypothesis draws KV geometries (odd head
dims, every element size, both layouts on both sides, padded block strides, zero-length and
single-token requests, tiny tiles) and weight specs (1-4 dims, any split dim, misaligned
offsets); the lowered descriptors are interpreted in numpy and must reproduce the oracle's
bytes with every destination byte written exactly once."""
import numpy as np
from hypothesis import HealthCheck, given, settings, strategies as st

import oracle
import paper_2608_06007_b200 as tc
from helpers import planes_of, run_descriptors, run_tile_range

HOST = tc.TC_PLAN_HOST_ONLY
COMMON = dict(deadline=None, suppress_health_check=[HealthCheck.too_slow, HealthCheck.data_too_large])


@st.composite
def kv_cases(draw):
    L = draw(st.integers(1, 3))
    B = draw(st.sampled_from([1, 2, 3, 4, 8, 16]))
    H = draw(st.integers(1, 4))
    D = draw(st.sampled_from([1, 3, 4, 7, 8, 16, 33, 64]))
    E = draw(st.sampled_from([1, 2, 4, 8]))
    R = draw(st.integers(0, 5))
    T = [draw(st.sampled_from([0, 1, B, B + 1, 2 * B, 3 * B - 1, 5 * B + B // 2])) for _ in range(R)]
    pad = draw(st.sampled_from([0, E, 16, 48]))
    tile = draw(st.sampled_from([0, 512, 1024, 4096]))
    seed = draw(st.integers(0, 2 ** 31))
    h0 = draw(st.integers(0, H - 1))
    hs = draw(st.integers(0, H - h0))   # 0 = all heads from h0... (library: 0 means H - h0)
    order = draw(st.sampled_from([0, 1]))
    return (L, B, H, D, E), T, pad, tile, seed, draw(st.sampled_from([0, 1])), draw(st.sampled_from([0, 1])), draw(st.booleans()), h0, hs, order


@settings(max_examples=150, **COMMON)
@given(kv_cases())
def test_random_kv_pack_unpack_migrate(case):
    shape, T, pad, tile, seed, pool_l, other_l, one_slot, h0, hs, order = case
    L, B, H, D, E = shape
    rng = np.random.default_rng(seed)
    T = np.array(T, dtype=np.int64)
    off = np.concatenate([[0], np.cumsum((T + B - 1) // B)]).astype(np.int64)
    NB = int(off[-1]) + 3
    chunk = B * H * D * E
    stride = chunk + pad
    pool = rng.integers(0, 256, L * 2 * NB * stride, dtype=np.uint8)
    bt = rng.permutation(NB)[:off[-1]].astype(np.int32)
    bt2 = rng.permutation(NB)[:off[-1]].astype(np.int32)
    tune = dict(tile_bytes=tile) if tile else None
    if one_slot:
        pl = tc.pool(pool_l, NB, 1, plane_stride=NB * stride, block_stride=stride, slot_bytes=pool.size)
        tabs = lambda a: [a]
    else:
        pl = tc.pool(pool_l, NB, L * 2, block_stride=stride, slot_bytes=NB * stride)
        tabs = lambda a: planes_of(a, L * 2)
    # pack (the packed side holds heads [h0, h0+hs) in the drawn order)
    okw = dict(order=order, head_begin=h0, head_count=hs or None)
    lkw = dict(packed_order=order, head_begin=h0, head_count=hs)
    want = np.zeros(oracle.packed_nbytes(shape, T, hs or H - h0), dtype=np.uint8)
    oracle.kv_pack(shape, pool_l, stride, planes_of(pool, L * 2), T, off, bt, other_l, want, **okw)
    plan = tc.tc_plan_create(tc.kv_spec(tc.TC_KV_PACK, shape, src_pool=pl, packed_layout=other_l, T=T, bt_off=off, bt_src=bt, flags=HOST, tuning=tune, **lkw))
    got = np.full(want.size, 0xCC, dtype=np.uint8)
    cnt = [np.zeros(want.size, dtype=np.int32)]
    run_descriptors(plan.descriptors(0), tabs(pool), [got], cnt)
    assert np.array_equal(got, want) and (cnt[0] == 1).all()
    # unpack
    want_pool = np.full_like(pool, 0xA5)
    oracle.kv_unpack(shape, pool_l, stride, planes_of(want_pool, L * 2), T, off, bt2, other_l, want, **okw)
    plan = tc.tc_plan_create(tc.kv_spec(tc.TC_KV_UNPACK, shape, dst_pool=pl, packed_layout=other_l, T=T, bt_off=off, bt_dst=bt2, flags=HOST, tuning=tune, **lkw))
    got_pool = np.full_like(pool, 0xA5)
    run_descriptors(plan.descriptors(1), [want], tabs(got_pool))
    assert np.array_equal(got_pool, want_pool)
    # migrate into a pool of the other layout
    want_pool = np.full_like(pool, 0x5A)
    oracle.kv_migrate(shape, pool_l, stride, planes_of(pool, L * 2), other_l, stride, planes_of(want_pool, L * 2), T, off, bt, bt2)
    pl2 = tc.pool(other_l, NB, L * 2, block_stride=stride, slot_bytes=NB * stride)
    plan = tc.tc_plan_create(tc.kv_spec(tc.TC_KV_MIGRATE, shape, src_pool=pl, dst_pool=pl2, T=T, bt_off=off, bt_src=bt, bt_dst=bt2, flags=HOST, tuning=tune))
    got_pool = np.full_like(pool, 0x5A)
    run_descriptors(plan.descriptors(0), tabs(pool), planes_of(got_pool, L * 2))
    assert np.array_equal(got_pool, want_pool)
    st_ = plan.stats()
    assert st_.payload_bytes[0] == oracle.packed_nbytes(shape, T)


@st.composite
def weight_cases(draw):
    n = draw(st.integers(1, 4))
    tensors = []
    for _ in range(n):
        ndim = draw(st.integers(1, 4))
        shape = [draw(st.sampled_from([1, 2, 3, 4, 6, 8, 12])) for _ in range(ndim)] + [1] * (4 - ndim)
        E = draw(st.sampled_from([1, 2, 4, 8]))
        world = draw(st.sampled_from([1, 2, 3, 4]))
        dims_ok = [m for m in range(ndim) if shape[m] % world == 0]
        split = draw(st.sampled_from(dims_ok)) if dims_ok and draw(st.booleans()) else -1
        gap = draw(st.sampled_from([0, 1, 2, 16]))
        tensors.append((ndim, shape, E, split, gap))
    return tensors, draw(st.sampled_from([1, 2, 3, 4])), draw(st.integers(0, 2 ** 31)), draw(st.sampled_from([0, 512]))


@settings(max_examples=150, **COMMON)
@given(weight_cases())
def test_random_weight_specs(case):
    tensors, world, seed, tile = case
    rng = np.random.default_rng(seed)
    # keep only splits that divide by the drawn world
    offs, nbytes, E, ndim, shapes, split = [], [], [], [], [], []
    cur = 0
    for nd, shp, e, sd, gap in tensors:
        cur += gap
        if sd >= 0 and shp[sd] % world:
            sd = -1
        offs.append(cur)
        nb = int(np.prod(shp)) * e
        nbytes.append(nb)
        E.append(e)
        ndim.append(nd)
        shapes.append(shp)
        split.append(sd)
        cur += nb
    blob = rng.integers(0, 256, cur + 7, dtype=np.uint8)
    rank = int(rng.integers(0, world))
    sizes = [nb // (world if sd >= 0 else 1) for nb, sd in zip(nbytes, split)]
    want = [np.zeros(n, dtype=np.uint8) for n in sizes]
    oracle.weights(offs, E, shapes, split, rank, world, blob, want)
    plan = tc.tc_plan_create(tc.weights_spec(offs, nbytes, E, ndim, shapes, split_dim=split, rank=rank, world=world, blob_bytes=blob.size,
                                             flags=HOST, tuning=dict(tile_bytes=tile) if tile else None))
    got = [np.full(n, 0xEE, dtype=np.uint8) for n in sizes]
    cnt = [np.zeros(n, dtype=np.int32) for n in sizes]
    run_descriptors(plan.descriptors(0), [blob], got, cnt)
    for g, w, c in zip(got, want, cnt):
        assert np.array_equal(g, w) and (c == 1).all()
    # the same spec cut into chunks for streaming: every chunk's staging bytes cover what its tiles read
    plan = tc.tc_plan_create(tc.weights_spec(offs, nbytes, E, ndim, shapes, split_dim=split, rank=rank, world=world, blob_bytes=blob.size,
                                             flags=HOST | tc.TC_PLAN_STREAM, tuning=dict(tile_bytes=tile) if tile else None))
    got = [np.full(n, 0xEE, dtype=np.uint8) for n in sizes]
    cnt = [np.zeros(n, dtype=np.int32) for n in sizes]
    descs = plan.descriptors(0)
    for sg in plan.segments(0):
        assert sg.host_off % 4096 == 0 and sg.host_off + sg.bytes <= blob.size
        run_tile_range(descs, sg.tile0, sg.n_tiles, [blob[sg.host_off:sg.host_off + sg.bytes].copy()], got, cnt, src_shift=sg.host_off)
    for g, w, c in zip(got, want, cnt):
        assert np.array_equal(g, w) and (c == 1).all()
