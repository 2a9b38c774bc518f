"""tc_kv_pack_noalloc: the KV pack for callers that must not allocate device memory.

An engine that has given all free HBM to its KV pool, or a scheduler loop that cannot take
the stall of a cudaMalloc, cannot use tc_plan_create (which keeps a plan's descriptors in
freshly allocated device memory).  tc_kv_pack_noalloc runs the same kernel with the
descriptors in a fixed 1 MiB scratch area inside the library.  This test drives it through
the C ABI twice in a row - the second call reuses the scratch area the first one filled - and
requires byte-for-byte the output of the ordinary tc_plan_create + tc_kv_pack path; it checks
that the calls leave the amount of free device memory unchanged (the reason the entry point
exists), that requests which move nothing succeed, that pool-to-pool specs and ragged
geometries go through it too, and that an over-large request is refused.  It is collected
last on purpose."""
import numpy as np
import pytest
import torch

import paper_2608_06007_b200 as tc
import workloads as wl

pytestmark = pytest.mark.gpu


def _case(seed, packed_layout, T):
    shape = wl.KVShape(L=3, B=16, H=8, D=128, E=2)
    NB = 96
    T = np.array(T, dtype=np.int64)
    off = np.concatenate([[0], np.cumsum((T + shape.B - 1) // shape.B)]).astype(np.int64)
    bt = np.random.default_rng(seed).permutation(NB)[:off[-1]].astype(np.int32)
    pool = torch.empty(NB * shape.block_bytes, dtype=torch.uint8, device="cuda")
    wl.fill_torch(pool, seed)
    pl = tc.pool(tc.TC_NHD, NB, 1, plane_stride=NB * shape.chunk_bytes, slot_bytes=pool.numel())
    make = lambda: tc.kv_spec(tc.TC_KV_PACK, shape.tuple, src_pool=pl, packed_layout=packed_layout, T=T, bt_off=off, bt_src=bt)
    nbytes = int(T.sum()) * shape.token_bytes
    return make, pool, nbytes


def test_noalloc_pack_matches_planned_pack_on_two_calls_in_a_row():
    cases = [_case(31, tc.TC_HND, (200, 37, 0, 5, 400)), _case(32, tc.TC_NHD, (16, 333, 90))]
    stream = torch.cuda.Stream()
    for make, pool, nbytes in cases:
        want = torch.full((nbytes,), 0x11, dtype=torch.uint8, device="cuda")
        plan = tc.tc_plan_create(make())
        got = torch.full((nbytes + 512,), 0x22, dtype=torch.uint8, device="cuda")
        torch.cuda.synchronize()                           # the fills ran on the default stream
        tc.tc_kv_pack(plan, [pool], [want], stream.cuda_stream)
        spec, keep = make()
        tc.tc_kv_pack_noalloc(spec, [pool], [got], stream.cuda_stream)
        stream.synchronize()
        assert torch.equal(got[:nbytes], want)
        assert bool((got[nbytes:] == 0x22).all())          # nothing written past the packed bytes
        plan.destroy()


def test_noalloc_calls_leave_free_device_memory_unchanged():
    make, pool, nbytes = _case(33, tc.TC_HND, (100, 64, 7))
    got = torch.zeros(nbytes, dtype=torch.uint8, device="cuda")
    stream = torch.cuda.Stream()
    torch.cuda.synchronize()
    tc.tc_kv_pack_noalloc(make()[0], [pool], [got], stream.cuda_stream)   # first call on the device: resolves the scratch address
    stream.synchronize()
    free0 = torch.cuda.mem_get_info()[0]
    for _ in range(3):
        spec, keep = make()
        tc.tc_kv_pack_noalloc(spec, [pool], [got], stream.cuda_stream)
    stream.synchronize()
    assert torch.cuda.mem_get_info()[0] == free0


def test_noalloc_requests_that_move_nothing_return_ok():
    shape = wl.KVShape(L=2, B=16, H=8, D=128, E=2)
    pl = tc.pool(tc.TC_NHD, 8, 1, plane_stride=8 * shape.chunk_bytes)
    pool = torch.zeros(8 * shape.block_bytes, dtype=torch.uint8, device="cuda")
    out = torch.full((64,), 0x22, dtype=torch.uint8, device="cuda")
    empty = tc.kv_spec(tc.TC_KV_PACK, shape.tuple, src_pool=pl)                                        # R = 0
    zeros = tc.kv_spec(tc.TC_KV_PACK, shape.tuple, src_pool=pl, T=[0, 0, 0], bt_off=[0, 0, 0, 0],
                       bt_src=np.zeros(0, dtype=np.int32))                                             # every T_r = 0
    for spec, keep in (empty, zeros):
        tc.tc_kv_pack_noalloc(spec, [pool], [out])
    torch.cuda.synchronize()
    assert bool((out == 0x22).all())
    with pytest.raises(tc.TensorCastError) as e:                                                       # asks for a plan that is not run
        tc.tc_kv_pack_noalloc(tc.kv_spec(tc.TC_KV_PACK, shape.tuple, src_pool=pl, flags=tc.TC_PLAN_HOST_ONLY)[0], [pool], [out])
    assert e.value.status == tc.TC_ERR_INVALID_ARG


def test_noalloc_runs_migrate_specs_and_ragged_geometries():
    """Pool to pool through the same entry point, and a geometry whose descriptors own unequal
    numbers of tiles (36 KiB planes next to a short last block), which needs the tile list in the
    scratch area as well as the descriptors."""
    shape = wl.KVShape(L=2, B=18, H=8, D=128, E=2)          # 36 KiB planes: more than one tile part
    NB = 40
    T = np.array([18 * 5, 3, 18 * 2 + 1, 18], dtype=np.int64)
    off = np.concatenate([[0], np.cumsum((T + shape.B - 1) // shape.B)]).astype(np.int64)
    rng = np.random.default_rng(34)
    bt_s, bt_d = rng.permutation(NB)[:off[-1]].astype(np.int32), rng.permutation(NB)[:off[-1]].astype(np.int32)
    src = torch.empty(NB * shape.block_bytes, dtype=torch.uint8, device="cuda")
    wl.fill_torch(src, 34)
    pl = tc.pool(tc.TC_NHD, NB, 1, plane_stride=NB * shape.chunk_bytes, slot_bytes=src.numel())
    pl_h = tc.pool(tc.TC_HND, NB, 1, plane_stride=NB * shape.chunk_bytes, slot_bytes=src.numel())
    stream = torch.cuda.Stream()
    for dst_pool in (pl, pl_h):
        make = lambda: tc.kv_spec(tc.TC_KV_MIGRATE, shape.tuple, src_pool=pl, dst_pool=dst_pool, T=T, bt_off=off, bt_src=bt_s, bt_dst=bt_d)
        want = torch.full_like(src, 0xA5)
        plan = tc.tc_plan_create(make())
        torch.cuda.synchronize()                           # the fills ran on the default stream
        tc.tc_kv_pack(plan, [src], [want], stream.cuda_stream)
        for _ in range(2):
            got = torch.full_like(src, 0xA5)
            torch.cuda.synchronize()
            spec, keep = make()
            tc.tc_kv_pack_noalloc(spec, [src], [got], stream.cuda_stream)
            stream.synchronize()
            assert torch.equal(got, want)
        plan.destroy()
    # a PACK whose blocks own very unequal numbers of tiles: the plan then carries an explicit
    # tile -> descriptor list, which travels through the scratch area behind the descriptors
    T2 = np.array([18] + [1] * 8, dtype=np.int64)
    off2 = np.arange(len(T2) + 1, dtype=np.int64)
    make = lambda: tc.kv_spec(tc.TC_KV_PACK, shape.tuple, src_pool=pl, packed_layout=tc.TC_HND, T=T2, bt_off=off2, bt_src=bt_s[:len(T2)],
                              tuning=dict(tile_bytes=8192))
    nbytes = int(T2.sum()) * shape.token_bytes
    want = torch.zeros(nbytes, dtype=torch.uint8, device="cuda")
    plan = tc.tc_plan_create(make())
    assert plan.stats().n_tiles[0] == (5 + 8) * shape.L * 2          # listed: no padding tiles
    tc.tc_kv_pack(plan, [src], [want], stream.cuda_stream)
    got = torch.zeros(nbytes, dtype=torch.uint8, device="cuda")
    tc.tc_kv_pack_noalloc(make()[0], [src], [got], stream.cuda_stream)
    stream.synchronize()
    assert torch.equal(got, want)
    plan.destroy()


def test_noalloc_rejects_requests_beyond_its_scratch_capacity():
    shape = wl.KVShape(L=1, B=16, H=8, D=128, E=2)
    n_blocks = tc.TC_NOALLOC_SCRATCH_BYTES // 128 + 1       # one 128-byte descriptor per block
    T = np.array([n_blocks * shape.B], dtype=np.int64)
    off = np.array([0, n_blocks], dtype=np.int64)
    bt = np.arange(n_blocks, dtype=np.int32)
    pl = tc.pool(tc.TC_NHD, n_blocks, 2)
    spec, keep = tc.kv_spec(tc.TC_KV_PACK, shape.tuple, src_pool=pl, T=T, bt_off=off, bt_src=bt)
    buf = torch.zeros(64, dtype=torch.uint8, device="cuda")
    with pytest.raises(tc.TensorCastError) as e:
        tc.tc_kv_pack_noalloc(spec, [buf, buf], [buf])
    assert e.value.status == tc.TC_ERR_TOO_LARGE
    with pytest.raises(tc.TensorCastError) as e:
        tc.tc_kv_pack_noalloc(tc.kv_spec(tc.TC_KV_UNPACK, shape.tuple, dst_pool=pl), [buf], [buf, buf])
    assert e.value.status == tc.TC_ERR_KIND
