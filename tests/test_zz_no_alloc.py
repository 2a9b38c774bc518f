"""tc_kv_pack_noalloc: the KV pack for callers that must not allocate device memory.

An engine that has given all free HBM to its KV pool, or a scheduler loop that cannot take
the stall of a cudaMalloc, cannot use tc_plan_create (which keeps a plan's descriptors in
freshly allocated device memory).  tc_kv_pack_noalloc runs the same kernel with the
descriptors in a fixed 1 MiB scratch area inside the library.  This test drives it through
the C ABI twice in a row - the second call reuses the scratch area the first one filled - and
requires byte-for-byte the output of the ordinary tc_plan_create + tc_kv_pack path, then
checks that an over-large request is refused.  It is collected last on purpose."""
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
        tc.tc_kv_pack(plan, [pool], [want], stream.cuda_stream)
        got = torch.full((nbytes + 512,), 0x22, dtype=torch.uint8, device="cuda")
        spec, keep = make()
        tc.tc_kv_pack_noalloc(spec, [pool], [got], stream.cuda_stream)
        stream.synchronize()
        assert torch.equal(got[:nbytes], want)
        assert bool((got[nbytes:] == 0x22).all())          # nothing written past the packed bytes
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
