"""Host-side tests of the C-ABI library that need no GPU: the exported symbols, the plan
builder's validation (every error is raised before any launch) and its lowering, checked by
interpreting the lowered descriptors in numpy and comparing with the oracle byte for byte."""
import ctypes
import itertools
import os
import re
import time

import numpy as np
import pytest

import oracle
import paper_2608_06007_b200 as tc
import workloads as wl
from helpers import run_tile_range, run_window, ck_spec, kv_case, planes_of, run_descriptors, small_checkpoint

HOST = tc.TC_PLAN_HOST_ONLY
ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def test_library_exports_every_declared_symbol():
    header = open(os.path.join(ROOT, "include", "tensorcast.h")).read()
    declared = set(re.findall(r"TC_API\s+[\w\s\*]+?\b(tc_\w+)\s*\(", header))
    assert {"tc_plan_create", "tc_kv_pack", "tc_kv_unpack", "tc_weights_materialize", "tc_plan_destroy"} <= declared
    lib = tc.load_library()
    for name in declared:
        assert hasattr(lib, name), name
    assert declared == set(tc.EXPORTS)
    assert ctypes.sizeof(tc.binding.tc_index_entry_t) == 64


def test_header_is_plain_c_and_the_library_runs_from_a_c_client(tmp_path):
    """tests/c_abi_check.c is compiled as C11 against include/tensorcast.h and linked with the
    library; it lowers the worked micro-example and executes the descriptors by hand."""
    import subprocess
    lib = tc.build_library()
    exe = tmp_path / "c_abi_check"
    subprocess.check_call(["gcc", "-std=c11", "-Wall", "-Wextra", "-Werror", "-pedantic", "-I", os.path.join(ROOT, "include"),
                           os.path.join(ROOT, "tests", "c_abi_check.c"), "-o", str(exe), lib, "-Wl,-rpath," + os.path.dirname(lib)])
    out = subprocess.run([str(exe)], capture_output=True, text=True, timeout=60)
    assert out.returncode == 0 and out.stdout.strip() == "ok", out.stdout + out.stderr


def test_fast_division_constants_are_exact():
    # the kernels divide by runtime constants with a multiply-high; replay that arithmetic
    rng = np.random.default_rng(0)
    ds = np.unique(np.concatenate([np.arange(1, 300), rng.integers(1, 1 << 20, 300), [1 << 20, (1 << 20) - 1, 3584, 28672]]))
    ns = np.unique(np.concatenate([np.arange(0, 5000), rng.integers(0, 1 << 31, 5000), [(1 << 31) - 1]])).astype(np.uint64)
    for d in ds:
        d = int(d)
        s = 0
        while (1 << s) < d:
            s += 1
        mul = ((1 << 32) * ((1 << s) - d)) // d + 1
        assert mul < (1 << 32)
        q = (((ns * np.uint64(mul)) >> np.uint64(32)) + ns) >> np.uint64(s)
        assert np.array_equal(q, ns // np.uint64(d)), d


# --------------------------------------------------------------------------- KV lowering
LAYOUTS = [tc.TC_NHD, tc.TC_HND]


@pytest.mark.parametrize("pool_l,packed_l", list(itertools.product(LAYOUTS, LAYOUTS)))
@pytest.mark.parametrize("slots", ["planes", "one"])
def test_pack_and_unpack_lowering_match_oracle(pool_l, packed_l, slots):
    rng = np.random.default_rng(1)
    shape, NB, stride, pool, T, off, bt = kv_case(rng, T=(5, 0, 11, 1, 8), pad_blocks=16)
    L = shape[0]
    planes = planes_of(pool, L * 2)
    want = np.zeros(oracle.packed_nbytes(shape, T), dtype=np.uint8)
    oracle.kv_pack(shape, pool_l, stride, planes, T, off, bt, packed_l, want)
    if slots == "planes":
        pl = tc.pool(pool_l, NB, L * 2, block_stride=stride, slot_bytes=planes[0].size)
        tables = planes
    else:
        pl = tc.pool(pool_l, NB, 1, plane_stride=planes[0].size, block_stride=stride, slot_bytes=pool.size)
        tables = [pool]
    plan = tc.tc_plan_create(tc.kv_spec(tc.TC_KV_PACK, shape, src_pool=pl, packed_layout=packed_l, T=T, bt_off=off, bt_src=bt, flags=HOST, tuning=dict(tile_bytes=512)))
    st = plan.stats()
    assert st.packed_bytes_required == want.size and st.payload_bytes[0] == want.size and not st.executable
    got = np.full(want.size, 0xCC, dtype=np.uint8)
    cnt = [np.zeros(want.size, dtype=np.int32)]
    run_descriptors(plan.descriptors(0), tables, [got], cnt)
    assert np.array_equal(got, want) and (cnt[0] == 1).all()
    # unpack through a fresh table into a sentinel pool
    bt2 = rng.permutation(NB)[:off[-1]].astype(np.int32)
    want_pool = np.full_like(pool, 0xA5)
    oracle.kv_unpack(shape, pool_l, stride, planes_of(want_pool, L * 2), T, off, bt2, packed_l, want)
    plan2 = tc.tc_plan_create(tc.kv_spec(tc.TC_KV_UNPACK, shape, dst_pool=pl, packed_layout=packed_l, T=T, bt_off=off, bt_dst=bt2, flags=HOST))
    got_pool = np.full_like(pool, 0xA5)
    run_descriptors(plan2.descriptors(1), [want], planes_of(got_pool, L * 2) if slots == "planes" else [got_pool])
    assert np.array_equal(got_pool, want_pool)
    assert plan2.stats().n_descriptors[0] == 0 and plan2.stats().n_descriptors[1] > 0


@pytest.mark.parametrize("src_l,dst_l", list(itertools.product(LAYOUTS, LAYOUTS)))
def test_migrate_lowering_matches_oracle_including_page_first_pool(src_l, dst_l):
    rng = np.random.default_rng(2)
    shape, NB, stride, pool, T, off, bt = kv_case(rng, T=(7, 12, 2))
    L, B, H, D, E = shape
    chunk = B * H * D * E
    NB2 = NB + 2
    bt2 = rng.permutation(NB2)[:off[-1]].astype(np.int32)
    # destination: page-first pool [block][plane][chunk]
    dst = np.full(NB2 * L * 2 * chunk, 0x5A, dtype=np.uint8)
    want = dst.copy()
    oracle.kv_migrate(shape, src_l, stride, planes_of(pool, L * 2), dst_l, L * 2 * chunk,
                      [want[p * chunk:] for p in range(L * 2)], T, off, bt, bt2)
    sp = tc.pool(src_l, NB, L * 2, block_stride=stride)
    dp = tc.pool(dst_l, NB2, 1, plane_stride=chunk, block_stride=L * 2 * chunk, slot_bytes=dst.size)
    plan = tc.tc_plan_create(tc.kv_spec(tc.TC_KV_MIGRATE, shape, src_pool=sp, dst_pool=dp, T=T, bt_off=off, bt_src=bt, bt_dst=bt2, flags=HOST))
    run_descriptors(plan.descriptors(0), planes_of(pool, L * 2), [dst])
    assert np.array_equal(dst, want)


def test_same_layout_full_blocks_lower_to_one_run_per_block():
    shape, NB, src, dst = wl.config1()
    pl = tc.pool(tc.TC_NHD, NB, 1, plane_stride=NB * shape.chunk_bytes)
    plan = tc.tc_plan_create(tc.kv_spec(tc.TC_KV_PACK, shape.tuple, src_pool=pl, T=src.T, bt_off=src.bt_off, bt_src=src.bt, flags=HOST))
    ds = plan.descriptors(0)
    assert len(ds) == 24                                   # one descriptor per (request, block)
    assert all(d.rows == 1 and d.n_outer == 2 for d in ds)
    assert sorted(d.run_bytes for d in ds)[-1] == shape.chunk_bytes
    st = plan.stats()
    assert st.payload_bytes[0] == 1400832 and st.vec_bytes[0] == 16 and st.n_tiles[0] == 48


def test_mixed_plan_groups_match_oracle():
    shape = (2, 4, 2, 8, 2)
    L, B, H, D, E = shape
    chunk = B * H * D * E
    step = next(wl.config5(NB_dev=40, NB_host=60, sessions=5, steps=1, shape=wl.KVShape(*shape), p=0.5, max_prefix=4, max_new=2))
    rng = np.random.default_rng(3)
    dev = rng.integers(0, 256, L * 2 * 40 * chunk, dtype=np.uint8)        # plane-major, NHD
    host = rng.integers(0, 256, 60 * L * 2 * chunk, dtype=np.uint8)       # page-first, HND
    dev_pool = tc.pool(tc.TC_NHD, 40, 1, plane_stride=40 * chunk)
    host_pool = tc.pool(tc.TC_HND, 60, 1, plane_stride=chunk, block_stride=L * 2 * chunk)
    spec = tc.kv_spec(tc.TC_KV_MIXED, shape, src_pool=dev_pool, dst_pool=host_pool,
                      T=step.offload_T, bt_off=step.offload_off, bt_src=step.offload_dev, bt_dst=step.offload_host,
                      reload=dict(T=step.reload_T, bt_off=step.reload_off, bt_src=step.reload_host, bt_dst=step.reload_dev), flags=HOST)
    plan = tc.tc_plan_create(spec)
    want_dev, want_host = dev.copy(), host.copy()
    hp = lambda a: [a[p * chunk:] for p in range(L * 2)]
    oracle.kv_migrate(shape, oracle.NHD, chunk, planes_of(dev, L * 2), oracle.HND, L * 2 * chunk, hp(want_host),
                      step.offload_T, step.offload_off, step.offload_dev, step.offload_host)
    oracle.kv_migrate(shape, oracle.HND, L * 2 * chunk, hp(host), oracle.NHD, chunk, planes_of(want_dev, L * 2),
                      step.reload_T, step.reload_off, step.reload_host, step.reload_dev)
    got_dev, got_host = dev.copy(), host.copy()
    run_descriptors(plan.descriptors(0), [dev], [got_host])
    run_descriptors(plan.descriptors(1), [host], [got_dev])
    assert np.array_equal(got_dev, want_dev) and np.array_equal(got_host, want_host)
    # an offload target that the reload group reads is refused
    bad = step.offload_host.copy()
    bad[0] = step.reload_host[0]
    with pytest.raises(tc.TensorCastError) as e:
        tc.tc_plan_create(tc.kv_spec(tc.TC_KV_MIXED, shape, src_pool=dev_pool, dst_pool=host_pool,
                                     T=step.offload_T, bt_off=step.offload_off, bt_src=step.offload_dev, bt_dst=bad,
                                     reload=dict(T=step.reload_T, bt_off=step.reload_off, bt_src=step.reload_host, bt_dst=step.reload_dev), flags=HOST))
    assert e.value.status == tc.TC_ERR_OVERLAP


# --------------------------------------------------------------------------- weights lowering
@pytest.mark.parametrize("variant", ["tight", "permuted_misaligned"])
@pytest.mark.parametrize("world", [1, 4])
def test_weights_lowering_matches_oracle(variant, world):
    ck = small_checkpoint() if variant == "tight" else small_checkpoint(order_seed=3, pad_to=1, lead_pad=2)
    blob = np.random.default_rng(4).integers(0, 256, ck.nbytes_total, dtype=np.uint8)
    for rank in range(world):
        split = ck.split_dim if world > 1 else np.full(ck.N, -1)
        sizes = [ck.nbytes(i) // (world if split[i] >= 0 else 1) for i in range(ck.N)]
        want = [np.zeros(n, dtype=np.uint8) for n in sizes]
        oracle.weights(ck.byte_off, ck.E, ck.shapes, split, rank, world, blob, want)
        plan = tc.tc_plan_create(ck_spec(ck, split_dim=split, rank=rank, world=world, flags=HOST, tuning=dict(tile_bytes=1024)))
        got = [np.full(n, 0xEE, dtype=np.uint8) for n in sizes]
        cnt = [np.zeros(n, dtype=np.int32) for n in sizes]
        run_descriptors(plan.descriptors(0), [blob], got, cnt)
        for i in range(ck.N):
            assert np.array_equal(got[i], want[i]), ck.names[i]
            assert (cnt[i] == 1).all()
        st = plan.stats()
        assert st.payload_bytes[0] == sum(sizes)
        assert st.vec_bytes[0] == (16 if variant == "tight" else 2)


def test_weights_transform_into_fused_target():
    """q, k, v of one layer written side by side into one fused qkv buffer (dst_slot / dst_off),
    and a middle-dim split written into a strided window."""
    ck = small_checkpoint()
    blob = np.random.default_rng(5).integers(0, 256, ck.nbytes_total, dtype=np.uint8)
    ids = [ck.names.index(f"layers.0.{n}_proj") for n in "qkv"]
    sizes = [ck.nbytes(i) for i in ids]
    offs = np.concatenate([[0], np.cumsum(sizes)])
    nb = [ck.nbytes(i) for i in ids]
    spec = tc.weights_spec(ck.byte_off[ids], nb, ck.E[ids], ck.ndim[ids], ck.shapes[ids], blob_bytes=blob.size,
                           dst_slot=[0, 0, 0], dst_off=offs[:3], n_dst=1, dst_bytes=[offs[-1]], flags=HOST)
    plan = tc.tc_plan_create(spec)
    fused = np.zeros(offs[-1], dtype=np.uint8)
    run_descriptors(plan.descriptors(0), [blob], [fused])
    want = np.concatenate([blob[ck.byte_off[i]:ck.byte_off[i] + ck.nbytes(i)] for i in ids])
    assert np.array_equal(fused, want)
    # overlapping windows are refused
    with pytest.raises(tc.TensorCastError) as e:
        tc.tc_plan_create(tc.weights_spec(ck.byte_off[ids], nb, ck.E[ids], ck.ndim[ids], ck.shapes[ids], blob_bytes=blob.size,
                                          dst_slot=[0, 0, 0], dst_off=[0, sizes[0] - 2, offs[2]], n_dst=1, dst_bytes=[offs[-1]], flags=HOST))
    assert e.value.status == tc.TC_ERR_OVERLAP
    # strided window, middle-dim split: same case as the oracle pin
    rng = np.random.default_rng(4)
    full = rng.integers(0, 2 ** 32, (4, 6, 5), dtype=np.uint32)
    blob2 = np.concatenate([np.zeros(3, dtype=np.uint8), full.reshape(-1).view(np.uint8)])
    spec = tc.weights_spec([3], [full.nbytes], [4], [3], [[4, 6, 5, 1]], split_dim=[1], rank=2, world=3, blob_bytes=blob2.size,
                           dst_slot=[0], dst_off=[12], dst_stride=[[64, 32, 4, 4]], n_dst=1, dst_bytes=[4 * 2 * 8 * 4], flags=HOST)
    target = np.zeros((4, 2, 8), dtype=np.uint32)
    run_descriptors(tc.tc_plan_create(spec).descriptors(0), [blob2], [target.reshape(-1).view(np.uint8)])
    want = np.zeros_like(target)
    want[:, :, 3:8] = full[:, 4:6, :]
    assert np.array_equal(target, want)


def test_a_tensor_whose_own_destination_strides_overlap_is_refused():
    """dst_stride can make one tensor overlap itself: rows closer together than they are long, or
    elements closer than an element.  Those would write a destination byte twice with different
    values; strides that interleave without colliding stay legal."""
    blob = np.arange(4 * 8 * 2, dtype=np.uint8)
    def create(stride, dst_bytes, shape=(4, 8)):
        spec = tc.weights_spec([0], [shape[0] * shape[1] * 2], [2], [2], [[shape[0], shape[1], 1, 1]], blob_bytes=blob.size,
                               dst_slot=[0], dst_off=[0], dst_stride=[stride], n_dst=1, dst_bytes=[dst_bytes], flags=HOST)
        return tc.tc_plan_create(spec)
    for stride in ([8, 2, 2, 2], [2, 2, 2, 2], [16, 1, 1, 1]):      # rows 8 B apart but 16 B long; rows 2 B apart; elements 1 B apart
        with pytest.raises(tc.TensorCastError) as e:
            create(stride, 256)
        assert e.value.status == tc.TC_ERR_OVERLAP, stride
    # a transpose (strides nest the other way round) and padded rows are fine
    for stride, nbytes in (([2, 8, 2, 2], 64), ([32, 2, 2, 2], 128)):
        plan = create(stride, nbytes)
        out, cnt = np.zeros(nbytes, dtype=np.uint8), [np.zeros(nbytes, dtype=np.int32)]
        run_descriptors(plan.descriptors(0), [blob], [out], cnt)
        assert cnt[0].max() == 1 and cnt[0].sum() == 64
    # strides that do not nest but never collide: element (i, j) of a [2, 3] tensor at 3i + 2j
    plan = create([6, 4, 2, 2], 16, shape=(2, 3))
    out, cnt = np.zeros(16, dtype=np.uint8), [np.zeros(16, dtype=np.int32)]
    run_descriptors(plan.descriptors(0), [blob], [out], cnt)
    assert cnt[0].max() == 1 and cnt[0].sum() == 12
    src = blob[:12].view(np.uint16).reshape(2, 3)
    got = out.view(np.uint16)
    for i in range(2):
        for j in range(3):
            assert got[3 * i + 2 * j] == src[i, j]
    # ... and the same shape with a collision: 2i + 2j puts (0, 1) on (1, 0)
    with pytest.raises(tc.TensorCastError) as e:
        create([4, 4, 2, 2], 16, shape=(2, 3))
    assert e.value.status == tc.TC_ERR_OVERLAP


def test_tp_resharding_8_to_2_and_2_to_8_by_composition_of_rules():
    """A checkpoint saved as W shard blobs, loaded at another TP degree W'.  8 -> 2: rank r' of 2
    concatenates four source shards along the split dim (dst_off / dst_stride windows, one plan
    per source blob).  2 -> 8: rank r' of 8 takes a quarter of one source shard (split of the
    shard).  Both must equal the oracle's direct W' shard of the full tensor."""
    rng = np.random.default_rng(8)
    shp, E = (16, 24), 2                                   # one [out, in] matrix, bf16-sized elements
    full = rng.integers(0, 256, shp[0] * shp[1] * E, dtype=np.uint8)
    for dim in (0, 1):
        def shard(rank, world):
            out = np.zeros(full.size // world, dtype=np.uint8)
            oracle.weights([0], [E], [[shp[0], shp[1], 1, 1]], [dim], rank, world, full, [out])
            return out
        sshape = lambda world: [shp[0] // world if dim == 0 else shp[0], shp[1] // world if dim == 1 else shp[1], 1, 1]
        # 8 -> 2
        for r2 in range(2):
            want = shard(r2, 2)
            got = np.full(want.size, 0xEE, dtype=np.uint8)
            cnt = [np.zeros(want.size, dtype=np.int32)]
            d2 = sshape(2)
            for k in range(4):                              # source shards 4*r2 .. 4*r2+3
                src_blob = shard(4 * r2 + k, 8)
                s8 = sshape(8)
                if dim == 0:
                    off, stride = k * src_blob.size, [d2[1] * E, E, E, E]
                else:
                    off, stride = k * s8[1] * E, [d2[1] * E, E, E, E]
                spec = tc.weights_spec([0], [src_blob.size], [E], [2], [s8], blob_bytes=src_blob.size, dst_slot=[0], dst_off=[off],
                                       dst_stride=[stride], n_dst=1, dst_bytes=[want.size], flags=HOST)
                run_descriptors(tc.tc_plan_create(spec).descriptors(0), [src_blob], [got], cnt)
            assert np.array_equal(got, want) and (cnt[0] == 1).all(), (dim, r2)
        # 2 -> 8
        for r8 in range(8):
            src_blob = shard(r8 // 4, 2)
            spec = tc.weights_spec([0], [src_blob.size], [E], [2], [sshape(2)], split_dim=[dim], rank=r8 % 4, world=4, blob_bytes=src_blob.size, flags=HOST)
            got = np.full(full.size // 8, 0xEE, dtype=np.uint8)
            run_descriptors(tc.tc_plan_create(spec).descriptors(0), [src_blob], [got])
            assert np.array_equal(got, shard(r8, 8)), (dim, r8)


def test_interleaved_strided_destinations_pass_the_exact_overlap_check():
    # two [4][3] byte tensors interleaved column-wise into one [4][6] target: bounding spans
    # intersect but no byte is written twice
    blob = np.arange(24, dtype=np.uint8)
    spec = tc.weights_spec([0, 12], [12, 12], [1, 1], [2, 2], [[4, 3, 1, 1]] * 2, blob_bytes=24,
                           dst_slot=[0, 0], dst_off=[0, 3], dst_stride=[[6, 1, 1, 1]] * 2, n_dst=1, dst_bytes=[24], flags=HOST)
    out = np.zeros(24, dtype=np.uint8)
    cnt = [np.zeros(24, dtype=np.int32)]
    run_descriptors(tc.tc_plan_create(spec).descriptors(0), [blob], [out], cnt)
    assert (cnt[0] == 1).all()
    assert np.array_equal(out.reshape(4, 6), np.concatenate([blob[:12].reshape(4, 3), blob[12:].reshape(4, 3)], axis=1))


def test_llama3_8b_plans_have_the_expected_size():
    ck = wl.config3()
    full = tc.tc_plan_create(ck_spec(ck, flags=HOST)).stats()
    assert full.payload_bytes[0] == 16060522496 and full.vec_bytes[0] == 16
    shard = tc.tc_plan_create(ck_spec(ck, split_dim=ck.split_dim, rank=3, world=8, flags=HOST)).stats()
    assert shard.payload_bytes[0] == 2 * 1004015616
    # 65 norms of 8 KiB are one tile each; everything else is cut into 32 KiB tiles
    assert full.n_tiles[0] == (16060522496 - 65 * 8192) // 32768 + 65


def _extent(descs, side):
    """Largest byte any descriptor touches, per table slot (src or dst side), computed in closed form."""
    hi = {}
    for d in descs:
        off, outer, s0, s1 = ((d.src_off, d.src_outer, d.src_s0, d.src_s1) if side == "src" else (d.dst_off, d.dst_outer, d.dst_s0, d.dst_s1))
        slot0, step = (d.src_slot, d.src_slot_step) if side == "src" else (d.dst_slot, d.dst_slot_step)
        n1 = d.rows // d.n0
        assert off >= 0 and s0 >= 0 and s1 >= 0 and outer >= 0
        top = off + (n1 - 1) * s1 + (d.n0 - 1) * s0 + d.run_bytes
        for o in ((0, d.n_outer - 1) if step else (d.n_outer - 1,)):
            slot = slot0 + o * step
            hi[slot] = max(hi.get(slot, 0), top + (0 if step else o * outer))
    return hi


def test_full_size_plans_stay_inside_their_buffers():
    """Closed-form bounds of every descriptor of the full-size workloads (no sanitizer runs on the
    GPU pool, so out-of-bounds lowering has to be caught here)."""
    shape = wl.LLAMA3_8B_KV
    _, NB, _, waves = wl.config2(wave_blocks=8192, NB_dst=8192)
    pool_bytes = NB * shape.block_bytes
    plA = tc.pool(tc.TC_NHD, NB, 1, plane_stride=NB * shape.chunk_bytes, slot_bytes=pool_bytes)
    for src, dst in waves[:2]:
        payload = int(src.T.sum()) * shape.token_bytes
        for order in (tc.TC_REQUEST_MAJOR, tc.TC_LAYER_MAJOR):
            plan = tc.tc_plan_create(tc.kv_spec(tc.TC_KV_PACK, shape.tuple, src_pool=plA, packed_layout=tc.TC_HND, packed_order=order,
                                                T=src.T, bt_off=src.bt_off, bt_src=src.bt, flags=HOST))
            ds = plan.descriptors(0)
            assert max(_extent(ds, "src").values()) <= pool_bytes and _extent(ds, "dst") == {0: payload}
            assert plan.stats().payload_bytes[0] == payload
    shape4 = wl.LLAMA3_70B_KV
    _, NB4, _, w4 = wl.config4(max_waves=1)
    pl4 = tc.pool(tc.TC_NHD, NB4, shape4.L * 2, slot_bytes=NB4 * shape4.chunk_bytes)
    ds = tc.tc_plan_create(tc.kv_spec(tc.TC_KV_MIGRATE, shape4.tuple, src_pool=pl4, dst_pool=pl4, T=w4[0][0].T, bt_off=w4[0][0].bt_off,
                                      bt_src=w4[0][0].bt, bt_dst=w4[0][1].bt, flags=HOST)).descriptors(0)
    for side in ("src", "dst"):
        ext = _extent(ds, side)
        assert set(ext) == {0, shape4.L * 2 - 1} and max(ext.values()) <= NB4 * shape4.chunk_bytes   # first and last plane
    ck = wl.config3()
    for kw, total in ((dict(), ck.nbytes_total), (dict(split_dim=ck.split_dim, rank=7, world=8), 2 * 1004015616)):
        ds = tc.tc_plan_create(ck_spec(ck, flags=HOST, **kw)).descriptors(0)
        assert max(_extent(ds, "src").values()) <= ck.nbytes_total
        ext = _extent(ds, "dst")
        for i in range(ck.N):
            assert ext[i] == ck.nbytes(i) // (8 if kw and ck.split_dim[i] >= 0 else 1)
        assert sum(ext.values()) == total


def test_long_runs_and_wide_spans_are_cut_for_32_bit_row_offsets():
    # a 6 GiB contiguous tensor and a dim-1 slice whose rows are 3 GiB apart
    spec = tc.weights_spec([0], [6 << 30], [2], [1], [[3 << 30, 1, 1, 1]], blob_bytes=6 << 30, flags=HOST)
    ds = tc.tc_plan_create(spec).descriptors(0)
    assert sum(d.run_bytes * d.rows for d in ds) == 6 << 30
    for d in ds:
        assert (d.rows // d.n0) * max(d.src_s1, d.dst_s1) + d.n0 * max(d.src_s0, d.dst_s0) + d.run_bytes < 2 ** 31
    spec = tc.weights_spec([0], [3 * (3 << 30)], [1], [2], [[3, 3 << 30, 1, 1]], split_dim=[1], rank=1, world=3,
                           blob_bytes=9 << 30, flags=HOST)
    ds = tc.tc_plan_create(spec).descriptors(0)
    assert sum(d.run_bytes * d.rows for d in ds) == 3 << 30
    starts = sorted(d.src_off for d in ds)
    assert starts[0] == 1 << 30 and starts[-1] >= (6 << 30) + (1 << 30)


def test_staged_plans_are_cut_into_contiguous_segments():
    # L=4: 16 KiB per token.  Request 0 (5000 tokens, 80 MB) exceeds a 64 MiB staging buffer and
    # is cut at plane boundaries (10 MB planes -> 6 + 2 planes); the small requests share one.
    shape = (4, 16, 8, 128, 2)
    T = np.array([5000, 37, 0, 100, 700], dtype=np.int64)
    off = np.concatenate([[0], np.cumsum((T + 15) // 16)])
    bt = np.arange(off[-1], dtype=np.int32)
    pl = tc.pool(tc.TC_NHD, int(off[-1]), 1, plane_stride=int(off[-1]) * 16 * 8 * 128 * 2)
    for kind, kw in ((tc.TC_KV_PACK, dict(src_pool=pl, bt_src=bt)), (tc.TC_KV_UNPACK, dict(dst_pool=pl, bt_dst=bt))):
        st = tc.tc_plan_create(tc.kv_spec(kind, shape, packed_layout=tc.TC_HND, T=T, bt_off=off, flags=HOST | tc.TC_PLAN_STAGED, **kw)).stats()
        g = 0 if kind == tc.TC_KV_PACK else 1
        assert st.path[g] == 3 and st.launches_per_execute == 3
        st = tc.tc_plan_create(tc.kv_spec(kind, shape, packed_layout=tc.TC_HND, T=T, bt_off=off, flags=HOST, **kw)).stats()
        assert st.path[g] == 1 and st.launches_per_execute == 1
    with pytest.raises(tc.TensorCastError) as e:
        tc.tc_plan_create(tc.kv_spec(tc.TC_KV_MIGRATE, shape, src_pool=pl, dst_pool=pl, T=T, bt_off=off, bt_src=bt, bt_dst=bt, flags=HOST | tc.TC_PLAN_STAGED))
    assert e.value.status == tc.TC_ERR_KIND


@pytest.mark.parametrize("order,L,T,n_seg", [
    (tc.TC_REQUEST_MAJOR, 4, (5000, 37, 0, 100, 700), 3),      # 80 MB request cut at planes (6 + 2), small ones share one
    (tc.TC_LAYER_MAJOR, 4, (5000, 37, 0, 100, 700), 2),        # 12 MB per plane of all requests: 5 + 3 planes
    (tc.TC_LAYER_MAJOR, 1, (0, 20000, 15000, 0, 3000, 0), 4),  # 78 MB per plane: cut inside planes at requests
])
def test_staged_kv_segments_hold_every_byte_their_windows_touch(order, L, T, n_seg):
    """Emulate the staged path segment by segment against a staging array that holds only the
    segment's host bytes, for offload (pack) and reload (unpack)."""
    rng = np.random.default_rng(31)
    B, H, D, E = 16, 8, 128, 2
    shape = (L, B, H, D, E)
    T = np.array(T, dtype=np.int64)
    off = np.concatenate([[0], np.cumsum((T + B - 1) // B)]).astype(np.int64)
    NB = int(off[-1]) + 3
    chunk = B * H * D * E
    pool = rng.integers(0, 256, L * 2 * NB * chunk, dtype=np.uint8)
    bt = rng.permutation(NB)[:off[-1]].astype(np.int32)
    want = np.zeros(oracle.packed_nbytes(shape, T), dtype=np.uint8)
    oracle.kv_pack(shape, oracle.NHD, chunk, planes_of(pool, L * 2), T, off, bt, oracle.NHD, want, order=order, threads=8)
    pl = tc.pool(tc.TC_NHD, NB, L * 2, block_stride=chunk)
    kw = dict(packed_layout=tc.TC_NHD, packed_order=order, T=T, bt_off=off, flags=HOST | tc.TC_PLAN_STAGED)
    plan = tc.tc_plan_create(tc.kv_spec(tc.TC_KV_PACK, shape, src_pool=pl, bt_src=bt, **kw))
    segs = plan.segments(0)
    assert len(segs) == n_seg == plan.stats().launches_per_execute and plan.stats().path[0] == 3
    host = np.full(want.size, 0x77, dtype=np.uint8)
    cnt = np.zeros(want.size, dtype=np.int32)
    end = 0
    for sg in segs:
        assert sg.n_descs > 0 and sg.n_outer > 0 and sg.n_tiles == 0 and 0 < sg.bytes <= 64 << 20
        assert sg.host_off == end                             # segments follow the buffer order without gaps
        end = sg.host_off + sg.bytes
        stage, c = np.full(sg.bytes, 0x55, dtype=np.uint8), np.zeros(sg.bytes, dtype=np.int32)
        run_window(plan.descriptors(0), sg, planes_of(pool, L * 2), [stage], [c], dst_shift=sg.host_off)
        assert (c == 1).all()                                 # the copy back to the host carries no stale byte
        host[sg.host_off:end] = stage
        cnt[sg.host_off:end] += 1
    assert end == want.size and (cnt == 1).all() and np.array_equal(host, want)
    bt2 = rng.permutation(NB)[:off[-1]].astype(np.int32)
    want_pool = np.full_like(pool, 0xA5)
    oracle.kv_unpack(shape, oracle.NHD, chunk, planes_of(want_pool, L * 2), T, off, bt2, oracle.NHD, want, order=order, threads=8)
    plan = tc.tc_plan_create(tc.kv_spec(tc.TC_KV_UNPACK, shape, dst_pool=pl, bt_dst=bt2, **kw))
    segs = plan.segments(1)
    assert len(segs) == n_seg
    got_pool = np.full_like(pool, 0xA5)
    for sg in segs:
        stage = want[sg.host_off:sg.host_off + sg.bytes].copy()
        run_window(plan.descriptors(1), sg, [stage], planes_of(got_pool, L * 2), src_shift=sg.host_off)
    assert np.array_equal(got_pool, want_pool)


@pytest.mark.parametrize("variant", ["tight", "permuted_misaligned"])
@pytest.mark.parametrize("world", [1, 4])
@pytest.mark.parametrize("mode", ["stream", "staged"])
def test_weight_chunks_hold_every_byte_their_tiles_read(variant, world, mode):
    """Streamed (and staged) weight plans run chunk by chunk against a staging buffer that holds
    only the chunk's blob range: emulate exactly that, tile range by tile range."""
    ck = small_checkpoint() if variant == "tight" else small_checkpoint(order_seed=3, pad_to=1, lead_pad=2)
    blob = np.random.default_rng(4).integers(0, 256, ck.nbytes_total, dtype=np.uint8)
    flag = tc.TC_PLAN_STREAM if mode == "stream" else tc.TC_PLAN_STAGED
    for rank in range(world):
        split = ck.split_dim if world > 1 else np.full(ck.N, -1)
        sizes = [ck.nbytes(i) // (world if split[i] >= 0 else 1) for i in range(ck.N)]
        want = [np.zeros(n, dtype=np.uint8) for n in sizes]
        oracle.weights(ck.byte_off, ck.E, ck.shapes, split, rank, world, blob, want)
        plan = tc.tc_plan_create(ck_spec(ck, split_dim=split, rank=rank, world=world, flags=HOST | flag, tuning=dict(tile_bytes=512)))
        segs, descs, st = plan.segments(0), plan.descriptors(0), plan.stats()
        if mode == "staged" and world > 1:
            assert not segs and st.path[0] == 1          # strided slices: plain staging declines, zero copy
            continue
        assert segs and st.path[0] == 3 and st.launches_per_execute == len(segs)
        got = [np.full(n, 0xEE, dtype=np.uint8) for n in sizes]
        cnt = [np.zeros(n, dtype=np.int32) for n in sizes]
        end = 0
        for sg in segs:
            assert sg.n_tiles > 0 and sg.tile0 >= end          # ascending, disjoint tile ranges
            end = sg.tile0 + sg.n_tiles
            assert 0 <= sg.host_off and sg.host_off + sg.bytes <= blob.size and sg.bytes <= 64 << 20
            if mode == "stream":
                assert sg.host_off % 4096 == 0
            stage = blob[sg.host_off:sg.host_off + sg.bytes].copy()
            run_tile_range(descs, sg.tile0, sg.n_tiles, [stage], got, cnt, src_shift=sg.host_off)
        assert end <= st.n_tiles[0]
        for i in range(ck.N):
            assert np.array_equal(got[i], want[i]), ck.names[i]
            assert (cnt[i] == 1).all()                         # every tile ran in exactly one chunk
        if world > 1:                                          # slabs of different tensors are far apart: several chunks
            assert len(segs) > 1
            assert sum(sg.bytes for sg in segs) < blob.size    # ... that do not read the whole blob


def test_stream_flag_limits():
    # 2 KiB pieces of 8 MiB rows, 16 rows per 32 KiB tile: one tile's covering range is 120 MiB
    spec = tc.weights_spec([0], [64 * (8 << 20)], [2], [2], [[64, 4 << 20, 1, 1]], split_dim=[1], rank=5, world=4096,
                           blob_bytes=64 * (8 << 20), flags=HOST | tc.TC_PLAN_STREAM)
    with pytest.raises(tc.TensorCastError) as e:
        tc.tc_plan_create(spec)
    assert e.value.status == tc.TC_ERR_TOO_LARGE and "sparse" in str(e.value)
    spec = tc.weights_spec([0], [64 * (8 << 20)], [2], [2], [[64, 4 << 20, 1, 1]], split_dim=[1], rank=5, world=4096,
                           blob_bytes=64 * (8 << 20), flags=HOST | tc.TC_PLAN_STREAM, tuning=dict(tile_bytes=8192))
    segs = tc.tc_plan_create(spec).segments(0)                 # 4 rows per tile: 24 MiB per tile, two tiles per chunk
    assert len(segs) == 8 and all(sg.bytes <= 64 << 20 for sg in segs)
    shape = (1, 4, 2, 8, 2)
    pl = tc.pool(tc.TC_NHD, 4, 1, plane_stride=4 * 4 * 2 * 8 * 2)
    with pytest.raises(tc.TensorCastError) as e:
        tc.tc_plan_create(tc.kv_spec(tc.TC_KV_PACK, shape, src_pool=pl, bt_src=np.arange(2, dtype=np.int32), T=np.array([8]),
                                     bt_off=np.array([0, 2]), flags=HOST | tc.TC_PLAN_STREAM))
    assert e.value.status == tc.TC_ERR_KIND


def test_debug_bounds_flag_limits():
    shape = (1, 4, 2, 8, 2)
    pl = tc.pool(tc.TC_NHD, 4, 1, plane_stride=4 * 4 * 2 * 8 * 2)
    kw = dict(src_pool=pl, bt_src=np.arange(2, dtype=np.int32), T=np.array([8]), bt_off=np.array([0, 2]))
    plan = tc.tc_plan_create(tc.kv_spec(tc.TC_KV_PACK, shape, flags=HOST | tc.TC_PLAN_DEBUG_BOUNDS, **kw))
    plain = tc.tc_plan_create(tc.kv_spec(tc.TC_KV_PACK, shape, flags=HOST, **kw))
    assert plan.stats().n_tiles[:] == plain.stats().n_tiles[:]  # the flag changes nothing in the lowering
    with pytest.raises(tc.TensorCastError) as e:              # a host-only plan has nothing on a device to check
        tc.tc_plan_check_device(plan, 0)
    assert e.value.status == tc.TC_ERR_KIND
    with pytest.raises(tc.TensorCastError) as e:
        tc.tc_plan_create(tc.kv_spec(tc.TC_KV_PACK, shape, flags=HOST | tc.TC_PLAN_DEBUG_BOUNDS | tc.TC_PLAN_STAGED, **kw))
    assert e.value.status == tc.TC_ERR_INVALID_ARG and "DEBUG_BOUNDS" in str(e.value)


@pytest.mark.parametrize("pool_l,packed_l", list(itertools.product(LAYOUTS, LAYOUTS)))
@pytest.mark.parametrize("order", [tc.TC_REQUEST_MAJOR, tc.TC_LAYER_MAJOR])
def test_head_slice_and_layer_major_lowering_match_oracle(pool_l, packed_l, order):
    rng = np.random.default_rng(7)
    shape, NB, stride, pool, T, off, bt = kv_case(rng, L=2, NB=14, B=4, H=5, D=8, E=2, T=(5, 0, 11, 1, 8), pad_blocks=16)
    L = shape[0]
    for h0, hs in ((0, 0), (1, 3), (4, 1)):
        kw = dict(order=order, head_begin=h0, head_count=hs or None)
        want = np.zeros(oracle.packed_nbytes(shape, T, hs or None), dtype=np.uint8)
        oracle.kv_pack(shape, pool_l, stride, planes_of(pool, L * 2), T, off, bt, packed_l, want, **kw)
        pl = tc.pool(pool_l, NB, L * 2, block_stride=stride)
        lib_kw = dict(packed_layout=packed_l, packed_order=order, head_begin=h0, head_count=hs, T=T, bt_off=off, flags=HOST, tuning=dict(tile_bytes=512))
        plan = tc.tc_plan_create(tc.kv_spec(tc.TC_KV_PACK, shape, src_pool=pl, bt_src=bt, **lib_kw))
        assert plan.stats().packed_bytes_required == want.size
        got = np.full(want.size, 0xCC, dtype=np.uint8)
        cnt = [np.zeros(want.size, dtype=np.int32)]
        run_descriptors(plan.descriptors(0), planes_of(pool, L * 2), [got], cnt)
        assert np.array_equal(got, want) and (cnt[0] == 1).all()
        want_pool = np.full_like(pool, 0xA5)
        oracle.kv_unpack(shape, pool_l, stride, planes_of(want_pool, L * 2), T, off, bt, packed_l, want, **kw)
        plan = tc.tc_plan_create(tc.kv_spec(tc.TC_KV_UNPACK, shape, dst_pool=pl, bt_dst=bt, **lib_kw))
        got_pool = np.full_like(pool, 0xA5)
        run_descriptors(plan.descriptors(1), [want], planes_of(got_pool, L * 2))
        assert np.array_equal(got_pool, want_pool)
    with pytest.raises(tc.TensorCastError) as e:
        tc.tc_plan_create(tc.kv_spec(tc.TC_KV_PACK, shape, src_pool=pl, bt_src=bt, packed_layout=packed_l, head_begin=3, head_count=3, T=T, bt_off=off, flags=HOST))
    assert e.value.status == tc.TC_ERR_BOUNDS
    with pytest.raises(tc.TensorCastError) as e:
        tc.tc_plan_create(tc.kv_spec(tc.TC_KV_MIGRATE, shape, src_pool=pl, dst_pool=pl, bt_src=bt, bt_dst=bt, head_begin=1, head_count=2, T=T, bt_off=off, flags=HOST))
    assert e.value.status == tc.TC_ERR_INVALID_ARG


def test_small_planes_share_a_tile():
    """Few KV heads: one plane of a block is 4-16 KiB, so a tile takes several planes of its
    descriptor (planes_per_tile), in pools with one pointer and in pools with a pointer per plane."""
    T = np.array([40, 16, 5], dtype=np.int64)
    for H, want_ppt in ((1, 8), (2, 4), (4, 2), (8, 1)):
        shape = (16, 16, H, 128, 2)                               # 32 planes of H * 4 KiB per block
        off = np.concatenate([[0], np.cumsum((T + 15) // 16)])
        bt = np.arange(off[-1], dtype=np.int32)
        nb = int(off[-1])
        chunk = 16 * H * 128 * 2
        one = tc.pool(tc.TC_NHD, nb, 1, plane_stride=nb * chunk)
        plan = tc.tc_plan_create(tc.kv_spec(tc.TC_KV_MIGRATE, shape, src_pool=one, dst_pool=one, T=T, bt_off=off, bt_src=bt, bt_dst=bt[::-1].copy(), flags=HOST))
        ds, st = plan.descriptors(0), plan.stats()
        assert all(d.planes_per_tile == want_ppt for d in ds)
        assert st.n_tiles[0] == len(ds) * (32 // want_ppt) and st.payload_bytes[0] == int(T.sum()) * 32 * H * 256
        per_plane = tc.pool(tc.TC_NHD, nb, 32)
        plan = tc.tc_plan_create(tc.kv_spec(tc.TC_KV_MIGRATE, shape, src_pool=per_plane, dst_pool=per_plane, T=T, bt_off=off, bt_src=bt, bt_dst=bt[::-1].copy(), flags=HOST))
        assert all(d.planes_per_tile == want_ppt for d in plan.descriptors(0))
    # L = 3: six planes, tiles of four -> two tile rows per descriptor, the second one half full
    shape = (3, 16, 2, 128, 2)
    plan = tc.tc_plan_create(tc.kv_spec(tc.TC_KV_PACK, shape, src_pool=tc.pool(tc.TC_NHD, 6, 1, plane_stride=6 * 8192), packed_layout=tc.TC_HND,
                                        T=np.array([96]), bt_off=np.array([0, 6]), bt_src=np.arange(6, dtype=np.int32), flags=HOST))
    assert plan.descriptors(0)[0].planes_per_tile == 4 and plan.stats().n_tiles[0] == 6 * 2


@pytest.mark.parametrize("H,L,slots", [(1, 4, "one"), (2, 3, "planes"), (4, 2, "one"), (2, 16, "planes")])
@pytest.mark.parametrize("dst_l", [tc.TC_NHD, tc.TC_HND])
def test_multi_plane_tile_walk_matches_the_oracle(H, L, slots, dst_l):
    """The tile -> (descriptor, planes) -> byte -> (plane, row, column) arithmetic of tiles that
    take several small planes, replayed on the CPU with bounds checks and write counts, for pools
    with one pointer and with one pointer per plane, ragged last blocks, and a plane count that
    the planes per tile do not divide (L = 3)."""
    from helpers import run_multiplane_tiles
    rng = np.random.default_rng(60 + H + L)
    shape, NB, stride, pool, T, off, bt = kv_case(rng, L=L, NB=14, B=16, H=H, D=128, E=2, T=(37, 16, 5, 48))
    planes = L * 2
    bt2 = rng.permutation(NB)[:off[-1]].astype(np.int32)
    n_slots = planes if slots == "planes" else 1
    kw = {} if slots == "planes" else dict(plane_stride=NB * stride)
    src_pool = tc.pool(tc.TC_NHD, NB, n_slots, **kw)
    dst_pool = tc.pool(dst_l, NB, n_slots, **kw)
    plan = tc.tc_plan_create(tc.kv_spec(tc.TC_KV_MIGRATE, shape, src_pool=src_pool, dst_pool=dst_pool, T=T, bt_off=off, bt_src=bt, bt_dst=bt2, flags=HOST))
    ds = plan.descriptors(0)
    assert ds[0].planes_per_tile > 1
    want = np.full_like(pool, 0xA5)
    oracle.kv_migrate(shape, oracle.NHD, stride, planes_of(pool, planes), dst_l, stride, planes_of(want, planes), T, off, bt, bt2)
    got = np.full_like(pool, 0xA5)
    cnt = np.zeros(pool.size, dtype=np.int32)
    tables = (lambda a: planes_of(a, planes)) if slots == "planes" else (lambda a: [a])
    run_multiplane_tiles(ds, plan.stats().n_tiles[0], tables(pool), tables(got), tables(cnt))
    assert np.array_equal(got, want)
    assert cnt.max() == 1 and cnt.sum() == int(T.sum()) * planes * H * 256


@pytest.mark.parametrize("a,b", [(0, 1), (1, 0), (15, 15), (8, 4), (3, 9), (5, 5)])
def test_realigning_path_arithmetic_on_the_cpu(a, b):
    """Base pointers at addresses = a / b modulo 16 under aligned geometry: the chunk, shift,
    head / tail and shared-boundary-chunk arithmetic of the realigning path, replayed on the CPU
    for KV pack (256-byte rows, destination rows adjacent along tokens), unpack, a same-layout
    migration (whole-plane runs), and a staging area small enough to force several passes and
    column pieces.  Each destination byte must be written once, with the oracle's value."""
    from helpers import _Mem, run_realign_tile
    rng = np.random.default_rng(70 + a + b)
    shape, NB, stride, pool, T, off, bt = kv_case(rng, L=1, NB=10, B=16, H=4, D=64, E=2, T=(37, 16, 5))
    bt2 = rng.permutation(NB)[:off[-1]].astype(np.int32)
    pl = tc.pool(tc.TC_NHD, NB, 1, plane_stride=NB * stride)
    packed_n = oracle.packed_nbytes(shape, T)
    cases = []
    want = np.zeros(packed_n, dtype=np.uint8)
    oracle.kv_pack(shape, oracle.NHD, stride, planes_of(pool, 2), T, off, bt, oracle.HND, want)
    cases.append((tc.kv_spec(tc.TC_KV_PACK, shape, src_pool=pl, packed_layout=tc.TC_HND, T=T, bt_off=off, bt_src=bt, flags=HOST), 0, pool, want, 0))
    want_pool = np.full_like(pool, 0xA5)
    oracle.kv_unpack(shape, oracle.NHD, stride, planes_of(want_pool, 2), T, off, bt2, oracle.HND, want)
    cases.append((tc.kv_spec(tc.TC_KV_UNPACK, shape, dst_pool=pl, packed_layout=tc.TC_HND, T=T, bt_off=off, bt_dst=bt2, flags=HOST), 1, want, want_pool, 0xA5))
    want_mig = np.full_like(pool, 0xA5)
    oracle.kv_migrate(shape, oracle.NHD, stride, planes_of(pool, 2), oracle.NHD, stride, planes_of(want_mig, 2), T, off, bt, bt2)
    cases.append((tc.kv_spec(tc.TC_KV_MIGRATE, shape, src_pool=pl, dst_pool=pl, T=T, bt_off=off, bt_src=bt, bt_dst=bt2, flags=HOST), 0, pool, want_mig, 0xA5))
    for spec, group, source, expect, fill in cases:
        plan = tc.tc_plan_create(spec)
        for smem in (52 << 10, 1360, 592):                    # one pass per tile; five 256-byte rows per pass; column pieces
            got = np.full(expect.size, fill, dtype=np.uint8)
            cnt = np.zeros(expect.size, dtype=np.int32)
            src, dst = _Mem(source, 4096 + a), _Mem(got, 1 << 20 | b)
            how = set()
            for d in plan.descriptors(group):
                for o in range(d.n_outer):
                    for part in range(d.tiles_per_outer):
                        if part * d.rows_per_tile < d.rows:
                            how.add(run_realign_tile(d, o, part, src, dst, cnt, smem_bytes=smem))
            assert np.array_equal(got, expect), (group, smem)
            assert cnt.max() == 1 and cnt.sum() == int(T.sum()) * 2 * 4 * 128, (group, smem)
            # 256-byte rows walk the destination's chunks when the tile fits the staging area in one
            # pass and either the destination is misaligned or only the source is (pack: the pool's
            # heads are contiguous; unpack: the packed buffer's tokens); the migration moves whole planes
            kind = spec[0].kind if isinstance(spec, tuple) else spec.kind
            assert ("destination order" in how) == ((a, b) != (0, 0) and smem > 4096 and kind != tc.TC_KV_MIGRATE), (kind, smem, how)


@pytest.mark.parametrize("a,b", [(0, 1), (1, 0), (15, 15), (8, 4), (3, 9)])
def test_realigning_path_stages_long_destination_adjacent_rows_back_to_back(a, b):
    """Rows of 1 KiB: pack (groups of a head's tokens, one per head), unpack (the whole tile is
    one destination run) and a dim-1 weight slice (strided source rows, contiguous destination)
    take the back-to-back staging: no two bulk copies share a staged chunk, the barrier's byte
    count adds up, every consumed byte was loaded, every destination byte is written once with
    the oracle's value.  Ragged last tiles and a small staging area fall back to per-row slots."""
    from helpers import _Mem, run_realign_tile
    rng = np.random.default_rng(90 + a + b)
    shape, NB, stride, pool, T, off, bt = kv_case(rng, L=1, NB=10, B=8, H=4, D=256, E=4, T=(19, 8, 5, 24))
    bt2 = rng.permutation(NB)[:off[-1]].astype(np.int32)
    pl = tc.pool(tc.TC_NHD, NB, 1, plane_stride=NB * stride)
    want = np.zeros(oracle.packed_nbytes(shape, T), dtype=np.uint8)
    oracle.kv_pack(shape, oracle.NHD, stride, planes_of(pool, 2), T, off, bt, oracle.HND, want)
    cases = [(tc.kv_spec(tc.TC_KV_PACK, shape, src_pool=pl, packed_layout=tc.TC_HND, T=T, bt_off=off, bt_src=bt, flags=HOST), 0, pool, want, 0)]
    want_pool = np.full_like(pool, 0xA5)
    oracle.kv_unpack(shape, oracle.NHD, stride, planes_of(want_pool, 2), T, off, bt2, oracle.HND, want)
    cases.append((tc.kv_spec(tc.TC_KV_UNPACK, shape, dst_pool=pl, packed_layout=tc.TC_HND, T=T, bt_off=off, bt_dst=bt2, flags=HOST), 1, want, want_pool, 0xA5))
    # a [96, 4096] fp16 matrix split 4 ways along dim 1: 96 rows of 2 KiB, 8 KiB apart in the blob
    blob = rng.integers(0, 256, 96 * 8192, dtype=np.uint8)
    want_w = [np.zeros(96 * 2048, dtype=np.uint8)]
    oracle.weights([0], [2], [[96, 4096, 1, 1]], [1], 1, 4, blob, want_w)
    cases.append((tc.weights_spec([0], [blob.size], [2], [2], [[96, 4096, 1, 1]], split_dim=[1], rank=1, world=4, blob_bytes=blob.size, flags=HOST), 0, blob, want_w[0], 0))
    for spec, group, source, expect, fill in cases:
        plan = tc.tc_plan_create(spec)
        for smem in (52 << 10, 6000):
            got = np.full(expect.size, fill, dtype=np.uint8)
            cnt = np.zeros(expect.size, dtype=np.int32)
            src, dst = _Mem(source, 4096 + a), _Mem(got, 1 << 20 | b)
            how = []
            for d in plan.descriptors(group):
                for o in range(d.n_outer):
                    for part in range(d.tiles_per_outer):
                        if part * d.rows_per_tile < d.rows:
                            how.append(run_realign_tile(d, o, part, src, dst, cnt, smem_bytes=smem))
            assert np.array_equal(got, expect), (spec.kind, smem)
            assert cnt.max() == 1
            assert ("joined" in how) == (smem > 6000), (spec.kind, smem, how)


@pytest.mark.parametrize("seed", range(14))
def test_realigning_path_models_on_random_geometries(seed):
    """Random block sizes, head counts and row lengths (multiples of 16 bytes), random request
    lengths and random alignments of both sides: pack and unpack replayed tile by tile through
    the CPU models of the realigning path - whichever of its organisations the kernel would pick
    for the tile (per-row slots, rows staged back to back, the destination walk with slots
    completed from their neighbours, column-wise copies of a contiguous source) - against the
    oracle, every destination byte written exactly once."""
    from helpers import _Mem, run_realign_tile
    rng = np.random.default_rng(500 + seed)
    while True:                                               # one plane per tile: a plane is at least a tile
        B = int(rng.choice([2, 4, 8, 16, 5]))
        H = int(rng.choice([1, 2, 4, 8, 3]))
        D, E = int(rng.choice([8, 16, 32, 64, 24, 512])), int(rng.choice([2, 4]))
        tile = int(rng.choice([1024, 4096, 32768]))
        if B * H * D * E >= tile and D * E >= 32:
            break
    nreq = int(rng.integers(1, 4))
    T = tuple(int(x) for x in rng.integers(1, 4 * B + 1, nreq))
    NB = sum((t + B - 1) // B for t in T) + 2
    shape, NB, stride, pool, T, off, bt = kv_case(rng, L=1, NB=NB, B=B, H=H, D=D, E=E, T=T)
    bt2 = rng.permutation(NB)[:off[-1]].astype(np.int32)
    a, b = (int(x) for x in rng.integers(0, 16, 2))
    if (a, b) == (0, 0):
        b = 1
    pl = tc.pool(tc.TC_NHD, NB, 1, plane_stride=NB * stride)
    want = np.zeros(oracle.packed_nbytes(shape, T), dtype=np.uint8)
    oracle.kv_pack(shape, oracle.NHD, stride, planes_of(pool, 2), T, off, bt, oracle.HND, want)
    want_pool = np.full_like(pool, 0xA5)
    oracle.kv_unpack(shape, oracle.NHD, stride, planes_of(want_pool, 2), T, off, bt2, oracle.HND, want)
    tune = dict(tile_bytes=tile)
    cases = [(tc.kv_spec(tc.TC_KV_PACK, shape, src_pool=pl, packed_layout=tc.TC_HND, T=T, bt_off=off, bt_src=bt, flags=HOST, tuning=tune), 0, pool, want, 0),
             (tc.kv_spec(tc.TC_KV_UNPACK, shape, dst_pool=pl, packed_layout=tc.TC_HND, T=T, bt_off=off, bt_dst=bt2, flags=HOST, tuning=tune), 1, want, want_pool, 0xA5)]
    for spec, group, source, expect, fill in cases:
        plan = tc.tc_plan_create(spec)
        if plan.stats().n_tiles[group] == 0:
            continue
        got = np.full(expect.size, fill, dtype=np.uint8)
        cnt = np.zeros(expect.size, dtype=np.int32)
        src, dst = _Mem(source, 4096 + a), _Mem(got, 1 << 20 | b)
        descs = plan.descriptors(group)
        if any(d.planes_per_tile > 1 or d.run_bytes < 32 for d in descs):
            continue                                          # multi-plane tiles and the narrow loop have models of their own
        for d in descs:
            for o in range(d.n_outer):
                for part in range(d.tiles_per_outer):
                    if part * d.rows_per_tile < d.rows:
                        run_realign_tile(d, o, part, src, dst, cnt)
        assert np.array_equal(got, expect), (group, shape, T, a, b)
        assert cnt.max() == 1 and cnt.sum() == int(T.sum()) * 2 * H * D * E, (group, shape, T, a, b)


@pytest.mark.parametrize("D,E,a,b", [(40, 1, 0, 0), (50, 2, 3, 0), (33, 1, 7, 12), (36, 1, 0, 5), (100, 2, 1, 1)])
def test_realigning_path_arithmetic_for_rows_that_differ_in_alignment(D, E, a, b):
    """Rows of D * E bytes, not a multiple of 16: every row of a tile has its own source and
    destination alignment.  Pack, unpack and a same-layout migration replayed on the CPU with
    the kernel's per-chunk arithmetic, one pass and several passes per tile."""
    from helpers import _Mem, run_realign_tile_mixed
    rng = np.random.default_rng(80 + D + a)
    shape, NB, stride, pool, T, off, bt = kv_case(rng, L=1, NB=8, B=8, H=3, D=D, E=E, T=(19, 8, 3))
    bt2 = rng.permutation(NB)[:off[-1]].astype(np.int32)
    pl = tc.pool(tc.TC_NHD, NB, 1, plane_stride=NB * stride)
    want = np.zeros(oracle.packed_nbytes(shape, T), dtype=np.uint8)
    oracle.kv_pack(shape, oracle.NHD, stride, planes_of(pool, 2), T, off, bt, oracle.HND, want)
    want_pool = np.full_like(pool, 0xA5)
    oracle.kv_unpack(shape, oracle.NHD, stride, planes_of(want_pool, 2), T, off, bt2, oracle.HND, want)
    cases = [(tc.kv_spec(tc.TC_KV_PACK, shape, src_pool=pl, packed_layout=tc.TC_HND, T=T, bt_off=off, bt_src=bt, flags=HOST), 0, pool, want, 0),
             (tc.kv_spec(tc.TC_KV_UNPACK, shape, dst_pool=pl, packed_layout=tc.TC_HND, T=T, bt_off=off, bt_dst=bt2, flags=HOST), 1, want, want_pool, 0xA5)]
    for spec, group, source, expect, fill in cases:
        plan = tc.tc_plan_create(spec)
        for smem in (52 << 10, 704):
            got = np.full(expect.size, fill, dtype=np.uint8)
            cnt = np.zeros(expect.size, dtype=np.int32)
            src, dst = _Mem(source, 4096 + a), _Mem(got, 1 << 20 | b)
            for d in plan.descriptors(group):
                if d.run_bytes < 32:
                    pytest.skip("rows this short take the narrow-vector loop")
                for o in range(d.n_outer):
                    for part in range(d.tiles_per_outer):
                        if part * d.rows_per_tile < d.rows:
                            run_realign_tile_mixed(d, o, part, src, dst, cnt, smem_bytes=smem)
            assert np.array_equal(got, expect), (spec.kind, smem)
            assert cnt.max() == 1 and cnt.sum() == int(T.sum()) * 2 * 3 * D * E, (spec.kind, smem)


def test_same_pool_compaction_lowering_and_its_overlap_check():
    """Defragmentation: the requests' blocks move to the low block ids of the same pool."""
    rng = np.random.default_rng(6)
    shape, NB, stride, pool, T, off, bt = kv_case(rng, L=2, NB=30, B=4, H=3, D=8, E=2, T=(9, 4, 14))
    L = shape[0]
    n = int(off[-1])
    bt = (rng.permutation(NB - n)[:n] + n).astype(np.int32)       # sources live above the compacted region
    dst = np.arange(n, dtype=np.int32)
    want = pool.copy()
    oracle.kv_migrate(shape, oracle.NHD, stride, planes_of(pool, L * 2), oracle.NHD, stride, planes_of(want, L * 2), T, off, bt, dst)
    pl = tc.pool(tc.TC_NHD, NB, L * 2, block_stride=stride)
    plan = tc.tc_plan_create(tc.kv_spec(tc.TC_KV_MIGRATE, shape, src_pool=pl, dst_pool=pl, T=T, bt_off=off, bt_src=bt, bt_dst=dst, flags=HOST | tc.TC_PLAN_SAME_POOL))
    got = pool.copy()
    run_descriptors(plan.descriptors(0), planes_of(pool, L * 2), planes_of(got, L * 2))
    assert np.array_equal(got, want)
    clash = dst.copy()
    clash[0] = bt[3]
    with pytest.raises(tc.TensorCastError) as e:
        tc.tc_plan_create(tc.kv_spec(tc.TC_KV_MIGRATE, shape, src_pool=pl, dst_pool=pl, T=T, bt_off=off, bt_src=bt, bt_dst=clash, flags=HOST | tc.TC_PLAN_SAME_POOL))
    assert e.value.status == tc.TC_ERR_OVERLAP
    other = tc.pool(tc.TC_HND, NB, L * 2, block_stride=stride)
    with pytest.raises(tc.TensorCastError) as e:
        tc.tc_plan_create(tc.kv_spec(tc.TC_KV_MIGRATE, shape, src_pool=pl, dst_pool=other, T=T, bt_off=off, bt_src=bt, bt_dst=dst, flags=HOST | tc.TC_PLAN_SAME_POOL))
    assert e.value.status == tc.TC_ERR_INVALID_ARG


# --------------------------------------------------------------------------- validation
def _pack_spec(**over):
    shape, NB, src, dst = wl.config1()
    kw = dict(src_pool=tc.pool(tc.TC_NHD, NB, 2), T=src.T, bt_off=src.bt_off, bt_src=src.bt, flags=HOST)
    kw.update(over)
    return tc.kv_spec(kw.pop("kind", tc.TC_KV_PACK), kw.pop("shape", shape.tuple), **kw)


def _status(spec):
    with pytest.raises(tc.TensorCastError) as e:
        tc.tc_plan_create(spec)
    return e.value.status


def test_validation_rejects_bad_plans_before_any_launch():
    shape, NB, src, dst = wl.config1()
    assert _status(_pack_spec(shape=(1, 16, 8, 128, 3))) == tc.TC_ERR_SHAPE
    bad = src.bt.copy(); bad[5] = NB
    assert _status(_pack_spec(bt_src=bad)) == tc.TC_ERR_BOUNDS
    assert _status(_pack_spec(bt_src=None)) == tc.TC_ERR_INVALID_ARG
    assert _status(_pack_spec(T=[37, 100, 5, 300])) == tc.TC_ERR_INVALID_ARG          # table too short for T
    assert _status(_pack_spec(packed_bytes=1400831)) == tc.TC_ERR_BOUNDS
    assert _status(_pack_spec(src_pool=tc.pool(tc.TC_NHD, NB, 3))) == tc.TC_ERR_INVALID_ARG
    assert _status(_pack_spec(src_pool=tc.pool(tc.TC_NHD, NB, 2, block_stride=100))) == tc.TC_ERR_OVERLAP
    assert _status(_pack_spec(src_pool=tc.pool(tc.TC_NHD, NB, 2, slot_bytes=1000))) == tc.TC_ERR_BOUNDS
    assert _status(_pack_spec(src_pool=tc.pool(tc.TC_NHD, NB, 1, plane_stride=4096))) == tc.TC_ERR_OVERLAP
    assert _status(_pack_spec(kind=9)) == tc.TC_ERR_INVALID_ARG
    dup = dst.bt.copy(); dup[3] = dup[17]
    un = dict(kind=tc.TC_KV_UNPACK, src_pool=None, dst_pool=tc.pool(tc.TC_NHD, NB, 2), bt_src=None)
    assert _status(_pack_spec(bt_dst=dup, **un)) == tc.TC_ERR_OVERLAP                 # a block written twice
    tc.tc_plan_create(_pack_spec(bt_dst=dst.bt, **un))
    # prefix sharing on the read side is allowed
    shared = src.bt.copy(); shared[4] = shared[0]
    tc.tc_plan_create(_pack_spec(bt_src=shared))
    spec, keep = _pack_spec()
    spec.struct_size = 8
    assert _status(spec) == tc.TC_ERR_INVALID_ARG
    ck = small_checkpoint()
    assert _status(ck_spec(ck, split_dim=ck.split_dim, rank=0, world=7, flags=HOST)) == tc.TC_ERR_SHAPE
    assert _status(ck_spec(ck, split_dim=ck.split_dim, rank=4, world=4, flags=HOST)) == tc.TC_ERR_INVALID_ARG
    assert _status(ck_spec(ck, blob_bytes=ck.nbytes_total - 1, flags=HOST)) == tc.TC_ERR_BOUNDS
    nb = [ck.nbytes(i) for i in range(ck.N)]
    nb[2] += 2
    assert _status(tc.weights_spec(ck.byte_off, nb, ck.E, ck.ndim, ck.shapes, blob_bytes=ck.nbytes_total + 2, flags=HOST)) == tc.TC_ERR_SHAPE
    small = [ck.nbytes(i) for i in range(ck.N)]
    small[1] -= 2
    assert _status(ck_spec(ck, dst_bytes=small, flags=HOST)) == tc.TC_ERR_BOUNDS


def test_documented_limits_are_enforced():
    shape, NB, src, dst = wl.config1()
    # pointer-table capacity: L*2 planes per pool, src + dst slots of one call
    big_l = (1001, 16, 8, 128, 2)
    assert _status(tc.kv_spec(tc.TC_KV_PACK, big_l, src_pool=tc.pool(tc.TC_NHD, 4, 2002), flags=HOST)) == tc.TC_ERR_INVALID_ARG
    n = tc.TC_MAX_TABLE_SLOTS
    spec = tc.weights_spec(np.arange(n) * 16, [16] * n, [2] * n, [1] * n, [[8, 1, 1, 1]] * n, blob_bytes=16 * n, flags=HOST)
    assert _status(spec) == tc.TC_ERR_INVALID_ARG
    ok = n - 1
    plan = tc.tc_plan_create(tc.weights_spec(np.arange(ok) * 16, [16] * ok, [2] * ok, [1] * ok, [[8, 1, 1, 1]] * ok, blob_bytes=16 * ok, flags=HOST))
    assert plan.stats().n_descriptors[0] == ok
    # more than 2^31 tiles in one plan
    huge = 1 << 47
    assert _status(tc.weights_spec([0], [huge], [1], [1], [[huge, 1, 1, 1]], blob_bytes=huge, flags=HOST)) == tc.TC_ERR_INVALID_ARG
    # tile size knob must be a power of two in range
    assert _status(_pack_spec(tuning=dict(tile_bytes=3000))) == tc.TC_ERR_INVALID_ARG
    assert _status(_pack_spec(tuning=dict(tile_bytes=1 << 21))) == tc.TC_ERR_INVALID_ARG
    assert _status(_pack_spec(tuning=dict(tile_order=3))) == tc.TC_ERR_INVALID_ARG
    tc.tc_plan_create(_pack_spec(tuning=dict(tile_order=2))).destroy()
    # the longest request the configs allow (32 768 tokens) and a single-token one, in one plan
    T = np.array([32768, 1], dtype=np.int64)
    off = np.array([0, 2048, 2049], dtype=np.int64)
    bt = np.arange(2049, dtype=np.int32)
    s8 = wl.LLAMA3_8B_KV
    st = tc.tc_plan_create(tc.kv_spec(tc.TC_KV_PACK, s8.tuple, src_pool=tc.pool(tc.TC_NHD, 2049, 1, plane_stride=2049 * s8.chunk_bytes),
                                      packed_layout=tc.TC_HND, T=T, bt_off=off, bt_src=bt, flags=HOST)).stats()
    assert st.payload_bytes[0] == 32769 * s8.token_bytes and st.n_descriptors[0] == 2049 and st.n_tiles[0] == 2049 * 64


def test_empty_plans_deadline_and_kind_checks():
    shape, NB, src, dst = wl.config1()
    empty = tc.tc_plan_create(tc.kv_spec(tc.TC_KV_PACK, shape.tuple, src_pool=tc.pool(tc.TC_NHD, NB, 2), flags=HOST))
    assert empty.stats().n_tiles[0] == 0 and empty.stats().payload_bytes[0] == 0
    zero_len = tc.tc_plan_create(_pack_spec(T=[0, 0], bt_off=[0, 0, 0], bt_src=[]))
    assert zero_len.stats().n_descriptors[0] == 0
    past = time.clock_gettime_ns(time.CLOCK_MONOTONIC) - 1
    assert _status(_pack_spec(deadline_ns=past)) == tc.TC_ERR_DEADLINE
    plan = tc.tc_plan_create(_pack_spec(trace_id=77))
    assert plan.stats().trace_id == 77
    with pytest.raises(tc.TensorCastError) as e:
        tc.tc_kv_unpack(plan, [1], [1, 1])
    assert e.value.status == tc.TC_ERR_KIND
    with pytest.raises(tc.TensorCastError) as e:
        tc.tc_kv_pack(plan, [16, 16], [16])            # host-only plans never execute
    assert e.value.status == tc.TC_ERR_INVALID_ARG
    with pytest.raises(tc.TensorCastError) as e:
        tc.tc_weights_materialize(plan, 16, [16])
    assert e.value.status == tc.TC_ERR_KIND
    tc.tc_trim()                                        # nothing cached here: still fine
    plan.destroy()
    plan.destroy()                                      # idempotent; NULL destroy is a no-op
    assert tc.load_library().tc_plan_destroy(None) == 0


@pytest.mark.skipif(__import__("torch").cuda.is_available(), reason="only meaningful without a GPU")
def test_product_path_fails_loudly_without_a_device():
    """No CPU fallback: without a CUDA device an executable plan cannot even be created."""
    shape, NB, src, dst = wl.config1()
    spec = tc.kv_spec(tc.TC_KV_PACK, shape.tuple, src_pool=tc.pool(tc.TC_NHD, NB, 2), T=src.T, bt_off=src.bt_off, bt_src=src.bt)
    assert _status(spec) == tc.TC_ERR_CUDA
