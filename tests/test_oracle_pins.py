"""Pins for the CPU oracle: everything here checks the oracle against something other than
itself - a hand-derived worked example, a brute-force model written a different way, numpy
library routines on the special cases that reduce to them, and invariants (exactly-once
writes, round trips, shards tiling the full tensor)."""
import itertools
import os

import numpy as np
import pytest

import oracle
import workloads as wl

GOLD = os.path.join(os.path.dirname(__file__), "golden")
LAY = {"NHD": oracle.NHD, "HND": oracle.HND}


def planes_of(pool, n_planes):
    """Split one flat allocation into equal (l,c) planes (views)."""
    per = pool.size // n_planes
    return [pool[i * per:(i + 1) * per] for i in range(n_planes)]


# ------------------------------------------------------------------ worked micro-example
def _micro_rows():
    rows = []
    for line in open(os.path.join(GOLD, "kv_micro_example.txt")):
        if line.startswith("#") or not line.strip():
            continue
        f = line.split()
        rows.append((f[0], f[1], np.array([int(x) for x in f[2:]], dtype=np.uint8)))
    return rows


@pytest.mark.parametrize("pool_l,packed_l,expect_k", _micro_rows())
def test_micro_example_pack(pool_l, packed_l, expect_k):
    shape = (1, 2, 2, 2, 1)
    K = np.arange(24, dtype=np.uint8)
    V = (100 + np.arange(24)).astype(np.uint8)
    packed = np.full(24, 255, dtype=np.uint8)
    cnt = np.zeros(24, dtype=np.uint8)
    oracle.kv_pack(shape, LAY[pool_l], 8, [K, V], [3], [0, 2], [2, 0], LAY[packed_l], packed, cnt)
    assert packed[:12].tolist() == expect_k.tolist()
    assert packed[12:].tolist() == (expect_k + 100).tolist()
    assert (cnt == 1).all()


@pytest.mark.parametrize("pool_l,packed_l,expect_k", _micro_rows())
def test_micro_example_unpack_touches_only_valid_slots(pool_l, packed_l, expect_k):
    shape = (1, 2, 2, 2, 1)
    packed = np.concatenate([expect_k, expect_k + 100]).astype(np.uint8)
    K = np.full(24, 0xA5, dtype=np.uint8)
    V = np.full(24, 0xA5, dtype=np.uint8)
    cK, cV = np.zeros(24, dtype=np.uint8), np.zeros(24, dtype=np.uint8)
    oracle.kv_unpack(shape, LAY[pool_l], 8, [K, V], [3], [0, 2], [1, 2], LAY[packed_l], packed, [cK, cV])
    # exactly block 1 (both slots) and slot 0 of block 2 are written: 12 bytes per plane
    assert cK.sum() == 12 and cV.sum() == 12 and cK.max() == 1
    assert (K[:8] == 0xA5).all() and (cK[8:16] == 1).all()
    # read the tokens back through the new table: same content as through the old one
    back = np.zeros(24, dtype=np.uint8)
    oracle.kv_pack(shape, LAY[pool_l], 8, [K, V], [3], [0, 2], [1, 2], LAY[packed_l], back)
    assert back.tolist() == packed.tolist()


# ------------------------------------------------------------------ brute-force model
def brute_pack(shape, pool_layout, planes_dict, T, bt, packed_layout):
    """Model written with dicts of index tuples: no address arithmetic shared with the oracle.
    planes_dict[(l,c)][(b,n,h,d,e)] -> byte.  Returns the packed bytes as a list, ordered by
    sorting the logical keys in the packed layout's nesting order."""
    L, B, H, D, E = shape
    out = []
    for r, Tr in enumerate(T):
        entries = {}
        for l, c, t, h, d, e in itertools.product(range(L), range(2), range(Tr), range(H), range(D), range(E)):
            key = (l, c, t, h, d, e) if packed_layout == oracle.NHD else (l, c, h, t, d, e)
            entries[key] = planes_dict[(l, c)][(bt[r][t // B], t % B, h, d, e)]
        out += [entries[k] for k in sorted(entries)]
    return out


def dict_planes(shape, NB, layout, rng):
    """Random planes, as flat arrays (block stride tight) and as tuple-keyed dicts."""
    L, B, H, D, E = shape
    flat, dicts = [], {}
    for l, c in itertools.product(range(L), range(2)):
        if layout == oracle.NHD:
            arr = rng.integers(0, 256, (NB, B, H, D, E), dtype=np.uint8)
            dicts[(l, c)] = {(b, n, h, d, e): int(arr[b, n, h, d, e]) for b, n, h, d, e in np.ndindex(arr.shape)}
        else:
            arr = rng.integers(0, 256, (NB, H, B, D, E), dtype=np.uint8)
            dicts[(l, c)] = {(b, n, h, d, e): int(arr[b, h, n, d, e]) for b, h, n, d, e in np.ndindex(arr.shape)}
        flat.append(arr.reshape(-1).copy())
    return flat, dicts


@pytest.mark.parametrize("pool_l", [oracle.NHD, oracle.HND])
@pytest.mark.parametrize("packed_l", [oracle.NHD, oracle.HND])
def test_brute_force_all_block_tables(pool_l, packed_l):
    shape = (2, 2, 3, 2, 2)  # L, B, H, D, E   (B != H on purpose)
    NB = 4
    rng = np.random.default_rng(7)
    flat, dicts = dict_planes(shape, NB, pool_l, rng)
    T = [3, 2, 1]  # 2 + 1 + 1 blocks: every ordered choice of 4 distinct blocks
    for perm in itertools.permutations(range(NB), 4):
        bt = [list(perm[:2]), [perm[2]], [perm[3]]]
        want = brute_pack(shape, pool_l, dicts, T, bt, packed_l)
        got = np.zeros(oracle.packed_nbytes(shape, T), dtype=np.uint8)
        oracle.kv_pack(shape, pool_l, flat[0].size // NB, flat, T, [0, 2, 3, 4], list(perm), packed_l, got)
        assert got.tolist() == want


def test_brute_force_odd_shapes_and_empty_requests():
    shape = (1, 3, 2, 3, 1)
    NB = 5
    rng = np.random.default_rng(11)
    for pool_l, packed_l in itertools.product([oracle.NHD, oracle.HND], repeat=2):
        flat, dicts = dict_planes(shape, NB, pool_l, rng)
        T = [0, 4, 0, 3]
        bt = [[], [4, 1], [], [0]]
        want = brute_pack(shape, pool_l, dicts, T, bt, packed_l)
        got = np.zeros(oracle.packed_nbytes(shape, T), dtype=np.uint8)
        oracle.kv_pack(shape, pool_l, flat[0].size // NB, flat, T, [0, 0, 2, 2, 3], [4, 1, 0], packed_l, got)
        assert got.tolist() == want


# ------------------------------------------------------------------ library special cases
def random_case(rng, L=2, NB=12, B=4, H=3, D=8, E=2, T=(8, 4, 12), pad_blocks=0):
    shape = (L, B, H, D, E)
    chunk = B * H * D * E
    stride = chunk + pad_blocks
    pool = rng.integers(0, 256, L * 2 * NB * stride, dtype=np.uint8)
    T = np.array(T, dtype=np.int64)
    off = np.concatenate([[0], np.cumsum((T + B - 1) // B)])
    bt = rng.permutation(NB)[:off[-1]].astype(np.int32)
    return shape, NB, stride, pool, T, off, bt


def test_pack_nhd_equals_numpy_gather_when_blocks_are_full():
    rng = np.random.default_rng(3)
    shape, NB, stride, pool, T, off, bt = random_case(rng)
    L, B, H, D, E = shape
    planes = planes_of(pool, L * 2)
    got = np.zeros(oracle.packed_nbytes(shape, T), dtype=np.uint8)
    oracle.kv_pack(shape, oracle.NHD, stride, planes, T, off, bt, oracle.NHD, got)
    p5 = pool.reshape(L * 2, NB, B, H, D * E)
    want = np.concatenate([p5[:, bt[off[r]:off[r + 1]]].reshape(-1) for r in range(len(T))])
    assert np.array_equal(got, want)
    # NHD pool -> request-level HND buffer is a transpose of (token, head) per plane
    got_h = np.zeros_like(got)
    oracle.kv_pack(shape, oracle.NHD, stride, planes, T, off, bt, oracle.HND, got_h)
    want_h = np.concatenate([
        p5[:, bt[off[r]:off[r + 1]]].reshape(L * 2, T[r], H, D * E).transpose(0, 2, 1, 3).reshape(-1)
        for r in range(len(T))])
    assert np.array_equal(got_h, want_h)


def test_unpack_equals_numpy_scatter_when_blocks_are_full():
    rng = np.random.default_rng(31)
    shape, NB, stride, pool, T, off, bt = random_case(rng)
    L, B, H, D, E = shape
    packed = rng.integers(0, 256, oracle.packed_nbytes(shape, T), dtype=np.uint8)
    for packed_l in (oracle.NHD, oracle.HND):
        got = np.full_like(pool, 0xA5)
        oracle.kv_unpack(shape, oracle.NHD, stride, planes_of(got, L * 2), T, off, bt, packed_l, packed)
        want = np.full_like(pool, 0xA5).reshape(L * 2, NB, B, H, D * E)
        pos = 0
        for r, t in enumerate(T):
            n = L * 2 * int(t) * H * D * E
            reg = packed[pos:pos + n]
            pos += n
            if packed_l == oracle.NHD:
                tok = reg.reshape(L * 2, int(t), H, D * E)
            else:
                tok = reg.reshape(L * 2, H, int(t), D * E).transpose(0, 2, 1, 3)
            want[:, bt[off[r]:off[r + 1]]] = tok.reshape(L * 2, -1, B, H, D * E)
        assert np.array_equal(got, want.reshape(-1))


def test_hnd_pool_is_per_block_transpose_of_nhd_pool():
    rng = np.random.default_rng(4)
    shape, NB, stride, pool, T, off, bt = random_case(rng, T=(7, 4, 9))
    L, B, H, D, E = shape
    pool_h = pool.reshape(L * 2, NB, B, H, D * E).transpose(0, 1, 3, 2, 4).reshape(-1).copy()
    for packed_l in (oracle.NHD, oracle.HND):
        a = np.zeros(oracle.packed_nbytes(shape, T), dtype=np.uint8)
        b = np.zeros_like(a)
        oracle.kv_pack(shape, oracle.NHD, stride, planes_of(pool, L * 2), T, off, bt, packed_l, a)
        oracle.kv_pack(shape, oracle.HND, stride, planes_of(pool_h, L * 2), T, off, bt, packed_l, b)
        assert np.array_equal(a, b)


# ------------------------------------------------------------------ invariants
@pytest.mark.parametrize("pool_l,packed_l", list(itertools.product([oracle.NHD, oracle.HND], repeat=2)))
def test_forward_and_inverse_formulations_agree(pool_l, packed_l):
    rng = np.random.default_rng(5)
    shape, NB, stride, pool, T, off, bt = random_case(rng, T=(5, 0, 11, 1), pad_blocks=6)
    planes = planes_of(pool, shape[0] * 2)
    a = np.zeros(oracle.packed_nbytes(shape, T), dtype=np.uint8)
    b = np.ones_like(a)
    cnt = np.zeros_like(a)
    oracle.kv_pack(shape, pool_l, stride, planes, T, off, bt, packed_l, a, cnt)
    oracle.kv_pack_inverse(shape, pool_l, stride, planes, T, off, bt, packed_l, b)
    assert np.array_equal(a, b)
    assert (cnt == 1).all()  # every packed byte written exactly once


@pytest.mark.parametrize("pool_l,packed_l", list(itertools.product([oracle.NHD, oracle.HND], repeat=2)))
def test_pack_unpack_round_trip_and_untouched_bytes(pool_l, packed_l):
    rng = np.random.default_rng(6)
    shape, NB, stride, pool, T, off, bt = random_case(rng, T=(5, 0, 11, 1), pad_blocks=6)
    L, B, H, D, E = shape
    planes = planes_of(pool, L * 2)
    packed = np.zeros(oracle.packed_nbytes(shape, T), dtype=np.uint8)
    oracle.kv_pack(shape, pool_l, stride, planes, T, off, bt, packed_l, packed)
    bt2 = rng.permutation(NB)[:off[-1]].astype(np.int32)
    pool2 = np.full_like(pool, 0xA5)
    cnt2 = np.zeros_like(pool)
    oracle.kv_unpack(shape, pool_l, stride, planes_of(pool2, L * 2), T, off, bt2, packed_l, packed,
                     planes_of(cnt2, L * 2))
    assert cnt2.max() == 1
    assert cnt2.sum() == packed.size                      # valid-token bytes, once each
    assert (pool2[cnt2 == 0] == 0xA5).all()               # everything else keeps the sentinel
    back = np.zeros_like(packed)
    oracle.kv_pack(shape, pool_l, stride, planes_of(pool2, L * 2), T, off, bt2, packed_l, back)
    assert np.array_equal(back, packed)                   # pack o unpack = identity on valid tokens


def test_layout_transform_there_and_back_is_identity():
    rng = np.random.default_rng(8)
    shape, NB, stride, pool, T, off, bt = random_case(rng, T=(6, 3, 10))
    L = shape[0]
    planes = planes_of(pool, L * 2)
    nhd = np.zeros(oracle.packed_nbytes(shape, T), dtype=np.uint8)
    hnd = np.zeros_like(nhd)
    oracle.kv_pack(shape, oracle.NHD, stride, planes, T, off, bt, oracle.NHD, nhd)
    oracle.kv_pack(shape, oracle.NHD, stride, planes, T, off, bt, oracle.HND, hnd)
    assert not np.array_equal(nhd, hnd)
    # NHD -> HND -> NHD : unpack the HND buffer into an NHD pool and re-pack as NHD
    pool2 = np.zeros_like(pool)
    oracle.kv_unpack(shape, oracle.NHD, stride, planes_of(pool2, L * 2), T, off, bt, oracle.HND, hnd)
    again = np.zeros_like(nhd)
    oracle.kv_pack(shape, oracle.NHD, stride, planes_of(pool2, L * 2), T, off, bt, oracle.NHD, again)
    assert np.array_equal(again, nhd)


@pytest.mark.parametrize("src_l,dst_l", list(itertools.product([oracle.NHD, oracle.HND], repeat=2)))
def test_migrate_equals_pack_then_unpack(src_l, dst_l):
    rng = np.random.default_rng(9)
    shape, NB, stride, pool, T, off, bt = random_case(rng, T=(5, 12, 2), pad_blocks=2)
    L, B, H, D, E = shape
    NB2, stride2 = NB + 3, stride + 10
    bt2 = rng.permutation(NB2)[:off[-1]].astype(np.int32)
    a = np.full(L * 2 * NB2 * stride2, 0x5A, dtype=np.uint8)
    b = a.copy()
    cnt = np.zeros_like(a)
    oracle.kv_migrate(shape, src_l, stride, planes_of(pool, L * 2), dst_l, stride2, planes_of(a, L * 2),
                      T, off, bt, bt2, planes_of(cnt, L * 2))
    packed = np.zeros(oracle.packed_nbytes(shape, T), dtype=np.uint8)
    oracle.kv_pack(shape, src_l, stride, planes_of(pool, L * 2), T, off, bt, oracle.NHD, packed)
    oracle.kv_unpack(shape, dst_l, stride2, planes_of(b, L * 2), T, off, bt2, oracle.NHD, packed)
    assert np.array_equal(a, b)
    assert cnt.max() == 1 and cnt.sum() == packed.size


def test_page_first_host_pool_is_a_block_stride():
    """A pool stored page-first ([block][layer][K|V][...]) is the same formula with plane
    bases one chunk apart and a block stride of L*2 chunks."""
    rng = np.random.default_rng(10)
    L, B, H, D, E, NB = 2, 2, 2, 4, 2, 5
    shape = (L, B, H, D, E)
    chunk = B * H * D * E
    page_first = rng.integers(0, 256, NB * L * 2 * chunk, dtype=np.uint8)
    planes = [page_first[p * chunk:] for p in range(L * 2)]
    T, off, bt = [4, 2], [0, 2, 3], [3, 0, 4]
    got = np.zeros(oracle.packed_nbytes(shape, T), dtype=np.uint8)
    oracle.kv_pack(shape, oracle.NHD, L * 2 * chunk, planes, T, off, bt, oracle.NHD, got)
    v = page_first.reshape(NB, L * 2, chunk)
    want = np.concatenate([v[bt[off[r]:off[r + 1]]].transpose(1, 0, 2).reshape(-1) for r in range(2)])
    assert np.array_equal(got, want)


# ------------------------------------------------------------------ weights
def small_checkpoint(**kw):
    return wl.llama_checkpoint(hidden=64, layers=2, q_heads=8, kv_heads=4, head_dim=8, mlp=96,
                               vocab=160, **kw)


def alloc_dst(ck, world=None):
    out = []
    for i in range(ck.N):
        n = ck.nbytes(i)
        if world and ck.split_dim[i] >= 0:
            n //= world
        out.append(np.full(n, 0xEE, dtype=np.uint8))
    return out


def test_weights_full_concatenation_reproduces_blob():
    ck = small_checkpoint()
    blob = np.random.default_rng(1).integers(0, 256, ck.nbytes_total, dtype=np.uint8)
    dst = alloc_dst(ck)
    cnt = [np.zeros_like(d) for d in dst]
    oracle.weights(ck.byte_off, ck.E, ck.shapes, np.full(ck.N, -1), 0, 1, blob, dst, dst_cnt=cnt)
    assert np.array_equal(np.concatenate(dst), blob)      # tight canonical order
    assert all((c == 1).all() for c in cnt)


def test_weights_permuted_and_padded_order():
    ck = small_checkpoint(order_seed=5, pad_to=64, lead_pad=2)
    blob = np.random.default_rng(2).integers(0, 256, ck.nbytes_total, dtype=np.uint8)
    dst = alloc_dst(ck)
    oracle.weights(ck.byte_off, ck.E, ck.shapes, np.full(ck.N, -1), 0, 1, blob, dst)
    for i in range(ck.N):
        assert np.array_equal(dst[i], blob[ck.byte_off[i]:ck.byte_off[i] + ck.nbytes(i)])


def test_weights_shards_equal_numpy_slices_and_tile_the_tensor():
    ck = small_checkpoint()
    W = 4
    blob = np.random.default_rng(3).integers(0, 256, ck.nbytes_total, dtype=np.uint8)
    shards = []
    for rank in range(W):
        dst = alloc_dst(ck, W)
        cnt = [np.zeros_like(d) for d in dst]
        oracle.weights(ck.byte_off, ck.E, ck.shapes, ck.split_dim, rank, W, blob, dst, dst_cnt=cnt)
        assert all((c == 1).all() for c in cnt)
        shards.append(dst)
    for i in range(ck.N):
        shp = [int(x) for x in ck.shapes[i][:ck.ndim[i]]]
        full = blob[ck.byte_off[i]:ck.byte_off[i] + ck.nbytes(i)].view(np.uint16).reshape(shp)
        sd = int(ck.split_dim[i])
        for rank in range(W):
            got = shards[rank][i].view(np.uint16)
            if sd < 0:
                assert np.array_equal(got, full.reshape(-1))          # replicated
            else:
                n = shp[sd] // W
                want = np.take(full, np.arange(rank * n, (rank + 1) * n), axis=sd)
                assert np.array_equal(got, want.reshape(-1))          # numpy narrow
        if sd >= 0:
            shp_s = list(shp)
            shp_s[sd] //= W
            cat = np.concatenate([shards[r][i].view(np.uint16).reshape(shp_s) for r in range(W)], axis=sd)
            assert np.array_equal(cat, full)                          # shards tile the tensor


def test_weights_split_of_a_middle_dim_and_strided_destination():
    # one 3-D tensor [4][6][5] of 4-byte elements, split on dim 1 into 3, written into a
    # window of a larger row-major target [4][2][8] (transform_into a caller-owned buffer)
    rng = np.random.default_rng(4)
    full = rng.integers(0, 2 ** 32, (4, 6, 5), dtype=np.uint32)
    blob = np.concatenate([np.zeros(3, dtype=np.uint8), full.reshape(-1).view(np.uint8)])
    target = np.zeros((4, 2, 8), dtype=np.uint32)
    tb = target.reshape(-1).view(np.uint8)
    oracle.weights([3], [4], [[4, 6, 5, 1]], [1], 2, 3, blob, [tb], dst_off=[3 * 4],
                   dst_stride=[[2 * 8 * 4, 8 * 4, 4, 4]])
    want = np.zeros_like(target)
    want[:, :, 3:8] = full[:, 4:6, :]
    assert np.array_equal(target, want)


def test_llama3_8b_index_matches_golden_offsets():
    g = {}
    for line in open(os.path.join(GOLD, "llama3_8b_blob_offsets.txt")):
        if not line.startswith("#") and line.strip():
            k, v = line.split()
            g[k] = int(v)
    ck = wl.config3()
    off = dict(zip(ck.names, ck.byte_off))
    assert ck.N == g["n_tensors"] and ck.nbytes_total == g["total_bytes"]
    assert sum(ck.nbytes(i) for i in range(ck.N)) // 2 == g["total_elements"]
    assert off["embed_tokens"] == g["embed_tokens"] and off["norm"] == g["norm"] and off["lm_head"] == g["lm_head"]
    for l in (0, 1, 31):
        base = g["layers.0.input_layernorm"] + l * g["layer_stride"]
        assert off[f"layers.{l}.input_layernorm"] == base
        for nm in ("q_proj", "k_proj", "v_proj", "o_proj", "post_attention_layernorm", "gate_proj", "up_proj", "down_proj"):
            assert off[f"layers.{l}.{nm}"] == base + g["in_layer." + nm]
    shard_el = sum(int(np.prod(wl.shard_shape(ck, i, 8))) for i in range(ck.N))
    assert shard_el == g["shard_elements_world8"]


# ------------------------------------------------------------------ packed-side views
@pytest.mark.parametrize("pool_l,packed_l", list(itertools.product([oracle.NHD, oracle.HND], repeat=2)))
def test_head_slice_is_a_numpy_slice_of_the_full_pack(pool_l, packed_l):
    rng = np.random.default_rng(14)
    shape, NB, stride, pool, T, off, bt = random_case(rng, H=5, T=(7, 0, 12, 1))
    L, B, H, D, E = shape
    planes = planes_of(pool, L * 2)
    full = np.zeros(oracle.packed_nbytes(shape, T), dtype=np.uint8)
    oracle.kv_pack(shape, pool_l, stride, planes, T, off, bt, packed_l, full)
    h0, hs = 1, 3
    part = np.zeros(oracle.packed_nbytes(shape, T, hs), dtype=np.uint8)
    cnt = np.zeros_like(part)
    oracle.kv_pack(shape, pool_l, stride, planes, T, off, bt, packed_l, part, cnt, head_begin=h0, head_count=hs)
    assert (cnt == 1).all()
    want, pos = [], 0
    for t in T:
        n = L * 2 * int(t) * H * D * E
        reg = full[pos:pos + n]
        pos += n
        if packed_l == oracle.NHD:
            want.append(reg.reshape(L * 2, int(t), H, D * E)[:, :, h0:h0 + hs].reshape(-1))
        else:
            want.append(reg.reshape(L * 2, H, int(t), D * E)[:, h0:h0 + hs].reshape(-1))
    assert np.array_equal(part, np.concatenate(want))
    # unpacking the slice writes exactly those heads: the others keep the sentinel
    pool2 = np.full_like(pool, 0xA5)
    cnt2 = np.zeros_like(pool)
    oracle.kv_unpack(shape, pool_l, stride, planes_of(pool2, L * 2), T, off, bt, packed_l, part, planes_of(cnt2, L * 2), head_begin=h0, head_count=hs)
    assert cnt2.sum() == part.size and cnt2.max() == 1 and (pool2[cnt2 == 0] == 0xA5).all()
    back = np.zeros_like(part)
    oracle.kv_pack(shape, pool_l, stride, planes_of(pool2, L * 2), T, off, bt, packed_l, back, head_begin=h0, head_count=hs)
    assert np.array_equal(back, part)


@pytest.mark.parametrize("packed_l", [oracle.NHD, oracle.HND])
def test_layer_major_order_is_a_regrouping_of_request_major(packed_l):
    rng = np.random.default_rng(15)
    shape, NB, stride, pool, T, off, bt = random_case(rng, T=(5, 0, 11, 2))
    L, B, H, D, E = shape
    planes = planes_of(pool, L * 2)
    rm = np.zeros(oracle.packed_nbytes(shape, T), dtype=np.uint8)
    lm = np.zeros_like(rm)
    cnt = np.zeros_like(rm)
    oracle.kv_pack(shape, oracle.NHD, stride, planes, T, off, bt, packed_l, rm)
    oracle.kv_pack(shape, oracle.NHD, stride, planes, T, off, bt, packed_l, lm, cnt, order=oracle.LAYER_MAJOR)
    assert (cnt == 1).all()
    per_req, pos = [], 0
    for t in T:
        n = L * 2 * int(t) * H * D * E
        per_req.append(rm[pos:pos + n].reshape(L * 2, -1))     # [plane][bytes of that plane]
        pos += n
    want = np.concatenate([np.concatenate([q[p] for q in per_req]) for p in range(L * 2)])
    assert np.array_equal(lm, want)
    pool2 = np.full_like(pool, 0xA5)
    oracle.kv_unpack(shape, oracle.NHD, stride, planes_of(pool2, L * 2), T, off, bt, packed_l, lm, order=oracle.LAYER_MAJOR)
    pool3 = np.full_like(pool, 0xA5)
    oracle.kv_unpack(shape, oracle.NHD, stride, planes_of(pool3, L * 2), T, off, bt, packed_l, rm)
    assert np.array_equal(pool2, pool3)


@pytest.mark.parametrize("pool_l,packed_l", list(itertools.product([oracle.NHD, oracle.HND], repeat=2)))
def test_layer_major_head_slice_is_a_regrouping_of_the_full_request_major_pack(pool_l, packed_l):
    """Layer-major order and a head slice together, on NHD and HND pools.  The expected bytes are
    cut out of the FULL request-major pack with numpy (slice the heads, then put plane p of every
    request side by side), so the combined branch of the packed-address formula is checked
    against the two options taken one at a time."""
    rng = np.random.default_rng(16)
    shape, NB, stride, pool, T, off, bt = random_case(rng, H=5, T=(6, 0, 9, 1, 13))
    L, B, H, D, E = shape
    planes = planes_of(pool, L * 2)
    full = np.zeros(oracle.packed_nbytes(shape, T), dtype=np.uint8)
    oracle.kv_pack(shape, pool_l, stride, planes, T, off, bt, packed_l, full)
    h0, hs = 2, 2
    got = np.zeros(oracle.packed_nbytes(shape, T, hs), dtype=np.uint8)
    cnt = np.zeros_like(got)
    oracle.kv_pack(shape, pool_l, stride, planes, T, off, bt, packed_l, got, cnt,
                   order=oracle.LAYER_MAJOR, head_begin=h0, head_count=hs)
    assert (cnt == 1).all()
    per_req, pos = [], 0
    for t in T:
        n = L * 2 * int(t) * H * D * E
        reg = full[pos:pos + n]
        pos += n
        if packed_l == oracle.NHD:
            per_req.append(reg.reshape(L * 2, int(t), H, D * E)[:, :, h0:h0 + hs].reshape(L * 2, -1))
        else:
            per_req.append(reg.reshape(L * 2, H, int(t), D * E)[:, h0:h0 + hs].reshape(L * 2, -1))
    want = np.concatenate([np.concatenate([q[p] for q in per_req]) for p in range(L * 2)])
    assert np.array_equal(got, want)
    # unpack of that buffer writes exactly the sliced heads of the valid tokens, each byte once,
    # and reading them back through the same table returns the buffer
    pool2 = np.full_like(pool, 0xA5)
    cnt2 = np.zeros_like(pool)
    oracle.kv_unpack(shape, pool_l, stride, planes_of(pool2, L * 2), T, off, bt, packed_l, got, planes_of(cnt2, L * 2),
                     order=oracle.LAYER_MAJOR, head_begin=h0, head_count=hs)
    assert cnt2.sum() == got.size and cnt2.max() == 1 and (pool2[cnt2 == 0] == 0xA5).all()
    assert np.array_equal(pool2[cnt2 == 1], pool[cnt2 == 1])
    back = np.zeros_like(got)
    oracle.kv_pack(shape, pool_l, stride, planes_of(pool2, L * 2), T, off, bt, packed_l, back,
                   order=oracle.LAYER_MAJOR, head_begin=h0, head_count=hs)
    assert np.array_equal(back, got)


# ------------------------------------------------------------------ integrity checksum
def test_checksum_shards_add_up_to_the_whole_and_replicas_equal_it():
    ck = small_checkpoint()
    blob = np.random.default_rng(12).integers(0, 256, ck.nbytes_total, dtype=np.uint8)
    none = np.full(ck.N, -1)
    full = oracle.weights_checksum(ck.byte_off, ck.E, ck.shapes, none, 0, 1, blob)
    W = 4
    parts = [oracle.weights_checksum(ck.byte_off, ck.E, ck.shapes, ck.split_dim, r, W, blob) for r in range(W)]
    with np.errstate(over="ignore"):
        total = np.sum(np.stack(parts), axis=0, dtype=np.uint64)
    for i in range(ck.N):
        if ck.split_dim[i] >= 0:
            assert total[i] == full[i], ck.names[i]          # position-keyed terms: slices partition the sum
        else:
            assert all(p[i] == full[i] for p in parts)        # replicated tensors


def test_checksum_depends_on_every_bit_and_on_position_but_not_on_the_shape_description():
    rng = np.random.default_rng(13)
    blob = rng.integers(0, 256, 4096, dtype=np.uint8)
    base = oracle.weights_checksum([0], [2], [[32, 64, 1, 1]], [-1], 0, 1, blob)[0]
    assert base == oracle.weights_checksum([0], [8], [[512, 1, 1, 1]], [-1], 0, 1, blob)[0]     # same bytes, other shape
    for pos in (0, 7, 8, 1234, 4095):
        for bit in (0, 7):
            b2 = blob.copy()
            b2[pos] ^= 1 << bit
            assert oracle.weights_checksum([0], [2], [[32, 64, 1, 1]], [-1], 0, 1, b2)[0] != base
    b2 = blob.copy()
    b2[0:4], b2[4:8] = blob[4:8], blob[0:4]                                                     # two words swapped
    assert oracle.weights_checksum([0], [2], [[32, 64, 1, 1]], [-1], 0, 1, b2)[0] != base
    # one non-zero word (value 3 at word index 2), by hand with Python integers
    one = np.zeros(16, dtype=np.uint8)
    one[8] = 3
    key2 = (((2 * 0x9E3779B1) << 1) | 1) % 2 ** 32
    assert oracle.weights_checksum([0], [4], [[4, 1, 1, 1]], [-1], 0, 1, one)[0] == 3 * key2
    # a slice that cuts words in half has no checksum
    with pytest.raises(ValueError):
        oracle.weights_checksum([0], [1], [[4, 6, 1, 1]], [1], 0, 3, blob)


# ------------------------------------------------------------------ workload generators
def test_config1_sizes():
    shape, NB, src, dst = wl.config1()
    assert src.n_blocks == 24 and int(src.T.sum()) == 342
    assert oracle.packed_nbytes(shape.tuple, src.T) == 1400832
    offs = np.concatenate([[0], np.cumsum(src.T * shape.token_bytes)])
    assert offs.tolist() == [0, 151552, 561152, 581632, 1400832]
    assert len(set(src.bt.tolist())) == 24 and len(set(dst.bt.tolist())) == 24
    assert wl.LLAMA3_8B_KV.token_bytes == 131072 and wl.LLAMA3_70B_KV.token_bytes == 327680


def test_lognormal_sampler_matches_table3_closed_forms():
    """Table 3 of the paper prints median / mean / P5 / P95 of its three log-normal presets;
    the sampler used for the context lengths must reproduce them."""
    table3 = {(2.1, 0.6): (8.2, 9.8, 3.0, 22.0), (3.0, 0.8): (20.1, 27.7, 5.4, 75.0),
              (4.1, 1.0): (60.3, 99.5, 11.6, 311.0)}
    rng = np.random.default_rng(0)
    for (mu, sigma), (med, mean, p5, p95) in table3.items():
        x = np.exp(mu + sigma * rng.standard_normal(400000))
        assert abs(np.median(x) / med - 1) < 0.02
        assert abs(x.mean() / mean - 1) < 0.03
        assert abs(np.percentile(x, 5) / p5 - 1) < 0.04
        assert abs(np.percentile(x, 95) / p95 - 1) < 0.03
    T = wl.lognormal_lengths(np.random.default_rng(1), 200000, np.log(2048), 1.0, 1, 32768)
    assert abs(np.median(T) / 2048 - 1) < 0.02 and T.max() == 32768 and T.min() >= 1


def test_clipped_geometric_mean():
    p, hi = 1 / 12, 64
    closed = (1 - (1 - p) ** hi) / p   # E[min(G, hi)] = sum_{k<hi} P(G > k)
    x = wl.clipped_geometric(np.random.default_rng(2), 400000, p, hi)
    assert abs(closed - 11.95) < 0.01 and abs(x.mean() / closed - 1) < 0.01 and x.max() == hi


def test_counter_based_fill_host_and_torch_agree():
    import torch
    for kind in ("bits16", "normal"):
        a = np.zeros(2 * 5000, dtype=np.uint8)
        wl.fill_np(a, 77, kind, chunk=1024)
        t = torch.zeros(2 * 5000, dtype=torch.uint8)
        wl.fill_torch(t, 77, kind, chunk=999)
        assert np.array_equal(a, t.numpy())
    vals = torch.from_numpy(wl.normal_bf16_np(5, 0, 200000).view(np.int16).copy()).view(torch.bfloat16).float()
    assert abs(vals.std().item() / 0.02 - 1) < 0.02 and abs(vals.mean().item()) < 2e-4
    bits = wl.bits16_np(5, 0, 1 << 16)
    assert len(np.unique(bits)) > 40000  # uniform 16-bit patterns, not a short cycle


def test_config_generators_are_consistent():
    shape, NB, T_all, waves = wl.config2(NB=2000, R=64, wave_blocks=1500)
    assert sum(len(w[0].T) for w in waves) == 64
    for src, dst in waves:
        assert src.n_blocks <= 1500 and len(set(src.bt.tolist())) == src.n_blocks
        assert len(set(dst.bt.tolist())) == dst.n_blocks and src.bt.max() < NB
    step = next(wl.config5(NB_dev=3000, NB_host=5000, sessions=32, steps=1))
    assert not set(step.reload_host.tolist()) & set(step.offload_host.tolist())
    assert not set(step.reload_dev.tolist()) & set(step.offload_dev.tolist())
