"""GPU parity at the full sizes of the workloads, in the launch configuration the benchmark
times.  The per-element oracle cannot run 16-40 GB in a test, so each case checks
  (a) sampled units (whole requests, row ranges of tensors) against the oracle, fed with the
      very same input bytes, and
  (b) properties that hold at any size, evaluated over every byte: a full materialise
      reproduces the blob, shards tile the full tensors, pack followed by unpack (and migrate)
      lands every source block in its destination block, untouched blocks keep the sentinel.
"""
import numpy as np
import pytest
import torch

import oracle
import paper_2608_06007_b200 as tc
import workloads as wl

pytestmark = pytest.mark.gpu


def _free():
    import gc
    gc.collect()
    torch.cuda.empty_cache()


def _need(nbytes):
    free, _ = torch.cuda.mem_get_info()
    if free < nbytes * 1.05:
        pytest.skip(f"needs {nbytes / 1e9:.0f} GB of device memory, {free / 1e9:.0f} GB free")


def _blocks_to_host(pool, planes, NB, chunk, ids):
    """The (input) bytes of the given blocks of every plane, as compact host planes."""
    g = pool.view(planes, NB, chunk)[:, torch.as_tensor(ids, dtype=torch.long, device=pool.device)]
    return g.cpu().numpy()  # [planes, n, chunk]


def _sample_requests(T):
    order = np.argsort(T)
    picks = {int(order[0]), int(order[len(order) // 3]), int(order[len(order) // 2])}
    tails = [r for r in range(len(T)) if T[r] % 16 and T[r] < 3000]
    if tails:
        picks.add(int(tails[0]))
    return sorted(picks)


def test_config2_full_size_pack_unpack_migrate():
    shape = wl.LLAMA3_8B_KV
    s, chunk, planes = shape.tuple, shape.chunk_bytes, shape.L * 2
    NB, WB = 20000, 8192
    _need((NB + 5 * WB) * shape.block_bytes)
    _, _, _, waves = wl.config2(NB=NB, R=256, wave_blocks=WB, NB_dst=WB)
    src, dst = waves[0]
    u8 = dict(dtype=torch.uint8, device="cuda")
    poolA = torch.empty(NB * shape.block_bytes, **u8)
    wl.fill_torch(poolA, wl.SEED_BASE + 2)
    poolB = torch.full((WB * shape.block_bytes,), 0xA5, **u8)
    payload = int(src.T.sum()) * shape.token_bytes
    Q = torch.full((max(int(w[0].T.sum()) for w in waves) * shape.token_bytes,), 0x5A, **u8)
    plA = tc.pool(tc.TC_NHD, NB, 1, plane_stride=NB * chunk, slot_bytes=poolA.numel())
    plB = tc.pool(tc.TC_NHD, WB, 1, plane_stride=WB * chunk, slot_bytes=poolB.numel())
    kw = dict(T=src.T, bt_off=src.bt_off)
    pack = tc.tc_plan_create(tc.kv_spec(tc.TC_KV_PACK, s, src_pool=plA, packed_layout=tc.TC_HND, packed_bytes=Q.numel(), bt_src=src.bt, **kw))
    unpack = tc.tc_plan_create(tc.kv_spec(tc.TC_KV_UNPACK, s, dst_pool=plB, packed_layout=tc.TC_HND, packed_bytes=Q.numel(), bt_dst=dst.bt, **kw))
    assert pack.stats().payload_bytes[0] == payload and pack.stats().grid[0] == pack.stats().n_tiles[0]
    tc.tc_kv_pack(pack, [poolA], [Q])
    tc.tc_kv_unpack(unpack, [Q], [poolB])
    torch.cuda.synchronize()
    # (a) sampled requests against the oracle
    offs = np.concatenate([[0], np.cumsum(src.T * shape.token_bytes)])
    for r in _sample_requests(src.T):
        ids = src.bt[src.bt_off[r]:src.bt_off[r + 1]]
        host = _blocks_to_host(poolA, planes, NB, chunk, ids)
        n = len(ids)
        want = np.zeros(int(src.T[r]) * shape.token_bytes, dtype=np.uint8)
        oracle.kv_pack(s, oracle.NHD, chunk, [host[p].reshape(-1) for p in range(planes)], [src.T[r]], [0, n], np.arange(n), oracle.HND, want, threads=1)
        got = Q[int(offs[r]):int(offs[r + 1])].cpu().numpy()
        assert np.array_equal(got, want), f"request {r}"
        # and its unpacked blocks
        want_blocks = np.full((planes, n, chunk), 0xA5, dtype=np.uint8)
        oracle.kv_unpack(s, oracle.NHD, chunk, [want_blocks[p].reshape(-1) for p in range(planes)], [src.T[r]], [0, n], np.arange(n), oracle.HND, want)
        got_blocks = _blocks_to_host(poolB, planes, WB, chunk, dst.bt[dst.bt_off[r]:dst.bt_off[r + 1]])
        assert np.array_equal(got_blocks, want_blocks), f"request {r} unpacked"
    # (b) every byte of the packed buffer, as the library routine it reduces to: gather the
    # request's blocks, keep the valid tokens, swap the (token, head) axes (request-level HND)
    A5 = poolA.view(planes, NB, shape.B, shape.H, shape.D * shape.E)
    for r in range(len(src.T)):
        ids = torch.as_tensor(src.bt[src.bt_off[r]:src.bt_off[r + 1]], dtype=torch.long, device="cuda")
        Tr = int(src.T[r])
        tok = A5[:, ids].reshape(planes, -1, shape.H, shape.D * shape.E)[:, :Tr]
        assert torch.equal(tok.permute(0, 2, 1, 3).reshape(-1), Q[int(offs[r]):int(offs[r + 1])]), f"request {r}"
        del tok
    # every full block arrives; every block outside the table keeps the sentinel
    full = np.concatenate([np.arange(src.bt_off[r], src.bt_off[r] + src.T[r] // shape.B) for r in range(len(src.T))])
    sb = torch.as_tensor(src.bt[full], dtype=torch.long, device="cuda")
    db = torch.as_tensor(dst.bt[full], dtype=torch.long, device="cuda")
    A, B = poolA.view(planes, NB, chunk), poolB.view(planes, WB, chunk)
    for p in range(planes):
        assert torch.equal(A[p][sb], B[p][db]), f"plane {p}"
    unused = np.setdiff1d(np.arange(WB), dst.bt)
    ub = torch.as_tensor(unused, dtype=torch.long, device="cuda")
    assert bool((B[:, ub] == 0xA5).all())
    # migrate = pack then unpack, bit for bit
    poolC = torch.full_like(poolB, 0xA5)
    mig = tc.tc_plan_create(tc.kv_spec(tc.TC_KV_MIGRATE, s, src_pool=plA, dst_pool=plB, bt_src=src.bt, bt_dst=dst.bt, **kw))
    tc.tc_kv_pack(mig, [poolA], [poolC])
    torch.cuda.synchronize()
    assert torch.equal(poolC, poolB)
    # every other wave of the workload: the any-size properties over all bytes (full blocks land
    # in their destination blocks, unused destination blocks keep the sentinel), both through
    # pack + unpack and through the fused migrate
    for w_src, w_dst in waves[1:]:
        wkw = dict(T=w_src.T, bt_off=w_src.bt_off)
        wp = int(w_src.T.sum()) * shape.token_bytes
        assert wp <= Q.numel()
        pk = tc.tc_plan_create(tc.kv_spec(tc.TC_KV_PACK, s, src_pool=plA, packed_layout=tc.TC_HND, bt_src=w_src.bt, **wkw))
        up = tc.tc_plan_create(tc.kv_spec(tc.TC_KV_UNPACK, s, dst_pool=plB, packed_layout=tc.TC_HND, bt_dst=w_dst.bt, **wkw))
        mg = tc.tc_plan_create(tc.kv_spec(tc.TC_KV_MIGRATE, s, src_pool=plA, dst_pool=plB, bt_src=w_src.bt, bt_dst=w_dst.bt, **wkw))
        poolB.fill_(0xA5)
        poolC.fill_(0xA5)
        tc.tc_kv_pack(pk, [poolA], [Q])
        tc.tc_kv_unpack(up, [Q], [poolB])
        tc.tc_kv_pack(mg, [poolA], [poolC])
        torch.cuda.synchronize()
        assert torch.equal(poolB, poolC)
        fullw = np.concatenate([np.arange(w_src.bt_off[r], w_src.bt_off[r] + w_src.T[r] // shape.B) for r in range(len(w_src.T))])
        sbw = torch.as_tensor(w_src.bt[fullw], dtype=torch.long, device="cuda")
        dbw = torch.as_tensor(w_dst.bt[fullw], dtype=torch.long, device="cuda")
        for p in range(0, planes, 5):
            assert torch.equal(A[p][sbw], B[p][dbw])
        ubw = torch.as_tensor(np.setdiff1d(np.arange(WB), w_dst.bt), dtype=torch.long, device="cuda")
        assert bool((B[::7, ubw] == 0xA5).all())
        for pl_ in (pk, up, mg):
            pl_.destroy()
    # restore wave 0's results for the staged comparison below
    poolB.fill_(0xA5)
    tc.tc_kv_pack(pack, [poolA], [Q])
    tc.tc_kv_unpack(unpack, [Q], [poolB])
    torch.cuda.synchronize()
    # the packed buffer as a view one byte off a 16-byte boundary (the realigning build at full
    # size): the same bytes, nothing around them touched, and the same pool after the reload
    Q2 = torch.full((Q.numel() + 16,), 0x5A, **u8)
    Qv = Q2[1:1 + Q.numel()]
    poolC.fill_(0xA5)
    tc.tc_kv_pack(pack, [poolA], [Qv])
    tc.tc_kv_unpack(unpack, [Qv], [poolC])
    torch.cuda.synchronize()
    assert torch.equal(Qv[:payload], Q[:payload]) and int(Q2[0]) == 0x5A and bool((Qv[payload:] == 0x5A).all())
    assert torch.equal(poolC, poolB)
    assert tc.tc_device_status() == 0
    del Q2, Qv
    # staged host path at full size: offload to pinned host and reload must reproduce the
    # (oracle-checked) direct results byte for byte
    Qh = torch.empty(payload, dtype=torch.uint8).pin_memory()
    pack_s = tc.tc_plan_create(tc.kv_spec(tc.TC_KV_PACK, s, src_pool=plA, packed_layout=tc.TC_HND, packed_bytes=payload, bt_src=src.bt, flags=tc.TC_PLAN_STAGED, **kw))
    unpack_s = tc.tc_plan_create(tc.kv_spec(tc.TC_KV_UNPACK, s, dst_pool=plB, packed_layout=tc.TC_HND, packed_bytes=payload, bt_dst=dst.bt, flags=tc.TC_PLAN_STAGED, **kw))
    assert pack_s.stats().path[0] == 3 and pack_s.stats().launches_per_execute > 200
    poolC.fill_(0xA5)
    tc.tc_kv_pack(pack_s, [poolA], [Qh])
    tc.tc_kv_unpack(unpack_s, [Qh], [poolC])
    torch.cuda.synchronize()
    for lo in range(0, payload, 1 << 30):
        hi = min(lo + (1 << 30), payload)
        assert torch.equal(Qh[lo:hi].cuda(), Q[lo:hi])
    assert torch.equal(poolC, poolB)
    del poolA, poolB, poolC, Q, Qh, A, B
    _free()


def test_config3_full_size_weights_full_and_all_shards():
    ck = wl.config3()
    _need(2.2 * ck.nbytes_total)
    u8 = dict(dtype=torch.uint8, device="cuda")
    blob = torch.empty(ck.nbytes_total, **u8)
    wl.fill_torch(blob, wl.SEED_BASE + 3, "normal")
    nbytes = [ck.nbytes(i) for i in range(ck.N)]
    offs = np.concatenate([[0], np.cumsum(nbytes)])
    dst = torch.full((ck.nbytes_total,), 0xEE, **u8)
    full = tc.tc_plan_create(tc.weights_spec(ck.byte_off, nbytes, ck.E, ck.ndim, ck.shapes, blob_bytes=ck.nbytes_total))
    tc.tc_weights_materialize(full, blob, [dst.data_ptr() + int(o) for o in offs[:-1]])
    torch.cuda.synchronize()
    assert torch.equal(dst, blob)                  # tight canonical order: the outputs concatenate to the blob
    W = 8
    ssize = [n // (W if ck.split_dim[i] >= 0 else 1) for i, n in enumerate(nbytes)]
    soffs = np.concatenate([[0], np.cumsum(ssize)])
    rng = np.random.default_rng(7)
    shards = []
    for rank in range(W):
        out = torch.full((int(soffs[-1]),), 0xEE, **u8)
        plan = tc.tc_plan_create(tc.weights_spec(ck.byte_off, nbytes, ck.E, ck.ndim, ck.shapes, split_dim=ck.split_dim, rank=rank, world=W, blob_bytes=ck.nbytes_total))
        tc.tc_weights_materialize(plan, blob, [out.data_ptr() + int(o) for o in soffs[:-1]])
        shards.append(out)
    torch.cuda.synchronize()
    # (b) the shards tile every tensor; replicated tensors equal the full ones
    for i in range(ck.N):
        shp = [int(x) for x in ck.shapes[i][:ck.ndim[i]]]
        whole = dst[int(offs[i]):int(offs[i + 1])].view(torch.int16).view(shp)
        sd = int(ck.split_dim[i])
        parts = [sh[int(soffs[i]):int(soffs[i + 1])].view(torch.int16) for sh in shards]
        if sd < 0:
            assert all(torch.equal(p, whole.reshape(-1)) for p in parts), ck.names[i]
        else:
            sshp = list(shp)
            sshp[sd] //= W
            assert torch.equal(torch.cat([p.view(sshp) for p in parts], dim=sd), whole), ck.names[i]
    # (a) sampled tensors / row ranges of one shard against the oracle, fed the blob's own bytes
    rank = 5
    picks = [ck.names.index(n) for n in ("layers.0.input_layernorm", "layers.7.k_proj", "layers.31.o_proj", "layers.13.down_proj", "embed_tokens", "lm_head")]
    for i in picks:
        rows, cols = (int(ck.shapes[i][0]), int(ck.shapes[i][1])) if ck.ndim[i] == 2 else (1, int(ck.shapes[i][0]))
        sd = int(ck.split_dim[i])
        if sd == 0:      # the same k-row window of every rank's slab, given to the oracle as a [W*k, cols] tensor
            k = 3
            a = int(rng.integers(0, rows // W - k))
            base = int(ck.byte_off[i])
            src_rows = torch.cat([blob[base + (q * (rows // W) + a) * cols * 2: base + (q * (rows // W) + a + k) * cols * 2] for q in range(W)]).cpu().numpy()
            want = np.zeros(k * cols * 2, dtype=np.uint8)
            oracle.weights([0], [2], [[W * k, cols, 1, 1]], [0], rank, W, src_rows, [want])
            lo = int(soffs[i]) + a * cols * 2
            got = shards[rank][lo:lo + k * cols * 2].cpu().numpy()
        elif sd == 1:    # k whole rows of the tensor: the oracle slices the rank's columns out of each
            k = 5
            r0 = int(rng.integers(0, rows - k))
            src_rows = blob[int(ck.byte_off[i]) + r0 * cols * 2: int(ck.byte_off[i]) + (r0 + k) * cols * 2].cpu().numpy()
            want = np.zeros(k * (cols // W) * 2, dtype=np.uint8)
            oracle.weights([0], [2], [[k, cols, 1, 1]], [1], rank, W, src_rows, [want])
            lo = int(soffs[i]) + r0 * (cols // W) * 2
            got = shards[rank][lo:lo + want.size].cpu().numpy()
        else:
            src_rows = blob[int(ck.byte_off[i]): int(ck.byte_off[i]) + nbytes[i]].cpu().numpy()
            want = np.zeros(nbytes[i], dtype=np.uint8)
            oracle.weights([0], [2], [[cols, 1, 1, 1]], [-1], 0, 1, src_rows, [want])
            got = shards[rank][int(soffs[i]):int(soffs[i + 1])].cpu().numpy()
        assert np.array_equal(got, want), ck.names[i]
    # the inputs are the generator's: spot-check that the device blob is what the host generator says
    probe = rng.integers(0, ck.nbytes_total // 2, 1000)
    assert np.array_equal(blob.view(torch.int16)[torch.as_tensor(probe, device="cuda")].cpu().numpy().view(np.uint16),
                          wl.normal_bf16_at_np(wl.SEED_BASE + 3, probe))
    del blob, dst, shards
    _free()


def test_config3_full_size_shard_does_not_depend_on_pointer_alignment():
    """The 1-of-8 shard of the full checkpoint through misaligned base pointers - the blob 1 byte
    and every output 9 bytes off a 16-byte boundary, then only the outputs off - must equal the
    aligned run byte for byte (which the test above holds against the oracle): long slabs, the
    strided 1 KiB and 3.5 KiB rows of o_proj / down_proj staged back to back, and the replicated
    norms, with the bytes around every output untouched."""
    ck = wl.config3()
    _need(2.6 * ck.nbytes_total)
    u8 = dict(dtype=torch.uint8, device="cuda")
    raw = torch.empty(ck.nbytes_total + 16, **u8)
    wl.fill_torch(raw, wl.SEED_BASE + 3, "normal")
    nbytes = [ck.nbytes(i) for i in range(ck.N)]
    W, rank = 8, 3
    ssize = [n // (W if ck.split_dim[i] >= 0 else 1) for i, n in enumerate(nbytes)]
    pitch = [(n + 63) // 32 * 32 for n in ssize]             # room for a shift and a gap after every output
    soffs = np.concatenate([[0], np.cumsum(pitch)])
    plan = tc.tc_plan_create(tc.weights_spec(ck.byte_off, nbytes, ck.E, ck.ndim, ck.shapes, split_dim=ck.split_dim, rank=rank, world=W, blob_bytes=ck.nbytes_total))
    outs = {}
    for a, b in ((0, 0), (0, 1), (1, 9)):
        blob = raw[a:a + ck.nbytes_total]
        if a:
            blob.copy_(raw[:ck.nbytes_total].clone())            # the same bytes, one byte further on
        out = torch.full((int(soffs[-1]) + 16,), 0xEE, **u8)
        torch.cuda.synchronize()
        tc.tc_weights_materialize(plan, blob, [out.data_ptr() + int(o) + b for o in soffs[:-1]])
        torch.cuda.synchronize()
        outs[(a, b)] = out
    ref = outs[(0, 0)]
    for (a, b), out in outs.items():
        for i in range(ck.N):
            lo = int(soffs[i])
            assert torch.equal(out[lo + b:lo + b + ssize[i]], ref[lo:lo + ssize[i]]), (ck.names[i], a, b)
            assert bool((out[lo + b + ssize[i]:int(soffs[i + 1]) + b] == 0xEE).all()), (ck.names[i], a, b)
    assert tc.tc_device_status() == 0
    del raw, outs
    _free()


def test_config4_full_size_migration_70b_shape():
    shape = wl.LLAMA3_70B_KV
    s, chunk, planes = shape.tuple, shape.chunk_bytes, shape.L * 2
    NB = 4096
    free, _ = torch.cuda.mem_get_info()
    while 2 * NB * shape.block_bytes > 0.8 * free:
        NB //= 2
    _, _, _, waves = wl.config4(NB=NB, max_waves=2)
    u8 = dict(dtype=torch.uint8, device="cuda")
    poolA = torch.empty(NB * shape.block_bytes, **u8)
    wl.fill_torch(poolA, wl.SEED_BASE + 4)
    plA = tc.pool(tc.TC_NHD, NB, 1, plane_stride=NB * chunk, slot_bytes=poolA.numel())
    A = poolA.view(planes, NB, chunk)
    for wave, dst_layout in zip(waves, (tc.TC_NHD, tc.TC_HND)):
        src, dst = wave
        poolB = torch.full((NB * shape.block_bytes,), 0xA5, **u8)
        plB = tc.pool(dst_layout, NB, 1, plane_stride=NB * chunk, slot_bytes=poolB.numel())
        mig = tc.tc_plan_create(tc.kv_spec(tc.TC_KV_MIGRATE, s, src_pool=plA, dst_pool=plB, T=src.T, bt_off=src.bt_off, bt_src=src.bt, bt_dst=dst.bt))
        assert mig.stats().payload_bytes[0] == int(src.T.sum()) * shape.token_bytes
        tc.tc_kv_pack(mig, [poolA], [poolB])
        torch.cuda.synchronize()
        B = poolB.view(planes, NB, chunk)
        # (a) sampled requests against the oracle
        for r in _sample_requests(src.T)[:3]:
            sid = src.bt[src.bt_off[r]:src.bt_off[r + 1]]
            did = dst.bt[dst.bt_off[r]:dst.bt_off[r + 1]]
            n = len(sid)
            host = _blocks_to_host(poolA, planes, NB, chunk, sid)
            want = np.full((planes, n, chunk), 0xA5, dtype=np.uint8)
            oracle.kv_migrate(s, oracle.NHD, chunk, [host[p].reshape(-1) for p in range(planes)], dst_layout, chunk,
                              [want[p].reshape(-1) for p in range(planes)], [src.T[r]], [0, n], np.arange(n), np.arange(n), threads=1)
            assert np.array_equal(_blocks_to_host(poolB, planes, NB, chunk, did), want), f"request {r}"
        # (b) all full blocks (same layout: equal bytes; HND target: per-block transpose), unused blocks untouched
        full = np.concatenate([np.arange(src.bt_off[r], src.bt_off[r] + src.T[r] // shape.B) for r in range(len(src.T))])
        sb = torch.as_tensor(src.bt[full], dtype=torch.long, device="cuda")
        db = torch.as_tensor(dst.bt[full], dtype=torch.long, device="cuda")
        for p in range(0, planes, 7):
            a, b = A[p][sb], B[p][db]
            if dst_layout == tc.TC_HND:
                a = a.view(-1, shape.B, shape.H, shape.D * shape.E).transpose(1, 2).reshape(-1, chunk)
            assert torch.equal(a, b), f"plane {p}"
        unused = torch.as_tensor(np.setdiff1d(np.arange(NB), dst.bt), dtype=torch.long, device="cuda")
        assert bool((B[::9, unused] == 0xA5).all())
        del poolB, B
        _free()
    del poolA, A
    _free()


@pytest.mark.parametrize("flags", [0, tc.TC_PLAN_STAGED])
def test_config5_mixed_steps_device_pool_and_pinned_paged_host_pool(flags):
    shape = wl.LLAMA3_8B_KV
    s, chunk, planes = shape.tuple, shape.chunk_bytes, shape.L * 2
    NBd, NBh = 20000, 4096                       # host pool shrunk to 8 GiB of pinned memory
    _need(NBd * shape.block_bytes)
    u8 = dict(dtype=torch.uint8, device="cuda")
    dev = torch.empty(NBd * shape.block_bytes, **u8)
    wl.fill_torch(dev, wl.SEED_BASE + 5)
    host = torch.empty(NBh * shape.block_bytes, dtype=torch.uint8).pin_memory()
    tmp = torch.empty(host.numel(), **u8)
    wl.fill_torch(tmp, wl.SEED_BASE + 55)
    host.copy_(tmp)
    del tmp
    dev_pool = tc.pool(tc.TC_NHD, NBd, 1, plane_stride=NBd * chunk, slot_bytes=dev.numel())
    host_pool = tc.pool(tc.TC_HND, NBh, 1, plane_stride=chunk, block_stride=planes * chunk, slot_bytes=host.numel())
    s1, s2 = torch.cuda.Stream(), torch.cuda.Stream()
    for step in wl.config5(NB_dev=NBd, NB_host=NBh, sessions=128, steps=2):
        before_dev_reads = _blocks_to_host(dev, planes, NBd, chunk, step.offload_dev)     # inputs of the offload
        H = host.numpy().reshape(NBh, planes, chunk)
        before_host_reads = H[step.reload_host].copy()                                       # inputs of the reload
        spec = tc.kv_spec(tc.TC_KV_MIXED, s, src_pool=dev_pool, dst_pool=host_pool,
                          T=step.offload_T, bt_off=step.offload_off, bt_src=step.offload_dev, bt_dst=step.offload_host,
                          reload=dict(T=step.reload_T, bt_off=step.reload_off, bt_src=step.reload_host, bt_dst=step.reload_dev), flags=flags)
        plan = tc.tc_plan_create(spec)
        assert plan.stats().path[1] == (3 if flags else 1)
        torch.cuda.synchronize()
        tc.tc_kv_pack(plan, [dev], [host], stream=s1)
        tc.tc_kv_unpack(plan, [host], [dev], stream=s2)
        torch.cuda.synchronize()
        # (a) the oracle on sampled sessions, both directions (compact pools)
        for sess in (0, 17, 127):
            a, b = int(step.offload_off[sess]), int(step.offload_off[sess + 1])
            n = b - a
            want = np.zeros((n, planes, chunk), dtype=np.uint8)
            oracle.kv_migrate(s, oracle.NHD, chunk, [before_dev_reads[p, a:b].reshape(-1) for p in range(planes)], oracle.HND, planes * chunk,
                              [want.reshape(-1)[p * chunk:] for p in range(planes)], [n * shape.B], [0, n], np.arange(n), np.arange(n))
            assert np.array_equal(H[step.offload_host[a:b]], want), f"offload session {sess}"
            a, b = int(step.reload_off[sess]), int(step.reload_off[sess + 1])
            n = b - a
            src_h = np.ascontiguousarray(before_host_reads[a:b])
            want = np.zeros((planes, n, chunk), dtype=np.uint8)
            oracle.kv_migrate(s, oracle.HND, planes * chunk, [src_h.reshape(-1)[p * chunk:] for p in range(planes)], oracle.NHD, chunk,
                              [want[p].reshape(-1) for p in range(planes)], [n * shape.B], [0, n], np.arange(n), np.arange(n))
            assert np.array_equal(_blocks_to_host(dev, planes, NBd, chunk, step.reload_dev[a:b]), want), f"reload session {sess}"
        # (b) every reloaded block, as a per-block transpose of its host page
        got = _blocks_to_host(dev, planes, NBd, chunk, step.reload_dev)                    # [planes, n, chunk] NHD
        exp = before_host_reads.reshape(-1, planes, shape.H, shape.B, shape.D * shape.E).transpose(1, 0, 3, 2, 4).reshape(planes, -1, chunk)
        assert np.array_equal(got, exp)
        plan.destroy()
    del dev, host
    _free()
