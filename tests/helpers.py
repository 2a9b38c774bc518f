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
