"""CPU oracle for descriptor-driven batched tensor movement: TEST INFRASTRUCTURE ONLY.

This package wraps ``tc_oracle.c`` (plain per-element C loops, compiled with gcc) for
numpy callers.  It defines what KV pack (publish), KV unpack (hydrate), pool-to-pool
migration and weight materialisation (tensor_dict / view / transform_into, Table 2 of
the paper) must produce, byte for byte.  It imports nothing from the CUDA package and
the CUDA package imports nothing from here; only the tests, the smoke check and the
benchmark's CPU-baseline leg may use it.

All buffers are ``numpy.uint8`` arrays.  A paged pool is passed as a list of L*2 plane
arrays (index l*2+c, c=0 K, c=1 V); planes may be views into one allocation.
"""
from __future__ import annotations

import ctypes as C
import os
import subprocess
from concurrent.futures import ThreadPoolExecutor

import numpy as np

NHD, HND = 0, 1
REQUEST_MAJOR, LAYER_MAJOR = 0, 1

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "tc_oracle.c")
_SO = os.path.join(_HERE, "libtc_oracle.so")


def build(force: bool = False) -> str:
    """Compile tc_oracle.c into libtc_oracle.so next to it (gcc -O2) and return the path."""
    if force or not os.path.exists(_SO) or os.path.getmtime(_SO) < os.path.getmtime(_SRC):
        tmp = _SO + f".{os.getpid()}.tmp"
        subprocess.check_call(["gcc", "-O2", "-std=c11", "-Wall", "-Wextra", "-shared", "-fPIC",
                               "-o", tmp, _SRC])
        os.replace(tmp, _SO)
    return _SO


class _Shape(C.Structure):
    _fields_ = [(n, C.c_int64) for n in ("L", "B", "H", "D", "E")]


class _Geom(C.Structure):
    _fields_ = [("layout", C.c_int32), ("block_stride", C.c_int64)]


class _Packed(C.Structure):
    _fields_ = [("layout", C.c_int32), ("order", C.c_int32), ("h0", C.c_int64), ("hs", C.c_int64)]


def _packed_geom(shape, layout, order, head_begin, head_count):
    H = shape[2]
    hs = H - head_begin if head_count is None else head_count
    assert 0 <= head_begin and hs >= 0 and head_begin + hs <= H
    return _Packed(layout, order, head_begin, hs)


_lib = None


def _load():
    global _lib
    if _lib is None:
        _lib = C.CDLL(build())
    return _lib


def _u8(a: np.ndarray) -> np.ndarray:
    assert a.dtype == np.uint8 and a.ndim == 1 and (a.size == 0 or a.strides[0] == 1), "oracle buffers are flat uint8"
    return a


def _ptr_table(arrs):
    t = (C.c_void_p * len(arrs))()
    for i, a in enumerate(arrs):
        t[i] = None if a is None else _u8(a).ctypes.data
    return t


def _i64(a):
    return np.ascontiguousarray(np.asarray(a, dtype=np.int64))


def _i32(a):
    return np.ascontiguousarray(np.asarray(a, dtype=np.int32))


def _split(n_items: int, threads: int):
    threads = max(1, min(threads, n_items))
    edges = np.linspace(0, n_items, threads + 1).astype(np.int64)
    return [(int(edges[k]), int(edges[k + 1])) for k in range(threads) if edges[k] < edges[k + 1]]


def _ranges(R, threads, requests):
    if requests is None:
        return _split(R, threads)
    r0, r1 = requests
    return [(r0 + a, r0 + b) for a, b in _split(r1 - r0, threads)]


def _run(fn, ranges, threads):
    if threads <= 1 or len(ranges) <= 1:
        for a, b in ranges:
            fn(a, b)
    else:
        with ThreadPoolExecutor(max_workers=threads) as ex:
            list(ex.map(lambda ab: fn(*ab), ranges))


def packed_nbytes(shape, T, head_count=None) -> int:
    """Size of the packed buffer: sum over requests of L*2*T_r*Hs*D*E (Hs = heads it holds)."""
    L, B, H, D, E = shape
    H = H if head_count is None else head_count
    return int(sum(L * 2 * int(t) * H * D * E for t in T))


def kv_pack(shape, pool_layout, block_stride, planes, T, bt_off, bt, packed_layout,
            packed, packed_cnt=None, threads=1, requests=None, order=REQUEST_MAJOR,
            head_begin=0, head_count=None):
    """publish / offload: pool planes -> packed buffer (written in place).
    requests=(r0, r1) restricts the loops to requests [r0, r1) (same arithmetic).
    order / head_begin / head_count: layer-major packed order, head slice of the packed side."""
    lib = _load()
    s, g = _Shape(*shape), _Geom(pool_layout, block_stride)
    pg = _packed_geom(shape, packed_layout, order, head_begin, head_count)
    T, bt_off, bt = _i64(T), _i64(bt_off), _i32(bt)
    tbl = _ptr_table(planes)
    R = len(T)

    def go(r0, r1):
        lib.oracle_kv_pack(C.byref(s), C.byref(g), tbl, C.c_int64(R), T.ctypes, bt_off.ctypes,
                           bt.ctypes, C.byref(pg), C.c_void_p(_u8(packed).ctypes.data),
                           C.c_void_p(None if packed_cnt is None else _u8(packed_cnt).ctypes.data),
                           C.c_int64(r0), C.c_int64(r1))
    _run(go, _ranges(R, threads, requests), threads)


def kv_pack_inverse(shape, pool_layout, block_stride, planes, T, bt_off, bt, packed_layout, packed):
    """Second formulation of pack: decode every packed byte offset (cross-check only)."""
    lib = _load()
    s, g = _Shape(*shape), _Geom(pool_layout, block_stride)
    T, bt_off, bt = _i64(T), _i64(bt_off), _i32(bt)
    tbl = _ptr_table(planes)
    lib.oracle_kv_pack_inverse(C.byref(s), C.byref(g), tbl, C.c_int64(len(T)), T.ctypes,
                               bt_off.ctypes, bt.ctypes, C.c_int32(packed_layout),
                               C.c_void_p(_u8(packed).ctypes.data), C.c_int64(0),
                               C.c_int64(packed.size))


def kv_unpack(shape, pool_layout, block_stride, planes, T, bt_off, bt, packed_layout,
              packed, plane_cnt=None, threads=1, requests=None, order=REQUEST_MAJOR,
              head_begin=0, head_count=None):
    """hydrate / reload: packed buffer -> pool planes (written in place)."""
    lib = _load()
    s, g = _Shape(*shape), _Geom(pool_layout, block_stride)
    pg = _packed_geom(shape, packed_layout, order, head_begin, head_count)
    T, bt_off, bt = _i64(T), _i64(bt_off), _i32(bt)
    tbl = _ptr_table(planes)
    cnt = None if plane_cnt is None else _ptr_table(plane_cnt)
    R = len(T)

    def go(r0, r1):
        lib.oracle_kv_unpack(C.byref(s), C.byref(g), tbl, cnt, C.c_int64(R), T.ctypes,
                             bt_off.ctypes, bt.ctypes, C.byref(pg),
                             C.c_void_p(_u8(packed).ctypes.data), C.c_int64(r0), C.c_int64(r1))
    _run(go, _ranges(R, threads, requests), threads)


def kv_migrate(shape, src_layout, src_block_stride, src_planes, dst_layout, dst_block_stride,
               dst_planes, T, bt_off, bt_src, bt_dst, dst_cnt=None, threads=1, requests=None):
    """publish then hydrate, fused: src pool -> dst pool through two block tables."""
    lib = _load()
    s = _Shape(*shape)
    gs, gd = _Geom(src_layout, src_block_stride), _Geom(dst_layout, dst_block_stride)
    T, bt_off, bt_src, bt_dst = _i64(T), _i64(bt_off), _i32(bt_src), _i32(bt_dst)
    ts, td = _ptr_table(src_planes), _ptr_table(dst_planes)
    cnt = None if dst_cnt is None else _ptr_table(dst_cnt)
    R = len(T)

    def go(r0, r1):
        lib.oracle_kv_migrate(C.byref(s), C.byref(gs), ts, C.byref(gd), td, cnt, C.c_int64(R),
                              T.ctypes, bt_off.ctypes, bt_src.ctypes, bt_dst.ctypes,
                              C.c_int64(r0), C.c_int64(r1))
    _run(go, _ranges(R, threads, requests), threads)


def weights(blob_off, E, shapes, split_dim, rank, world, blob, dst, dst_off=None,
            dst_stride=None, dst_cnt=None, threads=1):
    """Materialise tensors (whole, or rank's slab of split_dim) from the flat blob into dst[i].

    shapes: [N][4] (unused dims 1).  dst_stride: [N][4] byte strides; default = tight
    row-major strides of the destination shape.  dst_off: [N] byte offsets (default 0).
    """
    lib = _load()
    N = len(blob_off)
    blob_off, E = _i64(blob_off), _i64(E)
    shapes = _i64(shapes).reshape(N, 4)
    split_dim = _i32(split_dim)
    if dst_stride is None:
        dst_stride = np.zeros((N, 4), dtype=np.int64)
        for i in range(N):
            ext = [int(x) for x in shapes[i]]
            if split_dim[i] >= 0:
                ext[split_dim[i]] //= world
            st = int(E[i])
            for m in (3, 2, 1, 0):
                dst_stride[i, m] = st
                st *= ext[m]
    dst_stride = _i64(dst_stride).reshape(N, 4)
    dst_off = _i64(np.zeros(N) if dst_off is None else dst_off)
    td = _ptr_table(dst)
    cnt = None if dst_cnt is None else _ptr_table(dst_cnt)

    def go(i0, i1):
        lib.oracle_weights(C.c_int64(N), blob_off.ctypes, E.ctypes, shapes.ctypes, split_dim.ctypes,
                           C.c_int64(rank), C.c_int64(world), C.c_void_p(_u8(blob).ctypes.data),
                           td, dst_off.ctypes, dst_stride.ctypes, cnt, C.c_int64(i0), C.c_int64(i1))
    # split per tensor so that skewed sizes still spread over the threads
    _run(go, [(i, i + 1) for i in range(N)] if threads > 1 else [(0, N)], threads)


def weights_checksum(blob_off, E, shapes, split_dim, rank, world, blob):
    """Integrity checksums (uint64 per tensor) of the words the rank's slice covers; raises if a
    slice covers a 4-byte word only partly."""
    lib = _load()
    N = len(blob_off)
    blob_off, E = _i64(blob_off), _i64(E)
    shapes = _i64(shapes).reshape(N, 4)
    split_dim = _i32(split_dim)
    sums = np.zeros(N, dtype=np.uint64)
    biggest = int(max((int(np.prod(shapes[i])) * int(E[i]) for i in range(N)), default=0))
    scratch = np.zeros(max(biggest, 1), dtype=np.uint8)
    status = C.c_int32(0)
    lib.oracle_weights_checksum(C.c_int64(N), blob_off.ctypes, E.ctypes, shapes.ctypes, split_dim.ctypes,
                                C.c_int64(rank), C.c_int64(world), C.c_void_p(_u8(blob).ctypes.data),
                                sums.ctypes, scratch.ctypes, C.byref(status))
    if status.value != 0:
        raise ValueError("a slice covers a 4-byte word only partly: its checksum is undefined")
    return sums
