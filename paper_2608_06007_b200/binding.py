"""ctypes binding of libtensorcast_b200.so: argument marshalling only.

The functions carry the names of the C ABI (include/tensorcast.h): tc_plan_create, tc_kv_pack,
tc_kv_unpack, tc_weights_materialize, tc_plan_destroy, plus the inspection calls.  Every byte
is moved by the library's CUDA kernels; there is no fallback: a missing library or a failing
call raises.  Pointers may be given as ints or as objects with ``data_ptr()`` (torch tensors).
"""
from __future__ import annotations

import ctypes as C
import os

import numpy as np

from . import build as _build

TC_OK = 0
TC_ERR_INVALID_ARG, TC_ERR_SHAPE, TC_ERR_BOUNDS, TC_ERR_OVERLAP = -1, -2, -3, -4
TC_ERR_KIND, TC_ERR_OOM, TC_ERR_CUDA, TC_ERR_DEADLINE, TC_ERR_TOO_LARGE, TC_ERR_IO = -5, -6, -7, -8, -9, -10
TC_NOALLOC_SCRATCH_BYTES = 1 << 20
TC_KV_PACK, TC_KV_UNPACK, TC_KV_MIGRATE, TC_KV_MIXED, TC_WEIGHTS = 1, 2, 3, 4, 5
TC_NHD, TC_HND = 0, 1
TC_REQUEST_MAJOR, TC_LAYER_MAJOR = 0, 1
TC_PLAN_HOST_ONLY = 1
TC_PLAN_STAGED = 2
TC_PLAN_CHECKSUM = 4
TC_PLAN_SAME_POOL = 8
TC_PLAN_STREAM = 16
TC_PLAN_OFFLOAD_ZERO_COPY = 32
TC_PLAN_TRACE = 64
TC_PLAN_DEBUG_BOUNDS = 128
TC_MAX_TABLE_SLOTS = 4000
TC_DEVICE_BULK_WAIT_TIMEOUT = 1
TC_DEVICE_OUT_OF_BOUNDS = 2


class tc_kv_pool_t(C.Structure):
    _fields_ = [("layout", C.c_int32), ("reserved", C.c_int32), ("num_blocks", C.c_int64),
                ("n_slots", C.c_int64), ("plane_stride", C.c_int64), ("block_stride", C.c_int64),
                ("slot_bytes", C.c_int64)]


class tc_kv_group_t(C.Structure):
    _fields_ = [("R", C.c_int64), ("T", C.c_void_p), ("bt_off", C.c_void_p),
                ("bt_src", C.c_void_p), ("bt_dst", C.c_void_p)]


class tc_kv_spec_t(C.Structure):
    _fields_ = [("L", C.c_int64), ("B", C.c_int64), ("H", C.c_int64), ("D", C.c_int64), ("E", C.c_int64),
                ("src_pool", tc_kv_pool_t), ("dst_pool", tc_kv_pool_t),
                ("packed_layout", C.c_int32), ("packed_order", C.c_int32), ("packed_bytes", C.c_int64),
                ("head_begin", C.c_int64), ("head_count", C.c_int64),
                ("group", tc_kv_group_t), ("reload", tc_kv_group_t)]


class tc_index_entry_t(C.Structure):
    _fields_ = [("byte_off", C.c_uint64), ("nbytes", C.c_uint64), ("elem_bytes", C.c_uint32),
                ("ndim", C.c_uint32), ("shape", C.c_uint64 * 4), ("name_id", C.c_uint64)]


class tc_weight_rule_t(C.Structure):
    _fields_ = [("split_dim", C.c_int32), ("dst_slot", C.c_int32), ("dst_off", C.c_int64),
                ("dst_stride", C.c_int64 * 4)]


class tc_weights_spec_t(C.Structure):
    _fields_ = [("n_tensors", C.c_int64), ("index", C.c_void_p), ("rules", C.c_void_p),
                ("rank", C.c_int32), ("world", C.c_int32), ("blob_bytes", C.c_int64),
                ("n_dst", C.c_int64), ("dst_bytes", C.c_void_p)]


class tc_tuning_t(C.Structure):
    _fields_ = [("tile_bytes", C.c_int32), ("ctas_per_sm", C.c_int32), ("max_ctas", C.c_int32),
                ("tile_order", C.c_int32), ("copy_path", C.c_int32), ("reserved", C.c_int32)]


class tc_plan_spec_t(C.Structure):
    _fields_ = [("struct_size", C.c_uint32), ("kind", C.c_int32), ("flags", C.c_uint32),
                ("reserved", C.c_uint32), ("trace_id", C.c_uint64), ("deadline_ns", C.c_int64),
                ("tuning", tc_tuning_t), ("kv", tc_kv_spec_t), ("weights", tc_weights_spec_t)]


class tc_plan_stats_t(C.Structure):
    _fields_ = [("trace_id", C.c_uint64), ("kind", C.c_int32), ("executable", C.c_int32),
                ("n_descriptors", C.c_int64 * 2), ("n_tiles", C.c_int64 * 2),
                ("payload_bytes", C.c_int64 * 2), ("packed_bytes_required", C.c_int64),
                ("device_bytes", C.c_int64), ("vec_bytes", C.c_int32 * 2),
                ("launches_per_execute", C.c_int32), ("path", C.c_int32 * 2), ("grid", C.c_int32 * 2),
                ("last_device_us", C.c_double * 2)]


class tc_descriptor_t(C.Structure):
    _fields_ = [(n, C.c_int64) for n in ("src_off", "dst_off", "src_outer", "dst_outer",
                                          "src_s0", "src_s1", "dst_s0", "dst_s1")] + \
               [(n, C.c_uint32) for n in ("src_slot", "dst_slot", "src_slot_step", "dst_slot_step",
                                          "run_bytes", "n0", "rows", "n_outer",
                                          "rows_per_tile", "tiles_per_outer", "tile0", "planes_per_tile")]


class tc_segment_t(C.Structure):
    _fields_ = [("host_off", C.c_int64), ("bytes", C.c_int64), ("tile0", C.c_uint32), ("n_tiles", C.c_uint32),
                ("desc0", C.c_uint32), ("n_descs", C.c_uint32), ("outer0", C.c_uint32), ("n_outer", C.c_uint32)]


EXPORTS = ("tc_plan_create", "tc_kv_pack", "tc_kv_unpack", "tc_weights_materialize",
           "tc_plan_destroy", "tc_plan_stats", "tc_plan_descriptors", "tc_strerror", "tc_last_error",
           "tc_kv_pack_noalloc", "tc_weights_materialize_checksum", "tc_trim",
           "tc_weights_materialize_file", "tc_plan_segments", "tc_device_status", "tc_selftest_wait_timeout", "tc_plan_check_device")

_lib = None


def load_library(path: str | None = None):
    """Load (building first if stale) the C-ABI library.  Raises if it cannot be had."""
    global _lib
    if _lib is not None and path is None:
        return _lib
    path = path or _build.build_library()
    if not os.path.exists(path):
        raise RuntimeError(f"{path} is missing: build it with paper_2608_06007_b200.build")
    lib = C.CDLL(path)
    vp, sz = C.c_void_p, C.c_size_t
    lib.tc_plan_create.argtypes = [C.POINTER(tc_plan_spec_t), C.POINTER(vp)]
    lib.tc_kv_pack.argtypes = [vp, vp, sz, vp, sz, vp]
    lib.tc_kv_unpack.argtypes = [vp, vp, sz, vp, sz, vp]
    lib.tc_weights_materialize.argtypes = [vp, vp, vp, sz, vp]
    lib.tc_plan_destroy.argtypes = [vp]
    lib.tc_plan_stats.argtypes = [vp, C.POINTER(tc_plan_stats_t)]
    lib.tc_plan_descriptors.argtypes = [vp, C.c_int, vp, sz, C.POINTER(sz)]
    lib.tc_kv_pack_noalloc.argtypes = [C.POINTER(tc_plan_spec_t), vp, sz, vp, sz, vp]
    lib.tc_kv_pack_noalloc.restype = C.c_int
    lib.tc_weights_materialize_checksum.argtypes = [vp, vp, vp, sz, vp, vp]
    lib.tc_weights_materialize_checksum.restype = C.c_int
    lib.tc_weights_materialize_file.argtypes = [vp, C.c_int, C.c_int64, vp, sz, vp, vp]
    lib.tc_weights_materialize_file.restype = C.c_int
    lib.tc_plan_segments.argtypes = [vp, C.c_int, vp, sz, C.POINTER(sz)]
    lib.tc_plan_segments.restype = C.c_int
    lib.tc_device_status.argtypes = [C.POINTER(C.c_uint32)]
    lib.tc_device_status.restype = C.c_int
    lib.tc_plan_check_device.argtypes = [vp, C.c_int64, vp]
    lib.tc_plan_check_device.restype = C.c_int
    lib.tc_selftest_wait_timeout.argtypes = [vp]
    lib.tc_selftest_wait_timeout.restype = C.c_int
    lib.tc_trim.argtypes = []
    lib.tc_trim.restype = C.c_int
    lib.tc_strerror.argtypes = [C.c_int]
    lib.tc_strerror.restype = C.c_char_p
    lib.tc_last_error.restype = C.c_char_p
    for name in EXPORTS[:7]:
        getattr(lib, name).restype = C.c_int
    _lib = lib
    return lib


class TensorCastError(RuntimeError):
    def __init__(self, status: int, detail: str):
        self.status = status
        name = load_library().tc_strerror(status).decode()
        super().__init__(f"{name}: {detail}")


def _check(rc: int):
    if rc != TC_OK:
        raise TensorCastError(rc, load_library().tc_last_error().decode())


def _addr(p) -> int:
    if p is None:
        return 0
    if hasattr(p, "data_ptr"):
        return int(p.data_ptr())
    if isinstance(p, np.ndarray):
        return int(p.ctypes.data)
    return int(p)


def _table(ptrs):
    ptrs = list(ptrs) if not hasattr(ptrs, "data_ptr") and not isinstance(ptrs, int) else [ptrs]
    arr = (C.c_void_p * max(len(ptrs), 1))()
    for i, p in enumerate(ptrs):
        arr[i] = _addr(p)
    return arr, len(ptrs)


def _stream(stream) -> int:
    if stream is None:
        return 0
    return int(getattr(stream, "cuda_stream", stream))


def pool(layout, num_blocks, n_slots, plane_stride=0, block_stride=0, slot_bytes=0) -> tc_kv_pool_t:
    return tc_kv_pool_t(layout, 0, num_blocks, n_slots, plane_stride, block_stride, slot_bytes)


class _Keep:
    """Keeps the numpy arrays a spec points to alive while the spec is in use."""

    def __init__(self):
        self.refs = []

    def i64(self, a):
        a = np.ascontiguousarray(np.asarray(a, dtype=np.int64))
        self.refs.append(a)
        return a.ctypes.data

    def i32(self, a):
        if a is None:
            return None
        a = np.ascontiguousarray(np.asarray(a, dtype=np.int32))
        self.refs.append(a)
        return a.ctypes.data


def group(keep: _Keep, T, bt_off, bt_src=None, bt_dst=None) -> tc_kv_group_t:
    T = np.asarray(T, dtype=np.int64)
    return tc_kv_group_t(len(T), keep.i64(T), keep.i64(bt_off), keep.i32(bt_src), keep.i32(bt_dst))


def kv_spec(kind, shape, *, src_pool=None, dst_pool=None, packed_layout=TC_NHD, packed_bytes=0,
            T=(), bt_off=(0,), bt_src=None, bt_dst=None, reload=None, flags=0, trace_id=0,
            deadline_ns=0, tuning=None, packed_order=TC_REQUEST_MAJOR, head_begin=0, head_count=0):
    """Assemble a tc_plan_spec_t for the KV kinds.  shape = (L, B, H, D, E);
    reload = dict(T=, bt_off=, bt_src=, bt_dst=) for TC_KV_MIXED.  Returns (spec, keepalive)."""
    keep = _Keep()
    spec = tc_plan_spec_t()
    spec.struct_size = C.sizeof(tc_plan_spec_t)
    spec.kind, spec.flags, spec.trace_id, spec.deadline_ns = kind, flags, trace_id, deadline_ns
    if tuning:
        spec.tuning = tc_tuning_t(**tuning)
    kv = spec.kv
    kv.L, kv.B, kv.H, kv.D, kv.E = shape
    if src_pool is not None:
        kv.src_pool = src_pool
    if dst_pool is not None:
        kv.dst_pool = dst_pool
    kv.packed_layout, kv.packed_bytes = packed_layout, packed_bytes
    kv.packed_order, kv.head_begin, kv.head_count = packed_order, head_begin, head_count
    kv.group = group(keep, T, bt_off, bt_src, bt_dst)
    if reload is not None:
        kv.reload = group(keep, reload["T"], reload["bt_off"], reload["bt_src"], reload["bt_dst"])
    return spec, keep


def weights_spec(byte_off, nbytes, elem_bytes, ndim, shapes, *, split_dim=None, rank=0, world=1,
                 blob_bytes=0, dst_slot=None, dst_off=None, dst_stride=None, n_dst=0, dst_bytes=None,
                 flags=0, trace_id=0, deadline_ns=0, tuning=None):
    """Assemble a tc_plan_spec_t for TC_WEIGHTS from index arrays.  Returns (spec, keepalive)."""
    keep = _Keep()
    N = len(byte_off)
    index = (tc_index_entry_t * max(N, 1))()
    shapes = np.asarray(shapes, dtype=np.int64).reshape(N, 4)
    for i in range(N):
        index[i] = tc_index_entry_t(int(byte_off[i]), int(nbytes[i]), int(elem_bytes[i]), int(ndim[i]),
                                    (C.c_uint64 * 4)(*[int(x) for x in shapes[i]]), i)
    keep.refs.append(index)
    spec = tc_plan_spec_t()
    spec.struct_size = C.sizeof(tc_plan_spec_t)
    spec.kind, spec.flags, spec.trace_id, spec.deadline_ns = TC_WEIGHTS, flags, trace_id, deadline_ns
    if tuning:
        spec.tuning = tc_tuning_t(**tuning)
    w = spec.weights
    w.n_tensors, w.index = N, C.addressof(index)
    if split_dim is not None or dst_slot is not None or dst_off is not None or dst_stride is not None:
        rules = (tc_weight_rule_t * max(N, 1))()
        for i in range(N):
            rules[i].split_dim = -1 if split_dim is None else int(split_dim[i])
            rules[i].dst_slot = -1 if dst_slot is None else int(dst_slot[i])
            rules[i].dst_off = 0 if dst_off is None else int(dst_off[i])
            if dst_stride is not None:
                rules[i].dst_stride = (C.c_int64 * 4)(*[int(x) for x in dst_stride[i]])
        keep.refs.append(rules)
        w.rules = C.addressof(rules)
    w.rank, w.world, w.blob_bytes, w.n_dst = rank, world, blob_bytes, n_dst
    if dst_bytes is not None:
        w.dst_bytes = keep.i64(dst_bytes)
    return spec, keep


class Plan:
    """Owns a tc_plan_t*; destroyed explicitly or when collected."""

    def __init__(self, handle: int):
        self.handle = handle

    def destroy(self):
        if self.handle:
            _check(load_library().tc_plan_destroy(self.handle))
            self.handle = 0

    def __del__(self):
        try:
            self.destroy()
        except Exception:
            pass

    def stats(self) -> tc_plan_stats_t:
        return tc_plan_stats(self)

    def descriptors(self, group: int = 0):
        return tc_plan_descriptors(self, group)

    def segments(self, group: int = 0):
        return tc_plan_segments(self, group)


def tc_plan_create(spec, keep=None) -> Plan:
    if isinstance(spec, tuple):
        spec, keep = spec
    out = C.c_void_p()
    _check(load_library().tc_plan_create(C.byref(spec), C.byref(out)))
    return Plan(out.value)


def tc_plan_destroy(plan: Plan) -> None:
    plan.destroy()


def tc_kv_pack(plan: Plan, src_bases, dst_bases, stream=None) -> None:
    s, ns = _table(src_bases)
    d, nd = _table(dst_bases)
    _check(load_library().tc_kv_pack(plan.handle, s, ns, d, nd, _stream(stream)))


def tc_kv_pack_noalloc(spec, src_bases, dst_bases, stream=None) -> None:
    """tc_kv_pack for callers that must not allocate device memory: lowers `spec` and runs it
    in one call, with the descriptors in the library's fixed 1 MiB scratch area instead of a
    cudaMalloc'ed plan.  Calls whose GPU work may overlap race on that area; keep them on one
    stream.  Raises TC_ERR_TOO_LARGE when the request does not fit."""
    if isinstance(spec, tuple):
        spec = spec[0]
    s, ns = _table(src_bases)
    d, nd = _table(dst_bases)
    _check(load_library().tc_kv_pack_noalloc(C.byref(spec), s, ns, d, nd, _stream(stream)))


def tc_kv_unpack(plan: Plan, src_bases, dst_bases, stream=None) -> None:
    s, ns = _table(src_bases)
    d, nd = _table(dst_bases)
    _check(load_library().tc_kv_unpack(plan.handle, s, ns, d, nd, _stream(stream)))


def tc_weights_materialize(plan: Plan, blob, dst_ptrs, stream=None) -> None:
    d, nd = _table(dst_ptrs)
    _check(load_library().tc_weights_materialize(plan.handle, _addr(blob), d, nd, _stream(stream)))


def tc_weights_materialize_checksum(plan: Plan, blob, dst_ptrs, checksums, stream=None) -> None:
    """tc_weights_materialize that also fills `checksums` (device uint64[n_tensors]) in the same pass."""
    d, nd = _table(dst_ptrs)
    _check(load_library().tc_weights_materialize_checksum(plan.handle, _addr(blob), d, nd, _addr(checksums), _stream(stream)))


def tc_weights_materialize_file(plan: Plan, fd: int, file_offset: int, dst_ptrs, checksums=None, stream=None) -> None:
    """tc_weights_materialize with the blob read from file descriptor `fd`, starting at byte
    `file_offset` (plan created with TC_PLAN_STREAM).  Blocks while the file is read; the device
    work completes on `stream`."""
    d, nd = _table(dst_ptrs)
    cs = _addr(checksums) if checksums is not None else None
    _check(load_library().tc_weights_materialize_file(plan.handle, int(fd), int(file_offset), d, nd, cs, _stream(stream)))


def tc_plan_segments(plan: Plan, group: int = 0):
    """Chunks of a staged / streamed plan as a list of tc_segment_t."""
    lib = load_library()
    n = C.c_size_t()
    _check(lib.tc_plan_segments(plan.handle, group, None, 0, C.byref(n)))
    arr = (tc_segment_t * max(1, n.value))()
    _check(lib.tc_plan_segments(plan.handle, group, C.cast(arr, C.c_void_p), n.value, C.byref(n)))
    return list(arr[:n.value])


def tc_trim() -> None:
    """Release the device memory the library caches between plans (plan-storage blocks, idle staging rings)."""
    _check(load_library().tc_trim())


def tc_device_status() -> int:
    """Flags kernels have set on the current device since the last call (0 = none); waits for the device."""
    v = C.c_uint32()
    _check(load_library().tc_device_status(C.byref(v)))
    return int(v.value)


def tc_plan_check_device(plan: Plan, shrink: int = 0, stream=None) -> None:
    """Run the device-side bounds checker of a TC_PLAN_DEBUG_BOUNDS plan (slot extents less
    `shrink` bytes); the outcome is read with tc_device_status()."""
    _check(load_library().tc_plan_check_device(plan.handle, int(shrink), _stream(stream)))


def tc_selftest_wait_timeout(stream=None) -> None:
    """Run the self-test of the bounded device-side wait: afterwards tc_device_status() reports
    TC_DEVICE_BULK_WAIT_TIMEOUT once."""
    _check(load_library().tc_selftest_wait_timeout(_stream(stream)))


def tc_plan_stats(plan: Plan) -> tc_plan_stats_t:
    st = tc_plan_stats_t()
    _check(load_library().tc_plan_stats(plan.handle, C.byref(st)))
    return st


def tc_plan_descriptors(plan: Plan, group: int = 0):
    n = C.c_size_t()
    lib = load_library()
    _check(lib.tc_plan_descriptors(plan.handle, group, None, 0, C.byref(n)))
    arr = (tc_descriptor_t * max(n.value, 1))()
    _check(lib.tc_plan_descriptors(plan.handle, group, arr, n.value, C.byref(n)))
    return [arr[i] for i in range(n.value)]
