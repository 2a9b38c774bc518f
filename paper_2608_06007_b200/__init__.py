"""B200-native descriptor-driven batched tensor movement (KV pack / unpack / migrate and weight
materialisation) behind the C ABI of include/tensorcast.h.  This package is the thin Python
binding of that library; every byte is moved by its CUDA kernels."""
from .binding import (  # noqa: F401
    TC_ERR_BOUNDS, TC_ERR_CUDA, TC_ERR_DEADLINE, TC_ERR_INVALID_ARG, TC_ERR_KIND, TC_ERR_OOM,
    TC_ERR_OVERLAP, TC_ERR_SHAPE, TC_ERR_TOO_LARGE, TC_ERR_IO, TC_PLAN_STREAM, TC_PLAN_OFFLOAD_ZERO_COPY, TC_PLAN_TRACE, tc_weights_materialize_file, tc_plan_segments, TC_NOALLOC_SCRATCH_BYTES, tc_kv_pack_noalloc, TC_HND, TC_KV_MIGRATE, TC_KV_MIXED, TC_KV_PACK, TC_KV_UNPACK,
    TC_MAX_TABLE_SLOTS, TC_NHD, TC_OK, TC_REQUEST_MAJOR, TC_LAYER_MAJOR, TC_PLAN_HOST_ONLY, TC_PLAN_STAGED, TC_PLAN_CHECKSUM, TC_PLAN_SAME_POOL, tc_weights_materialize_checksum, tc_trim, TC_WEIGHTS, EXPORTS, Plan,
    TensorCastError, kv_spec, load_library, pool, tc_kv_pack, tc_kv_unpack, tc_plan_create,
    tc_plan_descriptors, tc_plan_destroy, tc_plan_stats, tc_device_status, tc_selftest_wait_timeout, tc_plan_check_device, TC_PLAN_DEBUG_BOUNDS, TC_DEVICE_OUT_OF_BOUNDS, TC_DEVICE_BULK_WAIT_TIMEOUT, tc_weights_materialize, weights_spec,
)
from .build import build_library  # noqa: F401
