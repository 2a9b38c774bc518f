// Internal interfaces between the library's translation units (not part of the public ABI):
//   launch.cu   picks the executor build and launches it
//   staging.cu  staged host path and file streaming (rings, reader threads)
//   exec.cu     plan lifecycle, argument checks and the extern "C" entry points
//   noalloc.cu  tc_kv_pack_noalloc
#pragma once

#include <cuda_runtime.h>

#include "plan.h"

namespace tc {

constexpr int kMaxDevices = 64;

// Three builds of the executor, chosen per group on the host, so that the common cases do not
// pay registers for the rare ones:
//   kModeRun   every tile is one 16-byte-aligned contiguous run (same-layout KV blocks, whole
//              tensors, dim-0 slabs): no row decoding
//   kModeRows  every access is 16-byte aligned, tiles hold strided rows (layout transforms,
//              dim-1 slices)
//   kModeAny   some descriptor or base pointer is less aligned: width picked per tile
enum { kModeRun = 0, kModeRows = 1, kModeAny = 2 };

int cuda_fail(cudaError_t e, const char *what);

// ---- launch.cu
// Which executor build a group needs, given the alignment shared by the call's base pointers.
int mode_for(const tc_plan *plan, const Group &g, uint32_t ptr_align, bool checksums = false);
// CTAs of each build that one SM holds, for a pointer table of n_ptrs slots (cached).
void resident_ctas_for(size_t n_ptrs, int out[3]);
// over_host_link: which side of a call has pinned host memory in its table (kHostSrc | kHostDst)
enum : int { kHostSrc = 1, kHostDst = 2 };
uint32_t grid_for(const tc_plan *plan, const Group &g, int mode, const Segment *win = nullptr, int over_host_link = 0);
// Launch group g (or the window / tile range `win` of it) on stream s.  sums: checksum
// accumulators or null.
int launch_any(const tc_plan *plan, const Group &g, const void *const *src, void *const *dst, uint32_t ptr_align, cudaStream_t s, const Segment *win,
               unsigned long long *sums = nullptr, int over_host_link = 0);

// The current device's sticky status word (flags set by kernels); reading clears it.
int read_device_status(unsigned int *out);

// TC_PLAN_DEBUG_BOUNDS: check group g's uploaded descriptors against its slot extents less
// `shrink` bytes; a violation sets the out-of-bounds flag of the device status word.
int launch_bounds_check(const Group &g, int64_t shrink, cudaStream_t s);

// Launch the self-test of the bounded wait (see tc_selftest_wait_timeout).
int launch_wait_timeout_probe(cudaStream_t s);

// ---- staging.cu
// Take / drop a reference on the device's staging rings (allocated on first use); *bytes
// receives the device memory the rings hold.
int stage_acquire(int device, int64_t *bytes);
void stage_release(int device);
// Free the rings of every device on which no staged plan is left.
void stage_trim();
int execute_staged(const tc_plan *plan, const Group &g, const void *const *src, void *const *dst, uint32_t ptr_align, cudaStream_t s,
                   unsigned long long *sums = nullptr);
int execute_streamed(const tc_plan *plan, const Group &g, int fd, int64_t file_off, void *const *dst, uint32_t ptr_align, cudaStream_t s,
                     unsigned long long *sums);

// ---- exec.cu
struct FileSource {
    int fd;
    int64_t offset;
};
// Checks shared by every execute entry point, then the launch (direct, staged or streamed).
int execute(const tc_plan *plan, int gi, const void *const *src, size_t n_src, void *const *dst, size_t n_dst, void *stream,
            unsigned long long *sums = nullptr, const FileSource *file = nullptr);

}  // namespace tc
