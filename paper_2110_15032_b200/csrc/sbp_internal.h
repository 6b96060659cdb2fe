// Internal helpers shared by the library's translation units (host side only).
#pragma once

#include <cuda_runtime.h>
#include <nvtx3/nvToolsExt.h>

#include <cstdarg>
#include <cstdint>
#include <cstdio>

#include "sbp.h"

namespace sbp {

// A named range around an entry point for tools that show NVTX ranges on a timeline (the header-only
// NVTX costs a null-pointer test per call when no tool is attached).
struct NvtxRange {
  explicit NvtxRange(const char* name) { nvtxRangePushA(name); }
  ~NvtxRange() { nvtxRangePop(); }
  NvtxRange(const NvtxRange&) = delete;
  NvtxRange& operator=(const NvtxRange&) = delete;
};
#define SBP_RANGE(name) ::sbp::NvtxRange sbp_range_guard_(name)

// Records the detail string returned by sbp_last_error() and passes the status through.
sbp_status fail(sbp_status s, const char* fmt, ...);
void count_launch(uint64_t n = 1);

inline int elem_size(int32_t dtype) {
  switch (dtype) {
    case SBP_F32: return 4;
    case SBP_BF16: return 2;
    case SBP_I64: return 8;
    default: return 0;
  }
}

// Balanced split (Section 3.1): start and length of shard r's piece of an axis of length n.
__host__ __device__ inline void split_range(int64_t n, int k, int r, int64_t* start, int64_t* len) {
  int64_t base = n / k, rem = n % k;
  *len = base + (r < rem ? 1 : 0);
  *start = r * base + (r < rem ? r : rem);
}

inline int placement_k(const sbp_tensor* t) {
  int k = 1;
  for (int p = 0; p < t->pdims; ++p) k *= t->pshape[p];
  return k;
}

inline bool same_sig(sbp_sig a, sbp_sig b) {
  return a.kind == b.kind && (a.kind != SBP_SPLIT || a.axis == b.axis);
}

// Local shape of device r under a 1-D or 2-D (hierarchical) placement: the signature of
// placement axis 0 is applied across the pshape[0] groups, then that of axis 1 inside a group;
// device r = i * pshape[1] + j.  out has SBP_MAX_DIMS entries (1 beyond ndim).
void local_shape_nd(const sbp_tensor* t, int r, int64_t out[SBP_MAX_DIMS]);

// Same checks as check_tensor but also accepts a two-axis placement (Section 3.3).
sbp_status check_tensor_nd(const sbp_tensor* t, const char* name, bool need_ptrs);

// Full validation of a descriptor (rank, dtype, placement, signature, pointers).
// need_ptrs: every local[r], r < k, must be non-null and aligned to the element size.
sbp_status check_tensor(const sbp_tensor* t, const char* name, bool need_ptrs);

inline int64_t numel(const sbp_tensor* t) {
  int64_t n = 1;
  for (int d = 0; d < t->ndim; ++d) n *= t->shape[d];
  return n;
}

// Elements of shard r's local tensor.
int64_t local_numel(const sbp_tensor* t, int r);

// Row pitch of shard r's local tensor in elements: local_ld[r], or its last local extent when dense.
int64_t local_pitch(const sbp_tensor* t, int r);

// True when some local tensor of t has a leading dimension other than its row length.
bool has_ld(const sbp_tensor* t);

// SBP_ERR_UNSUPPORTED (with the entry point's name in the message) when t is not dense.
sbp_status refuse_ld(const sbp_tensor* t, const char* name, const char* entry);

sbp_status cuda_fail(cudaError_t e, const char* what);

// Launch of `kernel` as a programmatic dependent of the kernel before it in the stream: if that
// kernel releases its dependents early (SBP_PDL_RELEASE), this one's CTAs may be set up while its
// last CTAs still run.  Such a kernel must execute SBP_PDL_WAIT before its first access to
// global memory; after any other kind of work the launch behaves like a plain one.
// Invariant the dependents rely on: several of them read their sources through the non-coherent
// path (ld.global.nc / __ldg), which is only sound for data that no thread of the SAME grid writes
// and that is complete before the grid's first read.  Both hold because every read comes after
// SBP_PDL_WAIT (the producer grid has finished and its writes are visible) and because no kernel
// of this library that releases its dependents early reads the buffers it writes.  A kernel that
// reads and then writes one buffer must use plain loads.  tests/test_boxing_gpu.py
// (test_ping_pong_between_two_buffers_without_a_host_sync) rewrites a source between two reads of
// it with no synchronisation in between.
template <typename... KArgs, typename... Args>
inline cudaError_t launch_dependent(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t st,
                                    Args&&... args) {
  cudaLaunchConfig_t cfg{};
  cfg.gridDim = grid;
  cfg.blockDim = block;
  cfg.dynamicSmemBytes = smem;
  cfg.stream = st;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  return cudaLaunchKernelEx(&cfg, kernel, static_cast<KArgs>(args)...);
}
#define SBP_PDL_RELEASE() asm volatile("griddepcontrol.launch_dependents;" ::: "memory")
#define SBP_PDL_WAIT() asm volatile("griddepcontrol.wait;" ::: "memory")

#define SBP_CUDA_TRY(expr)                                   \
  do {                                                       \
    cudaError_t _e = (expr);                                 \
    if (_e != cudaSuccess) return ::sbp::cuda_fail(_e, #expr); \
  } while (0)

}  // namespace sbp
