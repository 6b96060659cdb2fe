// Debug-bounds build of the library (compiled with -DSBP_DEBUG_BOUNDS into a library of its own).
//
// Every global-memory access of the library's kernels is preceded by SBP_GUARD(address, bytes).  In
// the normal build the macro is the constant `true` and leaves no trace in the code.  In the
// debug-bounds build it compares the address range with the list of buffers the host registered
// for the call -- every local tensor of every descriptor, sized from the shapes the host computed,
// and the workspace -- and, when the range lies in none of them, records the address in a device
// flag and makes the kernel SKIP the access.  Nothing traps and no out-of-range address is ever
// dereferenced, so the device stays usable; sbp_check_device_errors() reports SBP_ERR_BOUNDS.
// Accesses made by the copy engine are not covered: the tiled copies of the tensor-core kernel are
// clipped by the hardware to the extents of their descriptors (built from the same host-computed
// shapes), and the bulk-copy boxing engine is simply not selected in the debug-bounds build.
#pragma once

#include <cuda_runtime.h>

#include <cstddef>

#include "sbp.h"

namespace sbp {

constexpr int kBoundsMax = 160;   // ranges per call: up to 9 descriptors of 16 local tensors, plus scratch

struct BoundsTable {
  unsigned long long lo[kBoundsMax], hi[kBoundsMax];
  int n;
};

#ifdef SBP_DEBUG_BOUNDS

// Host side, shared by all translation units (defined in sbp_api.cu): the ranges of the call being set up.
void bounds_reset();
void bounds_add(const void* p, size_t bytes);
void bounds_add_tensor(const sbp_tensor* t);                 // every local tensor, by its shape and pitch
void bounds_add_tensor_shard(const sbp_tensor* t, int r);    // one local tensor
const BoundsTable& bounds_current();
typedef bool (*BoundsPollFn)(unsigned long long* addr);      // reads and clears one translation unit's flag
void bounds_register_poll(BoundsPollFn fn);

// Device side, one copy per translation unit (device symbols are not shared between them).
namespace {
__device__ BoundsTable tu_bounds;
__device__ int tu_bounds_bad = 0;
__device__ unsigned long long tu_bounds_addr = 0;

__device__ __forceinline__ bool bounds_ok(const void* p, size_t bytes) {
  const unsigned long long a = reinterpret_cast<unsigned long long>(p);
  for (int i = 0; i < tu_bounds.n; ++i)
    if (a >= tu_bounds.lo[i] && a + bytes <= tu_bounds.hi[i]) return true;
  if (atomicExch(&tu_bounds_bad, 1) == 0) tu_bounds_addr = a;
  return false;
}

inline cudaError_t bounds_upload(cudaStream_t st) {
  const BoundsTable& t = bounds_current();
  return cudaMemcpyToSymbolAsync(tu_bounds, &t, sizeof(BoundsTable), 0, cudaMemcpyHostToDevice, st);
}

inline bool bounds_poll(unsigned long long* addr) {
  int bad = 0, zero = 0;
  if (cudaMemcpyFromSymbol(&bad, tu_bounds_bad, sizeof(int)) != cudaSuccess) return false;
  if (!bad) return false;
  cudaMemcpyFromSymbol(addr, tu_bounds_addr, sizeof(unsigned long long));
  cudaMemcpyToSymbol(tu_bounds_bad, &zero, sizeof(int));
  return true;
}

struct BoundsRegistrar {
  BoundsRegistrar() { bounds_register_poll(&bounds_poll); }
};
static BoundsRegistrar tu_bounds_registrar;
}  // namespace

#define SBP_GUARD(ptr, bytes) (::sbp::bounds_ok((const void*)(ptr), (size_t)(bytes)))
#define SBP_BOUNDS_UPLOAD(stream) ((void)::sbp::bounds_upload(stream))
#define SBP_BOUNDS_RESET() ::sbp::bounds_reset()
#define SBP_BOUNDS_ADD(ptr, bytes) ::sbp::bounds_add((ptr), (bytes))
#define SBP_BOUNDS_TENSOR(t) ::sbp::bounds_add_tensor(t)
#define SBP_BOUNDS_SHARD(t, r) ::sbp::bounds_add_tensor_shard((t), (r))

#else

#define SBP_GUARD(ptr, bytes) (true)
#define SBP_BOUNDS_UPLOAD(stream) ((void)0)
#define SBP_BOUNDS_RESET() ((void)0)
#define SBP_BOUNDS_ADD(ptr, bytes) ((void)0)
#define SBP_BOUNDS_TENSOR(t) ((void)0)
#define SBP_BOUNDS_SHARD(t, r) ((void)0)

#endif

}  // namespace sbp
