// Descriptor checks, the MatMul signature rule (Table 1) and error reporting.
#include <atomic>
#include <cstring>

#include "bounds_check.h"
#include "sbp_internal.h"

namespace sbp {

#ifdef SBP_DEBUG_BOUNDS
static thread_local BoundsTable g_bounds_host;
static BoundsPollFn g_bounds_polls[16];
static int g_bounds_npolls = 0;

void bounds_reset() { g_bounds_host.n = 0; }

void bounds_add(const void* p, size_t bytes) {
  if (!p || bytes == 0) return;
  BoundsTable& t = g_bounds_host;
  const unsigned long long lo = reinterpret_cast<uintptr_t>(p), hi = lo + bytes;
  for (int i = 0; i < t.n; ++i)
    if (t.lo[i] == lo && t.hi[i] >= hi) return;
  if (t.n < kBoundsMax) {
    t.lo[t.n] = lo;
    t.hi[t.n] = hi;
    ++t.n;
  }
}

void bounds_add_tensor_shard(const sbp_tensor* t, int r) {
  if (!t || !t->local[r]) return;
  int64_t shp[SBP_MAX_DIMS];
  local_shape_nd(t, r, shp);
  int64_t rows = 1;
  for (int d = 0; d + 1 < t->ndim; ++d) rows *= shp[d];
  const int64_t cols = shp[t->ndim - 1];
  if (rows == 0 || cols == 0) return;
  const int64_t elems = (rows - 1) * local_pitch(t, r) + cols;   // the last row ends where its data ends
  bounds_add(t->local[r], (size_t)elems * elem_size(t->dtype));
}

void bounds_add_tensor(const sbp_tensor* t) {
  if (!t) return;
  const int k = placement_k(t);
  for (int r = 0; r < k && r < SBP_MAX_K; ++r) bounds_add_tensor_shard(t, r);
}

const BoundsTable& bounds_current() { return g_bounds_host; }

void bounds_register_poll(BoundsPollFn fn) {
  if (g_bounds_npolls < 16) g_bounds_polls[g_bounds_npolls++] = fn;
}
#endif

static thread_local char g_err[512] = "";
static std::atomic<uint64_t> g_launches{0};

sbp_status fail(sbp_status s, const char* fmt, ...) {
  va_list ap;
  va_start(ap, fmt);
  vsnprintf(g_err, sizeof(g_err), fmt, ap);
  va_end(ap);
  return s;
}

void count_launch(uint64_t n) { g_launches.fetch_add(n, std::memory_order_relaxed); }

sbp_status cuda_fail(cudaError_t e, const char* what) {
  return fail(SBP_ERR_CUDA, "%s: %s", what, cudaGetErrorString(e));
}

static sbp_status check_common(const sbp_tensor* t, const char* name, bool need_ptrs, bool allow_2d) {
  if (!t) return fail(SBP_ERR_INVALID_ARG, "%s: null descriptor", name);
  if (t->ndim < 1 || t->ndim > SBP_MAX_DIMS)
    return fail(SBP_ERR_INVALID_ARG, "%s: ndim %d outside [1,%d]", name, t->ndim, SBP_MAX_DIMS);
  if (elem_size(t->dtype) == 0) return fail(SBP_ERR_DTYPE, "%s: unknown dtype %d", name, t->dtype);
  for (int d = 0; d < t->ndim; ++d)
    if (t->shape[d] < 0) return fail(SBP_ERR_SHAPE, "%s: negative extent on axis %d", name, d);
  if (t->pdims < 1 || t->pdims > SBP_MAX_PDIMS)
    return fail(SBP_ERR_INVALID_ARG, "%s: pdims %d outside [1,%d]", name, t->pdims, SBP_MAX_PDIMS);
  for (int p = 0; p < t->pdims; ++p)
    if (t->pshape[p] < 1) return fail(SBP_ERR_INVALID_ARG, "%s: placement extent < 1", name);
  int k = placement_k(t);
  if (k > SBP_MAX_K) return fail(SBP_ERR_INVALID_ARG, "%s: k = %d exceeds %d", name, k, SBP_MAX_K);
  if (t->pdims != 1 && !allow_2d)
    return fail(SBP_ERR_UNSUPPORTED, "%s: multi-dimensional SBP (pdims = %d) is not implemented by this entry point",
                name, t->pdims);
  for (int p = 0; p < t->pdims; ++p) {
    sbp_sig s = t->sbp[p];
    if (s.kind < SBP_SPLIT || s.kind > SBP_PARTIAL_MAX)
      return fail(SBP_ERR_SIGNATURE, "%s: unknown sbp kind %d", name, s.kind);
    if (s.kind == SBP_SPLIT && (s.axis < 0 || s.axis >= t->ndim))
      return fail(SBP_ERR_SIGNATURE, "%s: split axis %d outside [0,%d)", name, s.axis, t->ndim);
  }
  for (int r = 0; r < k; ++r) {
    if (t->local_ld[r] == 0) continue;
    int64_t shp[SBP_MAX_DIMS];
    local_shape_nd(t, r, shp);
    if (t->local_ld[r] < shp[t->ndim - 1])
      return fail(SBP_ERR_INVALID_ARG, "%s: local_ld[%d] = %lld is below the local row length %lld", name, r,
                  (long long)t->local_ld[r], (long long)shp[t->ndim - 1]);
  }
  if (need_ptrs) {
    for (int r = 0; r < k; ++r) {
      if (!t->local[r] && local_numel(t, r) > 0)
        return fail(SBP_ERR_INVALID_ARG, "%s: local[%d] is null", name, r);
      if (reinterpret_cast<uintptr_t>(t->local[r]) % elem_size(t->dtype) != 0)
        return fail(SBP_ERR_ALIGNMENT, "%s: local[%d] is not aligned to its element size", name, r);
    }
  }
  return SBP_OK;
}

sbp_status check_tensor(const sbp_tensor* t, const char* name, bool need_ptrs) {
  return check_common(t, name, need_ptrs, false);
}

sbp_status check_tensor_nd(const sbp_tensor* t, const char* name, bool need_ptrs) {
  return check_common(t, name, need_ptrs, true);
}

void local_shape_nd(const sbp_tensor* t, int r, int64_t out[SBP_MAX_DIMS]) {
  for (int d = 0; d < SBP_MAX_DIMS; ++d) out[d] = d < t->ndim ? t->shape[d] : 1;
  int idx[SBP_MAX_PDIMS] = {r, 0};
  if (t->pdims == 2) {
    idx[0] = r / t->pshape[1];
    idx[1] = r % t->pshape[1];
  }
  for (int p = 0; p < t->pdims; ++p) {
    if (t->sbp[p].kind != SBP_SPLIT) continue;
    int64_t start, len;
    split_range(out[t->sbp[p].axis], t->pshape[p], idx[p], &start, &len);
    out[t->sbp[p].axis] = len;
  }
}

int64_t local_numel(const sbp_tensor* t, int r) {
  int64_t shp[SBP_MAX_DIMS];
  local_shape_nd(t, r, shp);
  int64_t n = 1;
  for (int d = 0; d < t->ndim; ++d) n *= shp[d];
  return n;
}

int64_t local_pitch(const sbp_tensor* t, int r) {
  if (t->local_ld[r] != 0) return t->local_ld[r];
  int64_t shp[SBP_MAX_DIMS];
  local_shape_nd(t, r, shp);
  return shp[t->ndim - 1];
}

bool has_ld(const sbp_tensor* t) {
  if (t->ndim < 2) return false;           // a single row has no pitch
  const int k = placement_k(t);
  for (int r = 0; r < k; ++r) {
    if (t->local_ld[r] == 0) continue;
    int64_t shp[SBP_MAX_DIMS];
    local_shape_nd(t, r, shp);
    if (t->local_ld[r] != shp[t->ndim - 1]) return true;
  }
  return false;
}

sbp_status refuse_ld(const sbp_tensor* t, const char* name, const char* entry) {
  if (t && has_ld(t))
    return fail(SBP_ERR_UNSUPPORTED, "%s: %s takes dense local tensors only (local_ld must be 0 or the row length)", name, entry);
  return SBP_OK;
}

#ifdef SBP_DEBUG_BOUNDS
// Self-test of the debug-bounds report path: asks the checker about the byte just past a registered
// buffer.  The check fails, so the store below it is skipped: nothing outside the buffer is touched.
__global__ void bounds_selftest_kernel(unsigned char* buf, size_t bytes) {
  if (SBP_GUARD(buf, 1)) buf[0] = 1;                 // inside: performed
  if (SBP_GUARD(buf + bytes, 1)) buf[bytes] = 1;     // one past the end: refused and recorded
}
#endif

// Defined next to the kernels that own the flags.
sbp_status read_and_clear_bulk_timeout(bool* timed_out);
sbp_status read_and_clear_tc_timeout(bool* timed_out);
sbp_status launch_expire_wait(unsigned long long limit_ns, cudaStream_t st);

}  // namespace sbp

using namespace sbp;

extern "C" {

const char* sbp_status_string(sbp_status s) {
  switch (s) {
    case SBP_OK: return "SBP_OK";
    case SBP_ERR_INVALID_ARG: return "SBP_ERR_INVALID_ARG";
    case SBP_ERR_SHAPE: return "SBP_ERR_SHAPE";
    case SBP_ERR_DTYPE: return "SBP_ERR_DTYPE";
    case SBP_ERR_SIGNATURE: return "SBP_ERR_SIGNATURE";
    case SBP_ERR_UNSUPPORTED: return "SBP_ERR_UNSUPPORTED";
    case SBP_ERR_ALIGNMENT: return "SBP_ERR_ALIGNMENT";
    case SBP_ERR_WORKSPACE: return "SBP_ERR_WORKSPACE";
    case SBP_ERR_CUDA: return "SBP_ERR_CUDA";
    case SBP_ERR_TIMEOUT: return "SBP_ERR_TIMEOUT";
    case SBP_ERR_BOUNDS: return "SBP_ERR_BOUNDS";
  }
  return "SBP_ERR_?";
}

const char* sbp_last_error(void) { return g_err; }

int32_t sbp_debug_bounds_enabled(void) {
#ifdef SBP_DEBUG_BOUNDS
  return 1;
#else
  return 0;
#endif
}

uint64_t sbp_launch_count(void) { return g_launches.load(std::memory_order_relaxed); }

sbp_status sbp_check_device_errors(void) {
  bool bulk = false, tc = false;
  sbp_status st = read_and_clear_bulk_timeout(&bulk);
  if (st != SBP_OK) return st;
  st = read_and_clear_tc_timeout(&tc);
  if (st != SBP_OK) return st;
#ifdef SBP_DEBUG_BOUNDS
  if (cudaDeviceSynchronize() != cudaSuccess) return fail(SBP_ERR_CUDA, "device synchronisation failed");
  for (int i = 0; i < g_bounds_npolls; ++i) {
    unsigned long long addr = 0;
    if (g_bounds_polls[i](&addr))
      return fail(SBP_ERR_BOUNDS, "a kernel computed the address 0x%llx, which lies in none of its call's buffers; the access was skipped", addr);
  }
#endif
  if (bulk) return fail(SBP_ERR_TIMEOUT, "a bulk-copy boxing kernel gave up waiting for its loads");
  if (tc) return fail(SBP_ERR_TIMEOUT, "the tensor-core matmul kernel gave up waiting on one of its barriers");
  return SBP_OK;
}

sbp_status sbp_selftest_debug_bounds(void* buf, size_t bytes, void* cuda_stream) {
#ifdef SBP_DEBUG_BOUNDS
  if (!buf || bytes == 0) return fail(SBP_ERR_INVALID_ARG, "a device buffer of at least one byte is needed");
  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
  SBP_BOUNDS_RESET();
  SBP_BOUNDS_ADD(buf, bytes);
  SBP_BOUNDS_UPLOAD(st);
  bounds_selftest_kernel<<<1, 1, 0, st>>>(static_cast<unsigned char*>(buf), bytes);
  cudaError_t e = cudaGetLastError();
  if (e != cudaSuccess) return cuda_fail(e, "bounds self-test launch");
  count_launch();
  return SBP_OK;
#else
  (void)buf; (void)bytes; (void)cuda_stream;
  return fail(SBP_ERR_UNSUPPORTED, "this is not the debug-bounds build of the library");
#endif
}

sbp_status sbp_selftest_wait_timeout(uint32_t limit_ms, void* cuda_stream) {
  if (limit_ms == 0 || limit_ms > 1000) return fail(SBP_ERR_INVALID_ARG, "limit_ms must be in [1, 1000]");
  return launch_expire_wait((unsigned long long)limit_ms * 1000000ull, static_cast<cudaStream_t>(cuda_stream));
}

sbp_status sbp_local_shape(const sbp_tensor* t, int32_t r, int64_t out_shape[SBP_MAX_DIMS]) {
  sbp_status st = check_tensor_nd(t, "t", false);
  if (st != SBP_OK) return st;
  if (!out_shape) return fail(SBP_ERR_INVALID_ARG, "out_shape is null");
  int k = placement_k(t);
  if (r < 0 || r >= k) return fail(SBP_ERR_INVALID_ARG, "shard %d outside [0,%d)", r, k);
  local_shape_nd(t, r, out_shape);
  return SBP_OK;
}

sbp_status sbp_view_b_to_s(const sbp_tensor* b, int32_t axis, sbp_tensor* view) {
  sbp_status st = check_tensor(b, "b", true);
  if (st != SBP_OK) return st;
  if (!view) return fail(SBP_ERR_INVALID_ARG, "view is null");
  if (b->sbp[0].kind != SBP_BROADCAST) return fail(SBP_ERR_SIGNATURE, "b must be a B tensor");
  if (axis < 0 || axis >= b->ndim) return fail(SBP_ERR_INVALID_ARG, "axis %d outside [0,%d)", axis, b->ndim);
  if (axis != 0 && axis != b->ndim - 1)
    return fail(SBP_ERR_UNSUPPORTED, "a view split along an inner axis of an N-D tensor needs two strides");
  const int k = placement_k(b);
  const int esz = elem_size(b->dtype);
  sbp_tensor v = *b;
  v.sbp[0].kind = SBP_SPLIT;
  v.sbp[0].axis = axis;
  int64_t inner = 1;   // elements in one step of axis 0, in a replica
  for (int d = 1; d < b->ndim; ++d) inner *= b->shape[d];
  for (int r = 0; r < k; ++r) {
    int64_t start, len;
    split_range(b->shape[axis], k, r, &start, &len);
    const int64_t pitch = local_pitch(b, r);             // row length of the replica
    char* base = static_cast<char*>(b->local[r]);
    if (axis == b->ndim - 1) {                            // a column block: rows stay `pitch` apart
      v.local[r] = base ? base + start * esz : nullptr;
      v.local_ld[r] = b->ndim >= 2 ? pitch : 0;          // a 1-D tensor is a single row: no pitch
    } else {                                              // a block of whole rows (ndim >= 2 here)
      const int64_t rows_per_step = inner / b->shape[b->ndim - 1];
      v.local[r] = base ? base + start * rows_per_step * pitch * esz : nullptr;
      v.local_ld[r] = b->local_ld[r];
    }
    if (len == 0) v.local[r] = b->local[r];               // an empty piece: any valid pointer
  }
  *view = v;
  return SBP_OK;
}

sbp_status sbp_transfer_cost(sbp_sig src, sbp_sig dst, int32_t p1, int32_t p2, int32_t disjoint, uint64_t t_bytes,
                             uint64_t* cost_bytes) {
  if (!cost_bytes) return fail(SBP_ERR_INVALID_ARG, "cost_bytes is null");
  if (p1 < 1 || p2 < 1) return fail(SBP_ERR_INVALID_ARG, "device counts must be >= 1");
  auto valid = [](sbp_sig s) { return s.kind >= SBP_SPLIT && s.kind <= SBP_PARTIAL_MAX; };
  if (!valid(src) || !valid(dst)) return fail(SBP_ERR_SIGNATURE, "unknown sbp kind");
  const bool ss = src.kind == SBP_SPLIT, sb = src.kind == SBP_BROADCAST, sp = !ss && !sb;
  const bool ds = dst.kind == SBP_SPLIT, db = dst.kind == SBP_BROADCAST, dp = !ds && !db;
  const uint64_t T = t_bytes, P1 = (uint64_t)p1, P2 = (uint64_t)p2;
  uint64_t c = 0;
  if (!disjoint) {
    if (p1 != p2) return fail(SBP_ERR_INVALID_ARG, "the same placement has p1 == p2");
    if (ss && ds) c = src.axis == dst.axis ? 0 : (P1 - 1) * T / P1;   // all2all
    else if (ss && db) c = (P1 - 1) * T;                               // all-gather
    else if (sp && ds) c = (P1 - 1) * T;                               // reduce-scatter
    else if (sp && db) c = 2 * (P1 - 1) * T;                           // all-reduce
    else c = 0;                                                        // S->P, B->S, B->B, B->P, P->P
  } else {
    if (ss && ds) c = T;
    else if (ss && db) c = P2 * T;
    else if (ss && dp) c = T;
    else if (sb && ds) c = T;
    else if (sb && db) c = P2 * T;
    else if (sb && dp) c = T;
    else if (sp && ds) c = P1 * T;
    else if (sp && db) c = (P1 + P2 - 1) * T;
    else c = P1 * T;                                                   // P -> P
  }
  *cost_bytes = c;
  return SBP_OK;
}

sbp_status sbp_matmul_infer(sbp_sig x, sbp_sig w, sbp_sig* y) {
  if (!y) return fail(SBP_ERR_INVALID_ARG, "y is null");
  auto is_s = [](sbp_sig s, int ax) { return s.kind == SBP_SPLIT && s.axis == ax; };
  auto is_b = [](sbp_sig s) { return s.kind == SBP_BROADCAST; };
  auto is_p = [](sbp_sig s) { return s.kind == SBP_PARTIAL_SUM; };
  sbp_sig out = {SBP_BROADCAST, 0};
  if (is_s(x, 0) && is_b(w)) out = {SBP_SPLIT, 0};            // data parallelism
  else if (is_b(x) && is_s(w, 1)) out = {SBP_SPLIT, 1};       // model parallelism
  else if (is_s(x, 1) && is_s(w, 0)) out = {SBP_PARTIAL_SUM, 0};
  else if (is_p(x) && is_b(w)) out = {SBP_PARTIAL_SUM, 0};
  else if (is_b(x) && is_p(w)) out = {SBP_PARTIAL_SUM, 0};
  else if (is_b(x) && is_b(w)) out = {SBP_BROADCAST, 0};
  else
    return fail(SBP_ERR_SIGNATURE, "(kind %d axis %d) x (kind %d axis %d) is not a valid MatMul signature",
                x.kind, x.axis, w.kind, w.axis);
  *y = out;
  return SBP_OK;
}

}  // extern "C"
