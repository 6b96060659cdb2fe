// Class-split softmax cross entropy (Section 6.3: classifier weight S(1) => logits S(1)).
//
// The paper's plan has two reductions inside the softmax, max and sum, each done locally per
// shard first and then across shards.  Here:
//   partial kernel   one CTA per (row, shard, column chunk) streams its piece of the logits
//                    once and leaves a local max m_p, a local exp-sum s_p = sum exp(z - m_p)
//                    and the label's logit t_p (0 when the label lies elsewhere);
//   combine kernel   per row, over the pieces p in fixed order (shard-major):
//                    m = max_p m_p            (the P(max) -> B boxing of the local maxima)
//                    S = sum_p s_p exp(m_p-m) (the P(sum) -> B boxing, after rescaling)
//                    loss = log S + m - sum_p t_p.
// The local sums are taken relative to the local max (one pass over the logits); rescaling
// by exp(m_p - m) in the combine gives the same S as the literal max-then-sum order.
// Reductions inside a CTA use a fixed tree (thread-serial, warp butterfly, warps in order),
// so results are reproducible for a given shape.
#include <cuda_bf16.h>

#include <cfloat>

#include "sbp_internal.h"

namespace sbp {

constexpr int kThreads = 256;
constexpr int kLoadsPerThread = 8;

struct XentParams {
  const char* logits[SBP_MAX_K];
  const long long* labels;
  float* part_m;   // [parts][rows]
  float* part_s;
  float* part_t;
  long long rows, classes;
  int k, nsplit;
  long long chunk;   // elements per column chunk
};

struct XentCombineParams {
  const float* part_m;
  const float* part_s;
  const float* part_t;
  float* loss[SBP_MAX_K];
  float* row_max[SBP_MAX_K];
  float* row_sum[SBP_MAX_K];
  int n_loss, n_max, n_sum;
  long long rows;
  int parts;
};

template <typename T>
__device__ __forceinline__ float to_f32(T v);
template <>
__device__ __forceinline__ float to_f32<float>(float v) { return v; }
template <>
__device__ __forceinline__ float to_f32<__nv_bfloat16>(__nv_bfloat16 v) { return __bfloat162float(v); }

__device__ __forceinline__ void merge(float& m, float& s, float m2, float s2) {
  const float mm = fmaxf(m, m2);
  // exp(-inf - finite) = 0; a piece with no elements carries (m = -inf, s = 0).
  const float a = (m == -INFINITY) ? 0.f : s * __expf(m - mm);
  const float b = (m2 == -INFINITY) ? 0.f : s2 * __expf(m2 - mm);
  s = a + b;
  m = mm;
}

// T: element type.  VEC: elements per load (16 bytes / sizeof(T), or 1 on the unaligned path).
template <typename T, int VEC>
__global__ void __launch_bounds__(kThreads) xent_partial_kernel(const __grid_constant__ XentParams p) {
  const long long row = blockIdx.x;
  const int split = blockIdx.y;
  const int shard = blockIdx.z;
  long long c_start, c_len;
  split_range(p.classes, p.k, shard, (int64_t*)&c_start, (int64_t*)&c_len);
  const long long c0 = (long long)split * p.chunk;
  long long n = c_len - c0;
  if (n > p.chunk) n = p.chunk;
  const int part = shard * p.nsplit + split;

  const T* z = reinterpret_cast<const T*>(p.logits[shard]) + row * c_len + c0;

  struct alignas(sizeof(T) * VEC) Pack { T e[VEC]; };
  Pack raw[kLoadsPerThread];
  bool ok[kLoadsPerThread];
#pragma unroll
  for (int u = 0; u < kLoadsPerThread; ++u) {
    const long long e0 = ((long long)u * kThreads + threadIdx.x) * VEC;
    ok[u] = e0 < n;   // n is a multiple of VEC on the vector path
    if (ok[u]) raw[u] = *reinterpret_cast<const Pack*>(z + e0);
  }
  float m = -INFINITY;
#pragma unroll
  for (int u = 0; u < kLoadsPerThread; ++u)
    if (ok[u]) {
#pragma unroll
      for (int i = 0; i < VEC; ++i) m = fmaxf(m, to_f32<T>(raw[u].e[i]));
    }
  float s = 0.f;
#pragma unroll
  for (int u = 0; u < kLoadsPerThread; ++u)
    if (ok[u]) {
#pragma unroll
      for (int i = 0; i < VEC; ++i) s += __expf(to_f32<T>(raw[u].e[i]) - m);
    }

#pragma unroll
  for (int off = 16; off > 0; off >>= 1) {
    const float m2 = __shfl_xor_sync(0xffffffffu, m, off);
    const float s2 = __shfl_xor_sync(0xffffffffu, s, off);
    merge(m, s, m2, s2);
  }
  __shared__ float sm[kThreads / 32], ss[kThreads / 32];
  if ((threadIdx.x & 31) == 0) {
    sm[threadIdx.x >> 5] = m;
    ss[threadIdx.x >> 5] = s;
  }
  __syncthreads();
  if (threadIdx.x == 0) {
    float mm = sm[0], sv = ss[0];
#pragma unroll
    for (int w = 1; w < kThreads / 32; ++w) merge(mm, sv, sm[w], ss[w]);
    float t = 0.f;
    const long long y = p.labels[row] - c_start - c0;
    if (y >= 0 && y < n) t = to_f32<T>(z[y]);
    p.part_m[(long long)part * p.rows + row] = mm;
    p.part_s[(long long)part * p.rows + row] = sv;
    p.part_t[(long long)part * p.rows + row] = t;
  }
}

__global__ void __launch_bounds__(128) xent_combine_kernel(const __grid_constant__ XentCombineParams p) {
  const long long row = (long long)blockIdx.x * 128 + threadIdx.x;
  if (row >= p.rows) return;
  float m = -INFINITY;
  for (int q = 0; q < p.parts; ++q) m = fmaxf(m, p.part_m[(long long)q * p.rows + row]);
  float S = 0.f, zy = 0.f;
  for (int q = 0; q < p.parts; ++q) {
    const float mq = p.part_m[(long long)q * p.rows + row];
    if (mq != -INFINITY) S += p.part_s[(long long)q * p.rows + row] * expf(mq - m);
    zy += p.part_t[(long long)q * p.rows + row];
  }
  const float loss = logf(S) + m - zy;
  for (int j = 0; j < p.n_loss; ++j) p.loss[j][row] = loss;
  for (int j = 0; j < p.n_max; ++j) p.row_max[j][row] = m;
  for (int j = 0; j < p.n_sum; ++j) p.row_sum[j][row] = S;
}

static int nsplit_for(const sbp_tensor* logits, int vec) {
  const int k = placement_k(logits);
  const long long c_max = (logits->shape[1] + k - 1) / k;
  const long long chunk = (long long)kThreads * kLoadsPerThread * vec;
  long long ns = (c_max + chunk - 1) / chunk;
  return (int)(ns < 1 ? 1 : ns);
}

// Elements per load: 16 bytes worth when every shard's rows are 16-byte aligned, else 1.
static int pick_vec(const sbp_tensor* logits) {
  const int k = placement_k(logits), esz = elem_size(logits->dtype);
  for (int r = 0; r < k; ++r) {
    int64_t st, ln;
    split_range(logits->shape[1], k, r, &st, &ln);
    if ((ln * esz) % 16 != 0) return 1;
    if (logits->local[r] && reinterpret_cast<uintptr_t>(logits->local[r]) % 16 != 0) return 1;
  }
  return 16 / esz;
}

static int dedup(float** out, const sbp_tensor* t, int k) {
  int n = 0;
  for (int r = 0; r < k; ++r) {
    float* ptr = static_cast<float*>(t->local[r]);
    bool seen = false;
    for (int q = 0; q < n; ++q) seen = seen || out[q] == ptr;
    if (!seen) out[n++] = ptr;
  }
  return n;
}

static sbp_status check_row_vector(const sbp_tensor* t, const char* name, long long rows, int k) {
  sbp_status st = check_tensor(t, name, true);
  if (st != SBP_OK) return st;
  if (t->ndim != 1 || t->shape[0] != rows) return fail(SBP_ERR_SHAPE, "%s must be [rows]", name);
  if (t->dtype != SBP_F32) return fail(SBP_ERR_DTYPE, "%s must be F32", name);
  if (t->sbp[0].kind != SBP_BROADCAST) return fail(SBP_ERR_SIGNATURE, "%s must be B", name);
  if (placement_k(t) != k) return fail(SBP_ERR_INVALID_ARG, "%s differs in k", name);
  return SBP_OK;
}

}  // namespace sbp

using namespace sbp;

extern "C" {

size_t sbp_softmax_xent_workspace_bytes(const sbp_tensor* logits) {
  if (check_tensor(logits, "logits", false) != SBP_OK || logits->ndim != 2) return 0;
  // sized for the unaligned path as well, so the answer does not depend on pointer values
  const int k = placement_k(logits);
  const int esz = elem_size(logits->dtype);
  bool vec_ok = true;
  for (int r = 0; r < k; ++r) {
    int64_t st, ln;
    split_range(logits->shape[1], k, r, &st, &ln);
    vec_ok = vec_ok && (ln * esz) % 16 == 0;
  }
  const int ns = nsplit_for(logits, 1);
  const int ns_vec = nsplit_for(logits, 16 / esz);
  (void)vec_ok;
  const size_t parts = (size_t)k * (size_t)(ns > ns_vec ? ns : ns_vec);
  return 3 * parts * (size_t)logits->shape[0] * sizeof(float);
}

sbp_status sbp_softmax_xent(const sbp_tensor* logits, const sbp_tensor* labels, sbp_tensor* loss,
                            sbp_tensor* row_max, sbp_tensor* row_sum, void* ws, size_t ws_bytes,
                            void* cuda_stream) {
  sbp_status st = check_tensor(logits, "logits", true);
  if (st != SBP_OK) return st;
  st = check_tensor(labels, "labels", true);
  if (st != SBP_OK) return st;
  if (logits->ndim != 2) return fail(SBP_ERR_SHAPE, "logits must be [rows, classes]");
  if (logits->dtype != SBP_BF16 && logits->dtype != SBP_F32) return fail(SBP_ERR_DTYPE, "logits must be BF16 or F32");
  if (!(logits->sbp[0].kind == SBP_SPLIT && logits->sbp[0].axis == 1))
    return fail(SBP_ERR_SIGNATURE, "logits must be S(1)");
  const int k = placement_k(logits);
  const long long rows = logits->shape[0], classes = logits->shape[1];
  if (labels->ndim != 1 || labels->shape[0] != rows) return fail(SBP_ERR_SHAPE, "labels must be [rows]");
  if (labels->dtype != SBP_I64) return fail(SBP_ERR_DTYPE, "labels must be I64");
  if (labels->sbp[0].kind != SBP_BROADCAST) return fail(SBP_ERR_SIGNATURE, "labels must be B");
  if (placement_k(labels) != k) return fail(SBP_ERR_INVALID_ARG, "labels differ in k");
  st = check_row_vector(loss, "loss", rows, k);
  if (st != SBP_OK) return st;
  if (row_max && (st = check_row_vector(row_max, "row_max", rows, k)) != SBP_OK) return st;
  if (row_sum && (st = check_row_vector(row_sum, "row_sum", rows, k)) != SBP_OK) return st;
  if (classes < 1) return fail(SBP_ERR_SHAPE, "softmax over zero classes");
  if (rows == 0) return SBP_OK;

  const int vec = pick_vec(logits);
  const int nsplit = nsplit_for(logits, vec);
  const int parts = k * nsplit;
  const size_t need = 3 * (size_t)parts * rows * sizeof(float);
  if (!ws || ws_bytes < need) return fail(SBP_ERR_WORKSPACE, "workspace of %zu bytes needed, %zu given", need, ws_bytes);
  if (reinterpret_cast<uintptr_t>(ws) % 4 != 0) return fail(SBP_ERR_ALIGNMENT, "workspace must be 4-byte aligned");
  if (rows > 0x7fffffffLL || nsplit > 65535) return fail(SBP_ERR_UNSUPPORTED, "shape too large for one launch");

  XentParams p{};
  for (int r = 0; r < k; ++r) p.logits[r] = static_cast<const char*>(logits->local[r]);
  p.labels = static_cast<const long long*>(labels->local[0]);
  p.part_m = static_cast<float*>(ws);
  p.part_s = p.part_m + (size_t)parts * rows;
  p.part_t = p.part_s + (size_t)parts * rows;
  p.rows = rows;
  p.classes = classes;
  p.k = k;
  p.nsplit = nsplit;
  p.chunk = (long long)kThreads * kLoadsPerThread * vec;

  cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
  dim3 grid((unsigned)rows, (unsigned)nsplit, (unsigned)k);
  if (logits->dtype == SBP_BF16) {
    if (vec > 1) xent_partial_kernel<__nv_bfloat16, 8><<<grid, kThreads, 0, stream>>>(p);
    else xent_partial_kernel<__nv_bfloat16, 1><<<grid, kThreads, 0, stream>>>(p);
  } else {
    if (vec > 1) xent_partial_kernel<float, 4><<<grid, kThreads, 0, stream>>>(p);
    else xent_partial_kernel<float, 1><<<grid, kThreads, 0, stream>>>(p);
  }
  cudaError_t e = cudaGetLastError();
  if (e != cudaSuccess) return cuda_fail(e, "softmax partial launch");

  XentCombineParams c{};
  c.part_m = p.part_m;
  c.part_s = p.part_s;
  c.part_t = p.part_t;
  c.rows = rows;
  c.parts = parts;
  c.n_loss = dedup(c.loss, loss, k);
  c.n_max = row_max ? dedup(c.row_max, row_max, k) : 0;
  c.n_sum = row_sum ? dedup(c.row_sum, row_sum, k) : 0;
  xent_combine_kernel<<<(unsigned)((rows + 127) / 128), 128, 0, stream>>>(c);
  e = cudaGetLastError();
  if (e != cudaSuccess) return cuda_fail(e, "softmax combine launch");
  count_launch(2);
  return SBP_OK;
}

}  // extern "C"
