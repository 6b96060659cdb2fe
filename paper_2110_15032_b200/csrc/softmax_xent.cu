// Class-split softmax cross entropy (Section 6.3: classifier weight S(1) => logits S(1)).
//
// The paper's plan has two reductions inside the softmax, max and sum, each done locally per
// shard first and then across shards.  Here:
//   partial kernel   one CTA per (row, shard, column chunk) streams its piece of the logits
//                    once and leaves a local max m_p, a local exp-sum s_p = sum exp(z - m_p)
//                    and the label's logit t_p (0 when the label lies elsewhere);
//   combine kernel   per row, over the pieces p (one warp per row: the pieces of a lane in
//                    ascending order, then the lanes by a butterfly):
//                    m = max_p m_p            (the P(max) -> B boxing of the local maxima)
//                    S = sum_p s_p exp(m_p-m) (the P(sum) -> B boxing, after rescaling)
//                    loss = log S + m - sum_p t_p.
// The local sums are taken relative to the local max (one pass over the logits); rescaling
// by exp(m_p - m) in the combine gives the same S as the literal max-then-sum order.
// Reductions inside a CTA use a fixed tree (thread-serial, warp butterfly, warps in order),
// so results are reproducible for a given shape.
#include <cuda_bf16.h>

#include <cfloat>
#include <cmath>

#include <mutex>

#include "bounds_check.h"
#include "sbp_internal.h"

namespace sbp {

constexpr int kThreads = 256;
constexpr int kLoadsPerThread = 4;    // vectors per thread per chunk
constexpr int kMaxChunksPerCta = 16;  // a CTA walks up to this many chunks of one row

struct XentParams {
  const char* logits[SBP_MAX_K];
  const long long* labels;
  float* part_m;   // [parts][rows]
  float* part_s;
  float* part_t;
  long long rows, classes;
  long long pitch[SBP_MAX_K];   // elements between consecutive rows of shard r's logits
  int k, nsplit;
  long long chunk;   // elements per chunk (kThreads * kLoadsPerThread * VEC)
  long long span;    // elements per CTA (chunk * chunks per CTA)
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

constexpr float kLog2e = 1.4426950408889634f;

__device__ __forceinline__ float ex2(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}

// (m, s) <- merge with (m2, s2), where s is a sum of exp(z - m).  A piece with no elements
// carries (m = -inf, s = 0) and must not produce inf - inf.
__device__ __forceinline__ void merge(float& m, float& s, float m2, float s2) {
  const float mm = fmaxf(m, m2);
  const float a = (m == -INFINITY) ? 0.f : s * ex2((m - mm) * kLog2e);
  const float b = (m2 == -INFINITY) ? 0.f : s2 * ex2((m2 - mm) * kLog2e);
  s = a + b;
  m = mm;
}

// ---- chunk policies: how one thread loads, maxes and exp-sums its kLoadsPerThread vectors

// bf16, 8 elements per 16-byte load; max on packed pairs, exp in fp32.
struct ChunkBF16x8 {
  using T = __nv_bfloat16;
  static constexpr int VEC = 8;
  uint4 raw[kLoadsPerThread];
  __device__ __forceinline__ void load(const T* z, long long n, int tid) {
#pragma unroll
    for (int u = 0; u < kLoadsPerThread; ++u) {
      const long long e0 = ((long long)u * kThreads + tid) * VEC;
      if (e0 < n && SBP_GUARD(z + e0, 16)) {
        asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];"
                     : "=r"(raw[u].x), "=r"(raw[u].y), "=r"(raw[u].z), "=r"(raw[u].w)
                     : "l"(z + e0));
      } else {
        raw[u] = make_uint4(0xFF80FF80u, 0xFF80FF80u, 0xFF80FF80u, 0xFF80FF80u);   // -inf, -inf
      }
    }
  }
  __device__ __forceinline__ float max() const {
    __nv_bfloat162 mx = *reinterpret_cast<const __nv_bfloat162*>(&raw[0].x);
#pragma unroll
    for (int u = 0; u < kLoadsPerThread; ++u) {
      const uint32_t* w = reinterpret_cast<const uint32_t*>(&raw[u]);
#pragma unroll
      for (int i = 0; i < 4; ++i) mx = __hmax2(mx, *reinterpret_cast<const __nv_bfloat162*>(&w[i]));
    }
    return fmaxf(__low2float(mx), __high2float(mx));
  }
  // sum of 2^(z*log2e + neg_m_l2e) over the thread's elements
  __device__ __forceinline__ float expsum(float neg_m_l2e) const {
    float s0 = 0.f, s1 = 0.f;
#pragma unroll
    for (int u = 0; u < kLoadsPerThread; ++u) {
      const uint32_t* w = reinterpret_cast<const uint32_t*>(&raw[u]);
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        const float lo = __uint_as_float(w[i] << 16);
        const float hi = __uint_as_float(w[i] & 0xffff0000u);
        s0 += ex2(fmaf(lo, kLog2e, neg_m_l2e));
        s1 += ex2(fmaf(hi, kLog2e, neg_m_l2e));
      }
    }
    return s0 + s1;
  }
};

// Generic policy: element type TT, V elements per load (V * sizeof(TT) is 16 or sizeof(TT)).
template <typename TT, int V>
struct ChunkGeneric {
  using T = TT;
  static constexpr int VEC = V;
  struct alignas(sizeof(TT) * V) Pack { TT e[V]; };
  Pack raw[kLoadsPerThread];
  bool ok[kLoadsPerThread];
  __device__ __forceinline__ static float f32(float v) { return v; }
  __device__ __forceinline__ static float f32(__nv_bfloat16 v) { return __bfloat162float(v); }
  __device__ __forceinline__ void load(const T* z, long long n, int tid) {
#pragma unroll
    for (int u = 0; u < kLoadsPerThread; ++u) {
      const long long e0 = ((long long)u * kThreads + tid) * VEC;
      ok[u] = e0 < n && SBP_GUARD(z + e0, sizeof(Pack));
      if (ok[u]) raw[u] = *reinterpret_cast<const Pack*>(z + e0);
    }
  }
  __device__ __forceinline__ float max() const {
    float m = -INFINITY;
#pragma unroll
    for (int u = 0; u < kLoadsPerThread; ++u)
      if (ok[u]) {
#pragma unroll
        for (int i = 0; i < VEC; ++i) m = fmaxf(m, f32(raw[u].e[i]));
      }
    return m;
  }
  __device__ __forceinline__ float expsum(float neg_m_l2e) const {
    float s = 0.f;
#pragma unroll
    for (int u = 0; u < kLoadsPerThread; ++u)
      if (ok[u]) {
#pragma unroll
        for (int i = 0; i < VEC; ++i) s += ex2(fmaf(f32(raw[u].e[i]), kLog2e, neg_m_l2e));
      }
    return s;
  }
};

// One CTA per (row, shard, column span).  Each thread keeps a running (m, s) over the chunks
// of its span -- the loads of the next chunk are issued before the current one is reduced --
// and the CTA merges the 256 pairs with a fixed tree.
template <typename Chunk>
__global__ void __launch_bounds__(kThreads) xent_partial_kernel(const __grid_constant__ XentParams p) {
  using T = typename Chunk::T;
  const long long row = blockIdx.x;
  const int split = blockIdx.y;
  const int shard = blockIdx.z;
  long long c_start, c_len;
  split_range(p.classes, p.k, shard, (int64_t*)&c_start, (int64_t*)&c_len);
  const long long c0 = (long long)split * p.span;
  long long n = c_len - c0;       // elements of this CTA's span (may be <= 0 on uneven shards)
  if (n > p.span) n = p.span;
  const int part = shard * p.nsplit + split;
  const T* z = reinterpret_cast<const T*>(p.logits[shard]) + row * p.pitch[shard] + c0;
  const int tid = threadIdx.x;
  // The kernel that combines the partials may be set up while this one runs; it waits for
  // this grid to finish before it reads anything.
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");

  float m = -INFINITY, s = 0.f;
  Chunk cur, nxt;
  if (n > 0) cur.load(z, n, tid);
  for (long long off = 0; off < n; off += p.chunk) {
    const bool more = off + p.chunk < n;
    if (more) nxt.load(z + off + p.chunk, n - off - p.chunk, tid);
    const float cm = cur.max();
    if (cm != -INFINITY) {
      const float mm = fmaxf(m, cm);
      const float neg = -mm * kLog2e;
      const float carried = (m == -INFINITY) ? 0.f : s * ex2(fmaf(m, kLog2e, neg));
      s = carried + cur.expsum(neg);
      m = mm;
    }
    if (more) cur = nxt;
  }

#pragma unroll
  for (int off = 16; off > 0; off >>= 1) {
    const float m2 = __shfl_xor_sync(0xffffffffu, m, off);
    const float s2 = __shfl_xor_sync(0xffffffffu, s, off);
    merge(m, s, m2, s2);
  }
  __shared__ float sm[kThreads / 32], ss[kThreads / 32];
  if ((tid & 31) == 0) {
    sm[tid >> 5] = m;
    ss[tid >> 5] = s;
  }
  __syncthreads();
  if (tid == 0) {
    float mm = sm[0], sv = ss[0];
#pragma unroll
    for (int w = 1; w < kThreads / 32; ++w) merge(mm, sv, sm[w], ss[w]);
    float t = 0.f;
    const long long y = (SBP_GUARD(p.labels + row, 8) ? p.labels[row] : -1) - c_start - c0;
    if (y >= 0 && y < n && SBP_GUARD(z + y, sizeof(T))) t = static_cast<float>(z[y]);
    const long long at = (long long)part * p.rows + row;
    if (SBP_GUARD(p.part_m + at, 4)) p.part_m[at] = mm;
    if (SBP_GUARD(p.part_s + at, 4)) p.part_s[at] = sv;
    if (SBP_GUARD(p.part_t + at, 4)) p.part_t[at] = t;
  }
}

// One warp per row: lane j takes the parts j, j + 32, ... in ascending order, then the lanes
// are merged by a butterfly -- a fixed tree for a given number of parts.
constexpr int kCombineThreads = 256;

__global__ void __launch_bounds__(kCombineThreads) xent_combine_kernel(const __grid_constant__ XentCombineParams p) {
  // When launched as the programmatic dependent of the kernel that writes the partials, wait
  // here until that grid has finished and its writes are visible (a no-op otherwise).
  asm volatile("griddepcontrol.wait;" ::: "memory");
  const long long row = (long long)blockIdx.x * (kCombineThreads / 32) + (threadIdx.x >> 5);
  if (row >= p.rows) return;
  const int lane = threadIdx.x & 31;
  float m = -INFINITY, S = 0.f, zy = 0.f;
  for (int q = lane; q < p.parts; q += 32) {
    const long long at = (long long)q * p.rows + row;
    if (!SBP_GUARD(p.part_m + at, 4) || !SBP_GUARD(p.part_s + at, 4) || !SBP_GUARD(p.part_t + at, 4)) continue;
    merge(m, S, p.part_m[at], p.part_s[at]);
    zy += p.part_t[at];
  }
#pragma unroll
  for (int off = 16; off > 0; off >>= 1) {
    const float m2 = __shfl_xor_sync(0xffffffffu, m, off);
    const float s2 = __shfl_xor_sync(0xffffffffu, S, off);
    zy += __shfl_xor_sync(0xffffffffu, zy, off);
    merge(m, S, m2, s2);
  }
  if (lane == 0) {
    const float loss = logf(S) + m - zy;
    for (int j = 0; j < p.n_loss; ++j)
      if (SBP_GUARD(p.loss[j] + row, 4)) p.loss[j][row] = loss;
    for (int j = 0; j < p.n_max; ++j)
      if (SBP_GUARD(p.row_max[j] + row, 4)) p.row_max[j][row] = m;
    for (int j = 0; j < p.n_sum; ++j)
      if (SBP_GUARD(p.row_sum[j] + row, 4)) p.row_sum[j][row] = S;
  }
}

// Elements of one CTA's column span, and how many spans cover the widest shard.
static void tiling_for(const sbp_tensor* logits, int vec, long long* chunk, long long* span, int* nsplit) {
  const int k = placement_k(logits);
  const long long c_max = (logits->shape[1] + k - 1) / k;
  *chunk = (long long)kThreads * kLoadsPerThread * vec;
  long long chunks = (c_max + *chunk - 1) / *chunk;
  if (chunks < 1) chunks = 1;
  const long long per_cta = chunks < kMaxChunksPerCta ? chunks : kMaxChunksPerCta;
  *span = *chunk * per_cta;
  *nsplit = (int)((chunks + per_cta - 1) / per_cta);
}

static int nsplit_for(const sbp_tensor* logits, int vec) {
  long long chunk, span;
  int ns;
  tiling_for(logits, vec, &chunk, &span, &ns);
  return ns;
}

// Elements per load: 16 bytes worth when every shard's rows are 16-byte aligned, else 1.
static int pick_vec(const sbp_tensor* logits) {
  const int k = placement_k(logits), esz = elem_size(logits->dtype);
  for (int r = 0; r < k; ++r) {
    int64_t st, ln;
    split_range(logits->shape[1], k, r, &st, &ln);
    if ((ln * esz) % 16 != 0 || (local_pitch(logits, r) * esz) % 16 != 0) return 1;
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

// ---- second-level reduction for many partials per row (used after the fused classifier
// kernel, which leaves one partial per 128 classes).  Thread (tx, ty) of a 32 x 8 CTA owns row
// 32 bx + tx and walks the parts of slice `by` with stride 8 in ascending order; the 8 lanes
// of a row are then merged in lane order.  Output: one partial per (slice, row).
struct XentReduceParams {
  const float* in_m;
  const float* in_s;
  const float* in_t;
  float* out_m;
  float* out_s;
  float* out_t;
  long long rows;
  int parts, per_slice;
};

__global__ void __launch_bounds__(256) xent_reduce_parts_kernel(const __grid_constant__ XentReduceParams p) {
  const int tx = threadIdx.x & 31, ty = threadIdx.x >> 5;
  const long long row = (long long)blockIdx.x * 32 + tx;
  const int lo = blockIdx.y * p.per_slice;
  const int hi = min(p.parts, lo + p.per_slice);
  // The partials come from the kernel just before this one in the stream; when launched as its
  // programmatic dependent, wait for it here (a no-op otherwise), and let the combine kernel
  // that follows be set up meanwhile.
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
  asm volatile("griddepcontrol.wait;" ::: "memory");
  float m = -INFINITY, s = 0.f, t = 0.f;
  if (row < p.rows) {
    // four parts (stride 8) are loaded before they are merged, in ascending order
    for (int q = lo + ty; q < hi; q += 32) {
      float pm[4], ps[4], pt[4];
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        const int qq = q + 8 * j;
        const long long at = (long long)(qq < hi ? qq : q) * p.rows + row;
        const bool in_ok = SBP_GUARD(p.in_m + at, 4) && SBP_GUARD(p.in_s + at, 4) && SBP_GUARD(p.in_t + at, 4);
        pm[j] = in_ok ? p.in_m[at] : -INFINITY;
        ps[j] = in_ok ? p.in_s[at] : 0.f;
        pt[j] = in_ok ? p.in_t[at] : 0.f;
      }
#pragma unroll
      for (int j = 0; j < 4; ++j)
        if (q + 8 * j < hi) {
          merge(m, s, pm[j], ps[j]);
          t += pt[j];
        }
    }
  }
  __shared__ float sm[8][33], ss[8][33], st[8][33];
  sm[ty][tx] = m;
  ss[ty][tx] = s;
  st[ty][tx] = t;
  __syncthreads();
  if (ty == 0 && row < p.rows) {
#pragma unroll
    for (int j = 1; j < 8; ++j) {
      merge(m, s, sm[j][tx], ss[j][tx]);
      t += st[j][tx];
    }
    const long long at = (long long)blockIdx.y * p.rows + row;
    if (SBP_GUARD(p.out_m + at, 4)) p.out_m[at] = m;
    if (SBP_GUARD(p.out_s + at, 4)) p.out_s[at] = s;
    if (SBP_GUARD(p.out_t + at, 4)) p.out_t[at] = t;
  }
}

constexpr int kMaxSlices = 64;

static int slices_for(int parts) {
  int s = parts / 256;
  return s < 1 ? 1 : (s > kMaxSlices ? kMaxSlices : s);
}

size_t xent_finish_stage_floats(long long rows) { return 3 * (size_t)kMaxSlices * (size_t)rows; }

sbp_status check_xent_outputs(const sbp_tensor* labels, const sbp_tensor* loss, const sbp_tensor* row_max,
                              const sbp_tensor* row_sum, long long rows, int k) {
  sbp_status st = check_tensor(labels, "labels", true);
  if (st != SBP_OK) return st;
  if (labels->ndim != 1 || labels->shape[0] != rows) return fail(SBP_ERR_SHAPE, "labels must be [rows]");
  if (labels->dtype != SBP_I64) return fail(SBP_ERR_DTYPE, "labels must be I64");
  if (labels->sbp[0].kind != SBP_BROADCAST) return fail(SBP_ERR_SIGNATURE, "labels must be B");
  if (placement_k(labels) != k) return fail(SBP_ERR_INVALID_ARG, "labels differ in k");
  st = check_row_vector(loss, "loss", rows, k);
  if (st != SBP_OK) return st;
  if (row_max && (st = check_row_vector(row_max, "row_max", rows, k)) != SBP_OK) return st;
  if (row_sum && (st = check_row_vector(row_sum, "row_sum", rows, k)) != SBP_OK) return st;
  return SBP_OK;
}

// parts partials per row in part_* ([parts][rows]) -> loss / row_max / row_sum.
sbp_status launch_xent_finish(float* part_m, float* part_s, float* part_t, int parts, long long rows, float* stage,
                              sbp_tensor* loss, sbp_tensor* row_max, sbp_tensor* row_sum, int k, cudaStream_t st) {
  const int slices = slices_for(parts);
  XentReduceParams r{};
  r.in_m = part_m;
  r.in_s = part_s;
  r.in_t = part_t;
  r.out_m = stage;
  r.out_s = stage + (size_t)slices * rows;
  r.out_t = stage + 2 * (size_t)slices * rows;
  r.rows = rows;
  r.parts = parts;
  r.per_slice = (parts + slices - 1) / slices;
  // Both kernels are launched as programmatic dependents of their predecessors in the stream.
  cudaLaunchAttribute pdl[1];
  pdl[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  pdl[0].val.programmaticStreamSerializationAllowed = 1;
  cudaLaunchConfig_t cfg{};
  cfg.gridDim = dim3((unsigned)((rows + 31) / 32), (unsigned)slices);
  cfg.blockDim = dim3(256);
  cfg.dynamicSmemBytes = 0;
  cfg.stream = st;
  cfg.attrs = pdl;
  cfg.numAttrs = 1;
  SBP_BOUNDS_UPLOAD(st);
  cudaError_t e = cudaLaunchKernelEx(&cfg, xent_reduce_parts_kernel, r);
  if (e != cudaSuccess) return cuda_fail(e, "softmax reduce launch");
  XentCombineParams c{};
  c.part_m = r.out_m;
  c.part_s = r.out_s;
  c.part_t = r.out_t;
  c.rows = rows;
  c.parts = slices;
  c.n_loss = dedup(c.loss, loss, k);
  c.n_max = row_max ? dedup(c.row_max, row_max, k) : 0;
  c.n_sum = row_sum ? dedup(c.row_sum, row_sum, k) : 0;
  cfg.gridDim = dim3((unsigned)((rows + kCombineThreads / 32 - 1) / (kCombineThreads / 32)));
  cfg.blockDim = dim3(kCombineThreads);
  e = cudaLaunchKernelEx(&cfg, xent_combine_kernel, c);
  if (e != cudaSuccess) return cuda_fail(e, "softmax combine launch");
  count_launch(2);
  return SBP_OK;
}

// ---- backward of the per-row loss with respect to the logits: softmax - onehot, kept S(1).
// Element-wise given the row max and row sum of the forward pass: one read and one write of
// the logits' size.
struct XentBwdParams {
  const char* logits[SBP_MAX_K];
  char* grad[SBP_MAX_K];
  const long long* labels;
  const float* row_max;
  const float* row_sum;
  long long rows, classes;
  long long lpitch[SBP_MAX_K], gpitch[SBP_MAX_K];   // elements between consecutive rows: logits, gradient
  int k;
};

template <typename T, int VEC>
__global__ void __launch_bounds__(kThreads) xent_backward_kernel(const __grid_constant__ XentBwdParams p) {
  const long long row = blockIdx.x;
  const int shard = blockIdx.z;
  long long c_start, c_len;
  split_range(p.classes, p.k, shard, (int64_t*)&c_start, (int64_t*)&c_len);
  const T* z = reinterpret_cast<const T*>(p.logits[shard]) + row * p.lpitch[shard];
  T* g = reinterpret_cast<T*>(p.grad[shard]) + row * p.gpitch[shard];
  // softmax = 2^(z log2e - m log2e - log2 S): the division by the row sum is folded into the exponent
  if (!SBP_GUARD(p.row_max + row, 4) || !SBP_GUARD(p.row_sum + row, 4) || !SBP_GUARD(p.labels + row, 8)) return;
  const float neg = -p.row_max[row] * kLog2e - log2f(p.row_sum[row]);
  const long long y = p.labels[row] - c_start;      // label's column inside this shard, if any
  struct alignas(sizeof(T) * VEC) Pack { T e[VEC]; };
  for (long long e0 = ((long long)blockIdx.y * kThreads + threadIdx.x) * VEC; e0 < c_len;
       e0 += (long long)gridDim.y * kThreads * VEC) {
    if (!SBP_GUARD(z + e0, sizeof(Pack)) || !SBP_GUARD(g + e0, sizeof(Pack))) continue;
    Pack in = *reinterpret_cast<const Pack*>(z + e0), out;
    const int y_rel = (y >= e0 && y < e0 + VEC) ? (int)(y - e0) : -1;   // the label's place in this vector, if it is here
#pragma unroll
    for (int i = 0; i < VEC; ++i) {
      float v = ex2(fmaf(static_cast<float>(in.e[i]), kLog2e, neg));
      if (i == y_rel) v -= 1.0f;
      out.e[i] = static_cast<T>(v);
    }
    *reinterpret_cast<Pack*>(g + e0) = out;
  }
}

}  // namespace sbp

using namespace sbp;

extern "C" {

size_t sbp_softmax_xent_workspace_bytes(const sbp_tensor* logits) {
  if (check_tensor(logits, "logits", false) != SBP_OK || logits->ndim != 2) return 0;
  // sized for the element-wise path as well, so the answer does not depend on pointer values
  const int k = placement_k(logits);
  const int ns = nsplit_for(logits, 1);
  const int ns_vec = nsplit_for(logits, 16 / elem_size(logits->dtype));
  const size_t parts = (size_t)k * (size_t)(ns > ns_vec ? ns : ns_vec);
  return 3 * parts * (size_t)logits->shape[0] * sizeof(float);
}

sbp_status sbp_softmax_xent(const sbp_tensor* logits, const sbp_tensor* labels, sbp_tensor* loss,
                            sbp_tensor* row_max, sbp_tensor* row_sum, void* ws, size_t ws_bytes,
                            void* cuda_stream) {
  SBP_RANGE("sbp_softmax_xent");
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
  for (int r = 0; r < k; ++r) {
    p.logits[r] = static_cast<const char*>(logits->local[r]);
    p.pitch[r] = local_pitch(logits, r);
  }
  p.labels = static_cast<const long long*>(labels->local[0]);
  p.part_m = static_cast<float*>(ws);
  p.part_s = p.part_m + (size_t)parts * rows;
  p.part_t = p.part_s + (size_t)parts * rows;
  p.rows = rows;
  p.classes = classes;
  p.k = k;
  p.nsplit = nsplit;
  {
    int ns;
    tiling_for(logits, vec, &p.chunk, &p.span, &ns);
  }

  cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
  dim3 grid((unsigned)rows, (unsigned)nsplit, (unsigned)k);
  SBP_BOUNDS_RESET();
  SBP_BOUNDS_TENSOR(logits);
  SBP_BOUNDS_TENSOR(labels);
  SBP_BOUNDS_TENSOR(loss);
  SBP_BOUNDS_TENSOR(row_max);
  SBP_BOUNDS_TENSOR(row_sum);
  SBP_BOUNDS_ADD(ws, need);
  SBP_BOUNDS_UPLOAD(stream);
  if (logits->dtype == SBP_BF16) {
    if (vec > 1) xent_partial_kernel<ChunkBF16x8><<<grid, kThreads, 0, stream>>>(p);
    else xent_partial_kernel<ChunkGeneric<__nv_bfloat16, 1>><<<grid, kThreads, 0, stream>>>(p);
  } else {
    if (vec > 1) xent_partial_kernel<ChunkGeneric<float, 4>><<<grid, kThreads, 0, stream>>>(p);
    else xent_partial_kernel<ChunkGeneric<float, 1>><<<grid, kThreads, 0, stream>>>(p);
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
  // Launched as the programmatic dependent of the partial kernel: it may be set up while that
  // kernel still runs and waits, on the device, for it to finish before reading the partials.
  cudaLaunchConfig_t cfg{};
  cfg.gridDim = dim3((unsigned)((rows + kCombineThreads / 32 - 1) / (kCombineThreads / 32)));
  cfg.blockDim = dim3(kCombineThreads);
  cfg.dynamicSmemBytes = 0;
  cfg.stream = stream;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  e = cudaLaunchKernelEx(&cfg, xent_combine_kernel, c);
  if (e != cudaSuccess) return cuda_fail(e, "softmax combine launch");
  count_launch(2);
  return SBP_OK;
}

}  // extern "C"

// ------------------------------------------------------------------ built-in scratch variant
//
// Scratch for callers that cannot hand in a workspace.  It lives in the library's image, so
// every GPU that loads the library carries these 3 MiB until the process exits.
namespace sbp {
constexpr size_t kStaticScratchBytes = SBP_SOFTMAX_XENT_STATIC_SCRATCH_BYTES;
static __device__ __align__(256) float g_xent_static_scratch[kStaticScratchBytes / sizeof(float)];
constexpr int kMaxDevices = 64;
}  // namespace sbp

extern "C" sbp_status sbp_softmax_xent_static(const sbp_tensor* logits, const sbp_tensor* labels, sbp_tensor* loss,
                                              sbp_tensor* row_max, sbp_tensor* row_sum, void* cuda_stream) {
  SBP_RANGE("sbp_softmax_xent_static");
  // Size check first, so that an oversized request is refused before anything else happens.
  sbp_status st = check_tensor(logits, "logits", true);
  if (st != SBP_OK) return st;
  if (logits->ndim != 2) return fail(SBP_ERR_SHAPE, "logits must be [rows, classes]");
  const size_t need =
      3 * (size_t)placement_k(logits) * (size_t)nsplit_for(logits, pick_vec(logits)) * (size_t)logits->shape[0] * sizeof(float);
  if (need > kStaticScratchBytes)
    return fail(SBP_ERR_WORKSPACE,
                "this shape needs %zu bytes of scratch but the built-in array holds %zu; call sbp_softmax_xent "
                "with a workspace of your own instead",
                need, kStaticScratchBytes);

  // In host code the array's name is only a handle; its device address has to be looked up,
  // once per device, while that device is current.
  static float* dev_ptr[kMaxDevices] = {};
  static std::mutex mu;
  int dev = 0;
  SBP_CUDA_TRY(cudaGetDevice(&dev));
  if (dev < 0 || dev >= kMaxDevices) return fail(SBP_ERR_UNSUPPORTED, "device ordinal %d out of range", dev);
  float* scratch = nullptr;
  {
    std::lock_guard<std::mutex> lock(mu);
    if (!dev_ptr[dev]) {
      void* ptr = nullptr;
      SBP_CUDA_TRY(cudaGetSymbolAddress(&ptr, g_xent_static_scratch));
      dev_ptr[dev] = static_cast<float*>(ptr);
    }
    scratch = dev_ptr[dev];
  }
  return sbp_softmax_xent(logits, labels, loss, row_max, row_sum, scratch, kStaticScratchBytes, cuda_stream);
}

extern "C" sbp_status sbp_softmax_xent_backward(const sbp_tensor* logits, const sbp_tensor* labels,
                                                const sbp_tensor* row_max, const sbp_tensor* row_sum,
                                                sbp_tensor* grad_logits, void* cuda_stream) {
  SBP_RANGE("sbp_softmax_xent_backward");
  sbp_status st = check_tensor(logits, "logits", true);
  if (st != SBP_OK) return st;
  st = check_tensor(grad_logits, "grad_logits", true);
  if (st != SBP_OK) return st;
  if (logits->ndim != 2 || grad_logits->ndim != 2 || logits->shape[0] != grad_logits->shape[0] ||
      logits->shape[1] != grad_logits->shape[1])
    return fail(SBP_ERR_SHAPE, "logits and grad_logits must be [rows, classes] alike");
  if (logits->dtype != SBP_BF16 && logits->dtype != SBP_F32) return fail(SBP_ERR_DTYPE, "logits must be BF16 or F32");
  if (grad_logits->dtype != logits->dtype) return fail(SBP_ERR_DTYPE, "grad_logits and logits differ in dtype");
  const int k = placement_k(logits);
  if (placement_k(grad_logits) != k) return fail(SBP_ERR_INVALID_ARG, "operands differ in k");
  auto is_s1 = [](const sbp_tensor* t) { return t->sbp[0].kind == SBP_SPLIT && t->sbp[0].axis == 1; };
  if (!is_s1(logits) || !is_s1(grad_logits)) return fail(SBP_ERR_SIGNATURE, "logits and grad_logits must be S(1)");
  const long long rows = logits->shape[0], classes = logits->shape[1];
  if (!row_max || !row_sum) return fail(SBP_ERR_INVALID_ARG, "row_max and row_sum of the forward pass are required");
  st = check_xent_outputs(labels, row_max, row_max, row_sum, rows, k);
  if (st != SBP_OK) return st;
  if (rows == 0 || classes == 0) return SBP_OK;
  if (rows > 0x7fffffffLL) return fail(SBP_ERR_UNSUPPORTED, "too many rows for one launch");

  XentBwdParams p{};
  bool vec_ok = true;
  const int esz = elem_size(logits->dtype);
  for (int r = 0; r < k; ++r) {
    int64_t s0, ln;
    split_range(classes, k, r, &s0, &ln);
    p.lpitch[r] = local_pitch(logits, r);
    p.gpitch[r] = local_pitch(grad_logits, r);
    vec_ok = vec_ok && (ln * esz) % 16 == 0 && reinterpret_cast<uintptr_t>(logits->local[r]) % 16 == 0 &&
             reinterpret_cast<uintptr_t>(grad_logits->local[r]) % 16 == 0 && (p.lpitch[r] * esz) % 16 == 0 &&
             (p.gpitch[r] * esz) % 16 == 0;
    p.logits[r] = static_cast<const char*>(logits->local[r]);
    p.grad[r] = static_cast<char*>(grad_logits->local[r]);
  }
  p.labels = static_cast<const long long*>(labels->local[0]);
  p.row_max = static_cast<const float*>(row_max->local[0]);
  p.row_sum = static_cast<const float*>(row_sum->local[0]);
  p.rows = rows;
  p.classes = classes;
  p.k = k;
  const int vec = vec_ok ? 16 / esz : 1;
  const long long c_max = (classes + k - 1) / k;
  long long gy = (c_max + (long long)kThreads * vec * 4 - 1) / ((long long)kThreads * vec * 4);   // ~4 vectors per thread
  if (gy < 1) gy = 1;
  if (gy > 65535) gy = 65535;
  dim3 grid((unsigned)rows, (unsigned)gy, (unsigned)k);
  cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
  SBP_BOUNDS_RESET();
  SBP_BOUNDS_TENSOR(logits);
  SBP_BOUNDS_TENSOR(labels);
  SBP_BOUNDS_TENSOR(row_max);
  SBP_BOUNDS_TENSOR(row_sum);
  SBP_BOUNDS_TENSOR(grad_logits);
  SBP_BOUNDS_UPLOAD(stream);
  if (logits->dtype == SBP_BF16) {
    if (vec > 1) xent_backward_kernel<__nv_bfloat16, 8><<<grid, kThreads, 0, stream>>>(p);
    else xent_backward_kernel<__nv_bfloat16, 1><<<grid, kThreads, 0, stream>>>(p);
  } else {
    if (vec > 1) xent_backward_kernel<float, 4><<<grid, kThreads, 0, stream>>>(p);
    else xent_backward_kernel<float, 1><<<grid, kThreads, 0, stream>>>(p);
  }
  cudaError_t e = cudaGetLastError();
  if (e != cudaSuccess) return cuda_fail(e, "softmax backward launch");
  count_launch();
  return SBP_OK;
}
