// MatMul under the SBP signatures of Table 1: signature rule -> grouped-GEMM plan -> kernel.
//
// Two kernels execute a plan:
//   * the tensor-core kernel (matmul_tc.cu): bf16 operands, fp32 accumulation in tensor
//     memory, TMA-fed tiles; taken whenever the shapes meet its alignment rules;
//   * the FMA kernel in this file: fp32 operands (and bf16 operands whose shapes the tensor
//     core kernel cannot take), fp32 accumulation with fused multiply-adds, k ascending.
#include <cuda_bf16.h>

#include "bounds_check.h"
#include "matmul_plan.h"
#include "sbp_internal.h"

namespace sbp {

// Defined in matmul_tc.cu.  Returns SBP_ERR_UNSUPPORTED (without touching the error text)
// when the plan does not meet the tensor-core kernel's rules; the caller then falls back
// to the FMA kernel.
sbp_status launch_matmul_tc(const MatmulPlan& plan, const XentFusion* xf, cudaStream_t st, bool* taken);
// Defined in softmax_xent.cu: reduces the per-chunk partials left by the fused classifier kernel.
sbp_status launch_xent_finish(float* part_m, float* part_s, float* part_t, int parts, long long rows, float* stage,
                              sbp_tensor* loss, sbp_tensor* row_max, sbp_tensor* row_sum, int k, cudaStream_t st);
sbp_status check_xent_outputs(const sbp_tensor* labels, const sbp_tensor* loss, const sbp_tensor* row_max,
                              const sbp_tensor* row_sum, long long rows, int k);
size_t xent_finish_stage_floats(long long rows);
size_t matmul_tc_workspace_bytes(const MatmulPlan& plan);
void tensor_map_cache_stats(unsigned long long* hits, unsigned long long* encodes);
void tc_form_stats(unsigned long long out[3]);
void tc_set_form(int form, int max_pairs);
int tc_route(long long tiles_sq, long long tiles_tall, long long kb, int pairs, bool gelu, int n_rep, bool out_f32, int forced,
             long long* tall_tiles);

__device__ __forceinline__ float gelu_erf(float v) { return 0.5f * v * (1.0f + erff(v * 0.70710678118654752440f)); }

template <typename T>
__device__ __forceinline__ float ld_f32(const T* p);
template <>
__device__ __forceinline__ float ld_f32<float>(const float* p) { return *p; }
template <>
__device__ __forceinline__ float ld_f32<__nv_bfloat16>(const __nv_bfloat16* p) { return __bfloat162float(*p); }

template <typename T>
__device__ __forceinline__ void st_out(T* p, float v);
template <>
__device__ __forceinline__ void st_out<float>(float* p, float v) { *p = v; }
template <>
__device__ __forceinline__ void st_out<__nv_bfloat16>(__nv_bfloat16* p, float v) { *p = __float2bfloat16_rn(v); }

constexpr int BM = 64, BN = 64, BK = 16;

template <typename TI, typename TO>
__global__ void __launch_bounds__(256) matmul_fma_kernel(const __grid_constant__ MatmulPlan p) {
  const int g = blockIdx.z;
  const long long M = p.m[g], N = p.n[g];
  const long long m0 = (long long)blockIdx.y * BM, n0 = (long long)blockIdx.x * BN;
  if (m0 >= M || n0 >= N) return;
  __shared__ float As[BK][BM + 1];
  __shared__ float Bs[BK][BN + 1];
  const int tx = threadIdx.x & 15, ty = threadIdx.x >> 4;
  float acc[4][4];
#pragma unroll
  for (int i = 0; i < 4; ++i)
#pragma unroll
    for (int j = 0; j < 4; ++j) acc[i][j] = 0.f;

  const int s_lo = p.chain ? 0 : g, s_hi = p.chain ? p.nseg : g + 1;
  for (int s = s_lo; s < s_hi; ++s) {
    // element (row, kk) of the A tile and (kk, col) of the B tile, whichever way they are stored
    const TI* A = static_cast<const TI*>(p.a[s]) + (p.a_trans ? p.row_off[g] + m0 : (p.row_off[g] + m0) * p.lda[s]);
    const TI* Bm = static_cast<const TI*>(p.b[s]) + (p.b_trans ? (p.col_off[g] + n0) * p.ldb[s] : p.col_off[g] + n0);
    const long long a_rs = p.a_trans ? 1 : p.lda[s], a_ks = p.a_trans ? p.lda[s] : 1;
    const long long b_ks = p.b_trans ? 1 : p.ldb[s], b_cs = p.b_trans ? p.ldb[s] : 1;
    const long long K = p.kseg[s];
    for (long long k0 = 0; k0 < K; k0 += BK) {
      if (p.a_trans) {
        for (int e = threadIdx.x; e < BM * BK; e += 256) {
          const int c = e / BM, r = e % BM;   // consecutive threads walk the stored rows
          As[c][r] = (m0 + r < M && k0 + c < K && SBP_GUARD(A + r * a_rs + (k0 + c) * a_ks, sizeof(TI))) ? ld_f32<TI>(A + r * a_rs + (k0 + c) * a_ks) : 0.f;
        }
      } else {
        for (int e = threadIdx.x; e < BM * BK; e += 256) {
          const int r = e / BK, c = e % BK;
          As[c][r] = (m0 + r < M && k0 + c < K && SBP_GUARD(A + r * a_rs + (k0 + c) * a_ks, sizeof(TI))) ? ld_f32<TI>(A + r * a_rs + (k0 + c) * a_ks) : 0.f;
        }
      }
      if (p.b_trans) {
        for (int e = threadIdx.x; e < BK * BN; e += 256) {
          const int c = e / BK, r = e % BK;
          Bs[r][c] = (k0 + r < K && n0 + c < N && SBP_GUARD(Bm + (k0 + r) * b_ks + c * b_cs, sizeof(TI))) ? ld_f32<TI>(Bm + (k0 + r) * b_ks + c * b_cs) : 0.f;
        }
      } else {
        for (int e = threadIdx.x; e < BK * BN; e += 256) {
          const int r = e / BN, c = e % BN;
          Bs[r][c] = (k0 + r < K && n0 + c < N && SBP_GUARD(Bm + (k0 + r) * b_ks + c * b_cs, sizeof(TI))) ? ld_f32<TI>(Bm + (k0 + r) * b_ks + c * b_cs) : 0.f;
        }
      }
      __syncthreads();
#pragma unroll
      for (int kk = 0; kk < BK; ++kk) {
        float a[4], b[4];
#pragma unroll
        for (int i = 0; i < 4; ++i) a[i] = As[kk][ty * 4 + i];
#pragma unroll
        for (int j = 0; j < 4; ++j) b[j] = Bs[kk][tx * 4 + j];
#pragma unroll
        for (int i = 0; i < 4; ++i)
#pragma unroll
          for (int j = 0; j < 4; ++j) acc[i][j] = fmaf(a[i], b[j], acc[i][j]);
      }
      __syncthreads();
    }
  }
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    const long long r = m0 + ty * 4 + i;
    if (r >= M) continue;
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      const long long c = n0 + tx * 4 + j;
      if (c >= N) continue;
      float v = acc[i][j];
      if (p.gelu) v = gelu_erf(v);
      if (SBP_GUARD(static_cast<TO*>(p.y[g]) + r * p.ldy[g] + c, sizeof(TO))) st_out<TO>(static_cast<TO*>(p.y[g]) + r * p.ldy[g] + c, v);
      if (g == 0)
        for (int q = 0; q < p.n_rep; ++q)
          if (SBP_GUARD(static_cast<TO*>(p.y_rep[q]) + r * p.ldy[g] + c, sizeof(TO))) st_out<TO>(static_cast<TO*>(p.y_rep[q]) + r * p.ldy[g] + c, v);
    }
  }
}

static sbp_status launch_fma(const MatmulPlan& p, cudaStream_t st) {
  long long mmax = 0, nmax = 0;
  for (int g = 0; g < p.ngroups; ++g) {
    mmax = p.m[g] > mmax ? p.m[g] : mmax;
    nmax = p.n[g] > nmax ? p.n[g] : nmax;
  }
  if (mmax == 0 || nmax == 0) return SBP_OK;
  const long long gx = (nmax + BN - 1) / BN, gy = (mmax + BM - 1) / BM;
  if (gx > 0x7fffffffLL || gy > 65535) return fail(SBP_ERR_UNSUPPORTED, "matrix too large for the FMA kernel");
  dim3 grid((unsigned)gx, (unsigned)gy, (unsigned)p.ngroups);
  SBP_BOUNDS_UPLOAD(st);
  if (p.in_dtype == SBP_F32 && p.out_dtype == SBP_F32)
    matmul_fma_kernel<float, float><<<grid, 256, 0, st>>>(p);
  else if (p.in_dtype == SBP_BF16 && p.out_dtype == SBP_BF16)
    matmul_fma_kernel<__nv_bfloat16, __nv_bfloat16><<<grid, 256, 0, st>>>(p);
  else if (p.in_dtype == SBP_BF16 && p.out_dtype == SBP_F32)
    matmul_fma_kernel<__nv_bfloat16, float><<<grid, 256, 0, st>>>(p);
  else
    return fail(SBP_ERR_DTYPE, "F32 operands need an F32 result");
  cudaError_t e = cudaGetLastError();
  if (e != cudaSuccess) return cuda_fail(e, "matmul launch");
  count_launch();
  return SBP_OK;
}

// ------------------------------------------------------------------ operands the copy engine cannot address
//
// The tensor-core kernel reads its operands through tiled bulk copies, which need a 16-byte aligned
// base, a row pitch that is a multiple of 16 bytes and, for the operand whose contiguous index is M
// or N, a start column that is a multiple of 8 elements.  A bf16 operand that breaks one of these
// rules (a shard width of 333, an odd column offset of a fused S(1) result) is first copied into
// the caller's workspace in a layout that keeps them: rows padded to a multiple of 8 elements,
// every output group's column block starting on a multiple of 8.  The product then runs on the
// tensor cores from the copy instead of falling to the FMA kernel (two orders of magnitude slower
// at large sizes); the copy costs one read and one write of the operand.

struct PackBlock {
  const unsigned short* src;
  unsigned short* dst;
  long long rows, cols, src_ld, dst_ld;
};
constexpr int kPackBlocks = 64;
struct PackList {
  PackBlock b[kPackBlocks];
};

// One 16-byte store per thread and step: eight consecutive elements of a row, zeros past its end.
__global__ void __launch_bounds__(256) matmul_pack_kernel(const __grid_constant__ PackList L) {
  const PackBlock& B = L.b[blockIdx.y];
  const long long groups = (B.cols + 7) / 8;
  const long long total = B.rows * groups;
  for (long long i = (long long)blockIdx.x * 256 + threadIdx.x; i < total; i += (long long)gridDim.x * 256) {
    const long long row = i / groups, g8 = i - row * groups;
    const unsigned short* sp = B.src + row * B.src_ld + g8 * 8;
    unsigned short v[8];
#pragma unroll
    for (int e = 0; e < 8; ++e) v[e] = (g8 * 8 + e < B.cols && SBP_GUARD(sp + e, 2)) ? __ldg(sp + e) : (unsigned short)0;
    uint4 o;
    o.x = v[0] | ((unsigned)v[1] << 16);
    o.y = v[2] | ((unsigned)v[3] << 16);
    o.z = v[4] | ((unsigned)v[5] << 16);
    o.w = v[6] | ((unsigned)v[7] << 16);
    if (SBP_GUARD(B.dst + row * B.dst_ld + g8 * 8, 16)) *reinterpret_cast<uint4*>(B.dst + row * B.dst_ld + g8 * 8) = o;
  }
}

static long long pad8(long long v) { return (v + 7) / 8 * 8; }
static size_t align256(size_t v) { return (v + 255) & ~size_t(255); }
static bool aligned16p(const void* p) { return reinterpret_cast<uintptr_t>(p) % 16 == 0; }

// What has to be repacked for the tensor-core kernel to take a bf16 plan, and how large the copies are.
struct PackNeed {
  bool a, b;              // operand x / w needs a packed copy
  bool a_blocked, b_blocked;   // its M / N index is cut into one block per output group
  size_t bytes;
};

static PackNeed pack_need(const MatmulPlan& p, bool with_ptrs) {
  PackNeed n{};
  if (p.in_dtype != SBP_BF16) return n;
  for (int s = 0; s < p.nseg; ++s) {
    const bool used = p.chain || s < p.ngroups;
    if (!used || p.kseg[s] == 0) continue;
    if (p.lda[s] % 8 != 0 || (with_ptrs && !aligned16p(p.a[s]))) n.a = true;
    if (p.ldb[s] % 8 != 0 || (with_ptrs && !aligned16p(p.b[s]))) n.b = true;
  }
  for (int g = 0; g < p.ngroups; ++g) {
    if (p.a_trans && p.row_off[g] % 8 != 0) n.a = n.a_blocked = true;
    if (!p.b_trans && p.col_off[g] % 8 != 0) n.b = n.b_blocked = true;
  }
  // a packed operand whose M / N index is contiguous keeps the groups' blocks apart whenever offsets are in use
  if (n.a && p.a_trans && p.chain && p.ngroups > 1) n.a_blocked = true;
  if (n.b && !p.b_trans && p.chain && p.ngroups > 1) n.b_blocked = true;
  long long rows_a = 0, cols_b = 0, blocked_a = 0, blocked_b = 0;
  for (int g = 0; g < p.ngroups; ++g) {
    rows_a = rows_a > p.row_off[g] + p.m[g] ? rows_a : p.row_off[g] + p.m[g];
    cols_b = cols_b > p.col_off[g] + p.n[g] ? cols_b : p.col_off[g] + p.n[g];
    blocked_a += pad8(p.m[g]);
    blocked_b += pad8(p.n[g]);
  }
  for (int s = 0; s < p.nseg; ++s) {
    const bool used = p.chain || s < p.ngroups;
    if (!used || p.kseg[s] == 0) continue;
    const long long ra = p.chain ? rows_a : p.m[s], cb = p.chain ? cols_b : p.n[s];
    if (n.a) n.bytes += align256((size_t)(p.a_trans ? p.kseg[s] * (n.a_blocked ? blocked_a : pad8(ra)) : ra * pad8(p.kseg[s])) * 2);
    if (n.b) n.bytes += align256((size_t)(p.b_trans ? cb * pad8(p.kseg[s]) : p.kseg[s] * (n.b_blocked ? blocked_b : pad8(cb))) * 2);
  }
  return n;
}

// Copies the operands named by `need` into ws and rewrites the plan to read the copies.
static sbp_status pack_operands(MatmulPlan* plan, const PackNeed& need, void* ws, cudaStream_t st) {
  MatmulPlan& p = *plan;
  PackList list{};
  int nb = 0;
  auto flush = [&]() -> sbp_status {
    if (nb == 0) return SBP_OK;
    long long most = 0;
    for (int i = 0; i < nb; ++i) {
      const long long t = list.b[i].rows * ((list.b[i].cols + 7) / 8);
      most = t > most ? t : most;
    }
    long long gx = (most + 255) / 256;
    if (gx < 1) gx = 1;
    if (gx > 148 * 8) gx = 148 * 8;
    SBP_BOUNDS_UPLOAD(st);
    matmul_pack_kernel<<<dim3((unsigned)gx, (unsigned)nb), 256, 0, st>>>(list);
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) return cuda_fail(e, "operand repack launch");
    count_launch();
    nb = 0;
    return SBP_OK;
  };
  auto add = [&](const void* src, void* dst, long long rows, long long cols, long long sld, long long dld) -> sbp_status {
    if (rows == 0 || cols == 0) return SBP_OK;
    list.b[nb++] = PackBlock{static_cast<const unsigned short*>(src), static_cast<unsigned short*>(dst), rows, cols, sld, dld};
    return nb == kPackBlocks ? flush() : SBP_OK;
  };
  long long rows_a = 0, cols_b = 0, blocked_a = 0, blocked_b = 0;
  long long new_row_off[SBP_MAX_K], new_col_off[SBP_MAX_K];
  for (int g = 0; g < p.ngroups; ++g) {
    rows_a = rows_a > p.row_off[g] + p.m[g] ? rows_a : p.row_off[g] + p.m[g];
    cols_b = cols_b > p.col_off[g] + p.n[g] ? cols_b : p.col_off[g] + p.n[g];
    new_row_off[g] = blocked_a;
    new_col_off[g] = blocked_b;
    blocked_a += pad8(p.m[g]);
    blocked_b += pad8(p.n[g]);
  }
  char* cur = static_cast<char*>(ws);
  sbp_status stt;
  for (int s = 0; s < p.nseg; ++s) {
    const bool used = p.chain || s < p.ngroups;
    if (!used || p.kseg[s] == 0) continue;
    const long long K = p.kseg[s];
    const long long ra = p.chain ? rows_a : p.m[s], cb = p.chain ? cols_b : p.n[s];
    if (need.a) {
      const unsigned short* src = static_cast<const unsigned short*>(p.a[s]);
      unsigned short* dst = reinterpret_cast<unsigned short*>(cur);
      long long ld;
      if (!p.a_trans) {                       // stored [rows, K]
        ld = pad8(K);
        if ((stt = add(src, dst, ra, K, p.lda[s], ld)) != SBP_OK) return stt;
        cur += align256((size_t)ra * ld * 2);
      } else if (!need.a_blocked) {           // stored [K, rows]
        ld = pad8(ra);
        if ((stt = add(src, dst, K, ra, p.lda[s], ld)) != SBP_OK) return stt;
        cur += align256((size_t)K * ld * 2);
      } else {                                // stored [K, rows], one column block per output group
        ld = blocked_a;
        for (int g = 0; g < p.ngroups; ++g)
          if ((stt = add(src + p.row_off[g], dst + new_row_off[g], K, p.m[g], p.lda[s], ld)) != SBP_OK) return stt;
        cur += align256((size_t)K * ld * 2);
      }
      p.a[s] = dst;
      p.lda[s] = ld;
    }
    if (need.b) {
      const unsigned short* src = static_cast<const unsigned short*>(p.b[s]);
      unsigned short* dst = reinterpret_cast<unsigned short*>(cur);
      long long ld;
      if (p.b_trans) {                        // stored [cols, K]
        ld = pad8(K);
        if ((stt = add(src, dst, cb, K, p.ldb[s], ld)) != SBP_OK) return stt;
        cur += align256((size_t)cb * ld * 2);
      } else if (!need.b_blocked) {           // stored [K, cols]
        ld = pad8(cb);
        if ((stt = add(src, dst, K, cb, p.ldb[s], ld)) != SBP_OK) return stt;
        cur += align256((size_t)K * ld * 2);
      } else {
        ld = blocked_b;
        for (int g = 0; g < p.ngroups; ++g)
          if ((stt = add(src + p.col_off[g], dst + new_col_off[g], K, p.n[g], p.ldb[s], ld)) != SBP_OK) return stt;
        cur += align256((size_t)K * ld * 2);
      }
      p.b[s] = dst;
      p.ldb[s] = ld;
    }
  }
  if ((stt = flush()) != SBP_OK) return stt;
  for (int g = 0; g < p.ngroups; ++g) {
    if (need.a_blocked) p.row_off[g] = new_row_off[g];
    if (need.b_blocked) p.col_off[g] = new_col_off[g];
  }
  return SBP_OK;
}

static bool is_s(sbp_sig s, int ax) { return s.kind == SBP_SPLIT && s.axis == ax; }
static bool is_b(sbp_sig s) { return s.kind == SBP_BROADCAST; }
static bool is_p(sbp_sig s) { return s.kind == SBP_PARTIAL_SUM; }

// Validates the three descriptors and fills the plan.  need_ptrs = false for size queries.
static sbp_status build_plan(const sbp_tensor* x, const sbp_tensor* w, const sbp_tensor* y, uint32_t flags,
                             bool need_ptrs, MatmulPlan* plan) {
  sbp_status st = check_tensor(x, "x", need_ptrs);
  if (st != SBP_OK) return st;
  st = check_tensor(w, "w", need_ptrs);
  if (st != SBP_OK) return st;
  st = check_tensor(y, "y", need_ptrs);
  if (st != SBP_OK) return st;
  if (x->ndim != 2 || w->ndim != 2 || y->ndim != 2) return fail(SBP_ERR_SHAPE, "x, w and y must be 2-D");
  if (flags & ~(SBP_EPILOGUE_GELU | SBP_TRANS_X | SBP_TRANS_W)) return fail(SBP_ERR_INVALID_ARG, "unknown flags 0x%x", flags);
  const bool tx = (flags & SBP_TRANS_X) != 0, tw = (flags & SBP_TRANS_W) != 0;
  // the operands as they enter the product: [M,K] and [K,N]
  const long long M = x->shape[tx ? 1 : 0], K = x->shape[tx ? 0 : 1], N = w->shape[tw ? 0 : 1];
  if (w->shape[tw ? 1 : 0] != K)
    return fail(SBP_ERR_SHAPE, "x is [%lld,%lld] but w has %lld rows", M, K, (long long)w->shape[tw ? 1 : 0]);
  if (y->shape[0] != M || y->shape[1] != N) return fail(SBP_ERR_SHAPE, "y must be [%lld,%lld]", M, N);
  if (x->dtype != w->dtype) return fail(SBP_ERR_DTYPE, "x and w differ in dtype");
  if (x->dtype != SBP_F32 && x->dtype != SBP_BF16) return fail(SBP_ERR_DTYPE, "operands must be F32 or BF16");
  if (y->dtype != SBP_F32 && y->dtype != SBP_BF16) return fail(SBP_ERR_DTYPE, "y must be F32 or BF16");
  if (x->dtype == SBP_F32 && y->dtype != SBP_F32) return fail(SBP_ERR_DTYPE, "F32 operands need an F32 result");
  const int k = placement_k(x);
  if (placement_k(w) != k || placement_k(y) != k) return fail(SBP_ERR_INVALID_ARG, "operands differ in k");

  // signature of the operand that enters Table 1: a transposed operand swaps S(0) and S(1)
  auto effective = [](sbp_sig s, bool t) {
    if (t && s.kind == SBP_SPLIT) s.axis = 1 - s.axis;
    return s;
  };
  const sbp_sig xs = effective(x->sbp[0], tx), ws = effective(w->sbp[0], tw), ys = y->sbp[0];
  sbp_sig natural;
  st = sbp_matmul_infer(xs, ws, &natural);
  if (st != SBP_OK) return st;
  const bool fused = is_p(natural) && !is_p(ys);
  if (!fused && !same_sig(natural, ys))
    return fail(SBP_ERR_SIGNATURE, "y's signature is neither the one Table 1 deduces nor a fusable boxing of it");
  if (fused && !(is_b(ys) || ys.kind == SBP_SPLIT))
    return fail(SBP_ERR_SIGNATURE, "a P(sum) product can be written directly only as B or S(i)");
  if ((flags & SBP_EPILOGUE_GELU) && is_p(natural) && !fused)
    return fail(SBP_ERR_SIGNATURE, "GeLU is not linear: it cannot be applied to partial values");

  MatmulPlan& p = *plan;
  p = MatmulPlan{};
  p.gelu = (flags & SBP_EPILOGUE_GELU) ? 1 : 0;
  p.a_trans = tx ? 1 : 0;
  p.b_trans = tw ? 1 : 0;
  p.in_dtype = x->dtype;
  p.out_dtype = y->dtype;

  auto range = [&](long long n, int r, long long* start, long long* len) {
    int64_t s_, l_;
    split_range(n, k, r, &s_, &l_);
    *start = s_;
    *len = l_;
  };
  // K-segments = the local operands of each shard
  for (int r = 0; r < k; ++r) {
    long long st_, ln;
    p.a[r] = x->local[r];
    p.b[r] = w->local[r];
    // leading dimensions of the stored local tensors: the descriptor's, else their last local extent
    p.lda[r] = local_pitch(x, r);
    p.ldb[r] = local_pitch(w, r);
    p.kseg[r] = K;
    if (is_s(xs, 1)) { range(K, r, &st_, &ln); p.kseg[r] = ln; }
  }
  p.nseg = k;

  for (int r = 1; r < k; ++r)
    if (is_b(ys) && local_pitch(y, r) != local_pitch(y, 0))
      return fail(SBP_ERR_UNSUPPORTED, "the replicas of a B result must share one leading dimension");
  auto set_replicas = [&]() {   // one group, stored to every distinct B replica
    p.ngroups = 1;
    p.m[0] = M; p.n[0] = N; p.ldy[0] = local_pitch(y, 0);
    void* uniq[SBP_MAX_K];
    int nu = 0;
    for (int r = 0; r < k; ++r) {
      bool seen = false;
      for (int q = 0; q < nu; ++q) seen = seen || uniq[q] == y->local[r];
      if (!seen) uniq[nu++] = y->local[r];
    }
    p.y[0] = uniq[0];
    p.n_rep = nu - 1;
    for (int q = 1; q < nu; ++q) p.y_rep[q - 1] = uniq[q];
  };

  if (!fused) {
    p.chain = 0;
    if (is_b(natural)) {
      p.nseg = 1;
      set_replicas();
    } else {
      p.ngroups = k;
      for (int g = 0; g < k; ++g) {
        long long st_, ln;
        p.m[g] = M; p.n[g] = N; p.ldy[g] = local_pitch(y, g);
        if (is_s(natural, 0)) { range(M, g, &st_, &ln); p.m[g] = ln; }
        if (is_s(natural, 1)) { range(N, g, &st_, &ln); p.n[g] = ln; }
        p.y[g] = y->local[g];
      }
    }
  } else {
    p.chain = 1;
    if (is_b(ys)) {
      set_replicas();
    } else {
      p.ngroups = k;
      for (int g = 0; g < k; ++g) {
        long long st_, ln;
        p.m[g] = M; p.n[g] = N; p.ldy[g] = local_pitch(y, g);
        if (ys.axis == 0) { range(M, g, &st_, &ln); p.m[g] = ln; p.row_off[g] = st_; }
        else { range(N, g, &st_, &ln); p.n[g] = ln; p.col_off[g] = st_; }
        p.y[g] = y->local[g];
      }
    }
  }
  return SBP_OK;
}

// Two-axis placements (Section 3.3, Table 3): Table 1 is applied to each placement axis on its
// own -- e.g. (S(0),B) x (B,S(1)) -> (S(0),S(1)) and (S(0),S(1)) x (B,S(0)) -> (S(0),P(sum)) --
// and every device multiplies its local tensors.  No fused output boxing on this path.
static sbp_status build_plan_2d(const sbp_tensor* x, const sbp_tensor* w, const sbp_tensor* y, uint32_t flags,
                                bool need_ptrs, MatmulPlan* plan) {
  sbp_status st = check_tensor_nd(x, "x", need_ptrs);
  if (st != SBP_OK) return st;
  st = check_tensor_nd(w, "w", need_ptrs);
  if (st != SBP_OK) return st;
  st = check_tensor_nd(y, "y", need_ptrs);
  if (st != SBP_OK) return st;
  if (x->pdims != 2 || w->pdims != 2 || y->pdims != 2) return fail(SBP_ERR_INVALID_ARG, "x, w and y must share one two-axis placement");
  for (int p = 0; p < 2; ++p)
    if (x->pshape[p] != w->pshape[p] || x->pshape[p] != y->pshape[p])
      return fail(SBP_ERR_INVALID_ARG, "x, w and y must share one two-axis placement");
  if (x->ndim != 2 || w->ndim != 2 || y->ndim != 2) return fail(SBP_ERR_SHAPE, "x, w and y must be 2-D");
  const long long M = x->shape[0], K = x->shape[1], N = w->shape[1];
  if (w->shape[0] != K) return fail(SBP_ERR_SHAPE, "x is [%lld,%lld] but w has %lld rows", M, K, (long long)w->shape[0]);
  if (y->shape[0] != M || y->shape[1] != N) return fail(SBP_ERR_SHAPE, "y must be [%lld,%lld]", M, N);
  if (x->dtype != w->dtype) return fail(SBP_ERR_DTYPE, "x and w differ in dtype");
  if (x->dtype != SBP_F32 && x->dtype != SBP_BF16) return fail(SBP_ERR_DTYPE, "operands must be F32 or BF16");
  if (y->dtype != SBP_F32 && y->dtype != SBP_BF16) return fail(SBP_ERR_DTYPE, "y must be F32 or BF16");
  if (x->dtype == SBP_F32 && y->dtype != SBP_F32) return fail(SBP_ERR_DTYPE, "F32 operands need an F32 result");
  if (flags & (SBP_TRANS_X | SBP_TRANS_W)) return fail(SBP_ERR_UNSUPPORTED, "transposed operands on a two-axis placement");
  if (flags & ~SBP_EPILOGUE_GELU) return fail(SBP_ERR_INVALID_ARG, "unknown flags 0x%x", flags);
  for (int p = 0; p < 2; ++p) {
    sbp_sig natural;
    st = sbp_matmul_infer(x->sbp[p], w->sbp[p], &natural);
    if (st != SBP_OK) return st;
    if (!same_sig(natural, y->sbp[p]))
      return fail(SBP_ERR_SIGNATURE, "placement axis %d: y's signature is not the one Table 1 deduces", p);
    if ((flags & SBP_EPILOGUE_GELU) && is_p(natural))
      return fail(SBP_ERR_SIGNATURE, "GeLU is not linear: it cannot be applied to partial values");
  }
  const int k = placement_k(x);
  MatmulPlan& p = *plan;
  p = MatmulPlan{};
  p.gelu = (flags & SBP_EPILOGUE_GELU) ? 1 : 0;
  p.in_dtype = x->dtype;
  p.out_dtype = y->dtype;
  p.ngroups = k;
  p.nseg = k;
  p.chain = 0;
  for (int r = 0; r < k; ++r) {
    int64_t xs[SBP_MAX_DIMS], wsz[SBP_MAX_DIMS], ys[SBP_MAX_DIMS];
    local_shape_nd(x, r, xs);
    local_shape_nd(w, r, wsz);
    local_shape_nd(y, r, ys);
    if (xs[1] != wsz[0] || ys[0] != xs[0] || ys[1] != wsz[1])
      return fail(SBP_ERR_SHAPE, "device %d: local shapes [%lld,%lld] x [%lld,%lld] -> [%lld,%lld] do not fit", r,
                  (long long)xs[0], (long long)xs[1], (long long)wsz[0], (long long)wsz[1], (long long)ys[0],
                  (long long)ys[1]);
    p.a[r] = x->local[r];
    p.b[r] = w->local[r];
    p.lda[r] = local_pitch(x, r);
    p.ldb[r] = local_pitch(w, r);
    p.kseg[r] = xs[1];
    p.m[r] = xs[0];
    p.n[r] = wsz[1];
    p.ldy[r] = local_pitch(y, r);
    p.y[r] = y->local[r];
  }
  return SBP_OK;
}

}  // namespace sbp

using namespace sbp;

extern "C" {

size_t sbp_matmul_workspace_bytes_for(const sbp_tensor* x, const sbp_tensor* w, const sbp_tensor* y, uint32_t flags) {
  MatmulPlan plan;
  const bool two_axes = x && w && y && (x->pdims == 2 || w->pdims == 2 || y->pdims == 2);
  const sbp_status st = two_axes ? build_plan_2d(x, w, y, flags, false, &plan) : build_plan(x, w, y, flags, false, &plan);
  if (st != SBP_OK) return 0;
  // without pointers to look at, an operand counts as misaligned only by its shape
  return pack_need(plan, false).bytes + matmul_tc_workspace_bytes(plan);
}

size_t sbp_matmul_workspace_bytes(const sbp_tensor* x, const sbp_tensor* w, const sbp_tensor* y) {
  return sbp_matmul_workspace_bytes_for(x, w, y, 0);
}

void sbp_tensor_map_stats(uint64_t* reused, uint64_t* encoded) {
  unsigned long long h = 0, e = 0;
  tensor_map_cache_stats(&h, &e);
  if (reused) *reused = h;
  if (encoded) *encoded = e;
}

void sbp_matmul_set_form(int32_t form, int32_t max_pairs) { tc_set_form(form, max_pairs); }

int32_t sbp_matmul_route(int64_t m, int64_t n, int64_t k, int32_t pairs, uint32_t flags, int32_t replicas, int32_t out_f32,
                         int64_t* tall_tiles) {
  if (m <= 0 || n <= 0 || k <= 0 || pairs <= 0 || replicas < 1) {
    if (tall_tiles) *tall_tiles = 0;
    return -1;
  }
  const long long tn = (n + 255) / 256;
  return tc_route((m + 255) / 256 * tn, (m + 511) / 512 * tn, (k + 63) / 64, pairs, (flags & SBP_EPILOGUE_GELU) != 0, replicas - 1,
                  out_f32 != 0, 0, reinterpret_cast<long long*>(tall_tiles));
}

void sbp_matmul_form_stats(uint64_t launches[3]) {
  unsigned long long v[3] = {0, 0, 0};
  tc_form_stats(v);
  if (launches)
    for (int i = 0; i < 3; ++i) launches[i] = v[i];
}

sbp_status sbp_matmul(const sbp_tensor* x, const sbp_tensor* w, sbp_tensor* y, uint32_t flags, void* ws,
                      size_t ws_bytes, void* cuda_stream) {
  SBP_RANGE("sbp_matmul");
  MatmulPlan plan;
  const bool two_axes = x && w && y && (x->pdims == 2 || w->pdims == 2 || y->pdims == 2);
  sbp_status st = two_axes ? build_plan_2d(x, w, y, flags, true, &plan) : build_plan(x, w, y, flags, true, &plan);
  if (st != SBP_OK) return st;
  cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
  SBP_BOUNDS_RESET();
  SBP_BOUNDS_TENSOR(x);
  SBP_BOUNDS_TENSOR(w);
  SBP_BOUNDS_TENSOR(y);
  SBP_BOUNDS_ADD(ws, ws_bytes);
  bool taken = false;
  st = launch_matmul_tc(plan, nullptr, stream, &taken);
  if (taken) return st;
  // bf16 operands that only miss the copy engine's alignment rules: repack them into the workspace,
  // when the caller gave one that is large enough, and stay on the tensor cores
  const PackNeed need = pack_need(plan, true);
  if ((need.a || need.b) && ws && ws_bytes >= need.bytes && reinterpret_cast<uintptr_t>(ws) % 256 == 0) {
    MatmulPlan packed = plan;
    st = pack_operands(&packed, need, ws, stream);
    if (st != SBP_OK) return st;
    st = launch_matmul_tc(packed, nullptr, stream, &taken);
    if (taken) return st;
  }
  return launch_fma(plan, stream);
}

// ------------------------------------------------------------------ fused classifier

// Chunks of 128 classes per shard and in total, for the partial arrays of the fused path.
static int classifier_chunks(const sbp_tensor* w, int part_base[SBP_MAX_K], long long class_start[SBP_MAX_K]) {
  const int k = placement_k(w);
  int total = 0;
  for (int r = 0; r < k; ++r) {
    int64_t st, ln;
    split_range(w->shape[1], k, r, &st, &ln);
    part_base[r] = total;
    class_start[r] = st;
    total += (int)((ln + 127) / 128);
  }
  return total;
}

static sbp_status check_classifier(const sbp_tensor* f, const sbp_tensor* w, bool need_ptrs) {
  sbp_status st = check_tensor(f, "features", need_ptrs);
  if (st != SBP_OK) return st;
  st = check_tensor(w, "weight", need_ptrs);
  if (st != SBP_OK) return st;
  if (f->ndim != 2 || w->ndim != 2) return fail(SBP_ERR_SHAPE, "features and weight must be 2-D");
  if (f->shape[1] != w->shape[0]) return fail(SBP_ERR_SHAPE, "features are [rows,%lld] but weight has %lld rows",
                                              (long long)f->shape[1], (long long)w->shape[0]);
  if (f->dtype != SBP_BF16 || w->dtype != SBP_BF16) return fail(SBP_ERR_DTYPE, "the fused classifier takes BF16 operands");
  if (placement_k(f) != placement_k(w)) return fail(SBP_ERR_INVALID_ARG, "operands differ in k");
  if (!is_b(f->sbp[0]) || !is_s(w->sbp[0], 1))
    return fail(SBP_ERR_SIGNATURE, "the fused classifier needs features B and weight S(1)");
  if (w->shape[1] < 1) return fail(SBP_ERR_SHAPE, "softmax over zero classes");
  if (w->shape[1] / 128 + SBP_MAX_K > 0x3fffffffLL) return fail(SBP_ERR_UNSUPPORTED, "too many classes");
  return SBP_OK;
}

size_t sbp_matmul_softmax_xent_workspace_bytes(const sbp_tensor* features, const sbp_tensor* weight) {
  if (check_classifier(features, weight, false) != SBP_OK) return 0;
  int part_base[SBP_MAX_K];
  long long class_start[SBP_MAX_K];
  const int parts = classifier_chunks(weight, part_base, class_start);
  const size_t rows = (size_t)features->shape[0];
  return (3 * (size_t)parts * rows + xent_finish_stage_floats((long long)rows)) * sizeof(float);
}

sbp_status sbp_matmul_softmax_xent(const sbp_tensor* features, const sbp_tensor* weight, const sbp_tensor* labels,
                                   sbp_tensor* loss, sbp_tensor* row_max, sbp_tensor* row_sum, void* ws,
                                   size_t ws_bytes, void* cuda_stream) {
  SBP_RANGE("sbp_matmul_softmax_xent");
  sbp_status st = check_classifier(features, weight, true);
  if (st != SBP_OK) return st;
  const int k = placement_k(features);
  const long long rows = features->shape[0], K = features->shape[1], N = weight->shape[1];
  st = check_xent_outputs(labels, loss, row_max, row_sum, rows, k);
  if (st != SBP_OK) return st;
  if (rows == 0) return SBP_OK;
  const size_t need = sbp_matmul_softmax_xent_workspace_bytes(features, weight);
  if (!ws || ws_bytes < need) return fail(SBP_ERR_WORKSPACE, "workspace of %zu bytes needed, %zu given", need, ws_bytes);
  if (reinterpret_cast<uintptr_t>(ws) % 4 != 0) return fail(SBP_ERR_ALIGNMENT, "workspace must be 4-byte aligned");

  // (B, S(1)) -> S(1): one group per shard of the weight
  MatmulPlan plan{};
  plan.in_dtype = SBP_BF16;
  plan.out_dtype = SBP_F32;
  plan.ngroups = k;
  plan.nseg = k;
  plan.chain = 0;
  for (int r = 0; r < k; ++r) {
    int64_t s0, ln;
    split_range(N, k, r, &s0, &ln);
    plan.a[r] = features->local[r];
    plan.b[r] = weight->local[r];
    plan.lda[r] = local_pitch(features, r);
    plan.ldb[r] = local_pitch(weight, r);
    plan.kseg[r] = K;
    plan.m[r] = rows;
    plan.n[r] = ln;
    plan.ldy[r] = ln;
  }
  XentFusion xf{};
  const int parts = classifier_chunks(weight, xf.part_base, xf.class_start);
  xf.part_m = static_cast<float*>(ws);
  xf.part_s = xf.part_m + (size_t)parts * rows;
  xf.part_t = xf.part_s + (size_t)parts * rows;
  float* stage = xf.part_t + (size_t)parts * rows;
  xf.labels = static_cast<const long long*>(labels->local[0]);
  xf.rows = rows;
  cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
  SBP_BOUNDS_RESET();
  SBP_BOUNDS_TENSOR(features);
  SBP_BOUNDS_TENSOR(weight);
  SBP_BOUNDS_TENSOR(labels);
  SBP_BOUNDS_TENSOR(loss);
  SBP_BOUNDS_TENSOR(row_max);
  SBP_BOUNDS_TENSOR(row_sum);
  SBP_BOUNDS_ADD(ws, need);
  bool taken = false;
  st = launch_matmul_tc(plan, &xf, stream, &taken);
  if (!taken)
    return fail(SBP_ERR_UNSUPPORTED,
                "the fused classifier needs the tensor-core path (16-byte aligned operands, feature and per-shard class "
                "counts that are multiples of 8, a non-empty contraction); use sbp_matmul + sbp_softmax_xent instead");
  if (st != SBP_OK) return st;
  return launch_xent_finish(xf.part_m, xf.part_s, xf.part_t, parts, rows, stage, loss, row_max, row_sum, k, stream);
}

sbp_status sbp_matmul_softmax_xent_backward(const sbp_tensor* features, const sbp_tensor* weight,
                                            const sbp_tensor* labels, const sbp_tensor* row_max,
                                            const sbp_tensor* row_sum, sbp_tensor* grad_logits, void* cuda_stream) {
  SBP_RANGE("sbp_matmul_softmax_xent_backward");
  sbp_status st = check_classifier(features, weight, true);
  if (st != SBP_OK) return st;
  const int k = placement_k(features);
  const long long rows = features->shape[0], K = features->shape[1], N = weight->shape[1];
  st = check_tensor(grad_logits, "grad_logits", true);
  if (st != SBP_OK) return st;
  if (grad_logits->ndim != 2 || grad_logits->shape[0] != rows || grad_logits->shape[1] != N)
    return fail(SBP_ERR_SHAPE, "grad_logits must be [rows, classes]");
  if (grad_logits->dtype != SBP_BF16 && grad_logits->dtype != SBP_F32)
    return fail(SBP_ERR_DTYPE, "grad_logits must be BF16 or F32");
  if (placement_k(grad_logits) != k || !is_s(grad_logits->sbp[0], 1))
    return fail(SBP_ERR_SIGNATURE, "grad_logits must be S(1) on the operands' placement");
  const sbp_tensor* vecs[3] = {labels, row_max, row_sum};
  const char* names[3] = {"labels", "row_max", "row_sum"};
  for (int i = 0; i < 3; ++i) {
    st = check_tensor(vecs[i], names[i], true);
    if (st != SBP_OK) return st;
    if (vecs[i]->ndim != 1 || vecs[i]->shape[0] != rows) return fail(SBP_ERR_SHAPE, "%s must be [rows]", names[i]);
    if (placement_k(vecs[i]) != k || !is_b(vecs[i]->sbp[0])) return fail(SBP_ERR_SIGNATURE, "%s must be B", names[i]);
    if (vecs[i]->dtype != (i == 0 ? SBP_I64 : SBP_F32)) return fail(SBP_ERR_DTYPE, "%s has the wrong dtype", names[i]);
  }
  if (rows == 0) return SBP_OK;

  MatmulPlan plan{};
  plan.in_dtype = SBP_BF16;
  plan.out_dtype = grad_logits->dtype;
  plan.ngroups = k;
  plan.nseg = k;
  plan.chain = 0;
  XentFusion xf{};
  for (int r = 0; r < k; ++r) {
    int64_t s0, ln;
    split_range(N, k, r, &s0, &ln);
    plan.a[r] = features->local[r];
    plan.b[r] = weight->local[r];
    plan.lda[r] = local_pitch(features, r);
    plan.ldb[r] = local_pitch(weight, r);
    plan.kseg[r] = K;
    plan.m[r] = rows;
    plan.n[r] = ln;
    plan.ldy[r] = local_pitch(grad_logits, r);
    plan.y[r] = grad_logits->local[r];
    xf.class_start[r] = s0;
  }
  xf.grad = 1;
  xf.labels = static_cast<const long long*>(labels->local[0]);
  xf.row_max = static_cast<const float*>(row_max->local[0]);
  xf.row_sum = static_cast<const float*>(row_sum->local[0]);
  xf.rows = rows;
  SBP_BOUNDS_RESET();
  SBP_BOUNDS_TENSOR(features);
  SBP_BOUNDS_TENSOR(weight);
  SBP_BOUNDS_TENSOR(labels);
  SBP_BOUNDS_TENSOR(row_max);
  SBP_BOUNDS_TENSOR(row_sum);
  SBP_BOUNDS_TENSOR(grad_logits);
  bool taken = false;
  st = launch_matmul_tc(plan, &xf, static_cast<cudaStream_t>(cuda_stream), &taken);
  if (!taken)
    return fail(SBP_ERR_UNSUPPORTED,
                "the fused classifier backward needs the tensor-core path (16-byte aligned operands and result, feature "
                "and per-shard class counts that are multiples of 8, a non-empty contraction); store the logits and use "
                "sbp_softmax_xent_backward instead");
  return st;
}

}  // extern "C"
