// Boxing transforms between SBP signatures on k shards held in one GPU's memory
// (Section 3.2, Table 2 "same placement" column).
//
// Every transform is expressed on one canonical 5-D view of the logical tensor,
//     [A][Na][M][Nb][C],
// where at most the axes Na and Nb are restricted by a split signature (on the source
// side, the destination side, or both) and C is the contiguous tail.  A *task* is one
// (source shard, destination shard) pair; the elements it moves are the intersection of
// the two shards' regions: A * la * M contiguous segments of lb * C elements.  Tasks are
// cut into tiles of J*256 vectors (rows = segments, columns = vectors inside a segment);
// one CTA moves one tile, each thread J vectors with all loads issued before the stores.
//
//   data movement  S(i)->S(j), S(i)->B (one read, k writes), B->S(i), copies
//   reduction      P(sum)/P(max) -> B (k reads, k writes) or -> S(i) (k reads, 1 write);
//                  fp32 accumulator, shards added in rank order, one rounding at the end
#include <cuda_bf16.h>

#include <algorithm>
#include <atomic>

#include "bounds_check.h"
#include "boxing_arith.h"
#include "boxing_params.h"
#include "sbp_internal.h"

namespace sbp {

// ------------------------------------------------------------------ the tile kernel

struct TaskGeom {
  long long nseg, seg_vecs;   // segments in the task, vectors per segment
  long long la;
  long long Na_s, aoff_s, Nb_s, boff_s;
  long long Na_d, aoff_d, Nb_d, boff_d;
  long long Ps, Pd;           // row pitch on either side (the local Nb extent unless a leading dimension is given)
};

__device__ __forceinline__ void task_geometry(const BoxParams& p, int s, int d, int vbytes, TaskGeom* g) {
  long long a0 = 0, la = p.Na, b0 = 0, lb = p.Nb;
  if (p.src_a) split_range_pre(p.a_base, p.a_rem, s, &a0, &la);
  else if (p.dst_a) split_range_pre(p.a_base, p.a_rem, d, &a0, &la);
  if (p.src_b) split_range_pre(p.b_base, p.b_rem, s, &b0, &lb);
  else if (p.dst_b) split_range_pre(p.b_base, p.b_rem, d, &b0, &lb);
  g->la = la;
  g->nseg = p.A * la * p.M;
  g->seg_vecs = lb * p.C * p.esz / vbytes;
  g->Na_s = p.src_a ? la : p.Na;  g->aoff_s = p.src_a ? 0 : a0;
  g->Nb_s = p.src_b ? lb : p.Nb;  g->boff_s = p.src_b ? 0 : b0;
  g->Na_d = p.dst_a ? la : p.Na;  g->aoff_d = p.dst_a ? 0 : a0;
  g->Nb_d = p.dst_b ? lb : p.Nb;  g->boff_d = p.dst_b ? 0 : b0;
  g->Ps = p.src_pitch[s] ? p.src_pitch[s] : g->Nb_s;
  g->Pd = p.dst_pitch[d] ? p.dst_pitch[d] : g->Nb_d;
}

// V: vector type moved by one thread access.  OP: BoxOp.  J: vectors per thread.
// KT: compile-time number of source shards of a reduction (0 = read p.k at run time).
template <typename V, int OP, int J, int KT>
__global__ void __launch_bounds__(256) box_tile_kernel(const __grid_constant__ BoxParams p) {
  // Task index varies fastest: CTAs that run together then touch the same rows of every shard
  // (whole DRAM pages) instead of one column stripe of one shard.  The grid is below 2^31 tiles,
  // so this is 32-bit arithmetic.
  // Let the next kernel in the stream be set up while this one's last CTAs run; it waits, as
  // this one does below, for its predecessor to finish before it touches global memory.
  SBP_PDL_RELEASE();
  const unsigned u = blockIdx.x;
  const unsigned rem = u / (unsigned)p.ntasks;
  const int t = (int)(u - rem * (unsigned)p.ntasks);
  const unsigned row_tile_u = rem / (unsigned)p.col_tiles;
  const long long row_tile = row_tile_u;
  const long long col_tile = rem - row_tile_u * (unsigned)p.col_tiles;

  int s = t, d = t;
  if (p.one_dst) { d = p.dst_shard; if (p.mode == MODE_DIAG) s = p.dst_shard; }
  else if (p.mode == MODE_PAIRS) { s = t / p.k; d = t - s * p.k; }
  else if (p.mode == MODE_REDUCE_B) { s = 0; d = 0; }

  TaskGeom g;
  task_geometry(p, s, d, (int)sizeof(V), &g);
  const long long seg0 = row_tile * p.rows_per_tile;
  if (seg0 >= g.nseg) return;
  const long long col0 = col_tile << p.cv_log2;
  if (col0 >= g.seg_vecs) return;

  const long long cs = p.C * p.esz;   // bytes per unit step of the Nb axis
  const bool flat = (p.A == 1 && p.M == 1);

  long long so[J], dofs[J];
  bool ok[J];
#pragma unroll
  for (int j = 0; j < J; ++j) {
    const int f = threadIdx.x + j * 256;
    const long long seg = seg0 + (f >> p.cv_log2);
    const long long col = col0 + (f & ((1 << p.cv_log2) - 1));
    ok[j] = seg < g.nseg && col < g.seg_vecs;
    long long x = 0, ia = seg, m = 0;
    if (!flat) {
      const long long q = seg / p.M;
      m = seg - q * p.M;
      x = q / g.la;
      ia = q - x * g.la;
    }
    so[j] = ((((x * g.Na_s + g.aoff_s + ia) * p.M + m) * g.Ps + g.boff_s) * cs) / (long long)sizeof(V) + col;
    dofs[j] = ((((x * g.Na_d + g.aoff_d + ia) * p.M + m) * g.Pd + g.boff_d) * cs) / (long long)sizeof(V) + col;
  }

  SBP_PDL_WAIT();   // the previous kernel's results are visible from here on

  V val[J];
  if constexpr (OP == OP_COPY) {
    const V* sp = reinterpret_cast<const V*>(p.src[s]);
#pragma unroll
    for (int j = 0; j < J; ++j)
      if (ok[j] && SBP_GUARD(sp + so[j], sizeof(V))) val[j] = ld_stream(sp + so[j]);

  } else {
    using L = typename Lanes<OP, V>::type;
    const int kk = KT ? KT : p.k;
    if constexpr (KT != 0) {
      V raw[J][KT ? KT : 1];
#pragma unroll
      for (int j = 0; j < J; ++j)
#pragma unroll
        for (int r = 0; r < (KT ? KT : 1); ++r)
          if (ok[j] && SBP_GUARD(reinterpret_cast<const V*>(p.src[r]) + so[j], sizeof(V)))
            raw[j][r] = ld_stream(reinterpret_cast<const V*>(p.src[r]) + so[j]);
#pragma unroll
      for (int j = 0; j < J; ++j) {
        if (!ok[j]) continue;
        L acc;
        acc.load(raw[j][0]);
#pragma unroll
        for (int r = 1; r < (KT ? KT : 1); ++r) {
          L x;
          x.load(raw[j][r]);
          combine<OP>(acc, x);
        }
        val[j] = acc.store();
      }
    } else {
#pragma unroll
      for (int j = 0; j < J; ++j) {
        if (!ok[j]) continue;
        L acc;
        if (!SBP_GUARD(reinterpret_cast<const V*>(p.src[0]) + so[j], sizeof(V))) continue;
        acc.load(ld_stream(reinterpret_cast<const V*>(p.src[0]) + so[j]));
        for (int r = 1; r < kk; ++r) {
          L x;
          if (!SBP_GUARD(reinterpret_cast<const V*>(p.src[r]) + so[j], sizeof(V))) continue;
          x.load(ld_stream(reinterpret_cast<const V*>(p.src[r]) + so[j]));
          combine<OP>(acc, x);
        }
        val[j] = acc.store();
      }
    }
  }

  if (p.mode == MODE_GATHER || p.mode == MODE_REDUCE_B) {
    for (int r = 0; r < p.n_dst; ++r) {
      V* dp = reinterpret_cast<V*>(p.dst[r]);
#pragma unroll
      for (int j = 0; j < J; ++j)
        if (ok[j] && SBP_GUARD(dp + dofs[j], sizeof(V))) st_stream(dp + dofs[j], val[j]);
    }
  } else {
    V* dp = reinterpret_cast<V*>(p.dst[d]);
#pragma unroll
    for (int j = 0; j < J; ++j)
      if (ok[j] && SBP_GUARD(dp + dofs[j], sizeof(V))) st_stream(dp + dofs[j], val[j]);
  }
}

// row = c / per_row and the remainder; 32-bit arithmetic whenever both fit (a 64-bit division
// costs an order of magnitude more and sits in front of every chunk's loads).
__device__ __forceinline__ void chunk_row(long long c, long long per_row, long long* row, long long* within) {
  if (((unsigned long long)c | (unsigned long long)per_row) >> 32) {
    *row = c / per_row;
    *within = c - *row * per_row;
  } else {
    const unsigned r = (unsigned)c / (unsigned)per_row;
    *row = r;
    *within = (unsigned)c - r * (unsigned)per_row;
  }
}

// ------------------------------------------------------------------ S(i)/B -> P(sum)
//
// Destination shard d has the full shape: the vectors [own_lo, own_hi) of every row come from
// the source shard, everything else is written as zero.  Three quarters (for k = 4) of the work
// is plain zero stores, so the kernel keeps its index arithmetic out of the inner loop: the
// host precomputes the per-shard column ranges, a CTA walks 32 KiB chunks of rows.
struct ScatterParams {
  const char* src[SBP_MAX_K];
  char* dst[SBP_MAX_K];
  long long own_lo[SBP_MAX_K], own_hi[SBP_MAX_K];   // in vectors, inside a row
  long long nrows, row_vecs, chunks_per_row, total_chunks;
  int d0;                                           // first destination shard of the launch (grid.y counts from it)
};

constexpr int kScatterJ = 8;

template <typename V>
__global__ void __launch_bounds__(256) box_scatter_kernel(const __grid_constant__ ScatterParams p) {
  SBP_PDL_RELEASE();
  const int d = blockIdx.y + p.d0;
  const V* sp = reinterpret_cast<const V*>(p.src[d]);
  V* dp = reinterpret_cast<V*>(p.dst[d]);
  const long long lo = p.own_lo[d], hi = p.own_hi[d], w = hi - lo;
  SBP_PDL_WAIT();
  for (long long c = blockIdx.x; c < p.total_chunks; c += gridDim.x) {
    long long row, within;
    chunk_row(c, p.chunks_per_row, &row, &within);
    const long long col0 = within * (256 * kScatterJ) + threadIdx.x;
    V val[kScatterJ];
#pragma unroll
    for (int j = 0; j < kScatterJ; ++j) {
      const long long col = col0 + j * 256;
      val[j] = V{};
      if (col >= lo && col < hi && SBP_GUARD(sp + row * w + (col - lo), sizeof(V))) val[j] = ld_stream(sp + row * w + (col - lo));
    }
#pragma unroll
    for (int j = 0; j < kScatterJ; ++j) {
      const long long col = col0 + j * 256;
      if (col < p.row_vecs && SBP_GUARD(dp + row * p.row_vecs + col, sizeof(V))) dp[row * p.row_vecs + col] = val[j];
    }
  }
}

template <typename V>
static void launch_scatter_v(const ScatterParams& sp, int k, cudaStream_t st) {
  long long gx = sp.total_chunks < 148 * 6 ? sp.total_chunks : 148 * 6;
  if (gx < 1) gx = 1;
  SBP_BOUNDS_UPLOAD(st);
  launch_dependent(box_scatter_kernel<V>, dim3((unsigned)gx, (unsigned)k), dim3(256), 0, st, sp);
}

// ------------------------------------------------------------------ S(i) -> B with an fp32 -> bf16 cast
//
// Section 6.4 ("Parallelizing the Optimizer"): sharded fp32 model states are cast to half
// precision and all-gathered -- a cast op whose input is S(0) and whose output is B.  Here the
// cast is folded into the gather: every source shard is read once as fp32, rounded to bf16
// (nearest even) and written to its place in every replica.  EPV = bf16 elements per store.
struct GatherCastParams {
  const float* src[SBP_MAX_K];
  __nv_bfloat16* dst[SBP_MAX_K];
  long long own_lo[SBP_MAX_K], own_hi[SBP_MAX_K];   // in units of EPV elements, inside a full row
  long long nrows, row_units;
  int n_dst;
};

template <int EPV>
__global__ void __launch_bounds__(256) box_gather_cast_kernel(const __grid_constant__ GatherCastParams p) {
  constexpr int J = 4;
  SBP_PDL_RELEASE();
  const int s = blockIdx.y;
  const long long lo = p.own_lo[s], w = p.own_hi[s] - lo;
  if (w <= 0) return;
  SBP_PDL_WAIT();
  const long long chunks_per_row = (w + 256 * J - 1) / (256 * J);
  const long long total = p.nrows * chunks_per_row;
  for (long long c = blockIdx.x; c < total; c += gridDim.x) {
    long long row, within;
    chunk_row(c, chunks_per_row, &row, &within);
    const long long col0 = within * (256 * J) + threadIdx.x;
    const float* sp = p.src[s] + (row * w) * EPV;
    float v[J][EPV] = {};
#pragma unroll
    for (int j = 0; j < J; ++j) {
      const long long col = col0 + j * 256;
      if (col < w && SBP_GUARD(sp + col * EPV, EPV * sizeof(float))) {
        if (EPV == 8) {
          const float4 a = __ldg(reinterpret_cast<const float4*>(sp + col * 8));
          const float4 b = __ldg(reinterpret_cast<const float4*>(sp + col * 8) + 1);
          v[j][0] = a.x; v[j][1] = a.y; v[j][2] = a.z; v[j][3] = a.w;
          v[j][4 % EPV] = b.x; v[j][5 % EPV] = b.y; v[j][6 % EPV] = b.z; v[j][7 % EPV] = b.w;
        } else {
          v[j][0] = __ldg(sp + col);
        }
      }
    }
#pragma unroll
    for (int j = 0; j < J; ++j) {
      const long long col = col0 + j * 256;
      if (col >= w) continue;
      const long long at = row * p.row_units + lo + col;
      if (EPV == 8) {
        uint4 o;
        __nv_bfloat162 h;
        h = __floats2bfloat162_rn(v[j][0], v[j][1]); o.x = *reinterpret_cast<unsigned*>(&h);
        h = __floats2bfloat162_rn(v[j][2], v[j][3]); o.y = *reinterpret_cast<unsigned*>(&h);
        h = __floats2bfloat162_rn(v[j][4 % EPV], v[j][5 % EPV]); o.z = *reinterpret_cast<unsigned*>(&h);
        h = __floats2bfloat162_rn(v[j][6 % EPV], v[j][7 % EPV]); o.w = *reinterpret_cast<unsigned*>(&h);
        for (int q = 0; q < p.n_dst; ++q)
          if (SBP_GUARD(reinterpret_cast<uint4*>(p.dst[q]) + at, 16)) reinterpret_cast<uint4*>(p.dst[q])[at] = o;
      } else {
        const __nv_bfloat16 o = __float2bfloat16_rn(v[j][0]);
        for (int q = 0; q < p.n_dst; ++q)
          if (SBP_GUARD(p.dst[q] + at, 2)) p.dst[q][at] = o;
      }
    }
  }
}

// ------------------------------------------------------------------ host side

static std::atomic<int> g_copy_engine{0};

struct Plan {
  BoxParams p;
  bool pitched;     // some local tensor has a leading dimension: only the tile kernel applies
  int op;
  int vbytes;
  int ntasks;
  long long grid;
};

static int pick_vector_bytes(const BoxParams& p, const sbp_tensor* src, const sbp_tensor* dst, int k) {
  for (int vb = 16; vb > p.esz; vb >>= 1) {
    bool ok = true;
    for (int r = 0; r < k && ok; ++r) {
      ok = ok && reinterpret_cast<uintptr_t>(src->local[r]) % vb == 0;
      ok = ok && reinterpret_cast<uintptr_t>(dst->local[r]) % vb == 0;
      int64_t st, ln;
      if (p.src_b || p.dst_b) {
        split_range(p.Nb, k, r, &st, &ln);
        ok = ok && (st * p.C * p.esz) % vb == 0 && (ln * p.C * p.esz) % vb == 0;
      }
    }
    ok = ok && (p.Nb * p.C * p.esz) % vb == 0;
    for (int r = 0; r < k && ok; ++r)
      ok = (p.src_pitch[r] * p.C * p.esz) % vb == 0 && (p.dst_pitch[r] * p.C * p.esz) % vb == 0;
    if (ok) return vb;
  }
  return p.esz;
}

// Launch as a programmatic dependent of whatever kernel precedes it in the stream: if that
// kernel releases its dependents early (the tile kernel does), this one's CTAs are set up while
// the last CTAs of the other still run, and wait on the device (griddepcontrol.wait, before
// their first access to global memory) until it has finished.  After any other kind of work
// the launch behaves like a plain one.
template <typename V, int OP, int J, int KT>
static void launch_tile(const Plan& pl, cudaStream_t st) {
  SBP_BOUNDS_UPLOAD(st);
  launch_dependent(box_tile_kernel<V, OP, J, KT>, dim3((unsigned)pl.grid), dim3(256), 0, st, pl.p);   // errors are picked up by the caller's cudaGetLastError
}

template <typename V, int OP, int J>
static void launch_k(const Plan& pl, cudaStream_t st) {
  if (OP == OP_COPY) {
    launch_tile<V, OP, J, 0>(pl, st);
    return;
  }
  switch (pl.p.k) {
    case 1: launch_tile<V, OP, J, 1>(pl, st); break;
    case 2: launch_tile<V, OP, J, 2>(pl, st); break;
    case 4: launch_tile<V, OP, J, 4>(pl, st); break;
    case 8: launch_tile<V, OP, J, 8>(pl, st); break;
    default: launch_tile<V, OP, J, 0>(pl, st); break;
  }
}

template <int OP, int J>
static void launch_v(const Plan& pl, cudaStream_t st) {
  switch (pl.vbytes) {
    case 16: launch_k<uint4, OP, J>(pl, st); break;
    case 8: launch_k<uint2, OP, J>(pl, st); break;
    case 4: launch_k<uint32_t, OP, J>(pl, st); break;
    default: launch_k<uint16_t, OP, J>(pl, st); break;
  }
}

// 2-byte vectors cannot carry an fp32 lane, 8-byte+ copies of int64 never use 2/4.
template <int OP, int J>
static void launch_v_f32(const Plan& pl, cudaStream_t st) {
  switch (pl.vbytes) {
    case 16: launch_k<uint4, OP, J>(pl, st); break;
    case 8: launch_k<uint2, OP, J>(pl, st); break;
    default: launch_k<uint32_t, OP, J>(pl, st); break;
  }
}

constexpr int kJCopy = 4;
constexpr int kJReduce = 2;

static sbp_status make_plan(const sbp_tensor* src, const sbp_tensor* dst, int dst_shard, Plan* pl) {
  const int k = placement_k(src);
  const sbp_sig ss = src->sbp[0], ds = dst->sbp[0];
  BoxParams& p = pl->p;
  p = BoxParams{};
  p.k = k;
  p.esz = elem_size(src->dtype);
  p.one_dst = dst_shard >= 0 ? 1 : 0;
  p.dst_shard = dst_shard >= 0 ? dst_shard : 0;
  const bool src_p = ss.kind == SBP_PARTIAL_SUM || ss.kind == SBP_PARTIAL_MAX;
  const bool dst_p = ds.kind == SBP_PARTIAL_SUM || ds.kind == SBP_PARTIAL_MAX;

  pl->op = OP_COPY;
  if (src_p && dst_p) {
    if (ss.kind != ds.kind)
      return fail(SBP_ERR_UNSUPPORTED, "boxing between P(sum) and P(max) has no meaning");
    p.mode = MODE_DIAG;
  } else if (dst_p) {
    if (ds.kind != SBP_PARTIAL_SUM)
      return fail(SBP_ERR_UNSUPPORTED, "boxing S->P(max) / B->P(max) is not implemented (zero is not neutral for max)");
    p.mode = MODE_SCATTER_P;
  } else if (src_p) {
    if (src->dtype == SBP_I64) return fail(SBP_ERR_DTYPE, "partial-value reduction needs F32 or BF16");
    const bool bf = src->dtype == SBP_BF16;
    pl->op = ss.kind == SBP_PARTIAL_SUM ? (bf ? OP_SUM_BF16 : OP_SUM_F32) : (bf ? OP_MAX_BF16 : OP_MAX_F32);
    p.mode = ds.kind == SBP_BROADCAST ? MODE_REDUCE_B : MODE_REDUCE_S;
  } else if (ss.kind == SBP_SPLIT && ds.kind == SBP_BROADCAST) {
    p.mode = MODE_GATHER;
  } else if (ss.kind == SBP_SPLIT && ds.kind == SBP_SPLIT && ss.axis != ds.axis) {
    p.mode = MODE_PAIRS;
  } else {
    p.mode = MODE_DIAG;   // S(i)->S(i), B->S(i), B->B
  }

  // canonical 5-D view
  const int sa = ss.kind == SBP_SPLIT ? ss.axis : -1;
  const int da = ds.kind == SBP_SPLIT ? ds.axis : -1;
  auto prod = [&](int lo, int hi) {
    long long v = 1;
    for (int d = lo; d < hi; ++d) v *= src->shape[d];
    return v;
  };
  p.A = p.Na = p.M = p.Nb = 1;
  const bool pitched = has_ld(src) || has_ld(dst);
  pl->pitched = pitched;
  if (pitched) {
    // Local tensors with a leading dimension: rows are no longer back to back, so the view keeps
    // the two tensor axes apart ([1][n0][1][n1][1]) and every segment is (a piece of) one row.
    if (src->ndim != 2)
      return fail(SBP_ERR_UNSUPPORTED, "local tensors with a leading dimension are boxed as 2-D tensors only");
    if (p.mode == MODE_SCATTER_P || src->dtype != dst->dtype)
      return fail(SBP_ERR_UNSUPPORTED, "boxing to P(sum) and the cast-fused gather take dense local tensors only");
    p.Na = src->shape[0];
    p.Nb = src->shape[1];
    p.C = 1;
    p.src_a = sa == 0;  p.dst_a = da == 0;
    p.src_b = sa == 1;  p.dst_b = da == 1;
    for (int r = 0; r < k; ++r) {
      p.src_pitch[r] = local_pitch(src, r);
      if (dst_shard < 0 || r == dst_shard) p.dst_pitch[r] = local_pitch(dst, r);
    }
    // a reduction reads every source at one offset, a gather / all-reduce writes every replica at one
    for (int r = 1; r < k; ++r) {
      if (src_p && !dst_p && p.src_pitch[r] != p.src_pitch[0])
        return fail(SBP_ERR_UNSUPPORTED, "the partial values of a reduction must share one leading dimension");
      if ((p.mode == MODE_GATHER || p.mode == MODE_REDUCE_B) && dst_shard < 0 && p.dst_pitch[r] != p.dst_pitch[0])
        return fail(SBP_ERR_UNSUPPORTED, "the replicas of a B destination must share one leading dimension");
    }
  } else if (sa < 0 && da < 0) {
    p.C = prod(0, src->ndim);
  } else if (sa >= 0 && sa == da) {
    // Same split on both sides: shard r's local tensor is copied whole, and a local tensor
    // is one contiguous run of len_r * (all other extents) elements on both sides.
    p.Nb = src->shape[sa];
    p.C = prod(0, sa) * prod(sa + 1, src->ndim);
    p.src_b = p.dst_b = 1;
  } else if (sa < 0 || da < 0) {
    // One restricted axis: [1][Na = outer (unrestricted)][1][Nb = n_ax][C].
    const int ax = sa >= 0 ? sa : da;
    p.Na = prod(0, ax);
    p.Nb = src->shape[ax];
    p.C = prod(ax + 1, src->ndim);
    p.src_b = sa >= 0;
    p.dst_b = da >= 0;
  } else {
    const int lo = std::min(sa, da), hi = std::max(sa, da);
    p.A = prod(0, lo);
    p.Na = src->shape[lo];
    p.M = prod(lo + 1, hi);
    p.Nb = src->shape[hi];
    p.C = prod(hi + 1, src->ndim);
    p.src_a = sa == lo;  p.dst_a = da == lo;
    p.src_b = sa == hi;  p.dst_b = da == hi;
  }

  p.a_base = p.Na / k;  p.a_rem = p.Na % k;
  p.b_base = p.Nb / k;  p.b_rem = p.Nb % k;
  for (int r = 0; r < k; ++r) {
    p.src[r] = static_cast<const char*>(src->local[r]);
    p.dst[r] = static_cast<char*>(dst->local[r]);
  }
  pl->vbytes = pick_vector_bytes(p, src, dst, k);
  if (pl->op != OP_COPY && pl->vbytes < 4 && src->dtype == SBP_F32) pl->vbytes = 4;

  // distinct destination buffers for the one-read-many-writes modes
  p.n_dst = 0;
  if ((p.mode == MODE_GATHER || p.mode == MODE_REDUCE_B) && p.one_dst) {
    p.n_dst = 1;
    p.dst[0] = static_cast<char*>(dst->local[dst_shard]);
  } else if (p.mode == MODE_GATHER || p.mode == MODE_REDUCE_B) {
    char* uniq[SBP_MAX_K];
    for (int r = 0; r < k; ++r) {
      bool seen = false;
      for (int q = 0; q < p.n_dst; ++q) seen = seen || uniq[q] == p.dst[r];
      if (!seen) uniq[p.n_dst++] = p.dst[r];
    }
    for (int q = 0; q < p.n_dst; ++q) p.dst[q] = uniq[q];
  }

  // tiling: the largest segment / segment count over shards bounds the per-task grid
  const long long la_max = (p.src_a || p.dst_a) ? (p.Na + k - 1) / k : p.Na;
  const long long lb_max = ((p.src_b || p.dst_b) && p.mode != MODE_SCATTER_P) ? (p.Nb + k - 1) / k : p.Nb;
  const long long nseg_max = p.A * la_max * p.M;
  const long long seg_vecs_max = lb_max * p.C * p.esz / pl->vbytes;
  const int J = pl->op == OP_COPY ? kJCopy : kJReduce;
  const int tile_vecs = J * 256;
  int cv_log2 = 0;
  while ((1 << cv_log2) < tile_vecs && (1LL << cv_log2) < seg_vecs_max) ++cv_log2;
  p.cv_log2 = cv_log2;
  p.rows_per_tile = tile_vecs >> cv_log2;
  p.col_tiles = std::max(1LL, (seg_vecs_max + (1LL << cv_log2) - 1) >> cv_log2);
  const long long row_tiles = std::max(1LL, (nseg_max + p.rows_per_tile - 1) / p.rows_per_tile);
  p.tiles_per_task = p.col_tiles * row_tiles;
  pl->ntasks = p.mode == MODE_PAIRS ? k * k : (p.mode == MODE_REDUCE_B ? 1 : k);
  if (p.one_dst) pl->ntasks = (p.mode == MODE_PAIRS || p.mode == MODE_GATHER) ? k : 1;
  p.ntasks = pl->ntasks;
  pl->grid = p.tiles_per_task * pl->ntasks;
  if (pl->grid > 0x7fffffffLL) return fail(SBP_ERR_UNSUPPORTED, "tensor too large for one launch");
  return SBP_OK;
}

// Bulk-copy engine (defined in boxing_bulk.cu); returns false when it does not apply.
bool launch_bulk_copy(const BoxParams& p, int ntasks, cudaStream_t st);

// dst_shard >= 0: only that destination local tensor is produced, the other dst pointers are not looked at.
static sbp_status check_pair(const sbp_tensor* src, const sbp_tensor* dst, bool need_ptrs, int dst_shard = -1) {
  sbp_status st = check_tensor(src, "src", need_ptrs);
  if (st != SBP_OK) return st;
  st = check_tensor(dst, "dst", need_ptrs && dst_shard < 0);
  if (st != SBP_OK) return st;
  if (dst_shard >= 0) {
    if (dst->pdims != 1 || src->pdims != 1) return fail(SBP_ERR_UNSUPPORTED, "one-shard boxing needs one-axis placements");
    if (dst_shard >= placement_k(dst)) return fail(SBP_ERR_INVALID_ARG, "dst_shard %d outside the placement of %d", dst_shard, placement_k(dst));
    const void* ptr = dst->local[dst_shard];
    if (!ptr && local_numel(dst, dst_shard) > 0) return fail(SBP_ERR_INVALID_ARG, "dst local tensor %d is null", dst_shard);
    if (reinterpret_cast<uintptr_t>(ptr) % elem_size(dst->dtype) != 0) return fail(SBP_ERR_ALIGNMENT, "dst local tensor %d is misaligned", dst_shard);
  }
  if (src->ndim != dst->ndim) return fail(SBP_ERR_SHAPE, "src and dst differ in rank");
  for (int d = 0; d < src->ndim; ++d)
    if (src->shape[d] != dst->shape[d]) return fail(SBP_ERR_SHAPE, "src and dst differ on axis %d", d);
  const bool cast_gather = src->dtype == SBP_F32 && dst->dtype == SBP_BF16 && src->sbp[0].kind == SBP_SPLIT &&
                           dst->sbp[0].kind == SBP_BROADCAST;
  if (src->dtype != dst->dtype && !cast_gather)
    return fail(SBP_ERR_DTYPE, "src and dst differ in dtype (only S(i) -> B may cast, F32 -> BF16)");
  if (placement_k(src) != placement_k(dst)) {
    if (src->pdims != 1 || dst->pdims != 1)
      return fail(SBP_ERR_UNSUPPORTED, "boxing between different placements needs one-axis placements on both sides");
    if (src->dtype != dst->dtype)
      return fail(SBP_ERR_UNSUPPORTED, "the cast-fused gather needs src and dst on the same placement");
  }
  return SBP_OK;
}

// Different shard counts on the two sides (defined in boxing_disjoint.cu).
sbp_status boxing_disjoint(const sbp_tensor* src, sbp_tensor* dst, int dst_shard, cudaStream_t stream, bool dry);

}  // namespace sbp

using namespace sbp;

extern "C" {

void sbp_boxing_set_copy_engine(int32_t engine) { g_copy_engine.store(engine); }

// Two-axis placements (Section 3.3, multi-dimensional SBP): device (i, j) of a k0 x k1
// placement holds piece j, under sbp[1], of piece i, under sbp[0], of the global tensor.  A
// boxing op that changes the signature of ONE placement axis is a set of independent one-axis
// boxing ops: inside every group i when axis 1 changes, across the groups for every j when
// axis 0 changes (valid when the unchanged axis-1 mapping commutes with the change).
static bool is_partial(sbp_sig s) { return s.kind == SBP_PARTIAL_SUM || s.kind == SBP_PARTIAL_MAX; }

// dry: every check is made (descriptors, signature pair, sizes) and nothing is launched.
static sbp_status boxing_one_axis(const sbp_tensor* src, sbp_tensor* dst, int dst_shard, void* cuda_stream, bool dry);

static sbp_status boxing_2d(const sbp_tensor* src, sbp_tensor* dst, void* cuda_stream, bool dry) {
  sbp_status st = check_tensor_nd(src, "src", true);
  if (st != SBP_OK) return st;
  st = check_tensor_nd(dst, "dst", true);
  if (st != SBP_OK) return st;
  st = refuse_ld(src, "src", "boxing on a two-axis placement");
  if (st != SBP_OK) return st;
  st = refuse_ld(dst, "dst", "boxing on a two-axis placement");
  if (st != SBP_OK) return st;
  if (src->pdims != 2 || dst->pdims != 2 || src->pshape[0] != dst->pshape[0] || src->pshape[1] != dst->pshape[1])
    return fail(SBP_ERR_INVALID_ARG, "src and dst must live on the same two-axis placement");
  if (src->ndim != dst->ndim) return fail(SBP_ERR_SHAPE, "src and dst differ in rank");
  for (int d = 0; d < src->ndim; ++d)
    if (src->shape[d] != dst->shape[d]) return fail(SBP_ERR_SHAPE, "src and dst differ on axis %d", d);
  if (src->dtype != dst->dtype) return fail(SBP_ERR_DTYPE, "src and dst differ in dtype");
  const int k0 = src->pshape[0], k1 = src->pshape[1];
  const bool ch0 = !same_sig(src->sbp[0], dst->sbp[0]), ch1 = !same_sig(src->sbp[1], dst->sbp[1]);
  if (ch0 && ch1)
    return fail(SBP_ERR_UNSUPPORTED, "change one placement axis per boxing call (two calls for both)");

  sbp_tensor s1 = *src, d1 = *dst;
  s1.pdims = d1.pdims = 1;
  s1.pshape[1] = d1.pshape[1] = 1;
  for (int r = 0; r < SBP_MAX_K; ++r) s1.local_ld[r] = d1.local_ld[r] = 0;
  if (!ch0) {
    // axis 1 changes (or nothing does): one boxing op inside each group, on the group's tensor
    s1.pshape[0] = d1.pshape[0] = k1;
    s1.sbp[0] = src->sbp[1];
    d1.sbp[0] = dst->sbp[1];
    for (int i = 0; i < k0; ++i) {
      if (src->sbp[0].kind == SBP_SPLIT) {
        int64_t start, len;
        split_range(src->shape[src->sbp[0].axis], k0, i, &start, &len);
        s1.shape[src->sbp[0].axis] = d1.shape[src->sbp[0].axis] = len;
      }
      for (int j = 0; j < k1; ++j) {
        s1.local[j] = src->local[i * k1 + j];
        d1.local[j] = dst->local[i * k1 + j];
      }
      st = boxing_one_axis(&s1, &d1, -1, cuda_stream, dry);
      if (st != SBP_OK) return st;
    }
    return SBP_OK;
  }
  // axis 0 changes, axis 1 keeps signature c
  const sbp_sig c = src->sbp[1];
  if (c.kind == SBP_SPLIT) {
    if ((src->sbp[0].kind == SBP_SPLIT && src->sbp[0].axis == c.axis) ||
        (dst->sbp[0].kind == SBP_SPLIT && dst->sbp[0].axis == c.axis))
      return fail(SBP_ERR_UNSUPPORTED, "axis 0 cannot be re-boxed along the tensor axis that axis 1 splits");
  } else if (is_partial(c)) {
    if (is_partial(src->sbp[0]) && src->sbp[0].kind != c.kind)
      return fail(SBP_ERR_UNSUPPORTED, "a max over one placement axis does not commute with a sum over the other");
  }
  s1.pshape[0] = d1.pshape[0] = k0;
  s1.sbp[0] = src->sbp[0];
  d1.sbp[0] = dst->sbp[0];
  for (int j = 0; j < k1; ++j) {
    if (c.kind == SBP_SPLIT) {
      int64_t start, len;
      split_range(src->shape[c.axis], k1, j, &start, &len);
      s1.shape[c.axis] = d1.shape[c.axis] = len;
    }
    for (int i = 0; i < k0; ++i) {
      s1.local[i] = src->local[i * k1 + j];
      d1.local[i] = dst->local[i * k1 + j];
    }
    st = boxing_one_axis(&s1, &d1, -1, cuda_stream, dry);
    if (st != SBP_OK) return st;
  }
  return SBP_OK;
}

static sbp_status boxing_one_axis(const sbp_tensor* src, sbp_tensor* dst, int dst_shard, void* cuda_stream, bool dry) {
  sbp_status st = check_pair(src, dst, true, dst_shard);
  if (st != SBP_OK) return st;
  if (placement_k(src) != placement_k(dst))
    return boxing_disjoint(src, dst, dst_shard, static_cast<cudaStream_t>(cuda_stream), dry);
  Plan pl;
  st = make_plan(src, dst, dst_shard, &pl);
  if (st != SBP_OK) return st;
  if (dry || numel(src) == 0) return SBP_OK;
  cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
  SBP_BOUNDS_RESET();
  SBP_BOUNDS_TENSOR(src);
  if (dst_shard >= 0) SBP_BOUNDS_SHARD(dst, dst_shard);
  else SBP_BOUNDS_TENSOR(dst);

  bool done = false;
  if (src->dtype != dst->dtype) {   // S(i) -> B with the fp32 -> bf16 cast folded in
    const BoxParams& b = pl.p;      // planned with the source element size; only the view is used
    GatherCastParams gp{};
    gp.nrows = b.A * b.Na * b.M;
    bool vec = (b.Nb * b.C) % 8 == 0;
    for (int r = 0; r < b.k && vec; ++r) {
      int64_t start, len;
      split_range(b.Nb, b.k, r, &start, &len);
      vec = (start * b.C) % 8 == 0 && (len * b.C) % 8 == 0 && reinterpret_cast<uintptr_t>(src->local[r]) % 16 == 0 &&
            reinterpret_cast<uintptr_t>(dst->local[r]) % 16 == 0;
    }
    const int epv = vec ? 8 : 1;
    gp.row_units = b.Nb * b.C / epv;
    for (int r = 0; r < b.k; ++r) {
      int64_t start, len;
      split_range(b.Nb, b.k, r, &start, &len);
      gp.src[r] = static_cast<const float*>(src->local[r]);
      gp.own_lo[r] = start * b.C / epv;
      gp.own_hi[r] = (start + len) * b.C / epv;
    }
    gp.n_dst = b.n_dst;
    for (int q = 0; q < b.n_dst; ++q) gp.dst[q] = reinterpret_cast<__nv_bfloat16*>(b.dst[q]);
    dim3 grid(148 * 4, (unsigned)b.k);
    SBP_BOUNDS_UPLOAD(stream);
    if (vec) launch_dependent(box_gather_cast_kernel<8>, grid, dim3(256), 0, stream, gp);
    else launch_dependent(box_gather_cast_kernel<1>, grid, dim3(256), 0, stream, gp);
    done = true;
  } else if (pl.p.mode == MODE_SCATTER_P) {
    const BoxParams& b = pl.p;
    ScatterParams sp{};
    sp.nrows = b.A * b.Na * b.M;
    sp.row_vecs = b.Nb * b.C * b.esz / pl.vbytes;
    sp.chunks_per_row = (sp.row_vecs + 256 * kScatterJ - 1) / (256 * kScatterJ);
    sp.total_chunks = sp.nrows * sp.chunks_per_row;
    for (int d = 0; d < b.k; ++d) {
      sp.src[d] = b.src[d];
      sp.dst[d] = b.dst[d];
      if (b.src_b) {
        int64_t start, len;
        split_range(b.Nb, b.k, d, &start, &len);
        sp.own_lo[d] = start * b.C * b.esz / pl.vbytes;
        sp.own_hi[d] = (start + len) * b.C * b.esz / pl.vbytes;
      } else {
        sp.own_lo[d] = 0;
        sp.own_hi[d] = d == 0 ? sp.row_vecs : 0;
      }
    }
    const int ny = b.one_dst ? 1 : b.k;
    sp.d0 = b.one_dst ? b.dst_shard : 0;
    switch (pl.vbytes) {
      case 16: launch_scatter_v<uint4>(sp, ny, stream); break;
      case 8: launch_scatter_v<uint2>(sp, ny, stream); break;
      case 4: launch_scatter_v<uint32_t>(sp, ny, stream); break;
      default: launch_scatter_v<uint16_t>(sp, ny, stream); break;
    }
    done = true;
  }
  // Default choice, from measurement on B200: the load/store kernel (5.6 TB/s on 128 MiB
  // re-layouts, 6.5 TB/s on 512 MiB ones) is ahead of the bulk engine (5.2 / 5.9 TB/s), whose
  // issuing warp spends 600-800 clocks on each bulk-copy instruction; the bulk engine stays
  // available on request.
  const int engine = g_copy_engine.load();
  const bool want_bulk = engine == 2;
  if (!done && pl.op == OP_COPY && want_bulk && pl.vbytes == 16 && !pl.pitched)
    done = launch_bulk_copy(pl.p, pl.ntasks, stream);
  if (!done) {
    switch (pl.op) {
      case OP_COPY: launch_v<OP_COPY, kJCopy>(pl, stream); break;
      case OP_SUM_F32: launch_v_f32<OP_SUM_F32, kJReduce>(pl, stream); break;
      case OP_MAX_F32: launch_v_f32<OP_MAX_F32, kJReduce>(pl, stream); break;
      case OP_SUM_BF16: launch_v<OP_SUM_BF16, kJReduce>(pl, stream); break;
      case OP_MAX_BF16: launch_v<OP_MAX_BF16, kJReduce>(pl, stream); break;
    }
  }
  cudaError_t e = cudaGetLastError();
  if (e != cudaSuccess) return cuda_fail(e, "boxing launch");
  count_launch();
  return SBP_OK;
}

sbp_status sbp_boxing(const sbp_tensor* src, sbp_tensor* dst, void* cuda_stream) {
  SBP_RANGE("sbp_boxing");
  if (src && dst && (src->pdims == 2 || dst->pdims == 2)) {
    // every group's one-axis op is checked before the first of them is launched
    sbp_status st = boxing_2d(src, dst, cuda_stream, true);
    if (st != SBP_OK) return st;
    return boxing_2d(src, dst, cuda_stream, false);
  }
  return boxing_one_axis(src, dst, -1, cuda_stream, false);
}

sbp_status sbp_boxing_shard(const sbp_tensor* src, sbp_tensor* dst, int32_t dst_shard, void* cuda_stream) {
  SBP_RANGE("sbp_boxing_shard");
  if (dst_shard < 0) return fail(SBP_ERR_INVALID_ARG, "dst_shard %d is negative", dst_shard);
  return boxing_one_axis(src, dst, dst_shard, cuda_stream, false);
}

static size_t align256(size_t v) { return (v + 255) & ~size_t(255); }

size_t sbp_boxing_host_workspace_bytes(const sbp_tensor* src_host, const sbp_tensor* dst_host) {
  if (check_pair(src_host, dst_host, false) != SBP_OK) return 0;
  const int ks = placement_k(src_host), kd = placement_k(dst_host);
  size_t total = 0;
  for (int r = 0; r < ks; ++r) total += align256((size_t)local_numel(src_host, r) * elem_size(src_host->dtype));
  for (int r = 0; r < kd; ++r) total += align256((size_t)local_numel(dst_host, r) * elem_size(dst_host->dtype));
  return total;
}

// B -> S(axis) on equal one-axis placements reads, of source replica r, only the block that becomes
// destination shard r: the host path copies that block alone.  Geometry of replica r's block as a
// pitched 2-D copy: `outer` rows of `width` bytes, `pitch` bytes apart, starting at byte `offset`.
struct HostBlock {
  size_t offset, pitch, width, outer;
};

static bool host_copy_is_diagonal(const sbp_tensor* src, const sbp_tensor* dst) {
  return src->pdims <= 1 && dst->pdims <= 1 && placement_k(src) == placement_k(dst) && src->dtype == dst->dtype &&
         src->sbp[0].kind == SBP_BROADCAST && dst->sbp[0].kind == SBP_SPLIT;
}

static HostBlock host_diagonal_block(const sbp_tensor* src, int axis, int r) {
  int64_t start = 0, len = 0;
  split_range(src->shape[axis], placement_k(src), r, &start, &len);
  size_t outer = 1, inner = (size_t)elem_size(src->dtype);
  for (int d = 0; d < axis; ++d) outer *= (size_t)src->shape[d];
  for (int d = axis + 1; d < src->ndim; ++d) inner *= (size_t)src->shape[d];
  return HostBlock{(size_t)start * inner, (size_t)src->shape[axis] * inner, (size_t)len * inner, outer};
}

// One source, n destinations: the source crosses to the device once and every transform reads it
// there.  Only the diagonal blocks are sent when EVERY destination is a B -> S(axis) of the same
// axis on an equal placement.
static bool host_multi_is_diagonal(const sbp_tensor* src, const sbp_tensor* dsts, int n) {
  for (int i = 0; i < n; ++i)
    if (!host_copy_is_diagonal(src, &dsts[i]) || dsts[i].sbp[0].axis != dsts[0].sbp[0].axis) return false;
  return n > 0;
}

static sbp_status host_multi_check(const sbp_tensor* src, const sbp_tensor* dsts, int n, bool need_pointers) {
  if (!src || !dsts) return fail(SBP_ERR_INVALID_ARG, "null descriptor");
  if (n < 1 || n > 64) return fail(SBP_ERR_INVALID_ARG, "between 1 and 64 destinations, not %d", n);
  for (int i = 0; i < n; ++i) {
    sbp_status st = check_pair(src, &dsts[i], need_pointers);
    if (st != SBP_OK) return st;
  }
  return SBP_OK;
}

static uint64_t host_source_bytes(const sbp_tensor* src, const sbp_tensor* dsts, int n) {
  const bool diag = host_multi_is_diagonal(src, dsts, n);
  uint64_t in = 0;
  for (int r = 0; r < placement_k(src); ++r) {
    if (diag) {
      const HostBlock b = host_diagonal_block(src, dsts[0].sbp[0].axis, r);
      in += (uint64_t)b.width * b.outer;
    } else {
      in += (uint64_t)local_numel(src, r) * elem_size(src->dtype);
    }
  }
  return in;
}

static uint64_t host_result_bytes(const sbp_tensor* dst) {
  uint64_t out = 0;
  for (int r = 0; r < placement_k(dst); ++r) {
    bool dup = false;
    for (int q = 0; q < r; ++q) dup = dup || dst->local[q] == dst->local[r];
    if (!dup) out += (uint64_t)local_numel(dst, r) * elem_size(dst->dtype);
  }
  return out;
}

sbp_status sbp_boxing_host_multi_copy_bytes(const sbp_tensor* src_host, const sbp_tensor* dst_hosts, int32_t n, uint64_t* h2d,
                                            uint64_t* d2h) {
  sbp_status st = host_multi_check(src_host, dst_hosts, n, false);
  if (st != SBP_OK) return st;
  uint64_t out = 0;
  for (int i = 0; i < n; ++i) out += host_result_bytes(&dst_hosts[i]);
  if (h2d) *h2d = host_source_bytes(src_host, dst_hosts, n);
  if (d2h) *d2h = out;
  return SBP_OK;
}

sbp_status sbp_boxing_host_copy_bytes(const sbp_tensor* src_host, const sbp_tensor* dst_host, uint64_t* h2d, uint64_t* d2h) {
  return sbp_boxing_host_multi_copy_bytes(src_host, dst_host, 1, h2d, d2h);
}

size_t sbp_boxing_host_multi_workspace_bytes(const sbp_tensor* src_host, const sbp_tensor* dst_hosts, int32_t n) {
  if (host_multi_check(src_host, dst_hosts, n, false) != SBP_OK) return 0;
  size_t total = 0;
  for (int r = 0; r < placement_k(src_host); ++r) total += align256((size_t)local_numel(src_host, r) * elem_size(src_host->dtype));
  for (int i = 0; i < n; ++i)
    for (int r = 0; r < placement_k(&dst_hosts[i]); ++r)
      total += align256((size_t)local_numel(&dst_hosts[i], r) * elem_size(dst_hosts[i].dtype));
  return total;
}

sbp_status sbp_boxing_host_multi(const sbp_tensor* src_host, sbp_tensor* dst_hosts, int32_t n, void* dev_ws, size_t dev_ws_bytes,
                                 void* cuda_stream) {
  SBP_RANGE("sbp_boxing_host");
  sbp_status st = host_multi_check(src_host, dst_hosts, n, true);
  if (st != SBP_OK) return st;
  st = refuse_ld(src_host, "src_host", "sbp_boxing_host");
  if (st != SBP_OK) return st;
  for (int i = 0; i < n; ++i) {
    st = refuse_ld(&dst_hosts[i], "dst_host", "sbp_boxing_host");
    if (st != SBP_OK) return st;
  }
  const size_t need = sbp_boxing_host_multi_workspace_bytes(src_host, dst_hosts, n);
  if (need > 0 && (!dev_ws || dev_ws_bytes < need))
    return fail(SBP_ERR_WORKSPACE, "device workspace of %zu bytes needed, %zu given", need, dev_ws_bytes);
  if (reinterpret_cast<uintptr_t>(dev_ws) % 256 != 0)
    return fail(SBP_ERR_ALIGNMENT, "device workspace must be 256-byte aligned");
  const int ks = placement_k(src_host);
  cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
  sbp_tensor s = *src_host;
  static thread_local sbp_tensor d[64];
  char* cur = static_cast<char*>(dev_ws);
  const int esz = elem_size(src_host->dtype);
  for (int r = 0; r < ks; ++r) {
    s.local[r] = cur;
    cur += align256((size_t)local_numel(src_host, r) * esz);
  }
  for (int i = 0; i < n; ++i) {
    d[i] = dst_hosts[i];
    // Destination replicas that alias on the host alias on the device as well.
    for (int r = 0; r < placement_k(&d[i]); ++r) {
      d[i].local[r] = nullptr;
      for (int q = 0; q < r; ++q)
        if (dst_hosts[i].local[q] == dst_hosts[i].local[r]) d[i].local[r] = d[i].local[q];
      if (!d[i].local[r]) {
        d[i].local[r] = cur;
        cur += align256((size_t)local_numel(&dst_hosts[i], r) * elem_size(dst_hosts[i].dtype));
      }
    }
  }
  // every transform's own refusals (signature pair, sizes) come before the first copy is enqueued
  for (int i = 0; i < n; ++i) {
    if (s.pdims == 2 || d[i].pdims == 2) st = boxing_2d(&s, &d[i], cuda_stream, true);
    else st = boxing_one_axis(&s, &d[i], -1, cuda_stream, true);
    if (st != SBP_OK) return st;
  }
  const bool diag = host_multi_is_diagonal(src_host, dst_hosts, n);
  for (int r = 0; r < ks; ++r) {
    if (diag) {
      // the rest of this replica's device copy stays unwritten: the transforms never read it
      const HostBlock b = host_diagonal_block(src_host, dst_hosts[0].sbp[0].axis, r);
      if (b.width && b.outer)
        SBP_CUDA_TRY(cudaMemcpy2DAsync(static_cast<char*>(s.local[r]) + b.offset, b.pitch,
                                       static_cast<const char*>(src_host->local[r]) + b.offset, b.pitch, b.width, b.outer,
                                       cudaMemcpyHostToDevice, stream));
      continue;
    }
    const size_t bytes = (size_t)local_numel(src_host, r) * esz;
    if (bytes) SBP_CUDA_TRY(cudaMemcpyAsync(s.local[r], src_host->local[r], bytes, cudaMemcpyHostToDevice, stream));
  }
  for (int i = 0; i < n; ++i) {
    st = sbp_boxing(&s, &d[i], cuda_stream);
    if (st != SBP_OK) return st;
    for (int r = 0; r < placement_k(&d[i]); ++r) {
      bool dup = false;
      for (int q = 0; q < r; ++q) dup = dup || dst_hosts[i].local[q] == dst_hosts[i].local[r];
      const size_t bytes = (size_t)local_numel(&dst_hosts[i], r) * elem_size(dst_hosts[i].dtype);
      if (!dup && bytes)
        SBP_CUDA_TRY(cudaMemcpyAsync(dst_hosts[i].local[r], d[i].local[r], bytes, cudaMemcpyDeviceToHost, stream));
    }
  }
  return SBP_OK;
}

sbp_status sbp_boxing_host(const sbp_tensor* src_host, sbp_tensor* dst_host, void* dev_ws, size_t dev_ws_bytes,
                           void* cuda_stream) {
  return sbp_boxing_host_multi(src_host, dst_host, 1, dev_ws, dev_ws_bytes, cuda_stream);
}

}  // extern "C"
