// Boxing between two DIFFERENT placements (Section 3.2, Table 2, column "disjoint"): the source
// lives on ks logical shards, the destination on kd others, ks != kd in general.
//
// The logical tensor is viewed as [A][Na][M][Nb][C] exactly as in the same-placement kernels,
// but here either side may restrict either of the two axes, both sides may restrict the SAME
// axis (S(i) on ks shards -> S(i) on kd shards), and the two sides split with different shard
// counts.  A task is one (source shard s, destination shard d) pair; what it moves is the
// intersection of the two shards' index ranges on each restricted axis.  One CTA moves one tile
// of J*256 vectors of one task, all loads before the stores.
//
//   copy      S -> S (any axes), B -> S (replica d mod ks serves shard d), S -> B and B -> B
//             (one read, one write per distinct replica), S -> P(sum) (zero fill by one kernel first, then
//             piece d of the kd-way split of the source's axis lands in place in partial d)
//   reduce    P -> S / B (all ks partials in rank order, fp32 accumulator, one rounding),
//             P -> P (partial r goes to destination r mod kd, which adds what it gets in
//             ascending r; a destination that gets nothing is zero)
#include <algorithm>

#include "bounds_check.h"
#include "boxing_arith.h"
#include "sbp_internal.h"

namespace sbp {

enum DisjointMode : int {
  DJ_PAIRS = 0,      // task t: (s, d) from the pair table, or s = t / kd, d = t % kd
  DJ_FROM_REPLICA,   // task t: d = t, s = t % ks
  DJ_TO_ALL,         // task t: s = t, every distinct destination replica
  DJ_REDUCE,         // task t: d = t, sources red_first(t), += red_stride, ...
  DJ_REDUCE_ALL      // one task: all sources, every distinct destination replica
};

constexpr int kMaxPairs = 2 * SBP_MAX_K;

struct DisjointParams {
  const char* src[SBP_MAX_K];
  char* dst[SBP_MAX_K];
  long long A, Na, M, Nb, C;
  long long tiles_per_task, col_tiles;
  int ks, kd, esz, mode;
  int src_a, src_b, dst_a, dst_b;   // which side's split restricts axis Na / Nb (both may)
  int dst_full;                     // destination restricts by its split but is addressed at full shape
  int n_dst;                        // distinct replicas written by one task (DJ_TO_ALL, DJ_REDUCE_ALL)
  int red_by_dst;                   // DJ_REDUCE: sources d, d + kd, ... instead of 0 .. ks-1
  int n_pairs;                      // > 0: DJ_PAIRS tasks listed in pair_s / pair_d
  int one_dst, dst_shard;           // one_dst: only the tasks that produce destination shard dst_shard
  int cv_log2, rows_per_tile, ntasks;
  unsigned char pair_s[kMaxPairs], pair_d[kMaxPairs];
  // quotient and remainder of each axis by each side's shard count: the balanced split without a division
  long long a_base_s, a_rem_s, a_base_d, a_rem_d, b_base_s, b_rem_s, b_base_d, b_rem_d;
};

struct AxisCut {
  long long len;        // length of the intersection (<= 0: empty)
  long long n_s, off_s; // extent of the axis in the source local tensor, start of the cut inside it
  long long n_d, off_d; // same for the destination
};

__device__ __forceinline__ AxisCut cut_axis(long long n, bool by_src, long long base_s, long long rem_s, int s, bool by_dst,
                                            long long base_d, long long rem_d, int d, bool dst_full) {
  long long lo = 0, hi = n;
  AxisCut c;
  c.n_s = n; c.n_d = n;
  long long start_s = 0, start_d = 0;
  if (by_src) {
    const long long ln = base_s + (s < rem_s ? 1 : 0), st = s * base_s + (s < rem_s ? s : rem_s);
    lo = st; hi = st + ln;
    start_s = st; c.n_s = ln;
  }
  if (by_dst) {
    const long long ln = base_d + (d < rem_d ? 1 : 0), st = d * base_d + (d < rem_d ? d : rem_d);
    lo = lo > st ? lo : st;
    hi = hi < st + ln ? hi : st + ln;
    if (!dst_full) { start_d = st; c.n_d = ln; }
  }
  c.len = hi - lo;
  c.off_s = lo - start_s;
  c.off_d = lo - start_d;
  return c;
}

template <typename V, int OP>
__global__ void __launch_bounds__(256, OP == OP_COPY ? 4 : 3) box_disjoint_kernel(const __grid_constant__ DisjointParams p) {
  constexpr int J = OP == OP_COPY ? 4 : 2;
  SBP_PDL_RELEASE();                             // the next kernel of the stream may be set up from here on
  const unsigned u = blockIdx.x;                 // the grid is below 2^31 tiles: 32-bit arithmetic
  const unsigned rem = u / (unsigned)p.ntasks;   // task index varies fastest
  const int t = (int)(u - rem * (unsigned)p.ntasks);
  const unsigned row_tile_u = rem / (unsigned)p.col_tiles;
  const long long row_tile = row_tile_u;
  const long long col_tile = rem - row_tile_u * (unsigned)p.col_tiles;

  int s = 0, d = 0;
  switch (p.mode) {
    case DJ_PAIRS:
      if (p.n_pairs > 0) { s = p.pair_s[t]; d = p.pair_d[t]; }
      else if (p.one_dst) { s = t; d = p.dst_shard; }
      else { s = t / p.kd; d = t - s * p.kd; }
      break;
    case DJ_FROM_REPLICA: d = p.one_dst ? p.dst_shard : t; s = d % p.ks; break;
    case DJ_TO_ALL: s = t; break;
    case DJ_REDUCE: d = p.one_dst ? p.dst_shard : t; break;
    default: break;
  }

  const AxisCut ca = cut_axis(p.Na, p.src_a, p.a_base_s, p.a_rem_s, s, p.dst_a, p.a_base_d, p.a_rem_d, d, p.dst_full);
  const AxisCut cb = cut_axis(p.Nb, p.src_b, p.b_base_s, p.b_rem_s, s, p.dst_b, p.b_base_d, p.b_rem_d, d, p.dst_full);
  if (ca.len <= 0 || cb.len <= 0) return;
  const long long nseg = p.A * ca.len * p.M;
  const long long cs = p.C * p.esz;              // bytes per unit step of the Nb axis
  const long long seg_vecs = cb.len * cs / (long long)sizeof(V);
  const long long seg0 = row_tile * p.rows_per_tile;
  const long long col0 = col_tile << p.cv_log2;
  if (seg0 >= nseg || col0 >= seg_vecs) return;
  const bool flat = (p.A == 1 && p.M == 1);

  long long so[J], dofs[J];
  bool ok[J];
#pragma unroll
  for (int j = 0; j < J; ++j) {
    const int f = threadIdx.x + j * 256;
    const long long seg = seg0 + (f >> p.cv_log2);
    const long long col = col0 + (f & ((1 << p.cv_log2) - 1));
    ok[j] = seg < nseg && col < seg_vecs;
    long long x = 0, ia = seg, m = 0;
    if (!flat) {
      const long long q = seg / p.M;
      m = seg - q * p.M;
      x = q / ca.len;
      ia = q - x * ca.len;
    }
    so[j] = ((((x * ca.n_s + ca.off_s + ia) * p.M + m) * cb.n_s + cb.off_s) * cs) / (long long)sizeof(V) + col;
    dofs[j] = ((((x * ca.n_d + ca.off_d + ia) * p.M + m) * cb.n_d + cb.off_d) * cs) / (long long)sizeof(V) + col;
  }

  SBP_PDL_WAIT();                                // the kernel before this one has finished

  V val[J];
  if constexpr (OP == OP_COPY) {
    const V* sp = reinterpret_cast<const V*>(p.src[s]);
#pragma unroll
    for (int j = 0; j < J; ++j)
      if (ok[j] && SBP_GUARD(sp + so[j], sizeof(V))) val[j] = ld_stream(sp + so[j]);
  } else {
    using L = typename Lanes<OP, V>::type;
    int first = 0, stride = 1, count = p.ks;
    if (p.mode == DJ_REDUCE && p.red_by_dst) {
      first = d;
      stride = p.kd;
      count = d < p.ks ? (p.ks - d + p.kd - 1) / p.kd : 0;
    }
    // sources in ascending order, four at a time so that 4 * J loads are in flight per thread
    constexpr int kBatch = 4;
    L acc[J];
#pragma unroll
    for (int j = 0; j < J; ++j) val[j] = V{};
    for (int base = 0; base < count; base += kBatch) {
      V raw[J][kBatch];
#pragma unroll
      for (int j = 0; j < J; ++j)
#pragma unroll
        for (int i = 0; i < kBatch; ++i)
          if (ok[j] && base + i < count &&
              SBP_GUARD(reinterpret_cast<const V*>(p.src[first + (base + i) * stride]) + so[j], sizeof(V)))
            raw[j][i] = ld_stream(reinterpret_cast<const V*>(p.src[first + (base + i) * stride]) + so[j]);
#pragma unroll
      for (int j = 0; j < J; ++j)
#pragma unroll
        for (int i = 0; i < kBatch; ++i)
          if (ok[j] && base + i < count) {
            L x;
            x.load(raw[j][i]);
            if (base + i == 0) acc[j] = x;
            else combine<OP>(acc[j], x);
          }
    }
    if (count > 0) {
#pragma unroll
      for (int j = 0; j < J; ++j)
        if (ok[j]) val[j] = acc[j].store();
    }
  }

  if (p.mode == DJ_TO_ALL || p.mode == DJ_REDUCE_ALL) {
    for (int r = 0; r < p.n_dst; ++r) {
      V* dp = reinterpret_cast<V*>(p.dst[r]);
#pragma unroll
      for (int j = 0; j < J; ++j)
        if (ok[j] && SBP_GUARD(dp + dofs[j], sizeof(V))) dp[dofs[j]] = val[j];
    }
  } else {
    V* dp = reinterpret_cast<V*>(p.dst[d]);
#pragma unroll
    for (int j = 0; j < J; ++j)
      if (ok[j] && SBP_GUARD(dp + dofs[j], sizeof(V))) dp[dofs[j]] = val[j];
  }
}

// Clears n destination buffers of `bytes` bytes each (16-byte aligned, a multiple of 16 long):
// the starting value of P(sum) partials that then receive their piece.
struct ZeroParams {
  char* dst[SBP_MAX_K];
  long long bytes;
  int n;
};

__global__ void __launch_bounds__(256) box_zero_kernel(const __grid_constant__ ZeroParams z) {
  SBP_PDL_RELEASE();
  SBP_PDL_WAIT();
  uint4* d = reinterpret_cast<uint4*>(z.dst[blockIdx.y]);
  const long long n = z.bytes / 16;
  const uint4 zero = make_uint4(0u, 0u, 0u, 0u);
  for (long long i = (long long)blockIdx.x * 256 + threadIdx.x; i < n; i += (long long)gridDim.x * 256)
    if (SBP_GUARD(d + i, 16)) d[i] = zero;
}

template <int OP>
static void launch_disjoint(const DisjointParams& p, int vbytes, long long grid, cudaStream_t st) {
  SBP_BOUNDS_UPLOAD(st);
  const dim3 g((unsigned)grid), b(256);
  switch (vbytes) {
    case 16: launch_dependent(box_disjoint_kernel<uint4, OP>, g, b, 0, st, p); break;
    case 8: launch_dependent(box_disjoint_kernel<uint2, OP>, g, b, 0, st, p); break;
    case 4: launch_dependent(box_disjoint_kernel<uint32_t, OP>, g, b, 0, st, p); break;
    default:
      // a 2-byte vector cannot carry an fp32 lane; the fp32 reductions never get here
      if constexpr (OP != OP_SUM_F32 && OP != OP_MAX_F32) launch_dependent(box_disjoint_kernel<uint16_t, OP>, g, b, 0, st, p);
      break;
  }
}

// src and dst have been validated by the caller (same logical shape and dtype, one-axis
// placements, pointers present); ks != kd is the expected case but not required.
// dst_shard >= 0: only that destination local tensor is produced (the other dst pointers may be null).
// dry: every check is made and nothing is launched.
sbp_status boxing_disjoint(const sbp_tensor* src, sbp_tensor* dst, int dst_shard, cudaStream_t stream, bool dry) {
  const int ks = placement_k(src), kd = placement_k(dst);
  const sbp_sig ss = src->sbp[0], ds = dst->sbp[0];
  const bool src_p = ss.kind == SBP_PARTIAL_SUM || ss.kind == SBP_PARTIAL_MAX;
  const bool dst_p = ds.kind == SBP_PARTIAL_SUM || ds.kind == SBP_PARTIAL_MAX;
  const int esz = elem_size(src->dtype);
  if (src->dtype != dst->dtype)
    return fail(SBP_ERR_UNSUPPORTED, "the cast-fused gather needs src and dst on the same placement");
  sbp_status ld_st = refuse_ld(src, "src", "boxing between different placements");
  if (ld_st == SBP_OK) ld_st = refuse_ld(dst, "dst", "boxing between different placements");
  if (ld_st != SBP_OK) return ld_st;

  DisjointParams p{};
  p.ks = ks; p.kd = kd; p.esz = esz;
  p.one_dst = dst_shard >= 0 ? 1 : 0;
  p.dst_shard = dst_shard >= 0 ? dst_shard : 0;
  int op = OP_COPY;
  bool zero_first = false;
  if (src_p) {
    if (dst_p && ss.kind != ds.kind) return fail(SBP_ERR_UNSUPPORTED, "boxing between P(sum) and P(max) has no meaning");
    if (src->dtype == SBP_I64) return fail(SBP_ERR_DTYPE, "partial-value reduction needs F32 or BF16");
    if (dst_p && ss.kind == SBP_PARTIAL_MAX && kd > ks)
      return fail(SBP_ERR_UNSUPPORTED, "P(max) onto more shards than there are partials is undefined (zero is not neutral for max)");
    const bool bf = src->dtype == SBP_BF16;
    op = ss.kind == SBP_PARTIAL_SUM ? (bf ? OP_SUM_BF16 : OP_SUM_F32) : (bf ? OP_MAX_BF16 : OP_MAX_F32);
    if (ds.kind == SBP_BROADCAST) p.mode = DJ_REDUCE_ALL;
    else { p.mode = DJ_REDUCE; p.red_by_dst = dst_p ? 1 : 0; }
  } else if (dst_p) {
    if (ds.kind != SBP_PARTIAL_SUM)
      return fail(SBP_ERR_UNSUPPORTED, "boxing S->P(max) / B->P(max) is not implemented (zero is not neutral for max)");
    zero_first = true;
    p.dst_full = 1;
    p.mode = ss.kind == SBP_SPLIT ? DJ_PAIRS : DJ_TO_ALL;   // B -> P(sum): replica 0 -> partial 0
  } else if (ds.kind == SBP_BROADCAST) {
    p.mode = DJ_TO_ALL;
  } else if (ss.kind == SBP_BROADCAST) {
    p.mode = DJ_FROM_REPLICA;
  } else {
    p.mode = DJ_PAIRS;
  }

  // canonical view: sa / da are the tensor axes restricted by the source / destination
  const int sa = ss.kind == SBP_SPLIT ? ss.axis : -1;
  int da = ds.kind == SBP_SPLIT ? ds.axis : -1;
  if (zero_first && ss.kind == SBP_SPLIT) da = sa;          // S(i) -> P(sum): the virtual kd-way split of axis i
  auto prod = [&](int lo, int hi) {
    long long v = 1;
    for (int d = lo; d < hi; ++d) v *= src->shape[d];
    return v;
  };
  p.A = p.Na = p.M = p.Nb = 1;
  if (sa < 0 && da < 0) {
    p.C = prod(0, src->ndim);
  } else if (sa < 0 || da < 0 || sa == da) {
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
  if (numel(src) == 0) return SBP_OK;
  p.a_base_s = p.Na / ks;  p.a_rem_s = p.Na % ks;  p.a_base_d = p.Na / kd;  p.a_rem_d = p.Na % kd;
  p.b_base_s = p.Nb / ks;  p.b_rem_s = p.Nb % ks;  p.b_base_d = p.Nb / kd;  p.b_rem_d = p.Nb % kd;

  for (int r = 0; r < ks; ++r) p.src[r] = static_cast<const char*>(src->local[r]);
  for (int r = 0; r < kd; ++r) p.dst[r] = static_cast<char*>(dst->local[r]);

  // widest vector that every base pointer and every boundary of both splits on the Nb axis allows
  int vbytes = esz;
  for (int vb = 16; vb > esz; vb >>= 1) {
    bool ok = (p.Nb * p.C * esz) % vb == 0;
    for (int r = 0; r < ks && ok; ++r) ok = reinterpret_cast<uintptr_t>(src->local[r]) % vb == 0;
    for (int r = 0; r < kd && ok; ++r) ok = reinterpret_cast<uintptr_t>(dst->local[r]) % vb == 0;
    for (int side = 0; side < 2 && ok; ++side) {
      const bool by = side == 0 ? p.src_b : p.dst_b;
      const int k = side == 0 ? ks : kd;
      for (int r = 0; r < k && ok && by; ++r) {
        int64_t st, ln;
        split_range(p.Nb, k, r, &st, &ln);
        ok = (st * p.C * esz) % vb == 0;
      }
    }
    if (ok) { vbytes = vb; break; }
  }
  if ((op == OP_SUM_F32 || op == OP_MAX_F32) && vbytes < 4) vbytes = 4;

  // tasks
  if (p.mode == DJ_PAIRS) {
    const bool same_axis = p.src_b && p.dst_b;      // one axis cut by both sides: few pairs overlap
    if (same_axis) {
      for (int s = 0; s < ks; ++s)
        for (int d = 0; d < kd; ++d) {
          int64_t s0, sl, d0, dl;
          split_range(p.Nb, ks, s, &s0, &sl);
          split_range(p.Nb, kd, d, &d0, &dl);
          if (p.one_dst && d != dst_shard) continue;
          if (std::max(s0, d0) < std::min(s0 + sl, d0 + dl)) {
            p.pair_s[p.n_pairs] = (unsigned char)s;
            p.pair_d[p.n_pairs] = (unsigned char)d;
            ++p.n_pairs;
          }
        }
      p.ntasks = p.n_pairs;
    } else {
      p.ntasks = p.one_dst ? ks : ks * kd;
    }
  } else if (p.mode == DJ_FROM_REPLICA || p.mode == DJ_REDUCE) {
    p.ntasks = p.one_dst ? 1 : kd;
  } else if (p.mode == DJ_TO_ALL) {
    p.ntasks = ss.kind == SBP_SPLIT ? ks : 1;
  } else {
    p.ntasks = 1;
  }
  bool copy_needed = p.ntasks > 0;
  if ((p.mode == DJ_TO_ALL || p.mode == DJ_REDUCE_ALL) && p.one_dst) {
    p.n_dst = 1;
    if (zero_first) copy_needed = dst_shard == 0;   // B -> P(sum): only partial 0 receives the tensor
    else p.dst[0] = static_cast<char*>(dst->local[dst_shard]);
  } else if (p.mode == DJ_TO_ALL || p.mode == DJ_REDUCE_ALL) {
    const int n_out = zero_first ? 1 : kd;          // B -> P(sum) writes partial 0 only
    char* uniq[SBP_MAX_K];
    for (int r = 0; r < n_out; ++r) {
      bool seen = false;
      for (int q = 0; q < p.n_dst; ++q) seen = seen || uniq[q] == p.dst[r];
      if (!seen) uniq[p.n_dst++] = p.dst[r];
    }
    if (!zero_first)
      for (int q = 0; q < p.n_dst; ++q) p.dst[q] = uniq[q];
  }

  // tiling, sized by the largest cut any task can have
  auto max_cut = [&](long long n, bool by_src, bool by_dst) {
    long long m = n;
    if (by_src) m = std::min(m, (n + ks - 1) / ks);
    if (by_dst) m = std::min(m, (n + kd - 1) / kd);
    return m;
  };
  const long long nseg_max = p.A * max_cut(p.Na, p.src_a, p.dst_a) * p.M;
  const long long seg_vecs_max = max_cut(p.Nb, p.src_b, p.dst_b) * p.C * esz / vbytes;
  const int tile_vecs = (op == OP_COPY ? 4 : 2) * 256;
  int cv_log2 = 0;
  while ((1 << cv_log2) < tile_vecs && (1LL << cv_log2) < seg_vecs_max) ++cv_log2;
  p.cv_log2 = cv_log2;
  p.rows_per_tile = tile_vecs >> cv_log2;
  p.col_tiles = std::max(1LL, (seg_vecs_max + (1LL << cv_log2) - 1) >> cv_log2);
  const long long row_tiles = std::max(1LL, (nseg_max + p.rows_per_tile - 1) / p.rows_per_tile);
  p.tiles_per_task = p.col_tiles * row_tiles;
  const long long grid = p.tiles_per_task * p.ntasks;
  if (copy_needed && grid > 0x7fffffffLL) return fail(SBP_ERR_UNSUPPORTED, "tensor too large for one launch");
  if (dry) return SBP_OK;   // every refusal lies above this line, every launch below it
  SBP_BOUNDS_RESET();
  SBP_BOUNDS_TENSOR(src);
  if (dst_shard >= 0) SBP_BOUNDS_SHARD(dst, dst_shard);
  else SBP_BOUNDS_TENSOR(dst);


  if (zero_first) {
    // The partials start as zeros.  One kernel clears all of them when they are 16-byte
    // aligned (one launch instead of up to kd memsets with their gaps); else memsets do.
    ZeroParams z{};
    z.bytes = (long long)numel(dst) * esz;
    bool vec_ok = z.bytes % 16 == 0;
    for (int r = 0; r < kd; ++r) {
      if (p.one_dst && r != dst_shard) continue;
      if (p.mode == DJ_TO_ALL && r == 0) continue;  // overwritten in full by the copy
      z.dst[z.n++] = static_cast<char*>(dst->local[r]);
      vec_ok = vec_ok && reinterpret_cast<uintptr_t>(dst->local[r]) % 16 == 0;
    }
    if (z.n > 0 && z.bytes > 0) {
      if (vec_ok) {
        long long zb = (z.bytes / 16 + 256 * 8 - 1) / (256 * 8);
        if (zb > 148 * 16) zb = 148 * 16;
        SBP_BOUNDS_UPLOAD(stream);
        launch_dependent(box_zero_kernel, dim3((unsigned)zb, (unsigned)z.n), dim3(256), 0, stream, z);
        cudaError_t ze = cudaGetLastError();
        if (ze != cudaSuccess) return cuda_fail(ze, "zero fill launch");
        count_launch();
      } else {
        for (int q = 0; q < z.n; ++q) SBP_CUDA_TRY(cudaMemsetAsync(z.dst[q], 0, (size_t)z.bytes, stream));
      }
    }
  }
  if (!copy_needed) return SBP_OK;
  switch (op) {
    case OP_COPY: launch_disjoint<OP_COPY>(p, vbytes, grid, stream); break;
    case OP_SUM_F32: launch_disjoint<OP_SUM_F32>(p, vbytes, grid, stream); break;
    case OP_MAX_F32: launch_disjoint<OP_MAX_F32>(p, vbytes, grid, stream); break;
    case OP_SUM_BF16: launch_disjoint<OP_SUM_BF16>(p, vbytes, grid, stream); break;
    default: launch_disjoint<OP_MAX_BF16>(p, vbytes, grid, stream); break;
  }
  cudaError_t e = cudaGetLastError();
  if (e != cudaSuccess) return cuda_fail(e, "disjoint-placement boxing launch");
  count_launch();
  return SBP_OK;
}

}  // namespace sbp
