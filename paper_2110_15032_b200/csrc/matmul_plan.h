// Grouped-GEMM plan shared by the MatMul kernels of this library (host + device).
//
// Every MatMul signature of Table 1 -- and every fused "P(sum) result written directly as
// B or S(i)" variant -- is a list of independent output groups; a group's result is the sum
// over one or more K-segments, taken in segment order:
//
//   Y_g[M_g, N_g] = sum_{s in segs(g)}  A_s[row_off_g : row_off_g + M_g, 0 : K_s]
//                                     * B_s[0 : K_s, col_off_g : col_off_g + N_g]
// (A_s and B_s may each be stored transposed, see a_trans / b_trans)
//
//   unfused (chain == 0): segs(g) = {g}       one local product per shard
//   fused   (chain == 1): segs(g) = {0..nseg-1}  the partial products of all shards are
//                                              accumulated in rank order in the accumulator
#pragma once

#include <cstdint>

#include "sbp.h"

namespace sbp {

struct MatmulPlan {
  // per K-segment (= per source shard)
  const void* a[SBP_MAX_K];
  const void* b[SBP_MAX_K];
  long long lda[SBP_MAX_K], ldb[SBP_MAX_K], kseg[SBP_MAX_K];
  // per output group
  long long m[SBP_MAX_K], n[SBP_MAX_K], row_off[SBP_MAX_K], col_off[SBP_MAX_K], ldy[SBP_MAX_K];
  void* y[SBP_MAX_K];
  // extra destinations of group 0 when one result is stored to several B replicas
  void* y_rep[SBP_MAX_K];
  int n_rep;
  int ngroups, nseg, chain;
  // a_trans: A_s is stored transposed, A_s[row, kk] = a[kk * lda + row]; b_trans: B_s[kk, col] =
  // b[col * ldb + kk].  lda / ldb are always the leading dimensions of the stored arrays.
  int a_trans, b_trans;
  int gelu;
  int in_dtype, out_dtype;   // sbp_dtype
};

// Optional epilogue of the tensor-core kernel for the class-split classifier: instead of storing
// the logits, every 128-column chunk of a tile leaves, per row, a local max, a local
// sum of exp(z - max) and the label's logit (0 when the label lies elsewhere).
//   part_x[(part_base[g] + chunk) * rows + row],  chunk = column / 128 inside group g
struct XentFusion {
  float* part_m;
  float* part_s;
  float* part_t;
  const long long* labels;          // [rows], global class indices
  long long class_start[SBP_MAX_K]; // first class of group g
  int part_base[SBP_MAX_K];         // first chunk index of group g
  long long rows;
  // grad mode: the epilogue writes softmax - onehot of the recomputed logits instead of partials
  int grad;
  const float* row_max;             // [rows], from the forward pass
  const float* row_sum;             // [rows]
};

}  // namespace sbp
