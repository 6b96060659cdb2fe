// Parameter block shared by the two boxing copy engines (host + device, this library only).
#pragma once

#include "sbp.h"

namespace sbp {

enum BoxMode : int {
  MODE_PAIRS = 0,      // task t: source shard t / k, destination shard t % k
  MODE_DIAG = 1,       // task t: source shard t, destination shard t
  MODE_GATHER = 2,     // task t: source shard t, every destination replica
  MODE_REDUCE_S = 3,   // task t: all sources, destination shard t
  MODE_REDUCE_B = 4,   // one task: all sources, every destination replica
  MODE_SCATTER_P = 5   // task t: destination shard t is the full shape: own piece copied, rest zero
};

// The logical tensor is viewed as [A][Na][M][Nb][C] (elements); src_a/src_b/dst_a/dst_b say
// which side's split signature restricts the axes Na and Nb.
struct BoxParams {
  const char* src[SBP_MAX_K];
  char* dst[SBP_MAX_K];
  long long A, Na, M, Nb, C;
  long long tiles_per_task, col_tiles;
  int k, esz, mode;
  int src_a, src_b, dst_a, dst_b;
  int n_dst;                        // distinct destination buffers (GATHER / REDUCE_B)
  int cv_log2;                      // tile width in vectors, log2
  int rows_per_tile;
  int ntasks;                       // tasks of the transform; tiles are dealt task-fastest
  int one_dst, dst_shard;           // one_dst: only the tasks that produce destination shard dst_shard
  long long a_base, a_rem, b_base, b_rem;   // Na / k, Na % k, Nb / k, Nb % k: the balanced split without a division
  // Row pitch of every local tensor in units of C elements, 0 = dense (the pitch is then the local
  // extent of the Nb axis).  Non-zero only for 2-D tensors with a leading dimension (C == 1).
  long long src_pitch[SBP_MAX_K], dst_pitch[SBP_MAX_K];
};

// Start and length of shard r's piece of an axis whose n / k and n % k are known.
__host__ __device__ inline void split_range_pre(long long base, long long rem, int r, long long* start, long long* len) {
  *len = base + (r < rem ? 1 : 0);
  *start = r * base + (r < rem ? r : rem);
}

}  // namespace sbp
