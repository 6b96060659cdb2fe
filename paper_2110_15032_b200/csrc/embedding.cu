// Row-split embedding lookup (Section 6.3: table S(0), "splitting the vocabulary IDs").
//
//   unfused: out_r[l,:] = table_r[id_l - start_r,:] when id_l lies in shard r's row range and
//            zeros otherwise; the k outputs form a P(sum) tensor.  One pass over the lookups
//            writes all k of them (row read once, k stores).
//   fused:   the P(sum) -> B boxing folded into the gather.  Exactly one shard contributes
//            to a lookup, so the sum over shards is that shard's row; the kernel finds the
//            owning shard from the id, reads the row once and writes every B replica.
//
// One thread moves one 16-byte piece of a row (or one element on the unaligned path) for J
// lookups; all id loads, then all row loads, are issued before the first store.
#include <cuda_bf16.h>

#include "bounds_check.h"
#include "sbp_internal.h"

namespace sbp {

struct EmbParams {
  const char* table[SBP_MAX_K];
  const long long* ids[SBP_MAX_K];
  char* out[SBP_MAX_K];
  long long rows;         // logical table rows
  long long base, rem, big;   // balanced split of the rows, see owner_of_row
  int narrow;
  long long n_lookups;
  long long vpr;          // vectors per row
  int vpr_log2;           // >= 0 when vpr is a power of two, else -1
  int k, esz;
  int n_dst;              // fused: distinct replicas
  int canon_neg_zero;     // fused and k > 1: write -0.0 as +0.0 (what x + 0 gives)
  int* oob;
};

// Shard that owns table row `id` under the balanced split, and the first row of that shard.
// base = rows / k, rem = rows % k, big = rem * (base + 1) come precomputed from the host; tables
// below 2^31 rows (narrow = 1) take 32-bit divisions, which cost a fraction of 64-bit ones.
__device__ __forceinline__ int owner_of_row(long long id, long long base, long long rem, long long big, int narrow,
                                            long long* start) {
  if (narrow) {
    const unsigned uid = (unsigned)id, ubase = (unsigned)base, ubig = (unsigned)big;
    unsigned r;
    if (uid < ubig) {
      r = uid / (ubase + 1);
      *start = (long long)r * (ubase + 1);
    } else {
      r = (unsigned)rem + (uid - ubig) / ubase;
      *start = (long long)ubig + (long long)(r - (unsigned)rem) * ubase;
    }
    return (int)r;
  }
  int r;
  if (id < big) {
    r = (int)(id / (base + 1));
    *start = r * (base + 1);
  } else {
    r = (int)(rem + (id - big) / base);
    *start = big + (r - rem) * base;
  }
  return r;
}

// item = lookup * vpr + piece: a shift when vpr is a power of two, a 32-bit division when both
// fit, a 64-bit division (an order of magnitude dearer) only otherwise.
__device__ __forceinline__ void split_item(long long item, long long vpr, int vpr_log2, long long* look, long long* col) {
  if (vpr_log2 >= 0) {
    *look = item >> vpr_log2;
    *col = item & (vpr - 1);
  } else if (((unsigned long long)item | (unsigned long long)vpr) >> 32) {
    *look = item / vpr;
    *col = item - *look * vpr;
  } else {
    const unsigned q = (unsigned)item / (unsigned)vpr;
    *look = q;
    *col = (unsigned)item - q * (unsigned)vpr;
  }
}

template <typename V>
__device__ __forceinline__ V zero_vec() {
  V z;
  unsigned char* b = reinterpret_cast<unsigned char*>(&z);
#pragma unroll
  for (int i = 0; i < (int)sizeof(V); ++i) b[i] = 0;
  return z;
}

// Replaces every -0.0 lane by +0.0.  ESZ = 4 (fp32) or 2 (bf16).
template <typename V, int ESZ>
__device__ __forceinline__ V canon(V v) {
  if (ESZ == 4) {
    uint32_t* w = reinterpret_cast<uint32_t*>(&v);
#pragma unroll
    for (int i = 0; i < (int)(sizeof(V) / 4); ++i)
      if (w[i] == 0x80000000u) w[i] = 0;
  } else {
    uint16_t* h = reinterpret_cast<uint16_t*>(&v);
#pragma unroll
    for (int i = 0; i < (int)(sizeof(V) / 2); ++i)
      if (h[i] == 0x8000u) h[i] = 0;
  }
  return v;
}

// MINB: resident CTAs per SM the register allocation is held to (see launch_emb).
template <typename V, int ESZ, int J, bool FUSED, int MINB>
__global__ void __launch_bounds__(256, MINB) embedding_kernel(const __grid_constant__ EmbParams p) {
  const long long total = p.n_lookups * p.vpr;
  const long long stride = (long long)gridDim.x * 256;
  const long long base = (long long)blockIdx.x * 256 + threadIdx.x;
  // Both forms walk the lookups once and read every row once, from the shard that owns it.
  // Fused: the row goes to every B replica.  Unfused: it goes to the owner's P(sum) output and
  // zeros go to the others' -- the same k outputs as k devices looking up only their own rows.
  // The ids are taken from replica 0 (the replicas of a B tensor are equal by definition).
  const int shard = 0;

  long long item[J], look[J], col[J], id[J];
  int own[J];
  bool ok[J];
#pragma unroll
  for (int j = 0; j < J; ++j) {
    item[j] = base + j * stride;
    ok[j] = item[j] < total;
    split_item(item[j], p.vpr, p.vpr_log2, &look[j], &col[j]);
  }
#pragma unroll
  for (int j = 0; j < J; ++j) id[j] = (ok[j] && SBP_GUARD(p.ids[shard] + look[j], 8)) ? __ldg(p.ids[shard] + look[j]) : -1;

  V val[J];
#pragma unroll
  for (int j = 0; j < J; ++j) {
    val[j] = zero_vec<V>();
    own[j] = -1;
    if (!ok[j]) continue;
    const bool in_table = id[j] >= 0 && id[j] < p.rows;
    if (!in_table) {
      if (p.oob && col[j] == 0 && shard == 0 && SBP_GUARD(p.oob, 4)) atomicAdd(p.oob, 1);
      continue;
    }
    long long start;
    const int r = owner_of_row(id[j], p.base, p.rem, p.big, p.narrow, &start);
    own[j] = r;
    const V* src = reinterpret_cast<const V*>(p.table[r]) + (id[j] - start) * p.vpr + col[j];
    if (SBP_GUARD(src, sizeof(V))) val[j] = __ldg(src);
  }

  if (FUSED) {
    for (int q = 0; q < p.n_dst; ++q) {
      V* o = reinterpret_cast<V*>(p.out[q]);
#pragma unroll
      for (int j = 0; j < J; ++j)
        if (ok[j] && SBP_GUARD(o + item[j], sizeof(V))) o[item[j]] = p.canon_neg_zero ? canon<V, ESZ>(val[j]) : val[j];
    }
  } else {
    for (int q = 0; q < p.k; ++q) {
      V* o = reinterpret_cast<V*>(p.out[q]);
#pragma unroll
      for (int j = 0; j < J; ++j)
        if (ok[j] && SBP_GUARD(o + item[j], sizeof(V))) o[item[j]] = own[j] == q ? val[j] : zero_vec<V>();
    }
  }
}

// Fused gather with a single destination per row (k = 1, or all B replicas the same buffer).
// There the element-wise kernel above is bound by the latency of its id -> row -> store chain, not
// by bandwidth.  This form takes the id load out of the chain.  A persistent CTA walks chunks of
// 256 * J consecutive 16-byte pieces of the result (for 512-byte rows and J = 8: 64 consecutive
// lookups).  The ids of a chunk sit in shared memory before its rows are asked for; the ids of the
// CTA's next chunk are requested first (one coalesced load), then every thread puts J row loads in
// flight at once (a warp: J whole rows), stores them, and only then parks the next ids in the other
// half of the shared buffer -- so the id latency hides behind the rows.  The result is written with
// streaming (evict-first) stores so that the output, which is never read back, does not push the
// table's hot rows out of L2.  vpr (vectors per row) must be a power of two between 8 and 256 * J, so
// that a chunk starts on a row boundary and holds at most 256 lookups (one id per thread).
template <typename V, int ESZ, int J>
__global__ void __launch_bounds__(256) embedding_rows_kernel(const __grid_constant__ EmbParams p) {
  // Per lookup of the chunk: where its table row starts (null for an id outside the table).  The
  // owner of an id -- a division by the shard size -- is worked out once per lookup by the thread
  // that stages it, a chunk ahead, not by each of the row's 16-byte vectors on its way to the load.
  __shared__ const char* rows_s[2][256];
  auto resolve = [&](long long id) -> const char* {
    if (id < 0 || id >= p.rows) {
      if (p.oob && SBP_GUARD(p.oob, 4)) atomicAdd(p.oob, 1);
      return nullptr;
    }
    long long start;
    const int r = owner_of_row(id, p.base, p.rem, p.big, p.narrow, &start);
    return p.table[r] + (id - start) * p.vpr * (long long)sizeof(V);
  };
  const long long total = p.n_lookups * p.vpr;
  const long long n_chunks = (total + 256 * J - 1) / (256 * J);

  // first and last lookup of a chunk
  auto span = [&](long long chunk, long long* look0, int* n_ids) {
    const long long first = chunk * (256 * J);
    long long last = first + 256 * J - 1;
    if (last >= total) last = total - 1;
    *look0 = first >> p.vpr_log2;
    *n_ids = (int)((last >> p.vpr_log2) - *look0) + 1;
  };

  long long chunk = blockIdx.x;
  if (chunk >= n_chunks) return;
  int cur = 0;
  {
    long long look0;
    int n_ids;
    span(chunk, &look0, &n_ids);
    if ((int)threadIdx.x < n_ids)
      rows_s[0][threadIdx.x] = resolve(SBP_GUARD(p.ids[0] + look0 + threadIdx.x, 8) ? __ldcs(p.ids[0] + look0 + threadIdx.x) : -1);
  }
  __syncthreads();

  for (; chunk < n_chunks; chunk += gridDim.x) {
    const long long cta_base = chunk * (256 * J);
    long long look0;
    int n_ids;
    span(chunk, &look0, &n_ids);
    // request the next chunk's ids; they are not touched until this chunk's rows are stored
    const long long next = chunk + gridDim.x;
    long long nlook0 = 0, nid = 0;
    int nn = 0;
    if (next < n_chunks) {
      span(next, &nlook0, &nn);
      if ((int)threadIdx.x < nn && SBP_GUARD(p.ids[0] + nlook0 + threadIdx.x, 8)) nid = __ldcs(p.ids[0] + nlook0 + threadIdx.x);
    }

    V val[J];
    bool ok[J];
#pragma unroll
    for (int j = 0; j < J; ++j) {
      const long long item = cta_base + j * 256 + threadIdx.x;
      ok[j] = item < total;
      val[j] = zero_vec<V>();
      if (!ok[j]) continue;
      const long long look = item >> p.vpr_log2, col = item & (p.vpr - 1);
      const char* row = rows_s[cur][look - look0];
      if (!row) continue;
      const V* src = reinterpret_cast<const V*>(row) + col;
      if (SBP_GUARD(src, sizeof(V))) val[j] = __ldg(src);
    }
    V* o = reinterpret_cast<V*>(p.out[0]);
#pragma unroll
    for (int j = 0; j < J; ++j)
      if (ok[j] && SBP_GUARD(o + cta_base + j * 256 + threadIdx.x, sizeof(V)))
        __stcs(o + cta_base + j * 256 + threadIdx.x, p.canon_neg_zero ? canon<V, ESZ>(val[j]) : val[j]);

    if ((int)threadIdx.x < nn) rows_s[cur ^ 1][threadIdx.x] = resolve(nid);
    __syncthreads();
    cur ^= 1;
  }
}

// Two shapes of the same kernel.  With several destinations per row the kernel is bound by its
// stores and runs best with four lookups per thread; with a single destination (aliased
// replicas, k = 1) it is bound by the latency of the id -> row -> store chain and runs best
// with more resident warps: two lookups per thread, registers held to eight CTAs per SM
// (measured on the Zipf workload: 0.347 -> 0.272 ms for one destination, while the same
// shape costs the eight-replica case 4 %).
template <typename V, int ESZ>
static void launch_emb(const EmbParams& p, bool fused, cudaStream_t st) {
  const long long total = p.n_lookups * p.vpr;
  SBP_BOUNDS_UPLOAD(st);
  auto blocks_for = [&](int j) {
    long long b = (total + 256LL * j - 1) / (256LL * j);
    return (unsigned)(b < 1 ? 1 : b);
  };
  if (fused && p.n_dst == 1 && p.vpr_log2 >= 3 && p.vpr_log2 <= 11) {
    // persistent: as many CTAs as fit at once
    static int resident = 0;
    if (resident == 0) {
      int dev = 0, sms = 148, per_sm = 4;
      cudaGetDevice(&dev);
      cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
      if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, embedding_rows_kernel<V, ESZ, 8>, 256, 0) != cudaSuccess || per_sm < 1) {
        cudaGetLastError();
        per_sm = 4;
      }
      resident = sms * per_sm;
    }
    const unsigned chunks = blocks_for(8);
    embedding_rows_kernel<V, ESZ, 8><<<dim3(chunks < (unsigned)resident ? chunks : (unsigned)resident), 256, 0, st>>>(p);
  } else if (fused && p.n_dst == 1) {
    embedding_kernel<V, ESZ, 2, true, 8><<<dim3(blocks_for(2)), 256, 0, st>>>(p);
  } else if (fused) {
    embedding_kernel<V, ESZ, 4, true, 1><<<dim3(blocks_for(4)), 256, 0, st>>>(p);
  } else {
    embedding_kernel<V, ESZ, 4, false, 1><<<dim3(blocks_for(4)), 256, 0, st>>>(p);
  }
}

// ---- table split along the hidden axis: S(1) ("splitting the hidden dimension", Section 6.3).
// Shard r holds columns [start_r, start_r + len_r) of every row.  The lookup of one id touches
// every shard; its natural result is split along the last axis the same way, and writing whole
// rows to every B replica instead is the all-gather fused into the gather.
struct EmbS1Params {
  const char* table[SBP_MAX_K];
  const long long* ids[SBP_MAX_K];
  char* out[SBP_MAX_K];
  long long vstart[SBP_MAX_K + 1];   // first vector of shard r's piece inside a full row
  long long rows, n_lookups, vpr_total;
  int vpr_log2;                      // >= 0 when vpr_total is a power of two, else -1
  int k, n_dst;
  int* oob;
};

template <typename V, int J, bool FUSED>
__global__ void __launch_bounds__(256) embedding_s1_kernel(const __grid_constant__ EmbS1Params p) {
  const long long total = p.n_lookups * p.vpr_total;
  const long long stride = (long long)gridDim.x * 256;
  const long long base = (long long)blockIdx.x * 256 + threadIdx.x;
  long long item[J], look[J], col[J], id[J];
  int shard[J];
  bool ok[J];
#pragma unroll
  for (int j = 0; j < J; ++j) {
    item[j] = base + j * stride;
    ok[j] = item[j] < total;
    split_item(item[j], p.vpr_total, p.vpr_log2, &look[j], &col[j]);
    int r = 0;
    while (r + 1 < p.k && col[j] >= p.vstart[r + 1]) ++r;
    shard[j] = r;
  }
#pragma unroll
  for (int j = 0; j < J; ++j)
    id[j] = (ok[j] && SBP_GUARD(p.ids[FUSED ? 0 : shard[j]] + look[j], 8)) ? __ldg(p.ids[FUSED ? 0 : shard[j]] + look[j]) : -1;
  V val[J];
#pragma unroll
  for (int j = 0; j < J; ++j) {
    val[j] = zero_vec<V>();
    if (!ok[j]) continue;
    if (id[j] < 0 || id[j] >= p.rows) {
      if (p.oob && col[j] == 0 && SBP_GUARD(p.oob, 4)) atomicAdd(p.oob, 1);
      continue;
    }
    const long long w = p.vstart[shard[j] + 1] - p.vstart[shard[j]];
    const V* src = reinterpret_cast<const V*>(p.table[shard[j]]) + id[j] * w + (col[j] - p.vstart[shard[j]]);
    if (SBP_GUARD(src, sizeof(V))) val[j] = __ldg(src);
  }
  if (FUSED) {
    for (int q = 0; q < p.n_dst; ++q) {
      V* o = reinterpret_cast<V*>(p.out[q]);
#pragma unroll
      for (int j = 0; j < J; ++j)
        if (ok[j] && SBP_GUARD(o + item[j], sizeof(V))) o[item[j]] = val[j];
    }
  } else {
#pragma unroll
    for (int j = 0; j < J; ++j) {
      if (!ok[j]) continue;
      const long long w = p.vstart[shard[j] + 1] - p.vstart[shard[j]];
      V* dstp = reinterpret_cast<V*>(p.out[shard[j]]) + look[j] * w + (col[j] - p.vstart[shard[j]]);
      if (SBP_GUARD(dstp, sizeof(V))) *dstp = val[j];
    }
  }
}

template <typename V>
static void launch_emb_s1(const EmbS1Params& p, bool fused, cudaStream_t st) {
  constexpr int J = 4;
  const long long total = p.n_lookups * p.vpr_total;
  long long blocks = (total + 256LL * J - 1) / (256LL * J);
  if (blocks < 1) blocks = 1;
  SBP_BOUNDS_UPLOAD(st);
  if (fused) embedding_s1_kernel<V, J, true><<<(unsigned)blocks, 256, 0, st>>>(p);
  else embedding_s1_kernel<V, J, false><<<(unsigned)blocks, 256, 0, st>>>(p);
}

static sbp_status embedding_hidden_split(const sbp_tensor* table, const sbp_tensor* ids, sbp_tensor* out,
                                         int32_t* oob_count, cudaStream_t stream) {
  const int k = placement_k(table);
  const int esz = elem_size(table->dtype);
  const int last = out->ndim - 1;
  const bool fused = out->sbp[0].kind == SBP_BROADCAST;
  if (!fused && !(out->sbp[0].kind == SBP_SPLIT && out->sbp[0].axis == last))
    return fail(SBP_ERR_SIGNATURE, "with the table S(1), out must be split along its last axis, or B (gather fused in)");
  const long long n_lookups = numel(ids);
  if (n_lookups == 0 || table->shape[1] == 0) return SBP_OK;
  int vb = 16;
  for (; vb > esz; vb >>= 1) {
    bool ok = true;
    for (int r = 0; r < k && ok; ++r) {
      int64_t st, ln;
      split_range(table->shape[1], k, r, &st, &ln);
      ok = (st * esz) % vb == 0 && (ln * esz) % vb == 0;
      ok = ok && reinterpret_cast<uintptr_t>(table->local[r]) % vb == 0 && reinterpret_cast<uintptr_t>(out->local[r]) % vb == 0;
    }
    if (ok) break;
  }
  EmbS1Params p{};
  p.k = k;
  p.rows = table->shape[0];
  p.n_lookups = n_lookups;
  p.oob = oob_count;
  p.vpr_total = table->shape[1] * esz / vb;
  p.vpr_log2 = -1;
  for (int b = 0; b < 40; ++b)
    if ((1LL << b) == p.vpr_total) p.vpr_log2 = b;
  for (int r = 0; r < k; ++r) {
    int64_t st, ln;
    split_range(table->shape[1], k, r, &st, &ln);
    p.vstart[r] = st * esz / vb;
    p.table[r] = static_cast<const char*>(table->local[r]);
    p.ids[r] = static_cast<const long long*>(ids->local[r]);
    p.out[r] = static_cast<char*>(out->local[r]);
  }
  p.vstart[k] = p.vpr_total;
  if (fused) {
    char* uniq[SBP_MAX_K];
    for (int r = 0; r < k; ++r) {
      bool seen = false;
      for (int q = 0; q < p.n_dst; ++q) seen = seen || uniq[q] == p.out[r];
      if (!seen) uniq[p.n_dst++] = p.out[r];
    }
    for (int q = 0; q < p.n_dst; ++q) p.out[q] = uniq[q];
  }
  if ((n_lookups * p.vpr_total + 1023) / 1024 > 0x7fffffffLL) return fail(SBP_ERR_UNSUPPORTED, "too many lookups for one launch");
  switch (vb) {
    case 16: launch_emb_s1<uint4>(p, fused, stream); break;
    case 8: launch_emb_s1<uint2>(p, fused, stream); break;
    case 4: launch_emb_s1<uint32_t>(p, fused, stream); break;
    default: launch_emb_s1<uint16_t>(p, fused, stream); break;
  }
  cudaError_t e = cudaGetLastError();
  if (e != cudaSuccess) return cuda_fail(e, "embedding launch");
  count_launch();
  return SBP_OK;
}

// ---- backward of the row-split lookup: the gradient of the table, S(0) like the table.
// grad_table_r[row, :] = sum over the lookups l with id_l = start_r + row of grad_out[l, :].
// Each shard's gradient is zero-filled; then the lookups are taken in chunks, one CTA per chunk:
// the CTA sorts its chunk by (id, position), each warp sums the runs of equal ids in its part
// of the sorted chunk in registers (in lookup order) and adds one row per run into the owning
// shard with 16-byte fp32 atomic adds. Under a skewed id distribution this takes the repeated
// adds to the hot rows out of the L2 atomic units, which otherwise serialise them. The order of
// the atomic adds between chunks, hence the last bits of a sum with many terms, is not fixed.
struct EmbBwdParams {
  float* grad_table[SBP_MAX_K];
  long long shard_vecs[SBP_MAX_K];   // float4 vectors in each shard's gradient
  const long long* ids;
  const float* grad_out;
  long long rows, base, rem, big;
  int narrow;
  long long n_lookups, vpr;          // float4 vectors per row
  int k;
  int* oob;
};

__global__ void __launch_bounds__(256) embedding_zero_kernel(const __grid_constant__ EmbBwdParams p) {
  float4* g = reinterpret_cast<float4*>(p.grad_table[blockIdx.y]);
  const long long n = p.shard_vecs[blockIdx.y];
  const float4 z = make_float4(0.f, 0.f, 0.f, 0.f);
  for (long long i = (long long)blockIdx.x * 256 + threadIdx.x; i < n; i += (long long)gridDim.x * 256)
    if (SBP_GUARD(g + i, 16)) g[i] = z;
}

// CHUNK lookups per CTA pass (256 or 1024); key = id * CHUNK + position in the chunk, all ones
// for a position past the end or an id outside the table (sorted last, skipped).
template <int CHUNK>
__global__ void __launch_bounds__(256, 3) embedding_backward_kernel(const __grid_constant__ EmbBwdParams p) {
  constexpr int kShift = CHUNK == 1024 ? 10 : 8;
  constexpr int kPerWarp = CHUNK / 8;     // sorted positions walked by one warp
  constexpr int kBatch = 8;               // gradient rows in flight per lane
  constexpr unsigned long long kNone = ~0ull;
  __shared__ unsigned long long key[CHUNK];
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const long long n_chunks = (p.n_lookups + CHUNK - 1) / CHUNK;
  const float4* gout = reinterpret_cast<const float4*>(p.grad_out);
  for (long long chunk = blockIdx.x; chunk < n_chunks; chunk += gridDim.x) {
    const long long first = chunk * CHUNK;
    for (int i = tid; i < CHUNK; i += 256) {
      unsigned long long kv = kNone;
      if (first + i < p.n_lookups) {
        const long long id = SBP_GUARD(p.ids + first + i, 8) ? __ldg(p.ids + first + i) : -1;
        if (id >= 0 && id < p.rows) kv = ((unsigned long long)id << kShift) | (unsigned)i;
        else if (p.oob && SBP_GUARD(p.oob, 4)) atomicAdd(p.oob, 1);
      }
      key[i] = kv;
    }
    __syncthreads();
    // bitonic sort, ascending
    for (int size = 2; size <= CHUNK; size <<= 1) {
      for (int j = size >> 1; j > 0; j >>= 1) {
        for (int t = tid; t < CHUNK / 2; t += 256) {
          const int lo = 2 * t - (t & (j - 1)), hi = lo + j;
          const unsigned long long a = key[lo], b = key[hi];
          const bool up = (lo & size) == 0;
          if ((a > b) == up) { key[lo] = b; key[hi] = a; }
        }
        __syncthreads();
      }
    }
    // runs of equal ids -> one atomic row add each
    for (long long cb = 0; cb < p.vpr; cb += 32) {
      const long long col = cb + lane;
      const bool active = col < p.vpr;
      long long cur = -1;
      float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
      auto flush = [&]() {
        if (cur >= 0 && active) {
          long long start;
          const int r = owner_of_row(cur, p.base, p.rem, p.big, p.narrow, &start);
          float4* at = reinterpret_cast<float4*>(p.grad_table[r]) + (cur - start) * p.vpr + col;
          if (SBP_GUARD(at, 16)) atomicAdd(at, acc);
        }
      };
      for (int pos = warp * kPerWarp; pos < (warp + 1) * kPerWarp; pos += kBatch) {
        unsigned long long kv[kBatch];
        float4 gv[kBatch];
#pragma unroll
        for (int j = 0; j < kBatch; ++j) {
          kv[j] = key[pos + j];
          gv[j] = make_float4(0.f, 0.f, 0.f, 0.f);
          if (kv[j] != kNone && active && SBP_GUARD(gout + (first + (long long)(kv[j] & (CHUNK - 1))) * p.vpr + col, 16))
            gv[j] = __ldg(gout + (first + (long long)(kv[j] & (CHUNK - 1))) * p.vpr + col);
        }
#pragma unroll
        for (int j = 0; j < kBatch; ++j) {
          if (kv[j] == kNone) continue;
          const long long id = (long long)(kv[j] >> kShift);
          if (id != cur) {
            flush();
            cur = id;
            acc = gv[j];
          } else {
            acc.x += gv[j].x; acc.y += gv[j].y; acc.z += gv[j].z; acc.w += gv[j].w;
          }
        }
      }
      flush();
    }
    __syncthreads();
  }
}

}  // namespace sbp

using namespace sbp;

extern "C" sbp_status sbp_embedding(const sbp_tensor* table, const sbp_tensor* ids, sbp_tensor* out,
                                    int32_t* oob_count, void* cuda_stream) {
  SBP_RANGE("sbp_embedding");
  sbp_status st = check_tensor(table, "table", true);
  if (st != SBP_OK) return st;
  st = check_tensor(ids, "ids", true);
  if (st != SBP_OK) return st;
  st = check_tensor(out, "out", true);
  if (st != SBP_OK) return st;
  const sbp_tensor* dense_only[3] = {table, ids, out};
  const char* dense_names[3] = {"table", "ids", "out"};
  for (int i = 0; i < 3; ++i)
    if ((st = refuse_ld(dense_only[i], dense_names[i], "sbp_embedding")) != SBP_OK) return st;
  if (table->ndim != 2) return fail(SBP_ERR_SHAPE, "table must be [rows, dim]");
  if (table->dtype != SBP_F32 && table->dtype != SBP_BF16) return fail(SBP_ERR_DTYPE, "table must be F32 or BF16");
  if (out->dtype != table->dtype) return fail(SBP_ERR_DTYPE, "out and table differ in dtype");
  if (ids->dtype != SBP_I64) return fail(SBP_ERR_DTYPE, "ids must be I64");
  if (ids->ndim > 3) return fail(SBP_ERR_SHAPE, "ids rank %d > 3", ids->ndim);
  if (out->ndim != ids->ndim + 1) return fail(SBP_ERR_SHAPE, "out rank must be ids rank + 1");
  for (int d = 0; d < ids->ndim; ++d)
    if (out->shape[d] != ids->shape[d]) return fail(SBP_ERR_SHAPE, "out and ids differ on axis %d", d);
  if (out->shape[out->ndim - 1] != table->shape[1]) return fail(SBP_ERR_SHAPE, "out's last axis must equal dim");
  const int k = placement_k(table);
  if (placement_k(ids) != k || placement_k(out) != k) return fail(SBP_ERR_INVALID_ARG, "operands differ in k");
  if (table->sbp[0].kind != SBP_SPLIT) return fail(SBP_ERR_SIGNATURE, "table must be S(0) or S(1)");
  if (ids->sbp[0].kind != SBP_BROADCAST) return fail(SBP_ERR_SIGNATURE, "ids must be B");
  SBP_BOUNDS_RESET();
  SBP_BOUNDS_TENSOR(table);
  SBP_BOUNDS_TENSOR(ids);
  SBP_BOUNDS_TENSOR(out);
  SBP_BOUNDS_ADD(oob_count, 4);
  if (table->sbp[0].axis == 1)
    return embedding_hidden_split(table, ids, out, oob_count, static_cast<cudaStream_t>(cuda_stream));
  const bool fused = out->sbp[0].kind == SBP_BROADCAST;
  if (!fused && out->sbp[0].kind != SBP_PARTIAL_SUM)
    return fail(SBP_ERR_SIGNATURE, "out must be P(sum) (unfused) or B (boxing fused into the gather)");
  const long long n_lookups = numel(ids);
  if (n_lookups == 0 || table->shape[1] == 0) return SBP_OK;

  EmbParams p{};
  p.k = k;
  p.esz = elem_size(table->dtype);
  p.rows = table->shape[0];
  p.base = p.rows / k;
  p.rem = p.rows % k;
  p.big = p.rem * (p.base + 1);
  p.narrow = p.rows < (1LL << 31) ? 1 : 0;
  p.n_lookups = n_lookups;
  p.oob = oob_count;
  const long long row_bytes = table->shape[1] * p.esz;
  int vb = 16;
  for (; vb > p.esz; vb >>= 1) {
    bool ok = row_bytes % vb == 0;
    for (int r = 0; r < k && ok; ++r)
      ok = reinterpret_cast<uintptr_t>(table->local[r]) % vb == 0 && reinterpret_cast<uintptr_t>(out->local[r]) % vb == 0;
    if (ok) break;
  }
  p.vpr = row_bytes / vb;
  p.vpr_log2 = -1;
  for (int b = 0; b < 40; ++b)
    if ((1LL << b) == p.vpr) p.vpr_log2 = b;
  for (int r = 0; r < k; ++r) {
    p.table[r] = static_cast<const char*>(table->local[r]);
    p.ids[r] = static_cast<const long long*>(ids->local[r]);
    p.out[r] = static_cast<char*>(out->local[r]);
  }
  if (fused) {
    p.canon_neg_zero = k > 1;
    char* uniq[SBP_MAX_K];
    for (int r = 0; r < k; ++r) {
      bool seen = false;
      for (int q = 0; q < p.n_dst; ++q) seen = seen || uniq[q] == p.out[r];
      if (!seen) uniq[p.n_dst++] = p.out[r];
    }
    for (int q = 0; q < p.n_dst; ++q) p.out[q] = uniq[q];
  }
  if ((n_lookups * p.vpr + 511) / 512 > 0x7fffffffLL) return fail(SBP_ERR_UNSUPPORTED, "too many lookups for one launch");
  cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
  const bool f32 = table->dtype == SBP_F32;
  switch (vb) {
    case 16: f32 ? launch_emb<uint4, 4>(p, fused, stream) : launch_emb<uint4, 2>(p, fused, stream); break;
    case 8: f32 ? launch_emb<uint2, 4>(p, fused, stream) : launch_emb<uint2, 2>(p, fused, stream); break;
    case 4: f32 ? launch_emb<uint32_t, 4>(p, fused, stream) : launch_emb<uint32_t, 2>(p, fused, stream); break;
    default: launch_emb<uint16_t, 2>(p, fused, stream); break;
  }
  cudaError_t e = cudaGetLastError();
  if (e != cudaSuccess) return cuda_fail(e, "embedding launch");
  count_launch();
  return SBP_OK;
}

extern "C" sbp_status sbp_embedding_backward(const sbp_tensor* grad_out, const sbp_tensor* ids, sbp_tensor* grad_table,
                                             int32_t* oob_count, void* cuda_stream) {
  SBP_RANGE("sbp_embedding_backward");
  sbp_status st = check_tensor(grad_out, "grad_out", true);
  if (st != SBP_OK) return st;
  st = check_tensor(ids, "ids", true);
  if (st != SBP_OK) return st;
  st = check_tensor(grad_table, "grad_table", true);
  if (st != SBP_OK) return st;
  const sbp_tensor* dense_only[3] = {grad_out, ids, grad_table};
  const char* dense_names[3] = {"grad_out", "ids", "grad_table"};
  for (int i = 0; i < 3; ++i)
    if ((st = refuse_ld(dense_only[i], dense_names[i], "sbp_embedding_backward")) != SBP_OK) return st;
  if (grad_table->ndim != 2) return fail(SBP_ERR_SHAPE, "grad_table must be [rows, dim]");
  if (grad_table->dtype != SBP_F32 || grad_out->dtype != SBP_F32)
    return fail(SBP_ERR_DTYPE, "the embedding backward accumulates in F32: grad_out and grad_table must be F32");
  if (ids->dtype != SBP_I64) return fail(SBP_ERR_DTYPE, "ids must be I64");
  if (ids->ndim > 3 || grad_out->ndim != ids->ndim + 1) return fail(SBP_ERR_SHAPE, "grad_out rank must be ids rank + 1");
  for (int d = 0; d < ids->ndim; ++d)
    if (grad_out->shape[d] != ids->shape[d]) return fail(SBP_ERR_SHAPE, "grad_out and ids differ on axis %d", d);
  const long long dim = grad_table->shape[1];
  if (grad_out->shape[grad_out->ndim - 1] != dim) return fail(SBP_ERR_SHAPE, "grad_out's last axis must equal dim");
  const int k = placement_k(grad_table);
  if (placement_k(ids) != k || placement_k(grad_out) != k) return fail(SBP_ERR_INVALID_ARG, "operands differ in k");
  if (!(grad_table->sbp[0].kind == SBP_SPLIT && grad_table->sbp[0].axis == 0))
    return fail(SBP_ERR_SIGNATURE, "grad_table must be S(0), like the table");
  if (ids->sbp[0].kind != SBP_BROADCAST || grad_out->sbp[0].kind != SBP_BROADCAST)
    return fail(SBP_ERR_SIGNATURE, "ids and grad_out must be B");
  if (dim % 4 != 0) return fail(SBP_ERR_UNSUPPORTED, "dim must be a multiple of 4 (16-byte atomic adds)");
  for (int r = 0; r < k; ++r)
    if (reinterpret_cast<uintptr_t>(grad_table->local[r]) % 16 != 0)
      return fail(SBP_ERR_ALIGNMENT, "grad_table shards must be 16-byte aligned");
  if (reinterpret_cast<uintptr_t>(grad_out->local[0]) % 16 != 0) return fail(SBP_ERR_ALIGNMENT, "grad_out must be 16-byte aligned");
  if (dim == 0 || grad_table->shape[0] == 0) return SBP_OK;
  SBP_BOUNDS_RESET();
  SBP_BOUNDS_TENSOR(grad_out);
  SBP_BOUNDS_TENSOR(ids);
  SBP_BOUNDS_TENSOR(grad_table);
  SBP_BOUNDS_ADD(oob_count, 4);

  EmbBwdParams p{};
  p.k = k;
  p.rows = grad_table->shape[0];
  p.base = p.rows / k;
  p.rem = p.rows % k;
  p.big = p.rem * (p.base + 1);
  p.narrow = p.rows < (1LL << 31) ? 1 : 0;
  p.n_lookups = numel(ids);
  p.vpr = dim / 4;
  p.ids = static_cast<const long long*>(ids->local[0]);
  p.grad_out = static_cast<const float*>(grad_out->local[0]);
  p.oob = oob_count;
  long long max_vecs = 0;
  for (int r = 0; r < k; ++r) {
    p.grad_table[r] = static_cast<float*>(grad_table->local[r]);
    p.shard_vecs[r] = local_numel(grad_table, r) / 4;
    max_vecs = p.shard_vecs[r] > max_vecs ? p.shard_vecs[r] : max_vecs;
  }
  cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
  long long zb = (max_vecs + 256 * 8 - 1) / (256 * 8);
  if (zb < 1) zb = 1;
  if (zb > 148 * 16) zb = 148 * 16;
  SBP_BOUNDS_UPLOAD(stream);
  embedding_zero_kernel<<<dim3((unsigned)zb, (unsigned)k), 256, 0, stream>>>(p);
  cudaError_t e = cudaGetLastError();
  if (e != cudaSuccess) return cuda_fail(e, "embedding backward launch");
  count_launch();
  if (p.n_lookups > 0) {
    // 1024-lookup chunks once they fill the GPU a few times over, else 256-lookup chunks
    const bool big_chunks = p.n_lookups / 1024 >= 148 * 4;
    const long long chunks = (p.n_lookups + (big_chunks ? 1023 : 255)) / (big_chunks ? 1024 : 256);
    const unsigned sb = (unsigned)(chunks < 148 * 8 ? chunks : 148 * 8);
    if (big_chunks) embedding_backward_kernel<1024><<<sb, 256, 0, stream>>>(p);
    else embedding_backward_kernel<256><<<sb, 256, 0, stream>>>(p);
    e = cudaGetLastError();
    if (e != cudaSuccess) return cuda_fail(e, "embedding backward launch");
    count_launch();
  }
  return SBP_OK;
}

