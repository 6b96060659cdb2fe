// Bulk-copy engine for the pure data-movement boxing transforms (S(i)->S(j), S(i)->B,
// B->S(i)): the copy engine of the SM moves whole row segments global -> shared -> global
// (cp.async.bulk), so no register file traffic; one warp per CTA issues the copies.
//
// A persistent grid of small CTAs walks the same (task, segment rows, column chunk) tiles
// as the load/store kernel.  Each CTA owns a ring of kStages shared-memory buffers: the
// loads of tile i + kStages - 1 are in flight while tile i is being stored.  A tile is
// filled by one bulk load per segment (all signalling one mbarrier with the tile's byte
// count) and drained by one bulk store per segment per destination replica.
//
// Every wait is bounded.  If a wait expires the CTA records it in a device flag that
// sbp_check_device_errors() reports as SBP_ERR_TIMEOUT, drains its stores and returns.
#include <cuda_runtime.h>

#include "boxing_params.h"
#include "sbp_internal.h"

namespace sbp {

__device__ int g_bulk_timeout_flag = 0;

constexpr int kStages = 4;
constexpr int kStageBytes = 16 * 1024;
constexpr int kCtasPerSm = 3;
constexpr int kStoreSlack = 1;         // store groups that may still be reading shared memory when the next load is issued
constexpr unsigned long long kWaitLimitNs = 2000000000ull;   // 2 s

struct BulkParams {
  BoxParams b;
  long long row_tiles, col_tiles;   // tiling of one task for this engine
  long long tiles_per_task;
  int rows_per_tile;                // segments per tile
  long long chunk_bytes;            // column chunk of a segment (multiple of 16)
  long long total_tiles;
};

__device__ __forceinline__ unsigned smem_u32(const void* p) {
  return (unsigned)__cvta_generic_to_shared(p);
}

__device__ __forceinline__ unsigned long long global_ns() {
  unsigned long long t;
  asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
  return t;
}

// Waits for the phase with the given parity; gives up after kWaitLimitNs.
__device__ __forceinline__ bool mbar_wait(unsigned bar, unsigned parity) {
  const unsigned long long t0 = global_ns();
  for (;;) {
    unsigned done;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2, 0x10000;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(done)
        : "r"(bar), "r"(parity)
        : "memory");
    if (done) return true;
    if (global_ns() - t0 > kWaitLimitNs) return false;
  }
}

// One tile of one task: which shards, which segments, where they sit on both sides.  The fields
// below `cb` belong to the task and are the same for all of its tiles.
struct BulkTile {
  long long rows, bytes;      // segments in the tile, bytes of each segment piece
  long long seg0, cb;         // first segment, byte offset of the column chunk
  int s, d;
  long long nseg, seg_bytes;  // segments of the task, bytes of one segment
  long long la;
  long long Na_s, aoff_s, Nb_s, boff_s;
  long long Na_d, aoff_d, Nb_d, boff_d;
};

constexpr int kTaskCache = 64;   // tasks whose geometry a CTA keeps in shared memory

// The per-task part of a tile (several 64-bit divisions: worked out once per task, not per tile).
__device__ __forceinline__ BulkTile bulk_task(const BoxParams& p, int t) {
  BulkTile g;
  g.s = t;
  g.d = t;
  if (p.one_dst) { g.d = p.dst_shard; if (p.mode == MODE_DIAG) g.s = p.dst_shard; }
  else if (p.mode == MODE_PAIRS) { g.s = t / p.k; g.d = t - g.s * p.k; }
  long long a0 = 0, la = p.Na, b0 = 0, lb = p.Nb;
  if (p.src_a) split_range_pre(p.a_base, p.a_rem, g.s, &a0, &la);
  else if (p.dst_a) split_range_pre(p.a_base, p.a_rem, g.d, &a0, &la);
  if (p.src_b) split_range_pre(p.b_base, p.b_rem, g.s, &b0, &lb);
  else if (p.dst_b) split_range_pre(p.b_base, p.b_rem, g.d, &b0, &lb);
  g.nseg = p.A * la * p.M;
  g.seg_bytes = lb * p.C * p.esz;
  g.la = la;
  g.Na_s = p.src_a ? la : p.Na;  g.aoff_s = p.src_a ? 0 : a0;
  g.Nb_s = p.src_b ? lb : p.Nb;  g.boff_s = p.src_b ? 0 : b0;
  g.Na_d = p.dst_a ? la : p.Na;  g.aoff_d = p.dst_a ? 0 : a0;
  g.Nb_d = p.dst_b ? lb : p.Nb;  g.boff_d = p.dst_b ? 0 : b0;
  g.rows = g.bytes = g.seg0 = g.cb = 0;
  return g;
}

// Tile number u (below 2^31, checked on the host): task index fastest, then column chunk, then rows.
__device__ __forceinline__ BulkTile bulk_tile(const BulkParams& q, const BulkTile* task_cache, unsigned u) {
  const BoxParams& p = q.b;
  const unsigned ntasks = (unsigned)p.ntasks, col_tiles = (unsigned)q.col_tiles;
  const unsigned rem = u / ntasks, t = u - rem * ntasks;
  const unsigned row_tile = rem / col_tiles, col_tile = rem - row_tile * col_tiles;
  BulkTile g = t < (unsigned)kTaskCache ? task_cache[t] : bulk_task(p, (int)t);
  g.seg0 = (long long)row_tile * q.rows_per_tile;
  g.cb = (long long)col_tile * q.chunk_bytes;
  g.rows = g.nseg - g.seg0 < q.rows_per_tile ? g.nseg - g.seg0 : q.rows_per_tile;
  g.bytes = g.seg_bytes - g.cb < q.chunk_bytes ? g.seg_bytes - g.cb : q.chunk_bytes;
  return g;
}

// Byte offsets of the start of segment `seg` inside the source and destination buffers.
__device__ __forceinline__ void seg_offsets(const BoxParams& p, const BulkTile& g, long long seg, long long* so,
                                            long long* dofs) {
  const long long cs = p.C * p.esz;
  long long x = 0, ia = seg, m = 0;
  if (!(p.A == 1 && p.M == 1)) {
    const long long q = seg / p.M;
    m = seg - q * p.M;
    x = q / g.la;
    ia = q - x * g.la;
  }
  *so = (((x * g.Na_s + g.aoff_s + ia) * p.M + m) * g.Nb_s + g.boff_s) * cs;
  *dofs = (((x * g.Na_d + g.aoff_d + ia) * p.M + m) * g.Nb_d + g.boff_d) * cs;
}

__global__ void __launch_bounds__(32) box_bulk_kernel(const __grid_constant__ BulkParams q) {
  extern __shared__ __align__(128) unsigned char smem[];
  __shared__ __align__(8) unsigned long long bars[kStages];
  __shared__ BulkTile tiles[kStages];          // geometry of the tile in each ring slot, computed once
  __shared__ BulkTile task_cache[kTaskCache];  // per-task geometry
  const BoxParams& p = q.b;
  const int lane = threadIdx.x;

  if (lane == 0) {
    for (int i = 0; i < kStages; ++i)
      asm volatile("mbarrier.init.shared::cta.b64 [%0], 1;" ::"r"(smem_u32(&bars[i])) : "memory");
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  }
  for (int t = lane; t < p.ntasks && t < kTaskCache; t += 32) task_cache[t] = bulk_task(p, t);
  __syncwarp();

  const long long first = blockIdx.x, stride = gridDim.x;
  const long long n_mine = first < q.total_tiles ? (q.total_tiles - first + stride - 1) / stride : 0;
  bool timed_out = false;

  // Loads of my tile number `it` into its ring slot: one bulk copy per segment, lane r issuing
  // the copies of segments r, r + 32, ...  Lane 0 works out the tile and posts the byte count.
  auto issue_loads = [&](long long it) {
    const int slot = (int)(it % kStages);
    const unsigned bar = smem_u32(&bars[slot]);
    if (lane == 0) {
      const BulkTile t = bulk_tile(q, task_cache, (unsigned)(first + it * stride));
      tiles[slot] = t;
      if (t.rows <= 0 || t.bytes <= 0)           // tile outside an uneven shard: complete the phase empty
        asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
      else
        asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar),
                     "r"((unsigned)(t.rows * t.bytes))
                     : "memory");
    }
    __syncwarp();
    const BulkTile& g = tiles[slot];
    if (g.rows <= 0 || g.bytes <= 0) return;
    unsigned char* buf = smem + (size_t)slot * kStageBytes;
    for (long long r = lane; r < g.rows; r += 32) {
      long long so, dofs;
      seg_offsets(p, g, g.seg0 + r, &so, &dofs);
      asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(
                       smem_u32(buf + r * g.bytes)),
                   "l"(p.src[g.s] + so + g.cb), "r"((unsigned)g.bytes), "r"(bar)
                   : "memory");
    }
  };

  // Stores of my tile number `it` out of its ring slot, once per destination replica; every lane
  // commits its own (possibly empty) group so that the group counts of all lanes stay in step.
  auto issue_stores = [&](long long it) {
    const int slot = (int)(it % kStages);
    const BulkTile& g = tiles[slot];
    if (g.rows > 0 && g.bytes > 0) {
      unsigned char* buf = smem + (size_t)slot * kStageBytes;
      const int nd = p.mode == MODE_GATHER ? p.n_dst : 1;
      for (long long r = lane; r < g.rows; r += 32) {
        long long so, dofs;
        seg_offsets(p, g, g.seg0 + r, &so, &dofs);
        for (int j = 0; j < nd; ++j) {
          char* base = p.mode == MODE_GATHER ? p.dst[j] : p.dst[g.d];
          asm volatile("cp.async.bulk.global.shared::cta.bulk_group [%0], [%1], %2;" ::"l"(base + dofs + g.cb),
                       "r"(smem_u32(buf + r * g.bytes)), "r"((unsigned)g.bytes)
                       : "memory");
        }
      }
    }
    asm volatile("cp.async.bulk.commit_group;" ::: "memory");
  };

  const long long prologue = n_mine < kStages - kStoreSlack ? n_mine : kStages - kStoreSlack;
  for (long long it = 0; it < prologue; ++it) issue_loads(it);

  for (long long it = 0; it < n_mine; ++it) {
    const int slot = (int)(it % kStages);
    const unsigned parity = (unsigned)((it / kStages) & 1);
    // every lane observes the phase itself before it hands the buffer to its stores
    const bool ok = mbar_wait(smem_u32(&bars[slot]), parity);
    if (!__all_sync(0xffffffffu, ok)) {
      timed_out = true;
      break;
    }
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    issue_stores(it);
    // The slot that tile it + kStages - kStoreSlack will use was last drained by tile
    // it - kStoreSlack: every lane waits until all of its store groups except the newest
    // kStoreSlack have finished reading shared memory, and the warp meets before anyone loads
    // into that slot.
    const long long nxt = it + kStages - kStoreSlack;
    if (nxt < n_mine) {
      asm volatile("cp.async.bulk.wait_group.read %0;" ::"n"(kStoreSlack) : "memory");
      __syncwarp();
      issue_loads(nxt);
    }
  }
  asm volatile("cp.async.bulk.wait_group 0;" ::: "memory");
  if (timed_out && lane == 0) atomicExch(&g_bulk_timeout_flag, 1);
}

bool launch_bulk_copy(const BoxParams& p, int ntasks, cudaStream_t st) {
#ifdef SBP_DEBUG_BOUNDS
  // the copy engine's accesses cannot be checked one by one: the debug-bounds build keeps to the
  // load/store kernel, whose every address is
  (void)p; (void)ntasks; (void)st;
  return false;
#endif
  if (p.mode != MODE_PAIRS && p.mode != MODE_DIAG && p.mode != MODE_GATHER) return false;
  const int k = p.k;
  const long long la_max = (p.src_a || p.dst_a) ? (p.Na + k - 1) / k : p.Na;
  const long long lb_max = (p.src_b || p.dst_b) ? (p.Nb + k - 1) / k : p.Nb;
  const long long nseg_max = p.A * la_max * p.M;
  const long long seg_bytes_max = lb_max * p.C * p.esz;
  if (seg_bytes_max < 512) return false;   // too many tiny descriptors: the vector kernel is better
  BulkParams q;
  q.b = p;
  if (seg_bytes_max >= kStageBytes) {
    q.rows_per_tile = 1;
    q.chunk_bytes = kStageBytes;
  } else {
    q.rows_per_tile = (int)(kStageBytes / seg_bytes_max);
    q.chunk_bytes = seg_bytes_max;
  }
  q.col_tiles = (seg_bytes_max + q.chunk_bytes - 1) / q.chunk_bytes;
  q.row_tiles = (nseg_max + q.rows_per_tile - 1) / q.rows_per_tile;
  q.tiles_per_task = q.col_tiles * q.row_tiles;
  q.total_tiles = q.tiles_per_task * ntasks;
  if (q.total_tiles <= 0 || q.total_tiles > 0x7fffffffLL || q.col_tiles > 0x7fffffffLL) return false;

  // per device: SM count and the kernel's shared-memory opt-in
  static int sms_on_device[64] = {};
  const size_t smem = (size_t)kStages * kStageBytes;
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return false;
  if (sms_on_device[dev] == 0) {
    int sms = 0;
    if (cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess) return false;
    if (cudaFuncSetAttribute(box_bulk_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) !=
        cudaSuccess)
      return false;
    sms_on_device[dev] = sms;
  }
  const int sm_count = sms_on_device[dev];
  long long grid = (long long)sm_count * kCtasPerSm;
  if (grid > q.total_tiles) grid = q.total_tiles;
  box_bulk_kernel<<<(unsigned)grid, 32, smem, st>>>(q);
  return true;
}

// Self-test of the bounded-wait path: one thread waits on an mbarrier that nothing will ever
// signal, gives up after limit_ns and raises the same flag a real expiry raises.
__global__ void expire_wait_kernel(unsigned long long limit_ns) {
  __shared__ __align__(8) unsigned long long bar;
  if (threadIdx.x != 0) return;
  asm volatile("mbarrier.init.shared::cta.b64 [%0], 1;" ::"r"(smem_u32(&bar)) : "memory");
  asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  const unsigned long long t0 = global_ns();
  bool done = false;
  while (!done && global_ns() - t0 <= limit_ns) {
    unsigned ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2, 0x10000;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok)
        : "r"(smem_u32(&bar)), "r"(0u)
        : "memory");
    done = ok != 0;
  }
  if (!done) atomicExch(&g_bulk_timeout_flag, 1);
}

sbp_status launch_expire_wait(unsigned long long limit_ns, cudaStream_t st) {
  expire_wait_kernel<<<1, 32, 0, st>>>(limit_ns);
  cudaError_t e = cudaGetLastError();
  if (e != cudaSuccess) return cuda_fail(e, "self-test launch");
  count_launch();
  return SBP_OK;
}

sbp_status read_and_clear_bulk_timeout(bool* timed_out) {
  int flag = 0, zero = 0;
  SBP_CUDA_TRY(cudaMemcpyFromSymbol(&flag, g_bulk_timeout_flag, sizeof(int)));
  if (flag) SBP_CUDA_TRY(cudaMemcpyToSymbol(g_bulk_timeout_flag, &zero, sizeof(int)));
  *timed_out = flag != 0;
  return SBP_OK;
}

}  // namespace sbp
