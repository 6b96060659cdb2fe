// Tensor-core MatMul for sm_100a: bf16 operands, fp32 accumulation in tensor memory.
//
// Pairs of CTAs (a cluster of two SMs) walk the (group, m-tile, n-tile) list of a grouped-GEMM
// plan (matmul_plan.h).  A pair owns one 256 x 256 output tile at a time: CTA r of the pair
// holds rows 128 r .. 128 r + 127 of the A tile, columns 128 r .. 128 r + 127 of the B tile and
// rows 128 r .. of the accumulator in its own tensor memory; one tcgen05.mma.cta_group::2
// instruction, issued by the pair's first CTA, multiplies across both.  Per CTA and 64-deep
// K-block that is 16 KiB of A and 16 KiB of B through TMA for 2 x 128 x 256 x 64 MACs, two
// thirds of what two independent 128 x 256 CTAs would pull from L2.
//
//   warp 0     producer   TMA loads of this CTA's A and B halves into a kStages-deep ring; the
//                         transaction bytes of both CTAs land on the first CTA's "full" barrier
//   warp 1     MMA        (first CTA only) one thread issues four M256 N256 K16 MMAs per K-block
//                         into one of two 256-column accumulators; tcgen05.commit, delivered to
//                         both CTAs, frees the ring slot / publishes the accumulator
//   warps 2-9  epilogue   warp w drains lanes 32 (w mod 4) .. +31, columns 128 ((w-2)/4) .. +127
//                         of its CTA's accumulator (tcgen05.ld), applies GeLU when asked, rounds
//                         to the output type, stages 32 x 128-byte slabs in swizzled shared memory
//                         and writes them with TMA stores, once per destination replica, while
//                         the next tile's MMAs fill the other accumulator
//
// A fused "P(sum) product written as B / S(i)" plan simply chains the K-blocks of all shards'
// operands, in rank order, into the same accumulator: the partial products are never stored.
//
// Every barrier wait is bounded in time (the one wait that is not is the allocation of tensor memory
// at the start, which cannot block: the shared-memory footprint keeps the kernel to one CTA per SM,
// so the CTA is alone on its SM's tensor memory).  A wait that expires raises a flag that
// sbp_check_device_errors() reports; the CTA then stops issuing work, waits (bounded) for the
// loads it still has in flight, meets its partner at the closing cluster barrier, frees its
// tensor memory and returns.
#include <cuda.h>
#include <cuda_bf16.h>
#include <cuda_runtime.h>

#include <algorithm>
#include <atomic>
#include <cstdlib>
#include <mutex>
#include <type_traits>

#include "bounds_check.h"
#include "matmul_plan.h"
#include "sbp_internal.h"

namespace sbp {

constexpr int BM = 256, BN = 256, BK = 64;      // tile of a CTA pair
constexpr int BMH = BM / 2, BNH = BN / 2;       // what one CTA of the pair loads
constexpr int kStages = 6;                        // 6 slots + 1 staging slab per warp beat 5 + 2 once the hand-back of an accumulator was cheap
constexpr int kStageA = BMH * BK * 2;             // 16 KiB
constexpr int kStageB = BK * BNH * 2;             // 16 KiB
constexpr int kStageBytes = kStageA + kStageB;    // 32 KiB per CTA
constexpr int kEpiWarps = 8;
constexpr int kSlabBytes = 32 * 128;              // one epilogue slab: 32 rows x 128 bytes
constexpr int kEpiBufs = 1;                       // staging slabs per epilogue warp
constexpr int kEpiBytes = kEpiWarps * kEpiBufs * kSlabBytes;
constexpr int kSmemBytes = kStages * kStageBytes + kEpiBytes + 1024;   // + alignment slack
// The tall form (MH = 2): a CTA pair owns a 512 x 256 tile -- two m-halves of 256 rows that share
// every B slice -- with BOTH 256-column accumulators in use at once.  A 64-deep K-block then brings
// 48 KiB per CTA into shared memory for 2 x 4 MMAs (1024 clocks) instead of 32 KiB for 4 MMAs
// (512 clocks): a quarter less operand traffic per MMA clock, both from L2 and through shared
// memory.  At the square form's rate the shared-memory data path has to carry one 128-byte
// wavefront every clock (TMA writes + MMA reads) and the tensor pipe reaches 76 %; with the
// slack the tall form leaves it runs the main loop at full rate.  The price is that the
// epilogue of a tile no longer overlaps the next tile's MMAs in full (the second accumulator is
// not a spare any more), which a long contraction repays many times over and a short one does not:
// the host picks the form per product.
constexpr int kStagesTall = 4;
constexpr int kStageBytesTall = 2 * kStageA + kStageB;     // 48 KiB per CTA
constexpr int kEpiBufsTall = 1;
constexpr int kSmemBytesTall = kStagesTall * kStageBytesTall + kEpiWarps * kEpiBufsTall * kSlabBytes + 1024;
constexpr int kMaxStages = kStages > kStagesTall ? kStages : kStagesTall;
constexpr int kThreadsTc = 32 * (2 + kEpiWarps);
constexpr int kTmemCols = 512;
constexpr unsigned long long kWaitLimitNs = 2000000000ull;

__device__ int g_tc_timeout_flag = 0;

struct TcParams {
  CUtensorMap map_a[SBP_MAX_K];
  CUtensorMap map_b[SBP_MAX_K];
  CUtensorMap map_y[SBP_MAX_K];
  CUtensorMap map_rep[SBP_MAX_K];
  long long m[SBP_MAX_K], n[SBP_MAX_K], row_off[SBP_MAX_K], col_off[SBP_MAX_K];
  int kblocks[SBP_MAX_K];       // per segment
  int tile_begin[SBP_MAX_K + 1];   // prefix sum of tiles per group
  int tiles_m[SBP_MAX_K];
  int tiles_n[SBP_MAX_K];
  int mt_begin[SBP_MAX_K + 1];     // stacked == 1: prefix sum of m-tiles per group; == 2: of n-tiles
  int stacked;                     // the groups are row (1) / column (2) blocks of one result and are walked as one grid
  int ngroups, nseg, chain, gelu, n_rep;
  int out_f32;
  int total_tiles;
  unsigned panel_magic[SBP_MAX_K];   // floor(2^32 / (kPanelM * n-tiles)) of the group (stacked walks: entry 0, of the whole list)
  int walk_m;                   // rows of a walked tile: 256, or 512 (tall form and the square remainder of a mixed run)
  int tile_first;               // index of the first walked tile of this launch
  int half_split;               // square form over 512-row walked tiles: launch tile 2t + h is m-half h of walked tile t
  int xent;                     // 1: softmax partials instead of stored logits
  XentFusion xf;
  // Results the copy engine cannot address (a base or a row pitch that is not a multiple of 16
  // bytes): the epilogue then writes its staged slabs itself, row by row, with element-wise stores.
  int y_direct;
  void* y_ptr[SBP_MAX_K];
  void* rep_ptr[SBP_MAX_K];
  long long ldy[SBP_MAX_K];
};

// ------------------------------------------------------------------ PTX helpers

__device__ __forceinline__ unsigned smem_addr(const void* p) { return (unsigned)__cvta_generic_to_shared(p); }

__device__ __forceinline__ unsigned long long now_ns() {
  unsigned long long t;
  asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
  return t;
}

__device__ __forceinline__ void mbar_init(unsigned bar, unsigned count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}

// One try_wait with a suspend-time hint: the thread sleeps in hardware until the phase completes
// or the hint (in ns) runs out, instead of spinning and taking issue slots and power from the
// tensor pipe (measured: +8 % MatMul throughput against a bare polling loop).
__device__ __forceinline__ bool mbar_try(unsigned bar, unsigned parity) {
  unsigned done;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2, 0x10000;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(done)
      : "r"(bar), "r"(parity)
      : "memory");
  return done != 0;
}

// Bounded wait.  Returns false (and raises the abort flag) when the limit expires.
__device__ __forceinline__ bool mbar_wait(unsigned bar, unsigned parity, volatile int* abort_flag) {
  if (mbar_try(bar, parity)) return true;
  const unsigned long long t0 = now_ns();
  for (;;) {
    if (mbar_try(bar, parity)) return true;
    if (*abort_flag) return false;
    if (now_ns() - t0 > kWaitLimitNs) {
      *abort_flag = 1;
      atomicExch(&g_tc_timeout_flag, 1);
      return false;
    }
  }
}

__device__ __forceinline__ void mbar_expect_tx(unsigned bar, unsigned bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}

__device__ __forceinline__ void mbar_arrive(unsigned bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}

// Address of the same shared-memory object in CTA `rank` of this cluster.
__device__ __forceinline__ unsigned map_to_cta(unsigned addr, unsigned rank) {
  unsigned r;
  asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(addr), "r"(rank));
  return r;
}

// Arrive on an mbarrier that may live in the partner CTA (cluster-space address).  The arrive
// carries the default (CTA-scope) release: what it hands over is tensor memory whose reads have
// completed (tcgen05.wait::ld, then tcgen05.fence::before_thread_sync), not data in memory, and a
// cluster-scope release here cost every epilogue warp some thousand clocks per tile (fused
// classifier forward 0.472 -> 0.450 ms, backward 0.577 -> 0.533 ms).
__device__ __forceinline__ void mbar_arrive_cluster(unsigned cluster_addr) {
  asm volatile("mbarrier.arrive.shared::cluster.b64 _, [%0];" ::"r"(cluster_addr) : "memory");
}

__device__ __forceinline__ unsigned cluster_ctarank() {
  unsigned r;
  asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
  return r;
}

__device__ __forceinline__ void cluster_sync_all() {
  asm volatile("barrier.cluster.arrive.release;" ::: "memory");
  asm volatile("barrier.cluster.wait.acquire;" ::: "memory");
}

// TMA load into this CTA's shared memory; the byte count is credited to `bar`, which may be the
// partner CTA's barrier (pair form of the instruction; no multicast).
__device__ __forceinline__ void tma_load_2d(unsigned dst, const CUtensorMap* map, int x, int y, unsigned bar) {
  asm volatile(
      "cp.async.bulk.tensor.2d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];" ::"r"(dst),
      "l"(map), "r"(x), "r"(y), "r"(bar)
      : "memory");
}

__device__ __forceinline__ void tma_store_2d(const CUtensorMap* map, int x, int y, unsigned src) {
  asm volatile("cp.async.bulk.tensor.2d.global.shared::cta.bulk_group [%0, {%1, %2}], [%3];" ::"l"(map), "r"(x),
               "r"(y), "r"(src)
               : "memory");
}

// One MMA across the CTA pair: D[256 x 256] (+)= A[256 x 16] * B[16 x 256].
__device__ __forceinline__ void umma_bf16(unsigned d_tmem, unsigned long long a_desc, unsigned long long b_desc,
                                          unsigned idesc, unsigned accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::2.kind::f16 [%0], %1, %2, %3, p;\n\t}" ::"r"(d_tmem),
      "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate)
      : "memory");
}

// Arrives on the barrier at this offset in BOTH CTAs of the pair once every tcgen05 operation
// issued so far by this thread is done.
__device__ __forceinline__ void umma_commit_pair(unsigned bar) {
  const unsigned short mask = 3;
  asm volatile("tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.multicast::cluster.b64 [%0], %1;" ::"r"(bar),
               "h"(mask)
               : "memory");
}

__device__ __forceinline__ void tmem_ld32(unsigned taddr, float* v) {
  unsigned* r = reinterpret_cast<unsigned*>(v);
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
      "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
      "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]),
        "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]), "=r"(r[16]),
        "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]), "=r"(r[24]),
        "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
      : "r"(taddr)
      : "memory");
}

// Shared-memory matrix descriptor, 128-byte swizzle (lbo / sbo in bytes): bits 0-13 start address
// >> 4, bits 16-29 lbo >> 4, bits 32-45 sbo >> 4, bit 46 the descriptor version of this architecture,
// bits 61-63 = 2 the 128-byte swizzle.  It is handled in two parts: what never changes (the high
// word, and the leading-dimension field of the low word) and the start-address field, so that the
// MMA-issuing thread builds a descriptor with one add and one register pair.
__host__ __device__ constexpr unsigned desc_lo_fixed(unsigned lbo) { return (lbo >> 4) << 16; }
__host__ __device__ constexpr unsigned desc_hi_fixed(unsigned sbo) { return (sbo >> 4) | (1u << 14) | (2u << 29); }
__device__ __forceinline__ unsigned long long desc_pack(unsigned lo, unsigned hi) {
  unsigned long long d;
  asm("mov.b64 %0, {%1, %2};" : "=l"(d) : "r"(lo), "r"(hi));
  return d;
}

// Instruction descriptor: D fp32, A and B bf16, M = 256 (pair), N = 256.  Bit 15 / bit 16 say
// that A / B lies in shared memory with its M / N index contiguous ("MN-major") instead of its
// K index.  Operands as given: A [M,K] row-major is K-major, B [K,N] row-major is N-major; a
// transposed operand is the other way round.
constexpr unsigned kIdescBase = (1u << 4) | (1u << 7) | (1u << 10) | ((BN >> 3) << 17) | ((BM >> 4) << 24);
__host__ __device__ constexpr unsigned make_idesc(int a_trans, int b_trans) {
  return kIdescBase | ((a_trans ? 1u : 0u) << 15) | ((b_trans ? 0u : 1u) << 16);
}

// erf by the rational approximation 7.1.26 of Abramowitz & Stegun (|error| <= 1.5e-7), which is
// far below the rounding of the bf16 / fp32 store that follows and costs two special-function
// operations where erff costs a long polynomial.
__device__ __forceinline__ float erf_as(float x) {
  const float ax = fabsf(x);
  float t;
  asm("rcp.approx.ftz.f32 %0, %1;" : "=f"(t) : "f"(fmaf(0.3275911f, ax, 1.0f)));
  float poly = fmaf(1.061405429f, t, -1.453152027f);
  poly = fmaf(poly, t, 1.421413741f);
  poly = fmaf(poly, t, -0.284496736f);
  poly = fmaf(poly, t, 0.254829592f);
  poly *= t;
  float e;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(e) : "f"(-ax * ax * 1.4426950408889634f));
  return copysignf(fmaf(-poly, e, 1.0f), x);
}

__device__ __forceinline__ float gelu_erf_tc(float v) { return 0.5f * v * (1.0f + erf_as(v * 0.70710678118654752440f)); }

struct TileCoord {
  int g, m0, n0;
};

// Tiles of a group are walked in panels of kPanelM m-tiles: inside a panel the m-tile index varies
// fastest and the n-tile index steps once per column of the panel, so that the CTA pairs running at
// the same time cover a roughly square patch of the output and share both their A rows and their B
// columns in L2.
constexpr int kPanelM = 8;

// n / d for 0 <= n < 2^31 and d >= 2 with magic = floor(2^32 / d): the high product is short of the
// quotient by at most one or two, which the loop makes up.  (The tile walk divides twice per tile
// in each of three roles; the generic division is a few hundred clocks of the one thread that
// issues the MMAs.)
__device__ __forceinline__ int div_by(int n, int d, unsigned magic) {
  int q = (int)__umulhi((unsigned)n, magic);
  while (n - q * d >= d) ++q;
  return q;
}

// position inside a panel of pm m-tiles: pm is kPanelM everywhere but in a group's last panel
__device__ __forceinline__ int div_panel(int rem, int pm) { return pm == kPanelM ? rem / kPanelM : rem / pm; }

__device__ __forceinline__ TileCoord tile_coord(const TcParams& p, int tile) {
  int half_m = 0;
  if (p.half_split) {
    half_m = (tile & 1) * BM;
    tile >>= 1;
  }
  tile += p.tile_first;
  if (p.stacked == 2) {
    // The same for a fused product written as S(1): column blocks of one result, which share every
    // A row block; the n-tiles of all groups form one list.
    const int tm = p.tiles_m[0], tn = p.mt_begin[p.ngroups];
    const int panel = div_by(tile, kPanelM * tn, p.panel_magic[0]);
    const int rem = tile - panel * (kPanelM * tn);
    const int pm = min(kPanelM, tm - panel * kPanelM);
    const int nt = div_panel(rem, pm), mt = panel * kPanelM + (rem - nt * pm);
    int g = 0;
    while (g + 1 < p.ngroups && nt >= p.mt_begin[g + 1]) ++g;
    return TileCoord{g, mt * p.walk_m + half_m, (nt - p.mt_begin[g]) * BN};
  }
  if (p.stacked) {
    // A fused product written as S(0): the groups are the row blocks of ONE result and share every
    // B column block.  Walking them one after the other would stream the whole B operand once per
    // group; instead the m-tiles of all groups form one list and the panel walk runs over that.
    const int tm = p.mt_begin[p.ngroups], tn = p.tiles_n[0];
    const int panel = div_by(tile, kPanelM * tn, p.panel_magic[0]);
    const int rem = tile - panel * (kPanelM * tn);
    const int pm = min(kPanelM, tm - panel * kPanelM);
    const int nt = div_panel(rem, pm), mt = panel * kPanelM + (rem - nt * pm);
    int g = 0;
    while (g + 1 < p.ngroups && mt >= p.mt_begin[g + 1]) ++g;
    return TileCoord{g, (mt - p.mt_begin[g]) * p.walk_m + half_m, nt * BN};
  }
  int g = 0;
  while (g + 1 < p.ngroups && tile >= p.tile_begin[g + 1]) ++g;
  const int local = tile - p.tile_begin[g];
  const int tm = p.tiles_m[g], tn = p.tiles_n[g];
  const int panel = div_by(local, kPanelM * tn, p.panel_magic[g]);
  const int rem = local - panel * (kPanelM * tn);
  const int pm = min(kPanelM, tm - panel * kPanelM);   // m-tiles in this (possibly last) panel
  const int nt = div_panel(rem, pm), mt = panel * kPanelM + (rem - nt * pm);
  return TileCoord{g, mt * p.walk_m + half_m, nt * BN};
}

// ------------------------------------------------------------------ the kernel

// AT / BT: operand A / B is stored transposed.  They are compile-time so that the usual
// (untransposed) form carries no trace of the other three: as run-time switches they cost the
// MMA-issuing thread and the producer enough to slow every product by 6 %.
// MH: m-halves of 256 rows per pair tile (1 = square form, 2 = tall form, see kStageBytesTall).
template <int AT, int BT, int MH>
__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(kThreadsTc, 1)
    matmul_tc_kernel(const __grid_constant__ TcParams p) {
  constexpr int kSt = MH == 2 ? kStagesTall : kStages;                  // ring depth
  constexpr int kStA = MH * kStageA;                                    // bytes of A per ring slot
  constexpr int kStBytes = kStA + kStageB;
  constexpr int kEB = MH == 2 ? kEpiBufsTall : kEpiBufs;                // staging slabs per epilogue warp
  extern __shared__ unsigned char smem_raw[];
  __shared__ __align__(8) unsigned long long bar_full[kMaxStages], bar_empty[kMaxStages], bar_acc_full[2], bar_acc_empty[2];
  __shared__ unsigned tmem_base_slot;
  __shared__ int abort_flag_s;
  volatile int* abort_flag = &abort_flag_s;

  unsigned char* smem = reinterpret_cast<unsigned char*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  unsigned char* epi = smem + kSt * kStBytes;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const unsigned rank = cluster_ctarank();     // 0 = the CTA that issues the pair's MMAs

  if (threadIdx.x == 0) {
    abort_flag_s = 0;
    for (int i = 0; i < kSt; ++i) {
      mbar_init(smem_addr(&bar_full[i]), 1);      // used in CTA 0 only: one arrive + both CTAs' bytes
      mbar_init(smem_addr(&bar_empty[i]), 1);     // one commit per use, delivered to both CTAs
    }
    for (int i = 0; i < 2; ++i) {
      mbar_init(smem_addr(&bar_acc_full[i]), 1);
      mbar_init(smem_addr(&bar_acc_empty[i]), 2 * kEpiWarps);   // used in CTA 0 only: both CTAs' epilogue warps
    }
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  }
  if (warp == 1) {
    asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_addr(&tmem_base_slot)),
                 "r"(kTmemCols)
                 : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
  }
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
  __syncthreads();
  cluster_sync_all();                            // both CTAs' barriers exist before anyone signals them
  asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
  const unsigned tmem_base = tmem_base_slot;
  // A kernel launched behind this one as its programmatic dependent may be set up from here on;
  // it waits on the device for this grid to finish before it reads what this grid writes.
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");

  const int first = blockIdx.x >> 1, stride = gridDim.x >> 1;   // tiles are dealt to CTA pairs

  if (warp == 0) {
    // ------------------------------------------------ producer (both CTAs)
    if (lane == 0) {
      // ring position kept as (slot, round parity) and stepped, not divided out of a running count:
      // with a slot count that is not a power of two the division is a long instruction sequence,
      // once per K-block
      long long kb_iter = 0;
      int slot = 0;
      unsigned round = 0;
      for (int tile = first; tile < p.total_tiles && !*abort_flag; tile += stride) {
        const TileCoord tc = tile_coord(p, tile);
        const int s_lo = p.chain ? 0 : tc.g, s_hi = p.chain ? p.nseg : tc.g + 1;
        for (int s = s_lo; s < s_hi; ++s) {
          const int nkb = p.kblocks[s];
          for (int kb = 0; kb < nkb; ++kb, ++kb_iter, slot = slot + 1 == kSt ? 0 : slot + 1, round ^= (slot == 0)) {
            const unsigned parity = round ^ 1;
            if (!mbar_wait(smem_addr(&bar_empty[slot]), parity, abort_flag)) goto producer_done;
            const unsigned full0 = map_to_cta(smem_addr(&bar_full[slot]), 0);
            if (rank == 0) mbar_expect_tx(smem_addr(&bar_full[slot]), 2 * kStBytes);
            unsigned char* sa0 = smem + slot * kStBytes;
            unsigned char* sb = sa0 + kStA;
            const int bcol = (int)p.col_off[tc.g] + tc.n0 + (int)rank * BNH;
#pragma unroll
            for (int h = 0; h < MH; ++h) {       // this CTA's 128 rows of every m-half
              unsigned char* sa = sa0 + h * kStageA;
              const int arow = (int)p.row_off[tc.g] + tc.m0 + h * BM + (int)rank * BMH;
              if constexpr (!AT) {   // [rows, K] in memory: one box of 128 rows x 64 K
                tma_load_2d(smem_addr(sa), &p.map_a[s], kb * BK, arow, full0);
              } else {            // [K, rows] in memory: two boxes of 64 K x 64 rows
#pragma unroll
                for (int c = 0; c < BMH / 64; ++c)
                  tma_load_2d(smem_addr(sa + c * (BK * 128)), &p.map_a[s], arow + c * 64, kb * BK, full0);
              }
            }
            if constexpr (!BT) {   // [K, cols] in memory: two boxes of 64 K x 64 columns
#pragma unroll
              for (int c = 0; c < BNH / 64; ++c)
                tma_load_2d(smem_addr(sb + c * (BK * 128)), &p.map_b[s], bcol + c * 64, kb * BK, full0);
            } else {            // [cols, K] in memory: one box of 128 columns x 64 K
              tma_load_2d(smem_addr(sb), &p.map_b[s], kb * BK, bcol, full0);
            }
          }
        }
      }
    producer_done:
      if (*abort_flag && rank == 0) {
        // give the loads still in flight a bounded chance to land before the CTA goes away
        const long long issued = kb_iter;
        for (long long i = issued > kSt ? issued - kSt : 0; i < issued; ++i) {
          const unsigned long long t0 = now_ns();
          while (!mbar_try(smem_addr(&bar_full[i % kSt]), (unsigned)((i / kSt) & 1)) && now_ns() - t0 < 100000000ull) {
          }
        }
      }
    }
  } else if (warp == 1) {
    // ------------------------------------------------ MMA issuer (first CTA of the pair only)
    if (lane == 0 && rank == 0) {
      int slot = 0;
      unsigned round = 0;
      int tile_iter = 0;
      constexpr unsigned idesc = make_idesc(AT, BT);
      for (int tile = first; tile < p.total_tiles && !*abort_flag; tile += stride, ++tile_iter) {
        const TileCoord tc = tile_coord(p, tile);
        // Square form: the two accumulators take turns, so a tile's MMAs run while the tile before
        // it is drained.  Tall form: accumulator h belongs to m-half h of every tile; the first
        // m-half may start as soon as ITS accumulator has been drained, the second waits for its own.
        const int acc = MH == 2 ? 0 : (tile_iter & 1);
        const unsigned empty_parity = MH == 2 ? (unsigned)((tile_iter & 1) ^ 1) : (unsigned)(((tile_iter >> 1) & 1) ^ 1);
        if (!mbar_wait(smem_addr(&bar_acc_empty[acc]), empty_parity, abort_flag)) break;
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
        const int s_lo = p.chain ? 0 : tc.g, s_hi = p.chain ? p.nseg : tc.g + 1;
        unsigned accumulate = 0;
        bool ok = true;
        for (int s = s_lo; s < s_hi && ok; ++s) {
          const int nkb = p.kblocks[s];
          for (int kb = 0; kb < nkb; ++kb, slot = slot + 1 == kSt ? 0 : slot + 1, round ^= (slot == 0)) {
            if (!mbar_wait(smem_addr(&bar_full[slot]), round, abort_flag)) {
              ok = false;
              break;
            }
            asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
            const unsigned sa0 = smem_addr(smem + slot * kStBytes);
            const unsigned sb = sa0 + kStA;
#pragma unroll
            for (int h = 0; h < MH; ++h) {
            if (MH == 2 && h == 1 && accumulate == 0) {      // first K-block of the tile: the second accumulator must be free too
              if (!mbar_wait(smem_addr(&bar_acc_empty[1]), empty_parity, abort_flag)) {
                ok = false;
                break;
              }
              asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
            }
            const unsigned sa = sa0 + h * kStageA;
            const unsigned d_tmem = tmem_base + (MH == 2 ? h : acc) * BN;
#pragma unroll
            for (int kk = 0; kk < BK / 16; ++kk) {
              // K-major tile (A as given, B transposed): rows of 128 bytes = 64 K-elements, 8-row
              //    groups 1024 bytes apart; 16 K-elements = 32 bytes.
              // MN-major tile (B as given, A transposed): 64-element chunks of the M / N index
              //    BK*128 bytes apart, 8-row K groups 1024 bytes apart; 16 K-rows = 2048 bytes.
              // Each CTA holds its 128 of the pair's 256 rows (A) or columns (B).
              // (shared-memory addresses are below 256 KiB and the tiles 1024-byte aligned, so the
              //  start-address field is address >> 4 and stepping it cannot carry out of the field)
              constexpr unsigned a_lo = desc_lo_fixed(AT ? BK * 128 : 16), b_lo = desc_lo_fixed(BT ? 16 : BK * 128);
              constexpr unsigned hi = desc_hi_fixed(1024);
              const unsigned long long da = desc_pack(a_lo + (sa >> 4) + kk * (AT ? 128 : 2), hi);
              const unsigned long long db = desc_pack(b_lo + (sb >> 4) + kk * (BT ? 2 : 128), hi);
              umma_bf16(d_tmem, da, db, idesc, kk == 0 ? accumulate : 1u);
            }
            }
            if (!ok) break;
            accumulate = 1;
            umma_commit_pair(smem_addr(&bar_empty[slot]));   // slot reusable in both CTAs
          }
        }
        if (!ok) break;
        umma_commit_pair(smem_addr(&bar_acc_full[acc]));      // accumulator(s) complete in both CTAs
      }
    }
  } else {
    // ------------------------------------------------ epilogue (warps 2..9, both CTAs)
    const int q = warp & 3;                       // the 32 tensor-memory lanes this warp may read
    const int half = (warp - 2) >> 2;             // which 128 of the 256 columns
    unsigned char* my_epi = epi + (warp - 2) * kEB * kSlabBytes;
    const int cols_per_slab = p.out_f32 ? 32 : 64;
    const int nslabs = (BN / 2) / cols_per_slab;
    const unsigned acc_empty0[2] = {map_to_cta(smem_addr(&bar_acc_empty[0]), 0), map_to_cta(smem_addr(&bar_acc_empty[1]), 0)};
    int tile_iter = 0;
    unsigned slab_iter = 0;
    for (int tile = first; tile < p.total_tiles; tile += stride, ++tile_iter) {
      if (*abort_flag) break;
      const TileCoord tc = tile_coord(p, tile);
      const int facc = MH == 2 ? 0 : (tile_iter & 1);
      bool ok = true;
      if (lane == 0)
        ok = mbar_wait(smem_addr(&bar_acc_full[facc]), MH == 2 ? (unsigned)(tile_iter & 1) : (unsigned)((tile_iter >> 1) & 1), abort_flag);
      ok = __shfl_sync(0xffffffffu, ok ? 1 : 0, 0) != 0;
      if (!ok) break;
      asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
      const long long Mg = p.m[tc.g], Ng = p.n[tc.g];
      // tall form: the accumulator of the first m-half is drained (and handed back) before the second
#pragma unroll 1
      for (int h = 0; h < MH; ++h) {
      const int acc = MH == 2 ? h : facc;
      const int row0 = tc.m0 + h * BM + (int)rank * BMH + q * 32;
      const unsigned taddr = tmem_base + ((unsigned)(q * 32) << 16) + acc * BN + half * (BN / 2);
      if (p.xent == 1) {
        // Softmax partials of this warp's 32 rows x 128 columns; one thread owns one row, so
        // nothing crosses lanes.  Columns are taken 32 at a time: batch max, then the running
        // (m, s) is rescaled and the batch's exponentials are added.
        constexpr float kL2e = 1.4426950408889634f;
        const int colbase = tc.n0 + half * (BN / 2);
        const long long row = row0 + lane;
        if (row0 < Mg && colbase < Ng) {            // warp-uniform
          float m = -INFINITY, s = 0.f, t = 0.f;
          long long want = -1;
          if (row < Mg && SBP_GUARD(p.xf.labels + row, 8)) want = p.xf.labels[row] - p.xf.class_start[tc.g] - colbase;
          for (int b = 0; b < 4; ++b) {
            const int c0 = colbase + b * 32;
            if (c0 >= Ng) break;                      // warp-uniform
            float v[32];
            tmem_ld32(taddr + b * 32, v);
            asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
            const int nvalid = (int)min((long long)32, Ng - c0);
            if (nvalid < 32) {
#pragma unroll
              for (int i = 0; i < 32; ++i)
                if (i >= nvalid) v[i] = -INFINITY;
            }
            float bm = v[0];
#pragma unroll
            for (int i = 1; i < 32; ++i) bm = fmaxf(bm, v[i]);
            const float mm = fmaxf(m, bm);
            const float neg = -mm * kL2e;
            float carried = 0.f;
            if (m != -INFINITY) {
              float e;
              asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(e) : "f"(fmaf(m, kL2e, neg)));
              carried = s * e;
            }
            float s0 = 0.f, s1 = 0.f;
#pragma unroll
            for (int i = 0; i < 32; i += 2) {
              float e0, e1;
              asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(e0) : "f"(fmaf(v[i], kL2e, neg)));
              asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(e1) : "f"(fmaf(v[i + 1], kL2e, neg)));
              s0 += e0;
              s1 += e1;
            }
            s = carried + (s0 + s1);
            m = mm;
          }
          // The label's logit: rows whose label falls inside this chunk (rare) re-read that one
          // column from tensor memory, one row at a time so the load stays warp-uniform.
          const long long ncols = min((long long)(BN / 2), Ng - colbase);
          unsigned hits = __ballot_sync(0xffffffffu, want >= 0 && want < ncols);
          while (hits) {
            const int src_lane = __ffs(hits) - 1;
            hits &= hits - 1;
            const int col = __shfl_sync(0xffffffffu, (int)want, src_lane);
            unsigned bitsv;
            asm volatile("tcgen05.ld.sync.aligned.32x32b.x1.b32 {%0}, [%1];" : "=r"(bitsv) : "r"(taddr + col) : "memory");
            asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
            if (lane == src_lane) t = __uint_as_float(bitsv);
          }
          if (row < Mg) {
            const long long slot = (long long)(p.xf.part_base[tc.g] + colbase / 128) * p.xf.rows + row;
            if (SBP_GUARD(p.xf.part_m + slot, 4)) p.xf.part_m[slot] = m;
            if (SBP_GUARD(p.xf.part_s + slot, 4)) p.xf.part_s[slot] = s;
            if (SBP_GUARD(p.xf.part_t + slot, 4)) p.xf.part_t[slot] = t;
          }
        }
      } else {
      // The element-wise modes are compiled apart (MODE 0 plain, 1 GeLU, 2 softmax - onehot of the
      // recomputed logits) so that the plain store, which the short-K classifier product leans
      // on, carries none of the others' instructions.
      // softmax = 2^(z log2e - m log2e - log2 S): the division by the row sum is folded into the exponent
      float g_neg = 0.f;
      long long g_lab = -1;
      if (p.xent == 2 && row0 + lane < Mg && SBP_GUARD(p.xf.row_max + row0 + lane, 4) &&
          SBP_GUARD(p.xf.row_sum + row0 + lane, 4) && SBP_GUARD(p.xf.labels + row0 + lane, 8)) {      // this thread's row constants
        const long long row = row0 + lane;
        g_neg = -p.xf.row_max[row] * 1.4426950408889634f - log2f(p.xf.row_sum[row]);
        g_lab = p.xf.labels[row] - p.xf.class_start[tc.g];
      }
      auto slabs = [&](auto mode_tag) {
        constexpr int MODE = decltype(mode_tag)::value;
        int lab_rel = -1;   // the label's column inside the current slab, if it lies there
        auto xform = [&](float x, int idx) -> float {
          if constexpr (MODE == 2) {
            float e;
            asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(e) : "f"(fmaf(x, 1.4426950408889634f, g_neg)));
            return e;          // the label's column gets its -1 below, outside the per-element path
          } else if constexpr (MODE == 1) {
            return gelu_erf_tc(x);
          } else {
            return x;
          }
        };
        for (int sl = 0; sl < nslabs; ++sl) {
          const int col0 = tc.n0 + half * (BN / 2) + sl * cols_per_slab;
          const bool live = row0 < Mg && col0 < Ng;   // warp-uniform
          if constexpr (MODE == 2) lab_rel = (g_lab >= col0 && g_lab < col0 + cols_per_slab) ? (int)(g_lab - col0) : -1;
          float v[64];
          if (live) {
            tmem_ld32(taddr + sl * cols_per_slab, v);
            if (!p.out_f32) tmem_ld32(taddr + sl * cols_per_slab + 32, v + 32);
            asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
            unsigned char* buf = my_epi + (slab_iter % kEB) * kSlabBytes;
            // the store that last used this buffer must have finished reading it
            if (lane == 0) asm volatile("cp.async.bulk.wait_group.read %0;" ::"n"(kEB - 1) : "memory");
            __syncwarp();
            unsigned char* rowp = buf + lane * 128;
            if (p.out_f32) {
#pragma unroll
              for (int c = 0; c < 8; ++c) {
                float4 o;
                o.x = xform(v[4 * c + 0], 4 * c + 0); o.y = xform(v[4 * c + 1], 4 * c + 1);
                o.z = xform(v[4 * c + 2], 4 * c + 2); o.w = xform(v[4 * c + 3], 4 * c + 3);
                *reinterpret_cast<float4*>(rowp + ((c ^ (lane & 7)) << 4)) = o;
              }
            } else {
#pragma unroll
              for (int c = 0; c < 8; ++c) {
                float f[8];
#pragma unroll
                for (int e = 0; e < 8; ++e) f[e] = xform(v[8 * c + e], 8 * c + e);
                uint4 o;
                __nv_bfloat162 h;
                h = __floats2bfloat162_rn(f[0], f[1]); o.x = *reinterpret_cast<unsigned*>(&h);
                h = __floats2bfloat162_rn(f[2], f[3]); o.y = *reinterpret_cast<unsigned*>(&h);
                h = __floats2bfloat162_rn(f[4], f[5]); o.z = *reinterpret_cast<unsigned*>(&h);
                h = __floats2bfloat162_rn(f[6], f[7]); o.w = *reinterpret_cast<unsigned*>(&h);
                *reinterpret_cast<uint4*>(rowp + ((c ^ (lane & 7)) << 4)) = o;
              }
            }
            if constexpr (MODE == 2) {
              // softmax - onehot: a row's label falls into this slab once in 2^14 slabs, so the -1 is
              // not a compare and a select on every element but a rare fix-up: the column is read
              // again from tensor memory (one row at a time, so the load stays warp-uniform) and the
              // staged element rewritten with exp - 1 computed in fp32 as before.
              unsigned hits = __ballot_sync(0xffffffffu, lab_rel >= 0);
              while (hits) {
                const int src_lane = __ffs(hits) - 1;
                hits &= hits - 1;
                const int col = __shfl_sync(0xffffffffu, lab_rel, src_lane);
                unsigned bitsv;
                asm volatile("tcgen05.ld.sync.aligned.32x32b.x1.b32 {%0}, [%1];" : "=r"(bitsv) : "r"(taddr + sl * cols_per_slab + col) : "memory");
                asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
                if (lane == src_lane) {
                  float e;
                  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(e) : "f"(fmaf(__uint_as_float(bitsv), 1.4426950408889634f, g_neg)));
                  e -= 1.0f;
                  if (p.out_f32) *reinterpret_cast<float*>(rowp + (((col >> 2) ^ (lane & 7)) << 4) + ((col & 3) << 2)) = e;
                  else *reinterpret_cast<__nv_bfloat16*>(rowp + (((col >> 3) ^ (lane & 7)) << 4) + ((col & 7) << 1)) = __float2bfloat16_rn(e);
                }
              }
              __syncwarp();
            }
            if (p.y_direct) {
              // rows of the slab, one after the other; the lanes take consecutive elements of a row
              __syncwarp();
              const int n_out = (tc.g == 0 ? p.n_rep : 0) + 1;
              for (int o = 0; o < n_out; ++o) {
                unsigned char* yb = static_cast<unsigned char*>(o == 0 ? p.y_ptr[tc.g] : p.rep_ptr[o - 1]);
                const long long ld = p.ldy[tc.g];
                for (int r = 0; r < 32 && row0 + r < Mg; ++r) {
                  const unsigned char* srow = buf + r * 128;
                  if (p.out_f32) {
                    const int c = lane;
                    if (col0 + c < Ng && SBP_GUARD(reinterpret_cast<float*>(yb) + (row0 + r) * ld + col0 + c, 4))
                      reinterpret_cast<float*>(yb)[(row0 + r) * ld + col0 + c] =
                          *reinterpret_cast<const float*>(srow + ((((c >> 2) ^ (r & 7)) << 4) | ((c & 3) << 2)));
                  } else {
#pragma unroll
                    for (int h = 0; h < 2; ++h) {
                      const int c = lane + 32 * h;
                      if (col0 + c < Ng && SBP_GUARD(reinterpret_cast<unsigned short*>(yb) + (row0 + r) * ld + col0 + c, 2))
                        reinterpret_cast<unsigned short*>(yb)[(row0 + r) * ld + col0 + c] =
                            *reinterpret_cast<const unsigned short*>(srow + ((((c >> 3) ^ (r & 7)) << 4) | ((c & 7) << 1)));
                    }
                  }
                }
              }
              __syncwarp();      // the buffer is rewritten two slabs from now
            } else {
            asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
            __syncwarp();
            if (lane == 0) {
              tma_store_2d(&p.map_y[tc.g], col0, row0, smem_addr(buf));
              if (tc.g == 0)
                for (int r = 0; r < p.n_rep; ++r) tma_store_2d(&p.map_rep[r], col0, row0, smem_addr(buf));
              asm volatile("cp.async.bulk.commit_group;" ::: "memory");
            }
            }
            ++slab_iter;
          }
        }
      };
      if (p.xent == 2) slabs(std::integral_constant<int, 2>{});
      else if (p.gelu) slabs(std::integral_constant<int, 1>{});
      else slabs(std::integral_constant<int, 0>{});
      }
      asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
      __syncwarp();
      if (lane == 0) mbar_arrive_cluster(acc_empty0[acc]);   // tells CTA 0's MMA thread
      }
    }
    if (lane == 0) asm volatile("cp.async.bulk.wait_group 0;" ::: "memory");
  }

  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
  __syncthreads();
  cluster_sync_all();          // the partner may still signal this CTA's barriers or read its tiles
  if (warp == 1) {
    __syncwarp();
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(kTmemCols) : "memory");
  }
}

// ------------------------------------------------------------------ host side

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

static EncodeTiledFn encode_fn() {
  static EncodeTiledFn fn = nullptr;
  static std::once_flag once;
  std::call_once(once, [] {
    void* ptr = nullptr;
    cudaDriverEntryPointQueryResult qres;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &ptr, cudaEnableDefault, &qres) == cudaSuccess &&
        qres == cudaDriverEntryPointSuccess)
      fn = reinterpret_cast<EncodeTiledFn>(ptr);
  });
  return fn;
}

// Tensor maps already encoded by this process, keyed by everything that goes into one.  A map holds
// nothing but the address and the layout, so an entry stays valid for as long as its key recurs: a
// product that is called again on the same buffers (every step of a training loop) encodes nothing.
// Two-way set-associative; used with the parameter block's lock held.
struct MapKey {
  const void* base;
  long long rows, cols, ld;
  int esz, box_rows, box_cols;
  bool operator==(const MapKey& o) const {
    return base == o.base && rows == o.rows && cols == o.cols && ld == o.ld && esz == o.esz && box_rows == o.box_rows &&
           box_cols == o.box_cols;
  }
};
struct MapSlot {
  CUtensorMap map;
  MapKey key;
  bool used;
};
constexpr int kMapCacheSets = 2048, kMapCacheWays = 2;
static MapSlot g_map_cache[kMapCacheSets][kMapCacheWays];
static unsigned char g_map_victim[kMapCacheSets];
static unsigned long long g_map_hits = 0, g_map_encodes = 0;

static unsigned map_slot_of(const MapKey& k) {
  unsigned long long h = reinterpret_cast<uintptr_t>(k.base) >> 4;
  auto mix = [&](unsigned long long v) { h = (h ^ v) * 0x9E3779B97F4A7C15ull; h ^= h >> 29; };
  mix((unsigned long long)k.rows);
  mix((unsigned long long)k.cols);
  mix((unsigned long long)k.ld);
  mix((unsigned long long)(k.esz | (k.box_rows << 8) | (k.box_cols << 20)));
  return (unsigned)(h % kMapCacheSets);
}

void tensor_map_cache_stats(unsigned long long* hits, unsigned long long* encodes) {
  *hits = g_map_hits;
  *encodes = g_map_encodes;
}

// launches of the kernel by form: square, tall, square over the halves that a mixed run leaves
static std::atomic<unsigned long long> g_form_launches[3];

// Overrides of the form choice and of the CTA pairs a launch may use (tests and measurements):
// set by tc_set_form, else taken once from SBP_TC_FORM (square | tall | mixed) and SBP_TC_PAIRS.
static std::atomic<int> g_forced_form{-1}, g_pair_cap{-1};

static int forced_form() {
  int v = g_forced_form.load();
  if (v < 0) {
    const char* e = getenv("SBP_TC_FORM");
    v = e ? (e[0] == 's' ? 1 : (e[0] == 't' ? 2 : (e[0] == 'm' ? 3 : 0))) : 0;
    g_forced_form.store(v);
  }
  return v;
}

static int pair_cap() {
  int v = g_pair_cap.load();
  if (v < 0) {
    const char* e = getenv("SBP_TC_PAIRS");
    v = e ? std::max(0, atoi(e)) : 0;
    g_pair_cap.store(v);
  }
  return v;
}

void tc_set_form(int form, int max_pairs) {
  g_forced_form.store(form >= 0 && form <= 3 ? form : 0);
  g_pair_cap.store(max_pairs > 0 ? max_pairs : 0);
}

void tc_form_stats(unsigned long long out[3]) {
  for (int i = 0; i < 3; ++i) out[i] = g_form_launches[i].load();
}

// 2-D row-major tensor [rows, cols] with leading dimension ld (elements), box [box_rows, box_cols].
static bool make_map(CUtensorMap* map, const void* base, int esz, long long rows, long long cols, long long ld,
                     int box_rows, int box_cols) {
  const MapKey key{base, rows, cols, ld, esz, box_rows, box_cols};
  const unsigned set = map_slot_of(key);
  for (int w = 0; w < kMapCacheWays; ++w) {
    const MapSlot& hit = g_map_cache[set][w];
    if (hit.used && hit.key == key) {
      *map = hit.map;
      ++g_map_hits;
      return true;
    }
  }
  int way = (g_map_victim[set] + 1) % kMapCacheWays;      // the way not written last ...
  for (int w = kMapCacheWays - 1; w >= 0; --w)
    if (!g_map_cache[set][w].used) way = w;                 // ... unless one is still unused
  g_map_victim[set] = (unsigned char)way;
  MapSlot& slot = g_map_cache[set][way];
  EncodeTiledFn fn = encode_fn();
  if (!fn) return false;
  cuuint64_t dims[2] = {(cuuint64_t)cols, (cuuint64_t)rows};
  cuuint64_t strides[1] = {(cuuint64_t)ld * esz};
  cuuint32_t box[2] = {(cuuint32_t)box_cols, (cuuint32_t)box_rows};
  cuuint32_t estr[2] = {1, 1};
  CUtensorMapDataType dt = esz == 2 ? CU_TENSOR_MAP_DATA_TYPE_BFLOAT16 : CU_TENSOR_MAP_DATA_TYPE_FLOAT32;
  if (fn(map, dt, 2, const_cast<void*>(base), dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
         CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
    return false;
  ++g_map_encodes;
  slot.map = *map;
  slot.key = key;
  slot.used = true;
  return true;
}

size_t matmul_tc_workspace_bytes(const MatmulPlan&) { return 0; }

static bool aligned16(const void* p) { return reinterpret_cast<uintptr_t>(p) % 16 == 0; }

// Launch of one compiled form of the kernel (called with the parameter block's lock held), or,
// with p == nullptr, only the number of CTA pairs of that form the device holds at once.
template <int AT, int BT, int MH>
static sbp_status launch_tc_form(const TcParams* p, cudaStream_t st, int* capacity) {
  constexpr int kSmem = MH == 2 ? kSmemBytesTall : kSmemBytes;
  // per device: the kernel's shared-memory opt-in and the number of CTA pairs that fit at once
  static int pairs_on_device[64] = {};
  int dev = 0;
  SBP_CUDA_TRY(cudaGetDevice(&dev));
  if (dev < 0 || dev >= 64) return fail(SBP_ERR_UNSUPPORTED, "device ordinal %d out of range", dev);
  if (pairs_on_device[dev] == 0) {
    SBP_CUDA_TRY(cudaFuncSetAttribute(matmul_tc_kernel<AT, BT, MH>, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmem));
    int sms = 0;
    SBP_CUDA_TRY(cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev));
    // how many CTA pairs the device can hold at once (pairs must sit in one GPC)
    cudaLaunchConfig_t probe = {};
    probe.gridDim = dim3((unsigned)(2 * (sms / 2)));
    probe.blockDim = dim3(kThreadsTc);
    probe.dynamicSmemBytes = kSmem;
    cudaLaunchAttribute attr;
    attr.id = cudaLaunchAttributeClusterDimension;
    attr.val.clusterDim.x = 2;
    attr.val.clusterDim.y = 1;
    attr.val.clusterDim.z = 1;
    probe.attrs = &attr;
    probe.numAttrs = 1;
    int clusters = 0;
    if (cudaOccupancyMaxActiveClusters(&clusters, matmul_tc_kernel<AT, BT, MH>, &probe) != cudaSuccess || clusters < 1) {
      cudaGetLastError();
      clusters = sms / 2;
    }
    pairs_on_device[dev] = clusters;
  }
  // a cap on the pairs (test and measurement switch): a small one makes small products run many
  // waves, and so take the mixed route
  const int cap = pair_cap();
  const int max_pairs = cap > 0 && cap < pairs_on_device[dev] ? cap : pairs_on_device[dev];
  if (capacity) *capacity = max_pairs;
  if (!p) return SBP_OK;
  const int pairs = p->total_tiles < max_pairs ? p->total_tiles : max_pairs;
  SBP_BOUNDS_UPLOAD(st);
  matmul_tc_kernel<AT, BT, MH><<<2 * pairs, kThreadsTc, kSmem, st>>>(*p);
  cudaError_t e = cudaGetLastError();
  if (e != cudaSuccess) return cuda_fail(e, "tensor-core matmul launch");
  count_launch();
  g_form_launches[MH == 2 ? 1 : (p->half_split ? 2 : 0)]++;
  return SBP_OK;
}

static sbp_status launch_tc(bool tall, bool a_trans, bool b_trans, const TcParams* p, cudaStream_t st, int* capacity) {
  switch ((tall ? 4 : 0) | (a_trans ? 2 : 0) | (b_trans ? 1 : 0)) {
    case 0: return launch_tc_form<0, 0, 1>(p, st, capacity);
    case 1: return launch_tc_form<0, 1, 1>(p, st, capacity);
    case 2: return launch_tc_form<1, 0, 1>(p, st, capacity);
    case 3: return launch_tc_form<1, 1, 1>(p, st, capacity);
    case 4: return launch_tc_form<0, 0, 2>(p, st, capacity);
    case 5: return launch_tc_form<0, 1, 2>(p, st, capacity);
    case 6: return launch_tc_form<1, 0, 2>(p, st, capacity);
    default: return launch_tc_form<1, 1, 2>(p, st, capacity);
  }
}

// Which form runs a product.  Times in microseconds per wave (one tile on every CTA pair), fitted
// to this kernel's measured times on B200 under its power cap (the clock settles lower the busier
// the tensor pipe is -- about 1.6 GHz in the square form, 1.4 GHz in the tall one -- which is why
// these are times and not clock counts):
//   square form  0.388 per 64-deep K-block (about 590 clocks); the epilogue is hidden unless it is store-bound;
//   tall form    0.70 per K-block (1024 clocks) for twice the rows, plus an exposed epilogue of about 2.6.
// A run may be mixed: whole waves of tall tiles, then the rest of the walk in the square form (two
// 256-row halves per walked tile) -- a last wave that only half fills the device costs a whole
// tall wave otherwise.
struct FormChoice {
  bool walk_tall;      // tiles are walked 512 rows at a time
  int tall_tiles;      // the first so many walked tiles run in the tall form
};

static FormChoice choose_form(long long tiles_sq, long long tiles_tall, long long kb, int cap_sq, int cap_tall, bool gelu, int n_rep,
                              bool out_f32, int forced) {
  const double wave_sq = 0.388 * kb + (gelu ? 1.3 : 0.0) + 1.2 * n_rep + (out_f32 ? 1.0 : 0.0);
  const double wave_tall = 0.70 * kb + 2.6 + (gelu ? 8.6 : 0.0) + 2.5 * n_rep + (out_f32 ? 3.0 : 0.0);
  const double kRelaunch = 5.0;
  auto waves = [](long long tiles, int cap) { return (double)((tiles + cap - 1) / cap); };
  const double cost_sq = waves(tiles_sq, cap_sq) * wave_sq;
  const double cost_tall = waves(tiles_tall, cap_tall) * wave_tall;
  const long long full = tiles_tall / cap_tall * cap_tall;       // tall tiles in whole waves
  const double cost_mixed = full == 0 || full == tiles_tall
                                ? 1e30
                                : (double)(full / cap_tall) * wave_tall + waves(2 * (tiles_tall - full), cap_sq) * wave_sq + kRelaunch;
  int pick;      // 0 square, 1 tall, 2 mixed
  if (forced) pick = forced - 1;
  else {
    pick = 0;
    double best = cost_sq * 0.98;                                // ties go to the square form
    if (cost_tall < best) { best = cost_tall; pick = 1; }
    if (cost_mixed < best) { best = cost_mixed; pick = 2; }
  }
  if (pick == 2 && (full == 0 || full == tiles_tall)) pick = full == 0 ? 0 : 1;
  if (pick == 0) return FormChoice{false, 0};
  return FormChoice{true, (int)(pick == 1 ? tiles_tall : full)};
}

// choose_form for callers outside this file (the C ABI's planning query): 0 square, 1 tall, 2 mixed.
int tc_route(long long tiles_sq, long long tiles_tall, long long kb, int pairs, bool gelu, int n_rep, bool out_f32, int forced,
             long long* tall_tiles) {
  const FormChoice f = choose_form(tiles_sq, tiles_tall, kb, pairs, pairs, gelu, n_rep, out_f32, forced);
  if (tall_tiles) *tall_tiles = f.walk_tall ? f.tall_tiles : 0;
  return !f.walk_tall ? 0 : (f.tall_tiles == tiles_tall ? 1 : 2);
}

sbp_status launch_matmul_tc(const MatmulPlan& plan, const XentFusion* xf, cudaStream_t st, bool* taken) {
  *taken = false;
  if (plan.in_dtype != SBP_BF16) return SBP_ERR_UNSUPPORTED;
  const int oesz = plan.out_dtype == SBP_F32 ? 4 : 2;
  const bool stores_y = !xf || xf->grad;      // the softmax-partials mode writes no product

  // the rules of the TMA path: 16-byte aligned bases, leading dimensions and column offsets
  for (int s = 0; s < plan.nseg; ++s) {
    const bool used = plan.chain || s < plan.ngroups;
    if (!used) continue;
    if (plan.kseg[s] > 0 && (!aligned16(plan.a[s]) || !aligned16(plan.b[s]))) return SBP_ERR_UNSUPPORTED;
    if (plan.lda[s] % 8 != 0 || plan.ldb[s] % 8 != 0) return SBP_ERR_UNSUPPORTED;
    if (plan.lda[s] == 0 || plan.ldb[s] == 0) return SBP_ERR_UNSUPPORTED;
  }
  bool y_direct = false;
  long long ktotal_chain = 0;
  for (int s = 0; s < plan.nseg; ++s) ktotal_chain += plan.kseg[s];
  for (int g = 0; g < plan.ngroups; ++g) {
    if (plan.m[g] == 0 || plan.n[g] == 0) continue;
    if (stores_y && (!aligned16(plan.y[g]) || (plan.ldy[g] * oesz) % 16 != 0)) y_direct = true;
    if (!plan.b_trans && plan.col_off[g] % 8 != 0) return SBP_ERR_UNSUPPORTED;   // the x coordinate of a TMA load
    if (plan.a_trans && plan.row_off[g] % 8 != 0) return SBP_ERR_UNSUPPORTED;
    const long long kg = plan.chain ? ktotal_chain : plan.kseg[g];
    if (kg == 0) return SBP_ERR_UNSUPPORTED;   // an all-zero result: left to the FMA kernel
    if (plan.m[g] > 0x7fffffffLL || plan.n[g] > 0x7fffffffLL) return SBP_ERR_UNSUPPORTED;
  }
  for (int r = 0; r < plan.n_rep; ++r)
    if (!aligned16(plan.y_rep[r])) y_direct = true;
  if (!encode_fn()) return SBP_ERR_UNSUPPORTED;

  static TcParams p;          // large; filled under a lock and copied by value at launch
  static std::mutex mu;
  std::lock_guard<std::mutex> lock(mu);
  p.ngroups = plan.ngroups;
  p.nseg = plan.nseg;
  p.chain = plan.chain;
  p.gelu = plan.gelu;
  p.n_rep = plan.n_rep;
  p.out_f32 = plan.out_dtype == SBP_F32;
  p.xent = xf ? (xf->grad ? 2 : 1) : 0;
  if (xf) p.xf = *xf;
  p.y_direct = y_direct ? 1 : 0;

  for (int s = 0; s < plan.nseg; ++s) {
    p.kblocks[s] = (int)((plan.kseg[s] + BK - 1) / BK);
    const bool used = plan.chain || s < plan.ngroups;
    if (!used || plan.kseg[s] == 0) continue;
    long long rows_a = 0, cols_b = 0;
    if (plan.chain) {
      for (int g = 0; g < plan.ngroups; ++g) {
        rows_a = std::max(rows_a, plan.row_off[g] + plan.m[g]);
        cols_b = std::max(cols_b, plan.col_off[g] + plan.n[g]);
      }
    } else {
      rows_a = plan.m[s];
      cols_b = plan.n[s];
    }
    if (rows_a == 0 || cols_b == 0) { p.kblocks[s] = plan.chain ? p.kblocks[s] : 0; continue; }
    // as stored: A [rows, K] (transposed [K, rows]), B [K, cols] (transposed [cols, K])
    const bool ok_a = plan.a_trans ? make_map(&p.map_a[s], plan.a[s], 2, plan.kseg[s], rows_a, plan.lda[s], BK, 64)
                                   : make_map(&p.map_a[s], plan.a[s], 2, rows_a, plan.kseg[s], plan.lda[s], BMH, BK);
    if (!ok_a) return fail(SBP_ERR_CUDA, "cuTensorMapEncodeTiled failed for operand x of shard %d", s);
    const bool ok_b = plan.b_trans ? make_map(&p.map_b[s], plan.b[s], 2, cols_b, plan.kseg[s], plan.ldb[s], BNH, BK)
                                   : make_map(&p.map_b[s], plan.b[s], 2, plan.kseg[s], cols_b, plan.ldb[s], BK, 64);
    if (!ok_b) return fail(SBP_ERR_CUDA, "cuTensorMapEncodeTiled failed for operand w of shard %d", s);
  }
  // Which form (see choose_form).  The softmax epilogues are written for the square form, and so is
  // the element-wise store of a result the copy engine cannot address.
  long long kb_tile = 0, tiles_sq = 0, tiles_tall = 0;
  for (int s = 0; s < plan.nseg; ++s)
    if (plan.chain || s < plan.ngroups) kb_tile = plan.chain ? kb_tile + p.kblocks[s] : std::max<long long>(kb_tile, p.kblocks[s]);
  for (int g = 0; g < plan.ngroups; ++g) {
    if (plan.m[g] <= 0 || plan.n[g] <= 0) continue;
    const long long tn = (plan.n[g] + BN - 1) / BN;
    tiles_sq += (plan.m[g] + BM - 1) / BM * tn;
    tiles_tall += (plan.m[g] + 2 * BM - 1) / (2 * BM) * tn;
  }
  FormChoice form{false, 0};
  if (!xf && !y_direct && tiles_tall > 0 && tiles_sq <= 0x1fffffffLL) {
    int cap_sq = 0, cap_tall = 0;
    sbp_status qs = launch_tc(false, plan.a_trans, plan.b_trans, nullptr, st, &cap_sq);
    if (qs == SBP_OK) qs = launch_tc(true, plan.a_trans, plan.b_trans, nullptr, st, &cap_tall);
    if (qs != SBP_OK) return qs;
    form = choose_form(tiles_sq, tiles_tall, kb_tile, cap_sq, cap_tall, plan.gelu != 0, plan.n_rep, plan.out_dtype == SBP_F32, forced_form());
  }
  const int tile_m = form.walk_tall ? 2 * BM : BM;
  p.walk_m = tile_m;
  p.tile_first = 0;
  p.half_split = 0;

  int tiles = 0;
  const int box_cols = p.out_f32 ? 32 : 64;
  for (int g = 0; g < plan.ngroups; ++g) {
    p.m[g] = plan.m[g];
    p.n[g] = plan.n[g];
    p.row_off[g] = plan.row_off[g];
    p.col_off[g] = plan.col_off[g];
    p.tile_begin[g] = tiles;
    const long long tm = (plan.m[g] + tile_m - 1) / tile_m, tn = (plan.n[g] + BN - 1) / BN;
    p.tiles_m[g] = (int)std::max(1LL, tm);
    p.tiles_n[g] = (int)std::max(1LL, tn);
    if (plan.m[g] > 0 && plan.n[g] > 0) {
      if (tm * tn + tiles > 0x3fffffffLL) return SBP_ERR_UNSUPPORTED;
      tiles += (int)(tm * tn);
      p.y_ptr[g] = plan.y[g];
      p.ldy[g] = plan.ldy[g];
      if (stores_y && !y_direct && !make_map(&p.map_y[g], plan.y[g], oesz, plan.m[g], plan.n[g], plan.ldy[g], 32, box_cols))
        return fail(SBP_ERR_CUDA, "cuTensorMapEncodeTiled failed for the result of group %d", g);
    }
  }
  // row-block (or column-block) groups of one fused result: one grid for the walk
  bool rows_stack = plan.chain && plan.ngroups > 1, cols_stack = rows_stack;
  for (int g = 0; g < plan.ngroups; ++g) {
    if (plan.n[g] != plan.n[0] || plan.col_off[g] != 0 || plan.n[g] == 0) rows_stack = false;
    if (plan.m[g] != plan.m[0] || plan.row_off[g] != 0 || plan.m[g] == 0) cols_stack = false;
  }
  p.stacked = rows_stack ? 1 : (cols_stack ? 2 : 0);
  p.mt_begin[0] = 0;
  for (int g = 0; g < plan.ngroups; ++g) {
    const bool live = plan.m[g] > 0 && plan.n[g] > 0;
    p.mt_begin[g + 1] = p.mt_begin[g] + (live ? (p.stacked == 2 ? p.tiles_n[g] : p.tiles_m[g]) : 0);
  }
  for (int g = 0; g < plan.ngroups; ++g) {
    const long long tn_walk = p.stacked == 2 ? p.mt_begin[plan.ngroups] : (p.stacked ? p.tiles_n[0] : p.tiles_n[g]);
    p.panel_magic[g] = (unsigned)((1ull << 32) / (unsigned long long)(kPanelM * std::max(1LL, tn_walk)));
  }
  p.tile_begin[plan.ngroups] = tiles;
  for (int g = plan.ngroups + 1; g <= SBP_MAX_K; ++g) p.tile_begin[g] = tiles;
  p.total_tiles = tiles;
  for (int r = 0; r < plan.n_rep; ++r) {
    p.rep_ptr[r] = plan.y_rep[r];
    if (!y_direct && !make_map(&p.map_rep[r], plan.y_rep[r], oesz, plan.m[0], plan.n[0], plan.ldy[0], 32, box_cols))
      return fail(SBP_ERR_CUDA, "cuTensorMapEncodeTiled failed for a result replica");
  }
  *taken = true;
  if (tiles == 0) return SBP_OK;

  if (!form.walk_tall) return launch_tc(false, plan.a_trans, plan.b_trans, &p, st, nullptr);
  // tall form over the first walked tiles, then (mixed run) the square form over the halves of the rest
  const int tall_tiles = std::min(form.tall_tiles, tiles);
  p.total_tiles = tall_tiles;
  sbp_status rs = launch_tc(true, plan.a_trans, plan.b_trans, &p, st, nullptr);
  if (rs != SBP_OK || tall_tiles == tiles) return rs;
  p.tile_first = tall_tiles;
  p.half_split = 1;
  p.total_tiles = 2 * (tiles - tall_tiles);
  return launch_tc(false, plan.a_trans, plan.b_trans, &p, st, nullptr);
}

sbp_status read_and_clear_tc_timeout(bool* timed_out) {
  int flag = 0, zero = 0;
  SBP_CUDA_TRY(cudaMemcpyFromSymbol(&flag, g_tc_timeout_flag, sizeof(int)));
  if (flag) SBP_CUDA_TRY(cudaMemcpyToSymbol(g_tc_timeout_flag, &zero, sizeof(int)));
  *timed_out = flag != 0;
  return SBP_OK;
}

}  // namespace sbp
