/*
 * sbp.h -- C ABI of the B200 (sm_100a) SBP library.
 *
 * SBP is the paper's abstraction (Section 3.1) for how a *global* (logical) tensor maps
 * onto the *local* tensors of the k devices of a placement:
 *     S(i)   split along axis i in a balanced manner,
 *     B      broadcast: every local tensor is an exact copy of the global tensor,
 *     P(op)  partial-value: every local tensor has the global shape and the global tensor
 *            is the element-wise reduction (sum or max) over the local tensors.
 * In this library the k "devices" of a placement are k logical shards that all live in
 * ONE GPU's memory; there is no inter-GPU traffic.
 *
 * General conventions (hold for every entry point unless it says otherwise)
 *   - All pointers inside an sbp_tensor are DEVICE pointers owned by the caller.  Every
 *     local tensor is dense row-major with the local shape given by sbp_local_shape().
 *   - The library allocates no device memory and frees none.  Scratch memory, where an
 *     operation needs it, is passed in by the caller ("ws", "ws_bytes"); its required
 *     size comes from the matching *_workspace_bytes() query.
 *   - Work is enqueued on `cuda_stream` (a cudaStream_t passed as void*; NULL = the
 *     legacy default stream) and the call returns without waiting for it.
 *   - All argument checking happens on the host before anything is launched; when a
 *     call returns anything other than SBP_OK nothing has been written.
 *   - Source and destination buffers must not overlap.
 *   - Balanced split of an axis of length n over k shards: shard r holds
 *     ceil(n/k) elements if r < n mod k, else floor(n/k), contiguous, in rank order.
 *   - 16-byte aligned pointers and row segments take the 128-bit vector path; anything
 *     else takes an element-wise path with identical results.
 *   - sbp_last_error() returns a thread-local, human readable detail for the last
 *     non-OK status returned on the calling thread.
 */
#ifndef SBP_H_
#define SBP_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
  SBP_OK = 0,
  SBP_ERR_INVALID_ARG = 1, /* null pointer, bad rank, k out of range, ...                */
  SBP_ERR_SHAPE = 2,       /* logical shapes of the operands do not fit together         */
  SBP_ERR_DTYPE = 3,       /* dtype not supported by this operation                      */
  SBP_ERR_SIGNATURE = 4,   /* SBP signatures are not a valid combination                 */
  SBP_ERR_UNSUPPORTED = 5, /* valid request that the library does not implement          */
  SBP_ERR_ALIGNMENT = 6,   /* a pointer is not aligned to its element size               */
  SBP_ERR_WORKSPACE = 7,   /* workspace missing or too small                             */
  SBP_ERR_CUDA = 8,        /* a CUDA runtime / driver call failed (no device, launch...) */
  SBP_ERR_TIMEOUT = 9,     /* a bounded device-side wait expired                         */
  SBP_ERR_BOUNDS = 10      /* debug-bounds build only: a kernel computed an address outside
                              the buffers of its call (the access was skipped)           */
} sbp_status;

typedef enum { SBP_F32 = 0, SBP_BF16 = 1, SBP_I64 = 2 } sbp_dtype;

typedef enum {
  SBP_SPLIT = 0,
  SBP_BROADCAST = 1,
  SBP_PARTIAL_SUM = 2,
  SBP_PARTIAL_MAX = 3
} sbp_kind;

/* One SBP signature.  `axis` is read only when kind == SBP_SPLIT. */
typedef struct {
  int32_t kind; /* sbp_kind */
  int32_t axis;
} sbp_sig;

#define SBP_MAX_DIMS 4
#define SBP_MAX_K 16
#define SBP_MAX_PDIMS 2

/*
 * A global tensor together with its placement, signature and local tensors
 * (Section 3: "a global tensor is mapped to multiple local tensors"; Section 3.4: a
 * tensor carries a placement and an sbp attribute).  Plain data; the caller owns it.
 *
 *   shape[0..ndim)   LOGICAL (global) shape, 1 <= ndim <= SBP_MAX_DIMS.
 *   pdims, pshape    placement hierarchy; k = product of pshape[0..pdims).  pdims == 2 is the
 *                    paper's multi-dimensional SBP (Section 3.3): sbp[0] is applied across the
 *                    pshape[0] groups, sbp[1] inside a group, and device (i, j) is local[i *
 *                    pshape[1] + j].  sbp_local_shape, sbp_boxing and sbp_matmul accept
 *                    pdims == 2; every other entry point answers SBP_ERR_UNSUPPORTED.
 *   sbp[p]           one signature per placement axis.
 *   local[r]         device pointer of shard r's local tensor, r in [0, k).  For a B
 *                    tensor the k replicas may all be the same pointer; a kernel then
 *                    writes that buffer once.
 *   local_ld[r]      leading dimension of shard r's local tensor, in elements: the distance between
 *                    consecutive rows when the local tensor is viewed as [rows, cols] with cols its
 *                    last local extent and rows the product of the others.  0 means dense
 *                    (local_ld = cols); otherwise local_ld[r] >= cols.  A local tensor with a
 *                    leading dimension is a window into a larger buffer -- a column block of a
 *                    replica (Table 2: B -> S costs nothing, see sbp_view_b_to_s) or a sub-block of a
 *                    matrix.  Honoured by sbp_matmul (all three tensors), by sbp_boxing on 2-D tensors
 *                    of one placement (S / B / P on either side, except the P(sum)-destination and
 *                    cast rows) and by sbp_softmax_xent / sbp_softmax_xent_backward (logits, grad);
 *                    every other entry point answers SBP_ERR_UNSUPPORTED to a non-dense tensor.
 */
typedef struct {
  int32_t ndim;
  int32_t dtype; /* sbp_dtype */
  int64_t shape[SBP_MAX_DIMS];
  int32_t pdims;
  int32_t pshape[SBP_MAX_PDIMS];
  sbp_sig sbp[SBP_MAX_PDIMS];
  void* local[SBP_MAX_K];
  int64_t local_ld[SBP_MAX_K];
} sbp_tensor;

/* ---------------------------------------------------------------- descriptors, rules */

const char* sbp_status_string(sbp_status s);
const char* sbp_last_error(void);

/* Number of kernels this library has launched from the calling process so far (all
 * threads).  Lets a harness count launches inside a timed region. */
uint64_t sbp_launch_count(void);

/* Local shape of shard r under t's signature (Section 3.1).  Host only, no CUDA. */
sbp_status sbp_local_shape(const sbp_tensor* t, int32_t r, int64_t out_shape[SBP_MAX_DIMS]);

/* B -> S(axis) without moving anything (Table 2: "B -> S" costs 0; Section 3.2: such a boxing "may
 * not lead to data movement").  Fills *view with a descriptor of the same global tensor under
 * S(axis) whose local tensors are windows into b's replicas: view->local[r] points at shard r's
 * piece inside b->local[r] and view->local_ld[r] carries the replica's row length when the piece
 * is not contiguous (a split of the last axis).  b must be a B tensor on a one-axis placement;
 * axis 0 or the last axis (any other axis of an N-D tensor would need two strides:
 * SBP_ERR_UNSUPPORTED).  Nothing is launched or copied; the view aliases b's memory, so writing
 * through one is visible through the other.  Host only, no CUDA. */
sbp_status sbp_view_b_to_s(const sbp_tensor* b, int32_t axis, sbp_tensor* view);

/* Table 1 ("Valid SBP signatures for MatMul"): signature of Y = XW from those of X and
 * W, or SBP_ERR_SIGNATURE when the pair is not one of the table's six rows. */
sbp_status sbp_matmul_infer(sbp_sig x, sbp_sig w, sbp_sig* y);

/* Table 2 ("Data size transferred between successive SBP signatures"): bytes that cross between
 * devices when a tensor of t_bytes goes from signature src on p1 devices to signature dst on p2
 * devices -- the "same" column (disjoint == 0, p1 == p2) or the "disjoint" column.  The paper
 * offers these counts for choosing the signatures with the lowest communication cost
 * (Section 3.2); on the one-GPU placements of this library nothing crosses a link, so this is
 * a planning aid only.  Host only, no CUDA. */
sbp_status sbp_transfer_cost(sbp_sig src, sbp_sig dst, int32_t p1, int32_t p2, int32_t disjoint,
                             uint64_t t_bytes, uint64_t* cost_bytes);

/* ---------------------------------------------------------------- boxing (Section 3.2)
 *
 * A boxing op re-arranges or transforms the local tensors of a global tensor so that
 * the same global tensor is seen under another signature (Section 3.2; Table 2, column
 * "same" placement).  src and dst must agree in logical shape and dtype (one exception below);
 * with the same k on both sides the rows below apply, with different k the "disjoint" rows
 * further down.
 *
 *   src            dst        the collective it stands for (Table 2)
 *   P(sum)         B          all-reduce       out_j[e] = round(sum_r in_r[e])
 *   P(sum)         S(i)       reduce-scatter   out_r    = slice_r,i(sum_r' in_r')
 *   P(max)         B / S(i)   same with max; exact
 *   S(i)           B          all-gather       out_j    = concat_i(in_0 .. in_{k-1})
 *   S(i)           S(j)       all2all (i!=j);  plain copy when i == j
 *   B              S(i)       local slice of the shard's own replica
 *   B              B          copy of the shard's own replica
 *   P(op)          P(op)      copy
 *   S(i)           P(sum)     local (Table 2: cost 0): shard r = zeros with its own slice in place
 *   B              P(sum)     local (Table 2: cost 0): shard 0 = the tensor, every other shard zeros
 *   S(i) F32       B BF16     the cast op of Section 6.4 (sharded fp32 state -> half-precision
 *                             replicas) folded into the all-gather: read once as fp32, rounded to
 *                             bf16 (nearest even), written to every replica.  The only dtype change
 *                             sbp_boxing accepts.
 * Anything else (a P(max) destination from S or B, P(sum)<->P(max)) returns SBP_ERR_UNSUPPORTED.
 *
 * Two-axis placements: one call may change the signature of ONE placement axis (the other stays
 * as it is); the transform then runs as independent one-axis boxing ops, inside each group when
 * axis 1 changes, across the groups when axis 0 changes.  Changing axis 0 along the tensor axis
 * that axis 1 splits, or summing over one axis what is a max over the other, is refused with
 * SBP_ERR_UNSUPPORTED, as is changing both axes at once (make two calls).
 *
 * Different placements (Table 2, column "disjoint"): src on p = k(src) shards, dst on q = k(dst)
 * other shards, p != q allowed, one-axis placements on both sides, same dtype.  The table fixes
 * only the bytes that travel; the transforms are the plainest ones that move exactly those bytes:
 *   S / B   -> S(i) / B   the global tensor, mapped onto the q shards (balanced q-way split)
 *   P(op)   -> S(i) / B   all p partials reduced in rank order (arithmetic below), then mapped
 *   S(i)    -> P(sum)     partial j = zeros with piece j of the q-way split of axis i in place
 *   B       -> P(sum)     partial 0 = the tensor, the others zeros
 *   P(op)   -> P(op)      partial r travels to shard r mod q, which reduces what it receives in
 *                         ascending r; a shard that receives nothing is zero (so P(max) with
 *                         q > p is refused with SBP_ERR_UNSUPPORTED)
 * With q == p these give the same local tensors as the same-placement rows.
 *
 * P(sum) arithmetic: an fp32 accumulator starts as shard 0, shards 1..k-1 are added in
 * rank order with plain IEEE adds, and the result is rounded once (nearest even) to the
 * storage dtype.  P(max): acc = shard 0; shard r replaces acc only when strictly greater.
 * Reductions accept SBP_F32 and SBP_BF16; pure data movement accepts every dtype.
 */
sbp_status sbp_boxing(const sbp_tensor* src, sbp_tensor* dst, void* cuda_stream);

/* The part of a boxing op that ONE device of the destination placement executes: produces
 * dst->local[dst_shard] and nothing else (Section 3.2: a boxing op stands for a collective; on
 * real devices each member pulls what it needs from the others).  Same transforms, arithmetic
 * and errors as sbp_boxing on one-axis placements (same or different shard counts); the k calls
 * with dst_shard = 0..k-1 together write exactly what one sbp_boxing call writes.
 *
 *   src->local[*]          read: every source local tensor the transform needs for this shard must
 *                          be readable from the current device -- device memory of this GPU, or a
 *                          peer GPU's memory mapped into this process (plain loads cross NVLink;
 *                          nothing in the library assumes the sources are local)
 *   dst->local[dst_shard]  written, device memory of the current GPU; the other dst->local entries
 *                          are not looked at and may be null
 * Which source shards are read: S -> S / S -> B all that overlap the shard; P -> S / B all k
 * partials; B -> S / B -> B / P -> P / S(i) -> S(i) only source shard dst_shard (dst_shard mod k(src)
 * between different placements); S / B -> P(sum) the shard's own piece.  The caller orders the calls
 * of different devices (sources complete before anyone reads them): a stream or host barrier,
 * never a wait inside a kernel.  Two-axis placements: SBP_ERR_UNSUPPORTED. */
sbp_status sbp_boxing_shard(const sbp_tensor* src, sbp_tensor* dst, int32_t dst_shard, void* cuda_stream);

/* Same transform, but every local[] pointer of src_host and dst_host is a HOST pointer
 * (pinned memory recommended).  The source local tensors are copied to the device
 * workspace, transformed there and the destination local tensors copied back, all
 * enqueued on cuda_stream.  dev_ws must hold sbp_boxing_host_workspace_bytes() bytes.
 * Only what the transform reads crosses to the device: for B -> S(i) on equal placements that is,
 * of source replica r, the block that becomes shard r (Table 2: B -> S moves no data between
 * devices); every other transform reads all of every source local tensor.  Destination replicas
 * that share one host pointer are copied back once.  sbp_boxing_host_copy_bytes reports the bytes a
 * call copies in each direction (host pointers are only compared, never dereferenced). */
size_t sbp_boxing_host_workspace_bytes(const sbp_tensor* src_host, const sbp_tensor* dst_host);
sbp_status sbp_boxing_host_copy_bytes(const sbp_tensor* src_host, const sbp_tensor* dst_host, uint64_t* h2d_bytes,
                                      uint64_t* d2h_bytes);
/* One source, n destinations (1 <= n <= 64; dst_hosts is an array of n descriptors): the source is
 * copied to the device once and boxed into every destination there, each result copied back as
 * soon as its transform is enqueued -- what a caller does who needs one host tensor under several
 * signatures (Section 3.2: one boxing op per consumer whose signature differs from the producer's;
 * e.g. the P(sum) result of a product as B for one consumer and as S(0) for another).  Same
 * rules as sbp_boxing_host for every (src, dst[i]) pair; all n pairs are validated before the
 * first copy is enqueued; only the diagonal blocks of a B source are sent when every destination is
 * an S of the same axis.  The workspace holds the source and all n results at once.
 * sbp_boxing_host is this call with n = 1. */
size_t sbp_boxing_host_multi_workspace_bytes(const sbp_tensor* src_host, const sbp_tensor* dst_hosts, int32_t n);
sbp_status sbp_boxing_host_multi_copy_bytes(const sbp_tensor* src_host, const sbp_tensor* dst_hosts, int32_t n,
                                            uint64_t* h2d_bytes, uint64_t* d2h_bytes);
sbp_status sbp_boxing_host_multi(const sbp_tensor* src_host, sbp_tensor* dst_hosts, int32_t n, void* dev_ws,
                                 size_t dev_ws_bytes, void* cuda_stream);
sbp_status sbp_boxing_host(const sbp_tensor* src_host, sbp_tensor* dst_host, void* dev_ws,
                           size_t dev_ws_bytes, void* cuda_stream);

/* 1 when this library was compiled as the debug-bounds build, else 0.  In that build every
 * global-memory address a kernel computes is compared, before it is used, with the buffers of the
 * call (every local tensor by its host-computed extent, and the workspace); an address outside
 * them is recorded and the access skipped -- nothing traps -- and the next
 * sbp_check_device_errors() returns SBP_ERR_BOUNDS.  It is an order of magnitude slower than the
 * normal build and meant for small and ragged test shapes; it stands in for a memory checker where
 * none can be run.  Build it with `python -m paper_2110_15032_b200.build --debug-bounds`
 * (libsbp_b200_dbg.so) and select it with SBP_B200_LIBRARY=<path> before the package loads. */
int32_t sbp_debug_bounds_enabled(void);

/* Self-test of that report path, safe to run anywhere (debug-bounds build only; the normal build
 * answers SBP_ERR_UNSUPPORTED): registers the device buffer [buf, buf + bytes) and enqueues a
 * one-thread kernel that asks the checker about buf[0] (allowed: the byte is set to 1) and about
 * the byte just past the end (refused: recorded, and NOT accessed).  After the stream has drained,
 * sbp_check_device_errors() returns SBP_ERR_BOUNDS once. */
sbp_status sbp_selftest_debug_bounds(void* buf, size_t bytes, void* cuda_stream);

/* Kernels of this library bound every device-side wait.  When one expires the kernel sets a
 * device flag and returns; this call (which synchronises with the device) reads and clears
 * the flag: SBP_ERR_TIMEOUT if a wait expired since the last call, else SBP_OK (debug-bounds
 * build: SBP_ERR_BOUNDS first, if a kernel's address check failed). */
sbp_status sbp_check_device_errors(void);

/* Self-test of that path, safe to run anywhere: enqueues a one-thread kernel that waits on a
 * barrier nothing signals, gives up after limit_ms (1..1000) and raises the flag.  After the
 * stream has drained, sbp_check_device_errors() returns SBP_ERR_TIMEOUT once, and the device
 * stays fully usable. */
sbp_status sbp_selftest_wait_timeout(uint32_t limit_ms, void* cuda_stream);

/* Selects the copy engine of the pure data-movement transforms: 0 = choose (default; currently
 * always the load/store kernel, the faster one on B200), 1 = 128-bit load/store kernel,
 * 2 = bulk asynchronous copies staged through shared memory (needs 16-byte aligned segments
 * of at least 512 bytes, else falls back to 1).  Process-wide. */
void sbp_boxing_set_copy_engine(int32_t engine);

/* ---------------------------------------------------------------- MatMul (Table 1)
 *
 * Y = XW on the local tensors, under the signatures the descriptors carry:
 *   (S(0),B)->S(0)   (B,S(1))->S(1)   (S(1),S(0))->P(sum)
 *   (P(sum),B)->P(sum)   (B,P(sum))->P(sum)   (B,B)->B
 * y->sbp must be the signature Table 1 deduces, or -- for rows whose deduced signature is
 * P(sum) -- B or S(i): the partial products are then reduced in rank order inside the
 * kernel's accumulator and Y is written directly in that signature (the boxing op of
 * Section 3.2 fused into the producer).  Any other request is SBP_ERR_SIGNATURE; call
 * sbp_boxing afterwards instead.
 * Two-axis placements (Table 3, e.g. (S(0),B) x (B,S(1)) -> (S(0),S(1)) and (S(0),S(1)) x
 * (B,S(0)) -> (S(0),P(sum))): Table 1 is applied to each placement axis on its own, y must carry
 * exactly the deduced pair, and every device multiplies its local tensors (no fused boxing).
 *
 * x: [M,K], w: [K,N], y: [M,N] logical, all 2-D, same dtype for x and w:
 *   SBP_F32  : fp32 FMA accumulation, y SBP_F32.
 *   SBP_BF16 : bf16 operands, fp32 accumulation on the tensor cores, y SBP_BF16 or SBP_F32.
 * flags: SBP_EPILOGUE_GELU applies GeLU(v) = v/2 (1 + erf(v/sqrt 2)) to the fp32
 * accumulator before the store; only where Y is S or B (GeLU is not linear, so it cannot
 * be applied to partial values).  erf is evaluated to about 1.5e-7 absolute on the tensor-core
 * path (a rational approximation) and by the fp32 library erf on the FMA path, so the same call
 * may differ in the last bits of an fp32 result depending on which kernel its shapes select;
 * both are far inside the stated tolerance.
 *        SBP_TRANS_X / SBP_TRANS_W: the descriptor x (w) holds the transpose of the operand,
 * i.e. x is stored as [K,M] (w as [N,K]), logically and in every local tensor, and its
 * signature refers to the stored axes.  The operand that enters Table 1 is the transpose, so a
 * stored S(0) counts as S(1) and a stored S(1) as S(0); B and P(sum) are unchanged.  This is
 * what the backward products of a layer need without a transposed copy: with Y = X W,
 * dW = X^T dY (x = X with SBP_TRANS_X) and dX = dY W^T (w = W with SBP_TRANS_W).  Data
 * parallelism (Section 3.1: X S(0), W B) then gives dW = (S(1), S(0)) -> P(sum), and asking
 * for y as B folds the gradient all-reduce into the product.  One-axis placements only.
 * ws: scratch for the tensor-core path (see below; may be NULL when the query returns 0).
 * A result whose base or leading dimension the copy engine cannot address is written by the
 * kernel's own stores instead; that needs no workspace.
 */
#define SBP_EPILOGUE_GELU 1u
#define SBP_TRANS_X 2u
#define SBP_TRANS_W 4u
/* Workspace: bf16 operands that the tensor-core path cannot address in place -- a local tensor whose
 * base is not 16-byte aligned or whose leading dimension is not a multiple of 8 elements (a shard
 * width of 333), or a fused S(i) result whose shards start on an odd column -- are first copied
 * into `ws` in an aligned layout (one read and one write of the operand) so that the product stays
 * on the tensor cores.  sbp_matmul_workspace_bytes_for returns the bytes that needs for the given
 * descriptors and flags (0 when nothing has to be copied; judged from the shapes, so pass 256-byte
 * aligned local tensors or add the operands' sizes yourself); ws must be 256-byte aligned.  Without
 * a large enough workspace such a product runs on the FMA kernel: same results within the stated
 * tolerance, far slower.  sbp_matmul_workspace_bytes is the same query for flags = 0. */
size_t sbp_matmul_workspace_bytes_for(const sbp_tensor* x, const sbp_tensor* w, const sbp_tensor* y, uint32_t flags);
size_t sbp_matmul_workspace_bytes(const sbp_tensor* x, const sbp_tensor* w, const sbp_tensor* y);

/* The tensor-core path describes every operand and result tile layout to the copy engine with a
 * descriptor that the driver encodes on the host.  The library keeps the descriptors it has
 * encoded, keyed by address and layout, and re-uses them when a product is called again on the
 * same buffers.  This reports how many were re-used and how many encoded since the library was
 * loaded (process-wide), so that a harness can check that a steady-state call encodes nothing. */
void sbp_tensor_map_stats(uint64_t* reused, uint64_t* encoded);
/* (No counterpart in the paper either.)  The tensor-core kernel has two compiled forms: CTA pairs that own 256 x 256 tiles of the result
 * with a spare accumulator, so that a tile's epilogue runs under the next tile's MMAs ("square"),
 * and pairs that own 512 x 256 tiles with both accumulators in use ("tall": less operand traffic per
 * MMA, the epilogue exposed).  The library picks per product, from the tile count, the length of
 * the contraction and the epilogue, one of: square; tall; or a mixed run -- whole waves of tall
 * tiles, then the rest of the result in the square form as a second launch.  The results do not
 * depend on the choice (same accumulation order per element).  This reports the launches since the
 * library was loaded (process-wide): [0] square, [1] tall, [2] the square launch that ends a mixed run.
 * sbp_matmul_set_form overrides the choice for tests and measurements (process-wide, not a tuning
 * knob): form 0 = the library chooses, 1 = square, 2 = tall, 3 = mixed (where a product cannot run
 * the forced form -- softmax epilogues, results written element-wise, fewer tiles than one wave
 * for "mixed" -- it runs the nearest one that it can); max_pairs > 0 caps the CTA pairs of a
 * launch (0 = all the device holds), which makes small products run many waves.  Until it is
 * called, the environment variables SBP_TC_FORM = square | tall | mixed and SBP_TC_PAIRS, read
 * once, give the same two values. */
#define SBP_TC_FORM_AUTO 0
#define SBP_TC_FORM_SQUARE 1
#define SBP_TC_FORM_TALL 2
#define SBP_TC_FORM_MIXED 3
void sbp_matmul_set_form(int32_t form, int32_t max_pairs);
/* (The paper has no counterpart: this is about how THIS library runs a Table 1 product.)
 * The route the library's cost model picks for ONE bf16 output group of m x n with a contraction of
 * k on a device that holds `pairs` CTA pairs at once (74 on a B200), written to `replicas` >= 1
 * destinations: returns 0 square, 1 tall, 2 mixed (then *tall_tiles = the 512 x 256 tiles that run
 * in the tall form; 0 for square), -1 for arguments out of range.  Host arithmetic only: no
 * device is touched, overrides set with sbp_matmul_set_form are not applied, and products that
 * cannot leave the square form (softmax epilogues, element-wise stores) are not modelled. */
int32_t sbp_matmul_route(int64_t m, int64_t n, int64_t k, int32_t pairs, uint32_t flags, int32_t replicas, int32_t out_f32,
                         int64_t* tall_tiles);
void sbp_matmul_form_stats(uint64_t launches[3]);
sbp_status sbp_matmul(const sbp_tensor* x, const sbp_tensor* w, sbp_tensor* y, uint32_t flags,
                      void* ws, size_t ws_bytes, void* cuda_stream);

/* ---------------------------------------------------------------- split softmax cross entropy
 *
 * Section 6.3 (classifier weight S(1) => logits S(1)): the softmax has two reductions,
 * max and sum, each done locally per shard first and then across shards
 * (P(max)->B, P(sum)->B); the loss is the sparse cross entropy of the label's column.
 *
 *   logits  [rows, classes]  S(1), SBP_BF16 or SBP_F32
 *   labels  [rows]           B, SBP_I64, each in [0, classes)
 *   loss    [rows]           B, SBP_F32:  log(sum_j exp(z_ij - m_i)) + m_i - z_i,label_i
 *   row_max [rows]           B, SBP_F32, optional (NULL): m_i = max_j z_ij
 *   row_sum [rows]           B, SBP_F32, optional (NULL): sum_j exp(z_ij - m_i)
 * ws holds the per-shard partial max / exp-sum / label-logit vectors.
 * A label outside [0, classes) contributes a label logit of 0.
 */
size_t sbp_softmax_xent_workspace_bytes(const sbp_tensor* logits);
sbp_status sbp_softmax_xent(const sbp_tensor* logits, const sbp_tensor* labels, sbp_tensor* loss,
                            sbp_tensor* row_max, sbp_tensor* row_sum, void* ws, size_t ws_bytes,
                            void* cuda_stream);

/* Backward of that loss with respect to the logits, for per-row losses with unit upstream
 * gradient: grad[i, j] = exp(z_ij - m_i) / S_i - [j == label_i], i.e. softmax minus one-hot.
 * It is element-wise once the forward pass's row_max (m) and row_sum (S) are known, so the
 * gradient keeps the logits' signature S(1) and needs no reduction (Section 6.3's plan read
 * backwards).  grad_logits has the logits' shape, dtype and signature. */
sbp_status sbp_softmax_xent_backward(const sbp_tensor* logits, const sbp_tensor* labels,
                                     const sbp_tensor* row_max, const sbp_tensor* row_sum,
                                     sbp_tensor* grad_logits, void* cuda_stream);

/* The classifier of Section 6.3 in one call: logits = features x weight with the weight S(1)
 * (hence logits S(1)), then the split softmax cross entropy above -- without ever storing the
 * logits.  Each 128-class chunk of a shard's product leaves, per row, its local max, local
 * exp-sum and the label's logit straight from the fp32 accumulator; these partials are then
 * reduced across chunks and shards in a fixed order (the two reductions of Section 6.3).
 *
 *   features [rows, feat]     B,    SBP_BF16
 *   weight   [feat, classes]  S(1), SBP_BF16
 *   labels, loss, row_max, row_sum: as for sbp_softmax_xent
 * The logits are taken from the fp32 accumulator, i.e. they are not rounded to bf16 first.
 * Needs shapes the tensor-core path accepts (16-byte aligned operands; feat and every shard's
 * class count multiples of 8; feat > 0), else SBP_ERR_UNSUPPORTED and nothing is launched. */
size_t sbp_matmul_softmax_xent_workspace_bytes(const sbp_tensor* features, const sbp_tensor* weight);
sbp_status sbp_matmul_softmax_xent(const sbp_tensor* features, const sbp_tensor* weight,
                                   const sbp_tensor* labels, sbp_tensor* loss, sbp_tensor* row_max,
                                   sbp_tensor* row_sum, void* ws, size_t ws_bytes, void* cuda_stream);

/* Backward of the fused classifier with respect to the logits, again without storing them: the
 * product F W is recomputed on the tensor cores and the epilogue writes
 *   grad[i, j] = exp(z_ij - m_i) / S_i - [j == label_i]
 * (softmax minus one-hot, Section 6.3's plan read backwards) as S(1), BF16 or F32, from the forward
 * pass's row_max (m) and row_sum (S), both [rows] B F32.  Same operand rules and
 * SBP_ERR_UNSUPPORTED conditions as sbp_matmul_softmax_xent, plus 16-byte aligned result shards.
 * The gradient feeds dW = F^T grad and dF = grad W^T, which this library does not compute. */
sbp_status sbp_matmul_softmax_xent_backward(const sbp_tensor* features, const sbp_tensor* weight,
                                            const sbp_tensor* labels, const sbp_tensor* row_max,
                                            const sbp_tensor* row_sum, sbp_tensor* grad_logits, void* cuda_stream);

/* Variant of sbp_softmax_xent for callers that have no device workspace to give and may not
 * create one.  (The paper has no counterpart; this exists for programs that embed the library
 * under constraints the paper does not discuss.)  Typical cases: a plug-in that runs inside
 * someone else's memory plan, where every device byte was handed out up front and a fresh
 * allocation would either fail or stall the device; or a latency-critical path that must not
 * enter the allocator.  Same arguments, results and checks as sbp_softmax_xent, minus
 * ws / ws_bytes: the per-shard partial vectors go into an array that is part of the library.
 *
 *   - The array is SBP_SOFTMAX_XENT_STATIC_SCRATCH_BYTES large and every GPU that loads the
 *     library holds it until the process ends.  A shape whose partials need more is refused
 *     with SBP_ERR_WORKSPACE and nothing is launched; use sbp_softmax_xent for those.
 *   - The call allocates nothing on the device and frees nothing.
 *   - The first call on each device looks up the array's device address (that device must be
 *     current, as it must for the launch anyway).  Make that first call ahead of any stream
 *     capture.
 *   - All calls share the one array, and it keeps whatever the previous call left there.
 *     Nothing in it has to start at zero: each call overwrites every entry it later reads.
 *     Two calls that overlap on the GPU (different streams, no ordering between them) race on
 *     it and may both produce wrong results; keep calls ordered. */
#define SBP_SOFTMAX_XENT_STATIC_SCRATCH_BYTES (3u * 1024u * 1024u)
sbp_status sbp_softmax_xent_static(const sbp_tensor* logits, const sbp_tensor* labels, sbp_tensor* loss,
                                   sbp_tensor* row_max, sbp_tensor* row_sum, void* cuda_stream);

/* ---------------------------------------------------------------- row-split embedding
 *
 * Section 6.3 (embedding table S(0), "splitting the vocabulary IDs"):
 *   table [rows, dim]   S(0) (or S(1), see below), SBP_F32 or SBP_BF16
 *   ids   [...]         B, SBP_I64, 1 <= ndim <= 3
 *   out   [..., dim]    P(sum): shard r writes table row id where id falls in its own row
 *                       range and zeros elsewhere (the k outputs sum to the lookup);
 *                       or B: the lookup itself, written to every replica -- the
 *                       P(sum)->B boxing fused into the gather (exactly one shard
 *                       contributes to a row, so the sum is that row; a -0.0 entry is
 *                       written as +0.0 when k > 1, as x + 0 would give).
 * The table may instead be S(1) (Section 6.3: "splitting the hidden dimension"): every shard
 * then holds a column block of every row, and out is either split along its last axis the same
 * way (each shard's lookup in its own block) or B (whole rows assembled and written to every
 * replica: the all-gather fused into the gather).
 * An id outside [0, rows) produces a zero row and, when oob_count is not NULL, adds 1 to
 * the device int32 it points to (the caller zeroes it).
 */
sbp_status sbp_embedding(const sbp_tensor* table, const sbp_tensor* ids, sbp_tensor* out,
                         int32_t* oob_count, void* cuda_stream);

/* Backward of the row-split lookup: the gradient of the table, S(0) like the table itself.
 *   grad_out   [..., dim]   B, SBP_F32   gradient of the lookup's result
 *   ids        [...]        B, SBP_I64   the ids of the forward pass
 *   grad_table [rows, dim]  S(0), SBP_F32: row i = sum of grad_out over the lookups of id i,
 *                           zero for rows never looked up (the whole tensor is written)
 * dim must be a multiple of 4.  The sums are accumulated with fp32 atomic adds in no fixed
 * order, so a row that many lookups hit may differ in its last bits from run to run.  Ids
 * outside [0, rows) contribute nothing (and are counted in oob_count when it is not NULL).
 * Two launches (zero fill, then scatter-add): every argument check comes before the first, but
 * should the second LAUNCH itself fail (SBP_ERR_CUDA) the gradient has already been zeroed. */
sbp_status sbp_embedding_backward(const sbp_tensor* grad_out, const sbp_tensor* ids, sbp_tensor* grad_table,
                                  int32_t* oob_count, void* cuda_stream);

#ifdef __cplusplus
}
#endif
#endif /* SBP_H_ */
