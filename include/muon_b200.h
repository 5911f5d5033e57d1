/*
 * muon_b200.h -- C ABI of the B200-native layout-driven Muon step.
 *
 * The library implements the local compute core of the paper's distributed Muon
 * (Section 6, Algorithm 2): whole matrices are materialised from a padded flat
 * FSDP-style shard buffer, every 2-D matrix receives one Muon update
 * (momentum -> Frobenius normalisation -> Newton-Schulz iteration of Eq. 1 ->
 * shape-scaled, weight-decayed update), and results are scattered back.
 *
 * Conventions (all entry points)
 *  - Every call returns MUON_OK (0) or a negative MUON_ERR_* code.  Nothing is
 *    launched when validation fails.  No exception crosses this boundary.
 *  - "device pointer" = address in the current CUDA device's global memory, owned by
 *    the caller; "host pointer" = ordinary process memory, read during the call only
 *    unless stated otherwise.
 *  - Arrays of matrix pointers (params, grads, ...) are HOST arrays of DEVICE pointers.
 *  - Matrices are dense row-major with leading dimension == cols.
 *  - `stream` is a cudaStream_t passed as void* (NULL = the legacy default stream).
 *    All device work is enqueued on it; calls do not synchronise the stream, except
 *    that the library may wait on the host for one of its OWN earlier pointer-table
 *    uploads before re-using a staging slot.
 *  - The library allocates only small device tables (layout chunk tables, per-plan
 *    descriptors).  The Newton-Schulz workspace is caller-owned (muon_set_workspace).
 *  - A context is bound to the device that was current in muon_create and must be used
 *    with that device current; calls on one context must not overlap in time on the
 *    host (one thread at a time), and device work of consecutive calls must be ordered
 *    by the caller (same stream or events) because they share the workspace.
 */
#ifndef MUON_B200_H_
#define MUON_B200_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

/* ------------------------------------------------------------------ status codes */
#define MUON_OK                      0
#define MUON_ERR_INVALID_ARG        -1   /* null pointer, negative count, bad enum, misaligned buffer      */
#define MUON_ERR_BAD_LAYOUT         -2   /* segment table does not describe a valid flat-shard layout      */
#define MUON_ERR_UNSUPPORTED        -3   /* legal request the library does not implement                   */
#define MUON_ERR_WORKSPACE_TOO_SMALL -4  /* muon_set_workspace not called, or buffer smaller than required  */
#define MUON_ERR_CUDA               -5   /* a CUDA runtime/driver call failed (no usable device, launch...) */
#define MUON_ERR_DEVICE_TIMEOUT     -6   /* a bounded device-side wait gave up; returned by muon_synchronize_and_check only */
#define MUON_ERR_TOO_LARGE          -7   /* the matrix needs more than the fixed built-in scratch (muon_orthogonalize_static) */

/* ------------------------------------------------------------------ enums */
#define MUON_DTYPE_BF16 0
#define MUON_DTYPE_FP32 1

#define MUON_NS_BF16 0   /* bf16 operands, fp32 accumulation on the tensor cores (Section 6.6: "bf16 arithmetic") */
#define MUON_NS_FP32 1   /* every product and intermediate in fp32 (no counterpart in the paper; accuracy anchor)  */

#define MUON_ENGINE_TENSOR      0   /* tensor cores, CTA pairs (cta_group::2), one launch per product for all shape groups */
#define MUON_ENGINE_CUDA_CORE   1
#define MUON_ENGINE_TENSOR_1CTA 2   /* tensor cores, single-CTA kernel, one launch per product per shape group (cross-check) */

/* flags of muon_orthogonalize_batched */
#define MUON_ORTHO_NO_NORMALIZE 1u  /* treat the input as X_0 already (r = 1); used for single-step checks */

typedef struct muon_ctx    muon_ctx_t;
typedef struct muon_layout muon_layout_t;

/* Shape of one dense row-major matrix (Section 2.3: W in R^{m x n}). */
typedef struct { int32_t rows, cols; } muon_shape_t;

/* A logical matrix inside a larger physical parameter (the model adapter of Section 6.6:
 * storage layout and the matrices the optimizer works on are separate things, e.g. the heads of a
 * fused QKV projection, the gate and up halves of an MoE FC1 weight, the factors of an MLA
 * projection, the E planes of an [E, M, N] expert tensor, which Section 6.3 says are E separate matrices).  rows x cols elements, row r starting ld elements after row r-1. */
typedef struct { int32_t rows, cols; int64_t ld; } muon_view_t;

/* One contiguous piece of a matrix inside the flat buffer: elements
 * [elem_begin, elem_begin+elem_count) of the row-major linearisation of matrix
 * `matrix` live at flat[flat_offset, flat_offset+elem_count).  Units: elements. */
typedef struct {
  int32_t matrix;
  int32_t reserved;      /* must be 0 */
  int64_t elem_begin;
  int64_t elem_count;
  int64_t flat_offset;
} muon_segment_t;

/* Flat FSDP-style shard buffer (the aligned, padded fused buffer of Section 5.2; the staging buffer of the
 * fused gather, Section 6.4 step 1, which is aligned, bf16 and may be split unevenly): num_shards consecutive
 * shards of shard_len elements each; segment starts are multiples of align_elems;
 * everything not covered by a segment is padding that is never read nor written. */
typedef struct {
  int32_t elem_size;              /* 2 (bf16) or 4 (fp32) bytes per element                */
  int32_t align_elems;            /* > 0; every flat_offset must be a multiple of it        */
  int32_t num_shards;             /* >= 1                                                   */
  int32_t num_matrices;           /* >= 0                                                   */
  int64_t shard_len;              /* elements per shard, multiple of align_elems            */
  const muon_shape_t*   shapes;   /* host, num_matrices entries                             */
  int64_t num_segments;
  const muon_segment_t* segments; /* host, num_segments entries; copied by muon_layout_create */
} muon_layout_desc_t;

typedef struct {
  int32_t grad_dtype;      /* MUON_DTYPE_BF16 | MUON_DTYPE_FP32: element type of `grads`                     */
  int32_t ns_precision;    /* MUON_NS_BF16 | MUON_NS_FP32                                                    */
  int32_t nesterov;        /* 1: u = G + mu*M' (Section 7.4 set-up), 0: u = M'                                 */
  int32_t coeffs_per_step; /* 0: coeffs[3] used at every step; 1: coeffs[3*ns_steps], (a_k,b_k,c_k) per step */
  float   eps;             /* epsilon of Eq. 1, added to the Frobenius norm; default 1e-7                    */
  int32_t engine;          /* MUON_ENGINE_TENSOR (default) | MUON_ENGINE_TENSOR_1CTA | MUON_ENGINE_CUDA_CORE (bf16  */
                           /* products on CUDA cores; slow cross-check); fp32 NS always runs on CUDA cores          */
  int64_t chunk_elems;     /* batching cap in elements per batched NS invocation; default 1<<29 (Section 6.6) */
  int32_t coeffs_per_matrix; /* 1: `coeffs` holds one row per matrix of the call, [count][3] or [count][3*ns_steps]:   */
                           /* matrices of one call may iterate with different polynomials (a per-parameter-group  */
                           /* choice in the pluggable design of Section 6.2); they still share their launches       */
  int32_t launch_per_product; /* 0 (default): a launch set with only a few tiles per product runs its whole Newton-Schulz   */
                           /* iteration as ONE launch (grid barriers between the products); 1: every product is always   */
                           /* a launch of its own (15 per set for five steps) -- same tiles, same results                  */
} muon_options_t;

/* Fills *opt with the defaults: bf16 grads, bf16 NS, Nesterov, constant coefficients, eps 1e-7, cap 2^29. */
int muon_default_options(muon_options_t* opt);

/* Creates a context on the current CUDA device.  MUON_ERR_CUDA when no device is usable
 * (the library never falls back to the CPU). */
int  muon_create(muon_ctx_t** ctx, const muon_options_t* opt);
void muon_destroy(muon_ctx_t* ctx);

/* Bytes of device workspace that muon_step_batched / muon_orthogonalize_batched need for
 * this list of shapes under these options (one workspace per batched invocation rather than
 * per matrix, Section 6.6).  Pure host arithmetic; needs no device. */
int muon_workspace_bytes(const muon_options_t* opt, const muon_shape_t* shapes, int32_t count, size_t* bytes);

/* Hands the library a caller-owned device buffer (256-byte aligned) used as workspace by
 * every later call on this context until replaced.  The caller keeps ownership. */
int muon_set_workspace(muon_ctx_t* ctx, void* dev_ptr, size_t bytes);

/* Host-only description of how a shape list is batched: matrices are grouped by core
 * shape (min(m,n), max(m,n)) -- the paper's shape-fused batching, Section 6.6 -- and each
 * group is cut into chunks of at most chunk_elems elements (at least one matrix).
 * chunk_of[i] receives the chunk index of matrix i (may be NULL); *num_chunks the count. */
int muon_plan_describe(const muon_options_t* opt, const muon_shape_t* shapes, int32_t count,
                       int32_t* num_chunks, int32_t* chunk_of);

/* Host-only description of how the chunks are launched: chunks are packed (first fit, largest first) into
 * launch sets of at most chunk_elems elements in total -- the memory-safe cap of Section 6.6 then bounds what
 * is resident in the workspace at once -- and the tensor engine runs every Newton-Schulz product as ONE kernel
 * per launch set, over all its core shapes (3 * ns_steps product launches per set; small groups no longer
 * get launches of their own: "per-matrix NS launches starve the device for small matrices", Section 6.6).
 * set_of[i] receives the launch set of matrix i (-1 for empty matrices; may be NULL); *num_sets the count. */
int muon_plan_launch_sets(const muon_options_t* opt, const muon_shape_t* shapes, int32_t count,
                          int32_t* num_sets, int32_t* set_of);

/* Host-only description of what muon_step_flat_host runs: the launch sets of its plan -- the plan above with two
 * small sets (about 2^24 elements each) split off the group with the smallest matrices -- and the order in which the
 * pipeline runs them: one small set first and the other last, because the inbound copy before the first kernel and
 * the outbound copy after the last one are the only copies nothing overlaps; in between, largest first (the
 * descending-size order of Section 6.7).  set_of[i]: launch set of matrix i (-1 for empty matrices; may be NULL);
 * order[k]: the set that runs k-th (may be NULL; at most order_capacity entries are written). */
int muon_plan_pipeline(const muon_options_t* opt, const muon_shape_t* shapes, int32_t count, int32_t* num_sets,
                       int32_t* set_of, int32_t* order, int32_t order_capacity);

/* Host-only: the tile list the tensor engine uses for a symmetric product (A = X X^T, A A^T) whose result has
 * `blocks` x `blocks` blocks of 128 rows/columns.  Tile i is tiles[4i..4i+3] = (ra, rb, cc, cd): row blocks ra
 * and rb (one per CTA of a pair; 0xFFFF = none) against column blocks cc and cd (0xFFFF = the tile is 128
 * columns wide).  Every unordered pair of blocks is covered (the kernel mirrors off-diagonal blocks); the only
 * block computed twice is the lower-left one of each diagonal 2 x 2 tile, and a last odd column gets 128-wide
 * tiles instead of half-empty 256-wide ones.  *count receives the number of tiles; at most `capacity` are
 * written.  Exposed so that the combinatorics can be tested on a CPU. */
int muon_symmetric_tiles(int32_t blocks, uint16_t* tiles, int32_t capacity, int32_t* count);

/* Validates a layout description on the host (no device needed): every element of every
 * matrix covered exactly once; segments inside one shard, pairwise disjoint in the flat
 * buffer, starts aligned; reserved fields zero.  MUON_ERR_BAD_LAYOUT otherwise. */
int muon_layout_validate(const muon_layout_desc_t* desc);

/* Validates and uploads a layout; the handle is immutable and may be used by any number of
 * materialize/scatter calls.  `desc` and what it points to may be freed afterwards. */
int  muon_layout_create(muon_ctx_t* ctx, const muon_layout_desc_t* desc, muon_layout_t** out);
void muon_layout_destroy(muon_layout_t* layout);

/* muon_materialize: unpack the flat shard buffer into whole matrices -- the copy-out half
 * of a fused gather (Section 6.4 step 1; the copy-in / copy-out passes of Section 5.1).
 *   flat_buf : device, num_shards*shard_len elements of elem_size bytes, 16-byte aligned
 *   matrices : host array [num_matrices] of device pointers, each rows*cols elements
 * Bit-exact byte movement; padding is never read. */
int muon_materialize(muon_ctx_t* ctx, const void* flat_buf, const muon_layout_t* layout,
                     void* const* matrices, void* stream);

/* muon_scatter: the inverse -- pack whole matrices into the flat shard buffer (the pack
 * before the relay broadcast, Section 6.4 step 3).  Padding elements of flat_buf are
 * never written. */
int muon_scatter(muon_ctx_t* ctx, void* flat_buf, const muon_layout_t* layout,
                 const void* const* matrices, void* stream);

/* ------------------------------------------------------------------ owner-sharded step (several ranks)
 * The pieces of the paper's shard-domain deduplication (Section 6.4, Figure "Two-level deduplication" (a)) and of
 * its batch pipeline (Section 6.7, Algorithm 2), as calls a rank makes on the shard it holds.  The library does
 * no communication: the caller moves the staged shards and the updates between ranks (all-gather in, broadcast
 * out) and these calls do everything else.  One step of one batch on rank r of S:
 *     muon_shard_momentum(layout, r, G_r, M_r, U_r)            momentum on the local shard; U_r is what the
 *                                                              fused gather sends (step 1)
 *     [all-gather U_0..U_{S-1} into one flat buffer]
 *     muon_materialize_owned(flat U, layout, owned matrices)   only the owner materialises a matrix (step 2)
 *     muon_orthogonalize_batched(owned matrices)               batched Newton-Schulz over core-shape groups
 *     [broadcast every owner's updates]                        relay broadcast (step 3)
 *     muon_shard_apply(layout, r, W_r, updates)                slice extraction and update with decay (step 4)
 * Momentum and parameters stay sharded throughout.  Assembled this way the step is bit-identical to
 * muon_step_batched on the whole matrices. */

/* Host-only: compute-owner assignment and batching.  Matrices are packed into batches in descending size
 * (Section 6.7: large matrices first; a batch is closed when the next matrix would take it beyond batch_elems
 * elements; batch_elems <= 0: one batch), and inside a batch each matrix is assigned to exactly one of `ranks`
 * owners by greedy balancing of its Newton-Schulz work, 3 s^2 l + s^3 (Section 6.4 step 2: "greedy size
 * balancing"): matrices in descending work, each to the least-loaded rank, lowest rank on ties.  Deterministic;
 * a batch's largest load is within 4/3 - 1/(3 ranks) of the best possible.  owner_of[i], batch_of[i] receive
 * rank and batch of matrix i (-1 for empty matrices); *num_batches the number of batches. */
int muon_owner_plan(const muon_shape_t* shapes, int32_t count, int32_t ranks, int64_t batch_elems,
                    int32_t* owner_of, int32_t* batch_of, int32_t* num_batches);

/* Shard-local momentum (Section 6.4 step 1, the part before the gather): for every element of shard `shard`
 * of the layout,  M <- mu*M + G;  staged = cast(G + mu*M)  (opt.nesterov) or cast(M).
 *   local_grads   : device, opt.grad_dtype, the shard_len elements of this shard (element 0 = flat offset
 *                   shard*shard_len)
 *   local_momenta : device, fp32, same extent, in/out
 *   local_staged  : device, NS element type, same extent, out
 * Padding elements are neither read nor written. */
int muon_shard_momentum(muon_ctx_t* ctx, const muon_layout_t* layout, int32_t shard, const void* local_grads,
                        void* local_momenta, void* local_staged, float mu, void* stream);

/* muon_materialize / muon_scatter for a subset: entries of `matrices` that are NULL are skipped (an owner
 * materialises only the matrices assigned to it, Section 6.4 step 2, and packs only its own updates, step 3). */
int muon_materialize_owned(muon_ctx_t* ctx, const void* flat_buf, const muon_layout_t* layout,
                           void* const* matrices, void* stream);
int muon_scatter_owned(muon_ctx_t* ctx, void* flat_buf, const muon_layout_t* layout,
                       const void* const* matrices, void* stream);

/* Shard-local slice-and-apply (Section 6.4 step 4): for every element of shard `shard`,
 *     W <- W (1 - lr*wd) - lr * 0.2 sqrt(max(rows, cols)) * O[matrix][element]
 * where updates[i] is the whole rows x cols update of matrix i in the NS element type (the payload of the relay
 * broadcast, wherever the caller received it); the slice this shard holds is taken from it on the fly.
 *   local_params : device, fp32, the shard_len elements of this shard, in/out
 *   updates      : host array [num_matrices] of device pointers; NULL = leave that matrix's slice alone */
int muon_shard_apply(muon_ctx_t* ctx, const muon_layout_t* layout, int32_t shard, void* local_params,
                     const void* const* updates, float lr, float wd, void* stream);

/* muon_step_batched: one Muon update of `count` independent matrices (Section 2.3, Eq. 1;
 * the complete-matrix path of Algorithm 2: momentum, batched Newton-Schulz, apply):
 *     M <- mu*M + G;  u = G + mu*M (Nesterov) or M;  U = cast(u)
 *     X_0 = U / (||U||_F + eps), run on U^T when rows > cols (transpose-first, Section 6.6)
 *     X_{k+1} = a_k X_k + (b_k A + c_k A^2) X_k,  A = X_k X_k^T,  k = 0..ns_steps-1
 *       (evaluated as the matrix polynomial it is: X_{k+1} = P_k X_k with P_k = a_k I + b_k A + c_k A^2; in bf16 mode each
 *        produced matrix -- A, P_k, X_{k+1} -- is rounded once, products accumulate in fp32)
 *     W <- W (1 - lr*wd) - lr * 0.2 sqrt(max(rows, cols)) * X_ns
 *   params, momenta : host arrays [count] of device pointers to fp32 matrices (in/out)
 *   grads           : host array  [count] of device pointers, element type opt.grad_dtype
 *   shapes          : host, [count]; a matrix with rows==0 or cols==0 is skipped
 *   coeffs          : host, 3 floats (or 3*ns_steps when opt.coeffs_per_step); with opt.coeffs_per_matrix one such
 *                     row per matrix, row i for matrix i of this call
 * All matrix pointers must be 16-byte aligned.  Matrices are batched by core shape; the
 * results do not depend on how they are batched (bit-identical run to run). */
int muon_step_batched(muon_ctx_t* ctx, void* const* params, const void* const* grads, void* const* momenta,
                      const muon_shape_t* shapes, int32_t count, float lr, float mu, float wd,
                      int32_t ns_steps, const float* coeffs, void* stream);

/* muon_step_batched_out: muon_step_batched that additionally writes each matrix's orthogonalised
 * update O = X_ns (shape rows x cols, element type of the NS precision) to updates[i] -- the payload
 * owners pack for the relay broadcast (Section 6.4 step 3).  updates may be NULL (then identical to
 * muon_step_batched); otherwise a host array [count] of 16-byte-aligned device pointers. */
int muon_step_batched_out(muon_ctx_t* ctx, void* const* params, const void* const* grads, void* const* momenta,
                          void* const* updates, const muon_shape_t* shapes, int32_t count, float lr, float mu,
                          float wd, int32_t ns_steps, const float* coeffs, void* stream);

/* muon_step_batched_views: muon_step_batched_out on strided views, so that logical matrices are
 * updated in place inside their physical parameters without split/concatenate copies and without a
 * restore pass (the zero-copy view and the restore mapping of the model adapter, Section 6.6).
 * params[i], grads[i], momenta[i] and, when given, updates[i] point at element (0,0) of view i inside
 * tensors that share the physical layout; all use views[i].ld as row stride (ld >= cols).  Pointers must
 * be 16-byte aligned; the vectorised path also needs ld to be a multiple of 4 elements (other strides
 * run element-wise).  Elements outside the views are never touched.  Two views of one call that share an element of
 * params, momenta or updates are rejected with MUON_ERR_INVALID_ARG before anything is launched (the check is
 * muon_views_overlap applied to each of the three pointer arrays). */
int muon_step_batched_views(muon_ctx_t* ctx, void* const* params, const void* const* grads, void* const* momenta,
                            void* const* updates, const muon_view_t* views, int32_t count, float lr, float mu,
                            float wd, int32_t ns_steps, const float* coeffs, void* stream);

/* Host arithmetic only (needs no device): *overlap = 1 when two of the strided views -- view i has element (0,0)
 * at address bases[i], rows x cols elements of elem_size bytes, ld elements between rows -- share a byte, else 0.
 * Views with rows == 0, cols == 0 or a NULL base are ignored.  This is the check muon_step_batched_views applies to
 * what it writes, so that the logical matrices of one physical parameter (row blocks of a fused QKV, interleaved
 * gate/up rows, [E,M,N] planes: the model adapter of Section 6.6) can be validated once when a model is set up. */
int muon_views_overlap(const void* const* bases, const muon_view_t* views, int32_t count, int32_t elem_size, int32_t* overlap);

/* muon_step_flat: the sharded-state flow of Section 6.4 (steps 1 and 4) on one device -- parameters, momenta and
 * gradients STAY in flat shard buffers that share one layout (in the paper the momentum is never
 * un-sharded, and every rank applies the update to its own slice of the parameters).
 * The momentum rule reads and writes the flat momentum shards in place and stages the cast result
 * straight into the Newton-Schulz workspace (the gather is fused away); the update is applied straight
 * onto the flat fp32 parameter shards and, when flat_updates is given, O is written straight into it
 * (the scatter is fused away).  No whole-matrix copy of any state exists.
 *   flat_params, flat_momenta : device, fp32, num_shards*shard_len elements, in/out
 *   flat_grads                : device, opt.grad_dtype, same element layout
 *   flat_updates              : device or NULL, NS element type, same element layout; padding untouched
 * The layout's elem_size is irrelevant here (offsets are in elements).  Requires a layout whose segments
 * hold whole rows (per-parameter row splits do); otherwise MUON_ERR_UNSUPPORTED and nothing is launched.
 * Results are bit-identical to muon_materialize + muon_step_batched_out + muon_scatter. */
int muon_step_flat(muon_ctx_t* ctx, const muon_layout_t* layout, void* flat_params, const void* flat_grads,
                   void* flat_momenta, void* flat_updates, float lr, float mu, float wd, int32_t ns_steps,
                   const float* coeffs, void* stream);

/* muon_step_flat_host: the whole path on HOST flat buffers, for end-to-end use and timing.
 * host_flat_grads / host_flat_updates are host buffers of num_shards*shard_len elements in the
 * layout's format (pinned memory makes the copies asynchronous).  Per batch of matrices (the chunks of
 * muon_plan_describe) the gradient segments are copied by DMA straight into grads[] -- the copy engine
 * performs the gather of Section 6.4 step 1 -- the batch is updated as in muon_step_batched_out, and
 * its update segments are copied from updates[] straight into host_flat_updates (the pack of step 3).
 * Inbound copies of later batches and outbound copies of earlier ones overlap the Newton-Schulz work
 * on two internal copy streams; padding of host_flat_updates is never written.
 *   grads, updates : host arrays of device pointers to whole-matrix scratch the caller owns
 * The layout's element size must equal both the gradient and the NS element size (bf16/bf16 or
 * fp32/fp32).  Ordering: everything starts after prior work on `stream`, and later work on `stream`
 * waits for the last outbound copy; the host buffers may be touched again once `stream` has been
 * synchronised.  The two copy streams are created on the first call (which therefore allocates). */
int muon_step_flat_host(muon_ctx_t* ctx, const void* host_flat_grads, void* host_flat_updates,
                        const muon_layout_t* layout, void* const* params, void* const* grads, void* const* momenta,
                        void* const* updates, float lr, float mu, float wd, int32_t ns_steps, const float* coeffs,
                        void* stream);

/* muon_orthogonalize_batched: only the Newton-Schulz part of the step (Eq. 1) on given
 * inputs -- for per-kernel parity checks and timing.  Element type of in/out is bf16 under
 * MUON_NS_BF16 and fp32 under MUON_NS_FP32; out[i] has the shape of in[i]; in and out may
 * not alias. */
int muon_orthogonalize_batched(muon_ctx_t* ctx, const void* const* in, void* const* out,
                               const muon_shape_t* shapes, int32_t count,
                               int32_t ns_steps, const float* coeffs, uint32_t flags, void* stream);

/* muon_ns_product: the batched product primitive the Newton-Schulz iteration is built from (the
 * three products of one step of Eq. 1), exposed for per-kernel parity checks and timing:
 *     C[i] = gamma_i * (beta * D[i] + alpha * P[i] Q[i]^T)        nn = 0, P: m x k, Q: n x k
 *     C[i] = gamma_i * (beta * D[i] + alpha * P[i] Q[i])          nn = 1, P: m x k, Q: k x n
 *     C[i] = gamma_i * (beta * D[i] + alpha * P[i] P[i]^T)        nn = 2, symmetric rank-k form: q == p,
 *            m == n, D symmetric (or NULL); only tiles touching the upper triangle are computed and
 *            the strictly upper ones are mirrored, so C is exactly symmetric
 * for i < batch.  All operands are device pointers to row-major matrices of the NS element type
 * (bf16 under MUON_NS_BF16, fp32 under MUON_NS_FP32) with leading dimensions ldp, ldq, ldc in
 * elements (D shares ldc and stride_c; d may be NULL) and stride_* elements between consecutive
 * matrices.  gamma_i = 1 when gamma is NULL, else gamma[i] (gamma_mode 1) or gamma[i]^2
 * (gamma_mode 2), gamma being a device array of `batch` floats.  For the tensor-core engine bases
 * must be 16-byte aligned and every ld/stride a multiple of 8 elements; other cases run on CUDA
 * cores.  C must not alias P, Q or D.  The tensor engine stores C in 16-byte pieces: the padding
 * columns [n, ldc) of a row may be overwritten up to the next multiple of 8 elements. */
int muon_ns_product(muon_ctx_t* ctx, const void* p, const void* q, const void* d, void* c,
                    int32_t m, int32_t n, int32_t k, int32_t ldp, int32_t ldq, int32_t ldc,
                    int64_t stride_p, int64_t stride_q, int64_t stride_c, int32_t batch, int32_t nn,
                    float alpha, float beta, const float* gamma, int32_t gamma_mode, void* stream);

/* muon_orthogonalize_static: muon_orthogonalize_batched for ONE matrix, for callers that cannot
 * allocate device memory.  (The paper has no counterpart; it exists for integration reasons only.)
 *
 * Who needs it: code that runs where cudaMalloc is forbidden or unavailable -- inside a memory
 * pool or allocator callback, in a process whose device memory is fully pre-assigned by another
 * runtime, or in a latency-critical section where an allocation's implicit synchronisation is not
 * acceptable.  Such a caller can create no muon_ctx_t (creation allocates) and own no workspace.
 * This entry point therefore takes no context and allocates nothing: it calls neither cudaMalloc
 * nor cudaFree nor any allocating library routine, on the device or for pinned host memory.  All
 * scratch (the two X iterates, A, B, the norm partial sums and a small descriptor) lives in one
 * fixed array of MUON_STATIC_SCRATCH_BYTES that is part of the library image: every GPU that loads
 * the library holds that much memory until the process exits.
 *
 *   in, out : device, rows x cols row-major, bf16 under MUON_NS_BF16 / fp32 under MUON_NS_FP32,
 *             16-byte aligned, not aliased; the caller owns them
 *   status  : optional device int32 the caller has zeroed; a bounded device-side wait that expires
 *             writes a non-zero code there (NULL: such a code is dropped)
 *   flags   : MUON_ORTHO_NO_NORMALIZE or 0;  coeffs: host, 3 floats
 * Limits: a matrix whose Newton-Schulz workspace exceeds the array (for bf16 roughly
 * 4*rows*cols + 4*min(rows,cols)^2 bytes; 1024 x 1024 fits, 2048 x 2048 does not) is rejected
 * with MUON_ERR_TOO_LARGE and nothing is launched.
 * Set-up: the first call on each device resolves the array's device address and the driver's
 * tensor-map encoder (guarded by a mutex, so first calls may come from several host threads); make
 * that first call outside any stream capture.  The matrix descriptor and the engine's small tables
 * reach the device as kernel arguments, so no host-to-device copy of the call outlives it.
 * Sharing: all calls on a device use the same array, which keeps whatever the previous call left;
 * the entry point rewrites every element it later reads, so no clearing by the caller is needed,
 * but two calls whose device work overlaps in time (different streams without ordering) race. */
#define MUON_STATIC_SCRATCH_BYTES (16u * 1024u * 1024u + 16384u)
int muon_orthogonalize_static(const void* in, void* out, int32_t rows, int32_t cols, int32_t ns_precision,
                              int32_t ns_steps, const float* coeffs, float eps, uint32_t flags,
                              int32_t* status, void* stream);

/* Device-side status word: the tensor-core pipeline bounds every wait on a barrier; a wait
 * that gives up records a non-zero code here and the kernel exits cleanly.  Reads the word
 * after synchronising `stream`; 0 = no bounded wait ever expired on this context. */
int muon_last_device_status(muon_ctx_t* ctx, void* stream, int32_t* status);

/* Resets the status word to 0 (stream-ordered). */
int muon_clear_device_status(muon_ctx_t* ctx, void* stream);

/* Opt-in synchronous check: synchronises `stream`, then returns MUON_OK when no bounded wait has expired on this
 * context and MUON_ERR_DEVICE_TIMEOUT when one has (the results of the affected call are then incomplete).
 * The step entry points themselves never synchronise and therefore never return that code: a caller that wants
 * the guarantee calls this (or muon_last_device_status) before it consumes a step's results. */
int muon_synchronize_and_check(muon_ctx_t* ctx, void* stream);

/* Failure-detection self-test (a test hook, not part of the optimizer path): launches one tiny kernel that waits, with a limit of about a millisecond,
 * on a barrier nothing ever arrives at, using the same bounded-wait routine as the tensor-core pipelines.
 * The wait must expire, the kernel records code 100 in the status word and returns normally; the context
 * stays usable.  No real pipeline is involved and nothing can hang. */
int muon_self_test_bounded_wait(muon_ctx_t* ctx, void* stream);

/* Phase timing (off by default).  When on, the library brackets each phase with CUDA
 * events on the caller's stream; muon_profile_read synchronises those events and adds up,
 * per phase, device milliseconds and kernel launches since the last muon_profile_reset. */
#define MUON_PHASE_MOMENTUM 0   /* fused momentum + Nesterov + cast + sum of squares, and the norm finalise */
#define MUON_PHASE_NS       1   /* the Newton-Schulz product kernels                                      */
#define MUON_PHASE_UPDATE   2   /* fused scaled, weight-decayed update                                    */
#define MUON_PHASE_GATHER   3   /* muon_materialize                                                       */
#define MUON_PHASE_SCATTER  4   /* muon_scatter                                                           */
#define MUON_NUM_PHASES     5
int muon_profile_enable(muon_ctx_t* ctx, int32_t on);
int muon_profile_reset(muon_ctx_t* ctx);
int muon_profile_read(muon_ctx_t* ctx, int32_t phase, double* ms, int64_t* launches);

/* Total kernels this context has launched since creation. */
int64_t muon_launch_count(const muon_ctx_t* ctx);

/* Total tensor maps this context has encoded since creation.  The plan of a shape list encodes its maps once,
 * when it first runs on a workspace (Section 6.2: the plan is fixed when the optimizer is built and replayed
 * unchanged every step); in steady state the count does not move. */
int64_t muon_tensor_map_encodes(const muon_ctx_t* ctx);

const char* muon_status_string(int status);

#ifdef __cplusplus
}
#endif
#endif /* MUON_B200_H_ */
