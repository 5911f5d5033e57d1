// Internal declarations shared by the translation units of libmuon_b200.  Not part of the ABI.
#pragma once

#include <cuda_runtime.h>
#include <cuda_bf16.h>
#include <stdint.h>

#include <string>
#include <unordered_map>
#include <vector>

#include "../../include/muon_b200.h"

namespace muon {

constexpr int kElemTile = 64;       // elementwise kernels work on 64x64 tiles of the source matrix
constexpr int kCopyChunk = 16384;   // elements per gather/scatter work item

// Per-matrix record read by the elementwise kernels (device copy is uploaded per call).
struct alignas(16) MatDesc {
  void* w;          // step: fp32 params (in/out)        | orthogonalize: output matrix
  const void* g;    // step: gradients                   | orthogonalize: input matrix
  void* m;          // step: fp32 momenta (in/out)       | orthogonalize: unused
  void* o;          // step: optional copy of the NS output O in the NS element type (may be null)
  int64_t ld;           // elements between consecutive rows of w, g, m and o (== cols for dense matrices)
  int32_t rows, cols;
  int32_t transposed;   // rows > cols: X holds the transpose
  float scale;          // 0.2*sqrt(max(rows, cols))
  int32_t seg_begin;    // flat-shard mode: first RowSeg of this matrix; w, g, m, o are then the flat buffers' bases
  int32_t seg_count;    // 0 = dense/strided addressing through ld
};

// Rows [row_begin, row_begin + row_count) of a matrix live contiguously at flat_offset (elements) of a flat shard buffer.
struct alignas(16) RowSeg {
  int32_t row_begin, row_count;
  int64_t flat_offset;
};

// One shape group's share of a batched Newton-Schulz invocation: `count` matrices of one core shape (s <= l).
struct Chunk {
  int32_t s = 0, l = 0;  // core shape: s = min(rows, cols), l = max(rows, cols)
  int32_t ldx = 0, lda = 0;      // leading dimensions (elements) of X [s x ldx] and of A, B [s x lda]
  int32_t count = 0;
  int32_t tiles_per_mat = 0;     // elementwise 64x64 tiles per matrix
  int32_t desc_begin = 0;        // index of the first MatDesc of this chunk in the uploaded table
  int32_t set = 0;               // launch set this chunk belongs to
  bool pitch8 = true;            // every matrix of the chunk has a row pitch that is a multiple of 8 elements
  size_t off_x[2] = {0, 0}, off_a = 0, off_b = 0;   // byte offsets of the chunk's buffers in the workspace
  int64_t part_off = 0;          // float index of the chunk's tile partial sums inside the set's partial-sum area
  std::vector<int32_t> mats;     // caller indices, in caller order
};

// Chunks that are resident in the workspace together (at most chunk_elems elements in total): every
// product of a Newton-Schulz step is ONE launch over all of them.
struct LaunchSet {
  std::vector<int32_t> chunks;      // indices into Plan::chunks; their MatDescs are contiguous
  int32_t desc_begin = 0, count = 0;
  size_t off_partials = 0, off_rnorm = 0, bytes = 0;
  int64_t elems = 0;
};

struct SetTables;   // tensor-core tables of one launch set (tc_tables.h)

struct Plan {
  std::vector<Chunk> chunks;
  std::vector<LaunchSet> sets;
  size_t ws_bytes = 0;
  int32_t live = 0;      // matrices with rows > 0 and cols > 0
  bool pipeline_ordered = false;   // the sets are listed in the order the host-buffer pipeline runs them (ramps at both ends)
  // tensor-core tables: built when the plan first runs on a workspace, rebuilt when the workspace moves
  void* d_tables = nullptr;
  const void* tables_ws = nullptr;
  std::vector<SetTables>* set_tables = nullptr;   // owned; one entry per launch set
};

size_t elem_bytes_of_ns(int ns_precision);
int build_plan(const muon_options_t& opt, const muon_shape_t* shapes, int32_t count, Plan* plan,
               const uint8_t* odd_pitch = nullptr, int64_t edge_elems = 0);
// Lays the chunks of one launch set out in a workspace (fills Chunk::off_*, part_off and the set's offsets).
void layout_set(const muon_options_t& opt, std::vector<Chunk>* chunks, LaunchSet* set);
// Tile list of a symmetric product over nb x nb blocks of 128: every unordered pair of blocks exactly once.
struct TilePatHost {
  uint16_t ra, rb, cc, cd;
};
std::vector<TilePatHost> symmetric_tile_pattern(int nb);
int validate_layout_host(const muon_layout_desc_t* d);
// 1 when two of the strided views (element (0,0) at bases[i]) share an element, else 0.
int views_overlap_host(const void* const* bases, const muon_view_t* views, int32_t count, int32_t elem_size);
int owner_plan_host(const muon_shape_t* shapes, int32_t count, int32_t ranks, int64_t batch_elems, int32_t* owner_of,
                    int32_t* batch_of, int32_t* num_batches);

// Copy work item of the gather/scatter kernel.
struct alignas(16) CopyItem {
  int64_t flat_offset;   // elements
  int64_t elem_begin;    // elements, inside the matrix
  int32_t matrix;
  int32_t count;         // elements, <= kCopyChunk
};

struct StagingSlot {
  void* host = nullptr;
  void* dev = nullptr;
  size_t cap = 0;
  cudaEvent_t ev = nullptr;
  bool used = false;
};

struct PhaseSpan {
  int phase;
  cudaEvent_t a, b;
  int64_t launches;
};

}  // namespace muon

struct muon_layout {
  muon_layout_desc_t desc;            // shapes/segments pointers are nulled after create
  std::vector<muon_shape_t> shapes;
  muon::CopyItem* d_items = nullptr;                 // sorted by flat offset: the items of a shard are contiguous
  int64_t num_items = 0;
  std::vector<int64_t> shard_item_begin;              // num_shards + 1 entries into d_items
  float* d_scales = nullptr;                          // per matrix: 0.2 * sqrt(max(rows, cols))
  int device = 0;
  std::vector<std::vector<muon_segment_t>> segs_of;   // host copy of the segment table, grouped by matrix
  bool row_aligned = false;                           // every segment holds whole rows: the flat buffers can be addressed in place
  int32_t flat_vec = 1;                               // largest of 8, 4, 1 that divides every row segment's flat offset
  muon::RowSeg* d_rowsegs = nullptr;                  // device, all matrices' row segments, sorted by row inside a matrix
  std::vector<int32_t> rowseg_begin, rowseg_count;    // per matrix: its range in d_rowsegs
};

struct muon_ctx {
  muon_options_t opt;
  int device = 0;
  void* ws = nullptr;
  size_t ws_bytes = 0;
  int32_t* d_status = nullptr;                     // device status word of the bounded waits
  muon::StagingSlot slots[4];
  int next_slot = 0;
  std::unordered_map<std::string, muon::Plan> plans;
  bool profiling = false;
  std::vector<muon::PhaseSpan> spans;
  std::vector<cudaEvent_t> event_pool;
  double phase_ms[MUON_NUM_PHASES] = {0, 0, 0, 0, 0};
  int64_t phase_launches[MUON_NUM_PHASES] = {0, 0, 0, 0, 0};
  int64_t launches = 0;
  int64_t tmap_encodes = 0;                        // tensor maps encoded so far (plan binding and the per-launch engines)
  uint32_t barrier_count = 0;                      // arrivals the grid-barrier counter (d_status[16]) has seen so far
  int persist_pairs = -1;                          // CTA pairs a whole-iteration launch may use (-1: not asked yet, 0: off)
  void* tmap_encode = nullptr;                     // cuTensorMapEncodeTiled, resolved at run time
  cudaStream_t h2d_stream = nullptr, d2h_stream = nullptr;   // copy streams of the host-buffer path (created on first use)
  std::vector<cudaEvent_t> sync_events;            // untimed events that order the copy streams against the caller's stream
  size_t next_sync_event = 0;
};

namespace muon {

// ---- kernel launchers (defined in the .cu files); each returns the number of kernels launched or < 0
int launch_copy(const CopyItem* items, int64_t num_items, void* flat, void* const* d_mats, int elem_size,
                bool scatter, cudaStream_t st);

int launch_shard_momentum(const CopyItem* items, int64_t num_items, int64_t shard_base, const void* g, void* m, void* staged,
                          float mu, int nesterov, int grad_dtype, int ns_precision, cudaStream_t st);
int launch_shard_apply(const CopyItem* items, int64_t num_items, int64_t shard_base, void* w, const void* const* d_updates,
                       const float* d_scales, float lr, float decay, int ns_precision, cudaStream_t st);

// One shape group inside an elementwise launch.
struct ElemChunk {
  int32_t block_begin;   // first block of this chunk in the launch
  int32_t tiles;         // blocks per matrix
  int32_t desc_begin;    // first MatDesc / rnorm entry, relative to the launch set
  int32_t count;
  int32_t s, l, ldx, pad;
  int64_t x_off;         // byte offset in the workspace of the X iterate this launch writes (stage) or reads (apply)
  int64_t part_off;      // float index of the chunk's partial sums
};
constexpr int kMaxElemChunks = 8;

struct StageArgs {
  const RowSeg* segs;     // device row-segment table (flat-shard mode), else null
  const MatDesc* descs;   // device, first record of the launch set
  char* ws;               // device, workspace base
  double* partials;       // device, the set's tile sums of squares
  float* rnorm;           // device, one per matrix of the set
  float mu, eps;
  int32_t nesterov, grad_dtype, ns_precision;
  int32_t momentum;       // 1: full momentum rule; 0: plain staging of the input (orthogonalize)
  int32_t normalize;      // 0: rnorm = 1
  int32_t wide;           // 1: rows, cols and every row pitch are multiples of 8: the 8-elements-per-thread kernels apply
  int32_t flat_vec;       // flat-shard mode: every segment offset is a multiple of this many elements (8, 4 or 1)
  int32_t nchunks;
  ElemChunk ch[kMaxElemChunks];
};
int launch_stage(const StageArgs& a, cudaStream_t st);

struct ApplyArgs {
  const RowSeg* segs;     // device row-segment table (flat-shard mode), else null
  const MatDesc* descs;
  const char* ws;
  float lr, wd;
  float decay;            // 1 - lr*wd, computed once on the host so that every update route uses the same value
  int32_t ns_precision;
  int32_t update;         // 1: W <- W(1-lr*wd) - lr*scale*O ; 0: write O into descs[i].w in the NS element type
  int32_t wide;           // as in StageArgs
  int32_t flat_vec;
  int32_t nchunks;
  ElemChunk ch[kMaxElemChunks];
};
int launch_apply(const ApplyArgs& a, cudaStream_t st);

// Writes up to 3 KiB of host data into device memory with a kernel (the data travels as a kernel argument):
// no staging buffer, no host-to-device copy that could outlive its source.
int launch_poke(void* dst, const void* src, size_t bytes, cudaStream_t st);

// C[k] = gamma_k * (beta * D[k] + alpha * op(P[k], Q[k]) + diag * I),  op = P Q^T (nn=0) or P Q (nn=1)
struct GemmArgs {
  const void* p; const void* q; const void* d; void* c;
  int32_t m, n, kdim;
  int32_t ldp, ldq, ldc;           // D shares ldc
  int64_t stride_p, stride_q, stride_c;   // elements between consecutive matrices
  int32_t batch;
  const float* rnorm;  // device, per matrix
  int32_t gamma_mode;  // 0: 1, 1: r, 2: r*r
  float alpha, beta;
  float diag;          // added to the diagonal elements C[i][i] (square results)
  int32_t nn;
  int32_t symmetric;   // op is P P^T with symmetric result (kernels may exploit it)
  // per-matrix coefficients: matrix k takes alpha = coef[k * coef_stride + coef_a] (beta, diag likewise with coef_b, coef_d) when
  // coef is set and the index is >= 0
  const float* coef;   // device or null
  int32_t coef_a, coef_b, coef_d, coef_stride;   // coef_d: index that replaces diag
};
int launch_gemm_simt(const GemmArgs& a, int ns_precision, cudaStream_t st);
int launch_gemm_tc(muon_ctx* ctx, const GemmArgs& a, cudaStream_t st);   // tcgen05 engine, single-CTA kernel (bf16 only)
bool tc_supported(const GemmArgs& a);
int launch_bounded_wait_probe(muon_ctx* ctx, cudaStream_t st);            // a wait that must expire (self-test)

}  // namespace muon
