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

// One batched Newton-Schulz invocation: `count` matrices of one core shape (s <= l).
struct Chunk {
  int32_t s, l;          // core shape: s = min(rows, cols), l = max(rows, cols)
  int32_t ldx, lda;      // leading dimensions (elements) of X [s x ldx] and of A, B [s x lda]
  int32_t count;
  int32_t tiles_per_mat; // elementwise 64x64 tiles per matrix
  int32_t desc_begin;    // index of the first MatDesc of this chunk in the uploaded table
  std::vector<int32_t> mats;  // caller indices, in caller order
};

struct Plan {
  std::vector<Chunk> chunks;
  size_t ws_bytes = 0;
  int32_t live = 0;      // matrices with rows > 0 and cols > 0
};

// Carving of the caller's workspace for the largest chunk.
struct WsCarve {
  size_t x0, x1, a, b, partials, rnorm, total;
};

size_t elem_bytes_of_ns(int ns_precision);
int build_plan(const muon_options_t& opt, const muon_shape_t* shapes, int32_t count, Plan* plan);
WsCarve carve_chunk(const muon_options_t& opt, const Chunk& c);
int validate_layout_host(const muon_layout_desc_t* d);

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
  muon::CopyItem* d_items = nullptr;
  int64_t num_items = 0;
  int device = 0;
  std::vector<std::vector<muon_segment_t>> segs_of;   // host copy of the segment table, grouped by matrix
  bool row_aligned = false;                           // every segment holds whole rows: the flat buffers can be addressed in place
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
  void* tmap_encode = nullptr;                     // cuTensorMapEncodeTiled, resolved at run time
  cudaStream_t h2d_stream = nullptr, d2h_stream = nullptr;   // copy streams of the host-buffer path (created on first use)
  std::vector<cudaEvent_t> sync_events;            // untimed events that order the copy streams against the caller's stream
  size_t next_sync_event = 0;
};

namespace muon {

// ---- kernel launchers (defined in the .cu files); each returns the number of kernels launched or < 0
int launch_copy(const CopyItem* items, int64_t num_items, void* flat, void* const* d_mats, int elem_size,
                bool scatter, cudaStream_t st);

struct StageArgs {
  const RowSeg* segs;     // device row-segment table (flat-shard mode), else null
  const MatDesc* descs;   // device, first record of the chunk
  void* x;                // device, chunk X buffer (bf16 or fp32)
  float* partials;        // device, count*tiles_per_mat
  float* rnorm;           // device, count
  int32_t count, tiles_per_mat, s, l, ldx;
  float mu, eps;
  int32_t nesterov, grad_dtype, ns_precision;
  int32_t momentum;       // 1: full momentum rule; 0: plain staging of the input (orthogonalize)
  int32_t normalize;      // 0: rnorm = 1
  int32_t wide;           // 1: rows, cols and every row pitch are multiples of 8: the 8-elements-per-thread kernels apply
};
int launch_stage(const StageArgs& a, cudaStream_t st);

struct ApplyArgs {
  const RowSeg* segs;     // device row-segment table (flat-shard mode), else null
  const MatDesc* descs;
  const void* x;          // final NS iterate
  int32_t count, tiles_per_mat, s, l, ldx;
  float lr, wd;
  float decay;            // 1 - lr*wd, computed once on the host so that every update route uses the same value
  int32_t ns_precision;
  int32_t update;         // 1: W <- W(1-lr*wd) - lr*scale*O ; 0: write O into descs[i].w in the NS element type
  int32_t wide;           // as in StageArgs
};
int launch_apply(const ApplyArgs& a, cudaStream_t st);

// C[k] = gamma_k * (beta * D[k] + alpha * op(P[k], Q[k])),  op = P Q^T (nn=0) or P Q (nn=1)
struct GemmArgs {
  const void* p; const void* q; const void* d; void* c;
  int32_t m, n, kdim;
  int32_t ldp, ldq, ldc;           // D shares ldc
  int64_t stride_p, stride_q, stride_c;   // elements between consecutive matrices
  int32_t batch;
  const float* rnorm;  // device, per matrix
  int32_t gamma_mode;  // 0: 1, 1: r, 2: r*r
  float alpha, beta;
  int32_t nn;
  int32_t symmetric;   // op is P P^T with symmetric result (kernels may exploit it)
};
int launch_gemm_simt(const GemmArgs& a, int ns_precision, cudaStream_t st);
int launch_gemm_tc(muon_ctx* ctx, const GemmArgs& a, cudaStream_t st);   // tcgen05 engine (bf16 only)
bool tc_supported(const GemmArgs& a);
int launch_gemm_tc_pair(muon_ctx* ctx, const GemmArgs& a, cudaStream_t st);   // two-CTA (cta_group::2) variant
bool tc_pair_supported(const GemmArgs& a);
int launch_bounded_wait_probe(muon_ctx* ctx, cudaStream_t st);            // a wait that must expire (self-test)

}  // namespace muon
