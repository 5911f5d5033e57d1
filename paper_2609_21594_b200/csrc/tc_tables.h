// Problem tables of the grouped tensor-core engine and the host helpers that fill them.  Internal to the library.
#pragma once

#include <cuda.h>

#include "internal.h"

namespace muon {
namespace tc {

// One tile of the paired engine, in units of 128-row / 128-column blocks: CTA 0 of the pair computes row
// block ra, CTA 1 row block rb, both against column blocks cc (accumulator columns 0..127) and cd (128..255).
// kNoBlock in rb: CTA 1 has nothing to do; in cd: the tile is 128 columns wide (UMMA N = 128).
struct TilePat {
  uint16_t ra, rb, cc, cd;
};
constexpr uint16_t kNoBlock = 0xFFFFu;

// Tensor maps of one batched product of a grouped launch.  They are encoded once, when the plan is bound to a
// workspace, and stay in device memory (the TMA unit reads them from there).
struct alignas(128) TcMaps {
  CUtensorMap p;     // P: 128-row boxes
  CUtensorMap ph;    // P: 64 x 64 boxes (transposed reads of a half-stored symmetric P)
  CUtensorMap q;     // Q: 128-row boxes (nn = 0) or 64 k-rows x 64 columns (nn = 1)
  CUtensorMap qh;    // Q: 64 x 64 boxes (128-wide tiles; transposed reads of a half-stored symmetric Q)
  CUtensorMap d, c;  // aux matrix and result: 128 rows x 64 columns
};

// Everything else about the product travels by value with the launch (constant bank: decoding a tile costs no
// global-memory round trip on the MMA issuer's critical path).
struct TcProbInfo {
  const __nv_bfloat16* d;    // aux matrix (may be null)
  __nv_bfloat16* c;
  const float* rnorm;        // per matrix (gamma modes 1, 2)
  int64_t mat_begin;         // index of the problem's first matrix inside the launch set (row of per-matrix tables)
  const TilePat* pattern;    // explicit tile list per matrix (symmetric products); null: dense 2 x 2 block grid
  int64_t stride_c;
  int32_t m, n, kdim, ldc;
  int32_t batch, tiles_per_mat, tile_begin, row_pairs;
  int32_t symmetric, nn, rblocks, cblocks;
  // Half-stored symmetric matrices.  The Newton-Schulz products never need the whole of A or B in memory: a
  // symmetric result is written only where tiles compute it -- block (r, c) with (r >> 1) <= (c >> 1) in
  // 128-blocks -- and a consumer that needs block (r, k) below that line reads block (k, r) instead and feeds
  // it to the tensor core as an MN-major operand (the transpose costs nothing).
  int32_t mirror_out;        // 1: also write the transposed blocks (stand-alone symmetric product: full C)
  int32_t p_half, q_half;    // operand P / Q is such a half-stored symmetric matrix
  int32_t pad;
};
constexpr int kMaxProblems = kMaxElemChunks;

// The five product tables of a launch set in device memory, for the launch that runs a whole Newton-Schulz
// iteration by itself: [0], [1]: A = X X^T reading X iterate 0 / 1; [2]: P = aI + bA + cA A^T; [3], [4]: X' = P X
// reading iterate 0 / 1 and writing the other.
struct alignas(128) TcPersist {
  TcMaps maps[5][kMaxProblems];
  TcProbInfo info[5][kMaxProblems];
  int32_t nprob;
  int32_t total_tiles[5];
};
constexpr int kMaxPersistSteps = 16;

// By-value arguments of one grouped launch.
struct TcLaunch {
  TcMaps maps[kMaxProblems];
  TcProbInfo info[kMaxProblems];
  int32_t nprob, total_tiles;
  float alpha, beta;
  float diag;                // added to the diagonal of the result (the a_k I of P_k = a_k I + b_k A + c_k A^2)
  int32_t gamma_mode;        // 0: 1, 1: r, 2: r*r
  // Per-matrix coefficients: row (mat_begin + matrix) of coef_table, coef_stride floats per row, replaces the scalars:
  // alpha = row[coef_off + coef_a], beta = row[coef_off + coef_b], diag = row[coef_off + coef_d] (an index < 0 keeps the scalar).  A whole-iteration
  // launch derives the indices from the product it is in (coef_off = 3 * step when coef_per_step).
  const float* coef_table;   // device, first row of the launch set; null: scalars only
  int32_t coef_a, coef_b, coef_d, coef_off, coef_stride, coef_per_step;
  int32_t* status;
  // Whole-iteration mode (persist != null): the launch walks 3 * ns_steps products, a grid-wide barrier between
  // consecutive ones, and takes tables from device memory instead of maps / info above.
  const TcPersist* persist;
  int32_t ns_steps;
  uint32_t barrier_base;     // value of *barrier when the launch starts
  uint32_t* barrier;         // device counter: every CTA adds 1 per finished product
  float coef[kMaxPersistSteps][3];   // (a_k, b_k, c_k)
};

// Host view of one product launch of a launch set: the device maps plus the by-value problem records.
struct TcTable {
  TcMaps maps[kMaxProblems];
  TcProbInfo info[kMaxProblems];
  int32_t nprob = 0, total_tiles = 0;
};

// ------------------------------------------------------------------ host: tensor maps
typedef CUresult (*EncodeFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*, const cuuint64_t*,
                             const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                             CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

// 3-D map over a batch of row-major matrices: dims (cols, rows, batch), box (64, box_rows, 1), 128B swizzle.
inline bool encode_map(void* fn, CUtensorMap* map, const void* ptr, int cols, int rows, int batch, int ld, int64_t stride,
                int box_rows) {
  const cuuint64_t dims[3] = {cuuint64_t(cols), cuuint64_t(rows), cuuint64_t(batch)};
  const cuuint64_t strides[2] = {cuuint64_t(ld) * 2u, cuuint64_t(stride) * 2u};
  const cuuint32_t box[3] = {64u, cuuint32_t(box_rows), 1u};
  const cuuint32_t estr[3] = {1u, 1u, 1u};
  const CUresult r = reinterpret_cast<EncodeFn>(fn)(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void*>(ptr), dims,
                                                    strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
                                                    CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                                                    CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  return r == CUDA_SUCCESS;
}

}  // namespace tc

// Tables of one launch set (tensor-core engine): for each product the problem list, longest k first.
struct SetTables {
  tc::TcTable g1[2];   // A = X X^T, reading X iterate 0 / 1
  tc::TcTable g2;      // P = aI + bA + c A A^T
  tc::TcTable g3[2];   // X' = P X, reading iterate 0 / 1 and writing the other
  const tc::TcPersist* persist = nullptr;   // the same five tables in device memory (null: not built)
  int32_t max_tiles = 0;                    // largest tile count of a product
};

// Launches the paired engine on one product (tables by value).
int launch_tc_grouped(int device, const tc::TcLaunch& L, cudaStream_t st);
// Launches the paired engine on a whole Newton-Schulz iteration (L.persist set): a cooperative launch of `pairs`
// CTA pairs that must all be resident.  Returns 1, or < 0 when such a launch is not possible here.
int launch_tc_persistent(int device, const tc::TcLaunch& L, int pairs, cudaStream_t st);
// How many CTA pairs of the paired kernel can be resident at once on this device (0 when unknown).
int tc_pair_max_resident(int device);
// Number of SMs of the device (> 0), after making the paired kernel launchable there; < 0 on error.
int tc_pair_grid_setup(int device);

// Builds (or rebuilds, when the workspace moved) the tables of every launch set of `plan`:
// tensor maps over the workspace buffers (device memory), tile lists, per-product problem lists.
int bind_plan_tables(muon_ctx* ctx, Plan* plan);
void release_plan_tables(Plan* plan);

// Host image of the device part of the tables of ONE launch set (tile lists and tensor maps) laid out for device
// address `dev_base`; used by bind_plan_tables and by the allocation-free entry point, which places the image in
// its built-in scratch.
struct SetImage {
  std::vector<char> bytes;
  SetTables tables;       // device addresses inside refer to dev_base + offset
};
int build_set_image(void* encode_fn, const void* ws, const std::vector<Chunk>& chunks, const LaunchSet& set,
                    const void* dev_base, SetImage* out, int64_t* encodes, bool with_persist = true);

// Single stand-alone product (muon_ns_product): device image (maps and tile list) plus the by-value table.
int build_product_image(void* encode_fn, const GemmArgs& g, const void* dev_base, std::vector<char>* bytes, tc::TcTable* table,
                        int64_t* encodes);

}  // namespace muon
