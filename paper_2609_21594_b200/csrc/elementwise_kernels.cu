// Fused elementwise kernels around the Newton-Schulz engine.
//   stage : M <- mu*M + G, u = G + mu*M (Nesterov), U = cast(u) written into the NS workspace in
//           wide orientation (transposed through shared memory when rows > cols: the
//           transpose-first rule of Section 6.6), plus per-tile sums of U^2
//   norm  : r = 1 / (sqrt(sum U^2) + eps) per matrix, fixed-order reduction in double (Eq. 1, second line)
//   apply : W <- W (1 - lr*wd) - lr * 0.2 sqrt(max(m,n)) * O, O read back through the transpose
// All three are HBM-bound.  Reductions use a fixed shuffle/shared-memory tree and per-tile
// partial sums, never floating-point atomics, so results are bit-identical run to run.
#include <algorithm>
#include <cstring>

#include "internal.h"

namespace muon {

namespace {

constexpr int T = kElemTile;       // 64
constexpr int PADT = T + 2;        // shared tile row pitch (elements)

template <typename XT> struct XConv;
template <> struct XConv<__nv_bfloat16> {
  static __device__ __forceinline__ __nv_bfloat16 from(float v) { return __float2bfloat16_rn(v); }
  static __device__ __forceinline__ float to(__nv_bfloat16 v) { return __bfloat162float(v); }
};
template <> struct XConv<float> {
  static __device__ __forceinline__ float from(float v) { return v; }
  static __device__ __forceinline__ float to(float v) { return v; }
};

template <typename GT> __device__ __forceinline__ float load_g(const GT* p);
template <> __device__ __forceinline__ float load_g<__nv_bfloat16>(const __nv_bfloat16* p) { return __bfloat162float(*p); }
template <> __device__ __forceinline__ float load_g<float>(const float* p) { return *p; }

// Where the rows of a matrix live inside the buffers w/g/m/o point at.  Dense or strided matrices are one
// run of rows with pitch ld; in flat-shard mode a matrix is a few runs of whole rows (sorted by row, covering
// every row) with pitch cols.  A thread's four rows almost always fall into one run, so the cursor keeps the
// current run and only searches when a row leaves it.  The block first copies the matrix's run table into
// shared memory (one coalesced load instead of a chain of dependent global loads per thread); a table longer
// than kSegCache is searched in global memory.
constexpr int kSegCache = 32;

template <bool FLAT>
struct RowCursor {
  int row_begin, row_end;
  size_t base, pitch;
  const RowSeg* table;      // the matrix's runs: shared-memory copy or global table
  int count;
  // every thread of the block must call this (it contains a barrier in flat-shard mode)
  __device__ __forceinline__ void prepare(const MatDesc& d, const RowSeg* __restrict__ segs, RowSeg* cache) {
    if (!FLAT) return;
    count = d.seg_count;
    if (count <= kSegCache) {
      if (int(threadIdx.x) < count) cache[threadIdx.x] = segs[d.seg_begin + threadIdx.x];
      __syncthreads();
      table = cache;
    } else {
      table = segs + d.seg_begin;
    }
  }
  __device__ __forceinline__ void init(const MatDesc& d, int r) {
    if (!FLAT) {
      row_begin = 0; row_end = d.rows; base = 0; pitch = size_t(d.ld);
    } else {
      pitch = size_t(d.cols);
      seek(r);
    }
  }
  __device__ __forceinline__ void seek(int r) {
    row_begin = 0; row_end = 0; base = 0;
    for (int i = 0; i < count; ++i) {
      const RowSeg sg = table[i];
      if (r < sg.row_begin + sg.row_count) {
        row_begin = sg.row_begin; row_end = sg.row_begin + sg.row_count; base = size_t(sg.flat_offset);
        return;
      }
    }
  }
  // element offset of (r, 0); r must be a valid row of the matrix
  __device__ __forceinline__ size_t at(const MatDesc& d, int r) {
    if (!FLAT) return size_t(unsigned(r)) * unsigned(d.ld);
    if (r >= row_end) seek(r);
    return base + size_t(r - row_begin) * pitch;
  }
};

// Sums of squares are carried in double from the first addition on: a square of a bf16 or fp32 value is exact in
// double, and the accumulated rounding (about 1e-16 relative) is far below the final rounding of the reciprocal
// norm to fp32 -- so the norm a matrix gets does not depend on which kernel variant (or tiling) summed it.
__device__ __forceinline__ double block_sum_256(double v, double* red) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  const int w = threadIdx.x >> 5;
  if ((threadIdx.x & 31) == 0) red[w] = v;
  __syncthreads();
  double t = 0.0;
  if (threadIdx.x == 0) {
#pragma unroll
    for (int i = 0; i < 8; ++i) t += red[i];
  }
  return t;  // valid in thread 0
}

// Which shape group of the launch a block belongs to, and where inside it.
struct BlockPos {
  int ci, mat_local, tile;
};
template <typename Args>
__device__ __forceinline__ BlockPos locate_block(const Args& a) {
  int ci = 0;
  for (int i = 1; i < a.nchunks; ++i)
    if (int(blockIdx.x) >= a.ch[i].block_begin) ci = i;
  const int local = int(blockIdx.x) - a.ch[ci].block_begin;
  BlockPos p;
  p.ci = ci;
  p.mat_local = local / a.ch[ci].tiles;
  p.tile = local - p.mat_local * a.ch[ci].tiles;
  return p;
}

// Sum of squares of bf16 values, the same bits whichever kernel variant computes it.  A square of a bf16 value is exact in
// fp32; the squares of one aligned group of 8 consecutive source columns of a row are added in column order with one fp32
// fused multiply-add each (s = fma(q, q, s), starting from 0), and only the group sums are accumulated in double.  The
// 8-elements-per-thread kernels hold a group in one thread; here two neighbouring threads hold 4 columns each: the even
// one runs its half of the chain, hands the result to its neighbour, and the odd one finishes the chain and owns the sum.
// (Positions beyond the matrix hold 0, which leaves the chain unchanged.)
__device__ __forceinline__ double sum_of_squares_group(const float (&q)[4], int tx) {
  float s = 0.f;
#pragma unroll
  for (int i = 0; i < 4; ++i) s = __fmaf_rn(q[i], q[i], s);
  float t = __shfl_up_sync(0xffffffffu, s, 1);
  if ((tx & 1) == 0) return 0.0;
#pragma unroll
  for (int i = 0; i < 4; ++i) t = __fmaf_rn(q[i], q[i], t);
  return double(t);
}

// GT: gradient/input element type; XT: NS element type; MOM: momentum rule on/off.
// Thread (ty = tid/16, tx = tid%16) handles 4 consecutive columns tx*4.. of rows ty, ty+16, ty+32, ty+48.
template <typename GT, typename XT, bool MOM, bool FLAT>
__global__ void __launch_bounds__(256) stage_kernel(StageArgs a) {
  __shared__ XT tile[T][PADT];
  __shared__ double red[8];
  const BlockPos bp = locate_block(a);
  const ElemChunk ch = a.ch[bp.ci];
  const int t = bp.tile, ldx = ch.ldx;
  const MatDesc d = a.descs[ch.desc_begin + bp.mat_local];
  const int tiles_c = (d.cols + T - 1) / T;
  const int r0 = (t / tiles_c) * T, c0 = (t % tiles_c) * T;
  const GT* __restrict__ G = static_cast<const GT*>(d.g);
  float* __restrict__ M = static_cast<float*>(d.m);
  XT* __restrict__ X = reinterpret_cast<XT*>(a.ws + ch.x_off) + size_t(bp.mat_local) * ch.s * ldx;
  const int tx = threadIdx.x & 15, ty = threadIdx.x >> 4;
  // 16-byte (fp32) / 8-byte (bf16) accesses need columns, pitch and, in flat-shard mode, every segment offset in fours
  const bool vec = ((d.cols | int(d.ld)) & 3) == 0 && (!FLAT || a.flat_vec >= 4);
  double sum = 0.0;
  __shared__ RowSeg seg_cache[FLAT ? kSegCache : 1];
  RowCursor<FLAT> cur;
  cur.prepare(d, a.segs, seg_cache);
  cur.init(d, min(r0 + ty, d.rows - 1));
#pragma unroll
  for (int pass = 0; pass < 4; ++pass) {
    const int rr = ty + pass * 16, cc = tx * 4;
    const int r = r0 + rr, c = c0 + cc;
    float u[4] = {0.f, 0.f, 0.f, 0.f};
    float sq[4] = {0.f, 0.f, 0.f, 0.f};                   // this thread's rounded values of the row (0 where there is none)
    if (r < d.rows && c < d.cols) {
      const size_t off = cur.at(d, r) + c;
      float g[4], m[4] = {0.f, 0.f, 0.f, 0.f};
      const int nv = min(4, d.cols - c);
      if (vec) {
        if (sizeof(GT) == 2) {
          const uint2 raw = __ldcs(reinterpret_cast<const uint2*>(G + off));
          const __nv_bfloat162 p0 = *reinterpret_cast<const __nv_bfloat162*>(&raw.x);
          const __nv_bfloat162 p1 = *reinterpret_cast<const __nv_bfloat162*>(&raw.y);
          g[0] = __low2float(p0); g[1] = __high2float(p0); g[2] = __low2float(p1); g[3] = __high2float(p1);
        } else {
          const float4 raw = __ldcs(reinterpret_cast<const float4*>(G + off));
          g[0] = raw.x; g[1] = raw.y; g[2] = raw.z; g[3] = raw.w;
        }
        if (MOM) {
          const float4 mv = __ldcs(reinterpret_cast<const float4*>(M + off));
          m[0] = mv.x; m[1] = mv.y; m[2] = mv.z; m[3] = mv.w;
        }
      } else {
        for (int i = 0; i < 4; ++i) {
          g[i] = i < nv ? load_g<GT>(G + off + i) : 0.f;
          if (MOM) m[i] = i < nv ? M[off + i] : 0.f;
        }
      }
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        if (MOM) {
          m[i] = __fmaf_rn(a.mu, m[i], g[i]);             // explicit roundings: every route to M' and u computes the same bits
          u[i] = a.nesterov ? __fmaf_rn(a.mu, m[i], g[i]) : m[i];
        } else {
          u[i] = g[i];
        }
      }
      if (MOM) {
        if (vec) {
          __stcs(reinterpret_cast<float4*>(M + off), make_float4(m[0], m[1], m[2], m[3]));
        } else {
          for (int i = 0; i < nv; ++i) M[off + i] = m[i];
        }
      }
      alignas(16) XT xv[4];
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        xv[i] = XConv<XT>::from(u[i]);
        const float qf = XConv<XT>::to(xv[i]);
        if (sizeof(XT) == 2) {
          if (i < nv) sq[i] = qf;                         // summed below, by the group-of-8 rule
        } else {
          const double q = double(qf);
          if (i < nv) sum += q * q;
        }
      }
      if (!d.transposed) {
        XT* dst = X + size_t(r) * ldx + c;     // ldx % 8 == 0 and c % 4 == 0: 8/16-byte aligned
        if (nv == 4) {
          if (sizeof(XT) == 2) *reinterpret_cast<uint2*>(dst) = *reinterpret_cast<const uint2*>(xv);
          else *reinterpret_cast<float4*>(dst) = *reinterpret_cast<const float4*>(xv);
        } else {
          for (int i = 0; i < nv; ++i) dst[i] = xv[i];
        }
      } else {
#pragma unroll
        for (int i = 0; i < 4; ++i) tile[rr][cc + i] = xv[i];
      }
    }
    if (sizeof(XT) == 2) sum += sum_of_squares_group(sq, tx);   // every lane takes part (shuffle inside)
  }
  if (d.transposed) {
    __syncthreads();
    // X holds the transpose: X[c][r].  Thread writes 4 consecutive r for one c.
#pragma unroll
    for (int pass = 0; pass < 4; ++pass) {
      const int cc = ty + pass * 16, rr = tx * 4;
      const int c = c0 + cc, r = r0 + rr;
      if (c < d.cols && r < d.rows) {
        alignas(16) XT xv[4];
#pragma unroll
        for (int i = 0; i < 4; ++i) xv[i] = tile[rr + i][cc];
        XT* dst = X + size_t(c) * ldx + r;
        const int nv = min(4, d.rows - r);
        if (nv == 4) {
          if (sizeof(XT) == 2) *reinterpret_cast<uint2*>(dst) = *reinterpret_cast<const uint2*>(xv);
          else *reinterpret_cast<float4*>(dst) = *reinterpret_cast<const float4*>(xv);
        } else {
          for (int i = 0; i < nv; ++i) dst[i] = xv[i];
        }
      }
    }
  }
  const double tot = block_sum_256(sum, red);
  if (threadIdx.x == 0) a.partials[ch.part_off + int64_t(bp.mat_local) * ch.tiles + t] = tot;
}

// One block per matrix of the launch: fixed-order sum of the tile partials in double, then r = 1/(sqrt(.)+eps).
__global__ void __launch_bounds__(256) norm_kernel(StageArgs a) {
  __shared__ double red[256];
  int ci = 0, first = 0;
  for (int i = 0; i < a.nchunks; ++i) {
    if (int(blockIdx.x) >= first + a.ch[i].count) first += a.ch[i].count;
    else { ci = i; break; }
  }
  const ElemChunk ch = a.ch[ci];
  const int mat_local = int(blockIdx.x) - first;
  const double* p = a.partials + ch.part_off + int64_t(mat_local) * ch.tiles;
  double acc = 0.0;
  for (int i = threadIdx.x; i < ch.tiles; i += 256) acc += p[i];
  red[threadIdx.x] = acc;
  __syncthreads();
  for (int o = 128; o > 0; o >>= 1) {
    if (int(threadIdx.x) < o) red[threadIdx.x] += red[threadIdx.x + o];
    __syncthreads();
  }
  if (threadIdx.x == 0)
    a.rnorm[ch.desc_begin + mat_local] = a.normalize ? float(1.0 / (sqrt(red[0]) + double(a.eps))) : 1.0f;
}

// XT: NS element type; UPD: 1 = weight update, 0 = plain store of O into d.w (element type XT).
// The weights of all four passes are requested first, then the O tile (through shared memory when it has
// to be transposed back), then the arithmetic and the stores.
template <typename XT, bool UPD, bool FLAT>
__global__ void __launch_bounds__(256, FLAT ? 5 : 6) apply_kernel(ApplyArgs a) {
  __shared__ XT tile[T][PADT];
  const BlockPos bp = locate_block(a);
  const ElemChunk ch = a.ch[bp.ci];
  const int t = bp.tile, ldx = ch.ldx;
  const MatDesc d = a.descs[ch.desc_begin + bp.mat_local];
  const int tiles_c = (d.cols + T - 1) / T;
  const int r0 = (t / tiles_c) * T, c0 = (t % tiles_c) * T;
  const XT* __restrict__ X = reinterpret_cast<const XT*>(a.ws + ch.x_off) + size_t(bp.mat_local) * ch.s * ldx;
  float* __restrict__ W = static_cast<float*>(d.w);
  const int tx = threadIdx.x & 15, ty = threadIdx.x >> 4;
  const bool vec = ((d.cols | int(d.ld)) & 3) == 0 && (!FLAT || a.flat_vec >= 4);
  const int cc = tx * 4, c = c0 + cc;
  const int nv = min(4, d.cols - c);
  float w[4][4];
  alignas(16) XT xv[4][4];
  size_t offs[FLAT ? 4 : 1];
  __shared__ RowSeg seg_cache[FLAT ? kSegCache : 1];
  if (FLAT) {
    RowCursor<true> cur;
    cur.prepare(d, a.segs, seg_cache);
    cur.init(d, min(r0 + ty, d.rows - 1));
#pragma unroll
    for (int pass = 0; pass < 4; ++pass) {
      const int r = r0 + ty + pass * 16;
      offs[FLAT ? pass : 0] = r < d.rows ? cur.at(d, r) + c : 0;
    }
  }
  // ---- loads: W (update mode), then O
  if (UPD) {
#pragma unroll
    for (int pass = 0; pass < 4; ++pass) {
      const int r = r0 + ty + pass * 16;
#pragma unroll
      for (int i = 0; i < 4; ++i) w[pass][i] = 0.f;
      if (r < d.rows && nv > 0) {
        const size_t off = FLAT ? offs[FLAT ? pass : 0] : size_t(unsigned(r)) * unsigned(d.ld) + unsigned(c);
        if (vec) {
          const float4 wv = __ldcs(reinterpret_cast<const float4*>(W + off));
          w[pass][0] = wv.x; w[pass][1] = wv.y; w[pass][2] = wv.z; w[pass][3] = wv.w;
        } else {
          for (int i = 0; i < nv; ++i) w[pass][i] = W[off + i];
        }
      }
    }
  }
  if (d.transposed) {
    // load X[c][r] coalesced along r, then read it back transposed
#pragma unroll
    for (int pass = 0; pass < 4; ++pass) {
      const int cc2 = ty + pass * 16, rr = tx * 4;
      const int c2 = c0 + cc2, r = r0 + rr;
      if (c2 < d.cols && r < d.rows) {
        const XT* src = X + size_t(c2) * ldx + r;
        const int nr = min(4, d.rows - r);
        alignas(16) XT tv[4];
        if (nr == 4) {
          if (sizeof(XT) == 2) *reinterpret_cast<uint2*>(tv) = __ldcs(reinterpret_cast<const uint2*>(src));
          else *reinterpret_cast<float4*>(tv) = __ldcs(reinterpret_cast<const float4*>(src));
        } else {
          for (int i = 0; i < 4; ++i) tv[i] = i < nr ? src[i] : XConv<XT>::from(0.f);
        }
#pragma unroll
        for (int i = 0; i < 4; ++i) tile[rr + i][cc2] = tv[i];
      }
    }
    __syncthreads();
#pragma unroll
    for (int pass = 0; pass < 4; ++pass) {
      const int rr = ty + pass * 16;
#pragma unroll
      for (int i = 0; i < 4; ++i) xv[pass][i] = tile[rr][cc + i];
    }
  } else {
#pragma unroll
    for (int pass = 0; pass < 4; ++pass) {
      const int r = r0 + ty + pass * 16;
#pragma unroll
      for (int i = 0; i < 4; ++i) xv[pass][i] = XConv<XT>::from(0.f);
      if (r < d.rows && nv > 0) {
        const XT* src = X + size_t(r) * ldx + c;
        if (nv == 4) {
          if (sizeof(XT) == 2) *reinterpret_cast<uint2*>(xv[pass]) = __ldcs(reinterpret_cast<const uint2*>(src));
          else *reinterpret_cast<float4*>(xv[pass]) = __ldcs(reinterpret_cast<const float4*>(src));
        } else {
          for (int i = 0; i < nv; ++i) xv[pass][i] = src[i];
        }
      }
    }
  }
  // ---- arithmetic and stores
  const float decay = a.decay;
  const float step = a.lr * d.scale;
#pragma unroll
  for (int pass = 0; pass < 4; ++pass) {
    const int r = r0 + ty + pass * 16;
    if (r < d.rows && nv > 0) {
      const size_t off = FLAT ? offs[FLAT ? pass : 0] : size_t(unsigned(r)) * unsigned(d.ld) + unsigned(c);
      if (UPD) {
        // two explicit roundings (product, then fused multiply-add): the result does not depend on how the
        // compiler contracts the expression
        float4 o;
        o.x = __fmaf_rn(-step, XConv<XT>::to(xv[pass][0]), __fmul_rn(w[pass][0], decay));
        o.y = __fmaf_rn(-step, XConv<XT>::to(xv[pass][1]), __fmul_rn(w[pass][1], decay));
        o.z = __fmaf_rn(-step, XConv<XT>::to(xv[pass][2]), __fmul_rn(w[pass][2], decay));
        o.w = __fmaf_rn(-step, XConv<XT>::to(xv[pass][3]), __fmul_rn(w[pass][3], decay));
        if (vec) {
          __stcs(reinterpret_cast<float4*>(W + off), o);
        } else {
          const float ov[4] = {o.x, o.y, o.z, o.w};
          for (int i = 0; i < nv; ++i) W[off + i] = ov[i];
        }
        if (d.o) {   // the update itself, for the pack that follows (relay broadcast payload)
          XT* O = static_cast<XT*>(d.o);
          if (vec) {
            if (sizeof(XT) == 2) __stcs(reinterpret_cast<uint2*>(O + off), *reinterpret_cast<const uint2*>(xv[pass]));
            else __stcs(reinterpret_cast<float4*>(O + off), *reinterpret_cast<const float4*>(xv[pass]));
          } else {
            for (int i = 0; i < nv; ++i) O[off + i] = xv[pass][i];
          }
        }
      } else {
        XT* O = static_cast<XT*>(d.w);
        if (vec) {
          if (sizeof(XT) == 2) *reinterpret_cast<uint2*>(O + off) = *reinterpret_cast<const uint2*>(xv[pass]);
          else *reinterpret_cast<float4*>(O + off) = *reinterpret_cast<const float4*>(xv[pass]);
        } else {
          for (int i = 0; i < nv; ++i) O[off + i] = xv[pass][i];
        }
      }
    }
  }
}


// ---------------------------------------------------------------------------------------------------------------
// "Wide" variants for matrices whose rows, cols and row pitches are all multiples of 8: 64 x 128 tiles, every
// thread moves 8 consecutive elements per access (16-byte bf16 / 2 x 16-byte fp32 vectors), so the instruction
// count per byte is about a third of the generic kernels' -- which is what keeps these HBM-bound kernels at
// bandwidth when the SM clock sits low under the power cap of a Newton-Schulz-heavy step.
// Transposition goes through a 128 x 64 bf16 shared tile T[c][r] (128 bytes per c-row, no padding) whose
// 16-byte chunks are XOR-swizzled with bits 3..5 of c: the element-wise side (one c-row per thread column)
// then spreads over 8 bank groups, the vector side reads/writes whole 16-byte chunks without conflicts.
// ---------------------------------------------------------------------------------------------------------------
constexpr int WR = 64, WC = 128;

__device__ __forceinline__ uint32_t wide_tile_addr(int c_local, int r_local) {   // byte offset of T[c][r]
  return uint32_t(c_local) * 128u + (uint32_t((r_local >> 3) ^ ((c_local >> 3) & 7)) << 4) + uint32_t(r_local & 7) * 2u;
}

__host__ __device__ inline int wide_tiles(int rows, int cols) { return ((rows + WR - 1) / WR) * ((cols + WC - 1) / WC); }

template <typename GT, bool MOM, bool FLAT>
__global__ void __launch_bounds__(256, 6) stage_wide_kernel(StageArgs a) {
  __shared__ __align__(16) unsigned char tsm[WC * 128];
  __shared__ double red[8];
  const BlockPos bp = locate_block(a);
  const ElemChunk ch = a.ch[bp.ci];
  const int t = bp.tile, ldx = ch.ldx;
  const MatDesc d = a.descs[ch.desc_begin + bp.mat_local];
  const int tiles_c = (d.cols + WC - 1) / WC;
  double sum = 0.0;
  if (t < wide_tiles(d.rows, d.cols)) {                      // block-uniform: the grid is sized for the larger orientation
    const int r0 = (t / tiles_c) * WR, c0 = (t % tiles_c) * WC;
    const GT* __restrict__ G = static_cast<const GT*>(d.g);
    float* __restrict__ M = static_cast<float*>(d.m);
    __nv_bfloat16* __restrict__ X = reinterpret_cast<__nv_bfloat16*>(a.ws + ch.x_off) + size_t(bp.mat_local) * ch.s * ldx;
    const int tx = threadIdx.x & 15, ty = threadIdx.x >> 4;
    const int c = c0 + 8 * tx;
    __shared__ RowSeg seg_cache[FLAT ? kSegCache : 1];
    RowCursor<FLAT> cur;
    cur.prepare(d, a.segs, seg_cache);
    cur.init(d, min(r0 + ty, d.rows - 1));
    if (c < d.cols) {
#pragma unroll
      for (int pass = 0; pass < 4; ++pass) {
        const int rl = ty + pass * 16, r = r0 + rl;
        if (r < d.rows) {
          const size_t off = cur.at(d, r) + size_t(c);
          float g[8], m[8];
          if (sizeof(GT) == 2) {
            const uint4 raw = __ldcs(reinterpret_cast<const uint4*>(G + off));
            const uint32_t w[4] = {raw.x, raw.y, raw.z, raw.w};
#pragma unroll
            for (int i = 0; i < 4; ++i) {
              g[2 * i] = __uint_as_float(w[i] << 16);
              g[2 * i + 1] = __uint_as_float(w[i] & 0xffff0000u);
            }
          } else {
            const float4 g0 = __ldcs(reinterpret_cast<const float4*>(G + off));
            const float4 g1 = __ldcs(reinterpret_cast<const float4*>(G + off) + 1);
            g[0] = g0.x; g[1] = g0.y; g[2] = g0.z; g[3] = g0.w; g[4] = g1.x; g[5] = g1.y; g[6] = g1.z; g[7] = g1.w;
          }
          if (MOM) {
            const float4 m0 = __ldcs(reinterpret_cast<const float4*>(M + off));
            const float4 m1 = __ldcs(reinterpret_cast<const float4*>(M + off) + 1);
            m[0] = m0.x; m[1] = m0.y; m[2] = m0.z; m[3] = m0.w; m[4] = m1.x; m[5] = m1.y; m[6] = m1.z; m[7] = m1.w;
#pragma unroll
            for (int i = 0; i < 8; ++i) {
              m[i] = __fmaf_rn(a.mu, m[i], g[i]);                 // explicit roundings, as in every other route to M' and u
              g[i] = a.nesterov ? __fmaf_rn(a.mu, m[i], g[i]) : m[i];   // g now holds u
            }
            __stcs(reinterpret_cast<float4*>(M + off), make_float4(m[0], m[1], m[2], m[3]));
            __stcs(reinterpret_cast<float4*>(M + off) + 1, make_float4(m[4], m[5], m[6], m[7]));
          }
          uint32_t pk[4];
          float grp = 0.f;
#pragma unroll
          for (int i = 0; i < 4; ++i) {
            const __nv_bfloat162 b = __floats2bfloat162_rn(g[2 * i], g[2 * i + 1]);
            pk[i] = *reinterpret_cast<const uint32_t*>(&b);
            const float q0 = __uint_as_float(pk[i] << 16), q1 = __uint_as_float(pk[i] & 0xffff0000u);
            grp = __fmaf_rn(q0, q0, grp);                          // the group-of-8 rule: see sum_of_squares_group
            grp = __fmaf_rn(q1, q1, grp);
          }
          sum += double(grp);
          if (!d.transposed) {
            *reinterpret_cast<uint4*>(X + size_t(r) * ldx + c) = make_uint4(pk[0], pk[1], pk[2], pk[3]);
          } else {
#pragma unroll
            for (int i = 0; i < 8; ++i) {
              const uint16_t h = uint16_t(i & 1 ? pk[i >> 1] >> 16 : pk[i >> 1] & 0xffffu);
              *reinterpret_cast<uint16_t*>(tsm + wide_tile_addr(8 * tx + i, rl)) = h;
            }
          }
        }
      }
    }
    if (d.transposed) {
      __syncthreads();
#pragma unroll
      for (int pass = 0; pass < 4; ++pass) {                 // X[c][r0 + 8*og .. +7]: one 16-byte chunk per thread
        const int oc = (threadIdx.x >> 3) + 32 * pass, og = threadIdx.x & 7;
        const int cc = c0 + oc, r = r0 + 8 * og;
        if (cc < d.cols && r < d.rows)
          *reinterpret_cast<uint4*>(X + size_t(cc) * ldx + r) = *reinterpret_cast<const uint4*>(tsm + wide_tile_addr(oc, 8 * og));
      }
    }
  }
  const double tot = block_sum_256(sum, red);
  if (threadIdx.x == 0) a.partials[ch.part_off + int64_t(bp.mat_local) * ch.tiles + t] = tot;
}

template <bool UPD, bool FLAT>
__global__ void __launch_bounds__(256, 6) apply_wide_kernel(ApplyArgs a) {
  __shared__ __align__(16) unsigned char tsm[WC * 128];
  const BlockPos bp = locate_block(a);
  const ElemChunk ch = a.ch[bp.ci];
  const int t = bp.tile, ldx = ch.ldx;
  const MatDesc d = a.descs[ch.desc_begin + bp.mat_local];
  if (t >= wide_tiles(d.rows, d.cols)) return;               // block-uniform
  const int tiles_c = (d.cols + WC - 1) / WC;
  const int r0 = (t / tiles_c) * WR, c0 = (t % tiles_c) * WC;
  const __nv_bfloat16* __restrict__ X = reinterpret_cast<const __nv_bfloat16*>(a.ws + ch.x_off) + size_t(bp.mat_local) * ch.s * ldx;
  const int tx = threadIdx.x & 15, ty = threadIdx.x >> 4;
  const int c = c0 + 8 * tx;
  const bool col_ok = c < d.cols;
  size_t offs[4];
  __shared__ RowSeg seg_cache[FLAT ? kSegCache : 1];
  {
    RowCursor<FLAT> cur;
    cur.prepare(d, a.segs, seg_cache);
    cur.init(d, min(r0 + ty, d.rows - 1));
#pragma unroll
    for (int pass = 0; pass < 4; ++pass) {
      const int r = r0 + ty + pass * 16;
      offs[pass] = r < d.rows ? cur.at(d, r) + size_t(c) : 0;
    }
  }
  if (d.transposed) {
#pragma unroll
    for (int pass = 0; pass < 4; ++pass) {                   // X[c][r0 + 8*og .. +7] -> T[c][.]
      const int oc = (threadIdx.x >> 3) + 32 * pass, og = threadIdx.x & 7;
      const int cc = c0 + oc, r = r0 + 8 * og;
      if (cc < d.cols && r < d.rows)
        *reinterpret_cast<uint4*>(tsm + wide_tile_addr(oc, 8 * og)) = __ldcs(reinterpret_cast<const uint4*>(X + size_t(cc) * ldx + r));
    }
    __syncthreads();
  }
  const float decay = a.decay;
  const float step = a.lr * d.scale;
#pragma unroll
  for (int pass = 0; pass < 4; ++pass) {
    const int rl = ty + pass * 16, r = r0 + rl;
    if (!col_ok || r >= d.rows) continue;
    uint32_t pk[4];
    if (!d.transposed) {
      const uint4 v = __ldcs(reinterpret_cast<const uint4*>(X + size_t(r) * ldx + c));
      pk[0] = v.x; pk[1] = v.y; pk[2] = v.z; pk[3] = v.w;
    } else {
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        const uint32_t lo = *reinterpret_cast<const uint16_t*>(tsm + wide_tile_addr(8 * tx + 2 * i, rl));
        const uint32_t hi = *reinterpret_cast<const uint16_t*>(tsm + wide_tile_addr(8 * tx + 2 * i + 1, rl));
        pk[i] = lo | (hi << 16);
      }
    }
    const size_t off = offs[pass];
    if (UPD) {
      float4 w[1][2];
      {
        const float* __restrict__ Wr = static_cast<const float*>(d.w);
        w[0][0] = __ldcs(reinterpret_cast<const float4*>(Wr + off));
        w[0][1] = __ldcs(reinterpret_cast<const float4*>(Wr + off) + 1);
      }
      float o[8];
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        o[2 * i] = __uint_as_float(pk[i] << 16);
        o[2 * i + 1] = __uint_as_float(pk[i] & 0xffff0000u);
      }
      float* W = static_cast<float*>(d.w);
      float4 n0, n1;
      n0.x = __fmaf_rn(-step, o[0], __fmul_rn(w[0][0].x, decay));
      n0.y = __fmaf_rn(-step, o[1], __fmul_rn(w[0][0].y, decay));
      n0.z = __fmaf_rn(-step, o[2], __fmul_rn(w[0][0].z, decay));
      n0.w = __fmaf_rn(-step, o[3], __fmul_rn(w[0][0].w, decay));
      n1.x = __fmaf_rn(-step, o[4], __fmul_rn(w[0][1].x, decay));
      n1.y = __fmaf_rn(-step, o[5], __fmul_rn(w[0][1].y, decay));
      n1.z = __fmaf_rn(-step, o[6], __fmul_rn(w[0][1].z, decay));
      n1.w = __fmaf_rn(-step, o[7], __fmul_rn(w[0][1].w, decay));
      __stcs(reinterpret_cast<float4*>(W + off), n0);
      __stcs(reinterpret_cast<float4*>(W + off) + 1, n1);
      if (d.o) __stcs(reinterpret_cast<uint4*>(static_cast<__nv_bfloat16*>(d.o) + off), make_uint4(pk[0], pk[1], pk[2], pk[3]));
    } else {
      *reinterpret_cast<uint4*>(static_cast<__nv_bfloat16*>(d.w) + off) = make_uint4(pk[0], pk[1], pk[2], pk[3]);
    }
  }
}

}  // namespace

template <bool FLAT>
static void launch_stage_t(const StageArgs& a, unsigned g, cudaStream_t st) {
  const bool xbf = a.ns_precision == MUON_NS_BF16;
  if (a.momentum) {
    const bool gbf = a.grad_dtype == MUON_DTYPE_BF16;
    if (gbf && xbf) stage_kernel<__nv_bfloat16, __nv_bfloat16, true, FLAT><<<g, 256, 0, st>>>(a);
    else if (gbf && !xbf) stage_kernel<__nv_bfloat16, float, true, FLAT><<<g, 256, 0, st>>>(a);
    else if (!gbf && xbf) stage_kernel<float, __nv_bfloat16, true, FLAT><<<g, 256, 0, st>>>(a);
    else stage_kernel<float, float, true, FLAT><<<g, 256, 0, st>>>(a);
  } else {
    if (xbf) stage_kernel<__nv_bfloat16, __nv_bfloat16, false, FLAT><<<g, 256, 0, st>>>(a);
    else stage_kernel<float, float, false, FLAT><<<g, 256, 0, st>>>(a);
  }
}

template <bool FLAT>
static void launch_stage_wide_t(const StageArgs& a, unsigned g, cudaStream_t st) {
  if (a.momentum) {
    if (a.grad_dtype == MUON_DTYPE_BF16) stage_wide_kernel<__nv_bfloat16, true, FLAT><<<g, 256, 0, st>>>(a);
    else stage_wide_kernel<float, true, FLAT><<<g, 256, 0, st>>>(a);
  } else {
    stage_wide_kernel<__nv_bfloat16, false, FLAT><<<g, 256, 0, st>>>(a);
  }
}

// Tiles per matrix of the wide kernels: a chunk mixes both orientations of its core shape, the grid takes the larger count.
static int wide_tiles_of_chunk(int s, int l) { return std::max(wide_tiles(s, l), wide_tiles(l, s)); }

// Fills block_begin / tiles of every shape group of the launch; returns the grid size or < 0.
template <typename Args>
static int64_t finish_chunks(Args* a, bool wide) {
  int64_t blocks = 0;
  int matrices = 0;
  for (int i = 0; i < a->nchunks; ++i) {
    ElemChunk& c = a->ch[i];
    c.tiles = wide ? wide_tiles_of_chunk(c.s, c.l) : ((c.s + T - 1) / T) * ((c.l + T - 1) / T);
    if (blocks > 0x7fffffffLL) return -1;
    c.block_begin = int32_t(blocks);
    blocks += int64_t(c.count) * c.tiles;
    matrices += c.count;
  }
  return blocks > 0x7fffffffLL ? -1 : blocks;
}

int launch_stage(const StageArgs& a0, cudaStream_t st) {
  StageArgs a = a0;
  if (a.nchunks < 1 || a.nchunks > kMaxElemChunks) return MUON_ERR_INVALID_ARG;
  const bool wide = a.wide && a.ns_precision == MUON_NS_BF16 && (!a.segs || a.flat_vec >= 8);
  const int64_t blocks = finish_chunks(&a, wide);
  if (blocks < 0) return MUON_ERR_UNSUPPORTED;
  if (blocks == 0) return 0;
  if (wide) {
    if (a.segs) launch_stage_wide_t<true>(a, unsigned(blocks), st);
    else launch_stage_wide_t<false>(a, unsigned(blocks), st);
  } else {
    if (a.segs) launch_stage_t<true>(a, unsigned(blocks), st);
    else launch_stage_t<false>(a, unsigned(blocks), st);
  }
  if (cudaGetLastError() != cudaSuccess) return MUON_ERR_CUDA;
  int matrices = 0;
  for (int i = 0; i < a.nchunks; ++i) matrices += a.ch[i].count;
  norm_kernel<<<unsigned(matrices), 256, 0, st>>>(a);
  return cudaGetLastError() == cudaSuccess ? 2 : MUON_ERR_CUDA;
}

template <bool FLAT>
static void launch_apply_t(const ApplyArgs& a, unsigned g, cudaStream_t st) {
  const bool xbf = a.ns_precision == MUON_NS_BF16;
  if (a.update) {
    if (xbf) apply_kernel<__nv_bfloat16, true, FLAT><<<g, 256, 0, st>>>(a);
    else apply_kernel<float, true, FLAT><<<g, 256, 0, st>>>(a);
  } else {
    if (xbf) apply_kernel<__nv_bfloat16, false, FLAT><<<g, 256, 0, st>>>(a);
    else apply_kernel<float, false, FLAT><<<g, 256, 0, st>>>(a);
  }
}

int launch_apply(const ApplyArgs& a0, cudaStream_t st) {
  ApplyArgs a = a0;
  if (a.nchunks < 1 || a.nchunks > kMaxElemChunks) return MUON_ERR_INVALID_ARG;
  const bool wide = a.wide && a.ns_precision == MUON_NS_BF16 && (!a.segs || a.flat_vec >= 8);
  const int64_t blocks = finish_chunks(&a, wide);
  if (blocks < 0) return MUON_ERR_UNSUPPORTED;
  if (blocks == 0) return 0;
  const unsigned g = unsigned(blocks);
  if (wide) {
    if (a.update) {
      if (a.segs) apply_wide_kernel<true, true><<<g, 256, 0, st>>>(a);
      else apply_wide_kernel<true, false><<<g, 256, 0, st>>>(a);
    } else {
      if (a.segs) apply_wide_kernel<false, true><<<g, 256, 0, st>>>(a);
      else apply_wide_kernel<false, false><<<g, 256, 0, st>>>(a);
    }
  } else {
    if (a.segs) launch_apply_t<true>(a, g, st);
    else launch_apply_t<false>(a, g, st);
  }
  return cudaGetLastError() == cudaSuccess ? 1 : MUON_ERR_CUDA;
}

// ---- poke: small host data -> device memory, carried by the kernel's argument buffer
struct PokeBlob {
  uint4 v[192];      // 3 KiB
};
__global__ void __launch_bounds__(192) poke_kernel(uint4* dst, const PokeBlob b, int n16) {
  if (int(threadIdx.x) < n16) dst[threadIdx.x] = b.v[threadIdx.x];
}

int launch_poke(void* dst, const void* src, size_t bytes, cudaStream_t st) {
  if (bytes == 0) return 0;
  if (bytes > sizeof(PokeBlob) || (reinterpret_cast<uintptr_t>(dst) & 15u)) return MUON_ERR_INVALID_ARG;
  PokeBlob b;
  std::memset(&b, 0, sizeof(b));
  std::memcpy(&b, src, bytes);
  poke_kernel<<<1, 192, 0, st>>>(static_cast<uint4*>(dst), b, int((bytes + 15) / 16));
  return cudaGetLastError() == cudaSuccess ? 1 : MUON_ERR_CUDA;
}

}  // namespace muon
