// Shared pieces of the tensor-core Newton-Schulz kernels: argument block, PTX wrappers for
// mbarrier / TMA / tcgen05, shared-memory and instruction descriptors.  Internal to the library.
#pragma once

#include <cuda.h>

#include "internal.h"

namespace muon {
namespace tc {

constexpr long long WAIT_CYCLES = 4000000000LL;   // ~2 s at 1.9 GHz: far beyond any legitimate wait

struct TcArgs {
  const __nv_bfloat16* d;   // aux matrix (may be null)
  __nv_bfloat16* c;
  int32_t m, n, kdim, ldc;
  int64_t stride_c;
  int32_t batch, tiles_m, tiles_n;
  int32_t tiles_per_mat;    // tiles_m*tiles_n, or the number of tiles on/above the diagonal when symmetric
  int32_t symmetric;        // C = C^T: compute tiles that touch the upper triangle, mirror the strictly upper ones
  const float* rnorm;
  int32_t gamma_mode;
  float alpha, beta;
  int32_t* status;
};

// ------------------------------------------------------------------ PTX wrappers
__device__ __forceinline__ uint32_t smem_u32(const void* p) { return uint32_t(__cvta_generic_to_shared(p)); }

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count));
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ bool mbar_try(uint32_t bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(ok)
      : "r"(bar), "r"(parity)
      : "memory");
  return ok != 0;
}
// Bounded wait.  Returns false when the deadline passed or (honor_abort) another role gave up;
// the caller must then abandon the pipeline.
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile int* abort_flag,
                                          bool honor_abort = true, long long limit = WAIT_CYCLES) {
  if (mbar_try(bar, parity)) return true;
  const long long t0 = clock64();
  uint32_t spins = 0;
  while (!mbar_try(bar, parity)) {
    if ((++spins & 255u) == 0) {
      if (honor_abort && *abort_flag) return false;
      if (clock64() - t0 > limit) return false;
    }
  }
  return true;
}

__device__ __forceinline__ void tma_load_3d(uint32_t dst, const CUtensorMap* map, uint32_t bar, int c0, int c1, int c2) {
  asm volatile(
      "cp.async.bulk.tensor.3d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5}], [%2];"
      ::"r"(dst), "l"(map), "r"(bar), "r"(c0), "r"(c1), "r"(c2)
      : "memory");
}

__device__ __forceinline__ void tma_store_3d(const CUtensorMap* map, uint32_t src, int c0, int c1, int c2) {
  asm volatile("cp.async.bulk.tensor.3d.global.shared::cta.bulk_group [%0, {%2, %3, %4}], [%1];"
               ::"l"(map), "r"(src), "r"(c0), "r"(c1), "r"(c2)
               : "memory");
}
__device__ __forceinline__ void tma_commit() { asm volatile("cp.async.bulk.commit_group;" ::: "memory"); }
template <int N> __device__ __forceinline__ void tma_wait_read() {
  asm volatile("cp.async.bulk.wait_group.read %0;" ::"n"(N) : "memory");
}
__device__ __forceinline__ void tma_wait_all() { asm volatile("cp.async.bulk.wait_group 0;" ::: "memory"); }
__device__ __forceinline__ void fence_async_smem() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }

__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }

__device__ __forceinline__ void tc_commit(uint32_t bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}

__device__ __forceinline__ void tc_mma(uint32_t d_tmem, uint64_t adesc, uint64_t bdesc, uint32_t idesc, uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
      ::"r"(d_tmem), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate)
      : "memory");
}

__device__ __forceinline__ void tc_ld32(uint32_t taddr, uint32_t (&r)[32]) {
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
__device__ __forceinline__ void tc_wait_ld() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }

// Shared-memory matrix descriptor, 128-byte swizzle (layout type 2), descriptor version 1.
// lbo/sbo in bytes.  K-major: lbo is unused by the hardware for swizzled layouts (set to 16),
// sbo = distance between 8-row groups.  MN-major: lbo = distance between 64-element column
// chunks, sbo = distance between groups of 8 k-rows.
__device__ __forceinline__ uint64_t make_desc(uint32_t saddr, uint32_t lbo, uint32_t sbo) {
  uint64_t d = 0;
  d |= uint64_t((saddr & 0x3FFFFu) >> 4);
  d |= uint64_t((lbo >> 4) & 0x3FFFu) << 16;
  d |= uint64_t((sbo >> 4) & 0x3FFFu) << 32;
  d |= uint64_t(1) << 46;
  d |= uint64_t(2) << 61;
  return d;
}

// Instruction descriptor for kind::f16: fp32 accumulator, bf16 A and B, A K-major, B K- or MN-major.
__host__ __device__ constexpr uint32_t make_idesc(bool b_mn_major, int umma_m, int umma_n) {
  return (1u << 4) | (1u << 7) | (1u << 10) | (uint32_t(b_mn_major ? 1 : 0) << 16) | (uint32_t(umma_n >> 3) << 17) |
         (uint32_t(umma_m >> 4) << 24);
}


// ------------------------------------------------------------------ epilogue of one 128 x 256 accumulator tile
constexpr int EPI_TILE_N = 256;
constexpr int EPI_ROWS = 128;
constexpr int EPI_COLS = 64;                         // columns per chunk (one 128-byte swizzle row of bf16)
constexpr int EPI_BYTES = EPI_ROWS * EPI_COLS * 2;   // 16 KiB staging buffer
constexpr int EPI_BUFS = 3;                          // ring of staging buffers: chunk g uses buffer g % 3

// Where a tile of C lives: matrix, first row of this CTA's 128 rows, first column.
struct EpiTile {
  int mat, m0, n0;
  bool valid;
};

// State the four epilogue warps carry from tile to tile.
struct EpilogueState {
  uint32_t g = 0;            // chunks processed so far
  uint32_t eph = 0;          // phase of the group rendezvous
  bool d_in_flight = false;  // the D load of chunk g has already been issued (prefetched during chunk g-1)
};

// Thread = one accumulator row (TMEM lane).  The tile leaves in four 64-column chunks through a ring of three
// 128B-swizzled staging buffers: TMA brings the D chunk in (requested one chunk ahead, across tile boundaries,
// so its latency hides behind the previous chunk), every thread turns its own row of D into its row of C in
// place (one bf16 rounding of gamma*(beta*D + alpha*acc)), TMA stores the chunk; a strictly upper tile of a
// symmetric product is also written transposed with plain stores (64 contiguous bytes per warp instruction).
// `next` is the tile this CTA processes afterwards (for the prefetch).  Returns false when a bounded wait expired.
__device__ __forceinline__ bool epilogue_tile(const TcArgs& a, const CUtensorMap* map_d, const CUtensorMap* map_c,
                                              const EpiTile& cur, const EpiTile& next, bool mirror, uint32_t taddr,
                                              uint32_t epi_base, uint32_t dfull_bar0, uint32_t egroup_bar, uint32_t tfull_bar,
                                              uint32_t aph, volatile int* abort_flag, EpilogueState& st, int quad, int lane) {
  const bool leader = quad == 2 && lane == 0;        // warp 2 is the first epilogue warp
  const int lrow = quad * 32 + lane;
  auto group_sync = [&]() -> bool {                  // rendezvous of the four warps on an mbarrier: bounded like every wait
    __syncwarp();
    if (lane == 0) mbar_arrive(egroup_bar);
    const bool done = mbar_wait(egroup_bar, st.eph, abort_flag);
    st.eph ^= 1u;
    return done;
  };
  const int mat = cur.mat, m0 = cur.m0, n0 = cur.n0;
  float gamma = 1.f;
  if (a.gamma_mode) {
    const float r = a.rnorm[mat];
    gamma = a.gamma_mode == 1 ? r : r * r;
  }
  const int row = m0 + lrow;
  const bool row_ok = row < a.m;
  __nv_bfloat16* cmat = a.c + size_t(mat) * a.stride_c;
  bool acc_ready = false;
#pragma unroll 1
  for (int cb = 0; cb < EPI_TILE_N / EPI_COLS; ++cb, ++st.g) {
    const int c0 = n0 + cb * EPI_COLS;
    if (c0 >= a.n) break;                             // uniform over the group
    const uint32_t b = st.g % EPI_BUFS;
    const uint32_t ebuf = epi_base + b * EPI_BYTES;
    const uint32_t dbar = dfull_bar0 + b * 8u;
    // the chunk after this one: the next chunk of this tile, or the first chunk of the next tile
    const bool more_here = cb + 1 < EPI_TILE_N / EPI_COLS && c0 + EPI_COLS < a.n;
    const bool have_next = more_here || next.valid;
    if (leader) {
      if (a.d) {
        if (!st.d_in_flight) {                        // only the very first chunk of a CTA is not prefetched
          tma_wait_read<2>();                         // buffer b was last read by the store of chunk g-3
          mbar_expect_tx(dbar, EPI_BYTES);
          tma_load_3d(ebuf, map_d, dbar, c0, m0, mat);
        }
        if (have_next) {
          const uint32_t nb = (st.g + 1) % EPI_BUFS;
          tma_wait_read<1>();                         // buffer nb was last read by the store of chunk g-2
          mbar_expect_tx(dfull_bar0 + nb * 8u, EPI_BYTES);
          if (more_here) tma_load_3d(epi_base + nb * EPI_BYTES, map_d, dfull_bar0 + nb * 8u, c0 + EPI_COLS, m0, mat);
          else tma_load_3d(epi_base + nb * EPI_BYTES, map_d, dfull_bar0 + nb * 8u, next.n0, next.m0, next.mat);
        }
      } else {
        tma_wait_read<2>();                           // buffer b was last read by the store of chunk g-3
      }
    }
    if (!acc_ready) {
      if (!mbar_wait(tfull_bar, aph, abort_flag)) return false;
      tc_fence_after();
      acc_ready = true;
    }
    if (a.d) {
      if (!mbar_wait(dbar, (st.g / EPI_BUFS) & 1u, abort_flag)) return false;
    } else {
      if (!group_sync()) return false;                // the leader's wait_group above frees the buffer for everyone
    }
    st.d_in_flight = a.d && have_next;
    uint32_t v[64];
    tc_ld32(taddr + uint32_t(cb * EPI_COLS), *reinterpret_cast<uint32_t(*)[32]>(&v[0]));
    tc_ld32(taddr + uint32_t(cb * EPI_COLS + 32), *reinterpret_cast<uint32_t(*)[32]>(&v[32]));
    tc_wait_ld();
    const uint32_t srow = ebuf + uint32_t(lrow) * 128u;
#pragma unroll
    for (int q = 0; q < 8; ++q) {                     // 16-byte piece q of the row sits at piece q ^ (row & 7)
      const uint32_t addr = srow + (uint32_t(q ^ (lrow & 7)) << 4);
      uint32_t d0 = 0, d1 = 0, d2 = 0, d3 = 0;
      if (a.d) asm volatile("ld.shared.v4.b32 {%0, %1, %2, %3}, [%4];" : "=r"(d0), "=r"(d1), "=r"(d2), "=r"(d3) : "r"(addr));
      const uint32_t dd[4] = {d0, d1, d2, d3};
      uint32_t oo[4];
#pragma unroll
      for (int e = 0; e < 4; ++e) {
        float x0 = a.alpha * __uint_as_float(v[q * 8 + 2 * e]), x1 = a.alpha * __uint_as_float(v[q * 8 + 2 * e + 1]);
        if (a.d) {
          const __nv_bfloat162 dp = *reinterpret_cast<const __nv_bfloat162*>(&dd[e]);
          x0 += a.beta * __low2float(dp);
          x1 += a.beta * __high2float(dp);
        }
        const __nv_bfloat162 o = __floats2bfloat162_rn(gamma * x0, gamma * x1);
        oo[e] = *reinterpret_cast<const uint32_t*>(&o);
      }
      asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(addr), "r"(oo[0]), "r"(oo[1]), "r"(oo[2]), "r"(oo[3]) : "memory");
      if (mirror && row_ok) {                         // C[c][row] = C[row][c]
#pragma unroll
        for (int e = 0; e < 4; ++e) {
          const int c = c0 + q * 8 + 2 * e;
          const __nv_bfloat162 o = *reinterpret_cast<const __nv_bfloat162*>(&oo[e]);
          if (c < a.n) cmat[size_t(c) * a.ldc + row] = __low2bfloat16(o);
          if (c + 1 < a.n) cmat[size_t(c + 1) * a.ldc + row] = __high2bfloat16(o);
        }
      }
    }
    fence_async_smem();                               // generic-proxy writes -> visible to the TMA store
    if (!group_sync()) return false;                  // everyone is done with the buffer (reads of D, writes of C)
    if (leader) {
      tma_store_3d(map_c, ebuf, c0, m0, mat);         // rows/columns beyond the matrix are clipped
      tma_commit();
    }
  }
  return true;
}

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
}  // namespace muon
