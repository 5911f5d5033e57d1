// Shared pieces of the tensor-core Newton-Schulz kernels: argument block, PTX wrappers for
// mbarrier / TMA / tcgen05, shared-memory and instruction descriptors.  Internal to the library.
#pragma once

#include "tc_tables.h"

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
  float alpha, beta, diag;
  const float* coef;        // per-matrix coefficient rows (null: alpha, beta, diag above for every matrix)
  int32_t coef_a, coef_b, coef_d, coef_stride;
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

// Instruction descriptor for kind::f16: fp32 accumulator, bf16 A and B, each K- or MN-major.
__host__ __device__ constexpr uint32_t make_idesc(bool b_mn_major, int umma_m, int umma_n, bool a_mn_major = false) {
  return (1u << 4) | (1u << 7) | (1u << 10) | (uint32_t(a_mn_major ? 1 : 0) << 15) | (uint32_t(b_mn_major ? 1 : 0) << 16) |
         (uint32_t(umma_n >> 3) << 17) | (uint32_t(umma_m >> 4) << 24);
}


// ------------------------------------------------------------------ epilogue of one 128-row accumulator tile
constexpr int EPI_ROWS = 128;
constexpr int EPI_COLS = 64;                         // columns per chunk (one 128-byte swizzle row of bf16)
constexpr int EPI_BYTES = EPI_ROWS * EPI_COLS * 2;   // 16 KiB staging buffer
#ifndef MUON_EPI_BUFS
#define MUON_EPI_BUFS 3
#endif
constexpr int EPI_BUFS = MUON_EPI_BUFS;              // ring of staging buffers: chunk g uses buffer g % EPI_BUFS

// What the four epilogue warps of a CTA need to know about one accumulator tile: 128 rows (row block
// `rblk`) times one or two 128-column blocks (`cblk0` in TMEM columns [0,128), `cblk1` in [128,256);
// cblk1 < 0 = the tile is 128 columns wide).  valid = this CTA has rows to write for the tile.
struct EpiTile {
  const CUtensorMap* map_d;
  const CUtensorMap* map_c;
  const __nv_bfloat16* d;    // aux matrix D (may be null)
  __nv_bfloat16* c;
  int64_t stride_c;
  int32_t ldc, m, n;
  int32_t mat, rblk;
  int32_t cblk0, cblk1;
  bool mirror0, mirror1;     // also write the 128 x 128 block transposed (symmetric products, off-diagonal blocks)
  float alpha, beta, gamma;
  float diag;                // added to C[i][i] before gamma (0: nothing to add)
  bool valid;
};

struct DiagYes { static constexpr bool value = true; };
struct DiagNo { static constexpr bool value = false; };

// State the four epilogue warps carry from tile to tile.
struct EpilogueState {
  uint32_t g = 0;            // chunks processed so far
  uint32_t eph = 0;          // phase of the group rendezvous
  uint32_t dph = 0;          // bit b: phase of the D-chunk barrier of staging buffer b
  bool d_in_flight = false;  // the D load of chunk g has already been issued (prefetched during chunk g-1)
};

__device__ __forceinline__ int epi_chunk_col(const EpiTile& t, int cb) {          // first column of chunk cb, or -1
  const int blk = cb < 2 ? t.cblk0 : t.cblk1;
  if (blk < 0) return -1;
  const int c0 = blk * 128 + (cb & 1) * EPI_COLS;
  return c0 < t.n ? c0 : -1;
}

// Thread = one accumulator row (TMEM lane).  The tile leaves in 64-column chunks through a ring of three
// 128B-swizzled staging buffers: TMA brings the D chunk in (requested one chunk ahead, across tile boundaries,
// so its latency hides behind the previous chunk), every thread turns its own row of D into its row of C in
// place (one bf16 rounding of gamma*(beta*D + alpha*acc)), TMA stores the chunk; an off-diagonal block of a
// symmetric product is also written transposed with plain stores (64 contiguous bytes per warp instruction).
// `next` is the tile this CTA processes afterwards (for the prefetch).  Returns false when a bounded wait expired.
// SPLIT warps share a lane quadrant (they may all read its 32 TMEM lanes): warp `part` of them handles columns
// [part * 64 / SPLIT, (part + 1) * 64 / SPLIT) of every chunk, so a chunk's conversion work is spread over 4 * SPLIT warps.
// `leader`: the one thread of the group that issues TMA loads and stores.
template <int SPLIT>
__device__ __forceinline__ bool epilogue_tile(const EpiTile& cur, const EpiTile& next, uint32_t taddr, uint32_t epi_base,
                                              uint32_t dfull_bar0, uint32_t egroup_bar, uint32_t tfull_bar, uint32_t aph,
                                              volatile int* abort_flag, EpilogueState& st, int quad, int lane, int part,
                                              bool leader) {
  static_assert(SPLIT == 1 || SPLIT == 2, "one or two warps per lane quadrant");
  constexpr int WCOLS = EPI_COLS / SPLIT;            // columns of a chunk this warp converts
  const int lrow = quad * 32 + lane;
  auto group_sync = [&]() -> bool {                  // rendezvous of the four warps on an mbarrier: bounded like every wait
    __syncwarp();
    if (lane == 0) mbar_arrive(egroup_bar);
    const bool done = mbar_wait(egroup_bar, st.eph, abort_flag);
    st.eph ^= 1u;
    return done;
  };
  const int mat = cur.mat, m0 = cur.rblk * EPI_ROWS;
  const float alpha = cur.alpha, beta = cur.beta, gamma = cur.gamma;
  const int row = m0 + lrow;
  const bool row_ok = row < cur.m;
  __nv_bfloat16* cmat = cur.c + size_t(mat) * cur.stride_c;
  const bool next_d = next.valid && next.d != nullptr;
  bool acc_ready = false;
#pragma unroll 1
  for (int cb = 0; cb < 4; ++cb) {
    const int c0 = epi_chunk_col(cur, cb);
    if (c0 < 0) continue;                             // uniform over the group
    const uint32_t b = st.g % EPI_BUFS;
    const uint32_t ebuf = epi_base + b * EPI_BYTES;
    const uint32_t dbar = dfull_bar0 + b * 8u;
    // the chunk after this one: the next valid chunk of this tile, or the first chunk of the next tile
    int nc0 = -1;
    for (int k = cb + 1; k < 4 && nc0 < 0; ++k) nc0 = epi_chunk_col(cur, k);
    const bool more_here = nc0 >= 0;
    const bool prefetch = cur.d ? (more_here || next_d) : false;
    if (leader) {
      if (cur.d) {
        if (!st.d_in_flight) {                        // a chunk that nobody prefetched (the first of a CTA, or after a tile without D)
          tma_wait_read<EPI_BUFS - 1>();              // buffer b was last read by the store of chunk g - EPI_BUFS
          mbar_expect_tx(dbar, EPI_BYTES);
          tma_load_3d(ebuf, cur.map_d, dbar, c0, m0, mat);
        }
        if (prefetch) {
          const uint32_t nb = (st.g + 1) % EPI_BUFS;
          tma_wait_read<EPI_BUFS - 2>();              // buffer nb was last read by the store of chunk g + 1 - EPI_BUFS
          mbar_expect_tx(dfull_bar0 + nb * 8u, EPI_BYTES);
          if (more_here) tma_load_3d(epi_base + nb * EPI_BYTES, cur.map_d, dfull_bar0 + nb * 8u, nc0, m0, mat);
          else tma_load_3d(epi_base + nb * EPI_BYTES, next.map_d, dfull_bar0 + nb * 8u, epi_chunk_col(next, 0),
                           next.rblk * EPI_ROWS, next.mat);
        }
      } else {
        tma_wait_read<EPI_BUFS - 1>();                // buffer b was last read by the store of chunk g - EPI_BUFS
      }
    }
    if (!acc_ready) {
      if (!mbar_wait(tfull_bar, aph, abort_flag)) return false;
      tc_fence_after();
      acc_ready = true;
    }
    if (cur.d) {
      if (!mbar_wait(dbar, (st.dph >> b) & 1u, abort_flag)) return false;
      st.dph ^= 1u << b;
    } else {
      if (!group_sync()) return false;                // the leader's wait_group above frees the buffer for everyone
    }
    st.d_in_flight = prefetch;
    uint32_t v[WCOLS];
#pragma unroll
    for (int h = 0; h < WCOLS / 32; ++h)
      tc_ld32(taddr + uint32_t(cb * EPI_COLS + part * WCOLS + h * 32), *reinterpret_cast<uint32_t(*)[32]>(&v[h * 32]));
    tc_wait_ld();
    const bool mirror = cb < 2 ? cur.mirror0 : cur.mirror1;
    const uint32_t srow = ebuf + uint32_t(lrow) * 128u;
    // the chunk holds diagonal elements only when its column block is this CTA's row block
    const bool diag_chunk = cur.diag != 0.f && (c0 >> 7) == cur.rblk;
    auto convert = [&](auto with_diag) {
      constexpr bool DIAG = decltype(with_diag)::value;
#pragma unroll
      for (int qq = 0; qq < WCOLS / 8; ++qq) {        // 16-byte piece q of the row sits at piece q ^ (row & 7)
        const int q = part * (WCOLS / 8) + qq;
        const uint32_t addr = srow + (uint32_t(q ^ (lrow & 7)) << 4);
        uint32_t d0 = 0, d1 = 0, d2 = 0, d3 = 0;
        if (cur.d) asm volatile("ld.shared.v4.b32 {%0, %1, %2, %3}, [%4];" : "=r"(d0), "=r"(d1), "=r"(d2), "=r"(d3) : "r"(addr));
        const uint32_t dd[4] = {d0, d1, d2, d3};
        uint32_t oo[4];
#pragma unroll
        for (int e = 0; e < 4; ++e) {
          float x0 = alpha * __uint_as_float(v[qq * 8 + 2 * e]), x1 = alpha * __uint_as_float(v[qq * 8 + 2 * e + 1]);
          if (cur.d) {
            const __nv_bfloat162 dp = *reinterpret_cast<const __nv_bfloat162*>(&dd[e]);
            x0 += beta * __low2float(dp);
            x1 += beta * __high2float(dp);
          }
          if (DIAG) {
            const int c = c0 + q * 8 + 2 * e;
            if (c == row) x0 += cur.diag;
            if (c + 1 == row) x1 += cur.diag;
          }
          const __nv_bfloat162 o = __floats2bfloat162_rn(gamma * x0, gamma * x1);
          oo[e] = *reinterpret_cast<const uint32_t*>(&o);
        }
        asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(addr), "r"(oo[0]), "r"(oo[1]), "r"(oo[2]), "r"(oo[3]) : "memory");
        if (mirror && row_ok) {                       // C[c][row] = C[row][c]
#pragma unroll
          for (int e = 0; e < 4; ++e) {
            const int c = c0 + q * 8 + 2 * e;
            const __nv_bfloat162 o = *reinterpret_cast<const __nv_bfloat162*>(&oo[e]);
            if (c < cur.n) cmat[size_t(c) * cur.ldc + row] = __low2bfloat16(o);
            if (c + 1 < cur.n) cmat[size_t(c + 1) * cur.ldc + row] = __high2bfloat16(o);
          }
        }
      }
    };
    if (diag_chunk) convert(DiagYes());
    else convert(DiagNo());
    fence_async_smem();                               // generic-proxy writes -> visible to the TMA store
    if (!group_sync()) return false;                  // everyone is done with the buffer (reads of D, writes of C)
    if (leader) {
      tma_store_3d(cur.map_c, ebuf, c0, m0, mat);     // rows/columns beyond the matrix are clipped
      tma_commit();
    }
    ++st.g;
  }
  return true;
}

}  // namespace tc
}  // namespace muon
