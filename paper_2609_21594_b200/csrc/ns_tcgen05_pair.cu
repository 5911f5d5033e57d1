// Paired-CTA tensor-core kernel for the Newton-Schulz products (Eq. 1): the same operation as
// ns_tcgen05.cu, computed by clusters of two CTAs that drive one tcgen05.mma.cta_group::2 of shape
// M256 x N256 x K16 together.
//
//   C[k] = gamma_k * (beta * D[k] + alpha * P[k] Q[k]^T)   (nn = 0)      C[k] = ... P[k] Q[k]   (nn = 1)
//
// A pair owns a 256 x 256 output tile.  CTA r of the pair (r = 0, 1) owns rows [128 r, 128 r + 128):
// it loads those 128 rows of P and HALF of the Q tile (128 of the 256 columns of the output) per
// 64-wide k-block -- 32 KiB per stage instead of 48 KiB, so five stages and a three-buffer epilogue ring fit and the bytes that cross
// L2 -> shared memory per flop drop by a third.  The leader (r = 0) issues every MMA; the hardware
// reads each CTA's own P rows and both CTAs' Q halves.  Each CTA keeps its 128 x 256 fp32 accumulator
// in its own TMEM (double-buffered) and runs its own epilogue.
//
// Synchronisation (all waits bounded, as in the single-CTA kernel):
//   full[s]    leader only.  The leader's producer arms it with the bytes of BOTH CTAs; both producers'
//              TMA loads complete on it (cta_group::2 form, no multicast).
//   empty[s]   in each CTA; the leader's tcgen05.commit arrives on both (commit multicast).
//   tfull[a]   in each CTA; commit multicast after a tile's last k-block.
//   tempty[a]  leader only, 8 arrivals: the four epilogue warps of each CTA (remote arrive).
#include "tc_common.cuh"

namespace muon {
namespace {

using namespace tc;

constexpr int BM = 128;          // rows per CTA; the pair covers 256
constexpr int BN = 256;          // columns of the pair's tile
constexpr int BNH = 128;         // columns of Q each CTA stages
constexpr int BK = 64;
constexpr int UK = 16;
constexpr int STAGES = 5;
constexpr int A_BYTES = BM * BK * 2;          // 16 KiB
constexpr int B_BYTES = BNH * BK * 2;         // 16 KiB
constexpr int STAGE_BYTES = A_BYTES + B_BYTES;
constexpr int SMEM_BYTES = STAGES * STAGE_BYTES + EPI_BUFS * EPI_BYTES + 1024 + 256;
constexpr int TMEM_COLS = 512;
constexpr int NUM_THREADS = 192;

__device__ __forceinline__ uint32_t cluster_rank() {
  uint32_t r;
  asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
  return r;
}
__device__ __forceinline__ uint32_t map_to_cta(uint32_t local_addr, uint32_t rank) {
  uint32_t r;
  asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(local_addr), "r"(rank));
  return r;
}
__device__ __forceinline__ void cluster_sync_all() {
  asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory");
  asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory");
}
__device__ __forceinline__ void mbar_arrive_cluster(uint32_t cluster_addr) {
  asm volatile("mbarrier.arrive.release.cluster.shared::cluster.b64 _, [%0];" ::"r"(cluster_addr) : "memory");
}
// TMA load whose completion bytes are credited to a barrier that may live in the peer CTA.
__device__ __forceinline__ void tma_load_3d_pair(uint32_t dst, const CUtensorMap* map, uint32_t bar_cluster_addr, int c0,
                                                 int c1, int c2) {
  asm volatile(
      "cp.async.bulk.tensor.3d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5}], [%2];"
      ::"r"(dst), "l"(map), "r"(bar_cluster_addr), "r"(c0), "r"(c1), "r"(c2)
      : "memory");
}
__device__ __forceinline__ void tc_mma_pair(uint32_t d_tmem, uint64_t adesc, uint64_t bdesc, uint32_t idesc, uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::2.kind::f16 [%0], %1, %2, %3, p;\n\t}"
      ::"r"(d_tmem), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate)
      : "memory");
}
// Arrive on the barrier at this shared-memory offset in both CTAs of the pair once all MMAs issued so far are done.
__device__ __forceinline__ void tc_commit_pair(uint32_t bar) {
  asm volatile(
      "{\n\t.reg .b16 m;\n\t"
      "mov.b16 m, 3;\n\t"
      "tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.multicast::cluster.b64 [%0], m;\n\t}"
      ::"r"(bar)
      : "memory");
}

struct Tile {
  int mat, m0, n0;   // m0: first row of the PAIR's tile
};
// Tiles are 256 x 256.  Dense: row blocks vary fastest.  Symmetric: block row I needs block columns J >= I.
__device__ __forceinline__ Tile decode_tile(int t, const TcArgs& a) {
  Tile r;
  r.mat = t / a.tiles_per_mat;
  int u = t - r.mat * a.tiles_per_mat;
  if (!a.symmetric) {
    r.n0 = (u / a.tiles_m) * BN;
    r.m0 = (u % a.tiles_m) * (2 * BM);
    return r;
  }
  int i = 0;
  while (u >= a.tiles_n - i) {
    u -= a.tiles_n - i;
    ++i;
  }
  r.m0 = i * (2 * BM);
  r.n0 = (i + u) * BN;
  return r;
}

template <bool NN>
__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(NUM_THREADS, 1)
ns_product_pair_kernel(const __grid_constant__ CUtensorMap map_p, const __grid_constant__ CUtensorMap map_q,
                       const __grid_constant__ CUtensorMap map_d, const __grid_constant__ CUtensorMap map_c, const TcArgs a) {
  extern __shared__ uint8_t smem_raw[];
  const uint32_t raw = smem_u32(smem_raw);
  const uint32_t base = (raw + 1023u) & ~1023u;
  uint8_t* gen_base = smem_raw + (base - raw);
  const uint32_t epi_base = base + STAGES * STAGE_BYTES;
  constexpr int BAR_OFF = STAGES * STAGE_BYTES + EPI_BUFS * EPI_BYTES;
  const uint32_t bars = base + BAR_OFF;
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(gen_base + BAR_OFF + 192);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(gen_base + BAR_OFF + 200);
  auto full_bar = [&](int s) { return bars + uint32_t(s) * 8u; };
  auto empty_bar = [&](int s) { return bars + uint32_t(STAGES + s) * 8u; };
  auto tfull_bar = [&](int i) { return bars + uint32_t(2 * STAGES + i) * 8u; };
  auto tempty_bar = [&](int i) { return bars + uint32_t(2 * STAGES + 2 + i) * 8u; };
  auto dfull_bar = [&](int i) { return bars + uint32_t(2 * STAGES + 4 + i) * 8u; };
  const uint32_t egroup_bar = bars + uint32_t(2 * STAGES + 4 + EPI_BUFS) * 8u;

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const uint32_t rank = cluster_rank();
  const bool leader_cta = rank == 0;
  const int pair_id = blockIdx.x >> 1, num_pairs = gridDim.x >> 1;
  const int total_tiles = a.batch * a.tiles_per_mat;
  const int num_kb = (a.kdim + BK - 1) / BK;

  if (threadIdx.x == 0) {
    for (int s = 0; s < STAGES; ++s) {
      mbar_init(full_bar(s), 1);
      mbar_init(empty_bar(s), 1);
    }
    for (int i = 0; i < 2; ++i) {
      mbar_init(tfull_bar(i), 1);
      mbar_init(tempty_bar(i), 8);
    }
    for (int i = 0; i < EPI_BUFS; ++i) mbar_init(dfull_bar(i), 1);
    mbar_init(egroup_bar, 4);
    *abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  }
  if (warp == 1) {
    asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(tmem_slot)), "r"(TMEM_COLS)
                 : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  cluster_sync_all();            // both CTAs' barriers exist before any remote arrive or remote TMA completion
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;

  if (warp == 0) {
    // ------------------------------------------------------------------ TMA producer (one per CTA)
    if (lane == 0) {
      uint32_t it = 0;
      bool ok = true;
      const int mrow = int(rank) * BM;           // this CTA's rows inside the pair's tile
      const int ncol = int(rank) * BNH;          // this CTA's half of the Q tile
      for (int t = pair_id; t < total_tiles && ok; t += num_pairs) {
        const Tile tl = decode_tile(t, a);
        for (int kb = 0; kb < num_kb; ++kb, ++it) {
          const int s = int(it % STAGES);
          const uint32_t ph = (it / STAGES) & 1u;
          if (!mbar_wait(empty_bar(s), ph ^ 1u, abort_flag)) { ok = false; break; }
          const uint32_t sa = base + uint32_t(s) * STAGE_BYTES, sb = sa + A_BYTES;
          if (leader_cta) mbar_expect_tx(full_bar(s), 2 * STAGE_BYTES);
          const uint32_t fb = map_to_cta(full_bar(s), 0);
          const int k0 = kb * BK;
          tma_load_3d_pair(sa, &map_p, fb, k0, tl.m0 + mrow, tl.mat);
          if (!NN) {
            tma_load_3d_pair(sb, &map_q, fb, k0, tl.n0 + ncol, tl.mat);
          } else {
#pragma unroll
            for (int j = 0; j < BNH / 64; ++j)
              tma_load_3d_pair(sb + uint32_t(j) * (64 * BK * 2), &map_q, fb, tl.n0 + ncol + 64 * j, k0, tl.mat);
          }
        }
      }
      if (!ok) {
        *abort_flag = 1;
        atomicExch(a.status, 11);
      }
      if (leader_cta) {   // every armed stage (both CTAs' bytes) has landed before shared memory is released
        const uint32_t issued = it;
        for (uint32_t j = (issued > STAGES ? issued - STAGES : 0); j < issued; ++j) {
          const int s = int(j % STAGES);
          const uint32_t ph = (j / STAGES) & 1u;
          if (!mbar_wait(full_bar(s), ph, abort_flag, false, WAIT_CYCLES / 8)) atomicExch(a.status, 12);
        }
      }
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------------ MMA issuer (leader CTA only)
    if (lane == 0 && leader_cta) {
      constexpr uint32_t idesc = make_idesc(NN, 2 * BM, BN);
      uint32_t it = 0, tile_it = 0;
      bool ok = true;
      for (int t = pair_id; t < total_tiles && ok; t += num_pairs, ++tile_it) {
        const uint32_t acc = tile_it & 1u, aph = (tile_it >> 1) & 1u;
        if (!mbar_wait(tempty_bar(int(acc)), aph ^ 1u, abort_flag)) { ok = false; break; }
        tc_fence_after();
        const uint32_t d_tmem = tmem_base + acc * uint32_t(BN);
        for (int kb = 0; kb < num_kb; ++kb, ++it) {
          const int s = int(it % STAGES);
          const uint32_t ph = (it / STAGES) & 1u;
          if (!mbar_wait(full_bar(s), ph, abort_flag)) { ok = false; break; }
          tc_fence_after();
          const uint32_t sa = base + uint32_t(s) * STAGE_BYTES, sb = sa + A_BYTES;
#pragma unroll
          for (int k = 0; k < BK / UK; ++k) {
            const uint64_t ad = make_desc(sa + uint32_t(k) * (UK * 2), 16, 1024);
            const uint64_t bd = NN ? make_desc(sb + uint32_t(k) * (UK * 128), 64 * BK * 2, 1024)
                                   : make_desc(sb + uint32_t(k) * (UK * 2), 16, 1024);
            tc_mma_pair(d_tmem, ad, bd, idesc, (kb > 0 || k > 0) ? 1u : 0u);
          }
          tc_commit_pair(empty_bar(s));
        }
        if (ok) tc_commit_pair(tfull_bar(int(acc)));
      }
      if (!ok) {
        *abort_flag = 1;
        atomicExch(a.status, 13);
      }
    }
  } else {
    // ------------------------------------------------------------------ epilogue warps (per CTA: its 128 rows)
    const int quad = warp & 3;                     // TMEM lane quadrant this warp may read
    EpilogueState est;
    uint32_t tile_it = 0;
    bool ok = true;
    for (int t = pair_id; t < total_tiles && ok; t += num_pairs, ++tile_it) {
      const Tile tl = decode_tile(t, a);
      const uint32_t acc = tile_it & 1u, aph = (tile_it >> 1) & 1u;
      const bool mirror = a.symmetric && tl.n0 > tl.m0;          // pair tile strictly above the diagonal block
      const uint32_t taddr = tmem_base + acc * uint32_t(BN) + (uint32_t(quad * 32) << 16);
      const EpiTile cur{tl.mat, tl.m0 + int(rank) * BM, tl.n0, true};
      EpiTile nxt{0, 0, 0, false};
      if (t + num_pairs < total_tiles) {
        const Tile tn = decode_tile(t + num_pairs, a);
        nxt = EpiTile{tn.mat, tn.m0 + int(rank) * BM, tn.n0, true};
      }
      ok = epilogue_tile(a, &map_d, &map_c, cur, nxt, mirror, taddr, epi_base, dfull_bar(0), egroup_bar, tfull_bar(int(acc)),
                         aph, abort_flag, est, quad, lane);
      if (!ok) break;
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive_cluster(map_to_cta(tempty_bar(int(acc)), 0));   // the leader CTA counts both epilogues
    }
    if (quad == 2 && lane == 0) {
      tma_wait_all();                               // every store has landed before the CTA retires
      if (!ok)                                      // a prefetched D chunk may still be landing: give it (bounded) time
        for (int i = 0; i < 64; ++i) __nanosleep(1000);
    }
    if (!ok && lane == 0) {
      *abort_flag = 1;
      atomicExch(a.status, 14);
    }
  }
  tc_fence_before();
  __syncthreads();
  cluster_sync_all();            // neither CTA retires while its peer may still signal its barriers or read its tiles
  tc_fence_after();
  if (warp == 1) {
    __syncwarp();
    asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(TMEM_COLS) : "memory");
  }
}

// Per device ordinal: shared-memory attribute set and SM count looked up once.
constexpr int kMaxDevices = 64;
int g_num_sms[kMaxDevices] = {};

}  // namespace

bool tc_pair_supported(const GemmArgs& a) {
  // The pair kernel pays off once a matrix has at least one full 256-row tile; smaller ones keep the single-CTA kernel.
  return a.m > 128;
}

int launch_gemm_tc_pair(muon_ctx* ctx, const GemmArgs& a, cudaStream_t st) {
  if (!ctx->tmap_encode) return MUON_ERR_CUDA;
  if (ctx->device < 0 || ctx->device >= kMaxDevices) return MUON_ERR_UNSUPPORTED;
  if (!g_num_sms[ctx->device]) {
    if (cudaFuncSetAttribute(ns_product_pair_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, SMEM_BYTES) != cudaSuccess ||
        cudaFuncSetAttribute(ns_product_pair_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, SMEM_BYTES) != cudaSuccess)
      return MUON_ERR_CUDA;
    cudaDeviceProp prop;
    if (cudaGetDeviceProperties(&prop, ctx->device) != cudaSuccess) return MUON_ERR_CUDA;
    g_num_sms[ctx->device] = prop.multiProcessorCount;
  }
  CUtensorMap map_p, map_q, map_c, map_d;
  if (!encode_map(ctx->tmap_encode, &map_p, a.p, a.kdim, a.m, a.batch, a.ldp, a.stride_p, BM)) return MUON_ERR_CUDA;
  if (!a.nn) {
    if (!encode_map(ctx->tmap_encode, &map_q, a.q, a.kdim, a.n, a.batch, a.ldq, a.stride_q, BNH)) return MUON_ERR_CUDA;
  } else {
    if (!encode_map(ctx->tmap_encode, &map_q, a.q, a.n, a.kdim, a.batch, a.ldq, a.stride_q, BK)) return MUON_ERR_CUDA;
  }
  if (!encode_map(ctx->tmap_encode, &map_c, a.c, a.n, a.m, a.batch, a.ldc, a.stride_c, BM)) return MUON_ERR_CUDA;
  if (!encode_map(ctx->tmap_encode, &map_d, a.d ? a.d : a.c, a.n, a.m, a.batch, a.ldc, a.stride_c, BM)) return MUON_ERR_CUDA;
  TcArgs t;
  t.d = static_cast<const __nv_bfloat16*>(a.d);
  t.c = static_cast<__nv_bfloat16*>(a.c);
  t.m = a.m; t.n = a.n; t.kdim = a.kdim; t.ldc = a.ldc;
  t.stride_c = a.stride_c;
  t.batch = a.batch;
  t.tiles_m = (a.m + 2 * BM - 1) / (2 * BM);
  t.tiles_n = (a.n + BN - 1) / BN;
  t.symmetric = a.symmetric ? 1 : 0;
  t.tiles_per_mat = t.symmetric ? t.tiles_n * (t.tiles_n + 1) / 2 : t.tiles_m * t.tiles_n;
  t.rnorm = a.rnorm;
  t.gamma_mode = a.gamma_mode;
  t.alpha = a.alpha; t.beta = a.beta;
  t.status = ctx->d_status;
  const int64_t tiles = int64_t(t.tiles_per_mat) * t.batch;
  const int64_t pairs = g_num_sms[ctx->device] / 2;
  const unsigned grid = unsigned(2 * (tiles < pairs ? tiles : pairs));
  if (a.nn) ns_product_pair_kernel<true><<<grid, NUM_THREADS, SMEM_BYTES, st>>>(map_p, map_q, map_d, map_c, t);
  else ns_product_pair_kernel<false><<<grid, NUM_THREADS, SMEM_BYTES, st>>>(map_p, map_q, map_d, map_c, t);
  return cudaGetLastError() == cudaSuccess ? 1 : MUON_ERR_CUDA;
}

}  // namespace muon
