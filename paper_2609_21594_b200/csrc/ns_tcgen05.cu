// Tensor-core Newton-Schulz engine for sm_100a, single-CTA kernel: batched products of Eq. 1 with bf16
// operands and fp32 accumulation in tensor memory.  It serves matrices of at most 128 rows and is the
// cross-check of the paired-CTA kernel, which runs everything else.
//
//   C[k] = gamma_k * (beta * D[k] + alpha * P[k] Q[k]^T + diag * I)   nn = 0   (A = X X^T,  P = aI + bA + cA A^T)
//   C[k] = gamma_k * (beta * D[k] + alpha * P[k] Q[k])                nn = 1   (X' = P X)
//
// One persistent CTA per SM, 192 threads, warp-specialised:
//   warp 0      TMA producer: cp.async.bulk.tensor loads of 128B-swizzled operand tiles into a
//               3-stage shared-memory ring of 48 KiB stages (one mbarrier pair per stage)
//   warp 1      MMA issuer: one thread issues tcgen05.mma (M128 x N256 x K16, kind::f16) on shared-memory
//               descriptors; accumulators live in TMEM, double-buffered (2 x 256 columns)
//   warps 2..5  epilogue (shared with the paired kernel): tcgen05.ld of the accumulator, D chunk by TMA,
//               fused gamma*(beta*D + alpha*acc) with one bf16 rounding, TMA store; overlaps the next
//               tile's main loop
// P tiles are K-major.  Q tiles are K-major for nn = 0 and MN-major for nn = 1 (X is read as stored,
// row-major s x l, so no transposed copy of X is ever made).
// Every wait on an mbarrier is bounded: on expiry the CTA records a code in the context's status
// word, stops issuing work, waits (bounded) for its own TMA copies, frees its TMEM and returns.
#include "tc_common.cuh"

namespace muon {
namespace {

using namespace tc;

constexpr int BM = 128;          // tile rows   (UMMA M)
constexpr int BN = 256;          // tile cols   (UMMA N)
constexpr int BK = 64;           // k per stage (one 128-byte swizzle atom of bf16)
constexpr int UK = 16;           // k per tcgen05.mma for 16-bit inputs
constexpr int STAGES = 3;
constexpr int A_BYTES = BM * BK * 2;          // 16 KiB
constexpr int B_BYTES = BN * BK * 2;          // 32 KiB
constexpr int STAGE_BYTES = A_BYTES + B_BYTES;
constexpr int SMEM_BYTES = STAGES * STAGE_BYTES + EPI_BUFS * EPI_BYTES + 1024 /*alignment slack*/ + 256 /*barriers*/;
constexpr int TMEM_COLS = 512;
constexpr int NUM_THREADS = 192;

struct Tile {
  int mat, m0, n0;
};
// Dense: row blocks vary fastest, so concurrent CTAs share the Q tile.
// Symmetric (m == n): row block i (128 rows) needs column blocks j >= i/2 (256 columns): the tile then holds
// at least one element on or above the diagonal.  Rows 2q and 2q+1 both start at column block q; the pair
// owns 2*(tiles_n - q) tiles, so the pairs before q own 2*q*tiles_n - q*(q-1).
__device__ __forceinline__ Tile decode_tile(int t, const TcArgs& a) {
  Tile r;
  r.mat = t / a.tiles_per_mat;
  int u = t - r.mat * a.tiles_per_mat;
  if (!a.symmetric) {
    r.n0 = (u / a.tiles_m) * BN;
    r.m0 = (u % a.tiles_m) * BM;
    return r;
  }
  int q = 0;
  while (true) {
    const int rows_in_pair = (2 * q + 1 < a.tiles_m) ? 2 : 1;
    const int cnt = rows_in_pair * (a.tiles_n - q);
    if (u < cnt) break;
    u -= cnt;
    ++q;
  }
  const int w = a.tiles_n - q;
  r.m0 = (2 * q + u / w) * BM;
  r.n0 = (q + u % w) * BN;
  return r;
}

template <bool NN>
__global__ void __launch_bounds__(NUM_THREADS, 1)
ns_product_tc_kernel(const __grid_constant__ CUtensorMap map_p, const __grid_constant__ CUtensorMap map_q,
                     const __grid_constant__ CUtensorMap map_d, const __grid_constant__ CUtensorMap map_c, const TcArgs a) {
  extern __shared__ uint8_t smem_raw[];
  const uint32_t raw = smem_u32(smem_raw);
  const uint32_t base = (raw + 1023u) & ~1023u;            // swizzled tiles need 1024-byte alignment
  uint8_t* gen_base = smem_raw + (base - raw);
  const uint32_t epi_base = base + STAGES * STAGE_BYTES;    // the epilogue staging buffers follow the ring
  constexpr int BAR_OFF = STAGES * STAGE_BYTES + EPI_BUFS * EPI_BYTES;
  const uint32_t bars = base + BAR_OFF;                     // barrier block follows the buffers
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(gen_base + BAR_OFF + 128);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(gen_base + BAR_OFF + 136);
  auto dfull_bar = [&](int i) { return bars + uint32_t(2 * STAGES + 4 + i) * 8u; };
  const uint32_t egroup_bar = bars + uint32_t(2 * STAGES + 4 + EPI_BUFS) * 8u;   // 128-thread rendezvous of the epilogue group
  auto full_bar = [&](int s) { return bars + uint32_t(s) * 8u; };
  auto empty_bar = [&](int s) { return bars + uint32_t(STAGES + s) * 8u; };
  auto tfull_bar = [&](int i) { return bars + uint32_t(2 * STAGES + i) * 8u; };
  auto tempty_bar = [&](int i) { return bars + uint32_t(2 * STAGES + 2 + i) * 8u; };

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int total_tiles = a.batch * a.tiles_per_mat;
  const int num_kb = (a.kdim + BK - 1) / BK;

  if (threadIdx.x == 0) {
    for (int s = 0; s < STAGES; ++s) {
      mbar_init(full_bar(s), 1);
      mbar_init(empty_bar(s), 1);
    }
    for (int i = 0; i < 2; ++i) {
      mbar_init(tfull_bar(i), 1);
      mbar_init(tempty_bar(i), 4);
    }
    for (int i = 0; i < EPI_BUFS; ++i) mbar_init(dfull_bar(i), 1);
    mbar_init(egroup_bar, 4);
    *abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  }
  if (warp == 1) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(tmem_slot)), "r"(TMEM_COLS)
                 : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;

  if (warp == 0) {
    // ------------------------------------------------------------------ TMA producer
    if (lane == 0) {
      uint32_t it = 0;
      bool ok = true;
      for (int t = blockIdx.x; t < total_tiles && ok; t += gridDim.x) {
        const Tile tl = decode_tile(t, a);
        for (int kb = 0; kb < num_kb; ++kb, ++it) {
          const int s = int(it % STAGES);
          const uint32_t ph = (it / STAGES) & 1u;
          if (!mbar_wait(empty_bar(s), ph ^ 1u, abort_flag)) { ok = false; break; }
          const uint32_t sa = base + uint32_t(s) * STAGE_BYTES, sb = sa + A_BYTES;
          mbar_expect_tx(full_bar(s), STAGE_BYTES);
          const int k0 = kb * BK;
          tma_load_3d(sa, &map_p, full_bar(s), k0, tl.m0, tl.mat);                   // P rows m0.., k0..k0+63
          if (!NN) {
            tma_load_3d(sb, &map_q, full_bar(s), k0, tl.n0, tl.mat);                 // Q rows n0..n0+127
            tma_load_3d(sb + A_BYTES, &map_q, full_bar(s), k0, tl.n0 + 128, tl.mat); // Q rows n0+128..n0+255
          } else {
#pragma unroll
            for (int j = 0; j < BN / 64; ++j)                                        // Q[k0..k0+63][n0+64j..+63]
              tma_load_3d(sb + uint32_t(j) * (64 * BK * 2), &map_q, full_bar(s), tl.n0 + 64 * j, k0, tl.mat);
          }
        }
      }
      if (!ok) {
        *abort_flag = 1;
        atomicExch(a.status, 1);
      }
      // Drain: every armed stage must have landed before this CTA's shared memory is released.
      const uint32_t issued = it;
      for (uint32_t j = (issued > STAGES ? issued - STAGES : 0); j < issued; ++j) {
        const int s = int(j % STAGES);
        const uint32_t ph = (j / STAGES) & 1u;
        if (!mbar_wait(full_bar(s), ph, abort_flag, false, WAIT_CYCLES / 8)) atomicExch(a.status, 2);
      }
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------------ MMA issuer
    if (lane == 0) {
      constexpr uint32_t idesc = make_idesc(NN, BM, BN);
      uint32_t it = 0, tile_it = 0;
      bool ok = true;
      for (int t = blockIdx.x; t < total_tiles && ok; t += gridDim.x, ++tile_it) {
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
            tc_mma(d_tmem, ad, bd, idesc, (kb > 0 || k > 0) ? 1u : 0u);
          }
          tc_commit(empty_bar(s));             // stage reusable once these MMAs have read it
        }
        if (ok) tc_commit(tfull_bar(int(acc)));  // accumulator complete
      }
      if (!ok) {
        *abort_flag = 1;
        atomicExch(a.status, 3);
      }
    }
  } else {
    // ------------------------------------------------------------------ epilogue warps
    const int quad = warp & 3;                     // TMEM lane quadrant this warp may read
    EpilogueState est;
    uint32_t tile_it = 0;
    bool ok = true;
    auto epi_of = [&](const Tile& tl) {
      EpiTile e;
      e.map_d = &map_d; e.map_c = &map_c;
      e.d = a.d; e.c = a.c;
      e.stride_c = a.stride_c;
      e.ldc = a.ldc; e.m = a.m; e.n = a.n;
      e.mat = tl.mat;
      e.rblk = tl.m0 / BM;
      e.cblk0 = tl.n0 / 128;
      e.cblk1 = tl.n0 + 128 < a.n ? tl.n0 / 128 + 1 : -1;
      e.mirror0 = e.mirror1 = a.symmetric && tl.n0 >= tl.m0 + BM;       // tile lies strictly above the diagonal
      e.alpha = a.alpha; e.beta = a.beta; e.diag = a.diag; e.gamma = 1.f;
      if (a.coef) {
        const float* co = a.coef + size_t(tl.mat) * size_t(a.coef_stride);
        if (a.coef_a >= 0) e.alpha = co[a.coef_a];
        if (a.coef_b >= 0) e.beta = co[a.coef_b];
        if (a.coef_d >= 0) e.diag = co[a.coef_d];
      }
      if (a.gamma_mode) {
        const float r = a.rnorm[tl.mat];
        e.gamma = a.gamma_mode == 1 ? r : r * r;
      }
      e.valid = true;
      return e;
    };
    for (int t = blockIdx.x; t < total_tiles && ok; t += gridDim.x, ++tile_it) {
      const uint32_t acc = tile_it & 1u, aph = (tile_it >> 1) & 1u;
      const uint32_t taddr = tmem_base + acc * uint32_t(BN) + (uint32_t(quad * 32) << 16);
      const EpiTile cur = epi_of(decode_tile(t, a));
      EpiTile nxt;
      nxt.valid = false;
      nxt.d = nullptr;
      if (t + int(gridDim.x) < total_tiles) nxt = epi_of(decode_tile(t + int(gridDim.x), a));
      ok = epilogue_tile<1>(cur, nxt, taddr, epi_base, dfull_bar(0), egroup_bar, tfull_bar(int(acc)), aph, abort_flag, est, quad,
                            lane, 0, quad == 2 && lane == 0);
      if (!ok) break;
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(tempty_bar(int(acc)));
    }
    if (quad == 2 && lane == 0) {
      tma_wait_all();                               // every store has landed before the CTA retires
      if (!ok)                                      // a prefetched D chunk may still be landing: give it (bounded) time
        for (int i = 0; i < 64; ++i) __nanosleep(1000);
    }
    if (!ok && lane == 0) {
      *abort_flag = 1;
      atomicExch(a.status, 4);
    }
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  if (warp == 1) {
    __syncwarp();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(TMEM_COLS) : "memory");
  }
}

// ------------------------------------------------------------------ host side
// Per device ordinal: shared-memory attribute set and SM count looked up once.
constexpr int kMaxDevices = 64;
int g_num_sms[kMaxDevices] = {};

// A wait that nothing ever satisfies, with a short limit: exercises the bounded-wait machinery (deadline,
// status word, clean return) without putting any real pipeline at risk.
__global__ void bounded_wait_probe_kernel(int32_t* status, long long limit_cycles) {
  __shared__ alignas(8) uint64_t bar;
  __shared__ int abort_flag;
  if (threadIdx.x == 0) {
    mbar_init(smem_u32(&bar), 1);
    abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  __syncthreads();
  if (threadIdx.x == 0) {
    const bool done = mbar_wait(smem_u32(&bar), 0, &abort_flag, true, limit_cycles);   // nobody arrives: must expire
    if (!done) atomicExch(status, 100);
  }
}

}  // namespace

int launch_bounded_wait_probe(muon_ctx* ctx, cudaStream_t st) {
  bounded_wait_probe_kernel<<<1, 32, 0, st>>>(ctx->d_status, 2000000LL);   // about a millisecond
  return cudaGetLastError() == cudaSuccess ? 1 : MUON_ERR_CUDA;
}

bool tc_supported(const GemmArgs& a) {
  if (a.m < 1 || a.n < 1 || a.kdim < 1 || a.batch < 1) return false;
  // tensor-map strides must be multiples of 16 bytes, bases 16-byte aligned
  if ((a.ldp % 8) || (a.ldq % 8) || (a.ldc % 8) || (a.stride_p % 8) || (a.stride_q % 8) || (a.stride_c % 8)) return false;
  if ((reinterpret_cast<uintptr_t>(a.p) | reinterpret_cast<uintptr_t>(a.q) | reinterpret_cast<uintptr_t>(a.c) |
       reinterpret_cast<uintptr_t>(a.d)) & 15u)
    return false;
  if (a.symmetric && (a.nn || a.m != a.n || a.p != a.q || a.ldp != a.ldq || a.stride_p != a.stride_q)) return false;
  const int64_t tiles = int64_t((a.m + BM - 1) / BM) * ((a.n + BN - 1) / BN) * a.batch;
  return tiles < (int64_t(1) << 30);
}

int launch_gemm_tc(muon_ctx* ctx, const GemmArgs& a, cudaStream_t st) {
  if (!ctx->tmap_encode) return MUON_ERR_CUDA;
  if (ctx->device < 0 || ctx->device >= kMaxDevices) return MUON_ERR_UNSUPPORTED;
  if (!g_num_sms[ctx->device]) {
    if (cudaFuncSetAttribute(ns_product_tc_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, SMEM_BYTES) != cudaSuccess ||
        cudaFuncSetAttribute(ns_product_tc_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, SMEM_BYTES) != cudaSuccess)
      return MUON_ERR_CUDA;
    cudaDeviceProp prop;
    if (cudaGetDeviceProperties(&prop, ctx->device) != cudaSuccess) return MUON_ERR_CUDA;
    g_num_sms[ctx->device] = prop.multiProcessorCount;
  }
  CUtensorMap map_p, map_q;
  // P: rows = m, cols = kdim
  if (!encode_map(ctx->tmap_encode, &map_p, a.p, a.kdim, a.m, a.batch, a.ldp, a.stride_p, BM)) return MUON_ERR_CUDA;
  if (!a.nn) {  // Q: rows = n, cols = kdim; two 128-row boxes per stage
    if (!encode_map(ctx->tmap_encode, &map_q, a.q, a.kdim, a.n, a.batch, a.ldq, a.stride_q, 128)) return MUON_ERR_CUDA;
  } else {      // Q: rows = kdim, cols = n; four 64(k) x 64(n) boxes per stage
    if (!encode_map(ctx->tmap_encode, &map_q, a.q, a.n, a.kdim, a.batch, a.ldq, a.stride_q, BK)) return MUON_ERR_CUDA;
  }
  // C (store) and D (load) chunks: 128 rows x 64 columns
  CUtensorMap map_c, map_d;
  if (!encode_map(ctx->tmap_encode, &map_c, a.c, a.n, a.m, a.batch, a.ldc, a.stride_c, BM)) return MUON_ERR_CUDA;
  if (!encode_map(ctx->tmap_encode, &map_d, a.d ? a.d : a.c, a.n, a.m, a.batch, a.ldc, a.stride_c, BM)) return MUON_ERR_CUDA;
  ctx->tmap_encodes += 4;
  TcArgs t;
  t.d = static_cast<const __nv_bfloat16*>(a.d);
  t.c = static_cast<__nv_bfloat16*>(a.c);
  t.m = a.m; t.n = a.n; t.kdim = a.kdim; t.ldc = a.ldc;
  t.stride_c = a.stride_c;
  t.batch = a.batch;
  t.tiles_m = (a.m + BM - 1) / BM;
  t.tiles_n = (a.n + BN - 1) / BN;
  t.symmetric = a.symmetric ? 1 : 0;
  t.tiles_per_mat = t.tiles_m * t.tiles_n;
  if (t.symmetric) {
    int cnt = 0;
    for (int i = 0; i < t.tiles_m; ++i) cnt += t.tiles_n - i / 2;
    t.tiles_per_mat = cnt;
  }
  t.rnorm = a.rnorm;
  t.gamma_mode = a.gamma_mode;
  t.alpha = a.alpha; t.beta = a.beta; t.diag = a.diag;
  t.coef = a.coef; t.coef_a = a.coef_a; t.coef_b = a.coef_b; t.coef_d = a.coef_d; t.coef_stride = a.coef_stride;
  t.status = ctx->d_status;
  const int64_t tiles = int64_t(t.tiles_per_mat) * t.batch;
  const unsigned grid = unsigned(tiles < g_num_sms[ctx->device] ? tiles : g_num_sms[ctx->device]);
  if (a.nn) ns_product_tc_kernel<true><<<grid, NUM_THREADS, SMEM_BYTES, st>>>(map_p, map_q, map_d, map_c, t);
  else ns_product_tc_kernel<false><<<grid, NUM_THREADS, SMEM_BYTES, st>>>(map_p, map_q, map_d, map_c, t);
  return cudaGetLastError() == cudaSuccess ? 1 : MUON_ERR_CUDA;
}

}  // namespace muon
