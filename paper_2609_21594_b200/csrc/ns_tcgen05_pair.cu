// Paired-CTA tensor-core engine for the Newton-Schulz products (Eq. 1), grouped over heterogeneous
// shapes: ONE launch computes the same product (A = X X^T, P = aI + bA + cA A^T or X' = P X) for every
// shape group that is resident in the workspace (the shape-fused batching of Section 6.6, taken one
// step further: not one batched kernel per core shape but one per product for all core shapes).
//
//   C[k] = gamma_k * (beta * D[k] + alpha * P[k] Q[k]^T + diag * I)   (nn = 0)      C[k] = ... P[k] Q[k]   (nn = 1)
//
// The launch reads a table of problems from global memory (tensor maps encoded once per plan, shapes,
// tile counts) and walks one global tile list with persistent clusters of two CTAs.  A tile is given in
// 128-row / 128-column blocks: CTA r of the pair owns row block (ra, rb)[r] and loads those 128 rows of P;
// the tile spans column blocks cc and cd (N = 256) or cc alone (N = 128), and CTA r stages half of the
// N columns of Q per 64-wide k-block.  The leader (r = 0) issues tcgen05.mma.cta_group::2 of shape
// M256 x N x K16; each CTA keeps its 128 x N fp32 accumulator in its own TMEM (double-buffered) and runs
// its own epilogue with eight warps (two per TMEM lane quadrant, each converting half of every 64-column
// chunk: the epilogue of a tile is a chain of latencies, and tiles with few k-blocks wait for it).
// Symmetric products (P = Q, C = C^T) come with an explicit per-matrix tile list over the block triangle
// (2 x 2 block tiles, a ragged last column block gets 128-wide tiles); a symmetric result is stored only
// where tiles compute it and read transposed where a consumer needs the other half.
//
// Synchronisation (all waits bounded):
//   full[s]    leader only.  The leader's producer arms it with the bytes of BOTH CTAs; both producers'
//              TMA loads complete on it (cta_group::2 form, no multicast).
//   empty[s]   in each CTA; the leader's tcgen05.commit arrives on both (commit multicast).
//   tfull[a]   in each CTA; commit multicast after a tile's last k-block.
//   tempty[a]  leader only, 16 arrivals: the eight epilogue warps of each CTA (remote arrive).
//   drain      in each CTA; the issuer's last commit, awaited before TMEM is freed.
// A role that gives up sets the abort flag of BOTH CTAs (remote store), records a code in the status word
// and leaves; everybody else notices the flag inside its own bounded wait.
#include "tc_common.cuh"

namespace muon {
namespace {

using namespace tc;

constexpr int BM = 128;          // rows per CTA; the pair covers 256
constexpr int BK = 64;
constexpr int UK = 16;
#ifndef MUON_PAIR_STAGES
#define MUON_PAIR_STAGES 5
#endif
constexpr int STAGES = MUON_PAIR_STAGES;
constexpr int A_BYTES = BM * BK * 2;          // 16 KiB: this CTA's rows of P
constexpr int B_BYTES = 128 * BK * 2;         // 16 KiB: this CTA's half of the Q tile
constexpr int STAGE_BYTES = A_BYTES + B_BYTES;
constexpr int SMEM_BYTES = STAGES * STAGE_BYTES + EPI_BUFS * EPI_BYTES + 1024 + 256;
constexpr int TMEM_COLS = 512;
constexpr int EPI_SPLIT = 2;                      // epilogue warps per TMEM lane quadrant
constexpr int EPI_WARPS = 4 * EPI_SPLIT;
constexpr int NUM_THREADS = 64 + 32 * EPI_WARPS;   // warp 0: TMA producer, warp 1: MMA issuer, then the epilogue warps
// constant parts of the shared-memory matrix descriptors (see make_desc): K-major (LBO 16, SBO 1024) and
// MN-major (LBO 8 KiB between 64-element chunks, SBO 1024), 128-byte swizzle
constexpr uint64_t DESC_HI_K = (uint64_t(16 >> 4) << 16) | (uint64_t(1024 >> 4) << 32) | (uint64_t(1) << 46) | (uint64_t(2) << 61);
constexpr uint64_t DESC_HI_MN =
    (uint64_t((64 * BK * 2) >> 4) << 16) | (uint64_t(1024 >> 4) << 32) | (uint64_t(1) << 46) | (uint64_t(2) << 61);

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
__device__ __forceinline__ void st_cluster_u32(uint32_t cluster_addr, uint32_t v) {
  asm volatile("st.shared::cluster.u32 [%0], %1;" ::"r"(cluster_addr), "r"(v) : "memory");
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
  int prob;      // index into the launch's problem list
  int mat;
  int ra, rb;    // row block of CTA 0 / CTA 1 (rb = -1: none)
  int cc, cd;    // column blocks (cd = -1: the tile is 128 columns wide)
};

// What one product of the launch looks like to the kernel: its problem list and its epilogue scalars.
struct PhaseView {
  const TcMaps* maps;
  const TcProbInfo* info;
  int nprob, total_tiles;
  float alpha, beta, diag;
  int gamma_mode;
  int coef_a, coef_b, coef_d, coef_off;   // per-matrix coefficient rows: see TcLaunch
};

// Product `ph` of the launch.  A one-product launch carries its tables by value; a whole-iteration launch reads
// them from device memory and derives the scalars of step k = ph / 3 from the coefficient rows:
// A = gamma X X^T (gamma = r^2 at k = 0), P = a I + b A + c A A^T, X' = gamma P X (gamma = r at k = 0).
__device__ __forceinline__ PhaseView phase_view(const TcLaunch& L, int ph) {
  PhaseView v;
  if (!L.persist) {
    v.maps = L.maps; v.info = L.info; v.nprob = L.nprob; v.total_tiles = L.total_tiles;
    v.alpha = L.alpha; v.beta = L.beta; v.diag = L.diag; v.gamma_mode = L.gamma_mode;
    v.coef_a = L.coef_a; v.coef_b = L.coef_b; v.coef_d = L.coef_d; v.coef_off = L.coef_off;
    return v;
  }
  const int k = ph / 3, j = ph - 3 * k, cur = k & 1;
  const int kind = j == 0 ? cur : (j == 1 ? 2 : 3 + cur);
  v.maps = L.persist->maps[kind];
  v.info = L.persist->info[kind];
  v.nprob = L.persist->nprob;
  v.total_tiles = L.persist->total_tiles[kind];
  v.alpha = j == 1 ? L.coef[k][2] : 1.f;
  v.beta = j == 1 ? L.coef[k][1] : 0.f;
  v.diag = j == 1 ? L.coef[k][0] : 0.f;
  v.gamma_mode = k == 0 ? (j == 0 ? 2 : (j == 2 ? 1 : 0)) : 0;
  v.coef_a = j == 1 ? 2 : -1;
  v.coef_b = j == 1 ? 1 : -1;
  v.coef_d = j == 1 ? 0 : -1;
  v.coef_off = L.coef_per_step ? 3 * k : 0;
  return v;
}

__device__ __forceinline__ Tile decode_tile(int t, const PhaseView& V) {
  int pi = 0;
  for (int i = 1; i < V.nprob; ++i)
    if (t >= V.info[i].tile_begin) pi = i;
  const TcProbInfo& p = V.info[pi];
  Tile r;
  r.prob = pi;
  const int u = t - p.tile_begin;
  r.mat = u / p.tiles_per_mat;
  const int v = u - r.mat * p.tiles_per_mat;
  if (p.pattern) {
    const uint2 raw = __ldg(reinterpret_cast<const uint2*>(p.pattern + v));
    const uint32_t ra = raw.x & 0xffffu, rb = raw.x >> 16, cc = raw.y & 0xffffu, cd = raw.y >> 16;
    r.ra = int(ra);
    r.rb = rb == kNoBlock ? -1 : int(rb);
    r.cc = int(cc);
    r.cd = cd == kNoBlock ? -1 : int(cd);
  } else {   // dense: row pairs vary fastest, so concurrent pairs share the Q tile
    const int j = v / p.row_pairs, i = v - j * p.row_pairs;
    r.ra = 2 * i;
    r.rb = 2 * i + 1 < p.rblocks ? 2 * i + 1 : -1;
    r.cc = 2 * j;
    r.cd = 2 * j + 1 < p.cblocks ? 2 * j + 1 : -1;
  }
  return r;
}

__device__ __forceinline__ EpiTile make_epi(const Tile& tl, int rank, const PhaseView& V, const TcLaunch& L) {
  EpiTile e;
  const TcProbInfo& p = V.info[tl.prob];
  e.map_d = &V.maps[tl.prob].d;
  e.map_c = &V.maps[tl.prob].c;
  e.d = p.d;
  e.c = p.c;
  e.stride_c = p.stride_c;
  e.ldc = p.ldc; e.m = p.m; e.n = p.n;
  e.mat = tl.mat;
  e.rblk = rank ? tl.rb : tl.ra;
  e.cblk0 = tl.cc; e.cblk1 = tl.cd;
  const bool sym = p.symmetric != 0 && p.mirror_out != 0;
  // when the whole of a symmetric result is wanted, a block (r, c) is also written as (c, r) unless it lies on
  // the diagonal or this very tile computes (c, r) itself (the diagonal 2 x 2 tiles)
  const bool in_cols = e.rblk == tl.cc || e.rblk == tl.cd;
  e.mirror0 = sym && tl.cc != e.rblk && !(in_cols && (tl.cc == tl.ra || tl.cc == tl.rb));
  e.mirror1 = sym && tl.cd != e.rblk && !(in_cols && (tl.cd == tl.ra || tl.cd == tl.rb));
  e.valid = e.rblk >= 0;
  e.alpha = V.alpha; e.beta = V.beta; e.diag = V.diag; e.gamma = 1.f;
  if (e.valid) {
    if (V.gamma_mode) {
      const float r = p.rnorm[tl.mat];
      e.gamma = V.gamma_mode == 1 ? r : r * r;
    }
    if (L.coef_table) {
      const float* co = L.coef_table + size_t(p.mat_begin + tl.mat) * size_t(L.coef_stride) + V.coef_off;
      if (V.coef_a >= 0) e.alpha = __ldg(co + V.coef_a);
      if (V.coef_b >= 0) e.beta = __ldg(co + V.coef_b);
      if (V.coef_d >= 0) e.diag = __ldg(co + V.coef_d);
    }
  }
  return e;
}

// Grid-wide barrier of the whole-iteration launch (all CTAs are resident: cooperative launch).  Arrival: one
// thread per CTA, after its bulk stores have completed, publishes them and adds 1.  Wait: poll (bounded) until
// every CTA has arrived for product `ph - 1`, then order the bulk loads that follow behind the acquire.
__device__ __forceinline__ void grid_arrive(uint32_t* counter) {
  asm volatile("fence.proxy.async;" ::: "memory");
  __threadfence();
  atomicAdd(counter, 1u);
}
__device__ __forceinline__ bool grid_wait(const TcLaunch& L, int ph, volatile int* abort_flag) {
  const uint32_t target = L.barrier_base + uint32_t(ph) * gridDim.x;
  const long long t0 = clock64();
  uint32_t spins = 0;
  while (true) {
    uint32_t v;
    asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(L.barrier) : "memory");
    if (int32_t(v - target) >= 0) break;
    if ((++spins & 63u) == 0) {
      if (*abort_flag) return false;
      if (clock64() - t0 > WAIT_CYCLES) return false;
    }
  }
  asm volatile("fence.proxy.async;" ::: "memory");
  return true;
}

// ---- main-loop bodies, specialised at compile time on how the two operands are read (K-major as stored, or
// MN-major = transposed): the producer and the MMA issuer are single threads whose loop must stay short, so
// a tile's k-range is cut into at most three pieces with fixed operand forms instead of deciding per k-block.
struct LoopCtx {
  uint32_t base, bars;          // shared-memory addresses of the stage ring and of the barrier block
  volatile int* abort_flag;
  uint32_t it;                  // k-blocks processed so far by this role
  uint32_t s, ph;               // ring position and phase of k-block `it` (kept incrementally: no division in the loop)
  uint32_t full0_leader;        // cluster address of the leader CTA's full[0] barrier
  __device__ __forceinline__ void advance() {
    ++it;
    if (++s == uint32_t(STAGES)) {
      s = 0;
      ph ^= 1u;
    }
  }
};
__device__ __forceinline__ uint32_t full_bar_of(const LoopCtx& c, int s) { return c.bars + uint32_t(s) * 8u; }
__device__ __forceinline__ uint32_t empty_bar_of(const LoopCtx& c, int s) { return c.bars + uint32_t(STAGES + s) * 8u; }

struct LoadArgs {
  const TcMaps* mp;
  int mat, prow, qcol;
  uint32_t stage_tx;
  bool leader_cta, narrow;
};

// ALIAS: a diagonal tile of a symmetric product (column blocks == row blocks): each CTA's half of Q is its own P tile,
// so Q is not loaded at all and the MMA reads both operands from the P buffer.
template <bool A_MN, bool B_MN, bool ALIAS>
__device__ __forceinline__ bool produce_range(LoopCtx& c, const LoadArgs& a, int kb_begin, int kb_end) {
  for (int kb = kb_begin; kb < kb_end; ++kb, c.advance()) {
    const int s = int(c.s);
    if (!mbar_wait(empty_bar_of(c, s), c.ph ^ 1u, c.abort_flag)) return false;
    const uint32_t sa = c.base + uint32_t(s) * STAGE_BYTES, sb = sa + A_BYTES;
    if (a.leader_cta) mbar_expect_tx(full_bar_of(c, s), a.stage_tx);
    const uint32_t fb = c.full0_leader + uint32_t(s) * 8u;
    const int k0 = kb * BK;
    if (!A_MN) {                                   // 128 rows of P x 64 k
      tma_load_3d_pair(sa, &a.mp->p, fb, k0, a.prow, a.mat);
    } else {                                       // the same block read from its mirror image: 64 k-rows x 64 columns, twice
      tma_load_3d_pair(sa, &a.mp->ph, fb, a.prow, k0, a.mat);
      tma_load_3d_pair(sa + 64 * BK * 2, &a.mp->ph, fb, a.prow + 64, k0, a.mat);
    }
    if (ALIAS) continue;
    if (!B_MN) {                                   // 128 rows of Q, or the 64 a 128-wide tile needs
      tma_load_3d_pair(sb, a.narrow ? &a.mp->qh : &a.mp->q, fb, k0, a.qcol, a.mat);
    } else {                                       // 64 k-rows x 64 columns, twice for a 256-wide tile
      tma_load_3d_pair(sb, &a.mp->qh, fb, a.qcol, k0, a.mat);
      if (!a.narrow) tma_load_3d_pair(sb + 64 * BK * 2, &a.mp->qh, fb, a.qcol + 64, k0, a.mat);
    }
  }
  return true;
}

// A shared-memory descriptor is a constant high part (layout, strides) plus the start address in 16-byte units.
// K-major: 16 k = 32 bytes along a 128-byte row; MN-major: 16 k-rows of 128 bytes each.
template <bool A_MN, bool B_MN>
__device__ __forceinline__ bool issue_range(LoopCtx& c, uint32_t d_tmem, uint32_t idesc_base, uint32_t b_off, int kb_begin,
                                            int kb_end) {
  constexpr uint32_t idesc_major = (A_MN ? 1u << 15 : 0u) | (B_MN ? 1u << 16 : 0u);
  constexpr uint64_t a_hi = A_MN ? DESC_HI_MN : DESC_HI_K, b_hi = B_MN ? DESC_HI_MN : DESC_HI_K;
  constexpr uint32_t a_step = A_MN ? (UK * 128) >> 4 : (UK * 2) >> 4, b_step = B_MN ? (UK * 128) >> 4 : (UK * 2) >> 4;
  const uint32_t idesc = idesc_base | idesc_major;
  for (int kb = kb_begin; kb < kb_end; ++kb, c.advance()) {
    const int s = int(c.s);
    if (!mbar_wait(full_bar_of(c, s), c.ph, c.abort_flag)) return false;
    tc_fence_after();
    const uint32_t a0 = (c.base + uint32_t(s) * STAGE_BYTES) >> 4, b0 = a0 + b_off;
#pragma unroll
    for (int k = 0; k < BK / UK; ++k)
      tc_mma_pair(d_tmem, a_hi | uint64_t(a0 + uint32_t(k) * a_step), b_hi | uint64_t(b0 + uint32_t(k) * b_step), idesc,
                  (kb > 0 || k > 0) ? 1u : 0u);
    tc_commit_pair(empty_bar_of(c, s));
  }
  return true;
}

// k-blocks [0, p_flip) read P transposed, [0, q_flip) read Q transposed: three pieces with fixed forms.
#define MUON_FOR_K_PIECES(CALL)                                                              \
  {                                                                                          \
    const int lo_ = p_flip_kb < q_flip_kb ? p_flip_kb : q_flip_kb;                           \
    const int hi_ = p_flip_kb < q_flip_kb ? q_flip_kb : p_flip_kb;                           \
    if (ok && lo_ > 0) ok = CALL(true, true, 0, lo_);                                        \
    if (ok && hi_ > lo_) ok = p_flip_kb > q_flip_kb ? CALL(true, false, lo_, hi_) : CALL(false, true, lo_, hi_); \
    if (ok && num_kb > hi_) ok = CALL(false, false, hi_, num_kb);                            \
  }

__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(NUM_THREADS, 1)
ns_product_pair_kernel(const __grid_constant__ TcLaunch L) {
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
  const uint32_t drain_bar = bars + uint32_t(2 * STAGES + 5 + EPI_BUFS) * 8u;

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const uint32_t rank = cluster_rank();
  const bool leader_cta = rank == 0;
  const int pair_id = blockIdx.x >> 1, num_pairs = gridDim.x >> 1;
  const int nphase = L.persist ? 3 * L.ns_steps : 1;      // products this launch walks through
  const uint32_t peer_abort = map_to_cta(base + BAR_OFF + 200, rank ^ 1u);
  auto give_up = [&](int code) {                 // tell both CTAs of the pair, then the host
    *abort_flag = 1;
    st_cluster_u32(peer_abort, 1u);
    atomicExch(L.status, code);
  };

  if (threadIdx.x == 0) {
    for (int s = 0; s < STAGES; ++s) {
      mbar_init(full_bar(s), 1);
      mbar_init(empty_bar(s), 1);
    }
    for (int i = 0; i < 2; ++i) {
      mbar_init(tfull_bar(i), 1);
      mbar_init(tempty_bar(i), 2 * EPI_WARPS);     // every epilogue warp of both CTAs
    }
    for (int i = 0; i < EPI_BUFS; ++i) mbar_init(dfull_bar(i), 1);
    mbar_init(egroup_bar, EPI_WARPS);
    mbar_init(drain_bar, 1);
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
      LoopCtx lc{base, bars, abort_flag, 0u, 0u, 0u, map_to_cta(full_bar(0), 0)};
      bool ok = true;
      for (int ph = 0; ph < nphase && ok; ++ph) {
        const PhaseView V = phase_view(L, ph);
        if (ph > 0 && !grid_wait(L, ph, abort_flag)) { ok = false; break; }   // operands written by the product before
        for (int t = pair_id; t < V.total_tiles && ok; t += num_pairs) {
          const Tile tl = decode_tile(t, V);
          const TcProbInfo& p = V.info[tl.prob];
          const TcMaps* mp = &V.maps[tl.prob];
          const bool nn = p.nn != 0;
          const bool narrow = tl.cd < 0;
          const int num_kb = (p.kdim + BK - 1) / BK;
          // this CTA's 128 rows of P (a missing row block reads beyond the matrix: zero fill)
          const int rblk = rank ? tl.rb : tl.ra;
          const int prow = rblk >= 0 ? rblk * BM : p.rblocks * BM;
          // this CTA's half of the N columns: a whole column block of a 256-wide tile, half a block of a 128-wide one
          const int qcol = narrow ? tl.cc * 128 + int(rank) * 64 : (rank ? tl.cd : tl.cc) * 128;
          LoadArgs la;
          la.mp = mp; la.mat = tl.mat; la.prow = prow; la.qcol = qcol;
          const bool alias = p.symmetric != 0 && !nn && !narrow && tl.cc == tl.ra && tl.cd == tl.rb;
          la.stage_tx = alias ? 2 * A_BYTES : (narrow ? 2 * (A_BYTES + B_BYTES / 2) : 2 * STAGE_BYTES);
          la.leader_cta = leader_cta; la.narrow = narrow;
          // half-stored symmetric operands: k-blocks left of the tile's own block pair are read transposed
          int p_flip_kb = p.p_half ? (tl.ra >> 1) * 4 : 0;            // k-blocks [0, p_flip_kb) of P come MN-major
          int q_flip_kb = nn ? num_kb : (p.q_half ? (tl.cc >> 1) * 4 : 0);
          p_flip_kb = p_flip_kb < num_kb ? p_flip_kb : num_kb;
          q_flip_kb = q_flip_kb < num_kb ? q_flip_kb : num_kb;
#define MUON_PRODUCE(AM, BM_, B0, B1) \
  (alias ? produce_range<AM, BM_, true>(lc, la, B0, B1) : produce_range<AM, BM_, false>(lc, la, B0, B1))
          MUON_FOR_K_PIECES(MUON_PRODUCE)
#undef MUON_PRODUCE
        }
      }
      if (!ok) give_up(11);
      if (leader_cta) {   // every armed stage (both CTAs' bytes) has landed before shared memory is released
        const uint32_t issued = lc.it;
        for (uint32_t j = (issued > STAGES ? issued - STAGES : 0); j < issued; ++j) {
          const int s = int(j % STAGES);
          const uint32_t ph = (j / STAGES) & 1u;
          if (!mbar_wait(full_bar(s), ph, abort_flag, false, WAIT_CYCLES / 8)) atomicExch(L.status, 12);
        }
      }
      if (*abort_flag)    // loads this CTA issued for a stage the leader never armed: give them time to land
        for (int i = 0; i < 64; ++i) __nanosleep(1000);
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------------ MMA issuer (leader CTA only)
    if (lane == 0) {
      if (leader_cta) {
        LoopCtx lc{base, bars, abort_flag, 0u, 0u, 0u, 0u};
        uint32_t tile_it = 0;
        bool ok = true;
        for (int ph = 0; ph < nphase && ok; ++ph) {       // no barrier here: the issuer only consumes what the producers loaded
          const PhaseView V = phase_view(L, ph);
          for (int t = pair_id; t < V.total_tiles && ok; t += num_pairs, ++tile_it) {
            const Tile tl = decode_tile(t, V);
            const TcProbInfo& p = V.info[tl.prob];
            const bool nn = p.nn != 0;
            const int num_kb = (p.kdim + BK - 1) / BK;
            const uint32_t idesc_base = make_idesc(false, 2 * BM, tl.cd >= 0 ? 256 : 128);
            int p_flip_kb = p.p_half ? (tl.ra >> 1) * 4 : 0;
            int q_flip_kb = nn ? num_kb : (p.q_half ? (tl.cc >> 1) * 4 : 0);
            p_flip_kb = p_flip_kb < num_kb ? p_flip_kb : num_kb;
            q_flip_kb = q_flip_kb < num_kb ? q_flip_kb : num_kb;
            // diagonal tile of a symmetric product: Q was not loaded, both operands come from the P buffer
            const bool alias = p.symmetric != 0 && !nn && tl.cd >= 0 && tl.cc == tl.ra && tl.cd == tl.rb;
            const uint32_t b_off = alias ? 0u : uint32_t(A_BYTES >> 4);
            const uint32_t acc = tile_it & 1u, aph = (tile_it >> 1) & 1u;
            if (!mbar_wait(tempty_bar(int(acc)), aph ^ 1u, abort_flag)) { ok = false; break; }
            tc_fence_after();
            const uint32_t d_tmem = tmem_base + acc * 256u;
#define MUON_ISSUE(AM, BM_, B0, B1) issue_range<AM, BM_>(lc, d_tmem, idesc_base, b_off, B0, B1)
            MUON_FOR_K_PIECES(MUON_ISSUE)
#undef MUON_ISSUE
            if (ok) tc_commit_pair(tfull_bar(int(acc)));
          }
        }
        if (!ok) give_up(13);
        tc_commit_pair(drain_bar);       // arrives in both CTAs once every MMA issued above has finished
      }
      if (!mbar_wait(drain_bar, 0, abort_flag, false, WAIT_CYCLES / 8)) atomicExch(L.status, 15);
    }
  } else {
    // ------------------------------------------------------------------ epilogue warps (per CTA: its 128 rows)
    const int quad = warp & 3;                     // TMEM lane quadrant this warp may read
    const int part = (warp - 2) >> 2;              // which share of a chunk's columns this warp converts
    const bool epi_leader = warp == 2 && lane == 0;
    EpilogueState est;
    uint32_t tile_it = 0;
    bool ok = true;
    for (int ph = 0; ph < nphase && ok; ++ph) {
      const PhaseView V = phase_view(L, ph);
      if (ph > 0) {                                 // D chunks and result tiles of this product touch what the last one wrote
        bool go = true;
        if (lane == 0) go = grid_wait(L, ph, abort_flag);
        if (!__shfl_sync(0xffffffffu, go ? 1 : 0, 0)) { ok = false; break; }
      }
      bool have = pair_id < V.total_tiles;
      EpiTile cur, nxt;                             // each tile is decoded once: `nxt` becomes `cur`
      if (have) nxt = make_epi(decode_tile(pair_id, V), int(rank), V, L);
      for (int t = pair_id; have && ok; t += num_pairs, ++tile_it) {
        const uint32_t acc = tile_it & 1u, aph = (tile_it >> 1) & 1u;
        const uint32_t taddr = tmem_base + acc * 256u + (uint32_t(quad * 32) << 16);
        cur = nxt;
        nxt.valid = false;
        nxt.d = nullptr;
        have = t + num_pairs < V.total_tiles;       // the prefetch of D never crosses a product boundary
        if (have) nxt = make_epi(decode_tile(t + num_pairs, V), int(rank), V, L);
        if (cur.valid) {
          ok = epilogue_tile<EPI_SPLIT>(cur, nxt, taddr, epi_base, dfull_bar(0), egroup_bar, tfull_bar(int(acc)), aph, abort_flag,
                                        est, quad, lane, part, epi_leader);
        } else {                                    // no rows for this CTA: hand the accumulator straight back
          ok = mbar_wait(tfull_bar(int(acc)), aph, abort_flag);
        }
        if (!ok) break;
        tc_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive_cluster(map_to_cta(tempty_bar(int(acc)), 0));   // the leader CTA counts both epilogues
      }
      if (ok && L.persist && ph + 1 < nphase) {     // this CTA's part of the product is in memory: tell the grid
        // the four warps meet first, so that every store of the product has been issued by the leader thread
        __syncwarp();
        if (lane == 0) mbar_arrive(egroup_bar);
        ok = mbar_wait(egroup_bar, est.eph, abort_flag);
        est.eph ^= 1u;
        if (ok && epi_leader) {
          tma_wait_all();
          grid_arrive(L.barrier);
        }
      }
    }
    if (epi_leader) {
      tma_wait_all();                               // every store has landed before the CTA retires
      if (!ok)                                      // a prefetched D chunk may still be landing: give it (bounded) time
        for (int i = 0; i < 64; ++i) __nanosleep(1000);
    }
    if (!ok && lane == 0) give_up(14);
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

int tc_pair_grid_setup(int device) {
  if (device < 0 || device >= kMaxDevices) return MUON_ERR_UNSUPPORTED;
  if (!g_num_sms[device]) {
    if (cudaFuncSetAttribute(ns_product_pair_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, SMEM_BYTES) != cudaSuccess)
      return MUON_ERR_CUDA;
    int sms = 0;
    if (cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, device) != cudaSuccess || sms < 2) return MUON_ERR_CUDA;
    g_num_sms[device] = sms;
  }
  return g_num_sms[device];
}

int launch_tc_grouped(int device, const tc::TcLaunch& L, cudaStream_t st) {
  if (L.total_tiles <= 0) return 0;
  const int sms = tc_pair_grid_setup(device);
  if (sms < 0) return sms;
  const int64_t pairs = sms / 2;
  const unsigned grid = unsigned(2 * (L.total_tiles < pairs ? L.total_tiles : pairs));
  ns_product_pair_kernel<<<grid, NUM_THREADS, SMEM_BYTES, st>>>(L);
  return cudaGetLastError() == cudaSuccess ? 1 : MUON_ERR_CUDA;
}

int tc_pair_max_resident(int device) {
  if (tc_pair_grid_setup(device) < 0) return 0;
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(2, 1, 1);
  cfg.blockDim = dim3(NUM_THREADS, 1, 1);
  cfg.dynamicSmemBytes = SMEM_BYTES;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeClusterDimension;
  attr[0].val.clusterDim.x = 2;
  attr[0].val.clusterDim.y = 1;
  attr[0].val.clusterDim.z = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  int clusters = 0;
  if (cudaOccupancyMaxActiveClusters(&clusters, ns_product_pair_kernel, &cfg) != cudaSuccess) {
    cudaGetLastError();
    return 0;
  }
  return clusters;
}

int launch_tc_persistent(int device, const tc::TcLaunch& L, int pairs, cudaStream_t st) {
  if (!L.persist || pairs < 1) return MUON_ERR_INVALID_ARG;
  if (tc_pair_grid_setup(device) < 0) return MUON_ERR_CUDA;
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(unsigned(2 * pairs), 1, 1);
  cfg.blockDim = dim3(NUM_THREADS, 1, 1);
  cfg.dynamicSmemBytes = SMEM_BYTES;
  cfg.stream = st;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeCooperative;      // every CTA resident at once: the grid barrier relies on it
  attr[0].val.cooperative = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  if (cudaLaunchKernelEx(&cfg, ns_product_pair_kernel, L) != cudaSuccess) {
    cudaGetLastError();
    return MUON_ERR_UNSUPPORTED;
  }
  return 1;
}

}  // namespace muon
