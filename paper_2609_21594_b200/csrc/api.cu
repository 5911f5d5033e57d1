// extern "C" entry points of libmuon_b200: argument validation, plan lookup, kernel sequencing.
#include <algorithm>
#include <cmath>
#include <cstdio>
#include <cstring>
#include <new>

#include <mutex>

#include "tc_tables.h"

using namespace muon;

namespace {

struct DeviceGuardCheck {
  static bool ok(const muon_ctx* ctx) {
    int dev = -1;
    return cudaGetDevice(&dev) == cudaSuccess && dev == ctx->device;
  }
};

bool aligned(const void* p, size_t a) { return (reinterpret_cast<uintptr_t>(p) & (a - 1)) == 0; }

bool valid_options(const muon_options_t& o) {
  if (o.grad_dtype != MUON_DTYPE_BF16 && o.grad_dtype != MUON_DTYPE_FP32) return false;
  if (o.ns_precision != MUON_NS_BF16 && o.ns_precision != MUON_NS_FP32) return false;
  if (o.engine != MUON_ENGINE_TENSOR && o.engine != MUON_ENGINE_CUDA_CORE && o.engine != MUON_ENGINE_TENSOR_1CTA) return false;
  if (o.nesterov != 0 && o.nesterov != 1) return false;
  if (o.coeffs_per_step != 0 && o.coeffs_per_step != 1) return false;
  if (o.coeffs_per_matrix != 0 && o.coeffs_per_matrix != 1) return false;
  if (o.launch_per_product != 0 && o.launch_per_product != 1) return false;
  if (!(o.eps >= 0.f) || !std::isfinite(o.eps)) return false;
  if (o.chunk_elems < 0) return false;
  return true;
}

// Stream-ordered upload of a small host table through a ring of pinned staging slots, in two halves so that a
// caller may learn the device address before it fills the table in.
int acquire_slot(muon_ctx* ctx, size_t bytes, StagingSlot** out) {
  StagingSlot& s = ctx->slots[ctx->next_slot];
  ctx->next_slot = (ctx->next_slot + 1) % 4;
  if (s.used && cudaEventSynchronize(s.ev) != cudaSuccess) return MUON_ERR_CUDA;
  if (s.cap < bytes) {
    // a kernel of an earlier call may still read the old device table: drain before freeing it
    if (s.dev && cudaDeviceSynchronize() != cudaSuccess) return MUON_ERR_CUDA;
    if (s.host) cudaFreeHost(s.host);
    if (s.dev) cudaFree(s.dev);
    s.host = s.dev = nullptr;
    s.cap = 0;
    const size_t cap = (bytes + 4095) / 4096 * 4096;
    if (cudaMallocHost(&s.host, cap) != cudaSuccess) return MUON_ERR_CUDA;
    if (cudaMalloc(&s.dev, cap) != cudaSuccess) return MUON_ERR_CUDA;
    s.cap = cap;
  }
  if (!s.ev && cudaEventCreateWithFlags(&s.ev, cudaEventDisableTiming) != cudaSuccess) return MUON_ERR_CUDA;
  *out = &s;
  return MUON_OK;
}

int commit_slot(StagingSlot* s, const void* src, size_t bytes, cudaStream_t st) {
  std::memcpy(s->host, src, bytes);
  if (cudaMemcpyAsync(s->dev, s->host, bytes, cudaMemcpyHostToDevice, st) != cudaSuccess) return MUON_ERR_CUDA;
  if (cudaEventRecord(s->ev, st) != cudaSuccess) return MUON_ERR_CUDA;
  s->used = true;
  return MUON_OK;
}

int upload(muon_ctx* ctx, const void* src, size_t bytes, cudaStream_t st, void** dev_out) {
  StagingSlot* s = nullptr;
  int rc = acquire_slot(ctx, bytes, &s);
  if (rc != MUON_OK) return rc;
  rc = commit_slot(s, src, bytes, st);
  if (rc != MUON_OK) return rc;
  *dev_out = s->dev;
  return MUON_OK;
}

cudaEvent_t get_event(muon_ctx* ctx) {
  if (!ctx->event_pool.empty()) {
    cudaEvent_t e = ctx->event_pool.back();
    ctx->event_pool.pop_back();
    return e;
  }
  cudaEvent_t e = nullptr;
  cudaEventCreate(&e);
  return e;
}

struct Span {
  muon_ctx* ctx;
  int idx = -1;
  cudaStream_t st;
  Span(muon_ctx* c, int phase, cudaStream_t s) : ctx(c), st(s) {
    if (!c->profiling) return;
    PhaseSpan ps{phase, get_event(c), get_event(c), 0};
    if (!ps.a || !ps.b) return;
    cudaEventRecord(ps.a, st);
    c->spans.push_back(ps);
    idx = int(c->spans.size()) - 1;
  }
  void end(int64_t launches) {
    if (idx < 0) return;
    cudaEventRecord(ctx->spans[size_t(idx)].b, st);
    ctx->spans[size_t(idx)].launches = launches;
    idx = -1;
  }
};

Plan* get_plan(muon_ctx* ctx, const muon_shape_t* shapes, int32_t count, int* status, const uint8_t* odd_pitch = nullptr,
               int64_t edge_elems = 0) {
  std::string key(reinterpret_cast<const char*>(shapes), size_t(count) * sizeof(muon_shape_t));
  if (odd_pitch) key.append(reinterpret_cast<const char*>(odd_pitch), size_t(count));
  if (edge_elems) key.append("/edge").append(std::to_string(edge_elems));
  auto it = ctx->plans.find(key);
  if (it != ctx->plans.end()) {
    *status = MUON_OK;
    return &it->second;
  }
  Plan p;
  *status = build_plan(ctx->opt, shapes, count, &p, odd_pitch, edge_elems);
  if (*status != MUON_OK) return nullptr;
  if (ctx->plans.size() > 64) {
    for (auto& kv : ctx->plans) release_plan_tables(&kv.second);
    ctx->plans.clear();
  }
  return &ctx->plans.emplace(std::move(key), std::move(p)).first->second;
}

bool grouped_engine(const muon_ctx* ctx) {
  return ctx->opt.ns_precision == MUON_NS_BF16 && ctx->opt.engine == MUON_ENGINE_TENSOR;
}

// One product on the engines that launch per shape group (single-CTA tensor kernel, CUDA cores).
int run_gemm(muon_ctx* ctx, const GemmArgs& g, cudaStream_t st) {
  if (ctx->opt.ns_precision == MUON_NS_BF16 && ctx->opt.engine != MUON_ENGINE_CUDA_CORE && tc_supported(g))
    return launch_gemm_tc(ctx, g, st);
  return launch_gemm_simt(g, ctx->opt.ns_precision, st);
}

struct ChunkRun {
  int32_t momentum;     // 1: optimizer step, 0: orthogonalize only
  int32_t normalize;
  float lr, mu, wd;
  int32_t ns_steps;
  const float* coeffs;  // host: one row of `nco` floats, or one row per matrix of the call (opt.coeffs_per_matrix)
};

int coeff_row_len(const muon_ctx* ctx, int ns_steps) { return ctx->opt.coeffs_per_step ? 3 * ns_steps : 3; }

// Everything the kernels of one launch set need besides the plan.
struct SetRun {
  const std::vector<Chunk>* chunks;
  const LaunchSet* set;
  const SetTables* tables;      // null: per-group engines
  const MatDesc* d_descs;       // device, first record of the SET
  const RowSeg* d_segs;         // flat-shard mode, else null
  int32_t flat_vec;
  const float* d_coef;          // device, per-matrix coefficient rows, first row of the SET (null: one row for all)
  int32_t coef_stride;
};

int fill_elem_chunks(const SetRun& sr, bool want_wide, int x_index, ElemChunk* out) {
  int n = 0;
  for (int32_t ci : sr.set->chunks) {
    const Chunk& c = (*sr.chunks)[size_t(ci)];
    const bool wide = c.pitch8 && c.s % 8 == 0 && c.l % 8 == 0;
    if (wide != want_wide) continue;
    ElemChunk& e = out[n++];
    e.block_begin = 0;
    e.tiles = 0;
    e.desc_begin = c.desc_begin - sr.set->desc_begin;
    e.count = c.count;
    e.s = c.s; e.l = c.l; e.ldx = c.ldx; e.pad = 0;
    e.x_off = int64_t(c.off_x[x_index]);
    e.part_off = c.part_off;
  }
  return n;
}

// The three Newton-Schulz products of every step, for every shape group of the set.
int run_set_products(muon_ctx* ctx, const SetRun& sr, const ChunkRun& r, cudaStream_t st, int64_t* launches) {
  char* base = static_cast<char*>(ctx->ws);
  const float* rnorm = reinterpret_cast<const float*>(base + sr.set->off_rnorm);
  int n;
  if (sr.tables) {
    auto launch = [&](const tc::TcTable& tab, float alpha, float beta, float diag, int gamma_mode, int coef_a, int coef_b, int coef_d,
                      int coef_off) {
      tc::TcLaunch L;
      L.persist = nullptr;
      for (int i = 0; i < tab.nprob; ++i) {
        L.maps[i] = tab.maps[i];
        L.info[i] = tab.info[i];
      }
      L.nprob = tab.nprob;
      L.total_tiles = tab.total_tiles;
      L.alpha = alpha; L.beta = beta; L.diag = diag; L.gamma_mode = gamma_mode;
      L.coef_table = sr.d_coef;
      L.coef_a = coef_a; L.coef_b = coef_b; L.coef_d = coef_d; L.coef_off = coef_off;
      L.coef_stride = sr.coef_stride;
      L.coef_per_step = ctx->opt.coeffs_per_step;
      L.status = ctx->d_status;
      return launch_tc_grouped(ctx->device, L, st);
    };
    // Small sets: the whole iteration in ONE cooperative launch, products separated by grid barriers instead of
    // launch boundaries ("per-matrix NS launches starve the device for small matrices", Section 6.6 -- so do
    // per-product launches when a product is a handful of tiles).
    if (sr.tables->persist && !ctx->opt.launch_per_product && r.ns_steps <= tc::kMaxPersistSteps && ctx->persist_pairs != 0) {
      if (ctx->persist_pairs < 0) ctx->persist_pairs = std::max(0, tc_pair_max_resident(ctx->device));
      const int pairs = std::min(ctx->persist_pairs, sr.tables->max_tiles);
      if (pairs > 0 && sr.tables->max_tiles <= 2 * ctx->persist_pairs) {
        tc::TcLaunch L;
        std::memset(static_cast<void*>(&L), 0, sizeof(L));
        L.coef_a = L.coef_b = L.coef_d = -1;
        L.coef_table = sr.d_coef;
        L.coef_stride = sr.coef_stride;
        L.coef_per_step = ctx->opt.coeffs_per_step;
        L.status = ctx->d_status;
        L.persist = sr.tables->persist;
        L.ns_steps = r.ns_steps;
        L.barrier = reinterpret_cast<uint32_t*>(ctx->d_status + 16);
        L.barrier_base = ctx->barrier_count;
        for (int k = 0; k < r.ns_steps; ++k)
          for (int j = 0; j < 3; ++j) L.coef[k][j] = r.coeffs[(ctx->opt.coeffs_per_step ? 3 * k : 0) + j];
        n = launch_tc_persistent(ctx->device, L, pairs, st);
        if (n > 0) {
          ctx->barrier_count += uint32_t(3 * r.ns_steps - 1) * uint32_t(2 * pairs);
          *launches += n;
          return MUON_OK;
        }
        ctx->persist_pairs = 0;      // a cooperative launch is not possible here: one launch per product from now on
      }
    }
    for (int k = 0; k < r.ns_steps; ++k) {
      const int off = ctx->opt.coeffs_per_step ? 3 * k : 0;
      const float* co = r.coeffs + off;      // with per-matrix rows these scalars are replaced row by row on the device
      const int cur = k & 1;
      if ((n = launch(sr.tables->g1[cur], 1.f, 0.f, 0.f, k == 0 ? 2 : 0, -1, -1, -1, off)) < 0) return n;   // A = gamma X X^T
      *launches += n;
      if ((n = launch(sr.tables->g2, co[2], co[1], co[0], 0, 2, 1, 0, off)) < 0) return n;                  // P = a I + b A + c A A^T
      *launches += n;
      if ((n = launch(sr.tables->g3[cur], 1.f, 0.f, 0.f, k == 0 ? 1 : 0, -1, -1, -1, off)) < 0) return n;   // X' = gamma P X
      *launches += n;
    }
    return MUON_OK;
  }
  for (int32_t ci : sr.set->chunks) {
    const Chunk& ch = (*sr.chunks)[size_t(ci)];
    void* xs[2] = {base + ch.off_x[0], base + ch.off_x[1]};
    void* A = base + ch.off_a;
    void* B = base + ch.off_b;
    const float* rn = rnorm + (ch.desc_begin - sr.set->desc_begin);
    const int64_t sx = int64_t(ch.s) * ch.ldx, sa_ = int64_t(ch.s) * ch.lda;
    for (int k = 0; k < r.ns_steps; ++k) {
      const int off = ctx->opt.coeffs_per_step ? 3 * k : 0;
      const float* co = r.coeffs + off;
      void* cur = xs[k & 1];
      void* nxt = xs[(k & 1) ^ 1];
      GemmArgs g{};
      g.coef = sr.d_coef ? sr.d_coef + size_t(ch.desc_begin - sr.set->desc_begin) * size_t(sr.coef_stride) + off : nullptr;
      g.coef_stride = sr.coef_stride;
      g.coef_a = g.coef_b = g.coef_d = -1;
      g.diag = 0.f;
      g.p = cur; g.q = cur; g.d = nullptr; g.c = A;
      g.m = ch.s; g.n = ch.s; g.kdim = ch.l;
      g.ldp = ch.ldx; g.ldq = ch.ldx; g.ldc = ch.lda;
      g.stride_p = sx; g.stride_q = sx; g.stride_c = sa_;
      g.batch = ch.count; g.rnorm = rn; g.gamma_mode = (k == 0) ? 2 : 0;
      g.alpha = 1.f; g.beta = 0.f; g.nn = 0; g.symmetric = 1;
      if ((n = run_gemm(ctx, g, st)) < 0) return n;
      *launches += n;
      g.p = A; g.q = A; g.d = A; g.c = B;
      g.kdim = ch.s; g.ldp = ch.lda; g.ldq = ch.lda;
      g.stride_p = sa_; g.stride_q = sa_;
      g.gamma_mode = 0; g.alpha = co[2]; g.beta = co[1]; g.diag = co[0];         // P = a I + b A + c A A^T
      g.coef_a = 2; g.coef_b = 1; g.coef_d = 0;
      if ((n = run_gemm(ctx, g, st)) < 0) return n;
      *launches += n;
      g.p = B; g.q = cur; g.d = nullptr; g.c = nxt;                                  // X' = gamma P X
      g.m = ch.s; g.n = ch.l; g.kdim = ch.s;
      g.ldp = ch.lda; g.ldq = ch.ldx; g.ldc = ch.ldx;
      g.stride_p = sa_; g.stride_q = sx; g.stride_c = sx;
      g.gamma_mode = (k == 0) ? 1 : 0; g.alpha = 1.f; g.beta = 0.f; g.diag = 0.f; g.nn = 1; g.symmetric = 0;
      g.coef_a = g.coef_b = g.coef_d = -1;
      if ((n = run_gemm(ctx, g, st)) < 0) return n;
      *launches += n;
    }
  }
  return MUON_OK;
}

int run_set(muon_ctx* ctx, const SetRun& sr, const ChunkRun& r, cudaStream_t st) {
  char* base = static_cast<char*>(ctx->ws);
  int n;
  {
    Span sp(ctx, MUON_PHASE_MOMENTUM, st);
    int64_t total = 0;
    for (int w = 1; w >= 0; --w) {
      StageArgs sa;
      sa.nchunks = fill_elem_chunks(sr, w != 0, 0, sa.ch);
      if (sa.nchunks == 0) continue;
      sa.segs = sr.d_segs;
      sa.descs = sr.d_descs;
      sa.ws = base;
      sa.partials = reinterpret_cast<double*>(base + sr.set->off_partials);
      sa.rnorm = reinterpret_cast<float*>(base + sr.set->off_rnorm);
      sa.mu = r.mu; sa.eps = ctx->opt.eps;
      sa.nesterov = ctx->opt.nesterov;
      sa.grad_dtype = ctx->opt.grad_dtype;
      sa.ns_precision = ctx->opt.ns_precision;
      sa.momentum = r.momentum;
      sa.normalize = r.normalize;
      sa.wide = w;
      sa.flat_vec = sr.flat_vec;
      n = launch_stage(sa, st);
      if (n < 0) return n;
      total += n;
    }
    ctx->launches += total;
    sp.end(total);
  }
  {
    Span sp(ctx, MUON_PHASE_NS, st);
    int64_t total = 0;
    const int rc = run_set_products(ctx, sr, r, st, &total);
    if (rc != MUON_OK) return rc;
    ctx->launches += total;
    sp.end(total);
  }
  {
    Span sp(ctx, MUON_PHASE_UPDATE, st);
    int64_t total = 0;
    for (int w = 1; w >= 0; --w) {
      ApplyArgs aa;
      aa.nchunks = fill_elem_chunks(sr, w != 0, r.ns_steps & 1, aa.ch);
      if (aa.nchunks == 0) continue;
      aa.segs = sr.d_segs;
      aa.descs = sr.d_descs;
      aa.ws = base;
      aa.lr = r.lr; aa.wd = r.wd;
      aa.decay = 1.0f - r.lr * r.wd;
      aa.ns_precision = ctx->opt.ns_precision;
      aa.update = r.momentum;
      aa.wide = w;
      aa.flat_vec = sr.flat_vec;
      n = launch_apply(aa, st);
      if (n < 0) return n;
      total += n;
    }
    ctx->launches += total;
    sp.end(total);
  }
  return MUON_OK;
}

// Host-buffer pipeline: per launch set, gradients arrive by DMA straight into the whole-matrix buffers (the
// copy engine performs the gather) and updates leave the same way, on two copy streams that run ahead
// of / behind the compute stream.
constexpr int64_t kPipeEdgeElems = int64_t(1) << 24;

// Order in which the host-buffer pipeline runs the launch sets: only the first set's inbound copy and the last
// set's outbound copy are exposed, so the smallest set goes first and the second smallest last; the others keep the
// plan's order (largest first, the descending-size order of Section 6.7).
std::vector<size_t> pipeline_order(const Plan& plan) {
  std::vector<size_t> order(plan.sets.size());
  for (size_t c = 0; c < order.size(); ++c) order[c] = c;
  auto elems = [&](size_t c) { return plan.sets[c].elems; };
  if (plan.pipeline_ordered) return order;       // the plan was built with ramp sets at both ends, in running order
  if (order.size() > 2) {
    size_t small = 0;
    for (size_t c = 1; c < order.size(); ++c)
      if (elems(c) < elems(small)) small = c;
    order.erase(order.begin() + long(small));
    size_t second = 0;
    for (size_t k = 1; k < order.size(); ++k)
      if (elems(order[k]) < elems(order[second])) second = k;
    const size_t last = order[second];
    order.erase(order.begin() + long(second));
    order.insert(order.begin(), small);
    order.push_back(last);
  }
  return order;
}

struct HostPipe {
  const char* host_in;
  char* host_out;
  const muon_layout* layout;
};

cudaEvent_t next_sync_event(muon_ctx* ctx) {
  if (ctx->sync_events.size() < 1024) {
    cudaEvent_t e = nullptr;
    if (cudaEventCreateWithFlags(&e, cudaEventDisableTiming) != cudaSuccess) return nullptr;
    ctx->sync_events.push_back(e);
    return e;
  }
  // a recorded event may be re-recorded: earlier waits captured its earlier state
  cudaEvent_t e = ctx->sync_events[ctx->next_sync_event];
  ctx->next_sync_event = (ctx->next_sync_event + 1) % ctx->sync_events.size();
  return e;
}

int run_batched(muon_ctx* ctx, void* const* w, const void* const* g, void* const* m, void* const* o,
                const muon_shape_t* shapes, int32_t count, const ChunkRun& r, cudaStream_t st,
                const HostPipe* pipe = nullptr, const int64_t* lds = nullptr, const muon_layout* flat = nullptr) {
  int status;
  std::vector<uint8_t> odd;                            // strided views whose pitch rules out the 8-element kernels
  if (lds) {
    odd.resize(size_t(count), 0);
    bool any = false;
    for (int32_t i = 0; i < count; ++i)
      if (lds[i] % 8) odd[size_t(i)] = 1, any = true;
    if (!any) odd.clear();
  }
  // host-buffer pipeline: the first and the last batch are small (16 Mi elements), see build_plan
  Plan* plan = get_plan(ctx, shapes, count, &status, odd.empty() ? nullptr : odd.data(), pipe ? kPipeEdgeElems : 0);
  if (!plan) return status;
  if (plan->live == 0) return MUON_OK;
  if (!ctx->ws || ctx->ws_bytes < plan->ws_bytes) return MUON_ERR_WORKSPACE_TOO_SMALL;
  std::vector<MatDesc> descs(size_t(plan->live));
  for (const Chunk& ch : plan->chunks) {
    for (int32_t j = 0; j < ch.count; ++j) {
      const int32_t i = ch.mats[size_t(j)];
      MatDesc& d = descs[size_t(ch.desc_begin + j)];
      d.w = w[i];
      d.g = g[i];
      d.m = m ? m[i] : nullptr;
      d.o = o ? o[i] : nullptr;
      if (!d.w || !d.g || (r.momentum && !d.m) || (o && !d.o)) return MUON_ERR_INVALID_ARG;
      if (!aligned(d.w, 16) || !aligned(d.g, 16) || (d.m && !aligned(d.m, 16)) || (d.o && !aligned(d.o, 16)))
        return MUON_ERR_INVALID_ARG;
      d.rows = shapes[i].rows;
      d.cols = shapes[i].cols;
      d.ld = lds ? lds[i] : int64_t(d.cols);
      if (d.ld < d.cols || d.ld > 0x7fffffffLL) return MUON_ERR_INVALID_ARG;
      d.seg_begin = flat ? flat->rowseg_begin[size_t(i)] : 0;
      d.seg_count = flat ? flat->rowseg_count[size_t(i)] : 0;
      d.transposed = d.rows > d.cols ? 1 : 0;
      d.scale = float(0.2 * std::sqrt(double(std::max(d.rows, d.cols))));
    }
  }
  const bool grouped = grouped_engine(ctx);
  if (grouped) {
    if (tc_pair_grid_setup(ctx->device) < 0) return MUON_ERR_CUDA;
    status = bind_plan_tables(ctx, plan);
    if (status != MUON_OK) return status;
  }
  void* d_descs = nullptr;
  status = upload(ctx, descs.data(), descs.size() * sizeof(MatDesc), st, &d_descs);
  if (status != MUON_OK) return status;
  const float* d_coef = nullptr;
  const int nco = coeff_row_len(ctx, r.ns_steps);
  if (ctx->opt.coeffs_per_matrix) {                    // rows travel in the order of the matrix records
    std::vector<float> rows(size_t(plan->live) * size_t(nco));
    for (const Chunk& ch : plan->chunks)
      for (int32_t j = 0; j < ch.count; ++j)
        std::memcpy(&rows[size_t(ch.desc_begin + j) * size_t(nco)], r.coeffs + size_t(ch.mats[size_t(j)]) * size_t(nco),
                    size_t(nco) * sizeof(float));
    void* d = nullptr;
    status = upload(ctx, rows.data(), rows.size() * sizeof(float), st, &d);
    if (status != MUON_OK) return status;
    d_coef = static_cast<const float*>(d);
  }
  auto set_run = [&](size_t k) {
    SetRun sr;
    sr.d_coef = d_coef ? d_coef + size_t(plan->sets[k].desc_begin) * size_t(nco) : nullptr;
    sr.coef_stride = nco;
    sr.chunks = &plan->chunks;
    sr.set = &plan->sets[k];
    sr.tables = grouped ? &(*plan->set_tables)[k] : nullptr;
    sr.d_descs = static_cast<const MatDesc*>(d_descs) + plan->sets[k].desc_begin;
    sr.d_segs = flat ? flat->d_rowsegs : nullptr;
    sr.flat_vec = flat ? flat->flat_vec : 8;
    return sr;
  };
  if (!pipe) {
    for (size_t k = 0; k < plan->sets.size(); ++k) {
      status = run_set(ctx, set_run(k), r, st);
      if (status != MUON_OK) return status;
    }
    return MUON_OK;
  }
  // ---- pipelined host path
  const size_t es = size_t(pipe->layout->desc.elem_size);
  cudaEvent_t ev = next_sync_event(ctx);
  if (!ev || cudaEventRecord(ev, st) != cudaSuccess) return MUON_ERR_CUDA;
  if (cudaStreamWaitEvent(ctx->h2d_stream, ev, 0) != cudaSuccess || cudaStreamWaitEvent(ctx->d2h_stream, ev, 0) != cudaSuccess)
    return MUON_ERR_CUDA;
  const std::vector<size_t> order = pipeline_order(*plan);
  std::vector<cudaEvent_t> arrived(plan->sets.size());
  auto enqueue_inbound = [&](size_t c) {
    for (int32_t ci : plan->sets[c].chunks)
      for (int32_t i : plan->chunks[size_t(ci)].mats)
        for (const muon_segment_t& sg : pipe->layout->segs_of[size_t(i)])
          if (cudaMemcpyAsync(static_cast<char*>(const_cast<void*>(g[i])) + size_t(sg.elem_begin) * es,
                              pipe->host_in + size_t(sg.flat_offset) * es, size_t(sg.elem_count) * es, cudaMemcpyHostToDevice,
                              ctx->h2d_stream) != cudaSuccess)
            return false;
    arrived[c] = next_sync_event(ctx);
    return arrived[c] && cudaEventRecord(arrived[c], ctx->h2d_stream) == cudaSuccess;
  };
  // Inbound copies are queued a few sets ahead of the kernels that need them, not all up front: a stream takes
  // only so many pending operations before the enqueueing call blocks, and a host thread stuck queueing the copies of
  // late sets would launch the kernels of the early ones late.
  constexpr size_t kInboundAhead = 3;
  size_t queued = 0;
  for (size_t pos = 0; pos < order.size(); ++pos) {
    while (queued < order.size() && queued <= pos + kInboundAhead)
      if (!enqueue_inbound(order[queued++])) return MUON_ERR_CUDA;
    const size_t c = order[pos];
    if (cudaStreamWaitEvent(st, arrived[c], 0) != cudaSuccess) return MUON_ERR_CUDA;
    status = run_set(ctx, set_run(c), r, st);
    if (status != MUON_OK) return status;
    cudaEvent_t done = next_sync_event(ctx);
    if (!done || cudaEventRecord(done, st) != cudaSuccess || cudaStreamWaitEvent(ctx->d2h_stream, done, 0) != cudaSuccess)
      return MUON_ERR_CUDA;
    for (int32_t ci : plan->sets[c].chunks)
      for (int32_t i : plan->chunks[size_t(ci)].mats)
        for (const muon_segment_t& sg : pipe->layout->segs_of[size_t(i)])
          if (cudaMemcpyAsync(pipe->host_out + size_t(sg.flat_offset) * es,
                              static_cast<const char*>(o[i]) + size_t(sg.elem_begin) * es, size_t(sg.elem_count) * es,
                              cudaMemcpyDeviceToHost, ctx->d2h_stream) != cudaSuccess)
            return MUON_ERR_CUDA;
  }
  cudaEvent_t fin = next_sync_event(ctx);
  if (!fin || cudaEventRecord(fin, ctx->d2h_stream) != cudaSuccess || cudaStreamWaitEvent(st, fin, 0) != cudaSuccess)
    return MUON_ERR_CUDA;
  return MUON_OK;
}

}  // namespace

extern "C" {

int muon_default_options(muon_options_t* opt) {
  if (!opt) return MUON_ERR_INVALID_ARG;
  opt->grad_dtype = MUON_DTYPE_BF16;
  opt->ns_precision = MUON_NS_BF16;
  opt->nesterov = 1;
  opt->coeffs_per_step = 0;
  opt->coeffs_per_matrix = 0;
  opt->launch_per_product = 0;
  opt->eps = 1e-7f;
  opt->engine = MUON_ENGINE_TENSOR;
  opt->chunk_elems = int64_t(1) << 29;
  return MUON_OK;
}

int muon_create(muon_ctx_t** out, const muon_options_t* opt) {
  if (!out) return MUON_ERR_INVALID_ARG;
  *out = nullptr;
  muon_options_t o;
  muon_default_options(&o);
  if (opt) o = *opt;
  if (!valid_options(o)) return MUON_ERR_INVALID_ARG;
  if (o.chunk_elems == 0) o.chunk_elems = int64_t(1) << 29;
  int ndev = 0, dev = 0;
  if (cudaGetDeviceCount(&ndev) != cudaSuccess || ndev <= 0) return MUON_ERR_CUDA;
  if (cudaGetDevice(&dev) != cudaSuccess) return MUON_ERR_CUDA;
  cudaDeviceProp prop;
  if (cudaGetDeviceProperties(&prop, dev) != cudaSuccess) return MUON_ERR_CUDA;
  if (prop.major != 10) return MUON_ERR_UNSUPPORTED;   // built for sm_100a only
  muon_ctx* ctx = new (std::nothrow) muon_ctx();
  if (!ctx) return MUON_ERR_CUDA;
  ctx->opt = o;
  ctx->device = dev;
  if (cudaMalloc(&ctx->d_status, 256) != cudaSuccess || cudaMemset(ctx->d_status, 0, 256) != cudaSuccess) {
    delete ctx;
    return MUON_ERR_CUDA;
  }
  cudaDriverEntryPointQueryResult qres;
  void* fn = nullptr;
  if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &qres) == cudaSuccess &&
      qres == cudaDriverEntryPointSuccess)
    ctx->tmap_encode = fn;
  *out = ctx;
  return MUON_OK;
}

void muon_destroy(muon_ctx_t* ctx) {
  if (!ctx) return;
  cudaDeviceSynchronize();
  for (auto& kv : ctx->plans) release_plan_tables(&kv.second);
  for (StagingSlot& s : ctx->slots) {
    if (s.host) cudaFreeHost(s.host);
    if (s.dev) cudaFree(s.dev);
    if (s.ev) cudaEventDestroy(s.ev);
  }
  for (PhaseSpan& p : ctx->spans) {
    cudaEventDestroy(p.a);
    cudaEventDestroy(p.b);
  }
  for (cudaEvent_t e : ctx->event_pool) cudaEventDestroy(e);
  for (cudaEvent_t e : ctx->sync_events) cudaEventDestroy(e);
  if (ctx->h2d_stream) cudaStreamDestroy(ctx->h2d_stream);
  if (ctx->d2h_stream) cudaStreamDestroy(ctx->d2h_stream);
  if (ctx->d_status) cudaFree(ctx->d_status);
  delete ctx;
}

int muon_workspace_bytes(const muon_options_t* opt, const muon_shape_t* shapes, int32_t count, size_t* bytes) {
  if (!opt || !bytes || count < 0 || (count > 0 && !shapes)) return MUON_ERR_INVALID_ARG;
  if (!valid_options(*opt)) return MUON_ERR_INVALID_ARG;
  Plan p, q;
  int st = build_plan(*opt, shapes, count, &p);
  if (st != MUON_OK) return st;
  // the host-buffer pipeline packs the same matrices into other launch sets: the workspace covers both plans
  st = build_plan(*opt, shapes, count, &q, nullptr, kPipeEdgeElems);
  if (st != MUON_OK) return st;
  const size_t need = std::max(p.ws_bytes, q.ws_bytes);
  // strided views with an odd pitch form groups of their own; the slack covers the alignment of the extra pieces
  *bytes = need ? need + 4096 * std::max(p.chunks.size(), q.chunks.size()) : 0;
  return MUON_OK;
}

int muon_plan_describe(const muon_options_t* opt, const muon_shape_t* shapes, int32_t count, int32_t* num_chunks,
                       int32_t* chunk_of) {
  if (!opt || !num_chunks || count < 0 || (count > 0 && !shapes)) return MUON_ERR_INVALID_ARG;
  if (!valid_options(*opt)) return MUON_ERR_INVALID_ARG;
  Plan p;
  const int st = build_plan(*opt, shapes, count, &p);
  if (st != MUON_OK) return st;
  *num_chunks = int32_t(p.chunks.size());
  if (chunk_of) {
    for (int32_t i = 0; i < count; ++i) chunk_of[i] = -1;
    for (size_t c = 0; c < p.chunks.size(); ++c)
      for (int32_t i : p.chunks[c].mats) chunk_of[i] = int32_t(c);
  }
  return MUON_OK;
}

int muon_plan_launch_sets(const muon_options_t* opt, const muon_shape_t* shapes, int32_t count, int32_t* num_sets,
                          int32_t* set_of) {
  if (!opt || !num_sets || count < 0 || (count > 0 && !shapes)) return MUON_ERR_INVALID_ARG;
  if (!valid_options(*opt)) return MUON_ERR_INVALID_ARG;
  Plan p;
  const int st = build_plan(*opt, shapes, count, &p);
  if (st != MUON_OK) return st;
  *num_sets = int32_t(p.sets.size());
  if (set_of) {
    for (int32_t i = 0; i < count; ++i) set_of[i] = -1;
    for (const Chunk& c : p.chunks)
      for (int32_t i : c.mats) set_of[i] = c.set;
  }
  return MUON_OK;
}

int muon_plan_pipeline(const muon_options_t* opt, const muon_shape_t* shapes, int32_t count, int32_t* num_sets, int32_t* set_of,
                       int32_t* order, int32_t order_capacity) {
  if (!opt || !num_sets || count < 0 || (count > 0 && !shapes) || order_capacity < 0) return MUON_ERR_INVALID_ARG;
  if (!valid_options(*opt)) return MUON_ERR_INVALID_ARG;
  Plan p;
  const int st = build_plan(*opt, shapes, count, &p, nullptr, kPipeEdgeElems);
  if (st != MUON_OK) return st;
  *num_sets = int32_t(p.sets.size());
  if (set_of) {
    for (int32_t i = 0; i < count; ++i) set_of[i] = -1;
    for (const Chunk& c : p.chunks)
      for (int32_t i : c.mats) set_of[i] = c.set;
  }
  if (order) {
    const std::vector<size_t> ord = pipeline_order(p);
    for (size_t k = 0; k < ord.size() && k < size_t(order_capacity); ++k) order[k] = int32_t(ord[k]);
  }
  return MUON_OK;
}

int muon_symmetric_tiles(int32_t blocks, uint16_t* tiles, int32_t capacity, int32_t* count) {
  if (blocks < 0 || blocks > 4096 || !count || capacity < 0 || (capacity > 0 && !tiles)) return MUON_ERR_INVALID_ARG;
  const std::vector<TilePatHost> pat = symmetric_tile_pattern(blocks);
  *count = int32_t(pat.size());
  for (int32_t i = 0; i < *count && i < capacity; ++i) {
    tiles[4 * i + 0] = pat[size_t(i)].ra;
    tiles[4 * i + 1] = pat[size_t(i)].rb;
    tiles[4 * i + 2] = pat[size_t(i)].cc;
    tiles[4 * i + 3] = pat[size_t(i)].cd;
  }
  return MUON_OK;
}

int muon_set_workspace(muon_ctx_t* ctx, void* dev_ptr, size_t bytes) {
  if (!ctx) return MUON_ERR_INVALID_ARG;
  if (bytes > 0 && (!dev_ptr || !aligned(dev_ptr, 256))) return MUON_ERR_INVALID_ARG;
  ctx->ws = dev_ptr;
  ctx->ws_bytes = bytes;
  return MUON_OK;
}

int muon_layout_validate(const muon_layout_desc_t* desc) { return validate_layout_host(desc); }

int muon_layout_create(muon_ctx_t* ctx, const muon_layout_desc_t* desc, muon_layout_t** out) {
  if (!ctx || !out) return MUON_ERR_INVALID_ARG;
  *out = nullptr;
  const int st = validate_layout_host(desc);
  if (st != MUON_OK) return st;
  if (!DeviceGuardCheck::ok(ctx)) return MUON_ERR_CUDA;
  std::vector<CopyItem> items;
  for (int64_t k = 0; k < desc->num_segments; ++k) {
    const muon_segment_t& s = desc->segments[k];
    for (int64_t done = 0; done < s.elem_count; done += kCopyChunk) {
      CopyItem it;
      it.flat_offset = s.flat_offset + done;
      it.elem_begin = s.elem_begin + done;
      it.matrix = s.matrix;
      it.count = int32_t(std::min<int64_t>(kCopyChunk, s.elem_count - done));
      items.push_back(it);
    }
  }
  // items in flat order: the work of one shard is then a contiguous range (the shard-local kernels use it)
  std::stable_sort(items.begin(), items.end(), [](const CopyItem& a, const CopyItem& b) { return a.flat_offset < b.flat_offset; });
  muon_layout* L = new (std::nothrow) muon_layout();
  if (!L) return MUON_ERR_CUDA;
  L->shard_item_begin.assign(size_t(desc->num_shards) + 1, int64_t(items.size()));
  {
    size_t k = 0;
    for (int32_t r = 0; r <= desc->num_shards; ++r) {
      while (k < items.size() && items[k].flat_offset < int64_t(r) * desc->shard_len) ++k;
      L->shard_item_begin[size_t(r)] = int64_t(k);
    }
  }
  L->desc = *desc;
  L->shapes.assign(desc->shapes, desc->shapes + desc->num_matrices);
  L->desc.shapes = nullptr;
  L->desc.segments = nullptr;
  L->num_items = int64_t(items.size());
  L->device = ctx->device;
  L->segs_of.resize(size_t(desc->num_matrices));
  for (int64_t k = 0; k < desc->num_segments; ++k)
    if (desc->segments[k].elem_count > 0) L->segs_of[size_t(desc->segments[k].matrix)].push_back(desc->segments[k]);
  // Row-aligned layouts (every segment holds whole rows) can also be addressed in place by the step kernels.
  L->row_aligned = true;
  for (int64_t k = 0; k < desc->num_segments && L->row_aligned; ++k) {
    const muon_segment_t& sg = desc->segments[k];
    const int64_t cols = desc->shapes[sg.matrix].cols;
    if (sg.elem_count > 0 && (sg.elem_begin % cols || sg.elem_count % cols)) L->row_aligned = false;
  }
  if (L->row_aligned) {
    // how wide the step kernels may vectorise their accesses to flat buffers: every row segment must start on
    // a multiple of the vector width (segment starts are only guaranteed to be multiples of align_elems)
    L->flat_vec = 8;
    for (int64_t k = 0; k < desc->num_segments; ++k) {
      const muon_segment_t& sg = desc->segments[k];
      if (sg.elem_count == 0) continue;
      while (L->flat_vec > 1 && sg.flat_offset % L->flat_vec) L->flat_vec = L->flat_vec == 8 ? 4 : 1;
    }
    std::vector<RowSeg> rs;
    L->rowseg_begin.assign(size_t(desc->num_matrices), 0);
    L->rowseg_count.assign(size_t(desc->num_matrices), 0);
    for (int32_t i = 0; i < desc->num_matrices; ++i) {
      std::vector<muon_segment_t> v = L->segs_of[size_t(i)];
      std::sort(v.begin(), v.end(), [](const muon_segment_t& a, const muon_segment_t& b) { return a.elem_begin < b.elem_begin; });
      L->rowseg_begin[size_t(i)] = int32_t(rs.size());
      L->rowseg_count[size_t(i)] = int32_t(v.size());
      const int64_t cols = desc->shapes[i].cols;
      for (const muon_segment_t& sg : v)
        rs.push_back(RowSeg{int32_t(sg.elem_begin / cols), int32_t(sg.elem_count / cols), sg.flat_offset});
    }
    if (!rs.empty() && (cudaMalloc(&L->d_rowsegs, rs.size() * sizeof(RowSeg)) != cudaSuccess ||
                        cudaMemcpy(L->d_rowsegs, rs.data(), rs.size() * sizeof(RowSeg), cudaMemcpyHostToDevice) != cudaSuccess)) {
      if (L->d_rowsegs) cudaFree(L->d_rowsegs);
      delete L;
      return MUON_ERR_CUDA;
    }
  }
  if (desc->num_matrices > 0) {
    std::vector<float> scales(size_t(desc->num_matrices));
    for (int32_t i = 0; i < desc->num_matrices; ++i)
      scales[size_t(i)] = float(0.2 * std::sqrt(double(std::max(desc->shapes[i].rows, desc->shapes[i].cols))));
    if (cudaMalloc(&L->d_scales, scales.size() * sizeof(float)) != cudaSuccess ||
        cudaMemcpy(L->d_scales, scales.data(), scales.size() * sizeof(float), cudaMemcpyHostToDevice) != cudaSuccess) {
      if (L->d_scales) cudaFree(L->d_scales);
      if (L->d_rowsegs) cudaFree(L->d_rowsegs);
      delete L;
      return MUON_ERR_CUDA;
    }
  }
  if (!items.empty()) {
    if (cudaMalloc(&L->d_items, items.size() * sizeof(CopyItem)) != cudaSuccess ||
        cudaMemcpy(L->d_items, items.data(), items.size() * sizeof(CopyItem), cudaMemcpyHostToDevice) != cudaSuccess) {
      if (L->d_items) cudaFree(L->d_items);
      if (L->d_rowsegs) cudaFree(L->d_rowsegs);
      if (L->d_scales) cudaFree(L->d_scales);
      delete L;
      return MUON_ERR_CUDA;
    }
  }
  *out = L;
  return MUON_OK;
}

void muon_layout_destroy(muon_layout_t* L) {
  if (!L) return;
  if (L->d_items || L->d_rowsegs || L->d_scales) cudaDeviceSynchronize();
  if (L->d_items) cudaFree(L->d_items);
  if (L->d_rowsegs) cudaFree(L->d_rowsegs);
  if (L->d_scales) cudaFree(L->d_scales);
  delete L;
}

static int copy_common(muon_ctx_t* ctx, void* flat, const muon_layout_t* L, void* const* mats, bool scatter, void* stream,
                       bool subset = false) {
  if (!ctx || !L) return MUON_ERR_INVALID_ARG;
  if (L->num_items == 0) return MUON_OK;
  if (!flat || !mats || !aligned(flat, 16)) return MUON_ERR_INVALID_ARG;
  if (!DeviceGuardCheck::ok(ctx) || L->device != ctx->device) return MUON_ERR_CUDA;
  const size_t es = size_t(L->desc.elem_size);
  for (int32_t i = 0; i < L->desc.num_matrices; ++i) {
    const bool empty = L->shapes[size_t(i)].rows == 0 || L->shapes[size_t(i)].cols == 0;
    if (!empty && !mats[i] && !subset) return MUON_ERR_INVALID_ARG;
    if (mats[i] && !aligned(mats[i], es)) return MUON_ERR_INVALID_ARG;
  }
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  void* d_mats = nullptr;
  int status = upload(ctx, mats, size_t(L->desc.num_matrices) * sizeof(void*), st, &d_mats);
  if (status != MUON_OK) return status;
  Span sp(ctx, scatter ? MUON_PHASE_SCATTER : MUON_PHASE_GATHER, st);
  const int n = launch_copy(L->d_items, L->num_items, flat, static_cast<void* const*>(d_mats), int(es), scatter, st);
  if (n < 0) return n;
  ctx->launches += n;
  sp.end(n);
  return MUON_OK;
}

int muon_materialize(muon_ctx_t* ctx, const void* flat_buf, const muon_layout_t* layout, void* const* matrices,
                     void* stream) {
  return copy_common(ctx, const_cast<void*>(flat_buf), layout, matrices, false, stream);
}

int muon_scatter(muon_ctx_t* ctx, void* flat_buf, const muon_layout_t* layout, const void* const* matrices,
                 void* stream) {
  return copy_common(ctx, flat_buf, layout, const_cast<void* const*>(matrices), true, stream);
}

int muon_materialize_owned(muon_ctx_t* ctx, const void* flat_buf, const muon_layout_t* layout, void* const* matrices,
                           void* stream) {
  return copy_common(ctx, const_cast<void*>(flat_buf), layout, matrices, false, stream, true);
}

int muon_scatter_owned(muon_ctx_t* ctx, void* flat_buf, const muon_layout_t* layout, const void* const* matrices,
                       void* stream) {
  return copy_common(ctx, flat_buf, layout, const_cast<void* const*>(matrices), true, stream, true);
}

int muon_owner_plan(const muon_shape_t* shapes, int32_t count, int32_t ranks, int64_t batch_elems, int32_t* owner_of,
                    int32_t* batch_of, int32_t* num_batches) {
  return owner_plan_host(shapes, count, ranks, batch_elems, owner_of, batch_of, num_batches);
}

static int shard_common(muon_ctx_t* ctx, const muon_layout_t* L, int32_t shard) {
  if (!ctx || !L || shard < 0 || shard >= L->desc.num_shards) return MUON_ERR_INVALID_ARG;
  if (!DeviceGuardCheck::ok(ctx) || L->device != ctx->device) return MUON_ERR_CUDA;
  return MUON_OK;
}

int muon_shard_momentum(muon_ctx_t* ctx, const muon_layout_t* layout, int32_t shard, const void* local_grads,
                        void* local_momenta, void* local_staged, float mu, void* stream) {
  const int rc = shard_common(ctx, layout, shard);
  if (rc != MUON_OK) return rc;
  if (!std::isfinite(mu)) return MUON_ERR_INVALID_ARG;
  const int64_t b = layout->shard_item_begin[size_t(shard)], e = layout->shard_item_begin[size_t(shard) + 1];
  if (e == b) return MUON_OK;
  if (!local_grads || !local_momenta || !local_staged) return MUON_ERR_INVALID_ARG;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  Span sp(ctx, MUON_PHASE_MOMENTUM, st);
  const int n = launch_shard_momentum(layout->d_items + b, e - b, int64_t(shard) * layout->desc.shard_len, local_grads, local_momenta,
                                      local_staged, mu, ctx->opt.nesterov, ctx->opt.grad_dtype, ctx->opt.ns_precision, st);
  if (n < 0) return n;
  ctx->launches += n;
  sp.end(n);
  return MUON_OK;
}

int muon_shard_apply(muon_ctx_t* ctx, const muon_layout_t* layout, int32_t shard, void* local_params,
                     const void* const* updates, float lr, float wd, void* stream) {
  const int rc = shard_common(ctx, layout, shard);
  if (rc != MUON_OK) return rc;
  if (!std::isfinite(lr) || !std::isfinite(wd)) return MUON_ERR_INVALID_ARG;
  const int64_t b = layout->shard_item_begin[size_t(shard)], e = layout->shard_item_begin[size_t(shard) + 1];
  if (e == b) return MUON_OK;
  if (!local_params || !updates) return MUON_ERR_INVALID_ARG;
  const size_t es = elem_bytes_of_ns(ctx->opt.ns_precision);
  for (int32_t i = 0; i < layout->desc.num_matrices; ++i)
    if (updates[i] && !aligned(updates[i], es)) return MUON_ERR_INVALID_ARG;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  void* d_updates = nullptr;
  const int urc = upload(ctx, updates, size_t(layout->desc.num_matrices) * sizeof(void*), st, &d_updates);
  if (urc != MUON_OK) return urc;
  Span sp(ctx, MUON_PHASE_UPDATE, st);
  const int n = launch_shard_apply(layout->d_items + b, e - b, int64_t(shard) * layout->desc.shard_len, local_params,
                                   static_cast<const void* const*>(d_updates), layout->d_scales, lr, 1.0f - lr * wd,
                                   ctx->opt.ns_precision, st);
  if (n < 0) return n;
  ctx->launches += n;
  sp.end(n);
  return MUON_OK;
}

static int check_common(muon_ctx_t* ctx, const muon_shape_t* shapes, int32_t count, int32_t ns_steps, const float* coeffs) {
  if (!ctx || count < 0) return MUON_ERR_INVALID_ARG;
  if (count > 0 && !shapes) return MUON_ERR_INVALID_ARG;
  if (ns_steps < 1 || ns_steps > 64 || !coeffs) return MUON_ERR_INVALID_ARG;
  const int64_t nco = int64_t(ctx->opt.coeffs_per_step ? 3 * ns_steps : 3) * (ctx->opt.coeffs_per_matrix ? count : 1);
  for (int64_t i = 0; i < nco; ++i)
    if (!std::isfinite(coeffs[i])) return MUON_ERR_INVALID_ARG;
  if (!DeviceGuardCheck::ok(ctx)) return MUON_ERR_CUDA;
  return MUON_OK;
}

int muon_step_batched_out(muon_ctx_t* ctx, void* const* params, const void* const* grads, void* const* momenta,
                          void* const* updates, const muon_shape_t* shapes, int32_t count, float lr, float mu, float wd,
                          int32_t ns_steps, const float* coeffs, void* stream) {
  int st = check_common(ctx, shapes, count, ns_steps, coeffs);
  if (st != MUON_OK) return st;
  if (count == 0) return MUON_OK;
  if (!params || !grads || !momenta) return MUON_ERR_INVALID_ARG;
  if (!std::isfinite(lr) || !std::isfinite(mu) || !std::isfinite(wd)) return MUON_ERR_INVALID_ARG;
  ChunkRun r{1, 1, lr, mu, wd, ns_steps, coeffs};
  return run_batched(ctx, params, grads, momenta, updates, shapes, count, r, static_cast<cudaStream_t>(stream));
}

int muon_views_overlap(const void* const* bases, const muon_view_t* views, int32_t count, int32_t elem_size, int32_t* overlap) {
  if (count < 0 || (count > 0 && (!bases || !views)) || elem_size <= 0 || !overlap) return MUON_ERR_INVALID_ARG;
  for (int32_t i = 0; i < count; ++i)
    if (views[i].rows < 0 || views[i].cols < 0 || (views[i].rows > 0 && views[i].cols > 0 && views[i].ld < views[i].cols))
      return MUON_ERR_INVALID_ARG;
  *overlap = views_overlap_host(bases, views, count, elem_size);
  return MUON_OK;
}

int muon_step_batched_views(muon_ctx_t* ctx, void* const* params, const void* const* grads, void* const* momenta,
                            void* const* updates, const muon_view_t* views, int32_t count, float lr, float mu, float wd,
                            int32_t ns_steps, const float* coeffs, void* stream) {
  if (!ctx || count < 0 || (count > 0 && !views)) return MUON_ERR_INVALID_ARG;
  std::vector<muon_shape_t> shapes(static_cast<size_t>(count));
  std::vector<int64_t> lds(static_cast<size_t>(count));
  for (int32_t i = 0; i < count; ++i) {
    shapes[size_t(i)].rows = views[i].rows;
    shapes[size_t(i)].cols = views[i].cols;
    lds[size_t(i)] = views[i].ld;
  }
  int st = check_common(ctx, shapes.data(), count, ns_steps, coeffs);
  if (st != MUON_OK) return st;
  if (count == 0) return MUON_OK;
  if (!params || !grads || !momenta) return MUON_ERR_INVALID_ARG;
  if (!std::isfinite(lr) || !std::isfinite(mu) || !std::isfinite(wd)) return MUON_ERR_INVALID_ARG;
  for (int32_t i = 0; i < count; ++i)
    if (views[i].rows > 0 && views[i].cols > 0 && views[i].ld < views[i].cols) return MUON_ERR_INVALID_ARG;
  // everything the call writes must be written once: two views that share an element would race
  if (views_overlap_host(params, views, count, 4) || views_overlap_host(momenta, views, count, 4) ||
      (updates && views_overlap_host(updates, views, count, ctx->opt.ns_precision == MUON_NS_BF16 ? 2 : 4)))
    return MUON_ERR_INVALID_ARG;
  ChunkRun r{1, 1, lr, mu, wd, ns_steps, coeffs};
  return run_batched(ctx, params, grads, momenta, updates, shapes.data(), count, r, static_cast<cudaStream_t>(stream), nullptr,
                     lds.data());
}

int muon_step_batched(muon_ctx_t* ctx, void* const* params, const void* const* grads, void* const* momenta,
                      const muon_shape_t* shapes, int32_t count, float lr, float mu, float wd, int32_t ns_steps,
                      const float* coeffs, void* stream) {
  return muon_step_batched_out(ctx, params, grads, momenta, nullptr, shapes, count, lr, mu, wd, ns_steps, coeffs, stream);
}

int muon_step_flat(muon_ctx_t* ctx, const muon_layout_t* layout, void* flat_params, const void* flat_grads,
                   void* flat_momenta, void* flat_updates, float lr, float mu, float wd, int32_t ns_steps,
                   const float* coeffs, void* stream) {
  if (!ctx || !layout) return MUON_ERR_INVALID_ARG;
  const int32_t count = layout->desc.num_matrices;
  int rc = check_common(ctx, layout->shapes.data(), count, ns_steps, coeffs);
  if (rc != MUON_OK) return rc;
  if (count == 0) return MUON_OK;
  if (!flat_params || !flat_grads || !flat_momenta || layout->device != ctx->device) return MUON_ERR_INVALID_ARG;
  if (!std::isfinite(lr) || !std::isfinite(mu) || !std::isfinite(wd)) return MUON_ERR_INVALID_ARG;
  if (!layout->row_aligned) return MUON_ERR_UNSUPPORTED;   // a segment cuts through a row: use materialize / scatter
  // Every matrix addresses the flat buffers through its row segments; the per-matrix pointers are the bases.
  std::vector<void*> w(size_t(count), flat_params), m(size_t(count), flat_momenta), o(size_t(count), flat_updates);
  std::vector<const void*> g(size_t(count), flat_grads);
  ChunkRun r{1, 1, lr, mu, wd, ns_steps, coeffs};
  return run_batched(ctx, w.data(), g.data(), m.data(), flat_updates ? o.data() : nullptr, layout->shapes.data(), count, r,
                     static_cast<cudaStream_t>(stream), nullptr, nullptr, layout);
}

int muon_step_flat_host(muon_ctx_t* ctx, const void* host_flat_grads, void* host_flat_updates,
                        const muon_layout_t* layout, void* const* params, void* const* grads, void* const* momenta,
                        void* const* updates, float lr, float mu, float wd, int32_t ns_steps, const float* coeffs,
                        void* stream) {
  if (!ctx || !layout || !host_flat_grads || !host_flat_updates || !updates) return MUON_ERR_INVALID_ARG;
  const int want = ctx->opt.grad_dtype == MUON_DTYPE_BF16 ? 2 : 4;
  const int ns_es = ctx->opt.ns_precision == MUON_NS_BF16 ? 2 : 4;
  if (layout->desc.elem_size != want || ns_es != want) return MUON_ERR_INVALID_ARG;   // one flat format carries both ways
  const int32_t count = layout->desc.num_matrices;
  int rc = check_common(ctx, layout->shapes.data(), count, ns_steps, coeffs);
  if (rc != MUON_OK) return rc;
  if (count == 0) return MUON_OK;
  if (!params || !grads || !momenta || layout->device != ctx->device) return MUON_ERR_INVALID_ARG;
  if (!std::isfinite(lr) || !std::isfinite(mu) || !std::isfinite(wd)) return MUON_ERR_INVALID_ARG;
  if (!ctx->h2d_stream && cudaStreamCreateWithFlags(&ctx->h2d_stream, cudaStreamNonBlocking) != cudaSuccess) return MUON_ERR_CUDA;
  if (!ctx->d2h_stream && cudaStreamCreateWithFlags(&ctx->d2h_stream, cudaStreamNonBlocking) != cudaSuccess) return MUON_ERR_CUDA;
  HostPipe pipe{static_cast<const char*>(host_flat_grads), static_cast<char*>(host_flat_updates), layout};
  ChunkRun r{1, 1, lr, mu, wd, ns_steps, coeffs};
  return run_batched(ctx, params, const_cast<const void* const*>(grads), momenta, updates, layout->shapes.data(), count, r,
                     static_cast<cudaStream_t>(stream), &pipe);
}

int muon_orthogonalize_batched(muon_ctx_t* ctx, const void* const* in, void* const* out, const muon_shape_t* shapes,
                               int32_t count, int32_t ns_steps, const float* coeffs, uint32_t flags, void* stream) {
  int st = check_common(ctx, shapes, count, ns_steps, coeffs);
  if (st != MUON_OK) return st;
  if (count == 0) return MUON_OK;
  if (!in || !out || (flags & ~MUON_ORTHO_NO_NORMALIZE)) return MUON_ERR_INVALID_ARG;
  for (int32_t i = 0; i < count; ++i)
    if (shapes[i].rows > 0 && shapes[i].cols > 0 && in[i] == out[i]) return MUON_ERR_INVALID_ARG;
  ChunkRun r{0, (flags & MUON_ORTHO_NO_NORMALIZE) ? 0 : 1, 0.f, 0.f, 0.f, ns_steps, coeffs};
  return run_batched(ctx, out, in, nullptr, nullptr, shapes, count, r, static_cast<cudaStream_t>(stream));
}

int muon_ns_product(muon_ctx_t* ctx, const void* p, const void* q, const void* d, void* c, int32_t m, int32_t n,
                    int32_t k, int32_t ldp, int32_t ldq, int32_t ldc, int64_t stride_p, int64_t stride_q,
                    int64_t stride_c, int32_t batch, int32_t nn, float alpha, float beta, const float* gamma,
                    int32_t gamma_mode, void* stream) {
  if (!ctx || m < 0 || n < 0 || k < 0 || batch < 0) return MUON_ERR_INVALID_ARG;
  if (m == 0 || n == 0 || batch == 0) return MUON_OK;
  if (!p || !q || !c || k < 1) return MUON_ERR_INVALID_ARG;
  if (nn < 0 || nn > 2) return MUON_ERR_INVALID_ARG;
  if (nn == 2 && (m != n || p != q || ldp != ldq || stride_p != stride_q)) return MUON_ERR_INVALID_ARG;
  if (gamma_mode < 0 || gamma_mode > 2 || (gamma_mode && !gamma)) return MUON_ERR_INVALID_ARG;
  if (ldp < k || ldc < n || ldq < (nn == 1 ? n : k)) return MUON_ERR_INVALID_ARG;
  if (c == p || c == q || c == d) return MUON_ERR_INVALID_ARG;
  if (!DeviceGuardCheck::ok(ctx)) return MUON_ERR_CUDA;
  GemmArgs g{};
  g.p = p; g.q = q; g.d = d; g.c = c;
  g.m = m; g.n = n; g.kdim = k;
  g.ldp = ldp; g.ldq = ldq; g.ldc = ldc;
  g.stride_p = stride_p; g.stride_q = stride_q; g.stride_c = stride_c;
  g.batch = batch;
  g.rnorm = gamma;
  g.gamma_mode = gamma ? gamma_mode : 0;
  g.alpha = alpha; g.beta = beta; g.nn = nn == 1 ? 1 : 0; g.symmetric = nn == 2 ? 1 : 0;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  int nl;
  if (grouped_engine(ctx) && tc_supported(g)) {
    // the grouped engine reads its problem from device memory: a one-problem table goes through the staging ring
    if (tc_pair_grid_setup(ctx->device) < 0) return MUON_ERR_CUDA;
    std::vector<char> img;
    tc::TcTable tab;
    int rc = build_product_image(ctx->tmap_encode, g, nullptr, &img, &tab, nullptr);        // size only
    if (rc != MUON_OK) return rc;
    StagingSlot* slot = nullptr;
    rc = acquire_slot(ctx, img.size(), &slot);
    if (rc != MUON_OK) return rc;
    rc = build_product_image(ctx->tmap_encode, g, slot->dev, &img, &tab, &ctx->tmap_encodes);   // at its device address
    if (rc != MUON_OK) return rc;
    rc = commit_slot(slot, img.data(), img.size(), st);
    if (rc != MUON_OK) return rc;
    tc::TcLaunch L;
    L.persist = nullptr;
    L.maps[0] = tab.maps[0];
    L.info[0] = tab.info[0];
    L.nprob = 1;
    L.total_tiles = tab.total_tiles;
    L.alpha = g.alpha; L.beta = g.beta; L.gamma_mode = g.gamma_mode;
    L.coef_table = nullptr;
    L.diag = 0.f;
    L.coef_a = L.coef_b = L.coef_d = -1;
    L.coef_off = L.coef_stride = L.coef_per_step = 0;
    L.status = ctx->d_status;
    Span sp(ctx, MUON_PHASE_NS, st);
    nl = launch_tc_grouped(ctx->device, L, st);
    if (nl < 0) return nl;
    sp.end(nl);
  } else {
    Span sp(ctx, MUON_PHASE_NS, st);
    nl = run_gemm(ctx, g, st);
    if (nl < 0) return nl;
    sp.end(nl);
  }
  ctx->launches += nl;
  return MUON_OK;
}

int muon_last_device_status(muon_ctx_t* ctx, void* stream, int32_t* status) {
  if (!ctx || !status) return MUON_ERR_INVALID_ARG;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  int32_t v = 0;
  if (cudaMemcpyAsync(&v, ctx->d_status, sizeof(v), cudaMemcpyDeviceToHost, st) != cudaSuccess) return MUON_ERR_CUDA;
  if (cudaStreamSynchronize(st) != cudaSuccess) return MUON_ERR_CUDA;
  *status = v;
  return MUON_OK;
}

int muon_clear_device_status(muon_ctx_t* ctx, void* stream) {
  if (!ctx) return MUON_ERR_INVALID_ARG;
  return cudaMemsetAsync(ctx->d_status, 0, sizeof(int32_t), static_cast<cudaStream_t>(stream)) == cudaSuccess ? MUON_OK
                                                                                                               : MUON_ERR_CUDA;
}

int muon_synchronize_and_check(muon_ctx_t* ctx, void* stream) {
  int32_t v = 0;
  const int rc = muon_last_device_status(ctx, stream, &v);
  if (rc != MUON_OK) return rc;
  return v == 0 ? MUON_OK : MUON_ERR_DEVICE_TIMEOUT;
}

int64_t muon_tensor_map_encodes(const muon_ctx_t* ctx) { return ctx ? ctx->tmap_encodes : 0; }

int muon_self_test_bounded_wait(muon_ctx_t* ctx, void* stream) {
  if (!ctx) return MUON_ERR_INVALID_ARG;
  if (!DeviceGuardCheck::ok(ctx)) return MUON_ERR_CUDA;
  const int n = launch_bounded_wait_probe(ctx, static_cast<cudaStream_t>(stream));
  if (n < 0) return n;
  ctx->launches += n;
  return MUON_OK;
}

int muon_profile_enable(muon_ctx_t* ctx, int32_t on) {
  if (!ctx) return MUON_ERR_INVALID_ARG;
  ctx->profiling = on != 0;
  return MUON_OK;
}

static int drain_spans(muon_ctx_t* ctx) {
  for (PhaseSpan& p : ctx->spans) {
    float ms = 0.f;
    if (cudaEventSynchronize(p.b) != cudaSuccess || cudaEventElapsedTime(&ms, p.a, p.b) != cudaSuccess) return MUON_ERR_CUDA;
    ctx->phase_ms[p.phase] += double(ms);
    ctx->phase_launches[p.phase] += p.launches;
    ctx->event_pool.push_back(p.a);
    ctx->event_pool.push_back(p.b);
  }
  ctx->spans.clear();
  return MUON_OK;
}

int muon_profile_reset(muon_ctx_t* ctx) {
  if (!ctx) return MUON_ERR_INVALID_ARG;
  const int st = drain_spans(ctx);
  for (int i = 0; i < MUON_NUM_PHASES; ++i) {
    ctx->phase_ms[i] = 0.0;
    ctx->phase_launches[i] = 0;
  }
  return st;
}

int muon_profile_read(muon_ctx_t* ctx, int32_t phase, double* ms, int64_t* launches) {
  if (!ctx || phase < 0 || phase >= MUON_NUM_PHASES) return MUON_ERR_INVALID_ARG;
  const int st = drain_spans(ctx);
  if (st != MUON_OK) return st;
  if (ms) *ms = ctx->phase_ms[phase];
  if (launches) *launches = ctx->phase_launches[phase];
  return MUON_OK;
}

int64_t muon_launch_count(const muon_ctx_t* ctx) { return ctx ? ctx->launches : 0; }

const char* muon_status_string(int status) {
  switch (status) {
    case MUON_OK: return "ok";
    case MUON_ERR_INVALID_ARG: return "invalid argument";
    case MUON_ERR_BAD_LAYOUT: return "bad flat-shard layout";
    case MUON_ERR_UNSUPPORTED: return "unsupported";
    case MUON_ERR_WORKSPACE_TOO_SMALL: return "workspace missing or too small";
    case MUON_ERR_CUDA: return "CUDA error or no usable sm_100 device";
    case MUON_ERR_DEVICE_TIMEOUT: return "a bounded device-side wait expired";
    case MUON_ERR_TOO_LARGE: return "matrix too large for the fixed built-in scratch";
    default: return "unknown status";
  }
}

}  // extern "C"

// ---------------------------------------------------------------------------------------------
// Allocation-free variant: one matrix, all scratch in a fixed device array that ships with the
// library image.  The array's name is only a host-side handle here; kernels need its device
// address, which differs per GPU, so it is looked up once per device with that device current.
// ---------------------------------------------------------------------------------------------
static __device__ __align__(256) unsigned char g_static_scratch[MUON_STATIC_SCRATCH_BYTES];

namespace {

constexpr int kMaxDevices = 64;
// [0,256): spare status word; [256,512): matrix descriptor; [512, 16 KiB): problem tables of the tensor engine
constexpr size_t kStaticHeader = 16384;
constexpr size_t kStaticDescOff = 256, kStaticTablesOff = 512;
std::mutex g_static_mutex;                  // guards the one-time set-up below
void* g_static_ptr[kMaxDevices] = {};       // device address of g_static_scratch, per device ordinal
void* g_static_encode = nullptr;            // cuTensorMapEncodeTiled

int static_setup(int dev, void** ptr_out, void** encode_out) {
  if (dev < 0 || dev >= kMaxDevices) return MUON_ERR_UNSUPPORTED;
  std::lock_guard<std::mutex> lock(g_static_mutex);
  if (!g_static_ptr[dev]) {
    cudaDeviceProp prop;
    if (cudaGetDeviceProperties(&prop, dev) != cudaSuccess) return MUON_ERR_CUDA;
    if (prop.major != 10) return MUON_ERR_UNSUPPORTED;
    void* p = nullptr;
    if (cudaGetSymbolAddress(&p, g_static_scratch) != cudaSuccess || !p) return MUON_ERR_CUDA;
    if (!g_static_encode) {
      cudaDriverEntryPointQueryResult qres;
      void* fn = nullptr;
      if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &qres) != cudaSuccess ||
          qres != cudaDriverEntryPointSuccess || !fn)
        return MUON_ERR_CUDA;
      g_static_encode = fn;
    }
    if (tc_pair_grid_setup(dev) < 0) return MUON_ERR_CUDA;
    g_static_ptr[dev] = p;
  }
  *ptr_out = g_static_ptr[dev];
  *encode_out = g_static_encode;
  return MUON_OK;
}

}  // namespace

extern "C" int muon_orthogonalize_static(const void* in, void* out, int32_t rows, int32_t cols, int32_t ns_precision,
                                         int32_t ns_steps, const float* coeffs, float eps, uint32_t flags,
                                         int32_t* status, void* stream) {
  if (rows < 0 || cols < 0 || ns_steps < 1 || ns_steps > 64 || !coeffs) return MUON_ERR_INVALID_ARG;
  if (ns_precision != MUON_NS_BF16 && ns_precision != MUON_NS_FP32) return MUON_ERR_INVALID_ARG;
  if (flags & ~MUON_ORTHO_NO_NORMALIZE) return MUON_ERR_INVALID_ARG;
  if (!(eps >= 0.f) || !std::isfinite(eps)) return MUON_ERR_INVALID_ARG;
  for (int i = 0; i < 3; ++i)
    if (!std::isfinite(coeffs[i])) return MUON_ERR_INVALID_ARG;
  if (rows == 0 || cols == 0) return MUON_OK;
  if (!in || !out || in == out || !aligned(in, 16) || !aligned(out, 16)) return MUON_ERR_INVALID_ARG;

  // A stack context: it only carries options and pointers into the fixed array; nothing is allocated.
  muon_ctx ctx;
  muon_default_options(&ctx.opt);
  ctx.opt.ns_precision = ns_precision;
  ctx.opt.eps = eps;
  std::vector<Chunk> chunks(1);                // one matrix, one shape group, one launch set
  Chunk& ch = chunks[0];
  ch.s = std::min(rows, cols);
  ch.l = std::max(rows, cols);
  ch.ldx = (ch.l + 7) / 8 * 8;
  ch.lda = (ch.s + 7) / 8 * 8;
  ch.count = 1;
  ch.tiles_per_mat = ((ch.s + kElemTile - 1) / kElemTile) * ((ch.l + kElemTile - 1) / kElemTile);
  LaunchSet set;
  set.chunks.push_back(0);
  set.count = 1;
  layout_set(ctx.opt, &chunks, &set);
  if (set.bytes + kStaticHeader > size_t(MUON_STATIC_SCRATCH_BYTES)) return MUON_ERR_TOO_LARGE;

  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess) return MUON_ERR_CUDA;
  void* base = nullptr;
  void* encode = nullptr;
  int rc = static_setup(dev, &base, &encode);
  if (rc != MUON_OK) return rc;
  char* sb = static_cast<char*>(base);
  ctx.device = dev;
  ctx.tmap_encode = encode;
  ctx.d_status = status ? status : reinterpret_cast<int32_t*>(sb);
  ctx.ws = sb + kStaticHeader;
  ctx.ws_bytes = size_t(MUON_STATIC_SCRATCH_BYTES) - kStaticHeader;

  cudaStream_t st = static_cast<cudaStream_t>(stream);
  MatDesc d;
  std::memset(&d, 0, sizeof(d));
  d.w = out;
  d.g = in;
  d.rows = rows;
  d.cols = cols;
  d.ld = cols;
  d.transposed = rows > cols ? 1 : 0;
  d.scale = 0.f;
  d.seg_begin = d.seg_count = 0;
  // The descriptor and the problem tables reach the device as kernel arguments (no copy whose host source could
  // go out of scope, no staging buffer).
  MatDesc* d_desc = reinterpret_cast<MatDesc*>(sb + kStaticDescOff);
  if (launch_poke(d_desc, &d, sizeof(d), st) < 0) return MUON_ERR_CUDA;
  SetImage img;
  const bool grouped = grouped_engine(&ctx);
  if (grouped) {
    rc = build_set_image(encode, ctx.ws, chunks, set, sb + kStaticTablesOff, &img, nullptr, false);
    if (rc != MUON_OK) return rc;
    if (img.bytes.size() > kStaticHeader - kStaticTablesOff) return MUON_ERR_TOO_LARGE;
    img.bytes.resize((img.bytes.size() + 15) / 16 * 16, 0);
    for (size_t off = 0; off < img.bytes.size(); off += 3072)
      if (launch_poke(sb + kStaticTablesOff + off, img.bytes.data() + off, std::min<size_t>(3072, img.bytes.size() - off), st) < 0)
        return MUON_ERR_CUDA;
  }
  ChunkRun r{0, (flags & MUON_ORTHO_NO_NORMALIZE) ? 0 : 1, 0.f, 0.f, 0.f, ns_steps, coeffs};
  SetRun sr;
  sr.chunks = &chunks;
  sr.set = &set;
  sr.tables = grouped ? &img.tables : nullptr;
  sr.d_descs = d_desc;
  sr.d_segs = nullptr;
  sr.flat_vec = 8;
  sr.d_coef = nullptr;
  sr.coef_stride = 0;
  return run_set(&ctx, sr, r, st);
}
