// Host side of the grouped tensor-core engine: the static plan of Section 6.2 ("fixed when the optimizer
// is built, and replayed unchanged at every step") for the Newton-Schulz launches.  For every launch set the
// tensor maps over its workspace buffers, the tile lists and the per-product problem lists are built once
// and kept in device memory; a step then launches 3 * ns_steps kernels per set and encodes nothing.
#include <algorithm>
#include <cstring>
#include <map>

#include "tc_tables.h"

namespace muon {

using tc::TcMaps;
using tc::TcPersist;
using tc::TcProbInfo;
using tc::TcTable;
using tc::TilePat;

namespace {

size_t up(size_t x, size_t a) { return (x + a - 1) / a * a; }

struct ImageBuilder {
  std::vector<char> bytes;
  const char* dev_base;
  size_t reserve(size_t n, size_t align) {
    const size_t off = up(bytes.size(), align);
    bytes.resize(off + n, 0);
    return off;
  }
  const void* dev(size_t off) const { return dev_base + off; }
};

// Dense product over an m x n result: 2 x 2 block tiles, row pairs varying fastest.
void fill_dense(TcProbInfo* p, int m, int n) {
  p->rblocks = (m + 127) / 128;
  p->cblocks = (n + 127) / 128;
  p->row_pairs = (p->rblocks + 1) / 2;
  p->tiles_per_mat = p->row_pairs * ((p->cblocks + 1) / 2);
  p->pattern = nullptr;
  p->symmetric = 0;
}

size_t add_pattern(ImageBuilder* ib, int nb, int32_t* count) {
  const std::vector<TilePatHost> pat = symmetric_tile_pattern(nb);
  const size_t off = ib->reserve(pat.size() * sizeof(TilePat), 16);
  static_assert(sizeof(TilePat) == sizeof(TilePatHost), "tile record layout");
  std::memcpy(ib->bytes.data() + off, pat.data(), pat.size() * sizeof(TilePat));
  *count = int32_t(pat.size());
  return off;
}

}  // namespace

int build_set_image(void* encode_fn, const void* ws, const std::vector<Chunk>& chunks, const LaunchSet& set,
                    const void* dev_base, SetImage* out, int64_t* encodes, bool with_persist) {
  if (!encode_fn) return MUON_ERR_CUDA;
  ImageBuilder ib;
  ib.dev_base = static_cast<const char*>(dev_base);
  const char* wsb = static_cast<const char*>(ws);
  const int n = int(set.chunks.size());
  if (n > tc::kMaxProblems) return MUON_ERR_UNSUPPORTED;
  // tile lists of the symmetric products, one per distinct block count
  std::map<int, std::pair<size_t, int32_t>> patterns;
  for (int32_t ci : set.chunks) {
    const int nb = (chunks[size_t(ci)].s + 127) / 128;
    if (!patterns.count(nb)) {
      int32_t cnt = 0;
      const size_t off = add_pattern(&ib, nb, &cnt);
      patterns[nb] = {off, cnt};
    }
  }
  // tensor maps per chunk: X iterates as 128-row boxes (P, Q, D, C), as 64-row boxes (Q of a 128-wide tile) and as
  // 64 x 64 boxes (the MN-major operand of X' = P X); A as 128- and 64-row boxes, B as 128-row boxes
  struct Maps {
    CUtensorMap xr[2], xh[2], a, ah, b, bh;
  };
  std::vector<Maps> maps(static_cast<size_t>(n));
  for (int k = 0; k < n; ++k) {
    const Chunk& c = chunks[size_t(set.chunks[size_t(k)])];
    const int64_t sx = int64_t(c.s) * c.ldx, sa = int64_t(c.s) * c.lda;
    bool ok = true;
    for (int i = 0; i < 2; ++i) {
      ok = ok && tc::encode_map(encode_fn, &maps[size_t(k)].xr[i], wsb + c.off_x[i], c.l, c.s, c.count, c.ldx, sx, 128);
      ok = ok && tc::encode_map(encode_fn, &maps[size_t(k)].xh[i], wsb + c.off_x[i], c.l, c.s, c.count, c.ldx, sx, 64);
    }
    ok = ok && tc::encode_map(encode_fn, &maps[size_t(k)].a, wsb + c.off_a, c.s, c.s, c.count, c.lda, sa, 128);
    ok = ok && tc::encode_map(encode_fn, &maps[size_t(k)].ah, wsb + c.off_a, c.s, c.s, c.count, c.lda, sa, 64);
    ok = ok && tc::encode_map(encode_fn, &maps[size_t(k)].b, wsb + c.off_b, c.s, c.s, c.count, c.lda, sa, 128);
    ok = ok && tc::encode_map(encode_fn, &maps[size_t(k)].bh, wsb + c.off_b, c.s, c.s, c.count, c.lda, sa, 64);
    if (!ok) return MUON_ERR_CUDA;
    if (encodes) *encodes += 8;
  }
  // problem order inside a launch: longest accumulation first, so that short tiles fill the tail
  std::vector<int> by_l(static_cast<size_t>(n)), by_s(static_cast<size_t>(n));
  for (int k = 0; k < n; ++k) by_l[size_t(k)] = by_s[size_t(k)] = k;
  auto chunk_of = [&](int k) -> const Chunk& { return chunks[size_t(set.chunks[size_t(k)])]; };
  std::stable_sort(by_l.begin(), by_l.end(), [&](int a, int b) { return chunk_of(a).l > chunk_of(b).l; });
  std::stable_sort(by_s.begin(), by_s.end(), [&](int a, int b) { return chunk_of(a).s > chunk_of(b).s; });

  const float* rnorm_base = reinterpret_cast<const float*>(wsb + set.off_rnorm);
  SetTables T;
  for (int kind = 0; kind < 5; ++kind) {     // 0,1: G1 reading X0/X1; 2: G2; 3,4: G3 reading X0/X1
    TcTable& tab = kind < 2 ? T.g1[kind] : kind == 2 ? T.g2 : T.g3[kind - 3];
    tab.nprob = n;
    int32_t tile_begin = 0;
    const std::vector<int>& order = kind < 2 ? by_l : by_s;
    for (int j = 0; j < n; ++j) {
      const int k = order[size_t(j)];
      const Chunk& c = chunk_of(k);
      const Maps& mp = maps[size_t(k)];
      TcMaps m;
      std::memset(&m, 0, sizeof(m));
      TcProbInfo p;
      std::memset(&p, 0, sizeof(p));
      p.rnorm = rnorm_base + (c.desc_begin - set.desc_begin);
      p.mat_begin = c.desc_begin - set.desc_begin;
      p.batch = c.count;
      const auto& pat = patterns[(c.s + 127) / 128];
      if (kind < 2) {            // A = gamma X X^T
        m.p = m.q = mp.xr[kind];
        m.ph = m.qh = mp.xh[kind];
        m.c = m.d = mp.a;
        p.d = nullptr;
        p.c = reinterpret_cast<__nv_bfloat16*>(const_cast<char*>(wsb + c.off_a));
        p.m = p.n = c.s; p.kdim = c.l; p.ldc = c.lda; p.stride_c = int64_t(c.s) * c.lda;
        p.symmetric = 1; p.nn = 0;
        p.rblocks = p.cblocks = (c.s + 127) / 128;
        p.row_pairs = 0;
        p.pattern = static_cast<const TilePat*>(ib.dev(pat.first));
        p.tiles_per_mat = pat.second;
      } else if (kind == 2) {    // P = delta I + beta A + alpha A A^T
        m.p = m.q = m.d = mp.a;
        m.ph = m.qh = mp.ah;
        m.c = mp.b;
        p.p_half = p.q_half = 1;                   // A was written by the product before, half-stored
        p.d = reinterpret_cast<const __nv_bfloat16*>(wsb + c.off_a);
        p.c = reinterpret_cast<__nv_bfloat16*>(const_cast<char*>(wsb + c.off_b));
        p.m = p.n = p.kdim = c.s; p.ldc = c.lda; p.stride_c = int64_t(c.s) * c.lda;
        p.symmetric = 1; p.nn = 0;
        p.rblocks = p.cblocks = (c.s + 127) / 128;
        p.row_pairs = 0;
        p.pattern = static_cast<const TilePat*>(ib.dev(pat.first));
        p.tiles_per_mat = pat.second;
      } else {                   // X' = gamma P X
        const int cur = kind - 3;
        m.p = mp.b;
        m.ph = mp.bh;
        p.p_half = 1;                              // B is half-stored
        m.q = m.qh = mp.xh[cur];                   // 64 x 64 boxes: same geometry as the 64-row boxes
        m.d = mp.xr[cur];
        m.c = mp.xr[cur ^ 1];
        p.d = nullptr;
        p.c = reinterpret_cast<__nv_bfloat16*>(const_cast<char*>(wsb + c.off_x[cur ^ 1]));
        p.m = c.s; p.n = c.l; p.kdim = c.s; p.ldc = c.ldx; p.stride_c = int64_t(c.s) * c.ldx;
        p.nn = 1;
        fill_dense(&p, p.m, p.n);
      }
      p.tile_begin = tile_begin;
      const int64_t tiles = int64_t(p.tiles_per_mat) * p.batch;
      if (tile_begin + tiles > 0x3fffffffLL) return MUON_ERR_UNSUPPORTED;
      tile_begin += int32_t(tiles);
      tab.maps[j] = m;
      tab.info[j] = p;
    }
    tab.total_tiles = tile_begin;
  }
  if (with_persist) {  // the five tables once more, in device memory, for the whole-iteration launch
    const size_t off = ib.reserve(sizeof(TcPersist), 128);
    TcPersist* pp = new TcPersist();
    std::memset(static_cast<void*>(pp), 0, sizeof(TcPersist));
    const TcTable* tabs[5] = {&T.g1[0], &T.g1[1], &T.g2, &T.g3[0], &T.g3[1]};
    pp->nprob = n;
    for (int kind = 0; kind < 5; ++kind) {
      for (int j = 0; j < n; ++j) {
        pp->maps[kind][j] = tabs[kind]->maps[j];
        pp->info[kind][j] = tabs[kind]->info[j];
      }
      pp->total_tiles[kind] = tabs[kind]->total_tiles;
      T.max_tiles = std::max(T.max_tiles, tabs[kind]->total_tiles);
    }
    std::memcpy(ib.bytes.data() + off, pp, sizeof(TcPersist));
    delete pp;
    T.persist = static_cast<const TcPersist*>(ib.dev(off));
  }
  out->bytes = std::move(ib.bytes);
  out->tables = T;
  return MUON_OK;
}

int build_product_image(void* encode_fn, const GemmArgs& g, const void* dev_base, std::vector<char>* bytes, TcTable* table,
                        int64_t* encodes) {
  if (!encode_fn) return MUON_ERR_CUDA;
  ImageBuilder ib;
  ib.dev_base = static_cast<const char*>(dev_base);
  TcMaps m;
  std::memset(&m, 0, sizeof(m));
  TcProbInfo p;
  std::memset(&p, 0, sizeof(p));
  bool ok = tc::encode_map(encode_fn, &m.p, g.p, g.kdim, g.m, g.batch, g.ldp, g.stride_p, 128);
  m.ph = m.p;                                      // stand-alone products read P as stored
  if (!g.nn) {
    ok = ok && tc::encode_map(encode_fn, &m.q, g.q, g.kdim, g.n, g.batch, g.ldq, g.stride_q, 128);
    ok = ok && tc::encode_map(encode_fn, &m.qh, g.q, g.kdim, g.n, g.batch, g.ldq, g.stride_q, 64);
  } else {
    ok = ok && tc::encode_map(encode_fn, &m.q, g.q, g.n, g.kdim, g.batch, g.ldq, g.stride_q, 64);
    m.qh = m.q;
  }
  ok = ok && tc::encode_map(encode_fn, &m.c, g.c, g.n, g.m, g.batch, g.ldc, g.stride_c, 128);
  ok = ok && tc::encode_map(encode_fn, &m.d, g.d ? g.d : g.c, g.n, g.m, g.batch, g.ldc, g.stride_c, 128);
  if (!ok) return MUON_ERR_CUDA;
  if (encodes) *encodes += g.nn ? 4 : 5;
  p.d = static_cast<const __nv_bfloat16*>(g.d);
  p.c = static_cast<__nv_bfloat16*>(g.c);
  p.rnorm = g.rnorm;
  p.mat_begin = 0;
  p.stride_c = g.stride_c;
  p.m = g.m; p.n = g.n; p.kdim = g.kdim; p.ldc = g.ldc;
  p.batch = g.batch;
  p.nn = g.nn ? 1 : 0;
  p.tile_begin = 0;
  if (g.symmetric) {
    p.symmetric = 1;
    p.mirror_out = 1;                              // the caller gets the whole of C
    p.rblocks = p.cblocks = (g.m + 127) / 128;
    int32_t cnt = 0;
    const size_t poff = add_pattern(&ib, p.rblocks, &cnt);
    p.pattern = static_cast<const TilePat*>(ib.dev(poff));
    p.tiles_per_mat = cnt;
  } else {
    fill_dense(&p, g.m, g.n);
  }
  const int64_t tiles = int64_t(p.tiles_per_mat) * p.batch;
  if (tiles > 0x3fffffffLL) return MUON_ERR_UNSUPPORTED;
  table->maps[0] = m;
  table->info[0] = p;
  table->nprob = 1;
  table->total_tiles = int32_t(tiles);
  *bytes = std::move(ib.bytes);
  return MUON_OK;
}

void release_plan_tables(Plan* plan) {
  if (plan->d_tables) {
    cudaDeviceSynchronize();      // a kernel of an earlier call may still read the tables
    cudaFree(plan->d_tables);
  }
  delete plan->set_tables;
  plan->set_tables = nullptr;
  plan->d_tables = nullptr;
  plan->tables_ws = nullptr;
}

int bind_plan_tables(muon_ctx* ctx, Plan* plan) {
  if (plan->d_tables && plan->tables_ws == ctx->ws) return MUON_OK;
  release_plan_tables(plan);
  // two passes: sizes first (against a null base), then the images at their final device addresses
  std::vector<size_t> offs(plan->sets.size());
  size_t total = 0;
  for (size_t k = 0; k < plan->sets.size(); ++k) {
    SetImage img;
    const int rc = build_set_image(ctx->tmap_encode, ctx->ws, plan->chunks, plan->sets[k], nullptr, &img, nullptr);
    if (rc != MUON_OK) return rc;
    offs[k] = total;
    total += up(img.bytes.size(), 256);
  }
  if (total == 0) return MUON_OK;
  void* dev = nullptr;
  if (cudaMalloc(&dev, total) != cudaSuccess) return MUON_ERR_CUDA;
  std::vector<char> host(total, 0);
  std::vector<SetTables>* tabs = new std::vector<SetTables>(plan->sets.size());
  for (size_t k = 0; k < plan->sets.size(); ++k) {
    SetImage img;
    const int rc = build_set_image(ctx->tmap_encode, ctx->ws, plan->chunks, plan->sets[k], static_cast<char*>(dev) + offs[k], &img,
                                   &ctx->tmap_encodes);
    if (rc != MUON_OK) {
      cudaFree(dev);
      delete tabs;
      return rc;
    }
    std::memcpy(host.data() + offs[k], img.bytes.data(), img.bytes.size());
    (*tabs)[k] = img.tables;
  }
  if (cudaMemcpy(dev, host.data(), total, cudaMemcpyHostToDevice) != cudaSuccess) {
    cudaFree(dev);
    delete tabs;
    return MUON_ERR_CUDA;
  }
  plan->d_tables = dev;
  plan->tables_ws = ctx->ws;
  plan->set_tables = tabs;
  return MUON_OK;
}

}  // namespace muon
