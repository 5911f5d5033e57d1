// Host-side planning: shape-fused batching (Section 6.6), workspace carving, layout validation.
#include <algorithm>
#include <map>
#include <numeric>

#include "internal.h"

namespace muon {

static inline size_t up(size_t x, size_t a) { return (x + a - 1) / a * a; }

size_t elem_bytes_of_ns(int ns_precision) { return ns_precision == MUON_NS_FP32 ? 4 : 2; }

// Matrices sharing a core shape (s, l) form one group (tensors of shape [A,B], [A,1,B], [N,A,B]
// share the (A,B) group, Section 6.6); a tall matrix joins the group of its transpose because the
// iteration runs on the transpose anyway.  Each group is cut into chunks of at most chunk_elems
// elements (the 2^29-element batching cap of Section 6.6), never fewer than one matrix.
int build_plan(const muon_options_t& opt, const muon_shape_t* shapes, int32_t count, Plan* plan) {
  plan->chunks.clear();
  plan->ws_bytes = 0;
  plan->live = 0;
  std::map<std::pair<int32_t, int32_t>, std::vector<int32_t>> groups;
  std::vector<std::pair<int32_t, int32_t>> order;
  for (int32_t i = 0; i < count; ++i) {
    const int32_t r = shapes[i].rows, c = shapes[i].cols;
    if (r < 0 || c < 0) return MUON_ERR_INVALID_ARG;
    if (r == 0 || c == 0) continue;
    const std::pair<int32_t, int32_t> key(std::min(r, c), std::max(r, c));
    auto it = groups.find(key);
    if (it == groups.end()) {
      order.push_back(key);
      it = groups.emplace(key, std::vector<int32_t>()).first;
    }
    it->second.push_back(i);
    plan->live++;
  }
  const int64_t cap = opt.chunk_elems > 0 ? opt.chunk_elems : (int64_t(1) << 29);
  int32_t desc_begin = 0;
  for (const auto& key : order) {
    const std::vector<int32_t>& idx = groups[key];
    const int64_t per = int64_t(key.first) * key.second;
    // as few chunks as the cap allows, of (nearly) equal size: a short last chunk would run its fifteen
    // products on a mostly idle device
    const int64_t max_per_chunk = std::max<int64_t>(1, cap / per);
    const int64_t num_chunks = (int64_t(idx.size()) + max_per_chunk - 1) / max_per_chunk;
    const size_t base = idx.size() / size_t(num_chunks), rem = idx.size() % size_t(num_chunks);
    size_t b = 0;
    for (int64_t ci = 0; ci < num_chunks; ++ci) {
      Chunk ch;
      ch.s = key.first;
      ch.l = key.second;
      ch.ldx = int32_t(up(size_t(ch.l), 8));
      ch.lda = int32_t(up(size_t(ch.s), 8));
      const size_t e = b + base + (size_t(ci) < rem ? 1 : 0);
      ch.mats.assign(idx.begin() + long(b), idx.begin() + long(e));
      b = e;
      ch.count = int32_t(ch.mats.size());
      const int32_t ts = (ch.s + kElemTile - 1) / kElemTile, tl = (ch.l + kElemTile - 1) / kElemTile;
      ch.tiles_per_mat = ts * tl;
      ch.desc_begin = desc_begin;
      desc_begin += ch.count;
      plan->ws_bytes = std::max(plan->ws_bytes, carve_chunk(opt, ch).total);
      plan->chunks.push_back(std::move(ch));
    }
  }
  return MUON_OK;
}

WsCarve carve_chunk(const muon_options_t& opt, const Chunk& c) {
  const size_t eb = elem_bytes_of_ns(opt.ns_precision);
  const size_t xb = up(size_t(c.count) * c.s * c.ldx * eb, 256);
  const size_t ab = up(size_t(c.count) * c.s * c.lda * eb, 256);
  WsCarve w;
  w.x0 = 0;
  w.x1 = w.x0 + xb;
  w.a = w.x1 + xb;
  w.b = w.a + ab;
  w.partials = w.b + ab;
  w.rnorm = w.partials + up(size_t(c.count) * c.tiles_per_mat * sizeof(float), 256);
  w.total = w.rnorm + up(size_t(c.count) * sizeof(float), 256);
  return w;
}

int validate_layout_host(const muon_layout_desc_t* d) {
  if (!d) return MUON_ERR_INVALID_ARG;
  if (d->elem_size != 2 && d->elem_size != 4) return MUON_ERR_INVALID_ARG;
  if (d->align_elems <= 0 || d->num_shards < 1 || d->num_matrices < 0 || d->num_segments < 0) return MUON_ERR_INVALID_ARG;
  if (d->shard_len < 0 || d->shard_len % d->align_elems) return MUON_ERR_BAD_LAYOUT;
  if ((d->num_matrices > 0 && !d->shapes) || (d->num_segments > 0 && !d->segments)) return MUON_ERR_INVALID_ARG;
  std::vector<int64_t> size(size_t(d->num_matrices));
  for (int32_t i = 0; i < d->num_matrices; ++i) {
    if (d->shapes[i].rows < 0 || d->shapes[i].cols < 0) return MUON_ERR_INVALID_ARG;
    size[size_t(i)] = int64_t(d->shapes[i].rows) * d->shapes[i].cols;
  }
  const int64_t flat_len = int64_t(d->num_shards) * d->shard_len;
  std::vector<int64_t> live;
  live.reserve(size_t(d->num_segments));
  for (int64_t k = 0; k < d->num_segments; ++k) {
    const muon_segment_t& s = d->segments[k];
    if (s.reserved != 0) return MUON_ERR_BAD_LAYOUT;
    if (s.matrix < 0 || s.matrix >= d->num_matrices) return MUON_ERR_BAD_LAYOUT;
    if (s.elem_begin < 0 || s.elem_count < 0 || s.flat_offset < 0) return MUON_ERR_BAD_LAYOUT;
    if (s.elem_count == 0) continue;
    if (s.elem_begin + s.elem_count > size[size_t(s.matrix)]) return MUON_ERR_BAD_LAYOUT;
    if (s.flat_offset % d->align_elems) return MUON_ERR_BAD_LAYOUT;
    if (s.flat_offset + s.elem_count > flat_len) return MUON_ERR_BAD_LAYOUT;
    if (s.flat_offset / d->shard_len != (s.flat_offset + s.elem_count - 1) / d->shard_len) return MUON_ERR_BAD_LAYOUT;
    live.push_back(k);
  }
  // every matrix element exactly once: sort by (matrix, elem_begin) and require a gap-free, overlap-free chain
  std::vector<int64_t> by_mat = live;
  std::sort(by_mat.begin(), by_mat.end(), [&](int64_t x, int64_t y) {
    const muon_segment_t &a = d->segments[x], &b = d->segments[y];
    return a.matrix != b.matrix ? a.matrix < b.matrix : a.elem_begin < b.elem_begin;
  });
  std::vector<int64_t> covered(size_t(d->num_matrices), 0);
  for (int64_t k : by_mat) {
    const muon_segment_t& s = d->segments[k];
    if (s.elem_begin != covered[size_t(s.matrix)]) return MUON_ERR_BAD_LAYOUT;
    covered[size_t(s.matrix)] += s.elem_count;
  }
  for (int32_t i = 0; i < d->num_matrices; ++i)
    if (covered[size_t(i)] != size[size_t(i)]) return MUON_ERR_BAD_LAYOUT;
  // flat ranges pairwise disjoint
  std::vector<int64_t> by_flat = live;
  std::sort(by_flat.begin(), by_flat.end(),
            [&](int64_t x, int64_t y) { return d->segments[x].flat_offset < d->segments[y].flat_offset; });
  int64_t end = 0;
  for (int64_t k : by_flat) {
    const muon_segment_t& s = d->segments[k];
    if (s.flat_offset < end) return MUON_ERR_BAD_LAYOUT;
    end = s.flat_offset + s.elem_count;
  }
  return MUON_OK;
}

}  // namespace muon
