// Host-side planning: shape-fused batching (Section 6.6), workspace carving, layout validation.
#include <algorithm>
#include <cstdlib>
#include <iterator>
#include <map>
#include <numeric>

#include "internal.h"

namespace muon {

static inline size_t up(size_t x, size_t a) { return (x + a - 1) / a * a; }

size_t elem_bytes_of_ns(int ns_precision) { return ns_precision == MUON_NS_FP32 ? 4 : 2; }

// Matrices sharing a core shape (s, l) form one group (tensors of shape [A,B], [A,1,B], [N,A,B]
// share the (A,B) group, Section 6.6); a tall matrix joins the group of its transpose because the
// iteration runs on the transpose anyway.  Each group is cut into chunks of at most chunk_elems
// elements (the 2^29-element batching cap of Section 6.6), never fewer than one matrix.  Chunks are
// then packed into launch sets of at most chunk_elems elements in total (first fit, largest chunk
// first): the chunks of a set are resident in the workspace together and share every launch, so a
// set -- not a chunk -- is the unit the cap bounds.
// `odd_pitch` (may be null) marks strided views whose row pitch is not a multiple of 8 elements: they form groups
// of their own, so that the elementwise kernels chosen for a matrix -- and with them the order in which its norm is
// summed -- never depend on what else is in the call.
// `edge_elems` > 0 (the host-buffer pipeline): the sets come out in the order the pipeline runs them, with a ramp at
// either end.  Copies and kernels overlap only from the second set on, and a set's kernels cannot start before its own
// inbound copy has finished, so a pipeline that opens with a full-size set waits for its whole copy, and one that closes
// with a full-size set waits for that set's whole outbound copy.  The ramp sets start at about edge_elems elements and
// grow as fast as the kernels of the sets before them can cover the next copy; the sets in the middle are the ordinary
// ones, largest first (the descending-size order of Section 6.7).
int build_plan(const muon_options_t& opt, const muon_shape_t* shapes, int32_t count, Plan* plan, const uint8_t* odd_pitch,
               int64_t edge_elems) {
  plan->chunks.clear();
  plan->sets.clear();
  plan->ws_bytes = 0;
  plan->live = 0;
  plan->pipeline_ordered = false;
  typedef std::pair<std::pair<int32_t, int32_t>, int32_t> GroupKey;      // ((s, l), odd pitch)
  auto key_of = [&](int32_t i) {
    const int32_t r = shapes[i].rows, c = shapes[i].cols;
    return GroupKey(std::make_pair(std::min(r, c), std::max(r, c)), (odd_pitch && odd_pitch[i]) ? 1 : 0);
  };
  auto elems_of_mat = [&](int32_t i) { return int64_t(shapes[i].rows) * shapes[i].cols; };
  std::vector<int32_t> live;
  int64_t total = 0;
  for (int32_t i = 0; i < count; ++i) {
    if (shapes[i].rows < 0 || shapes[i].cols < 0) return MUON_ERR_INVALID_ARG;
    if (shapes[i].rows == 0 || shapes[i].cols == 0) continue;
    live.push_back(i);
    total += elems_of_mat(i);
  }
  plan->live = int32_t(live.size());
  const int64_t cap = opt.chunk_elems > 0 ? opt.chunk_elems : (int64_t(1) << 29);

  // a bin = the chunks of one launch set
  std::vector<std::vector<Chunk>> bins;
  auto make_chunk = [&](const GroupKey& key, std::vector<int32_t>::const_iterator b, std::vector<int32_t>::const_iterator e) {
    Chunk ch;
    ch.s = key.first.first;
    ch.l = key.first.second;
    ch.pitch8 = key.second == 0;
    ch.ldx = int32_t(up(size_t(ch.l), 8));
    ch.lda = int32_t(up(size_t(ch.s), 8));
    ch.mats.assign(b, e);
    ch.count = int32_t(ch.mats.size());
    const int32_t ts = (ch.s + kElemTile - 1) / kElemTile, tl = (ch.l + kElemTile - 1) / kElemTile;
    ch.tiles_per_mat = ts * tl;
    return ch;
  };
  auto elems_of = [](const Chunk& c) { return int64_t(c.count) * c.s * c.l; };

  // ---- ramps (pipeline plans only, and only when the ramps leave at least half of the work to full-size sets)
  std::vector<std::vector<int32_t>> ramp[2];       // [0]: opening sets, first to last; [1]: closing sets, last to first
  if (edge_elems > 0 && total >= 16 * edge_elems) {
    // Ramp sets are built from the matrices with the most Newton-Schulz work per element (their kernels hide the most
    // copy time per byte copied); matrices with little work per element stay in the middle of the pipeline.  A set may
    // hold edge_elems elements plus what the kernels of the sets before it can cover: kFlopsPerElem flops of kernel work
    // per element copied (about 1.3 PFLOP/s of products against 25 G elements/s over the host link, with a margin).
    constexpr double kFlopsPerElem = 65536.0;
    auto flops_of_mat = [&](int32_t i) {                    // five steps of (3 s^2 l + s^3) multiply-adds
      const double sm = double(std::min(shapes[i].rows, shapes[i].cols)), lg = double(std::max(shapes[i].rows, shapes[i].cols));
      return 10.0 * sm * sm * (3.0 * lg + sm);
    };
    std::vector<int32_t> asc = live;
    std::stable_sort(asc.begin(), asc.end(), [&](int32_t a, int32_t b) {
      const double da = flops_of_mat(a) / double(elems_of_mat(a)), db = flops_of_mat(b) / double(elems_of_mat(b));
      return da > db || (da == db && elems_of_mat(a) < elems_of_mat(b));
    });
    size_t cur = 0;
    int64_t used = 0;
    double work_before[2] = {0.0, 0.0};
    bool open[2] = {true, true};
    while (open[0] || open[1]) {
      for (int side = 0; side < 2; ++side) {
        if (!open[side]) continue;
        const int64_t target = std::min(edge_elems + int64_t(work_before[side] / kFlopsPerElem), cap);
        std::vector<int32_t> set;
        std::vector<GroupKey> keys;
        int64_t e = 0;
        double w = 0.0;
        size_t c = cur;
        while (c < asc.size() && e < target) {
          const int64_t m = elems_of_mat(asc[c]);
          if (!set.empty() && e + m > std::max(target, edge_elems)) break;      // never overshoot the target by a matrix
          const GroupKey k = key_of(asc[c]);
          if (std::find(keys.begin(), keys.end(), k) == keys.end()) {
            if (keys.size() == size_t(kMaxElemChunks)) break;
            keys.push_back(k);
          }
          set.push_back(asc[c]);
          e += m;
          w += flops_of_mat(asc[c]);
          ++c;
        }
        // the ramp ends where its sets reach half the cap, or where it would take more than a quarter of the work
        if (set.empty() || used + e > total / 4 || target >= cap / 2) {
          open[side] = false;
          continue;
        }
        cur = c;
        used += e;
        work_before[side] += w;
        ramp[side].push_back(std::move(set));
      }
    }
    std::vector<uint8_t> taken(size_t(count), 0);
    for (int side = 0; side < 2; ++side)
      for (const auto& set : ramp[side])
        for (int32_t i : set) taken[size_t(i)] = 1;
    live.erase(std::remove_if(live.begin(), live.end(), [&](int32_t i) { return taken[size_t(i)] != 0; }), live.end());
  }
  auto bin_of_set = [&](std::vector<int32_t> set) {         // one launch set from an explicit list of matrices
    std::sort(set.begin(), set.end());
    std::vector<GroupKey> keys;
    std::map<GroupKey, std::vector<int32_t>> by_key;
    for (int32_t i : set) {
      const GroupKey k = key_of(i);
      if (by_key.find(k) == by_key.end()) keys.push_back(k);
      by_key[k].push_back(i);
    }
    std::vector<Chunk> bin;
    for (const GroupKey& k : keys) bin.push_back(make_chunk(k, by_key[k].begin(), by_key[k].end()));
    std::stable_sort(bin.begin(), bin.end(), [&](const Chunk& a, const Chunk& b) { return elems_of(a) > elems_of(b); });
    return bin;
  };
  for (auto& set : ramp[0]) bins.push_back(bin_of_set(std::move(set)));

  // ---- the ordinary sets: shape groups, evenly cut at the cap, packed first fit (largest first)
  {
    std::map<GroupKey, std::vector<int32_t>> groups;
    std::vector<GroupKey> order;
    for (int32_t i : live) {
      const GroupKey key = key_of(i);
      auto it = groups.find(key);
      if (it == groups.end()) {
        order.push_back(key);
        it = groups.emplace(key, std::vector<int32_t>()).first;
      }
      it->second.push_back(i);
    }
    std::vector<Chunk> chunks;
    for (const auto& key : order) {
      const std::vector<int32_t>& idx = groups[key];
      const int64_t per = int64_t(key.first.first) * key.first.second;
      // as few chunks as the cap allows, of (nearly) equal size: a short last chunk would run its fifteen
      // products on a mostly idle device
      const int64_t max_per_chunk = std::max<int64_t>(1, cap / per);
      const int64_t num_chunks = (int64_t(idx.size()) + max_per_chunk - 1) / max_per_chunk;
      const size_t base = idx.size() / size_t(num_chunks), rem = idx.size() % size_t(num_chunks);
      size_t b = 0;
      for (int64_t ci = 0; ci < num_chunks; ++ci) {
        const size_t e = b + base + (size_t(ci) < rem ? 1 : 0);
        chunks.push_back(make_chunk(key, idx.begin() + long(b), idx.begin() + long(e)));
        b = e;
      }
    }
    // first-fit decreasing (stable for equal sizes, so the result is a pure function of the shape list)
    std::vector<size_t> by_size(chunks.size());
    std::iota(by_size.begin(), by_size.end(), size_t(0));
    std::stable_sort(by_size.begin(), by_size.end(), [&](size_t a, size_t b) { return elems_of(chunks[a]) > elems_of(chunks[b]); });
    std::vector<std::vector<size_t>> packed;
    std::vector<int64_t> fill;
    for (size_t ci : by_size) {
      const int64_t e = elems_of(chunks[ci]);
      size_t k = 0;
      while (k < packed.size() && (fill[k] + e > cap || packed[k].size() >= size_t(kMaxElemChunks))) ++k;
      if (k == packed.size()) {
        packed.emplace_back();
        fill.push_back(0);
      }
      packed[k].push_back(ci);
      fill[k] += e;
    }
    for (const auto& pk : packed) {
      std::vector<Chunk> bin;
      for (size_t ci : pk) bin.push_back(std::move(chunks[ci]));
      bins.push_back(std::move(bin));
    }
  }
  for (size_t k = ramp[1].size(); k-- > 0;) bins.push_back(bin_of_set(std::move(ramp[1][k])));
  plan->pipeline_ordered = !ramp[0].empty() || !ramp[1].empty();

  // final order: set by set, descriptors contiguous inside a set
  int32_t desc_begin = 0;
  for (size_t k = 0; k < bins.size(); ++k) {
    LaunchSet set;
    set.desc_begin = desc_begin;
    set.elems = 0;
    for (Chunk& src : bins[k]) {
      Chunk ch = std::move(src);
      ch.set = int32_t(k);
      ch.desc_begin = desc_begin;
      desc_begin += ch.count;
      set.elems += elems_of(ch);
      set.chunks.push_back(int32_t(plan->chunks.size()));
      plan->chunks.push_back(std::move(ch));
    }
    set.count = desc_begin - set.desc_begin;
    layout_set(opt, &plan->chunks, &set);
    plan->ws_bytes = std::max(plan->ws_bytes, set.bytes);
    plan->sets.push_back(std::move(set));
  }
  return MUON_OK;
}

// Workspace of a launch set: per chunk X0, X1 [K, s, ldx] and A, B [K, s, lda] in the NS element type
// (every piece 256-byte aligned), then the set's tile sums of squares (double) and one reciprocal norm per matrix.
void layout_set(const muon_options_t& opt, std::vector<Chunk>* chunks, LaunchSet* set) {
  const size_t eb = elem_bytes_of_ns(opt.ns_precision);
  size_t off = 0;
  int64_t parts = 0;
  for (int32_t ci : set->chunks) {
    Chunk& c = (*chunks)[size_t(ci)];
    const size_t xb = up(size_t(c.count) * c.s * c.ldx * eb, 256);
    const size_t ab = up(size_t(c.count) * c.s * c.lda * eb, 256);
    c.off_x[0] = off;
    c.off_x[1] = off + xb;
    c.off_a = off + 2 * xb;
    c.off_b = c.off_a + ab;
    off = c.off_b + ab;
    c.part_off = parts;
    // the wide elementwise kernels use 64 x 128 tiles (never more per matrix than the 64 x 64 count), so
    // tiles_per_mat partial sums per matrix cover both tilings
    parts += int64_t(c.count) * c.tiles_per_mat;
  }
  set->off_partials = off;
  off += up(size_t(parts) * sizeof(double), 256);
  set->off_rnorm = off;
  off += up(size_t(set->count) * sizeof(float), 256);
  set->bytes = off;
}

// Symmetric product over nb x nb blocks of 128 rows/columns.  Needed: every unordered pair {x, y}, x <= y,
// once (the epilogue mirrors off-diagonal blocks).  A tile is {ra, rb} x {cc, cd} (256 wide, four blocks) or
// {ra, rb} x {cc} (128 wide, two blocks).  256-wide tiles feed the tensor cores best (a 128-wide tile moves
// three quarters of the operand bytes for half the flops), so the list uses them wherever four useful blocks
// can be had, accepts one redundant block per diagonal 2 x 2 tile (1/(nb+1) of the work), and spends 128-wide
// tiles only on a last odd column, which a 256-wide tile would compute half empty:
//   column pairs (2j, 2j+1):  row pairs (2i, 2i+1), i < j: four needed blocks each;
//                             the diagonal tile {2j, 2j+1} x {2j, 2j+1}: three needed blocks, one computed twice;
//   last column L when nb is odd: {2i, 2i+1} x {L}, and {L, -} x {L} with an idle second CTA.
std::vector<TilePatHost> symmetric_tile_pattern(int nb) {
  std::vector<TilePatHost> tiles;
  const uint16_t none = 0xFFFFu;
  const int pairs = nb / 2;
  for (int j = 0; j < pairs; ++j)
    for (int i = 0; i <= j; ++i)
      tiles.push_back(TilePatHost{uint16_t(2 * i), uint16_t(2 * i + 1), uint16_t(2 * j), uint16_t(2 * j + 1)});
  if (nb % 2) {
    const int L = nb - 1;
    for (int i = 0; i < pairs; ++i) tiles.push_back(TilePatHost{uint16_t(2 * i), uint16_t(2 * i + 1), uint16_t(L), none});
    tiles.push_back(TilePatHost{uint16_t(L), none, uint16_t(L), none});
  }
  return tiles;
}

// Compute-owner assignment and batching of the owner-sharded step (Section 6.4 step 2; Section 6.7 and
// Algorithm 2).  Matrices are packed into batches in descending size (large matrices first, so that their result
// broadcasts have the longest window to hide in); a batch is closed when the next matrix would take it past
// batch_elems elements.  Inside a batch every matrix gets exactly one owner by greedy balancing of the
// Newton-Schulz work (longest processing time first: matrices in descending cost, each to the rank with the
// least work so far, lowest rank on ties), which keeps a batch's makespan within 4/3 - 1/(3 ranks) of optimal.
// The cost of a matrix is what the engine really computes per iteration: 3 s^2 l + s^3 multiply-adds.
int owner_plan_host(const muon_shape_t* shapes, int32_t count, int32_t ranks, int64_t batch_elems, int32_t* owner_of,
                    int32_t* batch_of, int32_t* num_batches) {
  if (count < 0 || ranks < 1 || (count > 0 && (!shapes || !owner_of || !batch_of)) || !num_batches) return MUON_ERR_INVALID_ARG;
  std::vector<int32_t> live;
  for (int32_t i = 0; i < count; ++i) {
    if (shapes[i].rows < 0 || shapes[i].cols < 0) return MUON_ERR_INVALID_ARG;
    owner_of[i] = batch_of[i] = -1;
    if (shapes[i].rows > 0 && shapes[i].cols > 0) live.push_back(i);
  }
  auto elems = [&](int32_t i) { return int64_t(shapes[i].rows) * shapes[i].cols; };
  auto cost = [&](int32_t i) {
    const double s = std::min(shapes[i].rows, shapes[i].cols), l = std::max(shapes[i].rows, shapes[i].cols);
    return 3.0 * s * s * l + s * s * s;
  };
  std::stable_sort(live.begin(), live.end(), [&](int32_t a, int32_t b) { return elems(a) > elems(b); });
  int32_t nb = 0;
  size_t pos = 0;
  while (pos < live.size()) {
    size_t end = pos;
    int64_t filled = 0;
    while (end < live.size() && (end == pos || batch_elems <= 0 || filled + elems(live[end]) <= batch_elems)) filled += elems(live[end++]);
    std::vector<int32_t> batch(live.begin() + long(pos), live.begin() + long(end));
    std::stable_sort(batch.begin(), batch.end(), [&](int32_t a, int32_t b) { return cost(a) > cost(b); });
    std::vector<double> load(static_cast<size_t>(ranks), 0.0);
    for (int32_t i : batch) {
      size_t best = 0;
      for (size_t r = 1; r < load.size(); ++r)
        if (load[r] < load[best]) best = r;
      load[best] += cost(i);
      owner_of[i] = int32_t(best);
      batch_of[i] = nb;
    }
    ++nb;
    pos = end;
  }
  *num_batches = nb;
  return MUON_OK;
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

// Do two strided views written by one call share an element?  View i covers, for every row r < rows, the bytes
// [base_i + r * ld * es, + cols * es).  Candidates are found by sweeping the views' bounding intervals in address order;
// a candidate pair is settled row by row (the rows of one view against the at most two rows of the other it can meet).
int views_overlap_host(const void* const* bases, const muon_view_t* views, int32_t count, int32_t elem_size) {
  struct Box {
    uintptr_t lo, hi;   // bounding interval [lo, hi)
    int32_t i;
  };
  std::vector<Box> boxes;
  boxes.reserve(size_t(count));
  const uintptr_t es = uintptr_t(elem_size);
  for (int32_t i = 0; i < count; ++i) {
    const muon_view_t& v = views[i];
    if (v.rows <= 0 || v.cols <= 0 || !bases[i]) continue;
    const uintptr_t lo = reinterpret_cast<uintptr_t>(bases[i]);
    boxes.push_back({lo, lo + (uintptr_t(v.rows - 1) * uintptr_t(v.ld) + uintptr_t(v.cols)) * es, i});
  }
  std::sort(boxes.begin(), boxes.end(), [](const Box& a, const Box& b) { return a.lo < b.lo || (a.lo == b.lo && a.i < b.i); });
  auto rows_meet = [&](const Box& a, const Box& b) {
    const muon_view_t& va = views[a.i];
    const muon_view_t& vb = views[b.i];
    const uintptr_t pa = uintptr_t(va.ld) * es, pb = uintptr_t(vb.ld) * es;
    const uintptr_t wa = uintptr_t(va.cols) * es, wb = uintptr_t(vb.cols) * es;
    for (int32_t r = 0; r < va.rows; ++r) {
      const uintptr_t lo = a.lo + uintptr_t(r) * pa, hi = lo + wa;
      if (hi <= b.lo || lo >= b.hi) continue;
      // rows of b that may meet [lo, hi): the one that starts last at or before lo, and every row starting inside
      int64_t j0 = lo > b.lo ? int64_t((lo - b.lo) / pb) : 0;
      for (int64_t j = j0; j < vb.rows; ++j) {
        const uintptr_t blo = b.lo + uintptr_t(j) * pb;
        if (blo >= hi) break;
        if (blo + wb > lo) return true;
      }
    }
    return false;
  };
  for (size_t x = 0; x < boxes.size(); ++x)
    for (size_t y = x + 1; y < boxes.size() && boxes[y].lo < boxes[x].hi; ++y)
      if (rows_meet(boxes[x], boxes[y])) return 1;
  return 0;
}

}  // namespace muon
