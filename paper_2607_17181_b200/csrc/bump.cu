// Stable-address HBM layout (Sec. 4.2 "bump-managed HBM layout"; Sec. 4.4 staging surface).
//
// One managed region serves every model of a cold-pool instance.  For the active model the
// weights grow up from the low end, the runtime buffers are anchored at the high end and the gap
// between them is the paged KV pool: num_layers * num_planes planes of num_blocks rows, a row
// being one block's chunk.  Every address is a pure function of (region, model), so a model
// finds its weights, KV planes and runtime buffers at the same addresses each time it is
// activated -- the property the paper's restore-time pointer check relies on.
//
// Block ids are handed out lowest first, which keeps the high rows of every plane clean; those
// tails are the staging surface for the next model's weights.  A staged chunk occupies a run of
// rows in ONE plane.  The allocator skips rows under an active staging write, and an allocation
// that takes rows of a staged chunk marks that chunk dirty.
//
// Pure host arithmetic: nothing here touches the GPU; `region_base` is only a number.
#include <algorithm>
#include <cstdint>
#include <mutex>
#include <new>
#include <set>
#include <vector>

#include "talaria.h"

namespace {

struct Slot {              // rows [row0, row0 + rows) of one plane hold one staged chunk
  int32_t plane;
  int64_t row0;
};

inline int64_t up(int64_t x, int64_t a) { return (x + a - 1) / a * a; }
inline bool bit(const uint8_t *bm, int64_t i) { return (bm[i >> 3] >> (i & 7)) & 1; }

}  // namespace

struct talaria_bump {
  std::mutex mu;
  uintptr_t base = 0;
  int64_t bytes = 0, align = 256;
  std::vector<talaria_model_desc_t> models;
  // state of the active model
  int32_t active = -1;
  int64_t num_blocks = 0;
  std::set<int32_t> free_ids;
  // staging placement for the next model (cleared by every activation)
  int32_t next_model = -1;
  int64_t stage_chunk = 0, rows_per_chunk = 0;
  std::vector<Slot> chunk_slot;                     // per chunk id; plane < 0 = not placed
  std::vector<std::vector<int32_t>> slot_chunk;     // [plane][tail slot] -> chunk id or -1
  std::vector<uint8_t> locked;                      // per chunk id: a staging write is in flight

  // ---- the layout of one model: a pure function ---------------------------------------
  talaria_status_t plan(int32_t m, talaria_bump_view_t *v) const {
    if (m < 0 || m >= (int32_t)models.size()) return TALARIA_ERR_INVALID_ARG;
    const talaria_model_desc_t &d = models[(size_t)m];
    const int64_t lp = (int64_t)d.num_layers * d.num_planes;
    const int64_t kv_off = up(d.weight_bytes, align);
    const int64_t rt_off = (bytes - d.runtime_bytes) / align * align;       // anchored high, aligned down
    if (rt_off < kv_off) return TALARIA_ERR_EXTENT;
    const int64_t nb = (rt_off - kv_off) / (lp * d.chunk_bytes);
    if (nb < 1) return TALARIA_ERR_EXTENT;
    v->weights_base = (void *)base;
    v->weights_bytes = d.weight_bytes;
    v->kv_base = (void *)(base + (uintptr_t)kv_off);
    v->kv_bytes = lp * nb * d.chunk_bytes;
    v->runtime_base = (void *)(base + (uintptr_t)rt_off);
    v->runtime_bytes = d.runtime_bytes;
    v->num_blocks = nb;
    return TALARIA_OK;
  }
  int64_t plane_off(const talaria_bump_view_t &v, const talaria_model_desc_t &d, int64_t k) const {
    return (int64_t)((uintptr_t)v.kv_base - base) + k * v.num_blocks * d.chunk_bytes;
  }
  // busy[r] = 1 when row r is allocated or lies under a staging write in flight; prefix sums of it
  // answer "is every row of [r0, r1) free and unlocked" in constant time
  std::vector<int32_t> busy_prefix() const {
    std::vector<uint8_t> busy((size_t)num_blocks, 1);
    for (int32_t id : free_ids) busy[(size_t)id] = 0;
    for (size_t c = 0; c < locked.size(); ++c)
      if (locked[c] && chunk_slot[c].plane >= 0)
        for (int64_t r = chunk_slot[c].row0; r < chunk_slot[c].row0 + rows_per_chunk; ++r) busy[(size_t)r] = 1;
    std::vector<int32_t> pre((size_t)num_blocks + 1, 0);
    for (int64_t r = 0; r < num_blocks; ++r) pre[(size_t)r + 1] = pre[(size_t)r] + busy[(size_t)r];
    return pre;
  }
};

extern "C" talaria_status_t talaria_bump_create(talaria_bump **out, void *region_base, int64_t region_bytes,
                                                int64_t align, const talaria_model_desc_t *models,
                                                int32_t n_models) {
  if (!out) return TALARIA_ERR_INVALID_ARG;
  *out = nullptr;
  if (region_bytes <= 0 || align <= 0 || (align & (align - 1)) != 0 || n_models <= 0 || !models ||
      ((uintptr_t)region_base & (uintptr_t)(align - 1)) != 0)
    return TALARIA_ERR_INVALID_ARG;
  talaria_bump *b = new (std::nothrow) talaria_bump();
  if (!b) return TALARIA_ERR_NO_MEMORY;
  b->base = (uintptr_t)region_base;
  b->bytes = region_bytes;
  b->align = align;
  b->models.assign(models, models + n_models);
  for (int32_t m = 0; m < n_models; ++m) {
    const talaria_model_desc_t &d = models[m];
    talaria_bump_view_t v;
    talaria_status_t st = TALARIA_ERR_INVALID_ARG;
    if (d.weight_bytes >= 0 && d.runtime_bytes >= 0 && d.num_layers > 0 && d.num_planes > 0 && d.chunk_bytes > 0 &&
        d.chunk_bytes % align == 0)
      st = b->plan(m, &v);                       // every model must fit the region on its own
    if (st != TALARIA_OK) {
      delete b;
      return st;
    }
  }
  *out = b;
  return TALARIA_OK;
}

extern "C" talaria_status_t talaria_bump_destroy(talaria_bump *b) {
  if (!b) return TALARIA_ERR_INVALID_ARG;
  delete b;
  return TALARIA_OK;
}

extern "C" talaria_status_t talaria_bump_view(talaria_bump *b, int32_t model, talaria_bump_view_t *view,
                                              void **plane_base_out) {
  if (!b || !view) return TALARIA_ERR_INVALID_ARG;
  std::lock_guard<std::mutex> lk(b->mu);
  talaria_status_t st = b->plan(model, view);
  if (st != TALARIA_OK) return st;
  if (plane_base_out) {
    const talaria_model_desc_t &d = b->models[(size_t)model];
    for (int64_t k = 0; k < (int64_t)d.num_layers * d.num_planes; ++k)
      plane_base_out[k] = (void *)(b->base + (uintptr_t)b->plane_off(*view, d, k));
  }
  return TALARIA_OK;
}

extern "C" talaria_status_t talaria_bump_activate(talaria_bump *b, int32_t model, talaria_bump_view_t *view) {
  if (!b) return TALARIA_ERR_INVALID_ARG;
  std::lock_guard<std::mutex> lk(b->mu);
  talaria_bump_view_t v;
  talaria_status_t st = b->plan(model, &v);
  if (st != TALARIA_OK) return st;
  b->active = model;
  b->num_blocks = v.num_blocks;
  b->free_ids.clear();
  for (int64_t i = 0; i < v.num_blocks; ++i) b->free_ids.insert(b->free_ids.end(), (int32_t)i);
  b->next_model = -1;
  b->chunk_slot.clear();
  b->slot_chunk.clear();
  b->locked.clear();
  b->stage_chunk = b->rows_per_chunk = 0;
  if (view) *view = v;
  return TALARIA_OK;
}

extern "C" talaria_status_t talaria_bump_alloc_blocks(talaria_bump *b, int64_t n, int32_t *ids_out,
                                                      const uint8_t *staged_bitmap, uint8_t *dirty_bitmap,
                                                      int64_t *n_dirtied) {
  if (!b || n < 0 || (n > 0 && !ids_out)) return TALARIA_ERR_INVALID_ARG;
  std::lock_guard<std::mutex> lk(b->mu);
  if (b->active < 0) return TALARIA_ERR_INVALID_ARG;
  if (n_dirtied) *n_dirtied = 0;
  // lowest ids first; rows under an active staging write are passed over
  std::vector<int32_t> got;
  got.reserve((size_t)n);
  bool any_lock = false;
  for (uint8_t l : b->locked) any_lock |= l != 0;
  std::vector<int32_t> pre;
  if (any_lock) pre = b->busy_prefix();
  for (auto it = b->free_ids.begin(); it != b->free_ids.end() && (int64_t)got.size() < n; ++it)
    if (!any_lock || pre[(size_t)*it + 1] == pre[(size_t)*it]) got.push_back(*it);
  if ((int64_t)got.size() < n) return TALARIA_ERR_NO_MEMORY;          // nothing is taken
  int64_t dirtied = 0;
  const int64_t lp = (int64_t)b->slot_chunk.size();
  for (int32_t id : got) {
    b->free_ids.erase(id);
    if (!dirty_bitmap || b->rows_per_chunk <= 0) continue;
    // block id = row index in EVERY plane: the tail slot that holds this row, plane by plane
    const int64_t t = (b->num_blocks - 1 - id) / b->rows_per_chunk;
    for (int64_t k = 0; k < lp; ++k) {
      if (t >= (int64_t)b->slot_chunk[(size_t)k].size()) continue;
      const int32_t c = b->slot_chunk[(size_t)k][(size_t)t];
      if (c < 0) continue;
      if (staged_bitmap && !bit(staged_bitmap, c)) continue;
      if (!bit(dirty_bitmap, c)) {
        dirty_bitmap[c >> 3] |= (uint8_t)(1u << (c & 7));
        ++dirtied;
      }
    }
  }
  std::copy(got.begin(), got.end(), ids_out);
  if (n_dirtied) *n_dirtied = dirtied;
  return TALARIA_OK;
}

extern "C" talaria_status_t talaria_bump_free_blocks(talaria_bump *b, const int32_t *ids, int64_t n) {
  if (!b || n < 0 || (n > 0 && !ids)) return TALARIA_ERR_INVALID_ARG;
  std::lock_guard<std::mutex> lk(b->mu);
  for (int64_t i = 0; i < n; ++i)
    if (ids[i] < 0 || ids[i] >= b->num_blocks || b->free_ids.count(ids[i])) return TALARIA_ERR_INVALID_ARG;
  for (int64_t i = 0; i < n; ++i)
    if (!b->free_ids.insert(ids[i]).second) return TALARIA_ERR_INVALID_ARG;   // the same id twice in one call
  return TALARIA_OK;
}

extern "C" int64_t talaria_bump_free_count(talaria_bump *b) {
  if (!b) return 0;
  std::lock_guard<std::mutex> lk(b->mu);
  return (int64_t)b->free_ids.size();
}

// Tail slot t of plane k is rows [NB - (t+1)*rpc, NB - t*rpc).  It can take a chunk when all of its
// rows are free and unlocked and none of its bytes lies inside the NEXT model's weights region
// (the switch copies staged chunks into that region, so a source there would be overwritten).
static bool slot_usable(const talaria_bump *b, const talaria_bump_view_t &v, const talaria_model_desc_t &d,
                        const std::vector<int32_t> &busy_pre, int64_t next_weights_end, int64_t k, int64_t t) {
  const int64_t row0 = b->num_blocks - (t + 1) * b->rows_per_chunk;
  if (row0 < 0) return false;
  if (b->plane_off(v, d, k) + row0 * d.chunk_bytes < next_weights_end) return false;
  return busy_pre[(size_t)(row0 + b->rows_per_chunk)] == busy_pre[(size_t)row0];
}

extern "C" talaria_status_t talaria_bump_stage_place(talaria_bump *b, int32_t next_model, int64_t chunk_bytes,
                                                     const void *host_weights, talaria_copy_t *plan_out,
                                                     int64_t plan_capacity, int64_t *n_chunks_out,
                                                     int64_t *n_placed_out) {
  if (!b || chunk_bytes <= 0 || !n_chunks_out) return TALARIA_ERR_INVALID_ARG;
  std::lock_guard<std::mutex> lk(b->mu);
  if (b->active < 0 || next_model < 0 || next_model >= (int32_t)b->models.size() || next_model == b->active)
    return TALARIA_ERR_INVALID_ARG;
  const talaria_model_desc_t &d = b->models[(size_t)b->active];
  const talaria_model_desc_t &nx = b->models[(size_t)next_model];
  const int64_t n_chunks = (nx.weight_bytes + chunk_bytes - 1) / chunk_bytes;
  *n_chunks_out = n_chunks;
  if (n_chunks > 0x7fffffffll) return TALARIA_ERR_INVALID_ARG;
  if (!plan_out || plan_capacity < n_chunks) return TALARIA_ERR_EXTENT;
  talaria_bump_view_t v, vn;
  talaria_status_t st = b->plan(b->active, &v);
  if (st == TALARIA_OK) st = b->plan(next_model, &vn);
  if (st != TALARIA_OK) return st;
  const int64_t lp = (int64_t)d.num_layers * d.num_planes;
  b->next_model = next_model;
  b->stage_chunk = chunk_bytes;
  b->rows_per_chunk = (chunk_bytes + d.chunk_bytes - 1) / d.chunk_bytes;
  b->chunk_slot.assign((size_t)n_chunks, Slot{-1, 0});
  b->locked.assign((size_t)n_chunks, 0);
  const int64_t max_slots = b->num_blocks / b->rows_per_chunk;
  b->slot_chunk.assign((size_t)lp, std::vector<int32_t>((size_t)max_slots, -1));
  const int64_t next_weights_end = up(nx.weight_bytes, b->align);
  const std::vector<int32_t> pre = b->busy_prefix();       // no chunk is placed or locked yet: allocated rows only
  // slots are taken tail slot by tail slot across all planes, so every tail stays equally shallow
  int64_t c = 0;
  for (int64_t t = 0; t < max_slots && c < n_chunks; ++t)
    for (int64_t k = 0; k < lp && c < n_chunks; ++k) {
      if (!slot_usable(b, v, d, pre, next_weights_end, k, t)) continue;
      b->chunk_slot[(size_t)c] = Slot{(int32_t)k, b->num_blocks - (t + 1) * b->rows_per_chunk};
      b->slot_chunk[(size_t)k][(size_t)t] = (int32_t)c;
      ++c;
    }
  for (int64_t j = 0; j < n_chunks; ++j) {
    const Slot &s = b->chunk_slot[(size_t)j];
    talaria_copy_t &e = plan_out[j];
    const int64_t off = j * chunk_bytes;
    e.bytes = std::min(chunk_bytes, nx.weight_bytes - off);
    e.chunk_id = (int32_t)j;
    e.reserved = 0;
    e.dst_dev = (void *)((uintptr_t)vn.weights_base + (uintptr_t)off);
    e.src_host = host_weights ? (const void *)((const char *)host_weights + off) : nullptr;
    e.src_dev = s.plane < 0 ? nullptr
                            : (const void *)(b->base + (uintptr_t)(b->plane_off(v, d, s.plane) + s.row0 * d.chunk_bytes));
  }
  if (n_placed_out) *n_placed_out = c;
  return TALARIA_OK;
}

extern "C" talaria_status_t talaria_bump_lock_chunk(talaria_bump *b, int32_t chunk_id, int32_t locked) {
  if (!b) return TALARIA_ERR_INVALID_ARG;
  std::lock_guard<std::mutex> lk(b->mu);
  if (chunk_id < 0 || chunk_id >= (int32_t)b->locked.size()) return TALARIA_ERR_INVALID_ARG;
  b->locked[(size_t)chunk_id] = locked ? 1 : 0;
  return TALARIA_OK;
}

extern "C" int64_t talaria_bump_staging_slack(talaria_bump *b, int32_t next_model, int64_t chunk_bytes) {
  if (!b || chunk_bytes <= 0) return 0;
  std::lock_guard<std::mutex> lk(b->mu);
  if (b->active < 0 || next_model < 0 || next_model >= (int32_t)b->models.size()) return 0;
  const talaria_model_desc_t &d = b->models[(size_t)b->active];
  talaria_bump_view_t v;
  if (b->plan(b->active, &v) != TALARIA_OK) return 0;
  // count with this chunk size, without disturbing an existing placement
  const std::vector<int32_t> pre = b->busy_prefix();
  const int64_t saved = b->rows_per_chunk;
  b->rows_per_chunk = (chunk_bytes + d.chunk_bytes - 1) / d.chunk_bytes;
  const int64_t lp = (int64_t)d.num_layers * d.num_planes, max_slots = b->num_blocks / b->rows_per_chunk;
  const int64_t next_weights_end = up(b->models[(size_t)next_model].weight_bytes, b->align);
  int64_t slots = 0;
  for (int64_t t = 0; t < max_slots; ++t)
    for (int64_t k = 0; k < lp; ++k) {
      const bool used = saved == b->rows_per_chunk && k < (int64_t)b->slot_chunk.size() &&
                        t < (int64_t)b->slot_chunk[(size_t)k].size() && b->slot_chunk[(size_t)k][(size_t)t] >= 0;
      if (!used && slot_usable(b, v, d, pre, next_weights_end, k, t)) ++slots;
    }
  b->rows_per_chunk = saved;
  return slots * chunk_bytes;
}
