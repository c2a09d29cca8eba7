// Host-side page registry (Sec. 4.3: a block's key is the model name plus its cumulative
// prefix hash): chained block hash -> byte offset of the block's page-first slab in the
// pinned host pool.  Open addressing with linear probing and tombstones; pure host code
// (the hashes arrive in host memory from talaria_prefix_match_host).  The model-name part
// of the key is already folded into the chained hash through its seed.
#include <cstdint>
#include <cstring>
#include <mutex>
#include <new>
#include <vector>

#include "talaria.h"

namespace {
enum : uint8_t { kEmpty = 0, kFull = 1, kTomb = 2 };

inline uint64_t spread(uint64_t h) {      // the keys are already well mixed; fold the high half in anyway
  return h ^ (h >> 32);
}
}  // namespace

struct talaria_registry {
  std::mutex mu;
  std::vector<uint64_t> keys;
  std::vector<int64_t> vals;
  std::vector<uint8_t> state;
  int64_t live = 0, used = 0;             // used counts full slots and tombstones
  uint64_t mask = 0;

  bool init(int64_t slots) {
    uint64_t cap = 16;
    while ((int64_t)cap < slots) cap <<= 1;
    try {
      keys.assign(cap, 0);
      vals.assign(cap, 0);
      state.assign(cap, kEmpty);
    } catch (const std::bad_alloc &) {
      return false;
    }
    mask = cap - 1;
    live = used = 0;
    return true;
  }
  // slot of key, or -1
  int64_t find(uint64_t key) const {
    for (uint64_t s = spread(key) & mask;; s = (s + 1) & mask) {
      if (state[s] == kEmpty) return -1;
      if (state[s] == kFull && keys[s] == key) return (int64_t)s;
    }
  }
  bool grow_if_needed() {
    if ((uint64_t)(used + 1) * 10 <= (mask + 1) * 7) return true;
    // the new table is built aside and swapped in only when it is complete, so a failed
    // allocation leaves the old one intact
    talaria_registry bigger;
    const int64_t want = live * 4 > 16 ? live * 4 : 16;      // also sheds tombstones
    if (!bigger.init(want)) return false;
    for (size_t s = 0; s < state.size(); ++s)
      if (state[s] == kFull) bigger.put(keys[s], vals[s]);
    keys.swap(bigger.keys);
    vals.swap(bigger.vals);
    state.swap(bigger.state);
    live = bigger.live;
    used = bigger.used;
    mask = bigger.mask;
    return true;
  }
  // first wins; returns true if the key is new
  bool put(uint64_t key, int64_t val) {
    for (uint64_t s = spread(key) & mask;; s = (s + 1) & mask) {
      if (state[s] == kFull && keys[s] == key) return false;
      if (state[s] == kEmpty) {
        keys[s] = key;
        vals[s] = val;
        state[s] = kFull;
        ++live;
        ++used;
        return true;
      }
    }
  }
};

extern "C" talaria_status_t talaria_registry_create(talaria_registry **out, int64_t expected_pages) {
  if (!out || expected_pages < 0) return TALARIA_ERR_INVALID_ARG;
  *out = nullptr;
  talaria_registry *r = new (std::nothrow) talaria_registry();
  if (!r) return TALARIA_ERR_NO_MEMORY;
  if (!r->init(expected_pages * 2)) {
    delete r;
    return TALARIA_ERR_NO_MEMORY;
  }
  *out = r;
  return TALARIA_OK;
}

extern "C" talaria_status_t talaria_registry_destroy(talaria_registry *r) {
  if (!r) return TALARIA_ERR_INVALID_ARG;
  delete r;
  return TALARIA_OK;
}

extern "C" talaria_status_t talaria_registry_insert(talaria_registry *r, const uint64_t *hashes,
                                                    const int64_t *page_offsets, int64_t n, int64_t *n_new) {
  if (!r || n < 0 || (n > 0 && (!hashes || !page_offsets))) return TALARIA_ERR_INVALID_ARG;
  std::lock_guard<std::mutex> lk(r->mu);
  int64_t added = 0;
  for (int64_t k = 0; k < n; ++k) {
    if (!r->grow_if_needed()) return TALARIA_ERR_NO_MEMORY;
    if (r->put(hashes[k], page_offsets[k])) ++added;
  }
  if (n_new) *n_new = added;
  return TALARIA_OK;
}

extern "C" int64_t talaria_registry_lookup_prefix(talaria_registry *r, const uint64_t *hashes, int64_t n,
                                                  int64_t *page_offsets_out) {
  if (!r || n <= 0 || !hashes) return 0;
  std::lock_guard<std::mutex> lk(r->mu);
  int64_t k = 0;
  for (; k < n; ++k) {
    const int64_t s = r->find(hashes[k]);
    if (s < 0) break;
    if (page_offsets_out) page_offsets_out[k] = r->vals[(size_t)s];
  }
  return k;
}

extern "C" talaria_status_t talaria_registry_erase(talaria_registry *r, const uint64_t *hashes, int64_t n,
                                                   int64_t *n_erased) {
  if (!r || n < 0 || (n > 0 && !hashes)) return TALARIA_ERR_INVALID_ARG;
  std::lock_guard<std::mutex> lk(r->mu);
  int64_t gone = 0;
  for (int64_t k = 0; k < n; ++k) {
    const int64_t s = r->find(hashes[k]);
    if (s >= 0) {
      r->state[(size_t)s] = kTomb;
      --r->live;
      ++gone;
    }
  }
  if (n_erased) *n_erased = gone;
  return TALARIA_OK;
}

extern "C" int64_t talaria_registry_size(talaria_registry *r) {
  if (!r) return 0;
  std::lock_guard<std::mutex> lk(r->mu);
  return r->live;
}
