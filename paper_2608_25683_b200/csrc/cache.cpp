// Dynamic Block Caching (paper Sec. 5.2): host-side liveness of the KV blocks of one worker over
// an ordered list of micro-batches.  See include/psrl_cache.h for the rules.
#include <algorithm>
#include <cstdint>
#include <new>
#include <vector>

#include "../../include/psrl_cache.h"

namespace {

struct Extent {
  int64_t start, count;
};

struct Cache {
  int32_t n = 0, M = 0;
  int64_t capacity = 0;
  std::vector<int32_t> parent, seg_len, mb, group, bs, refcount, gbs;
  std::vector<int64_t> extent, base;       // base -1 = not resident
  std::vector<uint8_t> sample_end, evicted;
  std::vector<int32_t> use_off, use_list;  // CSR: micro-batches that read or write a block (its subtree's)
  std::vector<Extent> free_list;           // address order, coalesced
  int32_t next_mb = 0;
  bool in_mb = false, dead = false;
  psrl_cache_stats_t stats{};
  // buffers behind the borrowed pointers
  std::vector<int32_t> o_seg, o_parent, o_len, o_gbs, o_base, o_new, o_reload, o_evict, o_evict_base, o_freed, local;
  std::vector<uint8_t> o_flags;

  int64_t alloc(int64_t size) {
    for (size_t i = 0; i < free_list.size(); ++i) {
      Extent& e = free_list[i];
      if (e.count >= size) {
        const int64_t at = e.start;
        e.start += size;
        e.count -= size;
        if (e.count == 0) free_list.erase(free_list.begin() + i);
        return at;
      }
    }
    return -1;
  }
  void release(int64_t at, int64_t size) {
    auto it = std::lower_bound(free_list.begin(), free_list.end(), at,
                               [](const Extent& e, int64_t a) { return e.start < a; });
    it = free_list.insert(it, Extent{at, size});
    if (it + 1 != free_list.end() && it->start + it->count == (it + 1)->start) {
      it->count += (it + 1)->count;
      free_list.erase(it + 1);
    }
    if (it != free_list.begin() && (it - 1)->start + (it - 1)->count == it->start) {
      (it - 1)->count += it->count;
      free_list.erase(it);
    }
  }
  bool uses(int32_t s, int32_t m) const {
    return std::binary_search(use_list.begin() + use_off[s], use_list.begin() + use_off[s + 1], m);
  }
  int32_t next_use(int32_t s, int32_t m) const {  // first use after m, -1 if none
    auto b = use_list.begin() + use_off[s], e = use_list.begin() + use_off[s + 1];
    auto it = std::upper_bound(b, e, m);
    return it == e ? -1 : *it;
  }
  int64_t live() const {
    int64_t v = 0;
    for (int32_t s = 0; s < n; ++s)
      if (base[s] >= 0) v += extent[s];
    return v;
  }
};

}  // namespace

struct psrl_cache {
  Cache c;
};

extern "C" {

psrl_status_t psrl_cache_create(const psrl_cache_desc_t* d, psrl_cache_t** out) {
  if (out) *out = nullptr;
  if (!d || !out || d->n_segments < 1 || !d->parent || !d->seg_len || !d->group_block_size || !d->mb_of_seg ||
      d->n_microbatches < 1 || d->capacity_slots < 0 || d->capacity_slots % 16)
    return PSRL_ERR_INVALID_ARG;
  psrl_cache* h = new (std::nothrow) psrl_cache;
  if (!h) return PSRL_ERR_HOST_OOM;
  Cache& c = h->c;
  psrl_status_t st = PSRL_OK;
  try {
    const int32_t n = d->n_segments;
    c.n = n; c.M = d->n_microbatches; c.capacity = d->capacity_slots;
    c.parent.assign(d->parent, d->parent + n);
    c.seg_len.assign(d->seg_len, d->seg_len + n);
    c.mb.assign(d->mb_of_seg, d->mb_of_seg + n);
    std::vector<uint8_t> has_child(n, 0);
    std::vector<int32_t> roots;
    for (int32_t s = 0; s < n && st == PSRL_OK; ++s) {
      const int32_t p = c.parent[s];
      if (p == -1) roots.push_back(s);
      else if (p >= 0 && p < s) has_child[p] = 1;
      else st = PSRL_ERR_BAD_TREE;
      if (st == PSRL_OK && c.seg_len[s] < 1) st = PSRL_ERR_BAD_TREE;
      if (st == PSRL_OK && (c.mb[s] < 0 || c.mb[s] >= c.M)) st = PSRL_ERR_INVALID_ARG;
      if (st == PSRL_OK && p >= 0 && c.mb[p] > c.mb[s]) st = PSRL_ERR_BAD_TREE;
    }
    if (st == PSRL_OK && d->n_groups != static_cast<int32_t>(roots.size())) st = PSRL_ERR_INVALID_ARG;
    if (st == PSRL_OK)
      for (int32_t g = 0; g < d->n_groups; ++g) {
        const int32_t b = d->group_block_size[g];
        if (b != 0 && (b < 16 || b > 256 || (b & (b - 1)))) st = PSRL_ERR_BAD_BLOCK_SIZE;
      }
    if (st == PSRL_OK) {
      c.gbs.assign(d->group_block_size, d->group_block_size + d->n_groups);
      c.group.assign(n, 0); c.bs.assign(n, 0); c.extent.assign(n, 0);
      int32_t g = 0;
      for (int32_t s = 0; s < n; ++s) {
        c.group[s] = c.parent[s] == -1 ? g++ : c.group[c.parent[s]];
        c.bs[s] = c.gbs[c.group[s]];
        const int64_t unit = c.bs[s] ? c.bs[s] : 16;   // block size 0 = adaptive: the span at 16-slot granularity
        c.extent[s] = (int64_t(c.seg_len[s]) + unit - 1) / unit * unit;
        c.stats.total_slots += c.extent[s];
      }
      c.sample_end.assign(n, 0);
      for (int32_t s = 0; s < n; ++s) {
        c.sample_end[s] = d->seg_flags ? ((d->seg_flags[s] & PSRL_SEG_SAMPLE_END) ? 1 : 0) : !has_child[s];
        if (!has_child[s] && !c.sample_end[s]) st = PSRL_ERR_BAD_TREE;
      }
    }
    if (st == PSRL_OK) {
      // reference count = number of samples that will read the block
      c.refcount.assign(n, 0);
      for (int32_t e = 0; e < n; ++e)
        if (c.sample_end[e])
          for (int32_t s = e; s != -1; s = c.parent[s]) ++c.refcount[s];
      // micro-batches of every block's subtree
      std::vector<std::vector<int32_t>> u(n);
      for (int32_t s = 0; s < n; ++s)
        for (int32_t a = s; a != -1; a = c.parent[a]) u[a].push_back(c.mb[s]);
      c.use_off.assign(n + 1, 0);
      for (int32_t s = 0; s < n; ++s) {
        std::sort(u[s].begin(), u[s].end());
        u[s].erase(std::unique(u[s].begin(), u[s].end()), u[s].end());
        c.use_off[s + 1] = c.use_off[s] + static_cast<int32_t>(u[s].size());
        c.use_list.insert(c.use_list.end(), u[s].begin(), u[s].end());
      }
      c.base.assign(n, -1);
      c.evicted.assign(n, 0);
      c.free_list.push_back(Extent{0, c.capacity ? c.capacity : (int64_t(1) << 40)});
      c.local.assign(n, -1);
    }
  } catch (const std::bad_alloc&) {
    st = PSRL_ERR_HOST_OOM;
  }
  if (st != PSRL_OK) {
    delete h;
    return st;
  }
  *out = h;
  return PSRL_OK;
}

psrl_status_t psrl_cache_begin(psrl_cache_t* h, int32_t m, psrl_cache_step_t* out) {
  if (!h || !out) return PSRL_ERR_INVALID_ARG;
  Cache& c = h->c;
  if (c.dead || c.in_mb || m != c.next_mb || m >= c.M) return PSRL_ERR_INVALID_ARG;
  try {
    c.o_seg.clear(); c.o_new.clear(); c.o_reload.clear(); c.o_evict.clear(); c.o_evict_base.clear();
    for (int32_t s = 0; s < c.n; ++s)
      if (c.uses(s, m)) c.o_seg.push_back(s);
    std::fill(c.local.begin(), c.local.end(), -1);
    for (size_t i = 0; i < c.o_seg.size(); ++i) c.local[c.o_seg[i]] = static_cast<int32_t>(i);
    for (int32_t s : c.o_seg) {
      if (c.base[s] >= 0) continue;
      int64_t at;
      while ((at = c.alloc(c.extent[s])) < 0) {
        // evict the resident block, not used now, whose next use lies farthest ahead
        int32_t victim = -1, far = -1;
        for (int32_t r = 0; r < c.n; ++r) {
          if (c.base[r] < 0 || c.local[r] >= 0) continue;
          const int32_t nu = c.next_use(r, m);
          if (nu > far || (nu == far && r > victim)) { far = nu; victim = r; }
        }
        if (victim < 0) {
          c.dead = true;
          return PSRL_ERR_POOL_FULL;
        }
        c.o_evict.push_back(victim);
        c.o_evict_base.push_back(static_cast<int32_t>(c.base[victim]));
        c.release(c.base[victim], c.extent[victim]);
        c.base[victim] = -1;
        c.evicted[victim] = 1;
        c.stats.evicted_slots += c.extent[victim];
      }
      if (at + c.extent[s] > INT32_MAX / 2) { c.dead = true; return PSRL_ERR_SHAPE; }
      c.base[s] = at;
      c.stats.pool_high_water = std::max(c.stats.pool_high_water, at + c.extent[s]);
      if (c.evicted[s]) {
        c.evicted[s] = 0;
        c.o_reload.push_back(s);
        c.stats.reloaded_slots += c.extent[s];
      } else {
        if (c.mb[s] != m) { c.dead = true; return PSRL_ERR_INTERNAL; }
        c.o_new.push_back(s);
      }
    }
    const size_t k = c.o_seg.size();
    c.o_parent.assign(k, -1); c.o_len.assign(k, 0); c.o_base.assign(k, 0); c.o_flags.assign(k, 0); c.o_gbs.clear();
    std::vector<uint8_t> has_child(k, 0);
    int64_t top = 0;
    for (size_t i = 0; i < k; ++i) {
      const int32_t s = c.o_seg[i];
      if (c.parent[s] >= 0) {
        c.o_parent[i] = c.local[c.parent[s]];
        has_child[c.o_parent[i]] = 1;
      } else {
        c.o_gbs.push_back(c.gbs[c.group[s]]);
      }
      c.o_len[i] = c.seg_len[s];
      c.o_base[i] = static_cast<int32_t>(c.base[s]);
      top = std::max(top, c.base[s] + c.extent[s]);
    }
    for (size_t i = 0; i < k; ++i) {
      const int32_t s = c.o_seg[i];
      const bool active = c.mb[s] == m;
      uint8_t f = active ? PSRL_SEG_HAS_Q : 0;
      if (!has_child[i] || (active && c.sample_end[s])) f |= PSRL_SEG_SAMPLE_END;
      c.o_flags[i] = f;
    }
    const int64_t live = c.live();
    c.stats.peak_slots = std::max(c.stats.peak_slots, live);
    out->n_segments = static_cast<int32_t>(k);
    out->seg_id = c.o_seg.data(); out->parent = c.o_parent.data(); out->seg_len = c.o_len.data();
    out->seg_flags = c.o_flags.data(); out->group_block_size = c.o_gbs.data();
    out->n_groups = static_cast<int32_t>(c.o_gbs.size()); out->seg_slot_base = c.o_base.data();
    out->n_new = static_cast<int32_t>(c.o_new.size()); out->n_reload = static_cast<int32_t>(c.o_reload.size());
    out->n_evict = static_cast<int32_t>(c.o_evict.size());
    out->new_seg = c.o_new.data(); out->reload_seg = c.o_reload.data();
    out->evict_seg = c.o_evict.data(); out->evict_base = c.o_evict_base.data();
    out->live_slots = live; out->pool_slots = top;
  } catch (const std::bad_alloc&) {
    c.dead = true;
    return PSRL_ERR_HOST_OOM;
  }
  c.in_mb = true;
  return PSRL_OK;
}

psrl_status_t psrl_cache_end(psrl_cache_t* h, int32_t m, int32_t* n_freed, const int32_t** freed_seg,
                             int64_t* live_slots) {
  if (!h) return PSRL_ERR_INVALID_ARG;
  Cache& c = h->c;
  if (c.dead || !c.in_mb || m != c.next_mb) return PSRL_ERR_INVALID_ARG;
  // remove the reference entries of the samples that completed in this micro-batch
  for (int32_t e = 0; e < c.n; ++e)
    if (c.sample_end[e] && c.mb[e] == m)
      for (int32_t s = e; s != -1; s = c.parent[s]) --c.refcount[s];
  c.o_freed.clear();
  for (int32_t s = 0; s < c.n; ++s) {
    if (c.refcount[s] != 0) continue;
    if (c.base[s] >= 0) {
      c.release(c.base[s], c.extent[s]);
      c.base[s] = -1;
      c.o_freed.push_back(s);
    }
    c.evicted[s] = 0;
  }
  c.in_mb = false;
  ++c.next_mb;
  if (n_freed) *n_freed = static_cast<int32_t>(c.o_freed.size());
  if (freed_seg) *freed_seg = c.o_freed.data();
  if (live_slots) *live_slots = c.live();
  return PSRL_OK;
}

psrl_status_t psrl_cache_stats(const psrl_cache_t* h, psrl_cache_stats_t* out) {
  if (!h || !out) return PSRL_ERR_INVALID_ARG;
  *out = h->c.stats;
  return PSRL_OK;
}

psrl_status_t psrl_cache_refcounts(const psrl_cache_t* h, const int32_t** refcount) {
  if (!h || !refcount) return PSRL_ERR_INVALID_ARG;
  *refcount = h->c.refcount.data();
  return PSRL_OK;
}

void psrl_cache_destroy(psrl_cache_t* h) { delete h; }

}  // extern "C"
