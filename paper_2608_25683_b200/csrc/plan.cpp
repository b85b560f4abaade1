// Host-side plan builder: prefix forest -> canonical plan (paged block table
// with a block size per group, reference counts) + device work schedule.
//
// Paper Sec. 5.1 (Adaptive Block Allocation): block boundaries follow the
// reusable prefix spans, so pages never straddle a segment boundary and a
// shared span is materialised once.  Sec. 6 (KV manager): per-block metadata
// = base address (page_slot), block size (page_bs / page_valid), position of
// the span in the full sequence (page_pos), reference count.  Sec. 5.2: the
// reference count is the number of samples that will read the block.  Eq. 1:
// the attention cost of a sequence is l_suf * l; the exact per-segment form
// len*anc + len(len+1)/2 is used for the pair statistics and the tile costs
// that order the work lists longest-first (the paper's greedy placement sorts
// by estimated workload, Sec. 4.2).
#include "plan.h"

#include <algorithm>
#include <new>
#include <numeric>

namespace psrl {
namespace {

bool pow2_in_range(int32_t b) { return b >= 16 && b <= 256 && (b & (b - 1)) == 0; }

struct Extent {
  int64_t start, count;
};

template <class T>
int32_t append_array(std::vector<int32_t>& blob, const std::vector<T>& v) {
  // every array starts on a 16-byte boundary
  while (blob.size() % 4) blob.push_back(0);
  int32_t off = static_cast<int32_t>(blob.size());
  const int32_t* p = reinterpret_cast<const int32_t*>(v.data());
  blob.insert(blob.end(), p, p + v.size() * (sizeof(T) / sizeof(int32_t)));
  return off;
}

}  // namespace

psrl_status_t build_plan(const psrl_tree_desc_t& desc, Plan*& out) {
  out = nullptr;
  const int32_t n = desc.n_segments;
  if (n < 1 || !desc.parent || !desc.seg_len || !desc.group_block_size) return PSRL_ERR_INVALID_ARG;
  if (desc.n_free < 0 || (desc.n_free > 0 && !desc.free_extents)) return PSRL_ERR_INVALID_ARG;
  if (desc.n_q_heads < 1 || desc.n_kv_heads < 1 || desc.n_q_heads % desc.n_kv_heads) return PSRL_ERR_SHAPE;
  if (desc.dtype == PSRL_F32) {
    if (desc.head_dim != 64 && desc.head_dim != 128) return PSRL_ERR_UNSUPPORTED;
  } else if (desc.dtype == PSRL_BF16) {
    if (desc.head_dim != 128) return PSRL_ERR_UNSUPPORTED;
  } else {
    return PSRL_ERR_UNSUPPORTED;
  }

  Plan* pl = new (std::nothrow) Plan();
  if (!pl) return PSRL_ERR_HOST_OOM;
  struct Guard {
    Plan* p;
    ~Guard() { delete p; }
  } guard{pl};
  try {
    Plan& P = *pl;
    P.Hq = desc.n_q_heads;
    P.Hkv = desc.n_kv_heads;
    P.d = desc.head_dim;
    P.dtype = desc.dtype;
    P.n_seg = n;

    // ---- validate the tree, collect children (ascending input index) ----
    std::vector<int32_t> first_child(n, -1), next_sibling(n, -1), last_child(n, -1), roots;
    for (int32_t s = 0; s < n; ++s) {
      const int32_t p = desc.parent[s];
      if (!(p == -1 || (p >= 0 && p < s))) return PSRL_ERR_BAD_TREE;
      if (desc.seg_len[s] < 1) return PSRL_ERR_BAD_TREE;
      if (p == -1) {
        roots.push_back(s);
      } else {
        if (first_child[p] < 0) first_child[p] = s; else next_sibling[last_child[p]] = s;
        last_child[p] = s;
      }
    }
    std::vector<int32_t> in_flags(n);
    for (int32_t s = 0; s < n; ++s) {
      const bool leaf = first_child[s] < 0;
      int32_t f = desc.seg_flags ? desc.seg_flags[s] : (PSRL_SEG_HAS_Q | (leaf ? PSRL_SEG_SAMPLE_END : 0));
      if (f & ~(PSRL_SEG_HAS_Q | PSRL_SEG_SAMPLE_END)) return PSRL_ERR_INVALID_ARG;
      if (leaf && !(f & PSRL_SEG_SAMPLE_END)) return PSRL_ERR_BAD_TREE;
      in_flags[s] = f;
    }
    P.n_groups = static_cast<int32_t>(roots.size());
    if (desc.n_groups != P.n_groups) return PSRL_ERR_INVALID_ARG;
    for (int32_t g = 0; g < P.n_groups; ++g)
      if (desc.group_block_size[g] != 0 && !pow2_in_range(desc.group_block_size[g])) return PSRL_ERR_BAD_BLOCK_SIZE;
    for (int32_t g = 0; g < P.n_groups; ++g)  // adaptive blocks: tensor-core path only
      if (desc.group_block_size[g] == 0 && desc.dtype != PSRL_BF16) return PSRL_ERR_UNSUPPORTED;
    std::vector<Extent> extents;
    const bool bump = desc.free_extents == nullptr;
    for (int32_t i = 0; i < desc.n_free; ++i) {
      const int64_t a = desc.free_extents[2 * i], c = desc.free_extents[2 * i + 1];
      if (a < 0 || c < 0 || a % 16 || c % 16) return PSRL_ERR_INVALID_ARG;
      extents.push_back({a, c});
    }

    if (desc.seg_slot_base)
      for (int32_t s = 0; s < n; ++s) {
        const int64_t b = desc.seg_slot_base[s];
        if (b < -1 || (b >= 0 && b % 16)) return PSRL_ERR_INVALID_ARG;
      }

    // ---- canonical order: preorder walk with sibling links ----
    P.input_of_canon.reserve(n);
    P.canon_of_input.assign(n, -1);
    P.seg_group.reserve(n);
    for (int32_t g = 0; g < P.n_groups; ++g) {
      int32_t s = roots[g];
      const int32_t root = s;
      while (s >= 0) {
        P.canon_of_input[s] = static_cast<int32_t>(P.input_of_canon.size());
        P.input_of_canon.push_back(s);
        P.seg_group.push_back(g);
        if (first_child[s] >= 0) {
          s = first_child[s];
        } else {
          // climb until a sibling exists or we are back at the root
          while (s != root && next_sibling[s] < 0) s = desc.parent[s];
          s = (s == root) ? -1 : next_sibling[s];
        }
      }
    }

    // ---- per-segment arrays ----
    P.seg_parent.resize(n); P.seg_len.resize(n); P.seg_flags.resize(n); P.seg_bs.resize(n);
    P.seg_depth.assign(n, 0); P.seg_anc_tokens.assign(n, 0); P.seg_sub_end.resize(n);
    P.seg_tok_off.resize(n); P.seg_q_off.resize(n); P.seg_refcount.assign(n, 0);
    int64_t tok = 0, qtok = 0;
    for (int32_t c = 0; c < n; ++c) {
      const int32_t s = P.input_of_canon[c];
      const int32_t p = desc.parent[s] < 0 ? -1 : P.canon_of_input[desc.parent[s]];
      P.seg_parent[c] = p;
      P.seg_len[c] = desc.seg_len[s];
      P.seg_flags[c] = in_flags[s];
      P.seg_bs[c] = desc.group_block_size[P.seg_group[c]];
      if (p >= 0) {
        P.seg_depth[c] = P.seg_depth[p] + 1;
        P.seg_anc_tokens[c] = P.seg_anc_tokens[p] + P.seg_len[p];
      }
      P.max_depth = std::max(P.max_depth, P.seg_depth[c]);
      P.seg_tok_off[c] = static_cast<int32_t>(tok);
      tok += P.seg_len[c];
      if (P.seg_flags[c] & PSRL_SEG_HAS_Q) {
        P.seg_q_off[c] = static_cast<int32_t>(qtok);
        qtok += P.seg_len[c];
      } else {
        P.seg_q_off[c] = -1;
      }
      if (tok > INT32_MAX / 2) return PSRL_ERR_SHAPE;
    }
    P.T = static_cast<int32_t>(tok);
    P.T_q = static_cast<int32_t>(qtok);
    // subtree ends and reference counts by one reverse sweep (children come after parents)
    for (int32_t c = 0; c < n; ++c) P.seg_sub_end[c] = c + 1;
    for (int32_t c = n - 1; c >= 0; --c) {
      if (P.seg_flags[c] & PSRL_SEG_SAMPLE_END) P.seg_refcount[c] += 1;
      const int32_t p = P.seg_parent[c];
      if (p >= 0) {
        P.seg_refcount[p] += P.seg_refcount[c];
        P.seg_sub_end[p] = std::max(P.seg_sub_end[p], P.seg_sub_end[c]);
      }
    }

    // ---- ancestor CSR ----
    P.anc_off.assign(n + 1, 0);
    for (int32_t c = 0; c < n; ++c) P.anc_off[c + 1] = P.anc_off[c] + P.seg_depth[c];
    P.anc_list.resize(P.anc_off[n]);
    for (int32_t c = 0; c < n; ++c) {
      int32_t at = P.anc_off[c + 1];
      for (int32_t a = P.seg_parent[c]; a >= 0; a = P.seg_parent[a]) P.anc_list[--at] = a;
    }

    // ---- pages ----
    P.seg_first_page.resize(n); P.seg_n_pages.resize(n);
    int64_t bump_at = 0, pool = 0;
    auto take = [&](int64_t size) -> int64_t {
      if (bump) {
        const int64_t slot = bump_at;
        bump_at += size;
        return slot;
      }
      for (Extent& e : extents) {
        if (e.count >= size) {
          const int64_t slot = e.start;
          e.start += size;
          e.count -= size;
          return slot;
        }
      }
      return -1;
    };
    std::vector<int32_t> sizes;
    for (int32_t c = 0; c < n; ++c) {
      const int32_t bs = P.seg_bs[c], len = P.seg_len[c];
      sizes.clear();
      int64_t total = 0;
      if (bs) {
        sizes.assign((len + bs - 1) / bs, bs);
      } else {  // adaptive (Sec. 5.1): the span in 128-slot pages, its tail in 16-slot pages, one extent
        sizes.assign(len / kTile, kTile);
        sizes.insert(sizes.end(), (len % kTile + 15) / 16, 16);
      }
      for (int32_t sz : sizes) total += sz;
      const int32_t npg = static_cast<int32_t>(sizes.size());
      P.seg_first_page[c] = static_cast<int32_t>(P.page_seg.size());
      P.seg_n_pages[c] = npg;
      const int64_t pinned = desc.seg_slot_base ? desc.seg_slot_base[P.input_of_canon[c]] : -1;
      int64_t at = pinned;
      if (at < 0 && !bs) {
        at = take(total);
        if (at < 0) return PSRL_ERR_POOL_FULL;
      }
      int32_t tok = 0;
      for (int32_t i = 0; i < npg; ++i) {
        int64_t slot;
        if (at >= 0) {
          slot = at;
          at += sizes[i];
        } else {
          slot = take(sizes[i]);
          if (slot < 0) return PSRL_ERR_POOL_FULL;
        }
        if (slot + sizes[i] > INT32_MAX / 2) return PSRL_ERR_SHAPE;
        P.page_seg.push_back(c);
        P.page_bs.push_back(sizes[i]);
        P.page_valid.push_back(std::min(sizes[i], len - tok));
        P.page_pos.push_back(P.seg_anc_tokens[c] + tok);
        P.page_refcount.push_back(P.seg_refcount[c]);
        P.page_slot.push_back(static_cast<int32_t>(slot));
        pool = std::max<int64_t>(pool, slot + sizes[i]);
        tok += sizes[i];
      }
    }
    P.n_pages = static_cast<int32_t>(P.page_seg.size());
    P.pool_slots = static_cast<int32_t>(pool);

    // ---- block table ----
    P.bt_off.assign(n + 1, 0);
    for (int32_t c = 0; c < n; ++c) {
      int32_t cnt = P.seg_n_pages[c];
      for (int32_t i = P.anc_off[c]; i < P.anc_off[c + 1]; ++i) cnt += P.seg_n_pages[P.anc_list[i]];
      P.bt_off[c + 1] = P.bt_off[c] + cnt;
    }
    P.bt_pages.resize(P.bt_off[n]);
    for (int32_t c = 0; c < n; ++c) {
      int32_t at = P.bt_off[c];
      auto emit = [&](int32_t seg) {
        for (int32_t i = 0; i < P.seg_n_pages[seg]; ++i) P.bt_pages[at++] = P.seg_first_page[seg] + i;
      };
      for (int32_t i = P.anc_off[c]; i < P.anc_off[c + 1]; ++i) emit(P.anc_list[i]);
      emit(c);
    }

    // ---- token -> slot ----
    P.tok_slot.resize(P.T);
    for (int32_t c = 0; c < n; ++c) {
      int32_t tok = P.seg_tok_off[c];
      for (int32_t pg = P.seg_first_page[c]; pg < P.seg_first_page[c] + P.seg_n_pages[c]; ++pg)
        for (int32_t j = 0; j < P.page_valid[pg]; ++j) P.tok_slot[tok++] = P.page_slot[pg] + j;
    }

    // ---- samples and statistics ----
    for (int32_t c = 0; c < n; ++c) {
      const int64_t len = P.seg_len[c], anc = P.seg_anc_tokens[c];
      if (P.seg_flags[c] & PSRL_SEG_SAMPLE_END) {
        P.sample_end_seg.push_back(c);
        P.sample_len.push_back(static_cast<int32_t>(anc + len));
        P.flat_tokens += anc + len;
        P.flat_pairs += (anc + len) * (anc + len + 1) / 2;
      }
      if (P.seg_flags[c] & PSRL_SEG_HAS_Q) P.tree_pairs += len * anc + len * (len + 1) / 2;
    }
    P.n_samples = static_cast<int32_t>(P.sample_end_seg.size());

    // ================= device work schedule =================
    // KV tiles
    P.seg_first_kvt.resize(n); P.seg_n_kvt.resize(n);
    for (int32_t c = 0; c < n; ++c) {
      const int32_t bs = P.seg_bs[c], len = P.seg_len[c];
      const int32_t nt = (len + kTile - 1) / kTile;
      P.seg_first_kvt[c] = static_cast<int32_t>(P.kv_tiles.size());
      P.seg_n_kvt[c] = nt;
      for (int32_t t = 0; t < nt; ++t) {
        KvTile kt{};
        const int32_t tok0 = t * kTile;
        kt.n_valid = std::min(kTile, len - tok0);
        kt.bs = bs;
        kt.seg = c;
        kt.tile_idx = t;
        if (bs == 0) {
          // adaptive block: full tiles are one 128-slot page, the tail tile a run of 16-slot pages
          const int32_t full = len / kTile;
          if (t < full) {
            kt.bs = kTile; kt.first_page = P.seg_first_page[c] + t; kt.n_pages = 1; kt.row_off = 0; kt.rows_loaded = kTile;
          } else {
            kt.bs = 16; kt.first_page = P.seg_first_page[c] + full; kt.n_pages = (kt.n_valid + 15) / 16;
            kt.row_off = 0; kt.rows_loaded = kt.n_pages * 16;
          }
        } else if (bs >= kTile) {
          kt.first_page = P.seg_first_page[c] + tok0 / bs;
          kt.n_pages = 1;
          kt.row_off = tok0 % bs;
          kt.rows_loaded = kTile;
          kt.zero_rows = (bs > kTile && kt.row_off == 0 && t == nt - 1) ? bs - kTile : 0;
        } else {
          kt.first_page = P.seg_first_page[c] + tok0 / bs;
          kt.n_pages = (kt.n_valid + bs - 1) / bs;
          kt.row_off = 0;
          kt.rows_loaded = kt.n_pages * bs;
        }
        P.kv_tiles.push_back(kt);
      }
    }
    // descendant query ranges (a subtree is a contiguous run of canonical indices)
    P.seg_desc_q_begin.assign(n, 0); P.seg_desc_q_end.assign(n, 0);
    std::vector<int64_t> desc_qtiles(n, 0);  // own query tiles of all strict descendants
    for (int32_t c = 0; c < n; ++c) {
      int32_t b = -1, e = -1;
      for (int32_t x = c + 1; x < P.seg_sub_end[c]; ++x) {
        if (P.seg_q_off[x] >= 0) {
          if (b < 0) b = P.seg_q_off[x];
          e = P.seg_q_off[x] + P.seg_len[x];
          desc_qtiles[c] += P.seg_n_kvt[x];
        }
      }
      if (b >= 0) { P.seg_desc_q_begin[c] = b; P.seg_desc_q_end[c] = e; }
    }
    // Which segments are cascaded (tensor-core path only).  Walking a's n_a KV tiles costs
    // n_a tile steps per query tile that has a on its path: desc_qtiles[a] * n_a in total, or
    // packed * n_a when the descendants' rows are packed 128 to a tile.  Cascade when packing
    // at least halves that, or when the descendants' tiles are too few to occupy the SMs while
    // a is long (the small-suffix / long-prefix case, which then also gets split over CTAs).
    constexpr int64_t kSms = 148;
    const int64_t cta_units = int64_t(P.Hkv) * ((P.Hq / P.Hkv + 1) / 2);  // forward CTAs per item
    P.seg_cascaded.assign(n, 0);
    if (P.dtype == PSRL_BF16) {
      for (int32_t c = 0; c < n; ++c) {
        const int64_t rows = P.seg_desc_q_end[c] - P.seg_desc_q_begin[c];
        if (rows <= 0) continue;
        const int64_t packed = (rows + kTile - 1) / kTile;
        const bool fewer = packed * 2 <= desc_qtiles[c] && P.seg_n_kvt[c] >= 4;
        const bool starved = desc_qtiles[c] * cta_units * 2 <= kSms && P.seg_n_kvt[c] >= 8;
        P.seg_cascaded[c] = (fewer || starved) ? 1 : 0;
      }
    }
    // per-segment list of KV tiles for the own items: non-cascaded ancestors root->parent, then own
    P.path_off.assign(n + 1, 0);
    std::vector<uint8_t> has_casc_anc(n, 0);
    for (int32_t c = 0; c < n; ++c) {
      int32_t cnt = P.seg_n_kvt[c];
      for (int32_t i = P.anc_off[c]; i < P.anc_off[c + 1]; ++i) {
        const int32_t a = P.anc_list[i];
        if (P.seg_cascaded[a]) has_casc_anc[c] = 1; else cnt += P.seg_n_kvt[a];
      }
      P.path_off[c + 1] = P.path_off[c] + cnt;
    }
    P.path_tiles.resize(P.path_off[n]);
    for (int32_t c = 0; c < n; ++c) {
      int32_t at = P.path_off[c];
      auto emit = [&](int32_t seg) {
        for (int32_t i = 0; i < P.seg_n_kvt[seg]; ++i) P.path_tiles[at++] = P.seg_first_kvt[seg] + i;
      };
      for (int32_t i = P.anc_off[c]; i < P.anc_off[c + 1]; ++i)
        if (!P.seg_cascaded[P.anc_list[i]]) emit(P.anc_list[i]);
      emit(c);
    }
    // own items
    P.qrow_seg.resize(P.T_q);
    std::vector<int32_t> own_part_base(n, -1);
    for (int32_t c = 0; c < n; ++c) {
      if (P.seg_q_off[c] < 0) continue;
      for (int32_t i = 0; i < P.seg_len[c]; ++i) P.qrow_seg[P.seg_q_off[c] + i] = c;
      if (has_casc_anc[c]) { own_part_base[c] = P.n_part_rows; P.n_part_rows += P.seg_len[c]; }
      const int32_t anc_tiles = (P.path_off[c + 1] - P.path_off[c]) - P.seg_n_kvt[c];
      for (int32_t t = 0; t < P.seg_n_kvt[c]; ++t) {
        QTile qt{};
        qt.seg = c;
        qt.tile_idx = t;
        qt.q_row0 = P.seg_q_off[c] + t * kTile;
        qt.n_rows = std::min(kTile, P.seg_len[c] - t * kTile);
        qt.pt_begin = P.path_off[c];
        qt.n_kv_tiles = anc_tiles + t + 1;
        qt.causal = 1;
        qt.part_row0 = has_casc_anc[c] ? own_part_base[c] + t * kTile : -1;
        P.q_tiles.push_back(qt);
      }
    }
    // packed items of the cascaded segments: chunk k of a's tiles x block b of 128 packed rows;
    // partial rows of chunk k are [base + k*rows, base + (k+1)*rows), in query-row order
    std::vector<int32_t> casc_part_base(n, -1), casc_chunks(n, 0);
    for (int32_t a = 0; a < n; ++a) {
      if (!P.seg_cascaded[a]) continue;
      const int32_t rows = P.seg_desc_q_end[a] - P.seg_desc_q_begin[a];
      const int32_t packed = (rows + kTile - 1) / kTile, nt = P.seg_n_kvt[a];
      // about half an SM count of forward CTAs for the packed part: the rows' own items need SMs too, and
      // every further chunk adds a partial row per query row to merge (measured on the small-suffix case:
      // 4 chunks 0.128 ms, 10 chunks 0.142 ms per step)
      int64_t chunks = kSms / (2 * packed * cta_units);
      chunks = std::max<int64_t>(1, std::min<int64_t>(chunks, nt / 2));
      casc_part_base[a] = P.n_part_rows;
      casc_chunks[a] = static_cast<int32_t>(chunks);
      for (int32_t k = 0; k < chunks; ++k) {
        const int32_t t0 = static_cast<int32_t>(int64_t(nt) * k / chunks), t1 = static_cast<int32_t>(int64_t(nt) * (k + 1) / chunks);
        const int32_t pt = static_cast<int32_t>(P.path_tiles.size());
        for (int32_t t = t0; t < t1; ++t) P.path_tiles.push_back(P.seg_first_kvt[a] + t);
        for (int32_t b = 0; b < packed; ++b) {
          QTile qt{};
          qt.seg = a;
          qt.tile_idx = k;
          qt.q_row0 = P.seg_desc_q_begin[a] + b * kTile;
          qt.n_rows = std::min(kTile, rows - b * kTile);
          qt.pt_begin = pt;
          qt.n_kv_tiles = t1 - t0;
          qt.causal = 0;
          qt.part_row0 = P.n_part_rows + k * rows + b * kTile;
          P.q_tiles.push_back(qt);
        }
      }
      P.n_part_rows += static_cast<int32_t>(chunks) * rows;
    }
    // merge lists: cascaded ancestors root->parent (chunks ascending), then the own item
    P.merge_off.push_back(0);
    for (int32_t c = 0; c < n; ++c) {
      if (P.seg_q_off[c] < 0 || !has_casc_anc[c]) continue;
      for (int32_t i = 0; i < P.seg_len[c]; ++i) {
        const int32_t r = P.seg_q_off[c] + i;
        P.merge_row.push_back(r);
        for (int32_t x = P.anc_off[c]; x < P.anc_off[c + 1]; ++x) {
          const int32_t a = P.anc_list[x];
          if (!P.seg_cascaded[a]) continue;
          const int32_t rows = P.seg_desc_q_end[a] - P.seg_desc_q_begin[a];
          for (int32_t k = 0; k < casc_chunks[a]; ++k)
            P.merge_parts.push_back(casc_part_base[a] + k * rows + (r - P.seg_desc_q_begin[a]));
        }
        P.merge_parts.push_back(own_part_base[c] + i);
        P.merge_off.push_back(static_cast<int32_t>(P.merge_parts.size()));
      }
    }
    std::stable_sort(P.q_tiles.begin(), P.q_tiles.end(),
                     [](const QTile& a, const QTile& b) { return a.n_kv_tiles > b.n_kv_tiles; });
    // dK/dV items.  Cost of a KV tile = number of 128-row query sub-tiles that attend to it
    // (the pair count of Eq. 1's attention term, in tile units).  Tiles much heavier
    // than an SM's fair share are split into parts so that the longest item cannot dominate
    // the makespan; the list is then ordered longest first.
    auto n_subs = [](const KvItem& it) {
      int64_t n = (it.desc_q_end - it.desc_q_begin + kSubRows - 1) / kSubRows;
      if (it.own_q_row0 >= 0) n += (it.own_q_end - it.own_q_row0 + kSubRows - 1) / kSubRows;
      return static_cast<int32_t>(n);
    };
    std::vector<KvItem> whole;
    int64_t total_sub = 0;
    for (size_t k = 0; k < P.kv_tiles.size(); ++k) {
      const KvTile& kt = P.kv_tiles[k];
      KvItem it{};
      it.kvt = static_cast<int32_t>(k);
      const int32_t c = kt.seg;
      if (P.seg_q_off[c] >= 0) {
        it.own_q_row0 = P.seg_q_off[c] + kt.tile_idx * kTile;
        it.own_q_end = P.seg_q_off[c] + P.seg_len[c];
      } else {
        it.own_q_row0 = -1;
        it.own_q_end = -1;
      }
      it.desc_q_begin = P.seg_desc_q_begin[c];
      it.desc_q_end = P.seg_desc_q_end[c];
      it.sub_begin = 0;
      it.sub_end = n_subs(it);
      it.slab = -1;
      total_sub += it.sub_end;
      whole.push_back(it);
    }
    constexpr int64_t kMinPart = 12;
    const int64_t fair = (total_sub * P.Hkv + kSms - 1) / kSms;       // sub-tiles per SM if perfectly balanced
    const int64_t part_max = std::max<int64_t>(kMinPart, fair / 2);
    for (const KvItem& it : whole) {
      const int32_t n = it.sub_end;
      if (n <= part_max + part_max / 2) {
        P.kv_items.push_back(it);
        continue;
      }
      const int32_t parts = static_cast<int32_t>((n + part_max - 1) / part_max);
      KvSplit sp{it.kvt, P.n_slabs, parts, 0};
      for (int32_t a = 0; a < parts; ++a) {
        KvItem part = it;
        part.sub_begin = static_cast<int32_t>(int64_t(n) * a / parts);
        part.sub_end = static_cast<int32_t>(int64_t(n) * (a + 1) / parts);
        part.slab = P.n_slabs + a;
        P.kv_items.push_back(part);
      }
      P.n_slabs += parts;
      P.kv_splits.push_back(sp);
    }
    std::stable_sort(P.kv_items.begin(), P.kv_items.end(), [](const KvItem& a, const KvItem& b) {
      return (a.sub_end - a.sub_begin) > (b.sub_end - b.sub_begin);
    });

    // ---- device blob ----
    DeviceHeader& H = P.hdr;
    H.magic = 0x5053524c;  // "PSRL"
    H.n_seg = n; H.n_pages = P.n_pages; H.n_kvt = static_cast<int32_t>(P.kv_tiles.size());
    H.n_qt = static_cast<int32_t>(P.q_tiles.size()); H.T = P.T; H.T_q = P.T_q;
    H.n_bt = static_cast<int32_t>(P.bt_pages.size());
    std::vector<int32_t>& B = P.blob;
    B.assign(sizeof(DeviceHeader) / sizeof(int32_t), 0);
    H.off_seg_len = append_array(B, P.seg_len);
    H.off_seg_q_off = append_array(B, P.seg_q_off);
    H.off_seg_tok_off = append_array(B, P.seg_tok_off);
    H.off_seg_flags = append_array(B, P.seg_flags);
    H.off_seg_first_page = append_array(B, P.seg_first_page);
    H.off_seg_n_pages = append_array(B, P.seg_n_pages);
    H.off_seg_bs = append_array(B, P.seg_bs);
    H.off_seg_first_kvt = append_array(B, P.seg_first_kvt);
    H.off_seg_n_kvt = append_array(B, P.seg_n_kvt);
    H.off_seg_desc_q_begin = append_array(B, P.seg_desc_q_begin);
    H.off_seg_desc_q_end = append_array(B, P.seg_desc_q_end);
    H.off_page_slot = append_array(B, P.page_slot);
    H.off_page_valid = append_array(B, P.page_valid);
    H.off_page_seg = append_array(B, P.page_seg);
    H.off_page_bs = append_array(B, P.page_bs);
    H.off_bt_off = append_array(B, P.bt_off);
    H.off_bt_pages = append_array(B, P.bt_pages);
    H.off_qrow_seg = append_array(B, P.qrow_seg);
    H.off_tok_slot = append_array(B, P.tok_slot);
    H.off_kvt = append_array(B, P.kv_tiles);
    H.off_qt = append_array(B, P.q_tiles);
    H.off_kvi = append_array(B, P.kv_items);
    H.off_path_off = append_array(B, P.path_off);
    H.off_path_tiles = append_array(B, P.path_tiles);
    P.path_nvalid.resize(P.path_tiles.size());
    for (size_t i = 0; i < P.path_tiles.size(); ++i) P.path_nvalid[i] = P.kv_tiles[P.path_tiles[i]].n_valid;
    H.off_path_nvalid = append_array(B, P.path_nvalid);
    P.path_loads.resize(P.path_tiles.size());
    for (size_t i = 0; i < P.path_tiles.size(); ++i) {
      const KvTile& kt = P.kv_tiles[P.path_tiles[i]];
      TileLoad& tl = P.path_loads[i];
      tl = TileLoad{};
      tl.n_pages = kt.n_pages; tl.bs = kt.bs; tl.rows_loaded = kt.rows_loaded;
      for (int32_t pg = 0; pg < kt.n_pages && pg < 8; ++pg) tl.row[pg] = P.page_slot[kt.first_page + pg] + kt.row_off;
      // Pages that follow one another in the pool (always, under bump allocation) are fetched as ONE box
      // when together they make a power-of-two number of rows: a TMA box costs ~135 cycles plus its bytes.
      const int32_t page_rows = kt.bs >= kTile ? kTile : kt.bs;
      bool contiguous = kt.n_pages > 1;
      for (int32_t pg = 1; pg < kt.n_pages && contiguous; ++pg) contiguous = tl.row[pg] == tl.row[pg - 1] + page_rows;
      if (contiguous && (kt.rows_loaded & (kt.rows_loaded - 1)) == 0) {
        tl.n_pages = 1;
        tl.bs = kt.rows_loaded;   // 32, 64 or 128: selects the box height
      }
    }
    H.off_path_loads = append_array(B, P.path_loads);
    H.n_kvi = static_cast<int32_t>(P.kv_items.size());
    H.off_split = append_array(B, P.kv_splits);
    H.n_split = static_cast<int32_t>(P.kv_splits.size());
    H.n_slabs = P.n_slabs;
    H.n_part_rows = P.n_part_rows;
    H.n_merge_rows = static_cast<int32_t>(P.merge_row.size());
    H.off_merge_row = append_array(B, P.merge_row);
    H.off_merge_off = append_array(B, P.merge_off);
    H.off_merge_parts = append_array(B, P.merge_parts);
    while (B.size() % 64) B.push_back(0);
    std::copy(reinterpret_cast<const int32_t*>(&H), reinterpret_cast<const int32_t*>(&H + 1), B.begin());
  } catch (const std::bad_alloc&) {
    return PSRL_ERR_HOST_OOM;
  }
  guard.p = nullptr;
  out = pl;
  return PSRL_OK;
}

}  // namespace psrl
