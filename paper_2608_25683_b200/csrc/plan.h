// Internal representation of a plan: the canonical arrays the C ABI exposes
// through psrl_plan_view_t plus the device work schedule the kernels consume.
#pragma once
#include <cstdint>
#include <vector>

#include "../../include/psrl.h"

namespace psrl {

constexpr int kTile = 128;  // rows of a query tile / keys of a KV tile on the tensor-core path

// One KV tile: up to 128 consecutive tokens of ONE segment (tiles never cross
// a segment boundary, so the valid rows are always a prefix of the tile).
struct KvTile {
  int32_t first_page;  // first page of the tile
  int32_t n_pages;     // pages the tile spans (1 when bs >= 128)
  int32_t bs;          // page size of the segment's group
  int32_t row_off;     // first row inside first_page (0, or 128 for the upper half of a 256-slot page)
  int32_t n_valid;     // valid keys in the tile (1..128)
  int32_t seg;         // canonical segment
  int32_t tile_idx;    // index of the tile inside its segment
  int32_t rows_loaded; // rows a gather brings in: n_pages * min(bs, 128)
  int32_t zero_rows;   // page slots after the tile's 128 rows that no tile covers (upper half of a 256-slot
                       // page whose segment ends in the lower half): the backward writes zeros there
  int32_t pad0, pad1, pad2;
};

// TMA coordinates of one entry of a KV-tile list, resolved on the host so that the producer
// thread of the forward / dQ kernels needs one load per tile instead of a chain of three
// (list entry -> tile record -> page slots): first pool row (slot) of each page of the tile.
struct TileLoad {
  int32_t n_pages, bs, rows_loaded, pad;
  int32_t row[8];   // a tile spans at most 8 pages (page size >= 16 slots)
};

// One work item of the forward and dQ kernels: up to 128 consecutive query rows
// and a list of KV tiles they attend to.
//  * own item: rows of one HAS_Q segment; the list holds the tiles of its
//    ancestors root->parent (those that are not cascaded, see below) and its own
//    tiles up to the diagonal tile, which is last and causal.
//  * packed item: rows of the contiguous query range of ALL strict descendants of
//    a "cascaded" segment a (rows of several short segments share one tile) and a
//    chunk of a's KV tiles, every key visible to every row.  A segment is cascaded
//    when its descendants' own tiles are mostly empty or too few to fill the GPU;
//    its KV tiles are then visited once per 128 packed rows instead of once per
//    descendant tile, and split into chunks over CTAs (split-KV).
// An item whose rows also get contributions from other items writes fp32 partial
// results to rows [part_row0, part_row0 + n_rows) of the workspace; the merge
// kernels combine the parts of a row in the fixed order of its merge list.
struct QTile {
  int32_t seg;        // segment of the rows (own item) or the cascaded ancestor (packed item)
  int32_t tile_idx;   // own item: rows [tile_idx*128, ...) of the segment; packed item: chunk index
  int32_t q_row0;     // first row in Q/O/dO/dQ
  int32_t n_rows;     // 1..128
  int32_t pt_begin;   // first entry in path_tiles
  int32_t n_kv_tiles; // tiles to visit
  int32_t causal;     // 1: the last tile is the diagonal tile of the rows' segment; 0: every key visible
  int32_t part_row0;  // -1: the item writes the final outputs; else its first partial row
};

constexpr int kSubRows = 128;  // query rows per step of the dK/dV kernel

// One dK/dV work item: a KV tile and (a contiguous part of) the query rows that
// attend to it.  The rows are walked in sub-tiles of kSubRows: first the own
// segment's rows from the tile's first key on, then the rows of all strict
// descendants.  A heavy tile is split into several items over disjoint
// sub-tile ranges; their fp32 partial sums go to slabs of the workspace and are
// added in part order by the reduce kernel (fixed order, bitwise reproducible).
struct KvItem {
  int32_t kvt;         // KV tile id
  int32_t own_q_row0;  // first own-segment query row (the tile's first key), -1 if the segment has no queries
  int32_t own_q_end;   // one past the segment's last query row
  int32_t desc_q_begin, desc_q_end;  // query rows of all strict descendants (contiguous), empty if none
  int32_t sub_begin, sub_end;        // this item's range of sub-tiles
  int32_t slab;                      // partial-sum slab, or -1 if the item owns the tile and writes the output
};

// A KV tile whose work was split: its partial slabs [slab0, slab0 + n_parts).
struct KvSplit {
  int32_t kvt, slab0, n_parts, pad;
};

// Offsets (in int32 units from the start of the device blob) of each array.
struct DeviceHeader {
  int32_t magic;
  int32_t n_seg, n_pages, n_kvt, n_qt, T, T_q, n_bt;
  int32_t off_seg_len, off_seg_q_off, off_seg_tok_off, off_seg_flags, off_seg_first_page, off_seg_n_pages;
  int32_t off_seg_bs, off_seg_first_kvt, off_seg_n_kvt, off_seg_desc_q_begin, off_seg_desc_q_end;
  int32_t off_page_slot, off_page_valid, off_page_seg, off_page_bs;
  int32_t off_bt_off, off_bt_pages;
  int32_t off_qrow_seg;  // [T_q] segment of every query row
  int32_t off_kvt, off_qt, off_kvi, off_path_off, off_path_tiles;
  int32_t off_path_nvalid;  // valid keys of every entry of path_tiles
  int32_t off_path_loads;   // TileLoad of every entry of path_tiles
  int32_t n_kvi;
  int32_t n_split, off_split, n_slabs;
  // merge lists of the rows that are assembled from partial results: row i of the list is
  // query row merge_row[i]; its parts are merge_parts[merge_off[i] .. merge_off[i+1]) (partial-row ids)
  int32_t n_part_rows, n_merge_rows, off_merge_row, off_merge_off, off_merge_parts;
  int32_t off_tok_slot;     // [T] pool slot of every token
};

struct Plan {
  // problem
  int32_t Hq = 0, Hkv = 0, d = 0;
  psrl_dtype_t dtype = PSRL_F32;
  // scalars
  int32_t n_seg = 0, n_groups = 0, n_pages = 0, n_samples = 0, max_depth = 0, T = 0, T_q = 0, pool_slots = 0;
  int64_t flat_tokens = 0, tree_pairs = 0, flat_pairs = 0;
  // canonical arrays
  std::vector<int32_t> canon_of_input, input_of_canon, seg_group, seg_bs, seg_parent, seg_len, seg_flags, seg_depth,
      seg_anc_tokens, seg_sub_end, seg_tok_off, seg_q_off, seg_refcount, anc_off, anc_list, seg_first_page,
      seg_n_pages, page_seg, page_bs, page_valid, page_pos, page_refcount, page_slot, bt_off, bt_pages, tok_slot,
      sample_end_seg, sample_len;
  // schedule (host copies)
  std::vector<KvTile> kv_tiles;
  std::vector<QTile> q_tiles;    // longest first
  std::vector<KvItem> kv_items;  // longest first
  std::vector<KvSplit> kv_splits;
  int32_t n_slabs = 0;
  std::vector<uint8_t> seg_cascaded;  // 1: the segment's KV tiles are handled by packed items
  int32_t n_part_rows = 0;
  std::vector<int32_t> merge_row, merge_off, merge_parts;
  std::vector<TileLoad> path_loads;
  std::vector<int32_t> seg_first_kvt, seg_n_kvt, seg_desc_q_begin, seg_desc_q_end, path_off, path_tiles, path_nvalid, qrow_seg;
  // device blob
  std::vector<int32_t> blob;
  DeviceHeader hdr{};
  const int32_t* dev = nullptr;  // bound device copy of blob
};

psrl_status_t build_plan(const psrl_tree_desc_t& desc, Plan*& out);

}  // namespace psrl

// The opaque handle of the C ABI (one definition for every translation unit that takes a plan).
struct psrl_plan {
  psrl::Plan* p;
};
