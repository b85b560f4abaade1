/*
 * psrl_cache.h - Dynamic Block Caching for prefix-shared KV (paper Sec. 5.2) over an ordered list of
 * micro-batches (Sec. 4.1 inter-batch and self-sequence sharing, Sec. 4.3 token-wise micro-batching).
 *
 * Host-only bookkeeping, no CUDA call, no data movement.  The caller owns one arena of KV slots per
 * worker (the K/V pools passed to psrl_tree_attn_fwd / _bwd).  Blocks are the segments of the prefix
 * forest (Sec. 5.1: one block per reusable prefix span); a segment occupies one contiguous extent of
 * ceil(len / block) * block slots.  For every micro-batch the manager says which segments take part
 * (those computed now issue queries, cached prefixes are read in place), where each one lives
 * (psrl_tree_desc_t::seg_slot_base), which blocks had to be evicted to make room and which have to be
 * brought back; after the micro-batch's backward pass it removes the reference entries of the samples
 * that completed and releases every block whose count reached zero.
 *
 * Rules (the paper's, with the readings it leaves open):
 *  - reference count of a block = number of training samples that will read it (Sec. 5.2);
 *  - a sample completes in the micro-batch that computes its last segment; its entries are removed
 *    after that micro-batch's backward pass; a block stays only while its count is positive;
 *  - when an extent cannot be found, the resident block that is not used by the current micro-batch
 *    and whose next use lies farthest ahead is evicted (ties: larger segment index); the caller must
 *    save it if needed, and restore it when the manager lists it under `reload`;
 *  - the arena is managed first-fit in address order, with coalescing.
 *
 * Every call returns a psrl_status_t and never throws, aborts or prints.  All pointers are HOST
 * pointers.  A cache object is not thread-safe.
 */
#ifndef PSRL_CACHE_H_
#define PSRL_CACHE_H_

#include "psrl.h"

#ifdef __cplusplus
extern "C" {
#endif

typedef struct psrl_cache psrl_cache_t;

typedef struct {
  int32_t n_segments;              /* >= 1 */
  const int32_t* parent;           /* [n_segments] -1 = root, else an index < own index */
  const int32_t* seg_len;          /* [n_segments] tokens, >= 1 */
  const uint8_t* seg_flags;        /* [n_segments] PSRL_SEG_SAMPLE_END bits, or NULL = leaves end samples */
  const int32_t* group_block_size; /* one per root, in input order; power of two in [16, 256], or 0 =
                                      adaptive (Sec. 5.1): one extent per segment sized to its span at 16-slot
                                      granularity (bf16 path only) */
  int32_t n_groups;                /* must equal the number of roots */
  int32_t n_microbatches;          /* >= 1 */
  const int32_t* mb_of_seg;        /* [n_segments] micro-batch that computes the segment; a prefix is
                                      computed no later than what follows it: mb[parent] <= mb[s] */
  int64_t capacity_slots;          /* arena size in slots (multiple of 16), 0 = unbounded */
} psrl_cache_desc_t;

/* What one micro-batch runs on.  Borrowed pointers, valid until the next call on the same cache. */
typedef struct {
  int32_t n_segments;              /* segments of this micro-batch's tree */
  const int32_t* seg_id;           /* [n_segments] forest index, ascending */
  const int32_t* parent;           /* [n_segments] parent inside this tree, -1 = root */
  const int32_t* seg_len;          /* [n_segments] */
  const uint8_t* seg_flags;        /* HAS_Q on the segments computed now; SAMPLE_END on the tree's leaves and
                                      on samples that end in this micro-batch */
  const int32_t* group_block_size; /* [n_groups] one per root of this tree */
  int32_t n_groups;
  const int32_t* seg_slot_base;    /* [n_segments] first slot of each segment's extent: pass as
                                      psrl_tree_desc_t::seg_slot_base (free_extents = NULL) */
  int32_t n_new, n_reload, n_evict;
  const int32_t* new_seg;          /* forest ids whose K/V this micro-batch writes for the first time */
  const int32_t* reload_seg;       /* forest ids evicted earlier: restore their K/V at seg_slot_base first */
  const int32_t* evict_seg;        /* forest ids evicted now, in order ... */
  const int32_t* evict_base;       /* ... and the first slot each one occupied (save from there first) */
  int64_t live_slots;              /* slots resident while this micro-batch runs */
  int64_t pool_slots;              /* one past the highest slot in use: the pools need at least this many */
} psrl_cache_step_t;

/* Errors: INVALID_ARG, BAD_TREE (also mb[parent] > mb[s]), BAD_BLOCK_SIZE, HOST_OOM. */
psrl_status_t psrl_cache_create(const psrl_cache_desc_t* desc, psrl_cache_t** out);

/* Micro-batches run in order 0, 1, ...: begin(m), the attention calls, end(m).
 * Errors: INVALID_ARG (out of order), POOL_FULL (the micro-batch does not fit even after evicting
 * everything it does not use; the cache is unusable afterwards). */
psrl_status_t psrl_cache_begin(psrl_cache_t* cache, int32_t microbatch, psrl_cache_step_t* out);

/* After the backward pass.  *freed_seg: forest ids released now (borrowed, valid until the next call);
 * *live_slots: slots still resident.  Any output pointer may be NULL. */
psrl_status_t psrl_cache_end(psrl_cache_t* cache, int32_t microbatch, int32_t* n_freed, const int32_t** freed_seg,
                             int64_t* live_slots);

typedef struct {
  int64_t peak_slots;       /* largest live_slots of any micro-batch so far */
  int64_t evicted_slots;    /* slots of blocks evicted while still referenced */
  int64_t reloaded_slots;   /* slots of blocks brought back */
  int64_t pool_high_water;  /* one past the highest slot ever handed out */
  int64_t total_slots;      /* sum of all extents: what keeping every block would take */
} psrl_cache_stats_t;
psrl_status_t psrl_cache_stats(const psrl_cache_t* cache, psrl_cache_stats_t* out);

/* Current reference count of every segment, [n_segments] (borrowed). */
psrl_status_t psrl_cache_refcounts(const psrl_cache_t* cache, const int32_t** refcount);

void psrl_cache_destroy(psrl_cache_t* cache);

#ifdef __cplusplus
}
#endif
#endif /* PSRL_CACHE_H_ */
