/*
 * psrl_sched.h - workload model and scheduling of prefix-shared training data (paper Sec. 4.2, 4.3).
 * Host-only, no CUDA call.  Every call returns a psrl_status_t and never throws, aborts or prints.
 * All pointers are HOST pointers; outputs are caller-allocated.
 *
 * Forest arguments are the ones of psrl_tree_desc_t: parent[s] = -1 or an index < s, seg_len[s] >= 1,
 * seg_flags NULL (leaves end samples) or PSRL_SEG_SAMPLE_END bits.  Inside a prefix group the samples
 * (root-to-SAMPLE_END paths) are taken in canonical (DFS) order; the cached prefix h of a sample is the
 * part of its path that earlier samples have already computed, its length l the whole path.
 */
#ifndef PSRL_SCHED_H_
#define PSRL_SCHED_H_

#include "psrl.h"

#ifdef __cplusplus
extern "C" {
#endif

/* Eq. 1: T(s) = a1 * l_suf * l + a2 * l_suf + a3 with l_suf = l - h (attention, per-token work, overhead);
 * the coefficients come from profiling (bench.py fits them to measured kernel times). */
typedef struct {
  double a1, a2, a3;
} psrl_cost_model_t;

double psrl_cost_sequence(const psrl_cost_model_t* model, int64_t l, int64_t h);

/* Workload of every prefix group (root): the sum of Eq. 1 over its samples.
 *   workload  [n_groups] out, n_groups must equal the number of roots
 * Errors: INVALID_ARG, BAD_TREE. */
psrl_status_t psrl_group_workloads(int32_t n_segments, const int32_t* parent, const int32_t* seg_len,
                                   const uint8_t* seg_flags, const psrl_cost_model_t* model, int32_t n_groups,
                                   double* workload);

/* Load balancing (Sec. 4.2): groups in descending order of workload (ties: lower index first), each, whole,
 * to the worker with the smallest load so far (ties: lower worker index).
 *   worker_of_group [n_groups] out;  worker_load [n_workers] out (may be NULL)
 * Errors: INVALID_ARG (n_groups < 0, n_workers < 1, negative or non-finite workload). */
psrl_status_t psrl_place_groups(int32_t n_groups, const double* workload, int32_t n_workers,
                                int32_t* worker_of_group, double* worker_load);

/* Token-wise micro-batching (Sec. 4.3) of one worker's forest.  Budget = total workload / n_microbatches.
 * Samples are walked in canonical order; a sample whose remaining tokens would exceed what is left of the
 * budget is cut at the token level (largest piece that still fits, at least one token on each side; an
 * empty micro-batch takes at least one token) and continues in the next micro-batch; the last micro-batch
 * takes whatever remains.  A piece [a, b) of a sample costs Eq. 1 with h = a, l = b.
 * The result is a forest of pieces in canonical order, ready for psrl_cache_create / psrl_plan_build:
 *   capacity      size of the output arrays; n_segments + n_microbatches always suffices
 *   *n_pieces     out
 *   piece_parent  [capacity] out, parent piece (-1 = root); pieces of one segment form a chain
 *   piece_len     [capacity] out, tokens
 *   piece_mb      [capacity] out, micro-batch; never decreases along the list
 *   piece_seg, piece_begin [capacity] out, the input segment and first token inside it
 *   budget        out (may be NULL)
 * Errors: INVALID_ARG, BAD_TREE, WORKSPACE (capacity too small). */
psrl_status_t psrl_microbatch_tokens(int32_t n_segments, const int32_t* parent, const int32_t* seg_len,
                                     const uint8_t* seg_flags, const psrl_cost_model_t* model,
                                     int32_t n_microbatches, int32_t capacity, int32_t* n_pieces,
                                     int32_t* piece_parent, int32_t* piece_len, int32_t* piece_mb,
                                     int32_t* piece_seg, int32_t* piece_begin, double* budget);

#ifdef __cplusplus
}
#endif
#endif /* PSRL_SCHED_H_ */
