/*
 * psrl.h - C ABI of the tree-causal prefix-shared attention library (libpsrl.so).
 *
 * The library implements the attention step of training-time prefix sharing:
 * samples of a step-wise or tree-structured RL batch share decision prefixes;
 * every shared token span ("segment") is stored once, its K/V in a paged KV
 * store, and each token attends to all tokens of its ancestor segments plus
 * the causal part of its own segment, which reproduces per-sequence causal
 * attention exactly (paper Sec. 2.5, "Prefix sharing in training").  Backward
 * accumulates the adjoints of every consumer on the shared K/V (paper Sec. 6,
 * "Prefix-sharing training runtime") in a fixed order, so results are bitwise
 * reproducible run to run.
 *
 * Conventions
 *  - Every call returns a psrl_status_t; nothing throws, aborts or prints.
 *  - "host" / "device" is stated for every pointer.  The library never
 *    allocates device memory in the entry points below: tensors, pools, the
 *    plan's device mirror and the workspace are the caller's.
 *  - Kernels are launched on the caller's stream; no entry point synchronises
 *    except psrl_device_status().
 *  - Only sm_100a devices are supported; there is no CPU or other fallback.
 */
#ifndef PSRL_H_
#define PSRL_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
  PSRL_OK = 0,
  PSRL_ERR_INVALID_ARG = 1,    /* null / misaligned pointer, bad count, bad flag bits */
  PSRL_ERR_BAD_TREE = 2,       /* parent >= own index, length < 1, leaf that ends no sample */
  PSRL_ERR_BAD_BLOCK_SIZE = 3, /* block size not a power of two in [16, 256], or 0 =
                                      adaptive (Sec. 5.1): one extent per segment sized to its span at 16-slot
                                      granularity (bf16 path only) */
  PSRL_ERR_SHAPE = 4,          /* head counts do not divide, pool smaller than the plan needs */
  PSRL_ERR_UNSUPPORTED = 5,    /* dtype x head_dim outside {f32 x {64,128}, bf16 x 128} */
  PSRL_ERR_POOL_FULL = 6,      /* no free extent fits a page */
  PSRL_ERR_WORKSPACE = 7,      /* workspace / device buffer too small, or plan not uploaded */
  PSRL_ERR_HOST_OOM = 8,
  PSRL_ERR_CUDA = 9,           /* a CUDA runtime / driver call failed */
  PSRL_ERR_TIMEOUT = 10,       /* a bounded device-side wait ran out (read via psrl_device_status) */
  PSRL_ERR_INTERNAL = 11
} psrl_status_t;

typedef enum { PSRL_F32 = 0, PSRL_BF16 = 1 } psrl_dtype_t;

/* Segment flags. */
enum {
  PSRL_SEG_HAS_Q = 1,     /* the segment's tokens issue queries (rows of Q/O/dO/dQ exist) */
  PSRL_SEG_SAMPLE_END = 2 /* a training sample ends at this segment (root-to-here path) */
};

/*
 * Problem statement: a forest of token segments.  A sample is the path from a
 * root to a SAMPLE_END segment (tree sampling: leaves; step / tree-step
 * sampling: every node - paper Sec. 2.3).  Roots are independent prefix groups
 * (paper Sec. 4.2, semantic groups).  All pointers are HOST pointers, read
 * during psrl_plan_build only.
 */
typedef struct {
  int32_t n_segments;              /* >= 1 */
  const int32_t* parent;           /* [n_segments] -1 = root, else an index < own index */
  const int32_t* seg_len;          /* [n_segments] tokens, >= 1 */
  const uint8_t* seg_flags;        /* [n_segments] or NULL = HAS_Q everywhere, SAMPLE_END on leaves */
  const int32_t* group_block_size; /* one per root, in input order; power of two in [16, 256], or 0 =
                                      adaptive (Sec. 5.1): one extent per segment sized to its span at 16-slot
                                      granularity (bf16 path only) */
  int32_t n_groups;                /* must equal the number of roots */
  int32_t n_q_heads, n_kv_heads;   /* n_q_heads % n_kv_heads == 0 */
  int32_t head_dim;                /* 64 or 128 (f32), 128 (bf16) */
  psrl_dtype_t dtype;
  const int32_t* free_extents;     /* [2 * n_free] (start_slot, n_slots), multiples of 16; NULL = bump from 0 */
  int32_t n_free;
  /* Optional [n_segments] (input order) or NULL: where a segment's K/V already lives.  A value >= 0
   * (a multiple of 16) pins the segment: its pages are the consecutive runs of block-size slots starting
   * there and take nothing from the free extents; -1 allocates as usual.  This is how a prefix cached
   * by an earlier micro-batch is reused in place (paper Sec. 4.1 inter-batch / self-sequence sharing,
   * Sec. 5.2): the cache manager (psrl_cache.h) hands out these bases. */
  const int32_t* seg_slot_base;
} psrl_tree_desc_t;

typedef struct psrl_plan psrl_plan_t;

/*
 * Borrowed HOST pointers into the plan's canonical arrays (valid until
 * psrl_plan_destroy).  Segments are indexed in canonical order = DFS preorder,
 * roots and siblings in ascending input index.  The per-page fields are the
 * block metadata of the paper's KV manager (Sec. 6: base address, block size,
 * position of the token span in the full sequence, reference count); pages
 * follow reusable prefix spans and never cross a segment boundary (Sec. 5.1).
 */
typedef struct {
  int32_t n_seg, n_groups, n_pages, n_samples, max_depth;
  int32_t T;          /* tokens stored (each shared token once) */
  int32_t T_q;        /* tokens that issue queries */
  int32_t pool_slots; /* slots per KV head the pools must hold: max(page_slot + page_bs) */
  int64_t flat_tokens; /* sum of sample lengths (the unshared layout) */
  int64_t tree_pairs;  /* attended (query, key) pairs, shared:   sum len*anc + len(len+1)/2  (cf. Eq. 1) */
  int64_t flat_pairs;  /* attended pairs, unshared: sum L(L+1)/2 */
  int32_t n_anc, n_bt; /* lengths of anc_list and bt_pages */
  const int32_t *canon_of_input, *input_of_canon;               /* [n_seg] */
  const int32_t *seg_group, *seg_bs, *seg_parent, *seg_len, *seg_flags, *seg_depth;
  const int32_t *seg_anc_tokens; /* tokens of strict ancestors = position of the span in the sequence */
  const int32_t *seg_sub_end;    /* subtree = canonical indices [c, seg_sub_end[c]) */
  const int32_t *seg_tok_off;    /* exclusive prefix sum of seg_len */
  const int32_t *seg_q_off;      /* first row in Q/O/dO/dQ, -1 if the segment has no queries */
  const int32_t *seg_refcount;   /* samples that pass through the segment (Sec. 5.2) */
  const int32_t *anc_off, *anc_list;         /* CSR: strict ancestors root -> parent */
  const int32_t *seg_first_page, *seg_n_pages;
  const int32_t *page_seg, *page_bs, *page_valid, *page_pos, *page_refcount, *page_slot; /* [n_pages] */
  const int32_t *bt_off, *bt_pages;          /* CSR block table: ancestors' pages root -> parent, then own */
  const int32_t *tok_slot;                   /* [T] slot of every token in the pools */
  const int32_t *sample_end_seg, *sample_len; /* [n_samples] */
} psrl_plan_view_t;

/*
 * psrl_plan_build - host-side plan builder (paper Sec. 5.1 Adaptive Block
 * Allocation, Sec. 5.2 reference counts, Sec. 6 block metadata).
 * Turns the forest into the canonical plan (paged block table with a block
 * size per group) and a device work schedule.  Pure host code, no CUDA call.
 *   desc      HOST, read only during the call
 *   out_plan  HOST, receives a plan owned by the library (psrl_plan_destroy)
 * Errors: INVALID_ARG, BAD_TREE, BAD_BLOCK_SIZE, SHAPE, UNSUPPORTED,
 * POOL_FULL, HOST_OOM.  On error *out_plan is NULL.
 */
psrl_status_t psrl_plan_build(const psrl_tree_desc_t* desc, psrl_plan_t** out_plan);

/* Fills *out with borrowed host pointers.  INVALID_ARG on NULL. */
psrl_status_t psrl_plan_view(const psrl_plan_t* plan, psrl_plan_view_t* out);

/*
 * Borrowed HOST pointer to the device work schedule as psrl_plan_upload would
 * copy it (int32 words; *n_words = psrl_plan_device_bytes / 4).  The layout is
 * internal (a header of offsets, then the arrays: KV tiles, forward/dQ work
 * items with their KV-tile lists, dK/dV work items and splits, merge lists)
 * and not part of the bit-exact plan contract; it is exposed so that tests can
 * check its invariants - every (query row, key) pair of the tree covered
 * exactly once, every reduction a fixed total order (cf. the workload
 * estimate of Eq. 1 that the schedule balances) - without a GPU.
 * Valid until psrl_plan_destroy.  INVALID_ARG on NULL.
 */
psrl_status_t psrl_plan_schedule(const psrl_plan_t* plan, const int32_t** words, size_t* n_words);

/* Bytes of DEVICE memory psrl_plan_upload needs (0 for a NULL plan). */
size_t psrl_plan_device_bytes(const psrl_plan_t* plan);

/*
 * Copies the device schedule into caller-owned DEVICE memory (256-byte
 * aligned, >= psrl_plan_device_bytes) with cudaMemcpyAsync on `stream`
 * (a cudaStream_t passed as void*; NULL = default stream) and binds the plan
 * to that buffer.  The buffer must outlive every launch that uses the plan.
 * Errors: INVALID_ARG, WORKSPACE (too small), CUDA.
 */
psrl_status_t psrl_plan_upload(psrl_plan_t* plan, void* dev_buf, size_t bytes, void* stream);

/* Bytes of DEVICE workspace the forward / backward call needs (>= 256). */
size_t psrl_fwd_workspace_bytes(const psrl_plan_t* plan);
size_t psrl_bwd_workspace_bytes(const psrl_plan_t* plan);

/*
 * psrl_tree_attn_fwd - tree-causal attention forward (paper Sec. 2.5 attention
 * masking; Sec. 6: the attention backend locates K/V through block metadata).
 * For every query row i of a HAS_Q segment c and query head h (KV head
 * h / (Hq/Hkv)):  keys = all tokens of c's ancestors + tokens 0..i of c;
 *   O_i = softmax_j(scale * q_i . k_j) V,   LSE_i = ln sum_j exp(scale * q_i . k_j).
 * All tensor pointers are DEVICE pointers, 16-byte aligned, dtype = plan dtype (the Q-shaped ones may
 * be NULL when the plan has no query row at all, T_q = 0):
 *   q        [T_q, Hq, d]  read only; rows of segment c start at seg_q_off[c]
 *   k_pool   [Hkv, pool_capacity, d] read only; token t lives at slot tok_slot[t]
 *   v_pool   same layout.  Slots that hold no token (page pads, free slots)
 *            may contain anything, NaN included; they never reach an output.
 *   pool_capacity  slots per KV head in the caller's pools, >= plan pool_slots
 *   o        [T_q, Hq, d]  fully overwritten
 *   lse      [Hq, T_q] fp32 fully overwritten (natural log, scale inside)
 *   workspace, workspace_bytes  >= psrl_fwd_workspace_bytes(plan), 256-byte
 *            aligned; holds the device status word.  Concurrent launches need
 *            distinct workspaces.
 *   stream   cudaStream_t as void*
 * Errors: INVALID_ARG, SHAPE, WORKSPACE, CUDA.  Asynchronous.
 */
psrl_status_t psrl_tree_attn_fwd(const psrl_plan_t* plan, const void* q, const void* k_pool, const void* v_pool,
                                 int64_t pool_capacity, void* o, float* lse, float softmax_scale,
                                 void* workspace, size_t workspace_bytes, void* stream);

/*
 * psrl_tree_attn_bwd - backward of the above (paper Sec. 6: consumer adjoints
 * are accumulated on the shared prefix before one backward pass through its
 * producer).  Given dO (one row per shared token, already summed over the
 * samples that contain it):
 *   P = exp(S - LSE), dV = P^T dO, dP = dO V^T, D_i = dO_i . O_i,
 *   dS = P o (dP - D), dQ = scale dS K, dK = scale dS^T Q,
 * where dK/dV of a token sum over every query row that attends to it (its own
 * segment's later rows and all rows of all descendant segments) and over the
 * Hq/Hkv query heads of its KV head, in a fixed order.
 * DEVICE pointers, 16-byte aligned:
 *   q, k_pool, v_pool, o, lse   as in / as produced by the forward; read only
 *   d_o      [T_q, Hq, d] read only
 *   d_q      [T_q, Hq, d] fully overwritten
 *   dk_pool, dv_pool [Hkv, pool_capacity, d]: every slot of every page of the
 *            plan is overwritten (token slots: gradient; pad slots: 0); slots
 *            outside the plan's pages are not touched
 *   workspace >= psrl_bwd_workspace_bytes(plan): status word + D [Hq, T_q] fp32
 * Errors: INVALID_ARG, SHAPE, WORKSPACE, CUDA.  Asynchronous.
 */
psrl_status_t psrl_tree_attn_bwd(const psrl_plan_t* plan, const void* q, const void* k_pool, const void* v_pool,
                                 int64_t pool_capacity, const void* o, const float* lse, const void* d_o,
                                 void* d_q, void* dk_pool, void* dv_pool, float softmax_scale, void* workspace,
                                 size_t workspace_bytes, void* stream);

/*
 * psrl_tree_attn_bwd_static - the backward pass for callers that cannot
 * allocate device memory.  (The paper has no counterpart: this is a
 * convenience of this library.)
 *
 * psrl_tree_attn_bwd needs a caller-provided device workspace.  Callers that
 * must not call cudaMalloc - a latency-critical loop where an allocation would
 * synchronise the device, a plug-in inside a process whose GPU memory belongs
 * to another framework's pool, a process with a fixed memory budget - can use
 * this variant instead: its workspace is a fixed array inside the library
 * image (16 MiB + 256 bytes of device memory on every GPU that loads the
 * library, held until the process exits).  The call itself performs no
 * cudaMalloc / cudaFree and calls no allocating library routine.
 *
 * Same mathematics, same arguments (NULL Q-shaped pointers are accepted for a
 * plan without query rows, as there) and bit-identical results as
 * psrl_tree_attn_bwd, except:
 *   - no workspace arguments;
 *   - limit: the array stands in for the whole workspace, so a plan fits when
 *       psrl_bwd_workspace_bytes(plan) <= PSRL_BWD_STATIC_SCRATCH_BYTES,
 *     i.e. 256 bytes of header + D (one float per query row and head, so
 *     n_q_heads * T_q <= 4,194,304 at the very most) + the fp32 slabs of split
 *     KV tiles (n_kv_heads * 128 KiB each) + the partial dQ rows of cascaded
 *     prefixes (n_q_heads * 512 bytes each), the last two only for plans whose
 *     schedule has them.  Larger plans return PSRL_ERR_WORKSPACE and must use
 *     psrl_tree_attn_bwd;
 *   - status_workspace (HOST pointer, may be NULL) receives the DEVICE address
 *     of the array's status header; pass it to psrl_device_status to read the
 *     launch's device status.
 * Set-up: the first call on each device looks up the array's device address
 * (with that device current) and caches it.  Make that first call outside any
 * CUDA stream capture.
 * Sharing: every call on a device uses the same array, which keeps the
 * previous call's contents (the library clears what has to start at zero).
 * Two calls that overlap on the GPU - different streams, or different host
 * threads - race on it; serialise them, or use psrl_tree_attn_bwd with
 * separate workspaces.
 * Errors: INVALID_ARG, SHAPE, WORKSPACE (plan not uploaded, or over the
 * limit), CUDA.  Asynchronous.
 */
#define PSRL_BWD_STATIC_SCRATCH_BYTES ((size_t)16777472) /* 16 MiB + 256 */
psrl_status_t psrl_tree_attn_bwd_static(const psrl_plan_t* plan, const void* q, const void* k_pool,
                                        const void* v_pool, int64_t pool_capacity, const void* o, const float* lse,
                                        const void* d_o, void* d_q, void* dk_pool, void* dv_pool,
                                        float softmax_scale, void** status_workspace, void* stream);

/*
 * Synchronises `stream`, then reads the status word the last launch that used
 * `workspace` left: PSRL_OK, PSRL_ERR_TIMEOUT (a bounded wait gave up; outputs
 * are invalid) or PSRL_ERR_INTERNAL.  CUDA errors map to PSRL_ERR_CUDA.
 */
psrl_status_t psrl_device_status(const void* workspace, void* stream);

/*
 * psrl_kv_scatter / psrl_kv_gather - the neighbours of the attention calls: K and V leave the
 * projections token-major, the attention reads them through the paged pools (Sec. 6, KV manager), and
 * the gradients of the pools go back token-major.  scatter writes token t of the plan's tree (canonical
 * order, rows of `k_tok` / `v_tok`) to slot tok_slot[t] of every KV head; gather is the inverse read.
 * Slots that hold no token are neither written (scatter) nor read (gather).
 *   k_tok, v_tok  [T, Hkv, d] DEVICE, plan dtype, 16-byte aligned (either pair member may be NULL: skipped)
 *   k_pool, v_pool [Hkv, pool_capacity, d] DEVICE
 * Errors: INVALID_ARG, SHAPE, WORKSPACE (plan not uploaded), CUDA.  Asynchronous on `stream`.
 */
psrl_status_t psrl_kv_scatter(const psrl_plan_t* plan, const void* k_tok, const void* v_tok, void* k_pool,
                              void* v_pool, int64_t pool_capacity, void* stream);
psrl_status_t psrl_kv_gather(const psrl_plan_t* plan, const void* k_pool, const void* v_pool,
                             int64_t pool_capacity, void* k_tok, void* v_tok, void* stream);

/*
 * Benchmark aid (no counterpart in the paper): psrl_tree_attn_bwd with a mask
 * of the backward kernels to launch, so that each can be timed on its own
 * with CUDA events.  Bit 0: D = rowsum(dO o O) pre-pass, bit 1: dQ kernel
 * (+ its merge), bit 2: dK/dV kernel (+ its reduce).  phases = 7 is exactly
 * psrl_tree_attn_bwd; with any other mask the outputs of the skipped kernels
 * are left untouched (and a skipped pre-pass leaves D as the previous call on
 * this workspace wrote it).  Stateless: the mask is an argument of the call.
 */
psrl_status_t psrl_bench_bwd_phases(const psrl_plan_t* plan, const void* q, const void* k_pool, const void* v_pool,
                                    int64_t pool_capacity, const void* o, const float* lse, const void* d_o,
                                    void* d_q, void* dk_pool, void* dv_pool, float softmax_scale, void* workspace,
                                    size_t workspace_bytes, void* stream, int phases);

/*
 * Number of kernels one psrl_tree_attn_fwd (backward == 0) or
 * psrl_tree_attn_bwd (backward != 0, all phases enabled) call launches for
 * this plan (no counterpart in the paper; bookkeeping for benchmarks).
 * Forward: 1, plus a merge when rows are assembled from partial results
 * (cascaded prefixes / split-KV).  Backward: D pre-pass + dQ + dK/dV, plus the
 * dQ merge, plus one fixed-order reduction when the bf16 schedule splits
 * heavy KV tiles.  0 for a NULL plan.
 */
int psrl_launch_count(const psrl_plan_t* plan, int backward);

/* Last CUDA error string seen by the library on this thread (HOST, static storage). */
const char* psrl_last_cuda_error(void);

void psrl_plan_destroy(psrl_plan_t* plan);
const char* psrl_status_string(psrl_status_t s);

#ifdef __cplusplus
}
#endif
#endif /* PSRL_H_ */
