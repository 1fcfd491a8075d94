/*
 * decode_attn.h - C ABI of the B200 (sm_100a) paged decode-attention library.
 *
 * The operation (Section 3.1 and Algorithm 1 step 2 of the vSkipper paper):
 * in one decode step every sequence ("row") has one query token that attends
 * over all of that sequence's cached keys and values, which live in a paged
 * KV cache and are found through per-sequence page mappings (Invariant 2).
 * The row's own K/V is written before attention, so the whole cached range
 * [0, seq_len) is attended and no causal mask is applied.  Query heads are
 * grouped: query head h reads KV head h / (num_q_heads / num_kv_heads).
 *
 *   s_t = sm_scale * <q[b,h,:], K[page(t), slot(t), g, :]>,  page(t) = block_table[b][t / page_size]
 *   out[b,h,:] = sum_t softmax_t(s)_t * V[page(t), slot(t), g, :],   lse[b,h] = log sum_t exp(s_t)
 *
 * The library splits each sequence's token range into partitions ("splits"),
 * computes one partial result per (sequence, KV head, split) with a running
 * maximum and sum of exponentials in fp32, and merges the partials of a
 * sequence by their log-sum-exp weights.  The paper does not describe the
 * split or the merge; they are an exact re-association of the formula above.
 *
 * Conventions
 *  - Every pointer marked "device" is caller-owned device memory of the
 *    current CUDA device; "host" is ordinary host memory.  The library never
 *    allocates or frees device memory in run/combine and never synchronises
 *    the caller's stream there.  It owns only the plan object.
 *  - Every function returns an int status (da_status_t); nothing throws or
 *    aborts across this boundary and no kernel traps.  Conditions detected on
 *    the device (stale lengths, page ids outside the pool, a wait that gave
 *    up) are recorded in a status word read by decode_attn_last_device_status.
 *  - Strides are in elements.  The innermost (head_dim) axis is contiguous.
 *  - There is no CPU fallback: without a usable CUDA device the compute entry
 *    points return DA_ERR_CUDA.
 */
#ifndef DECODE_ATTN_H_
#define DECODE_ATTN_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#if defined(__CUDACC__) || defined(__CUDA_RUNTIME_API_H__) || defined(__DRIVER_TYPES_H__)
#include <cuda_runtime_api.h>
#else
typedef struct CUstream_st *cudaStream_t;
#endif

typedef struct decode_attn_plan decode_attn_plan_t; /* opaque, library-owned */

typedef enum {
    DA_OK = 0,
    DA_ERR_INVALID_ARG = -1,         /* null pointer, non-positive size, misaligned pointer or stride */
    DA_ERR_UNSUPPORTED = -2,         /* a shape, dtype or policy this build has no kernel for          */
    DA_ERR_WORKSPACE_TOO_SMALL = -3,
    DA_ERR_STALE_PLAN = -4,          /* seq_lens differ from the ones the plan was made for            */
    DA_ERR_CUDA = -5,                /* a CUDA runtime/driver call failed, or no device                */
    DA_ERR_BAD_PAGE = -6,            /* a referenced block-table entry lies outside [0, num_pages)     */
    DA_ERR_TIMEOUT = -7              /* a bounded device-side wait gave up                             */
} da_status_t;

enum { DA_DTYPE_BF16 = 1, DA_DTYPE_FP32 = 2, DA_DTYPE_FP16 = 3 };

typedef enum {
    DA_SPLIT_AUTO = 0,          /* chunk length chosen from the length mix and the SM count          */
    DA_SPLIT_FIXED_COUNT = 1,   /* every sequence gets exactly fixed_count splits (some may be empty) */
    DA_SPLIT_DETERMINISTIC = 2  /* boundaries at multiples of chunk_tokens (of the longer chunk that
                                   max_splits asks for on a long sequence): a function of seq_len only */
} da_split_mode_t;

typedef enum {
    DA_KERNEL_AUTO = 0,     /* MMA_TMA (every supported head_dim and group size); with
                               shared_prefix_tokens: UMMA_PREFIX where it applies, else MMA_TMA       */
    DA_KERNEL_SIMT = 1,     /* CUDA-core kernel, 16-byte vectorised global loads; groups of up to 8   */
    DA_KERNEL_MMA_TMA = 2,  /* TMA-staged pages in shared memory, mma.sync (bf16 or fp16) for QK^T, PV;
                               groups of up to 16 heads (two 8-column tiles of heads above 8)         */
    DA_KERNEL_UMMA_PREFIX = 3 /* shared-prefix plans only (head_dim 128, groups of 1 to 16 heads): the prefix
                               units run on the tcgen05 tensor cores, 128 query rows at a time with
                               accumulators in tensor memory; what follows the prefix runs as MMA_TMA */
} da_kernel_t;

/* Split policy.  Zero-initialise for the defaults. */
typedef struct {
    int32_t split_mode;     /* da_split_mode_t                                                       */
    int32_t fixed_count;    /* FIXED_COUNT: splits per sequence (>= 1)                               */
    int32_t chunk_tokens;   /* DETERMINISTIC: chunk length, a multiple of 16 (0: 256; with the default
                               max_splits a sequence of L tokens then gets chunks of
                               max(256, L / 32 rounded up to 16) tokens).
                               AUTO: smallest chunk the planner may choose (0: 256)                  */
    int32_t max_splits;     /* upper bound on the splits of one sequence (0: 512, DETERMINISTIC 32;
                               at most 1024); a longer sequence gets longer chunks                   */
    int32_t sm_count;       /* 0: the current device's multiprocessor count                          */
    int32_t kernel;         /* da_kernel_t                                                           */
    int32_t fuse_combine;   /* 0: decode_attn_combine must follow decode_attn_run.
                               1: run's launch carries merge blocks behind the attending ones; they
                               wait (bounded, DA_ERR_TIMEOUT) for a sequence's records and merge them  */
    int32_t capacity_batch; /* > 0: the plan can be refreshed in place for any batch <= this value
                               (decode_attn_plan_update) and launches a fixed grid whose surplus
                               blocks exit at once (Algorithm 1 step 6, "grid exit")                  */
    int32_t capacity_tokens;/* with capacity_batch: upper bound on sum(seq_lens) of any refresh      */
    int32_t ctas_per_sm;    /* 0: from the occupancy of the chosen kernel                            */
    int32_t shared_prefix_tokens; /* > 0: the caller promises that the first this-many tokens of every
                               sequence live in the same physical pages (the block-table rows agree on
                               their first shared_prefix_tokens / page_size entries, as with few-shot
                               prompts served from a prefix cache).  A multiple of page_size, at most
                               every seq_len.  The prefix is then attended once per block of
                               sequences instead of once per sequence.  Tensor-core kernels only
                               (MMA_TMA: groups of up to 4 heads; UMMA_PREFIX: head_dim 128, groups of
                               up to 16), separate combine, no capacity plan, not FIXED_COUNT.         */
    int32_t reserved[5];
} decode_attn_policy_t;

typedef struct {
    int32_t batch;              /* live sequences B (rows of q, out, block_table)                    */
    int32_t num_q_heads;
    int32_t num_kv_heads;       /* divides num_q_heads; group size <= 16 (DA_ERR_UNSUPPORTED above)  */
    int32_t head_dim;           /* 64 or 128                                                         */
    int32_t page_size;          /* tokens per page: 16, 32, 64, 128 or 256                           */
    int32_t max_pages_per_seq;  /* row stride of block_table, in entries                             */
    int64_t num_pages;          /* pages in each pool                                                */
    int64_t k_stride_page, k_stride_token, k_stride_head;   /* elements; multiples of 8              */
    int64_t v_stride_page, v_stride_token, v_stride_head;
    int32_t kv_dtype;           /* DA_DTYPE_BF16 or DA_DTYPE_FP16 (the paper serves one model family in
                                   each, Section 4.1)                                                 */
    int32_t q_dtype;            /* the same as kv_dtype                                              */
    int32_t out_dtype;          /* DA_DTYPE_FP32, DA_DTYPE_BF16 or DA_DTYPE_FP16                     */
    float sm_scale;             /* 0: 1/sqrtf(head_dim) evaluated in fp32                            */
} decode_attn_shape_t;

/* One unit of work: one KV head of one sequence over one token range.  With
 * policy.shared_prefix_tokens a second kind exists: a chunk of the shared
 * prefix attended for a block of consecutive sequences at once; it has
 * kv_head = g | (sequences_in_block << 16), seq = the block's first sequence
 * and slot = -2 (each sequence's record goes to its own slots). */
typedef struct {
    int32_t seq;          /* b                                                                       */
    int32_t kv_head;      /* g (low 16 bits)                                                         */
    int32_t tok_begin;    /* first token, a multiple of 16 (of chunk_tokens in DETERMINISTIC mode)  */
    int32_t tok_end;      /* one past the last token; tok_end == tok_begin marks an empty split      */
    int32_t slot;         /* index of the partial in the workspace, -1: writes `out` directly        */
    int32_t seq_len;      /* the length the plan was made for (checked against device seq_lens)      */
    int32_t split_index;  /* position of this split within its sequence                              */
    int32_t n_splits;     /* splits of this sequence                                                 */
} decode_attn_unit_t;

typedef struct {
    int64_t n_units;          /* work units = thread blocks that do work                             */
    int64_t grid;             /* thread blocks launched: the tensor-core kernel walks the work list
                                 with at most sm_count * ctas_per_sm blocks; fixed for a capacity plan */
    int64_t n_slots;          /* partial results held in the workspace                               */
    int64_t workspace_bytes;
    int32_t chunk_tokens;     /* AUTO / DETERMINISTIC: the chunk length in use (0 for FIXED_COUNT)   */
    int32_t kernel;           /* the da_kernel_t actually used                                       */
    int32_t ctas_per_sm;      /* resident blocks per SM the planner assumed                          */
    int32_t sm_count;
    int32_t fuse_combine;
    int32_t max_splits_used;  /* largest split count of any sequence                                 */
    int32_t block_threads;
    int32_t dynamic_smem_bytes;
} decode_attn_plan_info_t;

/* ---------------------------------------------------------------------------
 * Planner.  The paper gives no split policy; it only requires that launch
 * metadata is never stale (Invariant 2) and that launches are capture-safe
 * (Algorithm 1 step 6).
 *
 * decode_attn_plan_layout is the pure host function behind decode_attn_plan:
 * from the length mix it chooses the splits of every sequence and emits the
 * work list.  It touches no device.  units_out may be NULL to query sizes;
 * otherwise it must hold max_units entries (DA_ERR_INVALID_ARG if too few).
 * splits_out and slot_base_out are [batch] or NULL.  The result is a
 * deterministic function of (shape, policy, seq_lens, sm_count, ctas_per_sm);
 * in DETERMINISTIC mode each sequence's boundaries depend on its own length
 * and policy.chunk_tokens only.
 * ------------------------------------------------------------------------- */
int decode_attn_plan_layout(const decode_attn_shape_t *shape, const decode_attn_policy_t *policy,
                            const int32_t *seq_lens_host, int32_t sm_count, int32_t ctas_per_sm,
                            decode_attn_unit_t *units_out, int64_t max_units, int64_t *n_units_out,
                            int32_t *splits_out, int32_t *slot_base_out, int64_t *n_slots_out,
                            int32_t *chunk_tokens_out);

/* Builds a plan for one decode step: validates shape and policy, runs the
 * planner on seq_lens_host [batch] (host), starts the upload of the work list
 * to a small device buffer the plan owns (on an internal stream, without
 * waiting for it: the plan's first launch on a caller's stream is ordered
 * behind the upload on the device) and reports the workspace size run/combine
 * need.  *plan_out is set only on DA_OK.  The device buffer, its pinned mirror
 * and the stream come from a small cache fed by destroyed plans, so
 * re-planning every step does not allocate.  A plan is tied to the CUDA device
 * current at creation and must not be used by two launches that overlap on
 * the GPU.
 *
 * Lifetime: plan / run / combine / destroy may follow one another without any
 * synchronisation - destroying a plan whose kernels are still queued or
 * running is allowed; its device buffer is handed to a later plan only behind
 * those kernels.  The one exception is stream capture: launches recorded into
 * a CUDA graph run when the graph is replayed, so a plan must outlive every
 * replay of a graph that holds its launches. */
int decode_attn_plan(const decode_attn_shape_t *shape, const decode_attn_policy_t *policy,
                     const int32_t *seq_lens_host, decode_attn_plan_t **plan_out,
                     size_t *workspace_bytes_out);

/* Re-plans in place for new lengths (and a new live batch <= capacity_batch)
 * and enqueues the upload of the refreshed work list on `stream`; the device
 * addresses, grid and kernel stay the same, so a CUDA graph captured around
 * run/combine keeps working.  Only for plans made with capacity_batch > 0.
 * The copy is ordered like any other work on `stream`: behind the launches
 * already queued there, ahead of those that follow; launches on another
 * stream are for the caller to order.  seq_lens_host must stay valid until
 * the call returns (it is copied). */
int decode_attn_plan_update(decode_attn_plan_t *plan, int32_t batch, const int32_t *seq_lens_host,
                            cudaStream_t stream);

int decode_attn_plan_get_info(const decode_attn_plan_t *plan, decode_attn_plan_info_t *info_out);

/* Copies the plan's work list (host copy) into units_out[max_units]. */
int decode_attn_plan_get_units(const decode_attn_plan_t *plan, decode_attn_unit_t *units_out,
                               int64_t max_units);

/* DA_OK if seq_lens_host [batch] equals the lengths the plan was made for,
 * DA_ERR_STALE_PLAN otherwise (Invariant 2: row metadata is never stale). */
int decode_attn_plan_check(const decode_attn_plan_t *plan, int32_t batch, const int32_t *seq_lens_host);

int decode_attn_plan_destroy(decode_attn_plan_t *plan);

/* ---------------------------------------------------------------------------
 * Split-KV partial kernel (Algorithm 1 step 2, the attention read).
 *
 *   q            device, shape.q_dtype (bf16 or fp16) [batch, num_q_heads, head_dim], contiguous, 16-byte aligned
 *   k_cache      device, shape.kv_dtype pool addressed by the k_stride_* of the shape, 16-byte aligned
 *   v_cache      device, same with v_stride_*
 *   block_table  device, int32 [batch, max_pages_per_seq]; entries at or beyond
 *                ceil(seq_len / page_size) are never read; pages may be shared by rows
 *   seq_lens     device, int32 [batch]; must equal the planned lengths (checked per block)
 *   out          device, [batch, num_q_heads, head_dim] in shape.out_dtype
 *   lse_or_null  device, fp32 [batch, num_q_heads] or NULL
 *   workspace    device, >= workspace_bytes from the plan, 256-byte aligned (may be NULL if 0)
 *
 * One launch on `stream`.  Sequences with a single split write `out` (and
 * lse) directly; the others write unnormalised fp32 partials with their
 * running maximum and sum into the workspace, and - with fuse_combine - the
 * merge blocks at the end of the same launch merge them into `out` as soon
 * as the records of a (sequence, KV head) have all been published.
 * Rows with seq_len 0 get zeros and lse = -inf.  Capture-safe.
 *
 * The kernel is launched with a programmatic dependency on whatever precedes
 * it on `stream`: its blocks may become resident and fetch the plan's work
 * list while that work drains, but what it computes with - q, K/V, seq_lens,
 * block_table and run_mask - is read only after it has completed, so ordinary
 * stream order holds for every caller-visible buffer.  One thing happens
 * earlier in the tensor-core kernel: block_table and run_mask are also read
 * before that point to choose a few K/V lines to prefetch into L2, and the
 * lines of q, seq_lens and block_table that the first unit of every block
 * needs are asked into L2 as well.  The early values are used for nothing
 * else and everything is read again afterwards (L2 is where the writes of
 * the kernel before arrive, so a line brought in early is never stale), so a
 * kernel that is still writing these buffers does no harm; they only have to
 * be mapped device memory when the launch is enqueued.
 *
 * With a run_mask the units are handed to the thread blocks at run time (a
 * queue in the plan's device buffer), so that the time a masked row saves
 * follows the bytes it saves; the results do not depend on which block ran
 * which unit.
 * ------------------------------------------------------------------------- */
int decode_attn_run(const decode_attn_plan_t *plan, const void *q, const void *k_cache,
                    const void *v_cache, const int32_t *block_table, const int32_t *seq_lens, void *out,
                    float *lse_or_null, void *workspace, size_t workspace_bytes, cudaStream_t stream);

/* Extended arguments; set struct_size = sizeof(decode_attn_run_args_t). */
typedef struct {
    uint32_t struct_size;
    uint32_t flags;             /* must be 0 */
    const void *q;
    const void *k_cache;
    const void *v_cache;
    const int32_t *block_table;
    const int32_t *seq_lens;
    const uint8_t *run_mask;    /* device, [batch] or NULL.  A row whose byte is 0 reads no KV and
                                   emits zero (lse = -inf): the RUN mask of Algorithm 1 step 2. */
    void *out;
    float *lse;
    void *workspace;
    size_t workspace_bytes;
    /* Fused own-layer KV write (both NULL: none; struct_size may also stop before these two
     * fields).  device, 16-bit (shape.kv_dtype) [batch, num_kv_heads, head_dim], 16-byte aligned:
     * every row's new K and V rows.  The launch stores them at logical position seq_lens[b] - 1
     * (as decode_attn_append_kv would: masked rows too, rows of length 0 not) and attends over
     * them in the same pass, so k_cache and v_cache are modified although they are declared
     * const here; the result is bit for bit that of decode_attn_append_kv followed by this call
     * without the two pointers (Algorithm 1 step 2: the row's K/V is written, then the row
     * attends).  Tensor-core kernel, plans without a shared prefix (DA_ERR_UNSUPPORTED else). */
    const void *new_k;
    const void *new_v;
} decode_attn_run_args_t;

int decode_attn_run_ex(const decode_attn_plan_t *plan, const decode_attn_run_args_t *args,
                       cudaStream_t stream);

/* Own-layer KV write (Invariant 1; Algorithm 1 step 2: every valid row's K/V
 * is written through the cache-write path before attention, whether or not
 * the row then attends).  Stores row b's new K and V rows at logical position
 * seq_lens[b] - 1: page block_table[b][(L-1) / page_size], slot
 * (L-1) % page_size.  Bit-exact copy; rows with seq_len 0 write nothing.
 *   new_k, new_v  device, 16-bit (shape.kv_dtype) [batch, num_kv_heads, head_dim], 16-byte aligned
 *   block_table, seq_lens  device (seq_lens are the lengths INCLUDING the new token)
 *   k_cache, v_cache  device pools of the shape, modified in place
 * One launch on `stream`; a decode_attn_run enqueued after it on the same
 * stream sees the new rows.  The run mask plays no part here. */
int decode_attn_append_kv(const decode_attn_shape_t *shape, const void *new_k, const void *new_v,
                          const int32_t *block_table, const int32_t *seq_lens, void *k_cache, void *v_cache,
                          cudaStream_t stream);

/* The same write with the device-side checks reported: a row whose page id lies
 * outside the pool, or whose position lies beyond max_pages_per_seq, is not
 * written (as above) and records DA_ERR_BAD_PAGE / DA_ERR_STALE_PLAN in the
 * status word of `plan`, which decode_attn_last_device_status reads.  The
 * shape is the plan's. */
int decode_attn_append_kv_checked(const decode_attn_plan_t *plan, const void *new_k, const void *new_v,
                                  const int32_t *block_table, const int32_t *seq_lens, void *k_cache,
                                  void *v_cache, cudaStream_t stream);

/* Merge of KV-range shards (context parallelism; the paper has no multi-GPU
 * path - this is the one exchange step the decode path has when a single
 * long sequence is sharded by token range).  Every shard attended its own
 * token range of the same (sequence, query head) rows with plan / run /
 * combine and holds a normalised output with its log-sum-exp; after the
 * shards' results were gathered (torch.distributed all_gather over NCCL, or
 * one process that ran the shards one after the other), this call writes
 *   M = max_r lse_r;  w_r = e^{lse_r - M};  out = sum_r w_r out_r / sum_r w_r;
 *   lse = M + log(sum_r w_r)
 * in ascending shard order (fixed: the result does not depend on timing).
 *   out_shards  device, fp32 [n_shards, batch, num_q_heads, head_dim], 16-byte aligned
 *   lse_shards  device, fp32 [n_shards, batch, num_q_heads]; -inf marks a shard
 *               whose range was empty for that row (it weighs exactly zero)
 *   out         device, [batch, num_q_heads, head_dim] in shape.out_dtype, 16-byte aligned
 *   lse_or_null device, fp32 [batch, num_q_heads] or NULL
 * Rows that are empty in every shard get zeros and lse = -inf.  1 <= n_shards
 * <= 1024.  One launch on `stream`, nothing is allocated, capture-safe. */
int decode_attn_merge_shards(const decode_attn_shape_t *shape, int32_t n_shards, const float *out_shards,
                             const float *lse_shards, void *out, float *lse_or_null, cudaStream_t stream);

/* LSE combine: merges the partials `run` left in the workspace, per
 * (sequence, query head), in ascending split order:
 *   M = max_i m_i;  out = sum_i e^{m_i-M} o_i / sum_i e^{m_i-M} l_i;  lse = M + log(sum_i e^{m_i-M} l_i)
 * Empty splits weigh exactly zero.  One launch on `stream` (none if no
 * sequence was split).  With a fuse_combine plan the call is redundant but
 * valid: it recomputes the same bits. */
int decode_attn_combine(const decode_attn_plan_t *plan, const void *workspace, void *out,
                        float *lse_or_null, cudaStream_t stream);

/* Synchronises `stream`, returns the worst condition the kernels recorded
 * since the last call (DA_OK, DA_ERR_STALE_PLAN, DA_ERR_BAD_PAGE,
 * DA_ERR_TIMEOUT) and clears it.  For tests and debugging.  plan == NULL
 * reads the status word of decode_attn_step_static (which has no plan) on the
 * current device instead. */
int decode_attn_last_device_status(const decode_attn_plan_t *plan, cudaStream_t stream);

/* Host-only check of a block table against the shape: every entry below
 * ceil(seq_len / page_size) must lie in [0, num_pages). */
int decode_attn_validate_block_table(const decode_attn_shape_t *shape, const int32_t *seq_lens_host,
                                     const int32_t *block_table_host);

/* Host-only check of the promise behind policy.shared_prefix_tokens: every
 * sequence is at least that long and every block-table row starts with the
 * same shared_prefix_tokens / page_size page ids as row 0 (DA_ERR_BAD_PAGE if
 * a row differs).  The prefix cache of the paper's engine serves few-shot
 * prompts this way (Appendix J). */
int decode_attn_validate_shared_prefix(const decode_attn_shape_t *shape, int32_t shared_prefix_tokens,
                                       const int32_t *seq_lens_host, const int32_t *block_table_host);

/* ---------------------------------------------------------------------------
 * Debug / measurement helpers that reuse the kernels' page addressing.
 * ------------------------------------------------------------------------- */

/* Writes sequence `seq`'s K and V rows in logical token order,
 * k_out / v_out: device, 16-bit like the pools, [seq_len, num_kv_heads, head_dim], fetched
 * through the same tensor maps and page lookups as the MMA/TMA kernel.
 * Must be bit-exact with a host gather. */
int decode_attn_debug_gather(const decode_attn_plan_t *plan, int32_t seq, const void *k_cache,
                             const void *v_cache, const int32_t *block_table, void *k_out, void *v_out,
                             cudaStream_t stream);

/* Gather-only probe: streams exactly the K/V bytes `run` would read, through
 * the same loads, and folds them into checksum_out (device, uint32 [n_units]);
 * no attention arithmetic.  Its time is the ceiling for this access pattern. */
int decode_attn_gather_probe(const decode_attn_plan_t *plan, const void *k_cache, const void *v_cache,
                             const int32_t *block_table, uint32_t *checksum_out, cudaStream_t stream);

/* Test hook for the bounded waits (failure detection without a fault): launches
 * the plan's partial kernel exactly as decode_attn_run_ex would, except that
 * its producer warps withhold their loads and every wait of the launch gives
 * up after limit_cycles clock cycles (clamped to [100,000, the ordinary limit
 * of about a second]) instead of the ordinary limit.  Nothing is at fault and
 * nothing hangs: the waits run out, the blocks void their results and leave,
 * DA_ERR_TIMEOUT is recorded in the plan's status word, and `out` holds no
 * valid result.  After decode_attn_last_device_status has read (and cleared)
 * that status the plan is good for ordinary launches again.  Plans of the
 * MMA_TMA kernel only (DA_ERR_UNSUPPORTED otherwise). */
int decode_attn_debug_expire_wait(const decode_attn_plan_t *plan, const decode_attn_run_args_t *args,
                                  int64_t limit_cycles, cudaStream_t stream);

/* ---------------------------------------------------------------------------
 * Whole step from host buffers: copies q, both pools, block table and
 * lengths to the device (into a grow-only arena the library keeps), plans,
 * runs, combines, copies `out` (and lse) back and synchronises.  pool_elems
 * is the element count of each pool.  For end-to-end measurement and simple
 * callers; serving engines keep the pools resident and use plan/run/combine.
 * ------------------------------------------------------------------------- */
int decode_attn_host_step(const decode_attn_shape_t *shape, const decode_attn_policy_t *policy,
                          const void *q_host, const void *k_cache_host, const void *v_cache_host,
                          int64_t pool_elems, const int32_t *block_table_host,
                          const int32_t *seq_lens_host, void *out_host, float *lse_host_or_null);

/* ---------------------------------------------------------------------------
 * Allocation-free step.  (The paper has no counterpart to this entry point;
 * it exists for integration, not for the method.)
 *
 * One whole decode-attention step - the split-KV partial kernel followed by
 * the combine kernel - that never asks the CUDA allocator for anything: no
 * plan object, no cudaMalloc / cudaFree, no pinned allocation, no workspace
 * argument.  It is meant for callers that cannot allocate device memory at
 * the point of the call: a serving engine that handed every remaining byte of
 * HBM to its KV pool at start-up (a later cudaMalloc simply fails), or a
 * latency-critical path that cannot accept the device-wide synchronisation an
 * allocation implies.
 *
 * The work list and the partial records live in a scratch array compiled
 * into the library (8 MiB of device memory, held by every GPU that loads the
 * library until the process exits).  The step is planned with the
 * deterministic split policy at its defaults, so its result equals
 * plan / run / combine with that policy.
 *
 * Limits: batch <= 1,024; at most 4,096 work units (batch x KV heads x
 * splits); the partial records must fit in about 7.8 MiB (e.g. 470 split
 * sequences' worth of slots at 8 KV heads x group 4 x head_dim 128).  A step
 * beyond these returns DA_ERR_WORKSPACE_TOO_SMALL and launches nothing.
 *
 * All calls share the one array, which keeps whatever the previous call left
 * there; nothing in it has to start at zero (every call uploads what its
 * kernels read and writes its records before reading them).  Two calls whose
 * kernels overlap on the GPU (different streams, no ordering) race on it -
 * order them.
 *
 * Not for stream capture: every call plans on the host and uploads its own
 * work list (two small copies from pageable memory, taken by the runtime
 * before the call returns), so a captured call would replay a stale list; a
 * call on a capturing stream returns DA_ERR_UNSUPPORTED.  The first call on a
 * device also looks up the array's device address and sets kernel attributes.
 *
 * Conditions its kernels detect on the device (lengths that differ from
 * seq_lens_host, page ids outside the pool, a wait that gave up) void the
 * affected rows and are recorded in a status word inside the array:
 * decode_attn_last_device_status(NULL, stream) returns and clears it.
 * Arguments are those of decode_attn_plan + decode_attn_run:
 * seq_lens_host [batch] on the host, everything else on the device.
 * ------------------------------------------------------------------------- */
int decode_attn_step_static(const decode_attn_shape_t *shape, const int32_t *seq_lens_host, const void *q,
                            const void *k_cache, const void *v_cache, const int32_t *block_table,
                            const int32_t *seq_lens, void *out, float *lse_or_null, cudaStream_t stream);

/* Frees what the library caches between calls: the arena of
 * decode_attn_host_step and the buffers parked by destroyed plans. */
int decode_attn_host_release(void);

/* ---------------------------------------------------------------------------
 * Decode profitability rule (Section 3.3, Appendix D): what the RUN mask is
 * worth.  A skipped row saves its KV read at each routed layer, so with a
 * fraction s of decisions skipping over L_r routed layers a step holding V
 * resident tokens saves s * L_r * b * V / BW seconds against a fixed per-step
 * cost tau; routing pays above V* = tau * BW / (s * L_r * b).  Host only.
 * ------------------------------------------------------------------------- */
int decode_attn_breakeven_tokens(double tau_seconds, double bandwidth_bytes_per_s, double skip_fraction,
                                 int32_t routed_layers, double kv_bytes_per_token_layer, double *v_star_out);

/* Served thresholds of the rule: exit at V*, enter at 1.25 V*, each rounded
 * half up to a multiple of round_to tokens (0: no rounding; the paper's
 * printed thresholds use 10,000). */
int decode_attn_switch_thresholds(double v_star, double round_to, double *exit_tokens_out,
                                  double *enter_tokens_out);

/* One step of the hysteresis: returns 1 (routed) once resident_tokens reaches
 * enter_tokens, 0 (dense for newly starting requests) once it falls to
 * exit_tokens, and routed_now in between. */
int decode_attn_switch_next(int32_t routed_now, double resident_tokens, double exit_tokens, double enter_tokens);

const char *decode_attn_strerror(int status);

/* "major.minor arch" of this build, e.g. "0.1 sm_100a". */
const char *decode_attn_version(void);

#ifdef __cplusplus
}
#endif
#endif /* DECODE_ATTN_H_ */
