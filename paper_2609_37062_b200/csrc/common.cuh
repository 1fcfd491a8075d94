// Device-side pieces shared by the partial kernels and the combine kernel:
// the launch parameter block, the plan's device header, the unit epilogue
// (partial write, ticket, in-kernel merge) and the LSE merge itself.
#pragma once

#include <cuda_bf16.h>
#include <cuda_fp16.h>
#include <cuda_runtime.h>

#include <cstdint>

#include "decode_attn.h"

namespace da {

// First words of the plan's device buffer, refreshed by every upload.
struct DevHeader {
    int32_t n_units;
    int32_t batch;
    int32_t n_ranked;       // entries of the rank-ordered unit list (0: none), see KernelParams::unit_rank
    int32_t first_binned;   // position of the first binned unit in the work list
};

struct SeqInfo {
    int32_t slot_base;  // -1: single split, written directly
    int32_t n_splits;
    int32_t seq_len;    // the length the plan was made for
    int32_t pad;
};

struct KernelParams {
    const __nv_bfloat16* q;
    const __nv_bfloat16* k;
    const __nv_bfloat16* v;
    const int32_t* block_table;
    const int32_t* seq_lens;
    const uint8_t* run_mask;
    // Own-layer KV write fused into the attention launch (NULL: none): new K and V rows [batch][Hkv][D] of the
    // 16-bit input type, stored at position seq_len - 1 of every row and attended from there.
    const __nv_bfloat16* new_k;
    const __nv_bfloat16* new_v;
    void* out;
    float* lse;
    float* ws;     // [n_slots][Hkv] partial records, see rec_floats()
    const DevHeader* header;
    const decode_attn_unit_t* units;
    const SeqInfo* seq_info;
    const int32_t* block_begin;  // [grid + 1]: block b walks units block_begin[b] .. block_begin[b+1]; NULL: unit b
    const int2* unit_rank;       // [n_ranked] the binned unit with cost rank j (0: the most expensive): its position in the
                                 // work list and its sequence (-1: no RUN mask applies, a shared-prefix unit); the order
                                 // in which launches with a RUN mask hand the units out
    int32_t* queue;              // two counters, zero between launches: units drawn from unit_rank beyond the first of
                                 // every block, blocks that have drawn their last (NULL: no rank list)
    int32_t n_ranked;            // entries of unit_rank (0: none); capacity plans read it from the header
    int32_t first_binned;        // position of the first binned unit in the work list
    int32_t may_rank;            // capacity plans: the rank list exists (how long it is changes with every refresh)
    int32_t* tickets;  // [2][batch][Hkv], zero between launches: records published / slices merged per (sequence, KV head)
    int32_t* status;   // worst da_status_t seen by any block (0 = ok)
    int64_t k_stride_page, k_stride_token, k_stride_head;
    int64_t v_stride_page, v_stride_token, v_stride_head;
    int64_t num_pages;
    int32_t num_q_heads, num_kv_heads, max_pages_per_seq, batch;
    float scale_log2;  // sm_scale * log2(e): logits are kept in the base-2 domain
    int32_t out_kind;
    int32_t in_f16;          // q, K and V are fp16 (else bf16)
    int32_t tile_shift;      // log2(page_size / 16): the kernels walk the cache in 16-token tiles, 1 << tile_shift per page
    int32_t fused;
    int32_t grid_exit;  // capacity plans: the unit count is read from header->n_units, surplus blocks leave at once
    int32_t n_units;    // otherwise: the unit count
    int32_t n_work_blocks;  // fused plans: blocks at or beyond this index merge records instead of attending
    int32_t ticket_stride;  // elements between the two ticket arrays
    int32_t hint_first_pages;  // tensor-core kernel: pages of a block's first unit asked into L2 ahead of the dependency wait
    // A plan that runs two partial kernels (shared prefix on tcgen05 + everything else) launches them as a
    // pair whose members do not depend on each other: the first lets its successor go as soon as its own
    // dependency wait is over (early_trigger), the second starts without waiting and waits before it exits
    // (late_wait), so that what follows the pair still sees both complete.
    int32_t early_trigger;
    int32_t late_wait;
    // Bounded waits of the tensor-core kernel and of the merge blocks give up after this many
    // clock cycles (kWaitLimitCycles in every ordinary launch).
    long long wait_limit;
    // Test hook (decode_attn_debug_expire_wait): the producer withholds its loads, so that the
    // waits of the launch run out and its give-up path is exercised with nothing at fault.
    int32_t debug_drop_loads;
#ifdef DA_TRACE
    unsigned long long* trace;  // debug builds: 32 stamps per block, or NULL
#endif
};

// Optional per-block timeline (builds with -DDA_TRACE only): stamps at a few
// points of each block.  Compiled out of the product library.
#ifdef DA_TRACE
#define DA_TRACE_STAMP(uid, slot)                                                \
    do {                                                                         \
        if (p.trace != nullptr) {                                                \
            unsigned long long t__;                                              \
            asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t__));              \
            p.trace[(long long)(uid) * 32 + (slot)] = t__;                       \
        }                                                                        \
    } while (0)
#define DA_TRACE_CLOCK(uid, slot)                                                                         \
    do {                                                                                                  \
        if (p.trace != nullptr) p.trace[(long long)(uid) * 32 + (slot)] = (unsigned long long)clock64();  \
    } while (0)
#else
#define DA_TRACE_STAMP(uid, slot) ((void)0)
#define DA_TRACE_CLOCK(uid, slot) ((void)0)
#endif


constexpr float kLn2 = 0.6931471805599453f;
constexpr float kLog2e = 1.4426950408889634f;

__device__ __forceinline__ float ex2f(float x)
{
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}

__device__ __forceinline__ void record_status(int32_t* status, int code)
{
    // codes are negative; keep the most negative (worst) one
    atomicMin(status, code);
}

__device__ __forceinline__ decode_attn_unit_t load_unit(const decode_attn_unit_t* units, int idx)
{
    const int4* p = reinterpret_cast<const int4*>(units + idx);
    int4 a = __ldg(p), b = __ldg(p + 1);
    decode_attn_unit_t u;
    u.seq = a.x; u.kv_head = a.y; u.tok_begin = a.z; u.tok_end = a.w;
    u.slot = b.x; u.seq_len = b.y; u.split_index = b.z; u.n_splits = b.w;
    return u;
}

// out_kind: 0 fp32, 1 bf16, 2 fp16 (round to nearest even).
__device__ __forceinline__ void store_out4(void* out, int64_t idx, float4 v, int out_kind)
{
    if (out_kind == 1) {
        __nv_bfloat162 lo = __floats2bfloat162_rn(v.x, v.y);
        __nv_bfloat162 hi = __floats2bfloat162_rn(v.z, v.w);
        uint2 w;
        w.x = *reinterpret_cast<uint32_t*>(&lo);
        w.y = *reinterpret_cast<uint32_t*>(&hi);
        *reinterpret_cast<uint2*>(reinterpret_cast<__nv_bfloat16*>(out) + idx) = w;
    } else if (out_kind == 2) {
        __half2 lo = __floats2half2_rn(v.x, v.y);
        __half2 hi = __floats2half2_rn(v.z, v.w);
        uint2 w;
        w.x = *reinterpret_cast<uint32_t*>(&lo);
        w.y = *reinterpret_cast<uint32_t*>(&hi);
        *reinterpret_cast<uint2*>(reinterpret_cast<__half*>(out) + idx) = w;
    } else {
        *reinterpret_cast<float4*>(reinterpret_cast<float*>(out) + idx) = v;
    }
}

// ---------------------------------------------------------------- programmatic dependent launch
//
// Kernels of this library are launched with a programmatic dependency on the
// kernel before them in the stream: a kernel lets its successor start being
// scheduled early (the partial kernel once every block is past its main loop,
// the combine kernel at once), and the successor waits (pdl_wait_primary) for
// its predecessor to finish and flush before it reads anything that
// predecessor may have written.  Both are no-ops without such a dependency.
__device__ __forceinline__ void pdl_launch_dependents() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }
__device__ __forceinline__ void pdl_wait_primary() { asm volatile("griddepcontrol.wait;" ::: "memory"); }

// Barrier over `nthreads` threads of the block (a multiple of 32) on hardware barrier `id`;
// id 0 with the whole block is __syncthreads().
__device__ __forceinline__ void block_sync(int id, int nthreads)
{
    asm volatile("bar.sync %0, %1;" ::"r"(id), "r"(nthreads) : "memory");
}

// The same barrier carrying a vote: true for every thread if `pred` was true for any.
__device__ __forceinline__ bool block_sync_or(int id, int nthreads, bool pred)
{
    uint32_t r;
    asm volatile(
        "{\n\t.reg .pred p, q;\n\t"
        "setp.ne.u32 p, %3, 0;\n\t"
        "bar.red.or.pred q, %1, %2, p;\n\t"
        "selp.u32 %0, 1, 0, q;\n\t}"
        : "=r"(r)
        : "r"(id), "r"(nthreads), "r"((uint32_t)pred)
        : "memory");
    return r != 0;
}

// ---------------------------------------------------------------- partial records
//
// The partial result of one (split, KV head) is one contiguous record:
// G x D floats of unnormalised output followed by (running max in the log2
// domain, sum of exponentials) for each of the G heads, padded to 16 bytes so
// a record can be moved with one bulk copy.  Record r = slot * Hkv + kv_head.
__host__ __device__ constexpr int rec_floats(int G, int D) { return (G * D + 2 * G + 3) / 4 * 4; }

// ---------------------------------------------------------------- mbarrier / bulk copy

__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count)
{
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count));
}

// A location that holds a live barrier must be invalidated before it is initialised again.
__device__ __forceinline__ void mbar_inval(uint32_t bar)
{
    asm volatile("mbarrier.inval.shared::cta.b64 [%0];" ::"r"(bar) : "memory");
}

__device__ __forceinline__ void mbar_init_fence()
{
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
}

__device__ __forceinline__ void mbar_arrive(uint32_t bar)
{
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}

__device__ __forceinline__ void mbar_arrive_expect_tx(uint32_t bar, uint32_t bytes)
{
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}

__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity)
{
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok)
        : "r"(bar), "r"(parity)
        : "memory");
    return ok != 0;
}

// One probe, never suspends.
__device__ __forceinline__ bool mbar_test_wait(uint32_t bar, uint32_t parity)
{
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.test_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok)
        : "r"(bar), "r"(parity)
        : "memory");
    return ok != 0;
}

constexpr long long kWaitLimitCycles = 2000000000LL;  // about one second

// Bounded wait: false if the phase did not complete within `limit` clock cycles.
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, long long limit = kWaitLimitCycles)
{
    if (mbar_try_wait(bar, parity)) return true;
    const long long t0 = clock64();
    while (!mbar_try_wait(bar, parity)) {
        if (clock64() - t0 > limit) return false;
    }
    return true;
}

// ---------------------------------------------------------------- LSE merge of one slice
//
// Merge of the records of one (sequence, KV head) for a slice of 32 output
// columns (a column is four consecutive output dims of one query head), by
// 128 threads = four chains x 32 columns: chain k of a column sums the splits
// with index k (mod 4) in ascending order, the four chains are added as
// ((c0 + c1) + c2) + c3.  All of a thread's loads (its column of up to
// kCombineBatch records and their (max, sum) pairs) are in flight before
// anything is used, so up to 4 * kCombineBatch splits cost one round trip to
// L2.  The combine kernel and the merge blocks of a fused launch both call
// this, so both paths give the same bits.  sm: 4 * 32 * 6 floats of shared
// memory; the 128 threads synchronise on hardware barrier `bar_id`.
constexpr int kCombineThreads = 128;
constexpr int kCombineBatch = 12;
constexpr int kCombineSmemFloats = 4 * 32 * 6;

// ONE_PASS: the caller knows S <= 4 * BATCH, so the code for further rounds is left out.
template <int D, int BATCH = kCombineBatch, bool ONE_PASS = false>
__device__ __forceinline__ void combine_slice(const KernelParams& p, int b, int g, int slice, int G, int slot_base,
                                              int S, int tid, float* sm, int bar_id)
{
    constexpr int kCombineBatch = BATCH;    // loads in flight per thread; does not change the order of the sums
    constexpr int D4 = D / 4;
    float* const sm_m = sm;                                    // [4][32]
    float* const sm_l = sm + 128;                              // [4][32]
    float4* const sm_acc = reinterpret_cast<float4*>(sm + 256);   // [4][32]
    const int q = tid >> 5, lane = tid & 31;
    const int col = slice * 32 + lane;
    const bool live = col < G * D4;
    const int h = live ? col / D4 : 0;
    const int RF = rec_floats(G, D);
    const float* const recs = p.ws + ((int64_t)slot_base * p.num_kv_heads + g) * RF;
    const int64_t rec_stride = (int64_t)p.num_kv_heads * RF;
    const float4* const colp = reinterpret_cast<const float4*>(recs) + (live ? col : 0);
    const float2* const mlp = reinterpret_cast<const float2*>(recs + G * D) + h;

    float2 ml[kCombineBatch];
    float4 v[kCombineBatch];
#pragma unroll
    for (int t = 0; t < kCombineBatch; ++t) {
        const int j = q + 4 * t;
        ml[t] = make_float2(-INFINITY, 0.f);
        v[t] = make_float4(0.f, 0.f, 0.f, 0.f);
        if (j < S) {
            ml[t] = __ldcg(mlp + j * (rec_stride / 2));
            v[t] = __ldcg(colp + j * (rec_stride / 4));
        }
    }
    float mloc = -INFINITY;
#pragma unroll
    for (int t = 0; t < kCombineBatch; ++t) mloc = fmaxf(mloc, ml[t].x);
    if (!ONE_PASS)
        for (int j = q + 4 * kCombineBatch; j < S; j += 4) mloc = fmaxf(mloc, __ldcg(mlp + j * (rec_stride / 2)).x);
    sm_m[q * 32 + lane] = mloc;
    if (tid == 0) DA_TRACE_STAMP(p.n_work_blocks + blockIdx.x, 3);
    block_sync(bar_id, kCombineThreads);
    if (tid == 0) DA_TRACE_STAMP(p.n_work_blocks + blockIdx.x, 4);
    const float M = fmaxf(fmaxf(sm_m[lane], sm_m[32 + lane]), fmaxf(sm_m[64 + lane], sm_m[96 + lane]));

    float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
    float lch = 0.f;
    for (int t0 = 0; q + 4 * t0 < S && (!ONE_PASS || t0 == 0); t0 += kCombineBatch) {
        if (!ONE_PASS && t0 > 0) {
#pragma unroll
            for (int t = 0; t < kCombineBatch; ++t) {
                const int j = q + 4 * (t0 + t);
                ml[t] = make_float2(-INFINITY, 0.f);
                v[t] = make_float4(0.f, 0.f, 0.f, 0.f);
                if (j < S) {
                    ml[t] = __ldcg(mlp + j * (rec_stride / 2));
                    v[t] = __ldcg(colp + j * (rec_stride / 4));
                }
            }
        }
#pragma unroll
        for (int t = 0; t < kCombineBatch; ++t) {
            if (q + 4 * (t0 + t) < S) {
                const float w = (M == -INFINITY) ? 0.f : ex2f(ml[t].x - M);   // empty split: m = -inf, w = 0
                acc.x = fmaf(w, v[t].x, acc.x);
                acc.y = fmaf(w, v[t].y, acc.y);
                acc.z = fmaf(w, v[t].z, acc.z);
                acc.w = fmaf(w, v[t].w, acc.w);
                lch = fmaf(w, ml[t].y, lch);
            }
        }
    }
    sm_acc[q * 32 + lane] = acc;
    sm_l[q * 32 + lane] = lch;
    if (tid == 0) DA_TRACE_STAMP(p.n_work_blocks + blockIdx.x, 5);
    block_sync(bar_id, kCombineThreads);
    if (q == 0 && live) {
        const int d4 = col % D4;
        const float ls = ((sm_l[lane] + sm_l[32 + lane]) + sm_l[64 + lane]) + sm_l[96 + lane];
        float4 o = make_float4(0.f, 0.f, 0.f, 0.f);
        if (M != -INFINITY && ls > 0.f) {
            const float inv = 1.0f / ls;
            const float4 a0 = sm_acc[lane], a1 = sm_acc[32 + lane], a2 = sm_acc[64 + lane], a3 = sm_acc[96 + lane];
            o.x = (((a0.x + a1.x) + a2.x) + a3.x) * inv;
            o.y = (((a0.y + a1.y) + a2.y) + a3.y) * inv;
            o.z = (((a0.z + a1.z) + a2.z) + a3.z) * inv;
            o.w = (((a0.w + a1.w) + a2.w) + a3.w) * inv;
        }
        store_out4(p.out, ((int64_t)b * p.num_q_heads + g * G + h) * D + d4 * 4, o, p.out_kind);
        if (p.lse != nullptr && d4 == 0)
            p.lse[(int64_t)b * p.num_q_heads + g * G + h] = (M != -INFINITY && ls > 0.f) ? (M + log2f(ls)) * kLn2 : -INFINITY;
    }
    block_sync(bar_id, kCombineThreads);                       // the scratch may be reused by the next slice
}

// The same merge for sequences of at most MAXS (<= 8) splits, one thread per output column and no
// shared memory: the thread keeps the four chains in registers and adds them in the same order,
// so the bits equal combine_slice's.  All of the thread's loads are in flight at once.
template <int D, int MAXS>
__device__ __forceinline__ void combine_column(const KernelParams& p, int b, int g, int col, int G, int slot_base, int S)
{
    constexpr int D4 = D / 4;
    const int h = col / D4, d4 = col % D4;
    const int RF = rec_floats(G, D);
    const float* const recs = p.ws + ((int64_t)slot_base * p.num_kv_heads + g) * RF;
    const int64_t rec_stride = (int64_t)p.num_kv_heads * RF;
    const float4* const colp = reinterpret_cast<const float4*>(recs) + col;
    const float2* const mlp = reinterpret_cast<const float2*>(recs + G * D) + h;
    float2 ml[MAXS];
    float4 v[MAXS];
#pragma unroll
    for (int j = 0; j < MAXS; ++j) {
        ml[j] = make_float2(-INFINITY, 0.f);
        v[j] = make_float4(0.f, 0.f, 0.f, 0.f);
        if (j < S) {
            ml[j] = __ldcg(mlp + j * (rec_stride / 2));
            v[j] = __ldcg(colp + j * (rec_stride / 4));
        }
    }
    float M = -INFINITY;
#pragma unroll
    for (int j = 0; j < MAXS; ++j) M = fmaxf(M, ml[j].x);
    float4 acc[4];
    float lch[4];
#pragma unroll
    for (int k = 0; k < 4; ++k) {
        acc[k] = make_float4(0.f, 0.f, 0.f, 0.f);
        lch[k] = 0.f;
    }
#pragma unroll
    for (int j = 0; j < MAXS; ++j) {
        if (j < S) {
            const float w = (M == -INFINITY) ? 0.f : ex2f(ml[j].x - M);   // empty split: m = -inf, w = 0
            acc[j & 3].x = fmaf(w, v[j].x, acc[j & 3].x);
            acc[j & 3].y = fmaf(w, v[j].y, acc[j & 3].y);
            acc[j & 3].z = fmaf(w, v[j].z, acc[j & 3].z);
            acc[j & 3].w = fmaf(w, v[j].w, acc[j & 3].w);
            lch[j & 3] = fmaf(w, ml[j].y, lch[j & 3]);
        }
    }
    const float ls = ((lch[0] + lch[1]) + lch[2]) + lch[3];
    float4 o = make_float4(0.f, 0.f, 0.f, 0.f);
    if (M != -INFINITY && ls > 0.f) {
        const float inv = 1.0f / ls;
        o.x = (((acc[0].x + acc[1].x) + acc[2].x) + acc[3].x) * inv;
        o.y = (((acc[0].y + acc[1].y) + acc[2].y) + acc[3].y) * inv;
        o.z = (((acc[0].z + acc[1].z) + acc[2].z) + acc[3].z) * inv;
        o.w = (((acc[0].w + acc[1].w) + acc[2].w) + acc[3].w) * inv;
    }
    store_out4(p.out, ((int64_t)b * p.num_q_heads + g * G + h) * D + d4 * 4, o, p.out_kind);
    if (p.lse != nullptr && d4 == 0)
        p.lse[(int64_t)b * p.num_q_heads + g * G + h] = (M != -INFINITY && ls > 0.f) ? (M + log2f(ls)) * kLn2 : -INFINITY;
}

__host__ __device__ inline int combine_slices(int D, int G) { return (G * (D / 4) + 31) / 32; }

__device__ __forceinline__ int32_t ld_acquire(const int32_t* ptr)
{
    int32_t v;
    asm volatile("ld.acquire.gpu.global.s32 %0, [%1];" : "=r"(v) : "l"(ptr) : "memory");
    return v;
}

// ---------------------------------------------------------------- merge blocks of a fused launch
//
// With fuse_combine the launch carries extra blocks behind the attending ones
// (blockIdx.x >= n_work_blocks).  They are dispatched after every attending
// block has been dispatched, take the merge tasks (sequence, KV head, slice)
// round-robin, and for each task poll the group's arrival counter - every
// attending block adds one after publishing a record - until all the group's
// records are in, then merge the slice exactly as the combine kernel would.
// The poll is bounded (about a second); giving up records DA_ERR_TIMEOUT.
// The block that merges a group's last slice resets the group's counters, so
// the plan can be launched again (or replayed from a graph) as it is.
template <int D>
__device__ __forceinline__ void fused_merge_blocks(const KernelParams& p, int G, int nthreads, float* sm, int* sm_flag)
{
    const int tid = threadIdx.x;
    const int n_slices = combine_slices(D, G);
    const int batch = p.grid_exit ? p.header->batch : p.batch;
    const int n_tasks = batch * p.num_kv_heads * n_slices;
    const int n_merge_blocks = gridDim.x - p.n_work_blocks;
    for (int t = blockIdx.x - p.n_work_blocks; t < n_tasks; t += n_merge_blocks) {
        const int slice = t % n_slices, bg = t / n_slices;
        const int b = bg / p.num_kv_heads, g = bg % p.num_kv_heads;
        const SeqInfo si = p.seq_info[b];
        if (si.slot_base < 0) continue;                        // a single split: written directly
        if (tid == 0) {
            const int32_t* arrivals = p.tickets + bg;
            const long long t0 = clock64();
            int ok = 1;
            while (ld_acquire(arrivals) < si.n_splits) {
                // give up after the limit, or at once when an attending block already gave up
                // on a wait of its own (it will not publish the rest of its records)
                if (clock64() - t0 > p.wait_limit || ld_acquire(p.status) <= DA_ERR_TIMEOUT) {
                    ok = 0;
                    break;
                }
                __nanosleep(100);
            }
            if (!ok) record_status(p.status, DA_ERR_TIMEOUT);
            *sm_flag = ok;
        }
        block_sync(0, nthreads);
        const int ok = *sm_flag;
        if (ok && tid < kCombineThreads) combine_slice<D>(p, b, g, slice, G, si.slot_base, si.n_splits, tid, sm, 2);
        block_sync(0, nthreads);
        if (tid == 0) {
            // count this slice; whoever completes the group puts its counters back to zero
            int32_t* done = p.tickets + p.ticket_stride + bg;
            if (atomicAdd(done, 1) == n_slices - 1) {
                *done = 0;
                p.tickets[bg] = 0;
            }
        }
    }
}

// ---------------------------------------------------------------- end of a unit
//
// The block's R partial states (one per warp or row group) sit in shared
// memory: src_o [R][COLS][D] unnormalised accumulators, src_m / src_l
// [R][COLS] running maxima (log2 domain, -inf if nothing was attended) and
// sums.  With DUP, columns h and h + 4 hold the high and low parts of the
// same head and are added.  The calling threads (`nthreads`, ids
// 0..nthreads-1) call this after a barrier that made the sources visible and
// synchronise on hardware barrier `bar_id`.  The states are merged in the
// fixed order r = 0..R-1 and the result goes straight to `out` (single
// split) or to the unit's record; with a fused plan the block then publishes
// the record: a device-wide fence and one more arrival on the counter of its
// (sequence, KV head), which the merge blocks of the launch poll.
template <int D, int R, int COLS, bool DUP>
__device__ __forceinline__ void block_finish(const KernelParams& p, const decode_attn_unit_t& u, int G,
                                             const float* src_o, const float* src_m, const float* src_l, int tid,
                                             int nthreads, int bar_id, int head_first = 0, int head_count = -1,
                                             bool publish = true)
{
    // heads [head_first, head_first + head_count) of the group, held in source columns 0 .. head_count - 1
    if (head_count < 0) head_count = G;
    constexpr int D4 = D / 4;
    constexpr int kUnroll = R <= 4 ? R : 1;     // many row groups: keep the loop rolled, registers matter more
    const int Hq = p.num_q_heads;
    const int h0 = u.kv_head * G;
    const int RF = rec_floats(G, D);
    float* const rec = (u.slot >= 0) ? p.ws + ((int64_t)u.slot * p.num_kv_heads + u.kv_head) * RF : nullptr;
    if (tid == 0) DA_TRACE_CLOCK(blockIdx.x + 4096, 0);
    for (int task = tid; task < head_count * D4; task += nthreads) {
        const int h = task / D4, d4 = task % D4;          // source column h is head head_first + h
        float M = -INFINITY;
#pragma unroll kUnroll
        for (int r = 0; r < R; ++r) M = fmaxf(M, src_m[r * COLS + h]);
        if (tid == 0) DA_TRACE_CLOCK(blockIdx.x + 4096, 1);
        float4 o = make_float4(0.f, 0.f, 0.f, 0.f);
        float ls = 0.f;
        if (M != -INFINITY) {
#pragma unroll kUnroll
            for (int r = 0; r < R; ++r) {
                const float w = ex2f(src_m[r * COLS + h] - M);          // a source that saw nothing: w = 0
                float4 v = reinterpret_cast<const float4*>(src_o)[(r * COLS + h) * D4 + d4];
                if (DUP) {
                    const float4 v2 = reinterpret_cast<const float4*>(src_o)[(r * COLS + h + 4) * D4 + d4];
                    v.x += v2.x; v.y += v2.y; v.z += v2.z; v.w += v2.w;
                }
                o.x = fmaf(w, v.x, o.x);
                o.y = fmaf(w, v.y, o.y);
                o.z = fmaf(w, v.z, o.z);
                o.w = fmaf(w, v.w, o.w);
                ls = fmaf(w, src_l[r * COLS + h], ls);
            }
        }
        if (tid == 0) DA_TRACE_CLOCK(blockIdx.x + 4096, 2);
        if (rec == nullptr) {
            if (ls > 0.f) {
                const float inv = 1.0f / ls;
                o.x *= inv; o.y *= inv; o.z *= inv; o.w *= inv;
            } else {
                o = make_float4(0.f, 0.f, 0.f, 0.f);
            }
            store_out4(p.out, ((int64_t)u.seq * Hq + h0 + head_first + h) * D + d4 * 4, o, p.out_kind);
            if (p.lse != nullptr && d4 == 0)
                p.lse[(int64_t)u.seq * Hq + h0 + head_first + h] = (ls > 0.f) ? (M + log2f(ls)) * kLn2 : -INFINITY;
        } else {
            __stcg(reinterpret_cast<float4*>(rec) + head_first * D4 + task, o);
            if (d4 == 0) __stcg(reinterpret_cast<float2*>(rec + G * D) + head_first + h, make_float2(M, ls));
        }
    }
    if (tid == 0) DA_TRACE_CLOCK(blockIdx.x + 4096, 3);
    if (rec == nullptr || !p.fused || !publish) return;
    // The barrier orders every thread's record stores before thread 0's fence, which publishes
    // them device-wide ahead of the arrival.
    block_sync(bar_id, nthreads);
    if (tid == 0) {
        __threadfence();
        atomicAdd(p.tickets + (int64_t)u.seq * p.num_kv_heads + u.kv_head, 1);
    }
}

// Own-layer KV write of one (sequence, KV head): the new K and V rows go to position seq_len - 1 of the paged
// pools (Invariant 1: every valid row writes its K/V whether or not it then attends).  One warp; the unit must
// be the one that holds the sequence's last token.  Page ids are range-checked like everywhere else.
template <int D>
__device__ __forceinline__ void append_new_row(const KernelParams& p, int seq, int g, int seq_len, int lane)
{
    if (p.new_k == nullptr || seq_len <= 0) return;
    const int t = seq_len - 1;
    const int page_shift = p.tile_shift + 4;
    if ((t >> page_shift) >= p.max_pages_per_seq) {
        if (lane == 0) record_status(p.status, DA_ERR_STALE_PLAN);
        return;
    }
    const int page = __ldg(p.block_table + (int64_t)seq * p.max_pages_per_seq + (t >> page_shift));
    if ((unsigned)page >= (unsigned)p.num_pages) {
        if (lane == 0) record_status(p.status, DA_ERR_BAD_PAGE);
        return;
    }
    const int slot = t & ((1 << page_shift) - 1);
    constexpr int CH = D / 8;                               // 16-byte chunks of a row
    const uint4* sk = reinterpret_cast<const uint4*>(p.new_k + ((int64_t)seq * p.num_kv_heads + g) * D);
    const uint4* sv = reinterpret_cast<const uint4*>(p.new_v + ((int64_t)seq * p.num_kv_heads + g) * D);
    uint4* dk = reinterpret_cast<uint4*>(const_cast<__nv_bfloat16*>(p.k) + (int64_t)page * p.k_stride_page +
                                         (int64_t)slot * p.k_stride_token + (int64_t)g * p.k_stride_head);
    uint4* dv = reinterpret_cast<uint4*>(const_cast<__nv_bfloat16*>(p.v) + (int64_t)page * p.v_stride_page +
                                         (int64_t)slot * p.v_stride_token + (int64_t)g * p.v_stride_head);
    if (lane < CH) dk[lane] = __ldg(sk + lane);
    else if (lane < 2 * CH) dv[lane - CH] = __ldg(sv + lane - CH);
}

// The result of a unit that read nothing: zeros (and lse = -inf) for a sequence with a single split,
// an empty record (maximum -inf, sum 0) otherwise; published like any other record in fused plans.
template <int D>
__device__ __forceinline__ void block_finish_empty(const KernelParams& p, const decode_attn_unit_t& u, int G, int tid,
                                                   int nthreads)
{
    constexpr int D4 = D / 4;
    const int Hq = p.num_q_heads;
    const int h0 = u.kv_head * G;
    const int RF = rec_floats(G, D);
    float* const rec = (u.slot >= 0) ? p.ws + ((int64_t)u.slot * p.num_kv_heads + u.kv_head) * RF : nullptr;
    const float4 zero = make_float4(0.f, 0.f, 0.f, 0.f);
    for (int task = tid; task < G * D4; task += nthreads) {
        const int h = task / D4, d4 = task % D4;
        if (rec == nullptr) {
            store_out4(p.out, ((int64_t)u.seq * Hq + h0 + h) * D + d4 * 4, zero, p.out_kind);
            if (p.lse != nullptr && d4 == 0) p.lse[(int64_t)u.seq * Hq + h0 + h] = -INFINITY;
        } else {
            __stcg(reinterpret_cast<float4*>(rec) + task, zero);
            if (d4 == 0) __stcg(reinterpret_cast<float2*>(rec + G * D) + h, make_float2(-INFINITY, 0.f));
        }
    }
    if (rec == nullptr || !p.fused) return;
    // fused plans: the record is published; the barrier orders every thread's stores before
    // thread 0's fence (the named barrier the ordinary finish uses, by the same threads; a single
    // warp synchronises by itself)
    if (nthreads == 32)
        __syncwarp();
    else
        block_sync(1, nthreads);
    if (tid == 0) {
        __threadfence();
        atomicAdd(p.tickets + (int64_t)u.seq * p.num_kv_heads + u.kv_head, 1);
    }
}

}  // namespace da
