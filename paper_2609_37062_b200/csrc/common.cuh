// Device-side pieces shared by the partial kernels and the combine kernel:
// the launch parameter block, the plan's device header, the unit epilogue
// (partial write, ticket, in-kernel merge) and the LSE merge itself.
#pragma once

#include <cuda_bf16.h>
#include <cuda_runtime.h>

#include <cstdint>

#include "decode_attn.h"

namespace da {

// First words of the plan's device buffer, refreshed by every upload.
struct DevHeader {
    int32_t n_units;
    int32_t batch;
    int32_t pad[2];
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
    void* out;
    float* lse;
    float* ws;     // [n_slots][Hkv] partial records, see rec_floats()
    const DevHeader* header;
    const decode_attn_unit_t* units;
    const SeqInfo* seq_info;
    const int32_t* block_begin;  // [grid + 1]: block b walks units block_begin[b] .. block_begin[b+1]; NULL: unit b
    int32_t* tickets;  // [batch][Hkv], zero between launches
    int32_t* status;   // worst da_status_t seen by any block (0 = ok)
    int64_t k_stride_page, k_stride_token, k_stride_head;
    int64_t v_stride_page, v_stride_token, v_stride_head;
    int64_t num_pages;
    int32_t num_q_heads, num_kv_heads, max_pages_per_seq;
    float scale_log2;  // sm_scale * log2(e): logits are kept in the base-2 domain
    int32_t out_bf16;
    int32_t fused;
    int32_t grid_exit;  // capacity plans: the unit count is read from header->n_units, surplus blocks leave at once
    int32_t n_units;    // otherwise: the unit count
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

__device__ __forceinline__ void store_out4(void* out, int64_t idx, float4 v, int out_bf16)
{
    if (out_bf16) {
        __nv_bfloat162 lo = __floats2bfloat162_rn(v.x, v.y);
        __nv_bfloat162 hi = __floats2bfloat162_rn(v.z, v.w);
        uint2 w;
        w.x = *reinterpret_cast<uint32_t*>(&lo);
        w.y = *reinterpret_cast<uint32_t*>(&hi);
        *reinterpret_cast<uint2*>(reinterpret_cast<__nv_bfloat16*>(out) + idx) = w;
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

// ---------------------------------------------------------------- partial records
//
// The partial result of one (split, KV head) is one contiguous record:
// G x D floats of unnormalised output followed by (running max in the log2
// domain, sum of exponentials) for each of the G heads, padded to 16 bytes so
// a record can be moved with one bulk copy.  Record r = slot * Hkv + kv_head.
__host__ __device__ constexpr int rec_floats(int G, int D) { return (G * D + 2 * G + 3) / 4 * 4; }

// Shared memory merge_group needs to stage `cap` records at a time.
__host__ __device__ constexpr int merge_stage_bytes(int G, int D, int cap)
{
    return cap * rec_floats(G, D) * 4 + cap * G * 4 + 64;
}

// ---------------------------------------------------------------- mbarrier / bulk copy

__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count)
{
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count));
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

constexpr long long kWaitLimitCycles = 2000000000LL;  // about one second

// Bounded wait: false if the phase did not complete within the limit.
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity)
{
    if (mbar_try_wait(bar, parity)) return true;
    const long long t0 = clock64();
    while (!mbar_try_wait(bar, parity)) {
        if (clock64() - t0 > kWaitLimitCycles) return false;
    }
    return true;
}

// 1-D bulk copy global -> shared, completion counted in bytes on `bar`.
// Addresses 16-byte aligned, size a multiple of 16.
__device__ __forceinline__ void bulk_copy_g2s(uint32_t dst, const void* src, uint32_t bytes, uint32_t bar)
{
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                 ::"r"(dst), "l"(src), "r"(bytes), "r"(bar)
                 : "memory");
}

// ---------------------------------------------------------------- LSE merge
//
// Merge of the splits of one (sequence, KV head): all G query heads of the
// group, ascending split order, by the `nthreads` threads of one block.  Used
// by the combine kernel and by the last block to finish in a fused launch, so
// both give the same bits: every output column is the sum of four chains,
// chain k taking the splits with index k (mod 4) in ascending order, added as
// ((c0 + c1) + c2) + c3; the sums of exponentials follow the same scheme.
// The records (written by other SMs) are pulled
// into shared memory `cap` at a time by bulk copies, one per record, issued
// by as many threads in parallel as there are records (a bulk copy costs its
// issuer about one round trip to L2); warp w reduces the running maxima of
// heads w, w + nwarps, ... by shuffles and leaves the weights e^{m_i - M} in
// shared memory.  The result does not depend on `cap` (a multiple of 4).
// The `nthreads` threads synchronise on hardware barrier `bar_id`.
// `stage`: merge_stage_bytes(G, D, cap) bytes of shared
// memory, 16-byte aligned, that no thread still reads.  `bar`: an initialised
// mbarrier (count 1) whose current phase parity is `parity` (updated).
template <int D>
__device__ __forceinline__ void merge_group(const KernelParams& p, int b, int g, int G, int slot_base, int S,
                                            int tid, int nthreads, int bar_id, uint8_t* stage, int cap, uint32_t bar,
                                            uint32_t& parity)
{
    constexpr int D4 = D / 4;
    constexpr int kMaxTasks = 2;                        // G * D4 <= 256 tasks over >= 128 threads
    const int Hq = p.num_q_heads, Hkv = p.num_kv_heads;
    const int RF = rec_floats(G, D), RF4 = RF / 4;
    const int GD4 = G * D4;
    const int lane = tid & 31, warp = tid >> 5, nwarps = nthreads >> 5;
    float* const st_rec = reinterpret_cast<float*>(stage);          // [cap][RF]
    float* const st_w = st_rec + (size_t)cap * RF;                  // [cap][G] weights
    float* const st_M = st_w + cap * G;                             // [8] maxima
    const float* const recs = p.ws + ((int64_t)slot_base * Hkv + g) * RF;
    const int64_t rec_stride = (int64_t)Hkv * RF;                   // next split of the same KV head

    float4 acc[kMaxTasks][4];                                       // four chains per column
    float lch[kMaxTasks][4];                                        // and per head (kept by every column thread)
#pragma unroll
    for (int k = 0; k < kMaxTasks; ++k)
#pragma unroll
        for (int q = 0; q < 4; ++q) {
            acc[k][q] = make_float4(0.f, 0.f, 0.f, 0.f);
            lch[k][q] = 0.f;
        }

    for (int i0 = 0; i0 < S; i0 += cap) {
        const int n = min(cap, S - i0);
        // The proxy fence orders the generic-proxy accesses made so far (this block's use of the
        // stage memory, other blocks' record stores seen through the ticket) before the copies.
        if (tid < n) asm volatile("fence.proxy.async;" ::: "memory");
        if (tid == 0) mbar_arrive_expect_tx(bar, (uint32_t)(n * RF * 4));
        for (int j = tid; j < n; j += nthreads)
            bulk_copy_g2s(smem_u32(st_rec + (size_t)j * RF), recs + (i0 + j) * rec_stride, (uint32_t)(RF * 4), bar);
        if (i0 == 0 && S > cap) {
            // several batches: the maximum of every head over ALL splits must be known before the
            // first weight, so read the maxima from global memory while the first batch flies
            for (int h = warp; h < G; h += nwarps) {
                float m = -INFINITY;
                for (int i = lane; i < S; i += 32) m = fmaxf(m, __ldcg(recs + i * rec_stride + G * D + 2 * h));
#pragma unroll
                for (int off = 16; off >= 1; off >>= 1) m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, off));
                if (lane == 0) st_M[h] = m;
            }
        }
        if (!mbar_wait(bar, parity) && tid == 0) record_status(p.status, DA_ERR_TIMEOUT);
        parity ^= 1u;
        if (S <= cap) {
            // one batch: every record is here, take the maxima from shared memory
            for (int h = warp; h < G; h += nwarps) {
                float m = -INFINITY;
                for (int j = lane; j < n; j += 32) m = fmaxf(m, st_rec[(size_t)j * RF + G * D + 2 * h]);
#pragma unroll
                for (int off = 16; off >= 1; off >>= 1) m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, off));
                if (lane == 0) st_M[h] = m;
            }
        }
        block_sync(bar_id, nthreads);
        // weights e^{m_i - M}, once per (split, head)
        for (int c = tid; c < n * G; c += nthreads) {
            const int j = c / G, h = c % G;
            const float M = st_M[h];
            st_w[c] = (M == -INFINITY) ? 0.f : ex2f(st_rec[(size_t)j * RF + G * D + 2 * h] - M);   // empty split: 0
        }
        block_sync(bar_id, nthreads);
#pragma unroll
        for (int k = 0; k < kMaxTasks; ++k) {
            const int task = tid + k * nthreads;
            if (task < GD4) {
                const int h = task / D4;
                const float4* o = reinterpret_cast<const float4*>(st_rec) + task;
                const float* wp = st_w + h;
                const float* lp = st_rec + G * D + 2 * h + 1;
                int j = 0;
                for (; j + 4 <= n; j += 4) {       // i0 and cap are multiples of 4: chain q takes j + q
#pragma unroll
                    for (int q = 0; q < 4; ++q) {
                        const float w = wp[(j + q) * G];
                        const float4 v = o[(j + q) * RF4];
                        acc[k][q].x = fmaf(w, v.x, acc[k][q].x);
                        acc[k][q].y = fmaf(w, v.y, acc[k][q].y);
                        acc[k][q].z = fmaf(w, v.z, acc[k][q].z);
                        acc[k][q].w = fmaf(w, v.w, acc[k][q].w);
                        lch[k][q] = fmaf(w, lp[(size_t)(j + q) * RF], lch[k][q]);
                    }
                }
#pragma unroll
                for (int q = 0; q < 3; ++q) {
                    if (j + q < n) {
                        const float w = wp[(j + q) * G];
                        const float4 v = o[(j + q) * RF4];
                        acc[k][q].x = fmaf(w, v.x, acc[k][q].x);
                        acc[k][q].y = fmaf(w, v.y, acc[k][q].y);
                        acc[k][q].z = fmaf(w, v.z, acc[k][q].z);
                        acc[k][q].w = fmaf(w, v.w, acc[k][q].w);
                        lch[k][q] = fmaf(w, lp[(size_t)(j + q) * RF], lch[k][q]);
                    }
                }
            }
        }
        block_sync(bar_id, nthreads);
    }
#pragma unroll
    for (int k = 0; k < kMaxTasks; ++k) {
        const int task = tid + k * nthreads;
        if (task < GD4) {
            const int h = task / D4, d4 = task % D4;
            const float M = st_M[h];
            const float ls = ((lch[k][0] + lch[k][1]) + lch[k][2]) + lch[k][3];
            float4 o = make_float4(0.f, 0.f, 0.f, 0.f);
            if (M != -INFINITY && ls > 0.f) {
                const float inv = 1.0f / ls;
                o.x = (((acc[k][0].x + acc[k][1].x) + acc[k][2].x) + acc[k][3].x) * inv;
                o.y = (((acc[k][0].y + acc[k][1].y) + acc[k][2].y) + acc[k][3].y) * inv;
                o.z = (((acc[k][0].z + acc[k][1].z) + acc[k][2].z) + acc[k][3].z) * inv;
                o.w = (((acc[k][0].w + acc[k][1].w) + acc[k][2].w) + acc[k][3].w) * inv;
            }
            store_out4(p.out, ((int64_t)b * Hq + g * G + h) * D + d4 * 4, o, p.out_bf16);
            if (p.lse != nullptr && d4 == 0)
                p.lse[(int64_t)b * Hq + g * G + h] = (M != -INFINITY && ls > 0.f) ? (M + log2f(ls)) * kLn2 : -INFINITY;
        }
    }
}

// ---------------------------------------------------------------- end of a unit
//
// The block's R partial states (one per warp or row group) sit in shared
// memory: src_o [R][COLS][D] unnormalised accumulators, src_m / src_l
// [R][COLS] running maxima (log2 domain, -inf if nothing was attended) and
// sums.  With DUP, columns h and h + 4 hold the high and low parts of the
// same head and are added.  All threads call this after a __syncthreads()
// that made the sources visible.  The states are merged in the fixed order
// r = 0..R-1 and the result goes straight to `out` (single split) or to the
// unit's record; with a fused plan the block then draws a ticket and, if it
// is the last of its (sequence, KV head), merges all records.  The calling
// threads (`nthreads`, ids 0..nthreads-1) synchronise on hardware barrier
// `bar_id`.  `stage` / `cap`: shared memory the merge may overwrite (it may
// alias the sources); cap == 0 means none is available (the block still has
// units to stream) and a fused plan must not get here.
template <int D, int R, int COLS, bool DUP>
__device__ __forceinline__ void block_finish(const KernelParams& p, const decode_attn_unit_t& u, int G,
                                             const float* src_o, const float* src_m, const float* src_l,
                                             int* sm_ticket, uint32_t merge_bar, uint32_t* merge_parity, int tid,
                                             int nthreads, int bar_id, uint8_t* stage, int cap)
{
    constexpr int D4 = D / 4;
    constexpr int kUnroll = R <= 4 ? R : 1;     // many row groups: keep the loop rolled, registers matter more
    const int Hq = p.num_q_heads;
    const int h0 = u.kv_head * G;
    const int RF = rec_floats(G, D);
    float* const rec = (u.slot >= 0) ? p.ws + ((int64_t)u.slot * p.num_kv_heads + u.kv_head) * RF : nullptr;
    for (int task = tid; task < G * D4; task += nthreads) {
        const int h = task / D4, d4 = task % D4;
        float M = -INFINITY;
#pragma unroll kUnroll
        for (int r = 0; r < R; ++r) M = fmaxf(M, src_m[r * COLS + h]);
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
        if (rec == nullptr) {
            if (ls > 0.f) {
                const float inv = 1.0f / ls;
                o.x *= inv; o.y *= inv; o.z *= inv; o.w *= inv;
            } else {
                o = make_float4(0.f, 0.f, 0.f, 0.f);
            }
            store_out4(p.out, ((int64_t)u.seq * Hq + h0 + h) * D + d4 * 4, o, p.out_bf16);
            if (p.lse != nullptr && d4 == 0)
                p.lse[(int64_t)u.seq * Hq + h0 + h] = (ls > 0.f) ? (M + log2f(ls)) * kLn2 : -INFINITY;
        } else {
            __stcg(reinterpret_cast<float4*>(rec) + task, o);
            if (d4 == 0) __stcg(reinterpret_cast<float2*>(rec + G * D) + h, make_float2(M, ls));
        }
    }
    if (rec == nullptr || !p.fused) return;
    // Ticket: nobody waits.  The block barrier orders every thread's record
    // stores before thread 0's fence, which publishes them device-wide ahead
    // of the ticket; the block that draws the last ticket of its (sequence,
    // KV head) therefore sees all the other records.
    block_sync(bar_id, nthreads);
    if (tid == 0) DA_TRACE_CLOCK(blockIdx.x, 13);
    int32_t* ticket = p.tickets + (int64_t)u.seq * p.num_kv_heads + u.kv_head;
    if (tid == 0) {
        __threadfence();
        *sm_ticket = atomicAdd(ticket, 1);
        __threadfence();
    }
    block_sync(bar_id, nthreads);
    if (tid == 0) DA_TRACE_CLOCK(blockIdx.x, 14);
    if (*sm_ticket != u.n_splits - 1) return;
    if (cap <= 0) {                              // host-side contract broken: fused plans run one unit per block
        if (tid == 0) record_status(p.status, DA_ERR_UNSUPPORTED);
        return;
    }
    uint32_t parity = *merge_parity;
    merge_group<D>(p, u.seq, u.kv_head, G, u.slot - u.split_index, u.n_splits, tid, nthreads, bar_id, stage, cap, merge_bar,
                   parity);
    *merge_parity = parity;
    if (tid == 0) DA_TRACE_CLOCK(blockIdx.x, 19);
    if (tid == 0) *ticket = 0;  // ready for the next launch
}

}  // namespace da
