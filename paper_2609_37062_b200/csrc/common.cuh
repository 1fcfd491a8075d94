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
    int32_t slot_base;  // -1: single split
    int32_t n_splits;
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
    float* ws_o;   // [n_slots][Hq][D]   unnormalised partial outputs
    float* ws_ml;  // [n_slots][Hq][2]   running max (log2 domain) and sum of exponentials
    const DevHeader* header;
    const decode_attn_unit_t* units;
    const SeqInfo* seq_info;
    int32_t* tickets;  // [batch][Hkv], zero between launches
    int32_t* status;   // worst da_status_t seen by any block (0 = ok)
    int64_t k_stride_page, k_stride_token, k_stride_head;
    int64_t v_stride_page, v_stride_token, v_stride_head;
    int64_t num_pages;
    int32_t num_q_heads, num_kv_heads, max_pages_per_seq;
    float scale_log2;  // sm_scale * log2(e): logits are kept in the base-2 domain
    int32_t out_bf16;
    int32_t fused;
};

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

template <typename T>
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

// LSE merge of the splits of one (sequence, KV head): all G query heads of
// the group, ascending split order, by `nthreads` threads of one block.  Used
// by the combine kernel and by the last block to finish in a fused launch, so
// both give the same bits.  Partials are read around L1 (they were written by
// other SMs in the same launch when fused).
template <int D>
__device__ __forceinline__ void merge_group(const KernelParams& p, int b, int g, int G, int slot_base, int S,
                                            int tid, int nthreads)
{
    constexpr int D4 = D / 4;
    const int Hq = p.num_q_heads;
    for (int task = tid; task < G * D4; task += nthreads) {
        const int h = g * G + task / D4;
        const int d4 = task % D4;
        const float2* ml = reinterpret_cast<const float2*>(p.ws_ml) + ((int64_t)slot_base * Hq + h);
        const float4* po = reinterpret_cast<const float4*>(p.ws_o) + ((int64_t)slot_base * Hq + h) * D4 + d4;
        float M = -INFINITY;
        for (int i = 0; i < S; ++i) M = fmaxf(M, __ldcg(ml + (int64_t)i * Hq).x);
        float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
        float lsum = 0.f;
        if (M != -INFINITY) {
#pragma unroll 8
            for (int i = 0; i < S; ++i) {
                const float2 mli = __ldcg(ml + (int64_t)i * Hq);
                const float4 o = __ldcg(po + (int64_t)i * Hq * D4);
                const float w = ex2f(mli.x - M);  // an empty split has m = -inf: w = 0 exactly
                lsum = fmaf(w, mli.y, lsum);
                acc.x = fmaf(w, o.x, acc.x);
                acc.y = fmaf(w, o.y, acc.y);
                acc.z = fmaf(w, o.z, acc.z);
                acc.w = fmaf(w, o.w, acc.w);
            }
            const float inv = 1.0f / lsum;
            acc.x *= inv; acc.y *= inv; acc.z *= inv; acc.w *= inv;
        }
        store_out4<void>(p.out, ((int64_t)b * Hq + h) * D + d4 * 4, acc, p.out_bf16);
        if (p.lse != nullptr && d4 == 0)
            p.lse[(int64_t)b * Hq + h] = (M != -INFINITY) ? (M + log2f(lsum)) * kLn2 : -INFINITY;
    }
}

// End of a unit.  sm_o [G][D] holds the block's unnormalised accumulator,
// sm_m [G] its running max (log2 domain, -inf if nothing was attended) and
// sm_l [G] its sum of exponentials; all threads of the block call this after
// a __syncthreads() that made those visible.
template <int D>
__device__ __forceinline__ void finish_unit(const KernelParams& p, const decode_attn_unit_t& u, int G,
                                            const float* sm_o, const float* sm_m, const float* sm_l,
                                            int* sm_ticket, int tid, int nthreads)
{
    constexpr int D4 = D / 4;
    const int Hq = p.num_q_heads;
    const int h0 = u.kv_head * G;
    if (u.slot < 0) {
        for (int task = tid; task < G * D4; task += nthreads) {
            const int h = task / D4, d4 = task % D4;
            const float l = sm_l[h];
            float4 o = reinterpret_cast<const float4*>(sm_o)[h * D4 + d4];
            if (l > 0.f) {
                const float inv = 1.0f / l;
                o.x *= inv; o.y *= inv; o.z *= inv; o.w *= inv;
            } else {
                o = make_float4(0.f, 0.f, 0.f, 0.f);
            }
            store_out4<void>(p.out, ((int64_t)u.seq * Hq + h0 + h) * D + d4 * 4, o, p.out_bf16);
        }
        if (p.lse != nullptr && tid < G) {
            const float l = sm_l[tid];
            p.lse[(int64_t)u.seq * Hq + h0 + tid] = (l > 0.f) ? (sm_m[tid] + log2f(l)) * kLn2 : -INFINITY;
        }
        return;
    }
    for (int task = tid; task < G * D4; task += nthreads) {
        const int h = task / D4, d4 = task % D4;
        reinterpret_cast<float4*>(p.ws_o)[((int64_t)u.slot * Hq + h0 + h) * D4 + d4] =
            reinterpret_cast<const float4*>(sm_o)[h * D4 + d4];
    }
    if (tid < G)
        reinterpret_cast<float2*>(p.ws_ml)[(int64_t)u.slot * Hq + h0 + tid] = make_float2(sm_m[tid], sm_l[tid]);
    if (!p.fused) return;
    // Ticket: nobody waits.  The block that draws the last ticket of its
    // (sequence, KV head) sees every other block's partials (fence before
    // the ticket, fence after) and merges them in ascending split order.
    __threadfence();
    __syncthreads();
    int32_t* ticket = p.tickets + (int64_t)u.seq * p.num_kv_heads + u.kv_head;
    if (tid == 0) *sm_ticket = atomicAdd(ticket, 1);
    __syncthreads();
    if (*sm_ticket != u.n_splits - 1) return;
    __threadfence();
    merge_group<D>(p, u.seq, u.kv_head, G, u.slot - u.split_index, u.n_splits, tid, nthreads);
    if (tid == 0) *ticket = 0;  // ready for the next launch
}

}  // namespace da
