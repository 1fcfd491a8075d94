// LSE combine kernel.
//
// One block per (sequence, KV head, slice of 32 output columns); a column is
// four consecutive output dims of one query head.  The 128 threads are four
// chains x 32 columns: chain k of a column sums the splits with index k
// (mod 4) in ascending order, the four chains are added as
// ((c0 + c1) + c2) + c3 - the same scheme as the in-kernel merge of a fused
// launch, so both paths give the same bits.  All of a thread's loads (its
// column of up to kCombineBatch records and their (max, sum) pairs) are put
// in flight before anything is used, so a sequence of up to 4 * kCombineBatch
// splits costs one round trip to L2.  The grid is spread over all SMs, and the
// kernel is launched with a programmatic dependency on the partial kernel:
// its blocks may already be resident, waiting at the top, while the partial
// kernel's last blocks write their records.
#pragma once

#include "common.cuh"

namespace da {

constexpr int kCombineThreads = 128;
constexpr int kCombineBatch = 12;

template <int D>
__global__ void __launch_bounds__(kCombineThreads) decode_attn_combine_kernel(const KernelParams p, int G, int n_slices)
{
    constexpr int D4 = D / 4;
    __shared__ float sm_m[4][32];
    __shared__ float sm_l[4][32];
    __shared__ float4 sm_acc[4][32];

    pdl_launch_dependents();                              // the next kernel may start its prologue
    pdl_wait_primary();                                   // the records of the launch before this one are complete
    const int slice = blockIdx.x % n_slices;
    const int bg = blockIdx.x / n_slices;
    const int b = bg / p.num_kv_heads, g = bg % p.num_kv_heads;
    if (b >= p.header->batch) return;                     // rows past the live batch of a capacity plan
    const SeqInfo si = p.seq_info[b];
    if (si.slot_base < 0) return;                         // a single split, written directly by the partial kernel
    const int S = si.n_splits;
    const int q = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int col = slice * 32 + lane;
    const bool live = col < G * D4;
    const int h = live ? col / D4 : 0;
    const int RF = rec_floats(G, D);
    const float* const recs = p.ws + ((int64_t)si.slot_base * p.num_kv_heads + g) * RF;
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
    for (int j = q + 4 * kCombineBatch; j < S; j += 4) mloc = fmaxf(mloc, __ldcg(mlp + j * (rec_stride / 2)).x);
    sm_m[q][lane] = mloc;
    __syncthreads();
    const float M = fmaxf(fmaxf(sm_m[0][lane], sm_m[1][lane]), fmaxf(sm_m[2][lane], sm_m[3][lane]));

    float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
    float lch = 0.f;
    for (int t0 = 0; q + 4 * t0 < S; t0 += kCombineBatch) {
        if (t0 > 0) {
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
    sm_acc[q][lane] = acc;
    sm_l[q][lane] = lch;
    __syncthreads();
    if (q == 0 && live) {
        const int d4 = col % D4;
        const float ls = ((sm_l[0][lane] + sm_l[1][lane]) + sm_l[2][lane]) + sm_l[3][lane];
        float4 o = make_float4(0.f, 0.f, 0.f, 0.f);
        if (M != -INFINITY && ls > 0.f) {
            const float inv = 1.0f / ls;
            const float4 a0 = sm_acc[0][lane], a1 = sm_acc[1][lane], a2 = sm_acc[2][lane], a3 = sm_acc[3][lane];
            o.x = (((a0.x + a1.x) + a2.x) + a3.x) * inv;
            o.y = (((a0.y + a1.y) + a2.y) + a3.y) * inv;
            o.z = (((a0.z + a1.z) + a2.z) + a3.z) * inv;
            o.w = (((a0.w + a1.w) + a2.w) + a3.w) * inv;
        }
        store_out4(p.out, ((int64_t)b * p.num_q_heads + g * G + h) * D + d4 * 4, o, p.out_bf16);
        if (p.lse != nullptr && d4 == 0)
            p.lse[(int64_t)b * p.num_q_heads + g * G + h] = (M != -INFINITY && ls > 0.f) ? (M + log2f(ls)) * kLn2 : -INFINITY;
    }
}

inline int combine_slices(int D, int G) { return (G * (D / 4) + 31) / 32; }

// Launches the combine kernel with a programmatic dependency on whatever was
// launched before it on `stream` (the partial kernel).
template <int D>
inline int combine_launch_dim(int G, const KernelParams& kp, unsigned groups, cudaStream_t stream)
{
    const int n_slices = combine_slices(D, G);
    cudaLaunchConfig_t cfg;
    cfg.gridDim = dim3(groups * (unsigned)n_slices, 1, 1);
    cfg.blockDim = dim3(kCombineThreads, 1, 1);
    cfg.dynamicSmemBytes = 0;
    cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    if (cudaLaunchKernelEx(&cfg, decode_attn_combine_kernel<D>, kp, G, n_slices) != cudaSuccess) {
        (void)cudaGetLastError();
        return DA_ERR_CUDA;
    }
    return DA_OK;
}

inline int combine_launch(int D, int G, const KernelParams& kp, unsigned groups, cudaStream_t stream)
{
    if (D == 64) return combine_launch_dim<64>(G, kp, groups, stream);
    if (D == 128) return combine_launch_dim<128>(G, kp, groups, stream);
    return DA_ERR_UNSUPPORTED;
}

}  // namespace da
