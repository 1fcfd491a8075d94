// LSE combine kernel: one block per (sequence, KV head, slice of 32 output
// columns), see combine_slice.  The grid is spread over all SMs, and the
// kernel is launched with a programmatic dependency on the partial kernel:
// its blocks may already be resident, waiting at the top, while the partial
// kernel's last blocks write their records.
#pragma once

#include "common.cuh"

namespace da {

// BATCH: records a thread keeps in flight (see combine_slice).
template <int D, int BATCH, bool ONE_PASS>
__global__ void __launch_bounds__(kCombineThreads) decode_attn_combine_kernel(const KernelParams p, int G, int n_slices)
{
    __shared__ __align__(16) float sm[kCombineSmemFloats];
    pdl_launch_dependents();                              // the next kernel may start its prologue
    // The plan's own tables (live batch, split table) do not depend on the launch before this
    // one: fetch them while it drains, and wait only before touching its records.
    const int slice = blockIdx.x % n_slices;
    const int bg = blockIdx.x / n_slices;
    const int b = bg / p.num_kv_heads, g = bg % p.num_kv_heads;
    const bool in_batch = b < p.header->batch;            // rows past the live batch of a capacity plan
    SeqInfo si;
    si.slot_base = -1;
    if (in_batch) si = p.seq_info[b];
    // (trace builds: the combine blocks' stamps follow the partial kernel's rows)
    if (threadIdx.x == 0) DA_TRACE_STAMP(p.n_work_blocks + blockIdx.x, 0);
    pdl_wait_primary();                                   // the records of the launch before this one are complete
    if (threadIdx.x == 0) DA_TRACE_STAMP(p.n_work_blocks + blockIdx.x, 1);
    if (si.slot_base < 0) return;                         // a single split, written directly by the partial kernel
    combine_slice<D, BATCH, ONE_PASS>(p, b, g, slice, G, si.slot_base, si.n_splits, threadIdx.x, sm, 0);
    if (threadIdx.x == 0) DA_TRACE_STAMP(p.n_work_blocks + blockIdx.x, 2);
}

// Plans whose sequences have at most MAXS (4 or 8) splits: one thread per output column, 128
// columns per block, nothing shared between threads (see combine_column).
template <int D, int MAXS>
__global__ void __launch_bounds__(kCombineThreads) decode_attn_combine_few_kernel(const KernelParams p, int G, int blocks_per_group)
{
    pdl_launch_dependents();
    const int bg = blockIdx.x / blocks_per_group;
    const int col = (blockIdx.x % blocks_per_group) * kCombineThreads + threadIdx.x;
    const int b = bg / p.num_kv_heads, g = bg % p.num_kv_heads;
    const bool in_batch = b < p.header->batch;
    SeqInfo si;
    si.slot_base = -1;
    if (in_batch) si = p.seq_info[b];
    if (threadIdx.x == 0) DA_TRACE_STAMP(p.n_work_blocks + blockIdx.x, 0);
    pdl_wait_primary();
    if (threadIdx.x == 0) DA_TRACE_STAMP(p.n_work_blocks + blockIdx.x, 1);
    if (si.slot_base < 0 || col >= G * (D / 4)) return;
    combine_column<D, MAXS>(p, b, g, col, G, si.slot_base, si.n_splits);
    if (threadIdx.x == 0) DA_TRACE_STAMP(p.n_work_blocks + blockIdx.x, 2);
}

// Merge of KV-range shards: every shard holds a normalised output and its log-sum-exp (natural
// log) for each row; one thread per four output dims, shards in ascending order.
__global__ void __launch_bounds__(128) decode_attn_merge_shards_kernel(const float* out_shards, const float* lse_shards,
                                                                       int n_shards, int64_t rows, int D4, void* out,
                                                                       float* lse, int out_kind)
{
    const int64_t idx = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (idx >= rows * D4) return;
    const int64_t row = idx / D4;
    const int d4 = (int)(idx % D4);
    float M = -INFINITY;
    for (int r = 0; r < n_shards; ++r) M = fmaxf(M, __ldg(lse_shards + (int64_t)r * rows + row));
    float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
    float ws = 0.f;
    if (M != -INFINITY) {
        for (int r = 0; r < n_shards; ++r) {
            const float w = ex2f((__ldg(lse_shards + (int64_t)r * rows + row) - M) * kLog2e);   // empty shard: w = 0
            const float4 v = __ldg(reinterpret_cast<const float4*>(out_shards) + ((int64_t)r * rows + row) * D4 + d4);
            acc.x = fmaf(w, v.x, acc.x);
            acc.y = fmaf(w, v.y, acc.y);
            acc.z = fmaf(w, v.z, acc.z);
            acc.w = fmaf(w, v.w, acc.w);
            ws += w;
        }
        const float inv = 1.0f / ws;                          // ws >= 1: the shard that holds the maximum weighs 1
        acc.x *= inv; acc.y *= inv; acc.z *= inv; acc.w *= inv;
    }
    store_out4(out, idx * 4, acc, out_kind);
    if (lse != nullptr && d4 == 0) lse[row] = (M != -INFINITY) ? M + log2f(ws) * kLn2 : -INFINITY;
}

// Launches the combine kernel with a programmatic dependency on whatever was
// launched before it on `stream` (the partial kernel).
template <int D>
inline int combine_launch_dim(int G, const KernelParams& kp, unsigned groups, cudaStream_t stream, int max_splits)
{
    const int n_slices = combine_slices(D, G);
    const int blocks_per_group = (G * (D / 4) + kCombineThreads - 1) / kCombineThreads;
    cudaLaunchConfig_t cfg;
    cfg.gridDim = dim3(groups * (unsigned)(max_splits <= 8 ? blocks_per_group : n_slices), 1, 1);
    cfg.blockDim = dim3(kCombineThreads, 1, 1);
    cfg.dynamicSmemBytes = 0;
    cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    // The slice kernel keeps a chain's records in flight all at once; instantiated for chains of up to 8, 10
    // and 12 records (32, 40, 48 splits; more splits take further rounds of 12), since the shorter variants are
    // smaller and start faster: one 32,768-token sequence in 37 splits 23.42 -> 23.26 us per step with 10
    // instead of 12.  The order of the sums, and with it every bit of the result, is the same in all of them.
    const cudaError_t e =
        max_splits <= 4    ? cudaLaunchKernelEx(&cfg, decode_attn_combine_few_kernel<D, 4>, kp, G, blocks_per_group)
        : max_splits <= 8  ? cudaLaunchKernelEx(&cfg, decode_attn_combine_few_kernel<D, 8>, kp, G, blocks_per_group)
        : max_splits <= 32 ? cudaLaunchKernelEx(&cfg, decode_attn_combine_kernel<D, 8, true>, kp, G, n_slices)
        : max_splits <= 40 ? cudaLaunchKernelEx(&cfg, decode_attn_combine_kernel<D, 10, true>, kp, G, n_slices)
        : max_splits <= 48 ? cudaLaunchKernelEx(&cfg, decode_attn_combine_kernel<D, kCombineBatch, true>, kp, G, n_slices)
                           : cudaLaunchKernelEx(&cfg, decode_attn_combine_kernel<D, kCombineBatch, false>, kp, G, n_slices);
    if (e != cudaSuccess) {
        (void)cudaGetLastError();
        return DA_ERR_CUDA;
    }
    return DA_OK;
}

// max_splits: the most splits any sequence of the plan (or of its capacity) can have.
inline int combine_launch(int D, int G, const KernelParams& kp, unsigned groups, cudaStream_t stream, int max_splits)
{
    if (D == 64) return combine_launch_dim<64>(G, kp, groups, stream, max_splits);
    if (D == 128) return combine_launch_dim<128>(G, kp, groups, stream, max_splits);
    return DA_ERR_UNSUPPORTED;
}

}  // namespace da
