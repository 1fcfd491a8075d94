// LSE combine kernel: one block per (sequence, KV head) merges the partials
// of the group's query heads in ascending split order.
#pragma once

#include "common.cuh"

namespace da {

constexpr int kCombineThreads = 128;

template <int D>
__global__ void __launch_bounds__(kCombineThreads) decode_attn_combine_kernel(const KernelParams p, int G)
{
    const int b = blockIdx.x / p.num_kv_heads;
    const int g = blockIdx.x % p.num_kv_heads;
    if (b >= p.header->batch) return;                  // rows past the live batch of a capacity plan
    const SeqInfo si = p.seq_info[b];
    if (si.n_splits <= 1 || si.slot_base < 0) return;  // written directly by the partial kernel
    merge_group<D>(p, b, g, G, si.slot_base, si.n_splits, threadIdx.x, kCombineThreads);
}

inline int combine_launch(int D, int G, const KernelParams& kp, unsigned grid, cudaStream_t stream)
{
    if (D == 64)
        decode_attn_combine_kernel<64><<<grid, kCombineThreads, 0, stream>>>(kp, G);
    else if (D == 128)
        decode_attn_combine_kernel<128><<<grid, kCombineThreads, 0, stream>>>(kp, G);
    else
        return DA_ERR_UNSUPPORTED;
    return DA_OK;
}

}  // namespace da
