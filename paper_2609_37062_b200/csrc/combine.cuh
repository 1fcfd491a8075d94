// LSE combine kernel: one block per (sequence, KV head) merges the partial
// records of the group's query heads in ascending split order.
#pragma once

#include <algorithm>

#include "common.cuh"

namespace da {

constexpr int kCombineThreads = 128;

template <int D>
__global__ void __launch_bounds__(kCombineThreads) decode_attn_combine_kernel(const KernelParams p, int G, int cap)
{
    const int b = blockIdx.x / p.num_kv_heads;
    const int g = blockIdx.x % p.num_kv_heads;
    if (b >= p.header->batch) return;                  // rows past the live batch of a capacity plan
    const SeqInfo si = p.seq_info[b];
    if (si.n_splits <= 1 || si.slot_base < 0) return;  // written directly by the partial kernel
    extern __shared__ __align__(16) uint8_t combine_stage[];
    __shared__ __align__(8) uint64_t bar;
    if (threadIdx.x == 0) {
        mbar_init(smem_u32(&bar), 1);
        mbar_init_fence();
    }
    __syncthreads();
    uint32_t parity = 0;
    merge_group<D>(p, b, g, G, si.slot_base, si.n_splits, threadIdx.x, kCombineThreads, combine_stage, cap,
                   smem_u32(&bar), parity);
}

inline int combine_cap(int D, int G) { return std::max(1, std::min(32, (64 * 1024) / (rec_floats(G, D) * 4))); }

template <int D>
inline int combine_launch_dim(int G, const KernelParams& kp, unsigned grid, cudaStream_t stream)
{
    const int cap = combine_cap(D, G);
    const int smem = merge_stage_bytes(G, D, cap);
    if (cudaFuncSetAttribute(decode_attn_combine_kernel<D>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem) !=
        cudaSuccess) {
        (void)cudaGetLastError();
        return DA_ERR_CUDA;
    }
    decode_attn_combine_kernel<D><<<grid, kCombineThreads, smem, stream>>>(kp, G, cap);
    return DA_OK;
}

inline int combine_launch(int D, int G, const KernelParams& kp, unsigned grid, cudaStream_t stream)
{
    if (D == 64) return combine_launch_dim<64>(G, kp, grid, stream);
    if (D == 128) return combine_launch_dim<128>(G, kp, grid, stream);
    return DA_ERR_UNSUPPORTED;
}

}  // namespace da
