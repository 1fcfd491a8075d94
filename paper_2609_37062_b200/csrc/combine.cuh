// LSE combine kernel: one block per (sequence, KV head, slice of 32 output
// columns), see combine_slice.  The grid is spread over all SMs, and the
// kernel is launched with a programmatic dependency on the partial kernel:
// its blocks may already be resident, waiting at the top, while the partial
// kernel's last blocks write their records.
#pragma once

#include "common.cuh"

namespace da {

// BATCH: records a thread keeps in flight (see combine_slice).  Plans with few splits per
// sequence launch the small variant, whose lower register count lets four times as many blocks
// be resident; the sums are the same either way.
template <int D, int BATCH>
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
    pdl_wait_primary();                                   // the records of the launch before this one are complete
    if (si.slot_base < 0) return;                         // a single split, written directly by the partial kernel
    combine_slice<D, BATCH>(p, b, g, slice, G, si.slot_base, si.n_splits, threadIdx.x, sm, 0);
}

// Launches the combine kernel with a programmatic dependency on whatever was
// launched before it on `stream` (the partial kernel).
template <int D>
inline int combine_launch_dim(int G, const KernelParams& kp, unsigned groups, cudaStream_t stream, bool few_splits)
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
    const cudaError_t e = few_splits ? cudaLaunchKernelEx(&cfg, decode_attn_combine_kernel<D, 2>, kp, G, n_slices)
                                     : cudaLaunchKernelEx(&cfg, decode_attn_combine_kernel<D, kCombineBatch>, kp, G, n_slices);
    if (e != cudaSuccess) {
        (void)cudaGetLastError();
        return DA_ERR_CUDA;
    }
    return DA_OK;
}

// max_splits: the most splits any sequence of the plan (or of its capacity) can have.
inline int combine_launch(int D, int G, const KernelParams& kp, unsigned groups, cudaStream_t stream, int max_splits)
{
    const bool few = max_splits <= 8;
    if (D == 64) return combine_launch_dim<64>(G, kp, groups, stream, few);
    if (D == 128) return combine_launch_dim<128>(G, kp, groups, stream, few);
    return DA_ERR_UNSUPPORTED;
}

}  // namespace da
