// Placeholder until the tensor-core kernel lands: nothing is supported.
#pragma once

#include "common.cuh"

namespace da {

inline bool mma_supports(int, int) { return false; }
inline int mma_query_occupancy(int, int, int*, int*) { return -1; }
inline int mma_launch(const decode_attn_shape_t&, int, const KernelParams&, unsigned, cudaStream_t) { return DA_ERR_UNSUPPORTED; }
inline int mma_debug_gather(const decode_attn_shape_t&, int, int, const void*, const void*, const int32_t*, void*, void*, int32_t*, cudaStream_t) { return DA_ERR_UNSUPPORTED; }
inline int mma_gather_probe(const decode_attn_shape_t&, int, const KernelParams&, uint32_t*, unsigned, cudaStream_t) { return DA_ERR_UNSUPPORTED; }

}  // namespace da
