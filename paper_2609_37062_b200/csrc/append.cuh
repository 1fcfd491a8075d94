// Own-layer KV write (Invariant 1): scatter every row's new K and V rows into
// the paged pools at logical position seq_len - 1.  One warp per (sequence,
// KV head); 16-byte stores; bit-exact.  Rows write whether or not the RUN
// mask lets them attend: skipped layers still own their KV.
#pragma once

#include "common.cuh"

namespace da {

constexpr int kAppendThreads = 128;

struct AppendParams {
    const __nv_bfloat16* new_k;   // [B][Hkv][D]
    const __nv_bfloat16* new_v;
    __nv_bfloat16* k;
    __nv_bfloat16* v;
    const int32_t* block_table;
    const int32_t* seq_lens;
    int32_t* status;              // may be NULL
    int64_t k_stride_page, k_stride_token, k_stride_head;
    int64_t v_stride_page, v_stride_token, v_stride_head;
    int64_t num_pages;
    int32_t batch, num_kv_heads, head_dim, max_pages_per_seq;
    int32_t page_shift;           // log2(page_size)
};

__global__ void __launch_bounds__(kAppendThreads) decode_attn_append_kernel(const AppendParams p)
{
    pdl_launch_dependents();      // the attention kernel may start its prologue; it waits before reading K/V
    pdl_wait_primary();           // the projections that produced new_k / new_v are complete
    const int row = blockIdx.x * (kAppendThreads / 32) + (threadIdx.x >> 5);
    const int lane = threadIdx.x & 31;
    if (row >= p.batch * p.num_kv_heads) return;
    const int b = row / p.num_kv_heads, g = row % p.num_kv_heads;
    const int L = __ldg(p.seq_lens + b);
    if (L <= 0) return;
    const int t = L - 1;
    if ((t >> p.page_shift) >= p.max_pages_per_seq) {
        if (lane == 0 && p.status) record_status(p.status, DA_ERR_STALE_PLAN);
        return;
    }
    const int page = __ldg(p.block_table + (int64_t)b * p.max_pages_per_seq + (t >> p.page_shift));
    if ((unsigned)page >= (unsigned)p.num_pages) {
        if (lane == 0 && p.status) record_status(p.status, DA_ERR_BAD_PAGE);
        return;
    }
    const int slot = t & ((1 << p.page_shift) - 1);
    const int chunks = p.head_dim / 8;                  // 16-byte chunks per row (<= 16: both rows fit one warp)
    const uint4* sk = reinterpret_cast<const uint4*>(p.new_k + (int64_t)row * p.head_dim);
    const uint4* sv = reinterpret_cast<const uint4*>(p.new_v + (int64_t)row * p.head_dim);
    uint4* dk = reinterpret_cast<uint4*>(p.k + (int64_t)page * p.k_stride_page + (int64_t)slot * p.k_stride_token + (int64_t)g * p.k_stride_head);
    uint4* dv = reinterpret_cast<uint4*>(p.v + (int64_t)page * p.v_stride_page + (int64_t)slot * p.v_stride_token + (int64_t)g * p.v_stride_head);
    if (lane < chunks) dk[lane] = __ldg(sk + lane);
    else if (lane < 2 * chunks) dv[lane - chunks] = __ldg(sv + lane - chunks);
}

}  // namespace da
