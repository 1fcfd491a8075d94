// CUDA-core split-KV partial kernel.
//
// One block per work unit (sequence, KV head, token range), 4 warps.  A K or
// V row of D bf16 is read by D/8 neighbouring lanes with one 16-byte load
// each (a warp covers 2 rows at D = 128, 4 at D = 64), straight from global
// memory into registers; U rows per thread are in flight before any is used.
// Each thread holds its 8-dim slice of all G query rows of the group in fp32
// (pre-multiplied by sm_scale * log2 e), so every K/V byte is used G times.
// Logit partial sums are reduced over the D/8 lanes by xor shuffles; running
// max and sum of exponentials live in fp32 registers per row group and the
// row groups of the block are merged in a fixed order through shared memory.
//
// This kernel serves group size 1 (no reuse, nothing for a tensor core to
// do) and is the CUDA-core reference point for the tensor-core kernel.
#pragma once

#include <cuda_fp16.h>

#include "common.cuh"

namespace da {

constexpr int kSimtThreads = 128;
constexpr int kSimtWarps = kSimtThreads / 32;

__device__ __forceinline__ uint4 ldg_stream16(const void* ptr)
{
    uint4 v;
    asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];"
                 : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w)
                 : "l"(ptr));
    return v;
}

// Eight 16-bit inputs to fp32: bf16 by shifts, fp16 by conversion (one flag for the whole launch).
__device__ __forceinline__ void unpack8(const uint4& w, float (&f)[8], int in_f16)
{
    if (in_f16) {
        const __half2* h = reinterpret_cast<const __half2*>(&w);
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            const float2 v = __half22float2(h[i]);
            f[2 * i] = v.x;
            f[2 * i + 1] = v.y;
        }
        return;
    }
    f[0] = __uint_as_float(w.x << 16); f[1] = __uint_as_float(w.x & 0xffff0000u);
    f[2] = __uint_as_float(w.y << 16); f[3] = __uint_as_float(w.y & 0xffff0000u);
    f[4] = __uint_as_float(w.z << 16); f[5] = __uint_as_float(w.z & 0xffff0000u);
    f[6] = __uint_as_float(w.w << 16); f[7] = __uint_as_float(w.w & 0xffff0000u);
}

template <int D, int G>
__global__ void __launch_bounds__(kSimtThreads) decode_attn_simt_kernel(const KernelParams p)
{
    constexpr int LPR = D / 8;                  // lanes per row
    constexpr int RPW = 32 / LPR;               // rows per warp step
    constexpr int ROWS = kSimtWarps * RPW;      // row groups per block
    constexpr int U = 4;                        // rows in flight per thread

    // one raw block so the in-kernel merge can reuse it as its staging area
    constexpr int kOwnBytes = ROWS * G * D * 4 + 2 * ROWS * G * 4;
    constexpr int kRawBytes = kOwnBytes > kCombineSmemFloats * 4 ? kOwnBytes : kCombineSmemFloats * 4;
    __shared__ __align__(16) uint8_t sm_raw[kRawBytes];
    float (*sm_acc)[G][D] = reinterpret_cast<float (*)[G][D]>(sm_raw);
    float (*sm_rm)[G] = reinterpret_cast<float (*)[G]>(sm_raw + ROWS * G * D * 4);
    float (*sm_rl)[G] = reinterpret_cast<float (*)[G]>(sm_raw + ROWS * G * D * 4 + ROWS * G * 4);
    __shared__ int sm_flag;

    const int uid = blockIdx.x;
    if (p.fused && uid >= p.n_work_blocks) {    // a merge block of a fused launch
        pdl_launch_dependents();
        pdl_wait_primary();
        fused_merge_blocks<D>(p, G, kSimtThreads, reinterpret_cast<float*>(sm_raw), &sm_flag);
        return;
    }
    if (uid >= (p.grid_exit ? p.header->n_units : p.n_units)) {   // surplus blocks of a capacity launch
        if (uid == 0) pdl_wait_primary();       // an empty launch still hands stream order on to its successors
        return;
    }
    const decode_attn_unit_t u = load_unit(p.units, uid);
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int rg = warp * RPW + lane / LPR;     // row group of this thread
    const int li = lane % LPR;                  // 8-dim slice within the row
    const int b = u.seq, g = u.kv_head;

    const int t0 = u.tok_begin;
    int t1 = u.tok_end;
    // Only the plan's work list was read so far; what the kernel launched before this one may
    // have produced (q, new K/V rows, lengths, page mappings) is read past this point.
    pdl_wait_primary();
    // Invariant 2 (never run on stale lengths): fetched now, compared in the epilogue so the
    // load stays off the critical path; page ids are range-checked, so nothing can fault.
    const int dev_len = __ldg(p.seq_lens + b);
    if (p.run_mask != nullptr && __ldg(p.run_mask + b) == 0) t1 = t0;   // masked row reads no KV

    float qf[G][8];
#pragma unroll
    for (int h = 0; h < G; ++h) {
        const uint4 w = *reinterpret_cast<const uint4*>(p.q + ((int64_t)b * p.num_q_heads + g * G + h) * D + li * 8);
        unpack8(w, qf[h], p.in_f16);
#pragma unroll
        for (int i = 0; i < 8; ++i) qf[h][i] *= p.scale_log2;
    }
    float m[G], l[G], acc[G][8];
#pragma unroll
    for (int h = 0; h < G; ++h) {
        m[h] = -INFINITY;
        l[h] = 0.f;
#pragma unroll
        for (int i = 0; i < 8; ++i) acc[h][i] = 0.f;
    }

    const int32_t* bt = p.block_table + (int64_t)b * p.max_pages_per_seq;
    const int page_shift = 4 + p.tile_shift, page_mask = (1 << page_shift) - 1;
    const __nv_bfloat16* kbase = p.k + (int64_t)g * p.k_stride_head + li * 8;
    const __nv_bfloat16* vbase = p.v + (int64_t)g * p.v_stride_head + li * 8;

    for (int tb = t0; tb < t1; tb += ROWS * U) {
        uint4 kk[U], vv[U];
        bool ok[U];
#pragma unroll
        for (int j = 0; j < U; ++j) {
            const int t = tb + j * ROWS + rg;
            ok[j] = t < t1;
            kk[j] = make_uint4(0, 0, 0, 0);
            vv[j] = make_uint4(0, 0, 0, 0);
            if (ok[j]) {
                const int page = __ldg(bt + (t >> page_shift));
                if ((unsigned)page >= (unsigned)p.num_pages) {
                    record_status(p.status, DA_ERR_BAD_PAGE);
                    ok[j] = false;
                } else {
                    const int slot = t & page_mask;
                    kk[j] = ldg_stream16(kbase + (int64_t)page * p.k_stride_page + (int64_t)slot * p.k_stride_token);
                    vv[j] = ldg_stream16(vbase + (int64_t)page * p.v_stride_page + (int64_t)slot * p.v_stride_token);
                }
            }
        }
        float s[U][G];
#pragma unroll
        for (int j = 0; j < U; ++j) {
            float kf[8];
            unpack8(kk[j], kf, p.in_f16);
#pragma unroll
            for (int h = 0; h < G; ++h) {
                float d = 0.f;
#pragma unroll
                for (int i = 0; i < 8; ++i) d = fmaf(qf[h][i], kf[i], d);
                s[j][h] = d;
            }
        }
#pragma unroll
        for (int off = LPR / 2; off >= 1; off >>= 1) {
#pragma unroll
            for (int j = 0; j < U; ++j)
#pragma unroll
                for (int h = 0; h < G; ++h) s[j][h] += __shfl_xor_sync(0xffffffffu, s[j][h], off);
        }
        float pr[U][G];
#pragma unroll
        for (int h = 0; h < G; ++h) {
            float mx = m[h];
#pragma unroll
            for (int j = 0; j < U; ++j) {
                s[j][h] = ok[j] ? s[j][h] : -INFINITY;
                mx = fmaxf(mx, s[j][h]);
            }
            const float m_safe = (mx == -INFINITY) ? 0.f : mx;
            const float alpha = ex2f(m[h] - m_safe);
            m[h] = mx;
            float lsum = 0.f;
#pragma unroll
            for (int j = 0; j < U; ++j) {
                pr[j][h] = ex2f(s[j][h] - m_safe);
                lsum += pr[j][h];
            }
            l[h] = fmaf(l[h], alpha, lsum);
#pragma unroll
            for (int i = 0; i < 8; ++i) acc[h][i] *= alpha;
        }
#pragma unroll
        for (int j = 0; j < U; ++j) {
            float vf[8];
            unpack8(vv[j], vf, p.in_f16);
#pragma unroll
            for (int h = 0; h < G; ++h)
#pragma unroll
                for (int i = 0; i < 8; ++i) acc[h][i] = fmaf(pr[j][h], vf[i], acc[h][i]);
        }
    }

    pdl_launch_dependents();                    // the combine kernel may start getting scheduled
    // the row groups' states go to shared memory; block_finish merges them in a fixed order
    if (dev_len != u.seq_len) {                 // stale plan: void the result, report it
        if (tid == 0) record_status(p.status, DA_ERR_STALE_PLAN);
#pragma unroll
        for (int h = 0; h < G; ++h) {
            m[h] = -INFINITY;
            l[h] = 0.f;
        }
    }
#pragma unroll
    for (int h = 0; h < G; ++h) {
        if (li == 0) {
            sm_rm[rg][h] = m[h];
            sm_rl[rg][h] = l[h];
        }
        float4* dst = reinterpret_cast<float4*>(&sm_acc[rg][h][li * 8]);
        dst[0] = make_float4(acc[h][0], acc[h][1], acc[h][2], acc[h][3]);
        dst[1] = make_float4(acc[h][4], acc[h][5], acc[h][6], acc[h][7]);
    }
    __syncthreads();
    block_finish<D, ROWS, G, false>(p, u, G, &sm_acc[0][0][0], &sm_rm[0][0], &sm_rl[0][0], tid, kSimtThreads, 0);
}

}  // namespace da
