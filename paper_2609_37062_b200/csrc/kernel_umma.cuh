// Shared-prefix units on the tcgen05 tensor cores.
//
// A prefix every sequence of the batch shares (few-shot prompts served from a
// prefix cache) is a dense contraction: for one KV head, the query rows of
// many sequences meet the same K/V pages.  One unit = (KV head, chunk of up to
// 384 prefix tokens, block of 128 / G sequences): the 128 query rows form the
// M dimension of the MMAs, so a prefix page is fetched once for 128 rows.
//
//   S = Q K^T   three 128 x 128 x 128 tiles, accumulators in tensor memory
//               columns [0, 384): row r of S in lane r, token t in column t
//   softmax     thread r owns row r: exact maximum over the chunk first, then
//               p = 2^(s * scale * log2 e - m); no running rescale is needed
//               because the whole chunk's logits are resident
//   P           must keep more than bf16 precision: bf16(p) and
//               bf16(p - bf16(p)) are written back over the logits (two bf16
//               per column; the 32 logit columns of 32 tokens become 16
//               columns of high parts and 16 of low parts)
//   O = P V     A = P from tensor memory, B = V tile from shared memory with
//               the head dimension contiguous; high and low parts accumulate
//               into the same 128 x 128 fp32 tile in columns [384, 512)
//   records     row r = (sequence r / G, head r mod G) goes to that
//               sequence's record of this prefix chunk, unnormalised, with
//               (m, l), exactly like any other split; the combine kernel
//               merges prefix and suffix splits.
//
// Threads: warps 0..3 each own 32 lanes of tensor memory (softmax, epilogue);
// warp 4 issues the TMA boxes and, from one lane, the MMAs.  K tile t and
// then V tile t use stage t of shared memory; V lands as soon as the MMAs
// that read K tile t have completed.  Every wait is bounded; a wait that gives
// up records DA_ERR_TIMEOUT, and the block still frees its tensor memory.
#pragma once

#include "kernel_mma.cuh"
#include "umma.cuh"

namespace da {

constexpr int kUmmaThreads = 160;
constexpr int kUmmaRows = 128;                    // query rows of a unit
constexpr int kUmmaTileTokens = 128;
constexpr int kUmmaMaxTiles = 3;
constexpr int kUmmaMaxTokens = kUmmaTileTokens * kUmmaMaxTiles;
constexpr int kUmmaHalfBytes = 128 * 128;         // 128 rows x 64 dims of bf16
constexpr int kUmmaTileBytes = 2 * kUmmaHalfBytes;   // [half of the head dim][row][64 dims]
constexpr int kUmmaSmemBytes = (1 + kUmmaMaxTiles) * kUmmaTileBytes + 1024 /* barriers */ + 1024 /* alignment */;
constexpr int kUmmaTmemCols = 512;
constexpr int kUmmaOutCol = kUmmaMaxTokens;       // first column of the output tile

inline bool umma_supports(int D, int G) { return D == 128 && (G == 1 || G == 2 || G == 4 || G == 8); }

__global__ void __launch_bounds__(kUmmaThreads, 1)
decode_attn_umma_prefix_kernel(const KernelParams p, const __grid_constant__ CUtensorMap k_map,
                               const __grid_constant__ CUtensorMap v_map, const int G)
{
    constexpr int D = 128;
    extern __shared__ uint8_t smem_raw[];
    const uint32_t raw = smem_u32(smem_raw);
    const uint32_t base = (raw + 1023u) & ~1023u;
    uint8_t* const gbase = smem_raw + (base - raw);
    const uint32_t q_base = base;
    const uint32_t tile_base = base + kUmmaTileBytes;                       // stage t at tile_base + t * tile bytes
    const uint32_t bar_base = base + (1 + kUmmaMaxTiles) * kUmmaTileBytes;
    // barriers: full_k[3], full_v[3], k_done[3], s_ready, p_ready, o_ready
    const uint32_t bar_full_k = bar_base, bar_full_v = bar_base + 24, bar_k_done = bar_base + 48;
    const uint32_t bar_s = bar_base + 72, bar_p = bar_base + 80, bar_o = bar_base + 88;
    volatile uint32_t* const sm_tmem = reinterpret_cast<volatile uint32_t*>(gbase + (bar_base - base) + 128);
    volatile int* const sm_abort = reinterpret_cast<volatile int*>(gbase + (bar_base - base) + 132);

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const decode_attn_unit_t u = load_unit(p.units, blockIdx.x);
    const int g = u.kv_head & 0xffff, nseq = u.kv_head >> 16;
    const int n_tok = u.tok_end - u.tok_begin;                              // whole pages, at most 384 tokens
    const int n_pages = n_tok >> 4;
    const int n_tiles = (n_tok + kUmmaTileTokens - 1) / kUmmaTileTokens;

    if (tid == 0) {
        tma_prefetch_descriptor(&k_map);
        tma_prefetch_descriptor(&v_map);
        for (int i = 0; i < 9; ++i) mbar_init(bar_base + 8 * i, 1);
        mbar_init(bar_s, 1);
        mbar_init(bar_p, kUmmaRows);
        mbar_init(bar_o, 1);
        *sm_abort = 0;
        mbar_init_fence();
    }
    if (warp == 4) umma::tmem_alloc(smem_u32(const_cast<uint32_t*>(sm_tmem)), kUmmaTmemCols);
    umma::fence_before_thread_sync();
    __syncthreads();
    umma::fence_after_thread_sync();
    const uint32_t tmem = *sm_tmem;
    // Only the plan's work list and this block's own state were touched so far.
    pdl_wait_primary();

    if (warp == 4) {
        // ------------------------------------------------------------ loads and MMAs
        const uint64_t l2_policy = l2_policy_evict_first();
        const int32_t* bt = p.block_table + (int64_t)u.seq * p.max_pages_per_seq + (u.tok_begin >> 4);
        // lane j < 16 issues box (page j / 2, half j % 2) of a tile; a page past the chunk is
        // fetched from outside the pool, which the TMA unit fills with zeros
        auto issue_tile = [&](const CUtensorMap* map, int t, uint32_t bar) {
            if (lane == 0) mbar_arrive_expect_tx(bar, kUmmaTileBytes);
            __syncwarp();
            if (lane < 16) {
                const int pg = lane >> 1, hf = lane & 1;
                const int gp = t * 8 + pg;
                int page_id = (int)p.num_pages;
                if (gp < n_pages) {
                    page_id = __ldg(bt + gp);
                    if ((unsigned)page_id >= (unsigned)p.num_pages) {       // never hand TMA a page outside the pool
                        record_status(p.status, DA_ERR_BAD_PAGE);
                        page_id = 0;
                    }
                }
                const uint32_t dst = tile_base + t * kUmmaTileBytes + hf * kUmmaHalfBytes + pg * 2048;
                tma_load_4d(dst, map, bar, hf * 64, 0, g, page_id, l2_policy);
            }
        };
        for (int t = 0; t < n_tiles; ++t) issue_tile(&k_map, t, bar_full_k + 8 * t);

        block_sync(1, kUmmaThreads);                                        // Q is in shared memory
        bool ok = true;
        constexpr uint32_t idesc_qk = umma::instr_desc_bf16(128, 128, false);
        constexpr uint32_t idesc_pv = umma::instr_desc_bf16(128, 128, true);
        if (lane == 0) {
            for (int t = 0; t < n_tiles && ok; ++t) {
                ok = mbar_wait(bar_full_k + 8 * t, 0);
                if (!ok) break;
                umma::fence_after_thread_sync();
#pragma unroll
                for (int ks = 0; ks < D / 16; ++ks) {
                    const uint32_t off = (ks >> 2) * kUmmaHalfBytes + (ks & 3) * 32;
                    const uint64_t a = umma::smem_desc_sw128(q_base + off, 16, 1024);
                    const uint64_t b = umma::smem_desc_sw128(tile_base + t * kUmmaTileBytes + off, 16, 1024);
                    umma::mma_ss(tmem + t * kUmmaTileTokens, a, b, idesc_qk, ks > 0);
                }
                umma::commit(bar_k_done + 8 * t);
            }
            if (ok) umma::commit(bar_s);
        }
        ok = __shfl_sync(0xffffffffu, (int)ok, 0) != 0;
        // V tile t may land once the MMAs reading K tile t are done
        for (int t = 0; t < n_tiles && ok; ++t) {
            if (lane == 0) ok = mbar_wait(bar_k_done + 8 * t, 0);
            ok = __shfl_sync(0xffffffffu, (int)ok, 0) != 0;
            if (ok) issue_tile(&v_map, t, bar_full_v + 8 * t);
        }
        if (lane == 0 && ok) {
            ok = mbar_wait(bar_p, 0);
            if (ok) umma::fence_after_thread_sync();
            for (int t = 0; t < n_tiles && ok; ++t) {
                ok = mbar_wait(bar_full_v + 8 * t, 0);
                if (!ok) break;
                umma::fence_after_thread_sync();
                const int ksteps = min(8, (n_tok - t * kUmmaTileTokens) >> 4);
                for (int j = 0; j < ksteps; ++j) {
                    // 16 tokens: two groups of 8 rows, 128 bytes a row; the upper 64 dims one half further
                    const uint64_t b = umma::smem_desc_sw128(tile_base + t * kUmmaTileBytes + j * 2048, kUmmaHalfBytes, 1024);
                    const int kj = t * 8 + j;                               // 16-token step within the chunk
                    const uint32_t a_hi = tmem + (kj >> 1) * 32 + (kj & 1) * 8;
                    umma::mma_ts(tmem + kUmmaOutCol, a_hi, b, idesc_pv, kj > 0);
                    umma::mma_ts(tmem + kUmmaOutCol, a_hi + 16, b, idesc_pv, true);
                }
            }
            if (ok) umma::commit(bar_o);
        }
        ok = __shfl_sync(0xffffffffu, (int)ok, 0) != 0;
        if (!ok && lane == 0) {
            record_status(p.status, DA_ERR_TIMEOUT);
            *sm_abort = 1;
        }
    } else {
        // ------------------------------------------------------------ query rows, softmax, epilogue
        const int r = tid;                                                  // row of the tile = lane of tensor memory
        const int sl = r / G, h = r % G;
        const bool valid = sl < nseq;
        const int seq = u.seq + (valid ? sl : 0);
        {
            // row r of Q, 16 chunks of 16 bytes, into the swizzled K-major tile
            const uint4* src = reinterpret_cast<const uint4*>(p.q + ((int64_t)seq * p.num_q_heads + g * G + h) * D);
            uint4 v[16];
#pragma unroll
            for (int c = 0; c < 16; ++c) v[c] = valid ? __ldg(src + c) : make_uint4(0u, 0u, 0u, 0u);
#pragma unroll
            for (int c = 0; c < 16; ++c) {
                const uint32_t off = (c >> 3) * kUmmaHalfBytes + r * 128 + (((c & 7) ^ (r & 7)) << 4);
                *reinterpret_cast<uint4*>(gbase + off) = v[c];
            }
            asm volatile("fence.proxy.async.shared::cta;" ::: "memory");     // visible to the tensor core's reads
        }
        block_sync(1, kUmmaThreads);

        const SeqInfo si = p.seq_info[seq];
        bool dead = p.run_mask != nullptr && __ldg(p.run_mask + seq) == 0;  // masked row: an empty record
        if (valid && __ldg(p.seq_lens + seq) != si.seq_len) {                // stale plan: void the result, report it
            dead = true;
            record_status(p.status, DA_ERR_STALE_PLAN);
        }

        const uint32_t lane_base = tmem + ((uint32_t)(warp * 32) << 16);
        bool ok = mbar_wait(bar_s, 0);
        float m2 = -INFINITY, l = 0.f;
        if (ok) {
            umma::fence_after_thread_sync();
            const int n_chunks = (n_tok + 31) >> 5;
            uint32_t s[32];
            float mx = -INFINITY;
            for (int c = 0; c < n_chunks; ++c) {
                umma::ld32(lane_base + c * 32, s);
                umma::wait_ld();
#pragma unroll
                for (int i = 0; i < 32; ++i)
                    if (c * 32 + i < n_tok) mx = fmaxf(mx, __uint_as_float(s[i]));
            }
            m2 = mx * p.scale_log2;                                          // the scale is positive
            for (int c = 0; c < n_chunks; ++c) {
                umma::ld32(lane_base + c * 32, s);
                umma::wait_ld();
                uint32_t hi[16], lo[16];
#pragma unroll
                for (int i = 0; i < 16; ++i) {
                    float p0 = 0.f, p1 = 0.f;
                    if (c * 32 + 2 * i < n_tok) p0 = ex2f(fmaf(__uint_as_float(s[2 * i]), p.scale_log2, -m2));
                    if (c * 32 + 2 * i + 1 < n_tok) p1 = ex2f(fmaf(__uint_as_float(s[2 * i + 1]), p.scale_log2, -m2));
                    l += p0 + p1;
                    const __nv_bfloat162 ph = __floats2bfloat162_rn(p0, p1);
                    const float2 phf = __bfloat1622float2(ph);
                    const __nv_bfloat162 pl = __floats2bfloat162_rn(p0 - phf.x, p1 - phf.y);
                    hi[i] = *reinterpret_cast<const uint32_t*>(&ph);
                    lo[i] = *reinterpret_cast<const uint32_t*>(&pl);
                }
                // the chunk's 32 logit columns become 16 columns of high parts, 16 of low parts
                umma::st16(lane_base + c * 32, hi);
                umma::st16(lane_base + c * 32 + 16, lo);
            }
            umma::wait_st();
            umma::fence_before_thread_sync();
            mbar_arrive(bar_p);
            ok = mbar_wait(bar_o, 0);
        }
        if (ok) {
            umma::fence_after_thread_sync();
            const int RF = rec_floats(G, D);
            float* const rec = p.ws + ((int64_t)(si.slot_base + u.split_index) * p.num_kv_heads + g) * RF;
            uint32_t o[32];
#pragma unroll 1
            for (int c = 0; c < D / 32; ++c) {
                umma::ld32(lane_base + kUmmaOutCol + c * 32, o);
                umma::wait_ld();
                if (valid) {
                    float4* dst = reinterpret_cast<float4*>(rec + h * D + c * 32);
#pragma unroll
                    for (int i = 0; i < 8; ++i) {
                        float4 v = make_float4(__uint_as_float(o[4 * i]), __uint_as_float(o[4 * i + 1]),
                                               __uint_as_float(o[4 * i + 2]), __uint_as_float(o[4 * i + 3]));
                        if (dead) v = make_float4(0.f, 0.f, 0.f, 0.f);
                        __stcg(dst + i, v);
                    }
                }
            }
            if (valid)
                __stcg(reinterpret_cast<float2*>(rec + G * D) + h, dead ? make_float2(-INFINITY, 0.f) : make_float2(m2, l));
        } else if (lane == 0 && *sm_abort == 0) {
            record_status(p.status, DA_ERR_TIMEOUT);
        }
    }
    pdl_launch_dependents();
    umma::fence_before_thread_sync();
    __syncthreads();
    if (warp == 4) umma::tmem_dealloc(tmem, kUmmaTmemCols);
}

// ---------------------------------------------------------------- host side

inline int umma_prepare()
{
    if (cudaFuncSetAttribute(decode_attn_umma_prefix_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                             kUmmaSmemBytes) != cudaSuccess) {
        (void)cudaGetLastError();
        return DA_ERR_CUDA;
    }
    return DA_OK;
}

// One block per prefix unit: units [0, n_prefix_units) of the plan's work list.
inline int umma_prefix_launch(const decode_attn_shape_t& s, int G, const KernelParams& kp, unsigned n_prefix_units,
                              cudaStream_t stream)
{
    if (n_prefix_units == 0) return DA_OK;
    int rc = umma_prepare();
    if (rc != DA_OK) return rc;
    CUtensorMap kmap, vmap;
    rc = make_pool_map(&kmap, kp.k, s, s.k_stride_page, s.k_stride_token, s.k_stride_head);
    if (rc != DA_OK) return rc;
    rc = make_pool_map(&vmap, kp.v, s, s.v_stride_page, s.v_stride_token, s.v_stride_head);
    if (rc != DA_OK) return rc;
    cudaLaunchConfig_t cfg;
    cfg.gridDim = dim3(n_prefix_units, 1, 1);
    cfg.blockDim = dim3(kUmmaThreads, 1, 1);
    cfg.dynamicSmemBytes = (size_t)kUmmaSmemBytes;
    cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    if (cudaLaunchKernelEx(&cfg, decode_attn_umma_prefix_kernel, kp, kmap, vmap, G) != cudaSuccess) {
        (void)cudaGetLastError();
        return DA_ERR_CUDA;
    }
    return DA_OK;
}

}  // namespace da
