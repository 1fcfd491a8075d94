// Shared-prefix units on the tcgen05 tensor cores.
//
// A prefix every sequence of the batch shares (few-shot prompts served from a
// prefix cache) is a dense contraction: for one KV head, the query rows of
// many sequences meet the same K/V pages.  One unit = (KV head, chunk of up to
// 384 prefix tokens, block of 128 / G sequences): the 128 query rows form the
// M dimension of the MMAs, so a prefix page is fetched once for 128 rows.
//
//   S = Q K^T   up to three 128 x 128 x 128 tiles, accumulators in tensor
//               memory columns [0, 384): row r of S in lane r, token t in
//               column t
//   softmax     thread r owns row r: exact maximum over the chunk first (tile
//               by tile as the MMAs finish), then p = 2^(s * scale * log2 e -
//               m); no running rescale is needed because the whole chunk's
//               logits are resident
//   P           must keep more than bf16 precision: the upper 16 bits of p and
//               the upper 16 bits of the (exact) remainder are written back
//               over the logits, two bf16 per column: the 32 logit columns of
//               32 tokens become 16 columns of high parts and 16 of low
//               parts.  What is dropped is below 2^-16 of p.
//   O = P V     A = P from tensor memory, B = V tile from shared memory with
//               the head dimension contiguous; high and low parts accumulate
//               into the same 128 x 128 fp32 tile in columns [384, 512); the
//               MMAs of a tile start as soon as that tile's P is written
//   records     row r = (sequence r / G, head r mod G) goes to that
//               sequence's record of this prefix chunk, unnormalised, with
//               (m, l), exactly like any other split; the combine kernel
//               merges prefix and suffix splits.  Each thread stages its row
//               in shared memory and sends it with one bulk copy.
//
// Threads: eight warps for softmax and epilogue, two per 32 lanes of tensor
// memory (one takes the even, one the odd 32-token groups of a row);
// a ninth warp issues the TMA boxes and, from one lane, the MMAs.  The 2 n tiles of a
// chunk of n token tiles (K_0 .. K_n-1, V_0 .. V_n-1) go through two stages of
// shared memory in that order; a stage is refilled when the MMAs that read
// its tile have completed.  Every barrier is used once.  Every wait is
// bounded; a wait that gives up records DA_ERR_TIMEOUT, and the block still
// frees its tensor memory.
#pragma once

#include "kernel_mma.cuh"
#include "umma.cuh"

namespace da {

constexpr int kUmmaTraceBase = 2048;              // debug timelines: rows of this kernel's units
constexpr int kUmmaSoftmaxWarps = 8;              // two per 32 lanes of tensor memory
constexpr int kUmmaSoftmaxThreads = kUmmaSoftmaxWarps * 32;
constexpr int kUmmaThreads = kUmmaSoftmaxThreads + 32;   // + the warp that issues loads and MMAs
constexpr int kUmmaRows = 128;                    // query rows of a unit
constexpr int kUmmaTileTokens = 128;
constexpr int kUmmaMaxTiles = 3;
constexpr int kUmmaMaxTokens = kUmmaTileTokens * kUmmaMaxTiles;
constexpr int kUmmaHalfBytes = 128 * 128;         // 128 rows x 64 dims of bf16
constexpr int kUmmaTileBytes = 2 * kUmmaHalfBytes;   // [half of the head dim][row][64 dims]
constexpr int kUmmaStages = 2;
constexpr int kUmmaBarrierBytes = 2048;           // barriers, page ids, the halves' maxima and sums
constexpr int kUmmaSmemUsed = (1 + kUmmaStages) * kUmmaTileBytes + kUmmaBarrierBytes + 1024 /* alignment */;
// Asked for: more than half an SM's shared memory, so that two of these blocks, each of which
// wants all of tensor memory, never share an SM.
constexpr int kUmmaSmemBytes = 116 * 1024;
static_assert(kUmmaSmemUsed <= kUmmaSmemBytes, "shared memory of the tcgen05 prefix kernel");
constexpr int kUmmaTmemCols = 512;
constexpr int kUmmaOutCol = kUmmaMaxTokens;       // first column of the output tile
constexpr int kUmmaOutRowBytes = 128 * 4 + 16;    // a staged output row; the pad spreads the rows over the banks

inline bool umma_supports(int D, int G) { return D == 128 && (G == 1 || G == 2 || G == 4 || G == 8); }

__device__ __forceinline__ void bulk_store_s2g(void* dst, uint32_t src, uint32_t bytes)
{
    asm volatile("cp.async.bulk.global.shared::cta.bulk_group [%0], [%1], %2;" ::"l"(dst), "r"(src), "r"(bytes) : "memory");
}
__device__ __forceinline__ void bulk_store_commit_and_wait_read()
{
    asm volatile("cp.async.bulk.commit_group;" ::: "memory");
    asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory");
}

// Shared-prefix units first_unit, first_unit + unit_stride, ... < n_units, one after the other, by
// the 288 threads of a block.  smem_raw: at least kUmmaSmemUsed bytes of dynamic shared memory.
__device__ __forceinline__ void umma_prefix_units(const KernelParams& p, const CUtensorMap* k_map, const CUtensorMap* v_map,
                                                  const int G, const int first_unit, const int unit_stride,
                                                  const int n_units, uint8_t* smem_raw)
{
    constexpr int D = 128;
    const uint32_t raw = smem_u32(smem_raw);
    const uint32_t base = (raw + 1023u) & ~1023u;
    uint8_t* const gbase = smem_raw + (base - raw);
    const uint32_t q_base = base;
    const uint32_t tile_base = base + kUmmaTileBytes;                       // stage s at tile_base + s * tile bytes
    const uint32_t bar_base = base + (1 + kUmmaStages) * kUmmaTileBytes;
    // single-use barriers: full[6] (a tile has landed), done[6] (the MMAs reading it have completed;
    // for a K tile that also means its logits are ready), p_ready[3], o_ready
    const uint32_t bar_full = bar_base, bar_done = bar_base + 48, bar_p = bar_base + 96, bar_o = bar_base + 120;
    uint8_t* const sm_misc = gbase + (bar_base - base);
    volatile uint32_t* const sm_tmem = reinterpret_cast<volatile uint32_t*>(sm_misc + 128);
    volatile int* const sm_abort = reinterpret_cast<volatile int*>(sm_misc + 132);
    int32_t* const sm_pages = reinterpret_cast<int32_t*>(sm_misc + 256);    // [24] page ids of the chunk
    float* const sm_part = reinterpret_cast<float*>(sm_misc + 512);         // [2][128]: the column halves' maxima, then sums

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    if (first_unit >= n_units) {
        if (blockIdx.x == 0) pdl_wait_primary();   // an empty launch still hands stream order on
        return;
    }
    if (tid == 0) {
        tma_prefetch_descriptor(k_map);
        tma_prefetch_descriptor(v_map);
        *sm_abort = 0;
    }
    if (warp == kUmmaSoftmaxWarps) umma::tmem_alloc(smem_u32(const_cast<uint32_t*>(sm_tmem)), kUmmaTmemCols);
    umma::fence_before_thread_sync();
    __syncthreads();
    umma::fence_after_thread_sync();
    const uint32_t tmem = *sm_tmem;
    // Only this block's own state was touched so far.
    pdl_wait_primary();

  for (int unit_index = first_unit; unit_index < n_units && *sm_abort == 0; unit_index += unit_stride) {
    const decode_attn_unit_t u = load_unit(p.units, unit_index);
    const int g = u.kv_head & 0xffff, nseq = u.kv_head >> 16;
    const int n_tok = u.tok_end - u.tok_begin;                              // whole pages, at most 384 tokens
    const int n_pages = n_tok >> 4;
    const int n_tiles = (n_tok + kUmmaTileTokens - 1) / kUmmaTileTokens;
    if (tid == 0) DA_TRACE_STAMP(kUmmaTraceBase + unit_index, 0);
    if (tid == 0) {
        // every barrier serves one unit: set up again for each (the block is past a barrier here,
        // nobody is still waiting on the previous unit's)
        if (unit_index != first_unit)
            for (int i = 0; i < 16; ++i) mbar_inval(bar_base + 8 * i);
        for (int i = 0; i < 12; ++i) mbar_init(bar_base + 8 * i, 1);
        for (int i = 0; i < 3; ++i) mbar_init(bar_p + 8 * i, kUmmaSoftmaxThreads);
        mbar_init(bar_o, 1);
        mbar_init_fence();
    }
    __syncthreads();
    if (tid == 0) DA_TRACE_STAMP(kUmmaTraceBase + unit_index, 1);

    if (warp == kUmmaSoftmaxWarps) {
        // ------------------------------------------------------------ loads and MMAs
        {
            // the chunk's page ids, checked once
            int page_id = (int)p.num_pages;   // a page past the chunk is fetched from outside the pool: zeros
            if (lane < n_pages) {
                page_id = __ldg(p.block_table + (int64_t)u.seq * p.max_pages_per_seq + (u.tok_begin >> 4) + lane);
                if ((unsigned)page_id >= (unsigned)p.num_pages) {           // never hand TMA a page outside the pool
                    record_status(p.status, DA_ERR_BAD_PAGE);
                    page_id = 0;
                }
            }
            if (lane < 24) sm_pages[lane] = page_id;
            __syncwarp();
        }
        const uint64_t l2_policy = l2_policy_evict_first();
        const int n_loads = 2 * n_tiles;
        // load i of the chunk: K tile i for i < n_tiles, else V tile i - n_tiles; stage i % 2.
        // Whole warp: lane j < 16 issues box (page j / 2, half j % 2).
        auto issue = [&](int i) {
            const bool is_v = i >= n_tiles;
            const int t = is_v ? i - n_tiles : i;
            const uint32_t bar = bar_full + 8 * i;
            if (lane == 0) mbar_arrive_expect_tx(bar, kUmmaTileBytes);
            __syncwarp();
            if (lane < 16) {
                const int pg = lane >> 1, hf = lane & 1;
                const uint32_t dst = tile_base + (i % kUmmaStages) * kUmmaTileBytes + hf * kUmmaHalfBytes + pg * 2048;
                tma_load_4d(dst, is_v ? v_map : k_map, bar, hf * 64, 0, g, sm_pages[t * 8 + pg], l2_policy);
            }
        };
        // lane 0 waits, the warp learns the outcome
        auto wait = [&](uint32_t bar) {
            bool r = true;
            if (lane == 0) r = mbar_wait(bar, 0);
            return __shfl_sync(0xffffffffu, (int)r, 0) != 0;
        };
        issue(0);
        issue(1);
        if (lane == 0) DA_TRACE_STAMP(kUmmaTraceBase + unit_index, 2);
        block_sync(1, kUmmaThreads);                                        // Q is in shared memory
        constexpr uint32_t idesc_qk = umma::instr_desc_bf16(128, 128, false);
        constexpr uint32_t idesc_pv = umma::instr_desc_bf16(128, 128, true);
        bool ok = true;
        // S_t = Q K_t^T
        for (int t = 0; t < n_tiles && ok; ++t) {
            ok = wait(bar_full + 8 * t);
            if (!ok) break;
            if (lane == 0) {
                if (t == n_tiles - 1) DA_TRACE_STAMP(kUmmaTraceBase + unit_index, 3);
                umma::fence_after_thread_sync();
                const uint32_t kt = tile_base + (t % kUmmaStages) * kUmmaTileBytes;
#pragma unroll
                for (int ks = 0; ks < D / 16; ++ks) {
                    const uint32_t off = (ks >> 2) * kUmmaHalfBytes + (ks & 3) * 32;
                    umma::mma_ss(tmem + t * kUmmaTileTokens, umma::smem_desc_sw128(q_base + off, 16, 1024),
                                 umma::smem_desc_sw128(kt + off, 16, 1024), idesc_qk, ks > 0);
                }
                umma::commit(bar_done + 8 * t);
            }
            __syncwarp();
            if (t + 2 < n_loads) {                                          // the stage is free once these MMAs are done
                ok = wait(bar_done + 8 * t);
                if (ok) issue(t + 2);
            }
        }
        if (lane == 0) DA_TRACE_STAMP(kUmmaTraceBase + unit_index, 4);
        // O += P_t V_t
        for (int t = 0; t < n_tiles && ok; ++t) {
            const int i = n_tiles + t;
            ok = wait(bar_p + 8 * t);
            if (lane == 0 && t == 0) DA_TRACE_STAMP(kUmmaTraceBase + unit_index, 9);
            if (ok) ok = wait(bar_full + 8 * i);
            if (!ok) break;
            if (lane == 0) {
                if (t == n_tiles - 1) DA_TRACE_STAMP(kUmmaTraceBase + unit_index, 10);
                umma::fence_after_thread_sync();
                const uint32_t vt = tile_base + (i % kUmmaStages) * kUmmaTileBytes;
                const int ksteps = min(8, (n_tok - t * kUmmaTileTokens) >> 4);
#pragma unroll 2
                for (int j = 0; j < ksteps; ++j) {
                    // 16 tokens: two groups of 8 rows, 128 bytes a row; the upper 64 dims one half further
                    const uint64_t b = umma::smem_desc_sw128(vt + j * 2048, kUmmaHalfBytes, 1024);
                    const int kj = t * 8 + j;                               // 16-token step within the chunk
                    const uint32_t a_hi = tmem + (kj >> 1) * 32 + (kj & 1) * 8;
                    umma::mma_ts(tmem + kUmmaOutCol, a_hi, b, idesc_pv, kj > 0);
                    umma::mma_ts(tmem + kUmmaOutCol, a_hi + 16, b, idesc_pv, true);
                }
                umma::commit(bar_done + 8 * i);
            }
            __syncwarp();
            if (lane == 0 && t == 1) DA_TRACE_STAMP(kUmmaTraceBase + unit_index, 15);
            if (i + 2 < n_loads) {
                ok = wait(bar_done + 8 * i);
                if (lane == 0) DA_TRACE_STAMP(kUmmaTraceBase + unit_index, 14);
                if (ok) issue(i + 2);
            }
        }
        if (lane == 0) {
            if (ok) {
                umma::commit(bar_o);
            } else {
                record_status(p.status, DA_ERR_TIMEOUT);
                *sm_abort = 1;
            }
        }
    } else {
        // ------------------------------------------------------------ query rows, softmax, epilogue
        // Two threads per row: thread (quarter q, lane) of column half hh = warp / 4 owns row
        // r = 32 q + lane, the even (hh = 0) or odd (hh = 1) 32-token groups of the logits, and
        // half of the output columns.
        const int hh = warp >> 2;
        const int r = (warp & 3) * 32 + lane;                               // row of the tile = lane of tensor memory
        const int sl = r / G, h = r % G;
        const bool valid = sl < nseq;
        const int seq = u.seq + (valid ? sl : 0);
        {
            // 64 dims of row r of Q, 8 chunks of 16 bytes, into the swizzled K-major tile
            const uint4* src = reinterpret_cast<const uint4*>(p.q + ((int64_t)seq * p.num_q_heads + g * G + h) * D) + hh * 8;
            uint4 v[8];
#pragma unroll
            for (int c = 0; c < 8; ++c) v[c] = valid ? __ldg(src + c) : make_uint4(0u, 0u, 0u, 0u);
#pragma unroll
            for (int c = 0; c < 8; ++c) {
                const uint32_t off = hh * kUmmaHalfBytes + r * 128 + ((c ^ (r & 7)) << 4);
                *reinterpret_cast<uint4*>(gbase + off) = v[c];
            }
            asm volatile("fence.proxy.async.shared::cta;" ::: "memory");     // visible to the tensor core's reads
        }
        if (tid == 0) DA_TRACE_STAMP(kUmmaTraceBase + unit_index, 5);
        block_sync(1, kUmmaThreads);

        const SeqInfo si = p.seq_info[seq];
        bool dead = p.run_mask != nullptr && __ldg(p.run_mask + seq) == 0;  // masked row: an empty record
        if (valid && __ldg(p.seq_lens + seq) != si.seq_len) {                // stale plan: void the result, report it
            dead = true;
            if (hh == 0) record_status(p.status, DA_ERR_STALE_PLAN);
        }

        const uint32_t lane_base = tmem + ((uint32_t)((warp & 3) * 32) << 16);
        const int n_chunks = (n_tok + 31) >> 5;
        uint32_t sa[32], sb[32];
        bool ok = true;
        float mx = -INFINITY, l = 0.f;
        // pass 1: the row maximum, tile by tile as the logits arrive
        for (int t = 0; t < n_tiles && ok; ++t) {
            ok = mbar_wait(bar_done + 8 * t, 0);
            if (!ok) break;
            if (tid == 0 && t == n_tiles - 1) DA_TRACE_STAMP(kUmmaTraceBase + unit_index, 6);
            umma::fence_after_thread_sync();
            const int c0 = 4 * t + hh, c1 = c0 + 2;                          // this thread's two groups of the tile
            if (c0 < n_chunks) umma::ld32(lane_base + c0 * 32, sa);
            if (c1 < n_chunks) umma::ld32(lane_base + c1 * 32, sb);
            umma::wait_ld();
            if (c0 < n_chunks) {
#pragma unroll
                for (int i = 0; i < 32; ++i)
                    if (c0 * 32 + i < n_tok) mx = fmaxf(mx, __uint_as_float(sa[i]));
            }
            if (c1 < n_chunks) {
#pragma unroll
                for (int i = 0; i < 32; ++i)
                    if (c1 * 32 + i < n_tok) mx = fmaxf(mx, __uint_as_float(sb[i]));
            }
        }
        sm_part[hh * 128 + r] = mx;
        block_sync(2, kUmmaSoftmaxThreads);
        const float m2 = fmaxf(sm_part[r], sm_part[128 + r]) * p.scale_log2;   // the scale is positive
        block_sync(2, kUmmaSoftmaxThreads);                                  // sm_part is reused for the sums
        if (tid == 0) DA_TRACE_STAMP(kUmmaTraceBase + unit_index, 7);
        // pass 2: weights, written back over the logits as bf16 high and low parts
        auto weights = [&](const uint32_t (&s)[32], int c) {
            uint32_t hi[16], lo[16];
#pragma unroll
            for (int i = 0; i < 16; ++i) {
                float p0 = 0.f, p1 = 0.f;
                if (c * 32 + 2 * i < n_tok) p0 = ex2f(fmaf(__uint_as_float(s[2 * i]), p.scale_log2, -m2));
                if (c * 32 + 2 * i + 1 < n_tok) p1 = ex2f(fmaf(__uint_as_float(s[2 * i + 1]), p.scale_log2, -m2));
                l += p0 + p1;
                const uint32_t b0 = __float_as_uint(p0), b1 = __float_as_uint(p1);
                const float r0 = p0 - __uint_as_float(b0 & 0xffff0000u);     // exact
                const float r1 = p1 - __uint_as_float(b1 & 0xffff0000u);
                hi[i] = __byte_perm(b0, b1, 0x7632);                         // upper halves: element 2i low, 2i+1 high
                lo[i] = __byte_perm(__float_as_uint(r0), __float_as_uint(r1), 0x7632);
            }
            // the group's 32 logit columns become 16 columns of high parts, 16 of low parts
            umma::st16(lane_base + c * 32, hi);
            umma::st16(lane_base + c * 32 + 16, lo);
        };
        for (int t = 0; t < n_tiles && ok; ++t) {
            const int c0 = 4 * t + hh, c1 = c0 + 2;
            if (c0 < n_chunks) umma::ld32(lane_base + c0 * 32, sa);
            if (c1 < n_chunks) umma::ld32(lane_base + c1 * 32, sb);
            umma::wait_ld();
            if (c0 < n_chunks) weights(sa, c0);
            if (c1 < n_chunks) weights(sb, c1);
            umma::wait_st();
            umma::fence_before_thread_sync();
            mbar_arrive(bar_p + 8 * t);                                       // this tile's P V may start
            if (tid == 0 && t < 2) DA_TRACE_STAMP(kUmmaTraceBase + unit_index, 16 + t);
        }
        if (tid == 0) DA_TRACE_STAMP(kUmmaTraceBase + unit_index, 8);
        sm_part[hh * 128 + r] = l;
        if (ok) ok = mbar_wait(bar_o, 0);
        if (tid == 0) DA_TRACE_STAMP(kUmmaTraceBase + unit_index, 11);
        block_sync(2, kUmmaSoftmaxThreads);                                  // the sums of both halves are visible
        if (ok) {
            umma::fence_after_thread_sync();
            // Every MMA has completed: the Q tile and the stages are free.  This thread's half
            // of the row is staged there and leaves with one bulk copy.
            const int RF = rec_floats(G, D);
            float* const rec = p.ws + ((int64_t)(si.slot_base + u.split_index) * p.num_kv_heads + g) * RF;
            uint8_t* const row = gbase + r * kUmmaOutRowBytes + hh * 256;
#pragma unroll 1
            for (int c = 0; c < 2; ++c) {
                umma::ld32(lane_base + kUmmaOutCol + hh * 64 + c * 32, sa);
                umma::wait_ld();
#pragma unroll
                for (int i = 0; i < 8; ++i) {
                    uint4 v = make_uint4(sa[4 * i], sa[4 * i + 1], sa[4 * i + 2], sa[4 * i + 3]);
                    if (dead) v = make_uint4(0u, 0u, 0u, 0u);
                    *reinterpret_cast<uint4*>(row + c * 128 + i * 16) = v;
                }
            }
            asm volatile("fence.proxy.async.shared::cta;" ::: "memory");     // visible to the bulk copy's reads
            if (valid) {
                bulk_store_s2g(rec + h * D + hh * 64, smem_u32(row), 256);
                if (hh == 0)
                    __stcg(reinterpret_cast<float2*>(rec + G * D) + h,
                           dead ? make_float2(-INFINITY, 0.f) : make_float2(m2, sm_part[r] + sm_part[128 + r]));
            }
            bulk_store_commit_and_wait_read();
        } else if (lane == 0 && *sm_abort == 0) {
            record_status(p.status, DA_ERR_TIMEOUT);
        }
        if (tid == 0) DA_TRACE_STAMP(kUmmaTraceBase + unit_index, 12);
    }
    // the next unit reuses shared memory, tensor memory and the barriers
    umma::fence_before_thread_sync();
    __syncthreads();
    umma::fence_after_thread_sync();
    if (tid == 0) DA_TRACE_STAMP(kUmmaTraceBase + unit_index, 13);
  }
    pdl_launch_dependents();
    if (warp == kUmmaSoftmaxWarps) umma::tmem_dealloc(tmem, kUmmaTmemCols);
}

__global__ void __launch_bounds__(kUmmaThreads, 1)
decode_attn_umma_prefix_kernel(const KernelParams p, const __grid_constant__ CUtensorMap k_map,
                               const __grid_constant__ CUtensorMap v_map, const int G, const int n_units)
{
    extern __shared__ uint8_t smem_raw[];
    umma_prefix_units(p, &k_map, &v_map, G, blockIdx.x, gridDim.x, n_units, smem_raw);
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

// Units [0, n_prefix_units) of the plan's work list, dealt round-robin to `grid` blocks (at most one per SM).
inline int umma_prefix_launch(const decode_attn_shape_t& s, int G, const KernelParams& kp, unsigned n_prefix_units,
                              unsigned grid, cudaStream_t stream)
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
    cfg.gridDim = dim3(grid, 1, 1);
    cfg.blockDim = dim3(kUmmaThreads, 1, 1);
    cfg.dynamicSmemBytes = (size_t)kUmmaSmemBytes;
    cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    if (cudaLaunchKernelEx(&cfg, decode_attn_umma_prefix_kernel, kp, kmap, vmap, G, (int)n_prefix_units) != cudaSuccess) {
        (void)cudaGetLastError();
        return DA_ERR_CUDA;
    }
    return DA_OK;
}

}  // namespace da
