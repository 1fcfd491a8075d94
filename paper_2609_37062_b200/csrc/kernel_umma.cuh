// Shared-prefix units on the tcgen05 tensor cores.
//
// A prefix every sequence of the batch shares (few-shot prompts served from a
// prefix cache) is a dense contraction: for one KV head, the query rows of
// many sequences meet the same K/V pages.  One unit = (KV head, block of
// 128 / G sequences, a range of prefix tokens): the 128 query rows form the M
// dimension of the MMAs, so a prefix page is fetched once for 128 rows.  The
// range is walked in tiles of 128 tokens, pipelined over two logit buffers and
// two output buffers in tensor memory:
//
//   S_j = Q K_j^T  128 x 128 x 128, accumulators in tensor memory columns
//                  [128 b, 128 b + 128), b = j mod 2: row r of S in lane r,
//                  token t of the tile in column t
//   softmax        two threads per row.  They exchange the maxima of their
//                  halves, so each has the exact maximum m_j of the row over
//                  the tile, then turns its 64 logits into
//                  p = 2^(s * scale * log2 e - m_j)
//   P_j            must keep more than bf16 precision: the upper 16 bits of p
//                  and the upper 16 bits of the (exact) remainder are written
//                  back over the logits, two bf16 per column: the 32 logit
//                  columns of 32 tokens become 16 columns of high parts and
//                  16 of low parts.  What is dropped is below 2^-16 of p.
//   O_j = P_j V_j  A = P_j from tensor memory, B = V tile from shared memory
//                  with the head dimension contiguous; high and low parts
//                  accumulate into one 128 x 128 fp32 tile in columns
//                  [256 + 128 b, 256 + 128 b + 128)
//   merge          while the tensor core works on tile j + 1, the softmax
//                  threads fetch O_j and fold it into their running state
//                  (M, L, acc[64]) in registers with the usual log-sum-exp
//                  rescale, in ascending tile order
//   record         row r = (sequence r / G, head r mod G) goes to that
//                  sequence's record of this prefix chunk, unnormalised, with
//                  (M, L), exactly like any other split; the combine kernel
//                  merges prefix and suffix splits.  Each thread stages its
//                  half row in shared memory and sends it with one bulk copy.
//
// Threads: eight warps for softmax, merge and epilogue, two per 32 lanes of
// tensor memory (each takes one half of a row's 128 tokens and one half of
// the output columns, and moves them with few, large tensor-memory accesses:
// a 64-column load, two 32-column stores); one warp whose first lane issues the MMAs,
// always the one - the next Q K^T or the next P V - whose inputs are ready;
// one warp that issues the TMA boxes.  K tiles and V tiles each go through a
// ring of two 32 KB stages, filled independently (a K stage comes back after
// Q K^T, a V stage only after P V); a stage is handed back by the
// tcgen05.commit of the MMAs that read it.  Blocks are persistent (one per SM: the buffers fill
// tensor memory); the barriers are invalidated and set up again for every
// unit.  Every wait is bounded and also ends when another thread of the block
// has given up; the block then records DA_ERR_TIMEOUT, skips its records and
// still frees its tensor memory.
#pragma once

#include <cuda_fp16.h>

#include <type_traits>

#include "kernel_mma.cuh"
#include "umma.cuh"

namespace da {

constexpr int kUmmaTraceBase = 2048;              // debug timelines: rows of this kernel's units
constexpr int kUmmaSoftmaxWarps = 8;              // 8 or 16 (measured: no faster): warps w, w + 4, ... share 32 lanes of tensor memory
constexpr int kUmmaThreadsPerRow = kUmmaSoftmaxWarps / 4;
constexpr int kUmmaGroupsPerThread = 4 / kUmmaThreadsPerRow;     // 32-token groups of a tile a thread owns
constexpr int kUmmaOutColsPerThread = 128 / kUmmaThreadsPerRow;  // output columns a thread owns
constexpr int kUmmaSoftmaxThreads = kUmmaSoftmaxWarps * 32;
constexpr int kUmmaMmaWarp = kUmmaSoftmaxWarps;       // lane 0 issues the MMAs
constexpr int kUmmaLoadWarp = kUmmaSoftmaxWarps + 1;  // issues the TMA boxes
constexpr int kUmmaThreads = kUmmaSoftmaxThreads + 64;
constexpr int kUmmaRows = 128;                    // query rows of a unit
constexpr int kUmmaTileTokens = 128;
constexpr int kUmmaHalfBytes = 128 * 128;         // 128 rows x 64 dims of bf16
constexpr int kUmmaTileBytes = 2 * kUmmaHalfBytes;   // [half of the head dim][row][64 dims]
constexpr int kUmmaStages = 4;
constexpr int kUmmaMiscBytes = 8192;              // barriers, small state, the threads' row maxima and sums
constexpr int kUmmaSmemBytes = (1 + kUmmaStages) * kUmmaTileBytes + kUmmaMiscBytes + 1024 /* alignment */;
static_assert(kUmmaSmemBytes > 114 * 1024, "two of these blocks, each wanting all of tensor memory, must not share an SM");
constexpr int kUmmaTmemCols = 512;
constexpr int kUmmaOutCol = 256;                  // first column of the output buffers
constexpr int kUmmaOutRowBytes = 128 * 4 + 16;    // a staged output row; the pad spreads the rows over the banks

// Any group of up to 16 heads: a unit takes floor(128 / G) sequences, rows past them stay empty.
inline bool umma_supports(int D, int G) { return D == 128 && G >= 1 && G <= 16; }

__device__ __forceinline__ void bulk_store_s2g(void* dst, uint32_t src, uint32_t bytes)
{
    asm volatile("cp.async.bulk.global.shared::cta.bulk_group [%0], [%1], %2;" ::"l"(dst), "r"(src), "r"(bytes) : "memory");
}
__device__ __forceinline__ void bulk_store_commit_and_wait_read()
{
    asm volatile("cp.async.bulk.commit_group;" ::: "memory");
    asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory");
}

// Bounded wait that also ends when the block has given up elsewhere.  The first thread to run
// out of time raises the flag.
__device__ __forceinline__ bool umma_wait(uint32_t bar, uint32_t parity, volatile int* abort_flag)
{
    if (mbar_try_wait(bar, parity)) return true;
    const long long t0 = clock64();
    while (!mbar_try_wait(bar, parity)) {
        if (*abort_flag != 0) return false;
        if (clock64() - t0 > kWaitLimitCycles) {
            *abort_flag = 1;
            return false;
        }
    }
    return true;
}

// Shared-prefix units first_unit, first_unit + unit_stride, ... < n_units, one after the other, by
// the threads of a block (kUmmaThreads).  smem_raw: at least kUmmaSmemBytes of dynamic shared memory.
template <bool F16>
__device__ __forceinline__ void umma_prefix_units(const KernelParams& p, const CUtensorMap* k_map, const CUtensorMap* v_map,
                                                  const int G, const int first_unit, const int unit_stride,
                                                  const int n_units, uint8_t* smem_raw)
{
    constexpr int D = 128;
    constexpr int NS = kUmmaStages;
    const uint32_t raw = smem_u32(smem_raw);
    const uint32_t base = (raw + 1023u) & ~1023u;
    uint8_t* const gbase = smem_raw + (base - raw);
    const uint32_t q_base = base;
    const uint32_t ring_base = base + kUmmaTileBytes;                       // stage s at ring_base + s * tile bytes
    uint8_t* const ring_ptr = gbase + kUmmaTileBytes;
    const uint32_t bar_base = base + (1 + NS) * kUmmaTileBytes;
    // full[4]: a tile has landed; empty[4]: the MMAs reading it have completed; s_ready[2]: the logits
    // of a tile are complete; p_ready[2]: its weights are written (all softmax threads); o_ready[2]:
    // its output tile is complete (and its weights consumed); o_free[2]: the output tile was read;
    // m_ready[2][4]: the threads that share 32 rows have published their maxima of the tile
    const uint32_t bar_full = bar_base, bar_empty = bar_base + 32, bar_s = bar_base + 64, bar_p = bar_base + 80;
    const uint32_t bar_o = bar_base + 96, bar_ofree = bar_base + 112, bar_m = bar_base + 128;   // m_ready: [2][4]
    constexpr int kBarriers = 24;
    uint8_t* const sm_misc = gbase + (bar_base - base);
    volatile uint32_t* const sm_tmem = reinterpret_cast<volatile uint32_t*>(sm_misc + 320);
    volatile int* const sm_abort = reinterpret_cast<volatile int*>(sm_misc + 324);
    constexpr int TPR = kUmmaThreadsPerRow, GP = kUmmaGroupsPerThread, OC = kUmmaOutColsPerThread;
    volatile float* const sm_max = reinterpret_cast<volatile float*>(sm_misc + 512);   // [2 buffers][TPR][128 rows]
    float* const sm_l = reinterpret_cast<float*>(sm_misc + 512 + 2 * TPR * 128 * 4);   // [TPR][128]: the threads' shares of the row sums

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
    if (warp == kUmmaMmaWarp) umma::tmem_alloc(smem_u32(const_cast<uint32_t*>(sm_tmem)), kUmmaTmemCols);
    umma::fence_before_thread_sync();
    __syncthreads();
    umma::fence_after_thread_sync();
    const uint32_t tmem = *sm_tmem;
    // Only this block's own state was touched so far.  As the second of a pair (see KernelParams)
    // the kernel was let go only after the first one's own wait, so what precedes the pair is
    // complete and nothing the first one writes is read here.
    if (!p.late_wait) pdl_wait_primary();

    for (int unit_index = first_unit; unit_index < n_units && *sm_abort == 0; unit_index += unit_stride) {
        const decode_attn_unit_t u = load_unit(p.units, unit_index);
        const int g = u.kv_head & 0xffff, nseq = u.kv_head >> 16;
        const int n_tok = u.tok_end - u.tok_begin;                          // whole pages
        const int n_pages = n_tok >> 4;
        const int T = (n_tok + kUmmaTileTokens - 1) / kUmmaTileTokens;      // tiles
        if (tid == 0) {
            DA_TRACE_CLOCK(kUmmaTraceBase + unit_index, 0);
            // the barriers serve one unit: set up again for each (the block is past a barrier here,
            // nobody is still waiting on the previous unit's, and every arrival on them has landed)
            if (unit_index != first_unit)
                for (int i = 0; i < kBarriers; ++i) mbar_inval(bar_base + 8 * i);
            for (int i = 0; i < 2 * NS + 2; ++i) mbar_init(bar_base + 8 * i, 1);      // full, empty, s_ready
            for (int i = 0; i < 2; ++i) mbar_init(bar_p + 8 * i, kUmmaSoftmaxThreads);
            for (int i = 0; i < 2; ++i) mbar_init(bar_o + 8 * i, 1);
            for (int i = 0; i < 2; ++i) mbar_init(bar_ofree + 8 * i, kUmmaSoftmaxThreads);
            for (int i = 0; i < 8; ++i) mbar_init(bar_m + 8 * i, 32 * kUmmaThreadsPerRow);
            mbar_init_fence();
        }
        __syncthreads();

        if (warp == kUmmaLoadWarp) {
            // -------------------------------------------------------- TMA: K tiles and V tiles
            // K_j goes to stage (2j) % 4, V_j to stage (2j + 1) % 4, so K and V each have a ring of
            // two.  A K stage comes back as soon as Q K^T of its tile has completed, a V stage only
            // after P V: the two rings are filled independently (K at most two tiles ahead of V), so
            // that K_{j+2} never queues behind the wait for V_{j+1}'s stage.  Page ids are fetched 32
            // at a time (four tiles), one batch ahead, off the path of the copies.
            const uint64_t l2_policy = l2_policy_evict_first();
            const int32_t* bt = p.block_table + (int64_t)u.seq * p.max_pages_per_seq;
            const int ts = p.tile_shift, tile0 = u.tok_begin >> 4;         // 16-token tiles: 1 << ts per page
            const int pg = (lane >> 1) & 7, hf = lane & 1;                  // lane j < 16: box (16 tokens j / 2, half j % 2)
            auto fetch_ids = [&](int batch) {                               // lane l: 16-token tile 32 batch + l
                const int i = batch * 32 + lane;
                return i < n_pages ? __ldg(bt + ((tile0 + i) >> ts)) : 0;
            };
            int cb = 0;                                                     // batch of the V cursor
            int ids0 = fetch_ids(0), ids1 = fetch_ids(1);
            auto issue = [&](int j, int n, const CUtensorMap* map) {
                const int st = n % NS;
                const int idx = j * 8 + pg;                                 // 16-token tile of this lane's box
                int page_id = __shfl_sync(0xffffffffu, (j >> 2) == cb ? ids0 : ids1, ((j & 3) * 8 + pg) & 31);
                if (idx >= n_pages) {
                    // past the range: fetched from outside the pool, which the TMA unit fills with zeros
                    page_id = (int)p.num_pages;
                } else if ((unsigned)page_id >= (unsigned)p.num_pages) {    // never hand TMA a page outside the pool
                    record_status(p.status, DA_ERR_BAD_PAGE);
                    page_id = 0;
                }
                const int slot0 = ((tile0 + idx) & ((1 << ts) - 1)) << 4;
                const uint32_t bar = bar_full + 8 * st;
                if (lane == 0) mbar_arrive_expect_tx(bar, kUmmaTileBytes);
                __syncwarp();
                if (lane < 16)
                    tma_load_4d(ring_base + st * kUmmaTileBytes + hf * kUmmaHalfBytes + pg * 2048, map, bar, hf * 64, slot0, g,
                                page_id, l2_policy);
            };
            auto stage_free = [&](int n) {                                  // the stage of copy n was handed back
                if (n < NS) return true;
                bool f = false;
                if (lane == 0) f = mbar_test_wait(bar_empty + 8 * (n % NS), ((n / NS) - 1) & 1);
                return __shfl_sync(0xffffffffu, (int)f, 0) != 0;
            };
            int jk = 0, jv = 0;                                             // next K tile, next V tile
            long long t_idle = clock64();
            while (jv < T) {
                bool did = false;
                if (jk < T && jk - jv < 2 && stage_free(2 * jk)) {
                    issue(jk, 2 * jk, k_map);
                    ++jk;
                    did = true;
                }
                if (jv < jk && stage_free(2 * jv + 1)) {
                    issue(jv, 2 * jv + 1, v_map);
                    ++jv;
                    did = true;
                    if ((jv & 3) == 0) {                                    // the V cursor enters the next batch
                        ids0 = ids1;
                        ++cb;
                        ids1 = fetch_ids(cb + 1);
                    }
                }
                if (did) {
                    t_idle = clock64();
                } else {
                    bool stop = false;
                    if (lane == 0) {
                        stop = *sm_abort != 0;
                        if (!stop && clock64() - t_idle > kWaitLimitCycles) {
                            *sm_abort = 1;
                            stop = true;
                        }
                    }
                    if (__shfl_sync(0xffffffffu, (int)stop, 0) != 0) break;
                }
            }
        } else if (warp == kUmmaMmaWarp) {
            // -------------------------------------------------------- MMAs (one lane)
            block_sync(1, kUmmaSoftmaxThreads + 32);                        // Q is in shared memory
            if (lane == 0) {
                constexpr uint32_t idesc_qk = umma::instr_desc_16(128, 128, false, F16);
                constexpr uint32_t idesc_pv = umma::instr_desc_16(128, 128, true, F16);
                bool ok = true;
                // Descriptors differ only in their address field (16-byte units, the low 14 bits):
                // stepping through a tile adds a constant to the low word.
                const uint64_t q_desc = umma::smem_desc_sw128(q_base, 16, 1024);
                const uint64_t k_desc0 = umma::smem_desc_sw128(ring_base, 16, 1024);
                const uint64_t v_desc0 = umma::smem_desc_sw128(ring_base, kUmmaHalfBytes, 1024);
                constexpr uint32_t kStageUnits = kUmmaTileBytes >> 4, kHalfUnits = kUmmaHalfBytes >> 4;
                // S_j = Q K_j^T into logit buffer j % 2
                auto qk = [&](int j) {
                    const int st = (2 * j) % NS, b = j & 1;
                    if (j < 8) DA_TRACE_CLOCK(kUmmaTraceBase + 512 + unit_index, j);
                    umma::fence_after_thread_sync();
                    const uint64_t kd = k_desc0 + (uint64_t)(st * kStageUnits);
#pragma unroll
                    for (int ks = 0; ks < D / 16; ++ks) {
                        const uint32_t off = (ks >> 2) * kHalfUnits + (ks & 3) * 2;      // 32 bytes a step, then the other half
                        umma::mma_ss(tmem + b * 128, q_desc + off, kd + off, idesc_qk, ks > 0);
                    }
                    umma::commit(bar_empty + 8 * st);
                    umma::commit(bar_s + 8 * b);
                };
                // O_j = P_j V_j into output buffer j % 2
                auto pv = [&](int j) {
                    const int st = (2 * j + 1) % NS, b = j & 1;
                    if (j < 8) DA_TRACE_CLOCK(kUmmaTraceBase + 512 + unit_index, 8 + j);
                    umma::fence_after_thread_sync();
                    const uint64_t vd = v_desc0 + (uint64_t)(st * kStageUnits);
                    const int ksteps = min(8, (n_tok - j * kUmmaTileTokens) >> 4);
                    const uint32_t pd = tmem + b * 128, od = tmem + kUmmaOutCol + b * 128;
#pragma unroll
                    for (int k = 0; k < 8; ++k) {
                        if (k < ksteps) {
                            // 16 tokens: two groups of 8 rows, 128 bytes a row (2 KB a step); the weights'
                            // high parts 8 columns a step within a 32-column group, the low parts 16 further
                            const uint32_t a_hi = pd + (k >> 1) * 32 + (k & 1) * 8;
                            umma::mma_ts(od, a_hi, vd + k * 128, idesc_pv, k > 0);
                            umma::mma_ts(od, a_hi + 16, vd + k * 128, idesc_pv, true);
                        }
                    }
                    if (j < 8) DA_TRACE_CLOCK(kUmmaTraceBase + 512 + unit_index, 16 + j);
                    umma::commit(bar_empty + 8 * st);
                    umma::commit(bar_o + 8 * b);
                };
                // Whichever of the next P V and the next Q K^T has its inputs is issued; the tensor
                // core never waits for this thread to finish waiting for something else.
                //   Q K^T of tile j: K_j landed; logit buffer free = P V of tile j - 2 complete
                //   P V of tile j:   its weights written; V_j landed; output buffer read (tile j - 2 folded in)
                int nq = 0, np = 0;
                long long t_idle = clock64();
                while (np < T) {
                    bool did = false;
                    // Q K^T first: the logits feed the softmax threads, which are the busier side;
                    // P V only gates the fold and the logit buffer two tiles on.
                    if (nq < T) {
                        const int j = nq, n = 2 * j, b = j & 1;
                        if (mbar_test_wait(bar_full + 8 * (n % NS), (n / NS) & 1) &&
                            (j < 2 || (np > j - 2 && mbar_test_wait(bar_o + 8 * b, ((j - 2) >> 1) & 1)))) {
                            qk(j);
                            ++nq;
                            did = true;
                        }
                    }
                    if (!did && np < nq) {
                        const int j = np, n = 2 * j + 1, b = j & 1;
                        if (mbar_test_wait(bar_p + 8 * b, (j >> 1) & 1) && mbar_test_wait(bar_full + 8 * (n % NS), (n / NS) & 1) &&
                            (j < 2 || mbar_test_wait(bar_ofree + 8 * b, ((j - 2) >> 1) & 1))) {
                            pv(j);
                            ++np;
                            did = true;
                        }
                    }
                    if (did) {
                        t_idle = clock64();
                    } else if (*sm_abort != 0 || clock64() - t_idle > kWaitLimitCycles) {
                        *sm_abort = 1;
                        ok = false;
                        break;
                    }
                }
                // nothing may arrive on a barrier after the unit: the last two stages' hand-backs
                if (ok) {
                    const int n1 = 2 * T - 1, n0 = 2 * T - 2;
                    ok = umma_wait(bar_empty + 8 * (n1 % NS), (n1 / NS) & 1, sm_abort);
                    if (ok) ok = umma_wait(bar_empty + 8 * (n0 % NS), (n0 / NS) & 1, sm_abort);
                }
            }
        } else {
            // -------------------------------------------------------- query rows, softmax, merge, epilogue
            // TPR threads per row: thread (quarter q, lane) of part hh = warp / 4 owns row r = 32 q +
            // lane, tokens [64 hh, 64 hh + 64) of a tile's logits, and output columns
            // [OC hh, OC hh + OC).
            const int hh = warp >> 2;
            const int r = (warp & 3) * 32 + lane;                           // row of the tile = lane of tensor memory
            const int sl = r / G, h = r % G;
            const bool valid = sl < nseq;
            const int seq = u.seq + (valid ? sl : 0);
            {
                // this thread's share of row r of Q, chunks of 16 bytes, into the swizzled K-major tile
                constexpr int NC = 16 / TPR;
                const uint4* src = reinterpret_cast<const uint4*>(p.q + ((int64_t)seq * p.num_q_heads + g * G + h) * D) + hh * NC;
                uint4 v[NC];
#pragma unroll
                for (int c = 0; c < NC; ++c) v[c] = valid ? __ldg(src + c) : make_uint4(0u, 0u, 0u, 0u);
#pragma unroll
                for (int c = 0; c < NC; ++c) {
                    const int ci = hh * NC + c;                                 // chunk of the row: half ci / 8, chunk ci % 8
                    const uint32_t off = (ci >> 3) * kUmmaHalfBytes + r * 128 + (((ci & 7) ^ (r & 7)) << 4);
                    *reinterpret_cast<uint4*>(gbase + off) = v[c];
                }
                asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); // visible to the tensor core's reads
            }
            block_sync(1, kUmmaSoftmaxThreads + 32);
            if (tid == 0) DA_TRACE_CLOCK(kUmmaTraceBase + unit_index, 1);

            const SeqInfo si = p.seq_info[seq];
            bool dead = p.run_mask != nullptr && __ldg(p.run_mask + seq) == 0;   // masked row: an empty record
            if (valid && __ldg(p.seq_lens + seq) != si.seq_len) {            // stale plan: void the result, report it
                dead = true;
                if (hh == 0) record_status(p.status, DA_ERR_STALE_PLAN);
            }

            const uint32_t lane_base = tmem + ((uint32_t)((warp & 3) * 32) << 16);
            float acc[OC];
#pragma unroll
            for (int i = 0; i < OC; ++i) acc[i] = 0.f;
            float M = -INFINITY, L = 0.f;       // running maximum (log2 domain), this thread's share of the row sum
            float m_prev = 0.f, l_prev = 0.f;   // of the tile whose output is still to be folded in
            static_assert(32 * GP == OC && (OC == 64 || OC == 32), "a thread owns as many consecutive logit columns as output columns");
            uint32_t sg[OC];                        // logits of the thread's columns; also the output tile on its way in
            auto ld_cols = [&](uint32_t taddr) { umma::ld_cols(taddr, sg); };
            bool ok = true;

            // folds tile i's output into the running state
            auto fold = [&](int i) {
                const int b = i & 1;
                ok = umma_wait(bar_o + 8 * b, (i >> 1) & 1, sm_abort);
                if (!ok) return;
                if (tid == 0 && i < 8) DA_TRACE_CLOCK(kUmmaTraceBase + 1024 + unit_index, 16 + i);
                umma::fence_after_thread_sync();
                const uint32_t oc = lane_base + kUmmaOutCol + b * 128 + hh * OC;
                ld_cols(oc);
                umma::wait_ld();
                umma::fence_before_thread_sync();
                mbar_arrive(bar_ofree + 8 * b);                              // the buffer may be overwritten
                const float Mn = fmaxf(M, m_prev);
                const float a = ex2f(M - Mn), c = ex2f(m_prev - Mn);        // M = -inf at first: a = 0
#pragma unroll
                for (int q = 0; q < OC / 32; ++q)
#pragma unroll
                    for (int k = 0; k < 32; ++k)
                        acc[32 * q + k] = fmaf(acc[32 * q + k], a, __uint_as_float(sg[32 * q + k]) * c);
                L = fmaf(L, a, l_prev * c);
                M = Mn;
                if (tid == 0 && i < 8) DA_TRACE_CLOCK(kUmmaTraceBase + 1024 + unit_index, 24 + i);
            };

            for (int j = 0; j < T && ok; ++j) {
                const int b = j & 1;
                const int tok0 = j * kUmmaTileTokens;                        // first token of the tile within the unit
                const int n_here = min(kUmmaTileTokens, n_tok - tok0);      // a multiple of 16
                ok = umma_wait(bar_s + 8 * b, (j >> 1) & 1, sm_abort);
                if (!ok) break;
                if (tid == 0 && j == 0) DA_TRACE_CLOCK(kUmmaTraceBase + unit_index, 2);
                if (tid == 0 && j < 8) DA_TRACE_CLOCK(kUmmaTraceBase + 1024 + unit_index, j);
                umma::fence_after_thread_sync();
                const uint32_t sc = lane_base + b * 128;
                float m2 = 0.f, lsum = 0.f;
                // A full tile (all but possibly a unit's last) needs no per-token bounds.
                auto softmax_tile = [&](auto full_tag) {
                    constexpr bool FULL = decltype(full_tag)::value;
                    // pass 1: the maximum of this thread's logits; the row's other parts are exchanged
                    // through shared memory (their logits may not be read once they start writing weights)
                    float mx = -INFINITY;
                    ld_cols(sc + hh * OC);                                  // columns OC hh .. OC hh + OC - 1
                    umma::wait_ld();
#pragma unroll
                    for (int q = 0; q < GP; ++q)
#pragma unroll
                        for (int i = 0; i < 32; ++i)
                            if (FULL || (hh * GP + q) * 32 + i < n_here) mx = fmaxf(mx, __uint_as_float(sg[32 * q + i]));
                    sm_max[(b * TPR + hh) * 128 + r] = mx;
                    const uint32_t bm = bar_m + 8 * (b * 4 + (warp & 3));       // of the warps sharing these rows
                    mbar_arrive(bm);
                    ok = umma_wait(bm, (j >> 1) & 1, sm_abort);
                    if (!ok) return;
#pragma unroll
                    for (int q = 0; q < TPR; ++q) mx = fmaxf(mx, sm_max[(b * TPR + q) * 128 + r]);
                    m2 = mx * p.scale_log2;                                      // the scale is positive
                    // pass 2: this thread's weights, written back over the logits as bf16 high and low parts
                    auto weights = [&](const uint32_t* s, int col0) {
                        uint32_t hl[32];                                     // 16 high parts, then 16 low parts
#pragma unroll
                        for (int i = 0; i < 16; ++i) {
                            float p0 = 0.f, p1 = 0.f;
                            if (FULL || col0 + 2 * i < n_here) p0 = ex2f(fmaf(__uint_as_float(s[2 * i]), p.scale_log2, -m2));
                            if (FULL || col0 + 2 * i + 1 < n_here) p1 = ex2f(fmaf(__uint_as_float(s[2 * i + 1]), p.scale_log2, -m2));
                            lsum += p0 + p1;
                            if (F16) {
                                // fp16 inputs: the weights are fp16 too, rounded, and so is the remainder
                                const __half2 ph = __floats2half2_rn(p0, p1);
                                const float2 pf = __half22float2(ph);
                                const __half2 pl = __floats2half2_rn(p0 - pf.x, p1 - pf.y);
                                hl[i] = *reinterpret_cast<const uint32_t*>(&ph);
                                hl[16 + i] = *reinterpret_cast<const uint32_t*>(&pl);
                            } else {
                                const uint32_t b0 = __float_as_uint(p0), b1 = __float_as_uint(p1);
                                const float r0 = p0 - __uint_as_float(b0 & 0xffff0000u);   // exact
                                const float r1 = p1 - __uint_as_float(b1 & 0xffff0000u);
                                hl[i] = __byte_perm(b0, b1, 0x7632);             // upper halves: element 2i low, 2i+1 high
                                hl[16 + i] = __byte_perm(__float_as_uint(r0), __float_as_uint(r1), 0x7632);
                            }
                        }
                        // the group's 32 logit columns become 16 columns of high parts, 16 of low parts, in one
                        // store: fewer, larger accesses to tensor memory disturb the MMAs less (four stores of
                        // 16 columns per thread and tile instead of two of 32 cost the kernel 2 us of 20)
                        umma::st32(sc + col0, hl);
                    };
#pragma unroll
                    for (int q = 0; q < GP; ++q) weights(sg + 32 * q, (hh * GP + q) * 32);
                };
                if (n_here == kUmmaTileTokens)
                    softmax_tile(std::true_type());
                else
                    softmax_tile(std::false_type());
                if (!ok) break;
                umma::wait_st();
                umma::fence_before_thread_sync();
                mbar_arrive(bar_p + 8 * b);                                   // this tile's P V may start
                if (tid == 0 && j < 8) DA_TRACE_CLOCK(kUmmaTraceBase + 1024 + unit_index, 8 + j);
                // while it runs, fold in the tile before
                if (j >= 1) fold(j - 1);
                m_prev = m2;
                l_prev = lsum;
            }
            if (ok) fold(T - 1);
            if (tid == 0) DA_TRACE_CLOCK(kUmmaTraceBase + unit_index, 3);
            // the row sum is the sum of the threads' shares, added in a fixed order
            sm_l[hh * 128 + r] = L;
            block_sync(2, kUmmaSoftmaxThreads);
            if (ok) {
                // Every MMA has completed and every tile was consumed: the ring is free.  This
                // thread's half of the row is staged there and leaves with one bulk copy.
                const int RF = rec_floats(G, D);
                float* const rec = p.ws + ((int64_t)(si.slot_base + u.split_index) * p.num_kv_heads + g) * RF;
                uint8_t* const row = ring_ptr + r * kUmmaOutRowBytes + hh * (OC * 4);
#pragma unroll
                for (int i = 0; i < OC / 4; ++i) {
                    float4 v = make_float4(acc[4 * i], acc[4 * i + 1], acc[4 * i + 2], acc[4 * i + 3]);
                    if (dead) v = make_float4(0.f, 0.f, 0.f, 0.f);
                    *reinterpret_cast<float4*>(row + i * 16) = v;
                }
                asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); // visible to the bulk copy's reads
                if (valid) {
                    bulk_store_s2g(rec + h * D + hh * OC, smem_u32(row), OC * 4);
                    if (hh == 0) {
                        float ls = sm_l[r];
#pragma unroll
                        for (int q = 1; q < TPR; ++q) ls += sm_l[q * 128 + r];
                        __stcg(reinterpret_cast<float2*>(rec + G * D) + h, dead ? make_float2(-INFINITY, 0.f) : make_float2(M, ls));
                    }
                }
                bulk_store_commit_and_wait_read();
            }
            if (tid == 0) DA_TRACE_CLOCK(kUmmaTraceBase + unit_index, 4);
        }
        // the next unit reuses shared memory, tensor memory and the barriers
        umma::fence_before_thread_sync();
        __syncthreads();
        umma::fence_after_thread_sync();
    }
    if (tid == 0 && *sm_abort != 0) record_status(p.status, DA_ERR_TIMEOUT);
    if (p.late_wait) pdl_wait_primary();                      // this kernel's end then implies the first one's
    pdl_launch_dependents();
    if (warp == kUmmaMmaWarp) umma::tmem_dealloc(tmem, kUmmaTmemCols);
}

template <bool F16>
__global__ void __launch_bounds__(kUmmaThreads, 1)
decode_attn_umma_prefix_kernel(const KernelParams p, const __grid_constant__ CUtensorMap k_map,
                               const __grid_constant__ CUtensorMap v_map, const int G, const int n_units)
{
    extern __shared__ uint8_t smem_raw[];
    umma_prefix_units<F16>(p, &k_map, &v_map, G, blockIdx.x, gridDim.x, n_units, smem_raw);
}

// ---------------------------------------------------------------- host side

typedef void (*umma_kernel_t)(const KernelParams, const CUtensorMap, const CUtensorMap, const int, const int);

inline int umma_prepare(bool f16, umma_kernel_t* fn_out)
{
    umma_kernel_t fn = f16 ? decode_attn_umma_prefix_kernel<true> : decode_attn_umma_prefix_kernel<false>;
    *fn_out = fn;
    if (cudaFuncSetAttribute(fn, cudaFuncAttributeMaxDynamicSharedMemorySize, kUmmaSmemBytes) != cudaSuccess) {
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
    umma_kernel_t fn;
    int rc = umma_prepare(s.kv_dtype == DA_DTYPE_FP16, &fn);
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
    if (cudaLaunchKernelEx(&cfg, fn, kp, kmap, vmap, G, (int)n_prefix_units) != cudaSuccess) {
        (void)cudaGetLastError();
        return DA_ERR_CUDA;
    }
    return DA_OK;
}

}  // namespace da
