// Tensor-core split-KV partial kernel with TMA-staged pages.
//
// A block is four consumer warps and one producer warp.  It works through
// its share of the work list - units block_begin[b] .. block_begin[b+1], packed
// by the planner so that every block gets about the same cost (a unit is one
// sequence, one KV head, a run of pages) - without ever draining its
// pipeline: the producer keeps filling the ring of stages with the next
// unit's pages while the consumers finish the previous unit.  With a grid as
// large as the work list every block has one unit.  The producer turns block-table entries into
// TMA tile loads (cp.async.bulk.tensor over a 4-D map [dim, slot, head, page]
// of each pool): one 16-token tile of one KV head - a whole page, or 16 slots
// of a larger one; "page" below means such a tile - lands in shared memory as
// 16 rows x 128 bytes per half of the head dimension, 128-byte swizzled, with
// an mbarrier counting the bytes.  A stage is four pages of K and of V; a
// ring of stages keeps tens of KB in flight per block with no register cost.
//
// Consumer warp w owns page w of every stage.  With the query heads of the
// group as the N dimension (padded to 8) and the 16 tokens of the page as M,
//   S^T[16 x 8]  = K_page[16 x D] . Q^T[D x 8]          (mma.sync m16n8k16 bf16, fp32 accumulate)
//   O^T[D x 8]  += V_page^T[D x 16] . P^T[16 x 8]
// so K and V are the A operands straight out of shared memory (ldmatrix, the
// V tile transposed on the way) and each K/V byte is used for all heads of
// the group.  Softmax runs on the accumulator fragments in fp32: running max
// and sum per head, column maxima over the 8 lanes that share a head by warp
// shuffles, exponentials in the base-2 domain.
//
// P must keep more than bf16 precision.  For groups of up to 4 heads the
// query is duplicated into columns 4..7, so those columns see the same logits
// and carry the low part: columns 0..3 hold bf16(p), columns 4..7 hold
// bf16(p - bf16(p)), and one PV mma accumulates both; the two halves are
// added at the end.  For groups of 5..8 heads the low part takes a second
// mma; groups of 9..16 heads are two such tiles of 8 columns side by side
// (every K and V fragment feeds both).  P^T reaches the B-operand layout
// with one movmatrix transpose per 8x8 block.
//
// Every wait on an mbarrier is bounded; a wait that gives up records
// DA_ERR_TIMEOUT and the block drains without touching the tiles.
#pragma once

#include <cuda.h>
#include <cuda_fp16.h>

#include "common.cuh"

namespace da {

constexpr int kMmaConsumerWarps = 4;
constexpr int kMmaThreads = (kMmaConsumerWarps + 1) * 32;
constexpr int kPagesPerStage = kMmaConsumerWarps;

enum MmaMode { kModeAttend = 0, kModeProbe = 1, kModeGather = 2 };

template <int D, bool DUP>
struct MmaCfg {
    static constexpr int kHalves = D / 64;                      // 128-byte column blocks per row
    static constexpr int kBoxBytes = 16 * 128;                  // one TMA box: 16 rows x 128 B
    static constexpr int kPageBytes = kHalves * kBoxBytes;      // one page of one tensor
    static constexpr int kTensorBytes = kPagesPerStage * kPageBytes;
    static constexpr int kStageBytes = 2 * kTensorBytes;        // K then V
    static constexpr int kColsOut = 4;                          // output columns a warp hands to the block merge at a time
    static constexpr int kStages = (D == 128) ? 3 : 6;         // two blocks per SM must fit
    static constexpr int kBarrierBytes = 1024;                  // barriers + small state, keeps tiles 1 KB aligned
    static constexpr int kScratchBytes = kMmaConsumerWarps * kColsOut * D * 4 + 256;   // warps' results for the merge
    static constexpr int kSmemBytes = kStages * kStageBytes + kBarrierBytes + kScratchBytes + 1024;  // + alignment slack
};

// ---------------------------------------------------------------- PTX wrappers

__device__ __forceinline__ void tma_load_4d(uint32_t dst, const CUtensorMap* map, uint32_t bar, int c0, int c1,
                                            int c2, int c3, uint64_t l2_policy)
{
    asm volatile(
        "cp.async.bulk.tensor.4d.shared::cluster.global.tile.mbarrier::complete_tx::bytes.L2::cache_hint"
        " [%0], [%1, {%3, %4, %5, %6}], [%2], %7;"
        ::"r"(dst), "l"(map), "r"(bar), "r"(c0), "r"(c1), "r"(c2), "r"(c3), "l"(l2_policy)
        : "memory");
}

// The same box brought into L2 only: no shared memory, no barrier, nothing to wait for.
__device__ __forceinline__ void tma_prefetch_l2_4d(const CUtensorMap* map, int c0, int c1, int c2, int c3, uint64_t l2_policy)
{
    asm volatile("cp.async.bulk.prefetch.tensor.4d.L2.global.tile.L2::cache_hint [%0, {%1, %2, %3, %4}], %5;"
                 ::"l"(map), "r"(c0), "r"(c1), "r"(c2), "r"(c3), "l"(l2_policy)
                 : "memory");
}

// A line of global memory asked into L2: a hint, nothing to wait for.
__device__ __forceinline__ void prefetch_l2(const void* ptr)
{
    asm volatile("prefetch.global.L2 [%0];" ::"l"(ptr) : "memory");
}

__device__ __forceinline__ void tma_prefetch_descriptor(const CUtensorMap* map)
{
    asm volatile("prefetch.tensormap [%0];" ::"l"(map) : "memory");
}

// K/V bytes are read once per step: mark their L2 lines first in line for
// eviction so the stream does not push out the work list, block tables,
// partial records and instructions that are reused.
__device__ __forceinline__ uint64_t l2_policy_evict_first()
{
    uint64_t pol;
    asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(pol));
    return pol;
}

__device__ __forceinline__ void ldsm_x4(uint32_t addr, uint32_t (&r)[4])
{
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3])
                 : "r"(addr));
}

__device__ __forceinline__ void ldsm_x4_trans(uint32_t addr, uint32_t (&r)[4])
{
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3])
                 : "r"(addr));
}

__device__ __forceinline__ uint32_t movmatrix_trans(uint32_t a)
{
    uint32_t d;
    asm("movmatrix.sync.aligned.m8n8.trans.b16 %0, %1;" : "=r"(d) : "r"(a));
    return d;
}

// The 16-bit input type of q, K and V: bf16, or fp16 (template parameter F16 of the kernel).  P
// takes the same type, because both operands of an mma must have it.
template <bool F16>
struct In16;

template <>
struct In16<false> {
    // a pure function of its register operands: left non-volatile so the compiler may interleave
    // independent mma chains with the surrounding arithmetic
    static __device__ __forceinline__ void mma(float (&c)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1)
    {
        asm("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
            : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
            : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
    }
    static __device__ __forceinline__ uint32_t pack(float lo, float hi)
    {
        __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
        return *reinterpret_cast<uint32_t*>(&v);
    }
    static __device__ __forceinline__ float low(uint32_t v) { return __uint_as_float(v << 16); }
    static __device__ __forceinline__ float high(uint32_t v) { return __uint_as_float(v & 0xffff0000u); }
};

template <>
struct In16<true> {
    static __device__ __forceinline__ void mma(float (&c)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1)
    {
        asm("mma.sync.aligned.m16n8k16.row.col.f32.f16.f16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
            : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
            : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
    }
    static __device__ __forceinline__ uint32_t pack(float lo, float hi)
    {
        __half2 v = __floats2half2_rn(lo, hi);
        return *reinterpret_cast<uint32_t*>(&v);
    }
    static __device__ __forceinline__ float low(uint32_t v) { return __low2float(*reinterpret_cast<const __half2*>(&v)); }
    static __device__ __forceinline__ float high(uint32_t v) { return __high2float(*reinterpret_cast<const __half2*>(&v)); }
};

// Byte offset, inside one 16 x 128 B box written by TMA with the 128-byte
// swizzle, of 16-byte chunk `chunk` (0..7) of row `row` (0..15).
__device__ __forceinline__ uint32_t swz(int row, int chunk) { return row * 128 + ((chunk ^ (row & 7)) << 4); }

// ---------------------------------------------------------------- the kernel

struct MmaExtra {
    // kModeProbe:  checksum [n_units] (uint32).  kModeGather: dense K / V rows of one sequence.
    uint32_t* checksum;
    __nv_bfloat16* k_out;
    __nv_bfloat16* v_out;
    int32_t gather_seq;
};

// MASKED: the variant launched when a RUN mask is given (ordinary attention plans): it can deal the
// work list out again among the blocks; kept apart so that launches without a mask carry none of it.
// WIDE: groups of 9..16 query heads: two 8-column tiles of heads per K/V tile instead of one.
template <int D, bool DUP, int MODE, bool PREFIX, bool F16 = false, bool MASKED = false, bool WIDE = false>
__global__ void __launch_bounds__(kMmaThreads, 2) decode_attn_mma_kernel(const KernelParams p,
                                                                      const __grid_constant__ CUtensorMap k_map,
                                                                      const __grid_constant__ CUtensorMap v_map,
                                                                      const int G, const MmaExtra ex)
{
    using Cfg = MmaCfg<D, DUP>;
    using In = In16<F16>;
    constexpr int NS = Cfg::kStages;
    constexpr int KSTEPS = D / 16;
    constexpr int COLS = Cfg::kColsOut;
    constexpr int kConsumerThreads = kMmaConsumerWarps * 32;
    constexpr int NT = WIDE ? 2 : 1;                          // 8-column tiles of query heads
    static_assert(!(WIDE && (DUP || PREFIX)), "wide groups: ordinary units, low parts of P in a second mma");

    extern __shared__ uint8_t smem_raw[];
    const uint32_t raw = smem_u32(smem_raw);
    const uint32_t base = (raw + 1023u) & ~1023u;             // 1 KB aligned: the swizzle atom
    uint8_t* const gbase = smem_raw + (base - raw);
    const uint32_t bar_base = base + NS * Cfg::kStageBytes;   // full[NS], empty[NS]
    volatile int* const sm_flags = reinterpret_cast<volatile int*>(gbase + NS * Cfg::kStageBytes + 256);
    int* const sm_ticket = reinterpret_cast<int*>(gbase + NS * Cfg::kStageBytes + 256 + 16);
    // Launches with a RUN mask take their units from a queue (see below): the producer warp hands the
    // consumers the descriptors of the units it drew through a small ring, sm_pub counting the entries
    // published so far.  The producer is never more than NS + 1 units ahead of the consumers.
    constexpr int kRing = 8;
    static_assert(kRing > NS + 1, "the ring of drawn units is too short for the stages in flight");
    volatile int* const sm_pub = reinterpret_cast<volatile int*>(gbase + NS * Cfg::kStageBytes + 256 + 32);
    int4* const sm_ring = reinterpret_cast<int4*>(gbase + NS * Cfg::kStageBytes + 384);   // [kRing][2], 256 bytes
    static_assert(384 + 32 * kRing <= Cfg::kBarrierBytes, "the unit ring overlaps the scratch");
    float* const sm_wo = reinterpret_cast<float*>(gbase + NS * Cfg::kStageBytes + Cfg::kBarrierBytes);   // [4][COLS][D]
    float* const sm_wm = sm_wo + kMmaConsumerWarps * COLS * D;                                           // [4][COLS]
    float* const sm_wl = sm_wm + kMmaConsumerWarps * COLS;                                               // [4][COLS]

    if (MODE == kModeAttend && p.fused && (int)blockIdx.x >= p.n_work_blocks) {
        // a merge block of a fused launch: no tiles, no pipeline
        pdl_launch_dependents();
        pdl_wait_primary();                                   // `out` may still be in use by the kernel before
        fused_merge_blocks<D>(p, G, kMmaThreads, sm_wo, sm_ticket);
        return;
    }
    // this block's units: a range of the work list (the planner's packing), or just unit blockIdx.x
    int ubeg, uend;
    if (p.block_begin != nullptr) {
        ubeg = __ldg(p.block_begin + blockIdx.x);
        uend = __ldg(p.block_begin + blockIdx.x + 1);
    } else {
        const int n_units = p.grid_exit ? p.header->n_units : p.n_units;
        ubeg = blockIdx.x;
        uend = min(n_units, (int)blockIdx.x + 1);
    }
    // With a RUN mask the planner's packing is off: it could not know which rows read nothing, and a
    // block whose rows all run would set the step's time.  Such launches (the MASKED variant) hand
    // the units out through a queue instead: in cost order, block b starts with the unit of rank b
    // and then draws the next rank with one atomic add on a counter the plan owns, one unit ahead
    // of its consumers.  A unit whose row is masked costs the drawing warp a look at the mask byte
    // and the stores of its empty result.  No block waits for another, and a unit's result does not
    // depend on which block ran it.  The last block to have drawn puts the counters back to zero,
    // so the launch can be repeated (or replayed from a graph) as it is.
    const bool queued = MASKED && MODE == kModeAttend && p.run_mask != nullptr && p.queue != nullptr &&
                        (p.grid_exit ? p.may_rank != 0 : p.n_ranked > 0);
    const int n_ranked = queued ? (p.grid_exit ? p.header->n_ranked : p.n_ranked) : 0;
    if (queued) {
        ubeg = (int)blockIdx.x < n_ranked ? __ldg(p.unit_rank + blockIdx.x).x : 0;
        uend = (int)blockIdx.x < n_ranked ? ubeg + 1 : ubeg;
    }
    const bool idle = ubeg >= uend;                           // no units: a surplus block of a capacity launch
    if (idle) {
        // Stream order reaches the kernels behind this one through the waits of this launch's
        // blocks; should every block be surplus, block 0 still carries it.
        if (blockIdx.x == 0) pdl_wait_primary();
        return;
    }
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    if (tid == 0) DA_TRACE_STAMP(blockIdx.x, 0);

    if (tid == 0) {
        tma_prefetch_descriptor(&k_map);
        tma_prefetch_descriptor(&v_map);
        for (int s = 0; s < NS; ++s) {
            mbar_init(bar_base + 8 * s, 1);                             // full: the producer's expect_tx arrival
            mbar_init(bar_base + 8 * (NS + s), kMmaConsumerWarps);      // empty: one arrival per consumer warp
        }
        sm_flags[0] = 0;
        sm_pub[0] = 0;
        mbar_init_fence();
    }
    decode_attn_unit_t u = load_unit(p.units, ubeg);
    __syncthreads();
    if (tid == 0) DA_TRACE_STAMP(blockIdx.x, 1);
    // Everything above touched only the plan's own work list and kernel parameters.  What the
    // kernel launched before this one may have produced (q, new K/V rows, lengths, page
    // mappings) is read only past this point; with a programmatic dependency the lines above
    // overlap that kernel's tail.
    if (MODE != kModeGather && warp == 0 && p.hint_first_pages != 0) {     // (the gather-only probe issues the same hints)
        // Hints, while the kernel before this one drains (from a consumer warp, which has nothing to do
        // until the first stage lands; the producer goes straight to its wait): the pages that will fill the ring first
        // are asked into L2.  The mask and the page ids read here may be about to change; they steer
        // prefetches only (the loads below read them again, behind the wait), and an L2 prefetch
        // of the wrong line is harmless.
        const int unit_pages = (u.tok_end - u.tok_begin + 15) >> 4;
        const int np = min(unit_pages, p.hint_first_pages);
        const bool masked = p.run_mask != nullptr && (u.kv_head >> 16) == 0 && __ldcg(p.run_mask + u.seq) == 0;
        // The same goes for what the first unit's critical path reads right behind the wait - the
        // producer's first 64 page ids, the group's query rows, the sequence's length: behind the
        // wait they are L2 hits instead of trips to DRAM (1.5 -> 0.6 us from the end of the wait to the
        // first copy on a single long sequence).  L2 is where writes of the kernel before arrive, so
        // a line brought in early is never stale there.
        if (!masked) {
            const int32_t* const row = p.block_table + (int64_t)u.seq * p.max_pages_per_seq;
            const int first = (u.tok_begin >> 4) >> p.tile_shift;
            const int last = ((u.tok_begin >> 4) + min(unit_pages, 64) - 1) >> p.tile_shift;      // entries first .. last
            if (unit_pages > 0 && lane * 32 <= last - first) prefetch_l2(row + first + lane * 32);
            if (MODE == kModeAttend) {
                const char* const qrows = reinterpret_cast<const char*>(
                    p.q + ((int64_t)u.seq * p.num_q_heads + (u.kv_head & 0xffff) * G) * D);
                if (lane * 128 < G * D * 2) prefetch_l2(qrows + lane * 128);
                if (lane == 31) prefetch_l2(p.seq_lens + u.seq);
            }
        }
        if (lane < np && !masked) {
            const int tile = (u.tok_begin >> 4) + lane;
            const int id = __ldcg(p.block_table + (int64_t)u.seq * p.max_pages_per_seq + (tile >> p.tile_shift));
            if ((unsigned)id < (unsigned)p.num_pages) {
                const int slot0 = (tile & ((1 << p.tile_shift) - 1)) << 4;
                const uint64_t hint_policy = l2_policy_evict_first();
#pragma unroll
                for (int hf = 0; hf < Cfg::kHalves; ++hf) {
                    tma_prefetch_l2_4d(&k_map, hf * 64, slot0, u.kv_head & 0xffff, id, hint_policy);
                    tma_prefetch_l2_4d(&v_map, hf * 64, slot0, u.kv_head & 0xffff, id, hint_policy);
                }
            }
        }
    }
    pdl_wait_primary();
    if (tid == 0) DA_TRACE_STAMP(blockIdx.x, 7);
    if (p.early_trigger) pdl_launch_dependents();             // first of a pair: see KernelParams

    if (warp == kMmaConsumerWarps) {
        // ------------------------------------------------------------ producer
        if (lane == 0) DA_TRACE_STAMP(blockIdx.x, 8);
        const uint64_t l2_policy = l2_policy_evict_first();
        const int ts = p.tile_shift;                          // 16-token tiles per page, as a shift
        uint32_t git = 0;                                     // stages issued so far, over all units
        bool alive = true;
        // range of a unit as this launch sees it: a masked row (or, in the gather mode, another
        // sequence) has nothing to read
        auto unit_end = [&](const decode_attn_unit_t& x) {
            int e = x.tok_end;
            if (MODE == kModeAttend && p.run_mask != nullptr && (x.kv_head >> 16) == 0 && __ldg(p.run_mask + x.seq) == 0)
                e = x.tok_begin;
            if (MODE == kModeGather && x.seq != ex.gather_seq) e = x.tok_begin;
            return e;
        };
        auto first_ids = [&](const decode_attn_unit_t& x, int end) {
            const int np = (end - x.tok_begin + 15) >> 4;
            const int32_t* t = p.block_table + (int64_t)x.seq * p.max_pages_per_seq;
            return (lane < np) ? __ldg(t + (((x.tok_begin >> 4) + lane) >> ts)) : 0;
        };
        // ---- launches with a RUN mask: the queue (see the top of the kernel)
        const int nb = p.n_work_blocks;
        int published = 0;
        // hands a drawn unit (or, with valid = false, the end of the queue) to the consumers
        auto publish = [&](const decode_attn_unit_t& x, bool valid) {
            if (lane == 0) {
                int4* const e = sm_ring + 2 * (published % kRing);
                e[0] = make_int4(valid ? x.seq : -1, x.kv_head, x.tok_begin, x.tok_end);
                e[1] = make_int4(x.slot, x.seq_len, x.split_index, x.n_splits);
                __threadfence_block();
                sm_pub[0] = published + 1;
            }
            ++published;
        };
        auto draw = [&]() {
            int j = 0;
            if (lane == 0) j = nb + atomicAdd(p.queue, 1);
            return __shfl_sync(0xffffffffu, j, 0);
        };
        // the unit of rank j: 1 if it runs (x, its end and its first page ids are set), 0 if it reads
        // nothing (its empty result is written here, by this warp), -1 if the queue is exhausted
        auto candidate = [&](int j, decode_attn_unit_t& x, int& end, int& ids) {
            if (j >= n_ranked) return -1;
            x = load_unit(p.units, __ldg(p.unit_rank + j).x);
            end = unit_end(x);
            if (end > x.tok_begin) {
                ids = first_ids(x, end);
                return 1;
            }
            if (x.tok_end == x.seq_len && x.tok_end > x.tok_begin && (x.kv_head >> 16) == 0)
                append_new_row<D>(p, x.seq, x.kv_head, x.seq_len, lane);     // a masked row still writes its K/V
            block_finish_empty<D>(p, x, G, lane, 32);
            return 0;
        };
        int t1 = 0, ids_first = 0;
        bool have = true;
        if (queued) {
            // the block's first unit is the one of rank blockIdx.x, whose descriptor is in hand: its mask
            // byte and its first page ids are asked for together
            ids_first = first_ids(u, u.tok_end);
            t1 = unit_end(u);
            int r = 1;
            if (t1 <= u.tok_begin) {
                if (u.tok_end == u.seq_len && u.tok_end > u.tok_begin && (u.kv_head >> 16) == 0)
                    append_new_row<D>(p, u.seq, u.kv_head, u.seq_len, lane);
                block_finish_empty<D>(p, u, G, lane, 32);
                r = 0;
            }
            while (r == 0) r = candidate(draw(), u, t1, ids_first);
            have = r == 1;
            publish(u, have);
        } else {
            t1 = unit_end(u);
            ids_first = first_ids(u, t1);
        }
        for (int uid = ubeg; (queued ? have : uid < uend) && alive; ++uid) {
            const bool has_next = queued || uid + 1 < uend;
            decode_attn_unit_t nu = u;
            if (!queued && has_next) nu = load_unit(p.units, uid + 1);    // lands while this unit streams
            int nt1 = 0, nids_first = 0;
            bool next_ready = false;
            int next_state = 0;                                           // queue: 0 still looking, 1 found, -1 none left
            // The look for the next unit is a chain of dependent reads (the counter, the rank list,
            // the descriptor and the mask byte, the first page ids).  It advances one link per stage
            // issued - each link's loads are asked for in one step and used in the next - so that
            // the chain's latency passes while the warp waits for stages anyway.
            int q_link = 0, q_j = 0, q_masked = 0;
            int2 q_rank = make_int2(0, 0);
            auto queue_step = [&]() {
                if (q_link == 0) {
                    if (lane == 0) q_j = nb + atomicAdd(p.queue, 1);
                    q_link = 1;
                } else if (q_link == 1) {
                    q_j = __shfl_sync(0xffffffffu, q_j, 0);
                    if (q_j >= n_ranked) {
                        next_state = -1;
                        publish(nu, false);
                    } else {
                        q_rank = __ldg(p.unit_rank + q_j);
                        q_link = 2;
                    }
                } else if (q_link == 2) {
                    nu = load_unit(p.units, q_rank.x);
                    q_masked = q_rank.y >= 0 ? (int)(__ldg(p.run_mask + q_rank.y) == 0) : 0;
                    q_link = 3;
                } else {
                    nt1 = q_masked ? nu.tok_begin : nu.tok_end;
                    if (nt1 > nu.tok_begin) {
                        nids_first = first_ids(nu, nt1);
                        next_state = 1;
                        publish(nu, true);
                    } else {
                        if (nu.tok_end == nu.seq_len && nu.tok_end > nu.tok_begin && (nu.kv_head >> 16) == 0)
                            append_new_row<D>(p, nu.seq, nu.kv_head, nu.seq_len, lane);
                        block_finish_empty<D>(p, nu, G, lane, 32);
                        q_link = 0;
                    }
                }
            };
            const int b = u.seq, g = u.kv_head & 0xffff;   // (a shared-prefix unit keeps its block size in the high half)
            const int t0 = u.tok_begin;
            const int n_pages = (t1 - t0 + 15) >> 4;
            const int n_iters = (n_pages + kPagesPerStage - 1) / kPagesPerStage;
            const int32_t* bt = p.block_table + (int64_t)b * p.max_pages_per_seq;
            const int tile0 = t0 >> 4;                                    // first 16-token tile of the unit
            int ids_next = ids_first;
            int ids_cur = 0;
            for (int it = 0; it < n_iters; ++it, ++git) {
                if ((it & 7) == 0) {                                      // 32 page ids per 8 stages, one batch ahead
                    ids_cur = ids_next;
                    const int nxt = (it + 8) * kPagesPerStage + lane;
                    ids_next = (nxt < n_pages) ? __ldg(bt + ((tile0 + nxt) >> ts)) : 0;
                }
                const int s = git % NS;
                if (git >= (uint32_t)NS) {
                    bool ok = true;
                    if (lane == 0) ok = mbar_wait(bar_base + 8 * (NS + s), ((git / NS) & 1) ^ 1, p.wait_limit);
                    ok = __shfl_sync(0xffffffffu, (int)ok, 0) != 0;
                    if (!ok) {
                        if (lane == 0) {
                            record_status(p.status, DA_ERR_TIMEOUT);
                            sm_flags[0] = 1;
                        }
                        alive = false;
                        break;
                    }
                }
                if (p.debug_drop_loads) continue;                         // test hook: nothing arrives, the waits run out
                const int pages_here = min(kPagesPerStage, n_pages - it * kPagesPerStage);
                const uint32_t full = bar_base + 8 * s;
                if (lane == 0) mbar_arrive_expect_tx(full, (uint32_t)pages_here * 2u * Cfg::kPageBytes);
                __syncwarp();
                // lane j issues one box: page j / (2*halves), tensor (K, V), half of the head dimension
                constexpr int OPS_PER_PAGE = 2 * Cfg::kHalves;
                const int pg = lane / OPS_PER_PAGE;
                const int which = (lane % OPS_PER_PAGE) / Cfg::kHalves;   // 0: K, 1: V
                const int hf = lane % Cfg::kHalves;
                int page_id = __shfl_sync(0xffffffffu, ids_cur, ((it & 7) * kPagesPerStage + pg) & 31);
#ifdef DA_TRACE
                if (git == 0 && lane == 0 && page_id >= 0) DA_TRACE_STAMP(blockIdx.x, 9);
#endif
                if (lane < pages_here * OPS_PER_PAGE) {
                    if ((unsigned)page_id >= (unsigned)p.num_pages) {     // never hand TMA a page outside the pool
                        record_status(p.status, DA_ERR_BAD_PAGE);
                        page_id = 0;
                    }
                    const uint32_t dst = base + s * Cfg::kStageBytes + which * Cfg::kTensorBytes +
                                         pg * Cfg::kPageBytes + hf * Cfg::kBoxBytes;
                    const int slot0 = ((tile0 + it * kPagesPerStage + pg) & ((1 << ts) - 1)) << 4;   // of the tile within its page
                    tma_load_4d(dst, which ? &v_map : &k_map, full, hf * 64, slot0, g, page_id, l2_policy);
                    if (git == 0 && lane == 0) DA_TRACE_STAMP(blockIdx.x, 2);
#ifdef DA_TRACE
                    if (lane == 0 && uid - ubeg == 1 && it == 0) DA_TRACE_CLOCK(blockIdx.x, 30);   // second unit's first copy
#endif
                }
                if (queued) {
                    // One link of the look at the queue per stage issued, so that a run of masked rows
                    // does not hold the loads up - and only over the unit's last stages: a block that
                    // draws its next unit early takes it away from a block that has nothing to do.
                    constexpr int kQueueLead = 8;
                    if (next_state == 0 && n_iters - it <= kQueueLead) queue_step();
                } else if (has_next && !next_ready) {                     // this unit is under way: look ahead
                    nt1 = unit_end(nu);
                    nids_first = first_ids(nu, nt1);
                    next_ready = true;
                }
            }
            if (queued) {
                while (next_state == 0 && alive) queue_step();
                if (next_state == 0) publish(nu, false);                  // a wait was given up: the consumers leave too
                have = next_state == 1;
            } else if (has_next && !next_ready) {
                nt1 = unit_end(nu);
                nids_first = first_ids(nu, nt1);
            }
            u = nu;
            t1 = nt1;
            ids_first = nids_first;
        }
        if (queued && lane == 0) {
            // this block has drawn its last: count it; whoever is last puts the counters back
            const int participants = min(nb, n_ranked);
            if (atomicAdd(p.queue + 1, 1) == participants - 1) {
                atomicExch(p.queue, 0);
                atomicExch(p.queue + 1, 0);
            }
        }
        return;
    }

    // ---------------------------------------------------------------- consumers
    const int r = lane >> 2, c = lane & 3;
    const bool lo_role = DUP && (c >= 2);
    uint32_t git = 0;                                         // stages consumed so far, over all units
    // what a unit needs before its first tile: lengths / mask of its sequence and Q^T as B
    // fragments (column n = r of tile nt is query head 8 nt + r, or r mod 4 when duplicated); fetched
    // one unit ahead
    struct Pre {
        int dev_len;
        int masked;
        uint32_t qb[KSTEPS][NT][2];
    };
    auto prefetch = [&](const decode_attn_unit_t& x, Pre& o) {
        o.dev_len = x.seq_len;
        o.masked = 0;
        if (MODE == kModeAttend) {
            o.dev_len = __ldg(p.seq_lens + x.seq);
            if (p.run_mask != nullptr) o.masked = __ldg(p.run_mask + x.seq) == 0;
#pragma unroll
            for (int nt = 0; nt < NT; ++nt) {
                const int head = DUP ? (r & 3) : nt * 8 + r;
                const bool live = head < G;
                const uint32_t* qrow = reinterpret_cast<const uint32_t*>(
                    p.q + ((int64_t)x.seq * p.num_q_heads + (x.kv_head & 0xffff) * G + (live ? head : 0)) * D);
#pragma unroll
                for (int ks = 0; ks < KSTEPS; ++ks) {
                    o.qb[ks][nt][0] = live ? __ldg(qrow + ks * 8 + c) : 0u;         // dims ks*16 + 2c, +1
                    o.qb[ks][nt][1] = live ? __ldg(qrow + ks * 8 + 4 + c) : 0u;     // dims ks*16 + 8 + 2c, +1
                }
            }
        }
    };
    // queue (launches with a RUN mask): entry `need - 1` of the producer's ring has been published
    auto wait_published = [&](int need) {
        if (sm_pub[0] < need) {
            const long long c0 = clock64();
            while (sm_pub[0] < need)
                if (sm_flags[0] != 0 || clock64() - c0 > p.wait_limit) return false;
        }
        __threadfence_block();
        return true;
    };
    auto ring_unit = [&](int k) {
        const int4 a = sm_ring[2 * (k % kRing)], b2 = sm_ring[2 * (k % kRing) + 1];
        decode_attn_unit_t x;
        x.seq = a.x; x.kv_head = a.y; x.tok_begin = a.z; x.tok_end = a.w;
        x.slot = b2.x; x.seq_len = b2.y; x.split_index = b2.z; x.n_splits = b2.w;
        return x;
    };
    if (queued) {
        // the block's first unit is the first one of its draws whose row runs, if any does
        const bool late = block_sync_or(1, kConsumerThreads, !wait_published(1));
        if (late) {
            if (tid == 0) {
                record_status(p.status, DA_ERR_TIMEOUT);
                sm_flags[0] = 1;
            }
            return;
        }
        u = ring_unit(0);
        if (u.seq < 0) return;
    }
    Pre cur;
    prefetch(u, cur);
    for (int uid = ubeg; queued || uid < uend; ++uid) {
        bool last_unit = !queued && uid + 1 >= uend;          // (queue: known once the next entry has been published)
        decode_attn_unit_t nu = u;
        if (!queued && !last_unit) nu = load_unit(p.units, uid + 1);      // lands while this unit is consumed
        Pre nxt = cur;
#ifdef DA_TRACE
        // per-unit cycle stamps of a block's first four units: slots 10 + 4k .. 13 + 4k = the unit is taken up, its
        // first stage has landed, its streaming loop is done, it is finished; slots 26 .. 29 split the second unit's
        // finish (before / behind the vote barrier, states in the scratch, behind the second barrier)
        const int trace_k = uid - ubeg;
        if (tid == 0 && trace_k < 4) DA_TRACE_CLOCK(blockIdx.x, 10 + trace_k * 4);
#endif
        const int b = u.seq, g = u.kv_head & 0xffff;
        const int nseq = u.kv_head >> 16;                                  // > 0: a shared-prefix unit
        const int t0 = u.tok_begin;
        int t1 = u.tok_end;
        // Invariant 2 (never run on stale lengths): the device length was fetched ahead and is
        // compared at the end of the unit, off the critical path; a mismatch voids the unit's
        // result.  Reads stay inside the planned range and page ids are range-checked.
        const int dev_len = cur.dev_len;
        if (cur.masked && nseq == 0) t1 = t0;                              // masked row reads no KV
        if (MODE == kModeGather && b != ex.gather_seq) t1 = t0;
        const int n_pages = (t1 - t0 + 15) >> 4;
        const int n_iters = (n_pages + kPagesPerStage - 1) / kPagesPerStage;
        uint32_t (&qb)[KSTEPS][NT][2] = cur.qb;

        if (PREFIX && MODE == kModeAttend && nseq > 0) {
            // -------------------------------------------------------- shared-prefix unit
            // The pages of this chunk are the same physical pages for every sequence of the block,
            // so the block's query rows (sequence j, head h -> column j*G + h, 16 columns in two
            // tiles) are attended in one pass: each K/V tile is read once for all of them.  P keeps
            // its low part through a second mma.
            constexpr int NT = 2;
            const int spb = 16 / G;                                         // sequences per block
            uint32_t pq[KSTEPS][NT][2];
#pragma unroll
            for (int nt = 0; nt < NT; ++nt) {
                const int col = nt * 8 + r, j = col / G, h = col - j * G;
                const bool live = j < nseq && j < spb;
                const uint32_t* qrow = reinterpret_cast<const uint32_t*>(
                    p.q + ((int64_t)(b + (live ? j : 0)) * p.num_q_heads + g * G + h) * D);
#pragma unroll
                for (int ks = 0; ks < KSTEPS; ++ks) {
                    pq[ks][nt][0] = live ? __ldg(qrow + ks * 8 + c) : 0u;
                    pq[ks][nt][1] = live ? __ldg(qrow + ks * 8 + 4 + c) : 0u;
                }
            }
            float pacc[D / 16][NT][4];
            float pm[NT][2], pl[NT][2];
#pragma unroll
            for (int nt = 0; nt < NT; ++nt) {
                pm[nt][0] = pm[nt][1] = -INFINITY;
                pl[nt][0] = pl[nt][1] = 0.f;
#pragma unroll
                for (int mt = 0; mt < D / 16; ++mt) pacc[mt][nt][0] = pacc[mt][nt][1] = pacc[mt][nt][2] = pacc[mt][nt][3] = 0.f;
            }
            bool pfailed = false;
            for (int it = 0; it < n_iters; ++it, ++git) {
                const int s = git % NS;
                if (!mbar_wait(bar_base + 8 * s, (git / NS) & 1, p.wait_limit) || sm_flags[0] != 0) {
                    if (lane == 0) {
                        record_status(p.status, DA_ERR_TIMEOUT);
                        sm_flags[0] = 1;
                    }
                    pfailed = true;
                    break;
                }
                const int page_idx = it * kPagesPerStage + warp;
                if (page_idx < n_pages) {                                   // prefix pages are always full
                    const uint32_t kpage = base + s * Cfg::kStageBytes + warp * Cfg::kPageBytes;
                    const uint32_t vpage = kpage + Cfg::kTensorBytes;
                    float sacc[NT][4];
#pragma unroll
                    for (int nt = 0; nt < NT; ++nt) sacc[nt][0] = sacc[nt][1] = sacc[nt][2] = sacc[nt][3] = 0.f;
                    const int arow = (lane & 7) + ((lane >> 3) & 1) * 8;
                    const int achk = lane >> 4;
#pragma unroll
                    for (int ks = 0; ks < KSTEPS; ++ks) {
                        uint32_t a[4];
                        ldsm_x4(kpage + (ks >> 2) * Cfg::kBoxBytes + swz(arow, (ks & 3) * 2 + achk), a);
#pragma unroll
                        for (int nt = 0; nt < NT; ++nt) In::mma(sacc[nt], a, pq[ks][nt][0], pq[ks][nt][1]);
                    }
                    uint32_t bh[NT][2], bl[NT][2];
#pragma unroll
                    for (int nt = 0; nt < NT; ++nt) {
                        const float s00 = sacc[nt][0] * p.scale_log2, s01 = sacc[nt][1] * p.scale_log2;
                        const float s10 = sacc[nt][2] * p.scale_log2, s11 = sacc[nt][3] * p.scale_log2;
                        float mx0 = fmaxf(s00, s10), mx1 = fmaxf(s01, s11);
#pragma unroll
                        for (int off = 4; off <= 16; off <<= 1) {
                            mx0 = fmaxf(mx0, __shfl_xor_sync(0xffffffffu, mx0, off));
                            mx1 = fmaxf(mx1, __shfl_xor_sync(0xffffffffu, mx1, off));
                        }
                        const float mn0 = fmaxf(pm[nt][0], mx0), mn1 = fmaxf(pm[nt][1], mx1);
                        const float al0 = ex2f(pm[nt][0] - mn0), al1 = ex2f(pm[nt][1] - mn1);
                        pm[nt][0] = mn0;
                        pm[nt][1] = mn1;
                        const float p00 = ex2f(s00 - mn0), p01 = ex2f(s01 - mn1);
                        const float p10 = ex2f(s10 - mn0), p11 = ex2f(s11 - mn1);
                        pl[nt][0] = fmaf(pl[nt][0], al0, p00 + p10);
                        pl[nt][1] = fmaf(pl[nt][1], al1, p01 + p11);
                        if (__any_sync(0xffffffffu, al0 != 1.f || al1 != 1.f)) {
#pragma unroll
                            for (int mt = 0; mt < D / 16; ++mt) {
                                pacc[mt][nt][0] *= al0; pacc[mt][nt][1] *= al1;
                                pacc[mt][nt][2] *= al0; pacc[mt][nt][3] *= al1;
                            }
                        }
                        const uint32_t hi0 = In::pack(p00, p01), hi1 = In::pack(p10, p11);
                        const uint32_t lo0 = In::pack(p00 - In::low(hi0), p01 - In::high(hi0));
                        const uint32_t lo1 = In::pack(p10 - In::low(hi1), p11 - In::high(hi1));
                        bh[nt][0] = movmatrix_trans(hi0);
                        bh[nt][1] = movmatrix_trans(hi1);
                        bl[nt][0] = movmatrix_trans(lo0);
                        bl[nt][1] = movmatrix_trans(lo1);
                    }
                    const int vrow = (lane & 7) + (lane >> 4) * 8;
                    const int vchk = (lane >> 3) & 1;
#pragma unroll
                    for (int mt = 0; mt < D / 16; ++mt) {
                        uint32_t a[4];
                        ldsm_x4_trans(vpage + (mt >> 2) * Cfg::kBoxBytes + swz(vrow, (mt & 3) * 2 + vchk), a);
#pragma unroll
                        for (int nt = 0; nt < NT; ++nt) {
                            In::mma(pacc[mt][nt], a, bh[nt][0], bh[nt][1]);
                            In::mma(pacc[mt][nt], a, bl[nt][0], bl[nt][1]);
                        }
                    }
                }
                __syncwarp();
                if (lane == 0) mbar_arrive(bar_base + 8 * (NS + s));
            }
            if (last_unit) pdl_launch_dependents();
            if (!last_unit) prefetch(nu, nxt);
            // one answer for the whole block on whether a wait was given up (see below)
            pfailed = block_sync_or(1, kConsumerThreads, pfailed || sm_flags[0] != 0);
#pragma unroll
            for (int nt = 0; nt < NT; ++nt) {
#pragma unroll
                for (int off = 4; off <= 16; off <<= 1) {
                    pl[nt][0] += __shfl_xor_sync(0xffffffffu, pl[nt][0], off);
                    pl[nt][1] += __shfl_xor_sync(0xffffffffu, pl[nt][1], off);
                }
                if (pfailed) {
                    pm[nt][0] = pm[nt][1] = -INFINITY;
                    pl[nt][0] = pl[nt][1] = 0.f;
                }
            }
            // The warps' results go through the block's scratch four columns at a time (it holds
            // [4 warps][4 columns][D]): columns 4q .. 4q+3 live in tile q / 2, lanes c = 2 (q % 2), +1.
            const int RF = rec_floats(G, D);
#pragma unroll
            for (int q = 0; q < 4; ++q) {
                const int nt = q >> 1;
                block_sync(1, kConsumerThreads);                            // the scratch is free again
                if ((c >> 1) == (q & 1)) {
                    const int lc = 2 * (c & 1);                             // local columns lc, lc + 1
                    if (r == 0) {
                        sm_wm[warp * COLS + lc] = pm[nt][0];
                        sm_wm[warp * COLS + lc + 1] = pm[nt][1];
                        sm_wl[warp * COLS + lc] = pl[nt][0];
                        sm_wl[warp * COLS + lc + 1] = pl[nt][1];
                    }
                    float* wo = sm_wo + (warp * COLS + lc) * D;
#pragma unroll
                    for (int mt = 0; mt < D / 16; ++mt) {
                        wo[mt * 16 + r] = pacc[mt][nt][0];
                        wo[D + mt * 16 + r] = pacc[mt][nt][1];
                        wo[mt * 16 + r + 8] = pacc[mt][nt][2];
                        wo[D + mt * 16 + r + 8] = pacc[mt][nt][3];
                    }
                }
                block_sync(1, kConsumerThreads);
                for (int task = tid; task < 4 * (D / 4); task += kConsumerThreads) {
                    const int lc = task / (D / 4), d4 = task % (D / 4);
                    const int col = 4 * q + lc;
                    const int j = col / G, h = col - j * G;
                    if (j >= nseq || j >= spb) continue;
                    const SeqInfo si = p.seq_info[b + j];
                    bool dead = p.run_mask != nullptr && __ldg(p.run_mask + b + j) == 0;      // masked row: an empty record
                    if (__ldg(p.seq_lens + b + j) != si.seq_len) {                            // stale plan: void, report
                        if (d4 == 0 && h == 0) record_status(p.status, DA_ERR_STALE_PLAN);
                        dead = true;
                    }
                    float M = -INFINITY;
#pragma unroll
                    for (int w = 0; w < kMmaConsumerWarps; ++w) M = fmaxf(M, sm_wm[w * COLS + lc]);
                    float4 o = make_float4(0.f, 0.f, 0.f, 0.f);
                    float ls = 0.f;
                    if (M != -INFINITY && !dead) {
#pragma unroll
                        for (int w = 0; w < kMmaConsumerWarps; ++w) {
                            const float wgt = ex2f(sm_wm[w * COLS + lc] - M);
                            const float4 v = reinterpret_cast<const float4*>(sm_wo)[(w * COLS + lc) * (D / 4) + d4];
                            o.x = fmaf(wgt, v.x, o.x);
                            o.y = fmaf(wgt, v.y, o.y);
                            o.z = fmaf(wgt, v.z, o.z);
                            o.w = fmaf(wgt, v.w, o.w);
                            ls = fmaf(wgt, sm_wl[w * COLS + lc], ls);
                        }
                    } else {
                        M = -INFINITY;
                    }
                    float* rec = p.ws + ((int64_t)(si.slot_base + u.split_index) * p.num_kv_heads + g) * RF;
                    __stcg(reinterpret_cast<float4*>(rec + h * D) + d4, o);
                    if (d4 == 0) __stcg(reinterpret_cast<float2*>(rec + G * D) + h, make_float2(M, ls));
                }
            }
            if (pfailed) return;
            u = nu;
            cur = nxt;
            continue;
        }

        float oacc[D / 16][NT][4];
        float m_run[NT][2], l_run[NT][2];
#pragma unroll
        for (int nt = 0; nt < NT; ++nt) {
            m_run[nt][0] = m_run[nt][1] = -INFINITY;
            l_run[nt][0] = l_run[nt][1] = 0.f;
#pragma unroll
            for (int i = 0; i < D / 16; ++i) oacc[i][nt][0] = oacc[i][nt][1] = oacc[i][nt][2] = oacc[i][nt][3] = 0.f;
        }
        uint32_t probe_sum = 0;
        bool failed = false;

        for (int it = 0; it < n_iters; ++it, ++git) {
            const int s = git % NS;
            if (!mbar_wait(bar_base + 8 * s, (git / NS) & 1, p.wait_limit) || sm_flags[0] != 0) {
                if (lane == 0) {
                    record_status(p.status, DA_ERR_TIMEOUT);
                    sm_flags[0] = 1;
                }
                failed = true;
                break;
            }
            if (git == 0 && tid == 0) DA_TRACE_STAMP(blockIdx.x, 3);
#ifdef DA_TRACE
            if (it == 0 && tid == 0 && trace_k < 4) DA_TRACE_CLOCK(blockIdx.x, 11 + trace_k * 4);
#endif
            const int page_idx = it * kPagesPerStage + warp;
            if (page_idx < n_pages) {
                const int tok0 = t0 + page_idx * 16;
                const int n_valid = min(16, t1 - tok0);
                const uint32_t kpage = base + s * Cfg::kStageBytes + warp * Cfg::kPageBytes;
                const uint32_t vpage = kpage + Cfg::kTensorBytes;
                if (MODE == kModeProbe) {
                    // fold every 16-byte chunk of the page's K and V tiles
                    for (int i = lane; i < 2 * Cfg::kPageBytes / 16; i += 32) {
                        const uint32_t a = (i < Cfg::kPageBytes / 16 ? kpage : vpage - Cfg::kPageBytes) + i * 16;
                        uint32_t x, y, z, w;
                        asm volatile("ld.shared.v4.u32 {%0,%1,%2,%3}, [%4];" : "=r"(x), "=r"(y), "=r"(z), "=r"(w) : "r"(a));
                        probe_sum ^= x ^ y ^ z ^ w;
                    }
                } else if (MODE == kModeGather) {
                    // un-swizzle: token row, 16-byte chunk -> dense [token][head][dim]
                    for (int i = lane; i < n_valid * (D / 8); i += 32) {
                        const int row = i / (D / 8), ch = i % (D / 8);
                        const uint32_t off = (ch >> 3) * Cfg::kBoxBytes + swz(row, ch & 7);
                        uint4 kv, vv;
                        asm volatile("ld.shared.v4.u32 {%0,%1,%2,%3}, [%4];" : "=r"(kv.x), "=r"(kv.y), "=r"(kv.z), "=r"(kv.w) : "r"(kpage + off));
                        asm volatile("ld.shared.v4.u32 {%0,%1,%2,%3}, [%4];" : "=r"(vv.x), "=r"(vv.y), "=r"(vv.z), "=r"(vv.w) : "r"(vpage + off));
                        const int64_t o = ((int64_t)(tok0 + row) * p.num_kv_heads + g) * D + ch * 8;
                        *reinterpret_cast<uint4*>(ex.k_out + o) = kv;
                        *reinterpret_cast<uint4*>(ex.v_out + o) = vv;
                    }
                } else {
                    if (p.new_k != nullptr && nseq == 0 && tok0 + n_valid == u.seq_len) {
                        // Fused own-layer KV write (Algorithm 1 step 2: the row's K/V is written, then the row
                        // attends over it).  This page holds the sequence's last position, whose K and V rows
                        // are the new ones: they replace what TMA brought from the pool in the staged tiles -
                        // same bits as a write to the pool followed by the load - and go to the pool for the
                        // steps to come.  The pool row belongs to this (sequence, KV head) unit alone.
                        const int row = n_valid - 1;
                        const uint4* nk = reinterpret_cast<const uint4*>(p.new_k + ((int64_t)b * p.num_kv_heads + g) * D);
                        const uint4* nv = reinterpret_cast<const uint4*>(p.new_v + ((int64_t)b * p.num_kv_heads + g) * D);
                        for (int i = lane; i < 2 * (D / 8); i += 32) {
                            const int which = i / (D / 8), ch = i % (D / 8);
                            const uint4 val = __ldg((which ? nv : nk) + ch);
                            const uint32_t a = (which ? vpage : kpage) + (ch >> 3) * Cfg::kBoxBytes + swz(row, ch & 7);
                            asm volatile("st.shared.v4.u32 [%0], {%1,%2,%3,%4};" ::"r"(a), "r"(val.x), "r"(val.y), "r"(val.z), "r"(val.w) : "memory");
                        }
                        append_new_row<D>(p, b, g, u.seq_len, lane);
                        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
                        __syncwarp();
                    }
                    if (n_valid < 16) {
                        // rows past the sequence end may hold anything (NaN patterns included) and a
                        // zero weight does not silence them in an mma: clear those V rows.  This is the
                        // sequence's last page; the async-proxy fence orders the stores before the TMA
                        // load that will reuse the stage for the next unit.
                        for (int i = lane; i < (16 - n_valid) * (D / 8); i += 32) {
                            const int row = n_valid + i / (D / 8), ch = i % (D / 8);
                            const uint32_t a = vpage + (ch >> 3) * Cfg::kBoxBytes + swz(row, ch & 7);
                            asm volatile("st.shared.v4.u32 [%0], {%1,%1,%1,%1};" ::"r"(a), "r"(0u) : "memory");
                        }
                        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
                        __syncwarp();
                    }
                    // ---- S^T = K . Q^T
                    float sacc[NT][4];
#pragma unroll
                    for (int nt = 0; nt < NT; ++nt) sacc[nt][0] = sacc[nt][1] = sacc[nt][2] = sacc[nt][3] = 0.f;
                    const int arow = (lane & 7) + ((lane >> 3) & 1) * 8;
                    const int achk = lane >> 4;
#pragma unroll
                    for (int ks = 0; ks < KSTEPS; ++ks) {
                        uint32_t a[4];
                        ldsm_x4(kpage + (ks >> 2) * Cfg::kBoxBytes + swz(arow, (ks & 3) * 2 + achk), a);
#pragma unroll
                        for (int nt = 0; nt < NT; ++nt) In::mma(sacc[nt], a, qb[ks][nt][0], qb[ks][nt][1]);
                    }
                    // ---- online softmax on the fragment: rows r, r+8 (tokens), columns 2c, 2c+1 (heads)
                    const bool v_lo = r < n_valid, v_hi = (r + 8) < n_valid;
                    uint32_t b0[NT], b1[NT], b0l[NT], b1l[NT];
#pragma unroll
                    for (int nt = 0; nt < NT; ++nt) {
                        float s00 = v_lo ? sacc[nt][0] * p.scale_log2 : -INFINITY;
                        float s01 = v_lo ? sacc[nt][1] * p.scale_log2 : -INFINITY;
                        float s10 = v_hi ? sacc[nt][2] * p.scale_log2 : -INFINITY;
                        float s11 = v_hi ? sacc[nt][3] * p.scale_log2 : -INFINITY;
                        float mx0 = fmaxf(s00, s10), mx1 = fmaxf(s01, s11);
#pragma unroll
                        for (int off = 4; off <= 16; off <<= 1) {
                            mx0 = fmaxf(mx0, __shfl_xor_sync(0xffffffffu, mx0, off));
                            mx1 = fmaxf(mx1, __shfl_xor_sync(0xffffffffu, mx1, off));
                        }
                        const float mn0 = fmaxf(m_run[nt][0], mx0), mn1 = fmaxf(m_run[nt][1], mx1);   // finite: token 0 of the page is valid
                        const float al0 = ex2f(m_run[nt][0] - mn0), al1 = ex2f(m_run[nt][1] - mn1);
                        m_run[nt][0] = mn0;
                        m_run[nt][1] = mn1;
                        const float p00 = ex2f(s00 - mn0), p01 = ex2f(s01 - mn1);
                        const float p10 = ex2f(s10 - mn0), p11 = ex2f(s11 - mn1);
                        l_run[nt][0] = fmaf(l_run[nt][0], al0, p00 + p10);
                        l_run[nt][1] = fmaf(l_run[nt][1], al1, p01 + p11);
                        if (__any_sync(0xffffffffu, al0 != 1.f || al1 != 1.f)) {
#pragma unroll
                            for (int mt = 0; mt < D / 16; ++mt) {
                                oacc[mt][nt][0] *= al0; oacc[mt][nt][1] *= al1;
                                oacc[mt][nt][2] *= al0; oacc[mt][nt][3] *= al1;
                            }
                        }
                        // ---- P^T as B fragments (high parts; low parts in the duplicated columns or a second set)
                        uint32_t hi0 = In::pack(p00, p01), hi1 = In::pack(p10, p11);
                        const float r00 = p00 - In::low(hi0), r01 = p01 - In::high(hi0);
                        const float r10 = p10 - In::low(hi1), r11 = p11 - In::high(hi1);
                        const uint32_t lo0 = In::pack(r00, r01), lo1 = In::pack(r10, r11);
                        b0l[nt] = b1l[nt] = 0;
                        if (DUP) {
                            b0[nt] = movmatrix_trans(lo_role ? lo0 : hi0);
                            b1[nt] = movmatrix_trans(lo_role ? lo1 : hi1);
                        } else {
                            b0[nt] = movmatrix_trans(hi0);
                            b1[nt] = movmatrix_trans(hi1);
                            b0l[nt] = movmatrix_trans(lo0);
                            b1l[nt] = movmatrix_trans(lo1);
                        }
                    }
                    // ---- O^T += V^T . P^T
                    const int vrow = (lane & 7) + (lane >> 4) * 8;
                    const int vchk = (lane >> 3) & 1;
#pragma unroll
                    for (int mt = 0; mt < D / 16; ++mt) {
                        uint32_t a[4];
                        ldsm_x4_trans(vpage + (mt >> 2) * Cfg::kBoxBytes + swz(vrow, (mt & 3) * 2 + vchk), a);
#pragma unroll
                        for (int nt = 0; nt < NT; ++nt) {
                            In::mma(oacc[mt][nt], a, b0[nt], b1[nt]);
                            if (!DUP) In::mma(oacc[mt][nt], a, b0l[nt], b1l[nt]);
                        }
                    }
                }
            }
            __syncwarp();
            if (lane == 0) mbar_arrive(bar_base + 8 * (NS + s));          // this warp is done with the stage
        }
        if (uid == ubeg && tid == 0) DA_TRACE_STAMP(blockIdx.x, 4);
#ifdef DA_TRACE
        if (tid == 0 && trace_k < 4) DA_TRACE_CLOCK(blockIdx.x, 12 + trace_k * 4);
#endif
        if (queued) {
            // the producer drew the next unit while this one streamed
            const int need = uid - ubeg + 2;
            if (!failed && !wait_published(need)) {
                if (lane == 0) {
                    record_status(p.status, DA_ERR_TIMEOUT);
                    sm_flags[0] = 1;
                }
                failed = true;
            }
            last_unit = true;
            if (!failed) {
                nu = ring_unit(need - 1);
                last_unit = nu.seq < 0;
            }
        }
        if (last_unit && MODE == kModeAttend) pdl_launch_dependents();    // the combine kernel may start getting scheduled
        if (!last_unit) prefetch(nu, nxt);                                // in flight during this unit's epilogue

        if (MODE == kModeProbe) {
#pragma unroll
            for (int off = 16; off >= 1; off >>= 1) probe_sum ^= __shfl_xor_sync(0xffffffffu, probe_sum, off);
            if (lane == 0) atomicXor(ex.checksum + uid, probe_sum);
        }
        if (MODE != kModeAttend) {
            if (failed) return;
            u = nu;
            cur = nxt;
            continue;
        }

        // ------------------------------------------------------------ end of the unit
        const bool stale = dev_len != u.seq_len;                  // stale plan: void the result, report it
        if (stale && tid == 0) record_status(p.status, DA_ERR_STALE_PLAN);
        if (n_pages == 0) {
            // Nothing was read (a masked row, an empty split, a sequence of length 0): the empty
            // result is written straight away - no states to merge, no barrier, the scratch untouched.
            if (MODE == kModeAttend && warp == 0 && nseq == 0 && u.tok_end == u.seq_len && u.tok_end > u.tok_begin)
                append_new_row<D>(p, b, g, u.seq_len, lane);              // a masked row still writes its K/V
            block_finish_empty<D>(p, u, G, tid, kConsumerThreads);
            if (uid == ubeg && tid == 0) DA_TRACE_STAMP(blockIdx.x, 6);
            if (queued && last_unit) break;
            u = nu;
            cur = nxt;
            continue;
        }
#pragma unroll
        for (int nt = 0; nt < NT; ++nt) {
#pragma unroll
            for (int off = 4; off <= 16; off <<= 1) {
                l_run[nt][0] += __shfl_xor_sync(0xffffffffu, l_run[nt][0], off);
                l_run[nt][1] += __shfl_xor_sync(0xffffffffu, l_run[nt][1], off);
            }
        }
        // Every warp is done reading the previous unit's results.  A warp may have given up on a
        // wait just before the others saw the flag: the barrier carries a vote, every warp gets
        // the same answer, the unit's result is voided and the block leaves together.
#ifdef DA_TRACE
        if (tid == 0 && trace_k == 1) DA_TRACE_CLOCK(blockIdx.x, 26);
#endif
        const bool gave_up = block_sync_or(1, kConsumerThreads, failed || sm_flags[0] != 0);
#ifdef DA_TRACE
        if (tid == 0 && trace_k == 1) DA_TRACE_CLOCK(blockIdx.x, 27);
#endif
        if (gave_up || stale) {
#pragma unroll
            for (int nt = 0; nt < NT; ++nt) {
                m_run[nt][0] = m_run[nt][1] = -INFINITY;
                l_run[nt][0] = l_run[nt][1] = 0.f;
            }
        }
        if (DUP) {
            // columns 4..7 carried the low parts of P for heads 0..3: lanes c = 2, 3 hand theirs to c = 0, 1
#pragma unroll
            for (int mt = 0; mt < D / 16; ++mt)
#pragma unroll
                for (int i = 0; i < 4; ++i) oacc[mt][0][i] += __shfl_down_sync(0xffffffffu, oacc[mt][0][i], 2);
        }
        // The warps' states meet in the block's scratch four heads at a time (it holds [4 warps][4
        // columns][D]): heads 4q .. 4q+3 live in tile q / 2, lanes c = 2 (q % 2), +1 (all of a duplicated
        // group in c = 0, 1).
#pragma unroll
        for (int q = 0; q < (DUP ? 1 : 2 * NT); ++q) {
            if (4 * q >= G) break;
            const int nt = q >> 1;
            if (q > 0) block_sync(1, kConsumerThreads);                     // the scratch is free again
            if ((c >> 1) == (q & 1)) {
                const int lc = 2 * (c & 1);                                 // local columns lc, lc + 1
                if (r == 0) {
                    sm_wm[warp * COLS + lc] = m_run[nt][0];
                    sm_wm[warp * COLS + lc + 1] = m_run[nt][1];
                    sm_wl[warp * COLS + lc] = l_run[nt][0];
                    sm_wl[warp * COLS + lc + 1] = l_run[nt][1];
                }
                float* wo = sm_wo + (warp * COLS + lc) * D;
#pragma unroll
                for (int mt = 0; mt < D / 16; ++mt) {
                    wo[mt * 16 + r] = oacc[mt][nt][0];
                    wo[D + mt * 16 + r] = oacc[mt][nt][1];
                    wo[mt * 16 + r + 8] = oacc[mt][nt][2];
                    wo[D + mt * 16 + r + 8] = oacc[mt][nt][3];
                }
            }
#ifdef DA_TRACE
            if (tid == 0 && trace_k == 1 && q == 0) DA_TRACE_CLOCK(blockIdx.x, 28);
#endif
            block_sync(1, kConsumerThreads);
#ifdef DA_TRACE
            if (tid == 0 && trace_k == 1 && q == 0) DA_TRACE_CLOCK(blockIdx.x, 29);
#endif
            block_finish<D, kMmaConsumerWarps, COLS, false>(p, u, G, sm_wo, sm_wm, sm_wl, tid, kConsumerThreads, 1, 4 * q,
                                                            min(4, G - 4 * q), DUP || 4 * (q + 1) >= G);
        }
        if (uid == ubeg && tid == 0) DA_TRACE_STAMP(blockIdx.x, 6);
#ifdef DA_TRACE
        if (tid == 0 && trace_k < 4) DA_TRACE_CLOCK(blockIdx.x, 13 + trace_k * 4);
#endif
        if (gave_up) return;
        if (queued && last_unit) break;
        u = nu;
        cur = nxt;
    }
    if (tid == 0) DA_TRACE_STAMP(blockIdx.x, 5);                  // (trace builds) the block's last unit is finished
}

// ---------------------------------------------------------------- host side

inline bool mma_supports(int D, int G) { return (D == 64 || D == 128) && G >= 1 && G <= 16; }

typedef CUresult (*encode_tiled_fn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                    const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                    CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

inline encode_tiled_fn get_encode_tiled()
{
    static encode_tiled_fn fn = [] {
        void* ptr = nullptr;
        cudaDriverEntryPointQueryResult q;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &ptr, cudaEnableDefault, &q) != cudaSuccess ||
            q != cudaDriverEntryPointSuccess) {
            (void)cudaGetLastError();
            ptr = nullptr;
        }
        return reinterpret_cast<encode_tiled_fn>(ptr);
    }();
    return fn;
}

// 4-D map of one pool: [head_dim, slot, kv head, page]; a box is 64 dims x 16 slots of one head of one page.
inline int make_pool_map(CUtensorMap* map, const void* pool, const decode_attn_shape_t& s, int64_t stride_page,
                         int64_t stride_token, int64_t stride_head)
{
    const CUtensorMapDataType dt =
        s.kv_dtype == DA_DTYPE_FP16 ? CU_TENSOR_MAP_DATA_TYPE_FLOAT16 : CU_TENSOR_MAP_DATA_TYPE_BFLOAT16;
    encode_tiled_fn enc = get_encode_tiled();
    if (!enc) return DA_ERR_CUDA;
    const cuuint64_t dims[4] = {(cuuint64_t)s.head_dim, (cuuint64_t)s.page_size, (cuuint64_t)s.num_kv_heads,
                                (cuuint64_t)s.num_pages};
    const cuuint64_t strides[3] = {(cuuint64_t)stride_token * 2, (cuuint64_t)stride_head * 2,
                                   (cuuint64_t)stride_page * 2};
    const cuuint32_t box[4] = {64, 16, 1, 1};
    const cuuint32_t estr[4] = {1, 1, 1, 1};
    CUresult r = enc(map, dt, 4, const_cast<void*>(pool), dims, strides, box, estr,
                     CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                     CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    return r == CUDA_SUCCESS ? DA_OK : DA_ERR_CUDA;
}

typedef void (*mma_kernel_t)(const KernelParams, const CUtensorMap, const CUtensorMap, const int, const MmaExtra);

// f16: q, K and V are fp16 (attention mode); else bf16.
template <int MODE>
inline mma_kernel_t mma_kernel_for(int D, int G, bool prefix = false, bool f16 = false, bool masked = false)
{
    const bool dup = G <= 4;
    if (G > 8 && MODE == kModeAttend) {   // two tiles of heads; ordinary plans only
        if (prefix) return nullptr;
        if (D == 128)
            return f16 ? (masked ? decode_attn_mma_kernel<128, false, kModeAttend, false, true, true, true>
                                 : decode_attn_mma_kernel<128, false, kModeAttend, false, true, false, true>)
                       : (masked ? decode_attn_mma_kernel<128, false, kModeAttend, false, false, true, true>
                                 : decode_attn_mma_kernel<128, false, kModeAttend, false, false, false, true>);
        if (D == 64)
            return f16 ? (masked ? decode_attn_mma_kernel<64, false, kModeAttend, false, true, true, true>
                                 : decode_attn_mma_kernel<64, false, kModeAttend, false, true, false, true>)
                       : (masked ? decode_attn_mma_kernel<64, false, kModeAttend, false, false, true, true>
                                 : decode_attn_mma_kernel<64, false, kModeAttend, false, false, false, true>);
        return nullptr;
    }
    if (masked && MODE == kModeAttend && !prefix) {
        if (D == 128)
            return f16 ? (dup ? decode_attn_mma_kernel<128, true, kModeAttend, false, true, true>
                              : decode_attn_mma_kernel<128, false, kModeAttend, false, true, true>)
                       : (dup ? decode_attn_mma_kernel<128, true, kModeAttend, false, false, true>
                              : decode_attn_mma_kernel<128, false, kModeAttend, false, false, true>);
        if (D == 64)
            return f16 ? (dup ? decode_attn_mma_kernel<64, true, kModeAttend, false, true, true>
                              : decode_attn_mma_kernel<64, false, kModeAttend, false, true, true>)
                       : (dup ? decode_attn_mma_kernel<64, true, kModeAttend, false, false, true>
                              : decode_attn_mma_kernel<64, false, kModeAttend, false, false, true>);
        return nullptr;
    }
    if (f16) {
        if (MODE != kModeAttend) return nullptr;
        if (prefix) {
            if (!dup) return nullptr;
            if (D == 128) return decode_attn_mma_kernel<128, true, kModeAttend, true, true>;
            if (D == 64) return decode_attn_mma_kernel<64, true, kModeAttend, true, true>;
            return nullptr;
        }
        if (D == 128) return dup ? decode_attn_mma_kernel<128, true, kModeAttend, false, true>
                                 : decode_attn_mma_kernel<128, false, kModeAttend, false, true>;
        if (D == 64) return dup ? decode_attn_mma_kernel<64, true, kModeAttend, false, true>
                                : decode_attn_mma_kernel<64, false, kModeAttend, false, true>;
        return nullptr;
    }
    if (prefix) {   // shared-prefix plans: attention mode, groups of up to 4 heads
        if (MODE != kModeAttend || !dup) return nullptr;
        if (D == 128) return decode_attn_mma_kernel<128, true, kModeAttend, true>;
        if (D == 64) return decode_attn_mma_kernel<64, true, kModeAttend, true>;
        return nullptr;
    }
    if (D == 128) return dup ? decode_attn_mma_kernel<128, true, MODE, false> : decode_attn_mma_kernel<128, false, MODE, false>;
    if (D == 64) return dup ? decode_attn_mma_kernel<64, true, MODE, false> : decode_attn_mma_kernel<64, false, MODE, false>;
    return nullptr;
}

inline int mma_smem_bytes(int D, int G)
{
    const bool dup = G <= 4;
    if (D == 128) return dup ? MmaCfg<128, true>::kSmemBytes : MmaCfg<128, false>::kSmemBytes;
    return dup ? MmaCfg<64, true>::kSmemBytes : MmaCfg<64, false>::kSmemBytes;
}

template <int MODE>
inline int mma_prepare(int D, int G, mma_kernel_t* fn_out, bool prefix = false, bool f16 = false, bool masked = false)
{
    mma_kernel_t fn = mma_kernel_for<MODE>(D, G, prefix, f16, masked);
    if (!fn) return DA_ERR_UNSUPPORTED;
    if (cudaFuncSetAttribute(fn, cudaFuncAttributeMaxDynamicSharedMemorySize, mma_smem_bytes(D, G)) != cudaSuccess) {
        (void)cudaGetLastError();
        return DA_ERR_CUDA;
    }
    *fn_out = fn;
    return DA_OK;
}

inline int mma_query_occupancy(int D, int G, int* block_threads, int* dyn_smem, bool prefix = false, bool f16 = false)
{
    mma_kernel_t fn;
    if (mma_prepare<kModeAttend>(D, G, &fn, prefix, f16) != DA_OK) return -1;
    *block_threads = kMmaThreads;
    *dyn_smem = mma_smem_bytes(D, G);
    int n = 0;
    if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&n, fn, kMmaThreads, mma_smem_bytes(D, G)) != cudaSuccess) {
        (void)cudaGetLastError();
        return -1;
    }
    return n;
}

template <int MODE>
inline int mma_launch_mode(const decode_attn_shape_t& s, int G, const KernelParams& kp, const MmaExtra& ex,
                           unsigned grid, cudaStream_t stream, bool prefix = false)
{
    mma_kernel_t fn;
    // (the probe and gather modes only move 16-bit words: one variant serves both input types)
    const bool masked = MODE == kModeAttend && !prefix && kp.run_mask != nullptr &&
                        (kp.grid_exit ? kp.may_rank != 0 : kp.n_ranked > 0);
    int rc = mma_prepare<MODE>(s.head_dim, G, &fn, prefix, MODE == kModeAttend && s.kv_dtype == DA_DTYPE_FP16, masked);
    if (rc != DA_OK) return rc;
    CUtensorMap kmap, vmap;
    rc = make_pool_map(&kmap, kp.k, s, s.k_stride_page, s.k_stride_token, s.k_stride_head);
    if (rc != DA_OK) return rc;
    rc = make_pool_map(&vmap, kp.v, s, s.v_stride_page, s.v_stride_token, s.v_stride_head);
    if (rc != DA_OK) return rc;
    // programmatic dependency on the kernel launched before: this kernel's blocks may become
    // resident and run their prologue while that kernel drains (see pdl_wait_primary above)
    cudaLaunchConfig_t cfg;
    cfg.gridDim = dim3(grid, 1, 1);
    cfg.blockDim = dim3(kMmaThreads, 1, 1);
    cfg.dynamicSmemBytes = (size_t)mma_smem_bytes(s.head_dim, G);
    cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    if (cudaLaunchKernelEx(&cfg, fn, kp, kmap, vmap, G, ex) != cudaSuccess) {
        (void)cudaGetLastError();
        return DA_ERR_CUDA;
    }
    return DA_OK;
}

inline int mma_launch(const decode_attn_shape_t& s, int G, const KernelParams& kp, unsigned grid, cudaStream_t stream,
                      bool prefix = false)
{
    MmaExtra ex = {nullptr, nullptr, nullptr, 0};
    return mma_launch_mode<kModeAttend>(s, G, kp, ex, grid, stream, prefix);
}

inline int mma_gather_probe(const decode_attn_shape_t& s, int G, const KernelParams& kp, uint32_t* checksum,
                            unsigned n_units, unsigned grid, cudaStream_t stream)
{
    if (cudaMemsetAsync(checksum, 0, sizeof(uint32_t) * n_units, stream) != cudaSuccess) {
        (void)cudaGetLastError();
        return DA_ERR_CUDA;
    }
    MmaExtra ex = {checksum, nullptr, nullptr, 0};
    return mma_launch_mode<kModeProbe>(s, G, kp, ex, grid, stream);
}

inline int mma_debug_gather(const decode_attn_shape_t& s, int G, const KernelParams& kp, int seq, void* k_out,
                            void* v_out, unsigned grid, cudaStream_t stream)
{
    MmaExtra ex = {nullptr, static_cast<__nv_bfloat16*>(k_out), static_cast<__nv_bfloat16*>(v_out), seq};
    return mma_launch_mode<kModeGather>(s, G, kp, ex, grid, stream);
}

}  // namespace da
