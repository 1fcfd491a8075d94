// Split-KV planner.  The paper leaves partitioning to the engine; what it
// demands is that launch metadata is rebuilt from the current rows whenever
// they change (Invariant 2) and that a fixed launch shape can serve any live
// size (Algorithm 1 step 6).  The policy implemented here:
//
//  * a work unit is (sequence, KV head, run of whole pages); all query heads
//    of the group are handled by the unit so each K/V byte is read once;
//  * AUTO picks one chunk length c (pages) for the whole batch: the smallest
//    c >= the policy's minimum for which the unit count fits in
//    waves * sm_count * ctas_per_sm resident blocks, waves being the smallest
//    integer for which that is possible at all (and a fraction of that c where
//    the waves do not divide and the units are long, see make_layout).  Each
//    sequence then gets ceil(pages / c) splits of near-equal size;
//  * DETERMINISTIC cuts every sequence at multiples of a chunk that depends on
//    the sequence's own length and the policy alone (policy.chunk_tokens, by
//    default 256 tokens, lengthened so that no sequence has more than
//    max_splits = 32 chunks), so its boundaries do not depend on the batch;
//  * FIXED_COUNT gives every sequence exactly n splits of ceil(pages / n)
//    pages; trailing splits may be empty;
//  * units are issued most expensive first, and the KV heads of one token
//    range next to each other so their blocks run at the same time and touch
//    neighbouring addresses of the same pages.
#include "planner.h"

#include <algorithm>
#include <cmath>
#include <functional>
#include <queue>
#include <utility>

namespace da {

static inline int64_t ceil_div(int64_t a, int64_t b) { return (a + b - 1) / b; }

int validate_shape(const decode_attn_shape_t& s)
{
    if (s.batch < 0 || s.num_q_heads <= 0 || s.num_kv_heads <= 0 || s.head_dim <= 0 || s.page_size <= 0 ||
        s.max_pages_per_seq < 0 || s.num_pages <= 0)
        return DA_ERR_INVALID_ARG;
    if (s.num_q_heads % s.num_kv_heads != 0) return DA_ERR_INVALID_ARG;
    if (!(s.sm_scale >= 0.0f) || std::isinf(s.sm_scale)) return DA_ERR_INVALID_ARG;
    const int64_t strides[6] = {s.k_stride_page, s.k_stride_token, s.k_stride_head,
                                s.v_stride_page, s.v_stride_token, s.v_stride_head};
    for (int64_t st : strides) {
        if (st <= 0) return DA_ERR_INVALID_ARG;
        if (st % 8 != 0) return DA_ERR_INVALID_ARG;  // 16-byte rows for vector loads and TMA
    }
    if (s.k_stride_token < s.head_dim || s.k_stride_head < s.head_dim || s.v_stride_token < s.head_dim ||
        s.v_stride_head < s.head_dim)
        return DA_ERR_INVALID_ARG;  // rows of head_dim contiguous elements must not overlap
    if (s.num_q_heads / s.num_kv_heads > kMaxGroup) return DA_ERR_UNSUPPORTED;
    if (s.head_dim != 64 && s.head_dim != 128) return DA_ERR_UNSUPPORTED;
    // the kernels walk the cache in 16-token tiles: a page holds a power-of-two number of them
    if (s.page_size < 16 || s.page_size > 256 || (s.page_size & (s.page_size - 1)) != 0) return DA_ERR_UNSUPPORTED;
    if ((s.kv_dtype != DA_DTYPE_BF16 && s.kv_dtype != DA_DTYPE_FP16) || s.q_dtype != s.kv_dtype) return DA_ERR_UNSUPPORTED;
    if (s.out_dtype != DA_DTYPE_FP32 && s.out_dtype != DA_DTYPE_BF16 && s.out_dtype != DA_DTYPE_FP16) return DA_ERR_UNSUPPORTED;
    if (s.num_pages > (int64_t)INT32_MAX) return DA_ERR_UNSUPPORTED;
    return DA_OK;
}

int validate_policy(const decode_attn_shape_t& s, const decode_attn_policy_t& p)
{
    if (p.split_mode < DA_SPLIT_AUTO || p.split_mode > DA_SPLIT_DETERMINISTIC) return DA_ERR_INVALID_ARG;
    if (p.kernel < DA_KERNEL_AUTO || p.kernel > DA_KERNEL_UMMA_PREFIX) return DA_ERR_INVALID_ARG;
    if (p.split_mode == DA_SPLIT_FIXED_COUNT && p.fixed_count < 1) return DA_ERR_INVALID_ARG;
    if (p.chunk_tokens < 0 || p.max_splits < 0 || p.sm_count < 0 || p.ctas_per_sm < 0 ||
        p.capacity_batch < 0 || p.capacity_tokens < 0)
        return DA_ERR_INVALID_ARG;
    if (p.chunk_tokens % kTileTokens != 0) return DA_ERR_INVALID_ARG;
    if (p.max_splits > kMaxSplits || (p.split_mode == DA_SPLIT_FIXED_COUNT && p.fixed_count > kMaxSplits))
        return DA_ERR_INVALID_ARG;
    if (p.fuse_combine != 0 && p.fuse_combine != 1) return DA_ERR_INVALID_ARG;
    if (p.capacity_batch > 0 && (p.capacity_tokens <= 0 || s.batch > p.capacity_batch))
        return DA_ERR_INVALID_ARG;
    if (p.shared_prefix_tokens < 0 || p.shared_prefix_tokens % s.page_size != 0) return DA_ERR_INVALID_ARG;
    if (p.shared_prefix_tokens > 0) {
        if (p.fuse_combine || p.capacity_batch > 0 || p.split_mode == DA_SPLIT_FIXED_COUNT) return DA_ERR_UNSUPPORTED;
        const int G = s.num_q_heads / s.num_kv_heads;
        if (p.kernel == DA_KERNEL_UMMA_PREFIX) {
            if (s.head_dim != 128) return DA_ERR_UNSUPPORTED;
        } else if (p.kernel == DA_KERNEL_SIMT || G > 4) {
            return DA_ERR_UNSUPPORTED;
        }
    } else if (p.kernel == DA_KERNEL_UMMA_PREFIX) {
        return DA_ERR_UNSUPPORTED;   // that kernel serves shared-prefix plans only
    }
    for (int32_t r : p.reserved)
        if (r != 0) return DA_ERR_INVALID_ARG;
    return DA_OK;
}

// DETERMINISTIC cuts at multiples of the chunk, so a long sequence would leave hundreds of records;
// its default bound keeps that at 32 (the chunk grows with the sequence's own length instead, still a
// function of that length alone): 131,072 tokens alone 90 -> 80 us, sixteen of them 1,284 -> 1,240 us.
// Together with the default chunk of 256 tokens the default rule is: chunk = max(256, length / 32
// rounded up to 16) - a short sequence served alone still spreads over the machine (2,048 tokens
// alone 18.5 -> 8.2 us, 8,192 alone 18.9 -> 10.3 us, both what AUTO gets), at 3-13 % on the largest
// batches of such sequences (8,192 x 256: 1,350 against 1,252 us with 1,024-token chunks).
static int max_splits_of(const decode_attn_policy_t& p)
{
    if (p.max_splits > 0) return p.max_splits;
    return p.split_mode == DA_SPLIT_DETERMINISTIC ? kDefaultDeterministicMaxSplits : kDefaultMaxSplits;
}

static int min_chunk_pages(const decode_attn_shape_t& s, const decode_attn_policy_t& p)
{
    int tokens;
    if (p.split_mode == DA_SPLIT_DETERMINISTIC)
        tokens = p.chunk_tokens > 0 ? p.chunk_tokens : kDefaultDeterministicChunk;
    else
        tokens = p.chunk_tokens > 0 ? p.chunk_tokens : kDefaultAutoMinChunk;
    (void)s;
    return (int)std::max<int64_t>(1, ceil_div(tokens, kTileTokens));
}

int64_t capacity_slots(const decode_attn_shape_t& s, const decode_attn_policy_t& p)
{
    if (p.capacity_batch <= 0) return 0;
    if (p.split_mode == DA_SPLIT_FIXED_COUNT) return (int64_t)p.fixed_count * p.capacity_batch;
    const int64_t chunk_tokens = (int64_t)min_chunk_pages(s, p) * kTileTokens;
    return ceil_div(p.capacity_tokens, chunk_tokens) + p.capacity_batch;
}

namespace {

struct SeqCut {
    int64_t pages;
    int64_t chunk;   // pages per split (upper bound)
    int32_t splits;
    bool even;       // spread the pages evenly instead of cutting at multiples of chunk
};

// (page counts are below 2^28: 32-bit divisions, which are several times cheaper than 64-bit ones)
int64_t units_for_chunk(const std::vector<int64_t>& pages, int64_t c, int max_splits)
{
    int64_t total = 0;
    const uint32_t c32 = (uint32_t)std::min<int64_t>(c, INT32_MAX), ms = (uint32_t)max_splits;
    for (int64_t pg64 : pages) {
        const uint32_t pg = (uint32_t)pg64;
        if (pg == 0) {
            total += 1;
            continue;
        }
        const uint32_t cb = std::max(c32, (pg + ms - 1) / ms);
        total += (pg + cb - 1) / cb;
    }
    return total;
}

}  // namespace

int make_layout(const decode_attn_shape_t& s, const decode_attn_policy_t& p, const int32_t* seq_lens,
                int sm_count, int ctas_per_sm, Layout& out, int max_bins)
{
    if (sm_count <= 0 || ctas_per_sm <= 0) return DA_ERR_INVALID_ARG;
    if (s.batch > 0 && seq_lens == nullptr) return DA_ERR_INVALID_ARG;
    // Everything below counts in 16-token tiles ("pages" of the planner): what the kernels fetch at
    // a time.  The pool's page size only bounds the block table, so a plan does not depend on it.
    const int B = s.batch, P = kTileTokens, H = s.num_kv_heads;
    const int max_splits = max_splits_of(p);
    // With a shared prefix the ordinary units cover only what follows it; the prefix itself is
    // cut into chunks attended once for a block of sequences at a time (see below).
    const int64_t prefix_tokens = p.shared_prefix_tokens;
    const int64_t prefix_pages = prefix_tokens / P;
    std::vector<int64_t> pages(B);
    for (int b = 0; b < B; ++b) {
        if (seq_lens[b] < 0) return DA_ERR_INVALID_ARG;
        if (ceil_div(seq_lens[b], s.page_size) > s.max_pages_per_seq) return DA_ERR_INVALID_ARG;
        if (seq_lens[b] < prefix_tokens) return DA_ERR_INVALID_ARG;   // every sequence contains the prefix
        pages[b] = ceil_div(seq_lens[b] - prefix_tokens, P);
    }

    std::vector<SeqCut> cuts(B);
    out.chunk_tokens = 0;
    if (p.split_mode == DA_SPLIT_FIXED_COUNT) {
        for (int b = 0; b < B; ++b) {
            cuts[b].pages = pages[b];
            cuts[b].chunk = std::max<int64_t>(1, ceil_div(pages[b], p.fixed_count));
            cuts[b].splits = p.fixed_count;
            cuts[b].even = false;
        }
    } else {
        int64_t c = min_chunk_pages(s, p);
        const int64_t c_min = c;                              // the policy's smallest chunk: nothing below goes
        if (p.split_mode == DA_SPLIT_AUTO && B > 0) {
            const int64_t slots = (int64_t)sm_count * ctas_per_sm;
            const int64_t floor_units = (int64_t)H * B;  // one unit per (sequence, KV head) at least
            const int64_t waves = std::max<int64_t>(1, ceil_div(floor_units, slots));
            const int64_t target = waves * slots;
            int64_t lo = c, hi = std::max<int64_t>(c, *std::max_element(pages.begin(), pages.end()));
            if (H * units_for_chunk(pages, lo, max_splits) > target) {
                while (lo < hi) {  // smallest chunk whose unit count fits
                    const int64_t mid = lo + (hi - lo) / 2;
                    if (H * units_for_chunk(pages, mid, max_splits) <= target)
                        hi = mid;
                    else
                        lo = mid + 1;
                }
            }
            c = lo;
            // Whole waves do not always divide: 64 long sequences x 8 heads are 512 units on 296 blocks,
            // so most blocks get two units and the rest one.  Where the units are long enough for a
            // cut to cost next to nothing (chunks stay at 2,048 tokens or more; 1,024 was measured and
            // loses), a chunk that is a fraction of c is taken when it brings the heaviest block's
            // load down by more than 3 % - load in pages, three pages per unit for its hand-over, 24
            // for a combine launch the plan did not need before (131,072 x 64: 5.11 -> 4.85 ms,
            // 32,768 x 64: 1.28 -> 1.23 ms, 8,192 x 64: 312 -> 308.5 us).
            const int64_t u0 = H * units_for_chunk(pages, c, max_splits);
            const int64_t waves0 = ceil_div(u0, slots);
            constexpr int64_t kLongChunk = 128, kUnitPages = 3, kCombinePages = 24;
            if (waves0 * slots * 100 > u0 * 106 && c >= 2 * kLongChunk) {
                const bool split0 = u0 > floor_units;
                int64_t best = c, best_cost = waves0 * (c + kUnitPages) + (split0 ? kCombinePages : 0);
                for (int k = 2; k <= 8; ++k) {
                    const int64_t ck = ceil_div(c, k);
                    if (ck < std::max(kLongChunk, c_min)) break;
                    const int64_t wk = ceil_div(H * units_for_chunk(pages, ck, max_splits), slots);
                    const int64_t cost = wk * (ck + kUnitPages) + kCombinePages;
                    if (cost * 100 < best_cost * 97) {
                        best = ck;
                        best_cost = cost;
                    }
                }
                c = best;
            }
        }
        out.chunk_tokens = (int32_t)std::min<int64_t>(c * P, INT32_MAX);
        for (int b = 0; b < B; ++b) {
            cuts[b].pages = pages[b];
            cuts[b].chunk = std::max(c, ceil_div(pages[b], max_splits));
            cuts[b].splits = (int32_t)std::max<int64_t>(1, ceil_div(pages[b], cuts[b].chunk));
            cuts[b].even = (p.split_mode == DA_SPLIT_AUTO);
        }
    }

    out.splits.assign(B, 1);
    out.slot_base.assign(B, -1);
    out.n_slots = 0;
    out.max_splits_used = B > 0 ? 1 : 0;
    // Units in creation order (shared-prefix units first, then sequence by sequence, split by split,
    // KV head by KV head) with their costs beside them; the launch order is found by sorting indices.
    // This runs every decode step: no per-unit allocation, no moving of units but the final placement.
    std::vector<decode_attn_unit_t>& made = out.scratch_units;
    std::vector<int32_t>& cost = out.scratch_cost;
    made.clear();
    cost.clear();
    {
        size_t expect = 0;
        for (int b = 0; b < B; ++b) expect += (size_t)cuts[b].splits;
        made.reserve((expect + (size_t)B) * (size_t)H + 64);
        cost.reserve(made.capacity());
    }

    // Shared prefix: a unit is (block of sequences, KV head, chunk of the prefix); the query rows
    // of the block's sequences form the columns of one tensor-core tile, so a prefix page is
    // fetched once per block instead of once per sequence.
    const int G = s.num_q_heads / s.num_kv_heads;
    const bool umma = p.kernel == DA_KERNEL_UMMA_PREFIX && prefix_tokens > 0;
    const int seqs_per_block = prefix_tokens > 0 ? (umma ? kUmmaPrefixRows : kPrefixColumns) / G : 1;
    int32_t PC = 0;
    size_t n_prefix_units = 0;
    if (prefix_tokens > 0 && B > 0) {
        const int64_t blocks = ceil_div(B, seqs_per_block);
        // the mma.sync kernel runs ctas_per_sm blocks on an SM, the tcgen05 kernel one
        const int64_t slots = umma ? sm_count : (int64_t)sm_count * ctas_per_sm;
        // chunks of >= 128 tokens; the tcgen05 kernel works in whole 128-token tiles
        const int64_t max_chunks = umma ? ceil_div(prefix_pages, 8) : std::max<int64_t>(1, prefix_pages / 8);
        PC = (int32_t)std::min<int64_t>(max_chunks, std::max<int64_t>(1, slots / (H * blocks)));
        if (p.split_mode == DA_SPLIT_DETERMINISTIC) {
            const int64_t c = min_chunk_pages(s, p);                             // cuts at multiples of the chunk
            PC = (int32_t)std::max<int64_t>(1, ceil_div(prefix_pages, c));
        }
        PC = std::min<int32_t>(PC, max_splits / 2);
        for (int64_t j = 0; j < blocks; ++j) {
            const int b0 = (int)(j * seqs_per_block);
            const int nseq = std::min(seqs_per_block, B - b0);
            for (int32_t i = 0; i < PC; ++i) {
                int64_t pb, pe;
                if (umma && p.split_mode != DA_SPLIT_DETERMINISTIC) {
                    // whole 128-token tiles (8 pages), dealt evenly; the last chunk takes the ragged end
                    const int64_t tiles = ceil_div(prefix_pages, 8);
                    const int64_t q = tiles / PC, r = tiles % PC;
                    pb = std::min<int64_t>(prefix_pages, (i * q + std::min<int64_t>(i, r)) * 8);
                    pe = std::min<int64_t>(prefix_pages, pb + (q + (i < r ? 1 : 0)) * 8);
                } else {
                    const int64_t q = prefix_pages / PC, r = prefix_pages % PC;
                    pb = i * q + std::min<int64_t>(i, r);
                    pe = pb + q + (i < r ? 1 : 0);
                }
                for (int g = 0; g < H; ++g) {
                    decode_attn_unit_t u;
                    u.seq = b0;
                    u.kv_head = g | (nseq << 16);          // high half: sequences in the block
                    u.tok_begin = (int32_t)(pb * P);
                    u.tok_end = (int32_t)(pe * P);
                    u.slot = -2;                            // records go to each sequence's own slots
                    u.seq_len = seq_lens[b0];
                    u.split_index = i;
                    u.n_splits = 0;
                    made.push_back(u);
                    cost.push_back((int32_t)((pe - pb) * 4));     // heavier per page: attended for a whole block of sequences
                }
            }
        }
        n_prefix_units = made.size();
    }

    for (int b = 0; b < B; ++b) {
        const SeqCut& cut = cuts[b];
        const bool has_suffix = prefix_tokens == 0 || cut.pages > 0;
        const int32_t S_own = has_suffix ? cut.splits : 0;
        const int32_t S = PC + S_own;
        out.splits[b] = S;
        out.max_splits_used = std::max(out.max_splits_used, S);
        int64_t base_slot = -1;
        if (S > 1 || prefix_tokens > 0) {
            base_slot = out.n_slots;
            out.slot_base[b] = (int32_t)base_slot;
            out.n_slots += S;
            if (out.n_slots > INT32_MAX) return DA_ERR_UNSUPPORTED;
        }
        const int64_t even_q = S_own > 0 ? cut.pages / S_own : 0, even_r = S_own > 0 ? cut.pages % S_own : 0;
        for (int32_t i = 0; i < S_own; ++i) {
            int64_t pb, pe;
            if (cut.even) {
                const int64_t q = even_q, r = even_r;
                pb = i * q + std::min<int64_t>(i, r);
                pe = pb + q + (i < r ? 1 : 0);
            } else {
                pb = std::min(cut.pages, (int64_t)i * cut.chunk);
                pe = std::min(cut.pages, (int64_t)(i + 1) * cut.chunk);
            }
            decode_attn_unit_t u;
            u.seq = b;
            u.tok_begin = (int32_t)((prefix_pages + pb) * P);
            u.tok_end = (int32_t)std::min<int64_t>((prefix_pages + pe) * P, seq_lens[b]);
            if (u.tok_end < u.tok_begin) u.tok_end = u.tok_begin;
            u.slot = base_slot >= 0 ? (int32_t)(base_slot + PC + i) : -1;
            u.seq_len = seq_lens[b];
            u.split_index = PC + i;
            u.n_splits = S;
            for (int g = 0; g < H; ++g) {
                u.kv_head = g;
                made.push_back(u);
                cost.push_back((int32_t)(pe - pb));
            }
        }
    }
    out.prefix_chunks = PC;
    // Launch order: shared-prefix units first, then most expensive unit first, ties in creation
    // order.  Costs are small integers (16-token tiles of a unit), so a counting sort does it.
    const size_t n = made.size();
    std::vector<uint32_t>& order = out.scratch_order;
    order.resize(n);
    for (size_t i = 0; i < n; ++i) order[i] = (uint32_t)i;
    auto sort_range = [&](size_t lo, size_t hi) {
        bool sorted = true;
        int32_t max_cost = 0;
        for (size_t i = lo; i < hi; ++i) {
            if (i > lo && cost[i - 1] < cost[i]) sorted = false;
            max_cost = std::max(max_cost, cost[i]);
        }
        if (sorted) return;
        if ((size_t)max_cost <= 4 * (hi - lo) + 1024) {
            std::vector<uint32_t>& cnt = out.scratch_count;
            cnt.assign((size_t)max_cost + 2, 0);
            for (size_t i = lo; i < hi; ++i) ++cnt[(size_t)(max_cost - cost[i]) + 1];      // descending cost
            for (size_t c = 1; c < cnt.size(); ++c) cnt[c] += cnt[c - 1];
            for (size_t i = lo; i < hi; ++i) order[lo + cnt[(size_t)(max_cost - cost[i])]++] = (uint32_t)i;
        } else {
            std::stable_sort(order.begin() + lo, order.begin() + hi,
                             [&cost](uint32_t x, uint32_t y) { return cost[x] > cost[y]; });
        }
    };
    sort_range(0, n_prefix_units);
    sort_range(n_prefix_units, n);
    out.units.resize(n);
    out.block_begin.clear();
    out.rank_pos.clear();
    out.n_front_units = 0;
    size_t first = 0;                       // units before this one stay out of the bins
    if (umma) {
        for (; first < n_prefix_units; ++first) out.units[first] = made[order[first]];
        out.n_front_units = (int32_t)first;
    }
    if (max_bins <= 0 || first == n) {
        for (size_t i = first; i < n; ++i) out.units[i] = made[order[i]];
        return DA_OK;
    }
    // Longest unit first onto the lightest bin.  A unit costs its pages (a shared-prefix page
    // counts four times) plus a fixed charge for the hand-over between units.  Loads are small
    // integers that only grow, so the lightest bin is found with a bucket queue: one list of bins
    // per load, the lightest non-empty list never moves down (ties: the bin that got there first).
    constexpr int32_t kHandOverPages = 24;
    const int bins = (int)std::min<int64_t>((int64_t)(n - first), max_bins);
    std::vector<int32_t>& bin_of = out.scratch_bin_of;
    std::vector<int32_t>& count = out.scratch_bin_count;
    bin_of.resize(n);
    count.assign((size_t)bins + 1, 0);
    const bool equal_costs = cost[order[first]] == cost[order[n - 1]] && (first >= n_prefix_units || n_prefix_units == n);
    if ((size_t)bins == n - first) {
        for (size_t i = first; i < n; ++i) bin_of[i] = (int32_t)(i - first);      // a bin for every unit
    } else if (equal_costs) {
        for (size_t i = first; i < n; ++i) bin_of[i] = (int32_t)((i - first) % bins);   // what the rule below would do
    } else {
        int64_t total = 0;
        int32_t biggest = 0;
        for (size_t i = first; i < n; ++i) {
            total += cost[order[i]] + kHandOverPages;
            biggest = std::max(biggest, cost[order[i]] + kHandOverPages);
        }
        // no bin's load passes the mean by more than the biggest unit (the lightest bin is never above the mean)
        const size_t levels = (size_t)(total / bins + 2 * (int64_t)biggest + 2);
        std::vector<int32_t>& head = out.scratch_level_head;     // first bin of each load's list, -1: empty
        std::vector<int32_t>& tail = out.scratch_level_tail;
        std::vector<int32_t>& next = out.scratch_bin_next;       // next bin in the same list
        std::vector<int32_t>& load = out.scratch_bin_load;
        head.assign(levels, -1);
        tail.assign(levels, -1);
        next.assign((size_t)bins, -1);
        load.assign((size_t)bins, 0);
        for (int i = 0; i < bins; ++i) {                         // all bins start at load 0, in index order
            next[i] = i + 1 < bins ? i + 1 : -1;
        }
        head[0] = 0;
        tail[0] = bins - 1;
        size_t lightest = 0;
        for (size_t i = first; i < n; ++i) {
            while (head[lightest] < 0) ++lightest;
            const int32_t b = head[lightest];
            head[lightest] = next[b];
            if (head[lightest] < 0) tail[lightest] = -1;
            bin_of[i] = b;
            load[b] += cost[order[i]] + kHandOverPages;
            const size_t l = (size_t)load[b];
            next[b] = -1;
            if (tail[l] < 0) head[l] = b; else next[tail[l]] = b;
            tail[l] = b;
        }
    }
    // counting sort by bin, keeping the order within a bin
    for (size_t i = first; i < n; ++i) ++count[bin_of[i] + 1];
    out.block_begin.resize(bins);
    int32_t run = (int32_t)first;
    for (int b = 0; b < bins; ++b) {
        out.block_begin[b] = run;
        run += count[b + 1];
        count[b + 1] = out.block_begin[b];      // becomes the bin's write cursor
    }
    out.rank_pos.resize(n - first);
    for (size_t i = first; i < n; ++i) {
        const int32_t pos = count[bin_of[i] + 1]++;
        out.units[pos] = made[order[i]];
        out.rank_pos[i - first] = pos;
    }
    out.block_begin.push_back((int32_t)out.units.size());
    return DA_OK;
}

}  // namespace da

extern "C" int decode_attn_plan_layout(const decode_attn_shape_t* shape, const decode_attn_policy_t* policy,
                                       const int32_t* seq_lens_host, int32_t sm_count, int32_t ctas_per_sm,
                                       decode_attn_unit_t* units_out, int64_t max_units, int64_t* n_units_out,
                                       int32_t* splits_out, int32_t* slot_base_out, int64_t* n_slots_out,
                                       int32_t* chunk_tokens_out)
{
    if (!shape || !policy) return DA_ERR_INVALID_ARG;
    int rc = da::validate_shape(*shape);
    if (rc != DA_OK) return rc;
    rc = da::validate_policy(*shape, *policy);
    if (rc != DA_OK) return rc;
    da::Layout lay;
    rc = da::make_layout(*shape, *policy, seq_lens_host, sm_count, ctas_per_sm, lay);
    if (rc != DA_OK) return rc;
    if (n_units_out) *n_units_out = (int64_t)lay.units.size();
    if (n_slots_out) *n_slots_out = lay.n_slots;
    if (chunk_tokens_out) *chunk_tokens_out = lay.chunk_tokens;
    for (int b = 0; b < shape->batch; ++b) {
        if (splits_out) splits_out[b] = lay.splits[b];
        if (slot_base_out) slot_base_out[b] = lay.slot_base[b];
    }
    if (units_out) {
        if (max_units < (int64_t)lay.units.size()) return DA_ERR_INVALID_ARG;
        std::copy(lay.units.begin(), lay.units.end(), units_out);
    }
    return DA_OK;
}

// ---------------------------------------------------------------------------
// Decode profitability rule (Section 3.3, Appendix D).  Host arithmetic only.
// ---------------------------------------------------------------------------
extern "C" int decode_attn_breakeven_tokens(double tau_seconds, double bandwidth_bytes_per_s, double skip_fraction,
                                            int32_t routed_layers, double kv_bytes_per_token_layer, double* v_star_out)
{
    if (!v_star_out) return DA_ERR_INVALID_ARG;
    if (!(tau_seconds >= 0.0) || !(bandwidth_bytes_per_s > 0.0) || !(skip_fraction > 0.0) || skip_fraction > 1.0 ||
        routed_layers <= 0 || !(kv_bytes_per_token_layer > 0.0))
        return DA_ERR_INVALID_ARG;
    *v_star_out = tau_seconds * bandwidth_bytes_per_s / (skip_fraction * (double)routed_layers * kv_bytes_per_token_layer);
    return DA_OK;
}

extern "C" int decode_attn_switch_thresholds(double v_star, double round_to, double* exit_tokens_out,
                                             double* enter_tokens_out)
{
    if (!exit_tokens_out || !enter_tokens_out || !(v_star >= 0.0) || !(round_to >= 0.0)) return DA_ERR_INVALID_ARG;
    double ex = v_star, en = 1.25 * v_star;
    if (round_to > 0.0) {
        ex = std::floor(ex / round_to + 0.5) * round_to;
        en = std::floor(en / round_to + 0.5) * round_to;
    }
    *exit_tokens_out = ex;
    *enter_tokens_out = en;
    return DA_OK;
}

extern "C" int decode_attn_switch_next(int32_t routed_now, double resident_tokens, double exit_tokens,
                                       double enter_tokens)
{
    if (resident_tokens >= enter_tokens) return 1;
    if (resident_tokens <= exit_tokens) return 0;
    return routed_now ? 1 : 0;
}
