// Host-side split-KV planner: length mix -> work list.  Pure integer work, no
// CUDA calls, so it is also what the CPU tests exercise.
#pragma once

#include <cstdint>
#include <vector>

#include "decode_attn.h"

namespace da {

constexpr int kDefaultDeterministicChunk = 256;   // tokens: the floor; the bound of 32 splits lengthens it above 8,192 tokens
constexpr int kTileTokens = 16;                  // what the kernels fetch at a time; pages hold a power-of-two number of these
constexpr int kDefaultAutoMinChunk = 256;         // tokens
constexpr int kDefaultMaxSplits = 512;
constexpr int kDefaultDeterministicMaxSplits = 32;
constexpr int kMaxSplits = 1024;  // hard bound on the splits of one sequence
constexpr int kMaxGroup = 16;
constexpr int kPrefixColumns = 16;  // query rows (sequence x head) one shared-prefix unit attends at once
constexpr int kUmmaPrefixRows = 128;       // the same for the tcgen05 prefix kernel (the M dimension of its MMAs)

struct Layout {
    std::vector<decode_attn_unit_t> units;  // launch order: most expensive first
    std::vector<int32_t> splits;            // [batch]
    std::vector<int32_t> slot_base;         // [batch], -1 when the sequence has one split
    int64_t n_slots = 0;
    int32_t chunk_tokens = 0;
    int32_t max_splits_used = 0;
    int32_t prefix_chunks = 0;              // chunks the shared prefix is cut into (0: no shared prefix)
    int32_t n_front_units = 0;              // shared-prefix units kept at the front, outside the bins, for a
                                            // kernel of their own (policy kernel DA_KERNEL_UMMA_PREFIX)
    std::vector<int32_t> block_begin;       // [bins + 1] when the units were packed into bins, else empty
    std::vector<int32_t> rank_pos;          // binned layouts: position in `units` of the binned unit with cost rank j
                                            // (j = 0: most expensive; ties in creation order)
    // working storage of make_layout, kept so that a layout that is refilled every step allocates nothing
    std::vector<decode_attn_unit_t> scratch_units;
    std::vector<int32_t> scratch_cost, scratch_bin_of, scratch_bin_count, scratch_level_head, scratch_level_tail,
        scratch_bin_next, scratch_bin_load;
    std::vector<uint32_t> scratch_order, scratch_count;
};

// Validates the fields the planner and the kernels rely on.
int validate_shape(const decode_attn_shape_t& s);
int validate_policy(const decode_attn_shape_t& s, const decode_attn_policy_t& p);

// Fills `out` for the given lengths.  sm_count and ctas_per_sm must be > 0.
// max_bins > 0: the units are additionally packed into min(units, max_bins) bins of about equal
// cost (longest unit first onto the lightest bin) and stored bin by bin; block b of the persistent
// kernel walks bin b.  With policy kernel DA_KERNEL_UMMA_PREFIX the shared-prefix units are cut for the
// tcgen05 kernel (128 query rows, chunks of whole 128-token tiles), come first in `units` and stay out of
// the bins; block_begin then indexes the units behind them.
int make_layout(const decode_attn_shape_t& s, const decode_attn_policy_t& p, const int32_t* seq_lens,
                int sm_count, int ctas_per_sm, Layout& out, int max_bins = 0);

// Upper bounds for a capacity plan (any batch <= capacity_batch and
// sum(seq_lens) <= capacity_tokens).
int64_t capacity_slots(const decode_attn_shape_t& s, const decode_attn_policy_t& p);

}  // namespace da
