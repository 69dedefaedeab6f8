// Host planner: turns the per-sequence lengths of one mixed batch into work items for the
// split-K decode kernel, the combine kernel and the chunked-prefill kernel.
// The batch is the one the paper's decode worker builds from its resident decode sequences plus
// its local prefill queue (Section 5); the planner only partitions work, it does no arithmetic
// on tensor data.
#pragma once
#include <cstdint>
#include <vector>

#include "../../include/crossflow_attn.h"

namespace cf {

struct DecodeItem {        // one (decode sequence, KV chunk); the kernel adds the KV-head index
    int32_t seq;
    int32_t q_row;         // packed row of the sequence's single query token
    int32_t kv_begin;      // first visible token of the chunk (multiple of block_size)
    int32_t kv_end;        // one past the last token (== context_len for the last chunk)
    int32_t part_slot;     // partial slot to write, or -1: the only chunk, write `out` directly
    int32_t chunk;         // index of this chunk within its sequence
    int32_t n_chunks;      // chunks of the sequence (its partial slots are part_slot - chunk + [0, n_chunks))
    int32_t pad;
};

struct CombineItem {       // one decode sequence that was split
    int32_t q_row;
    int32_t part_first;    // its chunks occupy slots [part_first, part_first + n_chunks)
    int32_t n_chunks;
};

struct PrefillItem {       // one q tile of one prefill chunk; the kernel adds the head index
    int32_t seq;
    int32_t q_row0;        // packed row of the tile's first row
    int32_t row0;          // index of that row inside the chunk (0-based)
    int32_t n_rows;        // rows in this tile (<= tile height)
};

struct PrefillTcItem {     // tcgen05 kernel: two 128-row q tiles that share one KV head (tile 1 may be absent)
    int32_t seq;
    int32_t kvh;
    int32_t q_row0[2];     // packed row of each tile's first row
    int32_t row0[2];       // index of that row inside the chunk
    int32_t n_rows[2];     // 0 = tile absent
    int32_t head[2];       // query head of each tile
    // KV split: this item covers KV tiles [j_begin, j_end) (128-token tiles; j_end clamps to the item's
    // own extent).  part_slot[t] >= 0: tile t writes an fp32 partial for row r into slot
    // part_slot[t] + r * part_k + part_c instead of the final output.
    int32_t j_begin, j_end;
    int32_t part_slot[2];
    int32_t part_k, part_c;
    int32_t prefix, ctx_len;   // of the sequence (copied here so that a role needs one load per item)
    int32_t pad[2];            // 80 bytes: five 16-byte words
};
static_assert(sizeof(PrefillTcItem) == 80, "PrefillTcItem is copied as five 16-byte words");

struct PrefillCombineItem { // one KV-split tcgen05 item: merges its part_k partials per row
    int32_t q_row0[2];
    int32_t n_rows[2];
    int32_t head[2];
    int32_t part_slot[2];
    int32_t part_k;
};

struct PlanConfig {
    int32_t num_sms = 148;
    int32_t decode_ctas_per_sm = 2;   // resident decode CTAs per SM the kernel is built for
    int32_t decode_waves = 4;         // target number of CTA waves (load balance vs. partial traffic)
    int32_t decode_min_chunk_pages = 32;
    int32_t decode_page_quantum = 4;  // chunk lengths are multiples of this many pages (warps per CTA)
    int32_t prefill_tile_rows = 64;   // tile height of the mma.sync prefill kernel
    bool prefill_tc = false;          // true: plan items for the tcgen05 kernel (128-row tile pairs)
    int32_t prefill_sms_mixed = 0;    // > 0: SMs the prefill items are balanced over when the batch also holds decode
                                      // work (spatial launch sequence: the first prefill grid's share); 0: num_sms
    int32_t prefill_force_split = 0;  // >= 2: split every tcgen05 item that many ways (tests); 0: cost model decides
};

struct Plan {
    std::vector<int32_t> q_start;     // [S+1] exclusive prefix sum of query_len
    std::vector<DecodeItem> decode;   // longest chunk first
    std::vector<CombineItem> combine;
    std::vector<PrefillItem> prefill; // longest KV extent first (mma.sync kernel)
    std::vector<PrefillTcItem> prefill_tc;   // longest KV extent first (tcgen05 kernel); KV-split items appear part_k times
    std::vector<PrefillCombineItem> prefill_combine;   // one per KV-split item
    int32_t n_pre_slots = 0;          // fp32 partial rows of KV-split prefill items (compact, D floats each)
    int32_t n_part_slots = 0;
    int32_t total_q = 0;
    int32_t n_decode_seqs = 0;
    int32_t n_prefill_seqs = 0;
};

// Validates geometry (supported head_dim / block_size / group / strides).
cf_status validate_desc(const cf_cache_desc* d);
// Validates lengths against the block-table width; fills q_start/total_q.
cf_status validate_lengths(const cf_cache_desc* d, const int32_t* context_len, const int32_t* query_len,
                           int32_t num_seqs, int32_t max_blocks_per_seq, Plan* plan);
// Full plan (calls validate_lengths).
cf_status build_plan(const cf_cache_desc* d, const int32_t* context_len, const int32_t* query_len,
                     int32_t num_seqs, int32_t max_blocks_per_seq, const PlanConfig& cfg, Plan* plan);

// Predicted device time of one cf_mixed_attention call, in microseconds, from a model fitted to this
// library's measured kernel times on B200 (decode: fixed cost + bytes at the sustained split-K rate;
// prefill: work items scheduled longest-first onto the SMs, each costing a fixed part plus a time per
// 128-token KV tile).  Meant for deriving a lease's compute credit from a latency headroom (Section 4.2).
struct Estimate {
    float us_decode = 0.f, us_combine = 0.f, us_prefill = 0.f;
};
// Time the tcgen05 prefill items would take spread evenly over num_sms SMs, divided by the time of the
// decode kernel (same constants as estimate_us; no scheduling, O(items)).  0 when either part is absent.
float prefill_to_decode_ratio(const cf_cache_desc* d, const int32_t* context_len, const int32_t* query_len, const Plan& plan,
                              int32_t num_sms);
Estimate estimate_us(const cf_cache_desc* d, const int32_t* context_len, const int32_t* query_len, const Plan& plan,
                     int32_t num_sms);

}  // namespace cf
