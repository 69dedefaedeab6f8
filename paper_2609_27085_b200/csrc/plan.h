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
    int32_t kv_lo;         // first visible token of the sequence (left edge of a sliding window; 0 without one):
                           // tokens of this chunk below it are masked (only the first chunk can hold any)
};

// Shared prefix (radix-cache reuse, Section 4.4: a lookup tells how much of a prompt is already resident; agent
// turns share long prefixes): decode sequences of one share group point at the same physical pages for the first
// `shared_len` tokens.  Those pages are streamed once per KV chunk for a whole set of members, whose query heads
// ride along as extra MMA columns; every member gets a partial per shared chunk, merged with the partials of
// its own suffix by the usual split-K merge.
struct SharedDecodeItem {  // one (share group, shared KV chunk, member set); the kernel adds the KV-head index
    int32_t seq;           // the member whose block-table row is read for the shared pages
    int32_t kv_begin;      // whole pages of the shared prefix: [kv_begin, kv_end)
    int32_t kv_end;
    int32_t chunk;         // index of this chunk in every member's chunk list (shared chunks come first)
    int32_t member_first;  // first entry of this set in the member list
    int32_t n_members;     // members in the set (<= kSharedColumns / G)
    int32_t pad[2];
};
struct ShareMember {       // one member of a set
    int32_t q_row;         // packed row of its query token
    int32_t part_first;    // first partial slot of the sequence (its chunk c writes slot part_first + c)
    int32_t n_chunks;      // chunks of the sequence, shared ones and its own
    int32_t pad;
};
constexpr int32_t kSharedColumns = 16;      // query-head columns a shared-prefix CTA carries (two 8-wide MMA operands)
constexpr int32_t kMinSharedPages = 16;     // shorter shared prefixes are not worth a separate pass

struct CombineItem {       // one decode sequence that was split
    int32_t q_row;
    int32_t part_first;    // its chunks occupy slots [part_first, part_first + n_chunks)
    int32_t n_chunks;
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
    int32_t page_lo;           // first page of the sequence any row of the item can see (sliding window; 0 without
                               // one): pages below it are neither fetched nor multiplied
    int32_t pad;               // pair items (two CTAs, four q tiles): offset of the second CTA's partial slots from
                               // part_slot[]; 0 otherwise.  80 bytes: five 16-byte words
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
    int32_t prefill_sms_mixed = 0;    // > 0: SMs the prefill items are balanced over when the batch also holds decode
                                      // work (spatial launch sequence: the first prefill grid's share); 0: num_sms
    int32_t prefill_force_split = 0;  // >= 2: split every tcgen05 item that many ways (tests); 0: cost model decides
    bool prefill_pair = false;        // plan for the two-CTA kernel where the geometry allows it (head_dim 128, group
                                      // size a multiple of 4): an item carries four heads, the machine has num_sms / 2 slots
};

struct Plan {
    std::vector<int32_t> q_start;     // [S+1] exclusive prefix sum of query_len
    std::vector<DecodeItem> decode;   // longest chunk first
    std::vector<CombineItem> combine;
    std::vector<SharedDecodeItem> shared_decode;   // shared-prefix chunks (empty unless the caller described sharing)
    std::vector<ShareMember> share_members;
    std::vector<PrefillTcItem> prefill_tc;   // longest KV extent first (tcgen05 kernel); KV-split items appear part_k times
    std::vector<PrefillCombineItem> prefill_combine;   // one per KV-split item
    int32_t n_pre_slots = 0;          // fp32 partial rows of KV-split prefill items (compact, D floats each)
    int32_t n_part_slots = 0;
    int32_t total_q = 0;
    int32_t n_decode_seqs = 0;
    int32_t n_prefill_seqs = 0;
    bool pair = false;                // prefill_tc items are pair items (four q tiles, two CTAs)
};

// Validates geometry (supported head_dim / block_size / group / strides).
cf_status validate_desc(const cf_cache_desc* d);
// Validates lengths against the block-table width; fills q_start/total_q.
cf_status validate_lengths(const cf_cache_desc* d, const int32_t* context_len, const int32_t* query_len,
                           int32_t num_seqs, int32_t max_blocks_per_seq, Plan* plan);
// Decode chunking, shared by build_plan and by the allocation-free entry point (plain loops over the
// caller's arrays: nothing here allocates).  `lc_of(s)` returns the context length of sequence s if it is
// a decode sequence and a negative number otherwise.
//   decode_target_pages: the chunk length (in pages) that fills the machine `decode_waves` times, or, for a
//     batch too small for that, the length from [min, 4 x min] with the smallest waves x CTA time.
//   decode_split: near-equal chunks of at most `target` pages, each a multiple of the page quantum.
template <class LcOf>
inline int64_t decode_target_pages(int32_t num_seqs, LcOf lc_of, int32_t B, int32_t Hkv, int32_t D, const PlanConfig& cfg,
                                   bool shares_sms, int64_t extra_pages = 0)
{
    const int64_t wave = (int64_t)(cfg.num_sms > 1 ? cfg.num_sms : 1) * (cfg.decode_ctas_per_sm > 1 ? cfg.decode_ctas_per_sm : 1);
    const int64_t slots = wave * (cfg.decode_waves > 1 ? cfg.decode_waves : 1);
    const int64_t quantum = cfg.decode_page_quantum > 1 ? cfg.decode_page_quantum : 1;
    const int64_t min_pages = cfg.decode_min_chunk_pages > 1 ? cfg.decode_min_chunk_pages : 1;
    int64_t total_pages = 0;
    for (int32_t s = 0; s < num_seqs; ++s) {
        const int64_t lc = lc_of(s);
        if (lc >= 0) total_pages += (lc + B - 1) / B;
    }
    total_pages += extra_pages;                         // pages streamed by shared-prefix items
    int64_t target = (total_pages * Hkv + slots - 1) / slots;
    if (target < min_pages && total_pages > 0 && !shares_sms && extra_pages == 0) {
        // A small batch: chunks of the minimum length would not fill `decode_waves` waves, and how many waves
        // of (num_sms x ctas_per_sm) CTAs they do fall into decides the time (a last wave that is a quarter
        // full costs a whole CTA time).  Try chunk lengths from the minimum to four times it and keep the
        // one with the smallest waves x (CTA start-up + chunk streaming time).  (Not when decode shares the SMs
        // with a prefill grid: there the short chunks measured better.)
        const double page_us = (2.0 * B * D * 2.0) / (7.56e6 / (double)wave);   // one (page, head) of K and V at a CTA's share of HBM
        const double cta_us = 2.5;
        double best = 1e30;
        int64_t best_c = min_pages;
        for (int64_t c = (min_pages + quantum - 1) / quantum * quantum; c <= 4 * min_pages; c += quantum) {
            int64_t ctas = 0, longest = 0;
            for (int32_t s = 0; s < num_seqs; ++s) {
                const int64_t lc = lc_of(s);
                if (lc < 0) continue;
                const int64_t pages = (lc + B - 1) / B;
                int64_t n = (pages + c - 1) / c;
                if (n < 1) n = 1;
                const int64_t per = ((pages + n - 1) / n + quantum - 1) / quantum * quantum;
                n = per > 0 ? (pages + per - 1) / per : 1;
                ctas += n;
                const int64_t len = per < pages ? per : pages;
                if (len > longest) longest = len;
            }
            ctas *= Hkv;
            const double t = (double)((ctas + wave - 1) / wave) * (cta_us + page_us * (double)longest);
            if (t < best * 0.999) { best = t; best_c = c; }
        }
        target = best_c;
    }
    if (target < min_pages) target = min_pages;
    return (target + quantum - 1) / quantum * quantum;
}
inline void decode_split(int64_t pages, int64_t target, int32_t quantum, int64_t* n_chunks, int64_t* pages_per_chunk)
{
    const int64_t qn = quantum > 1 ? quantum : 1;
    int64_t n = (pages + target - 1) / target;
    if (n < 1) n = 1;
    int64_t per = (pages + n - 1) / n;
    per = (per + qn - 1) / qn * qn;
    if (per < qn) per = qn;
    *n_chunks = (pages + per - 1) / per > 0 ? (pages + per - 1) / per : 1;
    *pages_per_chunk = per;
}

// Full plan (calls validate_lengths).
// share_group / shared_len (both or neither; HOST [num_seqs]): share_group[s] >= 0 names the group of sequence s,
// whose members have identical block-table entries for the first shared_len[s] tokens; < 0: shares nothing.
cf_status build_plan(const cf_cache_desc* d, const int32_t* context_len, const int32_t* query_len,
                     int32_t num_seqs, int32_t max_blocks_per_seq, const PlanConfig& cfg, Plan* plan,
                     const int32_t* share_group = nullptr, const int32_t* shared_len = nullptr);

// Predicted device time of one cf_mixed_attention call, in microseconds, from a model fitted to this
// library's measured kernel times on B200 (decode: fixed cost + bytes at the sustained split-K rate;
// prefill: work items scheduled longest-first onto the SMs, each costing a fixed part plus a time per
// 128-token KV tile).  Meant for deriving a lease's compute credit from a latency headroom (Section 4.2).
struct Estimate {
    float us_decode = 0.f, us_combine = 0.f, us_prefill = 0.f;
};
// Spatial launch sequence: how many SMs the first prefill grid takes when a batch holds decode and prefill work
// (0 when either part is absent).  Computed from the lengths alone, before the plan exists, because the planner
// balances the prefill items over this many SMs.  Decode gets what it needs to be done when the prefill is, and no
// more: it saturates HBM from k_sat SMs (about 65 with up to four heads per KV head, about 100 with eight, where the
// MMAs per byte double), so over a call of length T it needs k_sat * t_decode / T of them, taken with a margin of 1.15;
// the share of the prefill grid is clamped to [3/5, 7/8] of the SMs.  t_decode and the prefill work come from the
// constants of estimate_us.  Fitted against sweeps of the share on the bench configurations (within a few per
// cent of the best share on each).
int32_t spatial_front_sms(const cf_cache_desc* d, const int32_t* context_len, const int32_t* query_len, int32_t num_seqs,
                          int32_t num_sms);
Estimate estimate_us(const cf_cache_desc* d, const int32_t* context_len, const int32_t* query_len, const Plan& plan,
                     int32_t num_sms);

}  // namespace cf
