#include "plan.h"

#include <algorithm>
#include <climits>
#include <cmath>
#include <functional>
#include <queue>
#include <utility>
#include <cstdint>

#ifndef CF_KV_SET_BYTES
#define CF_KV_SET_BYTES (80ll << 20)
#endif
namespace cf {

// Makespan of jobs taken in the given order by whichever of m machines is free first (what the GPU's
// block scheduler does with a grid of one-CTA-per-SM work items).
static double list_schedule(const std::vector<double>& jobs, size_t m)
{
    if (jobs.size() <= m) return jobs.empty() ? 0.0 : *std::max_element(jobs.begin(), jobs.end());
    std::priority_queue<double, std::vector<double>, std::greater<double>> free_at;
    for (size_t i = 0; i < m; ++i) free_at.push(0.0);
    double end = 0.0;
    for (double j : jobs) {
        const double t = free_at.top() + j;
        free_at.pop();
        free_at.push(t);
        end = std::max(end, t);
    }
    return end;
}

cf_status validate_desc(const cf_cache_desc* d)
{
    if (!d) return CF_ERR_INVALID_ARG;
    if (d->num_q_heads <= 0 || d->num_kv_heads <= 0 || d->num_blocks <= 0) return CF_ERR_INVALID_ARG;
    if (d->num_q_heads % d->num_kv_heads != 0) return CF_ERR_INVALID_ARG;
    const int g = d->num_q_heads / d->num_kv_heads;
    if (d->head_dim != 64 && d->head_dim != 128) return CF_ERR_UNSUPPORTED;
    if (d->block_size != 16) return CF_ERR_UNSUPPORTED;
    if (g != 1 && g != 2 && g != 4 && g != 8) return CF_ERR_UNSUPPORTED;
    const int64_t st[6] = {d->k_stride_block, d->k_stride_head, d->k_stride_token,
                           d->v_stride_block, d->v_stride_head, d->v_stride_token};
    for (int i = 0; i < 6; ++i) {
        if (st[i] <= 0) return CF_ERR_INVALID_ARG;
        if (st[i] % 8 != 0) return CF_ERR_UNSUPPORTED;
    }
    if (d->k_stride_token < d->head_dim || d->v_stride_token < d->head_dim) return CF_ERR_INVALID_ARG;
    if (!(d->softmax_scale >= 0.0f)) return CF_ERR_INVALID_ARG;   // also rejects NaN
    if (d->window_size < 0) return CF_ERR_INVALID_ARG;
    if (d->kv_dtype != CF_KV_BF16 && d->kv_dtype != CF_KV_FP8_E4M3) return CF_ERR_INVALID_ARG;
    if (d->kv_dtype == CF_KV_FP8_E4M3) {
        if (d->head_dim != 128) return CF_ERR_UNSUPPORTED;
        if (!d->k_scale || !d->v_scale) return CF_ERR_INVALID_ARG;
        for (int i = 0; i < 6; ++i)
            if (st[i] % 16 != 0) return CF_ERR_UNSUPPORTED;          // 16-byte copies of one-byte elements
    }
    return CF_OK;
}

cf_status validate_lengths(const cf_cache_desc* d, const int32_t* context_len, const int32_t* query_len,
                           int32_t num_seqs, int32_t max_blocks_per_seq, Plan* plan)
{
    if (num_seqs < 0 || max_blocks_per_seq < 0) return CF_ERR_INVALID_ARG;
    if (num_seqs > 0 && (!context_len || !query_len)) return CF_ERR_INVALID_ARG;
    plan->q_start.assign((size_t)num_seqs + 1, 0);
    int64_t total = 0;
    for (int32_t s = 0; s < num_seqs; ++s) {
        const int32_t lq = query_len[s], lc = context_len[s];
        if (lq < 0 || lc < 0 || lq > lc) return CF_ERR_INVALID_ARG;
        if ((int64_t)lc > (int64_t)max_blocks_per_seq * d->block_size) return CF_ERR_OUT_OF_RANGE;
        total += lq;
        if (total > (int64_t)1 << 30) return CF_ERR_OUT_OF_RANGE;
        plan->q_start[(size_t)s + 1] = (int32_t)total;
    }
    plan->total_q = (int32_t)total;
    return CF_OK;
}

cf_status build_plan(const cf_cache_desc* d, const int32_t* context_len, const int32_t* query_len,
                     int32_t num_seqs, int32_t max_blocks_per_seq, const PlanConfig& cfg, Plan* plan,
                     const int32_t* share_group, const int32_t* shared_len)
{
    *plan = Plan();
    cf_status st = validate_lengths(d, context_len, query_len, num_seqs, max_blocks_per_seq, plan);
    if (st != CF_OK) return st;
    const int32_t B = d->block_size;

    // ---- decode: near-equal KV chunks, sized so that (chunks x kv heads) fills the machine a few times
    for (int32_t s = 0; s < num_seqs; ++s)
        if (query_len[s] == 1) ++plan->n_decode_seqs;
        else if (query_len[s] > 1) ++plan->n_prefill_seqs;
    const int32_t quantum = std::max(1, cfg.decode_page_quantum);
    const bool shares_sms = cfg.prefill_sms_mixed > 0 && plan->n_prefill_seqs > 0;   // spatial sequence: decode runs on part of the machine, beside prefill
    // With a sliding window a decode token at position Lc - 1 sees keys [Lc - W, Lc): the chunks cover the pages
    // from the one that holds the window's left edge onwards, and nothing left of it is ever touched.
    const int32_t W = d->window_size;
    auto first_page_of = [&](int32_t lc) -> int64_t { return (W > 0 && lc > W) ? (lc - W) / B : 0; };

    // Shared prefixes: decode sequences of a group (at least two, full attention) whose common prefix is at least
    // kMinSharedPages pages long leave those pages to shared items; their own chunks start behind them.
    // shared_pages[s] = pages of sequence s that a shared item covers (0: none).
    const int32_t G = d->num_q_heads / d->num_kv_heads;
    std::vector<int32_t> shared_pages;
    struct GroupInfo { int32_t group; int32_t pages; std::vector<int32_t> members; };
    std::vector<GroupInfo> groups_sh;
    int64_t extra_pages = 0;
    if (share_group != nullptr && shared_len != nullptr && W == 0 && d->kv_dtype == CF_KV_BF16) {
        std::vector<std::pair<int32_t, int32_t>> keyed;          // (group, sequence) of the decode sequences that share
        for (int32_t s = 0; s < num_seqs; ++s)
            if (query_len[s] == 1 && share_group[s] >= 0 && shared_len[s] > 0) keyed.emplace_back(share_group[s], s);
        std::sort(keyed.begin(), keyed.end());
        for (size_t i = 0; i < keyed.size();) {
            size_t j = i;
            int32_t pages = INT32_MAX;
            while (j < keyed.size() && keyed[j].first == keyed[i].first) {
                const int32_t s = keyed[j].second;
                // a sequence's new token is never part of the shared prefix
                pages = std::min(pages, std::min(shared_len[s], context_len[s] - 1) / B);
                ++j;
            }
            if (j - i >= 2 && pages >= kMinSharedPages) {
                GroupInfo gi;
                gi.group = keyed[i].first;
                gi.pages = pages;
                for (size_t m = i; m < j; ++m) gi.members.push_back(keyed[m].second);
                const int64_t sets = ((int64_t)gi.members.size() * G + kSharedColumns - 1) / kSharedColumns;
                extra_pages += sets * pages;
                groups_sh.push_back(std::move(gi));
            }
            i = j;
        }
        if (!groups_sh.empty()) {
            shared_pages.assign((size_t)num_seqs, 0);
            for (const GroupInfo& gi : groups_sh)
                for (int32_t s : gi.members) shared_pages[(size_t)s] = gi.pages;
        }
    }
    auto own_first_page = [&](int32_t s) -> int64_t {
        return shared_pages.empty() ? first_page_of(context_len[s]) : (int64_t)shared_pages[(size_t)s];
    };
    const int64_t target = decode_target_pages(
        num_seqs,
        [&](int32_t s) -> int64_t { return query_len[s] == 1 ? (int64_t)context_len[s] - own_first_page(s) * B : -1; },
        B, d->num_kv_heads, d->head_dim, cfg, shares_sms, extra_pages);

    // chunks of the shared part of every group, the same for all of its members
    std::vector<int32_t> n_shared_chunks;      // per sequence
    std::vector<int64_t> shared_per;           // per group: pages per shared chunk
    if (!groups_sh.empty()) {
        n_shared_chunks.assign((size_t)num_seqs, 0);
        for (const GroupInfo& gi : groups_sh) {
            int64_t n = 1, per = gi.pages;
            decode_split(gi.pages, target, quantum, &n, &per);
            shared_per.push_back(per);
            for (int32_t s : gi.members) n_shared_chunks[(size_t)s] = (int32_t)n;
        }
    }

    std::vector<int32_t> part_first_of, n_chunks_of;   // per sequence: its first partial slot (-1: writes out directly), its chunks
    if (!groups_sh.empty()) {
        part_first_of.assign((size_t)num_seqs, -1);
        n_chunks_of.assign((size_t)num_seqs, 0);
    }
    for (int32_t s = 0; s < num_seqs; ++s) {
        if (query_len[s] != 1) continue;
        const int32_t lc = context_len[s];
        const int64_t page0 = own_first_page(s);
        const int64_t pages = (lc + B - 1) / B - page0;
        const int32_t n_sh = n_shared_chunks.empty() ? 0 : n_shared_chunks[(size_t)s];
        int64_t n = 1, per = pages;
        decode_split(pages, target, quantum, &n, &per);
        const int32_t n_all = (int32_t)n + n_sh;
        int32_t first = -1;
        if (n_all > 1) {
            first = plan->n_part_slots;
            plan->combine.push_back(CombineItem{plan->q_start[s], first, n_all});
            plan->n_part_slots += n_all;
            if (!part_first_of.empty()) {
                part_first_of[(size_t)s] = first;
                n_chunks_of[(size_t)s] = n_all;
            }
        }
        for (int64_t c = 0; c < n; ++c) {
            DecodeItem it;
            it.seq = s;
            it.q_row = plan->q_start[s];
            it.kv_begin = (int32_t)((page0 + c * per) * B);
            it.kv_end = (int32_t)std::min<int64_t>((page0 + (c + 1) * per) * B, lc);
            it.part_slot = n_all > 1 ? first + n_sh + (int32_t)c : -1;
            it.chunk = n_sh + (int32_t)c;
            it.n_chunks = n_all;
            it.kv_lo = (W > 0 && lc > W) ? lc - W : 0;
            plan->decode.push_back(it);
        }
    }
    // shared items: per group, member sets of kSharedColumns / G sequences, one item per (set, shared chunk)
    for (size_t gi_idx = 0; gi_idx < groups_sh.size(); ++gi_idx) {
        const GroupInfo& gi = groups_sh[gi_idx];
        const int64_t per = shared_per[gi_idx];
        const int32_t n_sh = n_shared_chunks[(size_t)gi.members[0]];
        const int32_t per_set = std::max(1, kSharedColumns / G);
        for (size_t m0 = 0; m0 < gi.members.size(); m0 += (size_t)per_set) {
            const int32_t n_mem = (int32_t)std::min<size_t>((size_t)per_set, gi.members.size() - m0);
            const int32_t member_first = (int32_t)plan->share_members.size();
            for (int32_t m = 0; m < n_mem; ++m) {
                const int32_t s = gi.members[m0 + (size_t)m];
                plan->share_members.push_back(ShareMember{plan->q_start[s], part_first_of[(size_t)s], n_chunks_of[(size_t)s], 0});
            }
            for (int32_t c = 0; c < n_sh; ++c) {
                SharedDecodeItem it;
                it.seq = gi.members[m0];
                it.kv_begin = (int32_t)(c * per * B);
                it.kv_end = (int32_t)std::min<int64_t>((c + 1) * per, gi.pages) * B;
                it.chunk = c;
                it.member_first = member_first;
                it.n_members = n_mem;
                it.pad[0] = it.pad[1] = 0;
                plan->shared_decode.push_back(it);
            }
        }
    }
    std::stable_sort(plan->decode.begin(), plan->decode.end(), [](const DecodeItem& a, const DecodeItem& b) {
        return (a.kv_end - a.kv_begin) > (b.kv_end - b.kv_begin);
    });

    // ---- prefill: q tiles of every chunk, the tile with the longest visible KV range first
    {
        // pairs of 128-row tiles that share a KV head: two heads of a group over the same rows, or
        // (group size 1) two consecutive row tiles of one head
        constexpr int32_t TR = 128;
        // pair items: four heads of a group per item, run by two CTAs on two SMs
        const bool pair = cfg.prefill_pair && d->head_dim == 128 && G % 4 == 0;
        const int32_t heads_per_item = pair ? 4 : 2;
        plan->pair = pair;
        struct KeyedTc { int64_t extent; int32_t tiles; PrefillTcItem it; };   // extent: end of the visible keys; tiles: KV tiles to visit
        std::vector<KeyedTc> items;
        auto prefix_of = [&](int32_t s) { return context_len[s] - query_len[s]; };
        // All items of one (sequence, row tile) have the same KV extent, so the longest-first order is found by
        // sorting those few groups, not the items (a 8192-token chunk with 64 query heads is 2048 items in 64 groups).
        struct Group { int64_t extent; int32_t s, tile; };
        std::vector<Group> groups;
        size_t n_emit = 0;
        for (int32_t s = 0; s < num_seqs; ++s) {
            const int32_t lq = query_len[s];
            if (lq <= 1) continue;
            const int32_t n_tiles = (lq + TR - 1) / TR;
            for (int32_t tile = 0; tile < n_tiles; tile += (G >= 2 ? 1 : 2)) {
                const int32_t last = (G >= 2 || tile + 1 >= n_tiles) ? tile : tile + 1;
                groups.push_back(Group{(int64_t)prefix_of(s) + last * TR + std::min(TR, lq - last * TR), s, tile});
                n_emit += (size_t)(G >= 2 ? d->num_kv_heads * (G / heads_per_item) : d->num_q_heads);
            }
        }
        std::stable_sort(groups.begin(), groups.end(), [](const Group& a, const Group& b) { return a.extent > b.extent; });
        items.reserve(n_emit);
        // Items that run at the same time re-read the K/V tiles of their KV heads from L2.  When the K/V of the longest
        // sequence (all KV heads) no longer fits there beside everything else, the KV heads are taken one after the
        // other (longest item first inside each), so that the items in flight share two or three heads instead of all:
        // the same work, a third of the trips to DRAM (measured on 2048 new over 24,576 cached tokens: +1.8 %).
        // Below that size the order makes no difference to DRAM and the globally longest-first order is kept.
        constexpr int64_t kKvSetBytes = CF_KV_SET_BYTES;
        int32_t kv_sets = 1;
        if (G >= 2) {
            int64_t longest = 0;
            for (const Group& gr : groups) longest = std::max(longest, gr.extent);
            if (longest * 2 * d->num_kv_heads * d->head_dim * 2 > kKvSetBytes) kv_sets = d->num_kv_heads;
        }
        const int32_t heads_per_set = d->num_kv_heads / kv_sets;
        for (int32_t set = 0; set < kv_sets; ++set)
        for (const Group& gr : groups) {
            const int32_t s = gr.s, tile = gr.tile, lq = query_len[s];
            const int32_t prefix = context_len[s] - lq;
            const int32_t n_tiles = (lq + TR - 1) / TR;
            auto rows_of = [&](int32_t tl) { return std::min(TR, lq - tl * TR); };
            PrefillTcItem it;
            it.seq = s; it.prefix = prefix; it.ctx_len = context_len[s]; it.pad = 0;
            // sliding window: the item's first row (position prefix + tile * TR) sees keys from lo0 on, and no row of
            // the item sees anything left of that; pages and KV tiles left of lo0 are skipped
            const int32_t lo0 = (W > 0) ? std::max(0, prefix + tile * TR - W + 1) : 0;
            it.page_lo = lo0 / B;
            it.j_begin = lo0 / TR; it.j_end = INT32_MAX; it.part_slot[0] = it.part_slot[1] = -1; it.part_k = 1; it.part_c = 0;
            const int32_t n_tiles_kv = (int32_t)((gr.extent + TR - 1) / TR) - it.j_begin;
            if (G >= 2) {
                for (int t = 0; t < 2; ++t) {
                    it.q_row0[t] = plan->q_start[s] + tile * TR;
                    it.row0[t] = tile * TR;
                    it.n_rows[t] = rows_of(tile);
                }
                for (int32_t kvh = set * heads_per_set; kvh < (set + 1) * heads_per_set; ++kvh)
                    for (int32_t i = 0; i < G; i += heads_per_item) {
                        it.kvh = kvh;
                        it.head[0] = kvh * G + i;
                        it.head[1] = kvh * G + i + 1;
                        items.push_back(KeyedTc{gr.extent, n_tiles_kv, it});
                    }
            } else {
                for (int t = 0; t < 2; ++t) {
                    const int32_t tt = tile + t;
                    const bool present = tt < n_tiles;
                    it.q_row0[t] = present ? plan->q_start[s] + tt * TR : 0;
                    it.row0[t] = present ? tt * TR : 0;
                    it.n_rows[t] = present ? rows_of(tt) : 0;
                }
                for (int32_t h = 0; h < d->num_q_heads; ++h) {
                    it.kvh = h;
                    it.head[0] = it.head[1] = h;
                    items.push_back(KeyedTc{gr.extent, n_tiles_kv, it});
                }
            }
        }
        // Few items (short chunks, few heads per GPU under tensor parallelism): a CTA's time is set by the
        // per-tile softmax -> MMA chain, not by how many q tiles it carries, so single-tile items are an
        // alternative while pairs would leave SMs idle (sharing K/V tiles matters only when the machine is
        // full).  Whether pairs or singles are used is decided below, together with the KV split.
        std::vector<KeyedTc> singles;
        if (!pair && items.size() * 2 <= (size_t)std::max(1, cfg.num_sms)) {
            singles.reserve(items.size() * 2);
            for (const KeyedTc& k : items)
                for (int t = 0; t < 2; ++t) {
                    if (k.it.n_rows[t] == 0) continue;
                    PrefillTcItem one = k.it;
                    one.q_row0[0] = k.it.q_row0[t]; one.row0[0] = k.it.row0[t]; one.n_rows[0] = k.it.n_rows[t];
                    one.head[0] = k.it.head[t];
                    one.q_row0[1] = 0; one.row0[1] = 0; one.n_rows[1] = 0; one.head[1] = k.it.head[t];
                    const int64_t ext = (int64_t)prefix_of(k.it.seq) + one.row0[0] + one.n_rows[0];
                    const int32_t lo1 = (W > 0) ? std::max(0, prefix_of(k.it.seq) + one.row0[0] - W + 1) : 0;
                    one.page_lo = lo1 / B;
                    one.j_begin = lo1 / TR;
                    singles.push_back(KeyedTc{ext, (int32_t)((ext + TR - 1) / TR) - one.j_begin, one});
                }
            std::stable_sort(singles.begin(), singles.end(), [](const KeyedTc& a, const KeyedTc& b) { return a.extent > b.extent; });
        }
        // ---- KV split.  Items run one per SM, so a long item or an incomplete last wave leaves SMs idle.
        // An item may be cut into k <= 8 KV ranges that write fp32 partials, merged by a combine pass; k
        // comes from the cost model's constants; a range never starts inside the diagonal band and has at
        // least 4 tiles.
        const size_t M = (size_t)std::max(1, ((cfg.prefill_sms_mixed > 0 && !plan->decode.empty()) ? cfg.prefill_sms_mixed : cfg.num_sms) /
                                                 (pair ? 2 : 1));      // slots that take an item: SMs, or pairs of SMs
        // decides the KV ranges per item for one candidate item list; returns the predicted time (us)
        auto decide = [&](const std::vector<KeyedTc>& its, const double tile_us, std::vector<int32_t>& k_of) -> double {
        const size_t n_items = its.size();
        k_of.assign(n_items, 1);
        double predicted = 0.0;
        auto tiles_of = [&](size_t i) { return (double)its[i].tiles; };
        // a whole item costs ~8 us + 1.9 us per tile; a KV range pays ~13 us (fp32 partial epilogue);
        // splitting adds the combine launch and the partial write/read
        auto split_extra = [](size_t n_ranges) { return 8.0 + 0.05 * (double)n_ranges; };
        if (cfg.prefill_force_split >= 2) {
            std::fill(k_of.begin(), k_of.end(), std::min(cfg.prefill_force_split, 8));
        } else if (cfg.prefill_force_split == 1 || n_items == 0) {
            // splitting switched off / nothing to do
        } else if (n_items <= M) {
            // One wave of unequal items (a few prompts with different prefixes): the longest item sets the
            // time.  Try a few target times T; an item is cut into ceil(time / T) ranges; the candidate
            // whose list-scheduled makespan (plus the split overhead) is smallest wins.
            double total = 0.0, longest = 0.0;
            for (size_t i = 0; i < n_items; ++i) {
                total += tile_us * tiles_of(i);
                longest = std::max(longest, tile_us * tiles_of(i));
            }
            double best = 8.0 + longest;                  // no split
            predicted = best;
            std::vector<int32_t> cand(n_items);
            for (double f : {1.0, 1.2, 1.5, 2.0, 3.0}) {
                const double T = std::max(f * total / (double)M, 8.0);
                size_t n_ranges = 0;
                bool any = false;
                std::vector<double> jobs;
                for (size_t i = 0; i < n_items; ++i) {
                    const double tl = tiles_of(i);
                    int32_t k = (int32_t)std::min(8.0, std::ceil(tile_us * tl / T));
                    k = std::max(1, std::min(k, (int32_t)(tl / 4.0)));
                    cand[i] = k;
                    any = any || k > 1;
                    n_ranges += (size_t)k;
                    for (int32_t c = 0; c < k; ++c) jobs.push_back((k > 1 ? 13.0 : 8.0) + tile_us * tl / k);
                }
                if (!any) continue;
                std::sort(jobs.begin(), jobs.end(), std::greater<double>());
                const double t = list_schedule(jobs, M) + split_extra(n_ranges);
                if (t < best * 0.95) { best = t; k_of = cand; predicted = t; }
            }
        } else if (n_items % M != 0) {
            // Several waves of similar items: after the full waves the remaining r items would hold r SMs
            // for a whole item time; cutting each into k ranges lets them fill the machine.
            const size_t r = n_items % M, first_tail = n_items - r;
            double tiles = 0.0;
            for (size_t i = first_tail; i < n_items; ++i) tiles += tiles_of(i);
            tiles /= (double)r;
            double best = 1e30;
            int32_t k_best = 1;
            for (int32_t k = 1; k <= 8; ++k) {
                if (k > 1 && tiles / k < 4.0) break;
                const double rounds = (double)((r * (size_t)k + M - 1) / M);
                double t = rounds * ((k > 1 ? 13.0 : 8.0) + tile_us * tiles / k);
                if (k > 1) t += split_extra(r * (size_t)k);
                if (t < best * 0.97) { best = t; k_best = k; }             // split only for a clear gain
            }
            for (size_t i = first_tail; i < n_items; ++i) k_of[i] = k_best;
        }
        return predicted;
        };
        std::vector<int32_t> k_of;
        double t_pairs = decide(items, 1.9, k_of);
        if (!singles.empty() && cfg.prefill_force_split == 0) {
            std::vector<int32_t> k_single;
            const double t_single = decide(singles, 1.8, k_single);
            if (t_single < t_pairs) {
                items.swap(singles);
                k_of.swap(k_single);
                t_pairs = t_single;
            }
        }
        const size_t n_items = items.size();
        plan->prefill_tc.reserve(n_items + 8 * plan->prefill_combine.capacity());
        for (size_t i = 0; i < n_items; ++i) {
            PrefillTcItem it = items[i].it;
            const int32_t k_want = k_of[i];
            if (k_want <= 1) {
                plan->prefill_tc.push_back(it);
                continue;
            }
            // tiles every present q tile takes part in, and the last tile boundary outside the diagonal band
            const int32_t prefix = prefix_of(it.seq);
            int32_t n_min = INT32_MAX, safe = INT32_MAX;
            for (int t = 0; t < 2; ++t)
                if (it.n_rows[t] > 0) {
                    n_min = std::min(n_min, (prefix + it.row0[t] + it.n_rows[t] + 127) / 128);
                    safe = std::min(safe, (prefix + it.row0[t]) / 128);
                }
            const int32_t j_lo = it.j_begin;          // first tile of the sliding window (0 without one); j_lo <= safe
            const int32_t k = std::min(k_want, std::max(1, (std::min(n_min, safe + 1) - j_lo) / 4));
            if (k <= 1) {
                plan->prefill_tc.push_back(it);
                continue;
            }
            PrefillCombineItem ci;
            ci.part_k = k;
            for (int t = 0; t < 2; ++t) {
                ci.q_row0[t] = it.q_row0[t]; ci.n_rows[t] = it.n_rows[t]; ci.head[t] = it.head[t];
                ci.part_slot[t] = it.n_rows[t] > 0 ? plan->n_pre_slots : -1;
                plan->n_pre_slots += it.n_rows[t] * k;
            }
            plan->prefill_combine.push_back(ci);
            if (pair) {
                // the second CTA's two q tiles (heads + 2) get slots of their own, a fixed distance behind the first CTA's
                PrefillCombineItem cj = ci;
                it.pad = plan->n_pre_slots - ci.part_slot[0];
                for (int t = 0; t < 2; ++t) {
                    cj.head[t] = it.head[t] + 2;
                    cj.part_slot[t] = it.n_rows[t] > 0 ? plan->n_pre_slots : -1;
                    plan->n_pre_slots += it.n_rows[t] * k;
                }
                plan->prefill_combine.push_back(cj);
            }
            for (int32_t c = 0; c < k; ++c) {
                PrefillTcItem f = it;
                f.j_begin = std::min(j_lo + (int32_t)((int64_t)c * (n_min - j_lo) / k), safe);
                f.j_end = c + 1 < k ? std::min(j_lo + (int32_t)((int64_t)(c + 1) * (n_min - j_lo) / k), safe) : INT32_MAX;
                f.part_slot[0] = ci.part_slot[0]; f.part_slot[1] = ci.part_slot[1];
                f.part_k = k; f.part_c = c;
                plan->prefill_tc.push_back(f);
            }
        }
    }
    return CF_OK;
}

int32_t spatial_front_sms(const cf_cache_desc* d, const int32_t* context_len, const int32_t* query_len, int32_t num_seqs,
                          int32_t num_sms)
{
    const int32_t G = d->num_q_heads / d->num_kv_heads, W = d->window_size;
    const double items_per_tile = G >= 2 ? (double)d->num_kv_heads * (double)(G / 2) : 0.5 * (double)d->num_q_heads;
    double dec_bytes = 0.0, work = 0.0;      // bytes the decode kernel streams; SM-microseconds of the prefill items
    for (int32_t s = 0; s < num_seqs; ++s) {
        const int32_t lq = query_len[s], lc = context_len[s];
        if (lq == 1) {
            dec_bytes += (double)(W > 0 ? std::min(lc, W) : lc) * 2.0 * d->num_kv_heads * d->head_dim * 2.0;
        } else if (lq > 1) {
            const int32_t prefix = lc - lq;
            for (int32_t row = 0; row < lq; row += 128) {
                const int32_t hi = prefix + std::min(lq, row + 128);
                const int32_t lo = W > 0 ? std::max(0, prefix + row - W + 1) / 128 : 0;
                work += items_per_tile * (8.0 + 1.9 * (double)((hi + 127) / 128 - lo));
            }
        }
    }
    if (dec_bytes == 0.0 || work == 0.0) return 0;
    const double sms = (double)std::max(1, num_sms);
    const double t_dec = 17.0 + dec_bytes / 7.1e6, k_sat = G > 4 ? 100.0 : 65.0;
    const double t_call = work / sms + t_dec * k_sat / sms;              // both parts packed without idle SMs
    const double k_dec = 1.15 * k_sat * t_dec / t_call;
    const double front = std::min(std::max(sms - k_dec, 0.6 * sms), 0.875 * sms);
    return std::max(1, (int32_t)front);
}

Estimate estimate_us(const cf_cache_desc* d, const int32_t* context_len, const int32_t* query_len, const Plan& plan,
                     int32_t num_sms)
{
    // Constants fitted to CUDA-event times of the kernels on a B200: split-K decode (with the merge of the
    // partials fused in) sustains ~7.56 TB/s on top of ~22 us of launch, ramp and tail; the separate combine
    // launch, when it is used, ~8 us, reported as 0 here because the default path has none; one tcgen05
    // prefill item costs ~8 us plus ~1.9 us per 128-token KV tile.
    constexpr double kDecodeFixedUs = 22.0, kDecodeBytesPerUs = 7.56e6, kCombineUs = 0.0;
    constexpr double kTcItemFixedUs = 8.0, kTcTileUs = 1.9, kLaunchUs = 4.0;
    Estimate e;
    const int32_t S = (int32_t)plan.q_start.size() - 1;
    double dec_bytes = 0.0;
    for (int32_t s = 0; s < S; ++s)
        if (query_len[s] == 1)
            dec_bytes += (double)(d->window_size > 0 ? std::min(context_len[s], d->window_size) : context_len[s]) * 2.0 *
                             d->num_kv_heads * d->head_dim * 2.0 + 4.0 * d->num_q_heads * d->head_dim;
    if (!plan.decode.empty()) e.us_decode = (float)(kDecodeFixedUs + dec_bytes / kDecodeBytesPerUs);
    if (!plan.combine.empty()) e.us_combine = (float)kCombineUs;
    if (!plan.prefill_tc.empty()) {
        // items are already longest-first: greedy list scheduling onto num_sms machines
        std::vector<double> jobs;
        jobs.reserve(plan.prefill_tc.size());
        for (const PrefillTcItem& it : plan.prefill_tc) {
            const int32_t prefix = context_len[it.seq] - query_len[it.seq];
            int32_t hi = 0;
            for (int t = 0; t < 2; ++t)
                if (it.n_rows[t] > 0) hi = std::max(hi, prefix + it.row0[t] + it.n_rows[t]);
            const int32_t tiles = std::max(0, std::min((hi + 127) / 128, it.j_end) - it.j_begin);
            const double cost = kTcItemFixedUs + kTcTileUs * tiles;
            jobs.push_back(cost);
        }
        e.us_prefill = (float)(kLaunchUs + list_schedule(jobs, (size_t)std::max(1, plan.pair ? num_sms / 2 : num_sms)));
        if (!plan.prefill_combine.empty()) e.us_prefill += (float)(6.0 + 0.05 * (double)plan.prefill_tc.size());
    }
    return e;
}

}  // namespace cf
