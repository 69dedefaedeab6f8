// Host-callable launchers of the CUDA kernels (one translation unit per kernel family).
#pragma once
#include <cuda.h>
#include <cuda_runtime.h>

#include "device_common.cuh"

namespace cf {

struct AppendParams {
    __nv_bfloat16* k_cache;
    __nv_bfloat16* v_cache;
    const __nv_bfloat16* k_new;
    const __nv_bfloat16* v_new;
    const int32_t* block_table;
    int32_t max_blocks;
    int64_t ks_block, ks_head, ks_token;
    int64_t vs_block, vs_head, vs_token;
    int32_t Hkv, D, num_seqs, total_rows;
    int32_t num_blocks;               // pool size: a block id outside [0, num_blocks) is reported, its row not written
    const float* k_scale;             // fp8 cache (non-null): rows are stored as e4m3_rne_sat(x / scale[head])
    const float* v_scale;
    uint32_t* err;                    // device error word (may be null)
    const int32_t* context_len;
    const int32_t* query_len;
    const int32_t* q_start;
};

cudaError_t launch_kv_append(const AppendParams& p, cudaStream_t stream);
cudaError_t launch_validate_table(const int32_t* block_table, int32_t max_blocks, const int32_t* context_len_dev,
                                  int32_t num_seqs, int32_t num_blocks, uint32_t* bad_count, cudaStream_t stream);
cudaError_t launch_decode(const AttnParams& p, int head_dim, int n_items, cudaStream_t stream);
cudaError_t launch_combine(const AttnParams& p, int head_dim, int n_items, cudaStream_t stream);
// split-K decode over an fp8 (e4m3) cache, head_dim 128: same items, partials and merge as launch_decode
cudaError_t launch_decode_fp8(const AttnParams& p, int n_items, cudaStream_t stream);
// fp8 cache: expands the pages that prefill chunks need into bf16 staging pools [n_stage_pages, Hkv, 16, 128] (the codes
// exactly, without the scales) and fills the staging block table; one entry per prefill sequence
struct StageSeq {
    int32_t seq;         // sequence (row of the block tables)
    int32_t page0;       // first page of the sequence that is expanded
    int32_t n_pages;
    int32_t stage_base;  // staging page of page0
};
cudaError_t launch_kv_dequant_gather(const AttnParams& p, const StageSeq* seqs_dev, int n_seqs, int max_pages,
                                     __nv_bfloat16* stage_k, __nv_bfloat16* stage_v, int32_t* stage_table, cudaStream_t stream);
// a batch with shared prefixes: one grid whose first CTAs serve the shared-prefix chunks (one CTA per shared item
// and KV head streams the chunk once for all members of its set and writes one partial per member and head) and
// whose other CTAs serve the sequences' own chunks; n_shared_items = 0 is launch_decode
cudaError_t launch_decode_with_shared(const AttnParams& p, int head_dim, int n_shared_items, int n_items, cudaStream_t stream);

// tcgen05 / tensor-memory chunked prefill (head_dim 64 or 128): `n_ctas` persistent CTAs draw the `n_items`
// PrefillTcItems from the ticket counter p.pre_queue, which `queue_ctas` CTAs share in total (several
// launches may draw from one counter; the last CTA to leave resets it).  Ticket t stands for item
// ticket_base + t; with first_static set, CTA b starts on item b without a draw (then ticket_base = n_ctas of
// that grid, also for a second grid that shares the counter).  `resident`, when not null, is a device word that
// every CTA increments as it starts.
// The kernel reads q and the two pools through TMA tensor maps; a map depends only on the base address and the
// geometry, so the caller may build it once and keep it (encode_* return false when the driver refuses).
struct PrefillMaps {
    CUtensorMap q, k, v;
};
bool encode_q_map(CUtensorMap* m, const void* q, int head_dim, int total_rows, int num_q_heads);
bool encode_pool_map(CUtensorMap* m, const void* pool, int head_dim, int num_blocks, int num_kv_heads, int64_t stride_block,
                     int64_t stride_head, int64_t stride_token);
cudaError_t launch_prefill_tc(const AttnParams& p, const PrefillMaps& maps, int head_dim, int n_items, int n_ctas,
                              int queue_ctas, int first_static, int ticket_base, uint32_t* resident, cudaStream_t stream);

// The same work on pairs of SMs (tcgen05.mma.cta_group::2; head_dim 128, group size a multiple of 4): an item is four
// q tiles (four heads of a group over the same rows), CTA r of a pair taking heads head[t] + 2 r and partial slots
// part_slot[t] + r * pad; n_pairs persistent pairs (2 n_pairs CTAs), queue_pairs pairs drawing from the counter.
bool prefill_pair_supported(const cf_cache_desc* desc);
cudaError_t launch_prefill_tc2(const AttnParams& p, const PrefillMaps& maps, int n_items, int n_pairs, int queue_pairs,
                               int first_static, int ticket_base, uint32_t* resident, cudaStream_t stream);

// merges the fp32 partials of KV-split prefill items into `out` (one CTA per split item)
cudaError_t launch_prefill_combine(const AttnParams& p, int head_dim, int n_items, cudaStream_t stream);
// one CTA whose bounded wait must expire: sets *err and returns normally (status-path self-test)
cudaError_t launch_wait_selftest(uint32_t* err, cudaStream_t stream);

}  // namespace cf
