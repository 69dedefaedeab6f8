// C ABI of the library: context, plan upload and the launch sequence.
// See include/crossflow_attn.h for the contract of every entry point.
#include <cuda.h>

#include <atomic>
#include <chrono>
#include <cmath>
#include <cstdio>
#include <cstdlib>
#include <cstring>
#include <new>
#include <vector>

#include "../../include/crossflow_attn.h"
#include "kernels.h"
#include "plan.h"

namespace cf {

static constexpr int kRing = 4;                         // plan slots in flight
static constexpr size_t kDefaultWorkspace = 64u << 20;  // split-K partials
static constexpr size_t kDefaultPlanBytes = 1u << 20;
// The first kCounterBytes of a split-K workspace hold the fused-combine ticket counters of the decode kernel
// (one per first partial slot of a split sequence and KV head): zeroed when the buffer is allocated, put back
// to zero by the kernel.  A batch with more counters than fit uses the separate combine kernel.
static constexpr size_t kCounterBytes = 256u << 10;

struct TimedCall {
    cudaEvent_t ev[4] = {nullptr, nullptr, nullptr, nullptr};
    bool ran[3] = {false, false, false};
};

// Device staging of one host-buffer step (cf_mixed_step_host): inputs copied in on one copy stream,
// result copied out on another, so that the copies of neighbouring steps overlap the kernels.
static constexpr int kHostStages = 3;
struct HostStage {
    uint8_t* dev = nullptr;
    size_t bytes = 0;
    cudaEvent_t h2d_done = nullptr, h2d_kv_done = nullptr, compute_done = nullptr, d2h_done = nullptr;
    bool used = false;
};

// TMA tensor maps of the prefill kernel, kept per (base address, geometry): a serving loop passes the same
// pools and activation buffer call after call (one set per layer), and encoding three maps costs a few
// microseconds of host time per launch.
struct PoolMapEntry {
    const void* base = nullptr;
    int D = 0, num_blocks = 0, Hkv = 0;
    int64_t sb = 0, sh = 0, st = 0;
    uint64_t stamp = 0;
    CUtensorMap map;
};
struct QMapEntry {
    const void* base = nullptr;
    int D = 0, rows = 0, Hq = 0;
    uint64_t stamp = 0;
    CUtensorMap map;
};
static constexpr int kPoolMaps = 32, kQMaps = 8;

struct PlanSlot {
    uint8_t* host = nullptr;   // pinned
    uint8_t* dev = nullptr;
    cudaEvent_t done = nullptr;
    cudaEvent_t uploaded = nullptr;   // host-staged steps: the plan copy runs on the input copy stream
    bool used = false;
};

}  // namespace cf

struct cf_ctx {
    int device = 0;
    int num_sms = 0;
    cf::PlanConfig cfg;
    cf::PlanSlot slots[cf::kRing];
    size_t plan_bytes = 0;
    int next_slot = 0;
    float* workspace = nullptr;
    size_t workspace_bytes = 0;
    bool workspace_fixed = false;
    uint32_t* err_dev = nullptr;      // [0] device-side findings (bit 0: a wait expired, bit 1: block id outside the pool); [1] scratch counter of cf_validate_block_table
    bool fused_combine = true; // split-K merge inside the decode kernel (CF_DEBUG_SEPARATE_COMBINE: the separate combine kernel)
    bool use_pairs = false;    // CF_DEBUG_PREFILL_PAIRS: chunked prefill on pairs of SMs where the geometry allows it (measured slower
                               // than one CTA per item, see prefill_tc2.cu; kept as a tested alternative)
    std::atomic<int> live_plans{0};
    // concurrent execution of the prefill kernel beside decode + combine (side stream, fork/join events)
    bool overlap = true;
    cudaStream_t upload_stream = nullptr;      // plan uploads of cf_kv_append / cf_mixed_attention
    cudaStream_t plan_copy_stream = nullptr;   // set while cf_mixed_step_host runs
    bool in_host_step = false; // inside a cf_mixed_step_host call that keeps the serial sequence (a step bound by the host copies)
    bool spatial_wait = true;  // decode waits (stream memory operation) for the front prefill CTAs to be resident; CF_DEBUG_SPATIAL_NO_WAIT: launch order only
    int spatial_sms = 0;       // SMs given to the first prefill grid in that mode (0 = three fifths)
    int spatial_sms_default = 0;   // CF_SPATIAL_SMS at cf_create: what cf_set_overlap(ctx, 1) goes back to
    cudaStream_t side = nullptr;
    cudaEvent_t ev_fork = nullptr, ev_join = nullptr;
    // host-staged step
    cf::HostStage stage[cf::kHostStages];
    int next_stage = 0;
    cudaStream_t h2d_stream = nullptr, h2d_kv_stream = nullptr, d2h_stream = nullptr;
    // timing: one quad of events per timed call since the last cf_get_timing_sums
    bool timing = false;
    std::vector<cf::TimedCall> timed;
    size_t timed_used = 0;
    int launches = 0;
    // host time spent inside the entry points (benchmark instrumentation): nanoseconds and call counts
    int64_t host_ns_append = 0, host_ns_attention = 0, host_ns_planner = 0;
    int32_t host_calls_append = 0, host_calls_attention = 0;
    // tensor-map cache (least recently used entry is replaced)
    cf::PoolMapEntry pool_maps[cf::kPoolMaps];
    cf::QMapEntry q_maps[cf::kQMaps];
    uint64_t map_stamp = 0;
    int32_t last_counts[8] = {0, 0, 0, 0, 0, 0, 0, 0};   // item counts of the plan the last cf_mixed_attention built
};

// A plan that lives on the device for as long as the caller wants: built once per scheduler iteration
// and used by every layer's append + attention calls (the lengths are the same for all layers).
struct cf_plan {
    cf_ctx* ctx = nullptr;
    cf_cache_desc desc;
    int32_t num_seqs = 0, max_blocks = 0;
    uint8_t* host = nullptr;       // pinned copy (source of the one upload)
    uint8_t* dev = nullptr;
    float* part = nullptr;         // this plan's own split-K partials
    int n_part_slots = 0, n_pre_slots = 0;
    size_t off_stage = 0;
    int n_stage_seqs = 0, n_stage_pages = 0, max_stage_pages = 0;
    size_t off_qstart = 0, off_ctx = 0, off_qlen = 0, off_dec = 0, off_comb = 0, off_sh = 0, off_shm = 0, off_pre_tc = 0, off_pre_comb = 0, off_queue = 0, total = 0;
    int n_dec = 0, n_comb = 0, n_pre_tc = 0, n_pre_comb = 0, total_q = 0;
    bool pair = false;
    int front_sms = 0;          // spatial sequence: SMs of the first prefill grid (spatial_front_sms or cf_set_overlap)
};

namespace cf {

static int env_int(const char* name, int fallback)
{
    const char* v = std::getenv(name);
    if (!v || !*v) return fallback;
    char* end = nullptr;
    long x = std::strtol(v, &end, 10);
    return (end && *end == 0 && x > 0 && x < (1 << 20)) ? (int)x : fallback;
}

struct DeviceGuard {
    int prev = -1;
    bool ok = false;
    explicit DeviceGuard(int dev)
    {
        if (cudaGetDevice(&prev) != cudaSuccess) return;
        ok = (prev == dev) || cudaSetDevice(dev) == cudaSuccess;
    }
    ~DeviceGuard()
    {
        if (ok && prev >= 0) cudaSetDevice(prev);
    }
};

static size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

static cf_status ensure_plan_capacity(cf_ctx* c, size_t need)
{
    if (need <= c->plan_bytes) return CF_OK;
    size_t nb = c->plan_bytes ? c->plan_bytes : kDefaultPlanBytes;
    while (nb < need) nb *= 2;
    if (cudaDeviceSynchronize() != cudaSuccess) return CF_ERR_CUDA;
    for (int i = 0; i < kRing; ++i) {
        PlanSlot& s = c->slots[i];
        if (s.host) cudaFreeHost(s.host);
        if (s.dev) cudaFree(s.dev);
        s.host = s.dev = nullptr;
        s.used = false;
        if (cudaMallocHost((void**)&s.host, nb) != cudaSuccess) return CF_ERR_CUDA;
        if (cudaMalloc((void**)&s.dev, nb) != cudaSuccess) return CF_ERR_CUDA;
    }
    c->plan_bytes = nb;
    return CF_OK;
}

static cf_status ensure_workspace(cf_ctx* c, size_t need)
{
    if (need <= c->workspace_bytes) return CF_OK;
    if (c->workspace_fixed) return CF_ERR_WORKSPACE;
    if (cudaDeviceSynchronize() != cudaSuccess) return CF_ERR_CUDA;
    if (c->workspace) cudaFree(c->workspace);
    c->workspace = nullptr;
    c->workspace_bytes = 0;
    size_t nb = align_up(need + need / 4, 1u << 20);
    if (cudaMalloc((void**)&c->workspace, nb) != cudaSuccess) return CF_ERR_CUDA;
    // The ticket counters at its front start at zero.  cudaMemset runs on the legacy default stream, which is not
    // ordered against non-blocking streams: wait for it here, before any kernel of the caller's stream can count.
    if (cudaMemset(c->workspace, 0, kCounterBytes < nb ? kCounterBytes : nb) != cudaSuccess || cudaDeviceSynchronize() != cudaSuccess)
        return CF_ERR_CUDA;
    c->workspace_bytes = nb;
    return CF_OK;
}

// Layout of one uploaded plan: [q_start S+1][context_len S][query_len S][decode][combine][prefill]
struct PlanLayout {
    size_t off_qstart, off_ctx, off_qlen, off_dec, off_comb, off_sh, off_shm, off_pre_tc, off_pre_comb, off_stage, off_queue, total;
};

static PlanLayout layout_of(int32_t S, const Plan& pl, size_t n_stage_seqs = 0)
{
    PlanLayout L;
    size_t at = 0;
    L.off_qstart = at; at = align_up(at + sizeof(int32_t) * ((size_t)S + 1), 16);
    L.off_ctx = at;    at = align_up(at + sizeof(int32_t) * (size_t)S, 16);
    L.off_qlen = at;   at = align_up(at + sizeof(int32_t) * (size_t)S, 16);
    L.off_dec = at;    at = align_up(at + sizeof(DecodeItem) * pl.decode.size(), 16);
    L.off_comb = at;   at = align_up(at + sizeof(CombineItem) * pl.combine.size(), 16);
    L.off_sh = at;     at = align_up(at + sizeof(SharedDecodeItem) * pl.shared_decode.size(), 16);
    L.off_shm = at;    at = align_up(at + sizeof(ShareMember) * pl.share_members.size(), 16);
    L.off_pre_tc = at; at = align_up(at + sizeof(PrefillTcItem) * pl.prefill_tc.size(), 16);
    L.off_pre_comb = at; at = align_up(at + sizeof(PrefillCombineItem) * pl.prefill_combine.size(), 16);
    L.off_stage = at;  at = align_up(at + sizeof(StageSeq) * n_stage_seqs, 16);
    L.off_queue = at;  at += 16;   // ticket counter + exit counter of the persistent prefill CTAs; uploaded as zeros
    L.total = at;
    return L;
}

// Copies the plan into the next pinned slot and enqueues its upload.  Returns the device base.
static cf_status upload_plan(cf_ctx* c, int32_t S, const int32_t* context_len, const int32_t* query_len,
                             const Plan& pl, cudaStream_t stream, PlanLayout* L, uint8_t** dev_base, PlanSlot** slot_out,
                             const std::vector<StageSeq>* stage = nullptr)
{
    *L = layout_of(S, pl, stage ? stage->size() : 0);
    cf_status st = ensure_plan_capacity(c, L->total);
    if (st != CF_OK) return st;
    PlanSlot& s = c->slots[c->next_slot];
    c->next_slot = (c->next_slot + 1) % kRing;
    if (s.used && cudaEventSynchronize(s.done) != cudaSuccess) return CF_ERR_CUDA;   // slot still in flight
    std::memcpy(s.host + L->off_qstart, pl.q_start.data(), sizeof(int32_t) * ((size_t)S + 1));
    if (S > 0) {
        std::memcpy(s.host + L->off_ctx, context_len, sizeof(int32_t) * (size_t)S);
        std::memcpy(s.host + L->off_qlen, query_len, sizeof(int32_t) * (size_t)S);
    }
    if (!pl.decode.empty()) std::memcpy(s.host + L->off_dec, pl.decode.data(), sizeof(DecodeItem) * pl.decode.size());
    if (!pl.combine.empty()) std::memcpy(s.host + L->off_comb, pl.combine.data(), sizeof(CombineItem) * pl.combine.size());
    if (!pl.shared_decode.empty())
        std::memcpy(s.host + L->off_sh, pl.shared_decode.data(), sizeof(SharedDecodeItem) * pl.shared_decode.size());
    if (!pl.share_members.empty())
        std::memcpy(s.host + L->off_shm, pl.share_members.data(), sizeof(ShareMember) * pl.share_members.size());
    if (!pl.prefill_tc.empty())
        std::memcpy(s.host + L->off_pre_tc, pl.prefill_tc.data(), sizeof(PrefillTcItem) * pl.prefill_tc.size());
    if (!pl.prefill_combine.empty())
        std::memcpy(s.host + L->off_pre_comb, pl.prefill_combine.data(), sizeof(PrefillCombineItem) * pl.prefill_combine.size());
    if (stage && !stage->empty()) std::memcpy(s.host + L->off_stage, stage->data(), sizeof(StageSeq) * stage->size());
    std::memset(s.host + L->off_queue, 0, 16);
    // The copy does not go on the caller's stream: there it would start only when that stream's earlier
    // kernels are done (a few microseconds of copy-engine latency between kernels, every call) and, queued in
    // the copy engine meanwhile, hold back copies enqueued after it.  It runs on a context-owned stream (a
    // host-staged step: on its input copy stream) and the caller's stream waits for it through an event; the
    // slot's device buffer is free by then (the host waited for the slot's last use above).
    cudaStream_t copy_stream = c->plan_copy_stream ? c->plan_copy_stream : c->upload_stream;
    if (cudaMemcpyAsync(s.dev, s.host, L->total, cudaMemcpyHostToDevice, copy_stream) != cudaSuccess) return CF_ERR_CUDA;
    if (cudaEventRecord(s.uploaded, copy_stream) != cudaSuccess || cudaStreamWaitEvent(stream, s.uploaded, 0) != cudaSuccess)
        return CF_ERR_CUDA;
    *dev_base = s.dev;
    *slot_out = &s;
    return CF_OK;
}

static cf_status finish_slot(PlanSlot* s, cudaStream_t stream)
{
    if (cudaEventRecord(s->done, stream) != cudaSuccess) return CF_ERR_CUDA;
    s->used = true;
    return CF_OK;
}

// Stream memory operations of the driver API (the runtime has no counterpart), looked up once.
struct StreamMemOps {
    typedef CUresult (*Fn)(CUstream, CUdeviceptr, cuuint32_t, unsigned int);
    Fn wait = nullptr, write = nullptr;
    bool ok = false;
};
static StreamMemOps lookup_stream_mem_ops()
{
    StreamMemOps ops;
    void *w = nullptr, *r = nullptr;
    cudaDriverEntryPointQueryResult q1, q2;
    if (cudaGetDriverEntryPoint("cuStreamWaitValue32", &w, cudaEnableDefault, &q1) == cudaSuccess &&
        cudaGetDriverEntryPoint("cuStreamWriteValue32", &r, cudaEnableDefault, &q2) == cudaSuccess &&
        q1 == cudaDriverEntryPointSuccess && q2 == cudaDriverEntryPointSuccess && w && r) {
        ops.wait = reinterpret_cast<StreamMemOps::Fn>(w);
        ops.write = reinterpret_cast<StreamMemOps::Fn>(r);
        ops.ok = true;
    }
    return ops;
}
static const StreamMemOps& stream_mem_ops()
{
    static const StreamMemOps ops = lookup_stream_mem_ops();      // initialised once, thread-safe
    return ops;
}

static int64_t now_ns()
{
    return std::chrono::duration_cast<std::chrono::nanoseconds>(std::chrono::steady_clock::now().time_since_epoch()).count();
}

static const CUtensorMap* pool_map(cf_ctx* c, const void* base, const cf_cache_desc* d, int64_t sb, int64_t sh, int64_t st)
{
    PoolMapEntry* victim = &c->pool_maps[0];
    for (PoolMapEntry& e : c->pool_maps) {
        if (e.base == base && e.D == d->head_dim && e.num_blocks == d->num_blocks && e.Hkv == d->num_kv_heads && e.sb == sb &&
            e.sh == sh && e.st == st) {
            e.stamp = ++c->map_stamp;
            return &e.map;
        }
        if (e.stamp < victim->stamp) victim = &e;
    }
    if (!encode_pool_map(&victim->map, base, d->head_dim, d->num_blocks, d->num_kv_heads, sb, sh, st)) {
        victim->base = nullptr;
        return nullptr;
    }
    victim->base = base; victim->D = d->head_dim; victim->num_blocks = d->num_blocks; victim->Hkv = d->num_kv_heads;
    victim->sb = sb; victim->sh = sh; victim->st = st;
    victim->stamp = ++c->map_stamp;
    return &victim->map;
}

static const CUtensorMap* q_map(cf_ctx* c, const void* base, int D, int rows, int Hq)
{
    QMapEntry* victim = &c->q_maps[0];
    for (QMapEntry& e : c->q_maps) {
        if (e.base == base && e.D == D && e.rows == rows && e.Hq == Hq) {
            e.stamp = ++c->map_stamp;
            return &e.map;
        }
        if (e.stamp < victim->stamp) victim = &e;
    }
    if (!encode_q_map(&victim->map, base, D, rows, Hq)) {
        victim->base = nullptr;
        return nullptr;
    }
    victim->base = base; victim->D = D; victim->rows = rows; victim->Hq = Hq;
    victim->stamp = ++c->map_stamp;
    return &victim->map;
}

static float scale_log2_of(const cf_cache_desc* d)
{
    const float sc = d->softmax_scale > 0.f ? d->softmax_scale : 1.0f / std::sqrt((float)d->head_dim);
    return sc * 1.4426950408889634f;
}

}  // namespace cf

namespace cf {

struct PlanCounts {
    int n_dec = 0, n_comb = 0, n_shared = 0, n_pre_tc = 0, n_pre_comb = 0, total_q = 0;
    int n_stage_seqs = 0, n_stage_pages = 0, max_stage_pages = 0, num_seqs = 0;   // fp8 cache: pages to expand for the prefill chunks
    bool pair = false;          // the prefill items are pair items (two CTAs each)
    int front_sms = 0;          // spatial sequence: SMs of the first prefill grid, as the plan was balanced for
    int n_part_slots = 0;
};

// Split-K workspace: the ticket counters, decode partials [slot, Hq, D] + [slot, Hq, 2], then the compact
// partial rows of KV-split prefill items [row slot, D] + [row slot, 2].
// For an fp8 cache the workspace also holds the bf16 staging pools of the prefill chunks' pages (K and V,
// [stage page, Hkv, 16, D]) and the staging block table [S, max_blocks].
struct WsLayout {
    size_t dec_o = 0, dec_ml = 0, pre_o = 0, pre_ml = 0, stage_k = 0, stage_v = 0, stage_bt = 0, total = 0;
};
static WsLayout ws_layout(int n_part_slots, int n_pre_slots, int Hq, int D, int n_stage_pages = 0, int Hkv = 0, int64_t table_entries = 0)
{
    WsLayout w;
    w.dec_o = kCounterBytes;
    w.dec_ml = w.dec_o + align_up((size_t)n_part_slots * Hq * D * sizeof(float), 256);
    w.pre_o = w.dec_ml + align_up((size_t)n_part_slots * Hq * 2 * sizeof(float), 256);
    w.pre_ml = w.pre_o + align_up((size_t)n_pre_slots * D * sizeof(float), 256);
    w.stage_k = w.pre_ml + align_up((size_t)n_pre_slots * 2 * sizeof(float), 256);
    const size_t pool = n_stage_pages > 0 ? align_up((size_t)n_stage_pages * Hkv * 16 * D * 2, 1024) : 0;
    w.stage_v = w.stage_k + pool;
    w.stage_bt = w.stage_v + pool;
    w.total = w.stage_bt + (n_stage_pages > 0 ? align_up((size_t)table_entries * sizeof(int32_t), 256) : 0);
    return w;
}

// fp8 cache: which pages of which prefill sequences have to be expanded to bf16 for the prefill kernel (from the first
// page any row of the chunk can see - 0 without a sliding window - to the last page of the context)
static void stage_list(const cf_cache_desc* d, const int32_t* context_len, const int32_t* query_len, int32_t S,
                       std::vector<StageSeq>* seqs, int* n_pages, int* max_pages)
{
    seqs->clear();
    *n_pages = 0;
    *max_pages = 0;
    if (d->kv_dtype != CF_KV_FP8_E4M3) return;
    for (int32_t s = 0; s < S; ++s) {
        if (query_len[s] <= 1) continue;
        const int32_t prefix = context_len[s] - query_len[s];
        const int32_t lo = d->window_size > 0 ? std::max(0, prefix - d->window_size + 1) : 0;
        StageSeq q;
        q.seq = s;
        q.page0 = lo / 16;
        q.n_pages = (context_len[s] + 15) / 16 - q.page0;
        q.stage_base = *n_pages;
        *n_pages += q.n_pages;
        *max_pages = std::max(*max_pages, q.n_pages);
        seqs->push_back(q);
    }
}

// Enqueues decode -> combine -> prefill for a plan that already sits in device memory at `base`.
static cf_status launch_attention(cf_ctx* c, const cf_cache_desc* desc, const PlanCounts& n, const PlanLayout& L,
                                  uint8_t* base, float* ws, const WsLayout& W, const void* q, const void* k_cache,
                                  const void* v_cache, const int32_t* block_table, int32_t max_blocks_per_seq, void* out,
                                  float* lse, cudaStream_t stream, bool allow_timing)
{
    const int Hq = desc->num_q_heads, D = desc->head_dim;
    AttnParams p;
    p.q = (const __nv_bfloat16*)q;
    p.k_cache = (const __nv_bfloat16*)k_cache;
    p.v_cache = (const __nv_bfloat16*)v_cache;
    p.out = (__nv_bfloat16*)out;
    p.lse = lse;
    p.block_table = block_table;
    p.max_blocks = max_blocks_per_seq;
    p.num_blocks = desc->num_blocks;
    p.ks_block = desc->k_stride_block; p.ks_head = desc->k_stride_head; p.ks_token = desc->k_stride_token;
    p.vs_block = desc->v_stride_block; p.vs_head = desc->v_stride_head; p.vs_token = desc->v_stride_token;
    p.Hq = Hq; p.Hkv = desc->num_kv_heads; p.G = Hq / desc->num_kv_heads;
    p.scale_log2 = scale_log2_of(desc);
    p.window = desc->window_size;
    p.sinks = desc->sink_logits;
    const bool fp8 = desc->kv_dtype == CF_KV_FP8_E4M3;
    p.k_scale = fp8 ? desc->k_scale : nullptr;
    p.v_scale = fp8 ? desc->v_scale : nullptr;
    p.q_start = (const int32_t*)(base + L.off_qstart);
    p.context_len = (const int32_t*)(base + L.off_ctx);
    p.query_len = (const int32_t*)(base + L.off_qlen);
    p.dec_items = (const DecodeItem*)(base + L.off_dec);
    p.comb_items = (const CombineItem*)(base + L.off_comb);
    p.sh_items = (const SharedDecodeItem*)(base + L.off_sh);
    p.sh_members = (const ShareMember*)(base + L.off_shm);
    p.pre_tc_items = (const PrefillTcItem*)(base + L.off_pre_tc);
    p.part_o = (float*)((uint8_t*)ws + W.dec_o);
    p.part_ml = (float*)((uint8_t*)ws + W.dec_ml);
    const bool fused_combine = c->fused_combine && (size_t)n.n_part_slots * desc->num_kv_heads * sizeof(uint32_t) <= kCounterBytes;
    p.dec_counters = fused_combine ? (uint32_t*)ws : nullptr;
    p.pre_part_o = (float*)((uint8_t*)ws + W.pre_o);
    p.pre_part_ml = (float*)((uint8_t*)ws + W.pre_ml);
    p.pre_comb_items = (const PrefillCombineItem*)(base + L.off_pre_comb);
    p.pre_queue = (uint32_t*)(base + L.off_queue);
    p.err = c->err_dev;

    cudaError_t e = cudaSuccess;
    TimedCall* tc = nullptr;
    if (c->timing && allow_timing) {
        if (c->timed_used == c->timed.size()) {
            TimedCall fresh;
            bool ok = true;
            for (int i = 0; i < 4 && ok; ++i) ok = cudaEventCreate(&fresh.ev[i]) == cudaSuccess;
            if (!ok) return CF_ERR_CUDA;
            c->timed.push_back(fresh);
        }
        tc = &c->timed[c->timed_used++];
        tc->ran[0] = (n.n_dec > 0);
        tc->ran[1] = (n.n_comb > 0) && !fused_combine;
        tc->ran[2] = n.n_pre_tc > 0;
    }
    const bool has_prefill = n.n_pre_tc > 0;
    // the prefill kernels' view of the cache: the caller's pools, or (fp8 cache) the bf16 staging pools in the workspace
    AttnParams pp = p;
    cf_cache_desc pdesc = *desc;
    if (fp8 && has_prefill) {
        pp.k_cache = (const __nv_bfloat16*)((uint8_t*)ws + W.stage_k);
        pp.v_cache = (const __nv_bfloat16*)((uint8_t*)ws + W.stage_v);
        pp.block_table = (const int32_t*)((uint8_t*)ws + W.stage_bt);
        pp.num_blocks = n.n_stage_pages;
        pdesc.num_blocks = n.n_stage_pages;
        pdesc.k_stride_block = pdesc.v_stride_block = (int64_t)desc->num_kv_heads * 16 * D;
        pdesc.k_stride_head = pdesc.v_stride_head = 16 * D;
        pdesc.k_stride_token = pdesc.v_stride_token = D;
        pp.ks_block = pp.vs_block = pdesc.k_stride_block;
        pp.ks_head = pp.vs_head = pdesc.k_stride_head;
        pp.ks_token = pp.vs_token = pdesc.k_stride_token;
    }
    PrefillMaps maps;
    if (has_prefill) {
        const CUtensorMap* mq = q_map(c, q, D, n.total_q, Hq);
        const CUtensorMap* mk = pool_map(c, pp.k_cache, &pdesc, pdesc.k_stride_block, pdesc.k_stride_head, pdesc.k_stride_token);
        const CUtensorMap* mv = pool_map(c, pp.v_cache, &pdesc, pdesc.v_stride_block, pdesc.v_stride_head, pdesc.v_stride_token);
        if (!mq || !mk || !mv) return CF_ERR_CUDA;
        maps.q = *mq; maps.k = *mk; maps.v = *mv;
    }
    // fp8 cache: the pages of the prefill chunks are expanded first, on the caller's stream (the prefill kernel behind
    // it waits for the grid before it in the stream to complete before its first read)
    auto stage_pages = [&](cudaStream_t st) -> cudaError_t {
        if (!(fp8 && has_prefill)) return cudaSuccess;
        return launch_kv_dequant_gather(p, (const StageSeq*)(base + L.off_stage), n.n_stage_seqs, n.max_stage_pages,
                                        (__nv_bfloat16*)((uint8_t*)ws + W.stage_k), (__nv_bfloat16*)((uint8_t*)ws + W.stage_v),
                                        (int32_t*)((uint8_t*)ws + W.stage_bt), st);
    };
    auto decode_launch = [&](cudaStream_t st) -> cudaError_t {
        return fp8 ? launch_decode_fp8(p, n.n_dec, st) : launch_decode_with_shared(p, D, n.n_shared, n.n_dec, st);
    };
    int second_grid = 0;
    // Slots that take a prefill item: SMs, or pairs of SMs for pair items.  Grid sizes, the shared work queue and
    // the front / tail split below are counted in slots.
    const int per_slot = n.pair ? 2 : 1;
    const int sms = (c->num_sms > 0 ? c->num_sms : 148) / per_slot;
    const int pre_ctas = n.n_pre_tc < sms ? n.n_pre_tc : sms;      // persistent CTAs (pairs) of the serial sequence
    auto launch_prefill = [&](int n_slots, int queue_slots, int first_static, int ticket_base, uint32_t* resident, cudaStream_t st) {
        return n.pair ? launch_prefill_tc2(pp, maps, n.n_pre_tc, n_slots, queue_slots, first_static, ticket_base, resident, st)
                      : launch_prefill_tc(pp, maps, D, n.n_pre_tc, n_slots, queue_slots, first_static, ticket_base, resident, st);
    };
    if (c->overlap && !c->in_host_step && !tc && has_prefill && (n.n_dec > 0)) {
        // Spatial partition.  `front` persistent prefill CTAs (one per SM: a CTA takes an SM's whole shared
        // memory) go first, on the caller's stream; decode runs on the SMs left over, on a context-owned side
        // stream forked from the caller's; a second prefill grid behind decode on that stream draws from the
        // same ticket counter, so the SMs that decode frees join the prefill as soon as decode is done; the
        // side stream is joined back before the prefill combine.
        // The front grid's share comes from spatial_front_sms (or cf_set_overlap): decode keeps the SMs it needs to be
        // done by the time the prefill is.
        int front = (c->spatial_sms > 0 ? c->spatial_sms : n.front_sms > 0 ? n.front_sms : (c->num_sms * 3) / 5) / per_slot;
        if (front < 1) front = 1;
        if (front > sms) front = sms;
        if (front > n.n_pre_tc) front = n.n_pre_tc;
        int tail = n.n_pre_tc - front;
        if (tail > sms) tail = sms;
        second_grid = tail > 0;
        // Decode must not start before the front CTAs hold their SMs (its grid would otherwise fill the
        // machine first and the prefill CTAs, which need an SM to themselves, would wait for its end: the call
        // then takes longer than the serial sequence).  Enqueueing the front grid first, on the stream that needs
        // no cross-stream event, wins that race only some of the time, so the order is enforced: the front CTAs
        // count themselves in and the side stream waits for that count with a stream memory operation before
        // decode (a few microseconds per call; not while the stream is being captured: in a graph the two branches
        // start together, front grid first, and memory-operation nodes cost more than they return).
        uint32_t* resident = nullptr;
        const StreamMemOps& mo = stream_mem_ops();
        cudaStreamCaptureStatus cap = cudaStreamCaptureStatusNone;
        if (front > 0 && c->spatial_wait && mo.ok && cudaStreamIsCapturing(stream, &cap) == cudaSuccess && cap == cudaStreamCaptureStatusNone) {
            resident = p.pre_queue + 2;
            if (mo.write(stream, (CUdeviceptr)(uintptr_t)resident, 0u, 0u) != CUDA_SUCCESS) e = cudaErrorUnknown;
        }
        if (e == cudaSuccess) e = stage_pages(stream);      // before the fork: the second prefill grid on the side stream reads the staging area too
        if (cudaEventRecord(c->ev_fork, stream) != cudaSuccess || cudaStreamWaitEvent(c->side, c->ev_fork, 0) != cudaSuccess)
            e = cudaErrorUnknown;
        if (e == cudaSuccess) e = launch_prefill(front, front + tail, 1, front, resident, stream);
        // only after the front grid has been enqueued without an error, so that the count is certain to arrive
        if (e == cudaSuccess && resident &&
            mo.wait(c->side, (CUdeviceptr)(uintptr_t)resident, (cuuint32_t)(front * per_slot), CU_STREAM_WAIT_VALUE_GEQ) != CUDA_SUCCESS)
            e = cudaErrorUnknown;
        if (e == cudaSuccess) e = decode_launch(c->side);
        if (e == cudaSuccess) e = launch_combine(p, D, fused_combine ? 0 : n.n_comb, c->side);
        if (e == cudaSuccess) e = launch_prefill(tail, front + tail, 0, front, nullptr, c->side);
        if (cudaEventRecord(c->ev_join, c->side) != cudaSuccess && e == cudaSuccess) e = cudaErrorUnknown;
        if (cudaStreamWaitEvent(stream, c->ev_join, 0) != cudaSuccess && e == cudaSuccess) e = cudaErrorUnknown;
        if (e == cudaSuccess) e = launch_prefill_combine(pp, D, n.n_pre_comb, stream);
    } else {
        if (tc) cudaEventRecord(tc->ev[0], stream);
        if (e == cudaSuccess) e = decode_launch(stream);
        if (tc) cudaEventRecord(tc->ev[1], stream);
        if (e == cudaSuccess) e = launch_combine(p, D, fused_combine ? 0 : n.n_comb, stream);
        if (tc) cudaEventRecord(tc->ev[2], stream);
        if (e == cudaSuccess) e = stage_pages(stream);
        if (e == cudaSuccess) e = launch_prefill(pre_ctas, pre_ctas, 1, pre_ctas, nullptr, stream);
        if (e == cudaSuccess) e = launch_prefill_combine(pp, D, n.n_pre_comb, stream);
        if (tc) cudaEventRecord(tc->ev[3], stream);
    }
    c->launches = (int)(n.n_dec > 0) + (int)(n.n_comb > 0 && !fused_combine) + (int)(n.n_pre_tc > 0) + (int)(n.n_pre_comb > 0) + second_grid;
    return e == cudaSuccess ? CF_OK : CF_ERR_CUDA;
}

}  // namespace cf

using namespace cf;

extern "C" {

const char* cf_status_string(cf_status s)
{
    switch (s) {
        case CF_OK: return "CF_OK";
        case CF_ERR_INVALID_ARG: return "CF_ERR_INVALID_ARG";
        case CF_ERR_UNSUPPORTED: return "CF_ERR_UNSUPPORTED";
        case CF_ERR_OUT_OF_RANGE: return "CF_ERR_OUT_OF_RANGE";
        case CF_ERR_WORKSPACE: return "CF_ERR_WORKSPACE";
        case CF_ERR_CUDA: return "CF_ERR_CUDA";
        case CF_ERR_TIMEOUT: return "CF_ERR_TIMEOUT";
        case CF_ERR_ARCH: return "CF_ERR_ARCH";
        case CF_ERR_BUSY: return "CF_ERR_BUSY";
    }
    return "CF_ERR_UNKNOWN";
}

cf_status cf_create(cf_ctx** out, int device, size_t workspace_bytes)
{
    if (!out) return CF_ERR_INVALID_ARG;
    *out = nullptr;
    int count = 0;
    if (cudaGetDeviceCount(&count) != cudaSuccess || device < 0 || device >= count) {
        cudaGetLastError();
        return count == 0 ? CF_ERR_CUDA : CF_ERR_INVALID_ARG;
    }
    cudaDeviceProp prop;
    if (cudaGetDeviceProperties(&prop, device) != cudaSuccess) return CF_ERR_CUDA;
    if (prop.major != 10) return CF_ERR_ARCH;
    DeviceGuard guard(device);
    if (!guard.ok) return CF_ERR_CUDA;
    cf_ctx* c = new (std::nothrow) cf_ctx();
    if (!c) return CF_ERR_CUDA;
    c->device = device;
    c->num_sms = prop.multiProcessorCount;
    c->cfg.num_sms = c->num_sms;
    {
        const char* v = std::getenv("CF_OVERLAP");          // spatial sequence unless CF_OVERLAP=0
        c->overlap = !(v && v[0] == '0' && v[1] == 0);
    }
    c->spatial_sms = c->spatial_sms_default = env_int("CF_SPATIAL_SMS", 0);
    bool ok = true;
    for (int i = 0; i < kRing && ok; ++i)
        ok = cudaEventCreateWithFlags(&c->slots[i].done, cudaEventDisableTiming) == cudaSuccess &&
             cudaEventCreateWithFlags(&c->slots[i].uploaded, cudaEventDisableTiming) == cudaSuccess;
    ok = ok && ensure_plan_capacity(c, kDefaultPlanBytes) == CF_OK;
    c->workspace_fixed = false;
    ok = ok && ensure_workspace(c, workspace_bytes ? workspace_bytes : kDefaultWorkspace) == CF_OK;
    c->workspace_fixed = workspace_bytes != 0;
    ok = ok && cudaStreamCreateWithFlags(&c->side, cudaStreamNonBlocking) == cudaSuccess;
    ok = ok && cudaStreamCreateWithFlags(&c->upload_stream, cudaStreamNonBlocking) == cudaSuccess;
    ok = ok && cudaStreamCreateWithFlags(&c->h2d_stream, cudaStreamNonBlocking) == cudaSuccess;
    ok = ok && cudaStreamCreateWithFlags(&c->h2d_kv_stream, cudaStreamNonBlocking) == cudaSuccess;
    ok = ok && cudaStreamCreateWithFlags(&c->d2h_stream, cudaStreamNonBlocking) == cudaSuccess;
    for (int i = 0; i < kHostStages && ok; ++i) {
        ok = cudaEventCreateWithFlags(&c->stage[i].h2d_done, cudaEventDisableTiming) == cudaSuccess &&
             cudaEventCreateWithFlags(&c->stage[i].h2d_kv_done, cudaEventDisableTiming) == cudaSuccess &&
             cudaEventCreateWithFlags(&c->stage[i].compute_done, cudaEventDisableTiming) == cudaSuccess &&
             cudaEventCreateWithFlags(&c->stage[i].d2h_done, cudaEventDisableTiming) == cudaSuccess;
    }
    ok = ok && cudaEventCreateWithFlags(&c->ev_fork, cudaEventDisableTiming) == cudaSuccess;
    ok = ok && cudaEventCreateWithFlags(&c->ev_join, cudaEventDisableTiming) == cudaSuccess;
    ok = ok && cudaMalloc((void**)&c->err_dev, 2 * sizeof(uint32_t)) == cudaSuccess;
    ok = ok && cudaMemset(c->err_dev, 0, 2 * sizeof(uint32_t)) == cudaSuccess && cudaDeviceSynchronize() == cudaSuccess;
    if (!ok) {
        cf_destroy(c);
        return CF_ERR_CUDA;
    }
    *out = c;
    return CF_OK;
}

cf_status cf_destroy(cf_ctx* c)
{
    if (!c) return CF_ERR_INVALID_ARG;
    if (c->live_plans.load() > 0) return CF_ERR_BUSY;      // a plan holds a pointer to its context
    DeviceGuard guard(c->device);
    cudaDeviceSynchronize();
    for (int i = 0; i < kRing; ++i) {
        if (c->slots[i].host) cudaFreeHost(c->slots[i].host);
        if (c->slots[i].dev) cudaFree(c->slots[i].dev);
        if (c->slots[i].done) cudaEventDestroy(c->slots[i].done);
        if (c->slots[i].uploaded) cudaEventDestroy(c->slots[i].uploaded);
    }
    for (cf::TimedCall& tc : c->timed)
        for (int i = 0; i < 4; ++i)
            if (tc.ev[i]) cudaEventDestroy(tc.ev[i]);
    if (c->workspace) cudaFree(c->workspace);
    if (c->err_dev) cudaFree(c->err_dev);
    if (c->ev_fork) cudaEventDestroy(c->ev_fork);
    if (c->ev_join) cudaEventDestroy(c->ev_join);
    if (c->side) cudaStreamDestroy(c->side);
    if (c->upload_stream) cudaStreamDestroy(c->upload_stream);
    for (int i = 0; i < kHostStages; ++i) {
        HostStage& hs = c->stage[i];
        if (hs.dev) cudaFree(hs.dev);
        if (hs.h2d_done) cudaEventDestroy(hs.h2d_done);
        if (hs.h2d_kv_done) cudaEventDestroy(hs.h2d_kv_done);
        if (hs.compute_done) cudaEventDestroy(hs.compute_done);
        if (hs.d2h_done) cudaEventDestroy(hs.d2h_done);
    }
    if (c->h2d_stream) cudaStreamDestroy(c->h2d_stream);
    if (c->h2d_kv_stream) cudaStreamDestroy(c->h2d_kv_stream);
    if (c->d2h_stream) cudaStreamDestroy(c->d2h_stream);
    delete c;
    return CF_OK;
}

cf_status cf_kv_append(cf_ctx* c, const cf_cache_desc* desc, void* k_cache, void* v_cache,
                       const void* k_new, const void* v_new,
                       const int32_t* block_table, int32_t max_blocks_per_seq,
                       const int32_t* context_len, const int32_t* query_len,
                       int32_t num_seqs, void* cuda_stream)
{
    if (!c || !desc) return CF_ERR_INVALID_ARG;
    const int64_t t_in = now_ns();
    cf_status st = validate_desc(desc);
    if (st != CF_OK) return st;
    Plan pl;
    st = validate_lengths(desc, context_len, query_len, num_seqs, max_blocks_per_seq, &pl);
    if (st != CF_OK) return st;
    if (pl.total_q == 0) return CF_OK;
    if (!k_cache || !v_cache || !k_new || !v_new || !block_table) return CF_ERR_INVALID_ARG;
    DeviceGuard guard(c->device);
    if (!guard.ok) return CF_ERR_CUDA;
    cudaStream_t stream = (cudaStream_t)cuda_stream;
    PlanLayout L;
    uint8_t* base = nullptr;
    PlanSlot* slot = nullptr;
    st = upload_plan(c, num_seqs, context_len, query_len, pl, stream, &L, &base, &slot);
    if (st != CF_OK) return st;
    AppendParams p;
    p.k_cache = (__nv_bfloat16*)k_cache;
    p.v_cache = (__nv_bfloat16*)v_cache;
    p.k_new = (const __nv_bfloat16*)k_new;
    p.v_new = (const __nv_bfloat16*)v_new;
    p.block_table = block_table;
    p.max_blocks = max_blocks_per_seq;
    p.ks_block = desc->k_stride_block; p.ks_head = desc->k_stride_head; p.ks_token = desc->k_stride_token;
    p.vs_block = desc->v_stride_block; p.vs_head = desc->v_stride_head; p.vs_token = desc->v_stride_token;
    p.Hkv = desc->num_kv_heads; p.D = desc->head_dim; p.num_seqs = num_seqs; p.total_rows = pl.total_q;
    p.num_blocks = desc->num_blocks; p.err = c->err_dev;
    p.k_scale = desc->kv_dtype == CF_KV_FP8_E4M3 ? desc->k_scale : nullptr;
    p.v_scale = desc->kv_dtype == CF_KV_FP8_E4M3 ? desc->v_scale : nullptr;
    p.q_start = (const int32_t*)(base + L.off_qstart);
    p.context_len = (const int32_t*)(base + L.off_ctx);
    p.query_len = (const int32_t*)(base + L.off_qlen);
    const cudaError_t e = launch_kv_append(p, stream);
    const cf_status fs = finish_slot(slot, stream);
    c->host_ns_append += now_ns() - t_in;
    ++c->host_calls_append;
    if (e != cudaSuccess) return CF_ERR_CUDA;
    return fs;
}

cf_status cf_mixed_attention(cf_ctx* c, const cf_cache_desc* desc, const void* q,
                             const void* k_cache, const void* v_cache,
                             const int32_t* block_table, int32_t max_blocks_per_seq,
                             const int32_t* context_len, const int32_t* query_len, int32_t num_seqs,
                             void* out, float* lse, void* cuda_stream)
{
    return cf_mixed_attention_shared(c, desc, q, k_cache, v_cache, block_table, max_blocks_per_seq, context_len, query_len,
                                     nullptr, nullptr, num_seqs, out, lse, cuda_stream);
}

cf_status cf_mixed_attention_shared(cf_ctx* c, const cf_cache_desc* desc, const void* q,
                                    const void* k_cache, const void* v_cache,
                                    const int32_t* block_table, int32_t max_blocks_per_seq,
                                    const int32_t* context_len, const int32_t* query_len,
                                    const int32_t* share_group, const int32_t* shared_len, int32_t num_seqs,
                                    void* out, float* lse, void* cuda_stream)
{
    if (!c || !desc) return CF_ERR_INVALID_ARG;
    if ((share_group == nullptr) != (shared_len == nullptr)) return CF_ERR_INVALID_ARG;
    const int64_t t_in = now_ns();
    cf_status st = validate_desc(desc);
    if (st != CF_OK) return st;
    Plan pl;
    PlanConfig cfg = c->cfg;
    const int front_sms = !(c->overlap && !c->in_host_step) ? 0 : c->spatial_sms > 0 ? c->spatial_sms
                              : spatial_front_sms(desc, context_len, query_len, num_seqs, c->num_sms);
    cfg.prefill_sms_mixed = c->timing ? 0 : front_sms;
    cfg.prefill_pair = c->use_pairs && prefill_pair_supported(desc);
    st = build_plan(desc, context_len, query_len, num_seqs, max_blocks_per_seq, cfg, &pl, share_group, shared_len);
    if (st != CF_OK) return st;
    c->host_ns_planner += now_ns() - t_in;
    c->launches = 0;
    if (pl.total_q == 0) return CF_OK;
    if (!q || !k_cache || !v_cache || !block_table || !out) return CF_ERR_INVALID_ARG;
    DeviceGuard guard(c->device);
    if (!guard.ok) return CF_ERR_CUDA;
    cudaStream_t stream = (cudaStream_t)cuda_stream;

    const int Hq = desc->num_q_heads, D = desc->head_dim;
    std::vector<StageSeq> stage;
    int n_stage_pages = 0, max_stage_pages = 0;
    if (!pl.prefill_tc.empty()) stage_list(desc, context_len, query_len, num_seqs, &stage, &n_stage_pages, &max_stage_pages);
    const WsLayout W = ws_layout(pl.n_part_slots, pl.n_pre_slots, Hq, D, n_stage_pages, desc->num_kv_heads,
                                 (int64_t)num_seqs * max_blocks_per_seq);
    st = ensure_workspace(c, W.total);
    if (st != CF_OK) return st;

    PlanLayout L;
    uint8_t* base = nullptr;
    PlanSlot* slot = nullptr;
    st = upload_plan(c, num_seqs, context_len, query_len, pl, stream, &L, &base, &slot, &stage);
    if (st != CF_OK) return st;

    PlanCounts n;
    n.n_dec = (int)pl.decode.size(); n.n_comb = (int)pl.combine.size(); n.n_shared = (int)pl.shared_decode.size();
    n.n_pre_tc = (int)pl.prefill_tc.size(); n.n_pre_comb = (int)pl.prefill_combine.size(); n.total_q = pl.total_q;
    n.n_part_slots = pl.n_part_slots;
    n.pair = pl.pair;
    n.n_stage_seqs = (int)stage.size(); n.n_stage_pages = n_stage_pages; n.max_stage_pages = max_stage_pages; n.num_seqs = num_seqs;
    c->last_counts[0] = n.n_dec; c->last_counts[1] = n.n_comb; c->last_counts[2] = n.n_pre_tc; c->last_counts[3] = n.n_part_slots;
    c->last_counts[4] = n.n_pre_comb; c->last_counts[5] = n.n_shared; c->last_counts[6] = (int32_t)pl.share_members.size();
    c->last_counts[7] = pl.pair ? 1 : 0;
    n.front_sms = front_sms;
    const cf_status ls = launch_attention(c, desc, n, L, base, c->workspace, W,
                                          q, k_cache, v_cache, block_table, max_blocks_per_seq, out, lse, stream, true);
    const cf_status fs = finish_slot(slot, stream);
    c->host_ns_attention += now_ns() - t_in;
    ++c->host_calls_attention;
    return ls != CF_OK ? ls : fs;
}

cf_status cf_plan_create(cf_ctx* c, const cf_cache_desc* desc, const int32_t* context_len, const int32_t* query_len,
                         int32_t num_seqs, int32_t max_blocks_per_seq, void* cuda_stream, cf_plan** out)
{
    if (!c || !desc || !out) return CF_ERR_INVALID_ARG;
    *out = nullptr;
    cf_status st = validate_desc(desc);
    if (st != CF_OK) return st;
    Plan pl;
    PlanConfig cfg = c->cfg;
    const int front_sms = !(c->overlap && !c->in_host_step) ? 0 : c->spatial_sms > 0 ? c->spatial_sms
                              : spatial_front_sms(desc, context_len, query_len, num_seqs, c->num_sms);
    cfg.prefill_sms_mixed = front_sms;
    cfg.prefill_pair = c->use_pairs && prefill_pair_supported(desc);
    st = build_plan(desc, context_len, query_len, num_seqs, max_blocks_per_seq, cfg, &pl);
    if (st != CF_OK) return st;
    DeviceGuard guard(c->device);
    if (!guard.ok) return CF_ERR_CUDA;
    cf_plan* P = new (std::nothrow) cf_plan();
    if (!P) return CF_ERR_CUDA;
    P->ctx = c;
    P->desc = *desc;
    P->num_seqs = num_seqs;
    P->max_blocks = max_blocks_per_seq;
    std::vector<StageSeq> stage;
    int n_stage_pages = 0, max_stage_pages = 0;
    if (!pl.prefill_tc.empty()) stage_list(desc, context_len, query_len, num_seqs, &stage, &n_stage_pages, &max_stage_pages);
    const PlanLayout L = layout_of(num_seqs, pl, stage.size());
    P->off_stage = L.off_stage;
    P->n_stage_seqs = (int)stage.size(); P->n_stage_pages = n_stage_pages; P->max_stage_pages = max_stage_pages;
    P->off_qstart = L.off_qstart; P->off_ctx = L.off_ctx; P->off_qlen = L.off_qlen; P->off_dec = L.off_dec;
    P->off_comb = L.off_comb; P->off_sh = L.off_sh; P->off_shm = L.off_shm; P->off_pre_tc = L.off_pre_tc; P->off_pre_comb = L.off_pre_comb; P->off_queue = L.off_queue;
    P->total = L.total;
    P->n_dec = (int)pl.decode.size(); P->n_comb = (int)pl.combine.size();
    P->n_pre_tc = (int)pl.prefill_tc.size(); P->n_pre_comb = (int)pl.prefill_combine.size(); P->total_q = pl.total_q;
    P->front_sms = front_sms;
    P->n_part_slots = pl.n_part_slots; P->n_pre_slots = pl.n_pre_slots;
    P->pair = pl.pair;
    const size_t part_bytes = ws_layout(pl.n_part_slots, pl.n_pre_slots, desc->num_q_heads, desc->head_dim, n_stage_pages,
                                        desc->num_kv_heads, (int64_t)num_seqs * max_blocks_per_seq).total;
    bool ok = cudaMallocHost((void**)&P->host, L.total) == cudaSuccess && cudaMalloc((void**)&P->dev, L.total) == cudaSuccess;
    // the ticket counters are zeroed on the caller's stream, like the plan copy: every launch that uses the plan
    // is ordered behind this call on that stream (or by the caller)
    if (ok && part_bytes)
        ok = cudaMalloc((void**)&P->part, part_bytes) == cudaSuccess &&
             cudaMemsetAsync(P->part, 0, kCounterBytes, (cudaStream_t)cuda_stream) == cudaSuccess;
    if (ok) {
        std::memcpy(P->host + L.off_qstart, pl.q_start.data(), sizeof(int32_t) * ((size_t)num_seqs + 1));
        if (num_seqs > 0) {
            std::memcpy(P->host + L.off_ctx, context_len, sizeof(int32_t) * (size_t)num_seqs);
            std::memcpy(P->host + L.off_qlen, query_len, sizeof(int32_t) * (size_t)num_seqs);
        }
        if (P->n_dec) std::memcpy(P->host + L.off_dec, pl.decode.data(), sizeof(DecodeItem) * pl.decode.size());
        if (P->n_comb) std::memcpy(P->host + L.off_comb, pl.combine.data(), sizeof(CombineItem) * pl.combine.size());
        if (P->n_pre_tc) std::memcpy(P->host + L.off_pre_tc, pl.prefill_tc.data(), sizeof(PrefillTcItem) * pl.prefill_tc.size());
        if (P->n_pre_comb)
            std::memcpy(P->host + L.off_pre_comb, pl.prefill_combine.data(), sizeof(PrefillCombineItem) * pl.prefill_combine.size());
        if (!stage.empty()) std::memcpy(P->host + L.off_stage, stage.data(), sizeof(StageSeq) * stage.size());
        std::memset(P->host + L.off_queue, 0, 16);
        ok = cudaMemcpyAsync(P->dev, P->host, L.total, cudaMemcpyHostToDevice, (cudaStream_t)cuda_stream) == cudaSuccess;
    }
    c->live_plans.fetch_add(1);
    if (!ok) {
        cf_plan_destroy(P);
        return CF_ERR_CUDA;
    }
    *out = P;
    return CF_OK;
}

cf_status cf_plan_destroy(cf_plan* P)
{
    if (!P) return CF_ERR_INVALID_ARG;
    DeviceGuard guard(P->ctx->device);
    cudaDeviceSynchronize();
    if (P->host) cudaFreeHost(P->host);
    if (P->dev) cudaFree(P->dev);
    if (P->part) cudaFree(P->part);
    P->ctx->live_plans.fetch_sub(1);
    delete P;
    return CF_OK;
}

cf_status cf_kv_append_planned(cf_plan* P, void* k_cache, void* v_cache, const void* k_new, const void* v_new,
                               const int32_t* block_table, void* cuda_stream)
{
    if (!P) return CF_ERR_INVALID_ARG;
    if (P->total_q == 0) return CF_OK;
    if (!k_cache || !v_cache || !k_new || !v_new || !block_table) return CF_ERR_INVALID_ARG;
    DeviceGuard guard(P->ctx->device);
    if (!guard.ok) return CF_ERR_CUDA;
    const cf_cache_desc* desc = &P->desc;
    AppendParams p;
    p.k_cache = (__nv_bfloat16*)k_cache;
    p.v_cache = (__nv_bfloat16*)v_cache;
    p.k_new = (const __nv_bfloat16*)k_new;
    p.v_new = (const __nv_bfloat16*)v_new;
    p.block_table = block_table;
    p.max_blocks = P->max_blocks;
    p.ks_block = desc->k_stride_block; p.ks_head = desc->k_stride_head; p.ks_token = desc->k_stride_token;
    p.vs_block = desc->v_stride_block; p.vs_head = desc->v_stride_head; p.vs_token = desc->v_stride_token;
    p.Hkv = desc->num_kv_heads; p.D = desc->head_dim; p.num_seqs = P->num_seqs; p.total_rows = P->total_q;
    p.num_blocks = desc->num_blocks; p.err = P->ctx->err_dev;
    p.k_scale = desc->kv_dtype == CF_KV_FP8_E4M3 ? desc->k_scale : nullptr;
    p.v_scale = desc->kv_dtype == CF_KV_FP8_E4M3 ? desc->v_scale : nullptr;
    p.q_start = (const int32_t*)(P->dev + P->off_qstart);
    p.context_len = (const int32_t*)(P->dev + P->off_ctx);
    p.query_len = (const int32_t*)(P->dev + P->off_qlen);
    return launch_kv_append(p, (cudaStream_t)cuda_stream) == cudaSuccess ? CF_OK : CF_ERR_CUDA;
}

cf_status cf_mixed_attention_planned(cf_plan* P, const void* q, const void* k_cache, const void* v_cache,
                                     const int32_t* block_table, void* out, float* lse, void* cuda_stream)
{
    if (!P) return CF_ERR_INVALID_ARG;
    P->ctx->launches = 0;
    if (P->total_q == 0) return CF_OK;
    if (!q || !k_cache || !v_cache || !block_table || !out) return CF_ERR_INVALID_ARG;
    DeviceGuard guard(P->ctx->device);
    if (!guard.ok) return CF_ERR_CUDA;
    PlanLayout L;
    L.off_qstart = P->off_qstart; L.off_ctx = P->off_ctx; L.off_qlen = P->off_qlen; L.off_dec = P->off_dec;
    L.off_comb = P->off_comb; L.off_sh = P->off_sh; L.off_shm = P->off_shm; L.off_pre_tc = P->off_pre_tc; L.off_stage = P->off_stage; L.off_pre_comb = P->off_pre_comb; L.off_queue = P->off_queue;
    L.total = P->total;
    PlanCounts n;
    n.n_dec = P->n_dec; n.n_comb = P->n_comb; n.n_pre_tc = P->n_pre_tc; n.n_pre_comb = P->n_pre_comb;
    n.total_q = P->total_q;
    n.front_sms = P->front_sms;
    n.n_part_slots = P->n_part_slots;
    n.pair = P->pair;
    n.n_stage_seqs = P->n_stage_seqs; n.n_stage_pages = P->n_stage_pages; n.max_stage_pages = P->max_stage_pages; n.num_seqs = P->num_seqs;
    const WsLayout W = ws_layout(P->n_part_slots, P->n_pre_slots, P->desc.num_q_heads, P->desc.head_dim, P->n_stage_pages,
                                 P->desc.num_kv_heads, (int64_t)P->num_seqs * P->max_blocks);
    return launch_attention(P->ctx, &P->desc, n, L, P->dev, P->part, W, q, k_cache,
                            v_cache, block_table, P->max_blocks, out, lse, (cudaStream_t)cuda_stream, false);
}

cf_status cf_mixed_step_host(cf_ctx* c, const cf_cache_desc* desc,
                             const void* q_host, const void* k_new_host, const void* v_new_host,
                             void* k_cache, void* v_cache,
                             const int32_t* block_table, int32_t max_blocks_per_seq,
                             const int32_t* context_len, const int32_t* query_len, int32_t num_seqs,
                             void* out_host, void* cuda_stream)
{
    if (!c || !desc) return CF_ERR_INVALID_ARG;
    cf_status st = validate_desc(desc);
    if (st != CF_OK) return st;
    Plan pl;
    st = validate_lengths(desc, context_len, query_len, num_seqs, max_blocks_per_seq, &pl);
    if (st != CF_OK) return st;
    if (pl.total_q == 0) return CF_OK;
    if (!q_host || !k_new_host || !v_new_host || !out_host) return CF_ERR_INVALID_ARG;
    DeviceGuard guard(c->device);
    if (!guard.ok) return CF_ERR_CUDA;
    cudaStream_t stream = (cudaStream_t)cuda_stream;
    const size_t T = (size_t)pl.total_q;
    const size_t q_bytes = align_up(T * desc->num_q_heads * desc->head_dim * 2, 256);
    const size_t kv_bytes = align_up(T * desc->num_kv_heads * desc->head_dim * 2, 256);
    const size_t need = 2 * q_bytes + 2 * kv_bytes;
    HostStage& hs = c->stage[c->next_stage];
    c->next_stage = (c->next_stage + 1) % kHostStages;
    if (need > hs.bytes) {
        if (cudaDeviceSynchronize() != cudaSuccess) return CF_ERR_CUDA;
        if (hs.dev) cudaFree(hs.dev);
        hs.dev = nullptr;
        hs.bytes = 0;
        if (cudaMalloc((void**)&hs.dev, need) != cudaSuccess) return CF_ERR_CUDA;
        hs.bytes = need;
        hs.used = false;
    }
    uint8_t* dq = hs.dev;
    uint8_t* dk = dq + q_bytes;
    uint8_t* dv = dk + kv_bytes;
    uint8_t* dout = dv + kv_bytes;
    const size_t qb = T * desc->num_q_heads * desc->head_dim * 2, kb = T * desc->num_kv_heads * desc->head_dim * 2;
    // inputs: copy stream, after the kernels and the read-back that last used this staging set
    // (q on one copy stream, k_new and v_new on a second: the small copies run at two thirds of the link rate
    // on their own and fill in beside the large one)
    if (hs.used) {
        if (cudaStreamWaitEvent(c->h2d_stream, hs.compute_done, 0) != cudaSuccess) return CF_ERR_CUDA;
        if (cudaStreamWaitEvent(c->h2d_stream, hs.d2h_done, 0) != cudaSuccess) return CF_ERR_CUDA;
        if (cudaStreamWaitEvent(c->h2d_kv_stream, hs.compute_done, 0) != cudaSuccess) return CF_ERR_CUDA;
    }
    if (cudaMemcpyAsync(dk, k_new_host, kb, cudaMemcpyHostToDevice, c->h2d_kv_stream) != cudaSuccess) return CF_ERR_CUDA;
    if (cudaMemcpyAsync(dv, v_new_host, kb, cudaMemcpyHostToDevice, c->h2d_kv_stream) != cudaSuccess) return CF_ERR_CUDA;
    if (cudaEventRecord(hs.h2d_kv_done, c->h2d_kv_stream) != cudaSuccess) return CF_ERR_CUDA;
    if (cudaMemcpyAsync(dq, q_host, qb, cudaMemcpyHostToDevice, c->h2d_stream) != cudaSuccess) return CF_ERR_CUDA;
    if (cudaEventRecord(hs.h2d_done, c->h2d_stream) != cudaSuccess) return CF_ERR_CUDA;
    // kernels: the caller's stream
    if (cudaStreamWaitEvent(stream, hs.h2d_kv_done, 0) != cudaSuccess) return CF_ERR_CUDA;
    c->plan_copy_stream = c->h2d_stream;
    st = cf_kv_append(c, desc, k_cache, v_cache, dk, dv, block_table, max_blocks_per_seq, context_len, query_len,
                      num_seqs, cuda_stream);
    if (st != CF_OK) {
        c->plan_copy_stream = nullptr;
        return st;
    }
    // A step whose decode part weighs as much as its prefill part is bound by the copies over PCIe, not by the
    // kernels: measured on the chat-like workload the spatial sequence made it slower (0.40 ms against 0.355 ms),
    // so such steps keep the serial sequence.  A prefill-heavy step (the spatial share above its floor) is bound by
    // the kernels and runs the sequence cf_mixed_attention would run.
    if (cudaStreamWaitEvent(stream, hs.h2d_done, 0) != cudaSuccess) {
        c->plan_copy_stream = nullptr;
        return CF_ERR_CUDA;
    }
    c->in_host_step = spatial_front_sms(desc, context_len, query_len, num_seqs, c->num_sms) <= (c->num_sms * 3) / 5;
    st = cf_mixed_attention(c, desc, dq, k_cache, v_cache, block_table, max_blocks_per_seq, context_len, query_len,
                            num_seqs, dout, nullptr, cuda_stream);
    c->in_host_step = false;
    c->plan_copy_stream = nullptr;
    if (st != CF_OK) return st;
    if (cudaEventRecord(hs.compute_done, stream) != cudaSuccess) return CF_ERR_CUDA;
    // result: second copy stream
    if (cudaStreamWaitEvent(c->d2h_stream, hs.compute_done, 0) != cudaSuccess) return CF_ERR_CUDA;
    if (cudaMemcpyAsync(out_host, dout, qb, cudaMemcpyDeviceToHost, c->d2h_stream) != cudaSuccess) return CF_ERR_CUDA;
    if (cudaEventRecord(hs.d2h_done, c->d2h_stream) != cudaSuccess) return CF_ERR_CUDA;
    hs.used = true;
    return CF_OK;
}

cf_status cf_host_steps_flush(cf_ctx* c, void* cuda_stream)
{
    if (!c) return CF_ERR_INVALID_ARG;
    DeviceGuard guard(c->device);
    if (!guard.ok) return CF_ERR_CUDA;
    for (int i = 0; i < kHostStages; ++i)
        if (c->stage[i].used && cudaStreamWaitEvent((cudaStream_t)cuda_stream, c->stage[i].d2h_done, 0) != cudaSuccess)
            return CF_ERR_CUDA;
    return CF_OK;
}

cf_status cf_get_async_status(cf_ctx* c)
{
    if (!c) return CF_ERR_INVALID_ARG;
    DeviceGuard guard(c->device);
    uint32_t w = 0;
    if (cudaMemcpy(&w, c->err_dev, sizeof w, cudaMemcpyDeviceToHost) != cudaSuccess) return CF_ERR_CUDA;
    if (w == 0) return CF_OK;
    if (cudaMemset(c->err_dev, 0, sizeof w) != cudaSuccess || cudaDeviceSynchronize() != cudaSuccess) return CF_ERR_CUDA;
    if (w & kErrTimeout) return CF_ERR_TIMEOUT;
    if (w & kErrBlockId) return CF_ERR_OUT_OF_RANGE;
    return CF_ERR_CUDA;
}

cf_status cf_validate_block_table(cf_ctx* c, const cf_cache_desc* desc, const int32_t* block_table,
                                  int32_t max_blocks_per_seq, const int32_t* context_len, const int32_t* query_len,
                                  int32_t num_seqs, void* cuda_stream, int32_t* num_bad)
{
    if (!c || !desc || !num_bad) return CF_ERR_INVALID_ARG;
    *num_bad = 0;
    cf_status st = validate_desc(desc);
    if (st != CF_OK) return st;
    Plan pl;
    st = validate_lengths(desc, context_len, query_len, num_seqs, max_blocks_per_seq, &pl);
    if (st != CF_OK) return st;
    if (num_seqs == 0) return CF_OK;
    if (!block_table) return CF_ERR_INVALID_ARG;
    DeviceGuard guard(c->device);
    if (!guard.ok) return CF_ERR_CUDA;
    cudaStream_t stream = (cudaStream_t)cuda_stream;
    PlanLayout L;
    uint8_t* base = nullptr;
    PlanSlot* slot = nullptr;
    st = upload_plan(c, num_seqs, context_len, query_len, pl, stream, &L, &base, &slot);
    if (st != CF_OK) return st;
    uint32_t* counter = c->err_dev + 1;      // context-owned scratch word
    bool ok = cudaMemsetAsync(counter, 0, sizeof(uint32_t), stream) == cudaSuccess;
    ok = ok && launch_validate_table(block_table, max_blocks_per_seq, (const int32_t*)(base + L.off_ctx), num_seqs,
                                     desc->num_blocks, counter, stream) == cudaSuccess;
    finish_slot(slot, stream);
    uint32_t host = 0;
    ok = ok && cudaMemcpyAsync(&host, counter, sizeof host, cudaMemcpyDeviceToHost, stream) == cudaSuccess;
    ok = ok && cudaStreamSynchronize(stream) == cudaSuccess;
    if (!ok) return CF_ERR_CUDA;
    *num_bad = (int32_t)host;
    return host ? CF_ERR_OUT_OF_RANGE : CF_OK;
}

cf_status cf_set_overlap(cf_ctx* c, int enabled)
{
    if (!c) return CF_ERR_INVALID_ARG;
    if (enabled < 0) return CF_ERR_INVALID_ARG;
    c->overlap = enabled != 0;
    if (enabled > 1) c->spatial_sms = enabled;
    if (enabled == 1) c->spatial_sms = c->spatial_sms_default;
    return CF_OK;
}

cf_status cf_set_debug_option(cf_ctx* c, cf_debug_option option, int value)
{
    if (!c) return CF_ERR_INVALID_ARG;
    const PlanConfig defaults;
    switch (option) {
        case CF_DEBUG_PREFILL_SPLIT: c->cfg.prefill_force_split = value > 0 ? value : 0; return CF_OK;
        case CF_DEBUG_SEPARATE_COMBINE: c->fused_combine = value <= 0; return CF_OK;
        case CF_DEBUG_DECODE_WAVES: c->cfg.decode_waves = value > 0 ? value : defaults.decode_waves; return CF_OK;
        case CF_DEBUG_DECODE_MIN_CHUNK_PAGES:
            c->cfg.decode_min_chunk_pages = value > 0 ? value : defaults.decode_min_chunk_pages;
            return CF_OK;
        case CF_DEBUG_SPATIAL_NO_WAIT: c->spatial_wait = value <= 0; return CF_OK;
        case CF_DEBUG_PREFILL_PAIRS: c->use_pairs = value > 0; return CF_OK;
    }
    return CF_ERR_INVALID_ARG;
}

cf_status cf_selftest_bounded_wait(cf_ctx* c, void* cuda_stream)
{
    if (!c) return CF_ERR_INVALID_ARG;
    DeviceGuard guard(c->device);
    if (!guard.ok) return CF_ERR_CUDA;
    return launch_wait_selftest(c->err_dev, (cudaStream_t)cuda_stream) == cudaSuccess ? CF_OK : CF_ERR_CUDA;
}

cf_status cf_set_timing(cf_ctx* c, int enabled)
{
    if (!c) return CF_ERR_INVALID_ARG;
    c->timing = enabled != 0;
    c->timed_used = 0;
    return CF_OK;
}

cf_status cf_get_timing_sums(cf_ctx* c, float* ms_decode, float* ms_combine, float* ms_prefill, int32_t* num_calls)
{
    if (!c) return CF_ERR_INVALID_ARG;
    double t[3] = {0., 0., 0.};
    const size_t n = c->timed_used;
    if (n > 0) {
        DeviceGuard guard(c->device);
        if (cudaEventSynchronize(c->timed[n - 1].ev[3]) != cudaSuccess) return CF_ERR_CUDA;
        for (size_t k = 0; k < n; ++k)
            for (int i = 0; i < 3; ++i) {
                float ms = 0.f;
                if (c->timed[k].ran[i] && cudaEventElapsedTime(&ms, c->timed[k].ev[i], c->timed[k].ev[i + 1]) != cudaSuccess)
                    return CF_ERR_CUDA;
                t[i] += ms;
            }
    }
    c->timed_used = 0;
    if (ms_decode) *ms_decode = (float)t[0];
    if (ms_combine) *ms_combine = (float)t[1];
    if (ms_prefill) *ms_prefill = (float)t[2];
    if (num_calls) *num_calls = (int32_t)n;
    return CF_OK;
}

cf_status cf_get_host_time_sums(cf_ctx* c, double* us_append, double* us_attention, double* us_planner, int32_t* num_steps)
{
    if (!c) return CF_ERR_INVALID_ARG;
    if (us_append) *us_append = 1e-3 * (double)c->host_ns_append;
    if (us_attention) *us_attention = 1e-3 * (double)c->host_ns_attention;
    if (us_planner) *us_planner = 1e-3 * (double)c->host_ns_planner;
    if (num_steps) *num_steps = c->host_calls_attention;
    c->host_ns_append = c->host_ns_attention = c->host_ns_planner = 0;
    c->host_calls_append = c->host_calls_attention = 0;
    return CF_OK;
}

cf_status cf_get_last_plan_counts(cf_ctx* c, int32_t* counts)
{
    if (!c || !counts) return CF_ERR_INVALID_ARG;
    for (int i = 0; i < 8; ++i) counts[i] = c->last_counts[i];
    return CF_OK;
}

cf_status cf_get_last_launch_count(cf_ctx* c, int32_t* num_launches)
{
    if (!c || !num_launches) return CF_ERR_INVALID_ARG;
    *num_launches = c->launches;
    return CF_OK;
}

int32_t cf_spatial_share(const cf_cache_desc* desc, const int32_t* context_len, const int32_t* query_len,
                         int32_t num_seqs, int32_t num_sms)
{
    if (validate_desc(desc) != CF_OK || num_seqs < 0 || (num_seqs > 0 && (!context_len || !query_len))) return 0;
    return spatial_front_sms(desc, context_len, query_len, num_seqs, num_sms > 0 ? num_sms : 148);
}

cf_status cf_estimate_us(const cf_cache_desc* desc, const int32_t* context_len, const int32_t* query_len,
                         int32_t num_seqs, int32_t max_blocks_per_seq, int32_t num_sms,
                         float* us_decode, float* us_combine, float* us_prefill)
{
    cf_status st = validate_desc(desc);
    if (st != CF_OK) return st;
    PlanConfig cfg;
    cfg.num_sms = num_sms > 0 ? num_sms : 148;
    Plan pl;
    st = build_plan(desc, context_len, query_len, num_seqs, max_blocks_per_seq, cfg, &pl);
    if (st != CF_OK) return st;
    const Estimate e = estimate_us(desc, context_len, query_len, pl, cfg.num_sms);
    if (us_decode) *us_decode = e.us_decode;
    if (us_combine) *us_combine = e.us_combine;
    if (us_prefill) *us_prefill = e.us_prefill;
    return CF_OK;
}

cf_status cf_plan_inspect(const cf_cache_desc* desc, const int32_t* context_len, const int32_t* query_len,
                          int32_t num_seqs, int32_t max_blocks_per_seq, const cf_plan_options* opts,
                          int32_t* decode_items, int32_t* combine_items, int32_t* prefill_items,
                          int32_t cap, int32_t* counts)
{
    cf_status st = validate_desc(desc);
    if (st != CF_OK) return st;
    PlanConfig cfg;
    if (opts) {
        if (opts->num_sms > 0) cfg.num_sms = opts->num_sms;
        if (opts->prefill_sms_mixed > 0) cfg.prefill_sms_mixed = opts->prefill_sms_mixed;
        if (opts->prefill_force_split > 0) cfg.prefill_force_split = opts->prefill_force_split;
        if (opts->decode_waves > 0) cfg.decode_waves = opts->decode_waves;
        if (opts->decode_min_chunk_pages > 0) cfg.decode_min_chunk_pages = opts->decode_min_chunk_pages;
    }
    cfg.prefill_pair = prefill_pair_supported(desc) && opts && opts->prefill_pairs > 0;
    Plan pl;
    st = build_plan(desc, context_len, query_len, num_seqs, max_blocks_per_seq, cfg, &pl);
    if (st != CF_OK) return st;
    if (cap < 0) cap = 0;
    if (decode_items)
        for (size_t i = 0; i < pl.decode.size() && i < (size_t)cap; ++i) {
            const DecodeItem& d = pl.decode[i];
            int32_t* o = decode_items + 6 * i;
            o[0] = d.seq; o[1] = d.q_row; o[2] = d.kv_begin; o[3] = d.kv_end; o[4] = d.part_slot; o[5] = d.chunk;
        }
    if (combine_items)
        for (size_t i = 0; i < pl.combine.size() && i < (size_t)cap; ++i) {
            int32_t* o = combine_items + 3 * i;
            o[0] = pl.combine[i].q_row; o[1] = pl.combine[i].part_first; o[2] = pl.combine[i].n_chunks;
        }
    size_t n_pre = 0;
    for (const PrefillTcItem& it : pl.prefill_tc)
        for (int t = 0; t < 2; ++t) {
            if (it.n_rows[t] <= 0) continue;
            const int32_t tiles = (it.prefix + it.row0[t] + it.n_rows[t] + 127) / 128;      // KV tiles this q tile can see
            if (prefill_items && n_pre < (size_t)cap) {
                int32_t* o = prefill_items + 8 * n_pre;
                o[0] = it.seq; o[1] = it.q_row0[t]; o[2] = it.row0[t]; o[3] = it.n_rows[t]; o[4] = it.head[t]; o[5] = it.kvh;
                o[6] = it.j_begin < tiles ? it.j_begin : tiles;
                o[7] = it.j_end < tiles ? it.j_end : tiles;
            }
            ++n_pre;
            if (pl.pair) {                               // the second CTA of the pair: the same q tile for head + 2
                if (prefill_items && n_pre < (size_t)cap) {
                    int32_t* o = prefill_items + 8 * n_pre;
                    for (int i = 0; i < 8; ++i) o[i] = o[i - 8];
                    o[4] += 2;
                }
                ++n_pre;
            }
        }
    if (counts) {
        counts[0] = (int32_t)pl.decode.size();
        counts[1] = (int32_t)pl.combine.size();
        counts[2] = (int32_t)n_pre;
        counts[3] = pl.n_part_slots;
        counts[4] = (int32_t)pl.prefill_tc.size();          // prefill CTAs, KV ranges of split items included
        counts[5] = (int32_t)pl.prefill_combine.size();     // KV-split prefill items
    }
    return CF_OK;
}

}  // extern "C"
