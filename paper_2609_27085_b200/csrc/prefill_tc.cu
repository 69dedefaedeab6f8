// Chunked-prefill attention on the 5th-generation tensor cores (tcgen05.mma, accumulators in
// tensor memory), head_dim 128 or 64 (template parameter D; the sizes quoted below are those of D = 128).
//
// A work item = two 128-row q tiles that share a KV head (two query heads of one group over the same
// rows; for G = 1 two consecutive row tiles of one head), so every K/V tile fetched into shared memory
// feeds two S = Q K^T and two O += P V products.  CTAs are persistent (one per SM): CTA b starts on
// item b and then draws items from a ticket counter; the roles run from item to item without a
// CTA-wide barrier.  384 threads, warp-specialised (the first warpgroup hands most of its registers to
// the two softmax warpgroups with setmaxnreg):
//   warp 0      work queue; TMA producer of the Q tiles and of the 128-token K tiles, one 16-token
//               page-half per TMA box, gathered through the block table into a 128B-swizzled ring.
//   warp 2      TMA producer of the V tiles (same box shape, its own ring).
//   warp 1      MMA issuer (one elected lane): S_t = Q_t K^T, O_t += P_t V, in the order
//               PV_0(j) QK_0(j+1) PV_1(j) QK_1(j+1) so that the tensor pipe works on one tile while
//               the other tile's softmax runs.
//   warps 4-7   softmax of tile 0, one thread per q row; warps 8-11 softmax of tile 1.
// Tensor memory (512 columns): S_0 | S_1 | O_0 | O_1, 128 fp32 columns each; P_t (bf16) overwrites
// the first 64 columns of S_t and is consumed by the PV product straight from tensor memory.
// Softmax: scores leave tensor memory once (tcgen05.ld), exp2 with the scale folded in, the
// running maximum is only raised when it grows by more than 2^8 (then O_t is rescaled in tensor
// memory), so almost every tile costs no correction pass.  The causal comparison j <= P + i is
// evaluated only in warps whose rows can see a masked key of the tile; tiles above the diagonal
// are never loaded.
// Every wait is bounded: on expiry the CTA raises an abort flag, every role leaves its loop, the
// error word is set and tensor memory is released.
#include <atomic>
#include <type_traits>

#include "kernels.h"
#include "prefill_common.cuh"

namespace cf {

namespace {

// Per head dimension (128 or 64): a Q, K or V tile is 128 rows x D elements, stored as D / 64 halves of
// [128 rows][64 elements]; the O accumulator of a q tile takes D fp32 columns of tensor memory.
template <int D>
struct Geo {
    static_assert(D == 64 || D == 128, "head_dim 64 or 128");
    static constexpr int HALVES = D / 64;
    static constexpr int TILE_BYTES = HALVES * HALF_BYTES;                 // 32 KB / 16 KB
    static constexpr uint32_t SMEM_Q = 0;
    static constexpr uint32_t SMEM_K = 2 * TILE_BYTES;
    static constexpr uint32_t SMEM_V = SMEM_K + KV_STAGES * TILE_BYTES;
    static constexpr uint32_t SMEM_TOTAL = SMEM_V + KV_STAGES * TILE_BYTES;   // 192 KB / 96 KB
    static constexpr int KS = D / 16;                                      // K = 16 steps of S = Q K^T
};
constexpr uint32_t TM_S = 0, TM_O = 256;   // column offsets: S_t at TM_S + 128 t, O_t at TM_O + D t

struct Bars {
    uint64_t q_full, q_empty;
    uint64_t k_full[KV_STAGES], k_empty[KV_STAGES];
    uint64_t v_full[KV_STAGES], v_empty[KV_STAGES];
    uint64_t s_full[2], p_full[2], o_done[2];
    uint64_t item_full[2];    // the producer has put an item context into slot s
};

}  // namespace

// Persistent CTAs: every CTA of the launch sequence draws work items (longest first) from one ticket
// counter in global memory, p.pre_queue[0], until the tickets run out.  `queue_ctas` is the number of CTAs
// that draw from the counter (over all grids that share it); the last of them to leave puts the two
// counter words back to zero, so that a replay of the same launches needs no host-side reset.
// Ticket t stands for item ticket_base + t; with first_static set, CTA b starts on item b without a draw
// (the grid that is launched first takes items 0 .. gridDim.x - 1 this way, so ticket_base is its size).
// The roles run through the items without a CTA-wide barrier in between: every mbarrier keeps counting
// phases across items (each role carries the running phase of the barriers it uses), the producer is up
// to two K/V tiles and one item context ahead, the issuer puts the first S = Q K^T of the next item
// right behind the last P V of the current one, and a softmax thread goes from the epilogue of one item
// straight to the first tile of the next.
// VARIANT = false is the plain path (full causal attention, no sinks, bf16 cache): its softmax keeps the shorter
// instruction stream - one-sided mask, exact maximum on the item's first tile only - which is worth ~3 % of the
// kernel's time; VARIANT = true adds the sliding window's left edge, sinks and the fp8 cache's per-head scales.
template <int D, bool VARIANT>
__global__ void __launch_bounds__(NTHREADS, 1)
prefill_tc_kernel(const __grid_constant__ CUtensorMap map_q, const __grid_constant__ CUtensorMap map_k,
                  const __grid_constant__ CUtensorMap map_v, const AttnParams p, const int n_items, const int queue_ctas,
                  const int first_static, const int ticket_base, uint32_t* const resident)
{
    constexpr int HALVES = Geo<D>::HALVES, TILE_BYTES = Geo<D>::TILE_BYTES, KS = Geo<D>::KS;
    constexpr uint32_t kPolyMask = D == 64 ? CF_POLY_MASK_D64 : CF_POLY_MASK;
    constexpr uint32_t SMEM_Q = Geo<D>::SMEM_Q, SMEM_K = Geo<D>::SMEM_K, SMEM_V = Geo<D>::SMEM_V;
    extern __shared__ uint8_t smem_raw[];
    __shared__ __align__(16) ItemCtx ctx_s[2];
    __shared__ __align__(8) Bars bars;
    __shared__ uint32_t tmem_base_s;
    __shared__ uint32_t abort_s;
    __shared__ uint32_t issuer_state[4];

    const uint32_t smem = (smem_u32(smem_raw) + 1023u) & ~1023u;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    // the first item of a CTA that starts on a fixed item: fetched now, in use after the set-up below (the plan
    // was uploaded before the kernel that precedes this one in the stream, so it may be read this early)
    const bool has_static = first_static != 0 && (int)blockIdx.x < n_items;
    PrefillTcItem first_it;
    if (warp == 0 && has_static) {
        const uint4* src = reinterpret_cast<const uint4*>(p.pre_tc_items + blockIdx.x);
        uint4* dst = reinterpret_cast<uint4*>(&first_it);
#pragma unroll
        for (int i = 0; i < (int)(sizeof(PrefillTcItem) / 16); ++i) dst[i] = __ldg(src + i);
    }
    // lets the next grid of the stream become resident while this grid drains (it waits for this grid's
    // completion before it reads anything this grid wrote)
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    volatile uint32_t* abort_flag = &abort_s;

    if (threadIdx.x == 0) {
        abort_s = (p.err != nullptr && (*reinterpret_cast<volatile uint32_t*>(p.err) & kErrTimeout) != 0u) ? 2u : 0u;   // an earlier CTA gave up
        // spatial launch sequence: the stream that carries the decode kernel waits (a
        // stream memory operation, not a kernel) until every CTA of this grid holds its SM
        if (resident != nullptr) atomicAdd(resident, 1u);
        mbar_init(smem_u32(&bars.q_full), 1);
        mbar_init(smem_u32(&bars.q_empty), 1);
        for (int s = 0; s < KV_STAGES; ++s) {
            mbar_init(smem_u32(&bars.k_full[s]), 1);
            mbar_init(smem_u32(&bars.k_empty[s]), 1);
            mbar_init(smem_u32(&bars.v_full[s]), 1);
            mbar_init(smem_u32(&bars.v_empty[s]), 1);
        }
        for (int t = 0; t < 2; ++t) {
            mbar_init(smem_u32(&bars.s_full[t]), 1);
            mbar_init(smem_u32(&bars.p_full[t]), 4);      // one arrival per softmax warp
            mbar_init(smem_u32(&bars.o_done[t]), 1);
            mbar_init(smem_u32(&bars.item_full[t]), 1);
        }
        fence_mbar_init();
    }
    if (warp == 0) tmem_alloc<512>(smem_u32(&tmem_base_s));
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = tmem_base_s;
    // Launched with programmatic stream serialisation: everything above overlaps the tail of the kernel
    // before this one in the stream; from here on that kernel has completed and its writes are visible
    // (the K/V rows of cf_kv_append when the batch has no decode part).
    asm volatile("griddepcontrol.wait;" ::: "memory");

    // A block id outside the pool is not used as a TMA coordinate: page 0 is fetched in its place and the error
    // word is set (the rows of that sequence are then meaningless, but nothing is read outside the pool).
    auto checked_pid = [&](int32_t id) -> int32_t {
        if ((uint32_t)id < (uint32_t)p.num_blocks) return id;
        if (p.err) atomicOr(p.err, kErrBlockId);
        return 0;
    };
    // the context of a role's k-th item (slot k & 1, filled for the (k >> 1)-th time); null on an abort.
    // A role copies the fields it needs at once: the slot is rewritten two items later.
    auto wait_item = [&](int k) -> const ItemCtx* {
        if (!mbar_wait(smem_u32(&bars.item_full[k & 1]), (uint32_t)(k >> 1) & 1u, abort_flag)) return nullptr;
        return &ctx_s[k & 1];
    };

    if (warp < 4) {
      reg_dec<REGS_ROLE>();
      if (warp == 3) {
        // spare warp of the first warpgroup
      } else if (warp == 2) {
        // =========================================================== TMA producer of the V tiles
        // (a warp issues the 16 boxes of a tile one after the other; K and V from one warp would make the
        // producer as slow as the tensor pipe)
        uint32_t ub[2] = {0u, 0u};
        bool ok = true;
        for (int k = 0; ok; ++k) {
            const ItemCtx* cs = wait_item(k);
            if (cs == nullptr || cs->live == 0) break;
            const int n_max = cs->n_max, total_pages = cs->total_pages, jb = cs->it.j_begin, kvh = cs->it.kvh;
            const int page_lo = cs->it.page_lo;          // sliding window: pages below it are not fetched (their table entries may be stale)
            const int32_t* bt = p.block_table + (int64_t)cs->it.seq * p.max_blocks;
            int32_t pid = (lane < min(8, total_pages - 8 * jb) && 8 * jb + lane >= page_lo) ? checked_pid(__ldg(bt + 8 * jb + lane)) : 0;
            for (int j = 0; j < n_max && ok; ++j) {
                const int stage = j & 1;
                const uint32_t use = ub[stage] + (uint32_t)(j >> 1);
                const int np = min(8, total_pages - 8 * (jb + j));
                const int p0 = max(0, page_lo - 8 * (jb + j));            // first page of the tile that is fetched
                const int32_t my_pid = __shfl_sync(0xffffffffu, pid, lane / HALVES);
                if (j + 1 < n_max) pid = lane < min(8, total_pages - 8 * (jb + j + 1)) ? checked_pid(__ldg(bt + 8 * (jb + j + 1) + lane)) : 0;
                const uint32_t dst_off = (lane % HALVES) * HALF_BYTES + (lane / HALVES) * 2048;
                if (use > 0) ok = __all_sync(0xffffffffu, mbar_wait(smem_u32(&bars.v_empty[stage]), (use - 1) & 1u, abort_flag));
                if (!ok) break;
                if (lane == 0) mbar_arrive_expect_tx(smem_u32(&bars.v_full[stage]), (np - p0) * 16 * D * 2);
                __syncwarp();
                if (lane < HALVES * np && lane >= HALVES * p0)
                    tma_load_4d(smem + SMEM_V + stage * TILE_BYTES + dst_off, &map_v, (lane % HALVES) * 64, 0, kvh, my_pid,
                                smem_u32(&bars.v_full[stage]));
            }
            ok = __all_sync(0xffffffffu, ok);
            ub[0] += (uint32_t)(n_max + 1) >> 1;
            ub[1] += (uint32_t)n_max >> 1;
        }
      } else if (warp == 0) {
        // =========================================================== TMA producer of Q and the K tiles, keeper of the work queue
        if (lane == 0) {
            prefetch_tensormap(&map_q);
            prefetch_tensormap(&map_k);
            prefetch_tensormap(&map_v);
        }
        bool counted_out = false;
        // draws the next ticket; on the first empty draw the CTA is counted out and the last CTA resets the counters
        auto draw = [&](ItemCtx& cx) {
            int idx = n_items;
            if (lane == 0 && *abort_flag == 0u && !counted_out) idx = ticket_base + (int)atomicAdd(p.pre_queue, 1u);
            idx = __shfl_sync(0xffffffffu, idx, 0);
            if (idx < n_items) {
                const uint4* src = reinterpret_cast<const uint4*>(p.pre_tc_items + idx);
                uint4* dst = reinterpret_cast<uint4*>(&cx.it);
#pragma unroll
                for (int i = 0; i < (int)(sizeof(PrefillTcItem) / 16); ++i) dst[i] = __ldg(src + i);
                derive_item(cx);
            } else {
                cx.live = 0;
                if (!counted_out && lane == 0 && atomicAdd(p.pre_queue + 1, 1u) == (uint32_t)(queue_ctas - 1)) {
                    p.pre_queue[0] = 0u;      // every other CTA has made its last draw
                    p.pre_queue[1] = 0u;
                    __threadfence();
                }
                counted_out = true;
            }
        };
        ItemCtx cx, nx;
        if (has_static && *abort_flag == 0u) {
            cx.it = first_it;
            derive_item(cx);
        } else {
            draw(cx);
        }
        uint32_t ub[2] = {0u, 0u};              // how often each K/V ring stage has been filled before this item
        bool ok = true;
        for (int k = 0; ok; ++k) {
            // Q tiles and the context slot are free once every S = Q K^T of the previous item has completed
            if (k > 0) ok = __all_sync(0xffffffffu, mbar_wait(smem_u32(&bars.q_empty), (uint32_t)(k - 1) & 1u, abort_flag));
            if (!ok) break;
            if (lane == 0) {
                const uint4* src = reinterpret_cast<const uint4*>(&cx);
                uint4* dst = reinterpret_cast<uint4*>(&ctx_s[k & 1]);
#pragma unroll
                for (int i = 0; i < (int)(sizeof(ItemCtx) / 16); ++i) dst[i] = src[i];
                mbar_arrive(smem_u32(&bars.item_full[k & 1]));
            }
            if (!cx.live) break;
            const PrefillTcItem& it = cx.it;
            if (lane == 0) {
                const int nq = (it.n_rows[0] > 0) + (it.n_rows[1] > 0);
                mbar_arrive_expect_tx(smem_u32(&bars.q_full), nq * TILE_BYTES);
                for (int t = 0; t < 2; ++t)
                    if (it.n_rows[t] > 0)
                        for (int h = 0; h < HALVES; ++h)
                            tma_load_3d(smem + SMEM_Q + t * TILE_BYTES + h * HALF_BYTES, &map_q, h * 64, it.head[t],
                                        it.q_row0[t], smem_u32(&bars.q_full));
            }
            const int32_t* bt = p.block_table + (int64_t)it.seq * p.max_blocks;
            const int n_max = cx.n_max, total_pages = cx.total_pages, jb = it.j_begin, page_lo = it.page_lo;
            const int j_draw = min(2, n_max - 1);       // the next ticket is drawn once the first tiles are on their way
            bool drawn = false;
            // page ids of a tile are fetched while the tile before it is being issued (never those of pages left of a
            // sliding window: page_lo lies in the item's first tile)
            int32_t pid = (lane < min(8, total_pages - 8 * jb) && 8 * jb + lane >= page_lo) ? checked_pid(__ldg(bt + 8 * jb + lane)) : 0;
            for (int j = 0; j < n_max && ok; ++j) {
                const int stage = j & 1;
                const uint32_t use = ub[stage] + (uint32_t)(j >> 1);
                const int np = min(8, total_pages - 8 * (jb + j));
                const int p0 = max(0, page_lo - 8 * (jb + j));
                const int32_t my_pid = __shfl_sync(0xffffffffu, pid, lane / HALVES);
                if (j + 1 < n_max) pid = lane < min(8, total_pages - 8 * (jb + j + 1)) ? checked_pid(__ldg(bt + 8 * (jb + j + 1) + lane)) : 0;
                const uint32_t dst_off = (lane % HALVES) * HALF_BYTES + (lane / HALVES) * 2048;
                if (use > 0) ok = __all_sync(0xffffffffu, mbar_wait(smem_u32(&bars.k_empty[stage]), (use - 1) & 1u, abort_flag));
                if (!ok) break;
                if (lane == 0) mbar_arrive_expect_tx(smem_u32(&bars.k_full[stage]), (np - p0) * 16 * D * 2);
                __syncwarp();
                if (lane < HALVES * np && lane >= HALVES * p0)
                    tma_load_4d(smem + SMEM_K + stage * TILE_BYTES + dst_off, &map_k, (lane % HALVES) * 64, 0, it.kvh, my_pid,
                                smem_u32(&bars.k_full[stage]));
                if (j == j_draw) {
                    draw(nx);
                    drawn = true;
                }
            }
            ok = __all_sync(0xffffffffu, ok);
            if (ok && !drawn) draw(nx);
            ub[0] += (uint32_t)(n_max + 1) >> 1;
            ub[1] += (uint32_t)n_max >> 1;
            cx = nx;
        }
        if (!counted_out) draw(nx);               // left on an abort (the flag is up, so no ticket is taken): still count this CTA out
      } else {
        // =========================================================== MMA issuer
        constexpr uint32_t IDESC_QK = idesc_bf16(128, 128, false);
        constexpr uint32_t IDESC_PV = idesc_bf16(128, D, true);
        constexpr uint64_t HI64 = (uint64_t)desc_hi_sw128(1024) << 32;
        // The issuing lane shares its scheduler with two softmax warps and gets roughly one issue
        // slot in ten, while a 128x128x16 MMA lasts only 64 cycles.  Every shared-memory descriptor
        // (q tile x k-step, K/V stage x k-step) is therefore built once and kept in registers, and the
        // tile / stage indices are compile-time, so that a batch is MMAs back to back.
        uint64_t qd[2][KS], kd[KV_STAGES][KS], vd[KV_STAGES][8];
#pragma unroll
        for (int i = 0; i < 2; ++i) {
#pragma unroll
            for (int ks = 0; ks < KS; ++ks) {
                const uint32_t off = (uint32_t)(((ks >> 2) * HALF_BYTES + (ks & 3) * 32) >> 4);
                qd[i][ks] = HI64 | (desc_lo_sw128(smem + SMEM_Q + i * TILE_BYTES, 16) + off);
                kd[i][ks] = HI64 | (desc_lo_sw128(smem + SMEM_K + i * TILE_BYTES, 16) + off);
            }
#pragma unroll
            for (int ks = 0; ks < 8; ++ks)
                vd[i][ks] = HI64 | (desc_lo_sw128(smem + SMEM_V + i * TILE_BYTES, HALF_BYTES) + ks * (2048 >> 4));
        }
        const uint32_t bar_s[2] = {smem_u32(&bars.s_full[0]), smem_u32(&bars.s_full[1])};
        const uint32_t bar_o[2] = {smem_u32(&bars.o_done[0]), smem_u32(&bars.o_done[1])};
        const uint32_t bar_p[2] = {smem_u32(&bars.p_full[0]), smem_u32(&bars.p_full[1])};
        auto issue_qk = [&](auto T, auto S) {             // S_t = Q_t K^T over the head dimension (D / 16 steps of K = 16)
            constexpr int t = decltype(T)::value, st = decltype(S)::value;
            const uint32_t dS = tmem + TM_S + t * 128;
            umma_ss(dS, qd[t][0], kd[st][0], IDESC_QK, 0u);
#pragma unroll
            for (int ks = 1; ks < KS; ++ks) umma_ss(dS, qd[t][ks], kd[st][ks], IDESC_QK, 1u);
            umma_commit(bar_s[t]);
        };
        // O_t (+)= P_t V, one K = 16 step per fetched page: pages [ks0, n_steps) of the tile (ks0 > 0 only in the first
        // tile of a sliding window, n_steps < 8 only in a sequence's last tile)
        auto issue_pv = [&](auto T, auto S, int ks0, int n_steps, uint32_t acc0) {
            constexpr int t = decltype(T)::value, st = decltype(S)::value;
            const uint32_t dO = tmem + TM_O + t * D, aP = tmem + TM_S + t * 128;
            if (ks0 == 0 && n_steps == 8) {
                umma_ts(dO, aP, vd[st][0], IDESC_PV, acc0);
#pragma unroll
                for (int ks = 1; ks < 8; ++ks) umma_ts(dO, aP + ks * 8, vd[st][ks], IDESC_PV, 1u);
            } else {
#pragma unroll
                for (int ks = 0; ks < 8; ++ks)
                    if (ks >= ks0 && ks < n_steps) umma_ts(dO, aP + ks * 8, vd[st][ks], IDESC_PV, ks == ks0 ? acc0 : 1u);
            }
            umma_commit(bar_o[t]);
        };
        using I0 = std::integral_constant<int, 0>;
        using I1 = std::integral_constant<int, 1>;
        // One lane runs the whole role (the others go straight to the teardown barrier).  This lane is
        // the critical resource of the kernel: it is a single dependent instruction stream that is also
        // blocked while its MMAs queue up, so the work between two batches is kept to a handful of
        // instructions, with a lean loop for interior tiles and the general step for the rest.
        if (lane == 0) {
        const uint32_t bar_kf[2] = {smem_u32(&bars.k_full[0]), smem_u32(&bars.k_full[1])};
        const uint32_t bar_vf[2] = {smem_u32(&bars.v_full[0]), smem_u32(&bars.v_full[1])};
        const uint32_t bar_ke[2] = {smem_u32(&bars.k_empty[0]), smem_u32(&bars.k_empty[1])};
        const uint32_t bar_ve[2] = {smem_u32(&bars.v_empty[0]), smem_u32(&bars.v_empty[1])};
        const uint32_t bar_qe = smem_u32(&bars.q_empty);
        // Running phases: ub[s] = fills of K/V ring stage s before this item (tile j of an item sits in
        // stage j & 1 and is that stage's fill number ub[j & 1] + (j >> 1)); sb[t] = tiles of q tile t
        // before this item (s_full / p_full / o_done complete one phase per tile).
        // Only this lane touches issuer_state (= ub[0], ub[1], sb[0], sb[1]).  The lane has no registers to
        // spare beside its 48 descriptors, so the running phases live in shared memory, the item's fields are
        // read from the context slot where they are needed (the slot is not rewritten before this lane has
        // left the next item's last S = Q K^T behind), and only the interior loop keeps its parities in registers.
        volatile uint32_t* const ist = issuer_state;
        ist[0] = ist[1] = ist[2] = ist[3] = 0u;
        bool ok = true;
        for (int k = 0; ok; ++k) {
        const ItemCtx* cs = wait_item(k);
        if (cs == nullptr || cs->live == 0) break;
        const volatile ItemCtx* const vs = cs;
        const int n_max = cs->n_max;
        const int n_j[2] = {cs->n_j[0], cs->n_j[1]};
        ok = mbar_wait(smem_u32(&bars.q_full), (uint32_t)k & 1u, abort_flag);
        ok = ok && mbar_wait(bar_kf[0], ist[0] & 1u, abort_flag);
        if (!ok) break;
        tc_fence_after();
        if (n_j[0] > 0) issue_qk(I0{}, I0{});
        if (n_j[1] > 0) issue_qk(I1{}, I0{});
        umma_commit(bar_ke[0]);
        // q_empty: arrives when every S = Q K^T of the item has completed (the last one is issued in step n_max - 2)
        if (n_max <= 1) umma_commit(bar_qe);
        // ---- interior tiles: both q tiles present and continuing, all 8 pages loaded, not the last tile
        const int n_int = (n_j[0] > 0 && n_j[1] > 0) ? min(n_j[0], n_j[1]) - 1 : 0;
        auto lean_step = [&](auto S, uint32_t par_v, uint32_t par_k1, uint32_t par_p0, uint32_t par_p1, uint32_t acc0) -> bool {
            constexpr int st = decltype(S)::value, st1 = st ^ 1;
            using S1 = std::integral_constant<int, st1>;
            if (!mbar_wait(bar_vf[st], par_v, abort_flag)) return false;
            if (!mbar_wait(bar_kf[st1], par_k1, abort_flag)) return false;
            if (!mbar_wait(bar_p[0], par_p0, abort_flag)) return false;
            tc_fence_after();
            issue_pv(I0{}, S, 0, 8, acc0);
            issue_qk(I0{}, S1{});
            if (!mbar_wait(bar_p[1], par_p1, abort_flag)) return false;
            tc_fence_after();
            issue_pv(I1{}, S, 0, 8, acc0);
            issue_qk(I1{}, S1{});
            umma_commit(bar_ve[st]);
            umma_commit(bar_ke[st1]);
            return true;
        };
        // ---- general step: PV_0(j) QK_0(j+1) PV_1(j) QK_1(j+1) with every edge case
        auto kv_step = [&](auto S, int j) -> bool {
            constexpr int st = decltype(S)::value, st1 = st ^ 1;
            using S1 = std::integral_constant<int, st1>;
            const int jb = vs->it.j_begin, Lc = vs->it.ctx_len;
            const int np = min(8, vs->total_pages - 8 * (jb + j));
            const int ks0 = max(0, vs->it.page_lo - 8 * (jb + j));      // sliding window: the tile's first fetched page
            if (!mbar_wait(bar_vf[st], (ist[st] + (uint32_t)(j >> 1)) & 1u, abort_flag)) return false;
            if (j == n_max - 1 && Lc < (8 * (jb + j) + np) * 16) {
                // slack slots of the sequence's last page came in with the page: zero those V rows so
                // that a zero probability never multiplies a NaN
                const int r0 = Lc - (jb + j) * KT, r1 = np * 16;
                for (int idx = 0; idx < (r1 - r0) * (D / 8); ++idx) {
                    const int r = r0 + idx / (D / 8), c = idx % (D / 8);
                    uint8_t* dst = smem_raw + ((smem + SMEM_V + st * TILE_BYTES) - smem_u32(smem_raw)) +
                                   (c >> 3) * HALF_BYTES + r * 128 + (c & 7) * 16;
                    *reinterpret_cast<uint4*>(dst) = make_uint4(0u, 0u, 0u, 0u);
                }
                fence_proxy_async();
            }
            const uint32_t acc0 = j > 0 ? 1u : 0u;
            auto tile = [&](auto T) -> bool {
                constexpr int t = decltype(T)::value;
                if (j >= n_j[t]) return true;
                const bool more = j + 1 < n_j[t];
                if (more && !mbar_wait(bar_kf[st1], (ist[st1] + (uint32_t)((j + 1) >> 1)) & 1u, abort_flag)) return false;
                if (!mbar_wait(bar_p[t], (ist[2 + t] + (uint32_t)j) & 1u, abort_flag)) return false;
                tc_fence_after();
                issue_pv(T, S, ks0, np, acc0);
                if (more) issue_qk(T, S1{});
                return true;
            };
            if (!tile(I0{})) return false;
            if (!tile(I1{})) return false;
            umma_commit(bar_ve[st]);
            if (j + 1 < n_max) umma_commit(bar_ke[st1]);
            if (j + 1 == n_max - 1) umma_commit(bar_qe);
            return true;
        };
        int j = 0;
        // Sliding window: the item's first tile may start with pages that are not fetched; it (and the tile after it,
        // so that the pair loop below starts on an even tile) take the general step.
        const bool partial_first = vs->it.page_lo > 8 * vs->it.j_begin;
        if (partial_first) {
            for (; j < min(2, n_max) && ok; ++j) ok = (j & 1) ? kv_step(I1{}, j) : kv_step(I0{}, j);
        }
        const int j_pairs = j;                       // where the pair loop starts: 0 or 2
        if (ok) {
            // parities of the even tile j of a pair: stage 0 fill ub[0] + j/2 (V now), stage 1 fill ub[1] + j/2
            // (K of tile j + 1), softmax phases sb[t] + j; the odd tile j + 1 flips all but the stage-0 K
            // fill of tile j + 2, which is ub[0] + j/2 + 1
            uint32_t h0 = (ist[0] + (uint32_t)(j >> 1)) & 1u, h1 = (ist[1] + (uint32_t)(j >> 1)) & 1u;
            const uint32_t p0 = ist[2] & 1u, p1 = ist[3] & 1u;
            for (; ok && j + 1 < n_int; j += 2, h0 ^= 1u, h1 ^= 1u) {
                ok = lean_step(I0{}, h0, h1, p0, p1, j > 0 ? 1u : 0u);
                if (ok) ok = lean_step(I1{}, h1, h0 ^ 1u, p0 ^ 1u, p1 ^ 1u, 1u);
            }
            if (ok && j > j_pairs && j >= n_max - 1) umma_commit(bar_qe);     // the pair loop issued the item's last S = Q K^T
        }
        static_assert(KV_STAGES == 2, "the stage index is the parity of the tile index");
        for (; j < n_max && ok; ++j) {
            ok = (j & 1) ? kv_step(I1{}, j) : kv_step(I0{}, j);
        }
        ist[0] += (uint32_t)(n_max + 1) >> 1;
        ist[1] += (uint32_t)n_max >> 1;
        ist[2] += (uint32_t)n_j[0];
        ist[3] += (uint32_t)n_j[1];
        }
        }
      }
    } else {
      reg_inc<REGS_SOFTMAX>();
      // =========================================================== softmax + epilogue, one thread per q row
      const int t = (warp - 4) >> 2;
      const int row = (warp & 3) * 32 + lane;
      const uint32_t lanes = lane_field(warp);
      const uint32_t tS = tmem + TM_S + t * 128 + lanes, tO = tmem + TM_O + t * D + lanes;
      uint32_t sbt = 0u;                       // tiles of this q tile in earlier items: running phase of s_full / p_full / o_done
      bool ok = true;
      for (int k = 0; ok; ++k) {
        const ItemCtx* cs = wait_item(k);
        if (cs == nullptr || cs->live == 0) break;
        {
        // this q tile's fields of the item
        const int jb = cs->it.j_begin, n_jt = cs->n_j[t], kv_hi = cs->kv_hi_t[t];
        const int it_row0 = cs->it.row0[t], it_n_rows = cs->it.n_rows[t], it_q_row0 = cs->it.q_row0[t], it_head = cs->it.head[t];
        const int it_part_slot = cs->it.part_slot[t], it_part_k = cs->it.part_k, it_part_c = cs->it.part_c;
        // fp8 cache: the staged K/V hold the codes; their per-head scales join the softmax scale and the output here
        const float sc = (VARIANT && p.k_scale != nullptr) ? p.scale_log2 * __ldg(p.k_scale + cs->it.kvh) : p.scale_log2;
        const float v_scale = (VARIANT && p.v_scale != nullptr) ? __ldg(p.v_scale + cs->it.kvh) : 1.f;
        const int limit = min(cs->it.prefix + it_row0 + row, kv_hi - 1);   // last visible key of this row
        const int first_key = (VARIANT && p.window > 0) ? limit - p.window + 1 : -(1 << 30);   // first visible key (sliding window)
        const uint32_t span = (uint32_t)(limit - first_key);
        float m_used = -INFINITY, l_sum = 0.f;     // -inf: the row has not met a visible key yet
        for (int j = 0; j < n_jt; ++j) {
            ok = mbar_wait(smem_u32(&bars.s_full[t]), (sbt + (uint32_t)j) & 1u, abort_flag);
            if (!ok) break;
            tc_fence_after();
            float sv[128];
#pragma unroll
            for (int c = 0; c < 4; ++c) tmem_ld32(tS + c * 32, reinterpret_cast<uint32_t*>(&sv[c * 32]));
            tmem_wait_ld();
            const int col_limit = limit - (jb + j) * KT;     // columns [col_first, col_limit] are visible
            const int col_first = first_key - (jb + j) * KT;
            if (VARIANT) {
                if (__any_sync(0xffffffffu, col_limit < KT - 1 || col_first > 0)) {
#pragma unroll
                    for (int c = 0; c < 128; ++c) sv[c] = ((uint32_t)(c - col_first) <= span) ? sv[c] : -INFINITY;
                }
            } else if (__any_sync(0xffffffffu, col_limit < KT - 1)) {
#pragma unroll
                for (int c = 0; c < 128; ++c) sv[c] = (c <= col_limit) ? sv[c] : -INFINITY;
            }
            if (VARIANT ? __any_sync(0xffffffffu, m_used == -INFINITY) : (j == 0)) {
                // A row's first tile with a visible key: the exact row maximum becomes its reference.  Without a
                // sliding window that is the item's first tile for every row (key 0 of a whole item; the planner
                // never starts a KV range inside the diagonal band); with one, a row of the tile's lower part may
                // meet its first key one tile later and keeps -inf (all its probabilities are zero) until then.
                float mx4[4] = {sv[0], sv[1], sv[2], sv[3]};
#pragma unroll
                for (int c = 4; c < 128; c += 8) {
                    mx4[0] = max3(mx4[0], sv[c], sv[c + 1]);
                    mx4[1] = max3(mx4[1], sv[c + 2], sv[c + 3]);
                    if (c + 4 < 128) {
                        mx4[2] = max3(mx4[2], sv[c + 4], sv[c + 5]);
                        mx4[3] = max3(mx4[3], sv[c + 6], sv[c + 7]);
                    }
                }
                if (!VARIANT || m_used == -INFINITY) m_used = fmaxf(fmaxf(mx4[0], mx4[1]), fmaxf(mx4[2], mx4[3])) * sc;
            }
            // Optimistic pass: exponentials against the current reference maximum, packed two per
            // FMA-pipe instruction.  Whether the reference has to be raised is read off the tile's row
            // sum (a probability above 2^8 makes it exceed 2^15 long before anything can overflow); only
            // then is the exact maximum taken, O_t rescaled in tensor memory and the pass repeated.
            float2 acc2[4];
            auto exp_pass = [&](const float neg_m) {
                const float2 sc2 = make_float2(sc, sc), nm2 = make_float2(neg_m, neg_m);
#pragma unroll
                for (int i = 0; i < 4; ++i) acc2[i] = make_float2(0.f, 0.f);
#pragma unroll
                for (int c = 0; c < 4; ++c) {
                    uint32_t pk[16];
#pragma unroll
                    for (int i = 0; i < 16; ++i) {
                        const float2 x = fma2(make_float2(sv[c * 32 + 2 * i], sv[c * 32 + 2 * i + 1]), sc2, nm2);
                        const float2 pr = ((kPolyMask >> i) & 1u) ? exp2_poly2(x) : make_float2(fast_exp2(x.x), fast_exp2(x.y));
                        acc2[i & 3] = add2(acc2[i & 3], pr);
                        pk[i] = pack_bf16(pr.x, pr.y);
                    }
                    tmem_st16(tS + c * 16, pk);
                }
                const float2 a01 = add2(acc2[0], acc2[1]), a23 = add2(acc2[2], acc2[3]);
                return (a01.x + a01.y) + (a23.x + a23.y);
            };
            float tile_sum = exp_pass((VARIANT && m_used == -INFINITY) ? 0.f : -m_used);
            if (__any_sync(0xffffffffu, !(tile_sum <= 32768.f))) {
                float mx4[4] = {sv[0], sv[1], sv[2], sv[3]};
#pragma unroll
                for (int c = 4; c < 128; c += 4) {
                    mx4[0] = fmaxf(mx4[0], sv[c]);
                    mx4[1] = fmaxf(mx4[1], sv[c + 1]);
                    mx4[2] = fmaxf(mx4[2], sv[c + 2]);
                    mx4[3] = fmaxf(mx4[3], sv[c + 3]);
                }
                const float rise = fmaxf(fmaxf(mx4[0], mx4[1]), fmaxf(mx4[2], mx4[3])) * sc - m_used;
                const float d = fmaxf(rise, 0.f);            // rows that did not rise keep their reference (a row without
                                                             // a visible key so far: -inf - -inf is NaN, which fmaxf drops)
                const float f = fast_exp2(-d);
                m_used += d;
                l_sum *= f;
                if (j > 0) {
                    ok = mbar_wait(smem_u32(&bars.o_done[t]), (sbt + (uint32_t)(j - 1)) & 1u, abort_flag);
                    if (!ok) break;
                    tc_fence_after();
#pragma unroll 1
                    for (int c = 0; c < D / 16; ++c) {
                        float ov[16];
                        tmem_ld16(tO + c * 16, reinterpret_cast<uint32_t*>(ov));
                        tmem_wait_ld();
#pragma unroll
                        for (int i = 0; i < 16; ++i) ov[i] *= f;
                        tmem_st16(tO + c * 16, reinterpret_cast<const uint32_t*>(ov));
                    }
                }
                tmem_wait_st();
                tile_sum = exp_pass((VARIANT && m_used == -INFINITY) ? 0.f : -m_used);
            }
            l_sum += tile_sum;
            tmem_wait_st();
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(smem_u32(&bars.p_full[t]));
        }
        if (ok && n_jt > 0) ok = mbar_wait(smem_u32(&bars.o_done[t]), (sbt + (uint32_t)(n_jt - 1)) & 1u, abort_flag);
        if (ok && n_jt > 0) {
            tc_fence_after();
            const bool live = row < it_n_rows;
            const bool partial = it_part_slot >= 0;
            // a whole item joins the head's sink logit here; a KV range leaves it to the combine pass
            float m_fin = m_used, l_fin = l_sum, shrink = 1.f;
            if (VARIANT && !partial && p.sinks != nullptr) shrink = join_sink(__ldg(p.sinks + it_head) * kLog2e, m_fin, l_fin);
            const float inv = shrink * v_scale / l_fin;
            __nv_bfloat16* orow = p.out + ((int64_t)(it_q_row0 + row) * p.Hq + it_head) * D;
            // KV-split item: un-normalised fp32 row plus (reference maximum, sum) for the combine pass
            const int64_t pslot = (int64_t)it_part_slot + (int64_t)row * it_part_k + it_part_c;
            float* prow = p.pre_part_o + pslot * D;
#pragma unroll
            for (int c = 0; c < D / 32; ++c) {
                float ov[32];
                tmem_ld32(tO + c * 32, reinterpret_cast<uint32_t*>(ov));
                tmem_wait_ld();
                // a thread owns a row, so a warp's store touches 32 rows: 32-byte stores halve the number of
                // memory transactions of the 16-byte ones
                if (live && partial) {
#pragma unroll
                    for (int i = 0; i < 4; ++i) st_global_256(prow + c * 32 + i * 8, reinterpret_cast<const uint32_t*>(ov + 8 * i));
                } else if (live) {
#pragma unroll
                    for (int i = 0; i < 2; ++i) {
                        uint32_t w[8];
#pragma unroll
                        for (int e = 0; e < 8; ++e) w[e] = pack_bf16(ov[16 * i + 2 * e] * inv, ov[16 * i + 2 * e + 1] * inv);
                        st_global_256(orow + c * 32 + i * 16, w);
                    }
                }
            }
            if (live && partial) *reinterpret_cast<float2*>(p.pre_part_ml + pslot * 2) = make_float2(m_used, l_sum);
            else if (live && p.lse) p.lse[(int64_t)(it_q_row0 + row) * p.Hq + it_head] = (m_fin + log2f(l_fin)) * kLn2;
            // O_t has been read out: the p_full arrival of the next item's first tile, later in this thread's
            // program order, is what allows the issuer to overwrite it
            tc_fence_before();
        }
        sbt += (uint32_t)n_jt;
        }
      }
    }

    // ---- teardown: every role has left its loop (the tickets ran out, or the abort flag went up)
    tc_fence_before();
    __syncthreads();
    if (abort_s == 1u) {
        if (threadIdx.x == 0 && p.err) atomicOr(p.err, kErrTimeout);
        // let copies and MMAs that may still be in flight settle before tensor memory is handed back
        for (int i = 0; i < 64; ++i) __nanosleep(2000);
        __syncthreads();
    }
    if (warp == 0) tmem_dealloc<512>(tmem);
}

// ---------------------------------------------------------------------------------------------
// Merges the partials of KV-split prefill items: for every row of the item's q tiles,
//   M = max_c m_c ; O = sum_c 2^(m_c - M) o_c / sum_c 2^(m_c - M) l_c ; lse = (M + log2 sum) ln 2
// in fixed range order.  One warp per row (8 rows per CTA, 32 CTAs per split item), one float4 of the
// row per lane (D / 4 lanes take part); the partials of a row are fetched with independent loads (part_k <= 8).
constexpr int kMaxSplit = 8;
template <int D>
__global__ void __launch_bounds__(256) prefill_combine_kernel(const AttnParams p)
{
    const PrefillCombineItem it = p.pre_comb_items[blockIdx.x >> 5];
    asm volatile("griddepcontrol.wait;" ::: "memory");     // the prefill grid has completed and its partials are visible
    const int lane = threadIdx.x & 31;
    const int rb = blockIdx.x & 31;                  // 32 blocks of 8 rows = 2 tiles x 128 rows
    const int t = rb >> 4, r = (rb & 15) * 8 + (threadIdx.x >> 5);
    if (r >= it.n_rows[t]) return;
    const int k = it.part_k;
    const int64_t s0 = (int64_t)it.part_slot[t] + (int64_t)r * k;
    const bool holds = lane < D / 4;                 // head_dim 64: half of the lanes hold a float4 of the row
    float2 ml[kMaxSplit];
    float4 v[kMaxSplit];
#pragma unroll
    for (int c = 0; c < kMaxSplit; ++c)
        if (c < k) {
            ml[c] = __ldg(reinterpret_cast<const float2*>(p.pre_part_ml + (s0 + c) * 2));
            v[c] = holds ? __ldg(reinterpret_cast<const float4*>(p.pre_part_o + (s0 + c) * D + lane * 4)) : make_float4(0.f, 0.f, 0.f, 0.f);
        }
    float M = -INFINITY;
#pragma unroll
    for (int c = 0; c < kMaxSplit; ++c)
        if (c < k) M = fmaxf(M, ml[c].x);
    float L = 0.f;
    float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
    for (int c = 0; c < kMaxSplit; ++c)
        if (c < k) {
            const float f = fast_exp2(ml[c].x - M);
            L += ml[c].y * f;
            acc.x += v[c].x * f; acc.y += v[c].y * f; acc.z += v[c].z * f; acc.w += v[c].w * f;
        }
    float shrink = 1.f;
    if (p.sinks != nullptr) shrink = join_sink(__ldg(p.sinks + it.head[t]) * kLog2e, M, L);
    if (p.v_scale != nullptr) shrink *= __ldg(p.v_scale + it.head[t] / p.G);      // fp8 cache: the value scale of the head's KV head
    const float inv = shrink / L;
    uint2 w;
    w.x = pack_bf16(acc.x * inv, acc.y * inv);
    w.y = pack_bf16(acc.z * inv, acc.w * inv);
    const int64_t orow = (int64_t)(it.q_row0[t] + r) * p.Hq + it.head[t];
    if (holds) *reinterpret_cast<uint2*>(p.out + orow * D + lane * 4) = w;
    if (p.lse && lane == 0) p.lse[orow] = (M + log2f(L)) * kLn2;
}

cudaError_t launch_prefill_combine(const AttnParams& p, int head_dim, int n_items, cudaStream_t stream)
{
    if (n_items <= 0) return cudaSuccess;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(n_items * 32);
    cfg.blockDim = dim3(256);
    cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    return head_dim == 128 ? cudaLaunchKernelEx(&cfg, prefill_combine_kernel<128>, p) : cudaLaunchKernelEx(&cfg, prefill_combine_kernel<64>, p);
}

// ---------------------------------------------------------------------------------------------
// Self-test of the bounded-wait path: one CTA waits, with a limit of a few milliseconds, on an
// mbarrier that nothing ever arrives at, gives up, raises the error word and returns normally.
__global__ void __launch_bounds__(32) wait_selftest_kernel(uint32_t* err)
{
    __shared__ __align__(8) uint64_t bar;
    __shared__ uint32_t abort_s;
    if (threadIdx.x == 0) {
        abort_s = 0;
        mbar_init(smem_u32(&bar), 1);
        fence_mbar_init();
    }
    __syncwarp();
    const bool ok = mbar_wait(smem_u32(&bar), 0, &abort_s, 1ll << 23);
    __syncwarp();
    if (!ok && threadIdx.x == 0 && err) atomicOr(err, kErrTimeout);
}

cudaError_t launch_wait_selftest(uint32_t* err, cudaStream_t stream)
{
    wait_selftest_kernel<<<1, 32, 0, stream>>>(err);
    return cudaGetLastError();
}

namespace {

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn lookup_encode()
{
    void* ptr = nullptr;
    cudaDriverEntryPointQueryResult q;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &ptr, cudaEnableDefault, &q) == cudaSuccess &&
        q == cudaDriverEntryPointSuccess)
        return reinterpret_cast<EncodeTiledFn>(ptr);
    return nullptr;
}
EncodeTiledFn get_encode()
{
    static const EncodeTiledFn fn = lookup_encode();      // initialised once, thread-safe
    return fn;
}

}  // namespace

// pool viewed as (d, token-in-page, head, block); one box = 64 elements x 16 tokens of one head of one page
bool encode_pool_map(CUtensorMap* m, const void* base, int D, int num_blocks, int Hkv, int64_t s_block, int64_t s_head, int64_t s_token)
{
    EncodeTiledFn enc = get_encode();
    if (!enc) return false;
    cuuint64_t dims[4] = {(cuuint64_t)D, 16, (cuuint64_t)Hkv, (cuuint64_t)num_blocks};
    cuuint64_t strides[3] = {(cuuint64_t)s_token * 2, (cuuint64_t)s_head * 2, (cuuint64_t)s_block * 2};
    cuuint32_t box[4] = {64, 16, 1, 1}, es[4] = {1, 1, 1, 1};
    return enc(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4, const_cast<void*>(base), dims, strides, box, es,
               CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
               CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// q viewed as (d, head, row); one box = 64 elements x 1 head x 128 rows; rows past the end read as zero
bool encode_q_map(CUtensorMap* m, const void* base, int D, int total_rows, int Hq)
{
    EncodeTiledFn enc = get_encode();
    if (!enc) return false;
    cuuint64_t dims[3] = {(cuuint64_t)D, (cuuint64_t)Hq, (cuuint64_t)total_rows};
    cuuint64_t strides[2] = {(cuuint64_t)D * 2, (cuuint64_t)Hq * D * 2};
    cuuint32_t box[3] = {64, 1, (cuuint32_t)QT}, es[3] = {1, 1, 1};
    return enc(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void*>(base), dims, strides, box, es,
               CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
               CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

namespace {

template <int D, bool VARIANT>
cudaError_t launch_prefill_tc_t(const CUtensorMap& mq, const CUtensorMap& mk, const CUtensorMap& mv, const AttnParams& p,
                                int n_items, int n_ctas, int queue_ctas, int first_static, int ticket_base, uint32_t* resident,
                                cudaStream_t stream)
{
    const size_t smem = Geo<D>::SMEM_TOTAL + 1024;
    // The register hand-over inside the kernel (setmaxnreg) is sized for LAUNCH_REGS registers per thread at
    // launch; with any other count a grow request could block forever, so such a build is never launched.
    // (both are set once; host threads racing here compute and store the same values)
    static std::atomic<int> regs_ok{-1};
    if (regs_ok.load(std::memory_order_acquire) < 0) {
        cudaFuncAttributes fa;
        regs_ok.store((cudaFuncGetAttributes(&fa, prefill_tc_kernel<D, VARIANT>) == cudaSuccess && fa.numRegs == LAUNCH_REGS) ? 1 : 0,
                      std::memory_order_release);
    }
    if (!regs_ok.load(std::memory_order_acquire)) return cudaErrorLaunchOutOfResources;
    static std::atomic<bool> configured[64];
    int dev = 0;
    cudaGetDevice(&dev);
    if (dev >= 0 && dev < 64 && !configured[dev].load(std::memory_order_acquire)) {
        cudaError_t e = cudaFuncSetAttribute(prefill_tc_kernel<D, VARIANT>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
        if (e != cudaSuccess) return e;
        configured[dev].store(true, std::memory_order_release);
    }
    // Programmatic dependent launch: barrier set-up and tensor-memory allocation run while the kernel
    // before this one in the stream drains; the kernel waits (griddepcontrol.wait) before its first read.
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(n_ctas);
    cfg.blockDim = dim3(NTHREADS);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, prefill_tc_kernel<D, VARIANT>, mq, mk, mv, p, n_items, queue_ctas, first_static, ticket_base, resident);
}

}  // namespace

cudaError_t launch_prefill_tc(const AttnParams& p, const PrefillMaps& maps, int head_dim, int n_items, int n_ctas,
                              int queue_ctas, int first_static, int ticket_base, uint32_t* resident, cudaStream_t stream)
{
    if (n_items <= 0 || n_ctas <= 0) return cudaSuccess;
    const bool variant = p.window > 0 || p.sinks != nullptr || p.k_scale != nullptr;
    if (head_dim == 128)
        return variant ? launch_prefill_tc_t<128, true>(maps.q, maps.k, maps.v, p, n_items, n_ctas, queue_ctas, first_static, ticket_base, resident, stream)
                       : launch_prefill_tc_t<128, false>(maps.q, maps.k, maps.v, p, n_items, n_ctas, queue_ctas, first_static, ticket_base, resident, stream);
    return variant ? launch_prefill_tc_t<64, true>(maps.q, maps.k, maps.v, p, n_items, n_ctas, queue_ctas, first_static, ticket_base, resident, stream)
                   : launch_prefill_tc_t<64, false>(maps.q, maps.k, maps.v, p, n_items, n_ctas, queue_ctas, first_static, ticket_base, resident, stream);
}

}  // namespace cf
