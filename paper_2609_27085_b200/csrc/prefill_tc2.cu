// Chunked-prefill attention on pairs of SMs (tcgen05.mma.cta_group::2), head_dim 128, group size a multiple of 4.
//
// The one-CTA kernel (prefill_tc.cu) moves 256 KB through an SM's shared memory per 128-token KV tile for 2048
// cycles of MMA work: both operands of S = Q K^T come from shared memory at the SM's full 128 B/clk while TMA
// writes the next tiles into the same memory.  Here two CTAs on two SMs form a cluster and work on one item of
// FOUR 128-row q tiles that share a KV head (four query heads of a group over the same rows): every MMA has
// M = 256 - CTA r holds q tiles (heads) 2r and 2r + 1 and their accumulators in its own tensor memory - and the
// B operand is split between the CTAs: CTA r fetches tokens [64 r, 64 r + 64) of every K tile and columns
// [64 r, 64 r + 64) of every V tile, with the plain per-CTA TMA loads of the one-CTA kernel (no multicast).  Per SM
// and KV tile that is 96 KB of Q K^T operand reads, 32 KB of P V operand reads and 32 KB of TMA writes: 160 KB.
//
// Roles per CTA (384 threads; the first warpgroup hands registers to the softmax warpgroups as in prefill_tc.cu):
//   warp 0      TMA producer of this CTA's Q tiles and K half-tiles; in the even ("leader") CTA also keeper of the
//               work queue, handing every item's context to both CTAs
//   warp 1      leader only: MMA issuer (one lane) for the pair
//   warp 2      TMA producer of this CTA's V half-tiles; waits for each to land, zeroes slack rows of a sequence's
//               last page, and tells the leader
//   warp 3      tells the leader when this CTA's Q tiles and K half-tiles have landed
//   warps 4-11  softmax of this CTA's two q tiles, one thread per row, exactly as in prefill_tc.cu
// Barriers live at the same shared-memory offsets in both CTAs.  Completion of MMAs is multicast to both (s_full,
// o_done, q_empty, k_empty, v_empty); "operands in place" (q_ready, k_ready, v_ready: one arrival per CTA) and
// "probabilities written" (p_full: one arrival per softmax warp of either CTA) are collected on the leader's
// copies, the other CTA arriving through the cluster's shared window.
// Every wait is bounded; a CTA that gives up raises the abort flag of both CTAs, both leave their loops, meet at a
// cluster barrier, report through the error word and release tensor memory together.
//
// Status: correct (held to the oracle like the one-CTA kernel) but NOT the default.  Measured on a B200 it is about
// 20 % slower (a 4096-token chunk over an 8192-token prefix: 982 against 1230 TFLOP/s; the agentic chunk 989 against
// 1203).  What bounds a KV tile is not the shared-memory traffic this design halves but the dependency chain of one
// q tile - P V (j) -> Q K^T (j + 1) -> softmax (j + 1) -> P V (j + 1) - whose softmax leg runs at the exp unit's
// rate; putting a cluster-scope arrival (p_full from the other SM) and multicast completions into that chain
// lengthens it by more than the relieved shared memory returns.  Selected with CF_DEBUG_PREFILL_PAIRS.
#include <atomic>
#include <type_traits>

#include "kernels.h"
#include "prefill_common.cuh"

namespace cf {

namespace {

constexpr int D2 = 128;                            // head_dim of the pair kernel
constexpr int TILE2 = 2 * HALF_BYTES;              // a 128-row q tile: 32 KB
constexpr int KHALF = 64 * 128;                    // [64 tokens][64 elements]: 8 KB; a K half-tile is two of them
constexpr int KV2 = 2 * KHALF;                     // bytes of a K or V half-tile: 16 KB
constexpr uint32_t P_SMEM_Q = 0;
constexpr uint32_t P_SMEM_K = 2 * TILE2;
constexpr uint32_t P_SMEM_V = P_SMEM_K + KV_STAGES * KV2;
constexpr uint32_t P_SMEM_TOTAL = P_SMEM_V + KV_STAGES * KV2;     // 128 KB
constexpr uint32_t PT_S = 0, PT_O = 256;           // tensor-memory columns: S_t at PT_S + 128 t, O_t at PT_O + 128 t

struct Bars2 {
    uint64_t q_full, q_ready, q_empty;
    uint64_t k_full[KV_STAGES], k_ready[KV_STAGES], k_empty[KV_STAGES];
    uint64_t v_full[KV_STAGES], v_ready[KV_STAGES], v_empty[KV_STAGES];
    uint64_t s_full[2], p_full[2], o_done[2];
    uint64_t item_full[2];
};

}  // namespace

// n_items work items (PrefillTcItem with pair semantics: CTA r of a pair adds 2 r to head[] and r * pad to
// part_slot[]); the grid is 2 x (resident pairs); pair b starts on item b when first_static is set and then draws
// tickets from p.pre_queue like the one-CTA kernel (queue_pairs pairs draw in total; ticket t = item ticket_base + t).
__global__ void __launch_bounds__(NTHREADS, 1)
prefill_tc2_kernel(const __grid_constant__ CUtensorMap map_q, const __grid_constant__ CUtensorMap map_k,
                   const __grid_constant__ CUtensorMap map_v, const AttnParams p, const int n_items, const int queue_pairs,
                   const int first_static, const int ticket_base, uint32_t* const resident)
{
    constexpr int D = D2, KS = D / 16;
    constexpr uint32_t kPolyMask = CF_POLY_MASK;
    extern __shared__ uint8_t smem_raw[];
    __shared__ __align__(16) ItemCtx ctx_s[2];
    __shared__ __align__(8) Bars2 bars;
    __shared__ uint32_t tmem_base_s;
    __shared__ uint32_t abort_s;
    __shared__ uint32_t issuer_state[4];

    const uint32_t smem = (smem_u32(smem_raw) + 1023u) & ~1023u;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const uint32_t rank = cluster_ctarank();           // 0: leader (issues the MMAs), 1: its partner
    const bool leader = rank == 0;
    const int pair = (int)(blockIdx.x >> 1);
    const bool has_static = first_static != 0 && pair < n_items;
    PrefillTcItem first_it;
    if (warp == 0 && leader && has_static) {
        const uint4* src = reinterpret_cast<const uint4*>(p.pre_tc_items + pair);
        uint4* dst = reinterpret_cast<uint4*>(&first_it);
#pragma unroll
        for (int i = 0; i < (int)(sizeof(PrefillTcItem) / 16); ++i) dst[i] = __ldg(src + i);
    }
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    volatile uint32_t* abort_flag = &abort_s;
    const uint32_t peer_abort = mapa_cluster(smem_u32(&abort_s), rank ^ 1u);

    if (threadIdx.x == 0) {
        abort_s = (p.err != nullptr && (*reinterpret_cast<volatile uint32_t*>(p.err) & kErrTimeout) != 0u) ? 2u : 0u;
        if (resident != nullptr) atomicAdd(resident, 1u);
        mbar_init(smem_u32(&bars.q_full), 1);
        mbar_init(smem_u32(&bars.q_ready), 2);            // one arrival per CTA
        mbar_init(smem_u32(&bars.q_empty), 1);
        for (int s = 0; s < KV_STAGES; ++s) {
            mbar_init(smem_u32(&bars.k_full[s]), 1);
            mbar_init(smem_u32(&bars.k_ready[s]), 2);
            mbar_init(smem_u32(&bars.k_empty[s]), 1);
            mbar_init(smem_u32(&bars.v_full[s]), 1);
            mbar_init(smem_u32(&bars.v_ready[s]), 2);
            mbar_init(smem_u32(&bars.v_empty[s]), 1);
        }
        for (int t = 0; t < 2; ++t) {
            mbar_init(smem_u32(&bars.s_full[t]), 1);
            mbar_init(smem_u32(&bars.p_full[t]), 8);      // one arrival per softmax warp of either CTA
            mbar_init(smem_u32(&bars.o_done[t]), 1);
            mbar_init(smem_u32(&bars.item_full[t]), 1);
        }
        fence_mbar_init();
    }
    __syncwarp();
    if (warp == 0) tmem_alloc2<512>(smem_u32(&tmem_base_s));
    tc_fence_before();
    cluster_sync_all();                                   // both CTAs: barriers initialised, tensor memory allocated
    tc_fence_after();
    const uint32_t tmem = tmem_base_s;
    asm volatile("griddepcontrol.wait;" ::: "memory");

    // a wait that gave up raises the other CTA's abort flag as well, so that both leave together
    auto wait_local = [&](uint32_t bar, uint32_t parity) -> bool {
        if (mbar_wait(bar, parity, abort_flag)) return true;
        st_cluster_u32(peer_abort, 1u);
        return false;
    };
    auto wait_pair = [&](uint32_t bar, uint32_t parity) -> bool {       // arrivals may come from the other CTA
        if (mbar_wait_cl(bar, parity, abort_flag)) return true;
        st_cluster_u32(peer_abort, 1u);
        return false;
    };
    // one arrival on the LEADER's copy of a barrier
    auto arrive_leader = [&](uint32_t bar) {
        if (leader) mbar_arrive(bar);
        else mbar_arrive_cluster(mapa_cluster(bar, 0u));
    };
    auto checked_pid = [&](int32_t id) -> int32_t {
        if ((uint32_t)id < (uint32_t)p.num_blocks) return id;
        if (p.err) atomicOr(p.err, kErrBlockId);
        return 0;
    };
    auto wait_item = [&](int k) -> const ItemCtx* {
        if (!wait_pair(smem_u32(&bars.item_full[k & 1]), (uint32_t)(k >> 1) & 1u)) return nullptr;
        return &ctx_s[k & 1];
    };

    if (warp < 4) {
      reg_dec<REGS_ROLE>();
      if (warp == 3) {
        // =========================================================== tells the leader when this CTA's Q and K halves are in place
        uint32_t ub[2] = {0u, 0u};
        bool ok = true;
        for (int k = 0; ok; ++k) {
            const ItemCtx* cs = wait_item(k);
            if (cs == nullptr || cs->live == 0) break;
            const int n_max = cs->n_max;
            ok = __all_sync(0xffffffffu, wait_local(smem_u32(&bars.q_full), (uint32_t)k & 1u));
            if (!ok) break;
            if (lane == 0) arrive_leader(smem_u32(&bars.q_ready));
            for (int j = 0; j < n_max && ok; ++j) {
                const int stage = j & 1;
                ok = __all_sync(0xffffffffu, wait_local(smem_u32(&bars.k_full[stage]), (ub[stage] + (uint32_t)(j >> 1)) & 1u));
                if (ok && lane == 0) arrive_leader(smem_u32(&bars.k_ready[stage]));
            }
            ub[0] += (uint32_t)(n_max + 1) >> 1;
            ub[1] += (uint32_t)n_max >> 1;
        }
      } else if (warp == 2) {
        // =========================================================== V half-tiles: fetch, wait, zero slack rows, tell the leader
        // (this CTA's half = columns [64 rank, 64 rank + 64) of the head dimension for all tokens of the tile: one box per page)
        uint32_t ub[2] = {0u, 0u};
        bool ok = true;
        for (int k = 0; ok; ++k) {
            const ItemCtx* cs = wait_item(k);
            if (cs == nullptr || cs->live == 0) break;
            const int n_max = cs->n_max, total_pages = cs->total_pages, jb = cs->it.j_begin, kvh = cs->it.kvh;
            const int page_lo = cs->it.page_lo, Lc = cs->it.ctx_len;
            const int32_t* bt = p.block_table + (int64_t)cs->it.seq * p.max_blocks;
            int32_t pid = (lane < min(8, total_pages - 8 * jb) && 8 * jb + lane >= page_lo) ? checked_pid(__ldg(bt + 8 * jb + lane)) : 0;
            for (int j = 0; j < n_max && ok; ++j) {
                const int stage = j & 1;
                const uint32_t use = ub[stage] + (uint32_t)(j >> 1);
                const int np = min(8, total_pages - 8 * (jb + j));
                const int p0 = max(0, page_lo - 8 * (jb + j));
                const int32_t my_pid = pid;
                if (j + 1 < n_max) pid = lane < min(8, total_pages - 8 * (jb + j + 1)) ? checked_pid(__ldg(bt + 8 * (jb + j + 1) + lane)) : 0;
                if (use > 0) ok = __all_sync(0xffffffffu, wait_local(smem_u32(&bars.v_empty[stage]), (use - 1) & 1u));
                if (!ok) break;
                const uint32_t dst = smem + P_SMEM_V + stage * KV2;
                if (lane == 0) mbar_arrive_expect_tx(smem_u32(&bars.v_full[stage]), (np - p0) * 2048);
                __syncwarp();
                if (lane < np && lane >= p0)
                    tma_load_4d(dst + lane * 2048, &map_v, 64 * (int)rank, 0, kvh, my_pid, smem_u32(&bars.v_full[stage]));
                ok = __all_sync(0xffffffffu, wait_local(smem_u32(&bars.v_full[stage]), use & 1u));
                if (!ok) break;
                if (j == n_max - 1 && Lc < (8 * (jb + j) + np) * 16) {
                    // slack slots of the sequence's last page came in with the page: zero those rows so that a zero
                    // probability never multiplies a NaN
                    const int r0 = Lc - (jb + j) * KT, r1 = np * 16;
                    uint8_t* base = smem_raw + (dst - smem_u32(smem_raw));
                    for (int idx = lane; idx < (r1 - r0) * 8; idx += 32)
                        *reinterpret_cast<uint4*>(base + (r0 + (idx >> 3)) * 128 + (idx & 7) * 16) = make_uint4(0u, 0u, 0u, 0u);
                    fence_proxy_async();
                }
                __syncwarp();
                if (lane == 0) arrive_leader(smem_u32(&bars.v_ready[stage]));
            }
            ok = __all_sync(0xffffffffu, ok);
            ub[0] += (uint32_t)(n_max + 1) >> 1;
            ub[1] += (uint32_t)n_max >> 1;
        }
      } else if (warp == 0) {
        // =========================================================== Q tiles and K half-tiles; in the leader: the work queue
        if (lane == 0) {
            prefetch_tensormap(&map_q);
            prefetch_tensormap(&map_k);
            prefetch_tensormap(&map_v);
        }
        bool counted_out = false;
        auto draw = [&](ItemCtx& cx) {                 // leader only
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
                if (!counted_out && lane == 0 && atomicAdd(p.pre_queue + 1, 1u) == (uint32_t)(queue_pairs - 1)) {
                    p.pre_queue[0] = 0u;
                    p.pre_queue[1] = 0u;
                    __threadfence();
                }
                counted_out = true;
            }
        };
        ItemCtx cx, nx;
        cx.live = 0;
        if (leader) {
            if (has_static && *abort_flag == 0u) {
                cx.it = first_it;
                derive_item(cx);
            } else {
                draw(cx);
            }
        }
        uint32_t ub[2] = {0u, 0u};
        bool ok = true;
        for (int k = 0; ok; ++k) {
            // Q tiles and the context slot (of both CTAs) are free once every S = Q K^T of the previous item has completed
            if (k > 0) ok = __all_sync(0xffffffffu, wait_local(smem_u32(&bars.q_empty), (uint32_t)(k - 1) & 1u));
            if (!ok) break;
            if (leader) {
                if (lane == 0) {
                    const uint4* src = reinterpret_cast<const uint4*>(&cx);
                    uint4* dst = reinterpret_cast<uint4*>(&ctx_s[k & 1]);
                    const uint32_t peer_ctx = mapa_cluster(smem_u32(&ctx_s[k & 1]), 1u);
#pragma unroll
                    for (int i = 0; i < (int)(sizeof(ItemCtx) / 16); ++i) {
                        dst[i] = src[i];
                        st_cluster_v4(peer_ctx + 16 * i, src[i]);
                    }
                    mbar_arrive(smem_u32(&bars.item_full[k & 1]));
                    mbar_arrive_cluster(mapa_cluster(smem_u32(&bars.item_full[k & 1]), 1u));     // release: the stores above are visible
                }
            } else {
                const ItemCtx* cs = wait_item(k);
                if (cs == nullptr) break;
                cx = *cs;
            }
            if (!cx.live) break;
            const PrefillTcItem& it = cx.it;
            if (lane == 0) {
                const int nq = (it.n_rows[0] > 0) + (it.n_rows[1] > 0);
                mbar_arrive_expect_tx(smem_u32(&bars.q_full), nq * TILE2);
                for (int t = 0; t < 2; ++t)
                    if (it.n_rows[t] > 0)
                        for (int h = 0; h < 2; ++h)
                            tma_load_3d(smem + P_SMEM_Q + t * TILE2 + h * HALF_BYTES, &map_q, h * 64, it.head[t] + 2 * (int)rank,
                                        it.q_row0[t], smem_u32(&bars.q_full));
            }
            const int32_t* bt = p.block_table + (int64_t)it.seq * p.max_blocks;
            const int n_max = cx.n_max, total_pages = cx.total_pages, jb = it.j_begin, page_lo = it.page_lo;
            const int j_draw = min(2, n_max - 1);
            bool drawn = false;
            // this CTA's half of a K tile: pages 4 rank .. 4 rank + 3 of the tile (tokens [64 rank, 64 rank + 64)); lanes 0..3 hold their ids
            auto my_page_id = [&](int tile) -> int32_t {
                const int pg = 8 * tile + 4 * (int)rank + (lane & 3);
                return (lane < 4 && pg < total_pages && pg >= page_lo) ? checked_pid(__ldg(bt + pg)) : 0;
            };
            int32_t pid = my_page_id(jb);
            for (int j = 0; j < n_max && ok; ++j) {
                const int stage = j & 1;
                const uint32_t use = ub[stage] + (uint32_t)(j >> 1);
                const int np = min(8, total_pages - 8 * (jb + j));
                const int p0 = max(0, page_lo - 8 * (jb + j));
                // pages of the tile in this CTA's half that are fetched: local index in [lo, hi)
                const int lo = min(4, max(0, p0 - 4 * (int)rank)), hi = min(4, max(0, np - 4 * (int)rank));
                const int32_t my_pid = __shfl_sync(0xffffffffu, pid, lane >> 1);
                if (j + 1 < n_max) pid = my_page_id(jb + j + 1);
                if (use > 0) ok = __all_sync(0xffffffffu, wait_local(smem_u32(&bars.k_empty[stage]), (use - 1) & 1u));
                if (!ok) break;
                if (lane == 0) mbar_arrive_expect_tx(smem_u32(&bars.k_full[stage]), max(0, hi - lo) * 4096);
                __syncwarp();
                // lane = 2 * page + half: a box is one 64-element half of one page, 2 KB
                if (lane < 8 && (lane >> 1) >= lo && (lane >> 1) < hi)
                    tma_load_4d(smem + P_SMEM_K + stage * KV2 + (lane & 1) * KHALF + (lane >> 1) * 2048, &map_k, (lane & 1) * 64, 0,
                                it.kvh, my_pid, smem_u32(&bars.k_full[stage]));
                if (leader && j == j_draw) {
                    draw(nx);
                    drawn = true;
                }
            }
            ok = __all_sync(0xffffffffu, ok);
            if (leader) {
                if (ok && !drawn) draw(nx);
                cx = nx;
            }
            ub[0] += (uint32_t)(n_max + 1) >> 1;
            ub[1] += (uint32_t)n_max >> 1;
        }
        if (leader && !counted_out) draw(nx);
      } else if (leader) {
        // =========================================================== MMA issuer of the pair (warp 1 of the leader, one lane)
        constexpr uint32_t IDESC_QK = idesc_bf16(256, 128, false);
        constexpr uint32_t IDESC_PV = idesc_bf16(256, D, true);
        constexpr uint64_t HI64 = (uint64_t)desc_hi_sw128(1024) << 32;
        uint64_t qd[2][KS], kd[KV_STAGES][KS], vd[KV_STAGES][8];
#pragma unroll
        for (int i = 0; i < 2; ++i) {
#pragma unroll
            for (int ks = 0; ks < KS; ++ks) {
                qd[i][ks] = HI64 | (desc_lo_sw128(smem + P_SMEM_Q + i * TILE2, 16) + (uint32_t)(((ks >> 2) * HALF_BYTES + (ks & 3) * 32) >> 4));
                kd[i][ks] = HI64 | (desc_lo_sw128(smem + P_SMEM_K + i * KV2, 16) + (uint32_t)(((ks >> 2) * KHALF + (ks & 3) * 32) >> 4));
            }
#pragma unroll
            for (int ks = 0; ks < 8; ++ks)
                vd[i][ks] = HI64 | (desc_lo_sw128(smem + P_SMEM_V + i * KV2, KV2) + ks * (2048 >> 4));
        }
        const uint32_t bar_s[2] = {smem_u32(&bars.s_full[0]), smem_u32(&bars.s_full[1])};
        const uint32_t bar_o[2] = {smem_u32(&bars.o_done[0]), smem_u32(&bars.o_done[1])};
        const uint32_t bar_p[2] = {smem_u32(&bars.p_full[0]), smem_u32(&bars.p_full[1])};
        auto issue_qk = [&](auto T, auto S) {
            constexpr int t = decltype(T)::value, st = decltype(S)::value;
            const uint32_t dS = tmem + PT_S + t * 128;
            umma2_ss(dS, qd[t][0], kd[st][0], IDESC_QK, 0u);
#pragma unroll
            for (int ks = 1; ks < KS; ++ks) umma2_ss(dS, qd[t][ks], kd[st][ks], IDESC_QK, 1u);
            umma2_commit(bar_s[t]);
        };
        auto issue_pv = [&](auto T, auto S, int ks0, int n_steps, uint32_t acc0) {
            constexpr int t = decltype(T)::value, st = decltype(S)::value;
            const uint32_t dO = tmem + PT_O + t * D, aP = tmem + PT_S + t * 128;
            if (ks0 == 0 && n_steps == 8) {
                umma2_ts(dO, aP, vd[st][0], IDESC_PV, acc0);
#pragma unroll
                for (int ks = 1; ks < 8; ++ks) umma2_ts(dO, aP + ks * 8, vd[st][ks], IDESC_PV, 1u);
            } else {
#pragma unroll
                for (int ks = 0; ks < 8; ++ks)
                    if (ks >= ks0 && ks < n_steps) umma2_ts(dO, aP + ks * 8, vd[st][ks], IDESC_PV, ks == ks0 ? acc0 : 1u);
            }
            umma2_commit(bar_o[t]);
        };
        using I0 = std::integral_constant<int, 0>;
        using I1 = std::integral_constant<int, 1>;
        if (lane == 0) {
        const uint32_t bar_kf[2] = {smem_u32(&bars.k_ready[0]), smem_u32(&bars.k_ready[1])};
        const uint32_t bar_vf[2] = {smem_u32(&bars.v_ready[0]), smem_u32(&bars.v_ready[1])};
        const uint32_t bar_ke[2] = {smem_u32(&bars.k_empty[0]), smem_u32(&bars.k_empty[1])};
        const uint32_t bar_ve[2] = {smem_u32(&bars.v_empty[0]), smem_u32(&bars.v_empty[1])};
        const uint32_t bar_qe = smem_u32(&bars.q_empty);
        volatile uint32_t* const ist = issuer_state;     // running phases, as in the one-CTA kernel
        ist[0] = ist[1] = ist[2] = ist[3] = 0u;
        bool ok = true;
        for (int k = 0; ok; ++k) {
        const ItemCtx* cs = wait_item(k);
        if (cs == nullptr || cs->live == 0) break;
        const volatile ItemCtx* const vs = cs;
        const int n_max = cs->n_max;
        const int n_j[2] = {cs->n_j[0], cs->n_j[1]};
        ok = wait_pair(smem_u32(&bars.q_ready), (uint32_t)k & 1u);
        ok = ok && wait_pair(bar_kf[0], ist[0] & 1u);
        if (!ok) break;
        tc_fence_after();
        if (n_j[0] > 0) issue_qk(I0{}, I0{});
        if (n_j[1] > 0) issue_qk(I1{}, I0{});
        umma2_commit(bar_ke[0]);
        if (n_max <= 1) umma2_commit(bar_qe);
        const int n_int = (n_j[0] > 0 && n_j[1] > 0) ? min(n_j[0], n_j[1]) - 1 : 0;
        auto lean_step = [&](auto S, uint32_t par_v, uint32_t par_k1, uint32_t par_p0, uint32_t par_p1, uint32_t acc0) -> bool {
            constexpr int st = decltype(S)::value, st1 = st ^ 1;
            using S1 = std::integral_constant<int, st1>;
            if (!wait_pair(bar_vf[st], par_v)) return false;
            if (!wait_pair(bar_kf[st1], par_k1)) return false;
            if (!wait_pair(bar_p[0], par_p0)) return false;
            tc_fence_after();
            issue_pv(I0{}, S, 0, 8, acc0);
            issue_qk(I0{}, S1{});
            if (!wait_pair(bar_p[1], par_p1)) return false;
            tc_fence_after();
            issue_pv(I1{}, S, 0, 8, acc0);
            issue_qk(I1{}, S1{});
            umma2_commit(bar_ve[st]);
            umma2_commit(bar_ke[st1]);
            return true;
        };
        auto kv_step = [&](auto S, int j) -> bool {
            constexpr int st = decltype(S)::value, st1 = st ^ 1;
            using S1 = std::integral_constant<int, st1>;
            const int jb = vs->it.j_begin;
            const int np = min(8, vs->total_pages - 8 * (jb + j));
            const int ks0 = max(0, vs->it.page_lo - 8 * (jb + j));
            if (!wait_pair(bar_vf[st], (ist[st] + (uint32_t)(j >> 1)) & 1u)) return false;
            const uint32_t acc0 = j > 0 ? 1u : 0u;
            auto tile = [&](auto T) -> bool {
                constexpr int t = decltype(T)::value;
                if (j >= n_j[t]) return true;
                const bool more = j + 1 < n_j[t];
                if (more && !wait_pair(bar_kf[st1], (ist[st1] + (uint32_t)((j + 1) >> 1)) & 1u)) return false;
                if (!wait_pair(bar_p[t], (ist[2 + t] + (uint32_t)j) & 1u)) return false;
                tc_fence_after();
                issue_pv(T, S, ks0, np, acc0);
                if (more) issue_qk(T, S1{});
                return true;
            };
            if (!tile(I0{})) return false;
            if (!tile(I1{})) return false;
            umma2_commit(bar_ve[st]);
            if (j + 1 < n_max) umma2_commit(bar_ke[st1]);
            if (j + 1 == n_max - 1) umma2_commit(bar_qe);
            return true;
        };
        int j = 0;
        const bool partial_first = vs->it.page_lo > 8 * vs->it.j_begin;
        if (partial_first) {
            for (; j < min(2, n_max) && ok; ++j) ok = (j & 1) ? kv_step(I1{}, j) : kv_step(I0{}, j);
        }
        const int j_pairs = j;
        if (ok) {
            uint32_t h0 = (ist[0] + (uint32_t)(j >> 1)) & 1u, h1 = (ist[1] + (uint32_t)(j >> 1)) & 1u;
            const uint32_t p0 = ist[2] & 1u, p1 = ist[3] & 1u;
            for (; ok && j + 1 < n_int; j += 2, h0 ^= 1u, h1 ^= 1u) {
                ok = lean_step(I0{}, h0, h1, p0, p1, j > 0 ? 1u : 0u);
                if (ok) ok = lean_step(I1{}, h1, h0 ^ 1u, p0 ^ 1u, p1 ^ 1u, 1u);
            }
            if (ok && j > j_pairs && j >= n_max - 1) umma2_commit(bar_qe);
        }
        static_assert(KV_STAGES == 2, "the stage index is the parity of the tile index");
        for (; j < n_max && ok; ++j) ok = (j & 1) ? kv_step(I1{}, j) : kv_step(I0{}, j);
        ist[0] += (uint32_t)(n_max + 1) >> 1;
        ist[1] += (uint32_t)n_max >> 1;
        ist[2] += (uint32_t)n_j[0];
        ist[3] += (uint32_t)n_j[1];
        }
        }
      }
    } else {
      reg_inc<REGS_SOFTMAX>();
      // =========================================================== softmax + epilogue of this CTA's two q tiles, one thread per row
      const int t = (warp - 4) >> 2;
      const int row = (warp & 3) * 32 + lane;
      const uint32_t lanes = lane_field(warp);
      const uint32_t tS = tmem + PT_S + t * 128 + lanes, tO = tmem + PT_O + t * D + lanes;
      uint32_t sbt = 0u;
      bool ok = true;
      for (int k = 0; ok; ++k) {
        const ItemCtx* cs = wait_item(k);
        if (cs == nullptr || cs->live == 0) break;
        {
        const int jb = cs->it.j_begin, n_jt = cs->n_j[t], kv_hi = cs->kv_hi_t[t];
        const int it_row0 = cs->it.row0[t], it_n_rows = cs->it.n_rows[t], it_q_row0 = cs->it.q_row0[t];
        const int it_head = cs->it.head[t] + 2 * (int)rank;                                         // this CTA's heads of the group
        const int it_part_slot = cs->it.part_slot[t] < 0 ? -1 : cs->it.part_slot[t] + (int)rank * cs->it.pad;
        const int it_part_k = cs->it.part_k, it_part_c = cs->it.part_c;
        // fp8 cache: the staged K/V hold the codes; their per-head scales join the softmax scale and the output here
        const float sc = p.k_scale != nullptr ? p.scale_log2 * __ldg(p.k_scale + cs->it.kvh) : p.scale_log2;
        const float v_scale = p.v_scale != nullptr ? __ldg(p.v_scale + cs->it.kvh) : 1.f;
        const int limit = min(cs->it.prefix + it_row0 + row, kv_hi - 1);
        const int first_key = p.window > 0 ? limit - p.window + 1 : -(1 << 30);
        const uint32_t span = (uint32_t)(limit - first_key);
        float m_used = -INFINITY, l_sum = 0.f;
        for (int j = 0; j < n_jt; ++j) {
            ok = wait_local(smem_u32(&bars.s_full[t]), (sbt + (uint32_t)j) & 1u);
            if (!ok) break;
            tc_fence_after();
            float sv[128];
#pragma unroll
            for (int c = 0; c < 4; ++c) tmem_ld32(tS + c * 32, reinterpret_cast<uint32_t*>(&sv[c * 32]));
            tmem_wait_ld();
            const int col_limit = limit - (jb + j) * KT;
            const int col_first = first_key - (jb + j) * KT;
            if (__any_sync(0xffffffffu, col_limit < KT - 1 || col_first > 0)) {
#pragma unroll
                for (int c = 0; c < 128; ++c) sv[c] = ((uint32_t)(c - col_first) <= span) ? sv[c] : -INFINITY;
            }
            if (__any_sync(0xffffffffu, m_used == -INFINITY)) {
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
                if (m_used == -INFINITY) m_used = fmaxf(fmaxf(mx4[0], mx4[1]), fmaxf(mx4[2], mx4[3])) * sc;
            }
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
            float tile_sum = exp_pass(m_used == -INFINITY ? 0.f : -m_used);
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
                const float d = fmaxf(rise, 0.f);
                const float f = fast_exp2(-d);
                m_used += d;
                l_sum *= f;
                if (j > 0) {
                    ok = wait_local(smem_u32(&bars.o_done[t]), (sbt + (uint32_t)(j - 1)) & 1u);
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
                tile_sum = exp_pass(m_used == -INFINITY ? 0.f : -m_used);
            }
            l_sum += tile_sum;
            tmem_wait_st();
            tc_fence_before();
            __syncwarp();
            if (lane == 0) arrive_leader(smem_u32(&bars.p_full[t]));
        }
        if (ok && n_jt > 0) ok = wait_local(smem_u32(&bars.o_done[t]), (sbt + (uint32_t)(n_jt - 1)) & 1u);
        if (ok && n_jt > 0) {
            tc_fence_after();
            const bool live = row < it_n_rows;
            const bool partial = it_part_slot >= 0;
            float m_fin = m_used, l_fin = l_sum, shrink = 1.f;
            if (!partial && p.sinks != nullptr) shrink = join_sink(__ldg(p.sinks + it_head) * kLog2e, m_fin, l_fin);
            const float inv = shrink * v_scale / l_fin;
            __nv_bfloat16* orow = p.out + ((int64_t)(it_q_row0 + row) * p.Hq + it_head) * D;
            const int64_t pslot = (int64_t)it_part_slot + (int64_t)row * it_part_k + it_part_c;
            float* prow = p.pre_part_o + pslot * D;
#pragma unroll
            for (int c = 0; c < D / 32; ++c) {
                float ov[32];
                tmem_ld32(tO + c * 32, reinterpret_cast<uint32_t*>(ov));
                tmem_wait_ld();
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
            tc_fence_before();
        }
        sbt += (uint32_t)n_jt;
        }
      }
    }

    // ---- teardown: every role of both CTAs has left its loop (the tickets ran out, or an abort flag went up)
    __syncwarp();                                         // the cluster barrier wants whole warps (single-lane roles rejoin here)
    tc_fence_before();
    cluster_sync_all();
    if (abort_s == 1u) {
        if (threadIdx.x == 0 && p.err) atomicOr(p.err, kErrTimeout);
        // let copies and MMAs that may still be in flight settle before tensor memory is handed back
        for (int i = 0; i < 64; ++i) __nanosleep(2000);
    }
    cluster_sync_all();                                   // neither CTA leaves while the other may still touch its memory
    if (warp == 0) tmem_dealloc2<512>(tmem);
}

bool prefill_pair_supported(const cf_cache_desc* d)
{
    const int g = d->num_q_heads / d->num_kv_heads;
    return d->head_dim == D2 && d->block_size == 16 && g % 4 == 0;
}

cudaError_t launch_prefill_tc2(const AttnParams& p, const PrefillMaps& maps, int n_items, int n_pairs, int queue_pairs,
                               int first_static, int ticket_base, uint32_t* resident, cudaStream_t stream)
{
    if (n_items <= 0 || n_pairs <= 0) return cudaSuccess;
    const size_t smem = P_SMEM_TOTAL + 1024;
    // the register hand-over (setmaxnreg) is sized for LAUNCH_REGS registers per thread at launch: a build with any
    // other count is never launched (a grow request that cannot be met would block forever)
    static std::atomic<int> regs_ok{-1};
    if (regs_ok.load(std::memory_order_acquire) < 0) {
        cudaFuncAttributes fa;
        regs_ok.store((cudaFuncGetAttributes(&fa, prefill_tc2_kernel) == cudaSuccess && fa.numRegs == LAUNCH_REGS) ? 1 : 0,
                      std::memory_order_release);
    }
    if (!regs_ok.load(std::memory_order_acquire)) return cudaErrorLaunchOutOfResources;
    static std::atomic<bool> configured[64];
    int dev = 0;
    cudaGetDevice(&dev);
    if (dev >= 0 && dev < 64 && !configured[dev].load(std::memory_order_acquire)) {
        cudaError_t e = cudaFuncSetAttribute(prefill_tc2_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
        if (e != cudaSuccess) return e;
        configured[dev].store(true, std::memory_order_release);
    }
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(2 * n_pairs);
    cfg.blockDim = dim3(NTHREADS);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = stream;
    cudaLaunchAttribute attr[2];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    attr[1].id = cudaLaunchAttributeClusterDimension;
    attr[1].val.clusterDim.x = 2;
    attr[1].val.clusterDim.y = 1;
    attr[1].val.clusterDim.z = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 2;
    return cudaLaunchKernelEx(&cfg, prefill_tc2_kernel, maps.q, maps.k, maps.v, p, n_items, queue_pairs, first_static, ticket_base, resident);
}

}  // namespace cf
