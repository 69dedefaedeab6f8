// Split-K decode attention over the paged KV cache (HBM-bound).
//
// One CTA serves one (decode sequence, KV chunk, KV head).  The G query heads that share the KV
// head ride along as the N dimension of the tensor-core tiles, so every K/V byte is read from HBM
// exactly once.  Each warp walks its own pages (page = 16 tokens) through a private cp.async ring;
// there is no block-wide barrier in the main loop.
//
// Orientation.  With only G <= 8 query rows, the usual S = Q K^T wastes the 16-row MMA tile.  The
// kernel computes the transposes instead:
//     S^T[token, head] = K[token, :] . Q[head, :]        A = K page (16 x D),   B = Q^T (D x 8)
//     O^T[d, head]    += V^T[d, token] . P^T[token, head] A = V^T via ldmatrix.trans, B = P^T
// so one m16n8k16 covers a whole page against all (up to 8) heads with no padding rows, and the
// probabilities move from accumulator layout to B-operand layout with one movmatrix per 8 tokens.
// Softmax runs per head (a column of S^T): running max in the log2 domain, un-normalised sums.
//
// Output: a sequence with a single chunk writes bf16 `out` (and lse) directly; otherwise the CTA
// writes an fp32 partial (o, m, l) that the combine kernel merges in fixed chunk order.
#include <cuda_fp16.h>

#include <algorithm>
#include <atomic>
#include <mutex>

#include "device_common.cuh"
#include "kernels.h"

namespace cf {

// ---------------------------------------------------------------------------------------------
// Merge of the partials of one (split sequence, query head) in fixed chunk order (deterministic), one float4
// of the head per calling thread:
//   M = max_c m_c ; O = sum_c 2^(m_c - M) o_c / sum_c 2^(m_c - M) l_c ; lse = (M + log2 sum) ln 2
// evaluated as a running merge over groups of eight chunks.  Partials are fetched eight chunks at a time
// with independent L2 loads (a dependent load per chunk would cost a memory round trip each; L2 loads,
// because in the fused path other CTAs of the same grid wrote them).
template <int D>
__device__ __forceinline__ void merge_partials(const AttnParams& p, int q_row, int part_first, int n_chunks, int hq, int d,
                                               bool write_lse)
{
    constexpr int GROUP = 8;
    float M = -INFINITY, L = 0.f;
    float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
    for (int c0 = 0; c0 < n_chunks; c0 += GROUP) {
        float2 ml[GROUP];
        float4 v[GROUP];
#pragma unroll
        for (int i = 0; i < GROUP; ++i)
            if (c0 + i < n_chunks) {
                const int64_t pr = (int64_t)(part_first + c0 + i) * p.Hq + hq;
                ml[i] = __ldcg(reinterpret_cast<const float2*>(p.part_ml + pr * 2));
                v[i] = __ldcg(reinterpret_cast<const float4*>(p.part_o + pr * D + d));
            }
        float Mg = M;
#pragma unroll
        for (int i = 0; i < GROUP; ++i)
            if (c0 + i < n_chunks) Mg = fmaxf(Mg, ml[i].x);
        const float fold = fast_exp2(M - Mg);               // 0 on the first group (M = -inf)
        L *= fold;
        acc.x *= fold; acc.y *= fold; acc.z *= fold; acc.w *= fold;
        M = Mg;
#pragma unroll
        for (int i = 0; i < GROUP; ++i)
            if (c0 + i < n_chunks) {
                const float f = fast_exp2(ml[i].x - M);
                L += ml[i].y * f;
                acc.x += v[i].x * f; acc.y += v[i].y * f; acc.z += v[i].z * f; acc.w += v[i].w * f;
            }
    }
    float shrink = 1.f;
    if (p.sinks != nullptr) shrink = join_sink(__ldg(p.sinks + hq) * kLog2e, M, L);
    const float inv = shrink / L;
    __nv_bfloat162 lo = __floats2bfloat162_rn(acc.x * inv, acc.y * inv);
    __nv_bfloat162 hi = __floats2bfloat162_rn(acc.z * inv, acc.w * inv);
    uint2 packed;
    packed.x = *reinterpret_cast<uint32_t*>(&lo);
    packed.y = *reinterpret_cast<uint32_t*>(&hi);
    *reinterpret_cast<uint2*>(p.out + ((int64_t)q_row * p.Hq + hq) * D + d) = packed;
    if (p.lse && write_lse) p.lse[(int64_t)q_row * p.Hq + hq] = (M + log2f(L)) * kLn2;
}

template <int D, int NWARPS, int NSTAGE>
__device__ __forceinline__ void decode_cta(const AttnParams& p, const int cta)
{
    constexpr int CPR = D / 8;                  // 16-byte chunks per token row
    constexpr int PAGE_BYTES = 16 * D * 2;      // one (page, head) of K or of V
    constexpr int STAGE_BYTES = 2 * PAGE_BYTES;
    constexpr int WARP_BYTES = NSTAGE * STAGE_BYTES;
    constexpr int KSTEPS = D / 16;
    constexpr int DP = D + 4;                   // padded row of the merge buffer (bank-conflict free)
    extern __shared__ __align__(1024) uint8_t smem[];

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int item_id = cta / p.Hkv, kvh = cta % p.Hkv;
    const DecodeItem it = p.dec_items[item_id];
    const int G = p.G;
    // lets the combine kernel (launched with programmatic stream serialisation) become resident while
    // this grid drains; it still waits for this grid's completion before it reads a partial
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");

    // ---- Q^T fragments (B operand): thread holds Q[head = lane/4][d = 16*ks + 2*(lane%4) + {0,1} (+8)]
    uint32_t qf[KSTEPS][2];
    {
        const int head = lane >> 2;
        const uint32_t* qrow = reinterpret_cast<const uint32_t*>(
            p.q + ((int64_t)it.q_row * p.Hq + (int64_t)kvh * G + head) * D);
#pragma unroll
        for (int ks = 0; ks < KSTEPS; ++ks) {
            qf[ks][0] = head < G ? __ldg(qrow + ks * 8 + (lane & 3)) : 0u;
            qf[ks][1] = head < G ? __ldg(qrow + ks * 8 + 4 + (lane & 3)) : 0u;
        }
    }

    const int first_page = it.kv_begin >> 4;
    const int n_pages = (it.kv_end - it.kv_begin + 15) >> 4;
    const int my_n = n_pages > warp ? (n_pages - warp + NWARPS - 1) / NWARPS : 0;
    const int32_t* bt = p.block_table + (int64_t)it.seq * p.max_blocks + first_page + warp;
    const uint32_t wbase = smem_u32(smem) + warp * WARP_BYTES;
    const __nv_bfloat16* kbase = p.k_cache + (int64_t)kvh * p.ks_head;
    const __nv_bfloat16* vbase = p.v_cache + (int64_t)kvh * p.vs_head;

    // A block id outside the pool is never dereferenced: page 0 is read in its place and the error word is set
    // (the result of that sequence is then meaningless, but nothing faults).
    auto checked = [&](int32_t id) -> int32_t {
        if ((uint32_t)id < (uint32_t)p.num_blocks) return id;
        if (p.err) atomicOr(p.err, kErrBlockId);
        return 0;
    };
    int cache_base = 0;
    int32_t pid_cache = (lane < my_n) ? checked(__ldg(bt + lane * NWARPS)) : 0;
    const uint64_t stream_once = l2_policy_evict_first();

    auto issue = [&](int i) {
        if (i - cache_base == 32) {             // refill the per-lane page-id cache
            cache_base = i;
            pid_cache = (i + lane < my_n) ? checked(__ldg(bt + (i + lane) * NWARPS)) : 0;
        }
        const int32_t pid = __shfl_sync(0xffffffffu, pid_cache, i - cache_base);
        const int tok0 = it.kv_begin + (i * NWARPS + warp) * 16;
        const uint32_t sbase = wbase + (i % NSTAGE) * STAGE_BYTES;
        const __nv_bfloat16* kp = kbase + (int64_t)pid * p.ks_block;
        const __nv_bfloat16* vp = vbase + (int64_t)pid * p.vs_block;
#pragma unroll
        for (int r = 0; r < (16 * CPR) / 32; ++r) {
            const int id = r * 32 + lane;
            const int t = id / CPR, c = id % CPR;
            // slack slots of the last page and tokens left of a sliding window are zero-filled
            const bool ok = tok0 + t < it.kv_end && tok0 + t >= it.kv_lo;
            const int tt = ok ? t : 0;
            cp_async16_hint(sbase + tile_off<16>(t, c), kp + tt * p.ks_token + c * 8, ok ? 16 : 0, stream_once);
            cp_async16_hint(sbase + PAGE_BYTES + tile_off<16>(t, c), vp + tt * p.vs_token + c * 8, ok ? 16 : 0, stream_once);
        }
    };

    float o[KSTEPS][4];
#pragma unroll
    for (int mt = 0; mt < KSTEPS; ++mt) o[mt][0] = o[mt][1] = o[mt][2] = o[mt][3] = 0.f;
    float m_run[2] = {-INFINITY, -INFINITY};
    float l_run[2] = {0.f, 0.f};

#pragma unroll
    for (int s = 0; s < NSTAGE - 1; ++s) {
        if (s < my_n) issue(s);
        cp_async_commit();
    }

    for (int i = 0; i < my_n; ++i) {
        cp_async_wait<NSTAGE - 2>();
        __syncwarp();
        if (i + NSTAGE - 1 < my_n) issue(i + NSTAGE - 1);
        cp_async_commit();

        const uint32_t sK = wbase + (i % NSTAGE) * STAGE_BYTES;
        const uint32_t sV = sK + PAGE_BYTES;
        const int tok0 = it.kv_begin + (i * NWARPS + warp) * 16;

        // S^T = K Q^T ; two accumulators break the dependent MMA chain
        float s0[4] = {0.f, 0.f, 0.f, 0.f}, s1[4] = {0.f, 0.f, 0.f, 0.f};
        {
            const int t = (lane & 7) + ((lane >> 3) & 1) * 8;
#pragma unroll
            for (int ks = 0; ks < KSTEPS; ++ks) {
                uint32_t a[4];
                ldmatrix_x4(a, sK + tile_off<16>(t, 2 * ks + (lane >> 4)));
                if (ks & 1) mma_bf16_16816(s1, a, qf[ks][0], qf[ks][1]);
                else        mma_bf16_16816(s0, a, qf[ks][0], qf[ks][1]);
            }
        }
        float s[4];
        const int tA = tok0 + (lane >> 2);
#pragma unroll
        for (int e = 0; e < 4; ++e) {
            const int tok = tA + (e >> 1) * 8;
            const bool ok = tok < it.kv_end && tok >= it.kv_lo;
            s[e] = ok ? (s0[e] + s1[e]) * p.scale_log2 : -INFINITY;
        }
        // per-head (column) max over the 16 tokens of the page: 2 local rows, 8 lane groups
        float alpha[2];
#pragma unroll
        for (int j = 0; j < 2; ++j) {
            float mx = fmaxf(s[j], s[2 + j]);
            mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 4));
            mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 8));
            mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 16));
            const float mnew = fmaxf(m_run[j], mx);      // finite: a page always has a visible token
            alpha[j] = fast_exp2(m_run[j] - mnew);
            m_run[j] = mnew;
            s[j] = fast_exp2(s[j] - mnew);
            s[2 + j] = fast_exp2(s[2 + j] - mnew);
            l_run[j] = l_run[j] * alpha[j] + s[j] + s[2 + j];
        }
#pragma unroll
        for (int mt = 0; mt < KSTEPS; ++mt) {
            o[mt][0] *= alpha[0]; o[mt][1] *= alpha[1];
            o[mt][2] *= alpha[0]; o[mt][3] *= alpha[1];
        }
        // P^T as B operand: transpose the two 8x8 (token x head) blocks
        const uint32_t pb0 = movmatrix_trans(pack_bf16(s[0], s[1]));
        const uint32_t pb1 = movmatrix_trans(pack_bf16(s[2], s[3]));
        {
            const int t = (lane & 7) + (lane >> 4) * 8;
#pragma unroll
            for (int mt = 0; mt < KSTEPS; ++mt) {
                uint32_t a[4];
                ldmatrix_x4_trans(a, sV + tile_off<16>(t, 2 * mt + ((lane >> 3) & 1)));
                mma_bf16_16816(o[mt], a, pb0, pb1);
            }
        }
    }
    cp_async_wait<0>();

    // ---- reduce the sums over the 8 lane groups, then merge the warps through shared memory
#pragma unroll
    for (int j = 0; j < 2; ++j) {
        l_run[j] += __shfl_xor_sync(0xffffffffu, l_run[j], 4);
        l_run[j] += __shfl_xor_sync(0xffffffffu, l_run[j], 8);
        l_run[j] += __shfl_xor_sync(0xffffffffu, l_run[j], 16);
    }
    __syncthreads();                                  // every warp is done with its ring
    float* mo = reinterpret_cast<float*>(smem);       // [NWARPS][8][DP]
    float* mm = mo + NWARPS * 8 * DP;                 // [NWARPS][8]
    float* ml = mm + NWARPS * 8;                      // [NWARPS][8]
#pragma unroll
    for (int mt = 0; mt < KSTEPS; ++mt)
#pragma unroll
        for (int e = 0; e < 4; ++e) {
            const int d = mt * 16 + (lane >> 2) + (e >> 1) * 8;
            const int head = 2 * (lane & 3) + (e & 1);
            mo[(warp * 8 + head) * DP + d] = o[mt][e];
        }
    if (lane < 4) {
#pragma unroll
        for (int j = 0; j < 2; ++j) {
            mm[warp * 8 + 2 * lane + j] = m_run[j];
            ml[warp * 8 + 2 * lane + j] = l_run[j];
        }
    }
    __syncthreads();

    for (int idx = threadIdx.x; idx < G * (D / 2); idx += NWARPS * 32) {
        const int head = idx / (D / 2), d = (idx % (D / 2)) * 2;
        float M = -INFINITY;
#pragma unroll
        for (int w = 0; w < NWARPS; ++w) M = fmaxf(M, mm[w * 8 + head]);
        float L = 0.f, o0 = 0.f, o1 = 0.f;
#pragma unroll
        for (int w = 0; w < NWARPS; ++w) {
            const float f = fast_exp2(mm[w * 8 + head] - M);   // idle warps: 2^(-inf) = 0
            L += ml[w * 8 + head] * f;
            o0 += mo[(w * 8 + head) * DP + d] * f;
            o1 += mo[(w * 8 + head) * DP + d + 1] * f;
        }
        const int hq = kvh * G + head;
        if (it.part_slot < 0) {
            float shrink = 1.f;
            if (p.sinks != nullptr) shrink = join_sink(__ldg(p.sinks + hq) * kLog2e, M, L);     // the only chunk: the sink joins here
            const float inv = shrink / L;
            *reinterpret_cast<__nv_bfloat162*>(p.out + ((int64_t)it.q_row * p.Hq + hq) * D + d) =
                __floats2bfloat162_rn(o0 * inv, o1 * inv);
            if (p.lse && d == 0) p.lse[(int64_t)it.q_row * p.Hq + hq] = (M + log2f(L)) * kLn2;
        } else {
            const int64_t pr = (int64_t)it.part_slot * p.Hq + hq;
            *reinterpret_cast<float2*>(p.part_o + pr * D + d) = make_float2(o0, o1);
            if (d == 0) *reinterpret_cast<float2*>(p.part_ml + pr * 2) = make_float2(M, L);
        }
    }

    // ---- Fused combine: the CTA that finishes a (sequence, KV head) last merges that head group's partials.
    // Every CTA publishes its partial (fence), then takes a ticket; the one that draws the last ticket sees
    // all of them (fence again, L2 loads).  The merge walks the chunks in index order, so the result does
    // not depend on which CTA performs it; that CTA also puts the counter back to zero for the next launch.
    if (it.part_slot >= 0 && p.dec_counters != nullptr) {
        __shared__ int last_s;
        __threadfence();
        __syncthreads();
        uint32_t* counter = p.dec_counters + (int64_t)(it.part_slot - it.chunk) * p.Hkv + kvh;
        if (threadIdx.x == 0) last_s = (atomicAdd(counter, 1u) == (uint32_t)(it.n_chunks - 1)) ? 1 : 0;
        __syncthreads();
        if (last_s) {
            __threadfence();
            for (int idx = threadIdx.x; idx < G * (D / 4); idx += NWARPS * 32) {
                const int head = idx / (D / 4), d = (idx % (D / 4)) * 4;
                merge_partials<D>(p, it.q_row, it.part_slot - it.chunk, it.n_chunks, kvh * G + head, d, d == 0);
            }
            if (threadIdx.x == 0) *counter = 0u;
        }
    }
}

// ---------------------------------------------------------------------------------------------
// Split-K decode over an fp8 (e4m3) cache, head_dim 128: the same work items, online softmax, partials and merge as
// decode_splitk_kernel; a (page, head) of K or V is 2 KB instead of 4 KB, so the bytes to stream halve.
// The codes are turned into fp16 on the way into the MMA fragments (e4m3 -> fp16 is exact) and the MMAs run in
// fp16 with fp32 accumulation (Q is converted bf16 -> fp16 once, the probabilities are rounded to fp16); the per-head
// scales multiply the scores (k_scale) and the output (v_scale) in fp32.
// ldmatrix moves 16-bit elements and cannot gather bytes, so the fragments are loaded with plain 8- and 16-byte
// shared-memory loads, which wants each thread's elements contiguous.  Both contractions allow that, because a
// sum does not care about the order of its terms and an output row may be produced by any thread:
//   S^T = K Q^T: the 16 k-slots of MMA step ks are mapped to head-dim elements so that thread (g, c) - g = lane / 4,
//     c = lane % 4 - reads, per row, the 8 contiguous bytes d = 32 (ks / 2) + 8 c + 4 (ks % 2) + {0..3} for two steps;
//     the Q fragments use the same map.
//   O^T = V^T P^T: output row i of MMA mt is head-dim element d = 16 (i % 8) + 2 mt + (i / 8), so thread (g, c) owns
//     d in [16 g, 16 g + 16) and reads one 16-byte chunk per token for all 8 MMAs; byte pairs of two tokens are
//     brought together with one byte-permute.
__device__ __forceinline__ uint32_t e4m3x2_to_f16x2(uint32_t two_codes)
{
    uint32_t d;
    asm("{\n.reg .b16 lo;\ncvt.u16.u32 lo, %1;\ncvt.rn.f16x2.e4m3x2 %0, lo;\n}" : "=r"(d) : "r"(two_codes));
    return d;
}
__device__ __forceinline__ void mma_f16_16816(float (&c)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1)
{
    asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.f16.f16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};\n"
                 : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
                 : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}
__device__ __forceinline__ uint32_t pack_f16(float lo, float hi)
{
    __half2 v = __floats2half2_rn(lo, hi);
    return *reinterpret_cast<uint32_t*>(&v);
}
__device__ __forceinline__ uint32_t bf16x2_to_f16x2(uint32_t v)
{
    const float2 f = __bfloat1622float2(*reinterpret_cast<__nv_bfloat162*>(&v));
    return pack_f16(f.x, f.y);
}

template <int NWARPS, int NSTAGE>
__global__ void __launch_bounds__(NWARPS * 32, 2) decode_splitk_fp8_kernel(const AttnParams p)
{
    constexpr int D = 128;
    constexpr int PAGE_BYTES = 16 * D;          // one (page, head) of K or of V: 16 tokens x 128 one-byte codes
    constexpr int STAGE_BYTES = 2 * PAGE_BYTES;
    constexpr int WARP_BYTES = NSTAGE * STAGE_BYTES;
    constexpr int KSTEPS = D / 16;
    constexpr int DP = D + 4;
    extern __shared__ __align__(1024) uint8_t smem[];

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int g = lane >> 2, c = lane & 3;
    const int item_id = blockIdx.x / p.Hkv, kvh = blockIdx.x % p.Hkv;
    const DecodeItem it = p.dec_items[item_id];
    const int G = p.G;
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    const float score_scale = p.scale_log2 * __ldg(p.k_scale + kvh);
    const float out_scale = __ldg(p.v_scale + kvh);

    // ---- Q^T fragments (fp16), k-slots permuted like the K bytes: step ks, slots {2c, 2c+1 | 2c+8, 2c+9} <-> d0 + {0, 1 | 2, 3}
    uint32_t qf[KSTEPS][2];
    {
        const uint32_t* qrow = reinterpret_cast<const uint32_t*>(p.q + ((int64_t)it.q_row * p.Hq + (int64_t)kvh * G + g) * D);
#pragma unroll
        for (int ks = 0; ks < KSTEPS; ++ks) {
            const int d0 = 32 * (ks >> 1) + 8 * c + 4 * (ks & 1);
            qf[ks][0] = g < G ? bf16x2_to_f16x2(__ldg(qrow + (d0 >> 1))) : 0u;
            qf[ks][1] = g < G ? bf16x2_to_f16x2(__ldg(qrow + (d0 >> 1) + 1)) : 0u;
        }
    }

    const int first_page = it.kv_begin >> 4;
    const int n_pages = (it.kv_end - it.kv_begin + 15) >> 4;
    const int my_n = n_pages > warp ? (n_pages - warp + NWARPS - 1) / NWARPS : 0;
    const int32_t* bt = p.block_table + (int64_t)it.seq * p.max_blocks + first_page + warp;
    const uint32_t wbase = smem_u32(smem) + warp * WARP_BYTES;
    const uint8_t* kbase = reinterpret_cast<const uint8_t*>(p.k_cache) + (int64_t)kvh * p.ks_head;
    const uint8_t* vbase = reinterpret_cast<const uint8_t*>(p.v_cache) + (int64_t)kvh * p.vs_head;

    auto checked = [&](int32_t id) -> int32_t {
        if ((uint32_t)id < (uint32_t)p.num_blocks) return id;
        if (p.err) atomicOr(p.err, kErrBlockId);
        return 0;
    };
    int cache_base = 0;
    int32_t pid_cache = (lane < my_n) ? checked(__ldg(bt + lane * NWARPS)) : 0;
    const uint64_t stream_once = l2_policy_evict_first();

    // a page in shared memory: [16 tokens][128 bytes], the eight 16-byte chunks of a row XOR-swizzled by the row index
    auto issue = [&](int i) {
        if (i - cache_base == 32) {
            cache_base = i;
            pid_cache = (i + lane < my_n) ? checked(__ldg(bt + (i + lane) * NWARPS)) : 0;
        }
        const int32_t pid = __shfl_sync(0xffffffffu, pid_cache, i - cache_base);
        const int tok0 = it.kv_begin + (i * NWARPS + warp) * 16;
        const uint32_t sbase = wbase + (i % NSTAGE) * STAGE_BYTES;
        const uint8_t* kp = kbase + (int64_t)pid * p.ks_block;
        const uint8_t* vp = vbase + (int64_t)pid * p.vs_block;
#pragma unroll
        for (int r = 0; r < 4; ++r) {
            const int id = r * 32 + lane;
            const int t = id >> 3, ch = id & 7;
            const bool ok = tok0 + t < it.kv_end && tok0 + t >= it.kv_lo;     // slack slots and tokens left of a window: zero-filled
            const int tt = ok ? t : 0;
            const uint32_t off = (uint32_t)(t * 128 + ((ch ^ (t & 7)) << 4));
            cp_async16_hint(sbase + off, kp + tt * p.ks_token + ch * 16, ok ? 16 : 0, stream_once);
            cp_async16_hint(sbase + PAGE_BYTES + off, vp + tt * p.vs_token + ch * 16, ok ? 16 : 0, stream_once);
        }
    };

    float o[KSTEPS][4];
#pragma unroll
    for (int mt = 0; mt < KSTEPS; ++mt) o[mt][0] = o[mt][1] = o[mt][2] = o[mt][3] = 0.f;
    float m_run[2] = {-INFINITY, -INFINITY};
    float l_run[2] = {0.f, 0.f};

#pragma unroll
    for (int s = 0; s < NSTAGE - 1; ++s) {
        if (s < my_n) issue(s);
        cp_async_commit();
    }

    for (int i = 0; i < my_n; ++i) {
        cp_async_wait<NSTAGE - 2>();
        __syncwarp();
        if (i + NSTAGE - 1 < my_n) issue(i + NSTAGE - 1);
        cp_async_commit();

        const uint32_t sK = wbase + (i % NSTAGE) * STAGE_BYTES;
        const uint32_t sV = sK + PAGE_BYTES;
        const int tok0 = it.kv_begin + (i * NWARPS + warp) * 16;

        // S^T = K Q^T
        float s0[4] = {0.f, 0.f, 0.f, 0.f}, s1[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
        for (int m = 0; m < 4; ++m) {
            uint32_t lo[2], hi[2];                    // rows g and g + 8: bytes d = 32 m + 8 c + {0..7}
#pragma unroll
            for (int rh = 0; rh < 2; ++rh) {
                const int row = g + 8 * rh;
                const uint32_t addr = sK + row * 128 + (((2 * m + (c >> 1)) ^ (row & 7)) << 4) + 8 * (c & 1);
                asm volatile("ld.shared.v2.u32 {%0, %1}, [%2];" : "=r"(lo[rh]), "=r"(hi[rh]) : "r"(addr));
            }
            {
                const uint32_t a[4] = {e4m3x2_to_f16x2(lo[0]), e4m3x2_to_f16x2(lo[1]), e4m3x2_to_f16x2(lo[0] >> 16), e4m3x2_to_f16x2(lo[1] >> 16)};
                mma_f16_16816(s0, a, qf[2 * m][0], qf[2 * m][1]);
            }
            {
                const uint32_t a[4] = {e4m3x2_to_f16x2(hi[0]), e4m3x2_to_f16x2(hi[1]), e4m3x2_to_f16x2(hi[0] >> 16), e4m3x2_to_f16x2(hi[1] >> 16)};
                mma_f16_16816(s1, a, qf[2 * m + 1][0], qf[2 * m + 1][1]);
            }
        }
        float s[4];
        const int tA = tok0 + g;
#pragma unroll
        for (int e = 0; e < 4; ++e) {
            const int tok = tA + (e >> 1) * 8;
            const bool ok = tok < it.kv_end && tok >= it.kv_lo;
            s[e] = ok ? (s0[e] + s1[e]) * score_scale : -INFINITY;
        }
        float alpha[2];
#pragma unroll
        for (int j = 0; j < 2; ++j) {
            float mx = fmaxf(s[j], s[2 + j]);
            mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 4));
            mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 8));
            mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 16));
            const float mnew = fmaxf(m_run[j], mx);
            alpha[j] = fast_exp2(m_run[j] - mnew);
            m_run[j] = mnew;
            s[j] = fast_exp2(s[j] - mnew);
            s[2 + j] = fast_exp2(s[2 + j] - mnew);
            l_run[j] = l_run[j] * alpha[j] + s[j] + s[2 + j];
        }
#pragma unroll
        for (int mt = 0; mt < KSTEPS; ++mt) {
            o[mt][0] *= alpha[0]; o[mt][1] *= alpha[1];
            o[mt][2] *= alpha[0]; o[mt][3] *= alpha[1];
        }
        const uint32_t pb0 = movmatrix_trans(pack_f16(s[0], s[1]));
        const uint32_t pb1 = movmatrix_trans(pack_f16(s[2], s[3]));
        // O^T += V^T P^T: this thread's 16 head-dim elements of its four tokens (2c, 2c+1, 2c+8, 2c+9)
        uint32_t vw[4][4];
#pragma unroll
        for (int q4 = 0; q4 < 4; ++q4) {
            const int tk = 2 * c + (q4 & 1) + 8 * (q4 >> 1);
            const uint32_t addr = sV + tk * 128 + ((g ^ (tk & 7)) << 4);
            asm volatile("ld.shared.v4.u32 {%0, %1, %2, %3}, [%4];" : "=r"(vw[q4][0]), "=r"(vw[q4][1]), "=r"(vw[q4][2]), "=r"(vw[q4][3]) : "r"(addr));
        }
#pragma unroll
        for (int mt = 0; mt < KSTEPS; ++mt) {
            // bytes 2 mt (row d) and 2 mt + 1 (row d + 1) of both tokens of a pair -> {tokA[b], tokB[b], tokA[b+1], tokB[b+1]}
            const int w = mt >> 1;
            const uint32_t sel = (mt & 1) ? 0x7362u : 0x5140u;
            const uint32_t pa = __byte_perm(vw[0][w], vw[1][w], sel), pc = __byte_perm(vw[2][w], vw[3][w], sel);
            const uint32_t a[4] = {e4m3x2_to_f16x2(pa), e4m3x2_to_f16x2(pa >> 16), e4m3x2_to_f16x2(pc), e4m3x2_to_f16x2(pc >> 16)};
            mma_f16_16816(o[mt], a, pb0, pb1);
        }
    }
    cp_async_wait<0>();

#pragma unroll
    for (int j = 0; j < 2; ++j) {
        l_run[j] += __shfl_xor_sync(0xffffffffu, l_run[j], 4);
        l_run[j] += __shfl_xor_sync(0xffffffffu, l_run[j], 8);
        l_run[j] += __shfl_xor_sync(0xffffffffu, l_run[j], 16);
    }
    __syncthreads();
    float* mo = reinterpret_cast<float*>(smem);       // [NWARPS][8][DP]
    float* mm = mo + NWARPS * 8 * DP;
    float* ml = mm + NWARPS * 8;
#pragma unroll
    for (int mt = 0; mt < KSTEPS; ++mt)
#pragma unroll
        for (int e = 0; e < 4; ++e) {
            const int d = 16 * g + 2 * mt + (e >> 1);       // the output rows of MMA mt in this thread (see the head of the kernel)
            const int head = 2 * c + (e & 1);
            mo[(warp * 8 + head) * DP + d] = o[mt][e];
        }
    if (lane < 4) {
#pragma unroll
        for (int j = 0; j < 2; ++j) {
            mm[warp * 8 + 2 * lane + j] = m_run[j];
            ml[warp * 8 + 2 * lane + j] = l_run[j];
        }
    }
    __syncthreads();

    for (int idx = threadIdx.x; idx < G * (D / 2); idx += NWARPS * 32) {
        const int head = idx / (D / 2), d = (idx % (D / 2)) * 2;
        float M = -INFINITY;
#pragma unroll
        for (int w = 0; w < NWARPS; ++w) M = fmaxf(M, mm[w * 8 + head]);
        float L = 0.f, o0 = 0.f, o1 = 0.f;
#pragma unroll
        for (int w = 0; w < NWARPS; ++w) {
            const float f = fast_exp2(mm[w * 8 + head] - M);
            L += ml[w * 8 + head] * f;
            o0 += mo[(w * 8 + head) * DP + d] * f;
            o1 += mo[(w * 8 + head) * DP + d + 1] * f;
        }
        o0 *= out_scale;                                   // the value scale, once, in fp32
        o1 *= out_scale;
        const int hq = kvh * G + head;
        if (it.part_slot < 0) {
            float shrink = 1.f;
            if (p.sinks != nullptr) shrink = join_sink(__ldg(p.sinks + hq) * kLog2e, M, L);
            const float inv = shrink / L;
            *reinterpret_cast<__nv_bfloat162*>(p.out + ((int64_t)it.q_row * p.Hq + hq) * D + d) =
                __floats2bfloat162_rn(o0 * inv, o1 * inv);
            if (p.lse && d == 0) p.lse[(int64_t)it.q_row * p.Hq + hq] = (M + log2f(L)) * kLn2;
        } else {
            const int64_t pr = (int64_t)it.part_slot * p.Hq + hq;
            *reinterpret_cast<float2*>(p.part_o + pr * D + d) = make_float2(o0, o1);
            if (d == 0) *reinterpret_cast<float2*>(p.part_ml + pr * 2) = make_float2(M, L);
        }
    }

    if (it.part_slot >= 0 && p.dec_counters != nullptr) {
        __shared__ int last_s;
        __threadfence();
        __syncthreads();
        uint32_t* counter = p.dec_counters + (int64_t)(it.part_slot - it.chunk) * p.Hkv + kvh;
        if (threadIdx.x == 0) last_s = (atomicAdd(counter, 1u) == (uint32_t)(it.n_chunks - 1)) ? 1 : 0;
        __syncthreads();
        if (last_s) {
            __threadfence();
            for (int idx = threadIdx.x; idx < G * (D / 4); idx += NWARPS * 32) {
                const int head = idx / (D / 4), d = (idx % (D / 4)) * 4;
                merge_partials<D>(p, it.q_row, it.part_slot - it.chunk, it.n_chunks, kvh * G + head, d, d == 0);
            }
            if (threadIdx.x == 0) *counter = 0u;
        }
    }
}

// ---------------------------------------------------------------------------------------------
// Shared-prefix decode: one CTA serves one (share group, shared KV chunk, KV head) for a SET of member sequences.
// The chunk lies inside the prefix that all members have in common (same physical pages), so its K/V is streamed
// once and the members' query heads ride along as MMA columns: NCG column groups of 8, column c of the set =
// head c % G of member c / G.  Loop structure, ring and fragment layouts are those of decode_splitk_kernel; there
// is no masking at all (whole pages, every token visible to every member).  Every (member, head) gets an fp32
// partial in the member's slot for this chunk; the member's own chunks and the merge follow in the next kernel.
// Pages are fetched with the default L2 policy: other member sets of the group read them again.
template <int D, int NWARPS, int NSTAGE, int NCG>
__device__ __forceinline__ void decode_shared_cta(const AttnParams& p, const int cta)
{
    constexpr int CPR = D / 8;
    constexpr int PAGE_BYTES = 16 * D * 2;
    constexpr int STAGE_BYTES = 2 * PAGE_BYTES;
    constexpr int WARP_BYTES = NSTAGE * STAGE_BYTES;
    constexpr int KSTEPS = D / 16;
    constexpr int DP = D + 4;
    constexpr int NCOL = NCG * 8;
    extern __shared__ __align__(1024) uint8_t smem[];

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int item_id = cta / p.Hkv, kvh = cta % p.Hkv;
    const SharedDecodeItem it = p.sh_items[item_id];
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    const ShareMember* members = p.sh_members + it.member_first;
    const int G = p.G;

    // ---- Q^T fragments of every column group (B operands)
    uint32_t qf[NCG][KSTEPS][2];
#pragma unroll
    for (int cg = 0; cg < NCG; ++cg) {
        const int col = cg * 8 + (lane >> 2);
        const int m = col / G, head = col % G;
        const bool live = m < it.n_members;
        const int q_row = live ? __ldg(&members[m].q_row) : 0;
        const uint32_t* qrow = reinterpret_cast<const uint32_t*>(p.q + ((int64_t)q_row * p.Hq + (int64_t)kvh * G + head) * D);
#pragma unroll
        for (int ks = 0; ks < KSTEPS; ++ks) {
            qf[cg][ks][0] = live ? __ldg(qrow + ks * 8 + (lane & 3)) : 0u;
            qf[cg][ks][1] = live ? __ldg(qrow + ks * 8 + 4 + (lane & 3)) : 0u;
        }
    }

    const int first_page = it.kv_begin >> 4;
    const int n_pages = (it.kv_end - it.kv_begin) >> 4;
    const int my_n = n_pages > warp ? (n_pages - warp + NWARPS - 1) / NWARPS : 0;
    const int32_t* bt = p.block_table + (int64_t)it.seq * p.max_blocks + first_page + warp;
    const uint32_t wbase = smem_u32(smem) + warp * WARP_BYTES;
    const __nv_bfloat16* kbase = p.k_cache + (int64_t)kvh * p.ks_head;
    const __nv_bfloat16* vbase = p.v_cache + (int64_t)kvh * p.vs_head;

    auto checked = [&](int32_t id) -> int32_t {
        if ((uint32_t)id < (uint32_t)p.num_blocks) return id;
        if (p.err) atomicOr(p.err, kErrBlockId);
        return 0;
    };
    int cache_base = 0;
    int32_t pid_cache = (lane < my_n) ? checked(__ldg(bt + lane * NWARPS)) : 0;

    auto issue = [&](int i) {
        if (i - cache_base == 32) {
            cache_base = i;
            pid_cache = (i + lane < my_n) ? checked(__ldg(bt + (i + lane) * NWARPS)) : 0;
        }
        const int32_t pid = __shfl_sync(0xffffffffu, pid_cache, i - cache_base);
        const uint32_t sbase = wbase + (i % NSTAGE) * STAGE_BYTES;
        const __nv_bfloat16* kp = kbase + (int64_t)pid * p.ks_block;
        const __nv_bfloat16* vp = vbase + (int64_t)pid * p.vs_block;
#pragma unroll
        for (int r = 0; r < (16 * CPR) / 32; ++r) {
            const int id = r * 32 + lane;
            const int t = id / CPR, c = id % CPR;
            cp_async16(sbase + tile_off<16>(t, c), kp + t * p.ks_token + c * 8, 16);
            cp_async16(sbase + PAGE_BYTES + tile_off<16>(t, c), vp + t * p.vs_token + c * 8, 16);
        }
    };

    float o[NCG][KSTEPS][4];
    float m_run[NCG][2], l_run[NCG][2];
#pragma unroll
    for (int cg = 0; cg < NCG; ++cg) {
#pragma unroll
        for (int mt = 0; mt < KSTEPS; ++mt) o[cg][mt][0] = o[cg][mt][1] = o[cg][mt][2] = o[cg][mt][3] = 0.f;
        m_run[cg][0] = m_run[cg][1] = -INFINITY;
        l_run[cg][0] = l_run[cg][1] = 0.f;
    }

#pragma unroll
    for (int s = 0; s < NSTAGE - 1; ++s) {
        if (s < my_n) issue(s);
        cp_async_commit();
    }

    for (int i = 0; i < my_n; ++i) {
        cp_async_wait<NSTAGE - 2>();
        __syncwarp();
        if (i + NSTAGE - 1 < my_n) issue(i + NSTAGE - 1);
        cp_async_commit();

        const uint32_t sK = wbase + (i % NSTAGE) * STAGE_BYTES;
        const uint32_t sV = sK + PAGE_BYTES;

        // S^T = K Q^T: one K fragment feeds every column group
        float sacc[NCG][4];
#pragma unroll
        for (int cg = 0; cg < NCG; ++cg) sacc[cg][0] = sacc[cg][1] = sacc[cg][2] = sacc[cg][3] = 0.f;
        {
            const int t = (lane & 7) + ((lane >> 3) & 1) * 8;
#pragma unroll
            for (int ks = 0; ks < KSTEPS; ++ks) {
                uint32_t a[4];
                ldmatrix_x4(a, sK + tile_off<16>(t, 2 * ks + (lane >> 4)));
#pragma unroll
                for (int cg = 0; cg < NCG; ++cg) mma_bf16_16816(sacc[cg], a, qf[cg][ks][0], qf[cg][ks][1]);
            }
        }
        uint32_t pb[NCG][2];
#pragma unroll
        for (int cg = 0; cg < NCG; ++cg) {
            float s[4];
#pragma unroll
            for (int e = 0; e < 4; ++e) s[e] = sacc[cg][e] * p.scale_log2;
            float alpha[2];
#pragma unroll
            for (int j = 0; j < 2; ++j) {
                float mx = fmaxf(s[j], s[2 + j]);
                mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 4));
                mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 8));
                mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 16));
                const float mnew = fmaxf(m_run[cg][j], mx);
                alpha[j] = fast_exp2(m_run[cg][j] - mnew);
                m_run[cg][j] = mnew;
                s[j] = fast_exp2(s[j] - mnew);
                s[2 + j] = fast_exp2(s[2 + j] - mnew);
                l_run[cg][j] = l_run[cg][j] * alpha[j] + s[j] + s[2 + j];
            }
#pragma unroll
            for (int mt = 0; mt < KSTEPS; ++mt) {
                o[cg][mt][0] *= alpha[0]; o[cg][mt][1] *= alpha[1];
                o[cg][mt][2] *= alpha[0]; o[cg][mt][3] *= alpha[1];
            }
            pb[cg][0] = movmatrix_trans(pack_bf16(s[0], s[1]));
            pb[cg][1] = movmatrix_trans(pack_bf16(s[2], s[3]));
        }
        {
            const int t = (lane & 7) + (lane >> 4) * 8;
#pragma unroll
            for (int mt = 0; mt < KSTEPS; ++mt) {
                uint32_t a[4];
                ldmatrix_x4_trans(a, sV + tile_off<16>(t, 2 * mt + ((lane >> 3) & 1)));
#pragma unroll
                for (int cg = 0; cg < NCG; ++cg) mma_bf16_16816(o[cg][mt], a, pb[cg][0], pb[cg][1]);
            }
        }
    }
    cp_async_wait<0>();

#pragma unroll
    for (int cg = 0; cg < NCG; ++cg)
#pragma unroll
        for (int j = 0; j < 2; ++j) {
            l_run[cg][j] += __shfl_xor_sync(0xffffffffu, l_run[cg][j], 4);
            l_run[cg][j] += __shfl_xor_sync(0xffffffffu, l_run[cg][j], 8);
            l_run[cg][j] += __shfl_xor_sync(0xffffffffu, l_run[cg][j], 16);
        }
    __syncthreads();                                  // every warp is done with its ring
    float* mo = reinterpret_cast<float*>(smem);       // [NWARPS][NCOL][DP]
    float* mm = mo + NWARPS * NCOL * DP;              // [NWARPS][NCOL]
    float* ml = mm + NWARPS * NCOL;                   // [NWARPS][NCOL]
#pragma unroll
    for (int cg = 0; cg < NCG; ++cg) {
#pragma unroll
        for (int mt = 0; mt < KSTEPS; ++mt)
#pragma unroll
            for (int e = 0; e < 4; ++e) {
                const int d = mt * 16 + (lane >> 2) + (e >> 1) * 8;
                const int col = cg * 8 + 2 * (lane & 3) + (e & 1);
                mo[(warp * NCOL + col) * DP + d] = o[cg][mt][e];
            }
        if (lane < 4) {
#pragma unroll
            for (int j = 0; j < 2; ++j) {
                mm[warp * NCOL + cg * 8 + 2 * lane + j] = m_run[cg][j];
                ml[warp * NCOL + cg * 8 + 2 * lane + j] = l_run[cg][j];
            }
        }
    }
    __syncthreads();

    const int n_cols = it.n_members * G;
    for (int idx = threadIdx.x; idx < n_cols * (D / 2); idx += NWARPS * 32) {
        const int col = idx / (D / 2), d = (idx % (D / 2)) * 2;
        float M = -INFINITY;
#pragma unroll
        for (int w = 0; w < NWARPS; ++w) M = fmaxf(M, mm[w * NCOL + col]);
        float L = 0.f, o0 = 0.f, o1 = 0.f;
#pragma unroll
        for (int w = 0; w < NWARPS; ++w) {
            const float f = fast_exp2(mm[w * NCOL + col] - M);   // idle warps: 2^(-inf) = 0
            L += ml[w * NCOL + col] * f;
            o0 += mo[(w * NCOL + col) * DP + d] * f;
            o1 += mo[(w * NCOL + col) * DP + d + 1] * f;
        }
        const int m = col / G, hq = kvh * G + col % G;
        const int64_t pr = (int64_t)(__ldg(&members[m].part_first) + it.chunk) * p.Hq + hq;
        *reinterpret_cast<float2*>(p.part_o + pr * D + d) = make_float2(o0, o1);
        if (d == 0) *reinterpret_cast<float2*>(p.part_ml + pr * 2) = make_float2(M, L);
    }
    // Fused merge: this chunk counts as done for every member of the set.  The members' own chunks run in the
    // same grid; whichever CTA draws a member's last ticket - this one or one of those - merges that member's
    // partials for this KV head (all of them were published, fence + ticket, before the last ticket was drawn).
    if (p.dec_counters != nullptr) {
        __shared__ uint32_t last_mask_s;
        if (threadIdx.x == 0) last_mask_s = 0u;
        __threadfence();
        __syncthreads();
        if ((int)threadIdx.x < it.n_members) {
            uint32_t* counter = p.dec_counters + (int64_t)__ldg(&members[threadIdx.x].part_first) * p.Hkv + kvh;
            if (atomicAdd(counter, 1u) == (uint32_t)(__ldg(&members[threadIdx.x].n_chunks) - 1)) atomicOr(&last_mask_s, 1u << threadIdx.x);
        }
        __syncthreads();
        const uint32_t last_mask = last_mask_s;
        if (last_mask != 0u) {
            __threadfence();
            for (int m = 0; m < it.n_members; ++m) {
                if (!((last_mask >> m) & 1u)) continue;
                const int q_row = __ldg(&members[m].q_row), part_first = __ldg(&members[m].part_first);
                const int n_chunks = __ldg(&members[m].n_chunks);
                for (int idx = threadIdx.x; idx < G * (D / 4); idx += NWARPS * 32) {
                    const int head = idx / (D / 4), d = (idx % (D / 4)) * 4;
                    merge_partials<D>(p, q_row, part_first, n_chunks, kvh * G + head, d, d == 0);
                }
                if (threadIdx.x == 0) p.dec_counters[(int64_t)part_first * p.Hkv + kvh] = 0u;
            }
        }
    }
}

template <int D, int NWARPS, int NSTAGE>
__global__ void __launch_bounds__(NWARPS * 32, 2) decode_splitk_kernel(const AttnParams p)
{
    decode_cta<D, NWARPS, NSTAGE>(p, (int)blockIdx.x);
}

// One grid for a batch with shared prefixes: the first n_shared_ctas CTAs serve the shared chunks (longer items
// first), the rest the sequences' own chunks.  Both kinds need half an SM's shared memory, so the larger register
// footprint of the shared role costs no occupancy; batches without sharing launch decode_splitk_kernel.
template <int D, int NWARPS, int NSTAGE, int NCG>
__global__ void __launch_bounds__(NWARPS * 32, 2) decode_with_shared_kernel(const AttnParams p, const int n_shared_ctas)
{
    if ((int)blockIdx.x < n_shared_ctas) decode_shared_cta<D, NWARPS, NSTAGE, NCG>(p, (int)blockIdx.x);
    else decode_cta<D, NWARPS, NSTAGE>(p, (int)blockIdx.x - n_shared_ctas);
}

// ---------------------------------------------------------------------------------------------
// Combine: merges the partials of a split sequence in fixed chunk order (deterministic).
//   M = max_c m_c ; O = sum_c 2^(m_c - M) o_c / sum_c 2^(m_c - M) l_c ; lse = (M + log2 sum) ln 2
// (evaluated as a running merge over groups of eight chunks)
// grid (n_combine_items, Hq), D/4 threads, one float4 of the head each.
template <int D>
__global__ void __launch_bounds__(D / 4) combine_kernel(const AttnParams p)
{
    const CombineItem it = p.comb_items[blockIdx.x];
    const int hq = blockIdx.y;
    asm volatile("griddepcontrol.wait;" ::: "memory");     // the decode grid has completed and its partials are visible
    merge_partials<D>(p, it.q_row, it.part_first, it.n_chunks, hq, threadIdx.x * 4, threadIdx.x == 0);
}

// ---------------------------------------------------------------------------------------------
static constexpr int kDecWarps = 4;
static constexpr int kDecStages = 3;
#ifndef CF_FP8_STAGES
#define CF_FP8_STAGES 4
#endif
static constexpr int kDecStagesFp8 = CF_FP8_STAGES;   // pages of an fp8 cache are half the size: the ring can be deeper in the same shared memory

#ifndef CF_D64_STAGES
#define CF_D64_STAGES 4
#endif
// head_dim 64: a (page, head) is 2 KB, so four stages per warp fit in 64 KB per CTA and three CTAs on an SM (+3.5 %)
template <int D> constexpr int dec_stages() { return D == 64 ? CF_D64_STAGES : kDecStages; }

template <int D>
static size_t decode_smem_bytes()
{
    const size_t ring = (size_t)kDecWarps * dec_stages<D>() * 2 * 16 * D * 2;
    const size_t merge = (size_t)kDecWarps * 8 * (D + 4) * 4 + (size_t)kDecWarps * 8 * 4 * 2;
    return ring > merge ? ring : merge;
}

template <int D>
static cudaError_t launch_decode_t(const AttnParams& p, int n_items, cudaStream_t stream)
{
    auto kern = decode_splitk_kernel<D, kDecWarps, dec_stages<D>()>;
    const size_t smem = decode_smem_bytes<D>();
    // set once per device; two host threads racing here both set the same value
    static std::atomic<bool> configured[64];
    int dev = 0;
    cudaGetDevice(&dev);
    if (dev >= 0 && dev < 64 && !configured[dev].load(std::memory_order_acquire)) {
        cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
        if (e != cudaSuccess) return e;
        configured[dev].store(true, std::memory_order_release);
    }
    kern<<<n_items * p.Hkv, kDecWarps * 32, smem, stream>>>(p);
    return cudaGetLastError();
}

cudaError_t launch_decode_fp8(const AttnParams& p, int n_items, cudaStream_t stream)
{
    if (n_items <= 0) return cudaSuccess;
    auto kern = decode_splitk_fp8_kernel<kDecWarps, kDecStagesFp8>;
    const size_t ring = (size_t)kDecWarps * kDecStagesFp8 * 2 * 16 * 128;
    const size_t merge = (size_t)kDecWarps * 8 * (128 + 4) * 4 + (size_t)kDecWarps * 8 * 4 * 2;
    const size_t smem = ring > merge ? ring : merge;
    static std::atomic<bool> configured[64];
    int dev = 0;
    cudaGetDevice(&dev);
    if (dev >= 0 && dev < 64 && !configured[dev].load(std::memory_order_acquire)) {
        cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
        if (e != cudaSuccess) return e;
        configured[dev].store(true, std::memory_order_release);
    }
    kern<<<n_items * p.Hkv, kDecWarps * 32, smem, stream>>>(p);
    return cudaGetLastError();
}

cudaError_t launch_decode(const AttnParams& p, int head_dim, int n_items, cudaStream_t stream)
{
    if (n_items <= 0) return cudaSuccess;
    return head_dim == 128 ? launch_decode_t<128>(p, n_items, stream) : launch_decode_t<64>(p, n_items, stream);
}

template <int D>
static cudaError_t launch_decode_shared_t(const AttnParams& p, int n_shared_items, int n_items, cudaStream_t stream)
{
    constexpr int NCG = kSharedColumns / 8;
    auto kern = decode_with_shared_kernel<D, kDecWarps, kDecStages, NCG>;
    const size_t ring = (size_t)kDecWarps * kDecStages * 2 * 16 * D * 2;
    const size_t merge = (size_t)kDecWarps * kSharedColumns * (D + 4) * 4 + (size_t)kDecWarps * kSharedColumns * 4 * 2;
    const size_t smem = ring > merge ? ring : merge;
    static std::atomic<bool> configured[64];
    int dev = 0;
    cudaGetDevice(&dev);
    if (dev >= 0 && dev < 64 && !configured[dev].load(std::memory_order_acquire)) {
        cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
        if (e != cudaSuccess) return e;
        configured[dev].store(true, std::memory_order_release);
    }
    kern<<<(n_shared_items + n_items) * p.Hkv, kDecWarps * 32, smem, stream>>>(p, n_shared_items * p.Hkv);
    return cudaGetLastError();
}

cudaError_t launch_decode_with_shared(const AttnParams& p, int head_dim, int n_shared_items, int n_items, cudaStream_t stream)
{
    if (n_shared_items + n_items <= 0) return cudaSuccess;
    if (n_shared_items <= 0) return launch_decode(p, head_dim, n_items, stream);
    return head_dim == 128 ? launch_decode_shared_t<128>(p, n_shared_items, n_items, stream)
                           : launch_decode_shared_t<64>(p, n_shared_items, n_items, stream);
}

cudaError_t launch_combine(const AttnParams& p, int head_dim, int n_items, cudaStream_t stream)
{
    if (n_items <= 0) return cudaSuccess;
    dim3 grid(n_items, p.Hq);
    // programmatic dependent launch: the grid may be scheduled while the decode kernel drains; every CTA
    // executes griddepcontrol.wait before touching the partials
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid;
    cfg.blockDim = dim3(head_dim == 128 ? 32 : 16);
    cfg.dynamicSmemBytes = 0;
    cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    return head_dim == 128 ? cudaLaunchKernelEx(&cfg, combine_kernel<128>, p) : cudaLaunchKernelEx(&cfg, combine_kernel<64>, p);
}

}  // namespace cf

// =============================================================================================
// Allocation-free decode entry point.
//
// Some callers cannot allocate device memory at the point where they need attention: code that
// runs inside another framework's memory plan (every byte of the GPU already handed to a caching
// allocator), real-time loops that must not hit the driver's allocator lock, or plugins that are
// only given input and output buffers.  For them the split-K scratch (plan items and fp32
// partials) lives in a fixed array in the library's own device image instead of a cf_ctx
// workspace.  Every GPU that loads the library holds the array until the process exits.
//
// The array's name is a host-side handle in host code, not a device address; the address comes
// from cudaGetSymbolAddress, taken once per device (with that device current) on the first call.
// =============================================================================================
namespace {

constexpr size_t kStaticScratchBytes = (size_t)16 << 20;          // whole array
constexpr size_t kStaticPlanBytes = (size_t)128 << 10;            // items + combine items
constexpr int kStaticMaxSeqs = 1024;
constexpr int kStaticMaxItems = 3584;                             // 3584 x 32 B + 1024 x 12 B fits the plan region
constexpr int kMaxDevices = 64;

static __device__ __align__(256) unsigned char g_static_scratch[kStaticScratchBytes];

struct StaticSetup {
    bool ready = false;
    unsigned char* base = nullptr;   // device address of g_static_scratch on this device
    int num_sms = 0;
};
StaticSetup g_static_setup[kMaxDevices];
std::mutex g_static_setup_mutex;     // two host threads may make a device's first call at the same time

struct StaticPlan {                  // fixed capacity, lives on the caller's stack (about 124 KB)
    cf::DecodeItem items[kStaticMaxItems];
    cf::CombineItem comb[kStaticMaxSeqs];
    int n_items = 0, n_comb = 0, n_slots = 0;
};
static_assert(sizeof(cf::DecodeItem) * kStaticMaxItems + 256 + sizeof(cf::CombineItem) * kStaticMaxSeqs <= kStaticPlanBytes,
              "the plan region of the scratch array holds the largest plan");

}  // namespace

extern "C" cf_status cf_decode_attention_static(const cf_cache_desc* desc, const void* q,
                                                const void* k_cache, const void* v_cache,
                                                const int32_t* block_table, int32_t max_blocks_per_seq,
                                                const int32_t* context_len, int32_t num_seqs,
                                                void* out, float* lse, void* cuda_stream)
{
    using namespace cf;
    cf_status st = validate_desc(desc);
    if (st != CF_OK) return st;
    if (num_seqs < 0 || max_blocks_per_seq < 0) return CF_ERR_INVALID_ARG;
    if (num_seqs == 0) return CF_OK;
    if (!q || !k_cache || !v_cache || !block_table || !context_len || !out) return CF_ERR_INVALID_ARG;
    if (num_seqs > kStaticMaxSeqs) return CF_ERR_WORKSPACE;
    if (desc->kv_dtype != CF_KV_BF16) return CF_ERR_UNSUPPORTED;      // the fp8 cache is served by the context-based calls
    cudaStream_t stream = (cudaStream_t)cuda_stream;
    // The plan is copied from this function's stack frame: a captured copy node would read a dead frame on
    // every replay, so the call is refused while the stream is being captured.
    cudaStreamCaptureStatus cap = cudaStreamCaptureStatusNone;
    if (cudaStreamIsCapturing(stream, &cap) != cudaSuccess) return CF_ERR_CUDA;
    if (cap != cudaStreamCaptureStatusNone) return CF_ERR_UNSUPPORTED;

    // ---- once per device: resolve the scratch address, read the SM count (no allocation)
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return CF_ERR_CUDA;
    StaticSetup su;
    {
        std::lock_guard<std::mutex> lock(g_static_setup_mutex);
        StaticSetup& slot = g_static_setup[dev];
        if (!slot.ready) {
            int major = 0, sms = 0;
            if (cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev) != cudaSuccess) return CF_ERR_CUDA;
            if (major != 10) return CF_ERR_ARCH;
            if (cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess) return CF_ERR_CUDA;
            void* ptr = nullptr;
            if (cudaGetSymbolAddress(&ptr, g_static_scratch) != cudaSuccess || !ptr) return CF_ERR_CUDA;
            slot.base = static_cast<unsigned char*>(ptr);
            slot.num_sms = sms;
            slot.ready = true;
        }
        su = slot;
    }

    // ---- plan: the chunking routine of the context path (decode_target_pages / decode_split with the default
    // planner settings), into fixed-capacity arrays
    const int32_t B = desc->block_size, Hq = desc->num_q_heads, D = desc->head_dim;
    PlanConfig cfg;
    cfg.num_sms = su.num_sms;
    for (int32_t s = 0; s < num_seqs; ++s) {
        const int32_t lc = context_len[s];
        if (lc < 1) return CF_ERR_INVALID_ARG;                       // every sequence decodes one token
        if ((int64_t)lc > (int64_t)max_blocks_per_seq * B) return CF_ERR_OUT_OF_RANGE;
    }
    const int32_t W = desc->window_size;
    auto first_page_of = [&](int32_t lc) -> int64_t { return (W > 0 && lc > W) ? (lc - W) / B : 0; };
    const int64_t target = decode_target_pages(
        num_seqs, [&](int32_t s) -> int64_t { return (int64_t)context_len[s] - first_page_of(context_len[s]) * B; }, B,
        desc->num_kv_heads, D, cfg, false);

    StaticPlan pl;
    for (int32_t s = 0; s < num_seqs; ++s) {
        const int32_t lc = context_len[s];
        const int64_t page0 = first_page_of(lc);
        const int64_t pages = (lc + B - 1) / B - page0;
        int64_t n = 1, per = pages;
        decode_split(pages, target, cfg.decode_page_quantum, &n, &per);
        if (pl.n_items + n > kStaticMaxItems) return CF_ERR_WORKSPACE;
        int32_t first = -1;
        if (n > 1) {
            first = pl.n_slots;
            pl.comb[pl.n_comb++] = CombineItem{s, first, (int32_t)n};
            pl.n_slots += (int32_t)n;
        }
        for (int64_t c = 0; c < n; ++c) {
            DecodeItem& it = pl.items[pl.n_items++];
            it.seq = s;
            it.q_row = s;
            it.n_chunks = (int32_t)n;
            it.kv_lo = (W > 0 && lc > W) ? lc - W : 0;
            it.kv_begin = (int32_t)((page0 + c * per) * B);
            it.kv_end = (int32_t)(((page0 + (c + 1) * per) * B < lc) ? (page0 + (c + 1) * per) * B : lc);
            it.part_slot = n > 1 ? first + (int32_t)c : -1;
            it.chunk = (int32_t)c;
        }
    }
    // longest chunk first, like the context path (std::sort works in place: no temporary buffer); the order of
    // the items does not change any bit of the result
    std::sort(pl.items, pl.items + pl.n_items, [](const DecodeItem& a, const DecodeItem& b) {
        const int32_t la = a.kv_end - a.kv_begin, lb = b.kv_end - b.kv_begin;
        if (la != lb) return la > lb;
        return a.seq != b.seq ? a.seq < b.seq : a.chunk < b.chunk;
    });
    const size_t items_bytes = sizeof(DecodeItem) * (size_t)pl.n_items;
    const size_t comb_off = (items_bytes + 255) / 256 * 256;
    const size_t comb_bytes = sizeof(CombineItem) * (size_t)pl.n_comb;
    if (comb_off + comb_bytes > kStaticPlanBytes) return CF_ERR_WORKSPACE;
    const size_t part_o_bytes = ((size_t)pl.n_slots * Hq * D * sizeof(float) + 255) / 256 * 256;
    const size_t part_ml_bytes = (size_t)pl.n_slots * Hq * 2 * sizeof(float);
    if (kStaticPlanBytes + part_o_bytes + part_ml_bytes > kStaticScratchBytes) return CF_ERR_WORKSPACE;

    // Pageable-source copies: the runtime stages the bytes before returning, so the stack arrays
    // may go out of scope as soon as this function returns.
    if (cudaMemcpyAsync(su.base, pl.items, items_bytes, cudaMemcpyHostToDevice, stream) != cudaSuccess) return CF_ERR_CUDA;
    if (comb_bytes &&
        cudaMemcpyAsync(su.base + comb_off, pl.comb, comb_bytes, cudaMemcpyHostToDevice, stream) != cudaSuccess)
        return CF_ERR_CUDA;

    AttnParams p = {};
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
    p.scale_log2 = (desc->softmax_scale > 0.f ? desc->softmax_scale : 1.0f / sqrtf((float)D)) * 1.4426950408889634f;
    p.window = desc->window_size;
    p.sinks = desc->sink_logits;
    p.dec_items = reinterpret_cast<const DecodeItem*>(su.base);
    p.comb_items = reinterpret_cast<const CombineItem*>(su.base + comb_off);
    // Partials need no clearing: every slot the combine kernel reads is fully written by its decode CTA
    // in the same call.  This entry point keeps the separate combine kernel (no ticket counters), so nothing
    // in the array has to start at zero; the merge routine and its chunk order are those of the fused merge.
    p.part_o = reinterpret_cast<float*>(su.base + kStaticPlanBytes);
    p.part_ml = reinterpret_cast<float*>(su.base + kStaticPlanBytes + part_o_bytes);
    if (launch_decode(p, D, pl.n_items, stream) != cudaSuccess) return CF_ERR_CUDA;
    if (launch_combine(p, D, pl.n_comb, stream) != cudaSuccess) return CF_ERR_CUDA;
    return CF_OK;
}
