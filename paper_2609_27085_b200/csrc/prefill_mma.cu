// Chunked-prefill attention, warp-level tensor-core version (mma.sync m16n8k16).
//
// One CTA = one 64-row q tile of one prefill chunk for one query head; 4 warps x 16 rows.
// K/V tiles of 64 tokens (4 pages) are gathered through the block table with cp.async into a
// double-buffered, XOR-swizzled shared-memory tile and consumed with ldmatrix.  Row i of the chunk
// sees keys j <= P + i (P = cached prefix); the comparison is evaluated only on tiles that can
// contain a masked entry (the diagonal band and the ragged tail), tiles entirely above the
// diagonal are never visited.
#include "device_common.cuh"
#include "kernels.h"

namespace cf {

template <int D>
__global__ void __launch_bounds__(128) prefill_mma_kernel(const AttnParams p)
{
    constexpr int QT = 64, KT = 64;
    constexpr int CPR = D / 8;
    constexpr int KSTEPS = D / 16;
    constexpr int TILE_BYTES = KT * D * 2;
    constexpr int STAGE_BYTES = 2 * TILE_BYTES;
    extern __shared__ __align__(1024) uint8_t smem[];

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int item_id = blockIdx.x / p.Hq, hq = blockIdx.x % p.Hq;
    const PrefillItem it = p.pre_items[item_id];
    const int kvh = hq / p.G;
    const int Lq = __ldg(p.query_len + it.seq), Lc = __ldg(p.context_len + it.seq);
    const int prefix = Lc - Lq;
    const int kv_hi = prefix + it.row0 + it.n_rows;        // tokens [0, kv_hi) are visible to this tile
    const int n_tiles = (kv_hi + KT - 1) / KT;
    const int first_limit = prefix + it.row0;              // last key visible to the tile's first row
    const int32_t* bt = p.block_table + (int64_t)it.seq * p.max_blocks;
    const __nv_bfloat16* kbase = p.k_cache + (int64_t)kvh * p.ks_head;
    const __nv_bfloat16* vbase = p.v_cache + (int64_t)kvh * p.vs_head;
    const uint32_t sbase = smem_u32(smem);

    auto issue = [&](int kt) {
        const uint32_t st = sbase + (kt & 1) * STAGE_BYTES;
#pragma unroll
        for (int r = 0; r < (KT * CPR) / 128; ++r) {
            const int id = r * 128 + threadIdx.x;
            const int t = id / CPR, c = id % CPR;
            const int tok = kt * KT + t;
            const bool ok = tok < kv_hi;
            const int32_t pid = ok ? __ldg(bt + (tok >> 4)) : 0;
            const int slot = ok ? (tok & 15) : 0;
            cp_async16(st + tile_off<KT>(t, c), kbase + (int64_t)pid * p.ks_block + slot * p.ks_token + c * 8, ok ? 16 : 0);
            cp_async16(st + TILE_BYTES + tile_off<KT>(t, c), vbase + (int64_t)pid * p.vs_block + slot * p.vs_token + c * 8, ok ? 16 : 0);
        }
    };

    issue(0);
    cp_async_commit();

    // ---- Q fragments (A operand), rows beyond the chunk read as zero
    uint32_t qf[KSTEPS][4];
    const int r_lo = warp * 16 + (lane >> 2), r_hi = r_lo + 8;       // rows of this thread inside the tile
    {
        const uint32_t* q0 = reinterpret_cast<const uint32_t*>(p.q + ((int64_t)(it.q_row0 + r_lo) * p.Hq + hq) * D);
        const uint32_t* q1 = reinterpret_cast<const uint32_t*>(p.q + ((int64_t)(it.q_row0 + r_hi) * p.Hq + hq) * D);
        const bool ok0 = r_lo < it.n_rows, ok1 = r_hi < it.n_rows;
#pragma unroll
        for (int ks = 0; ks < KSTEPS; ++ks) {
            qf[ks][0] = ok0 ? __ldg(q0 + ks * 8 + (lane & 3)) : 0u;
            qf[ks][1] = ok1 ? __ldg(q1 + ks * 8 + (lane & 3)) : 0u;
            qf[ks][2] = ok0 ? __ldg(q0 + ks * 8 + 4 + (lane & 3)) : 0u;
            qf[ks][3] = ok1 ? __ldg(q1 + ks * 8 + 4 + (lane & 3)) : 0u;
        }
    }

    float o[D / 8][4];
#pragma unroll
    for (int n = 0; n < D / 8; ++n) o[n][0] = o[n][1] = o[n][2] = o[n][3] = 0.f;
    float m_run[2] = {-INFINITY, -INFINITY}, l_run[2] = {0.f, 0.f};
    const int lim0 = first_limit + r_lo, lim1 = first_limit + r_hi;   // last visible key of each row

    for (int kt = 0; kt < n_tiles; ++kt) {
        if (kt + 1 < n_tiles) issue(kt + 1);
        cp_async_commit();
        cp_async_wait<1>();
        __syncthreads();
        const uint32_t sK = sbase + (kt & 1) * STAGE_BYTES, sV = sK + TILE_BYTES;

        float s[KT / 8][4];
#pragma unroll
        for (int n = 0; n < KT / 8; ++n) s[n][0] = s[n][1] = s[n][2] = s[n][3] = 0.f;
#pragma unroll
        for (int ks = 0; ks < KSTEPS; ++ks) {
#pragma unroll
            for (int np = 0; np < KT / 16; ++np) {
                uint32_t b[4];
                const int t = np * 16 + (lane & 7) + ((lane >> 4) << 3);
                ldmatrix_x4(b, sK + tile_off<KT>(t, 2 * ks + ((lane >> 3) & 1)));
                mma_bf16_16816(s[2 * np], qf[ks], b[0], b[1]);
                mma_bf16_16816(s[2 * np + 1], qf[ks], b[2], b[3]);
            }
        }
        const bool need_mask = kt * KT + KT - 1 > first_limit;
        float mx0 = -INFINITY, mx1 = -INFINITY;
#pragma unroll
        for (int n = 0; n < KT / 8; ++n) {
#pragma unroll
            for (int e = 0; e < 4; ++e) {
                float v = s[n][e] * p.scale_log2;
                if (need_mask) {
                    const int j = kt * KT + n * 8 + 2 * (lane & 3) + (e & 1);
                    if (j > ((e >> 1) ? lim1 : lim0)) v = -INFINITY;
                }
                s[n][e] = v;
            }
            mx0 = fmaxf(mx0, fmaxf(s[n][0], s[n][1]));
            mx1 = fmaxf(mx1, fmaxf(s[n][2], s[n][3]));
        }
        mx0 = fmaxf(mx0, __shfl_xor_sync(0xffffffffu, mx0, 1));
        mx0 = fmaxf(mx0, __shfl_xor_sync(0xffffffffu, mx0, 2));
        mx1 = fmaxf(mx1, __shfl_xor_sync(0xffffffffu, mx1, 1));
        mx1 = fmaxf(mx1, __shfl_xor_sync(0xffffffffu, mx1, 2));
        // tile 0 always holds key 0, visible to every row, so the running max is finite from then on
        const float mn0 = fmaxf(m_run[0], mx0), mn1 = fmaxf(m_run[1], mx1);
        const float a0 = fast_exp2(m_run[0] - mn0), a1 = fast_exp2(m_run[1] - mn1);
        m_run[0] = mn0; m_run[1] = mn1;
        float sum0 = 0.f, sum1 = 0.f;
#pragma unroll
        for (int n = 0; n < KT / 8; ++n) {
            s[n][0] = fast_exp2(s[n][0] - mn0); s[n][1] = fast_exp2(s[n][1] - mn0);
            s[n][2] = fast_exp2(s[n][2] - mn1); s[n][3] = fast_exp2(s[n][3] - mn1);
            sum0 += s[n][0] + s[n][1];
            sum1 += s[n][2] + s[n][3];
        }
        l_run[0] = l_run[0] * a0 + sum0;
        l_run[1] = l_run[1] * a1 + sum1;
#pragma unroll
        for (int n = 0; n < D / 8; ++n) {
            o[n][0] *= a0; o[n][1] *= a0; o[n][2] *= a1; o[n][3] *= a1;
        }
#pragma unroll
        for (int kk = 0; kk < KT / 16; ++kk) {
            uint32_t a[4];
            a[0] = pack_bf16(s[2 * kk][0], s[2 * kk][1]);
            a[1] = pack_bf16(s[2 * kk][2], s[2 * kk][3]);
            a[2] = pack_bf16(s[2 * kk + 1][0], s[2 * kk + 1][1]);
            a[3] = pack_bf16(s[2 * kk + 1][2], s[2 * kk + 1][3]);
#pragma unroll
            for (int dp = 0; dp < D / 16; ++dp) {
                uint32_t b[4];
                const int t = kk * 16 + (lane & 7) + (((lane >> 3) & 1) << 3);
                ldmatrix_x4_trans(b, sV + tile_off<KT>(t, 2 * dp + (lane >> 4)));
                mma_bf16_16816(o[2 * dp], a, b[0], b[1]);
                mma_bf16_16816(o[2 * dp + 1], a, b[2], b[3]);
            }
        }
        __syncthreads();          // the stage is refilled two iterations from now by issue(kt + 2)
    }
    cp_async_wait<0>();

    l_run[0] += __shfl_xor_sync(0xffffffffu, l_run[0], 1);
    l_run[0] += __shfl_xor_sync(0xffffffffu, l_run[0], 2);
    l_run[1] += __shfl_xor_sync(0xffffffffu, l_run[1], 1);
    l_run[1] += __shfl_xor_sync(0xffffffffu, l_run[1], 2);
    const float inv0 = 1.f / l_run[0], inv1 = 1.f / l_run[1];
    if (r_lo < it.n_rows) {
        __nv_bfloat16* orow = p.out + ((int64_t)(it.q_row0 + r_lo) * p.Hq + hq) * D;
#pragma unroll
        for (int n = 0; n < D / 8; ++n)
            *reinterpret_cast<__nv_bfloat162*>(orow + n * 8 + 2 * (lane & 3)) = __floats2bfloat162_rn(o[n][0] * inv0, o[n][1] * inv0);
        if (p.lse && (lane & 3) == 0) p.lse[(int64_t)(it.q_row0 + r_lo) * p.Hq + hq] = (m_run[0] + log2f(l_run[0])) * kLn2;
    }
    if (r_hi < it.n_rows) {
        __nv_bfloat16* orow = p.out + ((int64_t)(it.q_row0 + r_hi) * p.Hq + hq) * D;
#pragma unroll
        for (int n = 0; n < D / 8; ++n)
            *reinterpret_cast<__nv_bfloat162*>(orow + n * 8 + 2 * (lane & 3)) = __floats2bfloat162_rn(o[n][2] * inv1, o[n][3] * inv1);
        if (p.lse && (lane & 3) == 0) p.lse[(int64_t)(it.q_row0 + r_hi) * p.Hq + hq] = (m_run[1] + log2f(l_run[1])) * kLn2;
    }
}

template <int D>
static cudaError_t launch_prefill_mma_t(const AttnParams& p, int n_items, cudaStream_t stream)
{
    auto kern = prefill_mma_kernel<D>;
    const size_t smem = (size_t)2 * 2 * 64 * D * 2;
    static bool configured[64] = {};
    int dev = 0;
    cudaGetDevice(&dev);
    if (dev >= 0 && dev < 64 && !configured[dev]) {
        cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
        if (e != cudaSuccess) return e;
        configured[dev] = true;
    }
    kern<<<n_items * p.Hq, 128, smem, stream>>>(p);
    return cudaGetLastError();
}

cudaError_t launch_prefill_mma(const AttnParams& p, int head_dim, int n_items, cudaStream_t stream)
{
    if (n_items <= 0) return cudaSuccess;
    return head_dim == 128 ? launch_prefill_mma_t<128>(p, n_items, stream) : launch_prefill_mma_t<64>(p, n_items, stream);
}

}  // namespace cf
