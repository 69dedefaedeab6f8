// KV append: scatters this iteration's new K/V rows into the paged cache through the block table.
// Pure 16-byte moves, bit-exact.  One CTA per packed row; thread t moves 16-byte chunk t of the
// row's K (first half of the block) or V (second half).
#include <cuda_fp16.h>

#include "kernels.h"

namespace cf {

__global__ void __launch_bounds__(256) kv_append_kernel(const AppendParams p)
{
    const int row = blockIdx.x;
    // sequence owning this row: last s with q_start[s] <= row (q_start is non-decreasing)
    int lo = 0, hi = p.num_seqs;
    while (hi - lo > 1) {
        const int mid = (lo + hi) >> 1;
        if (__ldg(p.q_start + mid) <= row) lo = mid; else hi = mid;
    }
    const int s = lo;
    const int i = row - __ldg(p.q_start + s);
    const int pos = __ldg(p.context_len + s) - __ldg(p.query_len + s) + i;
    const int64_t blk = __ldg(p.block_table + (int64_t)s * p.max_blocks + (pos >> 4));
    const int slot = pos & 15;
    if (blk < 0 || blk >= p.num_blocks) {        // never write outside the pool
        if (threadIdx.x == 0 && p.err) atomicOr(p.err, kErrBlockId);
        return;
    }

    if (p.k_scale != nullptr) {
        // fp8 cache: 16 new bf16 values -> 16 e4m3 codes per thread and step (one 16-byte store).  The quotient is an
        // IEEE fp32 division and the conversion rounds to nearest even and saturates: the code is an integer decision
        // that the CPU definition takes in the same precision.
        uint8_t* k8 = reinterpret_cast<uint8_t*>(p.k_cache);
        uint8_t* v8 = reinterpret_cast<uint8_t*>(p.v_cache);
        const int cph = p.D / 16, per = p.Hkv * cph;
        for (int t = threadIdx.x; t < 2 * per; t += blockDim.x) {
            const bool is_v = t >= per;
            const int u = is_v ? t - per : t;
            const int g = u / cph, c = u % cph;
            const float scale = __ldg((is_v ? p.v_scale : p.k_scale) + g);
            const __nv_bfloat16* src = (is_v ? p.v_new : p.k_new) + ((int64_t)row * p.Hkv + g) * p.D + c * 16;
            const uint4 in0 = __ldg(reinterpret_cast<const uint4*>(src)), in1 = __ldg(reinterpret_cast<const uint4*>(src) + 1);
            const uint32_t w[8] = {in0.x, in0.y, in0.z, in0.w, in1.x, in1.y, in1.z, in1.w};
            uint32_t packed[4];
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                uint32_t out = 0u;
#pragma unroll
                for (int h = 0; h < 2; ++h) {
                    const uint32_t pair = w[2 * i + h];
                    const float lo = __fdiv_rn(__uint_as_float(pair << 16), scale), hi = __fdiv_rn(__uint_as_float(pair & 0xffff0000u), scale);
                    uint16_t two;
                    asm("cvt.rn.satfinite.e4m3x2.f32 %0, %1, %2;" : "=h"(two) : "f"(hi), "f"(lo));     // first source -> upper byte
                    out |= (uint32_t)two << (16 * h);
                }
                packed[i] = out;
            }
            uint8_t* dst = is_v ? v8 + blk * p.vs_block + g * p.vs_head + slot * p.vs_token + c * 16
                                : k8 + blk * p.ks_block + g * p.ks_head + slot * p.ks_token + c * 16;
            *reinterpret_cast<uint4*>(dst) = make_uint4(packed[0], packed[1], packed[2], packed[3]);
        }
        return;
    }
    const int chunks_per_head = p.D / 8;
    const int per_tensor = p.Hkv * chunks_per_head;
    for (int t = threadIdx.x; t < 2 * per_tensor; t += blockDim.x) {
        const bool is_v = t >= per_tensor;
        const int u = is_v ? t - per_tensor : t;
        const int g = u / chunks_per_head, c = u % chunks_per_head;
        const int64_t src = ((int64_t)row * p.Hkv + g) * p.D + c * 8;
        if (is_v) {
            const uint4 val = __ldg(reinterpret_cast<const uint4*>(p.v_new + src));
            *reinterpret_cast<uint4*>(p.v_cache + blk * p.vs_block + g * p.vs_head + slot * p.vs_token + c * 8) = val;
        } else {
            const uint4 val = __ldg(reinterpret_cast<const uint4*>(p.k_new + src));
            *reinterpret_cast<uint4*>(p.k_cache + blk * p.ks_block + g * p.ks_head + slot * p.ks_token + c * 8) = val;
        }
    }
}

// Debug aid: counts the block-table entries that a call with these lengths would dereference and that
// fall outside [0, num_blocks).  Reads the table only; never touches the caches.
__global__ void validate_table_kernel(const int32_t* block_table, int32_t max_blocks, const int32_t* context_len,
                                      int32_t num_seqs, int32_t num_blocks, uint32_t* bad_count)
{
    const int s = blockIdx.x;
    if (s >= num_seqs) return;
    const int used = (context_len[s] + 15) >> 4;
    uint32_t bad = 0;
    for (int i = threadIdx.x; i < used && i < max_blocks; i += blockDim.x) {
        const int32_t b = block_table[(int64_t)s * max_blocks + i];
        bad += (b < 0 || b >= num_blocks) ? 1u : 0u;
    }
    if (bad) atomicAdd(bad_count, bad);
}

cudaError_t launch_validate_table(const int32_t* block_table, int32_t max_blocks, const int32_t* context_len_dev,
                                  int32_t num_seqs, int32_t num_blocks, uint32_t* bad_count, cudaStream_t stream)
{
    if (num_seqs <= 0) return cudaSuccess;
    validate_table_kernel<<<num_seqs, 128, 0, stream>>>(block_table, max_blocks, context_len_dev, num_seqs, num_blocks, bad_count);
    return cudaGetLastError();
}

cudaError_t launch_kv_append(const AppendParams& p, cudaStream_t stream)
{
    if (p.total_rows <= 0) return cudaSuccess;
    int threads = 2 * p.Hkv * (p.D / (p.k_scale != nullptr ? 16 : 8));
    threads = threads > 256 ? 256 : (threads + 31) / 32 * 32;
    kv_append_kernel<<<p.total_rows, threads, 0, stream>>>(p);
    return cudaGetLastError();
}

}  // namespace cf

namespace cf {

// fp8 cache, prefill path: one CTA per (page of a prefill sequence, KV head) expands the page's 16 x 128 e4m3 codes
// of K and of V into bf16 (exactly: every e4m3 value is a bf16 value; the per-head scales are applied later, in fp32)
// at the page's place in the staging pools, laid out [stage page, Hkv, 16, 128]; the CTA of head 0 also writes the
// staging block-table entry.  Pages left of a sliding window are not listed and never touched.
__global__ void __launch_bounds__(128) kv_dequant_gather_kernel(const AttnParams p, const StageSeq* __restrict__ seqs,
                                                                 __nv_bfloat16* __restrict__ stage_k, __nv_bfloat16* __restrict__ stage_v,
                                                                 int32_t* __restrict__ stage_table)
{
    const StageSeq sq = seqs[blockIdx.y];
    const int pg = blockIdx.x / p.Hkv, g = blockIdx.x % p.Hkv;
    if (pg >= sq.n_pages) return;
    int32_t blk = __ldg(p.block_table + (int64_t)sq.seq * p.max_blocks + sq.page0 + pg);
    if ((uint32_t)blk >= (uint32_t)p.num_blocks) {          // never dereferenced: page 0 stands in, the error word says so
        if (threadIdx.x == 0 && p.err) atomicOr(p.err, kErrBlockId);
        blk = 0;
    }
    const int spage = sq.stage_base + pg;
    if (g == 0 && threadIdx.x == 0) stage_table[(int64_t)sq.seq * p.max_blocks + sq.page0 + pg] = spage;
    const uint8_t* k8 = reinterpret_cast<const uint8_t*>(p.k_cache) + (int64_t)blk * p.ks_block + (int64_t)g * p.ks_head;
    const uint8_t* v8 = reinterpret_cast<const uint8_t*>(p.v_cache) + (int64_t)blk * p.vs_block + (int64_t)g * p.vs_head;
    // 16 tokens x 8 chunks of 16 codes = 128 chunks per tensor: one per thread
    const int t = threadIdx.x >> 3, c = threadIdx.x & 7;
#pragma unroll
    for (int which = 0; which < 2; ++which) {
        const uint4 in = __ldg(reinterpret_cast<const uint4*>((which ? v8 + t * p.vs_token : k8 + t * p.ks_token) + c * 16));
        const uint32_t w[4] = {in.x, in.y, in.z, in.w};
        uint32_t out[8];
#pragma unroll
        for (int i = 0; i < 4; ++i)
#pragma unroll
            for (int h = 0; h < 2; ++h) {
                uint32_t f16x2;
                const uint16_t two = (uint16_t)(w[i] >> (16 * h));
                asm("cvt.rn.f16x2.e4m3x2 %0, %1;" : "=r"(f16x2) : "h"(two));
                const float2 f = __half22float2(*reinterpret_cast<__half2*>(&f16x2));
                out[2 * i + h] = pack_bf16(f.x, f.y);
            }
        __nv_bfloat16* dst = (which ? stage_v : stage_k) + (((int64_t)spage * p.Hkv + g) * 16 + t) * 128 + c * 16;
        *reinterpret_cast<uint4*>(dst) = make_uint4(out[0], out[1], out[2], out[3]);
        *(reinterpret_cast<uint4*>(dst) + 1) = make_uint4(out[4], out[5], out[6], out[7]);
    }
}

cudaError_t launch_kv_dequant_gather(const AttnParams& p, const StageSeq* seqs_dev, int n_seqs, int max_pages,
                                     __nv_bfloat16* stage_k, __nv_bfloat16* stage_v, int32_t* stage_table, cudaStream_t stream)
{
    if (n_seqs <= 0 || max_pages <= 0) return cudaSuccess;
    dim3 grid((unsigned)(max_pages * p.Hkv), (unsigned)n_seqs);
    kv_dequant_gather_kernel<<<grid, 128, 0, stream>>>(p, seqs_dev, stage_k, stage_v, stage_table);
    return cudaGetLastError();
}

}  // namespace cf
