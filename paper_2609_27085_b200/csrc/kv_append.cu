// KV append: scatters this iteration's new K/V rows into the paged cache through the block table.
// Pure 16-byte moves, bit-exact.  One CTA per packed row; thread t moves 16-byte chunk t of the
// row's K (first half of the block) or V (second half).
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
    int threads = 2 * p.Hkv * (p.D / 8);
    threads = threads > 256 ? 256 : (threads + 31) / 32 * 32;
    kv_append_kernel<<<p.total_rows, threads, 0, stream>>>(p);
    return cudaGetLastError();
}

}  // namespace cf
