// Device-side helpers shared by the attention kernels: kernel parameter block and thin PTX wrappers.
#pragma once
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <cstdint>

#include "plan.h"

namespace cf {

struct AttnParams {
    const __nv_bfloat16* q;
    const __nv_bfloat16* k_cache;
    const __nv_bfloat16* v_cache;
    __nv_bfloat16* out;
    float* lse;                       // may be null
    const int32_t* block_table;
    int32_t max_blocks;
    int32_t num_blocks;               // pool size; block ids outside [0, num_blocks) are skipped and reported
    int64_t ks_block, ks_head, ks_token;
    int64_t vs_block, vs_head, vs_token;
    int32_t Hq, Hkv, G;
    float scale_log2;                 // softmax_scale * log2(e)
    int32_t window;                   // sliding window in tokens (0 = none): row at position p sees keys (p - window, p]
    const float* sinks;               // [Hq] per-head sink logits (natural-log units) or null
    const float* k_scale;             // fp8 cache: [Hkv] dequantisation scales (null: bf16 cache, or scale 1)
    const float* v_scale;
    const int32_t* context_len;       // device copies of the host arrays
    const int32_t* query_len;
    const int32_t* q_start;
    const DecodeItem* dec_items;
    const CombineItem* comb_items;
    const SharedDecodeItem* sh_items; // shared-prefix chunks and their member sets (null when the batch has none)
    const ShareMember* sh_members;
    const PrefillTcItem* pre_tc_items;
    float* part_o;                    // [slot, Hq, D] fp32 un-normalised partial outputs
    float* part_ml;                   // [slot, Hq, 2] running max (log2 domain) and sum
    uint32_t* dec_counters;           // [first slot of a split sequence, Hkv] chunks finished; null: the combine kernel merges
    float* pre_part_o;                // [row slot, D] fp32 partial rows of KV-split prefill items
    float* pre_part_ml;               // [row slot, 2]
    const PrefillCombineItem* pre_comb_items;
    uint32_t* pre_queue;              // [2] ticket counter of the persistent prefill CTAs, and how many of them have left
    uint32_t* err;                    // device error word (bits below); may be null
};

// Bits of the device error word
constexpr uint32_t kErrTimeout = 1u;      // a bounded wait expired
constexpr uint32_t kErrBlockId = 2u;      // a block-table entry in use lay outside the pool; its page was skipped

__device__ __forceinline__ uint32_t smem_u32(const void* p)
{
    return static_cast<uint32_t>(__cvta_generic_to_shared(p));
}

// 16-byte async copy global -> shared, L2 only; src_bytes = 0 zero-fills the destination.
__device__ __forceinline__ void cp_async16(uint32_t dst, const void* src, int src_bytes)
{
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;\n" ::"r"(dst), "l"(src), "r"(src_bytes) : "memory");
}
// The same with an L2 eviction policy (createpolicy): K/V pages that decode streams once are marked
// evict-first, so that they do not push the prefill kernel's re-read K/V tiles out of L2.
__device__ __forceinline__ uint64_t l2_policy_evict_first()
{
    uint64_t pol;
    asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;\n" : "=l"(pol));
    return pol;
}
__device__ __forceinline__ void cp_async16_hint(uint32_t dst, const void* src, int src_bytes, uint64_t policy)
{
    asm volatile("cp.async.cg.shared.global.L2::cache_hint [%0], [%1], 16, %2, %3;\n" ::"r"(dst), "l"(src), "r"(src_bytes), "l"(policy)
                 : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;\n" ::: "memory"); }
template <int N>
__device__ __forceinline__ void cp_async_wait()
{
    asm volatile("cp.async.wait_group %0;\n" ::"n"(N) : "memory");
}

__device__ __forceinline__ void ldmatrix_x4(uint32_t (&r)[4], uint32_t addr)
{
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];\n"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(addr));
}
__device__ __forceinline__ void ldmatrix_x4_trans(uint32_t (&r)[4], uint32_t addr)
{
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];\n"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(addr));
}
// transpose an 8x8 tile of 16-bit values held one row-pair per thread
__device__ __forceinline__ uint32_t movmatrix_trans(uint32_t a)
{
    uint32_t d;
    asm volatile("movmatrix.sync.aligned.m8n8.trans.b16 %0, %1;\n" : "=r"(d) : "r"(a));
    return d;
}
// D(16x8, f32) += A(16x16, bf16, row) * B(16x8, bf16, col)
__device__ __forceinline__ void mma_bf16_16816(float (&c)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1)
{
    asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};\n"
                 : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
                 : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}
__device__ __forceinline__ float fast_exp2(float x)
{
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;\n" : "=f"(y) : "f"(x));
    return y;
}
__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi)
{
    __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);   // .x = lo (low 16 bits), .y = hi
    return *reinterpret_cast<uint32_t*>(&v);
}

// Byte offset of 16-byte chunk `c` (0..D/8) of token row `t` inside a K/V tile stored as
// [D/64 halves][rows][64 elements] with the 16-byte chunks of every 128-byte row XOR-swizzled by
// the row index, so that 8 consecutive rows at one logical chunk hit 8 different bank groups.
template <int ROWS>
__device__ __forceinline__ uint32_t tile_off(int t, int c)
{
    return (uint32_t)((c >> 3) * (ROWS * 128) + t * 128 + (((c & 7) ^ (t & 7)) << 4));
}

constexpr float kLn2 = 0.6931471805599453f;
constexpr float kLog2e = 1.4426950408889634f;

// Joins a sink logit (log2 domain) to a softmax whose running maximum is M and un-normalised sum is L: the sink
// adds 2^(sink - M') to the sum and carries no value.  Returns the factor by which the un-normalised output
// must shrink (1 when the maximum does not move); M and L are updated.  M may be -inf only together with L = 0.
__device__ __forceinline__ float join_sink(float sink2, float& M, float& L)
{
    const float Mn = fmaxf(M, sink2);
    const float f = fast_exp2(M - Mn);
    L = L * f + fast_exp2(sink2 - Mn);
    M = Mn;
    return f;
}

}  // namespace cf
