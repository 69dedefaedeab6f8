// Pieces shared by the two tcgen05 prefill kernels (one CTA per work item; a pair of CTAs per work item):
// tile constants, the register hand-over figures, the packed exp2 polynomial, wide stores and the item context
// that the producer hands to the other roles.
#pragma once
#include "device_common.cuh"
#include "tc05.cuh"

namespace cf {

using namespace tc;

namespace {

constexpr int QT = 128;                    // rows per q tile
constexpr int KT = 128;                    // tokens per K/V tile
constexpr int HALF_BYTES = 128 * 128;      // [128 rows][64 elements] bf16
constexpr int KV_STAGES = 2;
constexpr int NTHREADS = 384;
// Register hand-over (setmaxnreg).  The kernel launches with LAUNCH_REGS registers per thread; the
// first warpgroup shrinks to REGS_ROLE and the two softmax warpgroups grow to REGS_SOFTMAX.  A grow
// request blocks until the CTA's pool holds enough released registers, so the released amount MUST
// cover the growth or the kernel never returns; the launcher also checks the compiled register count.
#ifndef CF_REGS_ROLE
#define CF_REGS_ROLE 136
#endif
#ifndef CF_REGS_SOFTMAX
#define CF_REGS_SOFTMAX 184
#endif
constexpr int LAUNCH_REGS = 168, REGS_ROLE = CF_REGS_ROLE, REGS_SOFTMAX = CF_REGS_SOFTMAX;
static_assert(4 * (LAUNCH_REGS - REGS_ROLE) >= 8 * (REGS_SOFTMAX - LAUNCH_REGS), "setmaxnreg.inc would block forever");
__device__ __forceinline__ uint32_t lane_field(int warp) { return (uint32_t)((warp & 3) * 32) << 16; }
template <int N> __device__ __forceinline__ void reg_dec() { asm volatile("setmaxnreg.dec.sync.aligned.u32 %0;" ::"n"(N)); }
template <int N> __device__ __forceinline__ void reg_inc() { asm volatile("setmaxnreg.inc.sync.aligned.u32 %0;" ::"n"(N)); }
// 2^x for a packed pair on the FMA and integer pipes (no special-function unit): x = n + f with
// n = round(x) taken from the low mantissa bits of x + 1.5*2^23, 2^f on [-1/2, 1/2] by a degree-4
// polynomial (relative error 2.7e-6), and n added into the exponent field.  x is clamped to
// [-126, 127]: masked scores are -inf, and a score far above a stale reference maximum (tiles after
// the first run against a reference that is only raised on demand) must come out as a huge finite
// value, >= 2^127, so that the tile's row sum exceeds the rescale threshold; unclamped, the exponent
// add would wrap into the sign bit and the key would silently vanish.
__device__ __forceinline__ float2 exp2_poly2(float2 x)
{
    const float kMagic = 12582912.f;
    x.x = fminf(fmaxf(x.x, -126.f), 127.f);
    x.y = fminf(fmaxf(x.y, -126.f), 127.f);
    const float2 t = add2(x, make_float2(kMagic, kMagic));
    const float2 n = add2(t, make_float2(-kMagic, -kMagic));
    const float2 f = fma2(n, make_float2(-1.f, -1.f), x);
    float2 r = fma2(f, make_float2(0.009570097550749779f, 0.009570097550749779f), make_float2(0.05591785907745361f, 0.05591785907745361f));
    r = fma2(r, f, make_float2(0.240247443318367f, 0.240247443318367f));
    r = fma2(r, f, make_float2(0.6931217908859253f, 0.6931217908859253f));
    r = fma2(r, f, make_float2(0.9999992847442627f, 0.9999992847442627f));
    r.x = __int_as_float(__float_as_int(r.x) + (__float_as_int(t.x) << 23));
    r.y = __int_as_float(__float_as_int(r.y) + (__float_as_int(t.y) << 23));
    return r;
}
// Of the 16 pairs of a 32-column chunk, the pairs whose bit is set here take the polynomial route.
// The exp2 unit (16 results per clock per SM) is shared by both softmax warpgroups and is the busiest
// unit next to the tensor pipe; measured on the multi-item prefill case against no polynomial at all: 1/16 of
// the pairs +1.7 % (any position in the chunk), 1/8 -0.7 %, 3/16 0 %, 1/4 -8 % (the extra FMA-pipe instructions
// lengthen the in-order instruction stream of each warp).
#ifndef CF_POLY_MASK
#define CF_POLY_MASK 0x0080u
#endif
#ifndef CF_POLY_MASK_D64
#define CF_POLY_MASK_D64 0x8080u
#endif
// 32-byte store (address 32-byte aligned)
__device__ __forceinline__ void st_global_256(void* p, const uint32_t* v)
{
    asm volatile("st.global.v8.b32 [%0], {%1,%2,%3,%4,%5,%6,%7,%8};" ::"l"(p), "r"(v[0]), "r"(v[1]), "r"(v[2]), "r"(v[3]), "r"(v[4]),
                 "r"(v[5]), "r"(v[6]), "r"(v[7])
                 : "memory");
}
__device__ __forceinline__ float max3(float a, float b, float c)
{
    float d;
    asm("max.f32 %0, %1, %2, %3;" : "=f"(d) : "f"(a), "f"(b), "f"(c));
    return d;
}

}  // namespace

// What a role needs to know about the work item it is on.  The producer warp builds it and hands it
// to the other roles through a two-slot ring in shared memory.
struct ItemCtx {
    PrefillTcItem it;
    int kv_hi_t[2], n_j[2];   // per q tile: end of its visible keys; number of KV tiles of [j_begin, j_end) it takes part in
    int n_max, total_pages;
    int live, pad;            // live = 0: no more work, every role leaves
};
static_assert(sizeof(ItemCtx) % 16 == 0, "copied as 16-byte words");
__device__ __forceinline__ void derive_item(ItemCtx& c)
{
#pragma unroll
    for (int t = 0; t < 2; ++t) {
        c.kv_hi_t[t] = c.it.n_rows[t] > 0 ? c.it.prefix + c.it.row0[t] + c.it.n_rows[t] : 0;
        c.n_j[t] = max(0, min((c.kv_hi_t[t] + KT - 1) / KT, c.it.j_end) - c.it.j_begin);
    }
    c.n_max = max(c.n_j[0], c.n_j[1]);
    c.total_pages = (max(c.kv_hi_t[0], c.kv_hi_t[1]) + 15) >> 4;
    c.live = 1;
    c.pad = 0;
}


}  // namespace cf
