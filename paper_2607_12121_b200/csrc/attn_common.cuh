// Device helpers shared by the tensor-core attention kernels: register re-balancing, two-wide fp32
// arithmetic, exponentials, the plan that cuts the items of a last, partly filled round along the keys.
#pragma once
#include <cuda_bf16.h>
#include <stdint.h>

namespace fd {
namespace attn {

// Register re-balancing between warpgroups: the kernel starts with 128 registers per thread (512 threads);
// the issuing and the epilogue warpgroups give most of theirs back and the two softmax warpgroups take them.
template <int N> __device__ __forceinline__ void reg_dec() { asm volatile("setmaxnreg.dec.sync.aligned.u32 %0;" ::"n"(N)); }
template <int N> __device__ __forceinline__ void reg_inc() { asm volatile("setmaxnreg.inc.sync.aligned.u32 %0;" ::"n"(N)); }

__device__ __forceinline__ float ex2(float x) {
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}
__device__ __forceinline__ float max3(float a, float b, float c) {
    float d;
    asm("max.f32 %0, %1, %2, %3;" : "=f"(d) : "f"(a), "f"(b), "f"(c));
    return d;
}
// ---- two fp32 values per instruction (add/sub/fma .f32x2) --------------------------------------------
__device__ __forceinline__ uint64_t pair(float a, float b) {
    uint64_t r;
    asm("mov.b64 %0, {%1, %2};" : "=l"(r) : "f"(a), "f"(b));
    return r;
}
__device__ __forceinline__ void unpair(uint64_t v, float& a, float& b) { asm("mov.b64 {%0, %1}, %2;" : "=f"(a), "=f"(b) : "l"(v)); }
__device__ __forceinline__ uint64_t fma2(uint64_t a, uint64_t b, uint64_t c) {
    uint64_t d;
    asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(d) : "l"(a), "l"(b), "l"(c));
    return d;
}
__device__ __forceinline__ uint64_t add2(uint64_t a, uint64_t b) {
    uint64_t d;
    asm("add.rn.f32x2 %0, %1, %2;" : "=l"(d) : "l"(a), "l"(b));
    return d;
}
__device__ __forceinline__ uint64_t sub2(uint64_t a, uint64_t b) {
    uint64_t d;
    asm("sub.rn.f32x2 %0, %1, %2;" : "=l"(d) : "l"(a), "l"(b));
    return d;
}
// 2^x for two arguments on the FMA pipe: x = n + f with n the nearest integer, 2^f as a cubic on [-1/2, 1/2]
// (relative error 7.5e-5, far below the bf16 rounding P gets), n added into the exponent field.  Arguments
// below -125 are clamped, so a masked score gives 2^-125 instead of 0: nothing a row sum can see.
__device__ __forceinline__ uint64_t ex2_poly2(uint64_t x) {
    float xa, xb;
    unpair(x, xa, xb);
    x = pair(fmaxf(xa, -125.0f), fmaxf(xb, -125.0f));
    const uint64_t magic = pair(12582912.0f, 12582912.0f);          // 1.5 * 2^23: the sum's low mantissa bits hold n
    const uint64_t xn = add2(x, magic);
    const uint64_t f = sub2(x, sub2(xn, magic));
    uint64_t pl = fma2(pair(0.0551716648042202f, 0.0551716648042202f), f, pair(0.2426111251115799f, 0.2426111251115799f));
    pl = fma2(pl, f, pair(0.6932609677314758f, 0.6932609677314758f));
    pl = fma2(pl, f, pair(0.9999280571937561f, 0.9999280571937561f));
    float pa, pb, na, nb;
    unpair(pl, pa, pb);
    unpair(xn, na, nb);
    pa = __int_as_float(__float_as_int(pa) + (__float_as_int(na) << 23));
    pb = __int_as_float(__float_as_int(pb) + (__float_as_int(nb) << 23));
    return pair(pa, pb);
}

__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi) {
    const __nv_bfloat162 h = __floats2bfloat162_rn(lo, hi);
    return *reinterpret_cast<const uint32_t*>(&h);
}

// The running maximum of a row is only replaced (and the accumulators rescaled, which stalls the pipeline on the
// previous product) when the new maximum exceeds it by this many powers of two.  P and the accumulators are
// floating point with an 8-bit exponent, so a stale maximum costs no precision; 2^24 times the key count times
// |V| stays far inside the fp32 range.
constexpr float RESCALE_LOG2 = 24.0f;

// Work of one CTA.  Item blockIdx.x + k * gridDim.x in round k, as long as whole rounds last.  The items left over
// for a last, partly filled round are cut along the key sequence into `parts` pieces of `steps` key tiles so that
// (nearly) all CTAs take part in that round too; a piece leaves its un-normalised accumulator and row statistics
// in the CTA's scratch slot and a small kernel launched behind this one puts the pieces of an item together.
struct CutPlan { int n_rounds, n_tail, parts, steps; };
__host__ __device__ inline CutPlan cut_plan(int n_items, int n_kv, int grid, bool may_cut) {
    CutPlan c;
    c.n_rounds = n_items / grid;
    c.n_tail = n_items - c.n_rounds * grid;
    c.parts = 1;
    c.steps = n_kv;
    if (may_cut && c.n_tail > 0) {
        const int s_max = (grid / c.n_tail) < n_kv ? (grid / c.n_tail) : n_kv;
        if (s_max >= 2) {
            c.steps = (n_kv + s_max - 1) / s_max;
            c.parts = (n_kv + c.steps - 1) / c.steps;
        }
    }
    return c;
}
struct Task { int w, j0, j1, piece; };      // piece: 1 = a cut item's piece (result goes to the scratch slot)
// scratch slot of a CTA: [128 rows][DP + 4] floats: the un-normalised output row, then running maximum, row sum,
// own-region mass
__host__ __device__ inline size_t split_slot_floats(int dp) { return (size_t)128 * (dp + 4); }

}  // namespace attn
}  // namespace fd
