// GEMM epilogues shared by the CUDA-core and tensor-core kernels.  Each call finishes four
// consecutive output columns of one compact row:
//   EPI_QKV   bias, then Q stays compact while K and V rows are scattered into the request's cache
//             (skipped tokens' rows are never written: they keep the previous step's K/V),
//   EPI_RESID bias, adaLN gate, residual add into the fp32 stream; the last block also scatters
//             the row into y,
//   EPI_GELU  bias and tanh-GELU.
#pragma once
#include "common.cuh"

namespace fd {

template <typename T> __device__ __forceinline__ void store4(T* p, float a, float b, float c, float d);
template <> __device__ __forceinline__ void store4<float>(float* p, float a, float b, float c, float d) {
    *reinterpret_cast<float4*>(p) = make_float4(a, b, c, d);
}
template <> __device__ __forceinline__ void store4<__nv_bfloat16>(__nv_bfloat16* p, float a, float b, float c, float d) {
    const __nv_bfloat162 lo = __floats2bfloat162_rn(a, b), hi = __floats2bfloat162_rn(c, d);
    uint2 u;
    u.x = *reinterpret_cast<const uint32_t*>(&lo);
    u.y = *reinterpret_cast<const uint32_t*>(&hi);
    *reinterpret_cast<uint2*>(p) = u;
}
template <typename T> __device__ __forceinline__ void load4(const T* p, float* f);
template <> __device__ __forceinline__ void load4<float>(const float* p, float* f) {
    const float4 v = *reinterpret_cast<const float4*>(p);
    f[0] = v.x; f[1] = v.y; f[2] = v.z; f[3] = v.w;
}
template <> __device__ __forceinline__ void load4<__nv_bfloat16>(const __nv_bfloat16* p, float* f) {
    const uint2 u = *reinterpret_cast<const uint2*>(p);
    f[0] = __uint_as_float(u.x << 16); f[1] = __uint_as_float(u.x & 0xffff0000u);
    f[2] = __uint_as_float(u.y << 16); f[3] = __uint_as_float(u.y & 0xffff0000u);
}

// row: compact row (< a_total), col: first of four columns, tok: active_idx[row]
template <typename T, int KIND>
__device__ __forceinline__ void epilogue4(const EpiParams& ep, int row, int col, int tok, const float* acc) {
    float bias[4];
    load4<T>(reinterpret_cast<const T*>(ep.bias) + col, bias);
    float v[4];
#pragma unroll
    for (int i = 0; i < 4; ++i) v[i] = acc[i] + bias[i];
    if constexpr (KIND == EPI_QKV) {
        const int sec = col / ep.H, c = col - sec * ep.H;
        if (sec == 0) {
            store4<T>(reinterpret_cast<T*>(ep.q) + (size_t)row * ep.q_ld + c, v[0], v[1], v[2], v[3]);
        } else {
            const int b = tok / ep.N, j = tok - b * ep.N;
            T* dst = reinterpret_cast<T*>(ep.kv) + (((size_t)b * 2 + (sec - 1)) * ep.N + j) * ep.H + c;
            store4<T>(dst, v[0], v[1], v[2], v[3]);
        }
    } else if constexpr (KIND == EPI_RESID) {
        const int b = tok / ep.N;
        const float4 g = *reinterpret_cast<const float4*>(ep.gate + (size_t)b * 6 * ep.H + col);
        float* rp = ep.resid + (size_t)row * ep.H + col;
        float4 r = *reinterpret_cast<const float4*>(rp);
        r.x = fmaf(g.x, v[0], r.x); r.y = fmaf(g.y, v[1], r.y);
        r.z = fmaf(g.z, v[2], r.z); r.w = fmaf(g.w, v[3], r.w);
        *reinterpret_cast<float4*>(rp) = r;
        if (ep.y) store4<T>(reinterpret_cast<T*>(ep.y) + (size_t)tok * ep.H + col, r.x, r.y, r.z, r.w);
    } else {
        store4<T>(reinterpret_cast<T*>(ep.out) + (size_t)row * ep.out_ld + col, gelu_tanh(v[0]), gelu_tanh(v[1]),
                  gelu_tanh(v[2]), gelu_tanh(v[3]));
    }
}

}  // namespace fd
