// Block variants applied to the fresh queries and keys of a block, between the QKV projection and the
// attention: per-head RMS normalisation with a learned channel weight (QK-RMSNorm) and rotary position
// embedding (channel pairs (2i, 2i+1) rotated by the angle tabulated for the token's position).  The paper's
// evaluated models use both; the paper does not define them, the conventions are stated in the C header.
// One warp per (active row, head): it normalises and rotates that head's slice of the compact Q row and of the
// K row the projection has just written into the cache, in place, so the cache holds keys in their final form
// and rows of skipped tokens are never touched.  Memory bound: reads and writes 2 * A * H elements.
#include "common.cuh"
#include "ptx.cuh"

namespace fd {

namespace {

constexpr int QKV_THREADS = 256;

template <typename T> struct Pair;
template <> struct Pair<float> {
    static __device__ __forceinline__ float2 load(const float* p) { return *reinterpret_cast<const float2*>(p); }
    static __device__ __forceinline__ void store(float* p, float2 v) { *reinterpret_cast<float2*>(p) = v; }
};
template <> struct Pair<__nv_bfloat16> {
    static __device__ __forceinline__ float2 load(const __nv_bfloat16* p) {
        return __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(p));
    }
    static __device__ __forceinline__ void store(__nv_bfloat16* p, float2 v) {
        *reinterpret_cast<__nv_bfloat162*>(p) = __floats2bfloat162_rn(v.x, v.y);
    }
};

// slice [dh] at `x`: x <- rope(rmsnorm(x) * gamma); MAXP = pairs per lane (dh / 2 <= 32 * MAXP)
template <typename T, int MAXP>
__device__ __forceinline__ void head_slice(T* x, int dh, const T* gamma, float eps, const float* cs, const float* sn, int lane) {
    const int half = dh >> 1;
    float2 v[MAXP];
    float ss = 0.f;
#pragma unroll
    for (int i = 0; i < MAXP; ++i) {
        const int p = lane + 32 * i;
        v[i] = make_float2(0.f, 0.f);
        if (p < half) {
            v[i] = Pair<T>::load(x + 2 * p);
            ss += v[i].x * v[i].x + v[i].y * v[i].y;
        }
    }
    float r = 1.f;
    if (gamma) {
        ss = warp_sum(ss);
        r = rsqrtf(ss / (float)dh + eps);
    }
#pragma unroll
    for (int i = 0; i < MAXP; ++i) {
        const int p = lane + 32 * i;
        if (p < half) {
            float a = v[i].x, b = v[i].y;
            if (gamma) {
                const float2 g = Pair<T>::load(gamma + 2 * p);
                a = a * r * g.x;
                b = b * r * g.y;
            }
            if (cs) {
                const float c = __ldg(cs + p), s = __ldg(sn + p);
                const float ra = a * c - b * s, rb = a * s + b * c;
                a = ra;
                b = rb;
            }
            Pair<T>::store(x + 2 * p, make_float2(a, b));
        }
    }
}

template <typename T, int MAXP>
__global__ void __launch_bounds__(QKV_THREADS)
qk_variants_kernel(T* __restrict__ q, int q_ld, int q_head_stride, T* __restrict__ kv, const int32_t* __restrict__ active_idx,
                   int N, int H, int heads, int dh, const T* __restrict__ qn_w, const T* __restrict__ kn_w, float eps,
                   const float* __restrict__ rope_cos, const float* __restrict__ rope_sin, const Control* __restrict__ ctl,
                   const T* __restrict__ qn_w_text, const T* __restrict__ kn_w_text, const int32_t* __restrict__ labels, int R) {
    const int lane = threadIdx.x & 31;
    const int warps = gridDim.x * (QKV_THREADS / 32);
    ptx::pdl_wait();                              // the rows come from the projection launched just before
    const long long units = (long long)ctl->a_total * heads;
    for (long long u = (long long)blockIdx.x * (QKV_THREADS / 32) + (threadIdx.x >> 5); u < units; u += warps) {
        const int row = (int)(u / heads), h = (int)(u - (long long)row * heads);
        const int tok = active_idx[row];
        const int b = tok / N, j = tok - b * N;
        const float* cs = rope_cos ? rope_cos + (size_t)j * (dh >> 1) : nullptr;
        const float* sn = rope_cos ? rope_sin + (size_t)j * (dh >> 1) : nullptr;
        const bool text = labels && qn_w_text && labels[tok] == R;        // dual stream: the second stream's norm weights
        head_slice<T, MAXP>(q + (size_t)row * q_ld + (size_t)h * q_head_stride, dh, text ? qn_w_text : qn_w, eps, cs, sn, lane);
        head_slice<T, MAXP>(kv + (((size_t)b * 2 + 0) * N + j) * H + (size_t)h * dh, dh, text ? kn_w_text : kn_w, eps, cs, sn, lane);
    }
    ptx::pdl_trigger();
}

}  // namespace

template <typename T>
cudaError_t launch_qk_variants(T* q, int q_ld, int q_head_stride, T* kv_block, const int32_t* active_idx, int N, int H,
                               int heads, int dh, const T* qn_w, const T* kn_w, float eps, const float* rope_cos,
                               const float* rope_sin, int rows_cap, const Control* ctl, cudaStream_t st, int* n_launch,
                               const T* qn_w_text, const T* kn_w_text, const int32_t* labels, int R, bool pdl) {
    const long long max_units = (long long)rows_cap * heads;
    const int grid = (int)max(1LL, min((max_units + QKV_THREADS / 32 - 1) / (QKV_THREADS / 32), 148LL * 16));
    // launched like its neighbours (programmatic stream serialization when the engine uses it): a plainly serialized
    // launch between the projection and the attention would also break their overlap
    cudaError_t e;
    if (dh <= 64)
        e = ptx::launch_kernel(qk_variants_kernel<T, 1>, grid, QKV_THREADS, 0, st, pdl, q, q_ld, q_head_stride, kv_block, active_idx, N,
                               H, heads, dh, qn_w, kn_w, eps, rope_cos, rope_sin, ctl, qn_w_text, kn_w_text, labels, R);
    else
        e = ptx::launch_kernel(qk_variants_kernel<T, 2>, grid, QKV_THREADS, 0, st, pdl, q, q_ld, q_head_stride, kv_block, active_idx, N,
                               H, heads, dh, qn_w, kn_w, eps, rope_cos, rope_sin, ctl, qn_w_text, kn_w_text, labels, R);
    ++*n_launch;
    return e;
}

template cudaError_t launch_qk_variants<float>(float*, int, int, float*, const int32_t*, int, int, int, int, const float*,
                                               const float*, float, const float*, const float*, int, const Control*,
                                               cudaStream_t, int*, const float*, const float*, const int32_t*, int, bool);
template cudaError_t launch_qk_variants<__nv_bfloat16>(__nv_bfloat16*, int, int, __nv_bfloat16*, const int32_t*, int, int, int,
                                                       int, const __nv_bfloat16*, const __nv_bfloat16*, float, const float*,
                                                       const float*, int, const Control*, cudaStream_t, int*,
                                                       const __nv_bfloat16*, const __nv_bfloat16*, const int32_t*, int, bool);

}  // namespace fd
