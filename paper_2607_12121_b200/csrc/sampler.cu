// Sampler closure around the regional step (Appendix A.1, Eq. sf-update): patch embedding of the latent
// before the block stack, final layer and latent update after it.  An active patch moves along the drift
// read off its fresh block-stack output, a skipped patch along the drift cached at its last active step.
//
// Three small kernels outside the step's hot loop:
//   embed_kernel        x[b,j,:] = z[b,j,:] W_in^T + b_in + pos[j,:]                  (writes B N H elements)
//   final_drift_kernel  drift[tok,:] = LayerNorm(y[tok,:]) W_out^T + b_out, active tokens only
//   euler_kernel        z_next = z + h[b] drift                                      (all tokens)
// The contractions are skinny (D <= 256 on one side), so they run on CUDA cores with shared-memory tiles.
#include "common.cuh"

namespace fd {

namespace {

constexpr int EMB_TOK = 32;        // tokens per CTA
constexpr int EMB_THREADS = 256;   // one output column per thread

template <typename T>
__global__ void __launch_bounds__(EMB_THREADS)
embed_kernel(const float* __restrict__ z, const T* __restrict__ w_in, const T* __restrict__ b_in,
             const T* __restrict__ pos, T* __restrict__ x, long long n_tok, int N, int D, int H) {
    extern __shared__ float s_z[];                       // [EMB_TOK][D]
    const long long t0 = (long long)blockIdx.x * EMB_TOK;
    const int nt = (int)min((long long)EMB_TOK, n_tok - t0);
    for (int i = threadIdx.x; i < nt * D; i += EMB_THREADS) s_z[i] = z[t0 * D + i];
    __syncthreads();
    const int h = blockIdx.y * EMB_THREADS + threadIdx.x;
    if (h >= H) return;
    float acc[EMB_TOK];
#pragma unroll
    for (int t = 0; t < EMB_TOK; ++t) acc[t] = 0.f;
    const T* wr = w_in + (size_t)h * D;
    for (int d = 0; d < D; d += 4) {                     // D is a multiple of 4
        const float w0 = to_f<T>(wr[d]), w1 = to_f<T>(wr[d + 1]), w2 = to_f<T>(wr[d + 2]), w3 = to_f<T>(wr[d + 3]);
#pragma unroll
        for (int t = 0; t < EMB_TOK; ++t) {
            const float4 zv = *reinterpret_cast<const float4*>(s_z + t * D + d);     // same address for the whole warp
            acc[t] = fmaf(w3, zv.w, fmaf(w2, zv.z, fmaf(w1, zv.y, fmaf(w0, zv.x, acc[t]))));
        }
    }
    const float bias = to_f<T>(b_in[h]);
#pragma unroll
    for (int t = 0; t < EMB_TOK; ++t) {
        if (t < nt) {
            const long long tok = t0 + t;
            const int j = (int)(tok % N);
            x[(size_t)tok * H + h] = from_f<T>(acc[t] + bias + to_f<T>(pos[(size_t)j * H + h]));
        }
    }
}

constexpr int FIN_ROWS = 32;       // active rows per CTA
constexpr int FIN_THREADS = 256;
constexpr int FIN_KC = 64;         // columns of y per shared-memory chunk

// Thread (ty, tx): rows 4 ty .. 4 ty + 3 of the CTA's 32, outputs tx, tx + 32, ... (D / 32 of them, at most 8).
template <typename T>
__global__ void __launch_bounds__(FIN_THREADS)
final_drift_kernel(const T* __restrict__ y, const int32_t* __restrict__ active_idx, const int32_t* __restrict__ cu_active,
                   int B, const T* __restrict__ w_out, const T* __restrict__ b_out, float* __restrict__ drift, int D,
                   int H, float ln_eps) {
    extern __shared__ float s_fin[];
    float* s_a = s_fin;                                  // [FIN_ROWS][FIN_KC + 1]  normalised rows, one chunk
    float* s_w = s_a + FIN_ROWS * (FIN_KC + 1);          // [D][FIN_KC + 1]
    float* s_mean = s_w + D * (FIN_KC + 1);              // [FIN_ROWS]
    float* s_rstd = s_mean + FIN_ROWS;
    __shared__ long long s_tok[FIN_ROWS];
    const int a_total = cu_active[B];
    const int row0 = blockIdx.x * FIN_ROWS;
    if (row0 >= a_total) return;
    const int nr = min(FIN_ROWS, a_total - row0);
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    // row statistics: warp w takes rows w, w + 8, ...
    for (int r = warp; r < FIN_ROWS; r += FIN_THREADS / 32) {
        if (r < nr) {
            const long long tok = active_idx[row0 + r];
            const T* yr = y + (size_t)tok * H;
            float sum = 0.f;
            for (int c = lane; c < H; c += 32) sum += to_f<T>(yr[c]);
            const float mean = warp_sum(sum) / (float)H;
            float sq = 0.f;
            for (int c = lane; c < H; c += 32) { const float d = to_f<T>(yr[c]) - mean; sq = fmaf(d, d, sq); }
            const float rstd = rsqrtf(warp_sum(sq) / (float)H + ln_eps);
            if (lane == 0) { s_mean[r] = mean; s_rstd[r] = rstd; s_tok[r] = tok; }
        } else if (lane == 0) {
            s_mean[r] = 0.f; s_rstd[r] = 0.f; s_tok[r] = -1;
        }
    }
    __syncthreads();
    const int ty = threadIdx.x >> 5, tx = lane;
    const int nd = D / 32 + (D % 32 ? 1 : 0);            // outputs per thread (<= 8)
    float acc[4][8];
#pragma unroll
    for (int i = 0; i < 4; ++i)
#pragma unroll
        for (int k = 0; k < 8; ++k) acc[i][k] = 0.f;
    for (int c0 = 0; c0 < H; c0 += FIN_KC) {
        const int kc = min(FIN_KC, H - c0);
        for (int i = threadIdx.x; i < FIN_ROWS * FIN_KC; i += FIN_THREADS) {
            const int r = i / FIN_KC, c = i % FIN_KC;
            float v = 0.f;
            if (r < nr && c < kc) v = (to_f<T>(y[(size_t)s_tok[r] * H + c0 + c]) - s_mean[r]) * s_rstd[r];
            s_a[r * (FIN_KC + 1) + c] = v;
        }
        for (int i = threadIdx.x; i < D * FIN_KC; i += FIN_THREADS) {
            const int d = i / FIN_KC, c = i % FIN_KC;
            s_w[d * (FIN_KC + 1) + c] = c < kc ? to_f<T>(w_out[(size_t)d * H + c0 + c]) : 0.f;
        }
        __syncthreads();
        for (int c = 0; c < FIN_KC; ++c) {
            float a[4];
#pragma unroll
            for (int i = 0; i < 4; ++i) a[i] = s_a[(4 * ty + i) * (FIN_KC + 1) + c];
#pragma unroll
            for (int k = 0; k < 8; ++k) {
                if (k < nd) {
                    const int d = tx + 32 * k;
                    const float w = d < D ? s_w[d * (FIN_KC + 1) + c] : 0.f;
#pragma unroll
                    for (int i = 0; i < 4; ++i) acc[i][k] = fmaf(a[i], w, acc[i][k]);
                }
            }
        }
        __syncthreads();
    }
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        const int r = 4 * ty + i;
        if (r < nr) {
#pragma unroll
            for (int k = 0; k < 8; ++k) {
                const int d = tx + 32 * k;
                if (k < nd && d < D) drift[(size_t)s_tok[r] * D + d] = acc[i][k] + to_f<T>(b_out[d]);
            }
        }
    }
}

__global__ void __launch_bounds__(256)
euler_kernel(const float4* __restrict__ z, const float4* __restrict__ drift, const float* __restrict__ h,
             float4* __restrict__ z_next, long long n_vec, long long vec_per_request) {
    for (long long i = blockIdx.x * (long long)blockDim.x + threadIdx.x; i < n_vec; i += (long long)gridDim.x * blockDim.x) {
        const float hb = __ldg(h + i / vec_per_request);
        const float4 a = z[i], d = drift[i];
        z_next[i] = make_float4(fmaf(hb, d.x, a.x), fmaf(hb, d.y, a.y), fmaf(hb, d.z, a.z), fmaf(hb, d.w, a.w));
    }
}

}  // namespace

template <typename T>
cudaError_t launch_embed(const float* z, const T* w_in, const T* b_in, const T* pos, T* x, int B, int N, int D, int H,
                         cudaStream_t st, int* n_launch) {
    const long long n_tok = (long long)B * N;
    dim3 grid((unsigned)((n_tok + EMB_TOK - 1) / EMB_TOK), (unsigned)((H + EMB_THREADS - 1) / EMB_THREADS));
    embed_kernel<T><<<grid, EMB_THREADS, (size_t)EMB_TOK * D * sizeof(float), st>>>(z, w_in, b_in, pos, x, n_tok, N, D, H);
    ++*n_launch;
    return cudaGetLastError();
}

template <typename T>
cudaError_t launch_update(const float* z, const T* y, const int32_t* active_idx, const int32_t* cu_active, const float* h,
                          const T* w_out, const T* b_out, float* drift, float* z_next, int B, int N, int D, int H,
                          float ln_eps, cudaStream_t st, int* n_launch) {
    const size_t smem = ((size_t)FIN_ROWS * (FIN_KC + 1) + (size_t)D * (FIN_KC + 1) + 2 * FIN_ROWS) * sizeof(float);
    cudaError_t e = cudaFuncSetAttribute(final_drift_kernel<T>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
    const long long rows_cap = (long long)B * N;
    final_drift_kernel<T><<<(unsigned)((rows_cap + FIN_ROWS - 1) / FIN_ROWS), FIN_THREADS, smem, st>>>(
        y, active_idx, cu_active, B, w_out, b_out, drift, D, H, ln_eps);
    ++*n_launch;
    e = cudaGetLastError();
    if (e != cudaSuccess) return e;
    const long long n_vec = rows_cap * D / 4;
    const long long want = (n_vec + 255) / 256;
    const int grid = (int)(want < 148 * 8 ? want : 148 * 8);
    euler_kernel<<<max(grid, 1), 256, 0, st>>>(reinterpret_cast<const float4*>(z), reinterpret_cast<const float4*>(drift), h,
                                               reinterpret_cast<float4*>(z_next), n_vec, (long long)N * D / 4);
    ++*n_launch;
    return cudaGetLastError();
}

template cudaError_t launch_embed<float>(const float*, const float*, const float*, const float*, float*, int, int, int, int,
                                         cudaStream_t, int*);
template cudaError_t launch_embed<__nv_bfloat16>(const float*, const __nv_bfloat16*, const __nv_bfloat16*, const __nv_bfloat16*,
                                                 __nv_bfloat16*, int, int, int, int, cudaStream_t, int*);
template cudaError_t launch_update<float>(const float*, const float*, const int32_t*, const int32_t*, const float*, const float*,
                                          const float*, float*, float*, int, int, int, int, float, cudaStream_t, int*);
template cudaError_t launch_update<__nv_bfloat16>(const float*, const __nv_bfloat16*, const int32_t*, const int32_t*, const float*,
                                                  const __nv_bfloat16*, const __nv_bfloat16*, float*, float*, int, int, int, int,
                                                  float, cudaStream_t, int*);

}  // namespace fd
