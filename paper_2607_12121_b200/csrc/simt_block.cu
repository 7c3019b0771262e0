// CUDA-core GEMM and attention.  They serve the fp32 configuration (whose matrices are far too
// small for the tensor-core tiles to matter) and act as the validation path for bf16.
//
// GEMM:      C[row, n] = sum_k A[row, k] W[n, k], 64x64x16 tiles, 4x4 outputs per thread.
// Attention: each active query attends to all N keys of its request, fresh K/V for active tokens
//            and the previous step's K/V for skipped ones (paper Sec. 5, Appendix A.6); online
//            softmax in fp32, one warp per query row, 32 keys per shared-memory tile.
#include "epilogue.cuh"

namespace fd {

namespace {

constexpr int GT = 64;       // tile rows / cols
constexpr int GK = 16;       // tile depth

template <typename T, int KIND>
__global__ void __launch_bounds__(256)
simt_gemm_kernel(const T* __restrict__ a, int lda, const T* __restrict__ w, int n_out, int k_dim, EpiParams ep,
                 const Control* __restrict__ ctl) {
    __shared__ float As[GK][GT + 4];
    __shared__ float Ws[GK][GT + 4];
    const int a_total = ctl->a_total;
    const int row0 = blockIdx.y * GT, col0 = blockIdx.x * GT;
    if (row0 >= a_total) return;
    const int tid = threadIdx.x;
    const int lr = tid >> 2, lk = (tid & 3) * 4;        // loader: row lr, k offset lk..lk+3
    const int ty = tid >> 4, tx = tid & 15;             // compute: rows ty*4.., cols tx*4..
    float acc[4][4];
#pragma unroll
    for (int i = 0; i < 4; ++i)
#pragma unroll
        for (int j = 0; j < 4; ++j) acc[i][j] = 0.f;
    const T* ap = a + (size_t)(row0 + lr) * lda + lk;
    const bool w_ok = (col0 + lr) < n_out;
    const T* wp = w + (size_t)(w_ok ? col0 + lr : 0) * k_dim + lk;
    for (int k0 = 0; k0 < k_dim; k0 += GK) {
        float fa[4], fw[4] = {0.f, 0.f, 0.f, 0.f};
        load4<T>(ap + k0, fa);
        if (w_ok) load4<T>(wp + k0, fw);
#pragma unroll
        for (int i = 0; i < 4; ++i) { As[lk + i][lr] = fa[i]; Ws[lk + i][lr] = fw[i]; }
        __syncthreads();
#pragma unroll
        for (int kk = 0; kk < GK; ++kk) {
            const float4 av = *reinterpret_cast<const float4*>(&As[kk][ty * 4]);
            const float4 wv = *reinterpret_cast<const float4*>(&Ws[kk][tx * 4]);
            const float ar[4] = {av.x, av.y, av.z, av.w}, wr[4] = {wv.x, wv.y, wv.z, wv.w};
#pragma unroll
            for (int i = 0; i < 4; ++i)
#pragma unroll
                for (int j = 0; j < 4; ++j) acc[i][j] = fmaf(ar[i], wr[j], acc[i][j]);
        }
        __syncthreads();
    }
    const int col = col0 + tx * 4;
    if (col >= n_out) return;
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        const int row = row0 + ty * 4 + i;
        if (row < a_total) {
            const int tok = ep.active_idx[row];
            // dual stream: a launch finishes only the rows of its stream, with that stream's adaLN vectors
            const int text = ep.group >= 0 && ep.labels[tok] == ep.R ? 1 : 0;
            if (ep.group < 0 || text == ep.group) {
                EpiParams e2 = ep;
                if (text && e2.gate && !ep.ungated) e2.gate += ep.text_mod_off;
                epilogue4<T, KIND>(e2, row, col, tok, acc[i]);
            }
        }
    }
}

constexpr int AT_ROWS = 16;      // query rows per work item
constexpr int AT_KEYS = 32;      // keys per shared-memory tile
constexpr int AT_MAXD = 128;

template <typename T>
__global__ void __launch_bounds__(128)
simt_attention_kernel(const T* __restrict__ q, int q_ld, int q_head_stride, const T* __restrict__ kv, T* __restrict__ o,
                      int o_ld, const QTile* __restrict__ tiles, int N, int H, int dh, float sm_scale,
                      const Control* __restrict__ ctl, const int32_t* __restrict__ labels,
                      const int32_t* __restrict__ active_idx, double* __restrict__ region_mass, int R, float inv_heads) {
    __shared__ float Qs[AT_ROWS][AT_MAXD];
    __shared__ float Ks[AT_KEYS][AT_MAXD + 1];
    __shared__ float Vs[AT_KEYS][AT_MAXD];
    if ((int)blockIdx.x >= ctl->n_qtiles) return;
    const QTile tile = tiles[blockIdx.x];
    const int head = blockIdx.y;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const T* Kb = kv + ((size_t)tile.b * 2 + 0) * N * H + (size_t)head * dh;
    const T* Vb = kv + ((size_t)tile.b * 2 + 1) * N * H + (size_t)head * dh;
    for (int i = threadIdx.x; i < AT_ROWS * dh; i += 128) {
        const int r = i / dh, c = i - r * dh;
        Qs[r][c] = r < tile.rows ? to_f<T>(q[(size_t)(tile.row0 + r) * q_ld + head * q_head_stride + c]) * sm_scale : 0.f;
    }
    constexpr int RPW = AT_ROWS / 4;           // rows per warp
    constexpr int CPL = AT_MAXD / 32;          // output channels per lane
    float m[RPW], l[RPW], acc[RPW][CPL];
    // paper Sec. 4.2: the part of a query's softmax mass that falls on keys of the query's own region
    // (accumulated like l, against the same running maximum); only when region_mass is given
    float own[RPW];
    int row_lab[RPW];
#pragma unroll
    for (int r = 0; r < RPW; ++r) {
        own[r] = 0.f;
        const int lr = warp * RPW + r;
        row_lab[r] = (region_mass && lr < tile.rows) ? labels[active_idx[tile.row0 + lr]] : -1;
    }
#pragma unroll
    for (int r = 0; r < RPW; ++r) {
        m[r] = -INFINITY; l[r] = 0.f;
#pragma unroll
        for (int c = 0; c < CPL; ++c) acc[r][c] = 0.f;
    }
    for (int t0 = 0; t0 < N; t0 += AT_KEYS) {
        __syncthreads();
        for (int i = threadIdx.x; i < AT_KEYS * dh; i += 128) {
            const int t = i / dh, c = i - t * dh;
            const bool ok = (t0 + t) < N;
            Ks[t][c] = ok ? to_f<T>(Kb[(size_t)(t0 + t) * H + c]) : 0.f;
            Vs[t][c] = ok ? to_f<T>(Vb[(size_t)(t0 + t) * H + c]) : 0.f;
        }
        __syncthreads();
        const bool key_ok = (t0 + lane) < N;
        const int key_lab = (region_mass && key_ok) ? labels[(size_t)tile.b * N + t0 + lane] : -2;
#pragma unroll
        for (int r = 0; r < RPW; ++r) {
            const float* qr = Qs[warp * RPW + r];
            float s = 0.f;
            for (int c = 0; c < dh; ++c) s = fmaf(qr[c], Ks[lane][c], s);
            s = key_ok ? s : -INFINITY;
            const float m_new = fmaxf(m[r], warp_max(s));
            const float p = key_ok ? __expf(s - m_new) : 0.f;
            const float corr = __expf(m[r] - m_new);     // m = -inf on the first tile gives 0
            l[r] = l[r] * corr + warp_sum(p);
            if (region_mass) own[r] = own[r] * corr + warp_sum(key_lab == row_lab[r] ? p : 0.f);
            m[r] = m_new;
#pragma unroll
            for (int c = 0; c < CPL; ++c) acc[r][c] *= corr;
            for (int t = 0; t < AT_KEYS; ++t) {
                const float pt = __shfl_sync(0xffffffffu, p, t);
#pragma unroll
                for (int c = 0; c < CPL; ++c) {
                    const int ch = lane + 32 * c;
                    if (ch < dh) acc[r][c] = fmaf(pt, Vs[t][ch], acc[r][c]);
                }
            }
        }
    }
#pragma unroll
    for (int r = 0; r < RPW; ++r) {
        const int lr = warp * RPW + r;
        if (lr < tile.rows) {
            const float inv = 1.0f / l[r];
#pragma unroll
            for (int c = 0; c < CPL; ++c) {
                const int ch = lane + 32 * c;
                if (ch < dh) o[(size_t)(tile.row0 + lr) * o_ld + head * dh + ch] = from_f<T>(acc[r][c] * inv);
            }
            if (region_mass && lane == 0 && row_lab[r] >= 0 && row_lab[r] < R)
                atomicAdd(&region_mass[(size_t)tile.b * R + row_lab[r]], (double)(own[r] * inv * inv_heads));
        }
    }
}

}  // namespace

template <typename T>
cudaError_t launch_simt_gemm(int kind, const T* a, int lda, const T* w, int n_out, int k, int rows_cap,
                             const EpiParams& ep, const Control* ctl, cudaStream_t st, int* n_launch) {
    dim3 grid((n_out + GT - 1) / GT, (rows_cap + GT - 1) / GT);
    switch (kind) {
        case EPI_QKV: simt_gemm_kernel<T, EPI_QKV><<<grid, 256, 0, st>>>(a, lda, w, n_out, k, ep, ctl); break;
        case EPI_RESID: simt_gemm_kernel<T, EPI_RESID><<<grid, 256, 0, st>>>(a, lda, w, n_out, k, ep, ctl); break;
        default: simt_gemm_kernel<T, EPI_GELU><<<grid, 256, 0, st>>>(a, lda, w, n_out, k, ep, ctl); break;
    }
    ++*n_launch;
    return cudaGetLastError();
}

template <typename T>
cudaError_t launch_simt_attention(const T* q, int q_ld, const T* kv, T* o, int o_ld, const QTile* tiles,
                                  int max_tiles, int N, int H, int heads, int dh, const Control* ctl,
                                  cudaStream_t st, int* n_launch, int q_head_stride, const int32_t* labels,
                                  const int32_t* active_idx, double* region_mass, int R) {
    dim3 grid(max_tiles, heads);
    simt_attention_kernel<T><<<grid, 128, 0, st>>>(q, q_ld, q_head_stride > 0 ? q_head_stride : dh, kv, o, o_ld, tiles, N, H, dh,
                                                  1.0f / sqrtf((float)dh), ctl, labels, active_idx, region_mass, R,
                                                  1.0f / (float)heads);
    ++*n_launch;
    return cudaGetLastError();
}

int simt_attention_tile_rows() { return AT_ROWS; }

template cudaError_t launch_simt_gemm<float>(int, const float*, int, const float*, int, int, int, const EpiParams&,
                                             const Control*, cudaStream_t, int*);
template cudaError_t launch_simt_gemm<__nv_bfloat16>(int, const __nv_bfloat16*, int, const __nv_bfloat16*, int, int,
                                                     int, const EpiParams&, const Control*, cudaStream_t, int*);
template cudaError_t launch_simt_attention<float>(const float*, int, const float*, float*, int, const QTile*, int, int,
                                                  int, int, int, const Control*, cudaStream_t, int*, int, const int32_t*,
                                                  const int32_t*, double*, int);
template cudaError_t launch_simt_attention<__nv_bfloat16>(const __nv_bfloat16*, int, const __nv_bfloat16*,
                                                          __nv_bfloat16*, int, const QTile*, int, int, int, int, int,
                                                          const Control*, cudaStream_t, int*, int, const int32_t*,
                                                          const int32_t*, double*, int);

}  // namespace fd
