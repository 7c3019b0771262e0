// Shared declarations of the libflashdiff kernels (device helpers, workspace layout, launch
// prototypes).  Everything here is internal to the library.
#pragma once

#include <cuda_bf16.h>
#include <cuda_fp8.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "../../include/flashdiff.h"

namespace fd {

// ---------------------------------------------------------------------------------------------
// device-side status: word 0 = first error code (fd_status), word 1 = detail
// ---------------------------------------------------------------------------------------------
struct Control {
    int32_t status;        // first device-side error, 0 = none
    int32_t detail;
    int32_t a_total;       // number of active rows of the current step
    int32_t n_qtiles;      // number of attention query tiles of the current step
    int32_t n_qtiles2;     // ... and of double-height tiles (the work list of the CTA-pair attention kernel)
    int32_t n_text_tiles[2];   // dual stream: row tiles (128 rows / 256 rows) that hold rows of the second stream
    int32_t pad[9];
};

__device__ __forceinline__ void report(Control* c, int code, int detail) {
    if (atomicCAS(&c->status, 0, code) == 0) c->detail = detail;
}

struct QTile {            // one attention work item: `rows` compact rows of one request
    int32_t b, row0, rows, pad;
};

// ---------------------------------------------------------------------------------------------
// storage-type helpers
// ---------------------------------------------------------------------------------------------
template <typename T> __device__ __forceinline__ float to_f(T v);
template <> __device__ __forceinline__ float to_f<float>(float v) { return v; }
template <> __device__ __forceinline__ float to_f<__nv_bfloat16>(__nv_bfloat16 v) { return __bfloat162float(v); }
template <typename T> __device__ __forceinline__ T from_f(float v);
template <> __device__ __forceinline__ float from_f<float>(float v) { return v; }
template <> __device__ __forceinline__ __nv_bfloat16 from_f<__nv_bfloat16>(float v) { return __float2bfloat16_rn(v); }

// four values to E4M3 bytes (round to nearest even, saturating at 448), first value in the low byte
__device__ __forceinline__ uint32_t pack4_e4m3(float a, float b, float c, float d) {
    const uint32_t lo = __nv_cvt_float2_to_fp8x2(make_float2(a, b), __NV_SATFINITE, __NV_E4M3);
    const uint32_t hi = __nv_cvt_float2_to_fp8x2(make_float2(c, d), __NV_SATFINITE, __NV_E4M3);
    return lo | (hi << 16);
}

__device__ __forceinline__ float gelu_tanh(float a) {
    const float c = 0.7978845608028654f;
    float u = c * (a + 0.044715f * a * a * a);
    return 0.5f * a * (1.0f + tanhf(u));
}

__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    return v;
}
__device__ __forceinline__ float warp_max(float v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, o));
    return v;
}

// ---------------------------------------------------------------------------------------------
// GEMM epilogues (shared by the CUDA-core and the tensor-core kernels)
// ---------------------------------------------------------------------------------------------
enum EpiKind { EPI_QKV = 0, EPI_RESID = 1, EPI_GELU = 2 };

struct EpiParams {
    const void* bias;          // [n_out] storage type
    const int32_t* active_idx; // [A] global token id of each compact row
    int32_t N;                 // tokens per request
    int32_t H;                 // hidden width
    // EPI_QKV
    void* q;                   // [Mcap, q_ld] storage type
    int32_t q_ld;
    int32_t q_head_dim;        // 0, or the head dim when each head of Q is stored padded to q_head_pad columns
    int32_t q_head_pad;
    void* kv;                  // this block's cache [B,2,N,H] storage type
    // EPI_RESID
    float* resid;              // [Mcap,H] fp32, in/out
    const float* gate;         // mod + chunk offset; row stride 6H per request
    void* y;                   // [B*N,H] storage type or nullptr (only the last block scatters)
    // EPI_GELU
    void* out;                 // [Mcap,n_out] storage type
    int32_t out_ld;
    // dual stream: a launch finishes only the rows of one stream (tokens with label R form the second one)
    const int32_t* labels;     // [B*N] or nullptr
    int32_t R;
    int32_t group;             // -1: every row; 0: rows of the first stream only; 1: rows of the second stream only
    int32_t text_mod_off;      // offset (floats) from a request's adaLN vectors to those of the second stream
    int32_t ungated;           // EPI_RESID: `gate` is one [H] vector for every row (cross-attention passes ones)
    // FP8 operands (the kernels built for them): the accumulator is scaled by col_scale[col] * act_scale before the
    // bias; EPI_GELU then writes `out` as E4M3 bytes of value * out_inv_scale (row stride out_ld bytes)
    const float* col_scale;    // [n_out] f32
    float act_scale;
    float out_inv_scale;
    // EPI_QKV with the block variants fused (qk_head_dim != 0: 64 or 128, heads aligned with the epilogue's column
    // chunks): per head slice of a query / key row, RMS normalisation with the channel weights qn_w / kn_w [head_dim]
    // (nullptr: none) and rotation of the channel pairs by the row's angles rope_cos/sin [N, head_dim / 2] (nullptr: none)
    int32_t qk_head_dim;
    float qk_eps;
    const void* qn_w;
    const void* kn_w;
    const float* rope_cos;
    const float* rope_sin;
    // dual stream in one launch (the grouped form of the CTA-pair kernel): what the second stream's tiles use instead
    const void* qn_w2;
    const void* kn_w2;
    const void* bias2;
    const float* col_scale2;
    float act_scale2;
    float out_inv_scale2;
};

// Per-row choice of the second stream's adaLN vectors in the row kernels (labels == nullptr: single stream).
struct TextSel {
    const int32_t* labels;     // [B*N]
    int32_t R;
    long long mod_off;         // offset (floats) from the first stream's vectors to the second stream's
    float fp8_inv_text;        // FP8 operands: the second stream's 1 / activation scale (its rows are quantised with it)
};

// ---------------------------------------------------------------------------------------------
// host-side launchers (one per .cu file)
// ---------------------------------------------------------------------------------------------
struct Shape {
    int L, H, heads, dh, M, Hc;
    int B, N, R;
    int Mcap;        // capacity (rows) of the compact buffers
    float ln_eps;
};

// activity.cu
cudaError_t launch_activity(const float* z_cur, const float* z_prev, const int32_t* labels, int B, int N,
                            int D, int R, const float* eps, float* delta, int32_t* skip_count,
                            uint8_t* prev_active, float* score, float* weight, uint8_t* mask, float eta,
                            int K, double* acc_ss, int32_t* acc_cnt, Control* ctl, cudaStream_t st,
                            int* n_launch);

cudaError_t noalloc_gate(const float* z_cur, const float* z_prev, const int32_t* labels, int B, int N, int D,
                         int R, const float* eps, float eta, int K, float* delta, int32_t* skip_count,
                         uint8_t* prev_active, float* score, float* weight, uint8_t* mask, int32_t* status_out,
                         cudaStream_t st);

// compact.cu
cudaError_t launch_compact(const uint8_t* mask, const int32_t* labels, int B, int N, int R,
                           int32_t* active_idx, int32_t* cu_active, int32_t* block_counts, QTile* tiles,
                           int tile_rows, Control* ctl, cudaStream_t st, int* n_launch, QTile* tiles2 = nullptr);
// dual stream: ascending lists of the 128-row and of the 256-row tiles of the compact rows that contain at least one
// row of the second stream (label R); counts go to ctl->n_text_tiles.  lists: [cap128 + cap256] ints.
cudaError_t launch_text_tiles(const int32_t* active_idx, const int32_t* labels, int R, int rows_cap, int32_t* list128,
                              int32_t* list256, Control* ctl, cudaStream_t st, int* n_launch);

// rowops.cu
template <typename T>
cudaError_t launch_adaln(const T* cond, const T* w_ada, const T* b_ada, float* mod, int L, int B, int H,
                         int Hc, void* act_scratch, cudaStream_t st, int* n_launch);
template <typename T>
cudaError_t launch_ln_modulate(const T* x_gather, const float* resid_in, float* resid_out, T* out,
                               const int32_t* active_idx, const float* shift, const float* scale,
                               int mod_stride, int N, int H, int rows_cap, float ln_eps, const Control* ctl,
                               cudaStream_t st, int* n_launch, bool pdl, TextSel ts = TextSel{nullptr, 0, 0, 0.f},
                               float fp8_inv_scale = 0.f);   // > 0 (bf16 engine): `out` receives E4M3 bytes of value * this

// qk_variants.cu: QK-RMSNorm and rotary embedding on the fresh Q rows and the K rows just written to the cache
template <typename T>
cudaError_t launch_qk_variants(T* q, int q_ld, int q_head_stride, T* kv_block, const int32_t* active_idx, int N, int H,
                               int heads, int dh, const T* qn_w, const T* kn_w, float eps, const float* rope_cos,
                               const float* rope_sin, int rows_cap, const Control* ctl, cudaStream_t st, int* n_launch,
                               const T* qn_w_text = nullptr, const T* kn_w_text = nullptr, const int32_t* labels = nullptr,
                               int R = 0, bool pdl = false);

// simt_block.cu
template <typename T>
cudaError_t launch_simt_gemm(int kind, const T* a, int lda, const T* w, int n_out, int k, int rows_cap,
                             const EpiParams& ep, const Control* ctl, cudaStream_t st, int* n_launch);
template <typename T>
cudaError_t launch_simt_attention(const T* q, int q_ld, const T* kv, T* o, int o_ld, const QTile* tiles,
                                  int max_tiles, int N, int H, int heads, int dh, const Control* ctl,
                                  cudaStream_t st, int* n_launch, int q_head_stride = 0, const int32_t* labels = nullptr,
                                  const int32_t* active_idx = nullptr, double* region_mass = nullptr, int R = 0);
// activity.cu: the gate on the attention-mass signal
cudaError_t launch_attn_gate(const double* region_mass, const int32_t* region_sizes, int B, int R, const float* eps,
                             float eta, int K, float* rbar, float* delta, int32_t* skip_count, uint8_t* prev_active,
                             float* importance, float* weight, uint8_t* mask, cudaStream_t st, int* n_launch);

// sampler.cu
template <typename T>
cudaError_t launch_embed(const float* z, const T* w_in, const T* b_in, const T* pos, T* x, int B, int N, int D, int H,
                         cudaStream_t st, int* n_launch);
template <typename T>
cudaError_t launch_update(const float* z, const T* y, const int32_t* active_idx, const int32_t* cu_active, const float* h,
                          const T* w_out, const T* b_out, float* drift, float* z_next, int B, int N, int D, int H,
                          float ln_eps, cudaStream_t st, int* n_launch);

// partition.cu
size_t partition_scratch_bytes(int max_batch, int max_tokens, int max_regions);
cudaError_t launch_partition(const float* attn_map, int B, int N, int T, const int32_t* salient_cols,
                             int T_s, int R, int m_min, int m_max, int32_t* labels, int32_t* sizes,
                             void* scratch, Control* ctl, cudaStream_t st, int* n_launch);

}  // namespace fd
