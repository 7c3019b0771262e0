// Interface of the tensor-core engine (tcgen05 + TMEM + TMA kernels for the dense contractions).
#pragma once
#include <cuda.h>

#include <string>

#include "common.cuh"

namespace fd {

struct TcPlan;      // TMA descriptors of weights and workspace tensors, built once per context

struct TcBuffers {  // compact activation buffers inside the workspace (bf16)
    void *act, *q, *o, *g;
    void* resid;    // fp32 residual stream [Mcap, hidden]
    int Mcap, q_ld;
    void* attn_ws;  // scratch of the attention kernel: one slot per CTA for the pieces of cut items (may be null)
    int attn_slots;
};

// the last two are the cross-attention's projections (query: activations -> Q buffer; out: attention output -> residual)
enum TcGemmKind { TC_GEMM_QKV = 0, TC_GEMM_OUT = 1, TC_GEMM_FC1 = 2, TC_GEMM_FC2 = 3, TC_GEMM_XQ = 4, TC_GEMM_XO = 5 };

bool tc_supported(const fd_config& cfg, std::string* why);
bool tc_attention_supported(const fd_config& cfg);
int tc_attention_tile_rows();
bool tc_plan_pdl(TcPlan* p);                // kernels of the step are launched with programmatic stream serialization
int tc_attention_head_pad(int head_dim);   // head dim as stored in the padded Q buffer
constexpr int TC_ATTENTION_SLOTS = 256;    // CTAs the attention scratch has room for
size_t tc_attention_scratch_bytes(int head_dim);
TcPlan* tc_plan_create(const fd_config& cfg, const fd_weights& w, const TcBuffers& buf, std::string* err);
void tc_plan_destroy(TcPlan* p);
// text_pass: the second stream's weights, over the row tiles that hold rows of that stream (dual stream)
cudaError_t tc_gemm(TcPlan* p, TcGemmKind kind, int blk, const EpiParams& ep, const Control* ctl, cudaStream_t st,
                    int* n_launch, bool text_pass = false);
bool tc_plan_set_text(TcPlan* p, const fd_weights* w, const int32_t* list128, const int32_t* list256, std::string* err);
// FP8 operands: QKV, fc1 and fc2 with E4M3 weights [L, n_out, K] bytes (all nullptr: off); tc_gemm_fp8 runs one of them
// (text: the second stream's set; text_pass: the launch over the row tiles that hold rows of the second stream)
bool tc_plan_set_fp8(TcPlan* p, const void* w8_qkv, const void* w8_fc1, const void* w8_fc2, std::string* err,
                     bool text = false);
cudaError_t tc_gemm_fp8(TcPlan* p, TcGemmKind kind, int blk, const EpiParams& ep, const Control* ctl, cudaStream_t st,
                        int* n_launch, bool text_pass = false);
// dual stream in one launch (the grouped form of the CTA-pair kernel): true where it can run this projection
bool tc_plan_grouped(TcPlan* p, TcGemmKind kind);
bool tc_plan_qk_fusable(TcPlan* p);          // the QKV epilogue applies QK-RMSNorm / rotary embedding itself
cudaError_t tc_gemm_both(TcPlan* p, TcGemmKind kind, int blk, const EpiParams& ep, const Control* ctl, cudaStream_t st,
                         int* n_launch, bool fp8);
// cross-attention: tensor maps of its two [L, H, H] projection weights (both nullptr: off)
bool tc_plan_set_cross(TcPlan* p, const void* w_q, const void* w_o, std::string* err);
// region_mass (optional): [B, R] f64, receives the own-region softmax mass
cudaError_t tc_attention(TcPlan* p, int blk, void* kv_block, int B, int N, const QTile* tiles, int max_tiles,
                         const Control* ctl, cudaStream_t st, int* n_launch, const int32_t* labels = nullptr,
                         const int32_t* active_idx = nullptr, double* region_mass = nullptr, int R = 0,
                         const QTile* tiles2 = nullptr);

// CTA-pair attention kernel (head dim 128): 256-row items from the `tiles2` list
bool tc_attention_pair_supported(const fd_config& cfg);
cudaError_t tc_attention_pair_setup(int* max_clusters, int sm_count);
cudaError_t tc_attention_pair_launch(const CUtensorMap& tm_q, void* kv_block, int B, int H, void* o, int o_ld,
                                     const QTile* tiles2, int max_tiles2, int heads, int N, float scale_log2, float* split_ws,
                                     int split_slots, int max_clusters, bool may_cut, Control* ctl, cudaStream_t st, bool pdl,
                                     int* n_launch);

cudaError_t launch_bounded_wait_selftest(Control* ctl, cudaStream_t st, int* n_launch);

// host helper shared by the GEMM and attention plans: encodes a tiled bf16 tensor map
// (rank <= 4; dims / strides innermost first; strides in bytes for dims 1..rank-1)
bool encode_tmap_bf16(CUtensorMap* out, void* base, int rank, const uint64_t* dims, const uint64_t* strides_bytes,
                      const uint32_t* box, int swizzle_bytes, std::string* err);

}  // namespace fd
