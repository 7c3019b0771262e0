// Interface of the tensor-core engine (tcgen05 + TMEM + TMA kernels for the dense contractions).
#pragma once
#include <string>

#include "common.cuh"

namespace fd {

struct TcPlan;      // TMA descriptors of weights and workspace tensors, built once per context

struct TcBuffers {  // compact activation buffers inside the workspace (bf16)
    void *act, *q, *o, *g;
    int Mcap, q_ld;
};

enum TcGemmKind { TC_GEMM_QKV = 0, TC_GEMM_OUT = 1, TC_GEMM_FC1 = 2, TC_GEMM_FC2 = 3 };

bool tc_supported(const fd_config& cfg, std::string* why);
int tc_attention_tile_rows();
TcPlan* tc_plan_create(const fd_config& cfg, const fd_weights& w, const TcBuffers& buf, std::string* err);
void tc_plan_destroy(TcPlan* p);
cudaError_t tc_gemm(TcPlan* p, TcGemmKind kind, int blk, const EpiParams& ep, const Control* ctl, cudaStream_t st,
                    int* n_launch);
cudaError_t tc_attention(TcPlan* p, int blk, void* kv_block, int B, int N, const QTile* tiles, int max_tiles,
                         const Control* ctl, cudaStream_t st, int* n_launch);

}  // namespace fd
