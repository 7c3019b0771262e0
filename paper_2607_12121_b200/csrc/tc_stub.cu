#include "tc.cuh"
namespace fd {
bool tc_supported(const fd_config&, std::string* why) { if (why) *why = "not built yet"; return false; }
int tc_attention_tile_rows() { return 128; }
TcPlan* tc_plan_create(const fd_config&, const fd_weights&, const TcBuffers&, std::string* err) { if (err) *err = "not built"; return nullptr; }
void tc_plan_destroy(TcPlan*) {}
cudaError_t tc_gemm(TcPlan*, TcGemmKind, int, const EpiParams&, const Control*, cudaStream_t, int*) { return cudaErrorNotSupported; }
cudaError_t tc_attention(TcPlan*, int, void*, int, int, const QTile*, int, const Control*, cudaStream_t, int*) { return cudaErrorNotSupported; }
size_t partition_scratch_bytes(int, int, int) { return 256; }
cudaError_t launch_partition(const float*, int, int, int, const int32_t*, int, int, int, int, int32_t*, int32_t*, void*, Control*, cudaStream_t, int*) { return cudaErrorNotSupported; }
}
