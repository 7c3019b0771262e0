// Tensor-core attention of the active queries against all keys of their request.
#include "ptx.cuh"
#include "tc.cuh"

namespace fd {

bool tc_attention_supported(const fd_config&) { return false; }
int tc_attention_tile_rows() { return 128; }
void* tc_attention_plan_create(const fd_config&, const TcBuffers&, std::string* err) {
    if (err) *err = "no tensor-core attention kernel for this configuration";
    return nullptr;
}
void tc_attention_plan_destroy(void*) {}
cudaError_t tc_attention(TcPlan*, int, void*, int, int, const QTile*, int, const Control*, cudaStream_t, int*) {
    return cudaErrorNotSupported;
}

}  // namespace fd
