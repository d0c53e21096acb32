#include "common.cuh"
namespace tl {
int pack_weights_bf16(treelstm*, cudaStream_t) { return TREELSTM_ERR_UNSUPPORTED; }
int launch_forward_bf16(treelstm*, int, const int32_t*, const int32_t*, const int32_t*, float*, float*,
                        const int32_t*, const int32_t*, const int32_t*, int, int, void*, const WsLayout&,
                        cudaStream_t) { return TREELSTM_ERR_UNSUPPORTED; }
}
