#include "common.cuh"
namespace tl {
int launch_backward(treelstm*, const int32_t*, float*, float*, float*, float*, float*, int32_t*, float*,
                    int32_t*, cudaStream_t) { return TREELSTM_ERR_UNSUPPORTED; }
}
