#include "common.cuh"
namespace optgqa {
int launch_prefill(void*, const void*, const int32_t*, int, const void*, const void*, const int32_t*, int,
                   const int32_t*, const float*, float, int, int, int, int, int, int*, cudaStream_t) {
    return OPT_GQA_ERR_SHAPE;
}
}  // namespace optgqa
