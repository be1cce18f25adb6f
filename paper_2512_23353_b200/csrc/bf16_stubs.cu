// Temporary: bf16 entry points before their tcgen05 kernels land.
#include "isopo_internal.h"
namespace isopo {
isopo_status bf16_gram(const void*, const void*, int64_t, int, int, const int32_t*, int, float*, int32_t*, cudaStream_t) { return ISOPO_ERR_UNSUPPORTED; }
isopo_status bf16_weight_grad(const void*, const void*, int64_t, int, int, const float*, const int32_t*, float*, float, int32_t*, cudaStream_t) { return ISOPO_ERR_UNSUPPORTED; }
}
