// Temporary: bf16 entry points before the tcgen05 kernels land.
#include "isopo_internal.h"
namespace isopo {
isopo_status bf16_seq_grad(const void*, const void*, int64_t, int, int, const int64_t*, const int64_t*, int,
                           const WsLayout&, void*, int32_t*, cudaStream_t) { return ISOPO_ERR_UNSUPPORTED; }
isopo_status bf16_ntk(const void*, const WsLayout&, int, float*, int32_t*, cudaStream_t) { return ISOPO_ERR_UNSUPPORTED; }
isopo_status bf16_combine(const void*, const WsLayout&, int, int, int, const float*, float*, float, cudaStream_t) { return ISOPO_ERR_UNSUPPORTED; }
isopo_status bf16_gram(const void*, const void*, int64_t, int, int, const int32_t*, int, float*, int32_t*, cudaStream_t) { return ISOPO_ERR_UNSUPPORTED; }
isopo_status bf16_weight_grad(const void*, const void*, int64_t, int, int, const float*, const int32_t*, float*, float, int32_t*, cudaStream_t) { return ISOPO_ERR_UNSUPPORTED; }
}
