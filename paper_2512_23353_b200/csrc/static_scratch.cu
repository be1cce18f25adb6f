// isopo_layer_gram_static: the Gram-route NTK for callers that cannot allocate device memory.
//
// Some hosts of this library are not allowed to call cudaMalloc at the point where a layer's
// hook fires: code running under a framework whose caching allocator owns all device memory and
// forbids raw allocations, a hook that runs while that allocator is locked or while allocation is
// being traced, or an embedder that has handed the whole device to another memory pool.  For them
// this entry point brings its own scratch: a fixed array that lives in the library's device image,
// so loading the library on a GPU reserves kStaticScratchBytes there until the process exits.
//
// The array's name is only meaningful in device code.  On the host it is a stand-in symbol, never
// an address a kernel may be given, so the device address is looked up with cudaGetSymbolAddress
// once per device (with that device current) and that pointer is what the kernels receive.
#include "isopo_internal.h"

namespace isopo {

namespace {

constexpr int64_t kStaticMaxT = ISOPO_STATIC_MAX_TOKENS;
constexpr int kStaticMaxB = ISOPO_STATIC_MAX_SEQS;
constexpr int kMaxDevices = 64;

// layout inside the array: offsets | token -> sequence map | float64 K accumulators (float32 route)
constexpr size_t kOffBytes = 4096;                                     // int64 [kStaticMaxB + 1], padded
constexpr size_t kTokseqBytes = sizeof(int32_t) * (size_t)kStaticMaxT;  // 256 KB
constexpr size_t kKaccBytes = sizeof(double) * (size_t)kStaticMaxB * kStaticMaxB;  // 512 KB
constexpr size_t kStaticScratchBytes = kOffBytes + kTokseqBytes + kKaccBytes;
static_assert(sizeof(int64_t) * (kStaticMaxB + 1) <= kOffBytes, "offset area too small");

static __device__ __align__(256) unsigned char g_static_scratch[kStaticScratchBytes];

// device address of g_static_scratch, per device ordinal; filled by the first call on that device
unsigned char* g_scratch_addr[kMaxDevices] = {};

isopo_status scratch_for_current_device(unsigned char** out) {
  int dev = -1;
  ISOPO_CUDA_TRY(cudaGetDevice(&dev));
  if (dev < 0 || dev >= kMaxDevices) return ISOPO_ERR_UNSUPPORTED;
  if (!g_scratch_addr[dev]) {
    void* p = nullptr;
    ISOPO_CUDA_TRY(cudaGetSymbolAddress(&p, g_static_scratch));
    if (!p) return ISOPO_ERR_CUDA;
    g_scratch_addr[dev] = static_cast<unsigned char*>(p);
  }
  *out = g_scratch_addr[dev];
  return ISOPO_OK;
}

}  // namespace
}  // namespace isopo

using namespace isopo;

extern "C" ISOPO_API isopo_status isopo_layer_gram_static(const void* X, const void* dY, isopo_dtype dtype, int64_t T, int d_in,
                                                int d_out, const int64_t* seq_offsets_host, int B, float* K,
                                                int32_t* info, void* cuda_stream) {
  if (!X || !dY || !seq_offsets_host || !K || !info) return ISOPO_ERR_INVALID_ARG;
  if (dtype != ISOPO_F32 && dtype != ISOPO_BF16) return ISOPO_ERR_INVALID_ARG;
  if (T < 1 || B < 1 || d_in < 1 || d_out < 1 || (int64_t)B > T) return ISOPO_ERR_INVALID_ARG;
  if (T > kStaticMaxT || B > kStaticMaxB) {
    set_cuda_error(cudaSuccess,
                   "isopo_layer_gram_static: at most ISOPO_STATIC_MAX_TOKENS tokens and ISOPO_STATIC_MAX_SEQS "
                   "sequences fit the built-in scratch; use isopo_layer_gram with a caller workspace");
    return ISOPO_ERR_UNSUPPORTED;
  }
  if (((uintptr_t)X & 15) || ((uintptr_t)dY & 15)) return ISOPO_ERR_INVALID_ARG;
  if (seq_offsets_host[0] != 0 || seq_offsets_host[B] != T) return ISOPO_ERR_INVALID_ARG;
  for (int i = 0; i < B; ++i)
    if (seq_offsets_host[i + 1] <= seq_offsets_host[i]) return ISOPO_ERR_INVALID_ARG;
  if (dtype == ISOPO_BF16 && ((d_in & 7) || (d_out & 7))) return ISOPO_ERR_UNSUPPORTED;

  unsigned char* scratch = nullptr;
  isopo_status s = scratch_for_current_device(&scratch);
  if (s != ISOPO_OK) return s;
  int64_t* off_dev = reinterpret_cast<int64_t*>(scratch);
  int32_t* tokseq = reinterpret_cast<int32_t*>(scratch + kOffBytes);
  double* kacc = reinterpret_cast<double*>(scratch + kOffBytes + kTokseqBytes);

  cudaStream_t st = (cudaStream_t)cuda_stream;
  ProfilingPause pause;  // event timing would create events: keep this call free of any allocation
  // Every region that is read is rewritten first: the offsets and the map for [0, T) here, the
  // accumulators by a memset inside the float32 route.  Nothing left by an earlier call is used.
  s = launch_prep(seq_offsets_host, B, T, off_dev, tokseq, st);
  if (s != ISOPO_OK) return s;
  if (dtype == ISOPO_F32)
    return f32_gram((const float*)X, (const float*)dY, T, d_in, d_out, tokseq, B, kacc, K, st);
  return bf16_gram(X, dY, T, d_in, d_out, tokseq, B, K, info, st);
}
