// Internal declarations shared by the translation units of libisopo (not part of the C ABI).
#pragma once

#include <cuda_runtime.h>
#include <stddef.h>
#include <stdint.h>

#include "isopo.h"

namespace isopo {

// Tile of the stored per-sequence gradients on the bf16 path: one tensor-core accumulator tile.
constexpr int kTileM = 128;  // rows of G (d_out)
constexpr int kTileN = 256;  // columns of G (d_in)
constexpr int kTileElems = kTileM * kTileN;

// Kernel identifiers: written to *info together with ISOPO_INFO_TIMEOUT, and the index of the
// per-kernel timing slots of isopo_profile_collect.
enum KernelId : int {
  kIdPrep = 0,
  kIdSeqGrad = 1,
  kIdNtk = 2,
  kIdGram = 3,
  kIdWeightGrad = 4,
  kIdCombine = 5,
  kIdTransform = 6,
  kIdMirror = 7,
  kIdF32SeqGrad = 8,
  kIdF32Ntk = 9,
  kIdF32Gram = 10,
  kIdF32WeightGrad = 11,
  kIdF32Combine = 12,
  kIdSampled = 13,     // M^T of the token-sampled estimator (tensor-core or float32 kernel)
  kIdSampledAux = 14,  // its gather and finishing kernels
  kIdScaleRows = 15,   // per-token scale of the narrower operand before the 2-CTA weight-gradient GEMM
  kIdWaitProbe = 16,   // isopo_selftest_bounded_wait
  kIdCount = 17
};

// Debug build (-DISOPO_DEBUG, libisopo_debug.so): every index a kernel computes for a global load, store or
// atomic of its own buffers (stored gradients, K, M^T, dW, the staged sequence tables) is compared with the
// buffer's extent first; an index outside it skips the access and records ISOPO_INFO_BOUNDS | kernel id in
// *info.  It stands in for a memory checker on the data-dependent addressing: ragged tails, the
// piece-blocked store, segment sums.  In the normal build the checks compile to nothing.
#ifdef ISOPO_DEBUG
__device__ __forceinline__ bool dbg_in_range(long long idx, long long n, int32_t* info, int id) {
  if (idx >= 0 && idx < n) return true;
  atomicCAS(info, 0, ISOPO_INFO_BOUNDS | id);
  return false;
}
#define ISOPO_IN_RANGE(idx, n, info, id) (::isopo::dbg_in_range((long long)(idx), (long long)(n), (info), (id)))
#else
#define ISOPO_IN_RANGE(idx, n, info, id) (true)
#endif

// Brackets one kernel launch with CUDA events while profiling is enabled (isopo_profile_enable);
// otherwise only counts the launch.
class LaunchScope {
 public:
  LaunchScope(int id, cudaStream_t st);
  ~LaunchScope();

 private:
  int slot_;
  cudaStream_t st_;
};

// Suspends event timing for the lifetime of the object (launch counting continues).
class ProfilingPause {
 public:
  ProfilingPause();
  ~ProfilingPause();

 private:
  bool was_on_;
};

// What isopo_layer_gram(MATERIALISE) leaves at the head of the workspace so that isopo_weight_grad can tell
// whether the stored gradients it is about to sum belong to the layer and microbatch it was called for.
struct WsTag {
  int64_t v[8];  // magic, dtype, T, d_in, d_out, B, hash of the offsets, 0
};
WsTag make_ws_tag(isopo_dtype dtype, int64_t T, int d_in, int d_out, int B, const int64_t* off_host);

// How the bf16 stored route keeps G_i.  Split (isopo_set_store_format(ISOPO_STORE_E4M3_SPLIT)): two e4m3 planes of
// one byte per element each - `hi` = round(s_i G_i), `lo` = round(16 (s_i G_i - hi)) with a power-of-two scale s_i per
// sequence - in the same piece order.  The K pass reads only `hi` (half the bytes, kind::f8f6f4 MMAs) and takes the
// diagonal from `kdiag`, which the gradient GEMM sums in float32 from its accumulators; the combine reads both planes.
struct StoreFmt {
  int split;             // 0: bf16 (2 bytes per element), 1: e4m3 hi / lo planes
  const float* scales;   // [B] s_i
  float* kdiag;          // [B] sum of squares of G_i
};

struct WsLayout {
  size_t off_tag;      // WsTag (materialised path)
  size_t off_aux;      // float scales[B] | float kdiag[B]  (bf16 materialised path, split store)
  size_t off_offsets;  // int64 [B+1]
  size_t off_order;    // int32 [B]       (bf16 materialised path: sequences, longest first)
  size_t off_tokseq;   // int32 [T]: token -> sequence; the bf16 weight-gradient GEMM keeps float32 per-token scales here
  size_t off_kacc;     // float64 [B*B]   (float32 path: K accumulators)
  size_t off_scaled;   // bf16 [T, min(d_in, d_out)]  (bf16 Gram path: the pre-scaled operand of the weight-gradient GEMM)
  size_t off_G;        // stored gradients (materialised path only)
  size_t off_kpart;    // per-CTA partial K (bf16 materialised path in deterministic mode only)
  size_t total;
  int tiles_m, tiles_n;  // bf16 materialised layout: tiles per gradient
  int64_t n_pad;         // elements per stored gradient (row stride of G_flat)
};

inline size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

WsLayout ws_layout(isopo_dtype dtype, int64_t T, int d_in, int d_out, int B, isopo_path resolved);

// Workspace of isopo_sampled_coefficients: the Gram-route prefix (offsets, order, token map), then
// the sampled row indices, the gathered rows a0 / g0, M^T and the denominator.
struct SampledLayout {
  size_t off_rows, off_a0, off_g0, off_mt, off_den, total;
};
SampledLayout sampled_layout(isopo_dtype dtype, int64_t T, int d_in, int d_out, int B, int n_samples);

void set_cuda_error(cudaError_t e, const char* where);
#define ISOPO_CUDA_TRY(expr)                                  \
  do {                                                        \
    cudaError_t e__ = (expr);                                 \
    if (e__ != cudaSuccess) {                                 \
      ::isopo::set_cuda_error(e__, #expr);                    \
      return ISOPO_ERR_CUDA;                                  \
    }                                                         \
  } while (0)

// ---- launchers (each enqueues on `st` and returns a status; none synchronises) ----

isopo_status launch_prep(const int64_t* off_host, int B, int64_t T, int64_t* off_dev, int32_t* tokseq, cudaStream_t st);
// bf16 materialised path (B <= 256) in one launch: offsets, the longest-first order, the workspace tag, K = 0
isopo_status launch_prep_stored(const int64_t* off_host, int B, const WsTag& tag, int64_t* off_dev, int32_t* order_dev,
                                WsTag* tag_dev, float* K, cudaStream_t st);
isopo_status launch_prep_stored_multi(const int64_t* off_host, int B, int n_proj, const WsTag* tag, int64_t* const* off_dev,
                                      int32_t* const* order_dev, WsTag* const* tag_dev, float* const* K, cudaStream_t st);
isopo_status store_tag(const WsTag& tag, WsTag* tag_dev, cudaStream_t st);
// offsets to the device and tokscale[t] = coeffs[sequence of token t] (float32 [T])
isopo_status launch_tokscale(const int64_t* off_host, int B, int64_t T, int64_t* off_dev, const float* coeffs,
                             float* tokscale, cudaStream_t st);
// n host values -> device array, passed as kernel arguments (no host-to-device copy)
isopo_status store_i64(const int64_t* host, int64_t n, int64_t* dev, cudaStream_t st);
// true when every word of the tag in the workspace equals `want`; otherwise the first thread of the grid
// records ISOPO_INFO_STALE_WORKSPACE (device code, used by the combine kernels)
__device__ __forceinline__ bool ws_tag_matches(const WsTag* __restrict__ have, const WsTag& want, int32_t* info) {
  bool ok = true;
#pragma unroll
  for (int k = 0; k < 8; ++k) ok = ok && have->v[k] == want.v[k];
  if (!ok && blockIdx.x == 0 && threadIdx.x == 0) atomicCAS(info, 0, ISOPO_INFO_STALE_WORKSPACE);
  return ok;
}

// float32 SIMT path
isopo_status f32_seq_grad(const float* X, const float* dY, int d_in, int d_out, const int64_t* off_dev, int B,
                          float* G, cudaStream_t st);
isopo_status f32_ntk(const float* G, int64_t N, int B, float* K, cudaStream_t st);
isopo_status f32_gram(const float* X, const float* dY, int64_t T, int d_in, int d_out, const int32_t* tokseq, int B,
                      double* kacc, float* K, cudaStream_t st);
isopo_status f32_combine(const float* G, int64_t N, int B, const float* coeffs, float* dW, float beta, const WsTag* tag_dev,
                         const WsTag& tag, int32_t* info, cudaStream_t st);
isopo_status f32_weight_grad(const float* X, const float* dY, int64_t T, int d_in, int d_out, const float* coeffs,
                             const int32_t* tokseq, float* dW, float beta, cudaStream_t st);

// bf16 tcgen05 path
isopo_status bf16_seq_grad(const void* X, const void* dY, int64_t T, int d_in, int d_out, const int64_t* off_host,
                           const int64_t* off_dev, const int32_t* order_dev, int B, const WsLayout& L, void* G,
                           const StoreFmt& fmt, int32_t* info, cudaStream_t st);
isopo_status bf16_seq_grad_pair(const void* X, const void* dY, int64_t T, int d_in, int d_out, const int64_t* off_dev,
                                const int32_t* order_dev, int B, const WsLayout& L, void* G, const StoreFmt& fmt,
                                int32_t* info, cudaStream_t st);
// whether a layer of this shape keeps its gradients in the split e4m3 format under the current settings
bool use_split_store(const WsLayout& L, int B);
StoreFmt store_fmt(const WsLayout& L, int B, void* ws);
// s_i of every sequence from a sample of its token rows, kdiag = 0 (split store)
isopo_status launch_seq_scales(const void* X, const void* dY, int d_in, int d_out, const int64_t* off_dev, int B, float* scales,
                               float* kdiag, cudaStream_t st);
// the same for up to three projections that read one X, in one launch (L, dY, d_out, G: one entry per projection)
isopo_status bf16_seq_grad_pair_shared(const void* X, int n_proj, const void* const* dY, const int* d_out, int64_t T, int d_in,
                                       const int64_t* off_dev, const int32_t* order_dev, int B, const WsLayout* L,
                                       void* const* G, const StoreFmt* fmt, int32_t* info, cudaStream_t st);
// k_is_zero: the caller has already cleared K on this stream.  kpart != NULL (deterministic mode): every CTA
// stores its partial upper triangle there ([kNtkMaxPartials][B * B] floats) and a second kernel sums them in order.
constexpr int kNtkMaxPartials = 160;
isopo_status bf16_ntk(const void* G, const WsLayout& L, int B, float* K, bool k_is_zero, float* kpart, const StoreFmt& fmt,
                      int32_t* info, cudaStream_t st);
bool deterministic_mode();
// K[i][j] = K[j][i] for j < i (the K kernels fill the upper triangle)
isopo_status mirror_upper(float* K, int B, cudaStream_t st, const float* kdiag = nullptr);
isopo_status bf16_combine(const void* G, const WsLayout& L, int d_in, int d_out, int B, const float* coeffs, float* dW,
                          float beta, const WsTag* tag_dev, const WsTag& tag, const StoreFmt& fmt, int32_t* info,
                          cudaStream_t st);
isopo_status bf16_gram(const void* X, const void* dY, int64_t T, int d_in, int d_out, const int32_t* tokseq, int B,
                       float* K, int32_t* info, cudaStream_t st);
isopo_status bf16_gram_shared(const void* X, const void* const* dY, int64_t T, int d_in, const int* d_out, int n_heads,
                              const int32_t* tokseq, int B, float* const* K, int32_t* info, cudaStream_t st);
isopo_status bf16_weight_grad(const void* X, const void* dY, int64_t T, int d_in, int d_out, const float* tokscale,
                              void* scaled, float* dW, float beta, int32_t* info, cudaStream_t st);

// dW with the per-sequence coefficient applied when a segment's accumulator is drained (no scaled operand copy)
bool bf16_weight_grad_fold_applies(int64_t T, int d_in, int d_out, int B);
isopo_status bf16_weight_grad_fold(const void* X, const void* dY, int64_t T, int d_in, int d_out, const int64_t* off_dev,
                                   const float* coeffs, int B, float* dW, float beta, int32_t* info, cudaStream_t st);
isopo_status bf16_weight_grad_pair(const void* X, const void* dY, int64_t T, int d_in, int d_out, const float* tokscale,
                                   void* scaled, float* dW, float beta, int32_t* info, cudaStream_t st);

// token-sampled estimator of Algorithm 1
isopo_status bf16_sampled(const void* X, const void* dY, int64_t T, int d_in, int d_out, const int32_t* tokseq, int B,
                          const void* A0, const void* G0, int n_samples, float* Mt, int32_t* info, cudaStream_t st);
isopo_status sampled_coefficients(const void* X, const void* dY, isopo_dtype dtype, int64_t T, int d_in, int d_out,
                                  const int32_t* tokseq, int B, const int64_t* rows_host, int n_samples, char* ws,
                                  const SampledLayout& S, const float* A, float lambda, float* coeffs, float* F2,
                                  int32_t* info, cudaStream_t st);

// transform (all variants)
size_t transform_large_workspace_bytes(int B);
isopo_status transform_large(const float* K, const float* A, int B, float lambda, float* coeffs, float* scratch,
                             int32_t* info, cudaStream_t st);
isopo_status transform(const float* K, const float* A, int B, isopo_variant v, float lambda, const float* pqr_regs_host,
                       const float* rel_state, float* coeffs, int32_t* info, cudaStream_t st);
isopo_status transform_batched(int n, const float* const* K, const float* A, int B, isopo_variant v, const float* lambda,
                               const float* pqr_regs_host, const float* const* rel_state, float* const* coeffs,
                               int32_t* info, cudaStream_t st);
size_t spectral_workspace_bytes();
isopo_status spectral(const float* K, const float* A, int B, float lambda, float rel_cutoff, float* coeffs, float* eig,
                      void* ws, int32_t* info, cudaStream_t st);
isopo_status spectral_batched(int n, const float* const* K, const float* A, int B, const float* lambda,
                              float rel_cutoff, float* const* coeffs, float* const* eig, void* ws, int32_t* info,
                              cudaStream_t st);
isopo_status wait_probe(long long limit_clocks, int32_t* info, int32_t* roles_at_teardown, cudaStream_t st);
isopo_status reg_ema_update(const float* K, int B, float decay, float* state, cudaStream_t st);

}  // namespace isopo
