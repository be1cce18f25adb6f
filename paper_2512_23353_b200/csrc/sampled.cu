// Token-sampled Fisher-norm estimator of Algorithm 1 (Sec. 2.2, "Efficient implementation"):
// with a0 = X[samples], g0 = dY[samples] (the rows the caller drew),
//   F_i^2 = sum_j (g0_j . G_i a0_j)^2 / sum_j (||g0_j|| ||a0_j||)^2 ,   c_i = A_i / sqrt(F_i^2 + lambda).
// G_i is never formed: g0_j . G_i a0_j = sum_{t in i} (g0_j . dY_t)(a0_j . x_t) =: M^T[j, i] (Eq. one), a
// rectangular cousin of the Gram route (tensor-core kernel in tc_gram.cu, float32 SIMT kernel here).
// This file holds what surrounds it: gathering the sampled rows (and the denominator, Eq. two),
// the float32 kernel, and the finishing step that turns M^T into F^2 and the coefficients.
#include <algorithm>

#include <cuda_bf16.h>

#include "isopo_internal.h"

namespace isopo {

namespace {

__device__ __forceinline__ float to_f32(float v) { return v; }
__device__ __forceinline__ float to_f32(__nv_bfloat16 v) { return __bfloat162float(v); }

__device__ __forceinline__ double block_sum_d(double v) {
  __shared__ double red[32];
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  const int w = threadIdx.x >> 5, l = threadIdx.x & 31;
  __syncthreads();
  if (l == 0) red[w] = v;
  __syncthreads();
  v = l < (blockDim.x >> 5) ? red[l] : 0.0;
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;
}

// Copies one token row and returns this thread's share of its sum of squares.  Rows whose byte length and both
// addresses are multiples of 16 (every bfloat16 layer the library accepts) move as 16-byte vectors.
template <typename T>
__device__ __forceinline__ double copy_row_sq(const T* __restrict__ src, T* __restrict__ dst, int d) {
  constexpr int kVec = 16 / (int)sizeof(T);
  double acc = 0.0;
  if (d % kVec == 0 && (((uintptr_t)src | (uintptr_t)dst) & 15) == 0) {
    const uint4* s4 = reinterpret_cast<const uint4*>(src);
    uint4* d4 = reinterpret_cast<uint4*>(dst);
    for (int c = threadIdx.x; c < d / kVec; c += blockDim.x) {
      const uint4 v = __ldg(s4 + c);
      d4[c] = v;
      const T* e = reinterpret_cast<const T*>(&v);
      float part = 0.f;  // at most 8 squares of bfloat16 / 4 of float32 values: exact enough before the float64 sum
#pragma unroll
      for (int k = 0; k < kVec; ++k) {
        const float f = to_f32(e[k]);
        if (sizeof(T) == 2) part = fmaf(f, f, part); else acc += (double)f * (double)f;
      }
      if (sizeof(T) == 2) acc += (double)part;
    }
    return acc;
  }
  for (int c = threadIdx.x; c < d; c += blockDim.x) {
    const T v = src[c];
    dst[c] = v;
    const double f = (double)to_f32(v);
    acc += f * f;
  }
  return acc;
}

// Block j copies token row rows[j] of X and dY into a0[j], g0[j] and adds ||g0_j||^2 ||a0_j||^2 to *den.
template <typename T>
__global__ void __launch_bounds__(256) k_gather_samples(const T* __restrict__ X, const T* __restrict__ dY, int d_in,
                                                        int d_out, const int64_t* __restrict__ rows,
                                                        T* __restrict__ a0, T* __restrict__ g0,
                                                        double* __restrict__ den) {
  const int j = blockIdx.x;
  const int64_t t = rows[j];
  double na = copy_row_sq(X + t * d_in, a0 + (size_t)j * d_in, d_in);
  double ng = copy_row_sq(dY + t * d_out, g0 + (size_t)j * d_out, d_out);
  na = block_sum_d(na);
  ng = block_sum_d(ng);
  if (threadIdx.x == 0) atomicAdd(den, na * ng);
}

// float32 route: for a 32 x 32 tile (samples x tokens) form P = a0 X^T and Q = g0 dY^T, multiply
// elementwise and add into M^T[sample, sequence of the token] (float64 accumulators).
constexpr int kST = 32;
__global__ void __launch_bounds__(256) k_f32_sampled(const float* __restrict__ X, const float* __restrict__ dY, int64_t T,
                                                     int d_in, int d_out, const float* __restrict__ a0,
                                                     const float* __restrict__ g0, int n_samples,
                                                     const int32_t* __restrict__ tokseq, int B,
                                                     double* __restrict__ Mt) {
  __shared__ float sA[kST][kST + 1];
  __shared__ float sB[kST][kST + 1];
  const int tid = threadIdx.x, tx = tid & 15, ty = tid >> 4;
  const int64_t j0 = (int64_t)blockIdx.y * kST, t0 = (int64_t)blockIdx.x * kST;
  float h[2][2];
  for (int pass = 0; pass < 2; ++pass) {
    const float* R = pass == 0 ? a0 : g0;
    const float* C = pass == 0 ? X : dY;
    const int d = pass == 0 ? d_in : d_out;
    float acc[2][2] = {};
    for (int k0 = 0; k0 < d; k0 += kST) {
      for (int e = tid; e < kST * kST; e += 256) {
        const int r = e / kST, c = e % kST;
        sA[r][c] = (j0 + r < n_samples && k0 + c < d) ? R[(j0 + r) * d + k0 + c] : 0.f;
        sB[r][c] = (t0 + r < T && k0 + c < d) ? C[(t0 + r) * d + k0 + c] : 0.f;
      }
      __syncthreads();
#pragma unroll 8
      for (int c = 0; c < kST; ++c) {
        const float r0 = sA[ty * 2][c], r1 = sA[ty * 2 + 1][c], c0 = sB[tx * 2][c], c1 = sB[tx * 2 + 1][c];
        acc[0][0] = fmaf(r0, c0, acc[0][0]);
        acc[0][1] = fmaf(r0, c1, acc[0][1]);
        acc[1][0] = fmaf(r1, c0, acc[1][0]);
        acc[1][1] = fmaf(r1, c1, acc[1][1]);
      }
      __syncthreads();
    }
    for (int p = 0; p < 2; ++p)
      for (int q = 0; q < 2; ++q) h[p][q] = pass == 0 ? acc[p][q] : h[p][q] * acc[p][q];
  }
  for (int p = 0; p < 2; ++p)
    for (int q = 0; q < 2; ++q) {
      const int64_t j = j0 + ty * 2 + p, t = t0 + tx * 2 + q;
      if (j < n_samples && t < T) atomicAdd(&Mt[(size_t)j * B + tokseq[t]], (double)h[p][q]);
    }
}

// F_i^2 = sum_j M^T[j, i]^2 / den,  c_i = A_i / sqrt(F_i^2 + lambda).  A block of 32 x 8 threads serves 32
// sequences: thread (x, y) sums the samples j = y, y + 8, ... of sequence x (loads coalesced over x), the eight
// partial sums meet in shared memory.
constexpr int kFinishSlices = 8;
template <typename TM>
__global__ void __launch_bounds__(32 * kFinishSlices) k_sampled_finish(const TM* __restrict__ Mt, int n_samples, int B,
                                                                       const double* __restrict__ den,
                                                                       const float* __restrict__ A, float lambda,
                                                                       float* __restrict__ coeffs, float* __restrict__ F2) {
  __shared__ double part[kFinishSlices][32];
  const int x = threadIdx.x & 31, y = threadIdx.x >> 5;
  const int i = blockIdx.x * 32 + x;
  double s = 0.0;
  if (i < B)
    for (int j = y; j < n_samples; j += kFinishSlices) {
      const double m = (double)Mt[(size_t)j * B + i];
      s += m * m;
    }
  part[y][x] = s;
  __syncthreads();
  if (y != 0 || i >= B) return;
  s = 0.0;
#pragma unroll
  for (int k = 0; k < kFinishSlices; ++k) s += part[k][x];
  const double f2 = s / *den;
  if (F2) F2[i] = (float)f2;
  coeffs[i] = (float)((double)A[i] / sqrt(f2 + (double)lambda));
}

}  // namespace

SampledLayout sampled_layout(isopo_dtype dtype, int64_t T, int d_in, int d_out, int B, int n_samples) {
  SampledLayout S{};
  const size_t elt = dtype == ISOPO_BF16 ? 2 : 4;
  size_t p = ws_layout(dtype, T, d_in, d_out, B, ISOPO_PATH_GRAM).total;  // offsets, order, token map (+ kacc)
  S.off_rows = p;
  p = align_up(p + sizeof(int64_t) * (size_t)n_samples, 1024);
  S.off_a0 = p;
  p = align_up(p + elt * (size_t)n_samples * d_in, 1024);
  S.off_g0 = p;
  p = align_up(p + elt * (size_t)n_samples * d_out, 1024);
  S.off_mt = p;
  p = align_up(p + (dtype == ISOPO_BF16 ? sizeof(float) : sizeof(double)) * (size_t)n_samples * B, 1024);
  S.off_den = p;
  p = align_up(p + sizeof(double), 1024);
  S.total = p;
  return S;
}

isopo_status sampled_coefficients(const void* X, const void* dY, isopo_dtype dtype, int64_t T, int d_in, int d_out,
                                  const int32_t* tokseq, int B, const int64_t* rows_host, int n_samples, char* ws,
                                  const SampledLayout& S, const float* A, float lambda, float* coeffs, float* F2,
                                  int32_t* info, cudaStream_t st) {
  int64_t* rows = (int64_t*)(ws + S.off_rows);
  double* den = (double*)(ws + S.off_den);
  isopo_status s = store_i64(rows_host, n_samples, rows, st);
  if (s != ISOPO_OK) return s;
  ISOPO_CUDA_TRY(cudaMemsetAsync(den, 0, sizeof(double), st));
  if (dtype == ISOPO_F32) {
    float* a0 = (float*)(ws + S.off_a0);
    float* g0 = (float*)(ws + S.off_g0);
    double* Mt = (double*)(ws + S.off_mt);
    const int64_t nt = (T + kST - 1) / kST, ns = (n_samples + kST - 1) / kST;
    if (ns > 65535) return ISOPO_ERR_UNSUPPORTED;
    ISOPO_CUDA_TRY(cudaMemsetAsync(Mt, 0, sizeof(double) * (size_t)n_samples * B, st));
    {
      LaunchScope scope(kIdSampledAux, st);
      k_gather_samples<float><<<n_samples, 256, 0, st>>>((const float*)X, (const float*)dY, d_in, d_out, rows, a0, g0, den);
    }
    ISOPO_CUDA_TRY(cudaGetLastError());
    {
      LaunchScope scope(kIdSampled, st);
      k_f32_sampled<<<dim3((unsigned)nt, (unsigned)ns), 256, 0, st>>>((const float*)X, (const float*)dY, T, d_in, d_out, a0,
                                                                      g0, n_samples, tokseq, B, Mt);
    }
    ISOPO_CUDA_TRY(cudaGetLastError());
    {
      LaunchScope scope(kIdSampledAux, st);
      k_sampled_finish<double><<<(B + 31) / 32, 32 * kFinishSlices, 0, st>>>(Mt, n_samples, B, den, A, lambda, coeffs, F2);
    }
    ISOPO_CUDA_TRY(cudaGetLastError());
    return ISOPO_OK;
  }
  __nv_bfloat16* a0 = (__nv_bfloat16*)(ws + S.off_a0);
  __nv_bfloat16* g0 = (__nv_bfloat16*)(ws + S.off_g0);
  float* Mt = (float*)(ws + S.off_mt);
  {
    LaunchScope scope(kIdSampledAux, st);
    k_gather_samples<__nv_bfloat16><<<n_samples, 256, 0, st>>>((const __nv_bfloat16*)X, (const __nv_bfloat16*)dY, d_in, d_out,
                                                               rows, a0, g0, den);
  }
  ISOPO_CUDA_TRY(cudaGetLastError());
  s = bf16_sampled(X, dY, T, d_in, d_out, tokseq, B, a0, g0, n_samples, Mt, info, st);
  if (s != ISOPO_OK) return s;
  {
    LaunchScope scope(kIdSampledAux, st);
    k_sampled_finish<float><<<(B + 31) / 32, 32 * kFinishSlices, 0, st>>>(Mt, n_samples, B, den, A, lambda, coeffs, F2);
  }
  ISOPO_CUDA_TRY(cudaGetLastError());
  return ISOPO_OK;
}

}  // namespace isopo
