// float32 SIMT kernels of the ISOPO layer path (small layers, parity to 1e-5), plus the
// token -> sequence map that both dtypes use.  Products are float32 FFMA; everything that sums
// over many products of products (K) is accumulated in float64.
#include <algorithm>

#include "isopo_internal.h"

namespace isopo {

namespace {

constexpr int kT = 64;   // output tile edge of the SIMT GEMMs
constexpr int kTK = 16;  // tokens staged per step

// Host values travel to the device as kernel arguments (no host-to-device copy, so no hidden
// synchronisation with the stream and nothing that reads the caller's array after the call returns).
constexpr int kArgChunk = 384;
struct OffsetArgs { int64_t v[kArgChunk]; };
__global__ void k_store_offsets(OffsetArgs a, int base, int n, int64_t* __restrict__ off) {
  const int t = threadIdx.x;
  if (t < n) off[base + t] = a.v[t];
}

// Everything the bf16 stored-gradient kernels need before they start, in one launch (B <= 256):
// CTA 0 leaves the offsets, the working order of the sequences and the workspace tag; all CTAs clear K.
// With several projections sharing one launch (same offsets, one workspace each) every workspace gets its copy.
struct StoredPrepArgs {
  int64_t off[257];
  WsTag tag[3];
  int64_t* off_dev[3];
  int32_t* order_dev[3];
  WsTag* tag_dev[3];
  float* K[3];
  uint8_t order[256];
};
__global__ void __launch_bounds__(256) k_prep_stored(StoredPrepArgs a, int B, int n_proj) {
  for (int h = 0; h < n_proj; ++h) {
    if (blockIdx.x == 0) {
      for (int i = threadIdx.x; i <= B; i += blockDim.x) a.off_dev[h][i] = a.off[i];
      for (int i = threadIdx.x; i < B; i += blockDim.x) a.order_dev[h][i] = a.order[i];
      if (threadIdx.x < 8) a.tag_dev[h]->v[threadIdx.x] = a.tag[h].v[threadIdx.x];
    }
    for (int e = blockIdx.x * blockDim.x + threadIdx.x; e < B * B; e += gridDim.x * blockDim.x) a.K[h][e] = 0.f;
  }
}
__global__ void k_store_tag(WsTag t, WsTag* __restrict__ tag) {
  if (threadIdx.x < 8) tag->v[threadIdx.x] = t.v[threadIdx.x];
}

__global__ void k_tokseq(const int64_t* __restrict__ off, int B, int64_t T, int32_t* __restrict__ tokseq) {
  for (int64_t t = blockIdx.x * (int64_t)blockDim.x + threadIdx.x; t < T; t += (int64_t)gridDim.x * blockDim.x) {
    int lo = 0, hi = B;  // invariant: off[lo] <= t < off[hi]
    while (hi - lo > 1) {
      int mid = (lo + hi) >> 1;
      if (off[mid] <= t) lo = mid; else hi = mid;
    }
    tokseq[t] = lo;
  }
}

// tokscale[t] = coeffs[sequence of token t]: what the folded weight-gradient GEMM multiplies row t by.
__global__ void k_tokscale(const int64_t* __restrict__ off, int B, int64_t T, const float* __restrict__ coeffs,
                           float* __restrict__ tokscale) {
  for (int64_t t = blockIdx.x * (int64_t)blockDim.x + threadIdx.x; t < T; t += (int64_t)gridDim.x * blockDim.x) {
    int lo = 0, hi = B;  // invariant: off[lo] <= t < off[hi]
    while (hi - lo > 1) {
      int mid = (lo + hi) >> 1;
      if (off[mid] <= t) lo = mid; else hi = mid;
    }
    tokscale[t] = coeffs[lo];
  }
}

// k_store_offsets + k_tokseq / k_tokscale in one launch when all B + 1 offsets fit one argument block:
// every CTA copies them to shared memory and searches there; CTA 0 also leaves them in the workspace.
template <bool kScale>
__global__ void __launch_bounds__(256) k_prep_small(OffsetArgs a, int B, int64_t T, int64_t* __restrict__ off_dev,
                                                    const float* __restrict__ coeffs, void* __restrict__ out) {
  __shared__ int64_t s_off[kArgChunk];
  for (int i = threadIdx.x; i <= B; i += blockDim.x) {
    s_off[i] = a.v[i];
    if (blockIdx.x == 0) off_dev[i] = a.v[i];
  }
  __syncthreads();
  for (int64_t t = blockIdx.x * (int64_t)blockDim.x + threadIdx.x; t < T; t += (int64_t)gridDim.x * blockDim.x) {
    int lo = 0, hi = B;  // invariant: off[lo] <= t < off[hi]
    while (hi - lo > 1) {
      int mid = (lo + hi) >> 1;
      if (s_off[mid] <= t) lo = mid; else hi = mid;
    }
    if (kScale) static_cast<float*>(out)[t] = coeffs[lo];
    else static_cast<int32_t*>(out)[t] = lo;
  }
}

// Accumulates, for tokens [t0, t1), acc[4][4] += w_t * dY[t, m0+4ty+a] * X[t, n0+4tx+b].
template <bool kScaled>
__device__ __forceinline__ void gemm_tokens(const float* __restrict__ X, const float* __restrict__ dY, int d_in,
                                            int d_out, int64_t t0, int64_t t1, int m0, int n0,
                                            const float* __restrict__ coeffs, const int32_t* __restrict__ tokseq,
                                            float (&acc)[4][4]) {
  __shared__ float sY[kTK][kT + 4];
  __shared__ float sX[kTK][kT + 4];
  const int tid = threadIdx.x, tx = tid & 15, ty = tid >> 4;
  for (int64_t tb = t0; tb < t1; tb += kTK) {
    for (int e = tid; e < kTK * kT; e += 256) {
      const int r = e / kT, c = e % kT;
      const int64_t t = tb + r;
      float y = 0.f, x = 0.f;
      if (t < t1) {
        if (m0 + c < d_out) y = dY[t * d_out + m0 + c];
        if (n0 + c < d_in) x = X[t * d_in + n0 + c];
        if (kScaled) y *= coeffs[tokseq[t]];
      }
      sY[r][c] = y;
      sX[r][c] = x;
    }
    __syncthreads();
#pragma unroll
    for (int r = 0; r < kTK; ++r) {
      float a[4], b[4];
#pragma unroll
      for (int q = 0; q < 4; ++q) { a[q] = sY[r][ty * 4 + q]; b[q] = sX[r][tx * 4 + q]; }
#pragma unroll
      for (int p = 0; p < 4; ++p)
#pragma unroll
        for (int q = 0; q < 4; ++q) acc[p][q] = fmaf(a[p], b[q], acc[p][q]);
    }
    __syncthreads();
  }
}

// G_i = dY_i^T X_i, one (64 x 64 tile, sequence) per CTA.
__global__ void __launch_bounds__(256) k_f32_seq_grad(const float* __restrict__ X, const float* __restrict__ dY,
                                                      int d_in, int d_out, const int64_t* __restrict__ off,
                                                      float* __restrict__ G) {
  const int i = blockIdx.z, m0 = blockIdx.y * kT, n0 = blockIdx.x * kT;
  float acc[4][4] = {};
  gemm_tokens<false>(X, dY, d_in, d_out, off[i], off[i + 1], m0, n0, nullptr, nullptr, acc);
  const int tx = threadIdx.x & 15, ty = threadIdx.x >> 4;
  float* Gi = G + (size_t)i * d_out * d_in;
  for (int p = 0; p < 4; ++p)
    for (int q = 0; q < 4; ++q) {
      const int m = m0 + ty * 4 + p, n = n0 + tx * 4 + q;
      if (m < d_out && n < d_in) Gi[(size_t)m * d_in + n] = acc[p][q];
    }
}

// dW += (c_seq(t) dY)^T X over a slab of tokens (split over blockIdx.z), float atomics.
__global__ void __launch_bounds__(256) k_f32_weight_grad(const float* __restrict__ X, const float* __restrict__ dY,
                                                         int64_t T, int d_in, int d_out,
                                                         const float* __restrict__ coeffs,
                                                         const int32_t* __restrict__ tokseq, float* __restrict__ dW,
                                                         int64_t slab) {
  const int m0 = blockIdx.y * kT, n0 = blockIdx.x * kT;
  const int64_t t0 = blockIdx.z * slab, t1 = min(T, t0 + slab);
  float acc[4][4] = {};
  gemm_tokens<true>(X, dY, d_in, d_out, t0, t1, m0, n0, coeffs, tokseq, acc);
  const int tx = threadIdx.x & 15, ty = threadIdx.x >> 4;
  for (int p = 0; p < 4; ++p)
    for (int q = 0; q < 4; ++q) {
      const int m = m0 + ty * 4 + p, n = n0 + tx * 4 + q;
      if (m < d_out && n < d_in) atomicAdd(&dW[(size_t)m * d_in + n], acc[p][q]);
    }
}

__device__ __forceinline__ double block_sum(double v) {
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

// K_ij = sum(G_i * G_j) for j >= i, mirrored.
__global__ void __launch_bounds__(256) k_f32_ntk(const float* __restrict__ G, int64_t N, int B, float* __restrict__ K) {
  const int i = blockIdx.y, j = blockIdx.x;
  if (j < i) return;
  const float* gi = G + (size_t)i * N;
  const float* gj = G + (size_t)j * N;
  double s = 0.0;
  for (int64_t e = threadIdx.x; e < N; e += blockDim.x) s += (double)(gi[e] * gj[e]);
  s = block_sum(s);
  if (threadIdx.x == 0) {
    K[(size_t)i * B + j] = (float)s;
    K[(size_t)j * B + i] = (float)s;
  }
}

// Gram route: for a pair of 32-token tiles (I <= J) form P = X_I X_J^T and Q = dY_I dY_J^T, multiply
// elementwise and add into the (seq t, seq s) accumulators.  Only token pairs t <= s are used; a
// pair inside one sequence with t < s stands for (t,s) and (s,t) and counts twice.
constexpr int kGT = 32;
__global__ void __launch_bounds__(256) k_f32_gram(const float* __restrict__ X, const float* __restrict__ dY, int64_t T,
                                                  int d_in, int d_out, const int32_t* __restrict__ tokseq, int B,
                                                  double* __restrict__ kacc) {
  const int I = blockIdx.y, J = blockIdx.x;
  if (J < I) return;
  __shared__ float sA[kGT][kGT + 1];
  __shared__ float sB[kGT][kGT + 1];
  const int tid = threadIdx.x, tx = tid & 15, ty = tid >> 4;
  const int64_t tI = (int64_t)I * kGT, tJ = (int64_t)J * kGT;
  float h[2][2];
  for (int pass = 0; pass < 2; ++pass) {
    const float* M = pass == 0 ? X : dY;
    const int d = pass == 0 ? d_in : d_out;
    float acc[2][2] = {};
    for (int k0 = 0; k0 < d; k0 += kGT) {
      for (int e = tid; e < kGT * kGT; e += 256) {
        const int r = e / kGT, c = e % kGT;
        sA[r][c] = (tI + r < T && k0 + c < d) ? M[(tI + r) * d + k0 + c] : 0.f;
        sB[r][c] = (tJ + r < T && k0 + c < d) ? M[(tJ + r) * d + k0 + c] : 0.f;
      }
      __syncthreads();
#pragma unroll 8
      for (int c = 0; c < kGT; ++c) {
        const float a0 = sA[ty * 2][c], a1 = sA[ty * 2 + 1][c], b0 = sB[tx * 2][c], b1 = sB[tx * 2 + 1][c];
        acc[0][0] = fmaf(a0, b0, acc[0][0]);
        acc[0][1] = fmaf(a0, b1, acc[0][1]);
        acc[1][0] = fmaf(a1, b0, acc[1][0]);
        acc[1][1] = fmaf(a1, b1, acc[1][1]);
      }
      __syncthreads();
    }
    for (int p = 0; p < 2; ++p)
      for (int q = 0; q < 2; ++q) h[p][q] = pass == 0 ? acc[p][q] : h[p][q] * acc[p][q];
  }
  for (int p = 0; p < 2; ++p)
    for (int q = 0; q < 2; ++q) {
      const int64_t t = tI + ty * 2 + p, s = tJ + tx * 2 + q;
      if (t >= T || s >= T || t > s) continue;
      const int st = tokseq[t], ss = tokseq[s];
      const double w = (st == ss && t < s) ? 2.0 : 1.0;
      atomicAdd(&kacc[(size_t)st * B + ss], w * (double)h[p][q]);
    }
}

__global__ void k_f32_gram_finish(const double* __restrict__ kacc, int B, float* __restrict__ K) {
  const int e = blockIdx.x * blockDim.x + threadIdx.x;
  if (e >= B * B) return;
  const int i = e / B, j = e % B;
  K[e] = (float)(i <= j ? kacc[(size_t)i * B + j] : kacc[(size_t)j * B + i]);
}

__global__ void k_f32_combine(const float* __restrict__ G, int64_t N, int B, const float* __restrict__ coeffs,
                              float* __restrict__ dW, float beta, const WsTag* __restrict__ tag_dev, WsTag tag,
                              int32_t* __restrict__ info) {
  if (!ws_tag_matches(tag_dev, tag, info)) return;
  for (int64_t e = blockIdx.x * (int64_t)blockDim.x + threadIdx.x; e < N; e += (int64_t)gridDim.x * blockDim.x) {
    double s = 0.0;
    for (int i = 0; i < B; ++i) s += (double)coeffs[i] * (double)G[(size_t)i * N + e];
    dW[e] = (float)(beta != 0.f ? (double)dW[e] + s : s);
  }
}

}  // namespace

isopo_status store_i64(const int64_t* host, int64_t n, int64_t* dev, cudaStream_t st) {
  for (int64_t base = 0; base < n; base += kArgChunk) {
    OffsetArgs a;
    const int m = (int)std::min<int64_t>(kArgChunk, n - base);
    for (int t = 0; t < m; ++t) a.v[t] = host[base + t];
    k_store_offsets<<<1, kArgChunk, 0, st>>>(a, (int)base, m, dev);
    ISOPO_CUDA_TRY(cudaGetLastError());
  }
  return ISOPO_OK;
}

template <bool kScale>
static isopo_status launch_prep_small(const int64_t* off_host, int B, int64_t T, int64_t* off_dev, const float* coeffs,
                                      void* out, cudaStream_t st) {
  OffsetArgs a;
  for (int t = 0; t <= B; ++t) a.v[t] = off_host[t];
  const int grid = (int)std::min<int64_t>((T + 255) / 256, 1184);
  {
    LaunchScope scope(kIdPrep, st);
    k_prep_small<kScale><<<grid, 256, 0, st>>>(a, B, T, off_dev, coeffs, out);
  }
  ISOPO_CUDA_TRY(cudaGetLastError());
  return ISOPO_OK;
}

isopo_status launch_prep(const int64_t* off_host, int B, int64_t T, int64_t* off_dev, int32_t* tokseq,
                         cudaStream_t st) {
  if (B + 1 <= kArgChunk) return launch_prep_small<false>(off_host, B, T, off_dev, nullptr, tokseq, st);
  isopo_status s = store_i64(off_host, (int64_t)B + 1, off_dev, st);
  if (s != ISOPO_OK) return s;
  const int grid = (int)std::min<int64_t>((T + 255) / 256, 1184);
  {
    LaunchScope scope(kIdPrep, st);
    k_tokseq<<<grid, 256, 0, st>>>(off_dev, B, T, tokseq);
  }
  ISOPO_CUDA_TRY(cudaGetLastError());
  return ISOPO_OK;
}

isopo_status launch_tokscale(const int64_t* off_host, int B, int64_t T, int64_t* off_dev, const float* coeffs,
                             float* tokscale, cudaStream_t st) {
  if (B + 1 <= kArgChunk) return launch_prep_small<true>(off_host, B, T, off_dev, coeffs, tokscale, st);
  isopo_status s = store_i64(off_host, (int64_t)B + 1, off_dev, st);
  if (s != ISOPO_OK) return s;
  const int grid = (int)std::min<int64_t>((T + 255) / 256, 1184);
  {
    LaunchScope scope(kIdPrep, st);
    k_tokscale<<<grid, 256, 0, st>>>(off_dev, B, T, coeffs, tokscale);
  }
  ISOPO_CUDA_TRY(cudaGetLastError());
  return ISOPO_OK;
}

isopo_status launch_prep_stored(const int64_t* off_host, int B, const WsTag& tag, int64_t* off_dev, int32_t* order_dev,
                                WsTag* tag_dev, float* K, cudaStream_t st) {
  return launch_prep_stored_multi(off_host, B, 1, &tag, &off_dev, &order_dev, &tag_dev, &K, st);
}

isopo_status launch_prep_stored_multi(const int64_t* off_host, int B, int n_proj, const WsTag* tag, int64_t* const* off_dev,
                                      int32_t* const* order_dev, WsTag* const* tag_dev, float* const* K, cudaStream_t st) {
  if (B > 256 || n_proj < 1 || n_proj > 3) return ISOPO_ERR_UNSUPPORTED;
  StoredPrepArgs a;
  for (int i = 0; i <= B; ++i) a.off[i] = off_host[i];
  for (int h = 0; h < 3; ++h) {
    const int hh = h < n_proj ? h : 0;
    a.tag[h] = tag[hh]; a.off_dev[h] = off_dev[hh]; a.order_dev[h] = order_dev[hh]; a.tag_dev[h] = tag_dev[hh]; a.K[h] = K[hh];
  }
  int idx[256];
  for (int i = 0; i < B; ++i) idx[i] = i;
  // longest first; equal lengths keep their order
  std::stable_sort(idx, idx + B, [&](int x, int y) { return off_host[x + 1] - off_host[x] > off_host[y + 1] - off_host[y]; });
  for (int i = 0; i < B; ++i) a.order[i] = (uint8_t)idx[i];
  {
    LaunchScope scope(kIdPrep, st);
    k_prep_stored<<<std::max(1, (B * B + 2047) / 2048), 256, 0, st>>>(a, B, n_proj);
  }
  ISOPO_CUDA_TRY(cudaGetLastError());
  return ISOPO_OK;
}

isopo_status store_tag(const WsTag& tag, WsTag* tag_dev, cudaStream_t st) {
  k_store_tag<<<1, 32, 0, st>>>(tag, tag_dev);
  ISOPO_CUDA_TRY(cudaGetLastError());
  return ISOPO_OK;
}

isopo_status f32_seq_grad(const float* X, const float* dY, int d_in, int d_out, const int64_t* off_dev, int B,
                          float* G, cudaStream_t st) {
  dim3 grid((d_in + kT - 1) / kT, (d_out + kT - 1) / kT, B);
  if (grid.y > 65535 || grid.z > 65535) return ISOPO_ERR_UNSUPPORTED;
  {
    LaunchScope scope(kIdF32SeqGrad, st);
    k_f32_seq_grad<<<grid, 256, 0, st>>>(X, dY, d_in, d_out, off_dev, G);
  }
  ISOPO_CUDA_TRY(cudaGetLastError());
  return ISOPO_OK;
}

isopo_status f32_ntk(const float* G, int64_t N, int B, float* K, cudaStream_t st) {
  if (B > 65535) return ISOPO_ERR_UNSUPPORTED;
  {
    LaunchScope scope(kIdF32Ntk, st);
    k_f32_ntk<<<dim3(B, B), 256, 0, st>>>(G, N, B, K);
  }
  ISOPO_CUDA_TRY(cudaGetLastError());
  return ISOPO_OK;
}

isopo_status f32_gram(const float* X, const float* dY, int64_t T, int d_in, int d_out, const int32_t* tokseq, int B,
                      double* kacc, float* K, cudaStream_t st) {
  const int64_t nt = (T + kGT - 1) / kGT;
  if (nt > 65535) return ISOPO_ERR_UNSUPPORTED;
  ISOPO_CUDA_TRY(cudaMemsetAsync(kacc, 0, sizeof(double) * (size_t)B * B, st));
  {
    LaunchScope scope(kIdF32Gram, st);
    k_f32_gram<<<dim3((unsigned)nt, (unsigned)nt), 256, 0, st>>>(X, dY, T, d_in, d_out, tokseq, B, kacc);
  }
  ISOPO_CUDA_TRY(cudaGetLastError());
  {
    LaunchScope scope(kIdMirror, st);
    k_f32_gram_finish<<<(B * B + 255) / 256, 256, 0, st>>>(kacc, B, K);
  }
  ISOPO_CUDA_TRY(cudaGetLastError());
  return ISOPO_OK;
}

isopo_status f32_combine(const float* G, int64_t N, int B, const float* coeffs, float* dW, float beta, const WsTag* tag_dev,
                         const WsTag& tag, int32_t* info, cudaStream_t st) {
  const int grid = (int)std::min<int64_t>((N + 255) / 256, 148 * 8);
  {
    LaunchScope scope(kIdF32Combine, st);
    k_f32_combine<<<grid, 256, 0, st>>>(G, N, B, coeffs, dW, beta, tag_dev, tag, info);
  }
  ISOPO_CUDA_TRY(cudaGetLastError());
  return ISOPO_OK;
}

isopo_status f32_weight_grad(const float* X, const float* dY, int64_t T, int d_in, int d_out, const float* coeffs,
                             const int32_t* tokseq, float* dW, float beta, cudaStream_t st) {
  if (beta == 0.f) ISOPO_CUDA_TRY(cudaMemsetAsync(dW, 0, sizeof(float) * (size_t)d_in * d_out, st));
  const int gx = (d_in + kT - 1) / kT, gy = (d_out + kT - 1) / kT;
  if (gy > 65535) return ISOPO_ERR_UNSUPPORTED;
  // enough token slabs to fill the machine, each a multiple of the staging depth
  int64_t splits = std::max<int64_t>(1, std::min<int64_t>((T + 255) / 256, (148 * 4 + gx * gy - 1) / (gx * gy)));
  int64_t slab = ((T + splits - 1) / splits + kTK - 1) / kTK * kTK;
  splits = (T + slab - 1) / slab;
  {
    LaunchScope scope(kIdF32WeightGrad, st);
    k_f32_weight_grad<<<dim3(gx, gy, (unsigned)splits), 256, 0, st>>>(X, dY, T, d_in, d_out, coeffs, tokseq, dW, slab);
  }
  ISOPO_CUDA_TRY(cudaGetLastError());
  return ISOPO_OK;
}

}  // namespace isopo
