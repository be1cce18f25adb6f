// Advantage transform: one CTA turns (K, A) into the per-sequence coefficients.
//   simple variants  - per-row sums of K in float64, one warp per row
//   interacting      - Cholesky of the packed lower triangle of K + lambda*I in shared memory
//                      (float32), triangular solves by one warp, two refinement rounds with
//                      float64 residuals taken from the float32 K in global memory
#include "isopo_internal.h"

namespace isopo {

namespace {

constexpr int kThreads = 256;
constexpr int kMaxB = 256;

struct TransformParams {
  const float* K;
  const float* A;
  float* coeffs;
  int32_t* info;
  int B;
  int variant;
  float lambda;
  float p, q, r, reg_F, reg_G, reg_rel;
};

__device__ __forceinline__ int tri(int i, int j) { return i * (i + 1) / 2 + j; }  // i >= j

__device__ __forceinline__ double warp_sum(double v) {
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;
}

// Solves L L^T x = b for one right-hand side held in shared memory (overwritten by x); warp 0 only.
// Each lane owns entries lane, lane+32, ...
__device__ void warp_cholesky_solve(const float* __restrict__ Lp, float* __restrict__ v, int B) {
  const int lane = threadIdx.x & 31;
  // forward: L y = b, column sweep
  for (int k = 0; k < B; ++k) {
    __syncwarp();
    const float yk = v[k] / Lp[tri(k, k)];
    __syncwarp();
    if (lane == (k & 31)) v[k] = yk;
    for (int i = k + 1 + lane; i < B; i += 32) v[i] = fmaf(-Lp[tri(i, k)], yk, v[i]);
  }
  // backward: L^T x = y, row sweep
  for (int k = B - 1; k >= 0; --k) {
    __syncwarp();
    const float xk = v[k] / Lp[tri(k, k)];
    __syncwarp();
    if (lane == (k & 31)) v[k] = xk;
    for (int i = lane; i < k; i += 32) v[i] = fmaf(-Lp[tri(k, i)], xk, v[i]);
  }
  __syncwarp();
}

__global__ void __launch_bounds__(kThreads) k_transform(TransformParams P) {
  extern __shared__ __align__(16) unsigned char smem_raw[];
  __shared__ double s_trace;
  __shared__ float s_pivot;
  __shared__ int s_fail;
  const int B = P.B, tid = threadIdx.x, lane = tid & 31, warp = tid >> 5, nwarps = kThreads / 32;
  const float* __restrict__ K = P.K;

  if (P.variant == ISOPO_VAR_REINFORCE) {
    for (int i = tid; i < B; i += kThreads) P.coeffs[i] = P.A[i];
    return;
  }

  if (P.variant != ISOPO_VAR_INTERACTING) {
    // trace of K
    double tr = 0.0;
    for (int i = tid; i < B; i += kThreads) tr += (double)K[(size_t)i * B + i];
    tr = warp_sum(tr);
    if (tid == 0) s_trace = 0.0;
    __syncthreads();
    if (lane == 0) atomicAdd(&s_trace, tr);
    __syncthreads();
    const double trace = s_trace;
    for (int i = warp; i < B; i += nwarps) {
      double sq = 0.0;
      for (int j = lane; j < B; j += 32) {
        const double kij = (double)K[(size_t)i * B + j];
        sq += kij * kij;
      }
      sq = warp_sum(sq);
      if (lane == 0) {
        const double n2 = (double)K[(size_t)i * B + i];
        const double F2 = P.variant == ISOPO_VAR_NORMALISED_RAW ? sq / (double)B : sq / trace;
        const double a = (double)P.A[i], lam = (double)P.lambda;
        double c;
        switch (P.variant) {
          case ISOPO_VAR_NORMALISED:
          case ISOPO_VAR_NORMALISED_RAW: c = a / sqrt(F2 + lam); break;
          case ISOPO_VAR_DIRECTION: c = a / (F2 / n2 + lam); break;
          case ISOPO_VAR_EUCLID: c = a / sqrt(n2 + lam); break;
          default: {  // ISOPO_VAR_GENERAL
            const double eps = 1e-8;
            const double rF = sqrt(F2 + (double)P.reg_F + eps);
            const double rG = sqrt(n2 + (double)P.reg_G + eps);
            const double rR = sqrt(F2 / n2 + (double)P.reg_rel + eps);
            c = a * pow(rF, (double)P.p) * pow(rG, (double)P.q) * pow(rR, (double)P.r);
          }
        }
        P.coeffs[i] = (float)c;
      }
    }
    return;
  }

  // ---------------- interacting: (K + lambda I) c = A ----------------
  float* Lp = reinterpret_cast<float*>(smem_raw);                    // packed lower triangle
  float* vec = Lp + (size_t)B * (B + 1) / 2;                          // right-hand side / correction
  double* sol = reinterpret_cast<double*>(vec + ((B + 3) & ~3) + ((((size_t)B * (B + 1) / 2) & 1) ? 1 : 0));
  if (tid == 0) s_fail = 0;
  for (int e = tid; e < B * B; e += kThreads) {
    const int i = e / B, j = e % B;
    if (j <= i) Lp[tri(i, j)] = K[e] + (i == j ? P.lambda : 0.f);
  }
  __syncthreads();
  // left-looking Cholesky, thread i owns row i
  for (int k = 0; k < B; ++k) {
    float s = 0.f;
    const int i = tid;
    if (i >= k && i < B) {
      const float* ri = Lp + tri(i, 0);
      const float* rk = Lp + tri(k, 0);
      s = ri[k];
      for (int p = 0; p < k; ++p) s = fmaf(-ri[p], rk[p], s);
      if (i == k) s_pivot = s;
    }
    __syncthreads();
    const float piv = s_pivot;
    if (!(piv > 0.f)) {
      if (tid == 0) { s_fail = 1; atomicCAS(P.info, 0, k + 1); }
      break;
    }
    if (i >= k && i < B) Lp[tri(i, k)] = i == k ? sqrtf(piv) : s * rsqrtf(piv);
    __syncthreads();
  }
  __syncthreads();
  if (s_fail) {
    for (int i = tid; i < B; i += kThreads) P.coeffs[i] = 0.f;
    return;
  }
  // initial solve + two refinement rounds
  for (int i = tid; i < B; i += kThreads) { vec[i] = P.A[i]; sol[i] = 0.0; }
  __syncthreads();
  for (int round = 0; round < 3; ++round) {
    if (warp == 0) warp_cholesky_solve(Lp, vec, B);
    __syncthreads();
    for (int i = tid; i < B; i += kThreads) sol[i] += (double)vec[i];
    __syncthreads();
    if (round == 2) break;
    // residual r = A - (K + lambda I) sol in float64
    for (int i = warp; i < B; i += nwarps) {
      double acc = 0.0;
      for (int j = lane; j < B; j += 32) acc += (double)K[(size_t)i * B + j] * sol[j];
      acc = warp_sum(acc);
      if (lane == 0) vec[i] = (float)((double)P.A[i] - acc - (double)P.lambda * sol[i]);
    }
    __syncthreads();
  }
  for (int i = tid; i < B; i += kThreads) P.coeffs[i] = (float)sol[i];
}

}  // namespace

isopo_status transform(const float* K, const float* A, int B, isopo_variant v, float lambda, const float* g,
                       float* coeffs, int32_t* info, cudaStream_t st) {
  TransformParams P{};
  P.K = K; P.A = A; P.coeffs = coeffs; P.info = info; P.B = B; P.variant = (int)v; P.lambda = lambda;
  if (v == ISOPO_VAR_GENERAL) { P.p = g[0]; P.q = g[1]; P.r = g[2]; P.reg_F = g[3]; P.reg_G = g[4]; P.reg_rel = g[5]; }
  size_t smem = 0;
  if (v == ISOPO_VAR_INTERACTING) {
    if (B > kMaxB) return ISOPO_ERR_UNSUPPORTED;
    smem = sizeof(float) * ((size_t)B * (B + 1) / 2 + (size_t)B + 8) + sizeof(double) * (size_t)B + 16;
    static bool attr_set = false;  // idempotent; a race only repeats the same call
    if (!attr_set) {
      ISOPO_CUDA_TRY(cudaFuncSetAttribute(k_transform, cudaFuncAttributeMaxDynamicSharedMemorySize, 200 * 1024));
      attr_set = true;
    }
  }
  k_transform<<<1, kThreads, smem, st>>>(P);
  ISOPO_CUDA_TRY(cudaGetLastError());
  return ISOPO_OK;
}

}  // namespace isopo
