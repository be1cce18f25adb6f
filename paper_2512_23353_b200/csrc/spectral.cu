// Spectral form of the interacting transform (Alg. 2, last block: symmetric eigendecomposition of the
// NTK, every eigen-direction of the advantages divided by its eigenvalue plus the regulariser, then
// back to the sequence basis), with the spectrum as a second output.
//
// A cluster of eight CTAs (128 warps) diagonalises K by one-sided (Hestenes) Jacobi: W starts as K, V as the identity;
// a rotation of columns p and q, applied to both, makes the two columns of W orthogonal and keeps
// W = K V.  When all columns of W are orthogonal, K V = V diag(d): the columns of V are eigenvectors
// and d_k = v_k . w_k.  Column pairs follow the round-robin tournament (n - 1 steps of n / 2 disjoint
// pairs per sweep), one pair per warp and step, a cluster barrier between steps; the three inner
// products of a pair are accumulated in float64 (the decision whether to rotate rests on their ratio),
// the columns are float32.  W and V (256 KB each at B = 256) do not fit one SM's shared memory and
// live in the caller's workspace, which stays in the L2 (loads bypass the L1, which is not coherent
// between the SMs of the cluster).  A sweep is latency-bound: 255 steps of one L2 round trip, a
// reduction and a barrier each, and ~10 sweeps are needed.  This is the diagnostic variant (it
// returns the spectrum and can leave small directions out), not the fast path: the Cholesky solve
// of transform.cu is far faster.
#include "isopo_internal.h"

namespace isopo {

namespace {

constexpr int kThreads = 512;
constexpr int kClusterSize = 8;  // the portable maximum; 8 x 16 warps = the 128 pairs of a step at B = 256
constexpr int kLd = 256;        // column stride of W and V (floats); B <= kLd
constexpr int kMaxSweeps = 30;

struct SpectralParams {
  const float* K;
  const float* A;
  float* coeffs;
  float* eig;   // NULL or [B]
  float* W;     // [kLd][kLd] column-major
  float* V;
  int* rotations;  // running count of rotations applied, zeroed by the launcher
  int32_t* info;
  int B;
  float lambda, rel_cutoff;
};

// One launch serves up to ISOPO_MAX_BATCH layers that share A and B: cluster l works on layer l.
struct SpectralBatch {
  SpectralParams common;  // K, coeffs, eig, W, V, rotations, lambda are taken per layer
  const float* K[ISOPO_MAX_BATCH];
  float* coeffs[ISOPO_MAX_BATCH];
  float* eig[ISOPO_MAX_BATCH];
  float lambda[ISOPO_MAX_BATCH];
  char* ws;          // layer l uses ws + l * ws_stride
  size_t ws_stride;
};

__device__ __forceinline__ double warp_sum_d(double v) {
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;
}

// One column of kLd floats per warp: lane l holds elements 4l .. 4l+3 and 128+4l .. 128+4l+3.
struct Col { float4 lo, hi; };
__device__ __forceinline__ Col load_col(const float* base) {
  const int lane = threadIdx.x & 31;
  Col c;
  c.lo = __ldcg(reinterpret_cast<const float4*>(base + 4 * lane));
  c.hi = __ldcg(reinterpret_cast<const float4*>(base + 128 + 4 * lane));
  return c;
}
__device__ __forceinline__ void store_col(float* base, const Col& c) {
  const int lane = threadIdx.x & 31;
  *reinterpret_cast<float4*>(base + 4 * lane) = c.lo;
  *reinterpret_cast<float4*>(base + 128 + 4 * lane) = c.hi;
}
__device__ __forceinline__ double dot_cols(const Col& a, const Col& b) {
  double s = (double)a.lo.x * b.lo.x + (double)a.lo.y * b.lo.y + (double)a.lo.z * b.lo.z + (double)a.lo.w * b.lo.w;
  s += (double)a.hi.x * b.hi.x + (double)a.hi.y * b.hi.y + (double)a.hi.z * b.hi.z + (double)a.hi.w * b.hi.w;
  return s;
}
__device__ __forceinline__ void rotate(Col& p, Col& q, float cs, float sn) {
#define ISOPO_ROT(f)                          \
  {                                           \
    const float x = p.f, y = q.f;             \
    p.f = fmaf(cs, x, -sn * y);               \
    q.f = fmaf(sn, x, cs * y);                \
  }
  ISOPO_ROT(lo.x) ISOPO_ROT(lo.y) ISOPO_ROT(lo.z) ISOPO_ROT(lo.w)
  ISOPO_ROT(hi.x) ISOPO_ROT(hi.y) ISOPO_ROT(hi.z) ISOPO_ROT(hi.w)
#undef ISOPO_ROT
}

__device__ __forceinline__ void cluster_barrier() {  // every thread of the cluster; orders the global writes before it
  asm volatile("barrier.cluster.arrive.release.aligned;\nbarrier.cluster.wait.acquire.aligned;" ::: "memory");
}

__global__ void __cluster_dims__(kClusterSize, 1, 1) __launch_bounds__(kThreads)
k_spectral(const __grid_constant__ SpectralBatch batch) {
  __shared__ double s_d[kLd], s_f[kLd];
  __shared__ double s_fro2;
  const int layer = blockIdx.x / kClusterSize, rank = blockIdx.x % kClusterSize;  // one cluster per layer
  SpectralParams P = batch.common;
  P.K = batch.K[layer];
  P.coeffs = batch.coeffs[layer];
  P.eig = batch.eig[layer];
  P.lambda = batch.lambda[layer];
  P.W = reinterpret_cast<float*>(batch.ws + (size_t)layer * batch.ws_stride);
  P.V = P.W + (size_t)kLd * kLd;
  P.rotations = reinterpret_cast<int*>(P.V + (size_t)kLd * kLd);
  const int B = P.B, tid = threadIdx.x, lane = tid & 31, warp = tid >> 5, nwarps = kThreads / 32;
  const int gtid = rank * kThreads + tid, gthreads = kClusterSize * kThreads;
  float* W = P.W;  // read and written by every warp: no restrict, no read-only loads
  float* V = P.V;
  // W = K (symmetric: column c is row c), V = I; rows and columns past B are zero
  if (tid == 0) s_fro2 = 0.0;
  __syncthreads();
  double fro2 = 0.0;
  for (int e = gtid; e < kLd * kLd; e += gthreads) {  // every CTA fills its share
    const int c = e / kLd, r = e % kLd;
    const bool in = c < B && r < B;
    W[e] = in ? P.K[(size_t)c * B + r] : 0.f;
    V[e] = (in && r == c) ? 1.f : 0.f;
  }
  for (int e = tid; e < B * B; e += kThreads) {  // and sums all of K for itself
    const float k = P.K[e];
    fro2 += (double)k * k;
  }
  fro2 = warp_sum_d(fro2);
  if (lane == 0) atomicAdd(&s_fro2, fro2);
  __syncthreads();
  cluster_barrier();
  // A column of W shorter than this is rounding noise of the rotations (a rank-deficient K): it is left
  // alone, or the sweeps would for ever rotate noise that every rotation renews.  V stays orthogonal
  // whatever is skipped, so such columns of V still span the null space.  ||K||_F <= sqrt(B) d_max.
  const double null2 = 9e-14 * s_fro2;  // (3e-7 ||K||_F)^2

  const int n = B + (B & 1);  // an odd B plays with a phantom last column
  int sweeps = 0, seen = 0;
  bool converged = B < 2;
  while (!converged && sweeps < kMaxSweeps) {
    int rotated = 0;
    for (int step = 0; step < n - 1; ++step) {
      const int i = rank * nwarps + warp;  // this warp's pair of the step
      if (i < n / 2) {
        const int p = (step + i) % (n - 1);
        const int q = i == 0 ? n - 1 : (step + n - 1 - i) % (n - 1);
        if (p < B && q < B) {
          Col wp = load_col(W + (size_t)p * kLd), wq = load_col(W + (size_t)q * kLd);
          Col vp = load_col(V + (size_t)p * kLd), vq = load_col(V + (size_t)q * kLd);
          const double al = warp_sum_d(dot_cols(wp, wp)), be = warp_sum_d(dot_cols(wq, wq));
          const double ga = warp_sum_d(dot_cols(wp, wq));
          // warp-uniform: the sums are the same in every lane
          if (!(ga == 0.0 || fabs(ga) <= 5e-7 * sqrt(al * be) || al <= null2 || be <= null2)) {
            ++rotated;
            const double zeta = (be - al) / (2.0 * ga);
            const double t = (zeta >= 0.0 ? 1.0 : -1.0) / (fabs(zeta) + sqrt(1.0 + zeta * zeta));
            const double csd = 1.0 / sqrt(1.0 + t * t);
            const float cs = (float)csd, sn = (float)(csd * t);
            rotate(wp, wq, cs, sn);
            store_col(W + (size_t)p * kLd, wp);
            store_col(W + (size_t)q * kLd, wq);
            rotate(vp, vq, cs, sn);
            store_col(V + (size_t)p * kLd, vp);
            store_col(V + (size_t)q * kLd, vq);
          }
        }
      }
      cluster_barrier();  // the pairs of a step are disjoint; the next step reads what this one wrote
    }
    if (lane == 0 && rotated) atomicAdd(P.rotations, rotated);
    cluster_barrier();
    const int total = __ldcg(P.rotations);  // the same in every thread of the cluster
    converged = total == seen;
    seen = total;
    ++sweeps;
  }
  if (rank != 0) return;  // the rest is one CTA's work
  if (!converged && tid == 0) atomicCAS(P.info, 0, ISOPO_INFO_NO_CONVERGENCE | (layer << 16) | sweeps);

  // d_k = v_k . w_k (= v_k^T K v_k), y_k = v_k . A
  for (int k = warp; k < B; k += nwarps) {
    const Col v = load_col(V + (size_t)k * kLd), w = load_col(W + (size_t)k * kLd);
    Col a;
    const int r0 = 4 * lane, r1 = 128 + 4 * lane;
    a.lo = make_float4(r0 < B ? P.A[r0] : 0.f, r0 + 1 < B ? P.A[r0 + 1] : 0.f, r0 + 2 < B ? P.A[r0 + 2] : 0.f,
                       r0 + 3 < B ? P.A[r0 + 3] : 0.f);
    a.hi = make_float4(r1 < B ? P.A[r1] : 0.f, r1 + 1 < B ? P.A[r1 + 1] : 0.f, r1 + 2 < B ? P.A[r1 + 2] : 0.f,
                       r1 + 3 < B ? P.A[r1 + 3] : 0.f);
    const double d = warp_sum_d(dot_cols(v, w)), y = warp_sum_d(dot_cols(v, a));
    if (lane == 0) { s_d[k] = d; s_f[k] = y; }
  }
  __syncthreads();
  double dmax = -1e300;
  for (int k = 0; k < B; ++k) dmax = fmax(dmax, s_d[k]);
  __syncthreads();
  if (tid < B) {
    const double d = s_d[tid];
    const bool keep = d > (double)P.rel_cutoff * dmax;
    s_f[tid] = keep ? s_f[tid] / (d + (double)P.lambda) : 0.0;
    if (P.eig) {  // spectrum from the largest down: the rank of d among all (ties by index)
      int rank = 0;
      for (int k = 0; k < B; ++k) rank += (s_d[k] > d || (s_d[k] == d && k < tid)) ? 1 : 0;
      P.eig[rank] = (float)d;
    }
  }
  __syncthreads();
  if (tid < B) {
    double c = 0.0;
    for (int k = 0; k < B; ++k) c += (double)__ldcg(V + (size_t)k * kLd + tid) * s_f[k];
    P.coeffs[tid] = (float)c;
  }
}

}  // namespace

size_t spectral_workspace_bytes() { return sizeof(float) * 2 * (size_t)kLd * kLd + 256; }

isopo_status spectral_batched(int n, const float* const* K, const float* A, int B, const float* lambda,
                              float rel_cutoff, float* const* coeffs, float* const* eig, void* ws, int32_t* info,
                              cudaStream_t st) {
  if (B > kLd) return ISOPO_ERR_UNSUPPORTED;
  SpectralBatch T{};
  T.common.A = A; T.common.info = info; T.common.B = B; T.common.rel_cutoff = rel_cutoff;
  T.ws = (char*)ws;
  T.ws_stride = spectral_workspace_bytes();
  for (int l = 0; l < n; ++l) {
    T.K[l] = K[l];
    T.coeffs[l] = coeffs[l];
    T.eig[l] = eig ? eig[l] : nullptr;
    T.lambda[l] = lambda[l];
    // the rotation counter of layer l sits behind its W and V
    ISOPO_CUDA_TRY(cudaMemsetAsync(T.ws + (size_t)l * T.ws_stride + sizeof(float) * 2 * (size_t)kLd * kLd, 0, sizeof(int), st));
  }
  {
    LaunchScope scope(kIdTransform, st);
    k_spectral<<<n * kClusterSize, kThreads, 0, st>>>(T);
  }
  ISOPO_CUDA_TRY(cudaGetLastError());
  return ISOPO_OK;
}

isopo_status spectral(const float* K, const float* A, int B, float lambda, float rel_cutoff, float* coeffs, float* eig,
                      void* ws, int32_t* info, cudaStream_t st) {
  return spectral_batched(1, &K, A, B, &lambda, rel_cutoff, &coeffs, eig ? &eig : nullptr, ws, info, st);
}

}  // namespace isopo
