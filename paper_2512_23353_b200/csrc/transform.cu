// Advantage transform: one CTA turns (K, A) into the per-sequence coefficients.
//   simple variants  - per-row sums of K in float64, one warp per row
//   interacting      - blocked Cholesky of K + lambda*I in shared memory (float32, 32 x 32 blocks,
//                      warp-level diagonal factorisation), blocked triangular solves, then up to
//                      two refinement rounds with float64 residuals taken from the float32 K,
//                      stopped once the relative residual is below 1e-7
#include "isopo_internal.h"

namespace isopo {

namespace {

constexpr int kThreads = 512;
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
  const float* rel_state;  // NULL, or the running means {E[F^2], E[||G||^2], E[F^2/||G||^2], updates}: the
                           // regularisers above are then factors of these (relative regularisation)
};

// One launch serves up to ISOPO_MAX_BATCH layers that share A and the variant: CTA l works on layer l.
struct TransformBatch {
  TransformParams common;  // K, coeffs, lambda, rel_state are taken from the arrays below
  const float* K[ISOPO_MAX_BATCH];
  float* coeffs[ISOPO_MAX_BATCH];
  const float* rel_state[ISOPO_MAX_BATCH];
  float lambda[ISOPO_MAX_BATCH];
};


__device__ __forceinline__ double warp_sum(double v) {
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;
}

// ---------------------------------------------------------------------------------------------
// Interacting variant: blocked Cholesky in shared memory.
//
// K + lambda*I is held as 32 x 32 blocks (lower block triangle, block (I,J) at slot I(I+1)/2+J),
// every block column-major: element (r, c) at [c*32 + r], so that a warp whose lane owns row r
// reads a block column without bank conflicts and 4 consecutive rows form one float4.
// Per block column J:  (1) one warp per block below the diagonal solves X L_JJ^T = A_IJ by
// substitution (lane = row), while a spare warp inverts L_JJ for the solve phase;  (2) one warp per
// trailing block does the rank-32 update with 4 x 8 register tiles; block (J+1, J+1) is updated
// first, by all warps together, and warp 0 then factors it in registers (shuffles), so the serial
// pivot chain of the next column runs beside the other warps' updates instead of after them.  The triangular solves with the
// right-hand side use the stored inverses of the diagonal blocks.
// ---------------------------------------------------------------------------------------------
constexpr int kNB = 32;
constexpr int kBlk = kNB * kNB;

__device__ __forceinline__ int blk_slot(int I, int J) { return I * (I + 1) / 2 + J; }

// Column sums over the warp: on entry lane l holds r[c] = M[l][c]; on return r[0] of lane c holds
// sum_l M[l][c].  Recursive halving: 31 shuffles for all 32 sums.
__device__ __forceinline__ float warp_column_sums(float (&r)[kNB]) {
  const int lane = threadIdx.x & 31;
#pragma unroll
  for (int o = 16; o >= 1; o >>= 1) {
    const bool up = (lane & o) != 0;
#pragma unroll
    for (int idx = 0; idx < o; ++idx) {
      const float send = up ? r[idx] : r[idx + o];
      const float keep = up ? r[idx + o] : r[idx];
      r[idx] = keep + __shfl_xor_sync(0xffffffffu, send, o);
    }
  }
  return r[0];
}

// Pointer types of the block helpers.  The factor lives either in this CTA's shared memory (no other writer: the
// pointers may be restrict-qualified) or, for more than 256 sequences, in a workspace that stays in the L2, where a
// block written by one warp is read by others after a CTA barrier: plain loads only, never the read-only path.
template <bool kInWorkspace> struct BlkPtr { typedef float* __restrict__ rw; typedef const float* __restrict__ ro; };
template <> struct BlkPtr<true> { typedef float* rw; typedef const float* ro; };

// Factors the 32 x 32 diagonal block D (column-major, symmetric input) in place into its lower
// Cholesky factor and writes 1 / L_kk to rd[k].  One warp.
// Returns 0, or the 1-based local index of the first non-positive pivot.
template <bool kW>
__device__ __noinline__ int warp_factor_diag(typename BlkPtr<kW>::rw D, float* __restrict__ rd) {
  const int lane = threadIdx.x & 31;
  float r[kNB];
#pragma unroll
  for (int c = 0; c < kNB; ++c) r[c] = D[c * kNB + lane];  // row `lane`
  int fail = 0;
  float rdiag = 0.f;  // 1 / L[lane][lane]
#pragma unroll
  for (int k = 0; k < kNB; ++k) {
    const float d = __shfl_sync(0xffffffffu, r[k], k);
    if (!(d > 0.f) && fail == 0) fail = k + 1;
    const float rs = rsqrtf(d);
    if (lane == k) rdiag = rs;
    r[k] = lane == k ? d * rs : r[k] * rs;  // L[lane][k] (rows above k hold junk, never used)
#pragma unroll
    for (int j = k + 1; j < kNB; ++j) {
      const float ljk = __shfl_sync(0xffffffffu, r[k], j);
      r[j] = fmaf(-r[k], ljk, r[j]);
    }
  }
#pragma unroll
  for (int c = 0; c < kNB; ++c) D[c * kNB + lane] = c <= lane ? r[c] : 0.f;
  rd[lane] = rdiag;
  return fail;
}

// Inv = L^-1 (column-major) for the factored diagonal block D with rd[k] = 1 / L_kk.  One warp.
// Column sweep: lane j solves L z = e_j; after step k, z[k] = Inv[k][j] is final.
template <bool kW>
__device__ __noinline__ void warp_invert_factor(typename BlkPtr<kW>::ro D, const float* __restrict__ rd,
                                                float* __restrict__ Inv) {
  const int lane = threadIdx.x & 31;
  float z[kNB];
#pragma unroll
  for (int i = 0; i < kNB; ++i) z[i] = i == lane ? 1.f : 0.f;
#pragma unroll
  for (int k = 0; k < kNB; ++k) {
    z[k] *= rd[k];
#pragma unroll
    for (int i = k + 1; i < kNB; ++i) z[i] = fmaf(-D[k * kNB + i], z[k], z[i]);  // L[i][k], broadcast
  }
#pragma unroll
  for (int i = 0; i < kNB; ++i) Inv[lane * kNB + i] = z[i];
}

// X L^T = A for one 32 x 32 block A (in place); lane owns a row.  L: factored diagonal block,
// rd[k] = 1 / L_kk.  Column k of X is final after step k and is eliminated from the later columns.
template <bool kW>
__device__ __noinline__ void warp_solve_panel(typename BlkPtr<kW>::rw A, typename BlkPtr<kW>::ro L,
                                              const float* __restrict__ rd) {
  const int lane = threadIdx.x & 31;
  float a[kNB];
#pragma unroll
  for (int c = 0; c < kNB; ++c) a[c] = A[c * kNB + lane];
#pragma unroll
  for (int k = 0; k < kNB; ++k) {
    a[k] *= rd[k];
#pragma unroll
    for (int j = k + 1; j < kNB; ++j) a[j] = fmaf(-a[k], L[k * kNB + j], a[j]);  // L[j][k], broadcast
  }
#pragma unroll
  for (int c = 0; c < kNB; ++c) A[c * kNB + lane] = a[c];
}

// C -= A * Bm^T for 32 x 32 blocks (all column-major); lane computes a 4 x 8 sub-tile.
template <bool kW>
__device__ __noinline__ void warp_rank32_update(typename BlkPtr<kW>::rw C, typename BlkPtr<kW>::ro A,
                                                typename BlkPtr<kW>::ro Bm) {
  const int lane = threadIdx.x & 31, r0 = (lane & 7) * 4, c0 = (lane >> 3) * 8;
  float4 acc[8];
#pragma unroll
  for (int c = 0; c < 8; ++c) acc[c] = *reinterpret_cast<const float4*>(C + (c0 + c) * kNB + r0);
#pragma unroll 8
  for (int p = 0; p < kNB; ++p) {
    const float4 a = *reinterpret_cast<const float4*>(A + p * kNB + r0);
    const float4 b0 = *reinterpret_cast<const float4*>(Bm + p * kNB + c0);
    const float4 b1 = *reinterpret_cast<const float4*>(Bm + p * kNB + c0 + 4);
    const float b[8] = {b0.x, b0.y, b0.z, b0.w, b1.x, b1.y, b1.z, b1.w};
#pragma unroll
    for (int c = 0; c < 8; ++c) {
      acc[c].x = fmaf(-a.x, b[c], acc[c].x);
      acc[c].y = fmaf(-a.y, b[c], acc[c].y);
      acc[c].z = fmaf(-a.z, b[c], acc[c].z);
      acc[c].w = fmaf(-a.w, b[c], acc[c].w);
    }
  }
#pragma unroll
  for (int c = 0; c < 8; ++c) *reinterpret_cast<float4*>(C + (c0 + c) * kNB + r0) = acc[c];
}

// Solves L L^T x = v in place (v in shared memory, nb*32 entries) with the blocked factor.
template <bool kW>
__device__ __noinline__ void block_cholesky_solve(typename BlkPtr<kW>::ro Lb, const float* __restrict__ InvD,
                                                  float* __restrict__ v, int nb) {
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, nwarps = blockDim.x >> 5;
  // forward: L y = v
  for (int J = 0; J < nb; ++J) {
    if (warp == 0) {
      const float* Inv = InvD + J * kBlk;
      float acc0 = 0.f, acc1 = 0.f;
#pragma unroll
      for (int k = 0; k < kNB; k += 2) {
        acc0 = fmaf(Inv[k * kNB + lane], v[J * kNB + k], acc0);
        acc1 = fmaf(Inv[(k + 1) * kNB + lane], v[J * kNB + k + 1], acc1);
      }
      __syncwarp();
      v[J * kNB + lane] = acc0 + acc1;
    }
    __syncthreads();
    for (int I = J + 1 + warp; I < nb; I += nwarps) {
      const float* L = Lb + blk_slot(I, J) * kBlk;
      float acc0 = v[I * kNB + lane], acc1 = 0.f;
#pragma unroll
      for (int p = 0; p < kNB; p += 2) {
        acc0 = fmaf(-L[p * kNB + lane], v[J * kNB + p], acc0);
        acc1 = fmaf(-L[(p + 1) * kNB + lane], v[J * kNB + p + 1], acc1);
      }
      v[I * kNB + lane] = acc0 + acc1;
    }
    __syncthreads();
  }
  // backward: L^T x = y; lane owns a row of the block, column sums by recursive halving
  for (int J = nb - 1; J >= 0; --J) {
    if (warp == 0) {
      const float* Inv = InvD + J * kBlk;
      const float yj = v[J * kNB + lane];
      float r[kNB];
#pragma unroll
      for (int i = 0; i < kNB; ++i) r[i] = Inv[i * kNB + lane] * yj;  // Inv[lane][i] y_lane
      v[J * kNB + lane] = warp_column_sums(r);                        // x_i = sum_k Inv[k][i] y_k
    }
    __syncthreads();
    for (int I = warp; I < J; I += nwarps) {
      const float* L = Lb + blk_slot(J, I) * kBlk;  // y_I -= L_JI^T x_J
      const float xj = v[J * kNB + lane];
      float r[kNB];
#pragma unroll
      for (int i = 0; i < kNB; ++i) r[i] = L[i * kNB + lane] * xj;
      v[I * kNB + lane] -= warp_column_sums(r);
    }
    __syncthreads();
  }
}

// Interacting variant, (K + lambda I) c = A: blocked Cholesky of the lower block triangle held at Lb (nb(nb+1)/2
// blocks; shared memory, or the workspace with kW), the inverse diagonal factors at InvD, then the solve and up to
// two refinement rounds.  Called by every thread of the CTA; `layer` tags a failed pivot in *info.
template <bool kW>
__device__ __forceinline__ void interacting_solve(const TransformParams& P, typename BlkPtr<kW>::rw Lb, float* InvD,
                                                  float* vec, double* sol, float* rdiag, double& s_trace, double& s_res,
                                                  int& s_fail, int layer) {
  const int B = P.B, tid = threadIdx.x, lane = tid & 31, warp = tid >> 5, nwarps = kThreads / 32;
  const float* __restrict__ K = P.K;
  const int nb = (B + kNB - 1) / kNB, Bp = nb * kNB;
  if (tid == 0) s_fail = 0;
  // load the lower block triangle.  K is symmetric, so row j of K read along i gives column j of
  // the blocks; float4 loads, eight in flight per thread, when B is a multiple of 4.
  if ((B & 3) == 0) {
    const int nvec = B * B / 4;
    for (int base = tid; base < nvec; base += kThreads * 8) {
      float4 val[8];
#pragma unroll
      for (int u = 0; u < 8; ++u) {
        const int e = base + u * kThreads;
        val[u] = e < nvec ? __ldg(reinterpret_cast<const float4*>(K) + e) : make_float4(0.f, 0.f, 0.f, 0.f);
      }
#pragma unroll
      for (int u = 0; u < 8; ++u) {
        const int e = base + u * kThreads;
        if (e >= nvec) continue;
        const int j = (e * 4) / B, i = (e * 4) % B, I = i / kNB, J = j / kNB;
        if (I < J) continue;
        float4 w = val[u];
        if (i == j) w.x += P.lambda;
        if (i + 1 == j) w.y += P.lambda;
        if (i + 2 == j) w.z += P.lambda;
        if (i + 3 == j) w.w += P.lambda;
        *reinterpret_cast<float4*>(Lb + blk_slot(I, J) * kBlk + (j % kNB) * kNB + (i % kNB)) = w;
      }
    }
  } else {
    for (int e = tid; e < B * B; e += kThreads) {
      const int j = e / B, i = e % B, I = i / kNB, J = j / kNB;
      if (I >= J) Lb[blk_slot(I, J) * kBlk + (j % kNB) * kNB + (i % kNB)] = K[e] + (i == j ? P.lambda : 0.f);
    }
  }
  // identity padding of the last block row / column
  for (int e = tid; e < (Bp - B) * Bp; e += kThreads) {
    const int i = B + e / Bp, j = e % Bp;  // rows B..Bp-1, all columns j <= i
    if (j <= i || j / kNB == i / kNB)
      Lb[blk_slot(i / kNB, j / kNB) * kBlk + (j % kNB) * kNB + (i % kNB)] = i == j ? 1.f : 0.f;
  }
  __syncthreads();
  if (warp == 0) {
    const int f = warp_factor_diag<kW>(Lb, rdiag);
    if (f != 0 && lane == 0) s_fail = f;
  }
  __syncthreads();
  for (int J = 0; J < nb && !s_fail; ++J) {
    const float* Ljj = Lb + blk_slot(J, J) * kBlk;
    // panel: blocks (I, J) below the diagonal on warps 0 .. nwarps-2; the last warp inverts L_JJ
    if (warp == nwarps - 1) warp_invert_factor<kW>(Ljj, rdiag + J * kNB, InvD + J * kBlk);
    else
      for (int I = J + 1 + warp; I < nb; I += nwarps - 1) warp_solve_panel<kW>(Lb + blk_slot(I, J) * kBlk, Ljj, rdiag + J * kNB);
    __syncthreads();
    // trailing blocks (I, Kc) with I >= Kc > J; t = a(a+1)/2 + rem -> I = J+1+a, Kc = J+1+rem.
    // t = 0 is the next diagonal block: all warps update it together, then warp 0 factors it while the
    // others work through the rest
    const int m = nb - 1 - J, ntrail = m * (m + 1) / 2;
    if (m > 0) {
      // all warps: rank-32 update of the next diagonal block, kNB / nwarps columns each (lane = row)
      float* Dn = Lb + blk_slot(J + 1, J + 1) * kBlk;
      const float* Pn = Lb + blk_slot(J + 1, J) * kBlk;
      constexpr int kColsPerWarp = kNB / (kThreads / 32);
      float acc[kColsPerWarp];
#pragma unroll
      for (int c = 0; c < kColsPerWarp; ++c) acc[c] = Dn[(warp * kColsPerWarp + c) * kNB + lane];
#pragma unroll 8
      for (int p = 0; p < kNB; ++p) {
        const float a = Pn[p * kNB + lane];
#pragma unroll
        for (int c = 0; c < kColsPerWarp; ++c) acc[c] = fmaf(-a, Pn[p * kNB + warp * kColsPerWarp + c], acc[c]);
      }
#pragma unroll
      for (int c = 0; c < kColsPerWarp; ++c) Dn[(warp * kColsPerWarp + c) * kNB + lane] = acc[c];
      __syncthreads();
      if (warp == 0) {
        const int f = warp_factor_diag<kW>(Dn, rdiag + (J + 1) * kNB);
        if (f != 0 && lane == 0) s_fail = (J + 1) * kNB + f;
      } else {
        for (int t = warp; t < ntrail; t += nwarps - 1) {
          int a = 0, rem = t;
          while (rem > a) { rem -= a + 1; ++a; }
          const int I = J + 1 + a, Kc = J + 1 + rem;
          warp_rank32_update<kW>(Lb + blk_slot(I, Kc) * kBlk, Lb + blk_slot(I, J) * kBlk, Lb + blk_slot(Kc, J) * kBlk);
        }
      }
    }
    __syncthreads();
  }
  __syncthreads();
  if (s_fail) {
    if (tid == 0) atomicCAS(P.info, 0, s_fail + (layer << 16));
    for (int i = tid; i < B; i += kThreads) P.coeffs[i] = 0.f;
    return;
  }
  // solve, then refinement rounds with a float64 residual while it is above float32 round-off
  double anorm2 = 0.0;
  for (int i = tid; i < Bp; i += kThreads) {
    const float a = i < B ? P.A[i] : 0.f;
    vec[i] = a;
    sol[i] = 0.0;
    anorm2 += (double)a * a;
  }
  anorm2 = warp_sum(anorm2);
  if (tid == 0) { s_trace = 0.0; s_res = 0.0; }
  __syncthreads();
  if (lane == 0) atomicAdd(&s_trace, anorm2);
  __syncthreads();
  anorm2 = s_trace;
  for (int round = 0; round < 3; ++round) {
    block_cholesky_solve<kW>(Lb, InvD, vec, nb);
    for (int i = tid; i < Bp; i += kThreads) sol[i] += (double)vec[i];
    __syncthreads();
    if (round == 2) break;
    double rn2 = 0.0;
    for (int i0 = warp * 4; i0 < B; i0 += nwarps * 4) {  // four rows per warp pass: independent loads
      double acc[4] = {0.0, 0.0, 0.0, 0.0};
      if ((B & 3) == 0) {
        for (int j0 = lane * 4; j0 < B; j0 += 256) {  // two float4 per lane and row in flight
          float4 kv[4][2];
#pragma unroll
          for (int u = 0; u < 4; ++u)
#pragma unroll
            for (int h = 0; h < 2; ++h) {
              const int j = j0 + h * 128;
              kv[u][h] = (i0 + u < B && j < B) ? __ldg(reinterpret_cast<const float4*>(K + (size_t)(i0 + u) * B + j))
                                              : make_float4(0.f, 0.f, 0.f, 0.f);
            }
#pragma unroll
          for (int h = 0; h < 2; ++h) {
            const int j = j0 + h * 128;
            if (j >= B) continue;
            const double s0 = sol[j], s1 = sol[j + 1], s2 = sol[j + 2], s3 = sol[j + 3];
#pragma unroll
            for (int u = 0; u < 4; ++u)
              acc[u] += (double)kv[u][h].x * s0 + (double)kv[u][h].y * s1 + (double)kv[u][h].z * s2 +
                        (double)kv[u][h].w * s3;
          }
        }
      } else {
        for (int j = lane; j < B; j += 32) {
          const double sj = sol[j];
#pragma unroll
          for (int u = 0; u < 4; ++u)
            if (i0 + u < B) acc[u] += (double)K[(size_t)(i0 + u) * B + j] * sj;
        }
      }
#pragma unroll
      for (int u = 0; u < 4; ++u) {
        const double a = warp_sum(acc[u]);
        if (lane == 0 && i0 + u < B) {
          const double r = (double)P.A[i0 + u] - a - (double)P.lambda * sol[i0 + u];
          vec[i0 + u] = (float)r;
          rn2 += r * r;
        }
      }
    }
    if (lane == 0) atomicAdd(&s_res, rn2);
    __syncthreads();
    const bool done = s_res <= 1e-14 * anorm2;  // relative residual below 1e-7
    __syncthreads();
    if (tid == 0) s_res = 0.0;
    if (done) break;
  }
  for (int i = tid; i < B; i += kThreads) P.coeffs[i] = (float)sol[i];
}

__global__ void __launch_bounds__(kThreads) k_transform(const __grid_constant__ TransformBatch batch) {
  extern __shared__ __align__(16) unsigned char smem_raw[];
  TransformParams P = batch.common;
  P.K = batch.K[blockIdx.x];
  P.coeffs = batch.coeffs[blockIdx.x];
  P.rel_state = batch.rel_state[blockIdx.x];
  P.lambda = batch.lambda[blockIdx.x];
  __shared__ double s_trace, s_res;
  __shared__ int s_fail;
  const int B = P.B, tid = threadIdx.x, lane = tid & 31, warp = tid >> 5, nwarps = kThreads / 32;
  const float* __restrict__ K = P.K;
  if (P.rel_state) {
    // reg(val) = val + regularization * expectation(val) of the generalised re-scaling figure: each
    // regulariser is its factor times the running mean of the quantity it is added to
    const float eF = P.rel_state[0], eG = P.rel_state[1], eR = P.rel_state[2];
    switch (P.variant) {
      case ISOPO_VAR_NORMALISED:
      case ISOPO_VAR_NORMALISED_RAW: P.lambda *= eF; break;
      case ISOPO_VAR_DIRECTION: P.lambda *= eR; break;
      case ISOPO_VAR_EUCLID:
      case ISOPO_VAR_INTERACTING: P.lambda *= eG; break;  // mean eigenvalue of K = tr K / B = E[||G||^2]
      default: P.reg_F *= eF; P.reg_G *= eG; P.reg_rel *= eR;
    }
  }

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
  const int nb = (B + kNB - 1) / kNB, Bp = nb * kNB;
  float* Lb = reinterpret_cast<float*>(smem_raw);           // nb(nb+1)/2 blocks
  float* InvD = Lb + (size_t)(nb * (nb + 1) / 2) * kBlk;    // nb inverse diagonal factors
  float* vec = InvD + (size_t)nb * kBlk;                    // Bp floats
  double* sol = reinterpret_cast<double*>(vec + Bp);        // Bp doubles (8-byte aligned: all counts even)
  float* rdiag = reinterpret_cast<float*>(sol + Bp);        // Bp floats: 1 / L_kk
  interacting_solve<false>(P, Lb, InvD, vec, sol, rdiag, s_trace, s_res, s_fail, (int)blockIdx.x);
}

// The interacting variant for more sequences than the shared-memory kernel holds: the block triangle (2.1 MB at
// 1024 sequences) lives in a workspace that stays in the L2, everything else as above.  One CTA.
constexpr int kMaxLargeB = ISOPO_MAX_LARGE_SEQS;
__global__ void __launch_bounds__(kThreads) k_transform_large(const TransformParams P, float* scratch) {
  extern __shared__ __align__(16) unsigned char smem_raw[];
  __shared__ double s_trace, s_res;
  __shared__ int s_fail;
  const int nb = (P.B + kNB - 1) / kNB, Bp = nb * kNB;
  float* InvD = reinterpret_cast<float*>(smem_raw);         // nb inverse diagonal factors
  float* vec = InvD + (size_t)nb * kBlk;                    // Bp floats
  double* sol = reinterpret_cast<double*>(vec + Bp);        // Bp doubles
  float* rdiag = reinterpret_cast<float*>(sol + Bp);        // Bp floats
  interacting_solve<true>(P, scratch, InvD, vec, sol, rdiag, s_trace, s_res, s_fail, 0);
}

// Running means for the relative regulariser.  state = {E[F^2], E[||G||^2], E[F^2 / ||G||^2], number of updates};
// the first update stores this microbatch's means, later ones blend: s <- decay * s + (1 - decay) * mean.
__global__ void __launch_bounds__(kThreads) k_reg_ema(const float* __restrict__ K, int B, float decay,
                                                      float* __restrict__ state) {
  __shared__ double s_trace, s_f2, s_rel;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5, nwarps = kThreads / 32;
  double tr = 0.0;
  for (int i = tid; i < B; i += kThreads) tr += (double)K[(size_t)i * B + i];
  tr = warp_sum(tr);
  if (tid == 0) { s_trace = 0.0; s_f2 = 0.0; s_rel = 0.0; }
  __syncthreads();
  if (lane == 0) atomicAdd(&s_trace, tr);
  __syncthreads();
  const double trace = s_trace;
  double f2_sum = 0.0, rel_sum = 0.0;
  for (int i = warp; i < B; i += nwarps) {
    double sq = 0.0;
    for (int j = lane; j < B; j += 32) {
      const double kij = (double)K[(size_t)i * B + j];
      sq += kij * kij;
    }
    sq = warp_sum(sq);
    const double F2 = sq / trace;
    f2_sum += F2;
    rel_sum += F2 / (double)K[(size_t)i * B + i];
  }
  if (lane == 0) { atomicAdd(&s_f2, f2_sum); atomicAdd(&s_rel, rel_sum); }
  __syncthreads();
  if (tid == 0) {
    const double m[3] = {s_f2 / B, trace / B, s_rel / B};
    const bool first = state[3] == 0.f;
    for (int k = 0; k < 3; ++k)
      state[k] = (float)(first ? m[k] : (double)decay * (double)state[k] + (1.0 - (double)decay) * m[k]);
    state[3] += 1.f;
  }
}

}  // namespace

isopo_status reg_ema_update(const float* K, int B, float decay, float* state, cudaStream_t st) {
  {
    LaunchScope scope(kIdTransform, st);
    k_reg_ema<<<1, kThreads, 0, st>>>(K, B, decay, state);
  }
  ISOPO_CUDA_TRY(cudaGetLastError());
  return ISOPO_OK;
}

isopo_status transform_batched(int n, const float* const* K, const float* A, int B, isopo_variant v, const float* lambda,
                               const float* g, const float* const* rel_state, float* const* coeffs, int32_t* info,
                               cudaStream_t st) {
  TransformBatch T{};
  TransformParams& P = T.common;
  P.A = A; P.info = info; P.B = B; P.variant = (int)v;
  if (v == ISOPO_VAR_GENERAL) { P.p = g[0]; P.q = g[1]; P.r = g[2]; P.reg_F = g[3]; P.reg_G = g[4]; P.reg_rel = g[5]; }
  for (int l = 0; l < n; ++l) {
    T.K[l] = K[l];
    T.coeffs[l] = coeffs[l];
    T.rel_state[l] = rel_state ? rel_state[l] : nullptr;
    T.lambda[l] = lambda[l];
  }
  size_t smem = 0;
  if (v == ISOPO_VAR_INTERACTING) {
    if (B > kMaxB) return ISOPO_ERR_UNSUPPORTED;
    const size_t nb = (size_t)(B + kNB - 1) / kNB;
    smem = sizeof(float) * ((nb * (nb + 1) / 2 + nb) * kBlk + 2 * nb * kNB) + sizeof(double) * nb * kNB;
    ISOPO_CUDA_TRY(cudaFuncSetAttribute(k_transform, cudaFuncAttributeMaxDynamicSharedMemorySize, 200 * 1024));
  }
  {
    LaunchScope scope(kIdTransform, st);
    k_transform<<<n, kThreads, smem, st>>>(T);
  }
  ISOPO_CUDA_TRY(cudaGetLastError());
  return ISOPO_OK;
}

size_t transform_large_workspace_bytes(int B) {
  const size_t nb = (size_t)(B + kNB - 1) / kNB;
  return sizeof(float) * (nb * (nb + 1) / 2) * kBlk;
}

isopo_status transform_large(const float* K, const float* A, int B, float lambda, float* coeffs, float* scratch,
                             int32_t* info, cudaStream_t st) {
  if (B < 1 || B > kMaxLargeB) return ISOPO_ERR_UNSUPPORTED;
  TransformParams P{};
  P.K = K; P.A = A; P.coeffs = coeffs; P.info = info; P.B = B; P.variant = (int)ISOPO_VAR_INTERACTING; P.lambda = lambda;
  const size_t nb = (size_t)(B + kNB - 1) / kNB;
  const size_t smem = sizeof(float) * (nb * kBlk + 2 * nb * kNB) + sizeof(double) * nb * kNB;
  ISOPO_CUDA_TRY(cudaFuncSetAttribute(k_transform_large, cudaFuncAttributeMaxDynamicSharedMemorySize, 200 * 1024));
  {
    LaunchScope scope(kIdTransform, st);
    k_transform_large<<<1, kThreads, smem, st>>>(P, scratch);
  }
  ISOPO_CUDA_TRY(cudaGetLastError());
  return ISOPO_OK;
}

isopo_status transform(const float* K, const float* A, int B, isopo_variant v, float lambda, const float* g,
                       const float* rel_state, float* coeffs, int32_t* info, cudaStream_t st) {
  return transform_batched(1, &K, A, B, v, &lambda, g, rel_state ? &rel_state : nullptr, &coeffs, info, st);
}

}  // namespace isopo
