// Gram route to the layer NTK on the tensor cores.
//
// Every token gradient is the rank-one matrix dY_t x_t^T (Eq. one / Eq. two), hence
//   K_ij = sum_{t in i, s in j} (dY_t . dY_s)(x_t . x_s) = [ S ((dY dY^T) o (X X^T)) S^T ]_ij
// with S the B x T sequence indicator.  For a pair of 128-token tiles (I <= J) this kernel forms
// P = X_I X_J^T (contraction over d_in) and Q = dY_I dY_J^T (contraction over d_out) as two
// 128 x 128 float32 accumulators in tensor memory, and its epilogue multiplies them elementwise and
// adds the products into K by (sequence of row token, sequence of column token).  Neither T x T
// matrix ever leaves the SM.
//
// Only token pairs t <= s are visited.  A pair t < s inside one sequence stands for (t,s) and
// (s,t) and counts twice; a pair across sequences i < j lands in K_ij once (K_ji is mirrored at the
// end); t = s counts once.
//
//   warp 0      TMA producer: [128 tokens] x [64 features] boxes of X then of dY, 6-stage ring
//   warp 1      MMA issuer: tcgen05.mma 128 x 128 x 16, K-major operands
//   warps 2-5   epilogue: tcgen05.ld of P and Q, product, segmented sums, float atomics into K

#include "tc_common.cuh"
#include "tc_gram_epilogue.cuh"

namespace isopo {

namespace {

using namespace tc;

constexpr int kTT = 128;                       // tokens per tile
constexpr int kKF = 64;                        // features per stage (128 bytes of bf16)
constexpr int kStages = 6;
constexpr int kOperandBytes = kTT * 128;       // 16 KB
constexpr int kStageBytes = 2 * kOperandBytes;
constexpr int kSmemBytes = kStages * kStageBytes + 1024 + 256;
constexpr int kThreads = 192;
constexpr uint32_t kTmemCols = 512;            // 2 buffers x (P 128 + Q 128) columns

struct GramParams {
  const int32_t* tokseq;
  float* K;       // Gram: K [B, B];  sampled: M^T [samples, B]
  int64_t T;
  int B, nT, d_in, d_out;
  int32_t* info;
  int n_rows, n_row_tiles;  // sampled: sample rows and their 128-row tiles
  int strip;                // Gram: tile columns per strip of the pair order
};

// Work unit -> (row tile I, column tile J).  Gram: pairs I <= J of token tiles in strip order.
// Sampled: every (sample tile, token tile).
template <bool kSampled>
__device__ __forceinline__ void decode_unit(const GramParams& p, long long u, int& I, int& J, bool& diag) {
  if (kSampled) {
    I = (int)(u % p.n_row_tiles);
    J = (int)(u / p.n_row_tiles);
    diag = false;
  } else {
    decode_pair_strips(u, p.nT, p.strip, I, J);
    diag = I == J;
  }
}

// kSampled = false: the Gram route, rows and columns are both token tiles (mapRX = mapX, mapRY = mapY).
// kSampled = true: the token-sampled Fisher estimator of Algorithm 1: the rows are the sampled token
// rows a0 = X[samples] (mapRX) and g0 = dY[samples] (mapRY), the columns all tokens, and
//   M^T[j, i] = sum_{t in sequence i} (g0_j . dY_t)(a0_j . x_t) = g0_j . G_i a0_j      (Eq. one)
// comes out of the same product-and-segment-sum epilogue without any symmetry weights.
template <bool kSampled>
__global__ void __launch_bounds__(kThreads, 1)
k_bf16_gram(const __grid_constant__ CUtensorMap mapRX, const __grid_constant__ CUtensorMap mapRY,
            const __grid_constant__ CUtensorMap mapX, const __grid_constant__ CUtensorMap mapY, GramParams p) {
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  const uint32_t smem_base = smem_u32(smem);
  uint64_t* bars = reinterpret_cast<uint64_t*>(smem + kStages * kStageBytes);
  const uint32_t bar0 = smem_u32(bars);
  auto full_bar = [&](int s) { return bar0 + 8u * s; };
  auto empty_bar = [&](int s) { return bar0 + 8u * (kStages + s); };
  auto accfull_bar = [&](int b) { return bar0 + 8u * (2 * kStages + b); };
  auto accempty_bar = [&](int b) { return bar0 + 8u * (2 * kStages + 2 + b); };
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + 2 * kStages + 4);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  if (threadIdx.x == 0) {
    for (int s = 0; s < kStages; ++s) { mbar_init(full_bar(s), 1); mbar_init(empty_bar(s), 1); }
    for (int b = 0; b < 2; ++b) { mbar_init(accfull_bar(b), 1); mbar_init(accempty_bar(b), 4); }
    *abort_flag = 0;
    fence_barrier_init();
  }
  if (warp == 1) tmem_alloc(smem_u32(tmem_slot), kTmemCols);
  tc_fence_before_sync();
  __syncthreads();
  tc_fence_after_sync();
  const uint32_t tmem_base = *tmem_slot;

  const long long total_units = kSampled ? (long long)p.n_row_tiles * p.nT : (long long)p.nT * (p.nT + 1) / 2;
  const int nkx = (p.d_in + kKF - 1) / kKF, nky = (p.d_out + kKF - 1) / kKF;

  if (warp == 0) {
    if (elect_one()) {
      prefetch_tensormap(&mapX);
      prefetch_tensormap(&mapY);
      if (kSampled) {
        prefetch_tensormap(&mapRX);
        prefetch_tensormap(&mapRY);
      }
      int stage = 0;
      uint32_t phase = 0;
      bool ok = true;
      for (long long u = blockIdx.x; u < total_units && ok; u += gridDim.x) {
        int I, J;
        bool diag;
        decode_unit<kSampled>(p, u, I, J, diag);
        for (int kb = 0; kb < nkx + nky; ++kb) {
          if (!(ok = mbar_wait(empty_bar(stage), phase ^ 1u, abort_flag, p.info, kIdGram))) break;
          const CUtensorMap* rmap = kb < nkx ? &mapRX : &mapRY;
          const CUtensorMap* cmap = kb < nkx ? &mapX : &mapY;
          const int x = (kb < nkx ? kb : kb - nkx) * kKF;
          const uint32_t dst = smem_base + stage * kStageBytes;
          mbar_arrive_expect_tx(full_bar(stage), diag ? kOperandBytes : kStageBytes);
          tma_load_2d(dst, rmap, x, I * kTT, full_bar(stage));
          if (!diag) tma_load_2d(dst + kOperandBytes, cmap, x, J * kTT, full_bar(stage));
          if (++stage == kStages) { stage = 0; phase ^= 1u; }
        }
      }
    }
  } else if (warp == 1) {
    if (elect_one()) {  // elected, not "lane 0": lets the compiler keep the MMA operands in uniform registers
      constexpr uint32_t idesc = make_idesc_bf16(kTT, kTT, false, false);
      int stage = 0, acc = 0;
      uint32_t phase = 0, acc_phase = 0;
      bool ok = true;
      for (long long u = blockIdx.x; u < total_units && ok; u += gridDim.x) {
        int I, J;
        bool diag;
        decode_unit<kSampled>(p, u, I, J, diag);
        if (!(ok = mbar_wait(accempty_bar(acc), acc_phase ^ 1u, abort_flag, p.info, kIdGram))) break;
        tc_fence_after_sync();
        for (int kb = 0; kb < nkx + nky; ++kb) {
          if (!(ok = mbar_wait(full_bar(stage), phase, abort_flag, p.info, kIdGram))) break;
          tc_fence_after_sync();
          const uint32_t a_addr = smem_base + stage * kStageBytes;
          const uint32_t b_addr = diag ? a_addr : a_addr + kOperandBytes;
          const bool second = kb >= nkx;  // accumulating Q
          const uint32_t d_tmem = tmem_base + (uint32_t)acc * 256 + (second ? 128u : 0u);
          const int kk = second ? kb - nkx : kb;
#pragma unroll
          for (int k16 = 0; k16 < kKF / 16; ++k16) {
            const uint64_t a_desc = make_sdesc_sw128(a_addr + k16 * 32, 16, 1024);
            const uint64_t b_desc = make_sdesc_sw128(b_addr + k16 * 32, 16, 1024);
            mma_bf16(d_tmem, a_desc, b_desc, idesc, (kk | k16) != 0);
          }
          mma_commit(empty_bar(stage));
          if (++stage == kStages) { stage = 0; phase ^= 1u; }
        }
        if (!ok) break;
        mma_commit(accfull_bar(acc));
        if (++acc == 2) { acc = 0; acc_phase ^= 1u; }
      }
    }
  } else {
    const int q = warp & 3, row = q * 32 + lane;
    int acc = 0;
    uint32_t acc_phase = 0;
    for (long long u = blockIdx.x; u < total_units; u += gridDim.x) {
      int I, J;
      bool diag;
      decode_unit<kSampled>(p, u, I, J, diag);
      // sequence of this thread's row token and of every column token (clamped past the end; those
      // rows and columns are zero in P and Q)
      // (sampled: the "row sequence" is the sample index, its results go to row `row_seq` of M^T;
      // rows past the last sample are zero in P and Q, and they are barred from writing outright: a
      // non-finite input would turn their zeros into NaN, and row `trow` of M^T does not exist)
      const int64_t trow = (int64_t)I * kTT + row;
      const int row_seq = kSampled ? (int)trow : __ldg(p.tokseq + min(trow, p.T - 1));
      auto col_seq = [&](int g) { return __ldg(p.tokseq + min((int64_t)J * kTT + g * 32 + lane, p.T - 1)); };
      int cs = col_seq(0);  // sequence of column token 32 g + lane
      if (!mbar_wait(accfull_bar(acc), acc_phase, abort_flag, p.info, kIdGram)) break;
      tc_fence_after_sync();
      const uint32_t taddr = tmem_base + ((uint32_t)(q * 32) << 16) + (uint32_t)acc * 256;
      const RowSegments rows = row_segments(row_seq, (long long)(kSampled ? p.n_rows : p.B) * p.B, p.info, !kSampled || trow < (int64_t)p.n_rows);
      int cur = __shfl_sync(0xffffffffu, cs, 0);
      float wseg = (!kSampled && row_seq == cur) ? 2.f : 1.f, run = 0.f;
#pragma unroll 1
      for (int g = 0; g < kTT / 32; ++g) {
        const int cs_next = g + 1 < kTT / 32 ? col_seq(g + 1) : 0;
        uint32_t pv[32], qv[32];
        tmem_ld32(taddr + g * 32, pv);
        tmem_ld32(taddr + 128 + g * 32, qv);
        tmem_ld_wait();
        gram_group<!kSampled>(pv, qv, cs, g * 32, row, diag, rows, p.K, p.B, cur, wseg, run);
        cs = cs_next;
      }
      flush_rows(p.K, p.B, rows, cur, run);
      tc_fence_before_sync();
      __syncwarp();
      if (lane == 0) mbar_arrive(accempty_bar(acc));
      if (++acc == 2) { acc = 0; acc_phase ^= 1u; }
    }
  }

  if (*abort_flag) __nanosleep(100000);
  tc_fence_before_sync();
  __syncthreads();
  if (warp == 1) tmem_dealloc(tmem_base, kTmemCols);
}


}  // namespace

isopo_status bf16_gram(const void* X, const void* dY, int64_t T, int d_in, int d_out, const int32_t* tokseq, int B,
                       float* K, int32_t* info, cudaStream_t st) {
  CUtensorMap mapX, mapY;
  isopo_status s = make_map_2d_bf16(&mapX, X, (uint64_t)T, (uint64_t)d_in, (uint64_t)d_in, 64, kTT);
  if (s != ISOPO_OK) return s;
  s = make_map_2d_bf16(&mapY, dY, (uint64_t)T, (uint64_t)d_out, (uint64_t)d_out, 64, kTT);
  if (s != ISOPO_OK) return s;
  int dev = 0, sms = 0;
  ISOPO_CUDA_TRY(cudaGetDevice(&dev));
  ISOPO_CUDA_TRY(cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev));
  ISOPO_CUDA_TRY(cudaFuncSetAttribute(k_bf16_gram<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBytes));
  ISOPO_CUDA_TRY(cudaMemsetAsync(K, 0, sizeof(float) * (size_t)B * B, st));
  GramParams p{tokseq, K, T, B, (int)((T + kTT - 1) / kTT), d_in, d_out, info, 0, 0, 0};
  const long long units = (long long)p.nT * (p.nT + 1) / 2;
  const int grid = (int)std::min<long long>(units, sms);
  p.strip = gram_strip_width(2.0 * kTT * (d_in + d_out), grid);
  {
    LaunchScope scope(kIdGram, st);
    k_bf16_gram<false><<<grid, kThreads, kSmemBytes, st>>>(mapX, mapY, mapX, mapY, p);
  }
  ISOPO_CUDA_TRY(cudaGetLastError());
  return mirror_upper(K, B, st);
}

isopo_status bf16_sampled(const void* X, const void* dY, int64_t T, int d_in, int d_out, const int32_t* tokseq, int B,
                          const void* A0, const void* G0, int n_samples, float* Mt, int32_t* info, cudaStream_t st) {
  CUtensorMap mapX, mapY, mapRX, mapRY;
  isopo_status s = make_map_2d_bf16(&mapX, X, (uint64_t)T, (uint64_t)d_in, (uint64_t)d_in, 64, kTT);
  if (s != ISOPO_OK) return s;
  if ((s = make_map_2d_bf16(&mapY, dY, (uint64_t)T, (uint64_t)d_out, (uint64_t)d_out, 64, kTT)) != ISOPO_OK) return s;
  // only the n_samples real rows are in bounds: the rest of the last 128-row tile reads as zero
  if ((s = make_map_2d_bf16(&mapRX, A0, (uint64_t)n_samples, (uint64_t)d_in, (uint64_t)d_in, 64, kTT)) != ISOPO_OK) return s;
  if ((s = make_map_2d_bf16(&mapRY, G0, (uint64_t)n_samples, (uint64_t)d_out, (uint64_t)d_out, 64, kTT)) != ISOPO_OK) return s;
  int dev = 0, sms = 0;
  ISOPO_CUDA_TRY(cudaGetDevice(&dev));
  ISOPO_CUDA_TRY(cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev));
  ISOPO_CUDA_TRY(cudaFuncSetAttribute(k_bf16_gram<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBytes));
  ISOPO_CUDA_TRY(cudaMemsetAsync(Mt, 0, sizeof(float) * (size_t)n_samples * B, st));
  GramParams p{tokseq, Mt, T, B, (int)((T + kTT - 1) / kTT), d_in, d_out, info, n_samples, (n_samples + kTT - 1) / kTT, 0};
  const long long units = (long long)p.n_row_tiles * p.nT;
  const int grid = (int)std::min<long long>(units, sms);
  {
    LaunchScope scope(kIdSampled, st);
    k_bf16_gram<true><<<grid, kThreads, kSmemBytes, st>>>(mapRX, mapRY, mapX, mapY, p);
  }
  ISOPO_CUDA_TRY(cudaGetLastError());
  return ISOPO_OK;
}

}  // namespace isopo
