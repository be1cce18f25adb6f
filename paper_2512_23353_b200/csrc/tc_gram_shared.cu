// Gram route for several projections that read the same input X (q/k/v, gate/up):
//   K^(h)_ij = sum_{t in i, s in j} (dY^(h)_t . dY^(h)_s)(x_t . x_s)             (Eq. one / Eq. two per layer)
// The factor P = X_I X_J^T of a pair of token tiles does not depend on the projection, so one unit forms
// it once and then Q^(h) = dY^(h)_I dY^(h)_J^T for one projection after the other.  Tensor memory holds
// two P and two Q accumulators (4 x 128 columns): while the epilogue multiplies Q^(h) with P and adds
// into projection h's K, the tensor core already fills the other Q (or, after the last projection,
// the other P for the next unit), so no epilogue is exposed.  Against one k_bf16_gram launch per
// projection this saves the X contraction of every projection but the first, and the loads of X that
// feed it.  Pipeline, tile order and epilogue are those of tc_gram.cu.
#include <algorithm>

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
constexpr uint32_t kTmemCols = 512;            // P0 | P1 | Q0 | Q1
constexpr int kMaxHeads = 3;

struct SharedGramParams {
  const int32_t* tokseq;
  float* K[kMaxHeads];
  int64_t T;
  int B, nT, d_in, n_heads;
  int d_out[kMaxHeads];
  int32_t* info;
  int strip;
};

__global__ void __launch_bounds__(kThreads, 1)
k_bf16_gram_shared(const __grid_constant__ CUtensorMap mapX, const __grid_constant__ CUtensorMap mapY0,
                   const __grid_constant__ CUtensorMap mapY1, const __grid_constant__ CUtensorMap mapY2,
                   SharedGramParams p) {
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  const uint32_t smem_base = smem_u32(smem);
  uint64_t* bars = reinterpret_cast<uint64_t*>(smem + kStages * kStageBytes);
  const uint32_t bar0 = smem_u32(bars);
  auto full_bar = [&](int s) { return bar0 + 8u * s; };
  auto empty_bar = [&](int s) { return bar0 + 8u * (kStages + s); };
  auto qfull_bar = [&](int b) { return bar0 + 8u * (2 * kStages + b); };
  auto qempty_bar = [&](int b) { return bar0 + 8u * (2 * kStages + 2 + b); };
  auto pempty_bar = [&](int b) { return bar0 + 8u * (2 * kStages + 4 + b); };
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + 2 * kStages + 6);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  if (threadIdx.x == 0) {
    for (int s = 0; s < kStages; ++s) { mbar_init(full_bar(s), 1); mbar_init(empty_bar(s), 1); }
    for (int b = 0; b < 2; ++b) { mbar_init(qfull_bar(b), 1); mbar_init(qempty_bar(b), 4); mbar_init(pempty_bar(b), 4); }
    *abort_flag = 0;
    fence_barrier_init();
  }
  if (warp == 1) tmem_alloc(smem_u32(tmem_slot), kTmemCols);
  tc_fence_before_sync();
  __syncthreads();
  tc_fence_after_sync();
  const uint32_t tmem_base = *tmem_slot;

  const long long total_units = (long long)p.nT * (p.nT + 1) / 2;
  // stage index inside a unit -> (segment, feature block): segment 0 is X, segment 1 + h is dY^(h)
  int nk[kMaxHeads + 1];
  nk[0] = (p.d_in + kKF - 1) / kKF;
  int nk_total = nk[0];
#pragma unroll
  for (int h = 0; h < kMaxHeads; ++h) {
    nk[1 + h] = h < p.n_heads ? (p.d_out[h] + kKF - 1) / kKF : 0;
    nk_total += nk[1 + h];
  }
  auto locate = [&](int kb, int& seg, int& kk) {
    seg = 0;
    kk = kb;
#pragma unroll
    for (int s = 0; s < kMaxHeads; ++s)
      if (seg == s && kk >= nk[s]) { kk -= nk[s]; seg = s + 1; }
  };

  if (warp == 0) {
    if (elect_one()) {
      prefetch_tensormap(&mapX);
      prefetch_tensormap(&mapY0);
      if (p.n_heads > 1) prefetch_tensormap(&mapY1);
      if (p.n_heads > 2) prefetch_tensormap(&mapY2);
      int stage = 0;
      uint32_t phase = 0;
      bool ok = true;
      for (long long u = blockIdx.x; u < total_units && ok; u += gridDim.x) {
        int I, J;
        decode_pair_strips(u, p.nT, p.strip, I, J);
        const bool diag = I == J;
        for (int kb = 0; kb < nk_total; ++kb) {
          int seg, kk;
          locate(kb, seg, kk);
          if (!(ok = mbar_wait(empty_bar(stage), phase ^ 1u, abort_flag, p.info, kIdGram))) break;
          const CUtensorMap* map = seg == 0 ? &mapX : seg == 1 ? &mapY0 : seg == 2 ? &mapY1 : &mapY2;
          const uint32_t dst = smem_base + stage * kStageBytes;
          mbar_arrive_expect_tx(full_bar(stage), diag ? kOperandBytes : kStageBytes);
          tma_load_2d(dst, map, kk * kKF, I * kTT, full_bar(stage));
          if (!diag) tma_load_2d(dst + kOperandBytes, map, kk * kKF, J * kTT, full_bar(stage));
          if (++stage == kStages) { stage = 0; phase ^= 1u; }
        }
      }
    }
  } else if (warp == 1) {
    if (elect_one()) {
      constexpr uint32_t idesc = make_idesc_bf16(kTT, kTT, false, false);
      int stage = 0;
      uint32_t phase = 0;
      unsigned ucount = 0, qcount = 0;  // units and Q accumulators started: buffer = count & 1, parity = count >> 1 & 1
      bool ok = true;
      for (long long u = blockIdx.x; u < total_units && ok; u += gridDim.x, ++ucount) {
        int I, J;
        decode_pair_strips(u, p.nT, p.strip, I, J);
        const bool diag = I == J;
        const unsigned pb = ucount & 1u;
        // P[pb] is free once every projection of the unit before last has been through the epilogue
        if (!(ok = mbar_wait(pempty_bar(pb), ((ucount >> 1) & 1u) ^ 1u, abort_flag, p.info, kIdGram))) break;
        tc_fence_after_sync();
        int seg_now = 0;
        unsigned qb = 0;
        for (int kb = 0; kb < nk_total; ++kb) {
          int seg, kk;
          locate(kb, seg, kk);
          if (seg != seg_now) {  // a projection begins: close the previous one, claim a Q accumulator
            if (seg_now > 0) { mma_commit(qfull_bar(qb)); ++qcount; }
            seg_now = seg;
            qb = qcount & 1u;
            if (!(ok = mbar_wait(qempty_bar(qb), ((qcount >> 1) & 1u) ^ 1u, abort_flag, p.info, kIdGram))) break;
            tc_fence_after_sync();
          }
          if (!(ok = mbar_wait(full_bar(stage), phase, abort_flag, p.info, kIdGram))) break;
          tc_fence_after_sync();
          const uint32_t a_addr = smem_base + stage * kStageBytes;
          const uint32_t b_addr = diag ? a_addr : a_addr + kOperandBytes;
          const uint32_t d_tmem = tmem_base + (seg == 0 ? pb * 128u : 256u + qb * 128u);
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
        mma_commit(qfull_bar(qb));  // the last projection of the unit
        ++qcount;
      }
    }
  } else {
    const int q = warp & 3, row = q * 32 + lane;
    unsigned ucount = 0, qcount = 0;
    bool ok = true;
    for (long long u = blockIdx.x; u < total_units && ok; u += gridDim.x, ++ucount) {
      int I, J;
      decode_pair_strips(u, p.nT, p.strip, I, J);
      const bool diag = I == J;
      const unsigned pb = ucount & 1u;
      const int64_t trow = (int64_t)I * kTT + row;
      const int row_seq = __ldg(p.tokseq + min(trow, p.T - 1));
      auto col_seq = [&](int g) { return __ldg(p.tokseq + min((int64_t)J * kTT + g * 32 + lane, p.T - 1)); };
      const RowSegments rows = row_segments(row_seq, (long long)p.B * p.B, p.info);
      const uint32_t taddr = tmem_base + ((uint32_t)(q * 32) << 16);
#pragma unroll 1
      for (int h = 0; h < p.n_heads; ++h, ++qcount) {
        const unsigned qb = qcount & 1u;
        int cs = col_seq(0);
        if (!(ok = mbar_wait(qfull_bar(qb), (qcount >> 1) & 1u, abort_flag, p.info, kIdGram))) break;
        tc_fence_after_sync();
        float* Kh = p.K[h];
        int cur = __shfl_sync(0xffffffffu, cs, 0);
        float wseg = row_seq == cur ? 2.f : 1.f, run = 0.f;
#pragma unroll 1
        for (int g = 0; g < kTT / 32; ++g) {
          const int cs_next = g + 1 < kTT / 32 ? col_seq(g + 1) : 0;
          uint32_t pv[32], qv[32];
          tmem_ld32(taddr + pb * 128u + g * 32, pv);
          tmem_ld32(taddr + 256u + qb * 128u + g * 32, qv);
          tmem_ld_wait();
          gram_group<true>(pv, qv, cs, g * 32, row, diag, rows, Kh, p.B, cur, wseg, run);
          cs = cs_next;
        }
        flush_rows(Kh, p.B, rows, cur, run);
        tc_fence_before_sync();
        __syncwarp();
        if (lane == 0) {
          mbar_arrive(qempty_bar(qb));
          if (h == p.n_heads - 1) mbar_arrive(pempty_bar(pb));
        }
      }
    }
  }

  if (*abort_flag) __nanosleep(100000);
  tc_fence_before_sync();
  __syncthreads();
  if (warp == 1) tmem_dealloc(tmem_base, kTmemCols);
}


}  // namespace

isopo_status bf16_gram_shared(const void* X, const void* const* dY, int64_t T, int d_in, const int* d_out, int n_heads,
                              const int32_t* tokseq, int B, float* const* K, int32_t* info, cudaStream_t st) {
  if (n_heads < 1 || n_heads > kMaxHeads) return ISOPO_ERR_INVALID_ARG;
  CUtensorMap mapX, mapY[kMaxHeads];
  isopo_status s = make_map_2d_bf16(&mapX, X, (uint64_t)T, (uint64_t)d_in, (uint64_t)d_in, 64, kTT);
  if (s != ISOPO_OK) return s;
  for (int h = 0; h < kMaxHeads; ++h) {
    const int hh = std::min(h, n_heads - 1);  // unused slots repeat the last projection's map
    s = make_map_2d_bf16(&mapY[h], dY[hh], (uint64_t)T, (uint64_t)d_out[hh], (uint64_t)d_out[hh], 64, kTT);
    if (s != ISOPO_OK) return s;
  }
  int dev = 0, sms = 0;
  ISOPO_CUDA_TRY(cudaGetDevice(&dev));
  ISOPO_CUDA_TRY(cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev));
  ISOPO_CUDA_TRY(cudaFuncSetAttribute(k_bf16_gram_shared, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBytes));
  SharedGramParams p{};
  p.tokseq = tokseq; p.T = T; p.B = B; p.nT = (int)((T + kTT - 1) / kTT); p.d_in = d_in; p.n_heads = n_heads; p.info = info;
  int d_sum = d_in;
  for (int h = 0; h < n_heads; ++h) {
    p.K[h] = K[h];
    p.d_out[h] = d_out[h];
    d_sum += d_out[h];
    ISOPO_CUDA_TRY(cudaMemsetAsync(K[h], 0, sizeof(float) * (size_t)B * B, st));
  }
  const long long units = (long long)p.nT * (p.nT + 1) / 2;
  const int grid = (int)std::min<long long>(units, sms);
  p.strip = gram_strip_width(2.0 * kTT * d_sum, grid);
  {
    LaunchScope scope(kIdGram, st);
    k_bf16_gram_shared<<<grid, kThreads, kSmemBytes, st>>>(mapX, mapY[0], mapY[1], mapY[2], p);
  }
  ISOPO_CUDA_TRY(cudaGetLastError());
  for (int h = 0; h < n_heads; ++h) {
    const isopo_status s = mirror_upper(K[h], B, st);
    if (s != ISOPO_OK) return s;
  }
  return ISOPO_OK;
}

}  // namespace isopo
