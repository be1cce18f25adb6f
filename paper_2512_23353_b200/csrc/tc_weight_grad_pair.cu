// Stand-alone weight gradient dW = (c_seq(t) dY)^T X (Alg. 1: "grad += advantages * rescaled
// gradient") with 2-CTA tensor-core tiles.
//
// The per-token scale is applied to the NARROWER operand in one streaming pass (k_scale_rows:
// T x min(d_in, d_out) elements read and written once, round to nearest even), after which the
// weight gradient is a plain GEMM over all tokens.  Scaling the landed rows in shared memory inside
// the GEMM (what the 1-CTA kernel of tc_seq_grad.cu does for small layers) was measured 15 % slower
// here: under the power cap the extra shared-memory traffic and the busy scaler warps cost more
// than the extra pass over 1/6 .. 1/35 of the operand bytes.
//
// The GEMM is the pipeline of tc_seq_grad_pair.cu with other work units: (256 x 512 block of dW, slab
// of tokens), slab-major so that the pairs running at one time read the same tokens out of L2.  The
// block is two 256 x 256 accumulators side by side that share the dY operand: all 512 columns of
// tensor memory, so a unit's epilogue is not overlapped, but a unit is a long token slab (there are
// only a few per pair).  Against one 256 x 256 tile per unit this moves 3/4 of the operand bytes
// from L2 to the SMs per flop and streams the inputs from HBM about half as often (every round of
// units re-reads its slab, and there are half as many units per slab); under the power cap both show
// up as clock.
//
//   warp 0          TMA producer; both CTAs' copies complete on the barrier in CTA 0
//   warp 1, CTA 0   MMA issuer (one elected thread), 2 x tcgen05.mma.cta_group::2 256 x 256 x 16 per step
//   warps 2-5       epilogue: TMEM -> float32 red.global.add.v4 into dW (token slabs of a block meet there)
//
// Every wait is bounded; the teardown is that of tc_seq_grad_pair.cu.
#include <algorithm>

#include "tc_common.cuh"

namespace isopo {

namespace {

using namespace tc;

constexpr int kKB = 64;                              // tokens per pipeline stage
constexpr int kStages = 4;
constexpr int kHalf = 128;
constexpr int kChunkBytes = kKB * 128;           // 64 tokens x 64 columns
constexpr int kOperandBytes = 2 * kChunkBytes;   // one CTA's 128 columns of an operand
constexpr int kStageBytes = 3 * kOperandBytes;   // dY half, X half of the left tile, X half of the right tile
constexpr int kSmemBytes = kStages * kStageBytes + 1024 /*alignment slack*/ + 512 /*barriers*/;
constexpr int kThreads = 192;
constexpr uint32_t kTmemCols = 512;
constexpr int kPairN = 256;
constexpr int kUnitOverhead = 16;  // a unit's epilogue and pipeline fill, in 64-token stages (host cost model)
static_assert(kSmemBytes <= 227 * 1024, "shared memory");

struct FoldedPairParams {
  float* dW;
  int64_t T, slab;  // tokens per work unit (a multiple of kKB)
  int nslabs, d_in, d_out;
  int ptiles_m, tiles_n;  // 256-row blocks of d_out; 512-column blocks of d_in
  int32_t* info;
};

__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(kThreads, 1)
k_bf16_weight_grad_pair(const __grid_constant__ CUtensorMap mapY, const __grid_constant__ CUtensorMap mapX,
                        FoldedPairParams p) {
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  const uint32_t smem_base = smem_u32(smem);
  uint64_t* bars = reinterpret_cast<uint64_t*>(smem + kStages * kStageBytes);
  const uint32_t bar0 = smem_u32(bars);
  auto full_bar = [&](int s) { return bar0 + 8u * s; };                          // used in CTA 0
  auto empty_bar = [&](int s) { return bar0 + 8u * (kStages + s); };             // both CTAs
  auto accfull_bar = [&](int b) { return bar0 + 8u * (2 * kStages + b); };       // both CTAs
  auto accempty_bar = [&](int b) { return bar0 + 8u * (2 * kStages + 2 + b); };  // used in CTA 0
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + 2 * kStages + 4);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const uint32_t rank = cluster_ctarank();
  const uint32_t peer_abort = map_to_cta(smem_u32(const_cast<int*>(abort_flag)), rank ^ 1u);
  if (threadIdx.x == 0) {
    for (int s = 0; s < kStages; ++s) {
      mbar_init(full_bar(s), 1);
      mbar_init(empty_bar(s), 1);
    }
    mbar_init(accfull_bar(0), 1);
    mbar_init(accempty_bar(0), 8);
    *abort_flag = 0;
    fence_barrier_init();
  }
  if (warp == 1) tmem_alloc_pair(smem_u32(tmem_slot), kTmemCols);
  tc_fence_before_sync();
  __syncthreads();
  __syncwarp();
  cluster_sync_all();
  tc_fence_after_sync();
  const uint32_t tmem_base = *tmem_slot;

  const int ptiles = p.ptiles_m * p.tiles_n;
  const long long total_units = (long long)p.nslabs * ptiles;
  const long long pair_id = blockIdx.x >> 1, npairs = gridDim.x >> 1;
  // unit u = slab * ptiles + pair tile
  auto unit_tokens = [&](long long u, int64_t& t0, int& nkb) {
    t0 = (u / ptiles) * p.slab;
    nkb = (int)((min(p.T, t0 + p.slab) - t0 + kKB - 1) / kKB);
  };

  if (warp == 0) {
    // ------------------------------------------------------------------ TMA producer (both CTAs)
    if (elect_one()) {
      prefetch_tensormap(&mapY);
      prefetch_tensormap(&mapX);
      const uint32_t full_at_leader = map_to_cta(full_bar(0), 0);
      int stage = 0;
      uint32_t phase = 0;
      bool ok = true;
      for (long long u = pair_id; u < total_units && ok; u += npairs) {
        const int pt = (int)(u % ptiles);
        const int ptm = pt / p.tiles_n, tn = pt % p.tiles_n;
        int64_t t0;
        int nkb;
        unit_tokens(u, t0, nkb);
        const int ycol = (2 * ptm + (int)rank) * kHalf, xcol = tn * 2 * kPairN + (int)rank * kHalf;
        for (int kb = 0; kb < nkb; ++kb) {
          if (!(ok = mbar_wait_pair(empty_bar(stage), phase ^ 1u, abort_flag, peer_abort, p.info, kIdWeightGrad))) break;
          const uint32_t a_dst = smem_base + stage * kStageBytes, b_dst = a_dst + kOperandBytes;
          const int y = (int)(t0 + (int64_t)kb * kKB);  // rows past T and columns past d_in read as zero
          if (rank == 0) mbar_arrive_expect_tx(full_bar(stage), 2 * kStageBytes);
          const uint32_t fb = full_at_leader + 8u * stage;
#pragma unroll
          for (int c = 0; c < 2; ++c) {
            tma_load_2d_pair(a_dst + c * kChunkBytes, &mapY, ycol + c * 64, y, fb);
            tma_load_2d_pair(b_dst + c * kChunkBytes, &mapX, xcol + c * 64, y, fb);
            tma_load_2d_pair(b_dst + kOperandBytes + c * kChunkBytes, &mapX, xcol + kPairN + c * 64, y, fb);
          }
          if (++stage == kStages) { stage = 0; phase ^= 1u; }
        }
      }
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------------ MMA issuer (one thread of CTA 0)
    if (rank == 0 && elect_one()) {
      constexpr uint32_t idesc = make_idesc_bf16(256, kPairN, /*a_mn=*/true, /*b_mn=*/true);
      int stage = 0;
      uint32_t phase = 0, acc_phase = 0;
      bool ok = true;
      for (long long u = pair_id; u < total_units && ok; u += npairs) {
        int64_t t0;
        int nkb;
        unit_tokens(u, t0, nkb);
        if (!(ok = mbar_wait_pair(accempty_bar(0), acc_phase ^ 1u, abort_flag, peer_abort, p.info, kIdWeightGrad))) break;
        tc_fence_after_sync();
        const uint32_t d_tmem = tmem_base;
        for (int kb = 0; kb < nkb; ++kb) {
          if (!(ok = mbar_wait_pair(full_bar(stage), phase, abort_flag, peer_abort, p.info, kIdWeightGrad))) break;
          tc_fence_after_sync();
          const uint32_t a_addr = smem_base + stage * kStageBytes, b_addr = a_addr + kOperandBytes;
#pragma unroll
          for (int k16 = 0; k16 < kKB / 16; ++k16) {
            const uint64_t a_desc = make_sdesc_sw128(a_addr + k16 * 2048, kChunkBytes, 1024);
            const uint64_t b_desc = make_sdesc_sw128(b_addr + k16 * 2048, kChunkBytes, 1024);
            const uint64_t b2_desc = make_sdesc_sw128(b_addr + kOperandBytes + k16 * 2048, kChunkBytes, 1024);
            mma_bf16_pair(d_tmem, a_desc, b_desc, idesc, (kb | k16) != 0);
            mma_bf16_pair(d_tmem + kPairN, a_desc, b2_desc, idesc, (kb | k16) != 0);
          }
          mma_commit_pair(empty_bar(stage));
          if (++stage == kStages) { stage = 0; phase ^= 1u; }
        }
        if (!ok) break;
        mma_commit_pair(accfull_bar(0));
        acc_phase ^= 1u;
      }
    }
  } else if (warp < 6) {
    // ------------------------------------------------------------------ epilogue (warps 2..5, both CTAs)
    const int q = warp & 3;
    const int row = q * 32 + lane;
    const uint32_t accempty_at_leader = map_to_cta(accempty_bar(0), 0);
    uint32_t acc_phase = 0;
    for (long long u = pair_id; u < total_units; u += npairs) {
      const int pt = (int)(u % ptiles);
      const int m = (2 * (pt / p.tiles_n) + (int)rank) * kHalf + row, n0 = (pt % p.tiles_n) * 2 * kPairN;
      if (!mbar_wait_pair(accfull_bar(0), acc_phase, abort_flag, peer_abort, p.info, kIdWeightGrad)) break;
      tc_fence_after_sync();
      const uint32_t taddr = tmem_base + ((uint32_t)(q * 32) << 16);
      float* dst = p.dW + (size_t)m * p.d_in + n0;
#pragma unroll 2
      for (int jc = 0; jc < 2 * kPairN / 32; ++jc) {
        uint32_t r[32];
        tmem_ld32(taddr + jc * 32, r);
        tmem_ld_wait();
        if (m < p.d_out) {
#pragma unroll
          for (int v = 0; v < 8; ++v) {
            const int n = n0 + jc * 32 + v * 4;
            if (n < p.d_in &&  // d_in is a multiple of 8, so a group of 4 is all in or all out
                ISOPO_IN_RANGE((long long)m * p.d_in + n + 3, (long long)p.d_out * p.d_in, p.info, kIdWeightGrad))
              asm volatile("red.global.add.v4.f32 [%0], {%1, %2, %3, %4};" ::"l"(dst + jc * 32 + v * 4),
                           "f"(__uint_as_float(r[v * 4 + 0])), "f"(__uint_as_float(r[v * 4 + 1])),
                           "f"(__uint_as_float(r[v * 4 + 2])), "f"(__uint_as_float(r[v * 4 + 3]))
                           : "memory");
          }
        }
      }
      tc_fence_before_sync();
      __syncwarp();
      if (lane == 0) mbar_arrive_remote(accempty_at_leader);
      acc_phase ^= 1u;
    }
  }

  // ---------------------------------------------------------------------- teardown
  if (*abort_flag) __nanosleep(100000);
  tc_fence_before_sync();
  __syncthreads();
  __syncwarp();
  cluster_sync_all();
  if (warp == 1) tmem_dealloc_pair(tmem_base, kTmemCols);
}

// dst[t, :] = bf16(tokscale[t] * src[t, :]) (round to nearest even), 8 elements per thread.
__global__ void __launch_bounds__(256) k_scale_rows(const uint4* __restrict__ src, const float* __restrict__ tokscale,
                                                    int64_t T, int d8 /* columns / 8 */, uint4* __restrict__ dst) {
  const int64_t n = T * d8;
  for (int64_t e = blockIdx.x * (int64_t)blockDim.x + threadIdx.x; e < n; e += (int64_t)gridDim.x * blockDim.x) {
    const float c = __ldg(tokscale + e / d8);
    uint4 v = __ldcs(src + e);
    uint32_t* w = reinterpret_cast<uint32_t*>(&v);
#pragma unroll
    for (int k = 0; k < 4; ++k)
      w[k] = pack_bf16x2(c * __uint_as_float(w[k] << 16), c * __uint_as_float(w[k] & 0xffff0000u));
    dst[e] = v;
  }
}

}  // namespace

isopo_status bf16_weight_grad_pair(const void* X, const void* dY, int64_t T, int d_in, int d_out, const float* tokscale,
                                   void* scaled, float* dW, float beta, int32_t* info, cudaStream_t st) {
  int dev = 0, sms = 0;
  ISOPO_CUDA_TRY(cudaGetDevice(&dev));
  ISOPO_CUDA_TRY(cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev));
  {  // scale the narrower operand into `scaled`
    const bool scale_y = d_out <= d_in;
    const int d8 = (scale_y ? d_out : d_in) / 8;
    const int grid = (int)std::min<int64_t>((T * d8 + 255) / 256, (int64_t)sms * 16);
    {
      LaunchScope scope(kIdScaleRows, st);
      k_scale_rows<<<grid, 256, 0, st>>>((const uint4*)(scale_y ? dY : X), tokscale, T, d8, (uint4*)scaled);
    }
    ISOPO_CUDA_TRY(cudaGetLastError());
    if (scale_y) dY = scaled; else X = scaled;
  }
  CUtensorMap mapY, mapX;
  isopo_status s = make_map_2d_bf16(&mapY, dY, (uint64_t)T, (uint64_t)d_out, (uint64_t)d_out, 64, kKB);
  if (s != ISOPO_OK) return s;
  s = make_map_2d_bf16(&mapX, X, (uint64_t)T, (uint64_t)d_in, (uint64_t)d_in, 64, kKB);
  if (s != ISOPO_OK) return s;
  ISOPO_CUDA_TRY(cudaFuncSetAttribute(k_bf16_weight_grad_pair, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBytes));
  if (beta == 0.f) ISOPO_CUDA_TRY(cudaMemsetAsync(dW, 0, sizeof(float) * (size_t)d_in * d_out, st));
  static int resident_pairs[64] = {};
  if (dev < 0 || dev >= 64) return ISOPO_ERR_UNSUPPORTED;
  if (resident_pairs[dev] == 0) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(2 * (unsigned)(sms / 2));
    cfg.blockDim = dim3(kThreads);
    cfg.dynamicSmemBytes = kSmemBytes;
    cudaLaunchAttribute attr;
    attr.id = cudaLaunchAttributeClusterDimension;
    attr.val.clusterDim.x = 2; attr.val.clusterDim.y = 1; attr.val.clusterDim.z = 1;
    cfg.attrs = &attr;
    cfg.numAttrs = 1;
    int n = 0;
    ISOPO_CUDA_TRY(cudaOccupancyMaxActiveClusters(&n, k_bf16_weight_grad_pair, &cfg));
    if (n < 1) return ISOPO_ERR_UNSUPPORTED;
    resident_pairs[dev] = std::min(n, sms / 2);
  }
  FoldedPairParams p{};
  p.dW = dW; p.T = T; p.d_in = d_in; p.d_out = d_out; p.info = info;
  p.ptiles_m = ((d_out + kHalf - 1) / kHalf + 1) / 2;
  p.tiles_n = (d_in + 2 * kPairN - 1) / (2 * kPairN);
  // token slabs: the count (up to 64) whose rounds of units take least, a round costing its slab plus the
  // unit's exposed epilogue and pipeline fill (about kUnitOverhead stages' worth); ties go to fewer slabs.  Every slab is a multiple of the stage depth.
  // (Slabs small enough for their rows to stay in L2 across the rounds were measured slower: the
  // float32 reductions into dW grow with the slab count.)
  const long long ptiles = (long long)p.ptiles_m * p.tiles_n, pairs = resident_pairs[dev];
  const long long kblocks = (T + kKB - 1) / kKB;
  long long nslabs = 1, best = -1;
  for (long long n = 1; n <= std::min<long long>(64, kblocks); ++n) {
    const long long per = (kblocks + n - 1) / n, rounds = (ptiles * n + pairs - 1) / pairs;
    const long long cost = rounds * (per + kUnitOverhead);
    if (best < 0 || cost < best) { best = cost; nslabs = n; }
  }
  const long long kb_per = (kblocks + nslabs - 1) / nslabs;
  nslabs = (kblocks + kb_per - 1) / kb_per;
  p.slab = kb_per * kKB;
  p.nslabs = (int)nslabs;
  const int npairs = (int)std::max<long long>(1, std::min<long long>(ptiles * nslabs, pairs));
  {
    LaunchScope scope(kIdWeightGrad, st);
    k_bf16_weight_grad_pair<<<2 * npairs, kThreads, kSmemBytes, st>>>(mapY, mapX, p);
  }
  ISOPO_CUDA_TRY(cudaGetLastError());
  return ISOPO_OK;
}

}  // namespace isopo
