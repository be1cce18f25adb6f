// Per-sequence weight gradients G_i = dY_i^T X_i on the 5th-generation tensor cores (Alg. 1/2
// reduce loop: `seq_logprob_grad = grad_out.T @ act_in`).
//
// A ragged batched GEMM whose contraction index is the token: both operands are read exactly as
// they sit in memory (token-major rows), i.e. as "MN-major" tcgen05 operands, so no transpose is
// ever materialised.  One persistent CTA per SM walks the work units (sequence i, 128 x 256 tile of
// G) in sequence-major order, so that the CTAs running at the same time share one sequence's
// tokens in L2.
//
//   warp 0      TMA producer: 64-token slabs of dY[:, 128 cols] and X[:, 256 cols] into a 4-stage ring
//   warp 1      MMA issuer: 4 x tcgen05.mma (128 x 256 x 16) per slab into one of two TMEM accumulators;
//               zeroes the token rows past the end of the sequence in the last slab
//   warps 2-5   epilogue: TMEM -> registers -> bf16 (round to nearest even) -> workspace
//
// Stored layout of one tile (64 KB, private to the library): element (m, n) of the tile sits at
// ((n / 8) * 128 + m) * 8 + n % 8, so that a warp's 32 rows write 512 contiguous bytes.
#include "tc_common.cuh"

namespace isopo {

namespace {

using namespace tc;

constexpr int kKB = 64;                                // tokens per pipeline stage
constexpr int kStages = 4;
constexpr int kABytes = kTileM * kKB * 2;              // 16 KB: 2 chunks of [64 tokens][64 cols]
constexpr int kBBytes = kTileN * kKB * 2;              // 32 KB: 4 chunks
constexpr int kStageBytes = kABytes + kBBytes;
constexpr int kChunkBytes = kKB * 128;                 // one [64 tokens][64 cols] box
constexpr int kSmemBytes = kStages * kStageBytes + 1024 /*alignment slack*/ + 256 /*barriers*/;
constexpr int kThreads = 192;
constexpr uint32_t kTmemCols = 512;                    // two 256-column float32 accumulators

struct SeqGradParams {
  const int64_t* off;
  __nv_bfloat16* G;
  int64_t n_pad;
  int B, tiles_m, tiles_n;
  int32_t* info;
};

__global__ void __launch_bounds__(kThreads, 1)
k_bf16_seq_grad(const __grid_constant__ CUtensorMap mapY, const __grid_constant__ CUtensorMap mapX, SeqGradParams p) {
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

  const int tiles_per_seq = p.tiles_m * p.tiles_n;
  const long long total_units = (long long)p.B * tiles_per_seq;

  if (warp == 0) {
    // ------------------------------------------------------------------ TMA producer
    if (lane == 0) {
      prefetch_tensormap(&mapY);
      prefetch_tensormap(&mapX);
      int stage = 0;
      uint32_t phase = 0;
      bool ok = true;
      for (long long u = blockIdx.x; u < total_units && ok; u += gridDim.x) {
        const int i = (int)(u / tiles_per_seq), tile = (int)(u % tiles_per_seq);
        const int tm = tile / p.tiles_n, tn = tile % p.tiles_n;
        const int64_t t0 = p.off[i], t1 = p.off[i + 1];
        const int nkb = (int)((t1 - t0 + kKB - 1) / kKB);
        for (int kb = 0; kb < nkb; ++kb) {
          if (!(ok = mbar_wait(empty_bar(stage), phase ^ 1u, abort_flag, p.info, kIdSeqGrad))) break;
          const uint32_t a_dst = smem_base + stage * kStageBytes, b_dst = a_dst + kABytes;
          const int y = (int)(t0 + (int64_t)kb * kKB);
          mbar_arrive_expect_tx(full_bar(stage), kStageBytes);
#pragma unroll
          for (int c = 0; c < kTileM / 64; ++c)
            tma_load_2d(a_dst + c * kChunkBytes, &mapY, tm * kTileM + c * 64, y, full_bar(stage));
#pragma unroll
          for (int c = 0; c < kTileN / 64; ++c)
            tma_load_2d(b_dst + c * kChunkBytes, &mapX, tn * kTileN + c * 64, y, full_bar(stage));
          if (++stage == kStages) { stage = 0; phase ^= 1u; }
        }
      }
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------------ MMA issuer
    constexpr uint32_t idesc = make_idesc_bf16(kTileM, kTileN, /*a_mn=*/true, /*b_mn=*/true);
    int stage = 0, acc = 0;
    uint32_t phase = 0, acc_phase = 0;
    bool ok = true;
    for (long long u = blockIdx.x; u < total_units && ok; u += gridDim.x) {
      const int i = (int)(u / tiles_per_seq);
      const int64_t t0 = p.off[i], t1 = p.off[i + 1];
      const int len = (int)(t1 - t0);
      const int nkb = (len + kKB - 1) / kKB;
      if (!(ok = mbar_wait(accempty_bar(acc), acc_phase ^ 1u, abort_flag, p.info, kIdSeqGrad))) break;
      tc_fence_after_sync();
      const uint32_t d_tmem = tmem_base + (uint32_t)acc * kTileN;
      for (int kb = 0; kb < nkb; ++kb) {
        if (!(ok = mbar_wait(full_bar(stage), phase, abort_flag, p.info, kIdSeqGrad))) break;
        tc_fence_after_sync();
        const uint32_t a_addr = smem_base + stage * kStageBytes, b_addr = a_addr + kABytes;
        const int valid = min(kKB, len - kb * kKB);  // token rows of this slab that belong to sequence i
        const int n16 = (valid + 15) >> 4;           // 16-token MMA steps that hold any of them
        if (valid < n16 * 16) {
          // rows [valid, n16*16) hold the next sequence's tokens: zero them in the dY tile
          const int nbytes = (n16 * 16 - valid) * 128;
#pragma unroll
          for (int c = 0; c < kTileM / 64; ++c) {
            const uint32_t base = a_addr + c * kChunkBytes + valid * 128;
            for (int o = lane * 16; o < nbytes; o += 32 * 16)
              asm volatile("st.shared.v4.b32 [%0], {%1, %1, %1, %1};" ::"r"(base + o), "r"(0u) : "memory");
          }
          fence_proxy_async_smem();
        }
        __syncwarp();
        if (lane == 0) {
          for (int k16 = 0; k16 < n16; ++k16) {
            const uint64_t a_desc = make_sdesc_sw128(a_addr + k16 * 2048, kChunkBytes, 1024);
            const uint64_t b_desc = make_sdesc_sw128(b_addr + k16 * 2048, kChunkBytes, 1024);
            mma_bf16(d_tmem, a_desc, b_desc, idesc, (kb | k16) != 0);
          }
          mma_commit(empty_bar(stage));  // frees the stage once these MMAs have read it
        }
        __syncwarp();
        if (++stage == kStages) { stage = 0; phase ^= 1u; }
      }
      if (!ok) break;
      if (lane == 0) mma_commit(accfull_bar(acc));
      __syncwarp();
      if (++acc == 2) { acc = 0; acc_phase ^= 1u; }
    }
  } else {
    // ------------------------------------------------------------------ epilogue (warps 2..5)
    const int q = warp & 3;  // TMEM lane quarter this warp may read
    const int row = q * 32 + lane;
    int acc = 0;
    uint32_t acc_phase = 0;
    for (long long u = blockIdx.x; u < total_units; u += gridDim.x) {
      const int i = (int)(u / tiles_per_seq), tile = (int)(u % tiles_per_seq);
      if (!mbar_wait(accfull_bar(acc), acc_phase, abort_flag, p.info, kIdSeqGrad)) break;
      tc_fence_after_sync();
      uint4* dst = reinterpret_cast<uint4*>(p.G + (size_t)i * p.n_pad + (size_t)tile * kTileElems) + row;
      const uint32_t taddr = tmem_base + ((uint32_t)(q * 32) << 16) + (uint32_t)acc * kTileN;
#pragma unroll 2
      for (int jc = 0; jc < kTileN / 32; ++jc) {
        uint32_t r[32];
        tmem_ld32(taddr + jc * 32, r);
        tmem_ld_wait();
#pragma unroll
        for (int v = 0; v < 4; ++v) {
          uint4 o;
          o.x = pack_bf16x2(__uint_as_float(r[v * 8 + 0]), __uint_as_float(r[v * 8 + 1]));
          o.y = pack_bf16x2(__uint_as_float(r[v * 8 + 2]), __uint_as_float(r[v * 8 + 3]));
          o.z = pack_bf16x2(__uint_as_float(r[v * 8 + 4]), __uint_as_float(r[v * 8 + 5]));
          o.w = pack_bf16x2(__uint_as_float(r[v * 8 + 6]), __uint_as_float(r[v * 8 + 7]));
          dst[(size_t)(jc * 4 + v) * kTileM] = o;
        }
      }
      tc_fence_before_sync();
      __syncwarp();
      if (lane == 0) mbar_arrive(accempty_bar(acc));
      if (++acc == 2) { acc = 0; acc_phase ^= 1u; }
    }
  }

  // ---------------------------------------------------------------------- teardown
  if (*abort_flag) __nanosleep(100000);  // let TMA copies already in flight land before the CTA exits
  tc_fence_before_sync();
  __syncthreads();
  if (warp == 1) tmem_dealloc(tmem_base, kTmemCols);
}

}  // namespace

isopo_status bf16_seq_grad(const void* X, const void* dY, int64_t T, int d_in, int d_out, const int64_t* off_host,
                           const int64_t* off_dev, int B, const WsLayout& L, void* G, int32_t* info, cudaStream_t st) {
  (void)off_host;
  CUtensorMap mapY, mapX;
  isopo_status s = make_map_2d_bf16(&mapY, dY, (uint64_t)T, (uint64_t)d_out, (uint64_t)d_out, 64, kKB);
  if (s != ISOPO_OK) return s;
  s = make_map_2d_bf16(&mapX, X, (uint64_t)T, (uint64_t)d_in, (uint64_t)d_in, 64, kKB);
  if (s != ISOPO_OK) return s;
  int dev = 0, sms = 0;
  ISOPO_CUDA_TRY(cudaGetDevice(&dev));
  ISOPO_CUDA_TRY(cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev));
  ISOPO_CUDA_TRY(cudaFuncSetAttribute(k_bf16_seq_grad, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBytes));
  SeqGradParams p{off_dev, (__nv_bfloat16*)G, L.n_pad, B, L.tiles_m, L.tiles_n, info};
  const long long units = (long long)B * L.tiles_m * L.tiles_n;
  const int grid = (int)std::min<long long>(units, sms);
  {
    LaunchScope scope(kIdSeqGrad, st);
    k_bf16_seq_grad<<<grid, kThreads, kSmemBytes, st>>>(mapY, mapX, p);
  }
  ISOPO_CUDA_TRY(cudaGetLastError());
  return ISOPO_OK;
}

}  // namespace isopo
