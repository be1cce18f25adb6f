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
// The same pipeline, instantiated with kFolded = true, is the stand-alone weight-gradient GEMM
// dW = (c_seq(t) dY)^T X (Alg. 1 "grad += advantages * rescaled gradient"): its work units are
// (tile, token slab), four extra warps multiply every dY row of a landed stage by its sequence's
// coefficient in shared memory (round to nearest even) before the MMA warp may read it, and the
// epilogue adds float32 tiles into the row-major dW.
//
// The stored layout of G (pieces of 32 rows x 8 columns, sequence-minor) is described in
// tc_common.cuh; one epilogue warp writes one 512-byte piece per store instruction.
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
constexpr int kMaxSeqs = 256;                          // sequences whose extents are staged in shared memory
constexpr int kSeqInfoBytes = kMaxSeqs * 16;           // int64 first token, int32 length, int32 index
constexpr int kSmemBytes = kStages * kStageBytes + 1024 /*alignment slack*/ + 256 /*barriers*/ + kSeqInfoBytes;
constexpr int kThreads = 192;
constexpr int kThreadsFolded = 320;                    // + 4 warps that scale the dY rows
constexpr uint32_t kTmemCols = 512;                    // two 256-column float32 accumulators

struct SeqGradParams {
  const int64_t* off;
  const int32_t* order;  // per-sequence mode: the k-th sequence to work on (longest first)
  __nv_bfloat16* G;
  int64_t n_pad;
  int B, tiles_m, tiles_n;
  int32_t* info;
  // folded weight-gradient GEMM only
  const float* tokscale;  // coefficient of every token's sequence
  float* dW;
  int64_t T, slab;  // tokens per work unit (a multiple of 64)
  int nslabs, d_in, d_out;
};

// Extents of the sequences in working order, staged in shared memory by the kernel (per-sequence mode).
struct SeqInfo {
  const int64_t* first;
  const int* len;
  const int* seq;
};

// Work unit u -> (token range, tile).  Per-sequence mode: sequence-major, u = k * tiles + tile with the
// sequences taken longest first: round-robin over the CTAs then gives every CTA a regular sample of
// the sorted lengths, i.e. nearly the same number of tokens.  Folded mode: u = slab * tiles + tile.
template <bool kFolded>
__device__ __forceinline__ void decode_unit(const SeqGradParams& p, const SeqInfo& si, long long u, int tiles, int& tile,
                                            int64_t& t0, int64_t& t1, int& seq) {
  const int k = (int)(u / tiles);
  tile = (int)(u % tiles);
  if (kFolded) {
    seq = k;
    t0 = (int64_t)k * p.slab;
    t1 = min(p.T, t0 + p.slab);
  } else {
    seq = si.seq[k];
    t0 = si.first[k];
    t1 = t0 + si.len[k];
  }
}

template <bool kFolded>
__global__ void __launch_bounds__(kFolded ? kThreadsFolded : kThreads, 1)
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
  auto scaled_bar = [&](int s) { return bar0 + 8u * (2 * kStages + 4 + s); };
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + 3 * kStages + 4);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);
  // read once: the roles look the extents up at every unit, and a global load there would stall
  // the MMA warp for longer than its queue of MMAs lasts
  int64_t* s_first = reinterpret_cast<int64_t*>(smem + kStages * kStageBytes + 256);
  int* s_len = reinterpret_cast<int*>(s_first + kMaxSeqs);
  int* s_seq = s_len + kMaxSeqs;
  if (!kFolded) {
    for (int k = threadIdx.x; k < p.B; k += blockDim.x) {
      const int i = p.order[k];
      const int64_t t0 = p.off[i];
      s_first[k] = t0;
      s_len[k] = (int)(p.off[i + 1] - t0);
      s_seq[k] = i;
    }
  }
  const SeqInfo si{s_first, s_len, s_seq};

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  if (threadIdx.x == 0) {
    for (int s = 0; s < kStages; ++s) {
      mbar_init(full_bar(s), 1);
      mbar_init(empty_bar(s), 1);
      mbar_init(scaled_bar(s), 4);
    }
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
  const long long total_units = (long long)(kFolded ? p.nslabs : p.B) * tiles_per_seq;

  if (warp == 0) {
    // ------------------------------------------------------------------ TMA producer
    if (elect_one()) {
      prefetch_tensormap(&mapY);
      prefetch_tensormap(&mapX);
      int stage = 0;
      uint32_t phase = 0;
      bool ok = true;
      for (long long u = blockIdx.x; u < total_units && ok; u += gridDim.x) {
        int i, tile;
        int64_t t0, t1;
        decode_unit<kFolded>(p, si, u, tiles_per_seq, tile, t0, t1, i);
        const int tm = tile / p.tiles_n, tn = tile % p.tiles_n;
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
      int i, tile;
      int64_t t0, t1;
      decode_unit<kFolded>(p, si, u, tiles_per_seq, tile, t0, t1, i);
      const int len = (int)(t1 - t0);
      const int nkb = (len + kKB - 1) / kKB;
      if (!(ok = mbar_wait(accempty_bar(acc), acc_phase ^ 1u, abort_flag, p.info, kIdSeqGrad))) break;
      tc_fence_after_sync();
      const uint32_t d_tmem = tmem_base + (uint32_t)acc * kTileN;
      for (int kb = 0; kb < nkb; ++kb) {
        // folded mode: the scaler warps hand the stage over (they have waited for the TMA bytes)
        if (!(ok = mbar_wait(kFolded ? scaled_bar(stage) : full_bar(stage), phase, abort_flag, p.info, kIdSeqGrad)))
          break;
        tc_fence_after_sync();
        const uint32_t a_addr = smem_base + stage * kStageBytes, b_addr = a_addr + kABytes;
        const int valid = min(kKB, len - kb * kKB);  // token rows of this slab that belong to the unit
        const int n16 = (valid + 15) >> 4;           // 16-token MMA steps that hold any of them
        if (!kFolded && valid < n16 * 16) {
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
        if (elect_one()) {  // elected, not "lane 0": lets the compiler keep the operands in uniform registers
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
      if (elect_one()) mma_commit(accfull_bar(acc));
      __syncwarp();
      if (++acc == 2) { acc = 0; acc_phase ^= 1u; }
    }
  } else if (warp < 6) {
    // ------------------------------------------------------------------ epilogue (warps 2..5)
    const int q = warp & 3;  // TMEM lane quarter this warp may read
    const int row = q * 32 + lane;
    int acc = 0;
    uint32_t acc_phase = 0;
    for (long long u = blockIdx.x; u < total_units; u += gridDim.x) {
      const int tile = (int)(u % tiles_per_seq);
      const int i = kFolded ? 0 : si.seq[u / tiles_per_seq];
      if (!mbar_wait(accfull_bar(acc), acc_phase, abort_flag, p.info, kIdSeqGrad)) break;
      tc_fence_after_sync();
      const uint32_t taddr = tmem_base + ((uint32_t)(q * 32) << 16) + (uint32_t)acc * kTileN;
      if (!kFolded) {
        uint4* dst = reinterpret_cast<uint4*>(p.G);
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
            const size_t slot = stored_slot(stored_piece(tile, jc * 4 + v, q), i, p.B, lane);
            if (ISOPO_IN_RANGE(i < 0 || i >= p.B ? -1 : (long long)slot, (long long)p.B * p.n_pad / 8, p.info, kIdSeqGrad))
              dst[slot] = o;
          }
        }
      } else {
        // dW[m, n0 .. n0+255] += accumulator row; token slabs of one tile meet here, hence atomics
        const int m = (tile / p.tiles_n) * kTileM + row, n0 = (tile % p.tiles_n) * kTileN;
        float* dst = p.dW + (size_t)m * p.d_in + n0;
#pragma unroll 2
        for (int jc = 0; jc < kTileN / 32; ++jc) {
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
      }
      tc_fence_before_sync();
      __syncwarp();
      if (lane == 0) mbar_arrive(accempty_bar(acc));
      if (++acc == 2) { acc = 0; acc_phase ^= 1u; }
    }
  } else if (kFolded) {
    // ------------------------------------------------------------------ scaler (warps 6..9)
    // Thread (r, h): token row r of the stage, half h of each 128-byte row, in both dY chunks.
    // The 128-byte swizzle permutes 16-byte pieces inside a row only, so a whole row can be scaled
    // in place without knowing the permutation.
    const int st = threadIdx.x - 192, r = st >> 1, h = st & 1;
    int stage = 0;
    uint32_t phase = 0;
    bool ok = true;
    for (long long u = blockIdx.x; u < total_units && ok; u += gridDim.x) {
      int i, tile;
      int64_t t0, t1;
      decode_unit<kFolded>(p, si, u, tiles_per_seq, tile, t0, t1, i);
      const int nkb = (int)((t1 - t0 + kKB - 1) / kKB);
      for (int kb = 0; kb < nkb; ++kb) {
        const int64_t t = t0 + (int64_t)kb * kKB + r;
        const float c = t < t1 ? __ldg(p.tokscale + t) : 0.f;
        if (!(ok = mbar_wait(full_bar(stage), phase, abort_flag, p.info, kIdSeqGrad))) break;
        const uint32_t a_addr = smem_base + stage * kStageBytes + r * 128 + h * 64;
#pragma unroll
        for (int ch = 0; ch < kTileM / 64; ++ch)
#pragma unroll
          for (int v = 0; v < 4; ++v) {
            const uint32_t addr = a_addr + ch * kChunkBytes + v * 16;
            uint32_t w[4];
            asm volatile("ld.shared.v4.b32 {%0, %1, %2, %3}, [%4];"
                         : "=r"(w[0]), "=r"(w[1]), "=r"(w[2]), "=r"(w[3]) : "r"(addr) : "memory");
#pragma unroll
            for (int e = 0; e < 4; ++e)
              w[e] = pack_bf16x2(c * __uint_as_float(w[e] << 16), c * __uint_as_float(w[e] & 0xffff0000u));
            asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(addr), "r"(w[0]), "r"(w[1]), "r"(w[2]),
                         "r"(w[3]) : "memory");
          }
        fence_proxy_async_smem();
        __syncwarp();
        if (lane == 0) mbar_arrive(scaled_bar(stage));
        if (++stage == kStages) { stage = 0; phase ^= 1u; }
      }
    }
  }

  // ---------------------------------------------------------------------- teardown
  if (*abort_flag) __nanosleep(100000);  // let TMA copies already in flight land before the CTA exits
  tc_fence_before_sync();
  __syncthreads();
  if (warp == 1) tmem_dealloc(tmem_base, kTmemCols);
}

}  // namespace

static isopo_status make_maps(CUtensorMap* mapY, CUtensorMap* mapX, const void* X, const void* dY, int64_t T, int d_in,
                              int d_out) {
  isopo_status s = make_map_2d_bf16(mapY, dY, (uint64_t)T, (uint64_t)d_out, (uint64_t)d_out, 64, kKB);
  if (s != ISOPO_OK) return s;
  return make_map_2d_bf16(mapX, X, (uint64_t)T, (uint64_t)d_in, (uint64_t)d_in, 64, kKB);
}

static isopo_status sm_count(int* sms) {
  int dev = 0;
  ISOPO_CUDA_TRY(cudaGetDevice(&dev));
  ISOPO_CUDA_TRY(cudaDeviceGetAttribute(sms, cudaDevAttrMultiProcessorCount, dev));
  return ISOPO_OK;
}

isopo_status bf16_seq_grad(const void* X, const void* dY, int64_t T, int d_in, int d_out, const int64_t* off_host,
                           const int64_t* off_dev, const int32_t* order_dev, int B, const WsLayout& L, void* G,
                           const StoreFmt& fmt, int32_t* info, cudaStream_t st) {
  (void)off_host;
  // 2-CTA tiles (256 rows of G per pair) when they waste little: an odd number of 128-row tiles
  // leaves half of the last pair idle.
  if (L.tiles_m % 2 == 0 || L.tiles_m >= 7)
    return bf16_seq_grad_pair(X, dY, T, d_in, d_out, off_dev, order_dev, B, L, G, fmt, info, st);
  if (fmt.split) return ISOPO_ERR_INVALID_ARG;  // the split store exists in the 2-CTA kernel only (use_split_store)
  CUtensorMap mapY, mapX;
  isopo_status s = make_maps(&mapY, &mapX, X, dY, T, d_in, d_out);
  if (s != ISOPO_OK) return s;
  int sms = 0;
  if ((s = sm_count(&sms)) != ISOPO_OK) return s;
  ISOPO_CUDA_TRY(cudaFuncSetAttribute(k_bf16_seq_grad<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBytes));
  SeqGradParams p{};
  p.off = off_dev; p.order = order_dev; p.G = (__nv_bfloat16*)G; p.n_pad = L.n_pad; p.B = B; p.tiles_m = L.tiles_m; p.tiles_n = L.tiles_n;
  p.info = info;
  const long long units = (long long)B * L.tiles_m * L.tiles_n;
  const int grid = (int)std::min<long long>(units, sms);
  {
    LaunchScope scope(kIdSeqGrad, st);
    k_bf16_seq_grad<false><<<grid, kThreads, kSmemBytes, st>>>(mapY, mapX, p);
  }
  ISOPO_CUDA_TRY(cudaGetLastError());
  return ISOPO_OK;
}

isopo_status bf16_weight_grad(const void* X, const void* dY, int64_t T, int d_in, int d_out, const float* tokscale,
                              void* scaled, float* dW, float beta, int32_t* info, cudaStream_t st) {
  {  // 2-CTA tiles when they waste little (see bf16_seq_grad)
    const int tiles_m = (d_out + kTileM - 1) / kTileM;
    if (tiles_m % 2 == 0 || tiles_m >= 7) return bf16_weight_grad_pair(X, dY, T, d_in, d_out, tokscale, scaled, dW, beta, info, st);
  }
  CUtensorMap mapY, mapX;
  isopo_status s = make_maps(&mapY, &mapX, X, dY, T, d_in, d_out);
  if (s != ISOPO_OK) return s;
  int sms = 0;
  if ((s = sm_count(&sms)) != ISOPO_OK) return s;
  ISOPO_CUDA_TRY(cudaFuncSetAttribute(k_bf16_seq_grad<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBytes));
  if (beta == 0.f) ISOPO_CUDA_TRY(cudaMemsetAsync(dW, 0, sizeof(float) * (size_t)d_in * d_out, st));
  SeqGradParams p{};
  p.tiles_m = (d_out + kTileM - 1) / kTileM;
  p.tiles_n = (d_in + kTileN - 1) / kTileN;
  p.info = info; p.tokscale = tokscale; p.dW = dW; p.T = T; p.d_in = d_in; p.d_out = d_out;
  // token slabs: enough (tile, slab) units to fill the machine about twice, each slab a multiple of 64 tokens
  const long long tiles = (long long)p.tiles_m * p.tiles_n;
  const long long kblocks = (T + kKB - 1) / kKB;
  long long nslabs = std::max<long long>(1, std::min<long long>(kblocks, (2ll * sms + tiles - 1) / tiles));
  const long long kb_per = (kblocks + nslabs - 1) / nslabs;
  nslabs = (kblocks + kb_per - 1) / kb_per;
  p.slab = kb_per * kKB;
  p.nslabs = (int)nslabs;
  const int grid = (int)std::min<long long>(tiles * nslabs, sms);
  {
    LaunchScope scope(kIdWeightGrad, st);
    k_bf16_seq_grad<true><<<grid, kThreadsFolded, kSmemBytes, st>>>(mapY, mapX, p);
  }
  ISOPO_CUDA_TRY(cudaGetLastError());
  return ISOPO_OK;
}

}  // namespace isopo
