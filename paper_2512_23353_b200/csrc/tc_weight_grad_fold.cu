// Stand-alone weight gradient dW = sum_i c_i G_i = (c_seq(t) dY)^T X (Alg. 1: "grad += advantages *
// rescaled gradient"; Sec. 3 display v = J^T c) with the per-sequence coefficient folded into the
// accumulator drain: no scaled copy of an operand is ever written.
//
// dW is a sum over sequences of c_i times a plain product dY_i^T X_i.  A pair of CTAs (cluster of two,
// tcgen05.mma.cta_group::2, 256 x 256 tiles, both operands token-major = "MN-major") takes a work unit
// (tile of dW, chunk of tokens) and walks the chunk one SEGMENT at a time, a segment being a maximal
// run of the chunk's tokens that belong to one sequence.  Every segment is accumulated from zero in
// one of two tensor-memory accumulators; when its last MMA has completed, the epilogue warps read the
// accumulator, multiply by the sequence's coefficient and add into a running sum that lives in
// REGISTERS (8 warps x 32 lanes x 128 columns = the CTA's 128 x 256 half of the tile) while the MMA
// thread is already filling the other accumulator with the next segment.  At the end of the unit
// the running sum is added into dW (float32 reductions: the token chunks of one tile meet there).
// The tile never leaves the SM between segments, so against the pre-scaled-operand GEMM this saves one
// pass over the narrower operand (read + write) and its launch.
//
//   warp 0          TMA producer; both CTAs' copies complete on the barrier in CTA 0
//   warp 1, CTA 0   MMA issuer (one elected thread)
//   warps 2-9       epilogue: warp w reads TMEM lanes 32 (w mod 4) .. +31, columns 128 ((w - 2) / 4) .. +127
//   warp 10         zeroes the dY rows past the end of a segment in its last slab
//
// Barriers are those of tc_seq_grad_pair.cu with "unit" read as "segment".  Every wait is bounded; a
// CTA that gives up raises the abort flag of both CTAs, and both meet at a cluster barrier before
// tensor memory is released.
#include <algorithm>

#include "tc_common.cuh"

namespace isopo {

namespace {

using namespace tc;

constexpr int kKB = 64;                              // tokens per pipeline stage
constexpr int kStages = 6;
constexpr int kHalf = 128;                           // operand columns staged per CTA (both operands)
constexpr int kChunkBytes = kKB * 128;               // one [kKB tokens][64 columns] box
constexpr int kOperandBytes = 2 * kChunkBytes;       // this CTA's half of dY or of X for one stage
constexpr int kStageBytes = 2 * kOperandBytes;
constexpr int kMaxSeqs = 2048;                       // sequences whose extents and coefficients are staged in shared memory
constexpr int kOffBytes = (kMaxSeqs + 1 + 63) / 64 * 64 * 4;
constexpr int kSmemBytes = kStages * kStageBytes + 1024 /*alignment slack*/ + 512 /*barriers*/ + kOffBytes + kMaxSeqs * 4;
constexpr int kEpiWarps = 8;
constexpr int kThreads = 32 * (2 + kEpiWarps + 1);
constexpr uint32_t kTmemCols = 512;                  // two 256-column float32 accumulators
constexpr int kPairN = 256;
constexpr int kUnitOverhead = 6;                     // a unit's pipeline fill and flush, in stages (host cost model)
static_assert(kSmemBytes <= 227 * 1024, "shared memory");

struct FoldParams {
  const int64_t* off;    // [B + 1] token offsets
  const float* coeffs;   // [B]
  float* dW;
  int64_t T, chunk;      // tokens per work unit (a multiple of kKB)
  int nchunks, B, d_in, d_out;
  int ptiles_m, tiles_n;  // 256-row and 256-column tiles of dW
  int group_m;            // tile rows per group of the tile order (see pair_tile)
  int32_t* info;
};

// Tiles are visited in groups of `group_m` rows, row index fastest inside a group, so that the pairs
// running at one time share about group_m row blocks of dY and npairs / group_m column blocks of X.
__device__ __forceinline__ void pair_tile(int pt, const FoldParams& p, int& ptm, int& tn) {
  const int per_group = p.group_m * p.tiles_n;
  const int first = (pt / per_group) * p.group_m, in_group = pt % per_group;
  const int gm = min(p.group_m, p.ptiles_m - first);
  ptm = first + in_group % gm;
  tn = in_group / gm;
}

// Shape of one segment's token loop, identical in every role.
struct SegShape {
  int nkb;         // slabs
  int tail_n16;    // 16-token MMA steps of the last slab
  int tail_valid;  // token rows of the last slab that belong to the segment
  bool fix;        // the last step holds rows of the next segment
};
__device__ __forceinline__ SegShape seg_shape(int len) {
  SegShape s;
  s.nkb = (len + kKB - 1) / kKB;
  s.tail_valid = len - (s.nkb - 1) * kKB;
  s.tail_n16 = (s.tail_valid + 15) >> 4;
  s.fix = s.tail_valid < s.tail_n16 * 16;
  return s;
}

// Walks the segments of the token range [t, t_end): sequence i holds tokens off[i] .. off[i+1]-1.
struct SegWalk {
  const int* off;
  int t, t_end, i;
  __device__ __forceinline__ SegWalk(const int* off32, int B, int t0, int t1) : off(off32), t(t0), t_end(t1) {
    int lo = 0, hi = B;  // invariant: off[lo] <= t0 < off[hi]
    while (hi - lo > 1) {
      const int mid = (lo + hi) >> 1;
      if (off[mid] <= t0) lo = mid; else hi = mid;
    }
    i = lo;
  }
  __device__ __forceinline__ bool done() const { return t >= t_end; }
  __device__ __forceinline__ int len() const { return min(off[i + 1], t_end) - t; }
  __device__ __forceinline__ void next() { t += len(); ++i; }
};

__device__ __forceinline__ void tmem_ld16(uint32_t taddr, uint32_t (&r)[16]) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x16.b32 "
      "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15}, [%16];"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]),
        "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15])
      : "r"(taddr)
      : "memory");
}

__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(kThreads, 1)
k_bf16_weight_grad_fold(const __grid_constant__ CUtensorMap mapY, const __grid_constant__ CUtensorMap mapX, FoldParams p) {
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  const uint32_t smem_base = smem_u32(smem);
  uint64_t* bars = reinterpret_cast<uint64_t*>(smem + kStages * kStageBytes);
  const uint32_t bar0 = smem_u32(bars);
  auto full_bar = [&](int s) { return bar0 + 8u * s; };                          // used in CTA 0
  auto empty_bar = [&](int s) { return bar0 + 8u * (kStages + s); };             // both CTAs
  auto tail_bar = [&](int s) { return bar0 + 8u * (2 * kStages + s); };          // both CTAs
  auto fixed_bar = [&](int s) { return bar0 + 8u * (3 * kStages + s); };         // used in CTA 0
  auto accfull_bar = [&](int b) { return bar0 + 8u * (4 * kStages + b); };       // both CTAs
  auto accempty_bar = [&](int b) { return bar0 + 8u * (4 * kStages + 2 + b); };  // used in CTA 0
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + 4 * kStages + 4);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);
  // offsets (as 32-bit token indices) and coefficients, read once: the roles look them up at every
  // segment, and a global load there would stall the MMA thread for longer than its queue of MMAs lasts
  int* s_off = reinterpret_cast<int*>(smem + kStages * kStageBytes + 512);
  float* s_coef = reinterpret_cast<float*>(smem + kStages * kStageBytes + 512 + kOffBytes);
  for (int k = threadIdx.x; k <= p.B; k += kThreads) s_off[k] = (int)p.off[k];
  for (int k = threadIdx.x; k < p.B; k += kThreads) s_coef[k] = p.coeffs[k];

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const uint32_t rank = cluster_ctarank();  // 0 issues the MMAs
  const uint32_t peer_abort = map_to_cta(smem_u32(const_cast<int*>(abort_flag)), rank ^ 1u);
  if (threadIdx.x == 0) {
    for (int s = 0; s < kStages; ++s) {
      mbar_init(full_bar(s), 1);
      mbar_init(empty_bar(s), 1);
      mbar_init(tail_bar(s), 1);
      mbar_init(fixed_bar(s), 2);
    }
    for (int b = 0; b < 2; ++b) { mbar_init(accfull_bar(b), 1); mbar_init(accempty_bar(b), 2 * kEpiWarps); }
    *abort_flag = 0;
    fence_barrier_init();
  }
  if (warp == 1) tmem_alloc_pair(smem_u32(tmem_slot), kTmemCols);
  tc_fence_before_sync();
  __syncthreads();
  __syncwarp();
  cluster_sync_all();  // the peer's barriers exist before anything can arrive on them
  tc_fence_after_sync();
  const uint32_t tmem_base = *tmem_slot;

  const int ptiles = p.ptiles_m * p.tiles_n;
  const long long total_units = (long long)p.nchunks * ptiles;
  const long long pair_id = blockIdx.x >> 1, npairs = gridDim.x >> 1;
  // unit u = chunk * ptiles + tile: the pairs running at one time read the same tokens out of L2
  auto unit_tokens = [&](long long u, int& t0, int& t1) {
    const int64_t a = (u / ptiles) * p.chunk;
    t0 = (int)a;
    t1 = (int)min(p.T, a + p.chunk);
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
        int ptm, tn, t0, t1;
        pair_tile((int)(u % ptiles), p, ptm, tn);
        unit_tokens(u, t0, t1);
        const int ycol = (2 * ptm + (int)rank) * kHalf, xcol = tn * kPairN + (int)rank * kHalf;
        for (SegWalk w(s_off, p.B, t0, t1); !w.done() && ok; w.next()) {
          const SegShape ss = seg_shape(w.len());
          for (int kb = 0; kb < ss.nkb; ++kb) {
            if (!(ok = mbar_wait_pair(empty_bar(stage), phase ^ 1u, abort_flag, peer_abort, p.info, kIdWeightGrad))) break;
            const uint32_t a_dst = smem_base + stage * kStageBytes, b_dst = a_dst + kOperandBytes;
            const int y = w.t + kb * kKB;  // rows past T and columns past the matrix read as zero
            const bool own_tail = ss.fix && kb == ss.nkb - 1;  // dY goes to this CTA's tail barrier
            if (own_tail) mbar_arrive_expect_tx(tail_bar(stage), kOperandBytes);
            if (rank == 0) mbar_arrive_expect_tx(full_bar(stage), own_tail ? 2 * kOperandBytes : 2 * kStageBytes);
            const uint32_t fb = full_at_leader + 8u * stage;
#pragma unroll
            for (int c = 0; c < 2; ++c) {
              if (own_tail) tma_load_2d(a_dst + c * kChunkBytes, &mapY, ycol + c * 64, y, tail_bar(stage));
              else tma_load_2d_pair(a_dst + c * kChunkBytes, &mapY, ycol + c * 64, y, fb);
              tma_load_2d_pair(b_dst + c * kChunkBytes, &mapX, xcol + c * 64, y, fb);
            }
            if (++stage == kStages) { stage = 0; phase ^= 1u; }
          }
        }
      }
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------------ MMA issuer (one thread of CTA 0)
    if (rank == 0 && elect_one()) {
      constexpr uint32_t idesc = make_idesc_bf16(256, kPairN, /*a_mn=*/true, /*b_mn=*/true);
      int stage = 0, acc = 0;
      uint32_t phase = 0, acc_phase = 0, fixed_phase = 0;  // fixed_phase: one bit per stage
      bool ok = true;
      for (long long u = pair_id; u < total_units && ok; u += npairs) {
        int t0, t1;
        unit_tokens(u, t0, t1);
        for (SegWalk w(s_off, p.B, t0, t1); !w.done() && ok; w.next()) {
          const SegShape ss = seg_shape(w.len());
          if (!(ok = mbar_wait_pair(accempty_bar(acc), acc_phase ^ 1u, abort_flag, peer_abort, p.info, kIdWeightGrad))) break;
          tc_fence_after_sync();
          const uint32_t d_tmem = tmem_base + (uint32_t)acc * kPairN;
          for (int kb = 0; kb < ss.nkb; ++kb) {
            const bool last = kb == ss.nkb - 1;
            if (!(ok = mbar_wait_pair(full_bar(stage), phase, abort_flag, peer_abort, p.info, kIdWeightGrad))) break;
            if (last && ss.fix) {
              // both CTAs' dY halves of this slab have landed and their stray rows are zero
              if (!(ok = mbar_wait_pair(fixed_bar(stage), (fixed_phase >> stage) & 1u, abort_flag, peer_abort, p.info,
                                        kIdWeightGrad)))
                break;
              fixed_phase ^= 1u << stage;
            }
            tc_fence_after_sync();
            const uint32_t a_addr = smem_base + stage * kStageBytes, b_addr = a_addr + kOperandBytes;
            const int n16 = last ? ss.tail_n16 : kKB / 16;
            for (int k16 = 0; k16 < n16; ++k16) {
              const uint64_t a_desc = make_sdesc_sw128(a_addr + k16 * 2048, kChunkBytes, 1024);
              const uint64_t b_desc = make_sdesc_sw128(b_addr + k16 * 2048, kChunkBytes, 1024);
              mma_bf16_pair(d_tmem, a_desc, b_desc, idesc, (kb | k16) != 0);
            }
            mma_commit_pair(empty_bar(stage));  // frees the stage in both CTAs once these MMAs have read it
            if (++stage == kStages) { stage = 0; phase ^= 1u; }
          }
          if (!ok) break;
          mma_commit_pair(accfull_bar(acc));
          if (++acc == 2) { acc = 0; acc_phase ^= 1u; }
        }
      }
    }
  } else if (warp < 2 + kEpiWarps) {
    // ------------------------------------------------------------------ epilogue (warps 2..9, both CTAs)
    const int q = warp & 3;            // TMEM lane quarter this warp may read
    const int h = (warp - 2) >> 2;     // column half of the tile
    const uint32_t accempty_at_leader = map_to_cta(accempty_bar(0), 0);
    float sum[128];
#pragma unroll
    for (int e = 0; e < 128; ++e) sum[e] = 0.f;
    int acc = 0;
    uint32_t acc_phase = 0;
    bool ok = true;
    for (long long u = pair_id; u < total_units && ok; u += npairs) {
      int ptm, tn, t0, t1;
      pair_tile((int)(u % ptiles), p, ptm, tn);
      unit_tokens(u, t0, t1);
      for (SegWalk w(s_off, p.B, t0, t1); !w.done(); w.next()) {
        const float c = ISOPO_IN_RANGE(w.i, p.B, p.info, kIdWeightGrad) ? s_coef[w.i] : 0.f;
        if (!(ok = mbar_wait_pair(accfull_bar(acc), acc_phase, abort_flag, peer_abort, p.info, kIdWeightGrad))) break;
        tc_fence_after_sync();
        const uint32_t taddr = tmem_base + ((uint32_t)(q * 32) << 16) + (uint32_t)(acc * kPairN + h * 128);
#pragma unroll
        for (int jc = 0; jc < 8; ++jc) {
          uint32_t r[16];
          tmem_ld16(taddr + jc * 16, r);
          tmem_ld_wait();
#pragma unroll
          for (int e = 0; e < 16; ++e) sum[jc * 16 + e] = fmaf(c, __uint_as_float(r[e]), sum[jc * 16 + e]);
        }
        tc_fence_before_sync();
        __syncwarp();
        if (lane == 0) mbar_arrive_remote(accempty_at_leader + 8u * acc);
        if (++acc == 2) { acc = 0; acc_phase ^= 1u; }
      }
      if (!ok) break;
      // the unit's share of this tile: dW[m, n0 .. n0 + 127] += sum
      const int m = (2 * ptm + (int)rank) * kHalf + q * 32 + lane, n0 = tn * kPairN + h * 128;
      float* dst = p.dW + (size_t)m * p.d_in + n0;
#pragma unroll
      for (int v = 0; v < 32; ++v) {
        if (m < p.d_out && n0 + v * 4 < p.d_in &&  // d_in is a multiple of 8, so a group of 4 is all in or all out
            ISOPO_IN_RANGE((long long)m * p.d_in + n0 + v * 4 + 3, (long long)p.d_out * p.d_in, p.info, kIdWeightGrad))
          asm volatile("red.global.add.v4.f32 [%0], {%1, %2, %3, %4};" ::"l"(dst + v * 4), "f"(sum[v * 4 + 0]),
                       "f"(sum[v * 4 + 1]), "f"(sum[v * 4 + 2]), "f"(sum[v * 4 + 3])
                       : "memory");
        sum[v * 4 + 0] = sum[v * 4 + 1] = sum[v * 4 + 2] = sum[v * 4 + 3] = 0.f;
      }
    }
  } else {
    // ------------------------------------------------------------------ tail warp (warp 10, both CTAs)
    // tail[s] is used only for last slabs that need the fix, so its phase is counted per stage; it
    // cannot run ahead: the stage is not reloaded before the MMA thread has passed fixed[s].
    const uint32_t fixed_at_leader = map_to_cta(fixed_bar(0), 0);
    int stage = 0;
    uint32_t tail_phase = 0;  // one bit per stage
    bool ok = true;
    for (long long u = pair_id; u < total_units && ok; u += npairs) {
      int t0, t1;
      unit_tokens(u, t0, t1);
      for (SegWalk w(s_off, p.B, t0, t1); !w.done(); w.next()) {
        const SegShape ss = seg_shape(w.len());
        const int ts = (stage + ss.nkb - 1) % kStages;  // ring position of the last slab
        if (ss.fix) {
          if (!(ok = mbar_wait_pair(tail_bar(ts), (tail_phase >> ts) & 1u, abort_flag, peer_abort, p.info, kIdWeightGrad))) break;
          tail_phase ^= 1u << ts;
          // rows [tail_valid, tail_n16*16) hold the next segment's tokens
          const int nbytes = (ss.tail_n16 * 16 - ss.tail_valid) * 128;
          const uint32_t a_addr = smem_base + ts * kStageBytes;
#pragma unroll
          for (int c = 0; c < 2; ++c) {
            const uint32_t base = a_addr + c * kChunkBytes + ss.tail_valid * 128;
            for (int o = lane * 16; o < nbytes; o += 32 * 16)
              asm volatile("st.shared.v4.b32 [%0], {%1, %1, %1, %1};" ::"r"(base + o), "r"(0u) : "memory");
          }
          fence_proxy_async_smem();
          __syncwarp();
          // the zeroed rows are in this CTA's shared memory and only this CTA's tensor core reads
          // them; the arrival (CTA scope) merely tells the MMA thread that they are there
          if (lane == 0) mbar_arrive_remote(fixed_at_leader + 8u * ts);
        }
        stage = (ts + 1) % kStages;
      }
    }
  }

  // ---------------------------------------------------------------------- teardown
  if (*abort_flag) __nanosleep(100000);  // let TMA copies already in flight land before the CTA exits
  tc_fence_before_sync();
  __syncthreads();
  __syncwarp();
  cluster_sync_all();  // neither CTA leaves (or frees tensor memory) while the other may still use it
  if (warp == 1) tmem_dealloc_pair(tmem_base, kTmemCols);
}

}  // namespace

// Where this kernel is the faster route (measured against the pre-scaled-operand GEMM of
// tc_weight_grad_pair.cu, interleaved on one B200 under its power cap): layers whose wider side is at
// most 2048 (the scaling pass there costs 10-25 % of the GEMM; q/o 1536 x 1536: 1.63-1.80 against
// 1.80-1.92 ms, 896 x 896: 0.068 against 0.083 ms).  On wider layers the other kernel's 256 x 512 blocks
// move a quarter fewer operand bytes from L2 per flop, which under the power cap outweighs its extra
// pass (8960 x 1536: 7.0-8.5 against 7.9-9.1 ms; 18944 x 3584: 34-40 against 37-48 ms).
bool bf16_weight_grad_fold_applies(int64_t T, int d_in, int d_out, int B) {
  const int tiles_m = (d_out + kHalf - 1) / kHalf;
  // 2-CTA tiles when they waste little; segments long enough that the drain per segment stays hidden
  return (tiles_m % 2 == 0 || tiles_m >= 7) && std::max(d_in, d_out) <= 2048 && B <= kMaxSeqs && T >= (int64_t)B * 96 &&
         T < ((int64_t)1 << 31) - 4096;
}

isopo_status bf16_weight_grad_fold(const void* X, const void* dY, int64_t T, int d_in, int d_out, const int64_t* off_dev,
                                   const float* coeffs, int B, float* dW, float beta, int32_t* info, cudaStream_t st) {
  int dev = 0, sms = 0;
  ISOPO_CUDA_TRY(cudaGetDevice(&dev));
  ISOPO_CUDA_TRY(cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev));
  CUtensorMap mapY, mapX;
  isopo_status s = make_map_2d_bf16(&mapY, dY, (uint64_t)T, (uint64_t)d_out, (uint64_t)d_out, 64, kKB);
  if (s != ISOPO_OK) return s;
  s = make_map_2d_bf16(&mapX, X, (uint64_t)T, (uint64_t)d_in, (uint64_t)d_in, 64, kKB);
  if (s != ISOPO_OK) return s;
  ISOPO_CUDA_TRY(cudaFuncSetAttribute(k_bf16_weight_grad_fold, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBytes));
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
    ISOPO_CUDA_TRY(cudaOccupancyMaxActiveClusters(&n, k_bf16_weight_grad_fold, &cfg));
    if (n < 1) return ISOPO_ERR_UNSUPPORTED;
    resident_pairs[dev] = std::min(n, sms / 2);
  }
  FoldParams p{};
  p.off = off_dev; p.coeffs = coeffs; p.dW = dW; p.T = T; p.B = B; p.d_in = d_in; p.d_out = d_out; p.info = info;
  p.ptiles_m = ((d_out + kHalf - 1) / kHalf + 1) / 2;
  p.tiles_n = (d_in + kPairN - 1) / kPairN;
  // token chunks: the count (up to 64) whose rounds of units take least, a round costing its chunk plus the
  // unit's pipeline fill and flush; ties go to fewer chunks.  Every chunk is a whole number of stages.
  // (Chunks small enough to stay in L2 while all tiles pass over them were measured slower: the float32
  // reductions into dW and the fills grow with the chunk count, and the inputs were still read 2.6 x.)
  const long long ptiles = (long long)p.ptiles_m * p.tiles_n, pairs = resident_pairs[dev];
  const long long kblocks = (T + kKB - 1) / kKB;
  long long nchunks = 1, best = -1;
  for (long long n = 1; n <= std::min<long long>(64, kblocks); ++n) {
    const long long per = (kblocks + n - 1) / n, rounds = (ptiles * n + pairs - 1) / pairs;
    const long long cost = rounds * (per + kUnitOverhead);
    if (best < 0 || cost < best) { best = cost; nchunks = n; }
  }
  const long long kb_per = (kblocks + nchunks - 1) / nchunks;
  nchunks = (kblocks + kb_per - 1) / kb_per;
  p.chunk = kb_per * kKB;
  p.nchunks = (int)nchunks;
  const int npairs = (int)std::max<long long>(1, std::min<long long>(ptiles * nchunks, pairs));
  int g = 1;
  while ((g + 1) * (g + 1) <= npairs) ++g;  // about sqrt(npairs) rows by sqrt(npairs) columns of tiles in flight
  p.group_m = std::max(1, std::min(g, p.ptiles_m));
  {
    LaunchScope scope(kIdWeightGrad, st);
    k_bf16_weight_grad_fold<<<2 * npairs, kThreads, kSmemBytes, st>>>(mapY, mapX, p);
  }
  ISOPO_CUDA_TRY(cudaGetLastError());
  return ISOPO_OK;
}

}  // namespace isopo
