// K = G_flat G_flat^T from the stored per-sequence gradients (Alg. 2 "make neural tangent kernel":
// K_ij = sum(G_i * G_j)), and dW = sum_i c_i G_i from the same store (Alg. 2 last line).
//
// k_bf16_ntk: the B <= 256 stored gradients form a [pieces][B][256] bf16 array (tc_common.cuh).  Each CTA
// takes a contiguous run of the long contraction dimension, streams [B rows] x [64 elements] boxes
// (four per piece, so a CTA walks memory front to back) through a TMA ring, and uses every box as BOTH tcgen05 operands (K-major): rows 0..127 against all rows,
// then rows 128..255 against rows 128..255 (the lower-left block is the mirror of the upper-right).
// The float32 accumulators stay in tensor memory for the whole slab and are added into K once, with
// reductions across CTAs by float atomics; a last tiny kernel mirrors the upper triangle.
// For B <= 128 a box holds only the rows that exist (32, 64 or 128 >= B) but spans 8, 4 or 2 pieces, so
// that every TMA copy still moves 32 KB (small boxes cost a fixed ~100 clocks each) and the stage is
// again 256 rows: rows 0..127 and rows 128..255 each go through ONE 128 x 128 MMA per 16 elements,
// which multiplies 4, 2 or 1 pieces at once.  Only the diagonal blocks of that product (a piece
// against itself) are wanted; the epilogue adds them into K and skips the cross-piece blocks.  The
// tensor pipe does up to four times the needed work this way, but in a quarter of the instructions:
// with one 128 x 64 MMA per piece the pass was bound by the MMA issue rate (4.0 TB/s at B = 64
// against 5.4 TB/s at B = 256 on the same clock), and the pipe has time to spare in an HBM-bound pass.
// The order of the blocks inside the long contraction does not matter.
//
// k_bf16_combine: pure streaming, one 16-byte slot of every G_i per thread; a warp reads 512
// contiguous bytes per sequence and the B sequences of a piece back to back.
#include "tc_common.cuh"

namespace isopo {

namespace {

using namespace tc;

constexpr int kKB = 64;               // contraction elements per stage (one 128-byte row)
constexpr int kStages = 6;
constexpr int kStageBytes = 256 * 128;  // 256 rows x 128 bytes
constexpr int kSmemBytes = kStages * kStageBytes + 1024 + 256;
constexpr int kThreads = 192;
constexpr uint32_t kTmemCols = 512;

struct NtkParams {
  float* kpart;   // deterministic mode: [CTA][B * B] partial sums, plain stores; NULL: float atomics into K
  const float* scales;  // split store: s_i per sequence (the `hi` plane holds s_i G_i); the diagonal is not written here
  float* K;
  int B;
  long long nkb;  // boxes in the contraction dimension: ceil(pieces / ppb) * 4
  int32_t* info;
  int box_rows;   // rows of a piece inside a box: 32, 64, 128 or 256, >= B
  int ppb;        // pieces per box = 256 / box_rows
};

// kE4m3: the operand is the `hi` plane of the split store: 128 one-byte elements per 128-byte box row (two boxes
// per piece instead of four), kind::f8f6f4 MMAs of 32 elements each - the same number of MMAs per byte, half the bytes.
template <bool kE4m3>
__global__ void __launch_bounds__(kThreads, 1) k_bf16_ntk(const __grid_constant__ CUtensorMap mapG, NtkParams p) {
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  const uint32_t smem_base = smem_u32(smem);
  uint64_t* bars = reinterpret_cast<uint64_t*>(smem + kStages * kStageBytes);
  const uint32_t bar0 = smem_u32(bars);
  auto full_bar = [&](int s) { return bar0 + 8u * s; };
  auto empty_bar = [&](int s) { return bar0 + 8u * (kStages + s); };
  const uint32_t accfull_bar = bar0 + 8u * (2 * kStages);
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + 2 * kStages + 1);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  if (threadIdx.x == 0) {
    for (int s = 0; s < kStages; ++s) { mbar_init(full_bar(s), 1); mbar_init(empty_bar(s), 1); }
    mbar_init(accfull_bar, 1);
    *abort_flag = 0;
    fence_barrier_init();
  }
  if (warp == 1) tmem_alloc(smem_u32(tmem_slot), kTmemCols);
  tc_fence_before_sync();
  __syncthreads();
  tc_fence_after_sync();
  const uint32_t tmem_base = *tmem_slot;

  // this CTA's slab of the contraction dimension
  const long long per = (p.nkb + gridDim.x - 1) / gridDim.x;
  const long long kb0 = (long long)blockIdx.x * per, kb1 = min(p.nkb, kb0 + per);
  const bool two = p.B > 128;                       // one piece per box, K in two row blocks
  const uint32_t stage_tx = kStageBytes;            // rows >= B and pieces past the end arrive as zeros and count
  // MMA 1: rows 0..127 against n1 rows from row 0; MMA 2: rows 128..255 against n2 rows from row 128
  const int n1 = two ? 256 : (p.box_rows == 128 ? max(16, (p.B + 15) & ~15) : 128);
  const int n2 = two ? max(16, (p.B - 128 + 15) & ~15) : n1;

  if (kb0 < kb1) {
    if (warp == 0) {
      if (elect_one()) {
        prefetch_tensormap(&mapG);
        int stage = 0;
        uint32_t phase = 0;
        for (long long kb = kb0; kb < kb1; ++kb) {
          if (!mbar_wait(empty_bar(stage), phase ^ 1u, abort_flag, p.info, kIdNtk)) break;
          mbar_arrive_expect_tx(full_bar(stage), stage_tx);
          if (kE4m3)
            tma_load_3d(smem_base + stage * kStageBytes, &mapG, (int)(kb & 1) * 128, 0, (int)(kb >> 1) * p.ppb, full_bar(stage));
          else
            tma_load_3d(smem_base + stage * kStageBytes, &mapG, (int)(kb & 3) * kKB, 0, (int)(kb >> 2) * p.ppb, full_bar(stage));
          if (++stage == kStages) { stage = 0; phase ^= 1u; }
        }
      }
    } else if (warp == 1) {
      if (elect_one()) {  // elected, not "lane 0": lets the compiler keep the MMA operands in uniform registers
        const uint32_t idesc1 = kE4m3 ? make_idesc_e4m3(128, n1) : make_idesc_bf16(128, n1, false, false);
        const uint32_t idesc2 = kE4m3 ? make_idesc_e4m3(128, n2) : make_idesc_bf16(128, n2, false, false);
        int stage = 0;
        uint32_t phase = 0;
        bool ok = true;
        for (long long kb = kb0; kb < kb1; ++kb) {
          if (!(ok = mbar_wait(full_bar(stage), phase, abort_flag, p.info, kIdNtk))) break;
          tc_fence_after_sync();
          const uint32_t base = smem_base + stage * kStageBytes;
#pragma unroll
          for (int k16 = 0; k16 < kKB / 16; ++k16) {
            const bool accum = (kb > kb0) || k16 > 0;
            const uint64_t d0 = make_sdesc_sw128(base + k16 * 32, 16, 1024);
            const uint64_t d1 = make_sdesc_sw128(base + 128 * 128 + k16 * 32, 16, 1024);
            if (kE4m3) {
              mma_e4m3(tmem_base, d0, d0, idesc1, accum);
              mma_e4m3(tmem_base + 256, d1, d1, idesc2, accum);
            } else {
              mma_bf16(tmem_base, d0, d0, idesc1, accum);
              mma_bf16(tmem_base + 256, d1, d1, idesc2, accum);
            }
          }
          mma_commit(empty_bar(stage));
          if (++stage == kStages) { stage = 0; phase ^= 1u; }
        }
        if (ok) mma_commit(accfull_bar);
      }
    } else {
      const int q = warp & 3;
      const int r = q * 32 + lane;
      // every (CTA, entry of the upper triangle) is produced by exactly one thread, once
      float* const mine = p.kpart ? p.kpart + (size_t)blockIdx.x * p.B * p.B : nullptr;
      auto add_to_k = [&](size_t idx, float v) {
        if (mine) mine[idx] = v; else atomicAdd(&p.K[idx], v);
      };
      // `ok` is false only after a wait ran out; every thread still reaches the named barriers below
      const bool ok = mbar_wait(accfull_bar, 0, abort_flag, p.info, kIdNtk);
      // split store: the accumulators hold s_i s_j <G_i, G_j>; 1 / s_i of every sequence goes to shared memory (the ring
      // is idle by now), and the diagonal is left to the gradient GEMM's float32 sums
      float* inv_s = reinterpret_cast<float*>(smem + 128 * 1024);
      if (kE4m3) {
        for (int i = r; i < 256; i += 128) inv_s[i] = i < p.B ? 1.f / __ldg(p.scales + i) : 0.f;
        asm volatile("bar.sync 2, 128;" ::: "memory");
      }
      auto unscale = [&](int row, int col, float v) { return kE4m3 ? v * inv_s[row] * inv_s[col] : v; };
      {
        tc_fence_after_sync();
        const uint32_t tlane = (uint32_t)(q * 32) << 16;
        if (two && ok) {
          // block A: rows 0..127 x columns 0..255 of K; keep the upper triangle c >= r
          for (int c0 = 0; c0 < n1; c0 += 32) {
            uint32_t v[32];
            tmem_ld32(tmem_base + tlane + c0, v);
            tmem_ld_wait();
            if (r < p.B) {
#pragma unroll
              for (int e = 0; e < 32; ++e) {
                const int c = c0 + e;
                if (c >= r + (kE4m3 ? 1 : 0) && c < p.B &&
                    ISOPO_IN_RANGE((long long)r * p.B + c, (long long)p.B * p.B, p.info, kIdNtk))
                  add_to_k((size_t)r * p.B + c, unscale(r, c, __uint_as_float(v[e])));
              }
            }
          }
          // block B: rows 128..255 x columns 128..255
          const int rr = 128 + r;
          for (int c0 = 0; c0 < n2; c0 += 32) {
            uint32_t v[32];
            tmem_ld32(tmem_base + tlane + 256 + c0, v);
            tmem_ld_wait();
            if (rr < p.B) {
#pragma unroll
              for (int e = 0; e < 32; ++e) {
                const int c = 128 + c0 + e;
                if (c >= rr + (kE4m3 ? 1 : 0) && c < p.B &&
                    ISOPO_IN_RANGE((long long)rr * p.B + c, (long long)p.B * p.B, p.info, kIdNtk))
                  add_to_k((size_t)rr * p.B + c, unscale(rr, c, __uint_as_float(v[e])));
              }
            }
          }
        } else if (!two) {
          // both accumulators hold 128 / box_rows pieces side by side: row r is sequence r mod box_rows of
          // piece-group g = r / box_rows, whose columns start at g * box_rows.  Every thread leaves the sum
          // of its two accumulator rows in shared memory (the ring is idle by now); then the 128 threads
          // walk the box_rows x box_rows block together, add the groups and update K.
          const int lr = 31 - __clz(p.box_rows), rows = 1 << lr;  // box_rows is a power of two
          const int seq = r & (rows - 1), g = r >> lr, coff = r - seq, ngroups = 128 >> lr;
          const int ncol = min(rows, p.B);
          float* red = reinterpret_cast<float*>(smem);  // [group][column][sequence]
          if (ok) {
            for (int c0 = 0; c0 < ncol; c0 += 32) {
              uint32_t v0[32], v1[32];
              tmem_ld32(tmem_base + tlane + coff + c0, v0);
              tmem_ld32(tmem_base + tlane + 256 + coff + c0, v1);
              tmem_ld_wait();
              float* dst = red + ((((g << lr) + c0) << lr) + seq);
#pragma unroll
              for (int e = 0; e < 32; ++e) dst[e << lr] = __uint_as_float(v0[e]) + __uint_as_float(v1[e]);
            }
          }
          asm volatile("bar.sync 1, 128;" ::: "memory");  // the four epilogue warps
          if (ok) {
            for (int idx = r; idx < (ncol << lr); idx += 128) {
              const int sq = idx & (rows - 1), c = idx >> lr;
              if (c < sq + (kE4m3 ? 1 : 0) || sq >= p.B) continue;  // upper triangle of the sequences that exist
              float sum = 0.f;
              for (int h = 0; h < ngroups; ++h) sum += red[(((h << lr) + c) << lr) + sq];
              if (ISOPO_IN_RANGE((long long)sq * p.B + c, (long long)p.B * p.B, p.info, kIdNtk))
                add_to_k((size_t)sq * p.B + c, unscale(sq, c, sum));
            }
          }
        }
      }
    }
  }

  if (*abort_flag) __nanosleep(100000);
  tc_fence_before_sync();
  __syncthreads();
  if (warp == 1) tmem_dealloc(tmem_base, kTmemCols);
}

// Deterministic mode: K[i][j] = K[j][i] = sum over the CTAs, in CTA order, of their partial entry (i, j), i <= j.
// One thread per entry of the upper triangle (its reads run along a row of every partial matrix), which also
// writes the mirrored entry.
__global__ void k_ntk_reduce(const float* __restrict__ kpart, int n_ctas, int B, float* __restrict__ K) {
  const int e = blockIdx.x * blockDim.x + threadIdx.x;
  if (e >= B * B) return;
  const int i = e / B, j = e % B;
  if (j < i) return;
  const size_t stride = (size_t)B * B;
  float s = 0.f;
  int c = 0;
  for (; c + 8 <= n_ctas; c += 8) {  // eight loads in flight; the additions keep the CTA order
    float v[8];
#pragma unroll
    for (int u = 0; u < 8; ++u) v[u] = __ldcs(kpart + (c + u) * stride + e);
#pragma unroll
    for (int u = 0; u < 8; ++u) s += v[u];
  }
  for (; c < n_ctas; ++c) s += __ldcs(kpart + c * stride + e);
  K[e] = s;
  K[(size_t)j * B + i] = s;
}

// kdiag != NULL (split store): the diagonal comes from the gradient GEMM's float32 sums of squares
__global__ void k_mirror_upper(float* __restrict__ K, int B, const float* __restrict__ kdiag) {
  const int e = blockIdx.x * blockDim.x + threadIdx.x;
  if (e >= B * B) return;
  const int i = e / B, j = e % B;
  if (j < i) K[e] = K[(size_t)j * B + i];
  else if (j == i && kdiag) K[e] = kdiag[i];
}

#ifndef ISOPO_COMBINE_IN_FLIGHT
#define ISOPO_COMBINE_IN_FLIGHT 16
#endif
constexpr int kCombineInFlight = ISOPO_COMBINE_IN_FLIGHT;  // 16-byte loads a thread has in flight
// dW = beta dW + sum_i c_i G_i.  One thread per 16-byte slot (8 elements of every G_i) of the piece-blocked store.
__global__ void __launch_bounds__(256) k_bf16_combine(const uint4* __restrict__ G, long long nchunks /* n_pad / 8 */,
                                                       int B, int tiles_n, int d_in, int d_out,
                                                       const float* __restrict__ coeffs, float* __restrict__ dW,
                                                       float beta, const WsTag* __restrict__ tag_dev, WsTag tag,
                                                       int32_t* __restrict__ info) {
  if (!ws_tag_matches(tag_dev, tag, info)) return;  // another layer's or microbatch's gradients: touch nothing
  __shared__ float sc[256];
  for (int i = threadIdx.x; i < B; i += blockDim.x) sc[i] = coeffs[i];
  __syncthreads();
  for (long long pos = blockIdx.x * (long long)blockDim.x + threadIdx.x; pos < nchunks;
       pos += (long long)gridDim.x * blockDim.x) {
    // pos = piece * 32 + slot in the order of one sequence; piece = (tile * 32 + j) * 4 + q
    const long long piece = pos >> 5;
    const int l = (int)(pos & 31), q = (int)(piece & 3), j = (int)((piece >> 2) & 31), tile = (int)(piece >> 7);
    const int m = (tile / tiles_n) * kTileM + q * 32 + l, n = (tile % tiles_n) * kTileN + j * 8;
    if (m >= d_out || n >= d_in) continue;
    if (!ISOPO_IN_RANGE((long long)stored_slot((size_t)piece, B - 1, B, l), nchunks * B, info, kIdCombine)) continue;
    if (!ISOPO_IN_RANGE((long long)m * d_in + n + 7, (long long)d_out * d_in, info, kIdCombine)) continue;
    float acc[8] = {};
    const uint4* src = G + stored_slot((size_t)piece, 0, B, l);
    const size_t stride = 32;  // slots between successive sequences of one piece
    auto add = [&](const uint4& v, float c) {
      const uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
      for (int h = 0; h < 4; ++h) {
        acc[2 * h] = fmaf(c, __uint_as_float(w[h] << 16), acc[2 * h]);
        acc[2 * h + 1] = fmaf(c, __uint_as_float(w[h] & 0xffff0000u), acc[2 * h + 1]);
      }
    };
    int i = 0;
    for (; i + kCombineInFlight <= B; i += kCombineInFlight) {
      uint4 v[kCombineInFlight];
#pragma unroll
      for (int u = 0; u < kCombineInFlight; ++u) v[u] = __ldcs(src + (size_t)(i + u) * stride);
#pragma unroll
      for (int u = 0; u < kCombineInFlight; ++u) add(v[u], sc[i + u]);
    }
    for (; i < B; ++i) add(__ldcs(src + (size_t)i * stride), sc[i]);
    float4* out = reinterpret_cast<float4*>(dW + (size_t)m * d_in + n);
    float4 o0 = make_float4(acc[0], acc[1], acc[2], acc[3]), o1 = make_float4(acc[4], acc[5], acc[6], acc[7]);
    if (beta != 0.f) {
      const float4 p0 = out[0], p1 = out[1];
      o0.x += p0.x; o0.y += p0.y; o0.z += p0.z; o0.w += p0.w;
      o1.x += p1.x; o1.y += p1.y; o1.z += p1.z; o1.w += p1.w;
    }
    out[0] = o0;
    out[1] = o1;
  }
}

// Split store: dW = beta dW + sum_i (c_i / s_i) (hi_i + lo_i / 16).  One thread per PAIR of slots (two tile rows x 8
// columns), so that every load is 16 bytes per plane: with one slot per thread the two planes cost twice the load
// instructions per byte of the bf16 store and the pass fell to 5.0 TB/s inside the step.
__global__ void __launch_bounds__(256) k_e4m3_combine(const uint2* __restrict__ planes, long long nchunks /* n_pad / 8 */,
                                                       int B, int tiles_n, int d_in, int d_out,
                                                       const float* __restrict__ coeffs, const float* __restrict__ scales,
                                                       float* __restrict__ dW, float beta,
                                                       const WsTag* __restrict__ tag_dev, WsTag tag,
                                                       int32_t* __restrict__ info) {
  if (!ws_tag_matches(tag_dev, tag, info)) return;  // another layer's or microbatch's gradients: touch nothing
  __shared__ float sc[256];
  for (int i = threadIdx.x; i < B; i += blockDim.x) sc[i] = coeffs[i] / scales[i];
  __syncthreads();
  const long long npairs = nchunks / 2;
  for (long long pos = blockIdx.x * (long long)blockDim.x + threadIdx.x; pos < npairs;
       pos += (long long)gridDim.x * blockDim.x) {
    // pos = piece * 16 + pair of slots; piece = (tile * 32 + j) * 4 + q
    const long long piece = pos >> 4;
    const int l = (int)(pos & 15) * 2, q = (int)(piece & 3), j = (int)((piece >> 2) & 31), tile = (int)(piece >> 7);
    const int m = (tile / tiles_n) * kTileM + q * 32 + l, n = (tile % tiles_n) * kTileN + j * 8;
    if (m >= d_out || n >= d_in) continue;
    if (!ISOPO_IN_RANGE((long long)stored_slot((size_t)piece, B - 1, B, l + 1), nchunks * B, info, kIdCombine)) continue;
    if (!ISOPO_IN_RANGE((long long)m * d_in + n + 7, (long long)d_out * d_in, info, kIdCombine)) continue;
    float acc[16] = {};
    const uint4* hi = reinterpret_cast<const uint4*>(planes + stored_slot((size_t)piece, 0, B, l));
    const uint4* lo = reinterpret_cast<const uint4*>(planes + (size_t)nchunks * B + stored_slot((size_t)piece, 0, B, l));
    const size_t stride = 16;  // 16-byte units between successive sequences of one piece
    auto add = [&](const uint4& hv, const uint4& lv, float c) {
      const uint32_t hw[8] = {hv.x & 0xffffu, hv.x >> 16, hv.y & 0xffffu, hv.y >> 16,
                              hv.z & 0xffffu, hv.z >> 16, hv.w & 0xffffu, hv.w >> 16};
      const uint32_t lw[8] = {lv.x & 0xffffu, lv.x >> 16, lv.y & 0xffffu, lv.y >> 16,
                              lv.z & 0xffffu, lv.z >> 16, lv.w & 0xffffu, lv.w >> 16};
#pragma unroll
      for (int h = 0; h < 8; ++h) {
        // hi + lo / 16 in half precision is exact (4 + 4 significant bits, at most 9 binades apart)
        const float2 g = __half22float2(__hfma2(e4m3x2_to_half2(lw[h]), __float2half2_rn(1.f / kLoScale), e4m3x2_to_half2(hw[h])));
        acc[2 * h] = fmaf(c, g.x, acc[2 * h]);
        acc[2 * h + 1] = fmaf(c, g.y, acc[2 * h + 1]);
      }
    };
    constexpr int kN = kCombineInFlight / 2;
    int i = 0;
    for (; i + kN <= B; i += kN) {
      uint4 hv[kN], lv[kN];
#pragma unroll
      for (int u = 0; u < kN; ++u) { hv[u] = __ldcs(hi + (size_t)(i + u) * stride); lv[u] = __ldcs(lo + (size_t)(i + u) * stride); }
#pragma unroll
      for (int u = 0; u < kN; ++u) add(hv[u], lv[u], sc[i + u]);
    }
    for (; i < B; ++i) add(__ldcs(hi + (size_t)i * stride), __ldcs(lo + (size_t)i * stride), sc[i]);
#pragma unroll
    for (int r = 0; r < 2; ++r) {
      if (m + r >= d_out) break;
      float4* out = reinterpret_cast<float4*>(dW + (size_t)(m + r) * d_in + n);
      float4 o0 = make_float4(acc[8 * r], acc[8 * r + 1], acc[8 * r + 2], acc[8 * r + 3]);
      float4 o1 = make_float4(acc[8 * r + 4], acc[8 * r + 5], acc[8 * r + 6], acc[8 * r + 7]);
      if (beta != 0.f) {
        const float4 p0 = out[0], p1 = out[1];
        o0.x += p0.x; o0.y += p0.y; o0.z += p0.z; o0.w += p0.w;
        o1.x += p1.x; o1.y += p1.y; o1.z += p1.z; o1.w += p1.w;
      }
      out[0] = o0;
      out[1] = o1;
    }
  }
}

}  // namespace

isopo_status bf16_ntk(const void* G, const WsLayout& L, int B, float* K, bool k_is_zero, float* kpart, const StoreFmt& fmt,
                      int32_t* info, cudaStream_t st) {
  if (B > 256) return ISOPO_ERR_UNSUPPORTED;
  if (fmt.split && kpart) return ISOPO_ERR_INVALID_ARG;  // the split store's diagonal is summed with float atomics
  CUtensorMap mapG;
  const uint32_t rows = B > 128 ? 256 : B > 64 ? 128 : B > 32 ? 64 : 32, ppb = 256 / rows;
  const long long pieces = L.n_pad / kPieceElems;
  isopo_status s = fmt.split ? make_map_pieces_u8(&mapG, G, (uint64_t)B, (uint64_t)pieces, rows, ppb)
                             : make_map_pieces_bf16(&mapG, G, (uint64_t)B, (uint64_t)pieces, rows, ppb);
  if (s != ISOPO_OK) return s;
  int dev = 0, sms = 0;
  ISOPO_CUDA_TRY(cudaGetDevice(&dev));
  ISOPO_CUDA_TRY(cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev));
  auto kernel = fmt.split ? k_bf16_ntk<true> : k_bf16_ntk<false>;
  ISOPO_CUDA_TRY(cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBytes));
  if (!k_is_zero && !kpart) ISOPO_CUDA_TRY(cudaMemsetAsync(K, 0, sizeof(float) * (size_t)B * B, st));
  // boxes along the contraction: four per piece group of bf16 (64 elements a row), two of e4m3 (128 elements a row)
  NtkParams p{kpart, fmt.split ? fmt.scales : nullptr, K, B, (pieces + ppb - 1) / ppb * (fmt.split ? 2 : 4), info, (int)rows,
              (int)ppb};
  int grid = (int)std::max<long long>(1, std::min<long long>(sms, p.nkb / 8));
  if (kpart) grid = std::min(grid, kNtkMaxPartials);
  {
    LaunchScope scope(kIdNtk, st);
    kernel<<<grid, kThreads, kSmemBytes, st>>>(mapG, p);
  }
  ISOPO_CUDA_TRY(cudaGetLastError());
  if (!kpart) return mirror_upper(K, B, st, fmt.split ? fmt.kdiag : nullptr);
  // CTAs whose slab of the contraction is empty wrote nothing: sum only those that had work
  const long long per = (p.nkb + grid - 1) / grid;
  const int n_active = (int)((p.nkb + per - 1) / per);
  {
    LaunchScope scope(kIdMirror, st);
    k_ntk_reduce<<<(B * B + 255) / 256, 256, 0, st>>>(kpart, n_active, B, K);
  }
  ISOPO_CUDA_TRY(cudaGetLastError());
  return ISOPO_OK;
}

isopo_status mirror_upper(float* K, int B, cudaStream_t st, const float* kdiag) {
  {
    LaunchScope scope(kIdMirror, st);
    k_mirror_upper<<<(B * B + 255) / 256, 256, 0, st>>>(K, B, kdiag);
  }
  ISOPO_CUDA_TRY(cudaGetLastError());
  return ISOPO_OK;
}

isopo_status bf16_combine(const void* G, const WsLayout& L, int d_in, int d_out, int B, const float* coeffs, float* dW,
                          float beta, const WsTag* tag_dev, const WsTag& tag, const StoreFmt& fmt, int32_t* info,
                          cudaStream_t st) {
  if (B > 256) return ISOPO_ERR_UNSUPPORTED;
  const long long chunks = L.n_pad / 8;
  int dev = 0, sms = 0;
  ISOPO_CUDA_TRY(cudaGetDevice(&dev));
  ISOPO_CUDA_TRY(cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev));
  const int grid = (int)std::min<long long>((chunks + 255) / 256, (long long)sms * 8);
  {
    LaunchScope scope(kIdCombine, st);
    if (fmt.split)
      k_e4m3_combine<<<grid, 256, 0, st>>>((const uint2*)G, chunks, B, L.tiles_n, d_in, d_out, coeffs, fmt.scales, dW, beta,
                                           tag_dev, tag, info);
    else
      k_bf16_combine<<<grid, 256, 0, st>>>((const uint4*)G, chunks, B, L.tiles_n, d_in, d_out, coeffs, dW, beta, tag_dev, tag,
                                           info);
  }
  ISOPO_CUDA_TRY(cudaGetLastError());
  return ISOPO_OK;
}

}  // namespace isopo
