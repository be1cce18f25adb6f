// Per-sequence weight gradients G_i = dY_i^T X_i (Alg. 1/2 reduce loop) with 2-CTA tensor-core tiles.
//
// Two CTAs on neighbouring SMs (a cluster of two) share one 256 x 256 tile of G_i: CTA r of the pair
// stages dY[:, 128 columns] (its half of the tile's rows) and X[:, 128 columns] (its half of the
// tile's columns), one thread of CTA 0 issues tcgen05.mma.cta_group::2 (256 x 256 x 16, both operands
// token-major = "MN-major"), and each CTA ends up with its 128 x 256 half of the accumulator in its
// own tensor memory.  A 128 x 256 tile per CTA needs 96 bytes of operands per tensor clock read from
// shared memory and as many written by TMA, more than shared memory can move; the pair tile needs 64.
//
// Work units are (sequence, pair tile), sequence-major with the sequences taken longest first, handed
// round-robin to the persistent pairs: the pairs running at one time read the same sequence's tokens
// out of L2, and every pair gets a regular sample of the sorted lengths, i.e. nearly the same number
// of tokens.
//
//   warp 0          TMA producer; both CTAs' copies complete on the barrier in CTA 0
//   warp 1, CTA 0   MMA issuer (one thread)
//   warps 2-5       epilogue: TMEM -> registers -> bf16 (round to nearest even) -> stored gradients
//   warp 6          zeroes the dY rows past the end of a sequence in its last slab
//
// Several projections that read the same X (q/k/v, gate/up of a transformer block) can share one launch:
// their pair-tile rows are stacked into one tile grid, the dY operand and the destination of a unit
// come from the projection its row belongs to, and X is staged exactly as for one projection, so the
// pairs running at one time share its tokens in L2 across projections as well.
//
// Barriers.  full[s] lives in CTA 0 and counts the bytes of both CTAs; tcgen05.commit releases
// empty[s] and raises accfull[b] in BOTH CTAs; accempty[b] in CTA 0 counts the eight epilogue warps
// of the pair.  In the last slab of a sequence whose length is not a multiple of 16 the dY copy of
// each CTA completes on that CTA's own tail[s] barrier instead; warp 6 waits for it, zeroes the rows
// and arrives on fixed[s] in CTA 0, which the MMA thread waits for in addition to full[s].
// Every wait is bounded; a CTA that gives up raises the abort flag of both CTAs, and both meet at
// a cluster barrier before tensor memory is released.
#include <algorithm>
#include <cstdio>
#include <cstdlib>

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
constexpr int kMaxSeqs = 256;                        // sequences whose extents are staged in shared memory
constexpr int kSeqInfoBytes = kMaxSeqs * 16;         // int64 first token, int32 length, int32 index
constexpr int kSmemBytes = kStages * kStageBytes + 1024 /*alignment slack*/ + 512 /*barriers*/ + kSeqInfoBytes;
constexpr int kThreads = 224;
constexpr uint32_t kTmemCols = 512;                  // two 256-column float32 accumulators
constexpr int kPairN = 256;                          // columns of a pair tile (= columns of a stored tile)
static_assert(kKB % 16 == 0 && kKB <= 256, "a stage is a whole number of 16-token MMA steps and one TMA box");
static_assert(kSmemBytes <= 227 * 1024, "shared memory");

constexpr int kMaxProj = 3;  // projections sharing X in one launch
struct PairParams {
  const int64_t* off;
  const int32_t* order;     // the k-th sequence to work on (longest first)
  __nv_bfloat16* G[kMaxProj];   // stored gradients of every projection
  int tiles_m[kMaxProj];        // stored 128-row tiles of every projection
  int ptm_first[kMaxProj + 1];  // first pair-tile row of every projection in the stacked grid
  int n_proj;
  int B, tiles_n;           // sequences; stored 256-column tiles per gradient (X is common)
  int ptiles_m;             // pair-tile rows of the stacked grid = sum over projections of ceil(tiles_m / 2)
  int32_t* info;
  int group_m;              // pair-tile rows per group of the tile order
  long long n_slots[kMaxProj];  // slots (8 elements each) of each projection's stored gradients
  // split e4m3 store (see StoreFmt; kernel instantiation kSplit): G[h] is then the `hi` plane, the `lo` plane follows it
  const float* scales[kMaxProj];
  float* kdiag[kMaxProj];
};

// projection that pair-tile row `ptm` of the stacked grid belongs to (no indexing by a run-time value anywhere
// below: that would move the parameter arrays to local memory)
__device__ __forceinline__ int proj_of(const PairParams& p, int ptm) {
  return (int)(p.n_proj > 1 && ptm >= p.ptm_first[1]) + (int)(p.n_proj > 2 && ptm >= p.ptm_first[2]);
}
template <typename T>
__device__ __forceinline__ T pick(const T (&a)[kMaxProj], int h) {
  return h == 0 ? a[0] : (h == 1 ? a[1] : a[2]);
}

// The pair tiles of one sequence are visited in groups of `group_m` rows, row index fastest inside a
// group: the ~74 pairs then work on about group_m row blocks of dY and 74 / group_m column blocks of X
// of the same tokens at a time, and what they stream stays in the L2.  Row by row instead, a layer
// with a wide input (74 column blocks) has a whole sequence of X in flight, more than the L2 holds,
// and reads it from HBM once per row of tiles.
__device__ __forceinline__ void pair_tile(int pt, const PairParams& p, int& ptm, int& tn) {
  const int per_group = p.group_m * p.tiles_n;
  const int first = (pt / per_group) * p.group_m, in_group = pt % per_group;
  const int gm = min(p.group_m, p.ptiles_m - first);
  ptm = first + in_group % gm;
  tn = in_group / gm;
}

// Shape of one unit's token loop, identical in every role.
struct UnitShape {
  int nkb;         // slabs
  int tail_n16;    // 16-token MMA steps of the last slab
  int tail_valid;  // token rows of the last slab that belong to the sequence
  bool fix;        // the last step holds rows of the next sequence
};
__device__ __forceinline__ UnitShape unit_shape(int len) {
  UnitShape s;
  s.nkb = (len + kKB - 1) / kKB;
  s.tail_valid = len - (s.nkb - 1) * kKB;
  s.tail_n16 = (s.tail_valid + 15) >> 4;
  s.fix = s.tail_valid < s.tail_n16 * 16;
  return s;
}

template <bool kSplit>
__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(kThreads, 1)
k_bf16_seq_grad_pair(const __grid_constant__ CUtensorMap mapY0, const __grid_constant__ CUtensorMap mapY1,
                     const __grid_constant__ CUtensorMap mapY2, const __grid_constant__ CUtensorMap mapX, PairParams p) {
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
  // extents of the sequences in working order, read once: the roles look them up at every unit,
  // and a global load there would stall the MMA thread for longer than its queue of MMAs lasts
  int64_t* s_first = reinterpret_cast<int64_t*>(smem + kStages * kStageBytes + 512);
  int* s_len = reinterpret_cast<int*>(s_first + kMaxSeqs);
  int* s_seq = s_len + kMaxSeqs;
  for (int k = threadIdx.x; k < p.B; k += kThreads) {
    const int i = p.order[k];
    const int64_t t0 = p.off[i];
    s_first[k] = t0;
    s_len[k] = (int)(p.off[i + 1] - t0);
    s_seq[k] = i;
  }

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
    for (int b = 0; b < 2; ++b) { mbar_init(accfull_bar(b), 1); mbar_init(accempty_bar(b), 8); }
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
  const long long total_units = (long long)p.B * ptiles;
  const long long pair_id = blockIdx.x >> 1, npairs = gridDim.x >> 1;

  if (warp == 0) {
    // ------------------------------------------------------------------ TMA producer (both CTAs)
    if (elect_one()) {
      prefetch_tensormap(&mapY0);
      if (p.n_proj > 1) prefetch_tensormap(&mapY1);
      if (p.n_proj > 2) prefetch_tensormap(&mapY2);
      prefetch_tensormap(&mapX);
      const uint32_t full_at_leader = map_to_cta(full_bar(0), 0);
      int stage = 0;
      uint32_t phase = 0;
      bool ok = true;
      for (long long u = pair_id; u < total_units && ok; u += npairs) {
        const int k = (int)(u / ptiles), pt = (int)(u % ptiles);
        int ptm, tn;
        pair_tile(pt, p, ptm, tn);
        const int64_t t0 = s_first[k];
        const UnitShape us = unit_shape(s_len[k]);
        const int h = proj_of(p, ptm);
        const CUtensorMap* mapY = h == 0 ? &mapY0 : h == 1 ? &mapY1 : &mapY2;
        const int ycol = (2 * (ptm - (h == 0 ? 0 : (h == 1 ? p.ptm_first[1] : p.ptm_first[2]))) + (int)rank) * kHalf, xcol = tn * kPairN + (int)rank * kHalf;
        for (int kb = 0; kb < us.nkb; ++kb) {
          if (!(ok = mbar_wait_pair(empty_bar(stage), phase ^ 1u, abort_flag, peer_abort, p.info, kIdSeqGrad))) break;
          const uint32_t a_dst = smem_base + stage * kStageBytes, b_dst = a_dst + kOperandBytes;
          const int y = (int)(t0 + (int64_t)kb * kKB);
          const bool own_tail = us.fix && kb == us.nkb - 1;  // dY goes to this CTA's tail barrier
          if (own_tail) mbar_arrive_expect_tx(tail_bar(stage), kOperandBytes);
          if (rank == 0) mbar_arrive_expect_tx(full_bar(stage), own_tail ? 2 * kOperandBytes : 2 * kStageBytes);
          const uint32_t fb = full_at_leader + 8u * stage;
#pragma unroll
          for (int c = 0; c < 2; ++c) {
            if (own_tail) tma_load_2d(a_dst + c * kChunkBytes, mapY, ycol + c * 64, y, tail_bar(stage));
            else tma_load_2d_pair(a_dst + c * kChunkBytes, mapY, ycol + c * 64, y, fb);
            tma_load_2d_pair(b_dst + c * kChunkBytes, &mapX, xcol + c * 64, y, fb);
          }
          if (++stage == kStages) { stage = 0; phase ^= 1u; }
        }
      }
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------------ MMA issuer (one thread of CTA 0)
    // elected, not "lane 0": lets the compiler keep the MMA operands in uniform registers
    if (rank == 0 && elect_one()) {
      constexpr uint32_t idesc = make_idesc_bf16(256, kPairN, /*a_mn=*/true, /*b_mn=*/true);
      int stage = 0, acc = 0;
      uint32_t phase = 0, acc_phase = 0, fixed_phase = 0;  // fixed_phase: one bit per stage
      bool ok = true;
      for (long long u = pair_id; u < total_units && ok; u += npairs) {
        const UnitShape us = unit_shape(s_len[u / ptiles]);
        if (!(ok = mbar_wait_pair(accempty_bar(acc), acc_phase ^ 1u, abort_flag, peer_abort, p.info, kIdSeqGrad))) break;
        const uint32_t d_tmem = tmem_base + (uint32_t)acc * kPairN;
        for (int kb = 0; kb < us.nkb; ++kb) {
          const bool last = kb == us.nkb - 1;
          if (!(ok = mbar_wait_pair(full_bar(stage), phase, abort_flag, peer_abort, p.info, kIdSeqGrad))) break;
          if (last && us.fix) {
            // both CTAs' dY halves of this slab have landed and their stray rows are zero
            if (!(ok = mbar_wait_pair(fixed_bar(stage), (fixed_phase >> stage) & 1u, abort_flag, peer_abort, p.info,
                                      kIdSeqGrad)))
              break;
            fixed_phase ^= 1u << stage;
          }
          tc_fence_after_sync();
          const uint32_t a_addr = smem_base + stage * kStageBytes, b_addr = a_addr + kOperandBytes;
          const int n16 = last ? us.tail_n16 : kKB / 16;
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
  } else if (warp < 6) {
    // ------------------------------------------------------------------ epilogue (warps 2..5, both CTAs)
    const int q = warp & 3;  // TMEM lane quarter this warp may read
    const uint32_t accempty_at_leader = map_to_cta(accempty_bar(0), 0);
    int acc = 0;
    uint32_t acc_phase = 0;
    for (long long u = pair_id; u < total_units; u += npairs) {
      const int i = s_seq[u / ptiles], pt = (int)(u % ptiles);
      int ptm, tn;
      pair_tile(pt, p, ptm, tn);
      const int h = proj_of(p, ptm);
      const int tm = 2 * (ptm - (h == 0 ? 0 : (h == 1 ? p.ptm_first[1] : p.ptm_first[2]))) + (int)rank;
      const int tile = tm * p.tiles_n + tn;
      uint4* dst = reinterpret_cast<uint4*>(pick(p.G, h));
      if (!mbar_wait_pair(accfull_bar(acc), acc_phase, abort_flag, peer_abort, p.info, kIdSeqGrad)) break;
      tc_fence_after_sync();
      if (kSplit && tm < pick(p.tiles_m, h)) {
        // split store: hi = e4m3(s_i g), lo = e4m3(16 (s_i g - hi)), 8 bytes per lane and plane; the sum of g^2 goes to kdiag
        const uint32_t taddr = tmem_base + ((uint32_t)(q * 32) << 16) + (uint32_t)acc * kPairN;
        const long long n_slots = pick(p.n_slots, h);
        uint2* hi_plane = reinterpret_cast<uint2*>(pick(p.G, h));
        uint2* lo_plane = hi_plane + n_slots;
        const float s_i = __ldg(pick(p.scales, h) + i);
        float ksum = 0.f, vmax = 0.f;
#pragma unroll 2
        for (int jc = 0; jc < kPairN / 32; ++jc) {
          uint32_t r[32];
          tmem_ld32(taddr + jc * 32, r);
          tmem_ld_wait();
#pragma unroll
          for (int v = 0; v < 4; ++v) {
            uint32_t hw[4], lw[4];
#pragma unroll
            for (int e = 0; e < 4; ++e) {
              const float g0 = __uint_as_float(r[v * 8 + 2 * e]), g1 = __uint_as_float(r[v * 8 + 2 * e + 1]);
              ksum = fmaf(g0, g0, fmaf(g1, g1, ksum));
              const float v0 = g0 * s_i, v1 = g1 * s_i;
              vmax = fmaxf(vmax, fmaxf(fabsf(v0), fabsf(v1)));
              hw[e] = pack_e4m3x2(v0, v1);
              const float2 hf = unpack_e4m3x2(hw[e]);
              lw[e] = pack_e4m3x2((v0 - hf.x) * kLoScale, (v1 - hf.y) * kLoScale);
            }
            const size_t slot = stored_slot(stored_piece(tile, jc * 4 + v, q), i, p.B, lane);
            if (ISOPO_IN_RANGE(i < 0 || i >= p.B ? -1 : (long long)slot, n_slots, p.info, kIdSeqGrad)) {
              hi_plane[slot] = make_uint2(hw[0] | (hw[1] << 16), hw[2] | (hw[3] << 16));
              lo_plane[slot] = make_uint2(lw[0] | (lw[1] << 16), lw[2] | (lw[3] << 16));
            }
          }
        }
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) ksum += __shfl_xor_sync(0xffffffffu, ksum, o);
        if (lane == 0 && ISOPO_IN_RANGE(i, p.B, p.info, kIdSeqGrad)) atomicAdd(pick(p.kdiag, h) + i, ksum);
        // an element beyond e4m3's largest value was clamped: K and dW are off by more than rounding, say so
        if (__any_sync(0xffffffffu, vmax > 448.f) && lane == 0) atomicCAS(p.info, 0, ISOPO_INFO_SATURATED | kIdSeqGrad);
      } else if (!kSplit && tm < pick(p.tiles_m, h)) {  // an odd number of row tiles leaves the last pair's second half empty
        const uint32_t taddr = tmem_base + ((uint32_t)(q * 32) << 16) + (uint32_t)acc * kPairN;
#pragma unroll 2
        for (int jc = 0; jc < kPairN / 32; ++jc) {
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
            if (ISOPO_IN_RANGE(i < 0 || i >= p.B ? -1 : (long long)slot, pick(p.n_slots, h), p.info, kIdSeqGrad)) dst[slot] = o;
          }
        }
      }
      tc_fence_before_sync();
      __syncwarp();
      if (lane == 0) mbar_arrive_remote(accempty_at_leader + 8u * acc);
      if (++acc == 2) { acc = 0; acc_phase ^= 1u; }
    }
  } else {
    // ------------------------------------------------------------------ tail warp (warp 6, both CTAs)
    // tail[s] is used only for last slabs that need the fix, so its phase is counted per stage; it
    // cannot run ahead: the stage is not reloaded before the MMA thread has passed fixed[s].
    const uint32_t fixed_at_leader = map_to_cta(fixed_bar(0), 0);
    int stage = 0;
    uint32_t tail_phase = 0;  // one bit per stage
    for (long long u = pair_id; u < total_units; u += npairs) {
      const UnitShape us = unit_shape(s_len[u / ptiles]);
      const int ts = (stage + us.nkb - 1) % kStages;  // ring position of the last slab
      if (us.fix) {
        if (!mbar_wait_pair(tail_bar(ts), (tail_phase >> ts) & 1u, abort_flag, peer_abort, p.info, kIdSeqGrad)) break;
        tail_phase ^= 1u << ts;
        // rows [tail_valid, tail_n16*16) hold the next sequence's tokens
        const int nbytes = (us.tail_n16 * 16 - us.tail_valid) * 128;
        const uint32_t a_addr = smem_base + ts * kStageBytes;
#pragma unroll
        for (int c = 0; c < 2; ++c) {
          const uint32_t base = a_addr + c * kChunkBytes + us.tail_valid * 128;
          for (int o = lane * 16; o < nbytes; o += 32 * 16)
            asm volatile("st.shared.v4.b32 [%0], {%1, %1, %1, %1};" ::"r"(base + o), "r"(0u) : "memory");
        }
        fence_proxy_async_smem();
        __syncwarp();
        // The stores above were performed in this CTA's shared memory before the proxy fence
        // returned, and only this CTA's tensor core reads them; the arrival merely tells the MMA
        // thread so.  A cluster-scope release here costs the MMA thread ~1500 clocks per unit.
        if (lane == 0) mbar_arrive_remote(fixed_at_leader + 8u * ts);
      }
      stage = (ts + 1) % kStages;
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

// Split store: a power-of-two scale per sequence that brings the typical element of G_i to about 2, where e4m3 has
// its 3 mantissa bits with 2^8 of headroom and 2^7 below (sum_t dY_t x_t^T over L independent tokens has
// elements of size sqrt(L) rms(dY) rms(x); fully correlated tokens give sqrt(L) times more, still in range).
// The rms values come from up to 16 evenly spaced token rows of the sequence (16-byte loads: d_in and d_out are
// multiples of 8).  Also clears kdiag.
__device__ __forceinline__ float sum_sq8(const uint4& v) {
  const uint32_t w[4] = {v.x, v.y, v.z, v.w};
  float s = 0.f;
#pragma unroll
  for (int h = 0; h < 4; ++h) {
    const float a = __uint_as_float(w[h] << 16), b = __uint_as_float(w[h] & 0xffff0000u);
    s = fmaf(a, a, fmaf(b, b, s));
  }
  return s;
}
__global__ void __launch_bounds__(512) k_seq_scales(const uint4* __restrict__ X, const uint4* __restrict__ dY, int d_in8,
                                                    int d_out8, const int64_t* __restrict__ off,
                                                    float* __restrict__ scales, float* __restrict__ kdiag) {
  const int i = blockIdx.x;
  const int64_t t0 = off[i], len = off[i + 1] - t0;
  const int n = (int)min((int64_t)16, len);
  float sx = 0.f, sy = 0.f;
  for (int e = threadIdx.x; e < n * d_in8; e += blockDim.x) {
    const int k = e / d_in8, c = e - k * d_in8;
    sx += sum_sq8(__ldg(X + (t0 + (len * k) / n) * d_in8 + c));
  }
  for (int e = threadIdx.x; e < n * d_out8; e += blockDim.x) {
    const int k = e / d_out8, c = e - k * d_out8;
    sy += sum_sq8(__ldg(dY + (t0 + (len * k) / n) * d_out8 + c));
  }
  __shared__ float red[2][16];
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) { sx += __shfl_xor_sync(0xffffffffu, sx, o); sy += __shfl_xor_sync(0xffffffffu, sy, o); }
  if ((threadIdx.x & 31) == 0) { red[0][threadIdx.x >> 5] = sx; red[1][threadIdx.x >> 5] = sy; }
  __syncthreads();
  if (threadIdx.x == 0) {
    sx = sy = 0.f;
    for (int w = 0; w < 16; ++w) { sx += red[0][w]; sy += red[1][w]; }
    const float typical = sqrtf((float)len * (sx / ((float)n * 8.f * d_in8)) * (sy / ((float)n * 8.f * d_out8)));
    // 2^k nearest to 2 / typical; inputs that are all zero (or not finite) keep the scale one
    float s = 1.f;
    if (typical > 0.f && typical < 3.0e38f) s = exp2f(rintf(log2f(2.f / typical)));
    scales[i] = fminf(fmaxf(s, 1.0e-30f), 1.0e30f);
    kdiag[i] = 0.f;
  }
}

}  // namespace

isopo_status launch_seq_scales(const void* X, const void* dY, int d_in, int d_out, const int64_t* off_dev, int B, float* scales,
                               float* kdiag, cudaStream_t st) {
  {
    LaunchScope scope(kIdPrep, st);
    k_seq_scales<<<B, 512, 0, st>>>((const uint4*)X, (const uint4*)dY, d_in / 8, d_out / 8, off_dev, scales, kdiag);
  }
  ISOPO_CUDA_TRY(cudaGetLastError());
  return ISOPO_OK;
}

isopo_status bf16_seq_grad_pair(const void* X, const void* dY, int64_t T, int d_in, int d_out, const int64_t* off_dev,
                                const int32_t* order_dev, int B, const WsLayout& L, void* G, const StoreFmt& fmt,
                                int32_t* info, cudaStream_t st) {
  const void* dYs[1] = {dY};
  const int d_outs[1] = {d_out};
  void* Gs[1] = {G};
  return bf16_seq_grad_pair_shared(X, 1, dYs, d_outs, T, d_in, off_dev, order_dev, B, &L, Gs, &fmt, info, st);
}

isopo_status bf16_seq_grad_pair_shared(const void* X, int n_proj, const void* const* dY, const int* d_out, int64_t T, int d_in,
                                       const int64_t* off_dev, const int32_t* order_dev, int B, const WsLayout* L,
                                       void* const* G, const StoreFmt* fmt, int32_t* info, cudaStream_t st) {
  if (n_proj < 1 || n_proj > kMaxProj) return ISOPO_ERR_INVALID_ARG;
  for (int h = 1; h < n_proj; ++h)
    if (fmt[h].split != fmt[0].split) return ISOPO_ERR_INVALID_ARG;  // one store format per launch
  CUtensorMap mapY[kMaxProj], mapX;
  PairParams p{};
  p.off = off_dev; p.order = order_dev; p.B = B; p.tiles_n = L[0].tiles_n; p.n_proj = n_proj; p.info = info;
  for (int h = 0; h < kMaxProj; ++h) {
    const int hh = h < n_proj ? h : 0;  // unused slots repeat the first projection (never addressed)
    isopo_status s = make_map_2d_bf16(&mapY[h], dY[hh], (uint64_t)T, (uint64_t)d_out[hh], (uint64_t)d_out[hh], 64, kKB);
    if (s != ISOPO_OK) return s;
    p.G[h] = (__nv_bfloat16*)G[hh];
    p.tiles_m[h] = L[hh].tiles_m;
    p.n_slots[h] = (long long)B * L[hh].n_pad / 8;
    p.scales[h] = fmt[hh].scales;
    p.kdiag[h] = fmt[hh].kdiag;
    p.ptm_first[h] = h == 0 ? 0 : p.ptm_first[h - 1] + (h - 1 < n_proj ? (L[h - 1].tiles_m + 1) / 2 : 0);
  }
  p.ptm_first[kMaxProj] = p.ptm_first[kMaxProj - 1] + (kMaxProj - 1 < n_proj ? (L[kMaxProj - 1].tiles_m + 1) / 2 : 0);
  p.ptiles_m = p.ptm_first[n_proj];
  isopo_status s = make_map_2d_bf16(&mapX, X, (uint64_t)T, (uint64_t)d_in, (uint64_t)d_in, 64, kKB);
  if (s != ISOPO_OK) return s;
  int dev = 0, sms = 0;
  ISOPO_CUDA_TRY(cudaGetDevice(&dev));
  ISOPO_CUDA_TRY(cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev));
  auto kernel = fmt[0].split ? k_bf16_seq_grad_pair<true> : k_bf16_seq_grad_pair<false>;
  ISOPO_CUDA_TRY(cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBytes));
  const long long units = (long long)B * p.ptiles_m * p.tiles_n;
  // Persistent pairs with a static share of the units each: launch only as many pairs as can be
  // resident at once (the hardware may place fewer 2-CTA clusters than there are SM pairs).
  static int resident[2][64] = {};
  if (dev < 0 || dev >= 64) return ISOPO_ERR_UNSUPPORTED;
  int* resident_pairs = resident[fmt[0].split ? 1 : 0];
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
    ISOPO_CUDA_TRY(cudaOccupancyMaxActiveClusters(&n, kernel, &cfg));
    if (n < 1) return ISOPO_ERR_UNSUPPORTED;
    resident_pairs[dev] = std::min(n, sms / 2);
  }
  const int npairs = (int)std::max<long long>(1, std::min<long long>(units, resident_pairs[dev]));
  int g = 1;
  while ((g + 1) * (g + 1) <= npairs) ++g;  // about sqrt(npairs) rows by sqrt(npairs) columns of tiles in flight
  p.group_m = std::max(1, std::min(g, p.ptiles_m));
  {
    LaunchScope scope(kIdSeqGrad, st);
    kernel<<<2 * npairs, kThreads, kSmemBytes, st>>>(mapY[0], mapY[1], mapY[2], mapX, p);
  }
  ISOPO_CUDA_TRY(cudaGetLastError());
  return ISOPO_OK;
}

}  // namespace isopo
