// Epilogue shared by the Gram-route kernels (tc_gram.cu, tc_gram_shared.cu): the elementwise product of
// the two accumulators P and Q, summed per (sequence of the row token, sequence of the column token).
//
// Every lane owns one accumulator row and walks the columns 32 at a time.  Column tokens are in
// packed order, so their sequence ids never decrease: the places where a new sequence starts are
// found with one ballot per 32 columns (warp-uniform, so branching on them costs no divergence),
// and the running sum of a lane is flushed only there.  A flush adds the lanes of one row sequence
// together first (rows are in packed order too: a segmented shuffle reduction, five steps) and
// issues one float atomic per row sequence present in the warp.
#pragma once

#include <stdint.h>

namespace isopo {
namespace tc {

// Order of the tile pairs (I <= J) of the token-Gram triangle.  The tiles running at one time must
// fit in L2 or every operand byte comes from HBM: the triangle is cut into strips of `S` tile
// columns; inside a strip the pairs go row by row (I outer, J inner), so about n concurrent units
// touch S column tiles and n / S row tiles.  Unit u -> (I, J).
__device__ __forceinline__ void decode_pair_strips(long long u, int nT, int S, int& I, int& J) {
  int J0 = 0;
  while (true) {
    const int w = min(S, nT - J0);
    const long long cnt = (long long)J0 * w + (long long)w * (w + 1) / 2;
    if (u < cnt || J0 + w >= nT) {
      const long long rect = (long long)J0 * w;
      if (u < rect) {
        I = (int)(u / w);
        J = J0 + (int)(u % w);
      } else {
        long long r = u - rect;
        int k = 0;
        while (k < w - 1 && r >= w - k) { r -= w - k; ++k; }  // row J0 + k holds w - k pairs
        I = J0 + k;
        J = I + (int)r;
      }
      return;
    }
    u -= cnt;
    J0 += w;
  }
}

// Strip width for tiles of `tile_bytes` (both operands' rows of one tile): column and row tiles of
// ~148 concurrent units should stay within about 48 MB.
inline int gram_strip_width(double tile_bytes, int concurrent_units) {
  int best = 0, fewest = 2;
  double fewest_tiles = 1e300;
  for (int S = 2; S <= 32; ++S) {
    const double tiles = S + (double)concurrent_units / S;
    if (tiles * tile_bytes <= 48e6) best = S;  // widest strip that still fits (fewer, longer strips)
    if (tiles < fewest_tiles) { fewest_tiles = tiles; fewest = S; }
  }
  return best ? best : fewest;  // nothing fits: the strip with the fewest tiles in flight
}

struct RowSegments {
  int seq;        // sequence of this lane's row token (sampled estimator: the sample index, all distinct)
  bool head;      // first lane of its run of equal `seq`
  unsigned same;  // bit k: lane + 2^k exists and has the same `seq`
  bool valid;     // the row exists (rows past the end of the row range never write, whatever their sums hold)
  long long n_out;  // elements of the output matrix (debug build: every flush is checked against it)
  int32_t* info;
};

__device__ __forceinline__ RowSegments row_segments(int seq, long long n_out, int32_t* info, bool valid = true) {
  RowSegments r;
  r.seq = seq;
  r.valid = valid;
  r.n_out = n_out;
  r.info = info;
  const int lane = threadIdx.x & 31;
  const int up = __shfl_up_sync(0xffffffffu, seq, 1);
  r.head = lane == 0 || up != seq;
  r.same = 0;
#pragma unroll
  for (int k = 0; k < 5; ++k) {
    const int other = __shfl_down_sync(0xffffffffu, seq, 1 << k);
    if (lane + (1 << k) < 32 && other == seq) r.same |= 1u << k;
  }
  return r;
}

// K[rows.seq][col_seq] += sum of v over the lanes of each run of equal rows.seq
__device__ __forceinline__ void flush_rows(float* __restrict__ K, int B, const RowSegments& rows, int col_seq, float v) {
#pragma unroll
  for (int k = 0; k < 5; ++k) {
    const float t = __shfl_down_sync(0xffffffffu, v, 1 << k);
    if ((rows.same >> k) & 1u) v += t;
  }
  if (rows.head && rows.valid && v != 0.f &&
      ISOPO_IN_RANGE(col_seq < 0 || col_seq >= B ? -1 : (long long)rows.seq * B + col_seq, rows.n_out, rows.info, kIdGram))
    atomicAdd(&K[(size_t)rows.seq * B + col_seq], v);
}

// One group of 32 columns.  pv/qv: this lane's 32 values of P and Q; cs: sequence of column c0 + lane;
// cur / wseg / run: the running segment (its sequence, this lane's weight for it, this lane's sum).
// kWeighted: the Gram route's symmetry weights (a pair inside one sequence stands for (t,s) and
// (s,t), weight two); on a diagonal tile only columns c >= row are used, c == row once.
// The segment boundaries of the group come from one ballot; the loop below runs once per segment
// (not per column), so the code stays small: this runs once per unit and a fully unrolled
// per-column version (hundreds of KB of instructions) was bound by instruction fetch.
template <bool kWeighted>
__device__ __forceinline__ void gram_group(const uint32_t (&pv)[32], const uint32_t (&qv)[32], int cs, int c0, int row,
                                           bool diag, const RowSegments& rows, float* __restrict__ K, int B, int& cur,
                                           float& wseg, float& run) {
  const int lane = threadIdx.x & 31;
  const int prev = __shfl_up_sync(0xffffffffu, cs, 1);
  unsigned starts = __ballot_sync(0xffffffffu, cs != (lane == 0 ? cur : prev));  // bit e: a new sequence starts at column e
  float h[32];
#pragma unroll
  for (int e = 0; e < 32; ++e) h[e] = __uint_as_float(pv[e]) * __uint_as_float(qv[e]);
  if (kWeighted && diag) {
    // column c == row is the pair (t, t): once, against the weight two of its own sequence
    const int d = row - c0;  // columns e < d are below the diagonal
#pragma unroll
    for (int e = 0; e < 32; ++e) h[e] = e > d ? h[e] : (e == d ? 0.5f * h[e] : 0.f);
  }
  if (starts == 0u) {
    float s = 0.f;
#pragma unroll
    for (int e = 0; e < 32; ++e) s += h[e];
    run = fmaf(wseg, s, run);
    return;
  }
  int lo = 0;
  while (true) {
    const int hi = starts ? __ffs(starts) - 1 : 32;  // columns lo .. hi - 1 continue the running segment
    const unsigned in = (hi < 32 ? (1u << hi) - 1u : 0xffffffffu) & ~((1u << lo) - 1u);
    float s = 0.f;
#pragma unroll
    for (int e = 0; e < 32; ++e) s += ((in >> e) & 1u) ? h[e] : 0.f;
    run = fmaf(wseg, s, run);
    if (hi == 32) break;
    flush_rows(K, B, rows, cur, run);
    run = 0.f;
    cur = __shfl_sync(0xffffffffu, cs, hi);
    wseg = (kWeighted && rows.seq == cur) ? 2.f : 1.f;
    starts &= starts - 1u;
    lo = hi;
  }
}

}  // namespace tc
}  // namespace isopo
