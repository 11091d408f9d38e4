// Rank-r projection of one input vector against the rank rows of one expert's packed INT4 factor
// U [E][r][len]:  out[p] = sum_c in[c] U_e[p][c].  A warp per rank row, lanes over the 32-element scale groups
// (codes decoded without integer conversions, lanes summed by shuffles in a fixed order).
#pragma once

#include <cuda_fp16.h>
#include <stdint.h>

#include "cmoe_internal.h"
#include "device_utils.cuh"

namespace cmoe {

// rows pr_first + warp, then + pr_step, ... of expert e; all code lines of the first pass are requested at once
// (into L2), so the loop meets DRAM latency once, not once per unrolled batch
__device__ __forceinline__ void lowrank_rows(const __half* __restrict__ xin, int e, int r, int len, int pr_first, int pr_step,
                                             const uint8_t* __restrict__ Uq, const __half* __restrict__ Us,
                                             float* __restrict__ out_item) {
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, nwarp = blockDim.x >> 5;
  {
    const int lines = len >> 8;                                   // 128-byte lines of one rank row (len / 2 bytes)
    const int nr = min(nwarp, r - pr_first);
    for (int i = threadIdx.x; i < nr * lines; i += blockDim.x) {
      const int rr = i / lines, l = i - rr * lines;
      asm volatile("prefetch.global.L2 [%0];" ::"l"(Uq + ((((long long)e * r + pr_first + rr) * len) >> 1) + (size_t)l * 128));
    }
  }
  for (int pr = pr_first + warp; pr < r; pr += pr_step) {
    const long long base = ((long long)e * r + pr) * len;
    float acc = 0.f;
#pragma unroll 8
    for (int grp = lane; grp * 32 < len; grp += 32) {
      const uint4 pk = __ldg(reinterpret_cast<const uint4*>(Uq + ((base + grp * 32) >> 1)));
      const float sc = __half2float(Us[(base >> 5) + grp]);
      const uint32_t w[4] = {pk.x, pk.y, pk.z, pk.w};
      float part = 0.f;
#pragma unroll
      for (int qd = 0; qd < 4; ++qd) {
        const uint4 xv = *reinterpret_cast<const uint4*>(xin + grp * 32 + qd * 8);
        const __half2* xh = reinterpret_cast<const __half2*>(&xv);
        float cf[8];
        int4x8_to_float(w[qd], cf);
#pragma unroll
        for (int n = 0; n < 4; ++n) {
          const float2 xf = __half22float2(xh[n]);
          part = fmaf(xf.x, cf[2 * n], part);
          part = fmaf(xf.y, cf[2 * n + 1], part);
        }
      }
      acc = fmaf(part, sc, acc);
    }
    acc = warp_sum(acc);
    if (lane == 0) out_item[pr] = acc;
  }
}

// t = x U1 per (token, kept expert), indexed by token: t[(tok * k + j) * r + p], j over the token's local expert
// indices in ascending order (the order of the permuted rows' slot table).  It needs the routes but not the
// permutation, so for small batches its blocks ride in the grid of the one-block permutation kernel.
struct LowrankTok {
  const __half* x;          // [T][len]
  const int* cluster_id;    // [T]
  const int* slot;          // [T][k] local expert indices, routing order
  const uint8_t* Uq;
  const __half* Us;
  float* out;               // [T][k][r]
  const int* live;          // [E] bit 0: the expert's up residual block is not zero (else t is not needed)
  int T, K, k, r, len;      // T == 0: nothing to do
};

constexpr int kLowrankTokThreads = 256;      // eight warps = eight rank rows per block

inline int lowrank_tok_blocks(const LowrankTok& a) { return a.T * a.k * ((a.r + 7) / 8); }

__device__ __forceinline__ void lowrank_tok_block(const LowrankTok& a, int b) {
  const int ny = (a.r + 7) / 8;
  const int item = b / ny, by = b - item * ny;
  const int tok = item / a.k, j = item - tok * a.k;
  int sl[kMaxKsel];
#pragma unroll
  for (int i = 0; i < kMaxKsel; ++i) sl[i] = i < a.k ? a.slot[(size_t)tok * a.k + i] : 0x7fffffff;
#pragma unroll
  for (int p = 1; p < kMaxKsel; ++p)
#pragma unroll
    for (int q = kMaxKsel - 1; q > 0; --q)
      if (q <= p && sl[q] < sl[q - 1]) { const int tmp = sl[q]; sl[q] = sl[q - 1]; sl[q - 1] = tmp; }
  int mine = sl[0];
#pragma unroll
  for (int i = 1; i < kMaxKsel; ++i) if (i == j) mine = sl[i];
  const int e = a.cluster_id[tok] * a.K + mine;
  if (!(a.live[e] & 1)) return;                 // zero residual block: the epilogue does not read this t
  const int nwarp = blockDim.x >> 5;
  lowrank_rows(a.x + (size_t)tok * a.len, e, a.r, a.len, by * nwarp, ny * nwarp, a.Uq, a.Us, a.out + (size_t)item * a.r);
}

}  // namespace cmoe
