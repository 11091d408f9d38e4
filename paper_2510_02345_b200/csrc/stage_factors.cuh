// INT4 factors of the layer -> fp16 operand matrices of the tensor-core residual products (one thread per
// 32-bit word = 8 codes):
//   U1f [G][64][d]   V1f [G][d_ff][64]   U2f [G][64][d_ff]   V2f [G][d][64]
// with the expanded rank index c = i*r + p (i = expert of the cluster, p = rank) 64 wide.  The work depends on
// the weights only, so it has no kernel of its own: its blocks ride in the grid of the permutation's one-block
// scan kernel, whose time they hide in.
#pragma once

#include <cuda_fp16.h>
#include <stdint.h>

#include "device_utils.cuh"

namespace cmoe {

constexpr int kStageKE = 64;       // width of the expanded rank index

struct FactorStage {
  const uint8_t* q[4];     // U1, V1, U2, V2
  const __half* s[4];
  __half* dst[4];
  long long words[4];      // 32-bit words of each packed factor (all zero: nothing to stage)
  int dim[4];              // non-rank extent: d, d_ff, d_ff, d
  int K, r;
};

// blocks of `threads` threads that the staging needs: one word per thread
inline int stage_blocks(const FactorStage& fs, int threads) {
  long long n = 0;
  for (int i = 0; i < 4; ++i) n += (fs.words[i] + threads - 1) / threads;
  return (int)n;
}

__device__ __forceinline__ void stage_word(const FactorStage& fs, int which, long long wd) {
  const int dim = fs.dim[which], K = fs.K, r = fs.r;
  const uint32_t word = reinterpret_cast<const uint32_t*>(fs.q[which])[wd];
  const long long flat0 = wd * 8;
  const float sc = __half2float(fs.s[which][flat0 >> 5]);
  __align__(16) __half v[8];
#pragma unroll
  for (int n = 0; n < 8; ++n) v[n] = __float2half_rn((float)sext4((int)(word >> (4 * n))) * sc);
  __half* dst = fs.dst[which];
  if ((which & 1) == 0) {
    // U [E][r][dim]: row (e, p) of length dim -> row g*64 + i*r + p
    const long long row = flat0 / dim;
    const int c = (int)(flat0 - row * dim);
    const long long g = row / (K * r);
    const int n = (int)(row - g * (K * r));
    *reinterpret_cast<uint4*>(dst + ((g * kStageKE + n) * dim + c)) = *reinterpret_cast<const uint4*>(v);
  } else if (r >= 8) {
    // V [E][dim][r]: (e, n, p0..p0+7) -> [g][n][i*r + p0 ..]
    const long long en = flat0 / r;
    const int p0 = (int)(flat0 - en * r);
    const long long e = en / dim;
    const int n = (int)(en - e * dim);
    const long long g = e / K;
    const int i = (int)(e - g * K);
    *reinterpret_cast<uint4*>(dst + ((g * dim + n) * kStageKE + i * r + p0)) = *reinterpret_cast<const uint4*>(v);
  } else {
    // r == 4: the word holds two output columns of four ranks each
#pragma unroll
    for (int h = 0; h < 2; ++h) {
      const long long en = (flat0 + 4 * h) / 4;
      const long long e = en / dim;
      const int n = (int)(en - e * dim);
      const long long g = e / K;
      const int i = (int)(e - g * K);
      *reinterpret_cast<uint2*>(dst + ((g * dim + n) * kStageKE + i * 4)) = reinterpret_cast<const uint2*>(v)[h];
    }
  }
}

// block `b` (0 <= b < stage_blocks(fs, blockDim.x)) of the staging work
__device__ __forceinline__ void stage_block(const FactorStage& fs, int b) {
  const int threads = (int)blockDim.x;
#pragma unroll
  for (int which = 0; which < 4; ++which) {
    const int nb = (int)((fs.words[which] + threads - 1) / threads);
    if (b < nb) {
      const long long wd = (long long)b * threads + threadIdx.x;
      if (wd < fs.words[which]) stage_word(fs, which, wd);
      return;
    }
    b -= nb;
  }
}

}  // namespace cmoe
