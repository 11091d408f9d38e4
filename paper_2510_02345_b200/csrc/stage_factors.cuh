// INT4 factors of the layer -> fp16 operand matrices of the tensor-core residual products (one thread per scale
// group: 32 codes = 16 bytes of packed codes and one fp16 scale):
//   U1f [G][64][d]   V1f [G][d_ff][64]   U2f [G][64][d_ff]   V2f [G][d][64]
// with the expanded rank index c = i*r + p (i = expert of the cluster, p = rank) 64 wide.  The work depends on
// the weights only, so it has no kernel of its own: its blocks ride in the grid of another kernel of the forward.
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
  long long words[4];      // scale groups (32 codes) of each packed factor (all zero: nothing to stage)
  int dim[4];              // non-rank extent: d, d_ff, d_ff, d
  int K, r;
};

// blocks of `threads` threads that the staging needs: one scale group per thread
inline int stage_blocks(const FactorStage& fs, int threads) {
  long long n = 0;
  for (int i = 0; i < 4; ++i) n += (fs.words[i] + threads - 1) / threads;
  return (int)n;
}

// scale group `grp` of factor `which`: codes flat0 = 32 grp .. + 31
__device__ __forceinline__ void stage_word(const FactorStage& fs, int which, long long grp) {
  const int dim = fs.dim[which], K = fs.K, r = fs.r;
  const uint4 pk = __ldg(reinterpret_cast<const uint4*>(fs.q[which]) + grp);
  const float sc = __half2float(fs.s[which][grp]);
  const uint32_t w[4] = {pk.x, pk.y, pk.z, pk.w};
  __align__(16) __half v[32];
#pragma unroll
  for (int qd = 0; qd < 4; ++qd)
#pragma unroll
    for (int n = 0; n < 8; ++n) v[qd * 8 + n] = __float2half_rn((float)sext4((int)(w[qd] >> (4 * n))) * sc);
  const uint4* vv = reinterpret_cast<const uint4*>(v);
  const long long flat0 = grp * 32;
  __half* dst = fs.dst[which];
  if ((which & 1) == 0) {
    // U [E][r][dim]: row (e, p) of length dim (a multiple of 32) -> row g*64 + i*r + p; 64 contiguous bytes
    const long long row = flat0 / dim;
    const int c = (int)(flat0 - row * dim);
    const long long g = row / (K * r);
    const int n = (int)(row - g * (K * r));
    uint4* o = reinterpret_cast<uint4*>(dst + ((g * kStageKE + n) * dim + c));
#pragma unroll
    for (int i = 0; i < 4; ++i) o[i] = vv[i];
  } else {
    // V [E][dim][r]: the group holds 32 / r consecutive output columns n of one expert (dim is a multiple of 32),
    // r ranks each -> [g][n][i*r ..]
    const int per = 32 / r;                          // 1 (r = 32), 2, 4, 8
    const long long en0 = flat0 / r;
    const long long e = en0 / dim;
    const int n0 = (int)(en0 - e * dim);
    const long long g = e / K;
    const int i = (int)(e - g * K);
#pragma unroll
    for (int h = 0; h < 8; ++h) {
      if (h >= per) break;
      __half* o = dst + ((g * dim + n0 + h) * kStageKE + i * r);
      if (r == 32)      { uint4* o4 = reinterpret_cast<uint4*>(o); o4[0] = vv[0]; o4[1] = vv[1]; o4[2] = vv[2]; o4[3] = vv[3]; }
      else if (r == 16) { if (h < 2) { uint4* o4 = reinterpret_cast<uint4*>(o); o4[0] = vv[2 * h]; o4[1] = vv[2 * h + 1]; } }
      else if (r == 8)  { if (h < 4) *reinterpret_cast<uint4*>(o) = vv[h]; }
      else              { *reinterpret_cast<uint2*>(o) = reinterpret_cast<const uint2*>(v)[h]; }
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
