// The permutation key of a token: cluster * nsub + (rank of its set of kept experts among the k-subsets of the
// cluster's K experts, or its lowest kept expert when there are too many subsets).  Shared by the tensor-core router
// kernel, which counts the keys of its token tile, and the permutation kernels.  Also: what a router kernel is handed
// when it runs as the first kernel of a forward (key counts, and the factor-staging work that rides in its grid).
#pragma once

#include "cmoe_internal.h"
#include "stage_factors.cuh"

namespace cmoe {

__device__ __forceinline__ int binom(int n, int m) {
  if (m > n) return 0;
  long long r = 1;
  for (int i = 1; i <= m; ++i) r = r * (n - m + i) / i;
  return (int)r;
}

// Sort the token's k local expert indices ascending (gates follow) and return the sub-key.
__device__ __forceinline__ int canonical_slots(const int* __restrict__ slot, const float* __restrict__ gate,
                                               int k, int sub_is_combo, int* cs, float* cg) {
#pragma unroll
  for (int j = 0; j < kMaxKsel; ++j)
    if (j < k) { cs[j] = slot[j]; cg[j] = gate[j]; }
#pragma unroll
  for (int a = 1; a < kMaxKsel; ++a)
    if (a < k) {
#pragma unroll
      for (int b = kMaxKsel - 1; b > 0; --b)
        if (b <= a && cs[b] < cs[b - 1]) {
          int ti = cs[b]; cs[b] = cs[b - 1]; cs[b - 1] = ti;
          float tg = cg[b]; cg[b] = cg[b - 1]; cg[b - 1] = tg;
        }
    }
  if (!sub_is_combo) return cs[0];
  int rank = 0;                    // combinatorial number system: sum_i C(c_i, i+1)
#pragma unroll
  for (int j = 0; j < kMaxKsel; ++j)
    if (j < k) rank += binom(cs[j], j + 1);
  return rank;
}

// Per-tile key counting inside a router kernel (null keys: routing only, as for cmoe_route)
struct KeyCount {
  int* keys;           // [T] key of every token
  int* block_counts;   // [tiles][nkey] tokens of every key in the router's tile of tile_tokens tokens
  int nsub, nkey, sub_is_combo;
};

}  // namespace cmoe
