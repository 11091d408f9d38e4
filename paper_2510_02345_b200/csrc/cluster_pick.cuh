// Two clusters per token (Sec. 3.3, "Top-g1 groups" with g1 = 2): the routers see every token twice (its row is
// repeated in x), virtual token 2 t + c goes to the token's c-th most probable cluster, and the gates of that
// cluster's kept experts are scaled by the cluster's weight, Eq. 9's p_g renormalised over the two kept clusters.
#pragma once

#include "cmoe_internal.h"

namespace cmoe {

// Running best and second-best cluster logit; clusters are added in ascending index and ties keep the lower index.
struct TwoBest {
  float z1, z2;
  int c1, c2;
};
__device__ __forceinline__ void two_best_init(TwoBest& b) { b.z1 = 0.f; b.z2 = 0.f; b.c1 = -1; b.c2 = -1; }
__device__ __forceinline__ void two_best_add(TwoBest& b, int g, float z) {
  if (b.c1 < 0 || z > b.z1) { b.z2 = b.z1; b.c2 = b.c1; b.z1 = z; b.c1 = g; }
  else if (b.c2 < 0 || z > b.z2) { b.z2 = z; b.c2 = g; }
}
// the cluster of virtual token `rank` (0: most probable, 1: second) and that cluster's weight
__device__ __forceinline__ void two_best_pick(const TwoBest& b, int rank, int& g, float& w) {
  const float e2 = expf(b.z2 - b.z1);            // p_second / p_first <= 1
  if (rank == 0) { g = b.c1; w = 1.f / (1.f + e2); }
  else           { g = b.c2; w = e2 / (1.f + e2); }
}

// Expert parts (Dims::split = 2 or 4): virtual token `part` (0 .. parts-1) of a token keeps those of the token's k
// experts that lie in that part of the cluster's K experts (part c = experts c K / parts ..), renumbered inside the
// part, and fills its remaining slots with other experts of the part (lowest index first) at gate zero.  sel / gate:
// in the token's k kept experts (local index 0 .. K-1, gates summing to one), out this virtual token's k slots (local
// index 0 .. K/parts-1).  Returns the number of kept experts in the part (0: the virtual token contributes nothing).
__device__ __forceinline__ int split_part(int K, int parts, int k, int part, int* sel, float* gate) {
  const int Kp = K / parts;
  int si[kMaxKsel];
  float gv[kMaxKsel];
  unsigned used = 0;
  int n = 0;
  for (int s = 0; s < k; ++s)
    if (sel[s] / Kp == part) { si[n] = sel[s] - part * Kp; gv[n] = gate[s]; used |= 1u << si[n]; ++n; }
  const int kept = n;
  for (int i = 0; n < k && i < Kp; ++i)
    if (!((used >> i) & 1u)) { si[n] = i; gv[n] = 0.f; ++n; }
  for (int s = 0; s < k; ++s) { sel[s] = si[s]; gate[s] = gv[s]; }
  return kept;          // how many of the token's experts lie in this part
}

}  // namespace cmoe
