// Virtual tokens.  Two clusters per token (Sec. 3.3, "Top-g1 groups"): the layer runs on g1 virtual tokens per token.  Before the
// router every row of x is written g1 times (virtual token g1 t + c is token t on its way to its c-th most
// probable cluster); after the un-permuting store the g1 output rows of a token are summed.  The gates already
// carry the clusters' weights, so the sum is the mixture.  Expert parts (Dims::split = 2 or 4) use the same two kernels:
// a token's virtual tokens carry the experts of one half, or one quarter, of its cluster each.
#include "cmoe_internal.h"
#include "cluster_pick.cuh"
#include "perm_keys.cuh"

namespace cmoe {

namespace {

__global__ void __launch_bounds__(256)
repeat_rows_kernel(const uint4* __restrict__ x, uint4* __restrict__ x_rep, long long vec_per_row, long long T, int g1) {
  const long long n = T * vec_per_row;
  for (long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x; i < n; i += (long long)gridDim.x * blockDim.x) {
    const long long t = i / vec_per_row, v = i - t * vec_per_row;
    const uint4 val = x[i];
    for (int c = 0; c < g1; ++c) x_rep[(t * g1 + c) * vec_per_row + v] = val;
  }
}

// y[t] = sum of the token's n output rows (fp32 sums, one rounding), eight columns per thread
__global__ void __launch_bounds__(256)
sum_rows_kernel(const uint4* __restrict__ y_rep, uint4* __restrict__ y, long long vec_per_row, long long T, int g1,
                const int* __restrict__ cluster_id) {
  const long long n = T * vec_per_row;
  for (long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x; i < n; i += (long long)gridDim.x * blockDim.x) {
    const long long t = i / vec_per_row, v = i - t * vec_per_row;
    float acc[8] = {0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f};
    for (int c = 0; c < g1; ++c) {
      if (cluster_id && cluster_id[t * g1 + c] < 0) continue;        // a virtual token that was dropped: no row
      const uint4 q = y_rep[(t * g1 + c) * vec_per_row + v];
      const __half2* h = reinterpret_cast<const __half2*>(&q);
#pragma unroll
      for (int u = 0; u < 4; ++u) {
        const float2 f = __half22float2(h[u]);
        acc[2 * u] += f.x;
        acc[2 * u + 1] += f.y;
      }
    }
    uint4 o;
    __half2* oh = reinterpret_cast<__half2*>(&o);
#pragma unroll
    for (int u = 0; u < 4; ++u) oh[u] = __floats2half2_rn(acc[2 * u], acc[2 * u + 1]);
    y[i] = o;
  }
}

// Expert parts: the token's own routes (real cluster g, k experts among its K, gates) -> the routes of its `parts`
// virtual tokens, a thread per virtual token.  A part without any of the token's experts gets cluster id -1: the
// permutation gives it no row.  With kc.keys the kernel also writes every virtual token's permutation key and counts
// the keys of its block's kSplitTile virtual tokens, so that the permutation starts from a finished histogram.
constexpr int kSplitTile = 256;

__global__ void __launch_bounds__(kSplitTile)
split_routes_kernel(int T, int K, int parts, int k, const int* __restrict__ r_cluster, const int* __restrict__ r_slot,
                    const float* __restrict__ r_gates, int* __restrict__ cluster_id, int* __restrict__ slot,
                    float* __restrict__ gates, const KeyCount kc) {
  __shared__ int cnt[kMaxKeys];
  if (kc.keys) {
    for (int i = threadIdx.x; i < kc.nkey; i += blockDim.x) cnt[i] = 0;
    __syncthreads();
  }
  const long long vt = (long long)blockIdx.x * kSplitTile + threadIdx.x;
  const int t = (int)(vt / parts), part = (int)(vt - (long long)t * parts);
  if (t < T) {
    const int g = r_cluster[t];
    int sel[kMaxKsel];
    float gv[kMaxKsel];
    for (int s = 0; s < k; ++s) { sel[s] = r_slot[(size_t)t * k + s]; gv[s] = r_gates[(size_t)t * k + s]; }
    const int kept = split_part(K, parts, k, part, sel, gv);
    const int vg = kept > 0 ? parts * g + part : -1;
    cluster_id[vt] = vg;
    for (int s = 0; s < k; ++s) { slot[vt * k + s] = sel[s]; gates[vt * k + s] = gv[s]; }
    if (kc.keys) {
      int cs[kMaxKsel];
      float cg[kMaxKsel];
      const int key = vg >= 0 ? vg * kc.nsub + canonical_slots(sel, gv, k, kc.sub_is_combo, cs, cg) : -1;
      kc.keys[vt] = key;
      if (key >= 0) atomicAdd(&cnt[key], 1);
    }
  }
  if (kc.keys) {
    __syncthreads();
    for (int i = threadIdx.x; i < kc.nkey; i += blockDim.x) kc.block_counts[(size_t)blockIdx.x * kc.nkey + i] = cnt[i];
  }
}

int grid_for(long long n, int sm_count) {
  const long long want = (n + 255) / 256, most = (long long)(sm_count > 0 ? sm_count : 148) * 8;
  return (int)(want < most ? (want > 0 ? want : 1) : most);
}

}  // namespace

cudaError_t launch_repeat_rows(const Dims& D, const __half* x, __half* x_rep, int T, int n, cudaStream_t st) {
  const long long vec = D.d / 8;
  repeat_rows_kernel<<<grid_for((long long)T * vec, D.sm_count), 256, 0, st>>>(
      reinterpret_cast<const uint4*>(x), reinterpret_cast<uint4*>(x_rep), vec, T, n);
  return cudaGetLastError();
}

cudaError_t launch_sum_rows(const Dims& D, const __half* y_rep, __half* y, int T, int n, const int* cluster_id, cudaStream_t st) {
  const long long vec = D.d / 8;
  sum_rows_kernel<<<grid_for((long long)T * vec, D.sm_count), 256, 0, st>>>(
      reinterpret_cast<const uint4*>(y_rep), reinterpret_cast<uint4*>(y), vec, T, n, cluster_id);
  return cudaGetLastError();
}

int split_routes_tile() { return kSplitTile; }

cudaError_t launch_split_routes(const Dims& D, const Scratch& S, int T, cudaStream_t st, const KeyCount* kc) {
  const long long vts = (long long)T * D.split;
  split_routes_kernel<<<(unsigned)((vts + kSplitTile - 1) / kSplitTile), kSplitTile, 0, st>>>(
      T, real_K(D), D.split, D.k, S.r_cluster, S.r_slot, S.r_gates, S.cluster_id, S.slot, S.gates, kc ? *kc : KeyCount{});
  return cudaGetLastError();
}

}  // namespace cmoe
