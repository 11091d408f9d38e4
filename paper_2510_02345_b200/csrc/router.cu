// Fused two-stage router (Sec. 3.3): cluster logits z = x C and top-1 cluster (Eq. 9), expert
// logits l = x R_g* over the K experts of that cluster, top-k and renormalised softmax gates
// (Eq. 10).  One warp per token; all dot products are fp32 FMAs in a fixed order, so the result
// does not depend on the launch shape.
#include "cmoe_internal.h"
#include "device_utils.cuh"

namespace cmoe {

namespace {

// dot of the token row with one fp32 router row, lanes striding 8-element chunks
__device__ __forceinline__ float row_dot(const __half* __restrict__ xr, const float* __restrict__ wr,
                                         int d, int lane) {
  float acc = 0.f;
  for (int c = lane * 8; c < d; c += 256) {
    uint4 xv = *reinterpret_cast<const uint4*>(xr + c);
    float4 w0 = *reinterpret_cast<const float4*>(wr + c);
    float4 w1 = *reinterpret_cast<const float4*>(wr + c + 4);
    const __half2* xh = reinterpret_cast<const __half2*>(&xv);
    float2 a = __half22float2(xh[0]), b = __half22float2(xh[1]);
    float2 c2 = __half22float2(xh[2]), e = __half22float2(xh[3]);
    acc = fmaf(a.x, w0.x, acc);  acc = fmaf(a.y, w0.y, acc);
    acc = fmaf(b.x, w0.z, acc);  acc = fmaf(b.y, w0.w, acc);
    acc = fmaf(c2.x, w1.x, acc); acc = fmaf(c2.y, w1.y, acc);
    acc = fmaf(e.x, w1.z, acc);  acc = fmaf(e.y, w1.w, acc);
  }
  return warp_sum(acc);
}

__global__ void __launch_bounds__(256)
router_kernel(const __half* __restrict__ x, int T, int d, int G, int K, int k,
              const float* __restrict__ Ct, const float* __restrict__ Rt,
              const float* __restrict__ bc, const float* __restrict__ be,
              const int* __restrict__ label,
              int* __restrict__ cluster_id, int* __restrict__ expert_ids,
              float* __restrict__ gates, int* __restrict__ slot_local) {
  const int lane = threadIdx.x & 31;
  const int warps_per_block = blockDim.x >> 5;
  for (int t = blockIdx.x * warps_per_block + (threadIdx.x >> 5); t < T;
       t += gridDim.x * warps_per_block) {
    const __half* xr = x + (size_t)t * d;
    // stage 1: top-1 cluster = argmax of the logits (softmax of Eq. 9 is monotone)
    int gs = 0;
    float zbest = 0.f;
    for (int g = 0; g < G; ++g) {
      float z = row_dot(xr, Ct + (size_t)g * d, d, lane) + bc[g];
      if (g == 0 || z > zbest) { zbest = z; gs = g; }   // strict >: lowest index wins ties
    }
    // stage 2: lane i keeps the logit of expert i of the chosen cluster
    float myl = -INFINITY;
    for (int i = 0; i < K; ++i) {
      float l = row_dot(xr, Rt + (size_t)(gs * K + i) * d, d, lane) + be[gs * K + i];
      if (lane == i) myl = l;
    }
    // top-k by k rounds of warp arg-max (ties: lowest index)
    float selv[kMaxKsel];
    int seli[kMaxKsel];
    bool taken = (lane >= K);
#pragma unroll
    for (int s = 0; s < kMaxKsel; ++s) {
      if (s < k) {
        float v = taken ? -INFINITY : myl;
        int idx = taken ? 64 : lane;
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) {
          float ov = __shfl_xor_sync(0xffffffffu, v, o);
          int oi = __shfl_xor_sync(0xffffffffu, idx, o);
          if (ov > v || (ov == v && oi < idx)) { v = ov; idx = oi; }
        }
        selv[s] = v;
        seli[s] = idx;
        if (lane == idx) taken = true;
      }
    }
    if (lane == 0) cluster_id[t] = gs;
    // gates: softmax over the kept logits (= Eq. 10 renormalised over the kept experts)
    {
      const float lmax = selv[0];
      float ev[kMaxKsel];
      float sum = 0.f;
#pragma unroll
      for (int s = 0; s < kMaxKsel; ++s)
        if (s < k) {
          ev[s] = expf(selv[s] - lmax);
          sum += ev[s];
        }
#pragma unroll
      for (int s = 0; s < kMaxKsel; ++s)
        if (s < k && lane == 0) {
          int slot = gs * K + seli[s];
          if (gates) gates[(size_t)t * k + s] = ev[s] / sum;
          if (expert_ids) expert_ids[(size_t)t * k + s] = label[slot];
          if (slot_local) slot_local[(size_t)t * k + s] = seli[s];
        }
    }
  }
}

}  // namespace

cudaError_t launch_router(const Dims& D, const Weights& W, const __half* x, int T,
                          int* cluster_id, int* expert_ids, float* gates, int* slot_local,
                          cudaStream_t st) {
  if (T <= 0) return cudaSuccess;
  const int warps = 8;
  int blocks = (T + warps - 1) / warps;
  if (blocks > 148 * 8) blocks = 148 * 8;
  router_kernel<<<blocks, warps * 32, 0, st>>>(x, T, D.d, D.G, D.K, D.k, W.Ct, W.Rt, W.bc, W.be,
                                               W.label, cluster_id, expert_ids, gates, slot_local);
  return cudaGetLastError();
}

}  // namespace cmoe
