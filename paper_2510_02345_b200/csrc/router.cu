// Fused two-stage router (Sec. 3.3): cluster logits z = x C and top-1 cluster (Eq. 9), expert
// logits l = x R_g* over the K experts of that cluster, top-k and renormalised softmax gates
// (Eq. 10).  All dot products are fp32 FMAs in a fixed order per kernel, so a token's route does not
// depend on where in the batch it sits; which kernel runs depends only on the batch size.
//
//   router_tile_kernel   many tokens: a block takes 64 tokens, a warp eight of them at a time, so
//                        that a router row fetched by a lane is used for eight tokens.  Stage 1
//                        reads the cluster prototypes from shared memory; for stage 2 the block
//                        orders its tokens by cluster, so that the eight tokens of a warp mostly
//                        share one cluster's expert rows.
//   router_token_kernel  few tokens (decode): one block per token, a warp per router row.
//
// In both, lane l of a warp owns the columns 256 s + 8 l .. + 7 of the 256-column segments it
// visits, a lane's partial sum runs over its columns in ascending order, and partial sums are
// combined by the same xor butterfly, so both kernels give a token the same logits.
#include "cmoe_internal.h"
#include "launch.cuh"
#include "device_utils.cuh"
#include "stage_factors.cuh"
#include "cluster_pick.cuh"

namespace cmoe {

namespace {

constexpr int kTokPerWarp = 8;
constexpr int kTileWarps = 8;
constexpr int kTileTokens = kTokPerWarp * kTileWarps;     // 64
constexpr int kGroup = 8;                                  // router rows accumulated at once

__device__ __forceinline__ void fma8(float& acc, const uint4& xv, const float4& w0, const float4& w1) {
  const __half2* xh = reinterpret_cast<const __half2*>(&xv);
  const float2 a = __half22float2(xh[0]), b = __half22float2(xh[1]);
  const float2 c = __half22float2(xh[2]), e = __half22float2(xh[3]);
  acc = fmaf(a.x, w0.x, acc); acc = fmaf(a.y, w0.y, acc);
  acc = fmaf(b.x, w0.z, acc); acc = fmaf(b.y, w0.w, acc);
  acc = fmaf(c.x, w1.x, acc); acc = fmaf(c.y, w1.y, acc);
  acc = fmaf(e.x, w1.z, acc); acc = fmaf(e.y, w1.w, acc);
}

// Top-k of K logits (ties: lowest index), gates = softmax over the kept logits (Eq. 10
// renormalised over the kept experts); one thread per token, logits read from `lg`.
__device__ __forceinline__ void select_and_store(const float* lg, int K, int k, int g, int t,
                                                 const int* __restrict__ label, int* __restrict__ expert_ids,
                                                 float* __restrict__ gates, int* __restrict__ slot_local,
                                                 float cluster_weight = 1.f) {
  unsigned taken = 0;
  float selv[kMaxKsel];
  int seli[kMaxKsel];
  for (int s = 0; s < k; ++s) {
    float best = -INFINITY;
    int bi = 0;
    bool have = false;
    for (int i = 0; i < K; ++i) {
      if ((taken >> i) & 1u) continue;
      const float v = lg[i];
      if (!have || v > best) { best = v; bi = i; have = true; }   // strict >: lowest index wins ties
    }
    taken |= 1u << bi;
    selv[s] = best;
    seli[s] = bi;
  }
  const float lmax = selv[0];
  float ev[kMaxKsel];
  float sum = 0.f;
  for (int s = 0; s < k; ++s) { ev[s] = expf(selv[s] - lmax); sum += ev[s]; }
  for (int s = 0; s < k; ++s) {
    if (gates) gates[(size_t)t * k + s] = cluster_weight == 1.f ? ev[s] / sum : cluster_weight * (ev[s] / sum);
    if (expert_ids) expert_ids[(size_t)t * k + s] = label[g * K + seli[s]];
    if (slot_local) slot_local[(size_t)t * k + s] = seli[s];
  }
}

struct RouterArgs {
  const __half* x;
  int T, d, G, K, k;
  const float *Ct, *Rt, *bc, *be;
  const int* label;
  int* cluster_id;
  int* expert_ids;
  float* gates;
  int* slot_local;
  FactorStage fs;  // per-token kernel only: factor staging that rides in the blocks past the router's own (all words zero: none)
  int n_route_blocks, n_riders;
  int g1;          // clusters per token: token index t is virtual token t % g1 of caller token t / g1 (x holds its row g1 times)
  int dc;          // columns of the cluster prototypes staged in shared memory at a time
  int crows;       // prototype rows staged at a time: min(G, 8)
};

__global__ void __launch_bounds__(kTileWarps * 32)
router_tile_kernel(const RouterArgs a) {
  pdl_wait();
  extern __shared__ float sm_f[];
  float* Cs = sm_f;                                        // [crows][dc]
  float* lg = Cs + (size_t)a.crows * a.dc;                 // [64][K] expert logits
  __shared__ int s_cid[kTileTokens];
  __shared__ int s_order[kTileTokens];
  __shared__ float s_zbest[kTileTokens];
  __shared__ float s_z2[kTileTokens];                      // two clusters per token: second-best logit, its cluster,
  __shared__ int s_cid2[kTileTokens];                      // and the weight of the cluster the virtual token goes to
  __shared__ float s_weight[kTileTokens];

  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int tok0 = blockIdx.x * kTileTokens;
  const int d = a.d, G = a.G, K = a.K;

  // ---- stage 1: cluster logits of the warp's eight tokens, clusters in groups of eight
  const int wt0 = tok0 + warp * kTokPerWarp;
  for (int g0 = 0; g0 < G; g0 += kGroup) {
    const int ng = min(kGroup, G - g0);
    float acc[kTokPerWarp][kGroup];
#pragma unroll
    for (int t = 0; t < kTokPerWarp; ++t)
#pragma unroll
      for (int j = 0; j < kGroup; ++j) acc[t][j] = 0.f;
    for (int c0 = 0; c0 < d; c0 += a.dc) {
      const int cw = min(a.dc, d - c0);
      __syncthreads();                                     // the previous chunk is no longer read
      for (int i = threadIdx.x * 4; i < ng * cw; i += blockDim.x * 4) {
        const int j = i / cw, c = i - j * cw;
        *reinterpret_cast<float4*>(Cs + (size_t)j * a.dc + c) =
            *reinterpret_cast<const float4*>(a.Ct + (size_t)(g0 + j) * d + c0 + c);
      }
      __syncthreads();
      for (int c = lane * 8; c < cw; c += 256) {
        uint4 xv[kTokPerWarp];
#pragma unroll
        for (int t = 0; t < kTokPerWarp; ++t) {
          const int tok = min(wt0 + t, a.T - 1);
          xv[t] = *reinterpret_cast<const uint4*>(a.x + (size_t)tok * d + c0 + c);
        }
#pragma unroll
        for (int j = 0; j < kGroup; ++j) {
          if (j < ng) {
            const float4 w0 = *reinterpret_cast<const float4*>(Cs + (size_t)j * a.dc + c);
            const float4 w1 = *reinterpret_cast<const float4*>(Cs + (size_t)j * a.dc + c + 4);
#pragma unroll
            for (int t = 0; t < kTokPerWarp; ++t) fma8(acc[t][j], xv[t], w0, w1);
          }
        }
      }
    }
    // combine the lanes' partial sums; lane t keeps the running arg-max of token t
#pragma unroll
    for (int t = 0; t < kTokPerWarp; ++t) {
#pragma unroll
      for (int j = 0; j < kGroup; ++j) {
        const float z = warp_sum(acc[t][j]);
        if (j < ng && lane == t) {
          const float zb = z + a.bc[g0 + j];
          const int slot = warp * kTokPerWarp + t;
          if (a.g1 < 2) {
            if ((g0 + j) == 0 || zb > s_zbest[slot]) { s_zbest[slot] = zb; s_cid[slot] = g0 + j; }   // strict >: lowest index wins ties
          } else {
            TwoBest b{s_zbest[slot], s_z2[slot], (g0 + j) == 0 ? -1 : s_cid[slot], (g0 + j) <= 1 ? -1 : s_cid2[slot]};
            two_best_add(b, g0 + j, zb);
            s_zbest[slot] = b.z1; s_z2[slot] = b.z2; s_cid[slot] = b.c1; s_cid2[slot] = b.c2;
          }
        }
      }
    }
    __syncwarp();
  }
  __syncthreads();
  if (a.g1 >= 2 && threadIdx.x < kTileTokens) {
    // virtual token 2 t + c takes the token's c-th most probable cluster
    const TwoBest b{s_zbest[threadIdx.x], s_z2[threadIdx.x], s_cid[threadIdx.x], s_cid2[threadIdx.x]};
    int g;
    float w;
    two_best_pick(b, (tok0 + threadIdx.x) & 1, g, w);
    s_cid[threadIdx.x] = g;
    s_weight[threadIdx.x] = w;
  }
  __syncthreads();

  // ---- order the block's tokens by cluster (stable), so that a warp's eight tokens share rows
  if (threadIdx.x < kTileTokens) {
    const int me = threadIdx.x, c = s_cid[me];
    int rank = 0;
    for (int u = 0; u < kTileTokens; ++u) {
      const int cu = s_cid[u];
      rank += (cu < c || (cu == c && u < me)) ? 1 : 0;
    }
    s_order[rank] = me;
    if (tok0 + me < a.T) a.cluster_id[tok0 + me] = c;
  }
  __syncthreads();

  // ---- stage 2: expert logits; the warp takes eight tokens of the ordered list, run by run
  int slot_of[kTokPerWarp], cl_of[kTokPerWarp];
#pragma unroll
  for (int t = 0; t < kTokPerWarp; ++t) {
    slot_of[t] = s_order[warp * kTokPerWarp + t];
    cl_of[t] = s_cid[slot_of[t]];
  }
  int j0 = 0;
  while (j0 < kTokPerWarp) {
    int g = 0;
#pragma unroll
    for (int t = 0; t < kTokPerWarp; ++t)
      if (t == j0) g = cl_of[t];
    unsigned active = 0;                                   // tokens of this run
    int j1 = j0;
#pragma unroll
    for (int t = 0; t < kTokPerWarp; ++t)
      if (t >= j0 && cl_of[t] == g) { active |= 1u << t; j1 = t + 1; }
    for (int i0 = 0; i0 < K; i0 += 4) {
      const int ni = min(4, K - i0);
      float acc[kTokPerWarp][4];
#pragma unroll
      for (int t = 0; t < kTokPerWarp; ++t)
#pragma unroll
        for (int i = 0; i < 4; ++i) acc[t][i] = 0.f;
      for (int c = lane * 8; c < d; c += 256) {
        uint4 xv[kTokPerWarp];
#pragma unroll
        for (int t = 0; t < kTokPerWarp; ++t) {
          xv[t] = make_uint4(0, 0, 0, 0);
          if ((active >> t) & 1u) {
            const int tok = min(tok0 + slot_of[t], a.T - 1);
            xv[t] = *reinterpret_cast<const uint4*>(a.x + (size_t)tok * d + c);
          }
        }
#pragma unroll
        for (int i = 0; i < 4; ++i) {
          if (i < ni) {
            const float* wr = a.Rt + (size_t)(g * K + i0 + i) * d + c;
            const float4 w0 = __ldg(reinterpret_cast<const float4*>(wr));
            const float4 w1 = __ldg(reinterpret_cast<const float4*>(wr + 4));
#pragma unroll
            for (int t = 0; t < kTokPerWarp; ++t) fma8(acc[t][i], xv[t], w0, w1);
          }
        }
      }
#pragma unroll
      for (int t = 0; t < kTokPerWarp; ++t) {
#pragma unroll
        for (int i = 0; i < 4; ++i) {
          const float l = warp_sum(acc[t][i]);
          if (i < ni && ((active >> t) & 1u) && lane == t)
            lg[(size_t)slot_of[t] * K + i0 + i] = l + a.be[g * K + i0 + i];
        }
      }
    }
    j0 = j1;
  }
  __syncthreads();

  // ---- top-k and gates: one thread per token
  if (threadIdx.x < kTileTokens && tok0 + threadIdx.x < a.T)
    select_and_store(lg + (size_t)threadIdx.x * K, K, a.k, s_cid[threadIdx.x], tok0 + threadIdx.x, a.label,
                     a.expert_ids, a.gates, a.slot_local, a.g1 >= 2 ? s_weight[threadIdx.x] : 1.f);
}

// One block per token; warp w computes the rows w, w + nwarp, ... of the router matrix, each over all of d
// (so a dot product is summed in the same order as in the tiled kernel).
__global__ void __launch_bounds__(256)
router_token_kernel(const RouterArgs a) {
  pdl_wait();
  if ((int)blockIdx.x >= a.n_route_blocks) { stage_block(a.fs, blockIdx.x - a.n_route_blocks); return; }
  __shared__ float lg[kMaxG];           // cluster logits, then the expert logits (kMaxK <= kMaxG)
  __shared__ int s_g;
  __shared__ float s_w;                 // weight of the chosen cluster (two clusters per token), else 1
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, nwarp = blockDim.x >> 5;
  const int t = blockIdx.x, d = a.d;
  const __half* xr = a.x + (size_t)t * d;
  {
    // the second pass reads the expert rows of a cluster that is not known yet: bring all of them into
    // L2 while the cluster logits are computed (every thread of the grid asks for one 128-byte line at a time)
    const size_t bytes = (size_t)a.G * a.K * d * sizeof(float);
    const size_t step = (size_t)gridDim.x * blockDim.x * 128;
    for (size_t off = ((size_t)blockIdx.x * blockDim.x + threadIdx.x) * 128; off < bytes; off += step)
      asm volatile("prefetch.global.L2 [%0];" ::"l"(reinterpret_cast<const char*>(a.Rt) + off));
    // the first pass itself: all lines of the cluster prototypes and of this token's row are requested now,
    // so its unrolled batches of loads meet DRAM latency once
    const size_t cbytes = (size_t)a.G * d * sizeof(float);
    for (size_t off = (size_t)threadIdx.x * 128; off < cbytes; off += (size_t)blockDim.x * 128)
      asm volatile("prefetch.global.L2 [%0];" ::"l"(reinterpret_cast<const char*>(a.Ct) + off));
    for (size_t off = (size_t)threadIdx.x * 128; off < (size_t)d * sizeof(__half); off += (size_t)blockDim.x * 128)
      asm volatile("prefetch.global.L2 [%0];" ::"l"(reinterpret_cast<const char*>(xr) + off));
  }
  for (int pass = 0; pass < 2; ++pass) {
    const int n = pass == 0 ? a.G : a.K;
    const float* W = pass == 0 ? a.Ct : a.Rt + (size_t)s_g * a.K * d;
    const float* bias = pass == 0 ? a.bc : a.be + s_g * a.K;
    for (int j = warp; j < n; j += nwarp) {
      const float* wr = W + (size_t)j * d;
      float acc = 0.f;
#pragma unroll 8
      for (int c = lane * 8; c < d; c += 256)
        fma8(acc, *reinterpret_cast<const uint4*>(xr + c), __ldg(reinterpret_cast<const float4*>(wr + c)),
             __ldg(reinterpret_cast<const float4*>(wr + c + 4)));
      acc = warp_sum(acc);
      if (lane == 0) lg[j] = acc + bias[j];
    }
    __syncthreads();
    if (pass == 0) {
      if (threadIdx.x == 0) {
        int gs = 0;
        float w = 1.f;
        if (a.g1 < 2) {
          float zb = lg[0];
          for (int g = 1; g < a.G; ++g)
            if (lg[g] > zb) { zb = lg[g]; gs = g; }        // strict >: lowest index wins ties
        } else {
          TwoBest b;
          two_best_init(b);
          for (int g = 0; g < a.G; ++g) two_best_add(b, g, lg[g]);
          two_best_pick(b, t & 1, gs, w);
        }
        s_g = gs;
        s_w = w;
        a.cluster_id[t] = gs;
      }
      __syncthreads();
    }
  }
  if (threadIdx.x == 0) select_and_store(lg, a.K, a.k, s_g, t, a.label, a.expert_ids, a.gates, a.slot_local, s_w);
}

}  // namespace

cudaError_t launch_router(const Dims& D, const Weights& W, const __half* x, int T,
                          int* cluster_id, int* expert_ids, float* gates, int* slot_local,
                          cudaStream_t st, const FactorStage* fs) {
  if (T <= 0) return cudaSuccess;
  RouterArgs a{};
  // (the staging of the tensor-core residual factors rides here for batches below 1024 tokens, else in the
  // permutation's row-move kernel)
  if (fs && T < 1024) a.fs = *fs;
  a.n_riders = stage_blocks(a.fs, 256);          // one 32-bit word of packed codes per thread
  a.x = x; a.T = T; a.d = D.d; a.G = real_G(D); a.K = real_K(D); a.k = D.k; a.g1 = D.g1;
  // (a layer on expert halves routes its tokens over the real clusters; the routes are split afterwards)
  a.Ct = W.Ct; a.Rt = W.Rt; a.bc = W.bc; a.be = W.be; a.label = W.label;
  a.cluster_id = cluster_id; a.expert_ids = expert_ids; a.gates = gates; a.slot_local = slot_local;
  if (T < 1024) {
    // few tokens: the per-token kernel puts every token on its own SM
    a.n_route_blocks = T;
    launch_chained(router_token_kernel, dim3(T + a.n_riders), dim3(256), 0, st, 1,
      a);
    return cudaGetLastError();
  }
  // chunk of the prototypes staged at a time: at most 32 KB for a group of eight clusters
  const int rows = a.G < kGroup ? a.G : kGroup;
  int dc = 32768 / (4 * rows) / 256 * 256;
  if (dc > D.d) dc = D.d;
  a.dc = dc;
  a.crows = rows;
  const size_t sh = sizeof(float) * ((size_t)rows * dc + (size_t)kTileTokens * a.K);      // at most 32 KB + 8 KB
  static std::atomic<unsigned long long> smem_set{0};      // devices the kernel's shared-memory limit has been raised on
  if (cudaError_t e = ensure_dynamic_smem(router_tile_kernel, 64 * 1024, smem_set)) return e;
  launch_chained(router_tile_kernel, dim3((T + kTileTokens - 1) / kTileTokens), dim3(kTileWarps * 32), sh, st, 1,
      a);
  return cudaGetLastError();
}

}  // namespace cmoe
