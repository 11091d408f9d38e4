// By-products of routing for the training-side clustering, and the self-test of the bounded waits.
//
// cmoe_expert_stats: expert loads, the per-expert mean of the routed tokens x-bar_i and the EMA update of
// the activation centroids mu_i (Sec. 3.1, Eq. 5), and the coefficient of variation of the loads (the
// expert load balance metric of Sec. 4.1).  Tokens are routed by the same kernels as cmoe_route; the sums
// run over the tokens in ascending order in fixed-shape partial sums, so the result is reproducible.
//
// cmoe_selftest_wait_timeout: a one-block kernel that runs the kernels' bounded mbarrier wait into its
// limit on purpose (nothing ever arrives on its barrier), to exercise the status word and its reporting.
#include "cmoe_internal.h"
#include "launch.cuh"
#include "tc_ptx.cuh"

namespace cmoe {

namespace {

constexpr int kStatThreads = 256;
constexpr int kStatCols = 256;          // columns of x a block sums: eight per lane

// loads[e] += tokens of this block routed to e (shared-memory histogram, one global atomic per expert and block)
__global__ void __launch_bounds__(kStatThreads)
loads_kernel(int T, int K, int k, int E, const int* __restrict__ cluster_id, const int* __restrict__ slot,
             int* __restrict__ loads) {
  pdl_wait();
  extern __shared__ int sh_cnt[];
  for (int i = threadIdx.x; i < E; i += blockDim.x) sh_cnt[i] = 0;
  __syncthreads();
  const int t = blockIdx.x * blockDim.x + threadIdx.x;
  if (t < T) {
    const int g = cluster_id[t];
    for (int j = 0; j < k; ++j) atomicAdd(&sh_cnt[g * K + slot[(size_t)t * k + j]], 1);
  }
  __syncthreads();
  for (int i = threadIdx.x; i < E; i += blockDim.x)
    if (sh_cnt[i]) atomicAdd(&loads[i], sh_cnt[i]);
}

// Block (e, c): columns 256 c .. of the sum of the tokens routed to expert e.  Warp w takes the tokens
// w, w + 8, ... in ascending order; the eight partial sums are added in warp order.  Then x-bar and Eq. 5.
__global__ void __launch_bounds__(kStatThreads)
xbar_kernel(int T, int d, int K, int k, const __half* __restrict__ x, const int* __restrict__ cluster_id,
            const int* __restrict__ slot, const int* __restrict__ loads, float* __restrict__ xbar,
            float* __restrict__ mu, float beta) {
  pdl_wait();
  __shared__ float part[kStatThreads / 32][kStatCols];
  const int e = blockIdx.x, g = e / K, i = e - g * K;
  const int c0 = blockIdx.y * kStatCols;
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, nwarp = blockDim.x >> 5;
  const int col = c0 + lane * 8;
  float acc[8];
#pragma unroll
  for (int n = 0; n < 8; ++n) acc[n] = 0.f;
  for (int t = warp; t < T; t += nwarp) {
    if (cluster_id[t] != g) continue;
    bool mine = false;
    for (int j = 0; j < k; ++j) mine |= slot[(size_t)t * k + j] == i;
    if (!mine || col >= d) continue;
    const uint4 v = *reinterpret_cast<const uint4*>(x + (size_t)t * d + col);
    const __half2* h = reinterpret_cast<const __half2*>(&v);
#pragma unroll
    for (int n = 0; n < 4; ++n) {
      const float2 f = __half22float2(h[n]);
      acc[2 * n] += f.x;
      acc[2 * n + 1] += f.y;
    }
  }
#pragma unroll
  for (int n = 0; n < 8; ++n) part[warp][lane * 8 + n] = acc[n];
  __syncthreads();
  const int cc = threadIdx.x;                 // one column per thread
  if (c0 + cc < d) {
    float sum = 0.f;
    for (int w = 0; w < nwarp; ++w) sum += part[w][cc];
    const int n = loads[e];
    const float mean = n > 0 ? sum / (float)n : 0.f;
    const size_t o = (size_t)e * d + c0 + cc;
    if (xbar) xbar[o] = mean;
    if (mu && n > 0) mu[o] = (1.f - beta) * mu[o] + beta * mean;       // Eq. 5; no tokens: mu_i stays
  }
}

// population standard deviation of the loads over their mean (one block)
__global__ void __launch_bounds__(kStatThreads)
cov_kernel(int E, const int* __restrict__ loads, float* __restrict__ cov) {
  pdl_wait();
  __shared__ double red[kStatThreads];
  double s = 0.0;
  for (int i = threadIdx.x; i < E; i += blockDim.x) s += (double)loads[i];
  red[threadIdx.x] = s;
  __syncthreads();
  for (int o = kStatThreads / 2; o > 0; o >>= 1) {
    if ((int)threadIdx.x < o) red[threadIdx.x] += red[threadIdx.x + o];
    __syncthreads();
  }
  const double mean = red[0] / (double)E;
  __syncthreads();
  double v = 0.0;
  for (int i = threadIdx.x; i < E; i += blockDim.x) { const double dlt = (double)loads[i] - mean; v += dlt * dlt; }
  red[threadIdx.x] = v;
  __syncthreads();
  for (int o = kStatThreads / 2; o > 0; o >>= 1) {
    if ((int)threadIdx.x < o) red[threadIdx.x] += red[threadIdx.x + o];
    __syncthreads();
  }
  if (threadIdx.x == 0) *cov = mean > 0.0 ? (float)(sqrt(red[0] / (double)E) / mean) : 0.f;
}

__global__ void wait_timeout_kernel(long long limit_cycles, int* status) {
  __shared__ uint64_t bar;
  __shared__ int abort_flag;
  if (threadIdx.x == 0) {
    abort_flag = 0;
    ptx::mbar_init(ptx::smem_u32(&bar), 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    // phase 0 of the barrier never completes: nobody arrives
    if (!ptx::mbar_wait(ptx::smem_u32(&bar), 0, &abort_flag, limit_cycles)) atomicExch(status, (int)CMOE_ERR_TIMEOUT);
  }
}

}  // namespace

}  // namespace cmoe

using namespace cmoe;

extern "C" int cmoe_selftest_wait_timeout(cmoe_layer* L, int64_t limit_cycles, void* cuda_stream) {
  if (!L || limit_cycles < 1 || limit_cycles > (1ll << 31)) return CMOE_ERR_INVALID_ARG;
  wait_timeout_kernel<<<1, 32, 0, static_cast<cudaStream_t>(cuda_stream)>>>((long long)limit_cycles, L->sc.status);
  const cudaError_t e = cudaGetLastError();
  if (e != cudaSuccess) { L->last_cuda_error = (int)e; return CMOE_ERR_CUDA; }
  return CMOE_OK;
}

extern "C" int cmoe_expert_stats(cmoe_layer* L, const void* x, int32_t T, int32_t* loads, float* xbar,
                                 float* mu, float beta, float* cov, void* cuda_stream) {
  if (!L || T < 0 || !loads) return CMOE_ERR_INVALID_ARG;
  if (T > L->dims.T_user) return CMOE_ERR_T_EXCEEDS_MAX;
  if (T > 0 && (!x || (reinterpret_cast<uintptr_t>(x) & 15))) return CMOE_ERR_INVALID_ARG;
  if (!(beta >= 0.f && beta <= 1.f)) return CMOE_ERR_INVALID_ARG;
  const Dims& D = L->dims;
  const Scratch& S = L->sc;
  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
  cudaError_t e;
#define STAT_CUDA(expr) do { e = (expr); if (e != cudaSuccess) { L->last_cuda_error = (int)e; return CMOE_ERR_CUDA; } } while (0)
  STAT_CUDA(cudaMemsetAsync(loads, 0, sizeof(int) * (size_t)D.E, st));
  if (T == 0) {
    if (xbar) STAT_CUDA(cudaMemsetAsync(xbar, 0, sizeof(float) * (size_t)D.E * D.d, st));
    if (cov) STAT_CUDA(cudaMemsetAsync(cov, 0, sizeof(float), st));
    return CMOE_OK;
  }
  const __half* xh = static_cast<const __half*>(x);
  if (D.g1 > 1) {
    // g1 virtual tokens per token: an expert's load counts the tokens that reach it through either kept cluster
    STAT_CUDA(launch_repeat_rows(D, xh, S.x_rep, T, D.g1, st));
    xh = S.x_rep;
    T *= D.g1;
  }
  // (the token's own routes, also when the layer works on expert halves)
  if (L->router_tc && T >= 1024) STAT_CUDA(launch_router_tc(L, xh, T, S.cluster_id, nullptr, S.gates, S.slot, st));
  else STAT_CUDA(launch_router(plain_dims(D), L->w, xh, T, S.cluster_id, nullptr, S.gates, S.slot, st));
  STAT_CUDA(launch_chained(loads_kernel, dim3((T + kStatThreads - 1) / kStatThreads), dim3(kStatThreads),
                           sizeof(int) * (size_t)D.E, st, 1, (int)T, real_K(D), D.k, D.E, (const int*)S.cluster_id,
                           (const int*)S.slot, (int*)loads));
  if (xbar || mu)
    STAT_CUDA(launch_chained(xbar_kernel, dim3(D.E, (D.d + kStatCols - 1) / kStatCols), dim3(kStatThreads), 0, st, 1,
                             (int)T, D.d, real_K(D), D.k, xh, (const int*)S.cluster_id, (const int*)S.slot,
                             (const int*)loads, xbar, mu, beta));
  if (cov) STAT_CUDA(launch_chained(cov_kernel, dim3(1), dim3(kStatThreads), 0, st, 1, D.E, (const int*)loads, cov));
#undef STAT_CUDA
  return CMOE_OK;
}
