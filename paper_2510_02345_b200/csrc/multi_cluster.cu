// Virtual tokens.  Two clusters per token (Sec. 3.3, "Top-g1 groups"): the layer runs on g1 virtual tokens per token.  Before the
// router every row of x is written g1 times (virtual token g1 t + c is token t on its way to its c-th most
// probable cluster); after the un-permuting store the g1 output rows of a token are summed.  The gates already
// carry the clusters' weights, so the sum is the mixture.  Expert halves (Dims::split) use the same two kernels: a
// token's two virtual tokens carry the experts of one half of its cluster each.
#include "cmoe_internal.h"

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

__global__ void __launch_bounds__(256)
sum_rows_kernel(const __half2* __restrict__ y_rep, __half2* __restrict__ y, long long pairs_per_row, long long T, int g1) {
  const long long n = T * pairs_per_row;
  for (long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x; i < n; i += (long long)gridDim.x * blockDim.x) {
    const long long t = i / pairs_per_row, v = i - t * pairs_per_row;
    float2 acc = make_float2(0.f, 0.f);
    for (int c = 0; c < g1; ++c) {
      const float2 f = __half22float2(y_rep[(t * g1 + c) * pairs_per_row + v]);
      acc.x += f.x;
      acc.y += f.y;
    }
    y[i] = __floats2half2_rn(acc.x, acc.y);
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

cudaError_t launch_sum_rows(const Dims& D, const __half* y_rep, __half* y, int T, int n, cudaStream_t st) {
  const long long pairs = D.d / 2;
  sum_rows_kernel<<<grid_for((long long)T * pairs, D.sm_count), 256, 0, st>>>(
      reinterpret_cast<const __half2*>(y_rep), reinterpret_cast<__half2*>(y), pairs, T, n);
  return cudaGetLastError();
}

}  // namespace cmoe
