// Create-time layout changes: batched matrix transposes that bring the router matrices and the
// FP16 bases into reduction-index-fastest order.
#include "cmoe_internal.h"

namespace cmoe {

namespace {

template <typename T>
__global__ void __launch_bounds__(256)
transpose_kernel(const T* __restrict__ src, T* __restrict__ dst, int rows, int cols) {
  __shared__ T tile[32][33];
  const size_t mat = (size_t)blockIdx.z * rows * cols;
  const int c0 = blockIdx.x * 32, r0 = blockIdx.y * 32;
  const int tx = threadIdx.x & 31, ty = threadIdx.x >> 5;   // 32 x 8
  for (int i = ty; i < 32; i += 8) {
    int r = r0 + i, c = c0 + tx;
    if (r < rows && c < cols) tile[i][tx] = src[mat + (size_t)r * cols + c];
  }
  __syncthreads();
  for (int i = ty; i < 32; i += 8) {
    int c = c0 + i, r = r0 + tx;
    if (r < rows && c < cols) dst[mat + (size_t)c * rows + r] = tile[tx][i];
  }
}

template <typename T>
cudaError_t launch_t(const T* src, T* dst, int batch, int rows, int cols, cudaStream_t st) {
  // grid.y and grid.z are limited to 65535: fold large batches / row counts by looping on the host
  const int gx = (cols + 31) / 32, gy = (rows + 31) / 32;
  if (gy > 65535 || gx <= 0) return cudaErrorInvalidValue;
  for (int b0 = 0; b0 < batch; b0 += 65535) {
    int nb = batch - b0 < 65535 ? batch - b0 : 65535;
    dim3 grid(gx, gy, nb);
    transpose_kernel<T><<<grid, 256, 0, st>>>(src + (size_t)b0 * rows * cols,
                                               dst + (size_t)b0 * rows * cols, rows, cols);
  }
  return cudaGetLastError();
}

}  // namespace

cudaError_t launch_transpose_fp16(const __half* src, __half* dst, int batch, int rows, int cols,
                                  cudaStream_t st) {
  return launch_t<__half>(src, dst, batch, rows, cols, st);
}
cudaError_t launch_transpose_f32(const float* src, float* dst, int batch, int rows, int cols,
                                 cudaStream_t st) {
  return launch_t<float>(src, dst, batch, rows, cols, st);
}

}  // namespace cmoe
