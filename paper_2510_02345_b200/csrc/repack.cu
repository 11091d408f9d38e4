// Create-time layout changes: batched matrix transposes that bring the router matrices and the
// FP16 bases into reduction-index-fastest order.
#include "cmoe_internal.h"

namespace cmoe {

namespace {

// conversion applied on the way (identity, or bfloat16 bits -> fp16)
struct KeepBits {
  template <typename T> __device__ static T apply(T v) { return v; }
};
struct Bf16ToHalf {
  // the bf16 bit pattern is the upper half of the fp32 pattern; fp16 holds every bf16 value of its normal range
  // exactly (8 significant bits into 11) and rounds the ones below 2^-14 to its subnormal grid
  __device__ static __half apply(__half v) {
    const unsigned short bits = *reinterpret_cast<const unsigned short*>(&v);
    return __float2half_rn(__uint_as_float((unsigned)bits << 16));
  }
};

template <typename T, typename Conv>
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
    if (r < rows && c < cols) dst[mat + (size_t)c * rows + r] = Conv::apply(tile[tx][i]);
  }
}

// Base matrices of the weight-streaming path: src [batch][rows][cols] (rows = reduction index) ->
// dst [rows / 128][batch * cols][128], i.e. for every 128 reduction indices (one pipeline stage of the kernel)
// the slab of all output features, 256 bytes each: the rows a CTA loads per stage are one contiguous piece of
// memory, and the CTAs of a launch, which walk the reduction index in step, read neighbouring pieces.
template <typename Conv>
__global__ void __launch_bounds__(256)
stage_major_kernel(const __half* __restrict__ src, __half* __restrict__ dst, int batch, int rows, int cols) {
  __shared__ __half tile[32][33];
  const size_t mat = (size_t)blockIdx.z * rows * cols;
  const int c0 = blockIdx.x * 32, r0 = blockIdx.y * 32;       // rows is a multiple of 128: a tile stays inside one stage
  const int tx = threadIdx.x & 31, ty = threadIdx.x >> 5;   // 32 x 8
  for (int i = ty; i < 32; i += 8) {
    const int r = r0 + i, c = c0 + tx;
    if (r < rows && c < cols) tile[i][tx] = src[mat + (size_t)r * cols + c];
  }
  __syncthreads();
  const size_t slab = (size_t)batch * cols * 128;
  for (int i = ty; i < 32; i += 8) {
    const int c = c0 + i, r = r0 + tx;
    if (r < rows && c < cols)
      dst[(size_t)(r >> 7) * slab + ((size_t)blockIdx.z * cols + c) * 128 + (r & 127)] = Conv::apply(tile[tx][i]);
  }
}

template <typename T, typename Conv = KeepBits>
cudaError_t launch_t(const T* src, T* dst, int batch, int rows, int cols, cudaStream_t st) {
  // grid.y and grid.z are limited to 65535: fold large batches / row counts by looping on the host
  const int gx = (cols + 31) / 32, gy = (rows + 31) / 32;
  if (gy > 65535 || gx <= 0) return cudaErrorInvalidValue;
  for (int b0 = 0; b0 < batch; b0 += 65535) {
    int nb = batch - b0 < 65535 ? batch - b0 : 65535;
    dim3 grid(gx, gy, nb);
    transpose_kernel<T, Conv><<<grid, 256, 0, st>>>(src + (size_t)b0 * rows * cols,
                                               dst + (size_t)b0 * rows * cols, rows, cols);
  }
  return cudaGetLastError();
}

// One block per expert: is any element of the factor non-zero (a non-zero code in a group with a non-zero scale)?
// live[e] bit 0 = U1_e and V1_e both have one, bit 1 = U2_e and V2_e: a residual block is zero as soon as one of its
// two factors is (Sec. 3.4: blocks zeroed by the cosine gate cost nothing).
__global__ void __launch_bounds__(256)
residual_live_kernel(int r, int d, int d_ff, const uint8_t* __restrict__ U1q, const uint8_t* __restrict__ V1q,
                     const uint8_t* __restrict__ U2q, const uint8_t* __restrict__ V2q, const __half* __restrict__ U1s,
                     const __half* __restrict__ V1s, const __half* __restrict__ U2s, const __half* __restrict__ V2s,
                     int* __restrict__ live) {
  const int e = blockIdx.x;
  const uint8_t* q[4] = {U1q, V1q, U2q, V2q};
  const __half* sc[4] = {U1s, V1s, U2s, V2s};
  const long long n[4] = {(long long)r * d, (long long)d_ff * r, (long long)r * d_ff, (long long)d * r};
  __shared__ int any[4];
  if (threadIdx.x < 4) any[threadIdx.x] = 0;
  __syncthreads();
  for (int f = 0; f < 4; ++f) {
    const long long groups = n[f] / 32;           // 16 bytes of codes and one scale each
    const uint4* codes = reinterpret_cast<const uint4*>(q[f]) + (long long)e * groups;
    const __half* scale = sc[f] + (long long)e * groups;
    bool mine = false;
    for (long long gi = threadIdx.x; gi < groups; gi += blockDim.x) {
      const uint4 c = codes[gi];
      if ((c.x | c.y | c.z | c.w) != 0u && __half2float(scale[gi]) != 0.f) mine = true;
    }
    if (mine) any[f] = 1;      // benign race: every writer stores 1
  }
  __syncthreads();
  if (threadIdx.x == 0) live[e] = ((any[0] && any[1]) ? 1 : 0) | ((any[2] && any[3]) ? 2 : 0);
}

}  // namespace

cudaError_t launch_residual_live(const Dims& D, const Weights& W, cudaStream_t st) {
  if (D.r == 0) return cudaMemsetAsync(const_cast<int*>(W.live), 0, sizeof(int) * (size_t)D.E, st);
  residual_live_kernel<<<D.E, 256, 0, st>>>(D.r, D.d, D.d_ff, W.U1q, W.V1q, W.U2q, W.V2q, W.U1s, W.V1s, W.U2s, W.V2s,
                                            const_cast<int*>(W.live));
  return cudaGetLastError();
}

cudaError_t launch_transpose_fp16(const __half* src, __half* dst, int batch, int rows, int cols,
                                  cudaStream_t st, bool src_is_bf16) {
  if (src_is_bf16) return launch_t<__half, Bf16ToHalf>(src, dst, batch, rows, cols, st);
  return launch_t<__half>(src, dst, batch, rows, cols, st);
}
cudaError_t launch_stage_major_fp16(const __half* src, __half* dst, int batch, int rows, int cols, cudaStream_t st,
                                    bool src_is_bf16) {
  const int gx = (cols + 31) / 32, gy = (rows + 31) / 32;
  if (rows % 128 != 0 || gy > 65535 || batch > 65535 || gx <= 0) return cudaErrorInvalidValue;
  dim3 grid(gx, gy, batch);
  if (src_is_bf16) stage_major_kernel<Bf16ToHalf><<<grid, 256, 0, st>>>(src, dst, batch, rows, cols);
  else             stage_major_kernel<KeepBits><<<grid, 256, 0, st>>>(src, dst, batch, rows, cols);
  return cudaGetLastError();
}
cudaError_t launch_transpose_f32(const float* src, float* dst, int batch, int rows, int cols,
                                 cudaStream_t st) {
  return launch_t<float>(src, dst, batch, rows, cols, st);
}

}  // namespace cmoe
