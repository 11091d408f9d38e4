// Shared pieces of the CTA-pair tensor-core kernels (tc2_path.cu, tc2_up_wide.cu): tile constants,
// small device helpers, the parameter block of the up kernels and the pair launcher.
#pragma once

#include "cmoe_internal.h"
#include "launch.cuh"
#include "device_utils.cuh"
#include "tc_ptx.cuh"

namespace cmoe {
namespace tc2c {

using namespace ptx;

constexpr int BM = 128;          // rows per CTA tile (UMMA M per CTA)
constexpr int BK = 64;           // halves per K chunk: one 128-byte swizzle row
constexpr int KE = 64;           // width of the expanded rank index
constexpr uint32_t kTmemCols = 512;
constexpr size_t kSmemLimit = 232448;   // 227 KB

// all lanes wait; the warp agrees on the outcome so that it never diverges around .sync.aligned code
__device__ __forceinline__ bool warp_wait(uint32_t bar, uint32_t parity, volatile int* abort_flag) {
  const bool ok = mbar_wait(bar, parity, abort_flag);
  return __all_sync(0xffffffffu, ok);
}

__device__ __forceinline__ uint32_t pack_half2(float a, float b) {
  __half2 h = __floats2half2_rn(a, b);
  return *reinterpret_cast<uint32_t*>(&h);
}

__device__ __forceinline__ void st_shared_v4(uint32_t addr, uint32_t a, uint32_t b, uint32_t c, uint32_t d) {
  asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(addr), "r"(a), "r"(b), "r"(c), "r"(d) : "memory");
}

// GELU(u) ~ u/2 (1 + tanh(u (c1 + c2 u^2))) on two fp16 values at once, with c1, c2 fitted to the erf
// form (max abs deviation 2.7e-4 over the reals) and the hardware tanh; the error is of the size of the
// fp16 rounding of the stored activation.
__device__ __forceinline__ __half2 gelu_fast2(__half2 u) {
  const __half2 u2 = __hmul2(u, u);
  const __half2 w = __hfma2(u2, __float2half2_rn(0.03470089f), __float2half2_rn(0.80015708f));
  const __half2 z = __hmul2(u, w);
  uint32_t zi = *reinterpret_cast<const uint32_t*>(&z), ti;
  asm("tanh.approx.f16x2 %0, %1;" : "=r"(ti) : "r"(zi));
  const __half2 th = *reinterpret_cast<const __half2*>(&ti);
  const __half2 hu = __hmul2(u, __float2half2_rn(0.5f));
  return __hfma2(hu, th, hu);
}
__device__ __forceinline__ uint32_t h2u(__half2 h) { return *reinterpret_cast<uint32_t*>(&h); }
__device__ __forceinline__ __half2 u2h(uint32_t u) { return *reinterpret_cast<__half2*>(&u); }

// parameters of the up kernels (both tile widths)
struct Up2Params {
  const int* n_rows;
  const int* tile_cluster;   // per 256-row tile
  const int* tile_mask;      // per 128-row tile, two words
  const int* row_slot;
  const float* row_gate;
  const int* row_token;
  float* s_out;        // [rows][k][r] fp32, zeroed by the caller
  __half* abar;        // [rows][N]
  int* status;
  int KC, NT, N, K, k, r, log2r;
  int unit;            // N tiles per work unit (divides NT)
  int bshift;          // the base of cluster g is that of g >> bshift (expert halves or quarters share their cluster's base)
  __half* As_direct;   // [rows][KE] or null.  Not null: a unit is a whole row tile (unit == NT), so S is complete at its
                       // end and the gated rows p_j s_j go straight into the down kernel's operand (zeroed by the caller)
};

// launch as thread-block clusters of two CTAs (grid = 2 x pairs)
template <typename... KArgs, typename... Args>
inline cudaError_t launch_pairs(void (*kern)(KArgs...), int grid, int threads, size_t smem, cudaStream_t st, Args... args) {
  return launch_chained(kern, dim3((unsigned)grid), dim3((unsigned)threads), smem, st, 2, args...);
}

// The tensor maps of the wide up kernel: x_perm and B1t as 3-D boxes of 64 halves x 128 rows x 2 K atoms,
// A0 / Ad [rows][KE] (128-row boxes), V1f (128-row boxes), U2f (32-row boxes).
struct UpWideMaps {
  const CUtensorMap *x3, *b13, *a0, *ad, *v1, *u2;
};

constexpr int BN_WIDE = 256;     // columns per tile of the wide up kernel

// tc2_up_wide.cu: h and the activations on 256 x 256 pair tiles (d_ff a multiple of 256)
cudaError_t launch_up_wide(bool has_r, int ksel, const UpWideMaps& maps, const Up2Params& p, int grid, cudaStream_t st);

}  // namespace tc2c
}  // namespace cmoe
