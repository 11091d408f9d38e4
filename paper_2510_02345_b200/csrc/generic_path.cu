// Generic CUDA-core path of the expert FFNs: works for every shape the descriptor allows and is
// the fallback for shapes the tensor-core and weight-streaming paths do not take (small d, odd
// ranks).  It uses the factored form of the text after Eq. 7 throughout and never forms W_e:
//
//   t_j   = x U1_e                    residual_t_kernel  (one warp per row and kept expert)
//   H     = x B1_g                    up kernel, shared by the row's k experts
//   h_j   = H + t_j V1_e ; a_j = GELU(h_j) ; abar = sum_j p_j a_j ; s_j = a_j U2_e
//   y     = abar B2_g + sum_j p_j s_j V2_e     down kernel (linear in a_j, so the base product
//                                              runs once on the gate-weighted sum)
#include "cmoe_internal.h"
#include "launch.cuh"
#include "device_utils.cuh"

namespace cmoe {

namespace {

constexpr int BM = 64, BN = 64, BK = 16;

// t[row][j][p] = sum_c x_perm[row][c] * deq(U1[e_j][p][c]);  lanes stride groups of 32 columns
__global__ void __launch_bounds__(256)
residual_t_kernel(int d, int k, int r, const int* __restrict__ n_rows,
                  const __half* __restrict__ x_perm, const int* __restrict__ row_slot,
                  const uint8_t* __restrict__ U1q, const __half* __restrict__ U1s,
                  float* __restrict__ t) {
  pdl_wait();
  const int lane = threadIdx.x & 31;
  const int wpb = blockDim.x >> 5;
  const int total = *n_rows * k;
  for (int item = blockIdx.x * wpb + (threadIdx.x >> 5); item < total; item += gridDim.x * wpb) {
    const int row = item / k;
    const int e = row_slot[item];
    const __half* xr = x_perm + (size_t)row * d;
    for (int p = 0; p < r; ++p) {
      const long long base = ((long long)e * r + p) * d;
      float acc = 0.f;
      for (int grp = lane; grp * 32 < d; grp += 32) {
        const uint4 pk = *reinterpret_cast<const uint4*>(U1q + ((base + grp * 32) >> 1));
        const float sc = __half2float(U1s[(base >> 5) + grp]);
        const uint32_t w[4] = {pk.x, pk.y, pk.z, pk.w};
        float part = 0.f;
#pragma unroll
        for (int q = 0; q < 4; ++q) {
          const uint4 xv = *reinterpret_cast<const uint4*>(xr + grp * 32 + q * 8);
          const __half* xh = reinterpret_cast<const __half*>(&xv);
#pragma unroll
          for (int n = 0; n < 8; ++n)
            part = fmaf(__half2float(xh[n]), (float)sext4((int)(w[q] >> (4 * n))), part);
        }
        acc = fmaf(part, sc, acc);
      }
      acc = warp_sum(acc);
      if (lane == 0) t[(size_t)item * r + p] = acc;
    }
  }
}

// One 64x64 tile of  A[rows][Kd] * Bt[g][cols][Kd]^T  in fp32 on CUDA cores.
// UP:   A = x_perm, Bt = B1t, epilogue = residual + GELU + gate-weighted sum + s partials
// DOWN: A = abar,   Bt = B2t, epilogue = rank-r update + un-permuting store
template <bool UP>
__global__ void __launch_bounds__(256)
ffn_tile_kernel(int Kd, int N, int K, int k, int r, int row_align,
                const int* __restrict__ n_rows, const int* __restrict__ tile_cluster,
                const __half* __restrict__ A, const __half* __restrict__ Bt,
                const int* __restrict__ row_slot, const float* __restrict__ row_gate,
                const int* __restrict__ row_token,
                const uint8_t* __restrict__ Vq, const __half* __restrict__ Vs,   // V1 (UP) / V2 (DOWN)
                const uint8_t* __restrict__ U2q, const __half* __restrict__ U2s, // UP only
                const float* __restrict__ coef,      // t (UP) / s (DOWN), [rows][k][r]
                float* __restrict__ s_out,           // UP only
                __half* __restrict__ out) {
  pdl_wait();          // abar [rows][N] (UP) / y [T][N] (DOWN)
  const int row0 = blockIdx.y * BM;
  if (row0 >= *n_rows) return;
  const int g = tile_cluster[row0 / row_align];
  const int col0 = blockIdx.x * BN;
  const __half* Bg = Bt + (size_t)g * N * Kd;

  __shared__ float As[BK][BM + 1];
  __shared__ float Bs[BK][BN + 1];
  const int tid = threadIdx.x;
  const int tx = tid & 15, ty = tid >> 4;
  const int lr = tid >> 2, lc = (tid & 3) * 4;   // loader: row/col of the tile, 4 reduction elements
  float acc[4][4];
#pragma unroll
  for (int i = 0; i < 4; ++i)
#pragma unroll
    for (int j = 0; j < 4; ++j) acc[i][j] = 0.f;

  for (int k0 = 0; k0 < Kd; k0 += BK) {
    {
      const uint2 av = *reinterpret_cast<const uint2*>(A + (size_t)(row0 + lr) * Kd + k0 + lc);
      const __half* ah = reinterpret_cast<const __half*>(&av);
#pragma unroll
      for (int i = 0; i < 4; ++i) As[lc + i][lr] = __half2float(ah[i]);
      uint2 bv = make_uint2(0, 0);
      if (col0 + lr < N) bv = *reinterpret_cast<const uint2*>(Bg + (size_t)(col0 + lr) * Kd + k0 + lc);
      const __half* bh = reinterpret_cast<const __half*>(&bv);
#pragma unroll
      for (int i = 0; i < 4; ++i) Bs[lc + i][lr] = __half2float(bh[i]);
    }
    __syncthreads();
#pragma unroll
    for (int kk = 0; kk < BK; ++kk) {
      float a[4], b[4];
#pragma unroll
      for (int i = 0; i < 4; ++i) a[i] = As[kk][ty * 4 + i];
#pragma unroll
      for (int j = 0; j < 4; ++j) b[j] = Bs[kk][tx * 4 + j];
#pragma unroll
      for (int i = 0; i < 4; ++i)
#pragma unroll
        for (int j = 0; j < 4; ++j) acc[i][j] = fmaf(a[i], b[j], acc[i][j]);
    }
    __syncthreads();
  }

  // epilogue: thread owns rows row0 + ty*4 + i, columns col0 + tx*4 + j
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    const int row = row0 + ty * 4 + i;
    if (UP) {
      float ab[4] = {0.f, 0.f, 0.f, 0.f};
      for (int j = 0; j < k; ++j) {
        const int e = row_slot[(size_t)row * k + j];
        const float gate = row_gate[(size_t)row * k + j];
        const float* tj = coef + ((size_t)row * k + j) * r;
        float a[4];
#pragma unroll
        for (int c = 0; c < 4; ++c) {
          const int col = col0 + tx * 4 + c;
          float h = acc[i][c];
          if (col < N)
            for (int p = 0; p < r; ++p)
              h = fmaf(tj[p], deq4(Vq, Vs, ((long long)e * N + col) * r + p), h);
          a[c] = (col < N) ? gelu_erf(h) : 0.f;
          ab[c] = fmaf(gate, a[c], ab[c]);
        }
        // s_j[p] += sum over this tile's columns of a_j * U2_e[p][col]; reduce over the 16 lanes of the row
        for (int p = 0; p < r; ++p) {
          float sp = 0.f;
#pragma unroll
          for (int c = 0; c < 4; ++c) {
            const int col = col0 + tx * 4 + c;
            if (col < N) sp = fmaf(a[c], deq4(U2q, U2s, ((long long)e * r + p) * N + col), sp);
          }
#pragma unroll
          for (int o = 8; o > 0; o >>= 1) sp += __shfl_xor_sync(0xffffffffu, sp, o);
          if (tx == 0) atomicAdd(&s_out[((size_t)row * k + j) * r + p], sp);
        }
      }
#pragma unroll
      for (int c = 0; c < 4; ++c) {
        const int col = col0 + tx * 4 + c;
        if (col < N) out[(size_t)row * N + col] = __float2half_rn(ab[c]);
      }
    } else {
      const int tok = row_token[row];
      float yv[4];
#pragma unroll
      for (int c = 0; c < 4; ++c) yv[c] = acc[i][c];
      for (int j = 0; j < k; ++j) {
        const int e = row_slot[(size_t)row * k + j];
        const float gate = row_gate[(size_t)row * k + j];
        const float* sj = coef + ((size_t)row * k + j) * r;
#pragma unroll
        for (int c = 0; c < 4; ++c) {
          const int col = col0 + tx * 4 + c;
          if (col < N) {
            float u = 0.f;
            for (int p = 0; p < r; ++p)
              u = fmaf(sj[p], deq4(Vq, Vs, ((long long)e * N + col) * r + p), u);
            yv[c] = fmaf(gate, u, yv[c]);
          }
        }
      }
      if (tok >= 0) {
#pragma unroll
        for (int c = 0; c < 4; ++c) {
          const int col = col0 + tx * 4 + c;
          if (col < N) out[(size_t)tok * N + col] = __float2half_rn(yv[c]);
        }
      }
    }
  }
}

}  // namespace

cudaError_t launch_residual_t(const Dims& D, const Weights& W, const Scratch& S, int T, cudaStream_t st) {
  if (D.r <= 0) return cudaSuccess;
  const int rows_bound = t_pad_bound(D, T);
  int blocks = (rows_bound * D.k + 7) / 8;
  const int cap = (D.sm_count > 0 ? D.sm_count : 148) * 16;      // grid-stride loop: a few resident rounds
  if (blocks > cap) blocks = cap;
  launch_chained(residual_t_kernel, dim3(blocks), dim3(256), 0, st, 1,
      D.d, D.k, D.r, S.n_rows, S.x_perm, S.row_slot, W.U1q,
                                            W.U1s, S.t);
  return cudaGetLastError();
}

cudaError_t launch_generic_ffn(const Dims& D, const Weights& W, const Scratch& S, int T, __half* y,
                               cudaStream_t st, cudaEvent_t* marks) {
  const int rows_bound = t_pad_bound(D, T);
  if (marks) cudaEventRecord(marks[0], st);
  cudaError_t e0 = launch_residual_t(D, W, S, T, st);
  if (e0 != cudaSuccess) return e0;
  if (marks) cudaEventRecord(marks[1], st);
  dim3 gu((D.d_ff + BN - 1) / BN, rows_bound / BM);
  launch_chained(ffn_tile_kernel<true>, dim3(gu), dim3(256), 0, st, 1,
      D.d, D.d_ff, D.K, D.k, D.r, D.row_align, S.n_rows,
                                            S.tile_cluster, S.x_perm, W.B1t, S.row_slot, S.row_gate,
                                            S.row_token, W.V1q, W.V1s, W.U2q, W.U2s, S.t, S.s, S.abar);
  if (marks) cudaEventRecord(marks[2], st);
  dim3 gd((D.d + BN - 1) / BN, rows_bound / BM);
  launch_chained(ffn_tile_kernel<false>, dim3(gd), dim3(256), 0, st, 1,
      D.d_ff, D.d, D.K, D.k, D.r, D.row_align, S.n_rows,
                                             S.tile_cluster, S.abar, W.B2t, S.row_slot, S.row_gate,
                                             S.row_token, W.V2q, W.V2s, nullptr, nullptr, S.s, nullptr,
                                             y);
  return cudaGetLastError();
}

}  // namespace cmoe
