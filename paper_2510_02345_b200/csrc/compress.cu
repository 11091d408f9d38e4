// Offline compressor (Sec. 3.2, Eq. 6-7; Sec. 3.4): E dense expert matrices -> the layer's stored form.
//
//   Eq. 6     W_base^g = mean of the cluster's experts, stored as fp16
//   Eq. 7     Delta W_e = W_e - W_base^g (against the base as stored)  ~  A_e B_e^T, rank r: the truncated SVD, here by
//             a randomised range finder with subspace iteration (Halko, Martinsson, Tropp 2011, Alg. 4.4 / 5.1):
//               Y = R Omega;  Q = orth(Y);  q times { Z = orth(R^T Q);  Q = orth(R Z) };
//               Z = R^T Q  (so that  Q^T R = Z^T);  Z^T Z = Ut Lambda Ut^T  (Jacobi);  sigma = sqrt(Lambda)
//               A = Q Ut_r sqrt(Sigma_r),   B^T = Sigma_r^(-1/2) Ut_r^T Z^T          (A B^T = Q Ut_r Ut_r^T Q^T R)
//             The Gaussian test matrices Omega are the caller's input (l = r + oversample columns per expert).
//   Sec. 3.4  A_e, B_e^T -> symmetric INT4, one fp16 scale per 32 consecutive elements of the flattened factor in the
//             descriptor's layouts U [E][r][d_in], V [E][d_out][r]; optional cosine gate (blocks below gamma: zeroed).
//
// All arithmetic is fp32 on CUDA cores: the work is a handful of tall-skinny products per expert (2 d_in d_out l
// flops each), done once per model, not per token.  One launch of every kernel covers all experts (grid.z / grid.x).
#include <cfloat>

#include "cmoe_internal.h"

namespace cmoe {

namespace {

constexpr int kMaxL = 48;          // r + oversample

__device__ __forceinline__ float block_sum(float v, float* sh) {
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, nw = (blockDim.x + 31) >> 5;
  __syncthreads();
  if (lane == 0) sh[warp] = v;
  __syncthreads();
  float t = 0.f;
  for (int w = 0; w < nw; ++w) t += sh[w];
  return t;
}

// base (fp16) of cluster g and the residuals of its K experts; norms[e] = {|dW|^2, <dW, B>, |B|^2 (per cluster), 0}
__global__ void __launch_bounds__(256)
base_residual_kernel(int K, long long n, const float* __restrict__ W, __half* __restrict__ B, float* __restrict__ R,
                     float* __restrict__ norms) {
  __shared__ float sh[32];
  const int g = blockIdx.y;
  float nb = 0.f, nd[kMaxK], ip[kMaxK];
#pragma unroll
  for (int i = 0; i < kMaxK; ++i) { nd[i] = 0.f; ip[i] = 0.f; }
  for (long long idx = (long long)blockIdx.x * blockDim.x + threadIdx.x; idx < n; idx += (long long)gridDim.x * blockDim.x) {
    float sum = 0.f;
    for (int i = 0; i < K; ++i) sum += W[((long long)g * K + i) * n + idx];
    const __half bh = __float2half_rn(sum / (float)K);
    B[(long long)g * n + idx] = bh;
    const float b = __half2float(bh);
    nb = fmaf(b, b, nb);
#pragma unroll
    for (int i = 0; i < kMaxK; ++i)
      if (i < K) {
        const float dw = W[((long long)g * K + i) * n + idx] - b;
        R[((long long)g * K + i) * n + idx] = dw;
        nd[i] = fmaf(dw, dw, nd[i]);
        ip[i] = fmaf(dw, b, ip[i]);
      }
  }
  const float tb = block_sum(nb, sh);
  for (int i = 0; i < K; ++i) {
    const float td = block_sum(nd[i], sh), ti = block_sum(ip[i], sh);
    if (threadIdx.x == 0) {
      atomicAdd(&norms[(g * K + i) * 4 + 0], td);
      atomicAdd(&norms[(g * K + i) * 4 + 1], ti);
      atomicAdd(&norms[(g * K + i) * 4 + 2], tb);
    }
  }
}

// C[e][m][n] = sum_k A_e(m, k) X[e][k][n], A_e(m, k) = A[e * sAe + m * sAm + k * sAk]; X row-major [Kd][N], N <= 48.
// A block computes 64 rows of C; a thread 4 rows x 3 columns (16 x 16 threads cover 64 x 48).
__global__ void __launch_bounds__(256)
skinny_gemm_kernel(int M, int Kd, int N, const float* __restrict__ A, long long sAe, long long sAm, long long sAk,
                   const float* __restrict__ X, float* __restrict__ C) {
  __shared__ float As[16][65];
  __shared__ float Xs[16][kMaxL];
  const int e = blockIdx.z, m0 = blockIdx.x * 64;
  const float* Ae = A + (long long)e * sAe;
  const float* Xe = X + (long long)e * Kd * N;
  const int tx = threadIdx.x & 15, ty = threadIdx.x >> 4;
  float acc[4][3];
#pragma unroll
  for (int i = 0; i < 4; ++i)
#pragma unroll
    for (int j = 0; j < 3; ++j) acc[i][j] = 0.f;
  for (int k0 = 0; k0 < Kd; k0 += 16) {
    // the tile of A: 64 x 16, read along whichever of m, k is contiguous
    for (int i = threadIdx.x; i < 64 * 16; i += 256) {
      int mm, kk;
      if (sAk == 1) { kk = i & 15; mm = i >> 4; } else { mm = i & 63; kk = i >> 6; }
      const int m = m0 + mm, k = k0 + kk;
      As[kk][mm] = (m < M && k < Kd) ? Ae[m * sAm + k * sAk] : 0.f;
    }
    for (int i = threadIdx.x; i < 16 * N; i += 256) {
      const int kk = i / N, nn = i - kk * N;
      Xs[kk][nn] = (k0 + kk < Kd) ? Xe[(long long)(k0 + kk) * N + nn] : 0.f;
    }
    __syncthreads();
#pragma unroll
    for (int kk = 0; kk < 16; ++kk) {
      float a[4], x[3];
#pragma unroll
      for (int i = 0; i < 4; ++i) a[i] = As[kk][ty * 4 + i];
#pragma unroll
      for (int j = 0; j < 3; ++j) x[j] = (tx * 3 + j < N) ? Xs[kk][tx * 3 + j] : 0.f;
#pragma unroll
      for (int i = 0; i < 4; ++i)
#pragma unroll
        for (int j = 0; j < 3; ++j) acc[i][j] = fmaf(a[i], x[j], acc[i][j]);
    }
    __syncthreads();
  }
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    const int m = m0 + ty * 4 + i;
    if (m >= M) continue;
#pragma unroll
    for (int j = 0; j < 3; ++j)
      if (tx * 3 + j < N) C[((long long)e * M + m) * N + tx * 3 + j] = acc[i][j];
  }
}

// Orthonormalise the columns of Y[e] ([n][l] row-major) in place: column by column, classical Gram-Schmidt applied
// twice (as stable as modified Gram-Schmidt, and each pass is one sweep over the rows).  A column that is (numerically)
// in the span of the earlier ones - the residual had rank below l - becomes zero.
__global__ void __launch_bounds__(1024)
orth_kernel(int n, int l, float* __restrict__ Yall) {
  __shared__ float sh[32];
  __shared__ float dots[kMaxL];
  float* Y = Yall + (long long)blockIdx.x * n * l;
  for (int j = 0; j < l; ++j) {
    float norm0 = 0.f;
    for (int pass = 0; pass < 2; ++pass) {
      // dots[k] = <y_k, y_j> for k < j, and |y_j|^2 (index j)
      for (int k = 0; k <= j; ++k) {
        float part = 0.f;
        for (int i = threadIdx.x; i < n; i += blockDim.x) part = fmaf(Y[(long long)i * l + k], Y[(long long)i * l + j], part);
        const float t = block_sum(part, sh);
        if (threadIdx.x == 0) dots[k] = t;
      }
      __syncthreads();
      if (pass == 0) norm0 = dots[j];
      for (int i = threadIdx.x; i < n; i += blockDim.x) {
        float v = Y[(long long)i * l + j];
        for (int k = 0; k < j; ++k) v = fmaf(-dots[k], Y[(long long)i * l + k], v);
        Y[(long long)i * l + j] = v;
      }
      __syncthreads();
    }
    float part = 0.f;
    for (int i = threadIdx.x; i < n; i += blockDim.x) { const float v = Y[(long long)i * l + j]; part = fmaf(v, v, part); }
    const float nn = block_sum(part, sh);
    const float inv = (nn > 1e-10f * norm0 && nn > 0.f) ? rsqrtf(nn) : 0.f;
    for (int i = threadIdx.x; i < n; i += blockDim.x) Y[(long long)i * l + j] *= inv;
    __syncthreads();
  }
}

// Symmetric eigen-decomposition of M[e] (l x l, l <= 48) by cyclic Jacobi rotations; eigenvalues sorted descending.
// Out: Ut[e][a][j] = component a of eigenvector j, sig[e][j] = sqrt(max(lambda_j, 0)).  One block of 64 threads.
__global__ void __launch_bounds__(64)
jacobi_kernel(int l, const float* __restrict__ Mall, float* __restrict__ Utall, float* __restrict__ sigall) {
  __shared__ float M[kMaxL][kMaxL + 1];
  __shared__ float V[kMaxL][kMaxL + 1];
  __shared__ float cs[2];
  __shared__ int order[kMaxL];
  const int e = blockIdx.x, t = threadIdx.x;
  for (int i = t; i < l * l; i += blockDim.x) { M[i / l][i % l] = Mall[(long long)e * l * l + i]; V[i / l][i % l] = (i / l == i % l) ? 1.f : 0.f; }
  __syncthreads();
  for (int sweep = 0; sweep < 30; ++sweep) {
    float off = 0.f;
    if (t == 0) { for (int a = 0; a < l; ++a) for (int b = a + 1; b < l; ++b) off += M[a][b] * M[a][b]; cs[0] = off; }
    __syncthreads();
    float diag = 0.f;
    for (int a = 0; a < l; ++a) diag += M[a][a] * M[a][a];
    if (cs[0] <= 1e-14f * diag) break;
    __syncthreads();
    for (int p = 0; p < l - 1; ++p)
      for (int q = p + 1; q < l; ++q) {
        if (t == 0) {
          const float apq = M[p][q];
          float c = 1.f, s = 0.f;
          if (fabsf(apq) > 1e-30f) {
            const float tau = (M[q][q] - M[p][p]) / (2.f * apq);
            const float tt = (tau >= 0.f ? 1.f : -1.f) / (fabsf(tau) + sqrtf(1.f + tau * tau));
            c = rsqrtf(1.f + tt * tt);
            s = tt * c;
          }
          cs[0] = c; cs[1] = s;
        }
        __syncthreads();
        const float c = cs[0], s = cs[1];
        if (t < l) {       // columns p, q of M and V
          const float mp = M[t][p], mq = M[t][q];
          M[t][p] = c * mp - s * mq; M[t][q] = s * mp + c * mq;
          const float vp = V[t][p], vq = V[t][q];
          V[t][p] = c * vp - s * vq; V[t][q] = s * vp + c * vq;
        }
        __syncthreads();
        if (t < l) {       // rows p, q of M
          const float mp = M[p][t], mq = M[q][t];
          M[p][t] = c * mp - s * mq; M[q][t] = s * mp + c * mq;
        }
        __syncthreads();
      }
  }
  __syncthreads();
  if (t == 0) {            // selection sort of the diagonal, descending
    bool used[kMaxL];
    for (int a = 0; a < l; ++a) used[a] = false;
    for (int j = 0; j < l; ++j) {
      int best = -1;
      for (int a = 0; a < l; ++a) if (!used[a] && (best < 0 || M[a][a] > M[best][best])) best = a;
      used[best] = true;
      order[j] = best;
    }
  }
  __syncthreads();
  for (int i = t; i < l * l; i += blockDim.x) { const int a = i / l, j = i % l; Utall[(long long)e * l * l + i] = V[a][order[j]]; }
  if (t < l) sigall[(long long)e * l + t] = sqrtf(fmaxf(M[order[t]][order[t]], 0.f));
}

// A[e][i][j] = sqrt(sigma_j) sum_a Q[e][i][a] Ut[e][a][j];   Bt[e][j][c] = sigma_j^(-1/2) sum_a Ut[e][a][j] Zt[e][c][a]
__global__ void __launch_bounds__(256)
factors_kernel(int d_in, int d_out, int l, int r, const float* __restrict__ Q, const float* __restrict__ Zt,
               const float* __restrict__ Ut, const float* __restrict__ sig, float* __restrict__ A, float* __restrict__ Bt) {
  const int e = blockIdx.y;
  const long long idx = (long long)blockIdx.x * blockDim.x + threadIdx.x;
  const float* U = Ut + (long long)e * l * l;
  if (idx < (long long)d_in * r) {
    const int i = (int)(idx / r), j = (int)(idx - (long long)i * r);
    float acc = 0.f;
    for (int a = 0; a < l; ++a) acc = fmaf(Q[((long long)e * d_in + i) * l + a], U[a * l + j], acc);
    A[((long long)e * d_in + i) * r + j] = acc * sqrtf(sig[(long long)e * l + j]);
  } else if (idx < (long long)d_in * r + (long long)r * d_out) {
    const long long k = idx - (long long)d_in * r;
    const int j = (int)(k / d_out), c = (int)(k - (long long)j * d_out);
    const float s = sig[(long long)e * l + j];
    float acc = 0.f;
    for (int a = 0; a < l; ++a) acc = fmaf(U[a * l + j], Zt[((long long)e * d_out + c) * l + a], acc);
    Bt[((long long)e * r + j) * d_out + c] = s > 1e-20f ? acc * rsqrtf(s) : 0.f;
  }
}

// norms[e][3] += |R_e - A_e Bt_e|^2
__global__ void __launch_bounds__(256)
error_kernel(int d_in, int d_out, int r, const float* __restrict__ R, const float* __restrict__ A,
             const float* __restrict__ Bt, float* __restrict__ norms) {
  __shared__ float sh[32];
  const int e = blockIdx.y;
  const long long n = (long long)d_in * d_out;
  float part = 0.f;
  for (long long idx = (long long)blockIdx.x * blockDim.x + threadIdx.x; idx < n; idx += (long long)gridDim.x * blockDim.x) {
    const int i = (int)(idx / d_out), c = (int)(idx - (long long)i * d_out);
    float v = R[(long long)e * n + idx];
    for (int j = 0; j < r; ++j) v = fmaf(-A[((long long)e * d_in + i) * r + j], Bt[((long long)e * r + j) * d_out + c], v);
    part = fmaf(v, v, part);
  }
  const float t = block_sum(part, sh);
  if (threadIdx.x == 0) atomicAdd(&norms[e * 4 + 3], t);
}

// cosine, the gate, the relative error and the singular values that are reported
__global__ void finish_kernel(int E, int l, int r, float gamma, const float* __restrict__ norms, const float* __restrict__ sig,
                              int* __restrict__ pruned, float* __restrict__ cosine, float* __restrict__ rel_err,
                              float* __restrict__ sigma_out) {
  const int e = blockIdx.x * blockDim.x + threadIdx.x;
  if (e >= E) return;
  const float nd = norms[e * 4], ip = norms[e * 4 + 1], nb = norms[e * 4 + 2], er = norms[e * 4 + 3];
  const float cs = (nd > 0.f && nb > 0.f) ? ip * rsqrtf(nd) * rsqrtf(nb) : 0.f;
  pruned[e] = (gamma > 0.f && cs < gamma) ? 1 : 0;
  if (cosine) cosine[e] = cs;
  if (rel_err) rel_err[e] = nd > 0.f ? sqrtf(er / nd) : 0.f;
  if (sigma_out) for (int j = 0; j < r; ++j) sigma_out[e * r + j] = sig[(long long)e * l + j];
}

// One scale group (32 consecutive elements of the flattened factor, stored layout) per thread:
// scale = fp16(absmax / 7), code = clamp(rint(w / scale), -8, 7), even flat index in the low nibble.
// which = 0: U [E][r][d_in] from A [E][d_in][r];  which = 1: V [E][d_out][r] from Bt [E][r][d_out];
// which = 2: the source is already in the stored layout (the stand-alone quantiser).
__global__ void __launch_bounds__(256)
quantize_kernel(int which, long long groups_per_expert, int dim, int r, const float* __restrict__ src,
                const int* __restrict__ pruned, uint8_t* __restrict__ q, __half* __restrict__ s) {
  const int e = blockIdx.y;
  const long long grp = (long long)blockIdx.x * blockDim.x + threadIdx.x;
  if (grp >= groups_per_expert) return;
  float w[32];
  const long long flat0 = grp * 32;
#pragma unroll
  for (int n = 0; n < 32; ++n) {
    const long long f = flat0 + n;
    float v;
    if (which == 0)      { const long long j = f / dim, i = f - j * dim; v = src[((long long)e * dim + i) * r + j]; }          // U[j][i] = A[i][j]
    else if (which == 1) { const long long c = f / r, j = f - c * r;     v = src[((long long)e * r + j) * dim + c]; }          // V[c][j] = Bt[j][c]
    else                 { v = src[(long long)e * groups_per_expert * 32 + f]; }
    w[n] = v;
  }
  float amax = 0.f;
#pragma unroll
  for (int n = 0; n < 32; ++n) amax = fmaxf(amax, fabsf(w[n]));
  __half sc = __float2half_rn(amax / 7.0f);
  if (pruned && pruned[e]) sc = __float2half_rn(0.f);
  const float sf = __half2float(sc);
  uint32_t words[4] = {0, 0, 0, 0};
  if (sf > 0.f) {
#pragma unroll
    for (int n = 0; n < 32; ++n) {
      float c = rintf(w[n] / sf);
      c = fminf(fmaxf(c, -8.f), 7.f);
      words[n >> 3] |= ((uint32_t)((int)c & 0xF)) << (4 * (n & 7));
    }
  }
  reinterpret_cast<uint4*>(q)[(long long)e * groups_per_expert + grp] = make_uint4(words[0], words[1], words[2], words[3]);
  s[(long long)e * groups_per_expert + grp] = sc;
}

size_t align256(size_t v) { return (v + 255) / 256 * 256; }

struct Plan {
  size_t R, Y, Z, M, Ut, sig, norms, A, Bt, pruned, total;
};

Plan plan_ws(const cmoe_compress_desc* d, int l) {
  Plan p{};
  const size_t E = d->E, di = d->d_in, dout = d->d_out, r = d->r;
  size_t off = 0;
  auto take = [&](size_t bytes) { const size_t o = off; off = align256(off + bytes); return o; };
  p.R = take(4 * E * di * dout);
  p.Y = take(4 * E * di * l);
  p.Z = take(4 * E * dout * l);
  p.M = take(4 * E * l * l);
  p.Ut = take(4 * E * l * l);
  p.sig = take(4 * E * l);
  p.norms = take(4 * E * 4);
  p.A = take(4 * E * di * r);
  p.Bt = take(4 * E * r * dout);
  p.pruned = take(4 * E);
  p.total = off;
  return p;
}

int check_desc(const cmoe_compress_desc* d, int* l_out) {
  if (!d) return CMOE_ERR_INVALID_ARG;
  if (d->d_in <= 0 || d->d_out <= 0 || d->E <= 0 || d->G <= 0 || d->r <= 0 || d->oversample < 0 || d->power_iters < 0)
    return CMOE_ERR_INVALID_ARG;
  if (d->E % d->G) return CMOE_ERR_UNSUPPORTED_SHAPE;
  const int K = d->E / d->G, l = d->r + d->oversample;
  if (K > kMaxK || d->G > kMaxG) return CMOE_ERR_UNSUPPORTED_SHAPE;
  if (d->d_in % 32 || d->d_out % 32) return CMOE_ERR_UNSUPPORTED_SHAPE;
  if (!(d->r == 4 || d->r == 8 || d->r == 16 || d->r == 32)) return CMOE_ERR_UNSUPPORTED_SHAPE;
  if (l > kMaxL || l > d->d_in || l > d->d_out || d->power_iters > 8) return CMOE_ERR_UNSUPPORTED_SHAPE;
  *l_out = l;
  return CMOE_OK;
}

}  // namespace

}  // namespace cmoe

using namespace cmoe;

extern "C" int cmoe_compress_workspace_bytes(const cmoe_compress_desc* d, size_t* out_bytes) {
  int l = 0;
  if (!out_bytes) return CMOE_ERR_INVALID_ARG;
  const int rc = check_desc(d, &l);
  if (rc) return rc;
  *out_bytes = plan_ws(d, l).total;
  return CMOE_OK;
}

extern "C" int cmoe_compress(const cmoe_compress_desc* d, void* cuda_stream) {
  int l = 0;
  int rc = check_desc(d, &l);
  if (rc) return rc;
  if (!d->W || !d->omega || !d->B || !d->Uq || !d->Us || !d->Vq || !d->Vs || !d->workspace) return CMOE_ERR_INVALID_ARG;
  if ((reinterpret_cast<uintptr_t>(d->workspace) & 255) || (reinterpret_cast<uintptr_t>(d->Uq) & 15) ||
      (reinterpret_cast<uintptr_t>(d->Vq) & 15))
    return CMOE_ERR_INVALID_ARG;
  const Plan p = plan_ws(d, l);
  if (d->workspace_bytes < p.total) return CMOE_ERR_WORKSPACE_TOO_SMALL;
  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
  char* ws = static_cast<char*>(d->workspace);
  float* R = reinterpret_cast<float*>(ws + p.R);
  float* Y = reinterpret_cast<float*>(ws + p.Y);
  float* Z = reinterpret_cast<float*>(ws + p.Z);
  float* M = reinterpret_cast<float*>(ws + p.M);
  float* Ut = reinterpret_cast<float*>(ws + p.Ut);
  float* sig = reinterpret_cast<float*>(ws + p.sig);
  float* norms = reinterpret_cast<float*>(ws + p.norms);
  float* A = reinterpret_cast<float*>(ws + p.A);
  float* Bt = reinterpret_cast<float*>(ws + p.Bt);
  int* pruned = reinterpret_cast<int*>(ws + p.pruned);
  const int E = d->E, G = d->G, K = E / G, di = d->d_in, dout = d->d_out, r = d->r;
  const long long n = (long long)di * dout;
#define CK(expr) do { if ((expr) != cudaSuccess) return CMOE_ERR_CUDA; } while (0)
  CK(cudaMemsetAsync(norms, 0, sizeof(float) * (size_t)E * 4, st));
  base_residual_kernel<<<dim3(512, G), 256, 0, st>>>(K, n, d->W, reinterpret_cast<__half*>(d->B), R, norms);
  // R X with X [d_out][l]: A_e(m, k) = R[e][m][k];   R^T X with X [d_in][l]: A_e(m, k) = R[e][k][m]
  auto rx = [&](const float* X, float* C) {
    skinny_gemm_kernel<<<dim3((di + 63) / 64, 1, E), 256, 0, st>>>(di, dout, l, R, n, (long long)dout, 1ll, X, C);
  };
  auto rtx = [&](const float* X, float* C) {
    skinny_gemm_kernel<<<dim3((dout + 63) / 64, 1, E), 256, 0, st>>>(dout, di, l, R, n, 1ll, (long long)dout, X, C);
  };
  rx(d->omega, Y);
  orth_kernel<<<E, 1024, 0, st>>>(di, l, Y);
  for (int it = 0; it < d->power_iters; ++it) {
    rtx(Y, Z);
    orth_kernel<<<E, 1024, 0, st>>>(dout, l, Z);
    rx(Z, Y);
    orth_kernel<<<E, 1024, 0, st>>>(di, l, Y);
  }
  rtx(Y, Z);                                     // Z = R^T Q: Q^T R = Z^T
  // M = Z^T Z: A_e(m, k) = Z[e][k][m], X = Z[e]
  skinny_gemm_kernel<<<dim3(1, 1, E), 256, 0, st>>>(l, dout, l, Z, (long long)dout * l, 1ll, (long long)l, Z, M);
  jacobi_kernel<<<E, 64, 0, st>>>(l, M, Ut, sig);
  {
    const long long items = (long long)di * r + (long long)r * dout;
    factors_kernel<<<dim3((unsigned)((items + 255) / 256), E), 256, 0, st>>>(di, dout, l, r, Y, Z, Ut, sig, A, Bt);
  }
  error_kernel<<<dim3(256, E), 256, 0, st>>>(di, dout, r, R, A, Bt, norms);
  finish_kernel<<<(E + 127) / 128, 128, 0, st>>>(E, l, r, d->gamma, norms, sig, pruned, d->cosine, d->rel_err, d->sigma);
  {
    const long long gu = (long long)r * di / 32, gv = (long long)dout * r / 32;
    quantize_kernel<<<dim3((unsigned)((gu + 255) / 256), E), 256, 0, st>>>(0, gu, di, r, A, pruned, d->Uq, reinterpret_cast<__half*>(d->Us));
    quantize_kernel<<<dim3((unsigned)((gv + 255) / 256), E), 256, 0, st>>>(1, gv, dout, r, Bt, pruned, d->Vq, reinterpret_cast<__half*>(d->Vs));
  }
  if (d->pruned) CK(cudaMemcpyAsync(d->pruned, pruned, sizeof(int) * (size_t)E, cudaMemcpyDeviceToDevice, st));
  if (d->A_out) CK(cudaMemcpyAsync(d->A_out, A, sizeof(float) * (size_t)E * di * r, cudaMemcpyDeviceToDevice, st));
  if (d->Bt_out) CK(cudaMemcpyAsync(d->Bt_out, Bt, sizeof(float) * (size_t)E * r * dout, cudaMemcpyDeviceToDevice, st));
  CK(cudaGetLastError());
#undef CK
  return CMOE_OK;
}

extern "C" int cmoe_quantize_int4(const float* w, int64_t n, uint8_t* q, uint16_t* s, void* cuda_stream) {
  if (n < 0 || n % 32) return CMOE_ERR_INVALID_ARG;
  if (n == 0) return CMOE_OK;
  if (!w || !q || !s || (reinterpret_cast<uintptr_t>(q) & 15)) return CMOE_ERR_INVALID_ARG;
  const long long groups = n / 32;
  quantize_kernel<<<dim3((unsigned)((groups + 255) / 256), 1), 256, 0, static_cast<cudaStream_t>(cuda_stream)>>>(
      2, groups, 0, 0, w, nullptr, q, reinterpret_cast<__half*>(s));
  return cudaGetLastError() == cudaSuccess ? CMOE_OK : CMOE_ERR_CUDA;
}
