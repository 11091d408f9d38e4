// Expert similarity of the clustering step (Sec. 3.1, Eq. 2-4), sm_100a:
//
//   S_param[i][j] = <w_i, w_j> / (|w_i| |w_j|)      w_i = expert i's weight matrix, flattened (Eq. 2)
//   S_task[i][j]  = <mu_i, mu_j> / (|mu_i| |mu_j|)  mu_i = expert i's activation centroid   (Eq. 3)
//   S             = alpha S_param + (1 - alpha) S_task                                       (Eq. 4)
//
// S_param is a tall-skinny Gram matrix: E rows of n = d_in d_out weights each, i.e. all of the layer's dense
// weights read once (HBM-bound) for E x E dot products.  gram_kernel streams W through shared memory with TMA
// and forms W W^T on the tensor cores (tcgen05, kind::tf32: the fp32 weights are used as they lie in memory,
// with the mantissa cut to 10 bits; A and B operand are the SAME shared-memory tile), every CTA over its own
// range of the flattened index, and adds its partial E x E block to the result with fp32 atomics.
// With few experts an MMA of E rows would spend its time reading operand rows that do not exist (the
// instruction spans 128 rows of shared memory whatever E is).  The K atoms of a stage lie in shared memory one
// after the other, `rows` (E rounded up to 8) rows of 128 bytes each, so 128 consecutive rows ARE a stack of
// 128 / rows atoms: one M = N = 128 instruction multiplies the whole stack by itself, the diagonal blocks of the
// result are the Gram contributions of the stacked atoms (summed by the epilogue), the off-diagonal blocks mix
// different slices of the flattened index and are ignored.  Three quarters of those flops are wasted at E = 32;
// the operand bytes read per weight fall by the stack height, and that is what bounds the kernel.
// The norms are the diagonal.  S_task is E x E dot products of length d on CUDA cores.  One block then
// normalises both and forms S.
// Every device wait is bounded; on expiry the kernel leaves its loops, frees its tensor memory and, when the
// caller gave a status word, stores CMOE_ERR_TIMEOUT there.
#include "cmoe_internal.h"
#include "launch.cuh"
#include "device_utils.cuh"
#include "tc_ptx.cuh"

namespace cmoe {

namespace {

using namespace ptx;

constexpr int GR_THREADS = 256;                  // warp 0 TMA, 1 MMA, 2 tensor-memory allocation, 4..7 epilogue
constexpr int GR_STAGES = 6;
constexpr uint32_t GR_STAGE_BYTES = 32768;
constexpr uint32_t GR_ATOM_COLS = 32;            // floats per K atom: one 128-byte swizzle row
constexpr uint32_t GR_TMEM_COLS = 128;
// the MMA spans 128 operand rows whatever E is: the rows past the loaded ones are read (and their accumulator
// lanes ignored), so the ring is followed by as many bytes as one atom of 128 rows
constexpr uint32_t GR_PAD = 128 * 128;
constexpr size_t GR_SMEM = 1024 + (size_t)GR_STAGES * GR_STAGE_BYTES + GR_PAD + 256;

struct GramParams {
  float* gram;            // [E][E], zeroed by the caller
  int* status;            // may be null
  int E;
  int rows;               // E rounded up to 8: rows per loaded atom
  int stack;              // atoms multiplied by one instruction: 128 / rows (rounded down)
  int KA;                 // atoms per stage, a multiple of stack
  long long n_stages;     // stages over the whole flattened index
};

// Instruction descriptor of kind::tf32: tf32 A and B (both K-major), fp32 accumulator, M x N tile.
__host__ __device__ constexpr uint32_t idesc_tf32(int M, int N) {
  return (1u << 4) | (2u << 7) | (2u << 10) | ((uint32_t)(N >> 3) << 17) | ((uint32_t)(M >> 4) << 24);
}
// D[tmem] (+)= A[smem] * B[smem]^T, fp32 operands read as tf32 (K = 8 per instruction), fp32 accumulate
__device__ __forceinline__ void umma_tf32(uint32_t d_tmem, uint64_t adesc, uint64_t bdesc, uint32_t idesc,
                                          uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::tf32 [%0], %1, %2, %3, p;\n\t}"
      ::"r"(d_tmem), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate) : "memory");
}

__global__ void __launch_bounds__(GR_THREADS, 1)
gram_kernel(const __grid_constant__ CUtensorMap tmW, const GramParams p) {
  extern __shared__ uint8_t smem_raw[];
  const uint32_t raw = smem_u32(smem_raw);
  const uint32_t base = (raw + 1023u) & ~1023u;
  uint8_t* sm = smem_raw + (base - raw);
  uint64_t* bars = reinterpret_cast<uint64_t*>(sm + (size_t)GR_STAGES * GR_STAGE_BYTES + GR_PAD);
  const uint32_t full0 = smem_u32(bars), empty0 = smem_u32(bars + 8), tfull = smem_u32(bars + 16);
  uint32_t* tmem_holder = reinterpret_cast<uint32_t*>(bars + 17);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_holder + 1);
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

  if (threadIdx.x == 0) {
    for (int s = 0; s < GR_STAGES; ++s) { mbar_init(full0 + 8 * s, 1); mbar_init(empty0 + 8 * s, 1); }
    mbar_init(tfull, 1);
    *abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 2) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;"
                 ::"r"(smem_u32(tmem_holder)), "r"(GR_TMEM_COLS) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_holder;

  // This CTA's stages: s0, s0 + grid, s0 + 2 grid, ...  Dealt round-robin, the CTAs of the launch read, at any
  // time, one contiguous window of every expert's row between them.
  const long long s0 = blockIdx.x, s1 = p.n_stages, sstep = gridDim.x;
  const uint32_t atom_bytes = (uint32_t)p.rows * 128u, stage_bytes = atom_bytes * (uint32_t)p.KA;
  bool failed = false;

  if (warp == 0) {
    if (lane == 0) {
      uint32_t s = 0, ph = 0;
      for (long long st = s0; st < s1; st += sstep) {
        if (!mbar_wait(empty0 + 8 * s, ph ^ 1u, abort_flag)) { failed = true; break; }
        mbar_expect_tx(full0 + 8 * s, stage_bytes);
        // KA atoms of 32 floats x `rows` experts; past the end of the flattened index the fill value (zero)
        tma_load_3d(base + s * GR_STAGE_BYTES, &tmW, full0 + 8 * s, 0, 0, (int)(st * p.KA));
        if (++s == GR_STAGES) { s = 0; ph ^= 1u; }
      }
    }
  } else if (warp == 1) {
    if (lane == 0 && s1 > s0) {
      const int N = (p.stack * p.rows + 15) & ~15;
      const uint32_t idesc = idesc_tf32(128, N);
      uint32_t s = 0, ph = 0;
      for (long long st = s0; st < s1; st += sstep) {
        if (!mbar_wait(full0 + 8 * s, ph, abort_flag)) { failed = true; break; }
        tc_fence_after();
        const uint64_t desc0 = umma_desc(base + s * GR_STAGE_BYTES);      // A and B are the same tile
        for (int a = 0; a < p.KA; a += p.stack) {                            // a stack of atoms per instruction
          const uint64_t desc = desc0 + (uint64_t)((atom_bytes >> 4) * (uint32_t)a);
#pragma unroll
          for (int ks = 0; ks < 4; ++ks)                                    // 8 floats = 32 bytes per step
            umma_tf32(tmem_base, desc + 2 * ks, desc + 2 * ks, idesc, (st != s0 || a != 0 || ks != 0) ? 1u : 0u);
        }
        umma_commit(empty0 + 8 * s);
        if (++s == GR_STAGES) { s = 0; ph ^= 1u; }
      }
      if (!failed) umma_commit(tfull);
    }
  } else if (warp >= 4 && s1 > s0) {
    // epilogue: accumulator lane = row e of stacked atom a; its Gram contribution is the diagonal block, columns
    // a rows .. a rows + E - 1, added to the result
    const int q = warp & 3;
    const bool ok = mbar_wait(tfull, 0, abort_flag);
    if (!__all_sync(0xffffffffu, ok)) {
      failed = true;
    } else if (q * 32 < p.stack * p.rows) {
      tc_fence_after();
      const int l = q * 32 + lane;
      const int a = l / p.rows, e = l - a * p.rows;
      const bool mine = a < p.stack && e < p.E;
      const int c_lo = a * p.rows;
      const uint32_t taddr = tmem_base + ((uint32_t)(q * 32) << 16);
      const int ncol = p.stack * p.rows;
      for (int j0 = 0; j0 < ncol; j0 += 16) {
        uint32_t v[16];
        tmem_ld16_nowait(taddr + j0, v);
        tmem_ld_wait();
        if (mine) {
#pragma unroll
          for (int j = 0; j < 16; ++j) {
            const int c = j0 + j - c_lo;
            if (c >= 0 && c < p.E) atomicAdd(p.gram + (size_t)e * p.E + c, __uint_as_float(v[j]));
          }
        }
      }
    }
  }

  if (failed) {
    *abort_flag = 1;
    if (p.status) atomicExch(p.status, (int)CMOE_ERR_TIMEOUT);
  }
  __syncthreads();
  if (*abort_flag) {
    const long long t0 = clock64();
    while (clock64() - t0 < 400000ll) { }       // let copies already issued land
    __syncthreads();
  }
  tc_fence_after();
  if (warp == 2)
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(GR_TMEM_COLS) : "memory");
}

// raw dot products of the centroids: a warp per pair (i, j), lanes over the features
__global__ void __launch_bounds__(256)
centroid_dots_kernel(const float* __restrict__ mu, int E, int d, float* __restrict__ out) {
  const int i = blockIdx.x, warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int j = blockIdx.y * (blockDim.x >> 5) + warp;
  if (j >= E) return;
  const float* mi = mu + (size_t)i * d;
  const float* mj = mu + (size_t)j * d;
  float acc = 0.f;
  for (int c = lane; c < d; c += 32) acc = fmaf(mi[c], mj[c], acc);
  acc = warp_sum(acc);
  if (lane == 0) out[(size_t)i * E + j] = acc;
}

// One block: raw Gram matrices -> cosine similarities (in place), then the fused score.  A vector of norm zero has
// similarity 0 to every other vector and 1 to itself.
__global__ void __launch_bounds__(1024)
similarity_finish_kernel(int E, float alpha, float* __restrict__ S_param, float* __restrict__ S_task, float* __restrict__ S) {
  __shared__ float dp[128], dt[128];
  for (int i = threadIdx.x; i < E; i += blockDim.x) {
    dp[i] = S_param ? S_param[(size_t)i * E + i] : 0.f;
    dt[i] = S_task ? S_task[(size_t)i * E + i] : 0.f;
  }
  __syncthreads();
  for (int idx = threadIdx.x; idx < E * E; idx += blockDim.x) {
    const int i = idx / E, j = idx - i * E;
    float sp = 0.f, stk = 0.f;
    if (S_param) {
      const float nn = dp[i] * dp[j];
      sp = nn > 0.f ? S_param[idx] * rsqrtf(nn) : (i == j ? 1.f : 0.f);
      if (i == j && nn > 0.f) sp = 1.f;
      S_param[idx] = sp;
    }
    if (S_task) {
      const float nn = dt[i] * dt[j];
      stk = nn > 0.f ? S_task[idx] * rsqrtf(nn) : (i == j ? 1.f : 0.f);
      if (i == j && nn > 0.f) stk = 1.f;
      S_task[idx] = stk;
    }
    if (S) S[idx] = alpha * sp + (1.f - alpha) * stk;
  }
}

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*,
                                  CUtensorMapInterleave, CUtensorMapSwizzle, CUtensorMapL2promotion,
                                  CUtensorMapFloatOOBfill);

EncodeTiledFn get_encode() {
  void* ptr = nullptr;
  cudaDriverEntryPointQueryResult qres;
  if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &ptr, cudaEnableDefault, &qres) != cudaSuccess ||
      qres != cudaDriverEntryPointSuccess)
    return nullptr;
  return reinterpret_cast<EncodeTiledFn>(ptr);
}

}  // namespace
}  // namespace cmoe

using namespace cmoe;

extern "C" int cmoe_expert_similarity(const cmoe_similarity_desc* q, void* cuda_stream) {
  if (!q) return CMOE_ERR_INVALID_ARG;
  const int E = q->E;
  if (E < 1 || E > 128 || !(q->alpha >= 0.f && q->alpha <= 1.f)) return CMOE_ERR_INVALID_ARG;
  if (q->W && (!q->S_param || q->n <= 0 || q->n % 32 != 0 || (reinterpret_cast<uintptr_t>(q->W) & 15))) return CMOE_ERR_INVALID_ARG;
  if (q->mu && (!q->S_task || q->d <= 0)) return CMOE_ERR_INVALID_ARG;
  if (q->S && (!q->W || !q->mu)) return CMOE_ERR_INVALID_ARG;
  if (!q->W && !q->mu) return CMOE_ERR_INVALID_ARG;
  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
  if (q->W) {
    EncodeTiledFn enc = get_encode();
    if (!enc) return CMOE_ERR_CUDA;
    GramParams p{};
    p.gram = q->S_param; p.status = q->status; p.E = E;
    p.rows = (E + 7) & ~7;
    p.stack = 128 / p.rows;
    p.KA = (int)(GR_STAGE_BYTES / ((uint32_t)p.rows * 128u)) / p.stack * p.stack;      // 32 KB stages, whole stacks
    const long long atoms = q->n / GR_ATOM_COLS;
    p.n_stages = (atoms + p.KA - 1) / p.KA;
    CUtensorMap map;
    cuuint64_t gdim[3] = {GR_ATOM_COLS, (cuuint64_t)E, (cuuint64_t)atoms};
    cuuint64_t gstride[2] = {(cuuint64_t)q->n * 4, (cuuint64_t)GR_ATOM_COLS * 4};
    cuuint32_t box[3] = {GR_ATOM_COLS, (cuuint32_t)p.rows, (cuuint32_t)p.KA};
    cuuint32_t estr[3] = {1, 1, 1};
    if (enc(&map, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 3, const_cast<float*>(q->W), gdim, gstride, box, estr,
            CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
      return CMOE_ERR_INVALID_ARG;
    int dev = 0, sms = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return CMOE_ERR_CUDA;
    if (cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess) return CMOE_ERR_CUDA;
    static std::atomic<unsigned long long> smem_set{0};
    if (ensure_dynamic_smem(gram_kernel, GR_SMEM, smem_set) != cudaSuccess) return CMOE_ERR_CUDA;
    if (cudaMemsetAsync(q->S_param, 0, sizeof(float) * (size_t)E * E, st) != cudaSuccess) return CMOE_ERR_CUDA;
    const int grid = (int)(p.n_stages < sms ? p.n_stages : sms);
    gram_kernel<<<grid, GR_THREADS, GR_SMEM, st>>>(map, p);
    if (cudaGetLastError() != cudaSuccess) return CMOE_ERR_CUDA;
  }
  if (q->mu) {
    centroid_dots_kernel<<<dim3(E, (E + 7) / 8), 256, 0, st>>>(q->mu, E, q->d, q->S_task);
    if (cudaGetLastError() != cudaSuccess) return CMOE_ERR_CUDA;
  }
  similarity_finish_kernel<<<1, 1024, 0, st>>>(E, q->alpha, q->W ? q->S_param : nullptr, q->mu ? q->S_task : nullptr, q->S);
  return cudaGetLastError() == cudaSuccess ? CMOE_OK : CMOE_ERR_CUDA;
}
