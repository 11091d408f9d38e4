// Tensor-core path of the expert FFNs for large token counts (sm_100a): per-cluster grouped GEMMs
// on tcgen05 with TMEM accumulators, operands staged in shared memory by TMA.
//
//   up    H = x_perm B1_g (128 x BN tiles, fp16 x fp16 -> fp32 in TMEM), computed once per token and
//         shared by the token's k experts (text after Eq. 7); epilogue: h_j = H + t_j V1_e,
//         a_j = GELU(h_j), abar = sum_j p_j a_j (fp16), s_j += a_j U2_e (fp32 atomics)
//   down  y = abar B2_g + sum_j p_j s_j V2_e, stored un-permuted (fp16)
//
// One persistent CTA per SM, 192 threads: warp 0 = TMA producer (and TMEM allocator), warp 1 = MMA
// issuer (one elected lane), warps 2..5 = epilogue (each owns the 32 TMEM lanes of its quadrant).
// Shared-memory operand ring of `stages` K-chunks of 64 halves (128-byte swizzled rows), two TMEM
// accumulators so that the epilogue of a tile overlaps the main loop of the next one.  The INT4
// factor tiles of the tile's cluster are decoded once per tile into shared memory by the epilogue
// warps.  Every wait is bounded: on expiry the kernel records CMOE_ERR_TIMEOUT in the status word,
// all roles leave their loops, TMEM is freed and the kernel returns.
#include <cuda.h>

#include "cmoe_internal.h"
#include "launch.cuh"
#include "device_utils.cuh"

namespace cmoe {

namespace {

constexpr int BM = 128;         // rows per tile (UMMA M)
constexpr int BK = 64;          // halves per K chunk: one 128-byte swizzle row
constexpr int kThreads = 192;
constexpr int kMaxStages = 8;
constexpr uint32_t kTmemCols = 512;
constexpr long long kWaitLimitCycles = 4000000000ll;          // about 2 s of SM clocks
constexpr size_t kSmemLimit = 232448;                        // 227 KB

struct TcParams {
  const int* n_rows;
  const int* tile_cluster;
  const int* row_slot;
  const float* row_gate;
  const int* row_token;
  const uint8_t* Vq;  const __half* Vs;    // V1 (up) / V2 (down)
  const uint8_t* U2q; const __half* U2s;   // up only
  const float* coef;                       // t (up) / s (down): [rows][k][r]
  float* s_out;                            // up only
  __half* out;                             // abar [rows][N] (up) / y [T][N] (down)
  int* status;
  int Kd, N, K, stages;
};

// ---------------------------------------------------------------- PTX wrappers
__device__ __forceinline__ uint32_t smem_u32(const void* p) {
  return (uint32_t)__cvta_generic_to_shared(p);
}
__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ uint32_t mbar_try_wait(uint32_t bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
  return ok;
}
__device__ __forceinline__ unsigned long long global_ns() {
  unsigned long long t;
  asm volatile("mov.u64 %0, %globaltimer;" : "=l"(t));
  return t;
}
// Bounded wait: false if the time limit ran out or another role already gave up.
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile int* abort_flag) {
  if (mbar_try_wait(bar, parity)) return true;
  const long long t0 = clock64();      // the SM's own counter: reading the global timer costs about a microsecond
  uint32_t spins = 0;
  while (!mbar_try_wait(bar, parity)) {
    if ((++spins & 63u) == 0) {
      if (*abort_flag) return false;
      if (clock64() - t0 > kWaitLimitCycles) return false;
    }
  }
  return true;
}
__device__ __forceinline__ void tma_load_2d(uint32_t dst, const CUtensorMap* map, uint32_t bar, int x, int y) {
  asm volatile(
      "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4}], [%2];"
      ::"r"(dst), "l"(reinterpret_cast<uint64_t>(map)), "r"(bar), "r"(x), "r"(y) : "memory");
}
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void umma_f16(uint32_t d_tmem, uint64_t adesc, uint64_t bdesc, uint32_t idesc, uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
      ::"r"(d_tmem), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate) : "memory");
}
__device__ __forceinline__ void umma_commit(uint32_t bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void tmem_ld32(uint32_t taddr, uint32_t* v) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
      "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
      "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
      : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]), "=r"(v[4]), "=r"(v[5]), "=r"(v[6]), "=r"(v[7]),
        "=r"(v[8]), "=r"(v[9]), "=r"(v[10]), "=r"(v[11]), "=r"(v[12]), "=r"(v[13]), "=r"(v[14]), "=r"(v[15]),
        "=r"(v[16]), "=r"(v[17]), "=r"(v[18]), "=r"(v[19]), "=r"(v[20]), "=r"(v[21]), "=r"(v[22]), "=r"(v[23]),
        "=r"(v[24]), "=r"(v[25]), "=r"(v[26]), "=r"(v[27]), "=r"(v[28]), "=r"(v[29]), "=r"(v[30]), "=r"(v[31])
      : "r"(taddr) : "memory");
  asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
}
// named barrier over the 128 epilogue threads that also ANDs a predicate
__device__ __forceinline__ bool epi_all(bool ok) {
  uint32_t r;
  asm volatile(
      "{\n\t.reg .pred p, q;\n\tsetp.ne.u32 q, %1, 0;\n\t"
      "barrier.cta.red.and.pred p, 1, 128, q;\n\tselp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(r) : "r"((uint32_t)ok) : "memory");
  return r != 0;
}
__device__ __forceinline__ void epi_sync() { asm volatile("bar.sync 1, 128;" ::: "memory"); }

// K-major, 128-byte-swizzled shared-memory matrix descriptor: rows of 64 halves at a 128-byte
// pitch, 8-row groups 1024 bytes apart; descriptor version 1 (sm_100).
__device__ __forceinline__ uint64_t umma_desc(uint32_t saddr) {
  return (uint64_t)((saddr & 0x3FFFFu) >> 4) | (1ull << 16) | (64ull << 32) | (1ull << 46) | (2ull << 61);
}

// Decode 8 consecutive INT4 codes (one 32-bit word) times a scale into 8 halves.
__device__ __forceinline__ void decode8(uint32_t word, float scale, __half* out8) {
#pragma unroll
  for (int n = 0; n < 8; ++n) out8[n] = __float2half_rn((float)sext4((int)(word >> (4 * n))) * scale);
}

template <int BN, int R, int KSEL, bool UP>
__global__ void __launch_bounds__(kThreads, 1)
tc_ffn_kernel(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmB,
              const TcParams p) {
  extern __shared__ uint8_t smem_raw[];
  constexpr uint32_t A_BYTES = BM * BK * 2;
  constexpr uint32_t B_BYTES = BN * BK * 2;
  constexpr uint32_t STAGE_BYTES = A_BYTES + B_BYTES;
  constexpr uint32_t IDESC = (1u << 4) | ((uint32_t)(BN >> 3) << 17) | ((uint32_t)(BM >> 4) << 24);

  const uint32_t raw = smem_u32(smem_raw);
  const uint32_t base = (raw + 1023u) & ~1023u;
  uint8_t* sm = smem_raw + (base - raw);
  const int stages = p.stages;
  const int K = p.K;
  const uint32_t fac_bytes = (uint32_t)K * BN * R * 2;
  __half* vst = reinterpret_cast<__half*>(sm + (size_t)stages * STAGE_BYTES);              // [K][BN][R]
  __half* ust = reinterpret_cast<__half*>(sm + (size_t)stages * STAGE_BYTES + fac_bytes);  // up only
  uint8_t* after = sm + (size_t)stages * STAGE_BYTES + (UP ? 2 : 1) * fac_bytes;
  uint64_t* bars = reinterpret_cast<uint64_t*>(after);
  const uint32_t full0 = smem_u32(bars), empty0 = smem_u32(bars + kMaxStages);
  const uint32_t tfull0 = smem_u32(bars + 2 * kMaxStages), tempty0 = smem_u32(bars + 2 * kMaxStages + 2);
  uint32_t* tmem_holder = reinterpret_cast<uint32_t*>(bars + 2 * kMaxStages + 4);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_holder + 1);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

  if (threadIdx.x == 0) {
    for (int s = 0; s < stages; ++s) { mbar_init(full0 + 8 * s, 1); mbar_init(empty0 + 8 * s, 1); }
    for (int a = 0; a < 2; ++a) { mbar_init(tfull0 + 8 * a, 1); mbar_init(tempty0 + 8 * a, 4); }
    *abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 0) {
    __syncwarp();
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;"
                 ::"r"(smem_u32(tmem_holder)), "r"(kTmemCols) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_holder;

  const int n_mt = *p.n_rows / BM;
  const int NT = p.N / BN;
  const int total = n_mt * NT;
  const int KC = p.Kd / BK;
  bool failed = false;

  if (warp == 0) {
    // ---------------- TMA producer
    if (lane == 0) {
      uint32_t it = 0;
      for (int w = blockIdx.x; w < total && !failed; w += gridDim.x) {
        const int mt = w / NT, nt = w % NT;
        const int g = p.tile_cluster[mt];
        for (int kc = 0; kc < KC; ++kc, ++it) {
          const uint32_t s = it % stages, ph = (it / stages) & 1u;
          if (!mbar_wait(empty0 + 8 * s, ph ^ 1u, abort_flag)) { failed = true; break; }
          const uint32_t a_dst = base + s * STAGE_BYTES, b_dst = a_dst + A_BYTES;
          mbar_expect_tx(full0 + 8 * s, STAGE_BYTES);
          tma_load_2d(a_dst, &tmA, full0 + 8 * s, kc * BK, mt * BM);
          tma_load_2d(b_dst, &tmB, full0 + 8 * s, kc * BK, g * p.N + nt * BN);
        }
      }
    }
  } else if (warp == 1) {
    // ---------------- MMA issuer
    if (lane == 0) {
      uint32_t it = 0, tile_i = 0;
      for (int w = blockIdx.x; w < total && !failed; w += gridDim.x, ++tile_i) {
        const uint32_t acc = tile_i & 1u, aph = (tile_i >> 1) & 1u;
        if (!mbar_wait(tempty0 + 8 * acc, aph ^ 1u, abort_flag)) { failed = true; break; }
        tc_fence_after();
        const uint32_t d_tmem = tmem_base + acc * BN;
        for (int kc = 0; kc < KC; ++kc, ++it) {
          const uint32_t s = it % stages, ph = (it / stages) & 1u;
          if (!mbar_wait(full0 + 8 * s, ph, abort_flag)) { failed = true; break; }
          tc_fence_after();
          const uint32_t a_src = base + s * STAGE_BYTES, b_src = a_src + A_BYTES;
          const uint64_t adesc = umma_desc(a_src), bdesc = umma_desc(b_src);
#pragma unroll
          for (int ks = 0; ks < BK / 16; ++ks)
            umma_f16(d_tmem, adesc + 2 * ks, bdesc + 2 * ks, IDESC, (kc | ks) != 0 ? 1u : 0u);
          umma_commit(empty0 + 8 * s);      // frees the smem stage once these MMAs have read it
        }
        if (failed) break;
        umma_commit(tfull0 + 8 * acc);      // accumulator complete
      }
    }
  } else {
    // ---------------- epilogue warps
    const int q = warp & 3;                       // TMEM lane quadrant this warp may read
    const int et = (warp - 2) * 32 + lane;        // 0..127 within the epilogue group
    uint32_t tile_i = 0;
    for (int w = blockIdx.x; w < total; w += gridDim.x, ++tile_i) {
      const int mt = w / NT, nt = w % NT;
      const int g = p.tile_cluster[mt];
      const int n0 = nt * BN;
      const uint32_t acc = tile_i & 1u, aph = (tile_i >> 1) & 1u;
      if (R > 0) {
        epi_sync();                               // readers of the previous tile's factor tiles are done
        // V tile: expert i, columns n0..n0+BN, all ranks: BN*R consecutive flat elements
        for (int i = 0; i < K; ++i) {
          const long long flat0 = ((long long)(g * K + i) * p.N + n0) * R;
          const uint32_t* src = reinterpret_cast<const uint32_t*>(p.Vq + (flat0 >> 1));
          const __half* sc = p.Vs + (flat0 >> 5);
          __half* dst = vst + (size_t)i * BN * R;
          for (int w8 = et; w8 < BN * R / 8; w8 += 128) {
            __align__(16) __half tmp[8];
            decode8(src[w8], __half2float(sc[w8 >> 2]), tmp);
            *reinterpret_cast<uint4*>(dst + w8 * 8) = *reinterpret_cast<const uint4*>(tmp);
          }
        }
        if (UP) {
          // U2 tile: expert i, rank p, columns n0..n0+BN (consecutive), stored transposed [col][rank]
          for (int i = 0; i < K; ++i)
            for (int pr = 0; pr < R; ++pr) {
              const long long flat0 = ((long long)(g * K + i) * R + pr) * p.N + n0;
              const uint32_t* src = reinterpret_cast<const uint32_t*>(p.U2q + (flat0 >> 1));
              const __half* sc = p.U2s + (flat0 >> 5);
              __half* dst = ust + (size_t)i * BN * R + pr;
              for (int w8 = et; w8 < BN / 8; w8 += 128) {
                __half tmp[8];
                decode8(src[w8], __half2float(sc[w8 >> 2]), tmp);
#pragma unroll
                for (int n = 0; n < 8; ++n) dst[(size_t)(w8 * 8 + n) * R] = tmp[n];
              }
            }
        }
        epi_sync();
      }
      const int row = mt * BM + q * 32 + lane;
      const int tok = p.row_token[row];
      int li[KSEL];
      float gate[KSEL];
      float co[KSEL][R > 0 ? R : 1];
      float sacc[KSEL][R > 0 ? R : 1];
#pragma unroll
      for (int j = 0; j < KSEL; ++j) {
        li[j] = p.row_slot[(size_t)row * KSEL + j] - g * K;
        gate[j] = p.row_gate[(size_t)row * KSEL + j];
#pragma unroll
        for (int pr = 0; pr < R; ++pr) {
          const float c = p.coef[((size_t)row * KSEL + j) * R + pr];
          co[j][pr] = UP ? c : c * gate[j];
          sacc[j][pr] = 0.f;
        }
      }
      const bool ok = mbar_wait(tfull0 + 8 * acc, aph, abort_flag);
      if (!epi_all(ok)) { failed = true; break; }
      tc_fence_after();
      const uint32_t t_row = tmem_base + ((uint32_t)(q * 32) << 16) + acc * BN;
#pragma unroll 1
      for (int c0 = 0; c0 < BN; c0 += 32) {
        uint32_t v[32];
        tmem_ld32(t_row + c0, v);
        __align__(16) __half outh[32];
#pragma unroll
        for (int c = 0; c < 32; ++c) {
          float hbase = __uint_as_float(v[c]);
          float res;
          if (UP) {
            res = 0.f;
#pragma unroll
            for (int j = 0; j < KSEL; ++j) {
              float h = hbase;
              if (R > 0) {
                const __half* vp = vst + ((size_t)li[j] * BN + c0 + c) * R;
#pragma unroll
                for (int pr = 0; pr < R; ++pr) h = fmaf(co[j][pr], __half2float(vp[pr]), h);
              }
              const float a = gelu_erf(h);
              res = fmaf(gate[j], a, res);
              if (R > 0) {
                const __half* up = ust + ((size_t)li[j] * BN + c0 + c) * R;
#pragma unroll
                for (int pr = 0; pr < R; ++pr) sacc[j][pr] = fmaf(a, __half2float(up[pr]), sacc[j][pr]);
              }
            }
          } else {
            res = hbase;
            if (R > 0) {
#pragma unroll
              for (int j = 0; j < KSEL; ++j) {
                const __half* vp = vst + ((size_t)li[j] * BN + c0 + c) * R;
#pragma unroll
                for (int pr = 0; pr < R; ++pr) res = fmaf(co[j][pr], __half2float(vp[pr]), res);
              }
            }
          }
          outh[c] = __float2half_rn(res);
        }
        if (UP || tok >= 0) {
          const size_t orow = UP ? (size_t)row : (size_t)tok;
          uint4* dst = reinterpret_cast<uint4*>(p.out + orow * p.N + n0 + c0);
          const uint4* srcv = reinterpret_cast<const uint4*>(outh);
#pragma unroll
          for (int i = 0; i < 4; ++i) dst[i] = srcv[i];
        }
      }
      // accumulator drained: hand it back to the MMA warp
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(tempty0 + 8 * acc);
      if (UP && R > 0 && tok >= 0) {
#pragma unroll
        for (int j = 0; j < KSEL; ++j)
#pragma unroll
          for (int pr = 0; pr < R; ++pr)
            atomicAdd(&p.s_out[((size_t)row * KSEL + j) * R + pr], sacc[j][pr]);
      }
    }
  }

  if (failed) {
    *abort_flag = 1;
    atomicExch(p.status, (int)CMOE_ERR_TIMEOUT);
  }
  __syncthreads();
  if (*abort_flag) {
    // let copies that were already issued land before the CTA's shared memory goes away
    const unsigned long long t0 = global_ns();
    while (global_ns() - t0 < 200000ull) { }
    __syncthreads();
  }
  tc_fence_after();
  if (warp == 0) {
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(kTmemCols) : "memory");
  }
}

// ---------------------------------------------------------------- host side
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*,
                                  CUtensorMapInterleave, CUtensorMapSwizzle, CUtensorMapL2promotion,
                                  CUtensorMapFloatOOBfill);

EncodeTiledFn get_encode() {
  static EncodeTiledFn fn = nullptr;
  if (!fn) {
    void* p = nullptr;
    cudaDriverEntryPointQueryResult qres;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &qres) != cudaSuccess ||
        qres != cudaDriverEntryPointSuccess)
      return nullptr;
    fn = reinterpret_cast<EncodeTiledFn>(p);
  }
  return fn;
}

// fp16 matrix [rows][cols] row-major; box = box_rows x 64 halves, 128-byte swizzle
bool make_map(CUtensorMap* map, const void* ptr, uint64_t rows, uint64_t cols, uint32_t box_rows) {
  EncodeTiledFn enc = get_encode();
  if (!enc) return false;
  cuuint64_t gdim[2] = {cols, rows};
  cuuint64_t gstride[1] = {cols * 2};
  cuuint32_t box[2] = {(cuuint32_t)BK, box_rows};
  cuuint32_t estr[2] = {1, 1};
  return enc(map, CU_TENSOR_MAP_DATA_TYPE_FLOAT16, 2, const_cast<void*>(ptr), gdim, gstride, box, estr,
             CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
             CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

size_t smem_bytes(int BN, int K, int R, bool up, int stages) {
  return 1024 + (size_t)stages * (BM * BK * 2 + BN * BK * 2) + (size_t)(up ? 2 : 1) * K * BN * R * 2 +
         (2 * kMaxStages + 4) * 8 + 16;
}
int pick_stages(int BN, int K, int R, bool up) {
  int s = kMaxStages;
  while (s > 0 && smem_bytes(BN, K, R, up, s) > kSmemLimit) --s;
  return s;
}

struct TcState {
  CUtensorMap mapA_up, mapB_up, mapA_dn, mapB_dn;
  int bn_down;
  int stages_up, stages_dn;
  int sm_count;
};
static_assert(sizeof(TcState) <= sizeof(((cmoe_layer*)nullptr)->tc_state), "tc_state too small");

constexpr int BN_UP = 128;

template <int BN, int R, int KSEL, bool UP>
cudaError_t launch_one(const TcState& ts, const TcParams& p, int grid, cudaStream_t st) {
  auto kern = tc_ffn_kernel<BN, R, KSEL, UP>;
  const size_t sm = smem_bytes(BN, p.K, R, UP, p.stages);
  static std::atomic<unsigned long long> smem_set{0};      // devices the kernel's shared-memory limit has been raised on
  if (cudaError_t e = ensure_dynamic_smem(kern, kSmemLimit, smem_set)) return e;
  kern<<<grid, kThreads, sm, st>>>(UP ? ts.mapA_up : ts.mapA_dn, UP ? ts.mapB_up : ts.mapB_dn, p);
  return cudaGetLastError();
}

template <int R, int KSEL>
cudaError_t launch_rk(const TcState& ts, const TcParams& up, const TcParams& dn, int grid_up, int grid_dn,
                      cudaStream_t st, cudaEvent_t* marks) {
  cudaError_t e = launch_one<BN_UP, R, KSEL, true>(ts, up, grid_up, st);
  if (e != cudaSuccess) return e;
  if (marks) cudaEventRecord(marks[2], st);
  if (ts.bn_down == 256) return launch_one<256, R, KSEL, false>(ts, dn, grid_dn, st);
  return launch_one<128, R, KSEL, false>(ts, dn, grid_dn, st);
}

bool rk_instantiated(int r, int k) {
  return (k == 1 || k == 2) && (r == 0 || r == 4 || r == 8 || r == 16 || r == 32);
}

}  // namespace

bool tc_supported(const Dims& D) {
  if (D.d % 128 || D.d_ff % 128) return false;
  if (!rk_instantiated(D.r, D.k)) return false;
  if (D.row_align != BM) return false;
  const int bn_dn = (D.d % 256 == 0) ? 256 : 128;
  if (pick_stages(BN_UP, D.K, D.r, true) < 3 || pick_stages(bn_dn, D.K, D.r, false) < 3) return false;
  return true;
}

cudaError_t tc_init(cmoe_layer* L) {
  const Dims& D = L->dims;
  TcState* ts = reinterpret_cast<TcState*>(L->tc_state);
  ts->bn_down = (D.d % 256 == 0) ? 256 : 128;
  ts->stages_up = pick_stages(BN_UP, D.K, D.r, true);
  ts->stages_dn = pick_stages(ts->bn_down, D.K, D.r, false);
  int dev = 0;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return e;
  e = cudaDeviceGetAttribute(&ts->sm_count, cudaDevAttrMultiProcessorCount, dev);
  if (e != cudaSuccess) return e;
  const uint64_t P = (uint64_t)D.T_pad_max;
  bool ok = make_map(&ts->mapA_up, L->sc.x_perm, P, D.d, BM) &&
            make_map(&ts->mapB_up, L->w.B1t, (uint64_t)D.G * D.d_ff, D.d, BN_UP) &&
            make_map(&ts->mapA_dn, L->sc.abar, P, D.d_ff, BM) &&
            make_map(&ts->mapB_dn, L->w.B2t, (uint64_t)D.G * D.d, D.d_ff, ts->bn_down);
  return ok ? cudaSuccess : cudaErrorInvalidValue;
}

cudaError_t launch_tc_ffn(const cmoe_layer* L, int T, __half* y, cudaStream_t st, cudaEvent_t* marks) {
  const Dims& D = L->dims;
  const Weights& W = L->w;
  const Scratch& S = L->sc;
  const TcState& ts = *reinterpret_cast<const TcState*>(L->tc_state);
  if (marks) cudaEventRecord(marks[0], st);
  cudaError_t e = launch_residual_t(D, W, S, T, st);
  if (e != cudaSuccess) return e;
  if (marks) cudaEventRecord(marks[1], st);
  const int mt_bound = t_pad_bound(D, T) / BM;
  TcParams up{};
  up.n_rows = S.n_rows; up.tile_cluster = S.tile_cluster; up.row_slot = S.row_slot; up.row_gate = S.row_gate;
  up.row_token = S.row_token; up.Vq = W.V1q; up.Vs = W.V1s; up.U2q = W.U2q; up.U2s = W.U2s; up.coef = S.t;
  up.s_out = S.s; up.out = S.abar; up.status = S.status; up.Kd = D.d; up.N = D.d_ff; up.K = D.K;
  up.stages = ts.stages_up;
  TcParams dn = up;
  dn.Vq = W.V2q; dn.Vs = W.V2s; dn.U2q = nullptr; dn.U2s = nullptr; dn.coef = S.s; dn.s_out = nullptr;
  dn.out = y; dn.Kd = D.d_ff; dn.N = D.d; dn.stages = ts.stages_dn;
  auto grid_for = [&](int ntile) {
    long long total = (long long)mt_bound * ntile;
    return (int)(total < ts.sm_count ? total : ts.sm_count);
  };
  const int grid_up = grid_for(D.d_ff / BN_UP), grid_dn = grid_for(D.d / ts.bn_down);
#define CMOE_RK(RR, KK) \
  if (D.r == RR && D.k == KK) return launch_rk<RR, KK>(ts, up, dn, grid_up, grid_dn, st, marks);
  CMOE_RK(0, 1) CMOE_RK(0, 2) CMOE_RK(4, 1) CMOE_RK(4, 2) CMOE_RK(8, 1) CMOE_RK(8, 2)
  CMOE_RK(16, 1) CMOE_RK(16, 2) CMOE_RK(32, 1) CMOE_RK(32, 2)
#undef CMOE_RK
  return cudaErrorInvalidValue;
}

}  // namespace cmoe
