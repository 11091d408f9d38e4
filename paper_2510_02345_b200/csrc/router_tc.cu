// Router for large batches on the tensor cores (sm_100a, tcgen05): all G + E router logits of a tile
// of 128 tokens as one GEMM, z = x [C | R], with fp32-grade accuracy from an error-compensated split of
// the fp32 router matrices into two fp16 pieces,
//
//     w = hi + 2^-11 lo,   hi = fp16(w),   lo = fp16((w - hi) 2^11)      (|w - hi - 2^-11 lo| <= 2^-24 |w|)
//
// so that logit = x.hi + 2^-11 x.lo with both products accumulated in fp32 by the MMA (the fp16 x
// fp16 products are exact in fp32).  The logits of a tile go through shared memory; one thread per
// token then takes the top-1 cluster (Eq. 9) and the top-k experts of that cluster with their
// renormalised softmax gates (Eq. 10), exactly as the CUDA-core kernels of router.cu do.
// Computing all E expert logits instead of the K of the chosen cluster costs tensor flops only
// (2 T d 2(G+E): 5 GFLOP at the GPT-2-medium shape); x is read once.
#include "cmoe_internal.h"
#include "device_utils.cuh"
#include "launch.cuh"
#include "tc_ptx.cuh"
#include "perm_keys.cuh"
#include "cluster_pick.cuh"

namespace cmoe {

namespace {

using namespace ptx;

constexpr int RBM = 128;          // tokens per tile
constexpr int RBK = 64;           // halves per K atom
constexpr int RKA = 2;            // K atoms per stage
constexpr int R_THREADS = 224;    // warps 0, 6 TMA (alternating stages), 1 MMA, 2..5 epilogue
constexpr int R_MAX_STAGES = 4;    // stages of the operand ring: as many as shared memory allows for the router's width (2..4)

struct RtcParams {
  int T, d, G, K, k, E;
  int rp;                        // G + E rounded up to 8 (to 16 beyond 128): the hi pieces are columns 0..rp-1, the lo pieces rp..2rp-1
  const float *bc, *be;
  const int* label;
  int* cluster_id;
  int* expert_ids;
  float* gates;
  int* slot_local;
  int* status;
  KeyCount kc;     // key counting for the permutation (keys == nullptr: routing only)
  int stages;      // stages of the operand ring
  int g1;          // clusters per token (token index = virtual token)
};

// fp32 router rows -> the two fp16 pieces, rows [hi_0 .. hi_{rp-1}, lo_0 .. lo_{rp-1}] x d (padding rows zero)
__global__ void __launch_bounds__(256)
router_split_kernel(const float* __restrict__ Ct, const float* __restrict__ Rt, int G, int E, int rp, int d,
                    __half* __restrict__ Ws) {
  const long long idx = (long long)blockIdx.x * blockDim.x + threadIdx.x;
  if (idx >= (long long)rp * d) return;
  const int j = (int)(idx / d), c = (int)(idx - (long long)j * d);
  float w = 0.f;
  if (j < G) w = Ct[(size_t)j * d + c];
  else if (j < G + E) w = Rt[(size_t)(j - G) * d + c];
  const __half hi = __float2half_rn(w);
  const __half lo = __float2half_rn((w - __half2float(hi)) * 2048.f);
  Ws[idx] = hi;
  Ws[(size_t)rp * d + idx] = lo;
}

__global__ void __launch_bounds__(R_THREADS, 1)
router_tc_kernel(const __grid_constant__ CUtensorMap tmX, const __grid_constant__ CUtensorMap tmW, const RtcParams p) {
  pdl_wait();
  pdl_release_dependents();
  extern __shared__ uint8_t smem_raw[];
  const uint32_t raw = smem_u32(smem_raw);
  const uint32_t base = (raw + 1023u) & ~1023u;
  uint8_t* sm = smem_raw + (base - raw);
  const int N = 2 * p.rp;
  // A router wider than one MMA (N > 256) is issued piece by piece: two MMAs of N / 2 columns per step, the pieces'
  // operand rows loaded by a TMA box each (a box has at most 256 rows) and lying one behind the other in the stage
  const int pieces = N > 256 ? 2 : 1, Np = N / pieces;
  const uint32_t tcols = N > 256 ? 512u : 256u;
  const uint32_t a_atom = RBM * RBK * 2, b_atom = (uint32_t)N * RBK * 2;
  const uint32_t a_bytes = RKA * a_atom, b_bytes = RKA * b_atom, st_bytes = a_bytes + b_bytes;   // b_atom is a multiple of 1024
  const int R_STAGES = p.stages;
  uint64_t* bars = reinterpret_cast<uint64_t*>(sm + (size_t)R_STAGES * st_bytes);
  const uint32_t full0 = smem_u32(bars), empty0 = smem_u32(bars + 8), tfull = smem_u32(bars + 16);
  uint32_t* tmem_holder = reinterpret_cast<uint32_t*>(bars + 17);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_holder + 1);
  float* lg = reinterpret_cast<float*>(sm);              // [128][N + 1] logits, reusing the operand ring after the main loop
  int* key_of = reinterpret_cast<int*>(lg + (size_t)RBM * (N + 1));   // [128] keys of the tile's tokens, then [nkey] counts
  int* cnt = key_of + RBM;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int tile = blockIdx.x;
  const int KC = p.d / (RBK * RKA);

  if (threadIdx.x == 0) {
    for (int s = 0; s < R_STAGES; ++s) { mbar_init(full0 + 8 * s, 1); mbar_init(empty0 + 8 * s, 1); }
    mbar_init(tfull, 1);
    *abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 1) {
    __syncwarp();
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;"
                 ::"r"(smem_u32(tmem_holder)), "r"(tcols) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_holder;
  bool failed = false;

  if (warp == 0 || warp == 6) {
    if (lane == 0) {
      for (int c = warp == 0 ? 0 : 1; c < KC; c += 2) {
        const uint32_t s = c % R_STAGES, ph = (c / R_STAGES) & 1u;
        if (!mbar_wait(empty0 + 8 * s, ph ^ 1u, abort_flag)) { failed = true; break; }
        const uint32_t a_dst = base + s * st_bytes, b_dst = a_dst + a_bytes;
        mbar_expect_tx(full0 + 8 * s, st_bytes);
        tma_load_3d(a_dst, &tmX, full0 + 8 * s, 0, tile * RBM, c * RKA);    // rows past T read as zeros
        for (int h = 0; h < pieces; ++h)
          tma_load_3d(b_dst + h * (b_bytes / pieces), &tmW, full0 + 8 * s, 0, h * Np, c * RKA);
      }
    }
  } else if (warp == 1) {
    if (lane == 0) {
      const uint32_t idesc = idesc_f16(RBM, Np);
      const uint32_t bp_atom = b_atom / pieces;          // one K atom of one piece
      for (int c = 0; c < KC; ++c) {
        const uint32_t s = c % R_STAGES, ph = (c / R_STAGES) & 1u;
        if (!mbar_wait(full0 + 8 * s, ph, abort_flag)) { failed = true; break; }
        tc_fence_after();
        const uint32_t a_src = base + s * st_bytes, b_src = a_src + a_bytes;
        const uint64_t adesc = umma_desc(a_src), bdesc = umma_desc(b_src);
#pragma unroll
        for (int a = 0; a < RKA; ++a)
#pragma unroll
          for (int ks = 0; ks < RBK / 16; ++ks)
            for (int h = 0; h < pieces; ++h)
              umma_f16(tmem_base + h * Np, adesc + a * (a_atom >> 4) + 2 * ks,
                       bdesc + ((h * RKA + a) * bp_atom >> 4) + 2 * ks, idesc, (c | a | ks) != 0 ? 1u : 0u);
        umma_commit(empty0 + 8 * s);
      }
      if (!failed) umma_commit(tfull);
    }
  } else {
    // ---------------- epilogue: thread = token; logits to shared memory, then the selection
    const int q = warp & 3;
    const int trow = q * 32 + lane;
    const int tok = tile * RBM + trow;
    const bool ok = mbar_wait(tfull, 0, abort_flag);
    int key = -1;
    if (__all_sync(0xffffffffu, ok)) {
      tc_fence_after();
      const uint32_t taddr = tmem_base + ((uint32_t)(q * 32) << 16);
      float* mine = lg + (size_t)trow * (N + 1);
      for (int c0 = 0; c0 < N; c0 += 8) {
        uint32_t v[8];
        tmem_ld8_nowait(taddr + c0, v);
        tmem_ld_wait();
#pragma unroll
        for (int c = 0; c < 8; ++c) mine[c0 + c] = __uint_as_float(v[c]);
      }
      if (tok < p.T) {
        const int rp = p.rp, G = p.G, K = p.K;
        int gs = 0;
        float cluster_weight = 1.f;
        if (p.g1 < 2) {
          float zbest = 0.f;
          for (int g = 0; g < G; ++g) {
            const float z = fmaf(mine[rp + g], 1.f / 2048.f, mine[g]) + p.bc[g];
            if (g == 0 || z > zbest) { zbest = z; gs = g; }        // strict >: lowest index wins ties
          }
        } else {
          // two clusters per token: this is virtual token tok % 2 of its token
          TwoBest b;
          two_best_init(b);
          for (int g = 0; g < G; ++g) two_best_add(b, g, fmaf(mine[rp + g], 1.f / 2048.f, mine[g]) + p.bc[g]);
          two_best_pick(b, tok & 1, gs, cluster_weight);
        }
        p.cluster_id[tok] = gs;
        // expert logits of the chosen cluster, in place over the cluster columns (no longer needed)
        const int e0 = G + gs * K;
        for (int i = 0; i < K; ++i) mine[i] = fmaf(mine[rp + e0 + i], 1.f / 2048.f, mine[e0 + i]) + p.be[gs * K + i];
        unsigned taken = 0;
        float selv[kMaxKsel];
        int seli[kMaxKsel];
        for (int s = 0; s < p.k; ++s) {
          float best = -INFINITY;
          int bi = 0;
          bool have = false;
          for (int i = 0; i < K; ++i) {
            if ((taken >> i) & 1u) continue;
            const float v = mine[i];
            if (!have || v > best) { best = v; bi = i; have = true; }
          }
          taken |= 1u << bi;
          selv[s] = best;
          seli[s] = bi;
        }
        const float lmax = selv[0];
        float ev[kMaxKsel];
        float sum = 0.f;
        for (int s = 0; s < p.k; ++s) { ev[s] = expf(selv[s] - lmax); sum += ev[s]; }
        for (int s = 0; s < p.k; ++s) ev[s] = cluster_weight == 1.f ? ev[s] / sum : cluster_weight * (ev[s] / sum);
        for (int s = 0; s < p.k; ++s) {
          if (p.gates) p.gates[(size_t)tok * p.k + s] = ev[s];
          if (p.expert_ids) p.expert_ids[(size_t)tok * p.k + s] = p.label[gs * K + seli[s]];
          if (p.slot_local) p.slot_local[(size_t)tok * p.k + s] = seli[s];
        }
        if (p.kc.keys) {
          int cs[kMaxKsel];
          float cg[kMaxKsel];
          key = gs * p.kc.nsub + canonical_slots(seli, ev, p.k, p.kc.sub_is_combo, cs, cg);
          p.kc.keys[tok] = key;
        }
      }
    } else {
      failed = true;
    }
    if (p.kc.keys) key_of[trow] = key;       // (its own logits row is no longer read; the key table lies past all rows)
    tc_fence_before();
  }

  if (failed) {
    *abort_flag = 1;
    atomicExch(p.status, (int)CMOE_ERR_TIMEOUT);
  }
  __syncthreads();
  if (*abort_flag) {
    const long long t0 = clock64();
    while (clock64() - t0 < 400000ll) { }       // let copies already issued land
    __syncthreads();
  }
  tc_fence_after();
  if (warp == 1)
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(tcols) : "memory");
  if (p.kc.keys) {
    // keys of this tile counted in shared memory: the permutation's histogram, for free
    for (int i = threadIdx.x; i < p.kc.nkey; i += blockDim.x) cnt[i] = 0;
    __syncthreads();
    if (threadIdx.x < RBM && key_of[threadIdx.x] >= 0) atomicAdd(&cnt[key_of[threadIdx.x]], 1);
    __syncthreads();
    for (int i = threadIdx.x; i < p.kc.nkey; i += blockDim.x) p.kc.block_counts[(size_t)tile * p.kc.nkey + i] = cnt[i];
  }
}

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*,
                                  CUtensorMapInterleave, CUtensorMapSwizzle, CUtensorMapL2promotion,
                                  CUtensorMapFloatOOBfill);

EncodeTiledFn get_encode() {
  static EncodeTiledFn fn = nullptr;
  if (!fn) {
    void* ptr = nullptr;
    cudaDriverEntryPointQueryResult qres;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &ptr, cudaEnableDefault, &qres) != cudaSuccess ||
        qres != cudaDriverEntryPointSuccess)
      return nullptr;
    fn = reinterpret_cast<EncodeTiledFn>(ptr);
  }
  return fn;
}

// fp16 matrix [rows][cols] seen as [cols / 64][rows][64]; box of 64 x box_rows x RKA
bool make_map3(CUtensorMap* map, const void* ptr, uint64_t rows, uint64_t cols, uint32_t box_rows) {
  EncodeTiledFn enc = get_encode();
  if (!enc) return false;
  cuuint64_t gdim[3] = {(cuuint64_t)RBK, rows, cols / RBK};
  cuuint64_t gstride[2] = {cols * 2, (cuuint64_t)RBK * 2};
  cuuint32_t box[3] = {(cuuint32_t)RBK, box_rows, (cuuint32_t)RKA};
  cuuint32_t estr[3] = {1, 1, 1};
  return enc(map, CU_TENSOR_MAP_DATA_TYPE_FLOAT16, 3, const_cast<void*>(ptr), gdim, gstride, box, estr,
             CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
             CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

size_t rtc_smem(int N, int stages) {
  const size_t ring = (size_t)stages * RKA * (RBM + N) * RBK * 2;
  const size_t logits = (size_t)RBM * (N + 1) * 4 + (size_t)(RBM + kMaxKeys) * 4;   // logits, keys of the tile, key counts
  return 1024 + (ring > logits ? ring : logits) + 32 * 8;
}

// the deepest ring that fits (0: the router is too wide for this kernel)
int rtc_stages(int N) {
  for (int st = R_MAX_STAGES; st >= 2; --st)
    if (rtc_smem(N, st) <= 232448) return st;
  return 0;
}

}  // namespace

int router_tc_rp(const Dims& D) {
  const int n = real_G(D) + D.E;
  return n <= 128 ? (n + 7) / 8 * 8 : (n + 15) / 16 * 16;      // (beyond 128 every piece is an MMA of its own: N a multiple of 16)
}

bool router_tc_supported(const Dims& D) {
  const int N = 2 * router_tc_rp(D);
  return D.d % (RBK * RKA) == 0 && N <= 512 && D.T_max >= 1024 && rtc_stages(N) > 0;
}

cudaError_t router_tc_init(cmoe_layer* L) {
  const Dims& D = L->dims;
  const int rp = router_tc_rp(D);
  const long long n = (long long)rp * D.d;
  router_split_kernel<<<(unsigned)((n + 255) / 256), 256>>>(L->w.Ct, L->w.Rt, real_G(D), D.E, rp, D.d, L->sc.Wsplit);
  cudaError_t e = cudaGetLastError();
  if (e != cudaSuccess) return e;
  if (!make_map3(&L->router_map_w, L->sc.Wsplit, (uint64_t)2 * rp, D.d, (uint32_t)(2 * rp > 256 ? rp : 2 * rp))) return cudaErrorInvalidValue;
  e = cudaFuncSetAttribute(router_tc_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)rtc_smem(2 * rp, rtc_stages(2 * rp)));
  if (e != cudaSuccess) return e;
  return cudaDeviceSynchronize();
}

int router_tc_tile_tokens() { return RBM; }

cudaError_t launch_router_tc(const cmoe_layer* L, const __half* x, int T, int* cluster_id, int* expert_ids, float* gates,
                             int* slot_local, cudaStream_t st, const KeyCount* kc) {
  const Dims& D = L->dims;
  CUtensorMap mx;
  if (!make_map3(&mx, x, (uint64_t)T, D.d, RBM)) return cudaErrorInvalidValue;   // x is the caller's buffer: a map per call
  RtcParams p{};
  p.T = T; p.d = D.d; p.G = real_G(D); p.K = real_K(D); p.k = D.k; p.E = D.E; p.rp = router_tc_rp(D); p.g1 = D.g1;
  p.bc = L->w.bc; p.be = L->w.be; p.label = L->w.label;
  p.cluster_id = cluster_id; p.expert_ids = expert_ids; p.gates = gates; p.slot_local = slot_local; p.status = L->sc.status;
  if (kc) p.kc = *kc;
  p.stages = rtc_stages(2 * p.rp);
  return launch_chained(router_tc_kernel, dim3((unsigned)((T + RBM - 1) / RBM)), dim3(R_THREADS), rtc_smem(2 * p.rp, p.stages), st, 1, mx,
                        L->router_map_w, p);
}

}  // namespace cmoe
