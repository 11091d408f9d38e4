// Tensor-core path of the expert FFNs with the rank-r residuals on the tensor cores as well
// (sm_100a: tcgen05 MMAs with TMEM accumulators, operands staged in shared memory by TMA).
//
// The factored form of the text after Eq. 7, x W_e = x B_g + (x U_e) V_e, is kept, but every
// rank-r product is phrased as a GEMM over an "expanded rank index" c = i*r + p (i = expert of the
// cluster, p = rank), KE = 64 wide, so that one tile may mix rows routed to different experts:
//
//   stage   INT4 factors of the layer -> fp16 operand matrices in scratch (decoded in registers; stage_factors.cuh:
//           the blocks ride in the permutation's scan kernel)
//             U1f [G][KE][d]   V1f [G][d_ff][KE]   U2f [G][KE][d_ff]   V2f [G][d][KE]
//   t       Tall = x_perm U1f_g^T (128 x KE per tile); row-wise selection writes
//             A0 [row][c] = t of the row's first kept expert inside that expert's block, else 0
//             Ad [row][c] = +t of the second kept expert in its block, -t of the first in its block
//   up      P = x_perm B1_g^T + A0 V1f^T  (= h of the first expert),  Q = Ad V1f^T  (h_2 - h_1);
//           epilogue: a_j = GELU(h_j), abar = sum_j p_j a_j (fp16 to HBM), a_j (fp16) to shared
//           memory as the A operand of  S_j += a_j U2f^T  (accumulated in TMEM over the N tiles of
//           a row tile, then the row's own block is added to s with fp32 atomics)
//   down    y = abar B2_g^T + As V2f^T, stored un-permuted, with As [row][c] = p_j s_j inside the block of expert
//           e_j (fp16): written by the up kernel when its work units are whole row tiles, else by this kernel's
//           epilogue warps from the fp32 sums s while they wait for a tile's main loop
//
// The up and down kernels run as CTA pairs (thread-block clusters of two, tcgen05 cta_group::2) on
// 256-row tiles: each CTA loads its 128 rows of A and half of the B tile, the leader CTA issues the
// MMAs, each CTA's 128 accumulator rows land in its own TMEM and are drained by its own epilogue
// warps.  This halves the B traffic from L2 per CTA, which is what bounds 128-wide tiles.  A
// cluster's rows therefore start at multiples of 256.
//
// The base product is computed once per token and shared by its k experts; the extra tensor work
// is the KE-deep steps (skipped per tile for experts no row of the tile uses) and the S products.
// Every device wait is bounded: on expiry the kernel records CMOE_ERR_TIMEOUT in the status word,
// all roles leave their loops, TMEM is freed and the kernel returns.
#include "tc2_common.cuh"
#include "stage_factors.cuh"

namespace cmoe {

namespace {

using namespace tc2c;

constexpr int BN_UP = 128;
constexpr int kMaxStages = 8;

// ------------------------------------------------------------------------------------------------
// t: Tall = x_perm U1f_g^T, one 128-row tile per CTA, then the row-wise selection into A0 / Ad
// ------------------------------------------------------------------------------------------------
struct TParams {
  const int* n_rows;
  const int* tile_cluster;
  const int* row_slot;
  const int* row_token;
  __half* A0;          // [rows][KE]
  __half* Ad;          // [rows][KE]  (k == 2 only)
  int* tile_mask;      // [tiles][2]  16-wide steps of the expanded index used by slot 0 / slot 1 (up projection)
  int* tile_mask_dn;   // [tiles]     steps the down projection needs
  const int* live;     // [E]         bit 0 / 1: the expert's up / down residual block is not zero
  int* status;
  int KC, K, r;
  int x_rows;          // gather mode: rows of x (the first row index that reads zeros)
};

constexpr int T_THREADS = 224;      // warps 0 and 6 TMA (alternating stages), 1 MMA, 2..5 epilogue
constexpr int T_STAGES = 6;
constexpr uint32_t T_STAGE_BYTES = BM * BK * 2 + KE * BK * 2;   // 24 KB

// GATHER: the kernel reads the tile's rows from x itself (TMA gather by row_token, zeros for padding rows) and, as
// each K chunk passes through shared memory, stores it to x_perm for the up kernel: the permuted copy of x is a
// by-product of this kernel instead of a pass of its own over x.
template <int KSEL, bool GATHER>
__global__ void __launch_bounds__(T_THREADS, 1)
tc2_t_kernel(const __grid_constant__ CUtensorMap tmX, const __grid_constant__ CUtensorMap tmU1,
             const __grid_constant__ CUtensorMap tmXsrc, const TParams p) {
  pdl_wait();
  pdl_release_dependents();
  const int mt = blockIdx.x;
  if (mt >= *p.n_rows / BM) return;
  extern __shared__ uint8_t smem_raw[];
  const uint32_t raw = smem_u32(smem_raw);
  const uint32_t base = (raw + 1023u) & ~1023u;
  uint8_t* sm = smem_raw + (base - raw);
  uint64_t* bars = reinterpret_cast<uint64_t*>(sm + (size_t)T_STAGES * T_STAGE_BYTES);
  const uint32_t full0 = smem_u32(bars), empty0 = smem_u32(bars + kMaxStages), tfull = smem_u32(bars + 2 * kMaxStages);
  uint32_t* tmem_holder = reinterpret_cast<uint32_t*>(bars + 2 * kMaxStages + 1);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_holder + 1);
  int* sh_mask = reinterpret_cast<int*>(tmem_holder + 2);     // [3]
  int* s_tok = sh_mask + 4;                                   // [BM] gather mode: source row of every row of the tile
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

  if (GATHER && threadIdx.x < BM) {
    const int tok = p.row_token[mt * BM + threadIdx.x];
    s_tok[threadIdx.x] = tok >= 0 ? tok : p.x_rows;           // padding rows: outside the tensor, i.e. zeros
  }
  if (threadIdx.x == 0) {
    for (int s = 0; s < T_STAGES; ++s) { mbar_init(full0 + 8 * s, 1); mbar_init(empty0 + 8 * s, 1); }
    mbar_init(tfull, 1);
    *abort_flag = 0;
    sh_mask[0] = 0; sh_mask[1] = 0; sh_mask[2] = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 0) {
    __syncwarp();
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;"
                 ::"r"(smem_u32(tmem_holder)), "r"(64u) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_holder;
  const int g = p.tile_cluster[mt >> 1];      // the cluster table has one entry per 256 rows
  const int KC = p.KC;
  bool failed = false;

  if (warp == 0 || warp == 6) {
    if (lane == 0) {
      for (int kc = warp == 0 ? 0 : 1; kc < KC; kc += 2) {
        const uint32_t s = kc % T_STAGES, ph = (kc / T_STAGES) & 1u;
        if (!mbar_wait(empty0 + 8 * s, ph ^ 1u, abort_flag)) { failed = true; break; }
        const uint32_t a_dst = base + s * T_STAGE_BYTES, b_dst = a_dst + BM * BK * 2;
        mbar_expect_tx(full0 + 8 * s, T_STAGE_BYTES);
        if (GATHER) {
          // four rows (512 bytes of the swizzled tile) per instruction
          for (int r4 = 0; r4 < BM; r4 += 4) {
            const int4 t4 = *reinterpret_cast<const int4*>(s_tok + r4);
            tma_gather4_2d(a_dst + r4 * (BK * 2), &tmXsrc, full0 + 8 * s, kc * BK, t4.x, t4.y, t4.z, t4.w);
          }
        } else {
          tma_load_2d(a_dst, &tmX, full0 + 8 * s, kc * BK, mt * BM);
        }
        tma_load_2d(b_dst, &tmU1, full0 + 8 * s, kc * BK, g * KE);
      }
    }
  } else if (warp == 1) {
    if (lane == 0) {
      constexpr uint32_t IDESC = idesc_f16(BM, KE);
      for (int kc = 0; kc < KC; ++kc) {
        const uint32_t s = kc % T_STAGES, ph = (kc / T_STAGES) & 1u;
        if (!mbar_wait(full0 + 8 * s, ph, abort_flag)) { failed = true; break; }
        tc_fence_after();
        const uint32_t a_src = base + s * T_STAGE_BYTES, b_src = a_src + BM * BK * 2;
        const uint64_t adesc = umma_desc(a_src), bdesc = umma_desc(b_src);
#pragma unroll
        for (int ks = 0; ks < BK / 16; ++ks)
          umma_f16(tmem_base, adesc + 2 * ks, bdesc + 2 * ks, IDESC, (kc | ks) != 0 ? 1u : 0u);
        if (GATHER) {
          // The chunk of x rows goes out to x_perm.  A stage is handed back once its store has read it: two
          // stores stay in flight, so the stage of chunk kc - 2 is released here (the commit also covers its MMAs,
          // issued long before).
          tma_store_2d(&tmX, a_src, kc * BK, mt * BM);
          bulk_commit_group();
          bulk_wait_read_but2();
          if (kc >= 2) umma_commit(empty0 + 8 * ((kc - 2) % T_STAGES));
        } else {
          umma_commit(empty0 + 8 * s);
        }
      }
      if (GATHER) {
        bulk_wait_read_all();
        // (the last two stages are not refilled: nothing waits for their release)
        bulk_wait_all();
      }
      if (!failed) umma_commit(tfull);
    }
  } else if (warp < 6) {
    const int q = warp & 3;
    const int row = mt * BM + q * 32 + lane;
    const int r = p.r;
    const int lo0 = (p.row_slot[(size_t)row * KSEL] - g * p.K) * r;
    const int lo1 = KSEL == 2 ? (p.row_slot[(size_t)row * KSEL + 1] - g * p.K) * r : -1;
    const bool real = p.row_token[row] >= 0;
    // residual blocks that are zero (pruned) need no step: bit 0 up, bit 1 down, per kept expert
    const int live0 = p.live[p.row_slot[(size_t)row * KSEL]];
    const int live1 = KSEL == 2 ? p.live[p.row_slot[(size_t)row * KSEL + 1]] : 0;
    if (warp_wait(tfull, 0, abort_flag)) {
      tc_fence_after();
      const uint32_t taddr = tmem_base + ((uint32_t)(q * 32) << 16);
#pragma unroll
      for (int half = 0; half < 2; ++half) {
        uint32_t v[32];
        tmem_ld32_nowait(taddr + half * 32, v);
        tmem_ld_wait();
        uint32_t o0[16], od[16];
#pragma unroll
        for (int c = 0; c < 32; c += 2) {
          float a[2], dl[2];
#pragma unroll
          for (int u = 0; u < 2; ++u) {
            const int cc = half * 32 + c + u;
            const float t = __uint_as_float(v[c + u]);
            const bool in0 = cc >= lo0 && cc < lo0 + r;
            const bool in1 = KSEL == 2 && cc >= lo1 && cc < lo1 + r;
            a[u] = in0 ? t : 0.f;
            dl[u] = in1 ? t : (in0 ? -t : 0.f);
          }
          o0[c >> 1] = pack_half2(a[0], a[1]);
          od[c >> 1] = pack_half2(dl[0], dl[1]);
        }
        uint4* d0 = reinterpret_cast<uint4*>(p.A0 + (size_t)row * KE + half * 32);
#pragma unroll
        for (int i = 0; i < 4; ++i) d0[i] = make_uint4(o0[4 * i], o0[4 * i + 1], o0[4 * i + 2], o0[4 * i + 3]);
        if (KSEL == 2) {
          uint4* dd = reinterpret_cast<uint4*>(p.Ad + (size_t)row * KE + half * 32);
#pragma unroll
          for (int i = 0; i < 4; ++i) dd[i] = make_uint4(od[4 * i], od[4 * i + 1], od[4 * i + 2], od[4 * i + 3]);
        }
      }
      // 16-wide steps of the expanded index that rows of this tile use
      int m0 = 0, m1 = 0, md = 0;
      if (real) {
        int s0 = 0, s1 = 0;
        for (int c = lo0; c < lo0 + r; c += (r < 16 ? r : 16)) s0 |= 1 << (c >> 4);
        if (KSEL == 2)
          for (int c = lo1; c < lo1 + r; c += (r < 16 ? r : 16)) s1 |= 1 << (c >> 4);
        if (live0 & 1) m0 = s0;
        if (live1 & 1) m1 = s1;
        // Ad carries -t of the first expert inside that expert's block: its steps are needed whenever the second pass runs
        if (KSEL == 2 && (live0 & 1)) m1 |= s0;
        md = ((live0 & 2) ? s0 : 0) | ((live1 & 2) ? s1 : 0);
      }
      m0 = __reduce_or_sync(0xffffffffu, (unsigned)m0);
      m1 = __reduce_or_sync(0xffffffffu, (unsigned)m1);
      md = __reduce_or_sync(0xffffffffu, (unsigned)md);
      if (lane == 0) { atomicOr(&sh_mask[0], m0); atomicOr(&sh_mask[1], m1); atomicOr(&sh_mask[2], md); }
    } else {
      failed = true;
    }
    tc_fence_before();
  }

  if (failed) {
    *abort_flag = 1;
    atomicExch(p.status, (int)CMOE_ERR_TIMEOUT);
  }
  __syncthreads();
  if (threadIdx.x == 64) { p.tile_mask[2 * mt] = sh_mask[0]; p.tile_mask[2 * mt + 1] = sh_mask[1]; p.tile_mask_dn[mt] = sh_mask[2]; }
  if (*abort_flag) {
    const unsigned long long t0 = global_ns();
    while (global_ns() - t0 < 200000ull) { }    // let copies already issued land
    __syncthreads();
  }
  tc_fence_after();
  if (warp == 0)
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(64u) : "memory");
}

// ------------------------------------------------------------------------------------------------
// up: CTA pairs (cta_group::2) on 256 x 128 tiles; each CTA owns 128 rows
// ------------------------------------------------------------------------------------------------
// Warp roles: 0 and 3 TMA (alternating stages), 1 MMA, 2 S products, 4..19 epilogue.
// One thread can issue a TMA tile load only every few hundred cycles, and everything a single
// thread does between two MMAs delays the next one, so a stage carries two 64-wide K atoms (eight
// MMAs per barrier round trip) and two threads feed the ring.  The epilogue is sixteen warps (four
// per scheduler) working in packed fp16, because with fewer it, not the tensor pipe, sets the pace.
constexpr int UP_THREADS = 640;
constexpr int UP_EPI_WARP0 = 4, UP_EPI_WARPS = 16;
constexpr int KA = 2;                                               // K atoms of 64 halves per stage
constexpr uint32_t UP_A_ATOM = BM * BK * 2;                         // 16 KB: this CTA's 128 rows, one atom
constexpr uint32_t UP_B_ATOM = (BN_UP / 2) * BK * 2;                //  8 KB: this CTA's half of the B tile
constexpr uint32_t UP_A_BYTES = KA * UP_A_ATOM;
constexpr uint32_t UP_B_BYTES = KA * UP_B_ATOM;
constexpr uint32_t UP_STAGE_BYTES = UP_A_BYTES + UP_B_BYTES;        // 48 KB
constexpr uint32_t A_CHUNK_BYTES = BM * BK * 2;                     // 16 KB: 128 rows x 64 activations
constexpr uint32_t U2_CHUNK_BYTES = (KE / 2) * BK * 2;              //  4 KB: this CTA's 32 rows of a 64 x 64 chunk
constexpr uint32_t U2_TILE_BYTES = 2 * U2_CHUNK_BYTES;

// barrier slots (64-bit words after the buffers)
enum : int { B_FULL = 0, B_EMPTY = 8, B_TFULL = 16, B_TEMPTY = 18, B_QEMPTY = 20, B_AFULL = 21, B_AEMPTY = 25,
             B_U2FULL = 29, B_U2EMPTY = 31, B_SFULL = 33, B_SEMPTY = 34, B_QFULL = 35, B_COUNT = 37 };

template <bool HAS_R, int KSEL>
struct UpCfg {
  static constexpr int STAGES = HAS_R ? 3 : 4;
  static constexpr int NA = HAS_R ? 2 * KSEL : 1;          // activation chunks per tile = ring size
  static constexpr int NEXT = HAS_R ? 1 : 0;               // one expanded-index stage after the main loop (atom j feeds P / Q)
  static constexpr uint32_t RING = STAGES * UP_STAGE_BYTES;
  static constexpr uint32_t ARING = HAS_R ? NA * A_CHUNK_BYTES : 0;
  static constexpr uint32_t U2 = HAS_R ? 2 * U2_TILE_BYTES : 0;
  static constexpr uint32_t BAR_OFF = RING + ARING + U2;
  static constexpr size_t SMEM = 1024 + BAR_OFF + 48 * 8;
};

template <bool HAS_R, int KSEL>
__global__ void __launch_bounds__(UP_THREADS, 1)
tc2_up_kernel(const __grid_constant__ CUtensorMap tmX3, const __grid_constant__ CUtensorMap tmB13,
              const __grid_constant__ CUtensorMap tmA0, const __grid_constant__ CUtensorMap tmAd,
              const __grid_constant__ CUtensorMap tmV1, const __grid_constant__ CUtensorMap tmU2,
              const Up2Params p) {
  pdl_wait();
  using Cfg = UpCfg<HAS_R, KSEL>;
  constexpr int STAGES = Cfg::STAGES;
  extern __shared__ uint8_t smem_raw[];
  const uint32_t raw = smem_u32(smem_raw);
  const uint32_t base = (raw + 1023u) & ~1023u;
  uint8_t* sm = smem_raw + (base - raw);
  const uint32_t aring = base + Cfg::RING;
  const uint32_t u2base = aring + Cfg::ARING;
  uint64_t* bars = reinterpret_cast<uint64_t*>(sm + Cfg::BAR_OFF);
  const uint32_t bar0 = smem_u32(bars);
  uint32_t* tmem_holder = reinterpret_cast<uint32_t*>(bars + B_COUNT);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_holder + 1);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const uint32_t rank = cluster_ctarank();
  const bool leader = rank == 0;
  // the same barrier words in the leader's and in the peer's shared memory (shared::cluster addresses)
  const uint32_t cbar[2] = {mapa(bar0, 0), mapa(bar0, 1)};
  const uint32_t lbar = cbar[0];
  auto local = [&](int slot) { return bar0 + 8u * slot; };
  auto lead = [&](int slot) { return lbar + 8u * slot; };
  auto commit_both = [&](int slot) { umma2_commit(cbar[0] + 8u * slot); umma2_commit(cbar[1] + 8u * slot); };

  if (threadIdx.x == 0) {
    for (int s = 0; s < STAGES; ++s) { mbar_init(local(B_FULL + s), 1); mbar_init(local(B_EMPTY + s), 1); }
    for (int a = 0; a < 2; ++a) { mbar_init(local(B_TFULL + a), 1); mbar_init(local(B_TEMPTY + a), 2 * UP_EPI_WARPS); }
    mbar_init(local(B_QEMPTY), 2 * UP_EPI_WARPS);
    mbar_init(local(B_QFULL), 1);
    for (int a = 0; a < 4; ++a) { mbar_init(local(B_AFULL + a), UP_EPI_WARPS); mbar_init(local(B_AEMPTY + a), 1); }
    for (int a = 0; a < 2; ++a) { mbar_init(local(B_U2FULL + a), 1); mbar_init(local(B_U2EMPTY + a), 1); }
    mbar_init(local(B_SFULL), 1);
    mbar_init(local(B_SEMPTY), UP_EPI_WARPS * KSEL);
    *abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 0) {
    __syncwarp();
    asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;"
                 ::"r"(smem_u32(tmem_holder)), "r"(kTmemCols) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  cluster_sync_all();          // both CTAs' barriers are initialised before either signals the other
  tc_fence_after();
  const uint32_t tmem_base = *tmem_holder;
  // TMEM columns: P (two buffers) 0..255, Q 256..383, S_0 384..447, S_1 448..511
  const uint32_t tmem_q = tmem_base + 256, tmem_s = tmem_base + 384;

  const int NT = p.NT, KC = p.KC;
  // Work units of `unit` consecutive N tiles of one 256-row tile, dealt round-robin to the CTA pairs:
  // at any time the pairs work on neighbouring row tiles, i.e. inside one or two clusters, whose base
  // then stays in L2.  Local tile i of this pair is tile i % unit of its (i / unit)-th unit.
  const int pair = blockIdx.x >> 1, npairs = gridDim.x >> 1;
  const int unit = p.unit, upm = NT / unit;
  const int n_units = (*p.n_rows / (2 * BM)) * upm;
  const int w1 = pair < n_units ? ((n_units - 1 - pair) / npairs + 1) * unit : 0;
  auto tile_of = [&](int i, int& pt, int& nt) {
    const int uu = i / unit, u = pair + uu * npairs;
    pt = u / upm;
    nt = (u - pt * upm) * unit + (i - uu * unit);
  };
  bool failed = false;

  if (warp == 0 || warp == 3) {
    // ---------------- TMA producers (both CTAs, two threads taking alternate stages): this CTA's rows
    // of A and its half of B; the bytes of both CTAs are counted on the leader's barrier
    if (lane == 0) {
      const int spt = KC + Cfg::NEXT;                   // stages per tile
      const uint32_t n_it = (uint32_t)w1 * spt;
      for (uint32_t it = warp == 0 ? 0u : 1u; it < n_it && !failed; it += 2) {
        const int w = it / spt, c = it - w * spt;
        int pt, nt;
        tile_of(w, pt, nt);
        const int g = p.tile_cluster[pt];
        const int arow = (2 * pt + (int)rank) * BM;
        const int ncol = nt * BN_UP + (int)rank * (BN_UP / 2);
        const int brow = (g >> p.bshift) * p.N + ncol;        // base rows: of the cluster that owns the base
        const int vrow = g * p.N + ncol;                      // staged factor rows: of this (virtual) cluster
        const uint32_t s = it % STAGES, ph = (it / STAGES) & 1u;
        if (!mbar_wait_cluster(local(B_EMPTY + s), ph ^ 1u, abort_flag)) { failed = true; break; }
        const uint32_t a_dst = base + s * UP_STAGE_BYTES, b_dst = a_dst + UP_A_BYTES;
        if (c < KC) {
          if (leader) mbar_expect_tx(local(B_FULL + s), 2 * UP_STAGE_BYTES);
          tma2_load_3d(a_dst, &tmX3, lead(B_FULL + s), 0, arow, c * KA);
          tma2_load_3d(b_dst, &tmB13, lead(B_FULL + s), 0, brow, c * KA);
        } else {
          // expanded-index stage: atom 0 = (A0, V1f) for P, atom 1 = (Ad, V1f) for Q
          if (leader) mbar_expect_tx(local(B_FULL + s), 2 * KSEL * (UP_A_ATOM + UP_B_ATOM));
          tma2_load_2d(a_dst, &tmA0, lead(B_FULL + s), 0, arow);
          tma2_load_2d(b_dst, &tmV1, lead(B_FULL + s), 0, vrow);
          if (KSEL == 2) {
            tma2_load_2d(a_dst + UP_A_ATOM, &tmAd, lead(B_FULL + s), 0, arow);
            tma2_load_2d(b_dst + UP_B_ATOM, &tmV1, lead(B_FULL + s), 0, vrow);
          }
        }
      }
    }
  } else if (warp == 1) {
    // ---------------- MMA issuer of P and Q (leader CTA only)
    if (lane == 0 && leader) {
      constexpr uint32_t IDESC = idesc_f16(2 * BM, BN_UP);
      uint32_t s = 0, ph = 0, tile_i = 0;
      for (int w = 0; w < w1 && !failed; ++w, ++tile_i) {
        int pt, nt_unused;
        tile_of(w, pt, nt_unused);
        const uint32_t acc = tile_i & 1u, aph = (tile_i >> 1) & 1u;
        const int m0 = HAS_R ? (p.tile_mask[4 * pt] | p.tile_mask[4 * pt + 2]) : 0;
        const int m1 = HAS_R ? (p.tile_mask[4 * pt + 1] | p.tile_mask[4 * pt + 3]) : 0;
        if (!mbar_wait_cluster(local(B_TEMPTY + acc), aph ^ 1u, abort_flag)) { failed = true; break; }
        tc_fence_after();
        const uint32_t d_tmem = tmem_base + acc * BN_UP;
        for (int c = 0; c < KC + Cfg::NEXT; ++c) {
          if (!mbar_wait_cluster(local(B_FULL + s), ph, abort_flag)) { failed = true; break; }
          tc_fence_after();
          const uint32_t a_src = base + s * UP_STAGE_BYTES, b_src = a_src + UP_A_BYTES;
          const uint64_t adesc = umma_desc(a_src), bdesc = umma_desc(b_src);
          if (c < KC) {
            // the second atom's tiles follow the first's: descriptor addresses are in 16-byte units
            umma2_f16(d_tmem, adesc, bdesc, IDESC, c != 0 ? 1u : 0u);
#pragma unroll
            for (int ks = 1; ks < BK / 16; ++ks) umma2_f16(d_tmem, adesc + 2 * ks, bdesc + 2 * ks, IDESC, 1u);
#pragma unroll
            for (int ks = 0; ks < BK / 16; ++ks)
              umma2_f16(d_tmem, adesc + (UP_A_ATOM >> 4) + 2 * ks, bdesc + (UP_B_ATOM >> 4) + 2 * ks, IDESC, 1u);
          } else {
#pragma unroll
            for (int ks = 0; ks < KE / 16; ++ks)
              if ((m0 >> ks) & 1) umma2_f16(d_tmem, adesc + 2 * ks, bdesc + 2 * ks, IDESC, 1u);
            commit_both(B_TFULL + acc);    // P is complete: the epilogues start on the first expert
            if (KSEL == 2) {
              // Q has one buffer: both epilogues of the previous tile must have drained it.  They are
              // then already busy with P of this tile, so the wait and the Q product hide behind that.
              if (!mbar_wait_cluster(local(B_QEMPTY), (tile_i & 1u) ^ 1u, abort_flag)) { failed = true; break; }
              tc_fence_after();
              int m = m0 | m1;
              if (m == 0) m = 1;           // Q must be written at least once (A is zero there)
              uint32_t accum = 0;
#pragma unroll
              for (int ks = 0; ks < KE / 16; ++ks)
                if ((m >> ks) & 1) {
                  umma2_f16(tmem_q, adesc + (UP_A_ATOM >> 4) + 2 * ks, bdesc + (UP_B_ATOM >> 4) + 2 * ks, IDESC, accum);
                  accum = 1;
                }
              commit_both(B_QFULL);
            }
          }
          commit_both(B_EMPTY + s);
          if (++s == STAGES) { s = 0; ph ^= 1u; }
        }
        if (failed) break;
        if (!HAS_R) commit_both(B_TFULL + acc);
      }
    }
  } else if (warp == 2) {
    // ---------------- S products: S_j += a_j U2f^T as the epilogues hand activation chunks over.
    // Both CTAs load their 32 rows of each U2f chunk; the leader issues the MMAs.
    if (HAS_R && lane == 0 && w1 > 0) {
      constexpr uint32_t IDESC_S = idesc_f16(2 * BM, KE);
      auto load_u2 = [&](int w, uint32_t ti) -> bool {
        int pt, nt;
        tile_of(w, pt, nt);
        const int g = p.tile_cluster[pt];
        const uint32_t ub = ti & 1u, uph = (ti >> 1) & 1u;
        if (!mbar_wait_cluster(local(B_U2EMPTY + ub), uph ^ 1u, abort_flag)) return false;
        const uint32_t dst = u2base + ub * U2_TILE_BYTES;
        if (leader) mbar_expect_tx(local(B_U2FULL + ub), 2 * U2_TILE_BYTES);
        tma2_load_2d(dst, &tmU2, lead(B_U2FULL + ub), nt * BN_UP, g * KE + (int)rank * (KE / 2));
        tma2_load_2d(dst + U2_CHUNK_BYTES, &tmU2, lead(B_U2FULL + ub), nt * BN_UP + BK, g * KE + (int)rank * (KE / 2));
        return true;
      };
      uint32_t tile_i = 0, flushes = 0;
      bool fresh = true;                    // the next product of each slot overwrites S
      uint32_t written = 0;                 // bit j: S_j has been written since the last flush
      if (!load_u2(0, 0)) failed = true;
      for (int w = 0; w < w1 && !failed; ++w, ++tile_i) {
        if (w + 1 < w1 && !load_u2(w + 1, tile_i + 1)) { failed = true; break; }
        if (!leader) continue;
        const uint32_t ub = tile_i & 1u, uph = (tile_i >> 1) & 1u;
        if (!mbar_wait_cluster(local(B_U2FULL + ub), uph, abort_flag)) { failed = true; break; }
        if (fresh && flushes > 0) {
          // both epilogues must have read the previous unit's S before it is overwritten
          if (!mbar_wait_cluster(local(B_SEMPTY), (flushes - 1) & 1u, abort_flag)) { failed = true; break; }
          tc_fence_after();
        }
        if (fresh) { written = 0; fresh = false; }
        for (int c = 0; c < 2 * KSEL; ++c) {
          const uint32_t n = tile_i * (2 * KSEL) + c;
          const uint32_t slot = n % Cfg::NA, aph = (n / Cfg::NA) & 1u;
          if (!mbar_wait_cluster(local(B_AFULL + slot), aph, abort_flag)) { failed = true; break; }
          tc_fence_after();
          const int j = c >> 1, hf = c & 1;      // first-expert chunks of both halves first: the order the epilogues hand them over
          const uint64_t adesc = umma_desc(aring + slot * A_CHUNK_BYTES);
          const uint64_t bdesc = umma_desc(u2base + ub * U2_TILE_BYTES + hf * U2_CHUNK_BYTES);
#pragma unroll
          for (int ks = 0; ks < BK / 16; ++ks) {
            umma2_f16(tmem_s + j * KE, adesc + 2 * ks, bdesc + 2 * ks, IDESC_S, (written >> j) & 1u);
            written |= 1u << j;
          }
          commit_both(B_AEMPTY + slot);
        }
        if (failed) break;
        commit_both(B_U2EMPTY + ub);
        if ((w + 1) % unit == 0) { commit_both(B_SFULL); fresh = true; ++flushes; }
      }
    }
  } else {
    // ---------------- epilogue warps (both CTAs): quadrant q of this CTA's TMEM lanes, 32 of the
    // tile's 128 columns (quarter cq); packed fp16 arithmetic after h_2 = P + Q in fp32
    const int ew = warp - UP_EPI_WARP0;
    const int q = warp & 3;                                // the TMEM lanes a warp may read: 32 (warp % 4) ..
    const int cq = ew >> 2;
    const int hf = cq >> 1;                                // which 64-column activation chunk
    const int rowc = q * 32 + lane;                        // row inside this CTA's 128 rows
    const uint32_t taddr = tmem_base + ((uint32_t)(q * 32) << 16);
    uint32_t tile_i = 0, flushes = 0;
    for (int w = 0; w < w1; ++w, ++tile_i) {
      int pt, nt;
      tile_of(w, pt, nt);
      const uint32_t acc = tile_i & 1u, aph = (tile_i >> 1) & 1u;
      const int row = (2 * pt + (int)rank) * BM + rowc;
      const float g0f = p.row_gate[(size_t)row * p.k];
      const float g1f = p.k == 2 ? p.row_gate[(size_t)row * p.k + 1] : 0.f;
      const __half2 g0 = __float2half2_rn((HAS_R && KSEL == 2) ? g0f : g0f + g1f), g1 = __float2half2_rn(g1f);
      {
        const bool ok = mbar_wait_cluster(local(B_TFULL + acc), aph, abort_flag);
        if (!__all_sync(0xffffffffu, ok)) { failed = true; break; }
      }
      tc_fence_after();
      // Phase A (needs P only): a_1 = GELU(h_1) of the first kept expert, its share of abar, its chunk
      // of the S operand.  Phase B (needs Q, which the leader issues meanwhile): h_2 = P + Q, a_2.
      uint32_t ob[2][8];                                   // abar, stored after the hand-overs below
      auto put_chunk = [&](int j, int sub, const uint32_t* src) {
        // a_j into its chunk as a K-major 128-byte-swizzled A operand: 16-byte unit u of row rowc sits at
        // rowc*128 + ((u ^ (rowc & 7)) << 4); this warp owns units 4 (cq & 1) + 2 sub + {0, 1}
        const uint32_t n = tile_i * (2 * KSEL) + j * 2 + hf;
        const uint32_t cb = aring + (n % Cfg::NA) * A_CHUNK_BYTES + rowc * 128;
#pragma unroll
        for (int i = 0; i < 2; ++i) {
          const uint32_t un = (uint32_t)((cq & 1) * 4 + sub * 2 + i);
          st_shared_v4(cb + ((un ^ (uint32_t)(rowc & 7)) << 4), src[4 * i], src[4 * i + 1], src[4 * i + 2], src[4 * i + 3]);
        }
      };
      auto chunk_free = [&](int j) {       // the S product that read this slot one tile ago has finished
        const uint32_t n = tile_i * (2 * KSEL) + j * 2 + hf;
        const bool ok = mbar_wait_cluster(local(B_AEMPTY + n % Cfg::NA), ((n / Cfg::NA) & 1u) ^ 1u, abort_flag);
        return __all_sync(0xffffffffu, ok);
      };
      auto chunk_done = [&](int j) {
        fence_async_smem();
        __syncwarp();
        const uint32_t n = tile_i * (2 * KSEL) + j * 2 + hf;
        if (lane == 0) mbar_arrive_cluster_relaxed(lead(B_AFULL + n % Cfg::NA));   // after fence.proxy.async
      };
      if (HAS_R && !chunk_free(0)) { failed = true; break; }
#pragma unroll
      for (int sub = 0; sub < 2; ++sub) {
        uint32_t vp[16], oa0[8];
        tmem_ld16_nowait(taddr + acc * BN_UP + cq * 32 + sub * 16, vp);
        tmem_ld_wait();
#pragma unroll
        for (int c = 0; c < 16; c += 2) {
          const __half2 a0 = gelu_fast2(__floats2half2_rn(__uint_as_float(vp[c]), __uint_as_float(vp[c + 1])));
          ob[sub][c >> 1] = h2u(__hmul2(g0, a0));
          oa0[c >> 1] = h2u(a0);
        }
        if (HAS_R) put_chunk(0, sub, oa0);
      }
      if (HAS_R) chunk_done(0);
      if (HAS_R && KSEL == 2) {
        {
          const bool ok = mbar_wait_cluster(local(B_QFULL), tile_i & 1u, abort_flag);
          if (!__all_sync(0xffffffffu, ok)) { failed = true; break; }
        }
        tc_fence_after();
        if (!chunk_free(1)) { failed = true; break; }
#pragma unroll
        for (int sub = 0; sub < 2; ++sub) {
          const int col0 = cq * 32 + sub * 16;
          uint32_t vp[16], vq[16], oa1[8];
          tmem_ld16_nowait(taddr + acc * BN_UP + col0, vp);
          tmem_ld16_nowait(taddr + 256 + col0, vq);
          tmem_ld_wait();
#pragma unroll
          for (int c = 0; c < 16; c += 2) {
            const __half2 a1 = gelu_fast2(__floats2half2_rn(__uint_as_float(vp[c]) + __uint_as_float(vq[c]),
                                                            __uint_as_float(vp[c + 1]) + __uint_as_float(vq[c + 1])));
            const uint32_t prev = ob[sub][c >> 1];
            ob[sub][c >> 1] = h2u(__hfma2(g1, a1, *reinterpret_cast<const __half2*>(&prev)));
            oa1[c >> 1] = h2u(a1);
          }
          put_chunk(1, sub, oa1);
        }
        chunk_done(1);
      }
      // accumulators drained: hand P (and Q) back to the leader's MMA warp
      tc_fence_before();
      __syncwarp();
      if (lane == 0) { mbar_arrive_cluster_relaxed(lead(B_TEMPTY + acc)); mbar_arrive_cluster_relaxed(lead(B_QEMPTY)); }
      // abar goes out last: a release at cluster scope waits for the thread's earlier global stores,
      // and by the next tile's hand-overs these have long landed
      {
        __half* dst = p.abar + (size_t)row * p.N + nt * BN_UP + cq * 32;     // 64-byte aligned: two whole sectors
#pragma unroll
        for (int sub = 0; sub < 2; ++sub) st_global_v8(dst + 16 * sub, ob[sub]);
      }
      if (HAS_R && (w + 1) % unit == 0) {
        if (hf < KSEL) {
          // S_hf is complete for this unit.  The warp walks over the expert blocks of the expanded
          // index (this warp: every other block); lanes whose row uses the block add it to s.
          const bool ok = mbar_wait_cluster(local(B_SFULL), flushes & 1u, abort_flag);
          if (!__all_sync(0xffffffffu, ok)) { failed = true; break; }
          tc_fence_after();
          const int g = p.tile_cluster[pt];
          const int e = p.row_slot[(size_t)row * KSEL + hf] - g * p.K;
          const bool real = p.row_token[row] >= 0;
          float* srow = p.s_out + ((size_t)row * KSEL + hf) * p.r;
          const int r = p.r;
          for (int i = cq & 1; i < p.K; i += 2) {
            const uint32_t ta = taddr + 384 + hf * KE + i * r;
            const bool mine = real && e == i;
            if (r == 16) {
              uint32_t v[16];
              tmem_ld16_nowait(ta, v);
              tmem_ld_wait();
              if (mine) {
#pragma unroll
                for (int c = 0; c < 16; c += 4)
                  red_add_v4(srow + c, __uint_as_float(v[c]), __uint_as_float(v[c + 1]), __uint_as_float(v[c + 2]), __uint_as_float(v[c + 3]));
              }
            } else if (r == 32) {
              uint32_t v[32];
              tmem_ld32_nowait(ta, v);
              tmem_ld_wait();
              if (mine) {
#pragma unroll
                for (int c = 0; c < 32; c += 4)
                  red_add_v4(srow + c, __uint_as_float(v[c]), __uint_as_float(v[c + 1]), __uint_as_float(v[c + 2]), __uint_as_float(v[c + 3]));
              }
            } else if (r == 8) {
              uint32_t v[8];
              tmem_ld8_nowait(ta, v);
              tmem_ld_wait();
              if (mine) {
                red_add_v4(srow, __uint_as_float(v[0]), __uint_as_float(v[1]), __uint_as_float(v[2]), __uint_as_float(v[3]));
                red_add_v4(srow + 4, __uint_as_float(v[4]), __uint_as_float(v[5]), __uint_as_float(v[6]), __uint_as_float(v[7]));
              }
            } else {
              uint32_t v[4];
              tmem_ld4_nowait(ta, v);
              tmem_ld_wait();
              if (mine) red_add_v4(srow, __uint_as_float(v[0]), __uint_as_float(v[1]), __uint_as_float(v[2]), __uint_as_float(v[3]));
            }
          }
          tc_fence_before();
          __syncwarp();
          if (lane == 0) mbar_arrive_cluster_relaxed(lead(B_SEMPTY));
        }
        ++flushes;
      }
    }
  }

  if (failed) {
    *abort_flag = 1;
    st_cluster_u32(mapa(smem_u32(const_cast<int*>(abort_flag)), rank ^ 1u), 1u);   // the peer gives up too
    atomicExch(p.status, (int)CMOE_ERR_TIMEOUT);
  }
  __syncthreads();
  if (*abort_flag) {
    const unsigned long long t0 = global_ns();
    while (global_ns() - t0 < 200000ull) { }    // let copies already issued land
  }
  tc_fence_before();
  cluster_sync_all();      // neither CTA leaves while the other may still use its shared memory or barriers
  tc_fence_after();
  if (warp == 0)
    asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(kTmemCols) : "memory");
}

// ------------------------------------------------------------------------------------------------
// down: CTA pairs on 256 x BN tiles
// ------------------------------------------------------------------------------------------------
struct Down2Params {
  const int* n_rows;
  const int* tile_cluster;   // per 256-row tile
  const int* tile_mask;      // per 128-row tile: 16-wide steps of As V2f^T in use
  const int* row_token;
  __half* y;           // [T][N], original token order
  int* status;
  int KC, NT, N;
  int bshift;          // the base of cluster g is that of g >> bshift (expert halves or quarters share their cluster's base)
  // Not null: the up kernel left the sums s = a_j U2_e in fp32 (its work units were parts of a row tile) and this
  // kernel turns them into its own operand As[row][block of e_j] = fp16(p_j s_j), row tile by row tile, in the
  // epilogue warps while they wait for the tile's main loop.
  const float* s;            // [rows][k][r]
  const int* row_slot;       // [rows][k]
  const float* row_gate;     // [rows][k]
  __half* As;                // [rows][KE]
  int K, k, r;
};

constexpr int DN_THREADS = 224;   // warps 0 and 6 TMA (alternating stages), warp 1 MMA, warps 2..5 epilogue

template <int BN, bool HAS_R>
struct DownCfg {
  static constexpr uint32_t A_ATOM = BM * BK * 2;
  static constexpr uint32_t B_ATOM = (BN / 2) * BK * 2;        // this CTA's half of the B tile, one K atom
  static constexpr uint32_t A_BYTES = KA * A_ATOM;
  static constexpr uint32_t B_BYTES = KA * B_ATOM;
  static constexpr uint32_t STAGE_BYTES = A_BYTES + B_BYTES;   // 64 KB (BN = 256) / 48 KB
  static constexpr int STAGES = BN == 256 ? 3 : 4;
  static constexpr size_t SMEM = 1024 + (size_t)STAGES * STAGE_BYTES + 32 * 8;
};

template <int BN, bool HAS_R>
__global__ void __launch_bounds__(DN_THREADS, 1)
tc2_down_kernel(const __grid_constant__ CUtensorMap tmA3, const __grid_constant__ CUtensorMap tmB23,
                const __grid_constant__ CUtensorMap tmAs, const __grid_constant__ CUtensorMap tmV2,
                const Down2Params p) {
  using Cfg = DownCfg<BN, HAS_R>;
  constexpr int STAGES = Cfg::STAGES;
  constexpr uint32_t STAGE_BYTES = Cfg::STAGE_BYTES;
  extern __shared__ uint8_t smem_raw[];
  const uint32_t raw = smem_u32(smem_raw);
  const uint32_t base = (raw + 1023u) & ~1023u;
  uint8_t* sm = smem_raw + (base - raw);
  uint64_t* bars = reinterpret_cast<uint64_t*>(sm + (size_t)STAGES * STAGE_BYTES);
  const uint32_t bar0 = smem_u32(bars);
  uint32_t* tmem_holder = reinterpret_cast<uint32_t*>(bars + 20);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_holder + 1);
  constexpr int B_ASREADY = 24;       // this CTA's rows of As have been written (four epilogue warps arrive)
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const uint32_t rank = cluster_ctarank();
  const bool leader = rank == 0;
  const uint32_t cbar[2] = {mapa(bar0, 0), mapa(bar0, 1)};
  auto local = [&](int slot) { return bar0 + 8u * slot; };
  auto lead = [&](int slot) { return cbar[0] + 8u * slot; };
  auto commit_both = [&](int slot) { umma2_commit(cbar[0] + 8u * slot); umma2_commit(cbar[1] + 8u * slot); };

  if (threadIdx.x == 0) {
    for (int s = 0; s < STAGES; ++s) { mbar_init(local(B_FULL + s), 1); mbar_init(local(B_EMPTY + s), 1); }
    for (int a = 0; a < 2; ++a) { mbar_init(local(B_TFULL + a), 1); mbar_init(local(B_TEMPTY + a), 8); }
    mbar_init(local(B_ASREADY), 4);
    *abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 0) {
    __syncwarp();
    asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;"
                 ::"r"(smem_u32(tmem_holder)), "r"(kTmemCols) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  cluster_sync_all();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_holder;
  pdl_wait();                  // nothing above reads what an earlier kernel wrote
  pdl_release_dependents();

  const int NT = p.NT, KC = p.KC;
  const int pair = blockIdx.x >> 1, npairs = gridDim.x >> 1;
  const int total = (*p.n_rows / (2 * BM)) * NT;
  constexpr int NEXT = HAS_R ? 1 : 0;
  bool failed = false;

  if (warp == 0 || warp == 6) {
    // two producer threads take alternate stages
    if (lane == 0) {
      const int spt = KC + NEXT;
      const int my_tiles = pair < total ? (total - 1 - pair) / npairs + 1 : 0;
      const uint32_t n_it = (uint32_t)my_tiles * spt;
      for (uint32_t it = warp == 0 ? 0u : 1u; it < n_it && !failed; it += 2) {
        const int ti = it / spt, c = it - ti * spt;
        const int w = pair + ti * npairs;
        const int pt = w / NT, nt = w - pt * NT;
        const int g = p.tile_cluster[pt];
        const int arow = (2 * pt + (int)rank) * BM;
        const int ncol = nt * BN + (int)rank * (BN / 2);
        const int brow = (g >> p.bshift) * p.N + ncol;        // base rows: of the cluster that owns the base
        const int vrow = g * p.N + ncol;                      // staged factor rows: of this (virtual) cluster
        const uint32_t s = it % STAGES, ph = (it / STAGES) & 1u;
        if (!mbar_wait_cluster(local(B_EMPTY + s), ph ^ 1u, abort_flag)) { failed = true; break; }
        const uint32_t a_dst = base + s * STAGE_BYTES, b_dst = a_dst + Cfg::A_BYTES;
        if (c < KC) {
          if (leader) mbar_expect_tx(local(B_FULL + s), 2 * STAGE_BYTES);
          tma2_load_3d(a_dst, &tmA3, lead(B_FULL + s), 0, arow, c * KA);
          tma2_load_3d(b_dst, &tmB23, lead(B_FULL + s), 0, brow, c * KA);
        } else {
          // (this CTA's epilogue warps have written the tile's rows of As, if that is this kernel's job)
          if (p.s && !mbar_wait(local(B_ASREADY), (uint32_t)ti & 1u, abort_flag)) { failed = true; break; }
          if (leader) mbar_expect_tx(local(B_FULL + s), 2 * (Cfg::A_ATOM + Cfg::B_ATOM));
          tma2_load_2d(a_dst, &tmAs, lead(B_FULL + s), 0, arow);
          tma2_load_2d(b_dst, &tmV2, lead(B_FULL + s), 0, vrow);
        }
      }
    }
  } else if (warp == 1) {
    if (lane == 0 && leader) {
      constexpr uint32_t IDESC = idesc_f16(2 * BM, BN);
      uint32_t it = 0, tile_i = 0;
      for (int w = pair; w < total && !failed; w += npairs, ++tile_i) {
        const int pt = w / NT;
        const uint32_t acc = tile_i & 1u, aph = (tile_i >> 1) & 1u;
        if (!mbar_wait_cluster(local(B_TEMPTY + acc), aph ^ 1u, abort_flag)) { failed = true; break; }
        tc_fence_after();
        const uint32_t d_tmem = tmem_base + acc * BN;
        for (int c = 0; c < KC + NEXT; ++c, ++it) {
          const uint32_t s = it % STAGES, ph = (it / STAGES) & 1u;
          if (!mbar_wait_cluster(local(B_FULL + s), ph, abort_flag)) { failed = true; break; }
          tc_fence_after();
          const uint32_t a_src = base + s * STAGE_BYTES, b_src = a_src + Cfg::A_BYTES;
          if (c < KC) {
#pragma unroll
            for (int a = 0; a < KA; ++a) {
              const uint64_t adesc = umma_desc(a_src + a * Cfg::A_ATOM), bdesc = umma_desc(b_src + a * Cfg::B_ATOM);
#pragma unroll
              for (int ks = 0; ks < BK / 16; ++ks)
                umma2_f16(d_tmem, adesc + 2 * ks, bdesc + 2 * ks, IDESC, (c | a | ks) != 0 ? 1u : 0u);
            }
          } else {
            const uint64_t adesc = umma_desc(a_src), bdesc = umma_desc(b_src);
            const int m = p.tile_mask[2 * pt] | p.tile_mask[2 * pt + 1];        // (the down projection's own table)
#pragma unroll
            for (int ks = 0; ks < KE / 16; ++ks)
              if ((m >> ks) & 1) umma2_f16(d_tmem, adesc + 2 * ks, bdesc + 2 * ks, IDESC, 1u);
          }
          commit_both(B_EMPTY + s);
        }
        if (failed) break;
        commit_both(B_TFULL + acc);
      }
    }
  } else {
    const int q = warp & 3;
    const uint32_t taddr = tmem_base + ((uint32_t)(q * 32) << 16);
    uint32_t tile_i = 0;
    for (int w = pair; w < total; w += npairs, ++tile_i) {
      const int pt = w / NT, nt = w - pt * NT;
      const uint32_t acc = tile_i & 1u, aph = (tile_i >> 1) & 1u;
      const int tok = p.row_token[(2 * pt + (int)rank) * BM + q * 32 + lane];
      if (HAS_R && p.s) {
        // As of this thread's row: fp16(p_j s_j) inside the block of e_j, zeros elsewhere (the whole row is written,
        // so As needs no clearing; tiles of the same row tile write the same values again)
        const int row = (2 * pt + (int)rank) * BM + q * 32 + lane;
        const int g = p.tile_cluster[pt];
        uint4* arow = reinterpret_cast<uint4*>(p.As + (size_t)row * KE);
#pragma unroll
        for (int u = 0; u < KE / 8; ++u) {
          float f[8];
#pragma unroll
          for (int n = 0; n < 8; ++n) f[n] = 0.f;
          if (tok >= 0) {
            for (int j = 0; j < p.k; ++j) {
              const int lo = (p.row_slot[(size_t)row * p.k + j] - g * p.K) * p.r;      // first column of the block of e_j
              const float gate = p.row_gate[(size_t)row * p.k + j];
              const float* sj = p.s + ((size_t)row * p.k + j) * p.r;
#pragma unroll
              for (int n = 0; n < 8; ++n) {
                const int c = 8 * u + n - lo;
                if (c >= 0 && c < p.r) f[n] = gate * __ldcg(sj + c);
              }
            }
          }
          arow[u] = make_uint4(pack_half2(f[0], f[1]), pack_half2(f[2], f[3]), pack_half2(f[4], f[5]), pack_half2(f[6], f[7]));
        }
        asm volatile("fence.proxy.async.global;" ::: "memory");      // the tile load of As (async proxy) comes after these writes
        __syncwarp();
        if (lane == 0) mbar_arrive(local(B_ASREADY));
      }
      {
        const bool ok = mbar_wait_cluster(local(B_TFULL + acc), aph, abort_flag);
        if (!__all_sync(0xffffffffu, ok)) { failed = true; break; }
      }
      tc_fence_after();
#pragma unroll 1
      for (int c0 = 0; c0 < BN; c0 += 32) {
        uint32_t v[32];
        tmem_ld32_nowait(taddr + acc * BN + c0, v);
        tmem_ld_wait();
        if (tok >= 0) {
          uint32_t o[16];
#pragma unroll
          for (int c = 0; c < 32; c += 2) o[c >> 1] = pack_half2(__uint_as_float(v[c]), __uint_as_float(v[c + 1]));
          __half* dst = p.y + (size_t)tok * p.N + nt * BN + c0;                 // 64-byte aligned: two whole sectors
          st_global_v8(dst, o);
          st_global_v8(dst + 16, o + 8);
        }
      }
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive_cluster_relaxed(lead(B_TEMPTY + acc));
    }
  }

  if (failed) {
    *abort_flag = 1;
    st_cluster_u32(mapa(smem_u32(const_cast<int*>(abort_flag)), rank ^ 1u), 1u);
    atomicExch(p.status, (int)CMOE_ERR_TIMEOUT);
  }
  __syncthreads();
  if (*abort_flag) {
    const unsigned long long t0 = global_ns();
    while (global_ns() - t0 < 200000ull) { }
  }
  tc_fence_before();
  cluster_sync_all();
  tc_fence_after();
  if (warp == 0)
    asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(kTmemCols) : "memory");
}

// ------------------------------------------------------------------------------------------------
// host side
// ------------------------------------------------------------------------------------------------
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

// The same matrix seen as [cols / 64][rows][64]: a box of 64 x box_rows x KA lands in shared memory as KA
// consecutive 128-byte-swizzled [box_rows][64] tiles, one per K atom.
bool make_map3(CUtensorMap* map, const void* ptr, uint64_t rows, uint64_t cols, uint32_t box_rows) {
  EncodeTiledFn enc = get_encode();
  if (!enc) return false;
  cuuint64_t gdim[3] = {(cuuint64_t)BK, rows, cols / BK};
  cuuint64_t gstride[2] = {cols * 2, (cuuint64_t)BK * 2};
  cuuint32_t box[3] = {(cuuint32_t)BK, box_rows, (cuuint32_t)KA};
  cuuint32_t estr[3] = {1, 1, 1};
  return enc(map, CU_TENSOR_MAP_DATA_TYPE_FLOAT16, 3, const_cast<void*>(ptr), gdim, gstride, box, estr,
             CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
             CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

struct Tc2State {
  CUtensorMap mX, mX3, mB13, mA0, mAd, mV1, mU2;   // up (mX: 2-D, for the t kernel and the wide up kernel)
  CUtensorMap mB13w, mV1w;                     // wide up kernel: 128-row boxes of B1t and V1f
  CUtensorMap mU1;                             // t
  CUtensorMap mAbar3, mB23, mAs, mV2;          // down
  int bn_down;
  int up_wide;       // d_ff is a multiple of 256: the up kernel on 256-column tiles (tc2_up_wide.cu)
  int sm_count;
  int log2r;
};
static_assert(sizeof(Tc2State) <= sizeof(((cmoe_layer*)nullptr)->tc_state), "tc_state too small");

template <bool HAS_R, int KSEL>
cudaError_t launch_up(const Tc2State& ts, const Up2Params& p, int grid, cudaStream_t st) {
  auto kern = tc2_up_kernel<HAS_R, KSEL>;
  constexpr size_t sm = UpCfg<HAS_R, KSEL>::SMEM;
  static_assert(sm <= kSmemLimit, "up kernel shared memory");
  static std::atomic<unsigned long long> smem_set{0};      // devices the kernel's shared-memory limit has been raised on
  if (cudaError_t e = ensure_dynamic_smem(kern, sm, smem_set)) return e;
  return launch_pairs(kern, grid, UP_THREADS, sm, st, ts.mX3, ts.mB13, ts.mA0, ts.mAd, ts.mV1, ts.mU2, p);
}

template <int BN, bool HAS_R>
cudaError_t launch_down(const Tc2State& ts, const Down2Params& p, int grid, cudaStream_t st) {
  auto kern = tc2_down_kernel<BN, HAS_R>;
  constexpr size_t sm = DownCfg<BN, HAS_R>::SMEM;
  static_assert(sm <= kSmemLimit, "down kernel shared memory");
  static std::atomic<unsigned long long> smem_set{0};      // devices the kernel's shared-memory limit has been raised on
  if (cudaError_t e = ensure_dynamic_smem(kern, sm, smem_set)) return e;
  return launch_pairs(kern, grid, DN_THREADS, sm, st, ts.mAbar3, ts.mB23, ts.mAs, ts.mV2, p);
}

template <int KSEL, bool GATHER>
cudaError_t launch_t(const Tc2State& ts, const CUtensorMap& x_src, const TParams& p, int grid, cudaStream_t st) {
  auto kern = tc2_t_kernel<KSEL, GATHER>;
  constexpr size_t sm = 1024 + (size_t)T_STAGES * T_STAGE_BYTES + 32 * 8 + BM * sizeof(int);
  static std::atomic<unsigned long long> smem_set{0};      // devices the kernel's shared-memory limit has been raised on
  if (cudaError_t e = ensure_dynamic_smem(kern, sm, smem_set)) return e;
  launch_chained(kern, dim3(grid), dim3(T_THREADS), sm, st, 1,
      ts.mX, ts.mU1, x_src, p);
  return cudaGetLastError();
}

// N tiles per work unit of the up kernel: the largest divisor of NT up to 4 (S is flushed once per
// unit) that still leaves every SM a unit
int pick_unit(int NT, int pt_bound, int pairs) {
  int unit = 1;
  for (int u = 2; u <= 4; ++u)
    if (NT % u == 0 && (long long)pt_bound * (NT / u) >= 2LL * pairs) unit = u;
  return unit;
}

int ilog2(int v) { int l = 0; while ((1 << l) < v) ++l; return l; }

// Launch shape of the up kernel for a batch of T tokens.  A unit that is a whole row tile (unit == NT) leaves
// S complete at its end: the wide kernel then writes the gated rows p_j s_j straight into the down kernel's
// operand (`direct`), without fp32 reductions into s and without the expansion kernel.  Whole-row units are
// taken when they keep the pairs as busy as the default units do.
struct UpPlan {
  int NT, unit, grid;
  bool direct;
};
UpPlan plan_up(const Tc2State& ts, const Dims& D, int T) {
  UpPlan u{};
  const int pt_bound = t_pad_bound(D, T) / (2 * BM), pairs = ts.sm_count / 2;
  u.NT = D.d_ff / (ts.up_wide ? BN_WIDE : BN_UP);
  u.unit = pick_unit(u.NT, pt_bound, pairs);
  if (ts.up_wide && D.r > 0 && u.unit != u.NT) {
    auto eff = [&](int unit) {
      const long long n = (long long)pt_bound * (u.NT / unit), rounds = (n + pairs - 1) / pairs;
      return (double)n / (double)(rounds * pairs);
    };
    if (eff(u.NT) >= eff(u.unit) - 0.02) u.unit = u.NT;
  }
  u.direct = ts.up_wide && D.r > 0 && u.unit == u.NT;
  const long long total = (long long)pt_bound * (u.NT / u.unit);
  u.grid = 2 * (int)(total < pairs ? total : pairs);
  return u;
}

}  // namespace

bool tc2_supported(const Dims& D) {
  if (D.d % 128 || D.d_ff % 128) return false;
  if (D.k != 1 && D.k != 2) return false;
  if (!(D.r == 0 || D.r == 4 || D.r == 8 || D.r == 16 || D.r == 32)) return false;
  if (D.K * D.r > KE) return false;
  return true;      // (cmoe_create then aligns the clusters' row segments to 256)
}

cudaError_t tc2_init(cmoe_layer* L) {
  const Dims& D = L->dims;
  const Scratch& S = L->sc;
  Tc2State* ts = reinterpret_cast<Tc2State*>(L->tc_state);
  ts->bn_down = (D.d % 256 == 0) ? 256 : 128;
  ts->up_wide = (D.d_ff % BN_WIDE == 0 && L->opt.up_tile != 128) ? 1 : 0;
  ts->log2r = D.r > 0 ? ilog2(D.r) : 0;
  ts->sm_count = D.sm_count;
  cudaError_t e;
  const uint64_t P = (uint64_t)D.T_pad_max, G = (uint64_t)D.G, Gb = (uint64_t)real_G(D);     // Gb: bases, one per real cluster
  bool ok = make_map(&ts->mX, S.x_perm, P, D.d, BM) &&
            make_map3(&ts->mX3, S.x_perm, P, D.d, BM) &&
            make_map3(&ts->mB13, L->w.B1t, Gb * D.d_ff, D.d, BN_UP / 2) &&
            make_map3(&ts->mB13w, L->w.B1t, Gb * D.d_ff, D.d, BN_WIDE / 2) &&
            make_map3(&ts->mAbar3, S.abar, P, D.d_ff, BM) &&
            make_map3(&ts->mB23, L->w.B2t, Gb * D.d, D.d_ff, ts->bn_down / 2);
  if (ok && D.r > 0) {
    ok = make_map(&ts->mA0, S.A0, P, KE, BM) && make_map(&ts->mAd, S.Ad, P, KE, BM) &&
         make_map(&ts->mAs, S.As, P, KE, BM) &&
         make_map(&ts->mV1, S.V1f, G * D.d_ff, KE, BN_UP / 2) &&
         make_map(&ts->mV1w, S.V1f, G * D.d_ff, KE, BN_WIDE / 2) &&
         make_map(&ts->mV2, S.V2f, G * D.d, KE, ts->bn_down / 2) &&
         make_map(&ts->mU1, S.U1f, G * KE, D.d, KE) &&
         make_map(&ts->mU2, S.U2f, G * KE, D.d_ff, KE / 2);
    // the padding rows / columns of the staged factors (K*r < 64) stay zero for the handle's life
    const size_t f16 = sizeof(__half);
    if (ok) {
      if ((e = cudaMemset(S.U1f, 0, G * KE * D.d * f16)) != cudaSuccess) return e;
      if ((e = cudaMemset(S.V1f, 0, G * D.d_ff * KE * f16)) != cudaSuccess) return e;
      if ((e = cudaMemset(S.U2f, 0, G * KE * D.d_ff * f16)) != cudaSuccess) return e;
      if ((e = cudaMemset(S.V2f, 0, G * D.d * KE * f16)) != cudaSuccess) return e;
    }
  } else if (ok) {
    // unused maps still have to be valid kernel arguments
    ts->mA0 = ts->mX; ts->mAd = ts->mX; ts->mV1 = ts->mX; ts->mU2 = ts->mX; ts->mU1 = ts->mX;
    ts->mAs = ts->mX; ts->mV2 = ts->mX; ts->mV1w = ts->mX;
  }
  return ok ? cudaSuccess : cudaErrorInvalidValue;
}

// what the permutation's scan kernel stages beside its own work (tc2 path with residuals; else nothing)
void tc2_factor_stage(const cmoe_layer* L, FactorStage* fs) {
  const Dims& D = L->dims;
  const Weights& W = L->w;
  const Scratch& S = L->sc;
  *fs = FactorStage{};
  if (D.r == 0) return;
  const uint8_t* q[4] = {W.U1q, W.V1q, W.U2q, W.V2q};
  const __half* sc[4] = {W.U1s, W.V1s, W.U2s, W.V2s};
  __half* dst[4] = {S.U1f, S.V1f, S.U2f, S.V2f};
  const int dim[4] = {D.d, D.d_ff, D.d_ff, D.d};
  for (int i = 0; i < 4; ++i) {
    fs->q[i] = q[i]; fs->s[i] = sc[i]; fs->dst[i] = dst[i]; fs->dim[i] = dim[i];
    fs->words[i] = (long long)D.E * D.r * dim[i] / 32;      // scale groups of 32 codes
  }
  fs->K = D.K; fs->r = D.r;
}

// (option) the t kernel reads x by row_token and writes x_perm itself: the permutation then moves no rows
bool tc2_gathers_rows(const cmoe_layer* L) { return L->dims.r > 0 && L->opt.row_gather == 1 && L->dims.split <= 1; }

int tc2_launch_count(const cmoe_layer* L) {
  const Dims& D = L->dims;
  if (D.r == 0) return 2;
  const Tc2State& ts = *reinterpret_cast<const Tc2State*>(L->tc_state);
  // t, up, down; the factor staging rides in the router's or the permutation's grid
  return 3;
}

// The buffer the forward's first kernels clear for this path: the fp32 sums s, or the down kernel's
// operand As when the up kernel writes it directly.
void tc2_accum_buffer(const cmoe_layer* L, int T, void** ptr, size_t* bytes) {
  const Dims& D = L->dims;
  const Tc2State& ts = *reinterpret_cast<const Tc2State*>(L->tc_state);
  const size_t rows = (size_t)t_pad_bound(D, T);
  if (D.r > 0 && plan_up(ts, D, T).direct) { *ptr = L->sc.As; *bytes = sizeof(__half) * rows * KE; }
  else { *ptr = L->sc.s; *bytes = sizeof(float) * rows * D.k * D.r; }
}

cudaError_t launch_tc2_ffn(const cmoe_layer* L, const __half* x_src, int T, __half* y, cudaStream_t st, cudaEvent_t* marks) {
  const Dims& D = L->dims;
  const Weights& W = L->w;
  const Scratch& S = L->sc;
  const Tc2State& ts = *reinterpret_cast<const Tc2State*>(L->tc_state);
  const int rows_bound = t_pad_bound(D, T);
  const int mt_bound = rows_bound / BM, pt_bound = rows_bound / (2 * BM);
  cudaError_t e;
  if (marks) cudaEventRecord(marks[0], st);
  if (D.r > 0) {
    TParams tp{};
    tp.n_rows = S.n_rows; tp.tile_cluster = S.tile_cluster; tp.row_slot = S.row_slot; tp.row_token = S.row_token;
    tp.A0 = S.A0; tp.Ad = S.Ad; tp.tile_mask = S.tile_mask; tp.tile_mask_dn = S.tile_mask_dn; tp.live = L->w.live; tp.status = S.status;
    tp.KC = D.d / BK; tp.K = D.K; tp.r = D.r; tp.x_rows = T;
    if (x_src) {
      // the t kernel gathers the rows of x itself (and writes x_perm): a map of this call's x, boxes of one row
      CUtensorMap mx;
      if (!make_map(&mx, x_src, (uint64_t)T, D.d, 1)) return cudaErrorInvalidValue;
      e = D.k == 2 ? launch_t<2, true>(ts, mx, tp, mt_bound, st) : launch_t<1, true>(ts, mx, tp, mt_bound, st);
    } else {
      e = D.k == 2 ? launch_t<2, false>(ts, ts.mX, tp, mt_bound, st) : launch_t<1, false>(ts, ts.mX, tp, mt_bound, st);
    }
    if (e != cudaSuccess) return e;
  }
  if (marks) cudaEventRecord(marks[1], st);
  Up2Params up{};
  up.n_rows = S.n_rows; up.tile_cluster = S.tile_cluster; up.tile_mask = S.tile_mask; up.row_slot = S.row_slot;
  up.row_gate = S.row_gate; up.row_token = S.row_token; up.s_out = S.s; up.abar = S.abar; up.status = S.status;
  up.KC = D.d / (BK * KA); up.NT = D.d_ff / BN_UP; up.N = D.d_ff; up.K = D.K; up.k = D.k; up.r = D.r; up.log2r = ts.log2r;
  up.bshift = D.split > 1 ? ilog2(D.split) : 0;
  const UpPlan plan = plan_up(ts, D, T);
  {
    up.NT = plan.NT;
    up.unit = plan.unit;
    up.As_direct = plan.direct ? S.As : nullptr;
    const int grid = plan.grid;
    if (ts.up_wide) {
      const UpWideMaps maps{&ts.mX3, &ts.mB13w, &ts.mA0, &ts.mAd, &ts.mV1w, &ts.mU2};
      e = launch_up_wide(D.r > 0, D.k, maps, up, grid, st);
    }
    else if (D.r == 0) e = launch_up<false, 1>(ts, up, grid, st);    // without residuals k only enters through the gates
    else if (D.k == 2) e = launch_up<true, 2>(ts, up, grid, st);
    else               e = launch_up<true, 1>(ts, up, grid, st);
    if (e != cudaSuccess) return e;
  }
  if (marks) cudaEventRecord(marks[2], st);
  Down2Params dn{};
  dn.n_rows = S.n_rows; dn.tile_cluster = S.tile_cluster; dn.tile_mask = S.tile_mask_dn; dn.row_token = S.row_token;
  dn.y = y; dn.status = S.status; dn.KC = D.d_ff / (BK * KA); dn.NT = D.d / ts.bn_down; dn.N = D.d;
  dn.bshift = D.split > 1 ? ilog2(D.split) : 0;
  if (D.r > 0 && !plan.direct) {
    dn.s = S.s; dn.row_slot = S.row_slot; dn.row_gate = S.row_gate; dn.As = S.As; dn.K = D.K; dn.k = D.k; dn.r = D.r;
  }
  {
    const int pairs = ts.sm_count / 2;
    const long long total = (long long)pt_bound * dn.NT;
    const int grid = 2 * (int)(total < pairs ? total : pairs);
    if (ts.bn_down == 256) e = D.r > 0 ? launch_down<256, true>(ts, dn, grid, st) : launch_down<256, false>(ts, dn, grid, st);
    else                   e = D.r > 0 ? launch_down<128, true>(ts, dn, grid, st) : launch_down<128, false>(ts, dn, grid, st);
  }
  return e;
}

}  // namespace cmoe
