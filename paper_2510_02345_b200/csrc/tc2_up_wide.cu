// Up projection of the CTA-pair path on 256 x 256 tiles (d_ff a multiple of 256), sm_100a.
//
// What bounds the 128-column up kernel is the SM's shared memory: an N = 128 pair MMA reads its
// operands at 96 B/clk while TMA refills the ring and the activation chunks cross shared memory
// twice.  A 256-column tile needs a third less shared-memory traffic per output element, but h_1 and
// h_2 - h_1 as two fp32 accumulators of 256 columns, plus the S accumulators, do not fit the 512
// TMEM columns.  So one accumulator serves both experts of a token (text after Eq. 7: one base
// product per token), in place:
//
//   P  = x_perm B1_g^T + A0 V1f^T          (= h of the first kept expert)      -> epilogues copy P out
//   P += Ad V1f^T                          (= h of the second kept expert)     -> epilogues copy P out
//
// The epilogue warps copy P into registers (packed fp16), hand P back at once and do GELU, the gated
// sum abar and the A operand of  S_j += a_j U2f^T  while the next tile's main loop runs.  a_j never
// touches shared memory: the epilogues store it (fp16 pairs) into spare TMEM columns and the S
// products read their A operand from there, which leaves shared memory to a ring of three 64 KB
// stages (two 64-wide K atoms each, 3-D TMA boxes) and the tile's U2f columns.
// S is accumulated in TMEM over a unit of N tiles; at the unit's end the row's own block of S_j is added
// to s (fp32 reductions) or, when the unit is a whole row tile, written as fp16(p_j s_j) straight into the
// down kernel's operand.
// TMEM columns: P 0..255, S_0 256..319, S_1 320..383, a_j 384..511 (four chunks of 64 activations).
// Warp roles: 0 and 3 TMA (alternating stages), 1 MMA, 2 S products and U2f loads, 4..19 epilogue
// (twenty warps: warps are allocated in fours, and 96 registers per thread fit 20 but not 24).
// Every device wait is bounded: on expiry the kernel records CMOE_ERR_TIMEOUT in the status word,
// all roles leave their loops, TMEM is freed and the kernel returns.
#include "tc2_common.cuh"

namespace cmoe {
namespace tc2c {

namespace {

constexpr int UW_THREADS = 640;
constexpr int UW_EPI_WARP0 = 4, UW_EPI_WARPS = 16;
constexpr int UW_PRODUCERS = 2;
constexpr int UW_KA = 2;                                         // K atoms of 64 halves per stage
constexpr uint32_t UW_A_ATOM = BM * BK * 2;                      // 16 KB: this CTA's 128 rows, one K atom
constexpr uint32_t UW_B_ATOM = (BN_WIDE / 2) * BK * 2;           // 16 KB: this CTA's half of the B tile
constexpr uint32_t UW_A_BYTES = UW_KA * UW_A_ATOM;
constexpr uint32_t UW_B_BYTES = UW_KA * UW_B_ATOM;
constexpr uint32_t UW_STAGE_BYTES = UW_A_BYTES + UW_B_BYTES;     // 64 KB
constexpr int UW_CHUNKS = BN_WIDE / BK;                          // activation chunks per tile and expert
constexpr uint32_t UW_U2_PIECE = (KE / 2) * BK * 2;              //  4 KB: this CTA's 32 rows of a 64 x 64 piece of U2f
constexpr uint32_t UW_U2_BYTES = UW_CHUNKS * UW_U2_PIECE;
constexpr uint32_t UW_TMEM_S = BN_WIDE, UW_TMEM_A = BN_WIDE + 2 * KE;   // first columns of S and of the a_j operand

enum : int { W_FULL = 0, W_EMPTY = 4, W_TFULL = 8, W_T2FULL = 9, W_PDRAIN = 10, W_TEMPTY = 11, W_AFULL = 12,
             W_AEMPTY = 16, W_U2FULL = 20, W_U2EMPTY = 22, W_SFULL = 24, W_SEMPTY = 25, W_COUNT = 26 };

template <bool HAS_R, int KSEL>
struct WideCfg {
  static constexpr int STAGES = 3;
  static constexpr int NEXT = HAS_R ? 1 : 0;               // one expanded-index stage after the main loop: A0, Ad, V1f
  static constexpr uint32_t RING = STAGES * UW_STAGE_BYTES;
  static constexpr uint32_t U2 = HAS_R ? 2 * UW_U2_BYTES : 0;
  static constexpr uint32_t BAR_OFF = RING + U2;
  static constexpr size_t SMEM = 1024 + BAR_OFF + 32 * 8;
};

template <bool HAS_R, int KSEL>
__global__ void __launch_bounds__(UW_THREADS, 1)
tc2_up_wide_kernel(const __grid_constant__ CUtensorMap tmX3, const __grid_constant__ CUtensorMap tmB13,
                   const __grid_constant__ CUtensorMap tmA0, const __grid_constant__ CUtensorMap tmAd,
                   const __grid_constant__ CUtensorMap tmV1, const __grid_constant__ CUtensorMap tmU2,
                   const Up2Params p) {
  using Cfg = WideCfg<HAS_R, KSEL>;
  constexpr int STAGES = Cfg::STAGES;
  constexpr bool TWO = HAS_R && KSEL == 2;                 // a second pass over P for the second expert
  extern __shared__ uint8_t smem_raw[];
  const uint32_t raw = smem_u32(smem_raw);
  const uint32_t base = (raw + 1023u) & ~1023u;
  uint8_t* sm = smem_raw + (base - raw);
  const uint32_t u2base = base + Cfg::RING;
  uint64_t* bars = reinterpret_cast<uint64_t*>(sm + Cfg::BAR_OFF);
  const uint32_t bar0 = smem_u32(bars);
  uint32_t* tmem_holder = reinterpret_cast<uint32_t*>(bars + W_COUNT);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_holder + 1);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const uint32_t rank = cluster_ctarank();
  const bool leader = rank == 0;
  // the same barrier words in the leader's and in the peer's shared memory (shared::cluster addresses)
  const uint32_t cbar[2] = {mapa(bar0, 0), mapa(bar0, 1)};
  auto local = [&](int slot) { return bar0 + 8u * slot; };
  auto lead = [&](int slot) { return cbar[0] + 8u * slot; };
  auto commit_both = [&](int slot) { umma2_commit(cbar[0] + 8u * slot); umma2_commit(cbar[1] + 8u * slot); };

  if (threadIdx.x == 0) {
    for (int s = 0; s < STAGES; ++s) { mbar_init(local(W_FULL + s), 1); mbar_init(local(W_EMPTY + s), 1); }
    mbar_init(local(W_TFULL), 1);
    mbar_init(local(W_T2FULL), 1);
    mbar_init(local(W_PDRAIN), 2 * UW_EPI_WARPS);
    mbar_init(local(W_TEMPTY), 2 * UW_EPI_WARPS);
    for (int a = 0; a < UW_CHUNKS; ++a) { mbar_init(local(W_AFULL + a), 2 * UW_EPI_WARPS); mbar_init(local(W_AEMPTY + a), 1); }
    for (int a = 0; a < 2; ++a) { mbar_init(local(W_U2FULL + a), 1); mbar_init(local(W_U2EMPTY + a), 1); }
    mbar_init(local(W_SFULL), 1);
    mbar_init(local(W_SEMPTY), UW_EPI_WARPS * KSEL);
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
  const uint32_t tmem_s = tmem_base + UW_TMEM_S, tmem_a = tmem_base + UW_TMEM_A;
  pdl_wait();                  // nothing above reads what an earlier kernel wrote
  pdl_release_dependents();

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
      // Global stage number it = w * spt + c; this thread takes it = pid, pid + 2, ...  Tile coordinates
      // are worked out once per tile and the ring slot advances by two: integer divisions in this loop
      // would cost the single issuing thread more than the loads themselves.
      const int pid = warp == 0 ? 0 : 1;
      const int spt = KC + Cfg::NEXT;                   // stages per tile
      uint32_t s = (uint32_t)pid, ph = 0;
      int c = pid;
      for (int w = 0; w < w1 && !failed; ++w) {
        int pt, nt;
        tile_of(w, pt, nt);
        const int g = p.tile_cluster[pt];
        const int arow = (2 * pt + (int)rank) * BM;
        const int ncol = nt * BN_WIDE + (int)rank * (BN_WIDE / 2);
        const int brow = (g >> p.bshift) * p.N + ncol;        // base rows: of the cluster that owns the base
        const int vrow = g * p.N + ncol;                      // staged factor rows: of this (virtual) cluster
        for (; c < spt; c += UW_PRODUCERS) {
          if (!mbar_wait_cluster(local(W_EMPTY + s), ph ^ 1u, abort_flag)) { failed = true; break; }
          const uint32_t a_dst = base + s * UW_STAGE_BYTES, b_dst = a_dst + UW_A_BYTES;
          if (c < KC) {
            if (leader) mbar_expect_tx(local(W_FULL + s), 2 * UW_STAGE_BYTES);
            tma2_load_3d(a_dst, &tmX3, lead(W_FULL + s), 0, arow, c * UW_KA);
            tma2_load_3d(b_dst, &tmB13, lead(W_FULL + s), 0, brow, c * UW_KA);
          } else {
            // expanded-index stage: A0 (completes h of the first expert), Ad (turns it into the second's), V1f
            if (leader) mbar_expect_tx(local(W_FULL + s), 2 * (KSEL * UW_A_ATOM + UW_B_ATOM));
            tma2_load_2d(a_dst, &tmA0, lead(W_FULL + s), 0, arow);
            if (KSEL == 2) tma2_load_2d(a_dst + UW_A_ATOM, &tmAd, lead(W_FULL + s), 0, arow);
            tma2_load_2d(b_dst, &tmV1, lead(W_FULL + s), 0, vrow);
          }
          s += UW_PRODUCERS;
          if (s >= (uint32_t)STAGES) { s -= STAGES; ph ^= 1u; }
        }
        c -= spt;
      }
    }
  } else if (warp == 1) {
    // ---------------- MMA issuer of P (leader CTA only)
    if (lane == 0 && leader) {
      constexpr uint32_t IDESC = idesc_f16(2 * BM, BN_WIDE);
      uint32_t s = 0, ph = 0;
      auto next_stage = [&]() { if (++s == (uint32_t)STAGES) { s = 0; ph ^= 1u; } };
      for (int w = 0; w < w1 && !failed; ++w) {
        int pt, nt_unused;
        tile_of(w, pt, nt_unused);
        const uint32_t tph = (uint32_t)w & 1u;
        const int m0 = HAS_R ? (p.tile_mask[4 * pt] | p.tile_mask[4 * pt + 2]) : 0;
        const int m1 = HAS_R ? (p.tile_mask[4 * pt + 1] | p.tile_mask[4 * pt + 3]) : 0;
        // both CTAs' epilogues have copied the previous tile out of P
        if (!mbar_wait_cluster(local(W_TEMPTY), tph ^ 1u, abort_flag)) { failed = true; break; }
        tc_fence_after();
        for (int c = 0; c < KC; ++c) {
          if (!mbar_wait_cluster(local(W_FULL + s), ph, abort_flag)) { failed = true; break; }
          tc_fence_after();
          const uint32_t a_src = base + s * UW_STAGE_BYTES, b_src = a_src + UW_A_BYTES;
          const uint64_t adesc = umma_desc(a_src), bdesc = umma_desc(b_src);
          // the second atom's tiles follow the first's: descriptor addresses are in 16-byte units
          umma2_f16(tmem_base, adesc, bdesc, IDESC, c != 0 ? 1u : 0u);
#pragma unroll
          for (int ks = 1; ks < BK / 16; ++ks) umma2_f16(tmem_base, adesc + 2 * ks, bdesc + 2 * ks, IDESC, 1u);
#pragma unroll
          for (int ks = 0; ks < BK / 16; ++ks)
            umma2_f16(tmem_base, adesc + (UW_A_ATOM >> 4) + 2 * ks, bdesc + (UW_B_ATOM >> 4) + 2 * ks, IDESC, 1u);
          commit_both(W_EMPTY + s);
          next_stage();
        }
        if (failed) break;
        if (HAS_R) {
          if (!mbar_wait_cluster(local(W_FULL + s), ph, abort_flag)) { failed = true; break; }
          tc_fence_after();
          const uint32_t a_src = base + s * UW_STAGE_BYTES, b_src = a_src + UW_A_BYTES;
          const uint64_t adesc = umma_desc(a_src), bdesc = umma_desc(b_src);
#pragma unroll
          for (int ks = 0; ks < KE / 16; ++ks)
            if ((m0 >> ks) & 1) umma2_f16(tmem_base, adesc + 2 * ks, bdesc + 2 * ks, IDESC, 1u);
          commit_both(W_TFULL);        // P = h of the first expert
          if (KSEL == 2) {
            // P is updated in place: both CTAs' epilogues must have copied h of the first expert out
            if (!mbar_wait_cluster(local(W_PDRAIN), tph, abort_flag)) { failed = true; break; }
            tc_fence_after();
            const int m = m0 | m1;
#pragma unroll
            for (int ks = 0; ks < KE / 16; ++ks)
              if ((m >> ks) & 1) umma2_f16(tmem_base, adesc + (UW_A_ATOM >> 4) + 2 * ks, bdesc + 2 * ks, IDESC, 1u);
            commit_both(W_T2FULL);     // P = h of the second expert
          }
          commit_both(W_EMPTY + s);
          next_stage();
        } else {
          commit_both(W_TFULL);
        }
      }
    }
  } else if (warp == 2) {
    // ---------------- S products: S_j += a_j U2f^T as the epilogues hand activation chunks over.
    // Both CTAs load their 32 rows of the tile's U2f columns; the leader issues the MMAs.
    if (HAS_R && lane == 0 && w1 > 0) {
      constexpr uint32_t IDESC_S = idesc_f16(2 * BM, KE);
      uint32_t flushes = 0;
      bool fresh = true;                    // the next product of each slot overwrites S
      uint32_t written = 0;                 // bit j: S_j has been written since the last flush
      auto load_u2 = [&](int w) -> bool {
        int pt, nt;
        tile_of(w, pt, nt);
        const int g = p.tile_cluster[pt];
        const uint32_t ub = (uint32_t)w & 1u, uph = ((uint32_t)w >> 1) & 1u;
        if (!mbar_wait_cluster(local(W_U2EMPTY + ub), uph ^ 1u, abort_flag)) return false;
        if (leader) mbar_expect_tx(local(W_U2FULL + ub), 2 * UW_U2_BYTES);
#pragma unroll
        for (int m = 0; m < UW_CHUNKS; ++m)
          tma2_load_2d(u2base + ub * UW_U2_BYTES + m * UW_U2_PIECE, &tmU2, lead(W_U2FULL + ub), nt * BN_WIDE + m * BK,
                       g * KE + (int)rank * (KE / 2));
        return true;
      };
      if (!load_u2(0)) failed = true;
      for (int w = 0; w < w1 && !failed; ++w) {
        if (w + 1 < w1 && !load_u2(w + 1)) { failed = true; break; }
        if (!leader) continue;
        const uint32_t ub = (uint32_t)w & 1u, uph = ((uint32_t)w >> 1) & 1u;
        if (!mbar_wait_cluster(local(W_U2FULL + ub), uph, abort_flag)) { failed = true; break; }
        if (fresh && flushes > 0) {
          // both epilogues must have read the previous unit's S before it is overwritten
          if (!mbar_wait_cluster(local(W_SEMPTY), (flushes - 1) & 1u, abort_flag)) { failed = true; break; }
          tc_fence_after();
        }
        if (fresh) { written = 0; fresh = false; }
        for (int c = 0; c < UW_CHUNKS * KSEL; ++c) {
          const int j = c / UW_CHUNKS, m = c % UW_CHUNKS;
          const uint32_t use = (uint32_t)w * KSEL + j;          // how often chunk slot m has been filled before
          if (!mbar_wait_cluster(local(W_AFULL + m), use & 1u, abort_flag)) { failed = true; break; }
          tc_fence_after();
          const uint64_t bdesc = umma_desc(u2base + ub * UW_U2_BYTES + m * UW_U2_PIECE);
#pragma unroll
          for (int ks = 0; ks < BK / 16; ++ks) {
            // A from tensor memory: 32 columns per chunk, 8 per 16-deep step
            umma2_f16_ts(tmem_s + j * KE, tmem_a + m * (BK / 2) + ks * 8, bdesc + 2 * ks, IDESC_S, (written >> j) & 1u);
            written |= 1u << j;
          }
          commit_both(W_AEMPTY + m);
        }
        if (failed) break;
        commit_both(W_U2EMPTY + ub);
        if ((w + 1) % unit == 0) { commit_both(W_SFULL); fresh = true; ++flushes; }
      }
    }
  } else {
    // ---------------- epilogue warps (both CTAs): quadrant q of this CTA's TMEM lanes; of every 64-column
    // chunk of the tile the 16 columns 16 cq .., so that all warps finish a chunk at about the same time
    const int ew = warp - UW_EPI_WARP0;
    const int q = warp & 3;                                // the TMEM lanes a warp may read: 32 (warp % 4) ..
    const int cq = ew >> 2;
    const int rowc = q * 32 + lane;                        // row inside this CTA's 128 rows
    const uint32_t taddr = tmem_base + ((uint32_t)(q * 32) << 16);
    uint32_t flushes = 0;
    for (int w = 0; w < w1; ++w) {
      int pt, nt;
      tile_of(w, pt, nt);
      const uint32_t tph = (uint32_t)w & 1u;
      const int row = (2 * pt + (int)rank) * BM + rowc;
      const float g0f = p.row_gate[(size_t)row * p.k];
      const float g1f = p.k == 2 ? p.row_gate[(size_t)row * p.k + 1] : 0.f;
      const __half2 g0 = __float2half2_rn(TWO ? g0f : g0f + g1f), g1 = __float2half2_rn(g1f);
      // P -> registers as packed fp16: h[8 m + i] holds columns 64 m + 16 cq + 2 i, + 1 of this thread's row
      auto copy_out = [&](uint32_t* h) {
#pragma unroll
        for (int half = 0; half < 2; ++half) {
          uint32_t va[16], vb[16];
          tmem_ld16_nowait(taddr + (2 * half) * BK + cq * 16, va);
          tmem_ld16_nowait(taddr + (2 * half + 1) * BK + cq * 16, vb);
          tmem_ld_wait();
#pragma unroll
          for (int i = 0; i < 8; ++i) {
            h[(2 * half) * 8 + i] = pack_half2(__uint_as_float(va[2 * i]), __uint_as_float(va[2 * i + 1]));
            h[(2 * half + 1) * 8 + i] = pack_half2(__uint_as_float(vb[2 * i]), __uint_as_float(vb[2 * i + 1]));
          }
        }
      };
      uint32_t h1[32], h2[TWO ? 32 : 1];
      {
        const bool ok = mbar_wait_cluster(local(W_TFULL), tph, abort_flag);
        if (!__all_sync(0xffffffffu, ok)) { failed = true; break; }
      }
      tc_fence_after();
      copy_out(h1);
      if (TWO) {
        tc_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive_cluster_relaxed(lead(W_PDRAIN));
        const bool ok = mbar_wait_cluster(local(W_T2FULL), tph, abort_flag);
        if (!__all_sync(0xffffffffu, ok)) { failed = true; break; }
        tc_fence_after();
        copy_out(h2);
      }
      // P is free for the next tile's main loop; everything below overlaps it
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive_cluster_relaxed(lead(W_TEMPTY));

      // a_j chunk m as the A operand of the S product: this thread's 16 activations (columns 64 m + 16 cq ..)
      // go into 8 columns of its TMEM lane as fp16 pairs
      auto hand_over = [&](int j, int m, const uint32_t* src) -> bool {
        const uint32_t use = (uint32_t)w * KSEL + j;
        // the S product that read this chunk's columns one expert ago has finished
        const bool ok = mbar_wait_cluster(local(W_AEMPTY + m), (use & 1u) ^ 1u, abort_flag);
        if (!__all_sync(0xffffffffu, ok)) return false;
        tc_fence_after();
        tmem_st8(taddr + UW_TMEM_A + m * (BK / 2) + cq * 8, src);
        tmem_st_wait();
        tc_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive_cluster_relaxed(lead(W_AFULL + m));
        return true;
      };
      // first expert: a_1 = GELU(h_1), its share of abar (kept in h1), its chunks of the S operand
#pragma unroll
      for (int m = 0; m < UW_CHUNKS; ++m) {
        uint32_t oa[8];
#pragma unroll
        for (int i = 0; i < 8; ++i) {
          const __half2 a = gelu_fast2(u2h(h1[m * 8 + i]));
          oa[i] = h2u(a);
          h1[m * 8 + i] = h2u(__hmul2(g0, a));
        }
        if (HAS_R && !hand_over(0, m, oa)) { failed = true; break; }
      }
      if (failed) break;
      if (TWO) {
#pragma unroll
        for (int m = 0; m < UW_CHUNKS; ++m) {
          uint32_t oa[8];
#pragma unroll
          for (int i = 0; i < 8; ++i) {
            const __half2 a = gelu_fast2(u2h(h2[m * 8 + i]));
            oa[i] = h2u(a);
            h1[m * 8 + i] = h2u(__hfma2(g1, a, u2h(h1[m * 8 + i])));
          }
          if (!hand_over(1, m, oa)) { failed = true; break; }
        }
        if (failed) break;
      }
      {
        __half* dst = p.abar + (size_t)row * p.N + nt * BN_WIDE + cq * 16;     // 32-byte pieces: whole sectors
#pragma unroll
        for (int m = 0; m < UW_CHUNKS; ++m) st_global_v8(dst + m * BK, h1 + m * 8);
      }
      if (HAS_R && (w + 1) % unit == 0) {
        const int j = cq >> 1;
        if (j < KSEL) {
          // S_j is complete for this unit.  The warp walks over the expert blocks of the expanded
          // index (this warp: every other block); lanes whose row uses the block add it to s.
          const bool ok = mbar_wait_cluster(local(W_SFULL), flushes & 1u, abort_flag);
          if (!__all_sync(0xffffffffu, ok)) { failed = true; break; }
          tc_fence_after();
          const int g = p.tile_cluster[pt];
          const int e = p.row_slot[(size_t)row * KSEL + j] - g * p.K;
          const bool real = p.row_token[row] >= 0;
          float* srow = p.s_out + ((size_t)row * KSEL + j) * p.r;
          const int r = p.r;
          const float gate = j == 0 ? g0f : g1f;
          for (int i = cq & 1; i < p.K; i += 2) {
            const uint32_t ta = taddr + UW_TMEM_S + j * KE + i * r;
            const bool mine = real && e == i;
            __half* arow = p.As_direct ? p.As_direct + (size_t)row * KE + i * r : nullptr;   // the row's block of the expanded index
            if (r == 16) {
              uint32_t v[16];
              tmem_ld16_nowait(ta, v);
              tmem_ld_wait();
              if (mine && arow) {
                uint32_t o[8];
#pragma unroll
                for (int c = 0; c < 8; ++c) o[c] = pack_half2(gate * __uint_as_float(v[2 * c]), gate * __uint_as_float(v[2 * c + 1]));
                st_global_v8(arow, o);
              } else if (mine) {
#pragma unroll
                for (int c = 0; c < 16; c += 4)
                  red_add_v4(srow + c, __uint_as_float(v[c]), __uint_as_float(v[c + 1]), __uint_as_float(v[c + 2]), __uint_as_float(v[c + 3]));
              }
            } else if (r == 32) {
              uint32_t v[32];
              tmem_ld32_nowait(ta, v);
              tmem_ld_wait();
              if (mine && arow) {
                uint32_t o[16];
#pragma unroll
                for (int c = 0; c < 16; ++c) o[c] = pack_half2(gate * __uint_as_float(v[2 * c]), gate * __uint_as_float(v[2 * c + 1]));
                st_global_v8(arow, o);
                st_global_v8(arow + 16, o + 8);
              } else if (mine) {
#pragma unroll
                for (int c = 0; c < 32; c += 4)
                  red_add_v4(srow + c, __uint_as_float(v[c]), __uint_as_float(v[c + 1]), __uint_as_float(v[c + 2]), __uint_as_float(v[c + 3]));
              }
            } else if (r == 8) {
              uint32_t v[8];
              tmem_ld8_nowait(ta, v);
              tmem_ld_wait();
              if (mine && arow) {
                *reinterpret_cast<uint4*>(arow) =
                    make_uint4(pack_half2(gate * __uint_as_float(v[0]), gate * __uint_as_float(v[1])),
                               pack_half2(gate * __uint_as_float(v[2]), gate * __uint_as_float(v[3])),
                               pack_half2(gate * __uint_as_float(v[4]), gate * __uint_as_float(v[5])),
                               pack_half2(gate * __uint_as_float(v[6]), gate * __uint_as_float(v[7])));
              } else if (mine) {
                red_add_v4(srow, __uint_as_float(v[0]), __uint_as_float(v[1]), __uint_as_float(v[2]), __uint_as_float(v[3]));
                red_add_v4(srow + 4, __uint_as_float(v[4]), __uint_as_float(v[5]), __uint_as_float(v[6]), __uint_as_float(v[7]));
              }
            } else {
              uint32_t v[4];
              tmem_ld4_nowait(ta, v);
              tmem_ld_wait();
              if (mine && arow) {
                *reinterpret_cast<uint2*>(arow) = make_uint2(pack_half2(gate * __uint_as_float(v[0]), gate * __uint_as_float(v[1])),
                                                             pack_half2(gate * __uint_as_float(v[2]), gate * __uint_as_float(v[3])));
              } else if (mine) {
                red_add_v4(srow, __uint_as_float(v[0]), __uint_as_float(v[1]), __uint_as_float(v[2]), __uint_as_float(v[3]));
              }
            }
          }
          tc_fence_before();
          __syncwarp();
          if (lane == 0) mbar_arrive_cluster_relaxed(lead(W_SEMPTY));
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

template <bool HAS_R, int KSEL>
cudaError_t launch_w(const UpWideMaps& m, const Up2Params& p, int grid, cudaStream_t st) {
  auto kern = tc2_up_wide_kernel<HAS_R, KSEL>;
  constexpr size_t sm = WideCfg<HAS_R, KSEL>::SMEM;
  static_assert(sm <= kSmemLimit, "wide up kernel shared memory");
  static std::atomic<unsigned long long> smem_set{0};      // devices the kernel's shared-memory limit has been raised on
  if (cudaError_t e = ensure_dynamic_smem(kern, sm, smem_set)) return e;
  return launch_pairs(kern, grid, UW_THREADS, sm, st, *m.x3, *m.b13, *m.a0, *m.ad, *m.v1, *m.u2, p);
}

}  // namespace

cudaError_t launch_up_wide(bool has_r, int ksel, const UpWideMaps& maps, const Up2Params& p, int grid, cudaStream_t st) {
  if (!has_r) return launch_w<false, 1>(maps, p, grid, st);     // without residuals k only enters through the gates
  return ksel == 2 ? launch_w<true, 2>(maps, p, grid, st) : launch_w<true, 1>(maps, p, grid, st);
}

}  // namespace tc2c
}  // namespace cmoe
