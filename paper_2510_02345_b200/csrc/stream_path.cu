// Weight-streaming path of the expert FFNs for small batches (decode): with a handful of tokens per
// cluster the layer is bound by reading the FP16 bases once from HBM, so the kernels are laid out
// around the weight stream (sm_100a: TMA into shared memory, tcgen05 MMAs with TMEM accumulators).
//
// The roles of the two GEMM operands are swapped with respect to the large-batch path: the WEIGHTS
// are the 128-row A operand (a tile of output features, streamed once), the cluster's few tokens
// are the narrow B operand (N = 16..64, re-read from L2), and the accumulator holds
// D[feature][token].  Tensor-core rows cost nothing here; bytes do.  The bases are stored for this
// path stage by stage, [reduction index / 128][feature][128], so that what a CTA loads per pipeline
// stage is one contiguous piece of memory.
//
//   t      t_j = x U1_e for every (row, kept expert)                 (CUDA cores, tiny)
//   up     D = B1t_g[f-tile] x_g^T; epilogue per feature f (one thread each): h_j = D + t_j V1_e[f],
//          a_j = GELU(h_j) (erf form) -> fp16, abar = sum_j p_j a_j -> fp16; the INT4 codes of
//          V1_e[f, :] are read and decoded in registers right here
//   s      s_j = a_j U2_e                                            (CUDA cores, tiny)
//   down   D = B2t_g[c-tile, K range] abar_g^T, split along K over several CTAs, added to a fp32
//          copy of y with atomics
//   final  y = fp16(y32 + sum_j p_j s_j V2_e), stored un-permuted
//
// A cluster's rows are aligned to 16 (the MMA's N granularity) and cut into segments of at most 64
// rows; a work unit is (segment, tile of features[, K range]), dealt round-robin to the CTAs.
// Every device wait is bounded (status word CMOE_ERR_TIMEOUT on expiry).
#include "cmoe_internal.h"
#include "launch.cuh"
#include "device_utils.cuh"
#include "tc_ptx.cuh"
#include "lowrank.cuh"

namespace cmoe {

namespace {

using namespace ptx;

constexpr int SBK = 64;            // halves per K atom: one 128-byte swizzle row
constexpr int SKA = 2;             // K atoms per stage
constexpr int SNB = 64;            // most token rows per segment (MMA N)
constexpr int SMAXSEG = 160;       // segments: at most G + T_pad / 64
constexpr int S_THREADS = 640;     // warps 0, 3 TMA (alternating stages), 1 MMA, 2 TMEM allocation, 4..19 epilogue
constexpr uint32_t S_B_ATOM = SNB * SBK * 2;             // 8 KB
constexpr uint32_t S_TMEM_COLS = 128;                    // two accumulators of up to 64 columns
constexpr int S_EPI_WARPS = 16;
constexpr int S_PJ = 2;            // kept experts per token the up epilogue stages operands for (more: read in place)

// What an epilogue warp needs of its four token columns of one block of 16, staged in shared memory by the
// warp itself before the accumulator is complete: token, expert slots, gates and (up) the rows of t.
struct __align__(16) WarpStage {
  float t[4][S_PJ][32];
  int tok[4];
  int slot[4][S_PJ];
  float gate[4][S_PJ];
};

struct StreamParams {
  const int* seg_off;        // [G+1] first permuted row of each cluster (multiples of 16)
  const int* row_slot;       // [rows][k]
  const float* row_gate;     // [rows][k]
  const int* row_token;      // [rows]
  // up
  const float* t;            // [rows][k][r]
  const uint8_t* V1q;        // packed INT4 in the boundary layout
  const int* live;           // [E] bit 0 / 1: the expert's up / down residual block is not zero
  const __half* V1s;
  __half* a_slot;            // [rows][k][d_ff]  GELU(h_j) of every kept expert
  __half* abar;              // [rows][d_ff]
  // down
  float* y32;                // [rows][d], zeroed by the caller
  int* status;
  int G, K, k, r;
  int Kd;                    // reduction length (d for up, d_ff for down)
  int M;                     // output features (d_ff for up, d for down)
  int ksplit;                // down: K ranges per tile
};

template <int MROWS>
struct SCfg {
  static constexpr uint32_t A_ATOM = MROWS * SBK * 2;
  static constexpr uint32_t A_BYTES = SKA * A_ATOM;
  static constexpr uint32_t B_BYTES = SKA * S_B_ATOM;
  static constexpr uint32_t STAGE_BYTES = A_BYTES + B_BYTES;
  static constexpr int STAGES = 4;                                   // 48 KB each
  static constexpr size_t TABLES = 64 * 8 + SMAXSEG * 12 + 64;         // barriers, segment table
  static constexpr size_t SMEM = 1024 + (size_t)STAGES * STAGE_BYTES + TABLES + S_EPI_WARPS * sizeof(WarpStage);
};

// The down kernel's tiles have 128 feature rows and its granularity comes from the K ranges.  The up kernel
// cannot split K (GELU needs the complete h), so it picks the tile height R, a multiple of 8 up to 128, for
// which the round-robin over the CTAs ends soonest: with 896 tiles of 128 rows on 148 CTAs the last of seven
// rounds would hold 8 tiles, with 1024 tiles of 112 rows all seven rounds are nearly full and an eighth
// shorter.  Tiles of R rows are loaded with the box of tmRows.m[R / 8 - 1]; the MMA still spans 128 rows and
// the rest of the accumulator is not read.  A tile that reaches past the cluster's last feature loads rows
// of the next cluster (or the fill value past the matrix) into accumulator lanes that are not read either.
struct RowMaps { CUtensorMap m[16]; };       // boxes of 8, 16, ..., 128 weight rows
template <bool UP>
__global__ void __launch_bounds__(S_THREADS, 1)
stream_kernel(const __grid_constant__ CUtensorMap tmW, const __grid_constant__ RowMaps tmRows,
              const __grid_constant__ CUtensorMap tmTok, const StreamParams p) {
  constexpr int MROWS = 128;
  using Cfg = SCfg<MROWS>;
  constexpr int STAGES = Cfg::STAGES;
  extern __shared__ uint8_t smem_raw[];
  const uint32_t raw = smem_u32(smem_raw);
  const uint32_t base = (raw + 1023u) & ~1023u;
  uint8_t* sm = smem_raw + (base - raw);
  uint64_t* bars = reinterpret_cast<uint64_t*>(sm + (size_t)STAGES * Cfg::STAGE_BYTES);
  const uint32_t full0 = smem_u32(bars), empty0 = smem_u32(bars + 8);
  const uint32_t tfull0 = smem_u32(bars + 16), tempty0 = smem_u32(bars + 18);
  uint32_t* tmem_holder = reinterpret_cast<uint32_t*>(bars + 20);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_holder + 1);
  int* n_seg_p = reinterpret_cast<int*>(tmem_holder + 2);
  int* seg_row0 = reinterpret_cast<int*>(bars + 64);       // [SMAXSEG]
  int* seg_rows = seg_row0 + SMAXSEG;
  int* seg_g = seg_rows + SMAXSEG;
  WarpStage* stage_area = reinterpret_cast<WarpStage*>(sm + (size_t)STAGES * Cfg::STAGE_BYTES + Cfg::TABLES);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  constexpr int kEpiWarps = S_EPI_WARPS;      // four warps per TMEM lane quadrant: token columns c with c mod 4 = 0, 1, 2, 3

  if (threadIdx.x == 0) {
    for (int s = 0; s < STAGES; ++s) { mbar_init(full0 + 8 * s, 1); mbar_init(empty0 + 8 * s, 1); }
    for (int a = 0; a < 2; ++a) { mbar_init(tfull0 + 8 * a, 1); mbar_init(tempty0 + 8 * a, kEpiWarps); }
    *abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 2) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;"
                 ::"r"(smem_u32(tmem_holder)), "r"(S_TMEM_COLS) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  pdl_wait();                  // nothing above reads what an earlier kernel wrote
  pdl_release_dependents();
  if (warp == 0) {
    // segments of at most SNB rows, in cluster order: a lane per cluster (32 at a time), so that the reads of
    // the offsets table are one round trip instead of G dependent ones
    __syncwarp();
    int n = 0;
    for (int g0 = 0; g0 < p.G; g0 += 32) {
      const int g = g0 + lane;
      int r0 = 0, r1 = 0;
      if (g < p.G) { r0 = p.seg_off[g]; r1 = p.seg_off[g + 1]; }
      const int cnt = (r1 - r0 + SNB - 1) / SNB;
      int incl = cnt;
#pragma unroll
      for (int o = 1; o < 32; o <<= 1) {
        const int up = __shfl_up_sync(0xffffffffu, incl, o);
        if (lane >= o) incl += up;
      }
      int at = n + incl - cnt;
      for (int r = r0; r < r1 && at < SMAXSEG; r += SNB, ++at) { seg_row0[at] = r; seg_rows[at] = min(SNB, r1 - r); seg_g[at] = g; }
      n += __shfl_sync(0xffffffffu, incl, 31);
    }
    if (lane == 0) *n_seg_p = min(n, SMAXSEG);
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_holder;

  // work units: u = (seg * n_mt + mt) * ksplit + ks
  const int ksplit = UP ? 1 : p.ksplit;
  const int KCH = p.Kd / (SBK * SKA);                    // stages in the whole reduction
  int R = MROWS;                                         // feature rows per tile
  if (UP) {
    // time ~ rounds x rows per tile; below about 64 rows a stage is too small to keep the memory pipe full
    // and a round costs as much as one of 64 rows.  Ties go to the taller tile.
    long long best = 0;
    for (int cand = MROWS; cand >= 8; cand -= 8) {
      const long long tiles = (long long)*n_seg_p * ((p.M + cand - 1) / cand);
      const long long cost = ((tiles + gridDim.x - 1) / gridDim.x) * (cand > 64 ? cand : 64);
      if (cand == MROWS || cost < best) { best = cost; R = cand; }
    }
  }
  const int n_mt = (p.M + R - 1) / R;
  const int n_units = *n_seg_p * n_mt * ksplit;
  const int my_units = (int)blockIdx.x < n_units ? (n_units - 1 - (int)blockIdx.x) / (int)gridDim.x + 1 : 0;
  auto unit_of = [&](int i, int& seg, int& mt, int& c_begin, int& c_end) {
    const int u = blockIdx.x + i * gridDim.x;
    const int ks = u % ksplit, sm_ = u / ksplit;
    mt = sm_ % n_mt;
    seg = sm_ / n_mt;
    c_begin = (int)((long long)KCH * ks / ksplit);
    c_end = (int)((long long)KCH * (ks + 1) / ksplit);
  };
  bool failed = false;

  if (warp == 0 || warp == 3) {
    // ---------------- TMA producers: two threads take alternate stages of the flattened stage sequence
    if (lane == 0) {
      uint32_t it = 0;                                     // stage counter over all units
      const uint32_t mine = warp == 0 ? 0u : 1u;
      for (int i = 0; i < my_units && !failed; ++i) {
        int seg, mt, c0, c1;
        unit_of(i, seg, mt, c0, c1);
        const int g = seg_g[seg], row0 = seg_row0[seg], nb = seg_rows[seg] / 16;
        const int wrow = g * p.M + mt * R;
        const uint32_t a_bytes = (uint32_t)R * SBK * 2 * SKA;
        const CUtensorMap* wmap = UP ? &tmRows.m[R / 8 - 1] : &tmW;
        for (int c = c0; c < c1; ++c, ++it) {
          if ((it & 1u) != mine) continue;
          const uint32_t s = it % STAGES, ph = (it / STAGES) & 1u;
          if (!mbar_wait(empty0 + 8 * s, ph ^ 1u, abort_flag)) { failed = true; break; }
          const uint32_t a_dst = base + s * Cfg::STAGE_BYTES, b_dst = a_dst + Cfg::A_BYTES;
          mbar_expect_tx(full0 + 8 * s, a_bytes + (uint32_t)nb * SKA * 16 * SBK * 2);
          tma_load_4d(a_dst, wmap, full0 + 8 * s, 0, wrow, 0, c);     // stage c of the weights: rows wrow .., both K atoms
          // the tokens: 16 rows per box; atom a of block b lands at atom a, rows 16 b .. of the B tile
          for (int b = 0; b < nb; ++b)
            for (int a = 0; a < SKA; ++a)
              tma_load_2d(b_dst + a * S_B_ATOM + b * (16 * SBK * 2), &tmTok, full0 + 8 * s, (c * SKA + a) * SBK, row0 + 16 * b);
        }
      }
    }
  } else if (warp == 1) {
    // ---------------- MMA issuer
    if (lane == 0) {
      uint32_t s = 0, ph = 0;
      for (int i = 0; i < my_units && !failed; ++i) {
        int seg, mt, c0, c1;
        unit_of(i, seg, mt, c0, c1);
        const uint32_t idesc = idesc_f16(128, seg_rows[seg]);
        const uint32_t a_atom16 = (uint32_t)(R * SBK * 2) >> 4;        // second K atom of the R-row box, in 16-byte units
        const uint32_t acc = (uint32_t)i & 1u, aph = ((uint32_t)i >> 1) & 1u;
        if (!mbar_wait(tempty0 + 8 * acc, aph ^ 1u, abort_flag)) { failed = true; break; }
        tc_fence_after();
        const uint32_t d_tmem = tmem_base + acc * SNB;
        for (int c = c0; c < c1; ++c) {
          if (!mbar_wait(full0 + 8 * s, ph, abort_flag)) { failed = true; break; }
          tc_fence_after();
          const uint32_t a_src = base + s * Cfg::STAGE_BYTES, b_src = a_src + Cfg::A_BYTES;
          const uint64_t adesc = umma_desc(a_src), bdesc = umma_desc(b_src);
          umma_f16(d_tmem, adesc, bdesc, idesc, c != c0 ? 1u : 0u);
#pragma unroll
          for (int ks = 1; ks < SBK / 16; ++ks) umma_f16(d_tmem, adesc + 2 * ks, bdesc + 2 * ks, idesc, 1u);
#pragma unroll
          for (int ks = 0; ks < SBK / 16; ++ks)
            umma_f16(d_tmem, adesc + a_atom16 + 2 * ks, bdesc + (S_B_ATOM >> 4) + 2 * ks, idesc, 1u);
          umma_commit(empty0 + 8 * s);
          if (++s == STAGES) { s = 0; ph ^= 1u; }
        }
        if (failed) break;
        umma_commit(tfull0 + 8 * acc);
      }
    }
  } else if (warp >= 4) {
    // ---------------- epilogue warps: one thread per output feature of the tile
    const int q = warp & 3;
    const int part = (warp - 4) >> 2;                    // which token columns of the accumulator this warp takes
    const uint32_t taddr = tmem_base + ((uint32_t)(q * 32) << 16);
    const int r = p.r, k = p.k, M = p.M;
    WarpStage* ws = stage_area + (warp - 4);
    for (int i = 0; i < my_units; ++i) {
      int seg, mt, c0, c1;
      unit_of(i, seg, mt, c0, c1);
      const int f = mt * R + q * 32 + lane;                // output feature (up) / output column (down)
      const bool mine = q * 32 + lane < R && f < M;        // only the tile's own accumulator lanes are real
      const int row0 = seg_row0[seg], nrows = q * 32 < R ? seg_rows[seg] : 0;
      const uint32_t acc = (uint32_t)i & 1u, aph = ((uint32_t)i >> 1) & 1u;
      // Everything the warp needs of one block of 16 token columns besides the accumulator is fetched before
      // the accumulator is complete, so that the latency of these reads (dependent table lookups, then scattered
      // reads of V1 from HBM) hides behind the tile's weight stream instead of adding up, column after column,
      // between two tiles and at the kernel's end: tokens, slots, gates and the rows of t go into the warp's
      // staging area (lanes in parallel), the r INT4 codes and the scale of this thread's feature row of V1, for
      // each of the four columns and up to two kept experts, into registers.
      constexpr int PJ = S_PJ;
      const bool pre = UP && r > 0 && k <= PJ;
      uint32_t wq[4][PJ][4];
      float wsc[4][PJ];
      auto load_codes = [&](int e, uint32_t (&w)[4], float& sc) {
        const long long flat = ((long long)e * M + f) * r;           // the r codes of (e, f) are one scale group
        const uint8_t* src = p.V1q + (flat >> 1);
        sc = __half2float(p.V1s[flat >> 5]);
        w[1] = w[2] = w[3] = 0u;
        if (r == 32) {
          const uint4 v4 = *reinterpret_cast<const uint4*>(src);
          w[0] = v4.x; w[1] = v4.y; w[2] = v4.z; w[3] = v4.w;
        } else if (r == 16) {
          const uint2 v2 = *reinterpret_cast<const uint2*>(src);
          w[0] = v2.x; w[1] = v2.y;
        } else if (r == 8) {
          w[0] = *reinterpret_cast<const uint32_t*>(src);
        } else {
          w[0] = *reinterpret_cast<const uint16_t*>(src);
        }
      };
      auto preload = [&](int tb) {
        __syncwarp();                                      // the warp has finished with the previous block's stage
        const int rowb = row0 + tb + part;                 // column c2 of this warp is row rowb + 4 c2
        if (lane < 4) ws->tok[lane] = p.row_token[rowb + 4 * lane];
        if (pre && lane < 4 * PJ) {
          const int c2 = lane / PJ, j = lane % PJ;
          if (j < k) {
            ws->slot[c2][j] = p.row_slot[(size_t)(rowb + 4 * c2) * k + j];       // (padding rows hold valid slots and gate 0)
            ws->gate[c2][j] = p.row_gate[(size_t)(rowb + 4 * c2) * k + j];
          }
        }
        __syncwarp();
        if (pre) {
          // the rows of t (indexed by token): k r floats per column, four floats per lane and step
          const int per_col = k * r / 4;
          for (int idx = lane; idx < 4 * per_col; idx += 32) {
            const int c2 = idx / per_col, rem = idx - c2 * per_col;
            const int j = rem / (r / 4), q4 = rem - j * (r / 4);
            const int tok = ws->tok[c2];
            if (tok >= 0)
              *reinterpret_cast<float4*>(&ws->t[c2][j][4 * q4]) = *reinterpret_cast<const float4*>(p.t + (size_t)tok * k * r + 4 * rem);
          }
#pragma unroll
          for (int c2 = 0; c2 < 4; ++c2) {
            const bool real = mine && ws->tok[c2] >= 0;
#pragma unroll
            for (int j = 0; j < PJ; ++j) {
              wsc[c2][j] = 0.f;
              wq[c2][j][0] = wq[c2][j][1] = wq[c2][j][2] = wq[c2][j][3] = 0u;
              if (real && j < k) {
                const int e = ws->slot[c2][j];
                if (p.live[e] & 1) load_codes(e, wq[c2][j], wsc[c2][j]);      // (a zero residual block is skipped: Sec. 3.4)
              }
            }
          }
        }
        __syncwarp();
      };
      // h = dv + sc (t_j . codes): the r codes decoded in registers
      auto residual = [&](float dv, const float4* tp, const uint32_t (&w)[4], float sc) -> float {
        float dot0 = 0.f, dot1 = 0.f;
        if (r >= 8) {
#pragma unroll
          for (int w8 = 0; w8 < 4; ++w8) {
            if (w8 < r / 8) {
              float cf[8];
              int4x8_to_float(w[w8], cf);
              const float4 ta = tp[2 * w8], tb4 = tp[2 * w8 + 1];
              dot0 = fmaf(ta.x, cf[0], dot0);
              dot1 = fmaf(ta.y, cf[1], dot1);
              dot0 = fmaf(ta.z, cf[2], dot0);
              dot1 = fmaf(ta.w, cf[3], dot1);
              dot0 = fmaf(tb4.x, cf[4], dot0);
              dot1 = fmaf(tb4.y, cf[5], dot1);
              dot0 = fmaf(tb4.z, cf[6], dot0);
              dot1 = fmaf(tb4.w, cf[7], dot1);
            }
          }
        } else {
          float cf[8];
          int4x8_to_float(w[0], cf);
          const float4 ta = tp[0];
          dot0 = fmaf(ta.x, cf[0], dot0);
          dot1 = fmaf(ta.y, cf[1], dot1);
          dot0 = fmaf(ta.z, cf[2], dot0);
          dot1 = fmaf(ta.w, cf[3], dot1);
        }
        return fmaf(sc, dot0 + dot1, dv);
      };
      if (nrows > 0) preload(0);
      {
        const bool ok = mbar_wait(tfull0 + 8 * acc, aph, abort_flag);
        if (!__all_sync(0xffffffffu, ok)) { failed = true; break; }
      }
      tc_fence_after();
      for (int tb = 0; tb < nrows; tb += 16) {
        if (tb > 0) preload(tb);
        uint32_t v[16];
        tmem_ld16_nowait(taddr + acc * SNB + tb, v);
        tmem_ld_wait();
#pragma unroll
        for (int c2 = 0; c2 < 4; ++c2) {
          const int c = 4 * c2 + part;
          const int row = row0 + tb + c;
          const int tok = ws->tok[c2];
          const bool real = mine && tok >= 0;
          const float dv = __uint_as_float(part == 0 ? v[4 * c2] : part == 1 ? v[4 * c2 + 1] : part == 2 ? v[4 * c2 + 2] : v[4 * c2 + 3]);
          if (UP) {
            float ab = 0.f;
            if (real && pre) {
#pragma unroll
              for (int j = 0; j < PJ; ++j) {
                if (j < k) {
                  // a zero residual block has scale and codes 0 here: h = dv
                  const float h = residual(dv, reinterpret_cast<const float4*>(ws->t[c2][j]), wq[c2][j], wsc[c2][j]);
                  const float a = gelu_erf(h);
                  ab = fmaf(ws->gate[c2][j], a, ab);
                  p.a_slot[((size_t)row * k + j) * M + f] = __float2half_rn(a);
                }
              }
            } else if (real) {
              for (int j = 0; j < k; ++j) {
                const int e = p.row_slot[(size_t)row * k + j];
                float h = dv;
                if (r > 0 && (p.live[e] & 1)) {
                  uint32_t w[4];
                  float sc;
                  load_codes(e, w, sc);
                  h = residual(dv, reinterpret_cast<const float4*>(p.t + ((size_t)tok * k + j) * r), w, sc);      // t is indexed by token
                }
                const float a = gelu_erf(h);
                ab = fmaf(p.row_gate[(size_t)row * k + j], a, ab);
                if (r > 0) p.a_slot[((size_t)row * k + j) * M + f] = __float2half_rn(a);
              }
            }
            if (mine) p.abar[(size_t)row * M + f] = __float2half_rn(ab);
          } else {
            if (real) atomicAdd(p.y32 + (size_t)row * M + f, dv);
          }
        }
      }
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(tempty0 + 8 * acc);
    }
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
  if (warp == 2)
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(S_TMEM_COLS) : "memory");
}

// ------------------------------------------------------------------------------------------------
// rank-r projections of one vector per (row, kept expert):  out[item][p] = sum_c in[item][c] U_e[p][c]
// with U packed INT4 [E][r][len].  t = x U1 (in = the row's activations) and s = a_j U2 (in = the
// activation of that row and slot).  A block per (item, eight rank indices), a warp per rank index,
// lanes over the 32-element scale groups.
// ------------------------------------------------------------------------------------------------
__device__ __forceinline__ void
lowrank_body(const int* __restrict__ seg_off, int G, int k, int r, int len, int in_per_slot,
             const __half* __restrict__ in, const int* __restrict__ row_slot, const int* __restrict__ row_token,
             const uint8_t* __restrict__ Uq, const __half* __restrict__ Us, float* __restrict__ out,
             const int* __restrict__ live, int live_bit) {
  const int item = blockIdx.x;
  const int row = item / k;
  // padding rows and rows whose expert's residual block is zero: the projection is zero
  if (row >= seg_off[G] || row_token[row] < 0 || !(live[row_slot[item]] & live_bit)) {
    if (row < seg_off[G] && blockIdx.y == 0) for (int pr = threadIdx.x; pr < r; pr += blockDim.x) out[(size_t)item * r + pr] = 0.f;
    return;
  }
  const int e = row_slot[item];
  const __half* xin = in + (size_t)(in_per_slot ? item : row) * len;
  const int nwarp = blockDim.x >> 5;
  lowrank_rows(xin, e, r, len, blockIdx.y * nwarp, gridDim.y * nwarp, Uq, Us, out + (size_t)item * r);
}

// On the second stream: s = a_j U2 is not needed before the last kernel of the forward, so it
// runs beside the down kernel.  That kernel holds 640 threads x 96 registers of every SM; four warps of
// 32 registers are what fits next to it.
constexpr int kSideThreads = 128;
__global__ void __launch_bounds__(kSideThreads, 16)
lowrank_side_kernel(const int* __restrict__ seg_off, int G, int k, int r, int len, int in_per_slot,
                    const __half* __restrict__ in, const int* __restrict__ row_slot, const int* __restrict__ row_token,
                    const uint8_t* __restrict__ Uq, const __half* __restrict__ Us, float* __restrict__ out,
                    const int* __restrict__ live, int live_bit) {
  lowrank_body(seg_off, G, k, r, len, in_per_slot, in, row_slot, row_token, Uq, Us, out, live, live_bit);
}

// Second stream, after s: the rank-r part of the down-projection, y32[row][c] += sum_j p_j s_j . V2_e[c, :],
// one thread per (row, output column), added with the same fp32 atomics as the K ranges of the down kernel
// running beside it.
__global__ void __launch_bounds__(kSideThreads, 16)
resid_side_kernel(const int* __restrict__ seg_off, int G, int d, int k, int r, float* __restrict__ y32,
                  const float* __restrict__ s, const int* __restrict__ row_slot, const float* __restrict__ row_gate,
                  const int* __restrict__ row_token, const uint8_t* __restrict__ V2q, const __half* __restrict__ V2s,
                  const int* __restrict__ live) {
  const int row = blockIdx.y;
  const int c = blockIdx.x * blockDim.x + threadIdx.x;
  if (row >= seg_off[G] || c >= d || row_token[row] < 0) return;
  float v = 0.f;
  for (int j = 0; j < k; ++j) {
    const int e = row_slot[(size_t)row * k + j];
    if (!(live[e] & 2)) continue;                            // zero residual block
    const float* sj = s + ((size_t)row * k + j) * r;
    const long long flat = ((long long)e * d + c) * r;      // the r codes of (e, c) share one scale group
    float u = 0.f;
    if (r >= 8) {
      const uint32_t* wq = reinterpret_cast<const uint32_t*>(V2q + (flat >> 1));
      for (int w8 = 0; w8 < r / 8; ++w8) {
        float cf[8];
        int4x8_to_float(wq[w8], cf);
#pragma unroll
        for (int n = 0; n < 8; ++n) u = fmaf(sj[w8 * 8 + n], cf[n], u);
      }
    } else {
      float cf[8];
      int4x8_to_float(*reinterpret_cast<const uint16_t*>(V2q + (flat >> 1)), cf);
#pragma unroll
      for (int n = 0; n < 4; ++n) u = fmaf(sj[n], cf[n], u);
    }
    v = fmaf(row_gate[(size_t)row * k + j] * __half2float(V2s[flat >> 5]), u, v);
  }
  atomicAdd(y32 + (size_t)row * d + c, v);
}

// y[tok] = fp16(y32[row] + sum_j p_j s_j V2_e), one thread per (row, output column)
__global__ void __launch_bounds__(256)
stream_final_kernel(const int* __restrict__ seg_off, int G, int d, int k, int r,
                    const float* __restrict__ y32, const float* __restrict__ s, const int* __restrict__ row_slot,
                    const float* __restrict__ row_gate, const int* __restrict__ row_token,
                    const uint8_t* __restrict__ V2q, const __half* __restrict__ V2s, __half* __restrict__ y) {
  pdl_wait();
  const int row = blockIdx.y;
  const int c = blockIdx.x * blockDim.x + threadIdx.x;
  if (row >= seg_off[G] || c >= d) return;
  const int tok = row_token[row];
  if (tok < 0) return;
  float v = y32[(size_t)row * d + c];
  for (int j = 0; j < k && r > 0; ++j) {
    const int e = row_slot[(size_t)row * k + j];
    const float* sj = s + ((size_t)row * k + j) * r;
    const long long flat = ((long long)e * d + c) * r;      // the r codes of (e, c) share one scale group
    float u = 0.f;
    if (r >= 8) {
      const uint32_t* wq = reinterpret_cast<const uint32_t*>(V2q + (flat >> 1));
      for (int w8 = 0; w8 < r / 8; ++w8) {
        float cf[8];
        int4x8_to_float(wq[w8], cf);
#pragma unroll
        for (int n = 0; n < 8; ++n) u = fmaf(sj[w8 * 8 + n], cf[n], u);
      }
    } else {
      const uint32_t word = *reinterpret_cast<const uint16_t*>(V2q + (flat >> 1));
#pragma unroll
      for (int n = 0; n < 4; ++n) u = fmaf(sj[n], (float)sext4((int)(word >> (4 * n))), u);
    }
    v = fmaf(row_gate[(size_t)row * k + j] * __half2float(V2s[flat >> 5]), u, v);
  }
  y[(size_t)tok * d + c] = __float2half_rn(v);
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

// the token operand: fp16 matrix [rows][cols], boxes of 16 rows x 64 halves (one K atom of one block of 16 tokens)
bool make_token_map(CUtensorMap* map, const void* ptr, uint64_t rows, uint64_t cols) {
  EncodeTiledFn enc = get_encode();
  if (!enc) return false;
  cuuint64_t gdim[2] = {cols, rows};
  cuuint64_t gstride[1] = {cols * 2};
  cuuint32_t box[2] = {(cuuint32_t)SBK, 16};
  cuuint32_t estr[2] = {1, 1};
  return enc(map, CU_TENSOR_MAP_DATA_TYPE_FLOAT16, 2, const_cast<void*>(ptr), gdim, gstride, box, estr,
             CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
             CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// The bases as the streaming kernels read them, [Kd / 128][rows][128] fp16 (stage-major): a 4-D view
// {64 halves, rows, 2 K atoms, Kd / 128 stages} whose box (64, box_rows, 2, 1) lands in shared memory as two
// consecutive swizzled [box_rows][64] tiles, read from one contiguous piece of box_rows x 256 bytes.
bool make_weight_map(CUtensorMap* map, const void* ptr, uint64_t rows, uint64_t Kd, uint32_t box_rows) {
  EncodeTiledFn enc = get_encode();
  if (!enc) return false;
  cuuint64_t gdim[4] = {(cuuint64_t)SBK, rows, (cuuint64_t)SKA, Kd / (SBK * SKA)};
  cuuint64_t gstride[3] = {(cuuint64_t)SBK * SKA * 2, (cuuint64_t)SBK * 2, rows * SBK * SKA * 2};
  cuuint32_t box[4] = {(cuuint32_t)SBK, box_rows, (cuuint32_t)SKA, 1};
  cuuint32_t estr[4] = {1, 1, 1, 1};
  return enc(map, CU_TENSOR_MAP_DATA_TYPE_FLOAT16, 4, const_cast<void*>(ptr), gdim, gstride, box, estr,
             CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
             CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

struct StreamState {
  CUtensorMap mW1, mX, mW2, mAbar;
  RowMaps mW1r;
  int sm_count;
  int ksplit;
};
static_assert(sizeof(StreamState) <= sizeof(((cmoe_layer*)nullptr)->tc_state), "tc_state too small");

template <bool UP>
cudaError_t launch_stream(const CUtensorMap& mW, const RowMaps& mWs, const CUtensorMap& mTok, const StreamParams& p, int grid,
                          cudaStream_t st) {
  auto kern = stream_kernel<UP>;
  constexpr size_t sm = SCfg<128>::SMEM;
  static_assert(sm <= 232448, "stream kernel shared memory");
  static std::atomic<unsigned long long> smem_set{0};      // devices the kernel's shared-memory limit has been raised on
  if (cudaError_t e = ensure_dynamic_smem(kern, sm, smem_set)) return e;
  launch_chained(kern, dim3(grid), dim3(S_THREADS), sm, st, 1,
      mW, mWs, mTok, p);
  return cudaGetLastError();
}

}  // namespace

bool stream_supported(const Dims& D) {
  return D.d % 128 == 0 && D.d_ff % 128 == 0 && D.T_max <= 128;
}

cudaError_t stream_init(cmoe_layer* L) {
  const Dims& D = L->dims;
  const Scratch& S = L->sc;
  StreamState* ts = reinterpret_cast<StreamState*>(L->tc_state);
  int dev = 0;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return e;
  e = cudaDeviceGetAttribute(&ts->sm_count, cudaDevAttrMultiProcessorCount, dev);
  if (e != cudaSuccess) return e;
  const uint64_t P = (uint64_t)D.T_pad_max, G = (uint64_t)D.G;
  bool ok = make_weight_map(&ts->mW1, L->w.B1t, G * D.d_ff, D.d, 128);
  for (int i = 0; i < 16 && ok; ++i) ok = make_weight_map(&ts->mW1r.m[i], L->w.B1t, G * D.d_ff, D.d, 8 * (i + 1));
  ok = ok && make_token_map(&ts->mX, S.x_perm, P, D.d) &&
                  make_weight_map(&ts->mW2, L->w.B2t, G * D.d, D.d_ff, 128) && make_token_map(&ts->mAbar, S.abar, P, D.d_ff);
  // K ranges per down tile: fill the SMs evenly, keep at least four stages per range
  const int kch = D.d_ff / (SBK * SKA);
  const long long tiles = (long long)D.G * (D.d / 128);
  int best = 1;
  double best_eff = 0.0;
  for (int ks = 1; ks <= 16 && kch / ks >= 4; ++ks) {
    const long long units = tiles * ks, waves = (units + ts->sm_count - 1) / ts->sm_count;
    const double eff = (double)units / (double)(waves * ts->sm_count);
    if (eff > best_eff + 1e-9) { best_eff = eff; best = ks; }
  }
  ts->ksplit = best;
  return ok ? cudaSuccess : cudaErrorInvalidValue;
}

int stream_launch_count(const Dims& D) { return D.r > 0 ? 5 : 3; }

// t = x U1 for the blocks that ride in the permutation kernel
void stream_lowrank_rider(const cmoe_layer* L, const __half* x, int T, LowrankTok* lr) {
  const Dims& D = L->dims;
  *lr = LowrankTok{};
  if (D.r == 0) return;
  lr->x = x; lr->cluster_id = L->sc.cluster_id; lr->slot = L->sc.slot; lr->Uq = L->w.U1q; lr->Us = L->w.U1s;
  lr->out = L->sc.t; lr->live = L->w.live; lr->T = T; lr->K = D.K; lr->k = D.k; lr->r = D.r; lr->len = D.d;
}

cudaError_t launch_stream_ffn(const cmoe_layer* L, int T, __half* y, cudaStream_t st, cudaEvent_t* marks) {
  const Dims& D = L->dims;
  const Weights& W = L->w;
  const Scratch& S = L->sc;
  const StreamState& ts = *reinterpret_cast<const StreamState*>(L->tc_state);
  const int rows_bound = t_pad_bound(D, T);
  cudaError_t e;
  if (marks) cudaEventRecord(marks[0], st);
  // t = x U1 was computed beside the permutation (stream_lowrank_rider)
  if (marks) cudaEventRecord(marks[1], st);
  StreamParams p{};
  p.seg_off = S.seg_off; p.row_slot = S.row_slot; p.row_gate = S.row_gate; p.row_token = S.row_token;
  p.t = S.t; p.V1q = W.V1q; p.V1s = W.V1s; p.live = W.live; p.a_slot = S.a_slot; p.abar = S.abar; p.y32 = S.y32; p.status = S.status;
  p.G = D.G; p.K = D.K; p.k = D.k; p.r = D.r;
  const int seg_bound = D.G + rows_bound / SNB;
  {
    p.Kd = D.d; p.M = D.d_ff; p.ksplit = 1;
    const long long units = (long long)seg_bound * (D.d_ff / 8);       // the kernel may choose tiles as low as 8 rows
    const int grid = (int)(units < ts.sm_count ? units : ts.sm_count);
    if ((e = launch_stream<true>(ts.mW1, ts.mW1r, ts.mX, p, grid, st)) != cudaSuccess) return e;
  }
  if (marks) cudaEventRecord(marks[2], st);
  if (D.r > 0) {
    // fork: s = a_j U2, then the rank-r part of y, on the second stream beside the down kernel
    if ((e = cudaEventRecord(L->side_fork, st)) != cudaSuccess) return e;
    if ((e = cudaStreamWaitEvent(L->side_stream, L->side_fork, 0)) != cudaSuccess) return e;
    const int nwarp = kSideThreads / 32;
    lowrank_side_kernel<<<dim3(rows_bound * D.k, (D.r + nwarp - 1) / nwarp), kSideThreads, 0, L->side_stream>>>(
        S.seg_off, D.G, D.k, D.r, D.d_ff, 1, S.a_slot, S.row_slot, S.row_token, W.U2q, W.U2s, S.s, W.live, 2);
    if ((e = cudaGetLastError()) != cudaSuccess) return e;
    resid_side_kernel<<<dim3((D.d + kSideThreads - 1) / kSideThreads, rows_bound), kSideThreads, 0, L->side_stream>>>(
        S.seg_off, D.G, D.d, D.k, D.r, S.y32, S.s, S.row_slot, S.row_gate, S.row_token, W.V2q, W.V2s, W.live);
    if ((e = cudaGetLastError()) != cudaSuccess) return e;
    if ((e = cudaEventRecord(L->side_join, L->side_stream)) != cudaSuccess) return e;
  }
  {
    p.Kd = D.d_ff; p.M = D.d; p.ksplit = ts.ksplit;
    const long long units = (long long)seg_bound * (D.d / 128) * ts.ksplit;
    const int grid = (int)(units < ts.sm_count ? units : ts.sm_count);
    if ((e = launch_stream<false>(ts.mW2, ts.mW1r, ts.mAbar, p, grid, st)) != cudaSuccess) return e;
  }
  if (D.r > 0 && (e = cudaStreamWaitEvent(st, L->side_join, 0)) != cudaSuccess) return e;     // join
  dim3 fgrid((D.d + 255) / 256, rows_bound);
  launch_chained(stream_final_kernel, dim3(fgrid), dim3(256), 0, st, 1,
      S.seg_off, D.G, D.d, D.k, 0 /* the rank-r part is already in y32 */, S.y32, S.s, S.row_slot, S.row_gate,
                                             S.row_token, W.V2q, W.V2s, y);
  return cudaGetLastError();
}

}  // namespace cmoe
