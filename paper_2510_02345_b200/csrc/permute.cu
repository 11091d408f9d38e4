// Token permutation: a stable counting sort of the tokens by (cluster, expert combination), with
// every cluster's segment of permuted rows starting at a multiple of row_align so that GEMM tiles
// never straddle two clusters.  The paper only implies this step ("tokens are assigned to a
// cluster, then to experts inside it", Sec. 3.3); the mechanism is this library's.
//
//   hist     per-block histogram of the keys (block = 256 consecutive tokens); for batches of 1024 tokens and
//            more the router kernel has counted the keys of its token tiles itself and this kernel is not launched
//   scan     one block: per-key running sums over blocks, cluster segment offsets, tile table, and the
//            table entries of the padding rows of each segment (no token, zero gates); when the table of counts
//            is small every scatter block does these sums for itself and this kernel is not launched either
//   scatter  each token's row = key offset + earlier blocks' count + its rank inside the block;
//            writes the row tables
//   move     copies every token's activations to its row with 16-byte vectors (a block per row;
//            padding rows get zeros) and clears the buffer the later stages accumulate into; when the scatter blocks
//            do the sums themselves they also move the rows of their own token tile and this kernel is not launched
//
// The result is deterministic: rows of one key keep the token order.
#include "cmoe_internal.h"
#include "launch.cuh"
#include "device_utils.cuh"
#include "stage_factors.cuh"
#include "lowrank.cuh"
#include "perm_keys.cuh"

namespace cmoe {

namespace {

__global__ void __launch_bounds__(kPermBlock)
hist_kernel(int T, int k, int nsub, int nkey, int sub_is_combo,
            const int* __restrict__ cluster_id, const int* __restrict__ slot,
            const float* __restrict__ gates, int* __restrict__ keys, int* __restrict__ block_counts) {
  pdl_wait();
  extern __shared__ int sh_cnt[];
  for (int i = threadIdx.x; i < nkey; i += blockDim.x) sh_cnt[i] = 0;
  __syncthreads();
  int t = blockIdx.x * kPermBlock + threadIdx.x;
  if (t < T) {
    int cs[kMaxKsel];
    float cg[kMaxKsel];
    int sub = canonical_slots(slot + (size_t)t * k, gates + (size_t)t * k, k, sub_is_combo, cs, cg);
    const int g = cluster_id[t];
    const int key = g >= 0 ? g * nsub + sub : -1;       // (a virtual token without a cluster gets no row)
    keys[t] = key;
    if (key >= 0) atomicAdd(&sh_cnt[key], 1);
  }
  __syncthreads();
  for (int i = threadIdx.x; i < nkey; i += blockDim.x)
    block_counts[(size_t)blockIdx.x * nkey + i] = sh_cnt[i];
}

__global__ void __launch_bounds__(1024)
scan_kernel(int nblk, int G, int nsub, int nkey, int row_align, int max_tiles,
            const int* __restrict__ block_counts, int* __restrict__ block_base,
            int* __restrict__ key_cnt, int* __restrict__ key_off, int* __restrict__ seg_off,
            int* __restrict__ seg_cnt, int* __restrict__ n_rows, int* __restrict__ tile_cluster, int K, int k,
            int* __restrict__ row_token, int* __restrict__ row_slot, float* __restrict__ row_gate) {
  pdl_wait();
  __shared__ int sh_seg[kMaxG + 1];
  __shared__ int sh_segcnt[kMaxG];
  __shared__ int sh_cnt[kMaxKeys];
  // a warp per key, lanes over the blocks: exclusive prefix sums of the key's per-block counts
  const int lane = threadIdx.x & 31, nwarp = blockDim.x >> 5;
  for (int key = threadIdx.x >> 5; key < nkey; key += nwarp) {
    int run = 0;
    for (int b0 = 0; b0 < nblk; b0 += 256) {
      // eight loads per lane in flight (blocks b0 + 32 i + lane), then eight warp scans
      int c[8];
#pragma unroll
      for (int i = 0; i < 8; ++i) {
        const int b = b0 + 32 * i + lane;
        c[i] = b < nblk ? block_counts[(size_t)b * nkey + key] : 0;
      }
#pragma unroll
      for (int i = 0; i < 8; ++i) {
        const int b = b0 + 32 * i + lane;
        int incl = c[i];
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
          const int up = __shfl_up_sync(0xffffffffu, incl, o);
          if (lane >= o) incl += up;
        }
        if (b < nblk) block_base[(size_t)b * nkey + key] = run + incl - c[i];
        run += __shfl_sync(0xffffffffu, incl, 31);
      }
    }
    if (lane == 0) { key_cnt[key] = run; sh_cnt[key] = run; }
  }
  __syncthreads();
  if (threadIdx.x == 0) {
    int off = 0;
    for (int g = 0; g < G; ++g) {
      sh_seg[g] = off;
      seg_off[g] = off;
      int cnt = 0;
      for (int s = 0; s < nsub; ++s) {
        key_off[g * nsub + s] = off + cnt;
        cnt += sh_cnt[g * nsub + s];
      }
      seg_cnt[g] = cnt;
      sh_segcnt[g] = cnt;
      off += (cnt + row_align - 1) / row_align * row_align;
    }
    sh_seg[G] = off;
    seg_off[G] = off;
    *n_rows = off;
  }
  __syncthreads();
  // table entries of the padding rows of every cluster (the scatter kernel writes the token rows only)
  for (int g = 0; g < G; ++g) {
    const int first = sh_seg[g] + sh_segcnt[g], last = sh_seg[g + 1];
    for (int row = first + (int)threadIdx.x; row < last; row += blockDim.x) {
      row_token[row] = -1;
      for (int j = 0; j < k; ++j) {
        row_slot[(size_t)row * k + j] = g * K + j;       // any valid experts of the cluster
        row_gate[(size_t)row * k + j] = 0.f;
      }
    }
  }
  const int ntile = sh_seg[G] / row_align;
  for (int tile = threadIdx.x; tile < max_tiles; tile += blockDim.x) {
    int g = -1;
    if (tile < ntile) {
      int row = tile * row_align;
      g = 0;
      while (g + 1 < G && sh_seg[g + 1] <= row) ++g;
    }
    tile_cluster[tile] = g;
  }
}

// What the scan computes, for the scatter kernel to work out itself when the count table is small (ScanInline.counts
// not null): every scatter block then sums the table for its own keys - the keys' totals and the counts of the blocks
// before it - and block 0 also writes the segment tables; one kernel and one launch gap less.
struct ScanInline {
  const int* counts;      // [nblk][nkey], or null: block_base / key_off come from the scan kernel
  int nblk, G, nsub, row_align, max_tiles;
  int *seg_off, *seg_cnt, *n_rows, *tile_cluster;
};

// The row move done by the scatter blocks themselves (MoveInline.on; only with ScanInline): a block copies the rows
// of its own token tile, which are contiguous in x, to their places in x_perm, zeroes its share of the clusters'
// padding rows and of the accumulation buffer; blocks nblk.. stage the INT4 factors.  One launch less, and the rows'
// places never travel through memory.
struct MoveInline {
  int on;
  int rep;             // rows of x are shared by `rep` consecutive (virtual) tokens: token t reads row t / rep
  uint4* zero_ptr;
  size_t zero_n;
  FactorStage fs;
};

__global__ void __launch_bounds__(512)      // at least `tile` threads: the token tile of the kernel that counted the keys
scatter_kernel(int T, int tile, int d, int K, int k, int nkey, int sub_is_combo,
               const __half* __restrict__ x, const int* __restrict__ cluster_id,
               const int* __restrict__ slot, const float* __restrict__ gates,
               const int* __restrict__ keys, const int* __restrict__ block_base,
               const int* __restrict__ key_off,
               int* __restrict__ row_token, int* __restrict__ row_slot, float* __restrict__ row_gate,
               __half* __restrict__ x_perm, const ScanInline si, const MoveInline mv) {
  pdl_wait();
  if (mv.on && (int)blockIdx.x >= si.nblk) { stage_block(mv.fs, blockIdx.x - si.nblk); return; }
  extern __shared__ int sh_next[];   // next free row of each key for this block
  __shared__ int sh_seg[kMaxG + 1];
  __shared__ int sh_segcnt[kMaxG];
  __shared__ int sh_row[512];        // fused move: the row of each token of this block's tile (-1: none)
  if (si.counts) {
    int* sh_tot = sh_next + nkey;    // [nkey] tokens of each key in the whole batch
    // Column sums of the count table, read along its rows: lanes over the keys (four columns of 32 keys per pass),
    // warps over the counting blocks; a key's total and the part of the blocks before this one.
    for (int key = threadIdx.x; key < nkey; key += blockDim.x) { sh_tot[key] = 0; sh_next[key] = 0; }
    __syncthreads();
    {
      const int lane_ = threadIdx.x & 31, warp_ = threadIdx.x >> 5, nwarp_ = blockDim.x >> 5;
      for (int k0 = 0; k0 < nkey; k0 += 128) {
        int tot[4] = {0, 0, 0, 0}, bef[4] = {0, 0, 0, 0};
#pragma unroll 4
        for (int b = warp_; b < si.nblk; b += nwarp_) {
          const bool before = b < (int)blockIdx.x;
#pragma unroll
          for (int j = 0; j < 4; ++j) {
            const int key = k0 + 32 * j + lane_;
            const int c = key < nkey ? si.counts[(size_t)b * nkey + key] : 0;
            tot[j] += c;
            bef[j] += before ? c : 0;
          }
        }
#pragma unroll
        for (int j = 0; j < 4; ++j) {
          const int key = k0 + 32 * j + lane_;
          if (key < nkey) { atomicAdd(&sh_tot[key], tot[j]); atomicAdd(&sh_next[key], bef[j]); }
        }
      }
    }
    __syncthreads();
    if (threadIdx.x < si.G) {
      // tokens of this thread's cluster, then (thread 0) the padded segment offsets
      int cnt = 0;
      for (int sb = 0; sb < si.nsub; ++sb) cnt += sh_tot[threadIdx.x * si.nsub + sb];
      sh_segcnt[threadIdx.x] = cnt;
    }
    __syncthreads();
    if (threadIdx.x == 0) {
      int off = 0;
      for (int g = 0; g < si.G; ++g) {
        sh_seg[g] = off;
        off += (sh_segcnt[g] + si.row_align - 1) / si.row_align * si.row_align;
      }
      sh_seg[si.G] = off;
    }
    __syncthreads();
    if (threadIdx.x < si.G) {
      // first row of every key of this thread's cluster, plus the rows of the blocks before this one
      int off = sh_seg[threadIdx.x];
      for (int sb = 0; sb < si.nsub; ++sb) {
        const int key = threadIdx.x * si.nsub + sb;
        sh_next[key] += off;
        off += sh_tot[key];
      }
    }
    if (blockIdx.x == 0) {
      // block 0 also writes the tables the later kernels read
      for (int g = threadIdx.x; g <= si.G; g += blockDim.x) {
        si.seg_off[g] = sh_seg[g];
        if (g < si.G) si.seg_cnt[g] = sh_segcnt[g];
      }
      if (threadIdx.x == 0) *si.n_rows = sh_seg[si.G];
      for (int g = 0; g < si.G; ++g) {
        const int first = sh_seg[g] + sh_segcnt[g], last = sh_seg[g + 1];
        for (int row = first + (int)threadIdx.x; row < last; row += blockDim.x) {
          row_token[row] = -1;
          for (int j = 0; j < k; ++j) {
            row_slot[(size_t)row * k + j] = g * K + j;       // any valid experts of the cluster
            row_gate[(size_t)row * k + j] = 0.f;
          }
        }
      }
      const int ntile = sh_seg[si.G] / si.row_align;
      for (int tile = threadIdx.x; tile < si.max_tiles; tile += blockDim.x) {
        int g = -1;
        if (tile < ntile) {
          const int row = tile * si.row_align;
          g = 0;
          while (g + 1 < si.G && sh_seg[g + 1] <= row) ++g;
        }
        si.tile_cluster[tile] = g;
      }
    }
  } else {
    for (int i = threadIdx.x; i < nkey; i += blockDim.x)
      sh_next[i] = key_off[i] + block_base[(size_t)blockIdx.x * nkey + i];
  }
  __syncthreads();
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int t = blockIdx.x * tile + threadIdx.x;              // a block takes the tokens one counting block took,
  const int my_key = ((int)threadIdx.x < tile && t < T) ? keys[t] : -1;       // a thread each (the block may have more threads: they help with the sums above)
  const bool live = my_key >= 0;                  // (a virtual token without a cluster has key -1 and gets no row)
  const int key = live ? my_key : -1 - lane;      // dead lanes get unique keys: groups of one
  const unsigned peers = __match_any_sync(0xffffffffu, key);
  const int rank_in_warp = __popc(peers & ((1u << lane) - 1u));
  const bool leader = rank_in_warp == 0;
  int row = -1;
  // warps take their rows in warp order, so rows of a key stay in token order
  for (int w = 0; w < (tile >> 5); ++w) {
    if (warp == w && live) {
      row = sh_next[key] + rank_in_warp;
    }
    __syncthreads();
    if (warp == w && live && leader) sh_next[key] += __popc(peers);
    __syncthreads();
  }
  if (live) {
    int cs[kMaxKsel];
    float cg[kMaxKsel];
    canonical_slots(slot + (size_t)t * k, gates + (size_t)t * k, k, sub_is_combo, cs, cg);
    const int g = cluster_id[t];
    row_token[row] = t;
#pragma unroll
    for (int j = 0; j < kMaxKsel; ++j)
      if (j < k) {
        row_slot[(size_t)row * k + j] = g * K + cs[j];
        row_gate[(size_t)row * k + j] = cg[j];
      }
  }
  if (!mv.on) return;
  // ---- the row move, by the block that placed the rows
  if ((int)threadIdx.x < tile) sh_row[threadIdx.x] = row;
  __syncthreads();
  const int vec_per_row = d / 8, nthr = (int)blockDim.x;
  {
    // this tile's tokens are consecutive rows of x (every row mv.rep times when the tokens are virtual ones): vector i
    // of the tile is vector i % vec_per_row of token i / vec_per_row
    const int t0 = blockIdx.x * tile, nt = min(tile, T - t0);
    const uint4* src = reinterpret_cast<const uint4*>(x);
    const int nvec = nt * vec_per_row, rdiv = mv.rep;
    for (int i0 = threadIdx.x; i0 < nvec; i0 += 8 * nthr) {
      uint4 val[8];
#pragma unroll
      for (int u = 0; u < 8; ++u) {
        const int i = i0 + u * nthr;
        if (i < nvec) {
          const int tt = i / vec_per_row;
          val[u] = src[(size_t)((t0 + tt) / rdiv) * vec_per_row + (i - tt * vec_per_row)];
        }
      }
#pragma unroll
      for (int u = 0; u < 8; ++u) {
        const int i = i0 + u * nthr;
        if (i < nvec) {
          const int tt = i / vec_per_row, r = sh_row[tt];
          if (r >= 0) reinterpret_cast<uint4*>(x_perm + (size_t)r * d)[i - tt * vec_per_row] = val[u];
        }
      }
    }
  }
  // padding rows of every cluster: block b takes every nblk-th of them
  for (int g = 0; g < si.G; ++g) {
    const int first = sh_seg[g] + sh_segcnt[g], last = sh_seg[g + 1];
    for (int prow = first + (int)blockIdx.x; prow < last; prow += si.nblk) {
      uint4* dstp = reinterpret_cast<uint4*>(x_perm + (size_t)prow * d);
      for (int v = threadIdx.x; v < vec_per_row; v += nthr) dstp[v] = make_uint4(0, 0, 0, 0);
    }
  }
  // the accumulation buffer of the later stages starts at zero
  for (size_t i = (size_t)blockIdx.x * nthr + threadIdx.x; i < mv.zero_n; i += (size_t)si.nblk * nthr)
    mv.zero_ptr[i] = make_uint4(0, 0, 0, 0);
}

// x_perm[row] = x[row_token[row]], zeros for padding rows; a block per row, 16 bytes per thread
__global__ void __launch_bounds__(128)
move_rows_kernel(int d, const int* __restrict__ n_rows, const int* __restrict__ row_token,
                 const __half* __restrict__ x, __half* __restrict__ x_perm, uint4* __restrict__ zero_ptr, size_t zero_n,
                 int n_move, const FactorStage fs, int rdiv) {
  pdl_wait();
  // blocks n_move.. decode the layer's INT4 factors for the tensor-core residual products (weights only; a few MB
  // more for a kernel that is bound by memory bandwidth anyway)
  if ((int)blockIdx.x >= n_move) { stage_block(fs, blockIdx.x - n_move); return; }
  const int vec_per_row = d / 8;
  const int rows = x != nullptr ? *n_rows : 0;                 // (no x: a later kernel gathers the rows)
  // four rows at a time: their token lookups, then their loads, are in flight together instead of one row's
  // lookup - load - store chain after the other
  for (int row0 = blockIdx.x; row0 < rows; row0 += 4 * n_move) {
    int tok[4];
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      const int row = row0 + i * n_move;
      tok[i] = row < rows ? row_token[row] : -2;               // -2: no such row
    }
    for (int v = threadIdx.x; v < vec_per_row; v += blockDim.x) {
      uint4 val[4];
#pragma unroll
      for (int i = 0; i < 4; ++i)
        val[i] = tok[i] >= 0 ? reinterpret_cast<const uint4*>(x + (size_t)(tok[i] / rdiv) * d)[v] : make_uint4(0, 0, 0, 0);
#pragma unroll
      for (int i = 0; i < 4; ++i)
        if (tok[i] != -2) reinterpret_cast<uint4*>(x_perm + (size_t)(row0 + i * n_move) * d)[v] = val[i];
    }
  }
  // the accumulation buffer of the later stages starts at zero
  for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < zero_n; i += (size_t)n_move * blockDim.x)
    zero_ptr[i] = make_uint4(0, 0, 0, 0);
}


// The whole permutation of a small batch (T <= 256) in one block: keys, counts, offsets, the stable
// rank of every token inside its key (by counting the earlier tokens with the same key), the row
// tables and the padding rows.  Gives exactly the tables the four kernels above give.
constexpr int kSmallT = 256;

__global__ void __launch_bounds__(kSmallT)
permute_small_kernel(int T, int G, int K, int k, int nsub, int nkey, int sub_is_combo, int row_align, int max_tiles,
                     const int* __restrict__ cluster_id, const int* __restrict__ slot, const float* __restrict__ gates,
                     int* __restrict__ seg_off, int* __restrict__ seg_cnt, int* __restrict__ n_rows,
                     int* __restrict__ tile_cluster, int* __restrict__ row_token, int* __restrict__ row_slot,
                     float* __restrict__ row_gate, const LowrankTok lr) {
  pdl_wait();
  // blocks 1.. : t = x U1 of every (token, kept expert) on the weight-streaming path: it needs the routes,
  // not the permutation, and hides in this block's latency
  if (blockIdx.x > 0) { lowrank_tok_block(lr, blockIdx.x - 1); return; }
  extern __shared__ int sh[];
  int* cnt = sh;                   // [nkey] tokens per key, then first row of the key
  int* keys = cnt + nkey;          // [kSmallT]
  __shared__ int s_seg[kMaxG + 1];
  __shared__ int s_cnt[kMaxG];
  const int t = threadIdx.x;
  for (int i = t; i < nkey; i += blockDim.x) cnt[i] = 0;
  __syncthreads();
  int cs[kMaxKsel];
  float cg[kMaxKsel];
  int key = -1, g = 0;
  if (t < T) {
    const int sub = canonical_slots(slot + (size_t)t * k, gates + (size_t)t * k, k, sub_is_combo, cs, cg);
    g = cluster_id[t];
    key = g >= 0 ? g * nsub + sub : -1;                  // (a virtual token without a cluster gets no row)
    if (key >= 0) atomicAdd(&cnt[key], 1);
  }
  keys[t] = key;
  __syncthreads();
  if (t == 0) {
    int off = 0;
    for (int c = 0; c < G; ++c) {
      s_seg[c] = off;
      seg_off[c] = off;
      int n = 0;
      for (int sb = 0; sb < nsub; ++sb) {
        const int here = cnt[c * nsub + sb];
        cnt[c * nsub + sb] = off + n;          // first row of the key
        n += here;
      }
      seg_cnt[c] = n;
      s_cnt[c] = n;
      off += (n + row_align - 1) / row_align * row_align;
    }
    s_seg[G] = off;
    seg_off[G] = off;
    *n_rows = off;
  }
  __syncthreads();
  if (t < T && key >= 0) {
    int rank = 0;
    for (int u = 0; u < t; ++u) rank += keys[u] == key ? 1 : 0;
    const int row = cnt[key] + rank;
    row_token[row] = t;
    for (int j = 0; j < k; ++j) {
      row_slot[(size_t)row * k + j] = g * K + cs[j];
      row_gate[(size_t)row * k + j] = cg[j];
    }
  }
  // padding rows of every cluster, and the cluster of every tile
  for (int row = t; row < s_seg[G]; row += blockDim.x) {
    int c = 0;
    while (c + 1 < G && s_seg[c + 1] <= row) ++c;
    if (row - s_seg[c] >= s_cnt[c]) {                  // past the cluster's tokens
      row_token[row] = -1;
      for (int j = 0; j < k; ++j) {
        row_slot[(size_t)row * k + j] = c * K + j;     // any valid experts of the cluster
        row_gate[(size_t)row * k + j] = 0.f;
      }
    }
  }
  const int ntile = s_seg[G] / row_align;
  for (int tile = t; tile < max_tiles; tile += blockDim.x) {
    int c = -1;
    if (tile < ntile) {
      const int row = tile * row_align;
      c = 0;
      while (c + 1 < G && s_seg[c + 1] <= row) ++c;
    }
    tile_cluster[tile] = c;
  }
}

// the count table is small enough for every scatter block to sum it itself
bool inline_scan_ok(const Dims& D, int nblk, int tile) { return (long long)nblk * D.nkey <= 65536 && D.G <= tile; }

}  // namespace

int permute_launches(const Dims& D, int T, int counted_tile, bool separate_move) {
  if (T <= kSmallT) return 2;
  if (counted_tile <= 0) return 4;
  const int nblk = (T + counted_tile - 1) / counted_tile, sms = D.sm_count > 0 ? D.sm_count : 148;
  const bool fused = !separate_move && counted_tile <= 512 && (long long)T * D.d * 2 / (nblk < sms ? nblk : sms) <= 600 * 1024;
  return inline_scan_ok(D, nblk, counted_tile) ? (fused ? 1 : 2) : 3;
}

cudaError_t launch_permute(const Dims& D, const Scratch& S, const __half* x, int T, cudaStream_t st, void* zero_ptr,
                           size_t zero_bytes, const FactorStage& fs, const LowrankTok& lr, int counted_tile, int x_div,
                           bool move_in_scatter) {
  if (x_div < 1) x_div = 1;

  const int rows_bound = t_pad_bound(D, T);
  if (T <= kSmallT) {
    // (the factor staging rode in the router kernel)
    launch_chained(permute_small_kernel, dim3(1 + lowrank_tok_blocks(lr)), dim3(kSmallT), sizeof(int) * ((size_t)D.nkey + kSmallT), st, 1,
      
        T, D.G, D.K, D.k, D.nsub, D.nkey, D.sub_is_combo, D.row_align, D.T_pad_max / D.row_align, S.cluster_id, S.slot,
        S.gates, S.seg_off, S.seg_cnt, S.n_rows, S.tile_cluster, S.row_token, S.row_slot, S.row_gate, lr);
    launch_chained(move_rows_kernel, dim3(rows_bound), dim3(128), 0, st, 1,
      D.d, S.n_rows, S.row_token, x, S.x_perm, static_cast<uint4*>(zero_ptr), zero_bytes / 16, rows_bound, FactorStage{}, x_div);
    return cudaGetLastError();
  }
  // counting blocks: the router's token tiles when it counted the keys itself (counted_tile tokens each), else
  // blocks of 256 tokens counted here
  const int tile = counted_tile > 0 ? counted_tile : kPermBlock;
  const int nblk = (T + tile - 1) / tile;
  const size_t sh = sizeof(int) * (size_t)D.nkey;
  if (counted_tile <= 0)
    launch_chained(hist_kernel, dim3(nblk), dim3(kPermBlock), sh, st, 1,
        T, D.k, D.nsub, D.nkey, D.sub_is_combo, S.cluster_id,
                                              S.slot, S.gates, S.keys, S.block_counts);
  // a small count table: every scatter block sums it for itself and the scan kernel is not launched
  ScanInline si{};
  const bool inline_scan = counted_tile > 0 && inline_scan_ok(D, nblk, tile);
  if (inline_scan) {
    si.counts = S.block_counts; si.nblk = nblk; si.G = D.G; si.nsub = D.nsub; si.row_align = D.row_align;
    si.max_tiles = D.T_pad_max / D.row_align;
    si.seg_off = S.seg_off; si.seg_cnt = S.seg_cnt; si.n_rows = S.n_rows; si.tile_cluster = S.tile_cluster;
  } else {
    launch_chained(scan_kernel, dim3(1), dim3(1024), 0, st, 1,
        nblk, D.G, D.nsub, D.nkey, D.row_align, D.T_pad_max / D.row_align,
                                    S.block_counts, S.block_base, S.key_cnt, S.key_off, S.seg_off,
                                    S.seg_cnt, S.n_rows, S.tile_cluster, D.K, D.k, S.row_token, S.row_slot, S.row_gate);
  }
  // on request (cmoe_options.move_in_scatter) the scatter blocks that do the sums also move their tile's rows
  MoveInline mv{};
  // (not when that would leave each of too few blocks with megabytes to move: the row-move kernel then does better)
  const int sms = D.sm_count > 0 ? D.sm_count : 148;
  const bool fused_move = move_in_scatter && inline_scan && x != nullptr && tile <= 512 &&
                          (long long)T * D.d * 2 / (nblk < sms ? nblk : sms) <= 600 * 1024;
  if (fused_move) { mv.on = 1; mv.rep = x_div; mv.zero_ptr = static_cast<uint4*>(zero_ptr); mv.zero_n = zero_bytes / 16; mv.fs = fs; }
  launch_chained(scatter_kernel, dim3(nblk + (fused_move ? stage_blocks(fs, 512) : 0)), dim3(inline_scan ? 512 : tile),
                 sh * (inline_scan ? 2 : 1), st, 1,
      T, tile, D.d, D.K, D.k, D.nkey, D.sub_is_combo, x,
                                               S.cluster_id, S.slot, S.gates, S.keys, S.block_base,
                                               S.key_off, S.row_token, S.row_slot, S.row_gate,
                                               S.x_perm, si, mv);
  if (fused_move) return cudaGetLastError();
  const int move_max = (D.sm_count > 0 ? D.sm_count : 148) * 32;      // resident blocks of 128 threads
  const int move_grid = rows_bound < move_max ? rows_bound : move_max;
  launch_chained(move_rows_kernel, dim3(move_grid + stage_blocks(fs, 128)), dim3(128), 0, st, 1,
      D.d, S.n_rows, S.row_token, x, S.x_perm, static_cast<uint4*>(zero_ptr), zero_bytes / 16, move_grid, fs, x_div);
  return cudaGetLastError();
}

}  // namespace cmoe
