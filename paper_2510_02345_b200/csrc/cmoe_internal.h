// Internal declarations shared by the translation units of libcmoe: the handle, the arena plan,
// the per-call scratch views and the kernel launchers.  Nothing here is part of the C boundary.
#pragma once

#include <cuda.h>
#include <cuda_fp16.h>
#include <cuda_runtime.h>
#include <stddef.h>
#include <stdint.h>

#include "cmoe.h"

namespace cmoe {

constexpr int kMaxG = 64;          // clusters
constexpr int kMaxK = 32;          // experts per cluster (one lane each in the router's top-k)
constexpr int kMaxKsel = 8;        // k
constexpr int kMaxKeys = 4096;     // permutation keys (cluster x expert combination)
constexpr int kMaxHostChunks = 8; // most chunks cmoe_forward_host cuts a batch into
constexpr int kSeqTokens = 384;    // largest T_max that is served in pieces of 128 tokens on the weight-streaming path (Dims::seq)
constexpr int kPermBlock = 256;    // tokens per block in the permutation kernels (when they count the keys themselves)
constexpr int kMinCountTile = 128; // token tile of the router kernel that counts keys (router_tc.cu)

enum Path { kPathGeneric = 0, kPathTensor = 1, kPathStream = 2 };

// Expert parts (split == 2 or 4): a cluster whose K r exceeds the 64 columns of the pair path's expanded rank index is
// handled as `split` virtual clusters of K / split experts (virtual cluster split g + c = experts c K / split .. of
// cluster g: the expert numbering e = g K + i does not change) that share the base of cluster g.  A token becomes
// `split` virtual tokens, one per part, each with those of its kept experts that lie in the part and, in its remaining
// slots, other experts of the part at gate zero; a part without any of the token's experts has no row; the outputs are
// summed.  G and K below are then the virtual counts (split G, K / split): everything behind the router sees an
// ordinary layer; the router and the bases use real_G / real_K.
struct Dims {
  int d, d_ff, E, G, K, r, k;
  int nsub;        // permutation sub-keys per cluster (expert combinations, or lowest expert)
  int nkey;        // G * nsub
  int T_max;       // most tokens of a call as the kernels see them: g1 virtual tokens per caller token
  int T_user;      // most tokens of a call as the caller counts them (T_max = g1 * T_user)
  int g1;          // clusters per token (Sec. 3.3); 0 and 1 both mean one
  int split;       // 2 or 4: the clusters are handled as that many parts of K / split experts each (above); else 0
  int rep;         // rows of the kernels' x per caller token: max(g1, split, 1)
  int seq;         // > 0: a call's tokens go through the layer in consecutive pieces of at most `seq` tokens (= T_max):
                   // few tokens on a layer whose clusters would have to be split (below) stream the weights once per
                   // piece instead of computing two to four base products per token
  int T_pad_max;   // rows of the permuted buffers
  int row_align;   // a cluster's rows start at a multiple of this
  int sub_is_combo;
  int tc2;         // the shape takes the tensor-core path with tensor-core residuals (tc2_path.cu)
  int stream;      // the shape takes the weight-streaming path (stream_path.cu)
  int sm_count;    // multiprocessors of the handle's device (set by cmoe_create; 0 in pure host queries)
};

// Weights as re-laid-out in the arena by cmoe_create.
struct Weights {
  const float* Ct;   // [G][d]     cluster prototypes, one row per cluster
  const float* Rt;   // [E][d]     expert router vectors, one row per expert slot
  const float* bc;   // [G]        (zeros when the caller passed NULL)
  const float* be;   // [E]
  const int* label;  // [E]        expert label written to expert_ids
  const __half* B1t; // [G][d_ff][d]   base of the up-projection, reduction index fastest
  const __half* B2t; // [G][d][d_ff]   base of the down-projection, reduction index fastest
  const uint8_t *U1q, *V1q, *U2q, *V2q;  // packed INT4 in the boundary layouts
  const __half *U1s, *V1s, *U2s, *V2s;   // fp16 scale per 32 flat elements
  const int* live;   // [E]  bit 0: the residual U1_e V1_e is not a zero block, bit 1: U2_e V2_e is not (Sec. 3.4's pruned blocks)
};

// Per-call scratch in the arena.
struct Scratch {
  // token order
  int* cluster_id;    // [T]
  int* slot;          // [T][k]  local expert index inside the cluster, routing order
  float* gates;       // [T][k]
  int* keys;          // [T]     permutation key = cluster * nsub + sub
  // permutation tables
  int* block_counts;  // [nblk][nkey]
  int* block_base;    // [nblk][nkey]  rows of this key owned by earlier blocks
  int* key_cnt;       // [nkey]
  int* key_off;       // [nkey]  first permuted row of the key
  int* seg_off;       // [G+1]   first permuted row of each cluster (multiple of row_align)
  int* seg_cnt;       // [G]     tokens of each cluster
  int* n_rows;        // [1]     seg_off[G]
  int* tile_cluster;  // [T_pad_max / row_align]
  // permuted-row order
  int* row_token;     // [T_pad]     source token, -1 for padding rows
  int* row_slot;      // [T_pad][k]  expert slot ids (g*K+i), ascending
  float* row_gate;    // [T_pad][k]  gates in the same order (0 for padding rows)
  __half* x_perm;     // [T_pad][d]
  __half* x_rep;      // [T_max][d]  g1 > 1: every token's row g1 times (one virtual token per kept cluster)
  __half* y_rep;      // [T_max][d]  g1 > 1: the virtual tokens' outputs, summed per token at the end
  int* r_cluster;     // [T_user]     expert halves: the token's own routes, before they are split
  int* r_slot;        // [T_user][k]
  float* r_gates;     // [T_user][k]
  float* t;           // [T_pad][k][r]   x U1_e
  __half* abar;       // [T_pad][d_ff]   sum_j p_j GELU(h_j)
  float* s;           // [T_pad][k][r]   GELU(h_j) U2_e, accumulated with atomics
  int* status;        // [1]
  // tensor-core path with tensor-core residuals only (see tc2_path.cu)
  __half *U1f, *V1f, *U2f, *V2f;   // INT4 factors decoded to fp16 operand matrices, per call
  __half *A0, *Ad, *As;            // [T_pad][64] expanded-rank-index operands
  int* tile_mask;                  // [T_pad / 128][2]  16-wide steps of the expanded index the up projection needs
  int* tile_mask_dn;               // [T_pad / 128]     the same for the down projection
  // weight-streaming path only (see stream_path.cu)
  __half* a_slot;                  // [T_pad][k][d_ff]  GELU(h_j) of every kept expert
  float* y32;                      // [T_pad][d]        fp32 sum of the K ranges of the down-projection
  // tensor-core router only (see router_tc.cu): the fp32 router rows split into two fp16 pieces
  __half* Wsplit;                  // [2 * rp][d]
};

}  // namespace cmoe

struct cmoe_layer {
  cmoe::Dims dims;
  cmoe::Weights w;
  cmoe::Scratch sc;
  cmoe_options opt;  // what cmoe_create_ex was given (defaults otherwise)
  int path;
  int tc_variant;   // 1: tc_path.cu, 2: tc2_path.cu (when path == kPathTensor)
  int router_tc;    // batches of at least 1024 tokens are routed by router_tc.cu
  int pruned_blocks; // residual blocks (an expert's U V of one matrix) found to be entirely zero at create time
  CUtensorMap router_map_w;
  int last_cuda_error;
  // optional stage timing (cmoe_profile_*)
  int profiling;
  int n_stages;
  const char* stage_names[CMOE_MAX_STAGES];
  cudaEvent_t events[CMOE_MAX_STAGES + 1];
  int events_created;
  int events_recorded;
  // a second stream for work that does not depend on the kernel running on the caller's stream (forked and
  // joined with the two events inside one forward); created with the handle, never allocated per call
  cudaStream_t side_stream;
  cudaEvent_t side_fork, side_join;
  int side_created;
  // cmoe_forward_host: a stream per copy direction and an event per chunk and direction
  cudaStream_t h2d_stream, d2h_stream;
  cudaEvent_t host_fork, host_join, chunk_in[cmoe::kMaxHostChunks], chunk_done[cmoe::kMaxHostChunks];
  int host_created;     // objects created so far, in the order above
  // tensor-core path: tensor maps and launch shapes (opaque here, see tc_path.cu)
  alignas(128) unsigned char tc_state[4096];
};

namespace cmoe {

inline int round_up(int a, int b) { return (a + b - 1) / b * b; }
inline int real_G(const Dims& D) { return D.split > 1 ? D.G / D.split : D.G; }
inline int real_K(const Dims& D) { return D.split > 1 ? D.K * D.split : D.K; }
inline int t_pad_bound(const Dims& D, int T) { return round_up(T, D.row_align) + D.G * D.row_align; }

// ---- launchers (each returns the cudaError_t of its launches) ----------------------------------
// router.cu
// fs (or null): factor staging that rides in the per-token kernel's grid (batches below 1024 tokens)
struct KeyCount;      // perm_keys.cuh
struct FactorStage;   // stage_factors.cuh
struct LowrankTok;    // lowrank.cuh
cudaError_t launch_router(const Dims& D, const Weights& W, const __half* x, int T,
                          int* cluster_id, int* expert_ids, float* gates, int* slot_local,
                          cudaStream_t st, const FactorStage* fs = nullptr);
// router_tc.cu : the same routing on the tensor cores (split fp16 router matrices), for large batches
int router_tc_rp(const Dims& D);
bool router_tc_supported(const Dims& D);
cudaError_t router_tc_init(cmoe_layer* L);
// kc (or null): the kernel also writes every token's permutation key and the key counts of its 128-token tiles
cudaError_t launch_router_tc(const cmoe_layer* L, const __half* x, int T, int* cluster_id, int* expert_ids, float* gates,
                             int* slot_local, cudaStream_t st, const KeyCount* kc = nullptr);
// the routers work on the real clusters, also when the layer behind them works on expert halves (Dims::split)
inline Dims plain_dims(const Dims& D) { Dims R = D; R.G = real_G(D); R.K = real_K(D); R.split = 0; return R; }
int router_tc_tile_tokens();
// permute.cu : histogram, scan, scatter (+ row gather), padding rows
// also clears zero_bytes (a multiple of 16) at zero_ptr: the buffer the later stages accumulate into
// counted_tile > 0: the router kernel has already written the keys and the key counts of its tiles of that many tokens
cudaError_t launch_permute(const Dims& D, const Scratch& S, const __half* x, int T, cudaStream_t st, void* zero_ptr,
                           size_t zero_bytes, const FactorStage& fs, const LowrankTok& lr, int counted_tile, int x_div = 1,
                           bool move_in_scatter = false);
// kernels of the permutation: 2 for batches of at most 256 tokens, 4 below 1024 tokens, else 3 (the router counts the
// keys) or 2 (and the scatter kernel sums the small count table itself; see launch_permute)
int permute_launches(const Dims& D, int T, int counted_tile, bool separate_move);
// generic_path.cu : CUDA-core path for any supported shape
// `marks` (or null): three events recorded before the residual-t, up and down stages
cudaError_t launch_generic_ffn(const Dims& D, const Weights& W, const Scratch& S, int T, __half* y,
                               cudaStream_t st, cudaEvent_t* marks);
constexpr int kGenericFfnLaunches = 3;
// t = x_perm U1_e for every permuted row and kept expert (no-op when r == 0)
cudaError_t launch_residual_t(const Dims& D, const Weights& W, const Scratch& S, int T, cudaStream_t st);
// tc_path.cu : tcgen05/TMEM/TMA grouped GEMMs with the fused epilogues
bool tc_supported(const Dims& D);
cudaError_t tc_init(cmoe_layer* L);
cudaError_t launch_tc_ffn(const cmoe_layer* L, int T, __half* y, cudaStream_t st, cudaEvent_t* marks);
// tc2_path.cu : the same with the rank-r residual products on the tensor cores as well
bool tc2_supported(const Dims& D);
cudaError_t tc2_init(cmoe_layer* L);
int tc2_launch_count(const cmoe_layer* L);
void tc2_accum_buffer(const cmoe_layer* L, int T, void** ptr, size_t* bytes);
void tc2_factor_stage(const cmoe_layer* L, FactorStage* fs);
// x_src: not null when the t kernel gathers the rows of x itself (tc2_gathers_rows)
cudaError_t launch_tc2_ffn(const cmoe_layer* L, const __half* x_src, int T, __half* y, cudaStream_t st, cudaEvent_t* marks);
bool tc2_gathers_rows(const cmoe_layer* L);

// multi_cluster.cu (virtual tokens): x_rep[n t + c] = x[t];  y[t] = sum_c y_rep[n t + c]
cudaError_t launch_repeat_rows(const Dims& D, const __half* x, __half* x_rep, int T, int n, cudaStream_t st);
// cluster_id (or null): virtual tokens whose entry is negative have no row
cudaError_t launch_sum_rows(const Dims& D, const __half* y_rep, __half* y, int T, int n, const int* cluster_id, cudaStream_t st);
// expert halves: the token's own routes in Scratch::r_* -> the virtual tokens' routes (cluster_id, slot, gates)
struct KeyCount;
// routes of the T tokens -> routes of their virtual tokens; with kc the kernel also writes the virtual tokens' permutation
// keys and counts them per block of split_routes_tile() virtual tokens
cudaError_t launch_split_routes(const Dims& D, const Scratch& S, int T, cudaStream_t st, const KeyCount* kc);
int split_routes_tile();
// stream_path.cu : small batches, bound by streaming the bases from HBM
bool stream_supported(const Dims& D);
cudaError_t stream_init(cmoe_layer* L);
int stream_launch_count(const Dims& D);
void stream_lowrank_rider(const cmoe_layer* L, const __half* x, int T, LowrankTok* lr);
cudaError_t launch_stream_ffn(const cmoe_layer* L, int T, __half* y, cudaStream_t st, cudaEvent_t* marks);
// repack.cu : create-time layout changes; residual blocks that are entirely zero
cudaError_t launch_residual_live(const Dims& D, const Weights& W, cudaStream_t st);

// src_is_bf16: the source holds bfloat16 bit patterns, converted to fp16 on the way
cudaError_t launch_transpose_fp16(const __half* src, __half* dst, int batch, int rows, int cols,
                                  cudaStream_t st, bool src_is_bf16 = false);
cudaError_t launch_transpose_f32(const float* src, float* dst, int batch, int rows, int cols,
                                 cudaStream_t st);
// src [batch][rows][cols] -> dst [rows / 128][batch * cols][128] (rows a multiple of 128): the layout the
// weight-streaming path reads its bases in
cudaError_t launch_stage_major_fp16(const __half* src, __half* dst, int batch, int rows, int cols, cudaStream_t st,
                                    bool src_is_bf16 = false);

}  // namespace cmoe
