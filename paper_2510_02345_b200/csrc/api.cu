// The C boundary of libcmoe (include/cmoe.h): descriptor validation, the arena plan, weight
// re-layout at create time and the launch sequences of cmoe_route / cmoe_forward.
#include <cstdlib>
#include <new>

#include <cmath>

#include "cmoe_internal.h"
#include "stage_factors.cuh"
#include "lowrank.cuh"
#include "perm_keys.cuh"

using namespace cmoe;

namespace {

constexpr int kDefaultHostChunks = 4;   // chunks of a large batch in cmoe_forward_host unless the options say otherwise

struct Arena {
  size_t used = 0;
  char* base = nullptr;
  template <typename T>
  T* take(size_t count) {
    size_t off = (used + 255) / 256 * 256;
    used = off + count * sizeof(T);
    return base ? reinterpret_cast<T*>(base + off) : nullptr;
  }
};

long long binom_ll(int n, int m) {
  if (m > n) return 0;
  long long r = 1;
  for (int i = 1; i <= m; ++i) {
    r = r * (n - m + i) / i;
    if (r > (1ll << 40)) return r;
  }
  return r;
}

// Few tokens on a layer whose clusters would be handled as `parts` parts: pieces of 128 tokens on the streaming
// kernels, or the parts on the pair kernels?  Estimates in us, fitted to measurements on a B200 (four layers from
// 134 MB to 1.9 GB of bases, 129 to 384 tokens; the constants do not depend on the device so that the host query and
// cmoe_create always agree):
//   a piece     80 + bytes of the bases / 6.0 TB/s      (one pass over the weights and the launch chain)
//   the parts   60 + rounds of 256 x 256 pair tiles on 74 CTA pairs: parts * G row tiles (one per virtual cluster at
//               these sizes), 8.6 us * d / 1024 per up tile, 6.7 us * d_ff / 1024 per down tile (half for 128 columns)
// Pieces are taken when they come out at least 15 % ahead.
bool pieces_win(const cmoe_desc& desc, int parts) {
  const double d = desc.d, f = desc.d_ff, G = desc.G;
  const double piece = 80.0 + 2.0 * G * d * f * 2.0 / 6.0e6;
  const double n_pieces = (desc.T_max + 127) / 128;
  const double row_tiles = (double)parts * G, pairs = 74.0;
  const double up_rounds = std::ceil(row_tiles * std::ceil(f / 256.0) / pairs);
  const bool dn_wide = desc.d % 256 == 0;
  const double dn_rounds = std::ceil(row_tiles * std::ceil(d / (dn_wide ? 256.0 : 128.0)) / pairs);
  const double split = 60.0 + up_rounds * 8.6 * d / 1024.0 + dn_rounds * (dn_wide ? 6.7 : 3.35) * f / 1024.0;
  return n_pieces * piece < 0.85 * split;
}

int validate_dims(const cmoe_desc* desc, int g1, bool allow_split, Dims* D) {
  if (!desc) return CMOE_ERR_INVALID_ARG;
  if (g1 < 0 || g1 > 2) return CMOE_ERR_INVALID_ARG;
  if (g1 < 1) g1 = 1;
  if (g1 > desc->G) return CMOE_ERR_UNSUPPORTED_SHAPE;
  if (desc->d <= 0 || desc->d_ff <= 0 || desc->E <= 0 || desc->G <= 0 || desc->k <= 0 ||
      desc->r < 0 || desc->T_max <= 0)
    return CMOE_ERR_INVALID_ARG;
  if (desc->E % desc->G) return CMOE_ERR_UNSUPPORTED_SHAPE;
  const int K = desc->E / desc->G;
  if (desc->G > kMaxG || K > kMaxK || desc->k > K || desc->k > kMaxKsel) return CMOE_ERR_UNSUPPORTED_SHAPE;
  if (desc->d % 32 || desc->d_ff % 32) return CMOE_ERR_UNSUPPORTED_SHAPE;
  if (!(desc->r == 0 || desc->r == 4 || desc->r == 8 || desc->r == 16 || desc->r == 32))
    return CMOE_ERR_UNSUPPORTED_SHAPE;
  if (desc->quant_group != 32) return CMOE_ERR_UNSUPPORTED_SHAPE;
  if ((long long)desc->T_max * g1 > (1 << 22)) return CMOE_ERR_UNSUPPORTED_SHAPE;
  D->d = desc->d; D->d_ff = desc->d_ff; D->E = desc->E; D->G = desc->G; D->K = K;
  // with g1 clusters per token everything below the entry points works on g1 virtual tokens per token
  D->r = desc->r; D->k = desc->k; D->g1 = g1; D->T_user = desc->T_max; D->T_max = desc->T_max * g1;
  D->split = 0; D->rep = g1; D->seq = 0;
  // K r beyond the pair path's expanded rank index: every cluster as two halves, else four quarters, of its experts
  // where that makes the shape fit
  if (allow_split && g1 == 1 && D->T_max > 128 && !tc2_supported(*D)) {
    for (int parts = 2; parts <= 4 && D->split == 0 && D->seq == 0; parts *= 2) {
      if (K % parts || desc->k > K / parts || parts * desc->G > kMaxG || (long long)desc->T_max * parts > (1 << 22)) continue;
      Dims V = *D;
      V.K = K / parts; V.G = parts * desc->G; V.T_max = parts * desc->T_max;
      if (!tc2_supported(V)) continue;
      // Few tokens (at most kSeqTokens): the weight-streaming path, taken in pieces of 128 tokens, reads the weights
      // once per piece, where the parts run parts * G row tiles that are mostly padding.  Which is faster depends
      // on the layer's size; pieces_win() compares two fitted estimates.
      Dims W = *D;
      W.T_max = 128;
      if (desc->T_max <= kSeqTokens && stream_supported(W) && pieces_win(*desc, parts)) { D->seq = 128; D->T_max = 128; continue; }
      D->split = parts; D->rep = parts; D->K = V.K; D->G = V.G; D->T_max = V.T_max;
    }
  }
  const long long combos = binom_ll(D->K, desc->k);
  if (combos <= 64) { D->nsub = (int)combos; D->sub_is_combo = 1; }
  else              { D->nsub = D->K;        D->sub_is_combo = 0; }
  D->nkey = D->G * D->nsub;
  if (D->nkey > kMaxKeys) return CMOE_ERR_UNSUPPORTED_SHAPE;
  D->tc2 = (tc2_supported(*D) && D->T_max > 128) ? 1 : 0;
  D->stream = (!D->tc2 && stream_supported(*D)) ? 1 : 0;
  // CTA pairs work on 256-row tiles of one cluster; the streaming path on 16-row token blocks
  D->row_align = D->tc2 ? 256 : (D->stream ? 16 : 128);
  D->T_pad_max = t_pad_bound(*D, D->T_max);
  return CMOE_OK;
}

// Lays the arena out; with a null base it only measures.
void plan(const Dims& D, Arena& A, Weights* W, Scratch* S) {
  const size_t d = D.d, f = D.d_ff, E = D.E, G = D.G, r = D.r, k = D.k;
  const size_t T = D.T_max, P = D.T_pad_max;
  const size_t Gb = real_G(D);                       // bases and cluster prototypes: one per real cluster
  const size_t nblk = (T + kMinCountTile - 1) / kMinCountTile;
  Weights w{};
  Scratch s{};
  w.Ct = A.take<float>(G * d);
  w.Rt = A.take<float>(E * d);
  w.bc = A.take<float>(G);
  w.be = A.take<float>(E);
  w.label = A.take<int>(E);
  w.live = A.take<int>(E);
  w.B1t = A.take<__half>(Gb * d * f);
  w.B2t = A.take<__half>(Gb * d * f);
  w.U1q = A.take<uint8_t>(E * r * d / 2 + 16);
  w.V1q = A.take<uint8_t>(E * f * r / 2 + 16);
  w.U2q = A.take<uint8_t>(E * r * f / 2 + 16);
  w.V2q = A.take<uint8_t>(E * d * r / 2 + 16);
  w.U1s = A.take<__half>(E * r * d / 32 + 8);
  w.V1s = A.take<__half>(E * f * r / 32 + 8);
  w.U2s = A.take<__half>(E * r * f / 32 + 8);
  w.V2s = A.take<__half>(E * d * r / 32 + 8);
  const size_t Tr = D.seq > 0 ? (size_t)D.T_user : T;      // (cmoe_expert_stats routes a whole call at once)
  s.cluster_id = A.take<int>(Tr);
  s.slot = A.take<int>(Tr * k);
  s.gates = A.take<float>(Tr * k);
  s.keys = A.take<int>(T);
  s.block_counts = A.take<int>(nblk * D.nkey);
  s.block_base = A.take<int>(nblk * D.nkey);
  s.key_cnt = A.take<int>(D.nkey);
  s.key_off = A.take<int>(D.nkey);
  s.seg_off = A.take<int>(G + 1);
  s.seg_cnt = A.take<int>(G);
  s.n_rows = A.take<int>(1);
  s.tile_cluster = A.take<int>(P / D.row_align);
  s.row_token = A.take<int>(P);
  s.row_slot = A.take<int>(P * k);
  s.row_gate = A.take<float>(P * k);
  s.x_perm = A.take<__half>(P * d);
  if (D.rep > 1) {
    if (D.g1 > 1) s.x_rep = A.take<__half>(T * d);       // (expert parts read the token's own row)
    s.y_rep = A.take<__half>(T * d);
  }
  if (D.split > 1) {
    s.r_cluster = A.take<int>(D.T_user);
    s.r_slot = A.take<int>((size_t)D.T_user * k);
    s.r_gates = A.take<float>((size_t)D.T_user * k);
  }
  s.t = A.take<float>(P * k * r + 4);
  s.abar = A.take<__half>(P * f);
  s.s = A.take<float>(P * k * r + 4);
  s.status = A.take<int>(1);
  if (D.tc2 && r > 0) {
    s.U1f = A.take<__half>(G * 64 * d);
    s.V1f = A.take<__half>(G * f * 64);
    s.U2f = A.take<__half>(G * 64 * f);
    s.V2f = A.take<__half>(G * d * 64);
    s.A0 = A.take<__half>(P * 64);
    s.Ad = A.take<__half>(P * 64);
    s.As = A.take<__half>(P * 64);
    s.tile_mask = A.take<int>(P / 128 * 2);
    s.tile_mask_dn = A.take<int>(P / 128);
  }
  if (router_tc_supported(D)) s.Wsplit = A.take<__half>((size_t)2 * router_tc_rp(D) * d);
  if (D.stream) {
    if (r > 0) s.a_slot = A.take<__half>(P * k * f);
    s.y32 = A.take<float>(P * d);
  }
  if (W) *W = w;
  if (S) *S = s;
}

bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15) == 0; }

#define CMOE_CUDA(layer, expr)                                   \
  do {                                                           \
    cudaError_t _e = (expr);                                     \
    if (_e != cudaSuccess) {                                     \
      (layer)->last_cuda_error = (int)_e;                        \
      return CMOE_ERR_CUDA;                                      \
    }                                                            \
  } while (0)

int check_call(cmoe_layer* L, const void* x, int32_t T) {
  if (!L) return CMOE_ERR_INVALID_ARG;
  if (T < 0) return CMOE_ERR_INVALID_ARG;
  if (T > L->dims.T_user) return CMOE_ERR_T_EXCEEDS_MAX;
  if (T > 0 && (!x || !aligned16(x))) return CMOE_ERR_INVALID_ARG;
  return CMOE_OK;
}

}  // namespace

extern "C" {

int cmoe_workspace_bytes(const cmoe_desc* desc, size_t* out_bytes) { return cmoe_workspace_bytes_ex(desc, nullptr, out_bytes); }

int cmoe_workspace_bytes_ex(const cmoe_desc* desc, const cmoe_options* opt, size_t* out_bytes) {
  if (!out_bytes) return CMOE_ERR_INVALID_ARG;
  Dims D{};
  int rc = validate_dims(desc, opt ? opt->clusters_per_token : 1, !opt || (opt->force_path != kPathGeneric && opt->force_path != 3), &D);
  if (rc) return rc;
  Arena A;
  plan(D, A, nullptr, nullptr);
  *out_bytes = (A.used + 255) / 256 * 256;
  return CMOE_OK;
}

int cmoe_create(const cmoe_desc* desc, cmoe_layer** out_layer) { return cmoe_create_ex(desc, nullptr, out_layer); }

int cmoe_create_ex(const cmoe_desc* desc, const cmoe_options* opt, cmoe_layer** out_layer) {
  if (!out_layer) return CMOE_ERR_INVALID_ARG;
  *out_layer = nullptr;
  Dims D{};
  int rc = validate_dims(desc, opt ? opt->clusters_per_token : 1, !opt || (opt->force_path != kPathGeneric && opt->force_path != 3), &D);
  if (rc) return rc;
  if (!desc->C || !desc->R || !desc->B1 || !desc->B2 || !desc->workspace) return CMOE_ERR_INVALID_ARG;
  if (D.r > 0 && (!desc->U1q || !desc->V1q || !desc->U2q || !desc->V2q || !desc->U1s ||
                  !desc->V1s || !desc->U2s || !desc->V2s))
    return CMOE_ERR_INVALID_ARG;
  if ((reinterpret_cast<uintptr_t>(desc->workspace) & 255) != 0) return CMOE_ERR_INVALID_ARG;
  const void* ptrs[] = {desc->C, desc->R, desc->B1, desc->B2};
  for (const void* p : ptrs)
    if (!aligned16(p)) return CMOE_ERR_INVALID_ARG;
  size_t need = 0;
  cmoe_workspace_bytes_ex(desc, opt, &need);
  if (desc->workspace_bytes < need) return CMOE_ERR_WORKSPACE_TOO_SMALL;

  cmoe_options o{};
  o.force_path = -1;
  if (opt) o = *opt;
  if (o.force_path < -1 || (o.force_path > 0 && o.force_path != 3) || (o.up_tile != 0 && o.up_tile != 128 && o.up_tile != 256) ||
      o.base_dtype < 0 || o.base_dtype > 1 || o.host_chunks < 0 || o.host_chunks > kMaxHostChunks || o.row_gather < 0 || o.row_gather > 1 ||
      o.move_in_scatter < 0 || o.move_in_scatter > 1) return CMOE_ERR_INVALID_ARG;
  {
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || cudaDeviceGetAttribute(&D.sm_count, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess)
      return CMOE_ERR_CUDA;
  }
  cmoe_layer* L = new (std::nothrow) cmoe_layer();
  if (!L) return CMOE_ERR_INVALID_ARG;
  L->dims = D;
  L->opt = o;
  L->path = kPathGeneric;
  L->last_cuda_error = 0;
  L->profiling = 0;
  L->events_created = 0;
  L->events_recorded = 0;
  L->side_created = 0;
  L->host_created = 0;
  L->n_stages = 5;
  L->stage_names[0] = "router";
  L->stage_names[1] = "permute";
  L->stage_names[2] = "residual_t";
  L->stage_names[3] = "up";
  L->stage_names[4] = "down";
  Arena A;
  A.base = static_cast<char*>(desc->workspace);
  plan(D, A, &L->w, &L->sc);

  cudaStream_t st = 0;
  const Weights& W = L->w;
  const size_t d = D.d, f = D.d_ff, E = D.E, G = real_G(D), r = D.r;      // (router weights and bases: real clusters)
  auto fail = [&](cudaError_t) {
    cmoe_destroy(L);
    return CMOE_ERR_CUDA;
  };
  cudaError_t e;
  if ((e = cudaStreamCreateWithFlags(&L->side_stream, cudaStreamNonBlocking))) return fail(e);
  L->side_created = 1;
  if ((e = cudaEventCreateWithFlags(&L->side_fork, cudaEventDisableTiming))) return fail(e);
  L->side_created = 2;
  if ((e = cudaEventCreateWithFlags(&L->side_join, cudaEventDisableTiming))) return fail(e);
  L->side_created = 3;
  if ((e = cudaStreamCreateWithFlags(&L->h2d_stream, cudaStreamNonBlocking))) return fail(e);
  L->host_created = 1;
  if ((e = cudaStreamCreateWithFlags(&L->d2h_stream, cudaStreamNonBlocking))) return fail(e);
  L->host_created = 2;
  {
    cudaEvent_t* ev[2 + 2 * kMaxHostChunks];
    int n = 0;
    ev[n++] = &L->host_fork; ev[n++] = &L->host_join;
    for (int c = 0; c < kMaxHostChunks; ++c) ev[n++] = &L->chunk_in[c];
    for (int c = 0; c < kMaxHostChunks; ++c) ev[n++] = &L->chunk_done[c];
    for (int i = 0; i < n; ++i) {
      if ((e = cudaEventCreateWithFlags(ev[i], cudaEventDisableTiming))) return fail(e);
      L->host_created = 3 + i;
    }
  }
  // router: C [d][G] -> Ct [G][d];  R [G][d][K] -> Rt [G][K][d]
  if ((e = launch_transpose_f32(desc->C, const_cast<float*>(W.Ct), 1, D.d, real_G(D), st))) return fail(e);
  if ((e = launch_transpose_f32(desc->R, const_cast<float*>(W.Rt), real_G(D), D.d, real_K(D), st))) return fail(e);
  if (desc->b_c) e = cudaMemcpyAsync(const_cast<float*>(W.bc), desc->b_c, G * 4, cudaMemcpyDeviceToDevice, st);
  else           e = cudaMemsetAsync(const_cast<float*>(W.bc), 0, G * 4, st);
  if (e) return fail(e);
  if (desc->b_e) e = cudaMemcpyAsync(const_cast<float*>(W.be), desc->b_e, E * 4, cudaMemcpyDeviceToDevice, st);
  else           e = cudaMemsetAsync(const_cast<float*>(W.be), 0, E * 4, st);
  if (e) return fail(e);
  if (desc->expert_global_id) {
    e = cudaMemcpyAsync(const_cast<int*>(W.label), desc->expert_global_id, E * 4, cudaMemcpyDeviceToDevice, st);
  } else {
    int* ids = new (std::nothrow) int[E];
    if (!ids) { cmoe_destroy(L); return CMOE_ERR_INVALID_ARG; }
    for (size_t i = 0; i < E; ++i) ids[i] = (int)i;
    e = cudaMemcpy(const_cast<int*>(W.label), ids, E * 4, cudaMemcpyHostToDevice);
    delete[] ids;
  }
  if (e) return fail(e);
  // bases: B1 [G][d][d_ff] -> B1t [G][d_ff][d];  B2 [G][d_ff][d] -> B2t [G][d][d_ff]; the weight-streaming path
  // reads them stage by stage instead: [d / 128][G d_ff][128] and [d_ff / 128][G d][128]
  const bool streamed = D.stream && o.force_path != kPathGeneric;
  const __half* B1src = reinterpret_cast<const __half*>(desc->B1);
  const __half* B2src = reinterpret_cast<const __half*>(desc->B2);
  if (streamed) {
    if ((e = launch_stage_major_fp16(B1src, const_cast<__half*>(W.B1t), real_G(D), D.d, D.d_ff, st, o.base_dtype == 1))) return fail(e);
    if ((e = launch_stage_major_fp16(B2src, const_cast<__half*>(W.B2t), real_G(D), D.d_ff, D.d, st, o.base_dtype == 1))) return fail(e);
  } else {
    if ((e = launch_transpose_fp16(B1src, const_cast<__half*>(W.B1t), real_G(D), D.d, D.d_ff, st, o.base_dtype == 1))) return fail(e);
    if ((e = launch_transpose_fp16(B2src, const_cast<__half*>(W.B2t), real_G(D), D.d_ff, D.d, st, o.base_dtype == 1))) return fail(e);
  }
  if (r > 0) {
    struct { const void* src; const void* dst; size_t bytes; } cp[] = {
        {desc->U1q, W.U1q, E * r * d / 2}, {desc->V1q, W.V1q, E * f * r / 2},
        {desc->U2q, W.U2q, E * r * f / 2}, {desc->V2q, W.V2q, E * d * r / 2},
        {desc->U1s, W.U1s, E * r * d / 32 * 2}, {desc->V1s, W.V1s, E * f * r / 32 * 2},
        {desc->U2s, W.U2s, E * r * f / 32 * 2}, {desc->V2s, W.V2s, E * d * r / 32 * 2}};
    for (auto& c : cp)
      if ((e = cudaMemcpyAsync(const_cast<void*>(c.dst), c.src, c.bytes, cudaMemcpyDeviceToDevice, st))) return fail(e);
  }
  if ((e = launch_residual_live(D, W, st))) return fail(e);
  if ((e = cudaMemsetAsync(L->sc.status, 0, sizeof(int), st))) return fail(e);
  if ((e = cudaStreamSynchronize(st))) return fail(e);
  {
    int* live_h = new (std::nothrow) int[E];
    if (!live_h) { cmoe_destroy(L); return CMOE_ERR_INVALID_ARG; }
    e = cudaMemcpy(live_h, W.live, E * sizeof(int), cudaMemcpyDeviceToHost);
    L->pruned_blocks = 0;
    for (size_t i = 0; i < E && r > 0; ++i) L->pruned_blocks += ((live_h[i] & 1) ? 0 : 1) + ((live_h[i] & 2) ? 0 : 1);
    delete[] live_h;
    if (e) return fail(e);
  }
  // path choice: tensor-core grouped GEMMs when the shape allows and there are enough tokens to
  // fill 128-row tiles; cmoe_options.force_path = 0 keeps the generic path (for A/B checks)
  const int forced = o.force_path;
  L->tc_variant = 0;
  if (D.tc2 && forced != kPathGeneric) {
    if ((e = tc2_init(L))) return fail(e);
    L->path = kPathTensor;
    L->tc_variant = 2;
  } else if (D.stream && forced != kPathGeneric) {
    if ((e = stream_init(L))) return fail(e);
    L->path = kPathStream;
  } else if (tc_supported(D) && D.T_max > 128 && forced != kPathGeneric) {
    if ((e = tc_init(L))) return fail(e);
    L->path = kPathTensor;
    L->tc_variant = 1;
  }
  L->router_tc = 0;
  if (router_tc_supported(D) && !o.router_fp32) {
    if ((e = router_tc_init(L))) return fail(e);
    L->router_tc = 1;
  }
  *out_layer = L;
  return CMOE_OK;
}

int cmoe_route(cmoe_layer* L, const void* x, int32_t T, int32_t* cluster_id, int32_t* expert_ids,
               float* gates, void* cuda_stream) {
  int rc = check_call(L, x, T);
  if (rc) return rc;
  if (T == 0) return CMOE_OK;
  if (!cluster_id || !expert_ids || !gates) return CMOE_ERR_INVALID_ARG;
  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
  if (L->dims.g1 > 1) {
    // g1 virtual tokens per token: the outputs are [T][g1], [T][g1][k], [T][g1][k]
    CMOE_CUDA(L, launch_repeat_rows(L->dims, static_cast<const __half*>(x), L->sc.x_rep, T, L->dims.g1, st));
    x = L->sc.x_rep;
    T *= L->dims.g1;
  }
  // (a layer that works on expert halves still reports the token's own routes)
  if (L->router_tc && T >= 1024)
    CMOE_CUDA(L, launch_router_tc(L, static_cast<const __half*>(x), T, cluster_id, expert_ids, gates, nullptr, st));
  else
    CMOE_CUDA(L, launch_router(plain_dims(L->dims), L->w, static_cast<const __half*>(x), T, cluster_id, expert_ids,
                               gates, nullptr, st));
  return CMOE_OK;
}

static int forward_rows(cmoe_layer* L, const void* x, int32_t T, void* y, void* cuda_stream, const void* x_tokens);

int cmoe_forward(cmoe_layer* L, const void* x, int32_t T, void* y, void* cuda_stream) {
  int rc = check_call(L, x, T);
  if (rc) return rc;
  if (T == 0) return CMOE_OK;
  if (!y || !aligned16(y)) return CMOE_ERR_INVALID_ARG;
  const int n = L->dims.rep;
  if (L->dims.seq > 0 && T > L->dims.seq) {
    // consecutive pieces of at most seq tokens, one after the other on the caller's stream
    const size_t row = sizeof(__half) * (size_t)L->dims.d;
    for (int t0 = 0; t0 < T; t0 += L->dims.seq) {
      const int tc = T - t0 < L->dims.seq ? T - t0 : L->dims.seq;
      rc = forward_rows(L, static_cast<const char*>(x) + row * t0, tc, static_cast<char*>(y) + row * t0, cuda_stream, nullptr);
      if (rc) return rc;
    }
    return CMOE_OK;
  }
  if (n <= 1) return forward_rows(L, x, T, y, cuda_stream, nullptr);
  // virtual tokens (g1 clusters per token, or expert halves): every row n times, the layer on the virtual
  // tokens, the n outputs of a token summed
  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
  if (L->dims.split > 1) {
    // expert parts: the virtual tokens of a token share its row of x (the row move reads row t / n)
    rc = forward_rows(L, x, T * n, L->sc.y_rep, cuda_stream, x);
  } else {
    CMOE_CUDA(L, launch_repeat_rows(L->dims, static_cast<const __half*>(x), L->sc.x_rep, T, n, st));
    rc = forward_rows(L, L->sc.x_rep, T * n, L->sc.y_rep, cuda_stream, nullptr);
  }
  if (rc) return rc;
  // (expert parts: a part without any of the token's experts has no row)
  CMOE_CUDA(L, launch_sum_rows(L->dims, L->sc.y_rep, static_cast<__half*>(y), T, n,
                               L->dims.split > 1 ? L->sc.cluster_id : nullptr, st));
  return CMOE_OK;
}

// The layer on T rows of x as the kernels see them (virtual tokens when Dims::rep > 1).  x_tokens: not null for a
// layer on expert halves or quarters: the caller's T / split tokens, which are routed once over the real clusters; their routes are
// then split into those of the virtual tokens.
static int forward_rows(cmoe_layer* L, const void* x, int32_t T, void* y, void* cuda_stream, const void* x_tokens) {
  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
  const Dims& D = L->dims;
  const Scratch& S = L->sc;
  const __half* xh = static_cast<const __half*>(x);
  int stage = 0;
#define CMOE_MARK()                                                        \
  do {                                                                     \
    if (L->profiling) CMOE_CUDA(L, cudaEventRecord(L->events[stage], st)); \
    ++stage;                                                               \
  } while (0)
  CMOE_MARK();
  FactorStage fs{};                     // nothing to stage unless the pair path has residual factors
  if (L->path == kPathTensor && L->tc_variant == 2) tc2_factor_stage(L, &fs);
  // batches of at least 1024 tokens: the router counts the permutation keys of its token tiles as it goes
  KeyCount kc{};
  kc.keys = S.keys; kc.block_counts = S.block_counts; kc.nsub = D.nsub; kc.nkey = D.nkey; kc.sub_is_combo = D.sub_is_combo;
  int counted_tile = 0;
  if (x_tokens) {
    const __half* xt = static_cast<const __half*>(x_tokens);
    const int Tt = T / D.split;
    if (L->router_tc && Tt >= 1024) CMOE_CUDA(L, launch_router_tc(L, xt, Tt, S.r_cluster, nullptr, S.r_gates, S.r_slot, st));
    else CMOE_CUDA(L, launch_router(plain_dims(D), L->w, xt, Tt, S.r_cluster, nullptr, S.r_gates, S.r_slot, st, &fs));
    // (the splitting kernel writes the virtual tokens' permutation keys and counts them per block)
    CMOE_CUDA(L, launch_split_routes(D, S, Tt, st, &kc));
    counted_tile = split_routes_tile();
    if (Tt < 1024) fs = FactorStage{};  // staged beside the per-token router (else by the row-move kernel)
  } else {
    if (L->router_tc && T >= 1024) {
      CMOE_CUDA(L, launch_router_tc(L, xh, T, S.cluster_id, nullptr, S.gates, S.slot, st, &kc));
      counted_tile = router_tc_tile_tokens();
    } else {
      CMOE_CUDA(L, launch_router(D, L->w, xh, T, S.cluster_id, nullptr, S.gates, S.slot, st, &fs));
    }
    if (T < 1024) fs = FactorStage{};   // staged beside the per-token router (else by the row-move kernel)
  }
  CMOE_MARK();
  {
    // fp32 buffer that later kernels add into: the K ranges of y on the streaming path, else s
    const size_t rows = (size_t)t_pad_bound(D, T);
    void* zp = L->path == kPathStream ? static_cast<void*>(S.y32) : static_cast<void*>(S.s);
    size_t zb = L->path == kPathStream ? sizeof(float) * rows * D.d : sizeof(float) * rows * D.k * D.r;
    if (L->path == kPathTensor && L->tc_variant == 2) tc2_accum_buffer(L, T, &zp, &zb);
    LowrankTok lr{};                      // nothing rides along unless the streaming path has residual factors
    if (L->path == kPathStream) stream_lowrank_rider(L, xh, T, &lr);
    const bool gather = L->path == kPathTensor && L->tc_variant == 2 && tc2_gathers_rows(L);
    CMOE_CUDA(L, launch_permute(D, S, gather ? nullptr : xh, T, st, zp, zb, fs, lr, counted_tile, x_tokens ? D.split : 1, L->opt.move_in_scatter == 1));
  }
  if (L->path == kPathTensor && L->tc_variant == 2)
    CMOE_CUDA(L, launch_tc2_ffn(L, tc2_gathers_rows(L) ? xh : nullptr, T, static_cast<__half*>(y), st, L->profiling ? L->events + stage : nullptr));
  else if (L->path == kPathStream)
    CMOE_CUDA(L, launch_stream_ffn(L, T, static_cast<__half*>(y), st, L->profiling ? L->events + stage : nullptr));
  else if (L->path == kPathTensor)
    CMOE_CUDA(L, launch_tc_ffn(L, T, static_cast<__half*>(y), st, L->profiling ? L->events + stage : nullptr));
  else
    CMOE_CUDA(L, launch_generic_ffn(D, L->w, S, T, static_cast<__half*>(y), st,
                                    L->profiling ? L->events + stage : nullptr));
  stage += 3;
  CMOE_MARK();   // end of the last stage
#undef CMOE_MARK
  if (L->profiling) L->events_recorded = 1;
  return CMOE_OK;
}

int cmoe_forward_host(cmoe_layer* L, const void* x_host, int32_t T, void* y_host,
                      void* x_stage, void* y_stage, void* cuda_stream) {
  if (!L) return CMOE_ERR_INVALID_ARG;
  if (T < 0) return CMOE_ERR_INVALID_ARG;
  if (T > L->dims.T_user) return CMOE_ERR_T_EXCEEDS_MAX;
  if (T == 0) return CMOE_OK;
  if (!x_host || !y_host || !x_stage || !y_stage || !aligned16(x_stage) || !aligned16(y_stage)) return CMOE_ERR_INVALID_ARG;
  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
  const size_t row = sizeof(__half) * (size_t)L->dims.d;
  // chunks of at least 2048 tokens, multiples of 256, at most kMaxHostChunks of them
  int n_chunks = T / 2048;
  const int most = L->opt.host_chunks > 0 ? L->opt.host_chunks : kDefaultHostChunks;
  if (n_chunks < 1) n_chunks = 1;
  if (n_chunks > most) n_chunks = most;
  const int per = ((T + n_chunks - 1) / n_chunks + 255) / 256 * 256;
  // the copy streams start after what is already queued on the caller's stream (it may still use the buffers)
  CMOE_CUDA(L, cudaEventRecord(L->host_fork, st));
  CMOE_CUDA(L, cudaStreamWaitEvent(L->h2d_stream, L->host_fork, 0));
  CMOE_CUDA(L, cudaStreamWaitEvent(L->d2h_stream, L->host_fork, 0));
  int n = 0;
  for (int t0 = 0; t0 < T; t0 += per, ++n) {
    const int tc = T - t0 < per ? T - t0 : per;
    CMOE_CUDA(L, cudaMemcpyAsync(static_cast<char*>(x_stage) + row * t0, static_cast<const char*>(x_host) + row * t0,
                                 row * tc, cudaMemcpyHostToDevice, L->h2d_stream));
    CMOE_CUDA(L, cudaEventRecord(L->chunk_in[n], L->h2d_stream));
  }
  n = 0;
  for (int t0 = 0; t0 < T; t0 += per, ++n) {
    const int tc = T - t0 < per ? T - t0 : per;
    CMOE_CUDA(L, cudaStreamWaitEvent(st, L->chunk_in[n], 0));
    const int rc = cmoe_forward(L, static_cast<char*>(x_stage) + row * t0, tc, static_cast<char*>(y_stage) + row * t0, st);
    if (rc != CMOE_OK) return rc;
    CMOE_CUDA(L, cudaEventRecord(L->chunk_done[n], st));
    CMOE_CUDA(L, cudaStreamWaitEvent(L->d2h_stream, L->chunk_done[n], 0));
    CMOE_CUDA(L, cudaMemcpyAsync(static_cast<char*>(y_host) + row * t0, static_cast<char*>(y_stage) + row * t0,
                                 row * tc, cudaMemcpyDeviceToHost, L->d2h_stream));
  }
  // join: the caller's stream ends after the last copy back
  CMOE_CUDA(L, cudaEventRecord(L->host_join, L->d2h_stream));
  CMOE_CUDA(L, cudaStreamWaitEvent(st, L->host_join, 0));
  return CMOE_OK;
}

int cmoe_status(cmoe_layer* L, void* cuda_stream) {
  if (!L) return CMOE_ERR_INVALID_ARG;
  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
  int word = 0;
  CMOE_CUDA(L, cudaMemcpyAsync(&word, L->sc.status, sizeof(int), cudaMemcpyDeviceToHost, st));
  CMOE_CUDA(L, cudaStreamSynchronize(st));
  if (word != 0) {
    CMOE_CUDA(L, cudaMemsetAsync(L->sc.status, 0, sizeof(int), st));
    CMOE_CUDA(L, cudaStreamSynchronize(st));
    return CMOE_ERR_TIMEOUT;
  }
  return CMOE_OK;
}

int cmoe_get_info(const cmoe_layer* L, cmoe_info* out) {
  if (!L || !out) return CMOE_ERR_INVALID_ARG;
  *out = cmoe_info{};
  out->path = L->path;
  out->launches_route = 1;
  out->launches_forward = 1 + permute_launches(L->dims, L->dims.T_max, L->dims.split > 1 ? split_routes_tile() : (L->dims.T_max >= 1024 && L->router_tc) ? router_tc_tile_tokens() : 0,
                                              (L->path == kPathTensor && L->tc_variant == 2 && tc2_gathers_rows(L)) || L->opt.move_in_scatter != 1) +
                          (L->path == kPathTensor && L->tc_variant == 2
                               ? tc2_launch_count(L)
                               : L->path == kPathStream ? stream_launch_count(L->dims) : (L->dims.r > 0 ? kGenericFfnLaunches : kGenericFfnLaunches - 1)) + (L->dims.rep > 1 ? 2 : 0);
  if (L->dims.seq > 0) out->launches_forward *= (L->dims.T_user + L->dims.seq - 1) / L->dims.seq;    // (a call of T_max tokens)
  out->memsets_forward = 0;
  out->n_stages = L->n_stages;
  out->row_align = L->dims.row_align;
  out->T_pad_max = L->dims.T_pad_max;
  out->pruned_blocks = L->pruned_blocks;
  return CMOE_OK;
}

int cmoe_profile_enable(cmoe_layer* L, int on) {
  if (!L) return CMOE_ERR_INVALID_ARG;
  if (on && !L->events_created) {
    for (int i = 0; i <= CMOE_MAX_STAGES; ++i) CMOE_CUDA(L, cudaEventCreate(&L->events[i]));
    L->events_created = 1;
  }
  L->profiling = on ? 1 : 0;
  L->events_recorded = 0;
  return CMOE_OK;
}

int cmoe_profile_read(cmoe_layer* L, float* stage_ms, int32_t* n_stages) {
  if (!L || !stage_ms || !n_stages) return CMOE_ERR_INVALID_ARG;
  if (!L->events_created || !L->events_recorded) return CMOE_ERR_INVALID_ARG;
  CMOE_CUDA(L, cudaEventSynchronize(L->events[L->n_stages]));
  for (int i = 0; i < L->n_stages; ++i)
    CMOE_CUDA(L, cudaEventElapsedTime(&stage_ms[i], L->events[i], L->events[i + 1]));
  *n_stages = L->n_stages;
  return CMOE_OK;
}

const char* cmoe_stage_name(const cmoe_layer* L, int32_t stage) {
  if (!L || stage < 0 || stage >= L->n_stages) return nullptr;
  return L->stage_names[stage];
}

int cmoe_last_cuda_error(const cmoe_layer* L) { return L ? L->last_cuda_error : 0; }

int cmoe_destroy(cmoe_layer* L) {
  if (!L) return CMOE_ERR_INVALID_ARG;
  if (L->events_created)
    for (int i = 0; i <= CMOE_MAX_STAGES; ++i) cudaEventDestroy(L->events[i]);
  {
    cudaEvent_t ev[2 + 2 * kMaxHostChunks];
    int n = 0;
    ev[n++] = L->host_fork; ev[n++] = L->host_join;
    for (int c = 0; c < kMaxHostChunks; ++c) ev[n++] = L->chunk_in[c];
    for (int c = 0; c < kMaxHostChunks; ++c) ev[n++] = L->chunk_done[c];
    for (int i = 0; i < n; ++i)
      if (L->host_created >= 3 + i) cudaEventDestroy(ev[i]);
    if (L->host_created >= 2) { cudaStreamSynchronize(L->d2h_stream); cudaStreamDestroy(L->d2h_stream); }
    if (L->host_created >= 1) { cudaStreamSynchronize(L->h2d_stream); cudaStreamDestroy(L->h2d_stream); }
  }
  if (L->side_created >= 3) cudaEventDestroy(L->side_join);
  if (L->side_created >= 2) cudaEventDestroy(L->side_fork);
  if (L->side_created >= 1) { cudaStreamSynchronize(L->side_stream); cudaStreamDestroy(L->side_stream); }
  delete L;
  return CMOE_OK;
}

const char* cmoe_strerror(int code) {
  switch (code) {
    case CMOE_OK: return "ok";
    case CMOE_ERR_INVALID_ARG: return "invalid argument";
    case CMOE_ERR_UNSUPPORTED_SHAPE: return "descriptor outside the supported envelope";
    case CMOE_ERR_WORKSPACE_TOO_SMALL: return "workspace too small";
    case CMOE_ERR_T_EXCEEDS_MAX: return "T exceeds T_max";
    case CMOE_ERR_CUDA: return "CUDA call failed";
    case CMOE_ERR_TIMEOUT: return "bounded device wait expired";
    default: return "unknown error";
  }
}

}  // extern "C"
