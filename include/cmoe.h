/*
 * cmoe - forward pass of a clustered Mixture-of-Experts layer on one NVIDIA B200 (sm_100a).
 *
 * The layer (row-vector convention, y = x W):
 *   routing   two-stage hierarchical routing (Sec. 3.3): each token picks its top-1 cluster
 *             g* = argmax_g u_g.x (Eq. 9), then the top-k of the K = E/G experts inside that
 *             cluster by l_i = v_i.x with a softmax over them (Eq. 10); the gates are that softmax
 *             renormalised over the k kept experts.
 *   experts   every expert weight is a shared base plus a low-rank residual (Eq. 6, Eq. 7):
 *             W1_e = B1_g + U1_e V1_e (d x d_ff),  W2_e = B2_g + U2_e V2_e (d_ff x d), bases in FP16,
 *             factors in symmetric INT4 with one FP16 scale per 32 elements (Sec. 3.4).  The library
 *             never forms W_e: it uses  x W_e = x B_g + (x U_e) V_e  so that the base product is
 *             computed once per token and shared by the token's k experts (text after Eq. 7).
 *   combine   y = sum_{e in top-k} p_e GELU(x W1_e) W2_e, GELU(u) = u/2 (1 + erf(u / sqrt 2)).
 *
 * Arithmetic.  Activations, bases and outputs are fp16, all products accumulate in fp32.  The paths for
 * small batches (T_max <= 128) and the CUDA-core path evaluate GELU in the erf form in fp32.  The
 * tensor-core path for large batches rounds h to fp16 and evaluates u/2 (1 + tanh(u (0.80015708 +
 * 0.03470089 u^2))) in packed fp16 with the hardware tanh: the two coefficients are fitted to the erf
 * form (largest deviation 2.7e-4, at |u| near 1.7), of the size of the fp16 rounding of the stored
 * activation.  On every path max|y - y_exact| <= 1e-2 max|y_exact| + 1e-3 for the layer as defined above.
 *
 * Conventions
 *   - Every pointer below is a DEVICE pointer on the current CUDA device unless it says "host".
 *   - All arrays are dense, row-major, last index fastest.  fp16 values are IEEE binary16 bits.
 *   - Expert slot e = g*K + i is expert i of cluster g.
 *   - The library allocates no device memory: the caller passes a workspace arena.  The query
 *     cmoe_workspace_bytes() says how large it must be for a descriptor.
 *   - Every function returns CMOE_OK (0) or a negative cmoe_error; nothing throws or aborts.
 *     Argument errors are found on the host before anything is launched.
 *   - cmoe_route / cmoe_forward are asynchronous on the given stream, issue only kernel launches (no
 *     memsets, no copies), never synchronise, and touch only the arena and the given outputs.
 *     For handles with T_max <= 128 and r > 0, cmoe_forward forks two of its kernels onto a second
 *     stream that the handle owns and joins them back with two events (created with the handle): the
 *     work is complete when the given stream reaches the end of the call, as for any other call.
 *     They are not re-entrant on one handle (the arena holds the call's scratch, and the handle's second
 *     stream and events serve one call at a time): use one handle per concurrent caller.
 */
#ifndef CMOE_H
#define CMOE_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
  CMOE_OK = 0,
  CMOE_ERR_INVALID_ARG = -1,         /* NULL pointer, negative size, misaligned pointer              */
  CMOE_ERR_UNSUPPORTED_SHAPE = -2,   /* descriptor outside the supported envelope (see cmoe_desc)    */
  CMOE_ERR_WORKSPACE_TOO_SMALL = -3, /* workspace_bytes < cmoe_workspace_bytes(desc)                 */
  CMOE_ERR_T_EXCEEDS_MAX = -4,       /* T > desc.T_max                                               */
  CMOE_ERR_CUDA = -5,                /* a CUDA runtime/driver call failed; see cmoe_last_cuda_error  */
  CMOE_ERR_TIMEOUT = -6              /* a bounded device-side wait expired (reported by cmoe_status) */
} cmoe_error;

typedef struct cmoe_layer cmoe_layer; /* opaque, host object owned by the library */

/*
 * Layer descriptor (Sec. 3.2-3.4).  Supported envelope: E % G == 0, K = E/G <= 32, G <= 64,
 * 1 <= k <= min(K, 8), d % 32 == 0, d_ff % 32 == 0, r in {0, 4, 8, 16, 32}, quant_group == 32,
 * T_max >= 1.  With r == 0 the factor pointers are ignored (plain shared-base experts).
 * Speed, not results, depends on the shape: the fastest large-batch kernels need d and d_ff multiples of 128, k <= 2
 * and K*r <= 64 (or, for n = 2 or 4 with K a multiple of n, k <= K/n and n*G <= 64, (K/n)*r <= 64: the clusters are then
 * handled as n parts of K/n experts sharing the cluster's base; with T_max <= 384 and enough weights for it to pay
 * such a layer instead runs a call's tokens in consecutive pieces of 128 on the kernels for small batches, which read
 * the weights once per piece).
 * All weight pointers must be 16-byte aligned.
 */
typedef struct {
  int32_t d, d_ff, E, G, r, k;
  int32_t quant_group;          /* must be 32                                                      */
  int32_t T_max;                /* largest T any later call may pass                               */
  const float* C;               /* [d][G]       fp32  cluster prototypes; column g is u_g (Eq. 9)  */
  const float* R;               /* [G][d][K]    fp32  in-cluster router; columns are v_i (Eq. 10)  */
  const float* b_c;             /* [G] or NULL        optional bias added to the cluster logits    */
  const float* b_e;             /* [G][K] or NULL     optional bias added to the expert logits     */
  const uint16_t* B1;           /* [G][d][d_ff] fp16  shared base of the up-projection (Eq. 6)     */
  const uint16_t* B2;           /* [G][d_ff][d] fp16  shared base of the down-projection           */
  /* Residual factors (Eq. 7), packed INT4: two codes per byte, even flat index in the low nibble,
   * two's complement in [-8, 7]; the reduction index is the fastest one:
   *   U1q [E][r][d]   (U1_e is d x r)      V1q [E][d_ff][r] (V1_e is r x d_ff)
   *   U2q [E][r][d_ff](U2_e is d_ff x r)   V2q [E][d][r]    (V2_e is r x d)                        */
  const uint8_t *U1q, *V1q, *U2q, *V2q;
  /* one fp16 scale per 32 consecutive elements of the flattened factor (value = code * scale)     */
  const uint16_t *U1s, *V1s, *U2s, *V2s;
  const int32_t* expert_global_id; /* [E] or NULL (identity): label written to expert_ids          */
  void* workspace;              /* caller-owned device arena, 256-byte aligned                     */
  size_t workspace_bytes;
} cmoe_desc;

/* Pure host query: bytes of workspace cmoe_create needs for this descriptor (pointer fields are
 * not read).  Returns CMOE_ERR_UNSUPPORTED_SHAPE / CMOE_ERR_INVALID_ARG for a bad descriptor. */
int cmoe_workspace_bytes(const cmoe_desc* desc, size_t* out_bytes);

/* Validates the descriptor, copies and re-lays-out all weights into the arena (bases transposed to
 * reduction-index-fastest), and returns a handle.  Synchronous: it runs its kernels on the legacy
 * default stream and waits for them; work queued by the caller on other non-blocking streams that
 * produces the weights must have finished.  After it returns the source weight buffers may be
 * freed; the arena must outlive the handle and must not be written by the caller. */
int cmoe_create(const cmoe_desc* desc, cmoe_layer** out_layer);

/* cmoe_create with kernel-selection switches for A/B measurements and tests (NULL options = cmoe_create).
 * Results stay within the same tolerances whatever is chosen; only speed changes.
 *   force_path   -1 automatic (default); 0 keeps the generic CUDA-core path for every shape
 *                 3 automatic, but clusters are never handled as halves or quarters: shapes with K*r > 64 then
 *                 take the tensor-core path that evaluates the rank-r terms in its epilogue
 *   router_fp32   1 keeps batches of 1024 tokens and more on the fp32 CUDA-core router instead of the
 *                 tensor-core router (which splits the fp32 router matrices into two fp16 pieces; logit error
 *                 about 1e-6)
 *   up_tile       0 automatic; 128 keeps the up projection of large batches on 128-column tiles where d_ff
 *                 would allow 256-column tiles
 *   host_chunks   0 automatic; 1..8: the most chunks cmoe_forward_host cuts a batch into (chunks stay >= 2048 tokens)
 *   row_gather    0 (default): a copy kernel permutes the rows of x; 1: on the CTA-pair path with residual factors
 *                 the kernel that projects the tokens onto U1 reads them from x by TMA row gather (four rows of 128
 *                 bytes per instruction) and writes the permuted copy as it goes: one pass over x less, but slower
 *                 as measured (the gathers are issued at a fraction of the rate of tiled loads)
 *   move_in_scatter  0 (default): large batches are permuted by a kernel that places the tokens and a kernel that
 *                 moves their rows; 1: the placing blocks move the rows of their own token tile themselves (one
 *                 launch less; measured equal on one B200 of the pool and 3-7 us slower on another, so off)
 * and one switch that changes what the descriptor means:
 *   base_dtype    0: desc.B1 / desc.B2 hold fp16 bits (the paper's storage format, Sec. 3.4); 1: they hold bfloat16
 *                 bits.  The tensor cores take both operands of a product in one 16-bit type and the activations
 *                 are fp16, so bf16 bases are converted to fp16 while cmoe_create re-lays them out: exact for
 *                 magnitudes from 2^-14 to 65504 (fp16 has the wider significand), rounded to the fp16 subnormal
 *                 grid below, overflowing above.
 *   clusters_per_token  0 or 1: one cluster per token (Eq. 9's top-1, the paper's "typically g1 = 1"); 2: the paper's
 *                 "Top-g1 groups" with g1 = 2 (needs G >= 2).  The paper spells out the second stage for one
 *                 selected cluster only; the reading implemented: the two clusters with the largest p_g of Eq. 9
 *                 (largest z_g, lowest index first on ties) are kept, the second stage runs in each exactly as for
 *                 one cluster (top-k of its K logits, Eq. 10 renormalised over the kept experts), and the two
 *                 clusters' outputs are mixed with p_g renormalised over the kept clusters: expert i of kept cluster g
 *                 has gate p~_g p~_{i|g}, and a token's 2k gates sum to one.  cmoe_route then writes
 *                 cluster_id [T][2] (most probable first), expert_ids and gates [T][2][k].  Internally the layer runs
 *                 on two virtual tokens per token (2 T rows through router, permutation and expert FFNs, then one
 *                 sum per token), so a call costs about what one of 2 T tokens costs, and the workspace must be sized
 *                 with cmoe_workspace_bytes_ex.
 * Other values: CMOE_ERR_INVALID_ARG.  */
typedef struct {
  int32_t force_path;
  int32_t router_fp32;
  int32_t up_tile;
  int32_t base_dtype;
  int32_t host_chunks;
  int32_t row_gather;
  int32_t clusters_per_token;
  int32_t move_in_scatter;
} cmoe_options;
int cmoe_create_ex(const cmoe_desc* desc, const cmoe_options* options, cmoe_layer** out_layer);
/* cmoe_workspace_bytes for a handle that cmoe_create_ex will make with these options (NULL = cmoe_workspace_bytes):
 * clusters_per_token = 2 needs a larger arena. */
int cmoe_workspace_bytes_ex(const cmoe_desc* desc, const cmoe_options* options, size_t* out_bytes);

/* Two-stage routing only (Sec. 3.3, Eq. 9-10) for x = fp16 [T][d]:
 *   cluster_id [T]     chosen cluster g*
 *   expert_ids [T][k]  labels of the kept experts, by descending logit (lowest index first on ties)
 *   gates      [T][k]  fp32, softmax over the kept logits (sums to 1 per token)
 * 0 <= T <= T_max; T == 0 is a successful no-op.  x must be 16-byte aligned. */
int cmoe_route(cmoe_layer* layer, const void* x, int32_t T,
               int32_t* cluster_id, int32_t* expert_ids, float* gates, void* cuda_stream);

/* Whole layer: y = fp16 [T][d] in the original token order, for x = fp16 [T][d].  Routing uses the
 * same kernel as cmoe_route, so the two can never disagree.  x and y must be 16-byte aligned and
 * must not overlap.  The rank-r partial sums of the down-projection are accumulated with floating
 * point atomics, so y is reproducible only up to fp32 summation order. */
int cmoe_forward(cmoe_layer* layer, const void* x, int32_t T, void* y, void* cuda_stream);

/* The same for HOST buffers: y_host = fp16 [T][d] for x_host = fp16 [T][d] (both host pointers; page-locked
 * memory makes the copies asynchronous and lets them overlap, pageable memory works but serialises).
 * x_stage and y_stage are caller-owned DEVICE buffers of T*d fp16 values each (16-byte aligned) that the
 * call uses as staging.  Tokens are independent (Eq. 9-10 act per token), so the batch is cut into up to
 * four chunks of at least 2048 tokens and pipelined: chunk c+1 is copied to the device and chunk c-1 back
 * to the host on two streams owned by the handle while chunk c is computed on the caller's stream.  The
 * call is asynchronous: when the work queued on cuda_stream has finished, y_host is complete and x_host
 * may be reused.  0 <= T <= T_max. */
int cmoe_forward_host(cmoe_layer* layer, const void* x_host, int32_t T, void* y_host,
                      void* x_stage, void* y_stage, void* cuda_stream);

/* Waits for the stream and returns the device status word of the handle: CMOE_OK, or
 * CMOE_ERR_TIMEOUT if a bounded wait inside a kernel gave up (the output of that call is then
 * undefined; the handle stays usable and the word is cleared). */
int cmoe_status(cmoe_layer* layer, void* cuda_stream);

/* Test hook for the error path of the bounded device waits.  Every wait inside the kernels (on an mbarrier
 * fed by TMA, by the tensor cores or by another warp) gives up after a cycle limit, records
 * CMOE_ERR_TIMEOUT in the handle's status word and lets the kernel return normally.  This call launches a
 * one-block kernel that waits, with the same primitive and a limit of limit_cycles SM clocks (1 .. 2^31),
 * on a barrier nothing ever arrives on: it returns after about limit_cycles, nothing faults, and the next
 * cmoe_status reports CMOE_ERR_TIMEOUT once.  Asynchronous on the given stream. */
int cmoe_selftest_wait_timeout(cmoe_layer* layer, int64_t limit_cycles, void* cuda_stream);

/* By-products of routing that the training-side clustering consumes (Sec. 3.1, Eq. 5; Sec. 4.1's expert load
 * balance), for x = fp16 [T][d].  Routes x with the same kernels as cmoe_route and writes
 *   loads   [E]     int32  tokens routed to each expert slot (sum = k*T)
 *   xbar    [E][d]  fp32   mean of the tokens routed to the expert (Eq. 5's x-bar_i); rows of experts without
 *                          tokens are zero.  May be NULL.
 *   mu      [E][d]  fp32   in/out, or NULL: activation centroids, updated in place by Eq. 5,
 *                          mu_i <- (1 - beta) mu_i + beta xbar_i, unchanged for experts without tokens
 *   cov     [1]     fp32   coefficient of variation of the loads, population standard deviation / mean.  May be NULL.
 * All four are device pointers.  Uses the handle's scratch like cmoe_route / cmoe_forward (not re-entrant
 * with them); asynchronous on the given stream; 0 <= T <= T_max (T == 0: loads, xbar, cov are zeroed, mu
 * untouched). */
int cmoe_expert_stats(cmoe_layer* layer, const void* x, int32_t T, int32_t* loads, float* xbar,
                      float* mu, float beta, float* cov, void* cuda_stream);

/* Per-handle facts for tests and benchmarks (host struct, filled by cmoe_get_info). */
typedef struct {
  int32_t path;              /* 0 generic CUDA-core path, 1 tcgen05 grouped-GEMM path (T_max > 128),
                                2 weight-streaming path (T_max <= 128); chosen by cmoe_create             */
  int32_t launches_route;    /* kernel launches one cmoe_route call enqueues                       */
  int32_t launches_forward;  /* kernel launches one cmoe_forward call enqueues (memsets excluded)  */
  int32_t row_align;         /* permuted-row alignment of a cluster segment                        */
  int32_t T_pad_max;         /* rows of the permuted activations buffers                           */
  int32_t memsets_forward;   /* cudaMemsetAsync calls one cmoe_forward enqueues                    */
  int32_t n_stages;          /* stages cmoe_profile_read reports for this handle                   */
  int32_t pruned_blocks;     /* residual blocks (an expert's U V for one of its two matrices) that cmoe_create
                                found entirely zero - pruned by the cosine gate of Sec. 3.4; their work is skipped */
} cmoe_info;
int cmoe_get_info(const cmoe_layer* layer, cmoe_info* out);

/* Stage timing for benchmarks.  While enabled, cmoe_forward records a CUDA event on the stream
 * before each of its stages and after the last one (no synchronisation).  cmoe_profile_read waits
 * for the last recorded forward and writes the milliseconds of each stage of that call to
 * stage_ms[0..n_stages-1] (n_stages <= CMOE_MAX_STAGES); cmoe_stage_name names a stage, or returns
 * NULL past the last one.  Enabling creates the events; it allocates no device memory. */
#define CMOE_MAX_STAGES 8
int cmoe_profile_enable(cmoe_layer* layer, int on);
int cmoe_profile_read(cmoe_layer* layer, float* stage_ms, int32_t* n_stages);
const char* cmoe_stage_name(const cmoe_layer* layer, int32_t stage);

/* cudaError_t (as int) of the last failed CUDA call on this handle, 0 if none. */
int cmoe_last_cuda_error(const cmoe_layer* layer);

/* Routing for callers that cannot allocate device memory at all.  (The paper has no counterpart
 * of this call; it exists for integration reasons only.)
 *
 * cmoe_route needs a handle, and a handle needs an arena that somebody allocated.  Code that runs
 * where allocation is off the table - a plugin inside a host application whose GPU memory pool is
 * frozen after start-up, a dispatcher that must place tokens before any layer has been created -
 * can call this instead.  It takes the router exactly as cmoe_desc describes it (C [d][G],
 * R [G][d][K], optional b_c [G] and b_e [G][K], all device pointers) plus x = fp16 [T][d], and
 * writes the same three outputs as cmoe_route, with identity expert labels.  Its only scratch is a
 * fixed array of CMOE_ROUTE_STATIC_BYTES inside the library image, which every GPU that loads the
 * library holds until the process exits; it calls no cudaMalloc/cudaFree and no allocating library
 * routine.
 *
 *   - Limit: 4*(G+E)*d bytes of router plus a few KB must fit in the array; a larger router is
 *     rejected with CMOE_ERR_WORKSPACE_TOO_SMALL before anything is launched.  The shape rules of
 *     cmoe_desc for d, E, G, k apply (CMOE_ERR_UNSUPPORTED_SHAPE otherwise).
 *   - The first call on each device looks up the array's device address (that device must be
 *     current); make that first call outside any stream capture.
 *   - All calls on a device share the array.  Each call rewrites everything it reads, so calls in
 *     stream order are independent of each other, but two calls whose GPU work overlaps (issued
 *     on different streams without ordering) race and give undefined routes.
 *   - Asynchronous on the given stream like cmoe_route; T == 0 is a successful no-op. */
#define CMOE_ROUTE_STATIC_BYTES (2u << 20)
int cmoe_route_static(int32_t d, int32_t E, int32_t G, int32_t k,
                      const float* C, const float* R, const float* b_c, const float* b_e,
                      const void* x, int32_t T,
                      int32_t* cluster_id, int32_t* expert_ids, float* gates, void* cuda_stream);

/* Expert similarity that the clustering step consumes (Sec. 3.1, Eq. 2-4), for E experts:
 *   S_param [E][E] fp32  cosine similarity of the experts' flattened weight matrices (Eq. 2),
 *                        W = fp32 [E][n], n = number of weights per expert (n % 32 == 0, W 16-byte aligned)
 *   S_task  [E][E] fp32  cosine similarity of the activation centroids (Eq. 3), mu = fp32 [E][d]
 *                        (the mu that cmoe_expert_stats maintains)
 *   S       [E][E] fp32  alpha S_param + (1 - alpha) S_task (Eq. 4), 0 <= alpha <= 1
 * W == NULL skips S_param, mu == NULL skips S_task; S needs both (else it must be NULL).  A vector of norm zero has
 * similarity 0 to every other vector and 1 to itself.  The dot products of S_param run on the tensor cores with the
 * weights cut to tf32 (10 mantissa bits) and fp32 accumulation, partial sums of different ranges of the flattened
 * index combined with atomic additions: results agree with exact arithmetic to about 1e-4 and may differ in the
 * last bits between calls.  status: optional device word (caller zeroes it) that receives CMOE_ERR_TIMEOUT if a
 * bounded wait inside the kernel expires (the outputs are then undefined); may be NULL.
 * All pointers are device pointers; 1 <= E <= 128; needs no workspace (S_param doubles as the accumulation
 * buffer); asynchronous on the given stream. */
typedef struct {
  int32_t E;
  int32_t d;
  int64_t n;
  float alpha;
  const float* W;
  const float* mu;
  float* S_param;
  float* S_task;
  float* S;
  int32_t* status;
} cmoe_similarity_desc;
int cmoe_expert_similarity(const cmoe_similarity_desc* desc, void* cuda_stream);

/* Offline compressor (Sec. 3.2, Eq. 6-7; Sec. 3.4): from E dense expert matrices W_e (d_in x d_out, row-vector
 * convention; expert slot e = g*K + i belongs to cluster g) to the stored form of one of the layer's two matrices:
 *   B   [G][d_in][d_out]  fp16  W_base^g = mean of the cluster's experts (Eq. 6)
 *   Uq  [E][r][d_in], Vq [E][d_out][r]  packed INT4 + fp16 scales Us, Vs (one per 32 consecutive elements), with
 *       deq(U_e)^T deq(V_e)^T ~ W_e - W_base^g: the rank-r truncated SVD of the residual against the base as stored
 *       (Eq. 7; singular values split evenly over the two factors), quantised as Sec. 3.4 stores them
 * so that the outputs of two calls (W1: d_in = d, d_out = d_ff; W2: d_in = d_ff, d_out = d) are the B1, U1q, V1q ... /
 * B2, U2q, V2q ... fields of cmoe_desc.  The SVD is a randomised range finder with subspace iteration; its Gaussian
 * test matrices are the caller's input:
 *   omega [E][d_out][r + oversample] fp32 (standard normal draws), r + oversample <= 48
 * gamma > 0 switches the cosine gate of Sec. 3.4 on: a residual whose cosine similarity to its base,
 * <dW, B>_F / (|dW|_F |B|_F), is below gamma becomes a zero block (all codes and scales zero).
 * Optional outputs (NULL = not wanted): sigma [E][r] singular values, rel_err [E] = |dW - A B^T|_F / |dW|_F before
 * quantisation, cosine [E], pruned [E], and the fp32 factors A_out [E][d_in][r], Bt_out [E][r][d_out].
 * All pointers are device pointers; workspace (256-byte aligned) of cmoe_compress_workspace_bytes() bytes is the
 * caller's; asynchronous on the given stream.  Shapes: E % G == 0, K <= 32, d_in % 32 == d_out % 32 == 0,
 * r in {4, 8, 16, 32}, power_iters <= 8. */
typedef struct {
  int32_t d_in, d_out, E, G, r;
  int32_t oversample;
  int32_t power_iters;
  float gamma;
  const float* W;
  const float* omega;
  uint16_t* B;
  uint8_t* Uq;
  uint16_t* Us;
  uint8_t* Vq;
  uint16_t* Vs;
  float* sigma;
  float* rel_err;
  float* cosine;
  int32_t* pruned;
  float* A_out;
  float* Bt_out;
  void* workspace;
  size_t workspace_bytes;
} cmoe_compress_desc;
int cmoe_compress_workspace_bytes(const cmoe_compress_desc* desc, size_t* out_bytes);
int cmoe_compress(const cmoe_compress_desc* desc, void* cuda_stream);

/* The INT4 quantiser of the stored factors on its own (Sec. 3.4): w [n] fp32 in the stored order, n a multiple of 32
 * -> q [n / 2] packed codes (16-byte aligned), s [n / 32] fp16 scales; scale = fp16(absmax / 7), code =
 * clamp(round-half-even(w / scale), -8, 7), even index in the low nibble.  Device pointers; asynchronous. */
int cmoe_quantize_int4(const float* w, int64_t n, uint8_t* q, uint16_t* s, void* cuda_stream);

/* Frees the host object.  The arena is the caller's. */
int cmoe_destroy(cmoe_layer* layer);

const char* cmoe_strerror(int code);

#ifdef __cplusplus
}
#endif
#endif /* CMOE_H */
