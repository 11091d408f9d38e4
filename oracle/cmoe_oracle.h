/*
 * CPU oracle for the clustered-MoE layer forward.  TEST INFRASTRUCTURE ONLY.
 *
 * Plain, slow, single-purpose C: it is the layer exactly as the paper defines
 * it, written so that each line can be checked against the paper by eye.  It
 * shares no code with the CUDA library and must never be called from the
 * product path; only the tests, the smoke check and the benchmark's CPU
 * baseline leg load it.
 *
 * What it computes, per token x (row-vector convention, y = x W):
 *   stage 1 (Eq. 9):   z_g = sum_j x_j C[j][g] (+ b_c[g]);  g* = argmax_g z_g
 *                      (softmax is monotone, so the top-1 cluster is the argmax)
 *   stage 2 (Eq. 10):  l_i = sum_j x_j R[g*][j][i] (+ b_e[g*][i]), i in the K
 *                      experts of g*; keep the k largest; gate p_i = softmax
 *                      renormalised over the kept ones
 *   experts (Eq. 7):   W1_e = B1_g + deq(U1_e) deq(V1_e)   (d    x d_ff), formed explicitly
 *                      W2_e = B2_g + deq(U2_e) deq(V2_e)   (d_ff x d   ), formed explicitly
 *   combine:           y = sum_{e in top-k} p_e * GELU(x W1_e) W2_e,  GELU(u) = u/2 (1 + erf(u/sqrt 2))
 *
 * Arithmetic: values are fp32, every dot product is accumulated in double and
 * rounded once to fp32.
 *
 * Pins (tests/test_oracle_pins.py): r = 0 against a library dense FFN; G = E
 * against an independent top-1 MoE; brute-force route enumeration; the factored
 * identity x(B+UV) = xB + (xU)V in fp64; a residual-only layer; exhaustive INT4
 * codec; the parameter-count closed form (Eq. 8); equivariance invariants;
 * for the routing by-products (loads, x-bar, Eq. 5, load CoV): conservation
 * sums, a hand-counted example and numpy bincount / mean on the routes.
 * The paper prints no numeric layer output, so the absolute value of y on
 * random weights is otherwise "parity unpinned".
 */
#ifndef CMOE_ORACLE_H
#define CMOE_ORACLE_H
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct {
  int32_t d, d_ff, E, G, r, k;
  const float* C;       /* [d][G]                      */
  const float* R;       /* [G][d][K]                   */
  const float* b_c;     /* [G] or NULL                 */
  const float* b_e;     /* [G][K] or NULL              */
  const uint16_t* B1;   /* [G][d][d_ff] fp16 bits      */
  const uint16_t* B2;   /* [G][d_ff][d] fp16 bits      */
  const uint8_t *U1q, *V1q, *U2q, *V2q;   /* packed INT4: U1 [E][r][d], V1 [E][d_ff][r], U2 [E][r][d_ff], V2 [E][d][r] */
  const uint16_t *U1s, *V1s, *U2s, *V2s;  /* fp16 scale per 32 consecutive flat elements */
  int32_t base_is_bf16; /* 0: B1, B2 hold fp16 bits (the paper's storage format, Sec. 3.4); 1: bfloat16 bits (a variant) */
} cmoe_ref_desc;

/* fp16 bits -> fp32 value (exact). */
float cmoe_ref_half_to_float(uint16_t h);
/* bfloat16 bits -> fp32 value (exact). */
float cmoe_ref_bf16_to_float(uint16_t h);

/* Element `idx` of a packed INT4 factor: code * scale of its 32-group (exact in fp32). */
float cmoe_ref_dequant(const uint8_t* q, const uint16_t* s, int64_t idx);

/* Routing for T tokens.  cluster_id [T]; expert_slot [T][k] (slot = g*K + i,
 * by descending logit, lowest index first on ties); gates [T][k];
 * z [T][G] and l [T][K] (logits, fp32) may be NULL. Returns 0, or -1 on a bad descriptor. */
int cmoe_ref_route(const cmoe_ref_desc* D, const uint16_t* x, int32_t T,
                   int32_t* cluster_id, int32_t* expert_slot, float* gates,
                   float* z, float* l);

/* W1_e (which = 1, d x d_ff) or W2_e (which = 2, d_ff x d) of expert slot e, row-major fp32. */
int cmoe_ref_form_weight(const cmoe_ref_desc* D, int32_t e, int32_t which, float* W);

/* Layer output for the n_idx tokens listed in token_idx (NULL = tokens 0..n_idx-1);
 * y [n_idx][d] fp32. */
int cmoe_ref_forward(const cmoe_ref_desc* D, const uint16_t* x, int32_t T,
                     const int32_t* token_idx, int32_t n_idx, float* y);

/* Stored parameter elements of the compressed layer and of the E dense experts it replaces
 * (routers excluded): the ingredients of the compression ratio of Eq. 8. */
void cmoe_ref_param_count(const cmoe_ref_desc* D, int64_t* stored, int64_t* dense);

/* Routing by-products for the clustering of Sec. 3.1: tokens per expert slot, the mean routed token
 * x-bar_i, the EMA centroid update of Eq. 5 applied in place to mu (NULL = skip), and the coefficient of
 * variation of the loads (population standard deviation / mean; Sec. 4.1).  loads [E]; xbar, mu [E][d]. */
int cmoe_ref_expert_stats(const cmoe_ref_desc* D, const uint16_t* x, int32_t T,
                          int32_t* loads, float* xbar, float* mu, float beta, float* cov);

/* More than one cluster per token (Sec. 3.3, "Top-g1 groups"; the reading is stated above the functions in
 * cmoe_oracle.c): cluster_id [T][g1] by descending z, expert_slot and gates [T][g1][k]; a token's g1 k gates
 * sum to one.  g1 = 1 reproduces cmoe_ref_route / cmoe_ref_forward. */
int cmoe_ref_route_g1(const cmoe_ref_desc* D, const uint16_t* x, int32_t T, int32_t g1,
                      int32_t* cluster_id, int32_t* expert_slot, float* gates);
int cmoe_ref_forward_g1(const cmoe_ref_desc* D, const uint16_t* x, int32_t T, int32_t g1,
                        const int32_t* token_idx, int32_t n_idx, float* y);

int cmoe_ref_num_threads(void);

#ifdef __cplusplus
}
#endif
#endif
