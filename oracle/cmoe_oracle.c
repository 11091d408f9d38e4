/*
 * CPU oracle for the clustered-MoE layer forward.  TEST INFRASTRUCTURE ONLY:
 * see cmoe_oracle.h for what it computes, its precision, and its pins.
 * Nothing here is blocked, fused or reordered beyond the definitions cited.
 */
#include "cmoe_oracle.h"

#include <math.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

/* IEEE binary16 -> binary32, exact: 1 sign, 5 exponent (bias 15), 10 mantissa bits. */
float cmoe_ref_half_to_float(uint16_t h) {
  uint32_t sign = (uint32_t)(h & 0x8000u) << 16;
  uint32_t expo = (h >> 10) & 0x1Fu;
  uint32_t mant = h & 0x3FFu;
  float v;
  if (expo == 0) {                      /* zero / subnormal: mant * 2^-24 */
    v = (float)mant * 5.9604644775390625e-8f;
    return sign ? -v : v;
  }
  uint32_t bits;
  if (expo == 31) bits = sign | 0x7F800000u | (mant << 13);          /* inf / nan */
  else            bits = sign | ((expo + 112u) << 23) | (mant << 13); /* rebias 15 -> 127 */
  memcpy(&v, &bits, sizeof v);
  return v;
}

/* bfloat16 -> binary32, exact: the 16 bits are the upper half of the binary32 pattern. */
float cmoe_ref_bf16_to_float(uint16_t h) {
  uint32_t bits = (uint32_t)h << 16;
  float v;
  memcpy(&v, &bits, sizeof v);
  return v;
}

/* INT4 storage format of the residual factors (Sec. 3.4 "Precision and Memory
 * Management"): two's-complement 4-bit code, even flat index in the low nibble,
 * times the fp16 scale shared by its group of 32 consecutive flat elements. */
float cmoe_ref_dequant(const uint8_t* q, const uint16_t* s, int64_t idx) {
  uint8_t byte = q[idx / 2];
  int code = (idx % 2 == 0) ? (byte & 0xF) : (byte >> 4);
  if (code >= 8) code -= 16;
  return (float)code * cmoe_ref_half_to_float(s[idx / 32]);
}

static int desc_ok(const cmoe_ref_desc* D) {
  if (!D || D->d <= 0 || D->d_ff <= 0 || D->E <= 0 || D->G <= 0 || D->r < 0) return 0;
  if (D->E % D->G) return 0;
  if (D->k < 1 || D->k > D->E / D->G) return 0;
  return 1;
}

int cmoe_ref_num_threads(void) {
#ifdef _OPENMP
  return omp_get_max_threads();
#else
  return 1;
#endif
}

/* Two-stage hierarchical routing (Sec. 3.3, Eq. 9 and Eq. 10). */
int cmoe_ref_route(const cmoe_ref_desc* D, const uint16_t* x, int32_t T,
                   int32_t* cluster_id, int32_t* expert_slot, float* gates,
                   float* z_out, float* l_out) {
  if (!desc_ok(D)) return -1;
  const int d = D->d, G = D->G, K = D->E / D->G, k = D->k;
#pragma omp parallel for schedule(static)
  for (int t = 0; t < T; ++t) {
    float* z = (float*)malloc(sizeof(float) * (size_t)G);
    float* l = (float*)malloc(sizeof(float) * (size_t)K);
    char* taken = (char*)calloc((size_t)K, 1);
    /* stage 1: z_g = u_g . x ; the softmax of Eq. 9 is monotone, top-1 = argmax */
    for (int g = 0; g < G; ++g) {
      double acc = 0.0;
      for (int j = 0; j < d; ++j)
        acc += (double)cmoe_ref_half_to_float(x[(size_t)t * d + j]) * (double)D->C[(size_t)j * G + g];
      if (D->b_c) acc += (double)D->b_c[g];
      z[g] = (float)acc;
    }
    int gs = 0;
    for (int g = 1; g < G; ++g) if (z[g] > z[gs]) gs = g;      /* lowest index wins ties */
    cluster_id[t] = gs;
    /* stage 2: l_i = v_i . x over the K experts of the chosen cluster */
    for (int i = 0; i < K; ++i) {
      double acc = 0.0;
      for (int j = 0; j < d; ++j)
        acc += (double)cmoe_ref_half_to_float(x[(size_t)t * d + j]) *
               (double)D->R[((size_t)gs * d + j) * K + i];
      if (D->b_e) acc += (double)D->b_e[(size_t)gs * K + i];
      l[i] = (float)acc;
    }
    /* top-k by repeated argmax: descending logit, lowest index first on ties */
    int sel[64];
    for (int s = 0; s < k; ++s) {
      int best = -1;
      for (int i = 0; i < K; ++i)
        if (!taken[i] && (best < 0 || l[i] > l[best])) best = i;
      taken[best] = 1;
      sel[s] = best;
      expert_slot[(size_t)t * k + s] = gs * K + best;
    }
    /* gates: softmax of Eq. 10 restricted to, and renormalised over, the kept experts */
    double lmax = (double)l[sel[0]], denom = 0.0;
    for (int s = 0; s < k; ++s) denom += exp((double)l[sel[s]] - lmax);
    for (int s = 0; s < k; ++s)
      gates[(size_t)t * k + s] = (float)(exp((double)l[sel[s]] - lmax) / denom);
    if (z_out) memcpy(z_out + (size_t)t * G, z, sizeof(float) * (size_t)G);
    if (l_out) memcpy(l_out + (size_t)t * K, l, sizeof(float) * (size_t)K);
    free(z); free(l); free(taken);
  }
  return 0;
}

/* Eq. 7: W_e = W_base^g + U_e V_e, formed explicitly.
 * which = 1: W1_e[j][f] = B1_g[j][f] + sum_p U1_e[j][p] V1_e[p][f],  U1 stored [E][r][d],    V1 stored [E][d_ff][r]
 * which = 2: W2_e[f][c] = B2_g[f][c] + sum_p U2_e[f][p] V2_e[p][c],  U2 stored [E][r][d_ff], V2 stored [E][d][r] */
int cmoe_ref_form_weight(const cmoe_ref_desc* D, int32_t e, int32_t which, float* W) {
  if (!desc_ok(D) || e < 0 || e >= D->E || (which != 1 && which != 2)) return -1;
  const int K = D->E / D->G, g = e / K, r = D->r;
  const int64_t din = (which == 1) ? D->d : D->d_ff;
  const int64_t dout = (which == 1) ? D->d_ff : D->d;
  const uint16_t* B = ((which == 1) ? D->B1 : D->B2) + (size_t)g * din * dout;
  const uint8_t* Uq = (which == 1) ? D->U1q : D->U2q;
  const uint16_t* Us = (which == 1) ? D->U1s : D->U2s;
  const uint8_t* Vq = (which == 1) ? D->V1q : D->V2q;
  const uint16_t* Vs = (which == 1) ? D->V1s : D->V2s;
  /* deq(U_e) as [din][r] and deq(V_e) as [r][dout] */
  float* Ud = (float*)malloc(sizeof(float) * (size_t)(din * r + 1));
  float* Vd = (float*)malloc(sizeof(float) * (size_t)(dout * r + 1));
  for (int64_t a = 0; a < din; ++a)
    for (int p = 0; p < r; ++p)       /* U_e[a][p] lives at flat index (e*r + p)*din + a */
      Ud[a * r + p] = cmoe_ref_dequant(Uq, Us, ((int64_t)e * r + p) * din + a);
  for (int p = 0; p < r; ++p)
    for (int64_t b = 0; b < dout; ++b) /* V_e[p][b] lives at flat index (e*dout + b)*r + p */
      Vd[p * dout + b] = cmoe_ref_dequant(Vq, Vs, ((int64_t)e * dout + b) * r + p);
#pragma omp parallel
  {
    double* acc = (double*)malloc(sizeof(double) * (size_t)dout);
#pragma omp for schedule(static)
    for (int64_t a = 0; a < din; ++a) {
      for (int64_t b = 0; b < dout; ++b)
        acc[b] = (double)(D->base_is_bf16 ? cmoe_ref_bf16_to_float(B[a * dout + b]) : cmoe_ref_half_to_float(B[a * dout + b]));
      for (int p = 0; p < r; ++p) {
        double u = (double)Ud[a * r + p];
        for (int64_t b = 0; b < dout; ++b) acc[b] += u * (double)Vd[p * dout + b];
      }
      for (int64_t b = 0; b < dout; ++b) W[a * dout + b] = (float)acc[b];
    }
    free(acc);
  }
  free(Ud); free(Vd);
  return 0;
}

static float gelu_erf(float u) {
  return (float)(0.5 * (double)u * (1.0 + erf((double)u / sqrt(2.0))));
}

/* y_t = sum_{e in top-k} p_e * GELU(x_t W1_e) W2_e  for the listed tokens. */
int cmoe_ref_forward(const cmoe_ref_desc* D, const uint16_t* x, int32_t T,
                     const int32_t* token_idx, int32_t n_idx, float* y) {
  if (!desc_ok(D)) return -1;
  const int d = D->d, d_ff = D->d_ff, k = D->k, E = D->E;
  if (n_idx <= 0) return 0;
  /* routes of the requested tokens */
  uint16_t* xs = (uint16_t*)malloc(sizeof(uint16_t) * (size_t)n_idx * d);
  for (int n = 0; n < n_idx; ++n) {
    int t = token_idx ? token_idx[n] : n;
    if (t < 0 || t >= T) { free(xs); return -1; }
    memcpy(xs + (size_t)n * d, x + (size_t)t * d, sizeof(uint16_t) * (size_t)d);
  }
  int32_t* cid = (int32_t*)malloc(sizeof(int32_t) * (size_t)n_idx);
  int32_t* slot = (int32_t*)malloc(sizeof(int32_t) * (size_t)n_idx * k);
  float* gate = (float*)malloc(sizeof(float) * (size_t)n_idx * k);
  cmoe_ref_route(D, xs, n_idx, cid, slot, gate, NULL, NULL);

  /* per (token, kept expert) output of that expert's FFN */
  float* f_out = (float*)calloc((size_t)n_idx * k * d, sizeof(float));
  float* W1 = (float*)malloc(sizeof(float) * (size_t)d * d_ff);
  float* W2 = (float*)malloc(sizeof(float) * (size_t)d_ff * d);
  for (int e = 0; e < E; ++e) {
    int used = 0;
    for (int64_t i = 0; i < (int64_t)n_idx * k; ++i) if (slot[i] == e) { used = 1; break; }
    if (!used) continue;                       /* experts without tokens are never formed */
    cmoe_ref_form_weight(D, e, 1, W1);
    cmoe_ref_form_weight(D, e, 2, W2);
#pragma omp parallel
    {
      double* acc = (double*)malloc(sizeof(double) * (size_t)(d_ff > d ? d_ff : d));
      float* a = (float*)malloc(sizeof(float) * (size_t)d_ff);
#pragma omp for schedule(dynamic, 1)
      for (int64_t i = 0; i < (int64_t)n_idx * k; ++i) {
        if (slot[i] != e) continue;
        const uint16_t* xt = xs + (size_t)(i / k) * d;
        /* h = x W1_e */
        for (int f = 0; f < d_ff; ++f) acc[f] = 0.0;
        for (int j = 0; j < d; ++j) {
          double xj = (double)cmoe_ref_half_to_float(xt[j]);
          const float* w = W1 + (size_t)j * d_ff;
          for (int f = 0; f < d_ff; ++f) acc[f] += xj * (double)w[f];
        }
        for (int f = 0; f < d_ff; ++f) a[f] = gelu_erf((float)acc[f]);
        /* out = a W2_e */
        for (int c = 0; c < d; ++c) acc[c] = 0.0;
        for (int f = 0; f < d_ff; ++f) {
          double af = (double)a[f];
          const float* w = W2 + (size_t)f * d;
          for (int c = 0; c < d; ++c) acc[c] += af * (double)w[c];
        }
        float* o = f_out + (size_t)i * d;
        for (int c = 0; c < d; ++c) o[c] = (float)acc[c];
      }
      free(acc); free(a);
    }
  }
  /* gated combine, in slot order */
  for (int n = 0; n < n_idx; ++n)
    for (int c = 0; c < d; ++c) {
      double acc = 0.0;
      for (int s = 0; s < k; ++s)
        acc += (double)gate[(size_t)n * k + s] * (double)f_out[((size_t)n * k + s) * d + c];
      y[(size_t)n * d + c] = (float)acc;
    }
  free(xs); free(cid); free(slot); free(gate); free(f_out); free(W1); free(W2);
  return 0;
}

/* Storage of the compressed layer vs the E dense experts it stands for (Eq. 8,
 * applied to both FFN matrices): per cluster one base of d*d_ff per matrix, per
 * expert r*(d + d_ff) factor elements per matrix. */
void cmoe_ref_param_count(const cmoe_ref_desc* D, int64_t* stored, int64_t* dense) {
  int64_t W = 2 * (int64_t)D->d * D->d_ff;
  *dense = (int64_t)D->E * W;
  *stored = (int64_t)D->G * W + (int64_t)D->E * 2 * D->r * ((int64_t)D->d + D->d_ff);
}

/* By-products of routing that the clustering of Sec. 3.1 consumes.
 *   loads[e]  = number of tokens whose kept experts include e              (sum = k T)
 *   xbar[e]   = (1/N) sum of the N tokens routed to e (text after Eq. 5); zero row when N = 0
 *   mu[e]    <- (1 - beta) mu[e] + beta xbar[e]   (Eq. 5), unchanged when no token arrived
 *   cov       = standard deviation of the loads / their mean (Sec. 4.1, expert load balance);
 *               the population form (divide by E) is this build's reading, the paper does not say which
 * Sums in double, one rounding to fp32.  xbar, mu and cov may be NULL. */
int cmoe_ref_expert_stats(const cmoe_ref_desc* D, const uint16_t* x, int32_t T,
                          int32_t* loads, float* xbar, float* mu, float beta, float* cov) {
  if (!desc_ok(D) || T < 0 || !loads) return -1;
  const int d = D->d, E = D->E, k = D->k;
  int32_t* cid = (int32_t*)malloc(sizeof(int32_t) * (size_t)(T + 1));
  int32_t* slot = (int32_t*)malloc(sizeof(int32_t) * ((size_t)T * k + 1));
  float* gates = (float*)malloc(sizeof(float) * ((size_t)T * k + 1));
  if (T > 0 && cmoe_ref_route(D, x, T, cid, slot, gates, NULL, NULL)) { free(cid); free(slot); free(gates); return -1; }
  for (int e = 0; e < E; ++e) loads[e] = 0;
  for (int t = 0; t < T; ++t)
    for (int s = 0; s < k; ++s) loads[slot[(size_t)t * k + s]] += 1;
  if (xbar || mu) {
    double* sum = (double*)malloc(sizeof(double) * (size_t)d);
    for (int e = 0; e < E; ++e) {
      for (int j = 0; j < d; ++j) sum[j] = 0.0;
      for (int t = 0; t < T; ++t)
        for (int s = 0; s < k; ++s)
          if (slot[(size_t)t * k + s] == e)
            for (int j = 0; j < d; ++j) sum[j] += (double)cmoe_ref_half_to_float(x[(size_t)t * d + j]);
      for (int j = 0; j < d; ++j) {
        const double mean = loads[e] > 0 ? sum[j] / (double)loads[e] : 0.0;
        if (xbar) xbar[(size_t)e * d + j] = (float)mean;
        if (mu && loads[e] > 0)
          mu[(size_t)e * d + j] = (float)((1.0 - (double)beta) * (double)mu[(size_t)e * d + j] + (double)beta * mean);
      }
    }
    free(sum);
  }
  if (cov) {
    double mean = 0.0, var = 0.0;
    for (int e = 0; e < E; ++e) mean += (double)loads[e];
    mean /= (double)E;
    for (int e = 0; e < E; ++e) var += ((double)loads[e] - mean) * ((double)loads[e] - mean);
    *cov = mean > 0.0 ? (float)(sqrt(var / (double)E) / mean) : 0.f;
  }
  free(cid); free(slot); free(gates);
  return 0;
}

/* ---------------------------------------------------------------------------------------------------------
 * More than one cluster per token (Sec. 3.3: "We select the Top-g1 groups (typically g1 = 1)").
 * The paper gives the second stage for one selected cluster only.  Reading taken here: the g1 clusters with the
 * largest p_g of Eq. 9 (= largest z_g; lowest index first on ties) are kept; inside each the second stage runs
 * exactly as for g1 = 1 (top-k of the cluster's K logits, Eq. 10 renormalised over the kept experts); the
 * clusters' outputs are mixed with p_g renormalised over the kept clusters, i.e. expert i of kept cluster g
 * weighs p~_g p~_{i|g}, and all g1 k weights of a token sum to one.  g1 = 1 gives cmoe_ref_route's result.
 * --------------------------------------------------------------------------------------------------------- */
int cmoe_ref_route_g1(const cmoe_ref_desc* D, const uint16_t* x, int32_t T, int32_t g1,
                      int32_t* cluster_id, int32_t* expert_slot, float* gates) {
  if (!desc_ok(D) || g1 < 1 || g1 > D->G || D->E / D->G > 64) return -1;
  const int d = D->d, G = D->G, K = D->E / D->G, k = D->k;
#pragma omp parallel for schedule(static)
  for (int t = 0; t < T; ++t) {
    float* z = (float*)malloc(sizeof(float) * (size_t)G);
    float* l = (float*)malloc(sizeof(float) * (size_t)K);
    char* gone = (char*)calloc((size_t)G, 1);
    int* gsel = (int*)malloc(sizeof(int) * (size_t)g1);
    for (int g = 0; g < G; ++g) {
      double acc = 0.0;
      for (int j = 0; j < d; ++j)
        acc += (double)cmoe_ref_half_to_float(x[(size_t)t * d + j]) * (double)D->C[(size_t)j * G + g];
      if (D->b_c) acc += (double)D->b_c[g];
      z[g] = (float)acc;
    }
    /* the g1 largest z_g by repeated argmax */
    for (int c = 0; c < g1; ++c) {
      int best = -1;
      for (int g = 0; g < G; ++g)
        if (!gone[g] && (best < 0 || z[g] > z[best])) best = g;
      gone[best] = 1;
      gsel[c] = best;
      cluster_id[(size_t)t * g1 + c] = best;
    }
    /* p_g of Eq. 9 renormalised over the kept clusters */
    double zden = 0.0;
    for (int c = 0; c < g1; ++c) zden += exp((double)z[gsel[c]] - (double)z[gsel[0]]);
    for (int c = 0; c < g1; ++c) {
      const int gs = gsel[c];
      const double pg = exp((double)z[gs] - (double)z[gsel[0]]) / zden;
      for (int i = 0; i < K; ++i) {
        double acc = 0.0;
        for (int j = 0; j < d; ++j)
          acc += (double)cmoe_ref_half_to_float(x[(size_t)t * d + j]) *
                 (double)D->R[((size_t)gs * d + j) * K + i];
        if (D->b_e) acc += (double)D->b_e[(size_t)gs * K + i];
        l[i] = (float)acc;
      }
      char taken[64];
      int sel[64];
      memset(taken, 0, sizeof(taken));
      for (int s = 0; s < k; ++s) {
        int best = -1;
        for (int i = 0; i < K; ++i)
          if (!taken[i] && (best < 0 || l[i] > l[best])) best = i;
        taken[best] = 1;
        sel[s] = best;
        expert_slot[((size_t)t * g1 + c) * k + s] = gs * K + best;
      }
      double lmax = (double)l[sel[0]], denom = 0.0;
      for (int s = 0; s < k; ++s) denom += exp((double)l[sel[s]] - lmax);
      for (int s = 0; s < k; ++s)
        gates[((size_t)t * g1 + c) * k + s] = (float)(pg * (exp((double)l[sel[s]] - lmax) / denom));
    }
    free(z); free(l); free(gone); free(gsel);
  }
  return 0;
}

/* Layer output with g1 clusters per token: y = sum over the g1 k routed experts of weight * FFN_e(x), the
 * expert FFNs formed and applied exactly as in cmoe_ref_forward. */
int cmoe_ref_forward_g1(const cmoe_ref_desc* D, const uint16_t* x, int32_t T, int32_t g1,
                        const int32_t* token_idx, int32_t n_idx, float* y) {
  if (!desc_ok(D) || g1 < 1 || g1 > D->G) return -1;
  const int d = D->d, d_ff = D->d_ff, kk = g1 * D->k, E = D->E;
  if (n_idx <= 0) return 0;
  uint16_t* xs = (uint16_t*)malloc(sizeof(uint16_t) * (size_t)n_idx * d);
  for (int n = 0; n < n_idx; ++n) {
    int t = token_idx ? token_idx[n] : n;
    if (t < 0 || t >= T) { free(xs); return -1; }
    memcpy(xs + (size_t)n * d, x + (size_t)t * d, sizeof(uint16_t) * (size_t)d);
  }
  int32_t* cid = (int32_t*)malloc(sizeof(int32_t) * (size_t)n_idx * g1);
  int32_t* slot = (int32_t*)malloc(sizeof(int32_t) * (size_t)n_idx * kk);
  float* gate = (float*)malloc(sizeof(float) * (size_t)n_idx * kk);
  if (cmoe_ref_route_g1(D, xs, n_idx, g1, cid, slot, gate)) { free(xs); free(cid); free(slot); free(gate); return -1; }

  float* W1 = (float*)malloc(sizeof(float) * (size_t)d * d_ff);
  float* W2 = (float*)malloc(sizeof(float) * (size_t)d_ff * d);
  double* ysum = (double*)calloc((size_t)n_idx * d, sizeof(double));
  for (int e = 0; e < E; ++e) {
    int used = 0;
    for (int64_t i = 0; i < (int64_t)n_idx * kk; ++i) if (slot[i] == e) { used = 1; break; }
    if (!used) continue;
    cmoe_ref_form_weight(D, e, 1, W1);
    cmoe_ref_form_weight(D, e, 2, W2);
#pragma omp parallel
    {
      double* acc = (double*)malloc(sizeof(double) * (size_t)(d_ff > d ? d_ff : d));
      float* a = (float*)malloc(sizeof(float) * (size_t)d_ff);
#pragma omp for schedule(dynamic, 1)
      for (int n = 0; n < n_idx; ++n) {
        for (int s = 0; s < kk; ++s) {
          if (slot[(size_t)n * kk + s] != e) continue;
          const uint16_t* xt = xs + (size_t)n * d;
          for (int f = 0; f < d_ff; ++f) acc[f] = 0.0;
          for (int j = 0; j < d; ++j) {
            double xj = (double)cmoe_ref_half_to_float(xt[j]);
            const float* w = W1 + (size_t)j * d_ff;
            for (int f = 0; f < d_ff; ++f) acc[f] += xj * (double)w[f];
          }
          for (int f = 0; f < d_ff; ++f) a[f] = gelu_erf((float)acc[f]);
          for (int c = 0; c < d; ++c) acc[c] = 0.0;
          for (int f = 0; f < d_ff; ++f) {
            double af = (double)a[f];
            const float* w = W2 + (size_t)f * d;
            for (int c = 0; c < d; ++c) acc[c] += af * (double)w[c];
          }
          /* an expert's output is an fp32 value, as in cmoe_ref_forward; the weighted sum runs in double */
          for (int c = 0; c < d; ++c)
            ysum[(size_t)n * d + c] += (double)gate[(size_t)n * kk + s] * (double)(float)acc[c];
        }
      }
      free(acc); free(a);
    }
  }
  for (int64_t i = 0; i < (int64_t)n_idx * d; ++i) y[i] = (float)ysum[i];
  free(xs); free(cid); free(slot); free(gate); free(W1); free(W2); free(ysum);
  return 0;
}
