/*
 * CPU oracle for the Dispatch->Combine MoE-FFN layer.  TEST INFRASTRUCTURE ONLY:
 * it exists so that tests, the smoke check and the bench's CPU-baseline leg have
 * something slow and obviously correct to compare against; the product path never
 * calls it.  It shares no code, table or helper with the CUDA library.
 *
 * The paper's method is a re-scheduling that keeps the layer's data dependencies
 * and mathematical semantics (Section 4.3, correctness paragraph), so the oracle is
 * the plain definition of the layer, written out from the paper's prose:
 *   routing   -- Section 2.2, first paragraph (router picks top-k experts, outputs
 *                are weighted by routing scores and combined);
 *   forward   -- Section 2.2, second paragraph (Dispatch, GMM gate+up, SwiGLU,
 *                GMM down, Combine accumulating the top-k contributions);
 *   backward  -- Section 2.2, third paragraph (backward Dispatch, act_grad, w2_grad,
 *                SwiGLU_grad, gate_grad, w1_grad, backward Combine).
 * All arithmetic is fp64, plain loops in definition order, no blocking, no fusion.
 * Every function below is pinned by tests/test_oracle_*.py (brute force, library
 * routines, closed-form special cases, finite differences, autograd).
 *
 * Readings where the paper is silent:
 *   - scores = softmax over all E logits; the k experts are the k largest raw
 *     logits, ties to the lower expert id, slots ordered by descending logit;
 *   - optional renormalisation of the k scores to sum 1;
 *   - S shared experts = experts E..E+S-1, taken by every token with weight 1;
 *   - rows inside an expert segment keep flat-slot order (stable);
 *   - weight gradients overwrite; an expert with no rows gets exact zeros.
 *
 * Layouts (all row-major): x[T][d], W_gate_up[E+S][2F][d] (rows 0..F-1 gate,
 * F..2F-1 up), W_down[E+S][d][F], ids[T][k], w[T][k].
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

#ifdef _OPENMP
#include <omp.h>
#endif

int moe_oracle_threads(void) {
#ifdef _OPENMP
  return omp_get_max_threads();
#else
  return 1;
#endif
}

/* ---- routing (Section 2.2, first paragraph: the router keeps the k best-scoring experts of each token) ---- */
int moe_oracle_route(const float* logits, int T, int E, int k, int renorm,
                     int32_t* topk_ids, double* topk_w) {
  if (k < 1 || k > E) return -1;
#pragma omp parallel for schedule(static)
  for (int t = 0; t < T; ++t) {
    const float* l = logits + (size_t)t * E;
    /* softmax over all E experts */
    double mx = l[0];
    for (int e = 1; e < E; ++e) if (l[e] > mx) mx = l[e];
    double den = 0.0;
    for (int e = 0; e < E; ++e) den += exp((double)l[e] - mx);
    /* k selections: each picks the largest not-yet-taken logit, lowest id on ties */
    double wsum = 0.0;
    for (int j = 0; j < k; ++j) {
      int best = -1;
      for (int e = 0; e < E; ++e) {
        int taken = 0;
        for (int jj = 0; jj < j; ++jj) if (topk_ids[(size_t)t * k + jj] == e) taken = 1;
        if (taken) continue;
        if (best < 0 || l[e] > l[best]) best = e;
      }
      topk_ids[(size_t)t * k + j] = best;
      double p = exp((double)l[best] - mx) / den;
      topk_w[(size_t)t * k + j] = p;
      wsum += p;
    }
    if (renorm)
      for (int j = 0; j < k; ++j) topk_w[(size_t)t * k + j] /= wsum;
  }
  return 0;
}

/* ---- router in the path (Section 2.2, first paragraph: the router scores every expert for each token
 * and keeps the top k).  The score function the paper leaves open is the usual linear router:
 * logits[t][e] = <x[t], W_r[e]>, W_r[E][d].  The routing decision itself is moe_oracle_route applied
 * to these logits rounded to fp32 (the precision in which the CUDA path decides). ---- */
int moe_oracle_router_logits(const double* x, const double* Wr, int T, int d, int E, double* logits) {
#pragma omp parallel for schedule(static)
  for (int t = 0; t < T; ++t)
    for (int e = 0; e < E; ++e) {
      double acc = 0.0;
      for (int c = 0; c < d; ++c) acc += x[(size_t)t * d + c] * Wr[(size_t)e * d + c];
      logits[(size_t)t * E + e] = acc;
    }
  return 0;
}

/* Gradient of the routing scores w.r.t. the logits, given g = dL/d topk_w (the selection is piecewise
 * constant and passes no gradient).  p = softmax(logits) over all E.
 *   without renormalisation  w_j = p[e_j]:
 *       dL/dl[e] = [e = e_j] g_j p[e]  -  p[e] * sum_j g_j p[e_j]
 *   with renormalisation     w_j = p[e_j] / sum_{i in S} p[e_i]  (a softmax over the selected set S only):
 *       dL/dl[e_j] = w_j (g_j - sum_i g_i w_i),  0 outside S. */
int moe_oracle_router_bwd(const float* logits, const int32_t* ids, const double* g, int T, int E, int k,
                          int renorm, double* dlogits) {
  if (k < 1 || k > E) return -1;
#pragma omp parallel for schedule(static)
  for (int t = 0; t < T; ++t) {
    const float* l = logits + (size_t)t * E;
    const int32_t* id = ids + (size_t)t * k;
    const double* gt = g + (size_t)t * k;
    double* dl = dlogits + (size_t)t * E;
    for (int e = 0; e < E; ++e) dl[e] = 0.0;
    double mx = l[0];
    for (int e = 1; e < E; ++e) if (l[e] > mx) mx = l[e];
    if (renorm) {
      double den = 0.0, dot = 0.0;
      for (int j = 0; j < k; ++j) den += exp((double)l[id[j]] - mx);
      for (int j = 0; j < k; ++j) dot += gt[j] * (exp((double)l[id[j]] - mx) / den);
      for (int j = 0; j < k; ++j) {
        double wj = exp((double)l[id[j]] - mx) / den;
        dl[id[j]] += wj * (gt[j] - dot);
      }
    } else {
      double den = 0.0, dot = 0.0;
      for (int e = 0; e < E; ++e) den += exp((double)l[e] - mx);
      for (int j = 0; j < k; ++j) dot += gt[j] * (exp((double)l[id[j]] - mx) / den);
      for (int e = 0; e < E; ++e) dl[e] = -(exp((double)l[e] - mx) / den) * dot;
      for (int j = 0; j < k; ++j) dl[id[j]] += gt[j] * (exp((double)l[id[j]] - mx) / den);
    }
  }
  return 0;
}

/* ---- sigmoid gating (a routing variant; the paper's router description, Section 2.2, fixes no score function):
 * score s_e = 1 / (1 + exp(-l_e)) per expert, independent of the other experts; the k experts are still the k
 * largest raw logits (the sigmoid is monotone), ties to the lower id, slots in descending order;
 * w_j = s_{e_j}, or s_{e_j} / sum_{i in S} s_{e_i} with renormalisation. ---- */
int moe_oracle_route_sigmoid(const float* logits, int T, int E, int k, int renorm, int32_t* topk_ids, double* topk_w) {
  if (k < 1 || k > E) return -1;
#pragma omp parallel for schedule(static)
  for (int t = 0; t < T; ++t) {
    const float* l = logits + (size_t)t * E;
    double wsum = 0.0;
    for (int j = 0; j < k; ++j) {
      int best = -1;
      for (int e = 0; e < E; ++e) {
        int taken = 0;
        for (int jj = 0; jj < j; ++jj) if (topk_ids[(size_t)t * k + jj] == e) taken = 1;
        if (taken) continue;
        if (best < 0 || l[e] > l[best]) best = e;
      }
      topk_ids[(size_t)t * k + j] = best;
      const double s = 1.0 / (1.0 + exp(-(double)l[best]));
      topk_w[(size_t)t * k + j] = s;
      wsum += s;
    }
    if (renorm)
      for (int j = 0; j < k; ++j) topk_w[(size_t)t * k + j] /= wsum;
  }
  return 0;
}

/* Gradient of the sigmoid-gated scores w.r.t. the logits, g = dL/d topk_w; s' = s (1 - s).
 *   without renormalisation  dL/dl[e_j] = g_j s_j (1 - s_j)
 *   with renormalisation     w_j = s_j / Z, Z = sum_i s_i:  dL/dl[e_i] = s_i (1 - s_i) / Z * (g_i - sum_j g_j w_j)
 * Experts outside the selection get 0 in both cases. */
int moe_oracle_router_bwd_sigmoid(const float* logits, const int32_t* ids, const double* g, int T, int E, int k,
                                  int renorm, double* dlogits) {
  if (k < 1 || k > E) return -1;
#pragma omp parallel for schedule(static)
  for (int t = 0; t < T; ++t) {
    const float* l = logits + (size_t)t * E;
    const int32_t* id = ids + (size_t)t * k;
    const double* gt = g + (size_t)t * k;
    double* dl = dlogits + (size_t)t * E;
    for (int e = 0; e < E; ++e) dl[e] = 0.0;
    double Z = 0.0, dot = 0.0;
    for (int j = 0; j < k; ++j) Z += 1.0 / (1.0 + exp(-(double)l[id[j]]));
    for (int j = 0; j < k; ++j) dot += gt[j] * (1.0 / (1.0 + exp(-(double)l[id[j]]))) / Z;
    for (int j = 0; j < k; ++j) {
      const double s = 1.0 / (1.0 + exp(-(double)l[id[j]]));
      dl[id[j]] += renorm ? s * (1.0 - s) / Z * (gt[j] - dot) : gt[j] * s * (1.0 - s);
    }
  }
  return 0;
}

/* expert id of flat slot i = t*(k+S)+j: routed slots first, then the S shared experts */
static inline int slot_expert(const int32_t* ids, int k, int S, int E, int t, int j) {
  return j < k ? ids[(size_t)t * k + j] : E + (j - k);
}

/* ---- dispatch layout (Section 2.2, Dispatch: the expert-ordered row of every routed token copy) ---- */
int moe_oracle_layout(const int32_t* ids, int T, int E, int k, int S,
                      int32_t* counts, int32_t* offsets, int32_t* row_of, int32_t* src_of) {
  const int Ep = E + S, kp = k + S;
  for (int e = 0; e < Ep; ++e) counts[e] = 0;
  for (int t = 0; t < T; ++t)
    for (int j = 0; j < kp; ++j) {
      int e = slot_expert(ids, k, S, E, t, j);
      if (e < 0 || e >= Ep) return -1;
      counts[e]++;
    }
  offsets[0] = 0;
  for (int e = 0; e < Ep; ++e) offsets[e + 1] = offsets[e] + counts[e];
  int32_t* next = (int32_t*)malloc(sizeof(int32_t) * (size_t)Ep);
  for (int e = 0; e < Ep; ++e) next[e] = offsets[e];
  for (int t = 0; t < T; ++t)
    for (int j = 0; j < kp; ++j) {
      int i = t * kp + j;
      int e = slot_expert(ids, k, S, E, t, j);
      row_of[i] = next[e]++;
      src_of[row_of[i]] = i;
    }
  free(next);
  return 0;
}

static inline double sigmoid(double v) { return 1.0 / (1.0 + exp(-v)); }

/* one row through one expert: h = x.W_gate_up[e]^T, a = silu(g)*u, y = a.W_down[e]^T */
static void expert_row_fwd(const double* x, const double* Wgu, const double* Wd, int d, int F,
                           double* h, double* a, double* y) {
  for (int n = 0; n < 2 * F; ++n) {
    const double* wr = Wgu + (size_t)n * d;
    double s = 0.0;
    for (int c = 0; c < d; ++c) s += x[c] * wr[c];
    h[n] = s;
  }
  for (int f = 0; f < F; ++f) {
    double g = h[f], u = h[F + f];
    a[f] = g * sigmoid(g) * u;
  }
  if (y)
    for (int c = 0; c < d; ++c) {
      const double* wr = Wd + (size_t)c * F;
      double s = 0.0;
      for (int f = 0; f < F; ++f) s += a[f] * wr[f];
      y[c] = s;
    }
}

/* ---- forward (Section 2.2: Dispatch, GMM, SwiGLU, GMM, Combine) ----
 * out[t] = sum_j w(t,j) * y(t,j), j in slot order.  Optional per-slot saves (may be NULL):
 * H[T*kp][2F], A[T*kp][F], Y[T*kp][d], indexed by flat slot. */
int moe_oracle_fwd(const double* x, const int32_t* ids, const double* w,
                   const double* Wgu, const double* Wd,
                   int T, int d, int E, int k, int S, int F,
                   double* out, double* H, double* A, double* Y) {
  const int kp = k + S, Ep = E + S;
  int bad = 0;
#pragma omp parallel
  {
    double* h = (double*)malloc(sizeof(double) * (size_t)(2 * F));
    double* a = (double*)malloc(sizeof(double) * (size_t)F);
    double* y = (double*)malloc(sizeof(double) * (size_t)d);
#pragma omp for schedule(dynamic, 4)
    for (int t = 0; t < T; ++t) {
      double* o = out + (size_t)t * d;
      for (int c = 0; c < d; ++c) o[c] = 0.0;
      for (int j = 0; j < kp; ++j) {
        int e = slot_expert(ids, k, S, E, t, j);
        if (e < 0 || e >= Ep) { bad = 1; continue; }
        double wt = j < k ? w[(size_t)t * k + j] : 1.0;
        expert_row_fwd(x + (size_t)t * d, Wgu + (size_t)e * 2 * F * d, Wd + (size_t)e * d * F, d, F, h, a, y);
        for (int c = 0; c < d; ++c) o[c] += wt * y[c];
        size_t i = (size_t)t * kp + j;
        if (H) memcpy(H + i * 2 * F, h, sizeof(double) * (size_t)(2 * F));
        if (A) memcpy(A + i * F, a, sizeof(double) * (size_t)F);
        if (Y) memcpy(Y + i * d, y, sizeof(double) * (size_t)d);
      }
    }
    free(h); free(a); free(y);
  }
  return bad ? -1 : 0;
}

/* ---- backward (Section 2.2, the seven backward nodes) ----
 * Given dout[T][d]:  d_w(t,j) = <dout_t, y(t,j)>           (second output of Combine's gradient)
 *   dy = w * dout_t                                        (backward Dispatch)
 *   da = dy . W_down[e]                                    (GMM act_grad)
 *   dW_down[e][c][f]   = sum_rows dy[c] * a[f]             (GMM w2_grad)
 *   dg = da*u*s*(1+g*(1-s)), du = da*g*s, s = sigmoid(g)   (SwiGLU_grad)
 *   dxrow = dh . W_gate_up[e]                              (GMM gate_grad)
 *   dW_gate_up[e][n][c] = sum_rows dh[n] * x_t[c]          (GMM w1_grad)
 *   dx[t] = sum_j dxrow(t,j)                               (backward Combine)
 * Row sums run in increasing flat-slot order.  d_w may be NULL. */
int moe_oracle_bwd(const double* dout, const double* x, const int32_t* ids, const double* w,
                   const double* Wgu, const double* Wd,
                   int T, int d, int E, int k, int S, int F,
                   double* dx, double* dWgu, double* dWd, double* d_w) {
  const int kp = k + S, Ep = E + S;
  const size_t R = (size_t)T * kp;
  double* a_all = (double*)malloc(sizeof(double) * R * F);
  double* dh_all = (double*)malloc(sizeof(double) * R * 2 * F);
  double* dxrow = (double*)malloc(sizeof(double) * R * d);
  if (!a_all || !dh_all || !dxrow) { free(a_all); free(dh_all); free(dxrow); return -2; }
  int bad = 0;
  /* per-slot quantities */
#pragma omp parallel
  {
    double* h = (double*)malloc(sizeof(double) * (size_t)(2 * F));
    double* y = (double*)malloc(sizeof(double) * (size_t)d);
    double* dy = (double*)malloc(sizeof(double) * (size_t)d);
    double* da = (double*)malloc(sizeof(double) * (size_t)F);
#pragma omp for schedule(dynamic, 4)
    for (long i = 0; i < (long)R; ++i) {
      int t = (int)(i / kp), j = (int)(i % kp);
      int e = slot_expert(ids, k, S, E, t, j);
      if (e < 0 || e >= Ep) { bad = 1; continue; }
      const double* We1 = Wgu + (size_t)e * 2 * F * d;
      const double* We2 = Wd + (size_t)e * d * F;
      const double* xt = x + (size_t)t * d;
      const double* go = dout + (size_t)t * d;
      double* a = a_all + (size_t)i * F;
      double* dh = dh_all + (size_t)i * 2 * F;
      double wt = j < k ? w[(size_t)t * k + j] : 1.0;
      expert_row_fwd(xt, We1, We2, d, F, h, a, y);
      if (d_w && j < k) {
        double s = 0.0;
        for (int c = 0; c < d; ++c) s += go[c] * y[c];
        d_w[(size_t)t * k + j] = s;
      }
      for (int c = 0; c < d; ++c) dy[c] = wt * go[c];
      for (int f = 0; f < F; ++f) {
        double s = 0.0;
        for (int c = 0; c < d; ++c) s += dy[c] * We2[(size_t)c * F + f];
        da[f] = s;
      }
      for (int f = 0; f < F; ++f) {
        double g = h[f], u = h[F + f], s = sigmoid(g);
        dh[f] = da[f] * u * s * (1.0 + g * (1.0 - s));
        dh[F + f] = da[f] * g * s;
      }
      double* dr = dxrow + (size_t)i * d;
      for (int c = 0; c < d; ++c) {
        double s = 0.0;
        for (int n = 0; n < 2 * F; ++n) s += dh[n] * We1[(size_t)n * d + c];
        dr[c] = s;
      }
    }
    free(h); free(y); free(dy); free(da);
  }
  /* backward Combine */
#pragma omp parallel for schedule(static)
  for (int t = 0; t < T; ++t)
    for (int c = 0; c < d; ++c) {
      double s = 0.0;
      for (int j = 0; j < kp; ++j) s += dxrow[((size_t)t * kp + j) * d + c];
      dx[(size_t)t * d + c] = s;
    }
  /* weight gradients: one expert per thread, rows in increasing slot order */
#pragma omp parallel for schedule(dynamic, 1)
  for (int e = 0; e < Ep; ++e) {
    double* g1 = dWgu + (size_t)e * 2 * F * d;
    double* g2 = dWd + (size_t)e * d * F;
    for (size_t q = 0; q < (size_t)2 * F * d; ++q) g1[q] = 0.0;
    for (size_t q = 0; q < (size_t)d * F; ++q) g2[q] = 0.0;
    for (long i = 0; i < (long)R; ++i) {
      int t = (int)(i / kp), j = (int)(i % kp);
      if (slot_expert(ids, k, S, E, t, j) != e) continue;
      const double* xt = x + (size_t)t * d;
      const double* go = dout + (size_t)t * d;
      const double* a = a_all + (size_t)i * F;
      const double* dh = dh_all + (size_t)i * 2 * F;
      double wt = j < k ? w[(size_t)t * k + j] : 1.0;
      for (int c = 0; c < d; ++c) {
        double dyc = wt * go[c];
        for (int f = 0; f < F; ++f) g2[(size_t)c * F + f] += dyc * a[f];
      }
      for (int n = 0; n < 2 * F; ++n)
        for (int c = 0; c < d; ++c) g1[(size_t)n * d + c] += dh[n] * xt[c];
    }
  }
  free(a_all); free(dh_all); free(dxrow);
  return bad ? -1 : 0;
}

/* ---- SwiGLU + Add operator pair (Section 6, microbenchmarks): the producer/consumer pair the paper
 * uses to study tile interleaving and scheduling cost.  x[M][2C] holds the gate half (columns 0..C-1)
 * and the up half (columns C..2C-1); s = silu(gate) * up; z = s + r.  fp64, no intermediate rounding. */
int moe_oracle_swiglu_add(const double* x, const double* r, int M, int C, double* s_out, double* z) {
  if (M < 0 || C < 1) return -1;
#pragma omp parallel for schedule(static)
  for (long m = 0; m < (long)M; ++m)
    for (int c = 0; c < C; ++c) {
      const double g = x[(size_t)m * 2 * C + c], u = x[(size_t)m * 2 * C + C + c];
      const double s = g / (1.0 + exp(-g)) * u;
      if (s_out) s_out[(size_t)m * C + c] = s;
      z[(size_t)m * C + c] = s + r[(size_t)m * C + c];
    }
  return 0;
}
