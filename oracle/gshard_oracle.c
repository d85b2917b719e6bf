/*
 * CPU oracle for the GShard top-2 gated Mixture-of-Experts FFN layer.
 *
 * TEST INFRASTRUCTURE ONLY.  This file is the slow, plain statement of what the
 * layer computes; the tests, the smoke check and the benchmark's CPU-baseline leg
 * are its only callers.  It shares no code with the CUDA library and the CUDA
 * library never calls it.
 *
 * Every function follows one passage of the GShard paper (arxiv 2006.16668):
 *   - Algorithm 1  (group-level top-2 gating with auxiliary loss)
 *   - Eq. (1)-(3)  (the MoE layer: y_s = sum_e G_{s,e} * FFN_e(x_s),
 *                   FFN_e(x) = wo_e . ReLU(wi_e . x), no bias)
 *   - Algorithm 2  (tensor layouts: inputs [G,S,M], wg [M,E], wi [E,M,H],
 *                   wo [E,H,M], dispatched inputs [E,G,C,M])
 * Floating point: inputs arrive as float (bf16 inputs are widened exactly by
 * the caller) and every sum is accumulated in double.  There is no blocking,
 * fusion or reordering beyond what the paper's steps state.
 *
 * Readings where the paper is silent:
 *   - top_2 ties: the lowest expert index wins, for both picks.
 *   - the pass-2 counters continue from the (unclipped) pass-1 counts;
 *     Algorithm 1 initialises c_E once.
 *   - "default" reading of the second loop: the counter of e2 advances for
 *     every token, as the listing has it (the increment is outside the `if`).
 *     variant_a != 0 selects the other reading: only tokens that pass the
 *     random-routing test advance the counter.
 *   - the weight of a kept choice stays g/(g1+g2) when the other is dropped.
 *   - layer l_aux = mean over groups of the group value.
 *   - backward: the paper gives none; it is the derivative of
 *     L = <dy, y> + k * l_aux with the routing (e1, e2, slots, kept flags and
 *     the counts c_e) held constant.  c_e is stated to be non-differentiable
 *     in the paragraph that motivates the auxiliary loss.
 *
 * Pins: tests/test_oracle_*.py (hand-worked example with exact fractions,
 * brute-force rank formulas, invariants, closed forms, a dense einsum
 * restatement of Algorithm 2 with autograd, finite differences).
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

int gso_num_threads(void) {
#ifdef _OPENMP
  return omp_get_max_threads();
#else
  return 1;
#endif
}

/* ------------------------------------------------------------------------- */
/* Algorithm 1, "g_{S,E} <- softmax(wg . x_S)" for ONE group.                  */
/* x [S,M], wg [M,E] -> logits [S,E] (optional), p [S,E]                        */
void gso_gates(const float* x, const float* wg, int S, int M, int E,
               double* logits_out, double* p) {
#pragma omp parallel for schedule(static)
  for (int s = 0; s < S; ++s) {
    double* row = p + (size_t)s * E;
    for (int e = 0; e < E; ++e) row[e] = 0.0;
    for (int m = 0; m < M; ++m) {
      const double xv = (double)x[(size_t)s * M + m];
      const float* wrow = wg + (size_t)m * E;
      for (int e = 0; e < E; ++e) row[e] += xv * (double)wrow[e];
    }
    if (logits_out) memcpy(logits_out + (size_t)s * E, row, sizeof(double) * E);
    double mx = row[0];
    for (int e = 1; e < E; ++e) if (row[e] > mx) mx = row[e];
    double z = 0.0;
    for (int e = 0; e < E; ++e) { row[e] = exp(row[e] - mx); z += row[e]; }
    for (int e = 0; e < E; ++e) row[e] /= z;
  }
}

/* Algorithm 1, "m_E <- (1/S) sum_s g_{s,E}" for one group. */
void gso_mean_gates(const double* p, int S, int E, double* m) {
  for (int e = 0; e < E; ++e) {
    double acc = 0.0;
    for (int s = 0; s < S; ++s) acc += p[(size_t)s * E + e];
    m[e] = acc / (double)S;
  }
}

/* Algorithm 1, "g1, e1, g2, e2 = top_2(g_{s,E})" for every token of a group.
 * Lowest index wins ties.  g3 (third largest gate, -1 when E == 2) is returned
 * so that callers can compute the near-tie margin min(g1-g2, g2-g3). */
void gso_top2(const double* p, int S, int E, int32_t* e1, int32_t* e2,
              double* g1, double* g2, double* g3) {
  for (int s = 0; s < S; ++s) {
    const double* row = p + (size_t)s * E;
    int a = 0;
    for (int e = 1; e < E; ++e) if (row[e] > row[a]) a = e;
    int b = -1;
    for (int e = 0; e < E; ++e) {
      if (e == a) continue;
      if (b < 0 || row[e] > row[b]) b = e;
    }
    int c = -1;
    for (int e = 0; e < E; ++e) {
      if (e == a || e == b) continue;
      if (c < 0 || row[e] > row[c]) c = e;
    }
    e1[s] = a; e2[s] = b; g1[s] = row[a]; g2[s] = row[b];
    if (g3) g3[s] = (c >= 0) ? row[c] : -1.0;
  }
}

/* Algorithm 1, the two token loops and the auxiliary loss, for ONE group.
 *
 * in : e1,e2 [S]; g1,g2 [S] raw (un-normalised) top-2 gates; u [S] uniform noise;
 *      m [E] mean gates; pass_override [S] or NULL (-1: decide by 2*w2 > u,
 *      0 / 1: forced outcome of the random-routing test -- used only by the
 *      near-tie replay in the parity tests).
 * out: slot [S,2] buffer position or -1; weight [S,2] normalised g1, g2 (always
 *      the normalised values, kept or not); flags [S] bit0 first kept, bit1
 *      random test passed, bit2 second kept; first_count [E] = c_E after the
 *      first loop (unclipped); total_count [E] = c_E after the second loop;
 *      returns the group's l_aux = (1/E) sum_e (c_e/S) m_e with c_e taken
 *      after the first loop.
 */
double gso_capacity(int S, int E, int C, const int32_t* e1, const int32_t* e2,
                    const double* g1, const double* g2, const float* u,
                    const double* m, const int8_t* pass_override, int variant_a,
                    int32_t* slot, double* weight, uint8_t* flags,
                    int32_t* first_count, int32_t* total_count) {
  int32_t* c = (int32_t*)calloc((size_t)E, sizeof(int32_t));   /* c_E <- 0 */
  /* first loop: first choices */
  for (int s = 0; s < S; ++s) {
    const double w1 = g1[s] / (g1[s] + g2[s]);
    const int32_t pos = c[e1[s]];
    weight[2 * s + 0] = w1;
    flags[s] = 0;
    if (pos < C) { slot[2 * s + 0] = pos; flags[s] |= 1u; }
    else         { slot[2 * s + 0] = -1; }
    c[e1[s]] = pos + 1;
  }
  memcpy(first_count, c, sizeof(int32_t) * (size_t)E);
  /* l_aux, before the second choices are dispatched */
  double l_aux = 0.0;
  for (int e = 0; e < E; ++e) l_aux += ((double)c[e] / (double)S) * m[e];
  l_aux /= (double)E;
  /* second loop: second choices with random routing */
  for (int s = 0; s < S; ++s) {
    const double w2 = g2[s] / (g1[s] + g2[s]);
    int pass;
    if (pass_override && pass_override[s] >= 0) pass = pass_override[s];
    else pass = (2.0 * w2 > (double)u[s]) ? 1 : 0;
    const int32_t pos = c[e2[s]];
    weight[2 * s + 1] = w2;
    if (pass) flags[s] |= 2u;
    if (pos < C && pass) { slot[2 * s + 1] = pos; flags[s] |= 4u; }
    else                 { slot[2 * s + 1] = -1; }
    if (!variant_a || pass) c[e2[s]] = pos + 1;
  }
  memcpy(total_count, c, sizeof(int32_t) * (size_t)E);
  free(c);
  return l_aux;
}

/* Eq. (2): FFN_e(x) = wo_e . ReLU(wi_e . x) for `rows` input rows.
 * xrows [rows,M], wi_e [M,H], wo_e [H,M] -> out [rows,M]; optional h [rows,H]
 * receives the pre-activation wi_e . x. */
void gso_ffn_rows(const float* xrows, int rows, const float* wi_e, const float* wo_e,
                  int M, int H, double* out, double* h_pre) {
#pragma omp parallel for schedule(dynamic, 1)
  for (int r = 0; r < rows; ++r) {
    double* h = (double*)malloc(sizeof(double) * (size_t)H);
    for (int j = 0; j < H; ++j) h[j] = 0.0;
    for (int m = 0; m < M; ++m) {
      const double xv = (double)xrows[(size_t)r * M + m];
      const float* w = wi_e + (size_t)m * H;
      for (int j = 0; j < H; ++j) h[j] += xv * (double)w[j];
    }
    if (h_pre) memcpy(h_pre + (size_t)r * H, h, sizeof(double) * (size_t)H);
    double* o = out + (size_t)r * M;
    for (int i = 0; i < M; ++i) o[i] = 0.0;
    for (int j = 0; j < H; ++j) {
      const double a = h[j] > 0.0 ? h[j] : 0.0;
      if (a == 0.0) continue;
      const float* w = wo_e + (size_t)j * M;
      for (int i = 0; i < M; ++i) o[i] += a * (double)w[i];
    }
    free(h);
  }
}

/* The whole layer forward: Algorithm 1 per group, then eq. (3)
 * y_s = sum over kept choices of weight * FFN_e(x_s).
 * Routing outputs use the layouts of Algorithm 2:
 *   expert_idx [G,S,2], slot [G,S,2], weight [G,S,2] (double), flags [G,S],
 *   first_count/total_count [G,E], slot_token [E,G,C] (token index s or -1,
 *   the paper's s_indices), m [G,E], l_aux_group [G].
 * Returns the layer l_aux = mean over groups.  y may be NULL (routing only). */
double gso_forward(int G, int S, int M, int H, int E, int C, const float* x,
                   const float* wg, const float* wi, const float* wo, const float* u,
                   int variant_a, double* y, int32_t* expert_idx, int32_t* slot,
                   double* weight, uint8_t* flags, int32_t* first_count,
                   int32_t* total_count, int32_t* slot_token, double* m,
                   double* l_aux_group) {
  double l_aux = 0.0;
  for (size_t i = 0; i < (size_t)E * G * C; ++i) slot_token[i] = -1;
  double* p = (double*)malloc(sizeof(double) * (size_t)S * E);
  int32_t* e1 = (int32_t*)malloc(sizeof(int32_t) * S);
  int32_t* e2 = (int32_t*)malloc(sizeof(int32_t) * S);
  double* g1 = (double*)malloc(sizeof(double) * S);
  double* g2 = (double*)malloc(sizeof(double) * S);
  for (int g = 0; g < G; ++g) {
    gso_gates(x + (size_t)g * S * M, wg, S, M, E, NULL, p);
    gso_mean_gates(p, S, E, m + (size_t)g * E);
    gso_top2(p, S, E, e1, e2, g1, g2, NULL);
    l_aux_group[g] = gso_capacity(S, E, C, e1, e2, g1, g2, u + (size_t)g * S,
                                  m + (size_t)g * E, NULL, variant_a,
                                  slot + (size_t)g * S * 2, weight + (size_t)g * S * 2,
                                  flags + (size_t)g * S, first_count + (size_t)g * E,
                                  total_count + (size_t)g * E);
    l_aux += l_aux_group[g];
    for (int s = 0; s < S; ++s) {
      expert_idx[((size_t)g * S + s) * 2 + 0] = e1[s];
      expert_idx[((size_t)g * S + s) * 2 + 1] = e2[s];
      for (int k = 0; k < 2; ++k) {
        const int32_t pos = slot[((size_t)g * S + s) * 2 + k];
        const int32_t e = k ? e2[s] : e1[s];
        if (pos >= 0) slot_token[((size_t)e * G + g) * C + pos] = s;
      }
    }
  }
  free(p); free(e1); free(e2); free(g1); free(g2);
  l_aux /= (double)G;
  if (!y) return l_aux;
  /* eq. (3) token by token */
  double* tmp = (double*)malloc(sizeof(double) * (size_t)M);
  for (size_t t = 0; t < (size_t)G * S; ++t) {
    double* yrow = y + t * M;
    for (int i = 0; i < M; ++i) yrow[i] = 0.0;
    for (int k = 0; k < 2; ++k) {
      if (slot[t * 2 + k] < 0) continue;
      const int32_t e = expert_idx[t * 2 + k];
      gso_ffn_rows(x + t * M, 1, wi + (size_t)e * M * H, wo + (size_t)e * H * M, M, H, tmp, NULL);
      for (int i = 0; i < M; ++i) yrow[i] += weight[t * 2 + k] * tmp[i];
    }
  }
  free(tmp);
  return l_aux;
}

/* Backward of L = <dy, y> + k * l_aux with the routing frozen.
 *
 * Per token, with raw top-2 gates a = g_{s,e1}, b = g_{s,e2}, D = a + b, kept
 * flags k1, k2 and expert outputs o1 = FFN_{e1}(x_s), o2 = FFN_{e2}(x_s):
 *   y_s = k1 (a/D) o1 + k2 (b/D) o2
 *   dL/dw1 = k1 <dy_s, o1>,  dL/dw2 = k2 <dy_s, o2>
 *   dL/da = (b/D^2)(dw1 - dw2),  dL/db = (a/D^2)(dw2 - dw1)
 * l_aux = (1/G) sum_g (1/E) sum_e (c_{g,e}/S) (1/S) sum_s g_{g,s,e}  gives the
 * dense term  dL/dg_{g,s,e} += k (1/G)(1/E)(c_{g,e}/S)(1/S).
 * Softmax: dlogit_{s,e} = g_{s,e} (dg_{s,e} - sum_e' g_{s,e'} dg_{s,e'}).
 * Gating GEMM: dwg = sum_tokens x^T dlogit;  dx += dlogit . wg^T.
 * Expert path for a kept choice with weight w: dout = w dy_s,
 *   dh = (dout . wo_e^T) * 1[pre-activation > 0], dwo_e += relu(h)^T dout,
 *   dwi_e += x_s^T dh, dx_s += dh . wi_e^T.
 */

/* Expert path backward for `rows` rows of ONE expert (eq. (2) differentiated):
 * xrows [rows,M] inputs, dout [rows,M] upstream gradient of FFN_e's output.
 * ACCUMULATES into dxrows [rows,M], dwi_e [M,H], dwo_e [H,M]. */
void gso_ffn_rows_backward(const float* xrows, const double* dout, int rows, const float* wi_e,
                           const float* wo_e, int M, int H, double* dxrows, double* dwi_e,
                           double* dwo_e) {
  double* hpre = (double*)malloc(sizeof(double) * (size_t)H);
  double* dh = (double*)malloc(sizeof(double) * (size_t)H);
  double* o = (double*)malloc(sizeof(double) * (size_t)M);
  for (int r = 0; r < rows; ++r) {
    const float* xs = xrows + (size_t)r * M;
    const double* dor = dout + (size_t)r * M;
    gso_ffn_rows(xs, 1, wi_e, wo_e, M, H, o, hpre);
#pragma omp parallel for schedule(static)
    for (int j = 0; j < H; ++j) {
      double acc = 0.0;
      const double act = hpre[j] > 0.0 ? hpre[j] : 0.0;
      for (int i = 0; i < M; ++i) {
        acc += dor[i] * (double)wo_e[(size_t)j * M + i];
        dwo_e[(size_t)j * M + i] += act * dor[i];
      }
      dh[j] = hpre[j] > 0.0 ? acc : 0.0;
    }
#pragma omp parallel for schedule(static)
    for (int mm = 0; mm < M; ++mm) {
      double acc = 0.0;
      for (int j = 0; j < H; ++j) {
        dwi_e[(size_t)mm * H + j] += (double)xs[mm] * dh[j];
        acc += dh[j] * (double)wi_e[(size_t)mm * H + j];
      }
      dxrows[(size_t)r * M + mm] += acc;
    }
  }
  free(hpre); free(dh); free(o);
}

/* Gate backward for ONE token: p [E] its softmax gates, (e1,e2) its top-2, dw1/dw2 the
 * gradients of its two combine weights (0 for a dropped choice), first_count_g [E] the
 * group's c_e.  Writes dlogit [E]. */
void gso_gate_row_backward(const double* p, int E, int e1, int e2, double dw1, double dw2,
                           const int32_t* first_count_g, int S, int G, double k_aux,
                           double* dlogit) {
  const double a = p[e1], b = p[e2], D = a + b;
  for (int e = 0; e < E; ++e)
    dlogit[e] = k_aux * (1.0 / G) * (1.0 / E) * ((double)first_count_g[e] / (double)S) * (1.0 / S);
  dlogit[e1] += (b / (D * D)) * (dw1 - dw2);
  dlogit[e2] += (a / (D * D)) * (dw2 - dw1);
  double dot = 0.0;
  for (int e = 0; e < E; ++e) dot += p[e] * dlogit[e];
  for (int e = 0; e < E; ++e) dlogit[e] = p[e] * (dlogit[e] - dot);
}

/* Whole-layer backward.  Inputs are the forward inputs plus the frozen routing
 * (expert_idx, slot, first_count).  Outputs: dx [G,S,M], dwg [M,E], dwi [E,M,H],
 * dwo [E,H,M]. */
void gso_backward(int G, int S, int M, int H, int E, int C, const float* x,
                  const float* wg, const float* wi, const float* wo,
                  const int32_t* expert_idx, const int32_t* slot,
                  const int32_t* first_count, const float* dy, double k_aux,
                  double* dx, double* dwg, double* dwi, double* dwo) {
  (void)C;
  const size_t N = (size_t)G * S;
  memset(dx, 0, sizeof(double) * N * M);
  memset(dwg, 0, sizeof(double) * (size_t)M * E);
  memset(dwi, 0, sizeof(double) * (size_t)E * M * H);
  memset(dwo, 0, sizeof(double) * (size_t)E * H * M);
  double* p = (double*)malloc(sizeof(double) * (size_t)S * E);
  double* dlogit = (double*)malloc(sizeof(double) * (size_t)E);
  double* o = (double*)malloc(sizeof(double) * (size_t)M);
  double* dout = (double*)malloc(sizeof(double) * (size_t)M);
  for (int g = 0; g < G; ++g) {
    gso_gates(x + (size_t)g * S * M, wg, S, M, E, NULL, p);
    for (int s = 0; s < S; ++s) {
      const size_t t = (size_t)g * S + s;
      const float* xs = x + t * M;
      const float* dys = dy + t * M;
      const double* ps = p + (size_t)s * E;
      const int32_t ea = expert_idx[2 * t], eb = expert_idx[2 * t + 1];
      const double a = ps[ea], b = ps[eb], D = a + b;
      const double wgt[2] = {a / D, b / D};
      double dw[2] = {0.0, 0.0};
      for (int k = 0; k < 2; ++k) {
        if (slot[2 * t + k] < 0) continue;
        const int32_t e = k ? eb : ea;
        const float* wie = wi + (size_t)e * M * H;
        const float* woe = wo + (size_t)e * H * M;
        gso_ffn_rows(xs, 1, wie, woe, M, H, o, NULL);
        for (int i = 0; i < M; ++i) { dw[k] += (double)dys[i] * o[i]; dout[i] = wgt[k] * (double)dys[i]; }
        gso_ffn_rows_backward(xs, dout, 1, wie, woe, M, H, dx + t * M,
                              dwi + (size_t)e * M * H, dwo + (size_t)e * H * M);
      }
      gso_gate_row_backward(ps, E, ea, eb, dw[0], dw[1], first_count + (size_t)g * E, S, G, k_aux, dlogit);
      for (int mm = 0; mm < M; ++mm) {
        double acc = 0.0;
        for (int e = 0; e < E; ++e) {
          dwg[(size_t)mm * E + e] += (double)xs[mm] * dlogit[e];
          acc += dlogit[e] * (double)wg[(size_t)mm * E + e];
        }
        dx[t * M + mm] += acc;
      }
    }
  }
  free(p); free(dlogit); free(o); free(dout);
}
