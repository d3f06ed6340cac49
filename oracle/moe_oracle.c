/*
 * CPU oracle for the per-layer top-k Mixture-of-Experts forward pass.
 *
 * TEST INFRASTRUCTURE ONLY.  This file is the slow, plain, obviously-correct
 * statement of what the MoE layer computes; it exists so that the CUDA library
 * can be checked against it.  It shares no code, header, table or helper with
 * the CUDA path, and the CUDA path never calls it.
 *
 * What it follows: the paper's Section 2, paragraph "Mixture of Experts":
 *     y = sum_{i in top-k} G(x)_i * E_i(x),   G(x) = Softmax(TopK[x . W_g]),
 * with the number of active experts k given per layer (Algorithm 1's
 * UpdateTopk step; the search space {1..k_base} of Section 3).  The paper says
 * E_i is "typically an FFN"; the FFN used here is the bias-free SwiGLU block
 * of the models in the paper's Table 1:  E(x) = W_down (silu(W_gate x) * (W_up x)).
 *
 * Every sum is taken in IEEE double, in index order, on the exact values of the
 * inputs (fp32 and bf16 inputs are widened exactly); nothing is rounded in
 * between.  There is no blocking, tiling or fusion: each function is a loop
 * nest that can be read against the formula it cites.  The only parallelism is
 * an OpenMP "parallel for" over tokens, which are independent.
 *
 * Pins (tests/test_oracle_pins.py): dense-mixture identity at k = E without
 * renormalisation, brute-force subset enumeration for TopK, literal
 * Softmax(TopK[z]) against the renormalised form, k = 1 reduces to one expert,
 * E = 1 reduces to a plain SwiGLU MLP evaluated with numpy, W_up = 0 gives 0,
 * linearity in W_down, shared-expert concatenation identity, dispatch
 * invariants.  The paper prints no numeric worked example of a layer output,
 * so no printed value pins the numbers: "parity unpinned by a printed value",
 * pinned by closed forms and brute force instead.
 */
#include <math.h>
#include <stddef.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

enum { ORC_F32 = 0, ORC_BF16 = 1, ORC_F64 = 2 };

/* exact widening of one stored element to double */
static inline double ld(const void *p, int dt, size_t i)
{
    if (dt == ORC_F64) return ((const double *)p)[i];
    if (dt == ORC_F32) return (double)((const float *)p)[i];
    /* bf16: the upper 16 bits of an IEEE binary32 */
    uint32_t bits = ((uint32_t)((const uint16_t *)p)[i]) << 16;
    float f;
    memcpy(&f, &bits, sizeof f);
    return (double)f;
}

int orc_num_threads(void)
{
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}

/* ---------------------------------------------------------------------------
 * Router logits, z = x . W_g (+ b): Section 2, "G(x) := Softmax(TopK[x . W_g])".
 * x [T,d], W_g [E,d] (row e is expert e's gating vector), b [E] or NULL.
 * z [T,E] double.
 * ------------------------------------------------------------------------- */
void orc_router_logits(const void *x, int dt_x, const void *Wg, int dt_w,
                       const float *bias, int T, int d, int E, double *z)
{
#pragma omp parallel for schedule(static)
    for (int t = 0; t < T; ++t)
        for (int e = 0; e < E; ++e) {
            double acc = 0.0;
            for (int c = 0; c < d; ++c)
                acc += ld(x, dt_x, (size_t)t * d + c) * ld(Wg, dt_w, (size_t)e * d + c);
            if (bias) acc += (double)bias[e];
            z[(size_t)t * E + e] = acc;
        }
}

/* ---------------------------------------------------------------------------
 * TopK and the gate values, Section 2: TopK[.] keeps the k experts with the
 * highest gating scores and Softmax turns their scores into weights.
 *
 *   S      = the k indices with the largest logit; order: logit descending,
 *            equal logits -> lower index first (the paper is silent on ties).
 *   renorm = 1: g_i = exp(z_i) / sum_{j in S} exp(z_j)    (the paper's formula:
 *               softmax over the selected logits only)
 *   renorm = 0: g_i = exp(z_i) / sum_{j < E} exp(z_j)     (softmax over all
 *               experts, selected entries kept as they are)
 *
 * select_f32 = 1 takes the comparison on the logits rounded to binary32, the
 * precision in which the CUDA router decides; the gate values always come from
 * the unrounded z.  margin[t] = z_(k) - z_(k+1) in the comparison precision
 * (+inf when k = E); callers use it to set aside near-ties.
 * idx [T,k] int32, gate [T,k] double, margin [T] double (nullable).
 * ------------------------------------------------------------------------- */
void orc_topk_gates(const double *z, int T, int E, int k, int renorm, int select_f32,
                    int32_t *idx, double *gate, double *margin)
{
#pragma omp parallel for schedule(static)
    for (int t = 0; t < T; ++t) {
        const double *zt = z + (size_t)t * E;
        double *key = (double *)malloc(sizeof(double) * (size_t)E);
        char *taken = (char *)calloc((size_t)E, 1);
        for (int e = 0; e < E; ++e) key[e] = select_f32 ? (double)(float)zt[e] : zt[e];

        /* selection: k passes, each picks the largest remaining key; the scan
         * runs in ascending index and only a strictly larger key replaces the
         * incumbent, so equal keys resolve to the lower index */
        for (int j = 0; j < k; ++j) {
            int best = -1;
            for (int e = 0; e < E; ++e) {
                if (taken[e]) continue;
                if (best < 0 || key[e] > key[best]) best = e;
            }
            taken[best] = 1;
            idx[(size_t)t * k + j] = best;
        }
        if (margin) {
            if (k == E) {
                margin[t] = INFINITY;
            } else {
                int nxt = -1;
                for (int e = 0; e < E; ++e) {
                    if (taken[e]) continue;
                    if (nxt < 0 || key[e] > key[nxt]) nxt = e;
                }
                margin[t] = key[idx[(size_t)t * k + k - 1]] - key[nxt];
            }
        }

        /* gates */
        double zmax = zt[0];
        for (int e = 1; e < E; ++e) if (zt[e] > zmax) zmax = zt[e];
        double denom = 0.0;
        if (renorm) {
            for (int j = 0; j < k; ++j) denom += exp(zt[idx[(size_t)t * k + j]] - zmax);
        } else {
            for (int e = 0; e < E; ++e) denom += exp(zt[e] - zmax);
        }
        for (int j = 0; j < k; ++j)
            gate[(size_t)t * k + j] = exp(zt[idx[(size_t)t * k + j]] - zmax) / denom;
        free(key);
        free(taken);
    }
}

/* ---------------------------------------------------------------------------
 * Dispatch bookkeeping (integer, exact).  The paper only says that tokens are
 * routed to experts and that the per-expert token load decides the time
 * (Introduction; Section 3's latency discussion); the artefacts below are the
 * plain definition of "group the (token, slot) pairs by expert":
 *   counts[e]  = number of pairs (t,j) with idx[t,j] = e
 *   offsets    = exclusive prefix sum of counts, offsets[E] = T*k
 *   perm[r]    = flat pair id t*k+j of the r-th row in expert-major order,
 *                pairs of one expert in ascending t
 *   inv_perm   = inverse of perm
 * Written as a literal two-level loop (for each expert, for each pair in
 * ascending order), not as a counting sort.
 * ------------------------------------------------------------------------- */
void orc_dispatch(const int32_t *idx, int T, int k, int E, int32_t *counts,
                  int32_t *offsets, int32_t *perm, int32_t *inv_perm)
{
    int r = 0;
    for (int e = 0; e < E; ++e) {
        offsets[e] = r;
        int c = 0;
        for (int p = 0; p < T * k; ++p)
            if (idx[p] == e) {
                perm[r] = p;
                inv_perm[p] = r;
                ++r;
                ++c;
            }
        counts[e] = c;
    }
    offsets[E] = r;
}

/* ---------------------------------------------------------------------------
 * One expert on one token: E(x) = W_down ( silu(W_gate x) * (W_up x) ),
 * silu(a) = a / (1 + exp(-a)).  W_gate, W_up [I,d]; W_down [d,I]; all three
 * start at element offset given by the caller (expert e of a stacked tensor).
 * Section 2: "each expert E_i is typically an FFN".
 * ------------------------------------------------------------------------- */
static void expert_ffn(const double *x, const void *Wgate, const void *Wup, const void *Wdown,
                       int dt_w, size_t off_gu, size_t off_dn, int d, int I,
                       double *hbuf, double *out)
{
    for (int i = 0; i < I; ++i) {
        double a = 0.0, b = 0.0;
        for (int c = 0; c < d; ++c) {
            a += ld(Wgate, dt_w, off_gu + (size_t)i * d + c) * x[c];
            b += ld(Wup, dt_w, off_gu + (size_t)i * d + c) * x[c];
        }
        hbuf[i] = (a / (1.0 + exp(-a))) * b;
    }
    for (int c = 0; c < d; ++c) {
        double acc = 0.0;
        for (int i = 0; i < I; ++i)
            acc += ld(Wdown, dt_w, off_dn + (size_t)c * I + i) * hbuf[i];
        out[c] = acc;
    }
}

/* exported for the pins: one expert applied to one token */
void orc_expert_ffn(const void *x, int dt_x, const void *Wgate, const void *Wup,
                    const void *Wdown, int dt_w, int e, int d, int I, double *out)
{
    double *xr = (double *)malloc(sizeof(double) * (size_t)d);
    double *hb = (double *)malloc(sizeof(double) * (size_t)I);
    for (int c = 0; c < d; ++c) xr[c] = ld(x, dt_x, (size_t)c);
    expert_ffn(xr, Wgate, Wup, Wdown, dt_w, (size_t)e * I * d, (size_t)e * d * I, d, I, hb, out);
    free(xr);
    free(hb);
}

/* ---------------------------------------------------------------------------
 * The MoE layer on a list of tokens (tokens are independent, so any subset can
 * be evaluated alone):
 *   y[t] = routed_scale * sum_{j<k} g[t,j] * E_{idx[t,j]}(x[t])
 *          + gamma(x[t]) * E_shared(x[t])
 * Section 2's weighted sum over the active experts, summed in slot order
 * j = 0..k-1.  The shared expert is not in the paper; it is the always-on
 * SwiGLU expert of the Qwen1.5-MoE and DeepSeek-V2-Lite rows of Table 1, with
 * gamma = sigmoid(x . w_s) (shared_gate = 1) or 1 (shared_gate = 0), added
 * after the routed scaling.  I_s = 0 means no shared expert.
 *
 * idx/gate [T,k] come from orc_topk_gates.  tokens[n_tok] lists the token ids
 * to evaluate (NULL = 0..n_tok-1).  y [n_tok, d] double.
 * ------------------------------------------------------------------------- */
void orc_moe_layer(const void *x, int dt_x, int dt_w,
                   const void *Wgate, const void *Wup, const void *Wdown,
                   const void *Ws_gate, const void *Ws_up, const void *Ws_down, const void *w_s,
                   int d, int E, int I, int I_s, int shared_gate, double routed_scale,
                   int k, const int32_t *idx, const double *gate,
                   const int32_t *tokens, int n_tok, double *y)
{
    (void)E;
    int Imax = I > I_s ? I : I_s;
#pragma omp parallel
    {
        double *xr = (double *)malloc(sizeof(double) * (size_t)d);
        double *hb = (double *)malloc(sizeof(double) * (size_t)Imax);
        double *eo = (double *)malloc(sizeof(double) * (size_t)d);
#pragma omp for schedule(dynamic, 1)
        for (int n = 0; n < n_tok; ++n) {
            int t = tokens ? tokens[n] : n;
            double *yt = y + (size_t)n * d;
            for (int c = 0; c < d; ++c) {
                xr[c] = ld(x, dt_x, (size_t)t * d + c);
                yt[c] = 0.0;
            }
            for (int j = 0; j < k; ++j) {
                int e = idx[(size_t)t * k + j];
                double g = gate[(size_t)t * k + j];
                expert_ffn(xr, Wgate, Wup, Wdown, dt_w, (size_t)e * I * d, (size_t)e * d * I,
                           d, I, hb, eo);
                for (int c = 0; c < d; ++c) yt[c] += g * eo[c];
            }
            for (int c = 0; c < d; ++c) yt[c] *= routed_scale;
            if (I_s > 0) {
                double gamma = 1.0;
                if (shared_gate) {
                    double s = 0.0;
                    for (int c = 0; c < d; ++c) s += xr[c] * ld(w_s, dt_w, (size_t)c);
                    gamma = 1.0 / (1.0 + exp(-s));
                }
                expert_ffn(xr, Ws_gate, Ws_up, Ws_down, dt_w, 0, 0, d, I_s, hb, eo);
                for (int c = 0; c < d; ++c) yt[c] += gamma * eo[c];
            }
        }
        free(xr);
        free(hb);
        free(eo);
    }
}
