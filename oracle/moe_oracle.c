/*
 * CPU oracle for the sparse-MoE FFN layer run by speculative-decoding verification.
 *
 * THIS IS TEST INFRASTRUCTURE, NOT THE PRODUCT.  It is a plain, slow, token-major
 * restatement of what the layer computes, written from the paper's description of the
 * method (Sec. 1: a router activates K experts per token and only those experts' FFNs
 * run; Sec. 3.2: each token activates K of E experts, experts that receive no token are
 * never touched; Eq. N(t), Eq. T_exp, Eq. T_thres) and from the layer math the workload
 * configurations state (softmax or sigmoid scoring, optional top-k renormalisation,
 * SwiGLU experts, optional shared expert with an optional sigmoid scalar gate).
 *
 * It shares no code, header, table or helper with the CUDA path.  All floating-point
 * work is fp64 over exactly widened bf16 / fp32 inputs; nothing is blocked, fused or
 * reordered beyond the definition; there is no grouping step in the layer functions (a
 * token simply runs its own k experts), so the layer cannot share a bug with the
 * permutation.  OpenMP parallelises over tokens only.
 *
 * Pins (tests marked "not gpu"): dense-masked brute force, numpy/torch library
 * reductions for special cases, invariants, exact enumeration and the closed forms.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

#define ORACLE_SCORE_SOFTMAX 0
#define ORACLE_SCORE_SIGMOID 1

/* bf16 is the upper 16 bits of an IEEE-754 binary32: widening is exact. */
static double bf16_to_f64(uint16_t v)
{
    uint32_t bits = ((uint32_t)v) << 16;
    float f;
    memcpy(&f, &bits, sizeof f);
    return (double)f;
}

int oracle_num_threads(void)
{
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}

/* ------------------------------------------------------------------------------------
 * Closed forms of Sec. 3.2.
 * ---------------------------------------------------------------------------------- */

/* Eq. N(t): expected number of activated experts after t tokens, each activating K of E
 * experts uniformly:  N(t) = E * (1 - ((E-K)/E)^t). */
double oracle_expected_active(int E, int K, double t)
{
    return (double)E * (1.0 - pow((double)(E - K) / (double)E, t));
}

/* Eq. T_exp: mean tokens per activated expert, t*K/N(t) = rho*t / (1 - (1-rho)^t). */
double oracle_mean_tokens_per_expert(double rho, double t)
{
    return rho * t / (1.0 - pow(1.0 - rho, t));
}

/* Eq. T_thres: smallest token count with N(t) >= tau*E:  ceil(log_{1-rho}(1-tau)). */
int oracle_token_threshold(double rho, double tau)
{
    return (int)ceil(log(1.0 - tau) / log(1.0 - rho));
}

/* ------------------------------------------------------------------------------------
 * Step 1: router logits  z[t,e] = sum_h x[t,h] * Wg[e,h] (+ b[e]), fp64, rounded once
 * to fp32 (the router works on fp32 logits).
 * ---------------------------------------------------------------------------------- */
void oracle_router_logits(const uint16_t *x, const float *w_router, const float *bias,
                          int T, int H, int E, float *z)
{
#pragma omp parallel for schedule(static)
    for (int t = 0; t < T; ++t) {
        for (int e = 0; e < E; ++e) {
            double acc = 0.0;
            for (int h = 0; h < H; ++h)
                acc += bf16_to_f64(x[(size_t)t * H + h]) * (double)w_router[(size_t)e * H + h];
            if (bias)
                acc += (double)bias[e];
            z[(size_t)t * E + e] = (float)acc;
        }
    }
}

/* Scalar shared-expert gate  s[t] = sigmoid(sum_h x[t,h] * w_sg[h]). */
void oracle_shared_gate(const uint16_t *x, const uint16_t *w_sg, int T, int H, double *s)
{
    for (int t = 0; t < T; ++t) {
        double acc = 0.0;
        for (int h = 0; h < H; ++h)
            acc += bf16_to_f64(x[(size_t)t * H + h]) * bf16_to_f64(w_sg[h]);
        s[t] = 1.0 / (1.0 + exp(-acc));
    }
}

/* ------------------------------------------------------------------------------------
 * Steps 2-3: selection on the fp32 logits, then scores.
 *   - S_t = the k experts with the largest z; slot j holds the j-th largest;
 *     equal logits: the lower expert index comes first.
 *   - softmax scores are over ALL E experts; sigmoid scores are per expert.
 *   - renormalize != 0 divides the k selected scores by their sum.
 *   - the result is multiplied by routed_scale.
 * Both score functions increase strictly with z, so selecting on z selects the same set
 * as selecting on the scores, without fp collisions between nearly equal scores.
 * ---------------------------------------------------------------------------------- */
void oracle_route_topk(const float *z, int T, int E, int k, int score_fn, int renormalize,
                       double routed_scale, int32_t *topk_idx, double *topk_w)
{
    for (int t = 0; t < T; ++t) {
        const float *zt = z + (size_t)t * E;
        int32_t *it = topk_idx + (size_t)t * k;
        double *wt = topk_w + (size_t)t * k;
        /* selection: k passes, each taking the best not-yet-taken expert */
        for (int j = 0; j < k; ++j) {
            int best = -1;
            for (int e = 0; e < E; ++e) {
                int taken = 0;
                for (int q = 0; q < j; ++q)
                    if (it[q] == e)
                        taken = 1;
                if (taken)
                    continue;
                if (best < 0 || zt[e] > zt[best])
                    best = e; /* strict '>' keeps the lower index on ties */
            }
            it[j] = best;
        }
        /* scores */
        if (score_fn == ORACLE_SCORE_SOFTMAX) {
            double zmax = (double)zt[0];
            for (int e = 1; e < E; ++e)
                if ((double)zt[e] > zmax)
                    zmax = (double)zt[e];
            double denom = 0.0;
            for (int e = 0; e < E; ++e)
                denom += exp((double)zt[e] - zmax);
            for (int j = 0; j < k; ++j)
                wt[j] = exp((double)zt[it[j]] - zmax) / denom;
        } else {
            for (int j = 0; j < k; ++j)
                wt[j] = 1.0 / (1.0 + exp(-(double)zt[it[j]]));
        }
        if (renormalize) {
            double s = 0.0;
            for (int j = 0; j < k; ++j)
                s += wt[j];
            for (int j = 0; j < k; ++j)
                wt[j] /= s;
        }
        for (int j = 0; j < k; ++j)
            wt[j] *= routed_scale;
    }
}

/* ------------------------------------------------------------------------------------
 * Step 7: reference grouping (integers only).  Assignment a = t*k + j goes to expert
 * topk_idx[a].  counts[e] = assignments of e; offsets = exclusive prefix sum with
 * offsets[E] = A; perm lists the assignments ordered by (expert, a) ascending;
 * inv_perm[perm[i]] = i; active = ascending list of experts with counts > 0, the rest
 * of the array filled with -1.
 * ---------------------------------------------------------------------------------- */
void oracle_permute(const int32_t *topk_idx, int T, int k, int E, int32_t *counts,
                    int32_t *offsets, int32_t *perm, int32_t *inv_perm, int32_t *active,
                    int32_t *n_active)
{
    const int A = T * k;
    for (int e = 0; e < E; ++e)
        counts[e] = 0;
    for (int a = 0; a < A; ++a)
        counts[topk_idx[a]] += 1;
    offsets[0] = 0;
    for (int e = 0; e < E; ++e)
        offsets[e + 1] = offsets[e] + counts[e];
    int pos = 0;
    for (int e = 0; e < E; ++e)
        for (int a = 0; a < A; ++a)
            if (topk_idx[a] == e) {
                perm[pos] = a;
                inv_perm[a] = pos;
                ++pos;
            }
    int n = 0;
    for (int e = 0; e < E; ++e)
        if (counts[e] > 0)
            active[n++] = e;
    *n_active = n;
    for (int i = n; i < E; ++i)
        active[i] = -1;
}

/* ------------------------------------------------------------------------------------
 * Step 4: one SwiGLU expert on one token row.
 *   g = Wgate x, u = Wup x (length I);  h = g * sigmoid(g) * u;  y = Wdown h (length H).
 * Wgate, Wup are [I,H] (H contiguous), Wdown is [H,I] (I contiguous); no intermediate
 * rounding.  scratch holds I doubles.
 * ---------------------------------------------------------------------------------- */
static void expert_ffn_row(const uint16_t *x_row, const uint16_t *w_gate, const uint16_t *w_up,
                           const uint16_t *w_down, int H, int I, double *scratch, double *y)
{
    for (int i = 0; i < I; ++i) {
        double g = 0.0, u = 0.0;
        for (int h = 0; h < H; ++h) {
            double xv = bf16_to_f64(x_row[h]);
            g += bf16_to_f64(w_gate[(size_t)i * H + h]) * xv;
            u += bf16_to_f64(w_up[(size_t)i * H + h]) * xv;
        }
        scratch[i] = g / (1.0 + exp(-g)) * u;
    }
    for (int h = 0; h < H; ++h) {
        double acc = 0.0;
        for (int i = 0; i < I; ++i)
            acc += bf16_to_f64(w_down[(size_t)h * I + i]) * scratch[i];
        y[h] = acc;
    }
}

/* One expert applied to T rows (used by tests of the expert alone). */
void oracle_expert_ffn(const uint16_t *x, const uint16_t *w_gate, const uint16_t *w_up,
                       const uint16_t *w_down, int T, int H, int I, double *y)
{
#pragma omp parallel
    {
        double *scratch = (double *)malloc(sizeof(double) * (size_t)I);
#pragma omp for schedule(static)
        for (int t = 0; t < T; ++t)
            expert_ffn_row(x + (size_t)t * H, w_gate, w_up, w_down, H, I, scratch,
                           y + (size_t)t * H);
        free(scratch);
    }
}

/* ------------------------------------------------------------------------------------
 * Steps 4-6: the layer, token-major.
 *   out[t] = sum_{j<k} w[t,j] * FFN_{idx[t,j]}(x[t])  (accumulated in slot order j)
 *          + s[t] * FFN_shared(x[t])                   (if I_s > 0; s = 1 when not given)
 * rows: optional list of n_rows token ids to evaluate (NULL = all T tokens in order);
 * out is [n_rows, H] in that order.  The layer is token-wise, so a row sample is exact.
 * ---------------------------------------------------------------------------------- */
void oracle_layer(const uint16_t *x, int T, int H, int E, int k, int I, int I_s,
                  const uint16_t *w_gate, const uint16_t *w_up, const uint16_t *w_down,
                  const uint16_t *ws_gate, const uint16_t *ws_up, const uint16_t *ws_down,
                  const int32_t *topk_idx, const double *topk_w, const double *shared_scale,
                  const int32_t *rows, int n_rows, double *out)
{
    (void)E;
    const int n = rows ? n_rows : T;
    const int Imax = I > I_s ? I : I_s;
#pragma omp parallel
    {
        double *scratch = (double *)malloc(sizeof(double) * (size_t)Imax);
        double *y = (double *)malloc(sizeof(double) * (size_t)H);
#pragma omp for schedule(dynamic, 1)
        for (int r = 0; r < n; ++r) {
            const int t = rows ? rows[r] : r;
            const uint16_t *xt = x + (size_t)t * H;
            double *ot = out + (size_t)r * H;
            for (int h = 0; h < H; ++h)
                ot[h] = 0.0;
            for (int j = 0; j < k; ++j) {
                const size_t e = (size_t)topk_idx[(size_t)t * k + j];
                expert_ffn_row(xt, w_gate + e * I * H, w_up + e * I * H, w_down + e * H * I, H, I,
                               scratch, y);
                const double w = topk_w[(size_t)t * k + j];
                for (int h = 0; h < H; ++h)
                    ot[h] += w * y[h];
            }
            if (I_s > 0) {
                expert_ffn_row(xt, ws_gate, ws_up, ws_down, H, I_s, scratch, y);
                const double s = shared_scale ? shared_scale[t] : 1.0;
                for (int h = 0; h < H; ++h)
                    ot[h] += s * y[h];
            }
        }
        free(scratch);
        free(y);
    }
}

/* ------------------------------------------------------------------------------------
 * Step 8: brute force for tiny inputs.  Every one of the E experts runs on every token;
 * a dense mask m[t,e] (= w[t,j] where e = idx[t,j], else 0) picks the result:
 *   out[t] = sum_e m[t,e] * FFN_e(x[t]) + s[t] * FFN_shared(x[t]).
 * ---------------------------------------------------------------------------------- */
void oracle_layer_dense_masked(const uint16_t *x, int T, int H, int E, int k, int I, int I_s,
                               const uint16_t *w_gate, const uint16_t *w_up,
                               const uint16_t *w_down, const uint16_t *ws_gate,
                               const uint16_t *ws_up, const uint16_t *ws_down,
                               const int32_t *topk_idx, const double *topk_w,
                               const double *shared_scale, double *out)
{
    const int Imax = I > I_s ? I : I_s;
    double *mask = (double *)calloc((size_t)T * E, sizeof(double));
    double *all_y = (double *)malloc(sizeof(double) * (size_t)E * H);
    double *scratch = (double *)malloc(sizeof(double) * (size_t)Imax);
    double *y = (double *)malloc(sizeof(double) * (size_t)H);
    for (int t = 0; t < T; ++t)
        for (int j = 0; j < k; ++j)
            mask[(size_t)t * E + topk_idx[(size_t)t * k + j]] = topk_w[(size_t)t * k + j];
    for (int t = 0; t < T; ++t) {
        const uint16_t *xt = x + (size_t)t * H;
        for (int e = 0; e < E; ++e)
            expert_ffn_row(xt, w_gate + (size_t)e * I * H, w_up + (size_t)e * I * H,
                           w_down + (size_t)e * H * I, H, I, scratch, all_y + (size_t)e * H);
        for (int h = 0; h < H; ++h) {
            double acc = 0.0;
            for (int e = 0; e < E; ++e)
                acc += mask[(size_t)t * E + e] * all_y[(size_t)e * H + h];
            out[(size_t)t * H + h] = acc;
        }
        if (I_s > 0) {
            expert_ffn_row(xt, ws_gate, ws_up, ws_down, H, I_s, scratch, y);
            const double s = shared_scale ? shared_scale[t] : 1.0;
            for (int h = 0; h < H; ++h)
                out[(size_t)t * H + h] += s * y[h];
        }
    }
    free(mask);
    free(all_y);
    free(scratch);
    free(y);
}
