/*
 * CPU oracle for the folded Mixture-of-Experts layer (ExFold).
 *
 * TEST INFRASTRUCTURE ONLY. This file is the slow, plain reference that the
 * CUDA library is checked against. Nothing in the product path may call it;
 * only the tests, the smoke check and the benchmark's cpu-baseline leg do.
 * It shares no code with the CUDA path.
 *
 * It follows the paper's equations in the paper's order:
 *   Eq. 1  gated (SwiGLU) expert            -> expert_ffn()
 *   Eq. 2  Top-K routing + restricted softmax -> gate_token()
 *   Eq. 3  MoE output                        -> orc_moe_apply() on Eq. 2's routes
 *   Eq. 4  folded output, literal form        -> orc_prefill_eq4(), orc_decode_eq4()
 *   Eq. 6-9 scalar projector calibration      -> orc_calibrate()
 *   Eq. 10 prefill retained set               -> prefill_select()
 *   Eq. 11 decode pool                        -> orc_decode_fold()
 *   Eq. 12 minimum-loss assignment            -> argmin_loss()
 *   Eq. 13 prefill fold                       -> orc_prefill_fold()
 *   Eq. 14 decode remap (and the appendix's remapping listing) -> orc_decode_fold()
 *
 * Precision: tensors are fp32 or bf16 (bf16 is widened exactly); every sum,
 * product, exp and division is done in double. The one exception is the
 * prefill ranking key, which is DEFINED as a single fp32 addition
 * logit + ln(h) so that both sides of a parity test take the selection
 * decision in the same arithmetic. No blocking, no reordering: every
 * reduction is a plain left-to-right loop. OpenMP only spreads independent
 * tokens over threads.
 *
 * Readings of points the paper leaves open (each is listed in the design notes):
 *   - Top-K ties, ranking ties, argmin ties: the lower expert id wins.
 *   - h_e = mean L2 norm of expert e's output over the calibration tokens that
 *     route to it; an expert never routed gets the mean h of the others.
 *   - ranking by w*h is done on log scale: key = logit + ln h (same order, since
 *     the softmax denominator is common to the token and h > 0).
 *   - scalars are clipped first, the loss uses the clipped scalar, its numerator
 *     is clamped at 0, epsilon = 1e-12 by default; S_ee = 1, L_ee = 0;
 *     a pair never observed gets S = 0, L = 1e30.
 *   - decode pool = all of the union when the union has at most M experts.
 *   - no renormalisation after folding; negative scalars allowed.
 *   - the shared expert (index N) always runs with weight 1 and takes no part in folding.
 *   - "parity unpinned" by the paper itself: the h definition, the tie rules,
 *     epsilon and the S of unobserved pairs (fixed only by the readings above).
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

enum { ORC_F32 = 0, ORC_BF16 = 1 };

static inline double ldv(const void *p, int dtype, size_t i)
{
    if (dtype == ORC_BF16) {
        uint32_t b = ((const uint16_t *)p)[i];
        float f;
        b <<= 16;
        memcpy(&f, &b, 4);
        return (double)f;
    }
    return (double)((const float *)p)[i];
}

int orc_num_threads(void)
{
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}

/* ---- Eq. 2: Top-K set ordered by router score, softmax restricted to it ---- */
static void gate_token(const float *r, int N, int K, int32_t *ids, double *w)
{
    for (int k = 0; k < K; ++k) {
        int best = -1;
        for (int e = 0; e < N; ++e) {
            int taken = 0;
            for (int j = 0; j < k; ++j)
                if (ids[j] == e) taken = 1;
            if (taken) continue;
            if (best < 0 || r[e] > r[best]) best = e; /* strict >: lower id wins ties */
        }
        ids[k] = best;
    }
    double m = (double)r[ids[0]];
    double z = 0.0;
    for (int k = 0; k < K; ++k) {
        w[k] = exp((double)r[ids[k]] - m);
        z += w[k];
    }
    for (int k = 0; k < K; ++k) w[k] /= z;
}

int orc_gate(const float *logits, int64_t T, int N, int K, int32_t *ids, float *w, double *w64)
{
    if (K < 1 || K > N || K > 64) return -1;
#pragma omp parallel for schedule(static)
    for (int64_t i = 0; i < T; ++i) {
        int32_t id[64];
        double ww[64];
        gate_token(logits + i * N, N, K, id, ww);
        for (int k = 0; k < K; ++k) {
            ids[i * K + k] = id[k];
            if (w) w[i * K + k] = (float)ww[k];
            if (w64) w64[i * K + k] = ww[k];
        }
    }
    return 0;
}

/* ---- router scores entering Eq. 2: r_e(x) = <W_r[e], x>, summed in double in index order;
 *      out32 (fp32, what the layer consumes) and out64 may each be NULL ---- */
int orc_router_logits(const void *x, int dtype, int64_t T, int d, const void *wr, int N, float *out32, double *out64)
{
    if (T < 0 || d < 1 || N < 1) return -1;
#pragma omp parallel for schedule(static)
    for (int64_t i = 0; i < T; ++i)
        for (int e = 0; e < N; ++e) {
            double r = 0.0;
            for (int c = 0; c < d; ++c) r += ldv(wr, dtype, (size_t)e * d + c) * ldv(x, dtype, (size_t)i * d + c);
            if (out32) out32[i * N + e] = (float)r;
            if (out64) out64[i * N + e] = r;
        }
    return 0;
}

/* ---- Eq. 1: E_e(x) = W_down ( silu(W_gate x) * (W_up x) ) ---- */
static void expert_ffn(const void *x, size_t xoff, int dtype, int d, int I,
                       const void *wg, const void *wu, const void *wd, int e,
                       double *act /* [I] scratch */, double *out /* [d] */)
{
    size_t base_gu = (size_t)e * (size_t)I * (size_t)d;
    size_t base_dn = (size_t)e * (size_t)d * (size_t)I;
    for (int j = 0; j < I; ++j) {
        double g = 0.0, u = 0.0;
        size_t row = base_gu + (size_t)j * d;
        for (int c = 0; c < d; ++c) {
            double xv = ldv(x, dtype, xoff + c);
            g += ldv(wg, dtype, row + c) * xv;
            u += ldv(wu, dtype, row + c) * xv;
        }
        act[j] = (g / (1.0 + exp(-g))) * u;
    }
    for (int r = 0; r < d; ++r) {
        double o = 0.0;
        size_t row = base_dn + (size_t)r * I;
        for (int j = 0; j < I; ++j) o += ldv(wd, dtype, row + j) * act[j];
        out[r] = o;
    }
}

/*
 * Eq. 3 / the metadata form of Eq. 4: y_i = sum_j w[i][j] E_{ids[i][j]}(x_i)
 * (+ shared expert with weight 1). tok_idx selects which tokens are
 * evaluated (NULL: tokens 0..n_sel-1); y has n_sel rows.
 */
int orc_moe_apply(const void *x, int dtype, int64_t n_sel, const int64_t *tok_idx, int d, int I,
                  int N, int n_shared, const void *wg, const void *wu, const void *wd, int Kr,
                  const int32_t *ids, const float *w, float *y)
{
    int err = 0;
#pragma omp parallel
    {
        double *act = (double *)malloc(sizeof(double) * (size_t)I);
        double *o = (double *)malloc(sizeof(double) * (size_t)d);
        double *acc = (double *)malloc(sizeof(double) * (size_t)d);
#pragma omp for schedule(dynamic, 1)
        for (int64_t q = 0; q < n_sel; ++q) {
            int64_t i = tok_idx ? tok_idx[q] : q;
            for (int r = 0; r < d; ++r) acc[r] = 0.0;
            for (int j = 0; j < Kr; ++j) {
                int e = ids[i * Kr + j];
                if (e < 0 || e >= N) { err = 1; continue; }
                expert_ffn(x, (size_t)i * d, dtype, d, I, wg, wu, wd, e, act, o);
                double wj = (double)w[i * Kr + j];
                for (int r = 0; r < d; ++r) acc[r] += wj * o[r];
            }
            for (int s = 0; s < n_shared; ++s) {
                expert_ffn(x, (size_t)i * d, dtype, d, I, wg, wu, wd, N + s, act, o);
                for (int r = 0; r < d; ++r) acc[r] += o[r];
            }
            for (int r = 0; r < d; ++r) y[q * d + r] = (float)acc[r];
        }
        free(act); free(o); free(acc);
    }
    return err ? -2 : 0;
}

/* outputs of each routed expert, unweighted: out[i][k][:] = E_{ids[i][k]}(x_i), double */
int orc_expert_outputs(const void *x, int dtype, int64_t m, int d, int I, const void *wg,
                       const void *wu, const void *wd, int K, const int32_t *ids, double *out)
{
#pragma omp parallel
    {
        double *act = (double *)malloc(sizeof(double) * (size_t)I);
#pragma omp for schedule(dynamic, 1)
        for (int64_t i = 0; i < m; ++i)
            for (int k = 0; k < K; ++k)
                expert_ffn(x, (size_t)i * d, dtype, d, I, wg, wu, wd, ids[i * K + k], act,
                           out + ((size_t)i * K + k) * d);
        free(act);
    }
    return 0;
}

/*
 * Eq. 6-9 (and the appendix's shared-scalar / normalised-loss forms): pairwise scalar
 * calibration. mode 0: a pair (s,t) is observed on token i when both experts are in
 * the token's Top-K; mode 1: every expert sees every token.
 * Returns the number of routed experts never observed (>0 is a warning), <0 on error.
 * stats (optional) receives A, B, C as three [N][N] double planes.
 */
int orc_calibrate(const void *x, int dtype, int64_t m, int d, int I, int N, int K, const void *wg,
                  const void *wu, const void *wd, const float *logits, double lambda,
                  double clip_lo, double clip_hi, double eps, int mode, float *S, float *L,
                  float *h, float *lnh, int32_t *n_obs, double *stats)
{
    size_t NN = (size_t)N * N;
    double *A = (double *)calloc(NN, sizeof(double));  /* sum w <v,u>  */
    double *Bv = (double *)calloc(NN, sizeof(double)); /* sum w |v|^2  */
    double *C = (double *)calloc(NN, sizeof(double));  /* sum w |u|^2  */
    int32_t *cnt = (int32_t *)calloc(NN, sizeof(int32_t));
    double *H = (double *)calloc((size_t)N, sizeof(double));
    int64_t *hc = (int64_t *)calloc((size_t)N, sizeof(int64_t));
    int Ke = mode == 1 ? N : K;
    int32_t *ids = (int32_t *)malloc(sizeof(int32_t) * (size_t)Ke);
    double *gw = (double *)malloc(sizeof(double) * (size_t)(K > 0 ? K : 1));
    double *outs = (double *)malloc(sizeof(double) * (size_t)Ke * d);
    double *act = (double *)malloc(sizeof(double) * (size_t)I);
    if (!A || !Bv || !C || !cnt || !H || !hc || !ids || !outs || !act) return -3;

    /* tokens in order, so the statistics are plain left-to-right sums */
    for (int64_t i = 0; i < m; ++i) {
        if (mode == 1) {
            for (int e = 0; e < N; ++e) ids[e] = e;
        } else {
            gate_token(logits + i * N, N, K, ids, gw);
        }
        for (int k = 0; k < Ke; ++k)
            expert_ffn(x, (size_t)i * d, dtype, d, I, wg, wu, wd, ids[k], act, outs + (size_t)k * d);
        for (int a = 0; a < Ke; ++a) {
            const double *u = outs + (size_t)a * d; /* source output u_i = E_s(x_i) */
            double uu = 0.0;
            for (int r = 0; r < d; ++r) uu += u[r] * u[r];
            double wi = sqrt(uu); /* token weight = source output norm */
            H[ids[a]] += wi;
            hc[ids[a]] += 1;
            for (int b = 0; b < Ke; ++b) {
                if (a == b) continue;
                const double *v = outs + (size_t)b * d; /* target output v_i = E_t(x_i) */
                double vu = 0.0, vv = 0.0;
                for (int r = 0; r < d; ++r) { vu += v[r] * u[r]; vv += v[r] * v[r]; }
                size_t p = (size_t)ids[a] * N + ids[b];
                A[p] += wi * vu;
                Bv[p] += wi * vv;
                C[p] += wi * uu;
                cnt[p] += 1;
            }
        }
    }
    for (int s = 0; s < N; ++s)
        for (int t = 0; t < N; ++t) {
            size_t p = (size_t)s * N + t;
            if (s == t) { S[p] = 1.0f; L[p] = 0.0f; continue; }
            if (cnt[p] == 0) { S[p] = 0.0f; L[p] = 1e30f; continue; }
            double sc = A[p] / (Bv[p] + lambda);                      /* Eq. 8 */
            if (sc < clip_lo) sc = clip_lo;
            if (sc > clip_hi) sc = clip_hi;
            double num = C[p] - 2.0 * sc * A[p] + sc * sc * Bv[p];    /* Eq. 9 numerator, expanded */
            if (num < 0.0) num = 0.0;
            S[p] = (float)sc;
            L[p] = (float)(num / (C[p] + eps));
        }
    int unobserved = 0;
    double hsum = 0.0;
    int hn = 0;
    for (int e = 0; e < N; ++e)
        if (hc[e] > 0) { hsum += H[e] / (double)hc[e]; hn++; }
    for (int e = 0; e < N; ++e) {
        double he;
        if (hc[e] > 0) he = H[e] / (double)hc[e];
        else { he = hn ? hsum / hn : 1.0; unobserved++; }
        h[e] = (float)he;
        lnh[e] = (float)log((double)h[e]);
    }
    if (n_obs) memcpy(n_obs, cnt, NN * sizeof(int32_t));
    if (stats) {
        memcpy(stats, A, NN * sizeof(double));
        memcpy(stats + NN, Bv, NN * sizeof(double));
        memcpy(stats + 2 * NN, C, NN * sizeof(double));
    }
    free(A); free(Bv); free(C); free(cnt); free(H); free(hc); free(ids); free(gw); free(outs); free(act);
    return unobserved;
}

/* ---- Eq. 12: target with the smallest calibrated loss; ties -> lower expert id ---- */
static int argmin_loss(const float *L, int N, int s, const int32_t *cand, int n_cand)
{
    int best = -1;
    for (int j = 0; j < n_cand; ++j) {
        int t = cand[j];
        if (best < 0) { best = t; continue; }
        float lt = L[(size_t)s * N + t], lb = L[(size_t)s * N + best];
        if (lt < lb || (lt == lb && t < best)) best = t;
    }
    return best;
}

/*
 * Eq. 10 on log scale: order the token's K routes by key = logit + ln h (one fp32 add),
 * descending, ties -> lower expert id. order[] receives slot indices.
 */
static void prefill_select(const float *r, const int32_t *ids, int K, const float *lnh, int *order)
{
    float key[64];
    for (int k = 0; k < K; ++k) {
        volatile float s = r[ids[k]] + lnh[ids[k]];
        key[k] = s;
        order[k] = k;
    }
    for (int a = 0; a < K; ++a) /* selection sort, K is small */
        for (int b = a + 1; b < K; ++b) {
            int ia = order[a], ib = order[b];
            if (key[ib] > key[ia] || (key[ib] == key[ia] && ids[ib] < ids[ia])) {
                order[a] = ib;
                order[b] = ia;
            }
        }
}

/*
 * Prefill folding (Eq. 10, 12, 13). Outputs per token: the K' retained ids in
 * descending key order, their folded weights, and for each omitted route (in
 * descending key order) its source and its target.
 * mism (optional, one int64) counts tokens whose retained SET differs when the
 * ranking is done literally on w*h in double instead of on the fp32 log key.
 */
int orc_prefill_fold(const float *logits, int64_t T, int N, int K, int Kp, const float *S,
                     const float *L, const float *h, const float *lnh, int32_t *ids_out,
                     float *w_out, int32_t *omit_src, int32_t *omit_tgt, int64_t *mism)
{
    if (K < 1 || K > 64 || K > N || Kp < 1 || Kp > K) return -1;
    int64_t mismatch = 0;
    int Ko = K - Kp;
#pragma omp parallel for schedule(static) reduction(+ : mismatch)
    for (int64_t i = 0; i < T; ++i) {
        int32_t ids[64], kept[64];
        double w[64], wt[64];
        int order[64];
        const float *r = logits + i * N;
        gate_token(r, N, K, ids, w);
        prefill_select(r, ids, K, lnh, order);
        for (int j = 0; j < Kp; ++j) {
            kept[j] = ids[order[j]];
            wt[j] = w[order[j]];
        }
        for (int o = 0; o < Ko; ++o) {
            int slot = order[Kp + o];
            int s = ids[slot];
            int t = argmin_loss(L, N, s, kept, Kp);
            for (int j = 0; j < Kp; ++j)
                if (kept[j] == t) wt[j] += w[slot] * (double)S[(size_t)s * N + t]; /* Eq. 13 */
            if (omit_src) omit_src[i * Ko + o] = s;
            if (omit_tgt) omit_tgt[i * Ko + o] = t;
        }
        for (int j = 0; j < Kp; ++j) {
            ids_out[i * Kp + j] = kept[j];
            w_out[i * Kp + j] = (float)wt[j];
        }
        if (mism && h) { /* literal w*h ranking in double */
            int diff = 0;
            for (int j = 0; j < Kp && !diff; ++j) {
                int slot = order[j];
                double sj = w[slot] * (double)h[ids[slot]];
                for (int o = Kp; o < K; ++o) {
                    int so = order[o];
                    if (w[so] * (double)h[ids[so]] > sj) { diff = 1; break; }
                }
            }
            mismatch += diff;
        }
    }
    if (mism) *mism = mismatch;
    return 0;
}

/*
 * Prefill folding with the safeguards of the cross-model sections:
 *  - loss threshold (Qwen3.5 configuration): directed pairs whose calibrated loss exceeds
 *    loss_thr are excluded from target assignment; an omitted route with no admissible target
 *    is dropped (reading: the paper does not say);
 *  - rescale: after folding, the retained weights of a token are scaled by
 *    (sum of the original K routed weights) / (sum of the folded weights), so the original
 *    routed-weight sum is preserved (skipped when the folded sum is not positive: reading);
 *  - confidence split (DeepSeek-V4 appendix): with c_s = clip(1 - l_{s->t*}, 0, 1) for the
 *    minimum-loss target t*, the part w_s c_s S[s][t*] is folded onto t* and the rest
 *    w_s (1 - c_s) is spread over the retained routes in proportion to their original
 *    router weights.
 * loss_thr = +inf, rescale = 0, confidence = 0 is plain Eq. 13.
 */
int orc_prefill_fold_safe(const float *logits, int64_t T, int N, int K, int Kp, const float *S,
                          const float *L, const float *lnh, double loss_thr, int rescale,
                          int confidence, int32_t *ids_out, float *w_out, int32_t *omit_src,
                          int32_t *omit_tgt)
{
    if (K < 1 || K > 64 || K > N || Kp < 1 || Kp > K) return -1;
    int Ko = K - Kp;
#pragma omp parallel for schedule(static)
    for (int64_t i = 0; i < T; ++i) {
        int32_t ids[64], kept[64], adm[64];
        double w[64], wt[64], w0[64];
        int order[64];
        const float *r = logits + i * N;
        gate_token(r, N, K, ids, w);
        prefill_select(r, ids, K, lnh, order);
        double kept_sum = 0.0, all_sum = 0.0;
        for (int k = 0; k < K; ++k) all_sum += w[k];
        for (int j = 0; j < Kp; ++j) {
            kept[j] = ids[order[j]];
            wt[j] = w0[j] = w[order[j]];
            kept_sum += w0[j];
        }
        for (int o = 0; o < Ko; ++o) {
            int slot = order[Kp + o];
            int s = ids[slot];
            int na = 0;
            for (int j = 0; j < Kp; ++j)
                if (!((double)L[(size_t)s * N + kept[j]] > loss_thr)) adm[na++] = kept[j];
            int t = na ? argmin_loss(L, N, s, adm, na) : -1;
            if (t >= 0) {
                double c = 1.0;
                if (confidence) {
                    c = 1.0 - (double)L[(size_t)s * N + t];
                    if (c < 0.0) c = 0.0;
                    if (c > 1.0) c = 1.0;
                }
                for (int j = 0; j < Kp; ++j) {
                    if (kept[j] == t) wt[j] += w[slot] * c * (double)S[(size_t)s * N + t];
                    if (confidence) wt[j] += w[slot] * (1.0 - c) * (w0[j] / kept_sum);
                }
            }
            if (omit_src) omit_src[i * Ko + o] = s;
            if (omit_tgt) omit_tgt[i * Ko + o] = t;
        }
        if (rescale) {
            double fs = 0.0;
            for (int j = 0; j < Kp; ++j) fs += wt[j];
            if (fs > 0.0)
                for (int j = 0; j < Kp; ++j) wt[j] *= all_sum / fs;
        }
        for (int j = 0; j < Kp; ++j) {
            ids_out[i * Kp + j] = kept[j];
            w_out[i * Kp + j] = (float)wt[j];
        }
    }
    return 0;
}

/*
 * Eq. 4 written out for prefill: run every one of the token's K experts' targets and
 * scale: y = sum_{t kept} a_t E_t(x) + sum_{s omitted} a_s S[s][t_s] E_{t_s}(x) (+ shared).
 * Each term evaluates its expert anew; nothing is coalesced.
 */
int orc_prefill_eq4(const void *x, int dtype, int64_t T, int d, int I, int N, int n_shared,
                    const void *wg, const void *wu, const void *wd, const float *logits, int K,
                    int Kp, const float *S, const float *L, const float *lnh, float *y)
{
    if (K < 1 || K > 64 || Kp < 1 || Kp > K) return -1;
#pragma omp parallel
    {
        double *act = (double *)malloc(sizeof(double) * (size_t)I);
        double *o = (double *)malloc(sizeof(double) * (size_t)d);
        double *acc = (double *)malloc(sizeof(double) * (size_t)d);
#pragma omp for schedule(dynamic, 1)
        for (int64_t i = 0; i < T; ++i) {
            int32_t ids[64], kept[64];
            double w[64];
            int order[64];
            const float *r = logits + i * N;
            gate_token(r, N, K, ids, w);
            prefill_select(r, ids, K, lnh, order);
            for (int j = 0; j < Kp; ++j) kept[j] = ids[order[j]];
            for (int c = 0; c < d; ++c) acc[c] = 0.0;
            for (int j = 0; j < K; ++j) {
                int slot = order[j];
                int s = ids[slot];
                int t = s;
                double coef = w[slot];
                if (j >= Kp) {
                    t = argmin_loss(L, N, s, kept, Kp);
                    coef = w[slot] * (double)S[(size_t)s * N + t];
                }
                expert_ffn(x, (size_t)i * d, dtype, d, I, wg, wu, wd, t, act, o);
                for (int c = 0; c < d; ++c) acc[c] += coef * o[c];
            }
            for (int s = 0; s < n_shared; ++s) {
                expert_ffn(x, (size_t)i * d, dtype, d, I, wg, wu, wd, N + s, act, o);
                for (int c = 0; c < d; ++c) acc[c] += o[c];
            }
            for (int c = 0; c < d; ++c) y[i * d + c] = (float)acc[c];
        }
        free(act); free(o); free(acc);
    }
    return 0;
}

/*
 * Decode pool folding (Eq. 11, 12, 14).
 *  score_e = h_e * sum_i w_{i,e} over the batch (tokens ascending), in double;
 *  pool = the union when it has at most M experts, else its M best by score
 *         (ties -> lower id), listed in descending score;
 *  target[s] = s, scale[s] = 1 for s in the pool, else the minimum-loss pool expert
 *         and S[s][target]; every routed slot (id, w) becomes (target[id], w*scale[id]),
 *         the [B][K] layout is kept (duplicates inside a token stay separate slots).
 * pool_mask has ceil(N/32) words; score (optional) is [N] double.
 */
int orc_decode_fold(const float *logits, int64_t B, int N, int K, int M, const float *S,
                    const float *L, const float *h, int32_t *pool_ids, int32_t *pool_size,
                    uint32_t *pool_mask, int32_t *ids_out, float *w_out, int32_t *target,
                    float *scale, double *score_out, double *min_gap)
{
    if (K < 1 || K > 64 || K > N || M < 1 || M > N) return -1;
    int32_t *ids = (int32_t *)malloc(sizeof(int32_t) * (size_t)B * K);
    double *w = (double *)malloc(sizeof(double) * (size_t)B * K);
    double *score = (double *)calloc((size_t)N, sizeof(double));
    char *in_union = (char *)calloc((size_t)N, 1);
    char *in_pool = (char *)calloc((size_t)N, 1);
    int32_t *cand = (int32_t *)malloc(sizeof(int32_t) * (size_t)N);
    if (!ids || !w || !score || !in_union || !in_pool || !cand) return -3;
    for (int64_t i = 0; i < B; ++i) gate_token(logits + i * N, N, K, ids + i * K, w + i * K);
    for (int64_t i = 0; i < B; ++i)
        for (int k = 0; k < K; ++k) {
            int e = ids[i * K + k];
            in_union[e] = 1;
            score[e] += w[i * K + k]; /* sum_i w_{i,e} */
        }
    int n_union = 0;
    for (int e = 0; e < N; ++e) {
        score[e] *= (double)h[e];
        if (in_union[e]) cand[n_union++] = e;
    }
    /* order the union by (score desc, id asc) */
    for (int a = 0; a < n_union; ++a)
        for (int b = a + 1; b < n_union; ++b) {
            int ea = cand[a], eb = cand[b];
            if (score[eb] > score[ea] || (score[eb] == score[ea] && eb < ea)) {
                cand[a] = eb;
                cand[b] = ea;
            }
        }
    int P = n_union < M ? n_union : M;
    for (int w32 = 0; w32 < (N + 31) / 32; ++w32) pool_mask[w32] = 0u;
    for (int j = 0; j < M; ++j) pool_ids[j] = -1;
    for (int j = 0; j < P; ++j) {
        pool_ids[j] = cand[j];
        in_pool[cand[j]] = 1;
        pool_mask[cand[j] >> 5] |= 1u << (cand[j] & 31);
    }
    *pool_size = P;
    if (min_gap) { /* relative score gap at the pool boundary (input-quality check) */
        *min_gap = 1.0;
        if (P < n_union) {
            double a = score[cand[P - 1]], b = score[cand[P]];
            *min_gap = (a - b) / (fabs(a) > 0 ? fabs(a) : 1.0);
        }
    }
    for (int s = 0; s < N; ++s) {
        if (in_pool[s]) { target[s] = s; scale[s] = 1.0f; }
        else {
            int t = argmin_loss(L, N, s, cand, P);
            target[s] = t;
            scale[s] = S[(size_t)s * N + t];
        }
    }
    for (int64_t i = 0; i < B; ++i)
        for (int k = 0; k < K; ++k) {
            int e = ids[i * K + k];
            ids_out[i * K + k] = target[e];                                   /* Eq. 14 */
            w_out[i * K + k] = (float)(w[i * K + k] * (double)scale[e]);
        }
    if (score_out) memcpy(score_out, score, sizeof(double) * (size_t)N);
    free(ids); free(w); free(score); free(in_union); free(in_pool); free(cand);
    return 0;
}

/*
 * Static decode pool (appendix, "static implementation"): the pool is formed once from the
 * calibration-time norms, pool = TopK_e(h_e, M) over ALL experts (ties -> lower id, listed in
 * descending h), and one target and one scalar are precomputed for every possible source expert:
 * target[s] = s, scale[s] = 1 inside the pool, else the minimum-loss pool expert and S[s][target].
 */
int orc_static_pool(int N, int M, const float *S, const float *L, const float *h, int32_t *pool_ids,
                    int32_t *target, float *scale)
{
    if (M < 1 || M > N) return -1;
    char *in_pool = (char *)calloc((size_t)N, 1);
    if (!in_pool) return -3;
    for (int j = 0; j < M; ++j) {
        int best = -1;
        for (int e = 0; e < N; ++e) {
            if (in_pool[e]) continue;
            if (best < 0 || h[e] > h[best]) best = e; /* strict >: lower id wins ties */
        }
        pool_ids[j] = best;
        in_pool[best] = 1;
    }
    for (int s = 0; s < N; ++s) {
        if (in_pool[s]) { target[s] = s; scale[s] = 1.0f; }
        else {
            int t = argmin_loss(L, N, s, pool_ids, M);
            target[s] = t;
            scale[s] = S[(size_t)s * N + t];
        }
    }
    free(in_pool);
    return 0;
}

/*
 * Per-route remapping with precomputed tables (the appendix's remapping listing): every routed
 * slot (id, w) of Eq. 2 becomes (target[id], w * scale[id]); the [B][K] layout is kept.
 */
int orc_decode_static(const float *logits, int64_t B, int N, int K, const int32_t *target,
                      const float *scale, int32_t *ids_out, float *w_out)
{
    if (K < 1 || K > 64 || K > N) return -1;
#pragma omp parallel for schedule(static)
    for (int64_t i = 0; i < B; ++i) {
        int32_t ids[64];
        double w[64];
        gate_token(logits + i * N, N, K, ids, w);
        for (int k = 0; k < K; ++k) {
            ids_out[i * K + k] = target[ids[k]];
            w_out[i * K + k] = (float)(w[k] * (double)scale[ids[k]]);
        }
    }
    return 0;
}

/*
 * Eq. 4 written out for decode, given the pool: retained routes run their own expert,
 * routes outside the pool run their minimum-loss pool expert scaled by S. Nothing merged.
 */
int orc_decode_eq4(const void *x, int dtype, int64_t B, int d, int I, int N, int n_shared,
                   const void *wg, const void *wu, const void *wd, const float *logits, int K,
                   const int32_t *pool, int P, const float *S, const float *L, float *y)
{
    if (K < 1 || K > 64 || P < 1) return -1;
#pragma omp parallel
    {
        double *act = (double *)malloc(sizeof(double) * (size_t)I);
        double *o = (double *)malloc(sizeof(double) * (size_t)d);
        double *acc = (double *)malloc(sizeof(double) * (size_t)d);
#pragma omp for schedule(dynamic, 1)
        for (int64_t i = 0; i < B; ++i) {
            int32_t ids[64];
            double w[64];
            gate_token(logits + i * N, N, K, ids, w);
            for (int c = 0; c < d; ++c) acc[c] = 0.0;
            for (int k = 0; k < K; ++k) {
                int s = ids[k], t = s, inside = 0;
                double coef = w[k];
                for (int j = 0; j < P; ++j)
                    if (pool[j] == s) inside = 1;
                if (!inside) {
                    t = argmin_loss(L, N, s, pool, P);
                    coef = w[k] * (double)S[(size_t)s * N + t];
                }
                expert_ffn(x, (size_t)i * d, dtype, d, I, wg, wu, wd, t, act, o);
                for (int c = 0; c < d; ++c) acc[c] += coef * o[c];
            }
            for (int s = 0; s < n_shared; ++s) {
                expert_ffn(x, (size_t)i * d, dtype, d, I, wg, wu, wd, N + s, act, o);
                for (int c = 0; c < d; ++c) acc[c] += o[c];
            }
            for (int c = 0; c < d; ++c) y[i * d + c] = (float)acc[c];
        }
        free(act); free(o); free(acc);
    }
    return 0;
}

/*
 * Expert-sorted permutation of R routes: perm lists route indices ordered by
 * (group id, route index); offsets[g] is the first position of group g, offsets[G] = R.
 */
int orc_sort_routes(const int32_t *ids, int64_t R, int G, int32_t *perm, int32_t *offsets)
{
    int64_t p = 0;
    for (int g = 0; g < G; ++g) {
        offsets[g] = (int32_t)p;
        for (int64_t r = 0; r < R; ++r)
            if (ids[r] == g) perm[p++] = (int32_t)r;
    }
    offsets[G] = (int32_t)p;
    return p == R ? 0 : -2;
}
