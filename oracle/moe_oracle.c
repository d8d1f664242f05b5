/*
 * moe_oracle.c -- TEST INFRASTRUCTURE, NOT THE PRODUCT.
 *
 * A plain, slow, host-only evaluation of the top-k gated SwiGLU Mixture-of-Experts
 * layer forward pass, written out directly from its definition.  It exists only so
 * that tests, the smoke check and the benchmark's CPU-baseline leg have something
 * independent to compare the CUDA path against.  Nothing in the product may call it,
 * and it shares no code, header, table or helper with the CUDA sources.
 *
 * What it follows (paper: "Kernel Analysis: FP8 MoE Kernel (Blackwell)", the Sec. 4.5
 * description of the layer; Sec. 4.5 "Expert FFN computation" for the pipeline order):
 *   - per token, k experts are chosen out of E candidates from the router scores;
 *   - tokens are reordered so that each expert's tokens are contiguous
 *     ("sort-scatter"), experts with no token are skipped;
 *   - every chosen expert applies a gate and an up projection, combined through
 *     SiLU, followed by a down projection;
 *   - the k expert outputs of a token are summed with the routing weights.
 * The paper leaves the scoring function open; the build's stated reading is
 * softmax -> top-k -> renormalise with ties broken towards the lower expert index,
 * w13 rows [0,I) = gate and [I,2I) = up, weights applied at the combine.
 *
 * Arithmetic type: every floating-point operation is done in REAL, which the build
 * sets to float (liboracle_f32.so, the precision the layer is specified in) or to
 * double (liboracle_f64.so, used to put an error bar on the float build).  bf16
 * inputs are widened exactly.  No blocking, fusion or reordering: the loops below are
 * the sums of the definition in index order.  OpenMP only distributes independent
 * tokens over threads; it never splits a sum.
 *
 * Pins (tests/test_oracle_*.py): hand-computed closed forms, a NumPy float64
 * brute-force evaluation of all E experts per token, library reductions
 * (torch.softmax/topk, numpy stable argsort, torch matmul), and invariants
 * (identical experts with k=E collapse to one dense MLP, weights sum to one,
 * token-permutation equivariance, exact power-of-two scaling).
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

#ifndef REAL
#define REAL float
#endif

#define ORACLE_OK 0
#define ORACLE_ERR_ARG (-1)
#define ORACLE_ERR_MISSING_EXPERT (-2)
#define ORACLE_ERR_NOMEM (-3)

static inline REAL real_exp(REAL v) { return sizeof(REAL) == sizeof(float) ? (REAL)expf((float)v) : (REAL)exp((double)v); }

/* bfloat16 is the upper half of an IEEE binary32: widening is exact. */
static inline REAL bf16_to_real(uint16_t b) {
    uint32_t u = (uint32_t)b << 16;
    float f;
    memcpy(&f, &u, sizeof f);
    return (REAL)f;
}

int moe_oracle_real_bytes(void) { return (int)sizeof(REAL); }

int moe_oracle_num_threads(void) {
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}

/* Strict total order used for selection: expert a ranks before expert b when its
 * logit is larger, or when the logits compare equal and a has the lower index.
 * The comparison is on the raw fp32 logits (softmax is increasing, so this is the
 * order of the probabilities, without depending on how exp rounds). */
static inline int ranks_before(const float *l, int a, int b) {
    return l[a] > l[b] || (l[a] == l[b] && a < b);
}

/* Router for one token: softmax over E logits, the k best experts in rank order,
 * and their probabilities renormalised to sum to one.
 *   logits [E] f32 -> ids [k] i32 (rank order), w [k] REAL.
 * scratch p [E] REAL, taken [E] bytes. */
static void route_token(const float *l, int E, int k, int32_t *ids, REAL *w, REAL *p, unsigned char *taken) {
    /* softmax: p_e = exp(l_e - m) / sum_e' exp(l_e' - m), sums in ascending e */
    float m = l[0];
    for (int e = 1; e < E; ++e)
        if (l[e] > m) m = l[e];
    REAL S = 0;
    for (int e = 0; e < E; ++e) {
        p[e] = real_exp((REAL)l[e] - (REAL)m);
        S += p[e];
    }
    for (int e = 0; e < E; ++e) p[e] = p[e] / S;
    /* selection: k passes, each picking the best expert not yet taken */
    memset(taken, 0, (size_t)E);
    for (int j = 0; j < k; ++j) {
        int best = -1;
        for (int e = 0; e < E; ++e) {
            if (taken[e]) continue;
            if (best < 0 || ranks_before(l, e, best)) best = e;
        }
        taken[best] = 1;
        ids[j] = best;
    }
    /* renormalise over the selected experts, ascending rank */
    REAL D = 0;
    for (int j = 0; j < k; ++j) D += p[ids[j]];
    for (int j = 0; j < k; ++j) w[j] = p[ids[j]] / D;
}

/* Router for a batch.  router_logits [T,E] f32 -> topk_ids [T,k] i32, topk_w [T,k] REAL. */
int moe_oracle_route(const float *router_logits, int T, int E, int k, int32_t *topk_ids, REAL *topk_w) {
    if (T < 0 || E < 1 || k < 1 || k > E) return ORACLE_ERR_ARG;
    REAL *p = (REAL *)malloc(sizeof(REAL) * (size_t)E);
    unsigned char *taken = (unsigned char *)malloc((size_t)E);
    if (!p || !taken) { free(p); free(taken); return ORACLE_ERR_NOMEM; }
    for (int t = 0; t < T; ++t)
        route_token(router_logits + (size_t)t * E, E, k, topk_ids + (size_t)t * k, topk_w + (size_t)t * k, p, taken);
    free(p);
    free(taken);
    return ORACLE_OK;
}

/* ---- Grouped sigmoid router ("DeepSeek-V3 style, top-8 routing", Sec. 4.5) -------------------------------
 * The paper names the style without its formula; the build's reading is the routing published with
 * DeepSeek-V3, restated here with every constant as a parameter:
 *   score_e  = sigmoid(logit_e)                                    (the weight an expert gets if chosen)
 *   choice_e = score_e + bias_e                                    (used for selection only)
 *   the E experts form n_group contiguous groups of G = E / n_group; a group's score is the sum of its two
 *   largest choice values (the single value when G = 1); the topk_group best groups stay eligible;
 *   the k eligible experts with the largest choice values are selected, in rank order;
 *   w_j = score_{id_j} / (sum over the selected, in rank order) * route_scale.
 * Ties (groups and experts) go to the lower index.
 * Selection is an integer decision taken from floating-point values, so it is defined in ONE arithmetic,
 * binary32, for both builds of this file and for the CUDA kernel (which restates it on its own): every
 * operation below is a single correctly rounded IEEE operation (fmaf counts as one), exp included, which is
 * evaluated by the fixed recipe of exp_fixed.  Only the final division and scaling use REAL. */
typedef struct {
    int n_group, topk_group;
    const float *bias; /* [E] or NULL */
    float scale;
} GroupedRouter;

/* e^x in binary32 by a fixed sequence of correctly rounded operations (within 2 ulp of the true value):
 * x is clamped to [-87, 88]; n = nearest integer (ties to even) of x * log2(e); r = x - n * ln 2 with ln 2 in
 * two parts; e^r by the degree-7 Taylor polynomial in Horner form; the result is that times 2^n. */
static float exp_fixed(float x) {
    if (x < -87.0f) x = -87.0f;
    if (x > 88.0f) x = 88.0f;
    const float n = rintf(x * 1.44269502f);
    float r = fmaf(n, -0.693145752f, x);
    r = fmaf(n, -1.42860677e-06f, r);
    float p = 1.98412701e-04f;            /* 1/5040 */
    p = fmaf(p, r, 1.38888892e-03f);      /* 1/720 */
    p = fmaf(p, r, 8.33333377e-03f);      /* 1/120 */
    p = fmaf(p, r, 4.16666679e-02f);      /* 1/24 */
    p = fmaf(p, r, 1.66666672e-01f);      /* 1/6 */
    p = fmaf(p, r, 0.5f);
    p = fmaf(p, r, 1.0f);
    p = fmaf(p, r, 1.0f);
    return p * ldexpf(1.0f, (int)n);      /* 2^n is exact for n in [-126, 127] */
}

static float sigmoid_fixed(float l) { return 1.0f / (1.0f + exp_fixed(-l)); }

float moe_oracle_exp_fixed(float x) { return exp_fixed(x); }
float moe_oracle_sigmoid_fixed(float l) { return sigmoid_fixed(l); }

/* scratch: score [E], choice [E] floats; eligible [n_group], taken [E] bytes */
static void route_token_grouped(const float *l, int E, int k, const GroupedRouter *g, int32_t *ids, REAL *w, float *score,
                                float *choice, unsigned char *eligible, unsigned char *taken) {
    const int G = E / g->n_group;
    for (int e = 0; e < E; ++e) {
        score[e] = sigmoid_fixed(l[e]);
        choice[e] = g->bias ? score[e] + g->bias[e] : score[e];
    }
    /* group scores, then topk_group passes each picking the best group not yet eligible */
    float gscore[256];
    for (int q = 0; q < g->n_group; ++q) {
        float t1 = -INFINITY, t2 = -INFINITY; /* the two largest choice values of the group */
        for (int e = q * G; e < (q + 1) * G; ++e) {
            if (choice[e] > t1) { t2 = t1; t1 = choice[e]; }
            else if (choice[e] > t2) t2 = choice[e];
        }
        gscore[q] = G >= 2 ? t1 + t2 : t1;
        eligible[q] = 0;
    }
    for (int j = 0; j < g->topk_group; ++j) {
        int best = -1;
        for (int q = 0; q < g->n_group; ++q) {
            if (eligible[q]) continue;
            if (best < 0 || gscore[q] > gscore[best]) best = q; /* strict >: ties keep the lower index */
        }
        eligible[best] = 1;
    }
    memset(taken, 0, (size_t)E);
    for (int j = 0; j < k; ++j) {
        int best = -1;
        for (int e = 0; e < E; ++e) {
            if (taken[e] || !eligible[e / G]) continue;
            if (best < 0 || choice[e] > choice[best]) best = e;
        }
        taken[best] = 1;
        ids[j] = best;
    }
    float D = 0;
    for (int j = 0; j < k; ++j) D = D + score[ids[j]];
    for (int j = 0; j < k; ++j) w[j] = (REAL)score[ids[j]] / (REAL)D * (REAL)g->scale;
}

static int grouped_router_ok(int E, int k, int n_group, int topk_group) {
    return n_group >= 1 && n_group <= 256 && E % n_group == 0 && topk_group >= 1 && topk_group <= n_group &&
           (long)topk_group * (E / n_group) >= k;
}

/* Grouped router for a batch: router_logits [T,E] f32, bias [E] f32 or NULL -> topk_ids [T,k], topk_w [T,k] REAL. */
int moe_oracle_route_grouped(const float *router_logits, const float *bias, int T, int E, int k, int n_group, int topk_group,
                             float scale, int32_t *topk_ids, REAL *topk_w) {
    if (T < 0 || E < 1 || k < 1 || k > E || !grouped_router_ok(E, k, n_group, topk_group)) return ORACLE_ERR_ARG;
    float *score = (float *)malloc(sizeof(float) * 2 * (size_t)E);
    unsigned char *flags = (unsigned char *)malloc((size_t)E + 256);
    if (!score || !flags) { free(score); free(flags); return ORACLE_ERR_NOMEM; }
    const GroupedRouter g = {n_group, topk_group, bias, scale};
    for (int t = 0; t < T; ++t)
        route_token_grouped(router_logits + (size_t)t * E, E, k, &g, topk_ids + (size_t)t * k, topk_w + (size_t)t * k, score,
                            score + E, flags + E, flags);
    free(score);
    free(flags);
    return ORACLE_OK;
}

/* Stable counting sort of the A = T*k assignments by expert ("sort-scatter").
 * Flat assignment index a = t*k + j.
 *   expert_offsets [E+1]: exclusive prefix sum of the per-expert counts
 *   flat_to_sorted [A]  : position of assignment a in expert-contiguous order
 *   sorted_to_flat [A]  : its inverse
 * Within an expert, assignments keep their flat order. */
int moe_oracle_permute(const int32_t *topk_ids, int T, int k, int E, int32_t *expert_offsets,
                       int32_t *sorted_to_flat, int32_t *flat_to_sorted) {
    if (T < 0 || E < 1 || k < 1) return ORACLE_ERR_ARG;
    const long A = (long)T * k;
    for (int e = 0; e <= E; ++e) expert_offsets[e] = 0;
    for (long a = 0; a < A; ++a) {
        if (topk_ids[a] < 0 || topk_ids[a] >= E) return ORACLE_ERR_ARG;
        expert_offsets[topk_ids[a] + 1] += 1; /* counts, shifted by one */
    }
    for (int e = 0; e < E; ++e) expert_offsets[e + 1] += expert_offsets[e];
    int32_t *next = (int32_t *)malloc(sizeof(int32_t) * (size_t)E);
    if (!next) return ORACLE_ERR_NOMEM;
    for (int e = 0; e < E; ++e) next[e] = expert_offsets[e];
    for (long a = 0; a < A; ++a) {
        int32_t pos = next[topk_ids[a]]++;
        flat_to_sorted[a] = pos;
        sorted_to_flat[pos] = (int32_t)a;
    }
    free(next);
    return ORACLE_OK;
}

/* One expert applied to one token row (gate/up projections, SiLU, down projection):
 *   g_i = sum_h x_h * w13[i,h],  u_i = sum_h x_h * w13[I+i,h],
 *   s_i = g_i / (1 + exp(-g_i)) * u_i,
 *   y_n = sum_i s_i * w2[n,i].
 * x_row [H] bf16, w13_e [2I,H] bf16, w2_e [H,I] bf16 -> y [H] REAL; scratch s [I] REAL.
 * Nothing is rounded to bf16 on the way. */
static void expert_ffn_row(const uint16_t *x_row, const uint16_t *w13_e, const uint16_t *w2_e, int H, int I, REAL *y, REAL *s) {
    for (int i = 0; i < I; ++i) {
        const uint16_t *wg = w13_e + (size_t)i * H;
        const uint16_t *wu = w13_e + (size_t)(I + i) * H;
        REAL g = 0, u = 0;
        for (int h = 0; h < H; ++h) {
            REAL xv = bf16_to_real(x_row[h]);
            g += xv * bf16_to_real(wg[h]);
            u += xv * bf16_to_real(wu[h]);
        }
        s[i] = g / ((REAL)1 + real_exp(-g)) * u;
    }
    for (int n = 0; n < H; ++n) {
        const uint16_t *wd = w2_e + (size_t)n * I;
        REAL acc = 0;
        for (int i = 0; i < I; ++i) acc += s[i] * bf16_to_real(wd[i]);
        y[n] = acc;
    }
}

int moe_oracle_expert_ffn(const uint16_t *x_row, const uint16_t *w13_e, const uint16_t *w2_e, int H, int I, REAL *y) {
    if (H < 1 || I < 1) return ORACLE_ERR_ARG;
    REAL *s = (REAL *)malloc(sizeof(REAL) * (size_t)I);
    if (!s) return ORACLE_ERR_NOMEM;
    expert_ffn_row(x_row, w13_e, w2_e, H, I, y, s);
    free(s);
    return ORACLE_OK;
}

/* The layer for a chosen list of tokens, with the experts given as a table of
 * per-expert pointers (an entry may be NULL when no listed token routes to it, so a
 * caller can keep only the needed experts in host memory).
 *   x [T,H] bf16, router_logits [T,E] f32, w13_ptrs[e] -> [2I,H] bf16, w2_ptrs[e] -> [H,I] bf16,
 *   tokens [n_tokens] (indices into [0,T)), out [n_tokens,H] REAL.
 * out[i,:] = sum_{j ascending} topk_w[t,j] * expert_{ids[t,j]}(x[t,:]),  t = tokens[i]. */
static int forward_tokens(const uint16_t *x, const float *router_logits, const uint16_t *const *w13_ptrs,
                          const uint16_t *const *w2_ptrs, int T, int H, int I, int E, int k, const int32_t *tokens,
                          int n_tokens, int skip_missing, const GroupedRouter *grouped, REAL *out) {
    if (T < 0 || H < 1 || I < 1 || E < 1 || k < 1 || k > E || n_tokens < 0) return ORACLE_ERR_ARG;
    if (grouped && !grouped_router_ok(E, k, grouped->n_group, grouped->topk_group)) return ORACLE_ERR_ARG;
    int status = ORACLE_OK;
#pragma omp parallel
    {
        REAL *p = (REAL *)malloc(sizeof(REAL) * (size_t)E);
        unsigned char *taken = (unsigned char *)malloc((size_t)E);
        int32_t *ids = (int32_t *)malloc(sizeof(int32_t) * (size_t)k);
        REAL *w = (REAL *)malloc(sizeof(REAL) * (size_t)k);
        REAL *s = (REAL *)malloc(sizeof(REAL) * (size_t)I);
        REAL *y = (REAL *)malloc(sizeof(REAL) * (size_t)H);
        float *gs = (float *)malloc(sizeof(float) * 2 * (size_t)E);      /* grouped router: score, choice */
        unsigned char *elig = (unsigned char *)malloc(256);             /* grouped router: eligible groups */
        if (!p || !taken || !ids || !w || !s || !y || !gs || !elig) {
#pragma omp critical
            status = ORACLE_ERR_NOMEM;
        } else {
#pragma omp for schedule(dynamic, 1)
            for (int i = 0; i < n_tokens; ++i) {
                const int t = tokens[i];
                REAL *o = out + (size_t)i * H;
                for (int n = 0; n < H; ++n) o[n] = 0;
                if (t < 0 || t >= T) {
#pragma omp critical
                    status = ORACLE_ERR_ARG;
                    continue;
                }
                if (grouped)
                    route_token_grouped(router_logits + (size_t)t * E, E, k, grouped, ids, w, gs, gs + E, elig, taken);
                else
                    route_token(router_logits + (size_t)t * E, E, k, ids, w, p, taken);
                for (int j = 0; j < k; ++j) {
                    const int e = ids[j];
                    if (!w13_ptrs[e] || !w2_ptrs[e]) {
                        if (skip_missing) continue; /* expert not resident here: it contributes nothing */
#pragma omp critical
                        status = ORACLE_ERR_MISSING_EXPERT;
                        continue;
                    }
                    expert_ffn_row(x + (size_t)t * H, w13_ptrs[e], w2_ptrs[e], H, I, y, s);
                    for (int n = 0; n < H; ++n) o[n] += w[j] * y[n];
                }
            }
        }
        free(p); free(taken); free(ids); free(w); free(s); free(y); free(gs); free(elig);
    }
    return status;
}

int moe_oracle_forward_sampled(const uint16_t *x, const float *router_logits, const uint16_t *const *w13_ptrs,
                               const uint16_t *const *w2_ptrs, int T, int H, int I, int E, int k,
                               const int32_t *tokens, int n_tokens, REAL *out) {
    return forward_tokens(x, router_logits, w13_ptrs, w2_ptrs, T, H, I, E, k, tokens, n_tokens, 0, NULL, out);
}

/* The same with the grouped sigmoid router (bias [E] f32 or NULL). */
int moe_oracle_forward_sampled_grouped(const uint16_t *x, const float *router_logits, const float *bias, int n_group,
                                       int topk_group, float scale, const uint16_t *const *w13_ptrs,
                                       const uint16_t *const *w2_ptrs, int T, int H, int I, int E, int k,
                                       const int32_t *tokens, int n_tokens, REAL *out) {
    const GroupedRouter g = {n_group, topk_group, bias, scale};
    return forward_tokens(x, router_logits, w13_ptrs, w2_ptrs, T, H, I, E, k, tokens, n_tokens, 0, &g, out);
}

/* The layer restricted to the experts resident on one device (the paper's kernel computes "32 local
 * experts" of 256, Sec. 4.5): routing is over all E experts, but only assignments whose expert lies in
 * [local_offset, local_offset + n_local) are evaluated; the others contribute nothing, and the routing
 * weights are NOT renormalised over the local ones, so the partial outputs of devices that partition
 * the experts add up to the full layer.
 *   w13_local [n_local,2I,H] bf16, w2_local [n_local,H,I] bf16 -> out [T,H] REAL. */
int moe_oracle_forward_local(const uint16_t *x, const float *router_logits, const uint16_t *w13_local,
                             const uint16_t *w2_local, int T, int H, int I, int E, int k, int local_offset, int n_local,
                             REAL *out) {
    if (T < 0 || H < 1 || I < 1 || E < 1 || k < 1 || k > E || local_offset < 0 || n_local < 0 || local_offset + n_local > E)
        return ORACLE_ERR_ARG;
    const uint16_t **p13 = (const uint16_t **)calloc((size_t)E, sizeof(void *));
    const uint16_t **p2 = (const uint16_t **)calloc((size_t)E, sizeof(void *));
    int32_t *tokens = (int32_t *)malloc(sizeof(int32_t) * (size_t)(T > 0 ? T : 1));
    int status = ORACLE_ERR_NOMEM;
    if (p13 && p2 && tokens) {
        for (int l = 0; l < n_local; ++l) {
            p13[local_offset + l] = w13_local + (size_t)l * 2 * I * H;
            p2[local_offset + l] = w2_local + (size_t)l * H * I;
        }
        for (int t = 0; t < T; ++t) tokens[t] = t;
        status = forward_tokens(x, router_logits, p13, p2, T, H, I, E, k, tokens, T, 1, NULL, out);
    }
    free(p13); free(p2); free(tokens);
    return status;
}

/* Sort-scatter restricted to the local experts: a stable counting sort of the assignments whose
 * expert is local, by local expert index; dropped assignments get flat_to_sorted = -1, and the tail
 * of sorted_to_flat past expert_offsets[n_local] is -1. */
int moe_oracle_permute_local(const int32_t *topk_ids, int T, int k, int local_offset, int n_local,
                             int32_t *expert_offsets, int32_t *sorted_to_flat, int32_t *flat_to_sorted) {
    if (T < 0 || k < 1 || n_local < 0 || local_offset < 0) return ORACLE_ERR_ARG;
    const long A = (long)T * k;
    for (int e = 0; e <= n_local; ++e) expert_offsets[e] = 0;
    for (long a = 0; a < A; ++a) {
        const int l = topk_ids[a] - local_offset;
        if (l >= 0 && l < n_local) expert_offsets[l + 1] += 1;
    }
    for (int e = 0; e < n_local; ++e) expert_offsets[e + 1] += expert_offsets[e];
    int32_t *next = (int32_t *)malloc(sizeof(int32_t) * (size_t)(n_local > 0 ? n_local : 1));
    if (!next) return ORACLE_ERR_NOMEM;
    for (int e = 0; e < n_local; ++e) next[e] = expert_offsets[e];
    for (long a = 0; a < A; ++a) sorted_to_flat[a] = -1;
    for (long a = 0; a < A; ++a) {
        const int l = topk_ids[a] - local_offset;
        if (l >= 0 && l < n_local) {
            const int32_t pos = next[l]++;
            flat_to_sorted[a] = pos;
            sorted_to_flat[pos] = (int32_t)a;
        } else {
            flat_to_sorted[a] = -1;
        }
    }
    free(next);
    return ORACLE_OK;
}

/* The whole layer on contiguous weights: w13 [E,2I,H] bf16, w2 [E,H,I] bf16 -> out [T,H] REAL. */
int moe_oracle_forward(const uint16_t *x, const float *router_logits, const uint16_t *w13, const uint16_t *w2,
                       int T, int H, int I, int E, int k, REAL *out) {
    if (T < 0 || H < 1 || I < 1 || E < 1 || k < 1 || k > E) return ORACLE_ERR_ARG;
    const uint16_t **p13 = (const uint16_t **)malloc(sizeof(void *) * (size_t)E);
    const uint16_t **p2 = (const uint16_t **)malloc(sizeof(void *) * (size_t)E);
    int32_t *tokens = (int32_t *)malloc(sizeof(int32_t) * (size_t)(T > 0 ? T : 1));
    int status = ORACLE_ERR_NOMEM;
    if (p13 && p2 && tokens) {
        for (int e = 0; e < E; ++e) {
            p13[e] = w13 + (size_t)e * 2 * I * H;
            p2[e] = w2 + (size_t)e * H * I;
        }
        for (int t = 0; t < T; ++t) tokens[t] = t;
        status = forward_tokens(x, router_logits, p13, p2, T, H, I, E, k, tokens, T, 0, NULL, out);
    }
    free(p13); free(p2); free(tokens);
    return status;
}

/* The two halves of the layer around the sort-scatter, exposed so that tests can
 * compare the CUDA path's intermediates in expert-contiguous order:
 *   h [A,I]  = SiLU(gate) * up   per sorted assignment row,
 *   y [A,H]  = down projection   per sorted assignment row.
 * Row r of either belongs to flat assignment sorted_to_flat[r]. */
int moe_oracle_sorted_intermediates(const uint16_t *x, const uint16_t *w13, const uint16_t *w2, const int32_t *topk_ids,
                                    const int32_t *sorted_to_flat, int T, int H, int I, int E, int k, REAL *h, REAL *y) {
    if (T < 0 || H < 1 || I < 1 || E < 1 || k < 1) return ORACLE_ERR_ARG;
    const long A = (long)T * k;
#pragma omp parallel for schedule(dynamic, 1)
    for (long r = 0; r < A; ++r) {
        const int a = sorted_to_flat[r];
        const int t = a / k, e = topk_ids[a];
        const uint16_t *xr = x + (size_t)t * H;
        const uint16_t *w13_e = w13 + (size_t)e * 2 * I * H;
        const uint16_t *w2_e = w2 + (size_t)e * H * I;
        REAL *hr = h + (size_t)r * I;
        for (int i = 0; i < I; ++i) {
            REAL g = 0, u = 0;
            for (int c = 0; c < H; ++c) {
                REAL xv = bf16_to_real(xr[c]);
                g += xv * bf16_to_real(w13_e[(size_t)i * H + c]);
                u += xv * bf16_to_real(w13_e[(size_t)(I + i) * H + c]);
            }
            hr[i] = g / ((REAL)1 + real_exp(-g)) * u;
        }
        for (int n = 0; n < H; ++n) {
            REAL acc = 0;
            for (int i = 0; i < I; ++i) acc += hr[i] * bf16_to_real(w2_e[(size_t)n * I + i]);
            y[(size_t)r * H + n] = acc;
        }
    }
    return ORACLE_OK;
}

/* ---- FP8 block-scaled weights -------------------------------------------------------------------
 * The paper's workload stores the expert weights in FP8 ("FP8 MoE", Table 2; Sec. 4.5), and its kernel
 * feeds 16-bit tensor-core tiles, so the stored weights are converted and rescaled on the way in.  The
 * build's reading of the storage format: OCP E4M3 codes (1 sign, 4 exponent bits with bias 7, 3 mantissa
 * bits; no infinities, S.1111.111 is NaN) with one fp32 scale per 128 x 128 block of each expert's weight
 * matrix; the weight a code stands for is  decode(code) * scale[row / 128][col / 128].  Activations stay
 * bf16.  Everything else (router, sort-scatter, SwiGLU, combine) is unchanged. */
static inline REAL e4m3_decode(uint8_t b) {
    const int sign = b >> 7, e = (b >> 3) & 15, m = b & 7;
    REAL v;
    if (e == 15 && m == 7) v = (REAL)NAN;
    else if (e == 0) v = (REAL)m / (REAL)8 * (REAL)0.015625;                 /* subnormal: m/8 * 2^-6 */
    else v = ((REAL)1 + (REAL)m / (REAL)8) * (REAL)ldexp(1.0, e - 7);        /* (1 + m/8) * 2^(e-7) */
    return sign ? -v : v;
}

float moe_oracle_e4m3_decode(uint8_t code) { return (float)e4m3_decode(code); }

/* One expert with FP8 block-scaled weights applied to one token row.
 *   w13q_e [2I,H] codes, w13s_e [2I/128, H/128] scales; w2q_e [H,I] codes, w2s_e [H/128, I/128] scales. */
static void expert_ffn_row_fp8w(const uint16_t *x_row, const uint8_t *w13q_e, const float *w13s_e, const uint8_t *w2q_e,
                                const float *w2s_e, int H, int I, REAL *y, REAL *s) {
    const int hb = H / 128, ib = I / 128;
    for (int i = 0; i < I; ++i) {
        REAL g = 0, u = 0;
        for (int h = 0; h < H; ++h) {
            const REAL xv = bf16_to_real(x_row[h]);
            const REAL wg = e4m3_decode(w13q_e[(size_t)i * H + h]) * (REAL)w13s_e[(size_t)(i / 128) * hb + h / 128];
            const REAL wu = e4m3_decode(w13q_e[(size_t)(I + i) * H + h]) * (REAL)w13s_e[(size_t)((I + i) / 128) * hb + h / 128];
            g += xv * wg;
            u += xv * wu;
        }
        s[i] = g / ((REAL)1 + real_exp(-g)) * u;
    }
    for (int n = 0; n < H; ++n) {
        REAL acc = 0;
        for (int i = 0; i < I; ++i)
            acc += s[i] * (e4m3_decode(w2q_e[(size_t)n * I + i]) * (REAL)w2s_e[(size_t)(n / 128) * ib + i / 128]);
        y[n] = acc;
    }
}

/* The whole layer with FP8 block-scaled weights: w13_q [E,2I,H] codes, w13_scale [E,2I/128,H/128] f32,
 * w2_q [E,H,I] codes, w2_scale [E,H/128,I/128] f32 -> out [T,H] REAL.  H and I must be multiples of 128. */
int moe_oracle_forward_fp8w(const uint16_t *x, const float *router_logits, const uint8_t *w13_q, const float *w13_scale,
                            const uint8_t *w2_q, const float *w2_scale, int T, int H, int I, int E, int k, REAL *out) {
    if (T < 0 || H < 128 || I < 128 || H % 128 || I % 128 || E < 1 || k < 1 || k > E) return ORACLE_ERR_ARG;
    int status = ORACLE_OK;
    const size_t n13 = (size_t)2 * I * H, n2 = (size_t)H * I;
    const size_t s13 = (size_t)(2 * I / 128) * (H / 128), s2 = (size_t)(H / 128) * (I / 128);
#pragma omp parallel
    {
        REAL *p = (REAL *)malloc(sizeof(REAL) * (size_t)E);
        unsigned char *taken = (unsigned char *)malloc((size_t)E);
        int32_t *ids = (int32_t *)malloc(sizeof(int32_t) * (size_t)k);
        REAL *w = (REAL *)malloc(sizeof(REAL) * (size_t)k);
        REAL *s = (REAL *)malloc(sizeof(REAL) * (size_t)I);
        REAL *y = (REAL *)malloc(sizeof(REAL) * (size_t)H);
        if (!p || !taken || !ids || !w || !s || !y) {
#pragma omp critical
            status = ORACLE_ERR_NOMEM;
        } else {
#pragma omp for schedule(dynamic, 1)
            for (int t = 0; t < T; ++t) {
                REAL *o = out + (size_t)t * H;
                for (int n = 0; n < H; ++n) o[n] = 0;
                route_token(router_logits + (size_t)t * E, E, k, ids, w, p, taken);
                for (int j = 0; j < k; ++j) {
                    const int e = ids[j];
                    expert_ffn_row_fp8w(x + (size_t)t * H, w13_q + e * n13, w13_scale + e * s13, w2_q + e * n2,
                                        w2_scale + e * s2, H, I, y, s);
                    for (int n = 0; n < H; ++n) o[n] += w[j] * y[n];
                }
            }
        }
        free(p); free(taken); free(ids); free(w); free(s); free(y);
    }
    return status;
}

/* ---- MX FP8: weights AND activations in 8 bits, one power-of-two scale per 32 elements ---------------
 * The paper's MoE workload is an FP8 one ("FP8 MoE", Table 2; Sec. 4.5 names the cost of FP8 packing and
 * scaling).  It does not fix the scaling granularity.  The build's reading for a path whose products run
 * on the tensor cores in 8 bits is the OCP Microscaling format MXFP8: E4M3 element codes and, for every
 * 32 consecutive elements along the contraction dimension, one E8M0 scale byte b standing for 2^(b-127)
 * (b = 255 is NaN).  A stored value is decode(code) * 2^(b-127).
 *
 * Quantising 32 values v (MX specification, "conversion to MX formats"):
 *     shared exponent  s = floor(log2(max|v|)) - 8     (8 = exponent of the largest E4M3 binade),
 *     scale byte       b = clamp(s + 127, 0, 254),
 *     code_i           = E4M3 of v_i / 2^(b-127), round to nearest even, values beyond +-448 saturate.
 * An all-zero block gets b = 0; a block holding an infinity or a NaN gets b = 255 and NaN codes.
 *
 * The layer: the expert weights arrive quantised (inputs); the token rows x are quantised along H before
 * the gate/up projections, and h = SiLU(gate) * up is quantised along I before the down projection, both
 * with the rule above; every dot product is the plain sum, in index order, of products of stored values. */
static inline REAL e8m0_decode(uint8_t b) { return b == 255 ? (REAL)NAN : (REAL)ldexp(1.0, (int)b - 127); }

/* E4M3 code of v: round to nearest, ties to the even code, finite values beyond the largest magnitude
 * (448) saturate to it, NaN gives the NaN code. */
static uint8_t e4m3_encode(double v) {
    const uint8_t sign = signbit(v) ? 0x80 : 0;
    const double a = fabs(v);
    if (isnan(a)) return (uint8_t)(sign | 0x7F);
    if (a >= 448.0) return (uint8_t)(sign | 0x7E);
    if (a < 0.015625) return (uint8_t)(sign | (uint8_t)rint(a * 512.0)); /* multiples of 2^-9; 8 is the first normal */
    int ex;
    const double m = frexp(a, &ex);                  /* a = m * 2^ex, m in [0.5, 1) */
    int E = ex - 1;                                  /* a = (2m) * 2^E, 2m in [1, 2) */
    int mant = (int)rint((2.0 * m - 1.0) * 8.0);     /* eighths above one, nearest even */
    if (mant == 8) { mant = 0; E += 1; }
    return (uint8_t)(sign | ((E + 7) << 3) | mant);
}

uint8_t moe_oracle_e4m3_encode(float v) { return e4m3_encode((double)v); }

/* Quantise one block of n values (n = 32 in the layer) to codes and one scale byte. */
static void mx_quantize_block(const REAL *v, int n, uint8_t *codes, uint8_t *scale_byte) {
    double amax = 0;
    int nonfinite = 0;
    for (int i = 0; i < n; ++i) {
        const double a = fabs((double)v[i]);
        if (!isfinite(a)) nonfinite = 1;
        else if (a > amax) amax = a;
    }
    if (nonfinite) {
        *scale_byte = 255;
        for (int i = 0; i < n; ++i) codes[i] = 0x7F;
        return;
    }
    int b = 0;
    if (amax > 0) {
        int ex;
        (void)frexp(amax, &ex);       /* floor(log2(amax)) = ex - 1 */
        b = (ex - 1) - 8 + 127;
        if (b < 0) b = 0;
        if (b > 254) b = 254;
    }
    *scale_byte = (uint8_t)b;
    for (int i = 0; i < n; ++i) codes[i] = e4m3_encode(ldexp((double)v[i], 127 - b)); /* division by 2^(b-127) is exact */
}

/* Rows of fp32 values [R, K] -> codes [R, K] and scale bytes [R, K/32]; K a multiple of 32. */
int moe_oracle_mx_quantize(const float *v, int R, int K, uint8_t *codes, uint8_t *scales) {
    if (R < 0 || K < 32 || K % 32) return ORACLE_ERR_ARG;
    REAL tmp[32];
    for (long r = 0; r < R; ++r)
        for (int b = 0; b < K / 32; ++b) {
            for (int i = 0; i < 32; ++i) tmp[i] = (REAL)v[(size_t)r * K + 32 * b + i];
            mx_quantize_block(tmp, 32, codes + (size_t)r * K + 32 * b, scales + (size_t)r * (K / 32) + b);
        }
    return ORACLE_OK;
}

static inline REAL mx_value(const uint8_t *codes, const uint8_t *scales, int i) {
    return e4m3_decode(codes[i]) * e8m0_decode(scales[i / 32]);
}

/* One expert with MX weights applied to one quantised token row.
 *   xq [H] codes, xs [H/32]; w13q_e [2I,H], w13s_e [2I,H/32]; w2q_e [H,I], w2s_e [H,I/32]
 *   -> y [H] REAL; s [I] REAL receives h before quantisation, hq [I] / hs [I/32] its quantised form. */
static void expert_ffn_row_mx(const uint8_t *xq, const uint8_t *xs, const uint8_t *w13q_e, const uint8_t *w13s_e,
                              const uint8_t *w2q_e, const uint8_t *w2s_e, int H, int I, REAL *y, REAL *s, uint8_t *hq,
                              uint8_t *hs) {
    for (int i = 0; i < I; ++i) {
        const uint8_t *gq = w13q_e + (size_t)i * H, *gs = w13s_e + (size_t)i * (H / 32);
        const uint8_t *uq = w13q_e + (size_t)(I + i) * H, *us = w13s_e + (size_t)(I + i) * (H / 32);
        REAL g = 0, u = 0;
        for (int c = 0; c < H; ++c) {
            const REAL xv = mx_value(xq, xs, c);
            g += xv * mx_value(gq, gs, c);
            u += xv * mx_value(uq, us, c);
        }
        s[i] = g / ((REAL)1 + real_exp(-g)) * u;
    }
    for (int b = 0; b < I / 32; ++b) mx_quantize_block(s + 32 * b, 32, hq + 32 * b, hs + b);
    for (int n = 0; n < H; ++n) {
        const uint8_t *dq = w2q_e + (size_t)n * I, *ds = w2s_e + (size_t)n * (I / 32);
        REAL acc = 0;
        for (int i = 0; i < I; ++i) acc += mx_value(hq, hs, i) * mx_value(dq, ds, i);
        y[n] = acc;
    }
}

/* The MX FP8 layer for a chosen list of tokens, with the experts given as tables of per-expert pointers
 * (an entry may be NULL when no listed token routes to it).  out [n_tokens,H] REAL; the optional
 * intermediates are indexed by (position in `tokens`) * k + j. */
static int forward_tokens_mx(const uint16_t *x, const float *router_logits, const uint8_t *const *w13q, const uint8_t *const *w13s,
                             const uint8_t *const *w2q, const uint8_t *const *w2s, int T, int H, int I, int E, int k,
                             const int32_t *tokens, int n_tokens, REAL *out, REAL *h_pre, uint8_t *h_q, uint8_t *h_s) {
    if (T < 0 || H < 32 || I < 32 || H % 32 || I % 32 || E < 1 || k < 1 || k > E || n_tokens < 0) return ORACLE_ERR_ARG;
    int status = ORACLE_OK;
#pragma omp parallel
    {
        REAL *p = (REAL *)malloc(sizeof(REAL) * (size_t)E);
        unsigned char *taken = (unsigned char *)malloc((size_t)E);
        int32_t *ids = (int32_t *)malloc(sizeof(int32_t) * (size_t)k);
        REAL *w = (REAL *)malloc(sizeof(REAL) * (size_t)k);
        REAL *s = (REAL *)malloc(sizeof(REAL) * (size_t)I);
        REAL *y = (REAL *)malloc(sizeof(REAL) * (size_t)H);
        REAL *xr = (REAL *)malloc(sizeof(REAL) * (size_t)H);
        uint8_t *xq = (uint8_t *)malloc((size_t)H), *xs = (uint8_t *)malloc((size_t)(H / 32));
        uint8_t *hq = (uint8_t *)malloc((size_t)I), *hs = (uint8_t *)malloc((size_t)(I / 32));
        if (!p || !taken || !ids || !w || !s || !y || !xr || !xq || !xs || !hq || !hs) {
#pragma omp critical
            status = ORACLE_ERR_NOMEM;
        } else {
#pragma omp for schedule(dynamic, 1)
            for (int n_i = 0; n_i < n_tokens; ++n_i) {
                const int t = tokens[n_i];
                REAL *o = out + (size_t)n_i * H;
                for (int n = 0; n < H; ++n) o[n] = 0;
                if (t < 0 || t >= T) {
#pragma omp critical
                    status = ORACLE_ERR_ARG;
                    continue;
                }
                route_token(router_logits + (size_t)t * E, E, k, ids, w, p, taken);
                for (int c = 0; c < H; ++c) xr[c] = bf16_to_real(x[(size_t)t * H + c]);
                for (int b = 0; b < H / 32; ++b) mx_quantize_block(xr + 32 * b, 32, xq + 32 * b, xs + b);
                for (int j = 0; j < k; ++j) {
                    const int e = ids[j];
                    if (!w13q[e] || !w13s[e] || !w2q[e] || !w2s[e]) {
#pragma omp critical
                        status = ORACLE_ERR_MISSING_EXPERT;
                        continue;
                    }
                    expert_ffn_row_mx(xq, xs, w13q[e], w13s[e], w2q[e], w2s[e], H, I, y, s, hq, hs);
                    const size_t a = (size_t)n_i * k + j;
                    if (h_pre) memcpy(h_pre + a * I, s, sizeof(REAL) * (size_t)I);
                    if (h_q) memcpy(h_q + a * I, hq, (size_t)I);
                    if (h_s) memcpy(h_s + a * (I / 32), hs, (size_t)(I / 32));
                    for (int n = 0; n < H; ++n) o[n] += w[j] * y[n];
                }
            }
        }
        free(p); free(taken); free(ids); free(w); free(s); free(y); free(xr); free(xq); free(xs); free(hq); free(hs);
    }
    return status;
}

int moe_oracle_forward_mxfp8_sampled(const uint16_t *x, const float *router_logits, const uint8_t *const *w13q,
                                     const uint8_t *const *w13s, const uint8_t *const *w2q, const uint8_t *const *w2s, int T,
                                     int H, int I, int E, int k, const int32_t *tokens, int n_tokens, REAL *out) {
    return forward_tokens_mx(x, router_logits, w13q, w13s, w2q, w2s, T, H, I, E, k, tokens, n_tokens, out, NULL, NULL, NULL);
}

/* The whole layer in MX FP8.  x [T,H] bf16, router_logits [T,E] f32, w13_q [E,2I,H] codes, w13_s [E,2I,H/32]
 * scale bytes, w2_q [E,H,I], w2_s [E,H,I/32] -> out [T,H] REAL.  Optional (may be NULL), per flat assignment
 * a = t*k + j:  h_pre [A,I] REAL = h before quantisation, h_q [A,I] codes, h_s [A,I/32] scale bytes.
 * H and I must be multiples of 32. */
int moe_oracle_forward_mxfp8(const uint16_t *x, const float *router_logits, const uint8_t *w13_q, const uint8_t *w13_s,
                             const uint8_t *w2_q, const uint8_t *w2_s, int T, int H, int I, int E, int k, REAL *out,
                             REAL *h_pre, uint8_t *h_q, uint8_t *h_s) {
    if (T < 0 || H < 32 || I < 32 || H % 32 || I % 32 || E < 1 || k < 1 || k > E) return ORACLE_ERR_ARG;
    const size_t n13 = (size_t)2 * I * H, n2 = (size_t)H * I;
    const size_t s13 = (size_t)2 * I * (H / 32), s2 = (size_t)H * (I / 32);
    const uint8_t **tab = (const uint8_t **)malloc(sizeof(void *) * 4 * (size_t)E);
    int32_t *tokens = (int32_t *)malloc(sizeof(int32_t) * (size_t)(T > 0 ? T : 1));
    int status = ORACLE_ERR_NOMEM;
    if (tab && tokens) {
        for (int e = 0; e < E; ++e) {
            tab[e] = w13_q + e * n13;
            tab[E + e] = w13_s + e * s13;
            tab[2 * E + e] = w2_q + e * n2;
            tab[3 * E + e] = w2_s + e * s2;
        }
        for (int t = 0; t < T; ++t) tokens[t] = t;
        status = forward_tokens_mx(x, router_logits, tab, tab + E, tab + 2 * E, tab + 3 * E, T, H, I, E, k, tokens, T, out,
                                   h_pre, h_q, h_s);
    }
    free(tab); free(tokens);
    return status;
}
