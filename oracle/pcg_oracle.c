/*
 * PCG verification oracle -- TEST INFRASTRUCTURE, NOT PRODUCT CODE.
 *
 * A plain, slow, double-precision CPU statement of the group-level verification
 * step of Principled Coarse-Graining (PCG) speculative decoding.  It exists so
 * that the CUDA library can be checked against something that can be compared
 * with the paper by eye.  Only the tests, the smoke check and the CPU-baseline
 * leg of the benchmark may call it; the product path never does, and this file
 * shares no code, header, table or helper with the CUDA sources.
 *
 * Letters.  The paper's body calls the target model q and the draft model p.
 * This file (like the library's C interface) uses the opposite, unambiguous
 * convention: p = TARGET token distribution, q = DRAFT token distribution,
 * P[g] = target coarse mass of group g, Q[g] = draft coarse mass of group g.
 * The semantics are the paper's: accept with probability min(1, target/draft)
 * (acceptance equation of Sec. 2.2), residual proportional to
 * (target - draft)_+ over groups (residual equation of Sec. 2.2).
 *
 * No blocking, fusion or reordering: sums run sequentially in index order, in
 * double precision, exactly as the definitions are written.
 *
 * Parity status.  Every function below is pinned by the CPU test-suite to
 * facts that do not come from this file (a library softmax, dense-matrix brute
 * force in exact rationals, the exactness proposition checked by enumeration,
 * a separately written token-level speculative-sampling verifier).  The
 * general-weights branches (coarse-graining, label draw, within-group draw)
 * and the constant acceptance bias are pinned with unequal hand-made weights
 * the same way (exact rationals, hand-written labels, the coupling identity,
 * min(Q, P + bias Q) on a grid of uniforms).  The thinning sampler of
 * pcg_oracle_verify_thinning is pinned by the laws the
 * paper states for it, measured over many seeded uniforms (kept group ~
 * normalised residual, emitted group ~ target coarse distribution, mean
 * number of trials = 1/TV, token ~ target-conditional), by its singleton-group
 * special case and by its fallback equalling the enumerated draw.  What can
 * NOT be pinned: draw-by-draw agreement with the authors' own program (none is
 * published, and how it maps random numbers to draws is not stated) -- for
 * that comparison alone: "parity unpinned"; agreement in distribution is what
 * is pinned.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

#define ORACLE_F32 0
#define ORACLE_BF16 1
#define ORACLE_F16 2

/* flag bits written per sequence */
#define ORACLE_FLAG_ZERO_RESIDUAL 2 /* reject taken but sum of (P-Q)_+ was <= 0 */
#define ORACLE_FLAG_THINNING_EXHAUSTED 8 /* every supplied thinning trial was turned down; enumerated draw used */

/* IEEE binary16 bit pattern to double, from the format's definition: 1 sign, 5 exponent (bias 15), 10 fraction bits. */
static double half_bits_to_double(uint16_t h) {
    int sign = h >> 15, ex = (h >> 10) & 0x1f, frac = h & 0x3ff;
    double v;
    if (ex == 0)
        v = ldexp((double)frac, -24); /* zero and subnormals: frac * 2^-10 * 2^-14 */
    else if (ex == 31)
        v = frac ? NAN : INFINITY;
    else
        v = ldexp(1.0 + (double)frac / 1024.0, ex - 15);
    return sign ? -v : v;
}

/* Widen one stored logit to double exactly (bf16 = upper 16 bits of a float). */
static double load_logit(const void *base, int dtype, int64_t idx) {
    if (dtype == ORACLE_F32) {
        return (double)((const float *)base)[idx];
    } else if (dtype == ORACLE_F16) {
        return half_bits_to_double(((const uint16_t *)base)[idx]);
    } else {
        uint32_t bits = ((uint32_t)((const uint16_t *)base)[idx]) << 16;
        float f;
        memcpy(&f, &bits, sizeof f);
        return (double)f;
    }
}

/*
 * Softmax with temperature: p(t) = exp(l_t/T - m) / sum_t' exp(l_t'/T - m),
 * m = max_t l_t/T.  The paper only says that the token distributions are the
 * models' distributions at inference temperature 0.8 (Sec. 3.1); the softmax
 * itself is the textbook one.
 */
static void softmax_row(const void *logits, int dtype, int64_t row, int V, double T, double *p) {
    int64_t off = row * (int64_t)V;
    double m = -INFINITY;
    for (int t = 0; t < V; ++t) {
        p[t] = load_logit(logits, dtype, off + t) / T;
        if (p[t] > m) m = p[t];
    }
    double Z = 0.0;
    for (int t = 0; t < V; ++t) {
        p[t] = exp(p[t] - m);
        Z += p[t];
    }
    for (int t = 0; t < V; ++t) p[t] /= Z;
}

/*
 * Equal-split coarse-graining (Sec. 2.2, the equal-split form of the
 * coarse-grained distributions):  P[g] = sum_{t in G_g} p(t) / N(t),
 * N(t) = number of groups that contain t.  With general weights (the weight
 * equation of Sec. 2.2) the term is p(t) * w[k] for the k-th stored (g,t) pair.
 */
static void coarse_grain(const double *p, int M, const int32_t *group_ptr, const int32_t *group_tok,
                         const int32_t *tok_degree, const double *weights, double *P) {
    for (int g = 0; g < M; ++g) {
        double s = 0.0;
        for (int32_t k = group_ptr[g]; k < group_ptr[g + 1]; ++k) {
            int32_t t = group_tok[k];
            s += weights ? p[t] * weights[k] : p[t] / (double)tok_degree[t];
        }
        P[g] = s;
    }
}

int pcg_oracle_softmax(const void *logits, int dtype, int64_t rows, int V, float temperature, double *out) {
    if (!logits || !out || rows < 0 || V < 1 || !(temperature > 0.0f)) return 1;
    for (int64_t r = 0; r < rows; ++r) softmax_row(logits, dtype, r, V, (double)temperature, out + r * V);
    return 0;
}

int pcg_oracle_group_probs(const void *logits, int dtype, int64_t rows, int V, float temperature, int M,
                           const int32_t *group_ptr, const int32_t *group_tok, const int32_t *tok_degree,
                           const double *weights, double *out) {
    if (!logits || !out || rows < 0 || V < 1 || M < 1 || !(temperature > 0.0f)) return 1;
    double *p = (double *)malloc(sizeof(double) * (size_t)V);
    if (!p) return 2;
    for (int64_t r = 0; r < rows; ++r) {
        softmax_row(logits, dtype, r, V, (double)temperature, p);
        coarse_grain(p, M, group_ptr, group_tok, tok_degree, weights, out + r * M);
    }
    free(p);
    return 0;
}

/*
 * Inverse-CDF draw over n non-negative masses w[0..n): returns the first index
 * whose inclusive running sum strictly exceeds u * total; if rounding leaves
 * none, the last index with positive mass.  *margin receives the distance, on
 * the u scale, from u to the nearer edge of the chosen bin (how far u would
 * have to move for the draw to change).  The paper fixes only the law of the
 * draw; this mapping from a uniform to the draw is the library's reading.
 */
static int inverse_cdf(const double *w, int n, double u, double *total_out, double *margin) {
    double total = 0.0;
    for (int k = 0; k < n; ++k) total += w[k];
    if (total_out) *total_out = total;
    double target = u * total, run = 0.0, lo = 0.0;
    int pick = -1, last_pos = -1;
    for (int k = 0; k < n; ++k) {
        if (w[k] > 0.0) last_pos = k;
        double next = run + w[k];
        if (pick < 0 && next > target) {
            pick = k;
            lo = run;
            run = next;
            break;
        }
        run = next;
    }
    if (pick < 0) {
        pick = last_pos;
        if (margin) *margin = 0.0;
        return pick;
    }
    if (margin) {
        double d_lo = target - lo, d_hi = run - target;
        if (pick == 0 || lo <= 0.0) d_lo = INFINITY; /* nothing below the first positive bin */
        double d = d_lo < d_hi ? d_lo : d_hi;
        *margin = total > 0.0 ? d / total : 0.0;
    }
    return pick;
}

/*
 * Group-label coupling (Sec. 2.2): the label of token x is drawn from w_{.,x} over S(x), the groups containing
 * x in ascending group id.  Equal split: j = min(floor(u N), N-1); general weights: inverse CDF over them.
 * Returns the group id; *margin receives the distance from u to the nearest point where the label changes.
 */
static int32_t draw_label(int32_t x, double u, const double *weights, const int32_t *rev_ptr, const int32_t *rev_grp,
                          const int32_t *rev_nz, double *margin) {
    int32_t N = rev_ptr[x + 1] - rev_ptr[x];
    int j;
    if (!weights) {
        double uj = u * (double)N;
        j = (int)floor(uj);
        if (j > N - 1) j = N - 1;
        if (margin) {
            double d = INFINITY;
            for (int e = 1; e < N; ++e) {
                double dd = fabs(u - (double)e / (double)N);
                if (dd < d) d = dd;
            }
            *margin = d;
        }
    } else {
        /* inverse CDF over the weights of x's groups, ascending group id */
        double *wx = (double *)malloc(sizeof(double) * (size_t)N);
        for (int e = 0; e < N; ++e) wx[e] = weights[rev_nz[rev_ptr[x] + e]];
        j = inverse_cdf(wx, N, u, NULL, margin);
        free(wx);
    }
    return rev_grp[rev_ptr[x] + j];
}

/*
 * One sequence of Algorithm 1 with the randomness supplied from outside.
 *
 * uniforms[i][0], i < K : group-label draw for drafted position i
 * uniforms[i][1], i < K : accept draw for drafted position i
 * uniforms[K][0]        : terminal group draw (residual or bonus)
 * uniforms[K][1]        : terminal within-group token draw
 *
 * Terminal group, two ways.  thin == NULL: enumerate the residual over all groups and invert its CDF with
 * uniforms[K][0].  thin != NULL ([B, n_trials, 3]): the thinning sampler of the paper
 * (Sec. 2.2), which never enumerates the groups.  Trial r uses thin[r][0] to draw a token y from the target
 * row by inverse CDF over the tokens taken in the order cand_order[0], cand_order[1], ... (a permutation of the tokens
 * supplied by the caller, NULL = ascending token id: the paper fixes the law y ~ target, which no order can change,
 * not how a uniform is mapped to y), thin[r][1] to draw y's label k ~ w_{.,y} (so that k ~ the target's coarse
 * distribution), and keeps k if thin[r][2] < [1 - draft mass(k) / target mass(k)]_+; otherwise the next trial
 * draws a new (y, k).  After all accepted positions (no rejection) there is no draft mass: the first candidate
 * is kept, which draws the bonus group from the target's coarse distribution.  The paper's sampler is not
 * bounded; here the trials are: if all n_trials candidates are turned down the group is drawn by the enumerated
 * inverse CDF with uniforms[K][0] instead (same law) and the sequence is flagged.  The token inside the kept
 * group is then drawn from the target-conditional with uniforms[K][1], as the thinning paragraph prescribes.
 *
 * rev_ptr/rev_grp is the reverse membership S(t) (groups containing t, in
 * ascending group id) built by the caller of verify_sequence from the CSR.
 */
static void verify_sequence(const void *target_logits, const void *draft_logits, int dtype, int64_t b, int K, int V,
                            double T, const int32_t *draft_tokens, int M, const int32_t *group_ptr,
                            const int32_t *group_tok, const int32_t *tok_degree, const double *weights,
                            const int32_t *rev_ptr, const int32_t *rev_grp, const int32_t *rev_nz,
                            const float *uniforms, const float *thin, int n_trials, const int32_t *cand_order,
                            double *pm, double accept_bias, int32_t *accept_len, int32_t *tokens, int32_t *groups,
                            int32_t *flags, int32_t *trials, double *margins, double *p, double *q, double *P,
                            double *Q, double *R) {
    const float *u = uniforms + b * (int64_t)(K + 1) * 2;
    int32_t *tok_out = tokens + b * (int64_t)(K + 1);
    int32_t *grp_out = groups + b * (int64_t)(K + 1);
    double *mg = margins ? margins + b * (int64_t)(K + 1) * 2 : NULL;
    for (int i = 0; i <= K; ++i) {
        tok_out[i] = -1;
        grp_out[i] = -1;
        if (mg) mg[2 * i] = mg[2 * i + 1] = INFINITY;
    }
    int32_t fl = 0;
    int n = K;
    int have_Q = 0;
    for (int i = 0; i < K; ++i) { /* the loop of Algorithm 1 */
        softmax_row(target_logits, dtype, b * (int64_t)(K + 1) + i, V, T, p);
        softmax_row(draft_logits, dtype, b * (int64_t)K + i, V, T, q);
        coarse_grain(p, M, group_ptr, group_tok, tok_degree, weights, P);
        coarse_grain(q, M, group_ptr, group_tok, tok_degree, weights, Q);
        /* group-label coupling (Sec. 2.2): K_i ~ w_{.,x} over S(x) */
        int32_t x = draft_tokens[b * (int64_t)K + i];
        int32_t g = draw_label(x, (double)u[2 * i], weights, rev_ptr, rev_grp, rev_nz, mg ? &mg[2 * i] : NULL);
        grp_out[i] = g;
        /* acceptance (Sec. 2.2): u < min(1, target mass / draft mass); a constant
           bias on the ratio (the SSD comparison system of Sec. 3.2) is 0 for PCG */
        double ratio = Q[g] > 0.0 ? P[g] / Q[g] : INFINITY;
        int accept = (P[g] >= Q[g]) || ((double)u[2 * i + 1] < ratio + accept_bias);
        if (mg) mg[2 * i + 1] = fabs((double)u[2 * i + 1] - (ratio + accept_bias));
        if (accept) {
            tok_out[i] = x; /* the draft token is kept on acceptance (end of Sec. 2.2) */
        } else {
            n = i;
            have_Q = 1;
            break;
        }
    }
    /* terminal draw at position n: residual if a rejection happened, bonus otherwise */
    if (!have_Q) {
        softmax_row(target_logits, dtype, b * (int64_t)(K + 1) + K, V, T, p);
        coarse_grain(p, M, group_ptr, group_tok, tok_degree, weights, P);
    }
    int gs = -1;
    double m_group = INFINITY; /* smallest margin over the decisions that led to the terminal group */
    if (thin) {
        const float *tu = thin + b * (int64_t)n_trials * 3;
        int used = 0;
        for (int t = 0; t < V; ++t) pm[t] = p[cand_order ? cand_order[t] : t]; /* target masses in candidate order */
        for (int r = 0; r < n_trials && gs < 0; ++r) {
            double m_tok = INFINITY, m_lab = INFINITY, m_keep = INFINITY;
            int y = inverse_cdf(pm, V, (double)tu[3 * r], NULL, &m_tok); /* y ~ target */
            if (cand_order) y = cand_order[y];
            int32_t k = draw_label(y, (double)tu[3 * r + 1], weights, rev_ptr, rev_grp, rev_nz, &m_lab); /* k ~ w_{.,y} */
            int keep = 1;
            if (have_Q) { /* thinning probability a(k) = [1 - draft mass / target mass]_+ */
                double a = P[k] > 0.0 ? 1.0 - Q[k] / P[k] : 0.0;
                if (a < 0.0) a = 0.0;
                keep = (double)tu[3 * r + 2] < a;
                m_keep = fabs((double)tu[3 * r + 2] - a);
            }
            if (m_tok < m_group) m_group = m_tok;
            if (m_lab < m_group) m_group = m_lab;
            if (m_keep < m_group) m_group = m_keep;
            used = r + 1;
            if (keep) gs = k;
        }
        if (trials) trials[b] = used;
        if (gs < 0) fl |= ORACLE_FLAG_THINNING_EXHAUSTED;
    }
    if (gs < 0) { /* enumerated residual over all groups, inverse CDF in group order */
        if (!have_Q) {
            for (int g = 0; g < M; ++g) R[g] = P[g];
        } else {
            for (int g = 0; g < M; ++g) R[g] = P[g] > Q[g] ? P[g] - Q[g] : 0.0;
        }
        double Z = 0.0;
        for (int g = 0; g < M; ++g) Z += R[g];
        if (!(Z > 0.0)) { /* cannot happen in exact arithmetic after a rejection */
            for (int g = 0; g < M; ++g) R[g] = P[g];
            fl |= ORACLE_FLAG_ZERO_RESIDUAL;
        }
        double m_enum = INFINITY;
        gs = inverse_cdf(R, M, (double)u[2 * K], NULL, &m_enum);
        if (m_enum < m_group) m_group = m_enum;
    }
    if (mg) mg[2 * K] = m_group;
    /* within-group conditional (Sec. 2.2): Pr(z = t | g*) = p(t) w_{g*,t} / P[g*] */
    int32_t lo = group_ptr[gs], hi = group_ptr[gs + 1];
    int len = hi - lo;
    double *w = (double *)malloc(sizeof(double) * (size_t)(len > 0 ? len : 1));
    for (int k = 0; k < len; ++k) {
        int32_t t = group_tok[lo + k];
        w[k] = weights ? p[t] * weights[lo + k] : p[t] / (double)tok_degree[t];
    }
    int kz = inverse_cdf(w, len, (double)u[2 * K + 1], NULL, mg ? &mg[2 * K + 1] : NULL);
    free(w);
    tok_out[n] = group_tok[lo + kz];
    grp_out[n] = gs;
    accept_len[b] = n;
    if (flags) flags[b] = fl;
}

/*
 * Batched verification.  Layouts (all row-major, contiguous):
 *   target_logits [B, K+1, V], draft_logits [B, K, V]  (float or bf16 bit patterns)
 *   draft_tokens [B, K], uniforms [B, K+1, 2] (float in [0,1))
 *   group_ptr [M+1], group_tok [nnz] ascending inside a group, tok_degree [V]
 *   weights: NULL for equal split, else [nnz] (one per stored pair, summing to 1 per token)
 * Outputs: accept_len [B], tokens [B, K+1], groups [B, K+1] (unused slots -1),
 *   flags [B] (may be NULL), margins [B, K+1, 2] doubles (may be NULL).
 * threads <= 0 means "all cores".  Returns 0, or non-zero on bad arguments.
 */
static int verify_batch(const void *target_logits, const void *draft_logits, int dtype, int B, int K, int V,
                        const int32_t *draft_tokens, int M, const int32_t *group_ptr, const int32_t *group_tok,
                        const int32_t *tok_degree, const double *weights, const float *uniforms, const float *thin,
                        int n_trials, const int32_t *cand_order, float temperature, double accept_bias,
                        int32_t *accept_len, int32_t *tokens, int32_t *groups, int32_t *flags, int32_t *trials,
                        double *margins, int threads) {
    if (!target_logits || !draft_logits || !draft_tokens || !group_ptr || !group_tok || !tok_degree || !uniforms ||
        !accept_len || !tokens || !groups)
        return 1;
    if (B < 0 || K < 1 || V < 1 || M < 1 || !(temperature > 0.0f)) return 1;
    int64_t nnz = group_ptr[M];
    /* reverse membership S(t), ascending group id, by counting sort over the CSR */
    int32_t *rev_ptr = (int32_t *)calloc((size_t)V + 1, sizeof(int32_t));
    int32_t *rev_grp = (int32_t *)malloc(sizeof(int32_t) * (size_t)(nnz > 0 ? nnz : 1));
    int32_t *rev_nz = (int32_t *)malloc(sizeof(int32_t) * (size_t)(nnz > 0 ? nnz : 1));
    int32_t *fill = (int32_t *)calloc((size_t)V, sizeof(int32_t));
    if (!rev_ptr || !rev_grp || !rev_nz || !fill) return 2;
    for (int64_t k = 0; k < nnz; ++k) {
        if (group_tok[k] < 0 || group_tok[k] >= V) return 3;
        rev_ptr[group_tok[k] + 1]++;
    }
    for (int t = 0; t < V; ++t) {
        if (rev_ptr[t + 1] != tok_degree[t] || tok_degree[t] < 1) return 3; /* N(t) must match and be >= 1 */
        rev_ptr[t + 1] += rev_ptr[t];
    }
    for (int g = 0; g < M; ++g)
        for (int32_t k = group_ptr[g]; k < group_ptr[g + 1]; ++k) {
            int32_t t = group_tok[k];
            rev_grp[rev_ptr[t] + fill[t]] = g;
            rev_nz[rev_ptr[t] + fill[t]] = k;
            fill[t]++;
        }
    for (int64_t k = 0; k < (int64_t)B * K; ++k)
        if (draft_tokens[k] < 0 || draft_tokens[k] >= V) return 4;
    /* the candidate order of the thinning sampler must be a permutation of the tokens */
    if (thin && cand_order) {
        int bad = 0;
        for (int t = 0; t < V; ++t) fill[t] = 0;
        for (int t = 0; t < V; ++t) {
            if (cand_order[t] < 0 || cand_order[t] >= V || fill[cand_order[t]]++) bad = 1;
        }
        if (bad) {
            free(rev_ptr);
            free(rev_grp);
            free(rev_nz);
            free(fill);
            return 5;
        }
    }
    int nthreads = threads;
#ifdef _OPENMP
    if (nthreads <= 0) nthreads = omp_get_max_threads();
#else
    nthreads = 1;
#endif
    int failed = 0;
#pragma omp parallel num_threads(nthreads)
    {
        double *p = (double *)malloc(sizeof(double) * (size_t)V);
        double *q = (double *)malloc(sizeof(double) * (size_t)V);
        double *P = (double *)malloc(sizeof(double) * (size_t)M);
        double *Q = (double *)malloc(sizeof(double) * (size_t)M);
        double *R = (double *)malloc(sizeof(double) * (size_t)M);
        double *pm = (double *)malloc(sizeof(double) * (size_t)V);
        if (!p || !q || !P || !Q || !R || !pm) {
#pragma omp atomic write
            failed = 1;
        } else {
#pragma omp for schedule(dynamic, 1)
            for (int b = 0; b < B; ++b)
                verify_sequence(target_logits, draft_logits, dtype, b, K, V, (double)temperature, draft_tokens, M,
                                group_ptr, group_tok, tok_degree, weights, rev_ptr, rev_grp, rev_nz, uniforms,
                                thin, n_trials, cand_order, pm, accept_bias, accept_len, tokens, groups, flags,
                                trials, margins, p, q, P, Q, R);
        }
        free(p);
        free(q);
        free(P);
        free(Q);
        free(R);
        free(pm);
    }
    free(rev_ptr);
    free(rev_grp);
    free(rev_nz);
    free(fill);
    return failed ? 2 : 0;
}

int pcg_oracle_verify(const void *target_logits, const void *draft_logits, int dtype, int B, int K, int V,
                      const int32_t *draft_tokens, int M, const int32_t *group_ptr, const int32_t *group_tok,
                      const int32_t *tok_degree, const double *weights, const float *uniforms, float temperature,
                      double accept_bias, int32_t *accept_len, int32_t *tokens, int32_t *groups, int32_t *flags,
                      double *margins, int threads) {
    return verify_batch(target_logits, draft_logits, dtype, B, K, V, draft_tokens, M, group_ptr, group_tok,
                        tok_degree, weights, uniforms, NULL, 0, NULL, temperature, accept_bias, accept_len, tokens, groups,
                        flags, NULL, margins, threads);
}

/*
 * Batched verification with the thinning sampler for the terminal group (see verify_sequence).
 * thin_uniforms [B, n_trials, 3] floats in [0,1), n_trials >= 1; cand_order [V]: the order in which the
 * candidate draw walks the tokens, a permutation of 0..V-1, or NULL for ascending token id; trials [B] (may be
 * NULL) receives the number of candidates drawn (1 after an all-accepted sequence).  margins[b][K][0] is the smallest margin over every
 * decision that led to the terminal group.  Everything else as pcg_oracle_verify.
 */
int pcg_oracle_verify_thinning(const void *target_logits, const void *draft_logits, int dtype, int B, int K, int V,
                               const int32_t *draft_tokens, int M, const int32_t *group_ptr,
                               const int32_t *group_tok, const int32_t *tok_degree, const double *weights,
                               const float *uniforms, const float *thin_uniforms, int n_trials,
                               const int32_t *cand_order, float temperature, double accept_bias,
                               int32_t *accept_len, int32_t *tokens, int32_t *groups, int32_t *flags,
                               int32_t *trials, double *margins, int threads) {
    if (!thin_uniforms || n_trials < 1) return 1;
    return verify_batch(target_logits, draft_logits, dtype, B, K, V, draft_tokens, M, group_ptr, group_tok,
                        tok_degree, weights, uniforms, thin_uniforms, n_trials, cand_order, temperature, accept_bias,
                        accept_len, tokens, groups, flags, trials, margins, threads);
}

/* Number of threads pcg_oracle_verify uses for threads <= 0. */
int pcg_oracle_max_threads(void) {
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}
