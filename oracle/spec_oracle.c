/*
 * CPU oracle for the combined token/embedding speculator: draft-tree generation and
 * greedy multi-candidate verification (arXiv 2404.19124, Sec. 3.1 and Sec. 4.1).
 *
 * THIS IS TEST INFRASTRUCTURE.  It is a slow, plain restatement of the method used to
 * judge the CUDA library; it shares no code, header, table or helper with it and must
 * never be called from the product path.  Only the test-suite, the smoke check and the
 * CPU-baseline leg of the benchmark may load it.
 *
 * The paper gives the method in prose only (no equations, no algorithm box), so every
 * function below states which sentence of the paper it restates and which reading it
 * takes where the prose is silent.
 *
 * Arithmetic: weights / context states are bf16 bit patterns widened exactly to fp32;
 * every stored intermediate (projection, mix, LayerNorm output, state, logits,
 * log-sum-exp, scores) is fp32; reductions (dot products, mean/variance, sum of
 * exponentials) are accumulated in fp64 and rounded once to fp32.  The post-GELU state
 * is rounded to bf16 (round-to-nearest-even) once per stage when `round_state_bf16`
 * is set, because that vector is what a 16-bit implementation carries between stages
 * (Sec. 4.1: inference runs in 16-bit precision).
 *
 * Pins (see tests, marker "not gpu"): every stage step against float64 library
 * routines (embedding, linear, layer_norm, erf-GELU, log_softmax, topk), probability
 * mass of a full tree == 1, brute-force path enumeration, the no-token-conditioning
 * special case (Sec. 3.1, the parallel-head structure), a hand-built token-conditioning
 * case, hand-built exact ties of leaf scores (all scores equal; a tie across the K
 * boundary) for the prune's lower-leaf-first rule, and hand-built verification examples.
 * Parity unpinned: the behaviour of the authors' trained speculators (tokens per step
 * in Sec. 3.1 / Tables 1-2) - it needs their weights and data.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

#define ORACLE_MAX_HEADS 8

enum {
    ORACLE_OK = 0,
    ORACLE_ERR_ARG = 1,      /* null pointer / non-positive size            */
    ORACLE_ERR_SHAPE = 2,    /* K > number of leaves, topk > V, ...         */
    ORACLE_ERR_TOKEN = 3,    /* token id outside [0, V)                     */
    ORACLE_ERR_NOMEM = 4
};

enum { ORACLE_BF16 = 0, ORACLE_F32 = 1 };

/* One embedding table, one state projection, one LayerNorm and one output matrix per
 * head: Sec. 3.1 ("without any weight sharing").  All matrices row-major. */
typedef struct {
    int32_t n_heads, V, d_base, d_inner;
    const uint16_t *emb[ORACLE_MAX_HEADS];    /* bf16 [V, d_inner]                          */
    const uint16_t *proj[ORACLE_MAX_HEADS];   /* bf16 [d_inner, d_in]; d_in = d_base (head 0) else d_inner */
    const float *ln_gamma[ORACLE_MAX_HEADS];  /* fp32 [d_inner]                             */
    const float *ln_beta[ORACLE_MAX_HEADS];   /* fp32 [d_inner]                             */
    const uint16_t *head[ORACLE_MAX_HEADS];   /* bf16 [V, d_inner]                          */
    float state_weight;                       /* a: weight of the projected state (Sec. 4)  */
    float emb_weight;                         /* b: weight of the token embedding (Sec. 4)  */
    float ln_eps;
    int32_t round_state_bf16;                 /* 1: round the post-GELU state to bf16       */
} oracle_weights_t;

/* ---------- bf16 <-> fp32 (bf16 = upper 16 bits of an IEEE-754 binary32) ---------- */

static float bf16_to_f32(uint16_t h) {
    uint32_t u = (uint32_t)h << 16;
    float f;
    memcpy(&f, &u, 4);
    return f;
}

static uint16_t f32_to_bf16_rne(float f) {
    uint32_t u;
    memcpy(&u, &f, 4);
    if ((u & 0x7fffffffu) > 0x7f800000u) return (uint16_t)((u >> 16) | 0x0040u); /* quiet NaN */
    u += 0x7fffu + ((u >> 16) & 1u);
    return (uint16_t)(u >> 16);
}

float oracle_bf16_to_f32(uint16_t h) { return bf16_to_f32(h); }
uint16_t oracle_f32_to_bf16(float f) { return f32_to_bf16_rne(f); }

int oracle_d_in(const oracle_weights_t *w, int level) { return level == 0 ? w->d_base : w->d_inner; }

/* ---------- one stage of the multi-stage MLP (Sec. 3.1) ----------
 * "Each input pair (state plus sampled token embedding) is projected and passed through
 * a LayerNorm/GeLU activation, forming a new state vector."
 *   z = E_l[tok]                      embedding of the token sampled at the prior stage
 *   p = Wp_l . s_parent               linear projection of the prior state, no bias
 *   h = a p + b z                     weighted mix (Sec. 4: state/embedding weighting)
 *   y = gamma * (h - mean) / sqrt(var + eps) + beta     (biased variance over d_inner)
 *   s = y * Phi(y)                    exact (erf) GELU
 * Optional outputs p_out / h_out / y_out (each d_inner floats) may be NULL.
 */
int oracle_stage_state(const oracle_weights_t *w, int level, const float *s_parent, int32_t tok,
                       float *s_out, float *p_out, float *h_out, float *y_out) {
    if (!w || !s_parent || !s_out) return ORACLE_ERR_ARG;
    if (level < 0 || level >= w->n_heads) return ORACLE_ERR_SHAPE;
    if (tok < 0 || tok >= w->V) return ORACLE_ERR_TOKEN;
    const int d = w->d_inner, d_in = oracle_d_in(w, level);
    const uint16_t *E = w->emb[level], *Wp = w->proj[level];
    float *h = (float *)malloc(sizeof(float) * (size_t)d);
    if (!h) return ORACLE_ERR_NOMEM;

    for (int i = 0; i < d; ++i) {
        double acc = 0.0;
        const uint16_t *row = Wp + (size_t)i * d_in;
#pragma omp simd reduction(+ : acc)
        for (int c = 0; c < d_in; ++c) acc += (double)bf16_to_f32(row[c]) * (double)s_parent[c];
        float p = (float)acc;
        float z = bf16_to_f32(E[(size_t)tok * d + i]);
        h[i] = w->state_weight * p + w->emb_weight * z;
        if (p_out) p_out[i] = p;
        if (h_out) h_out[i] = h[i];
    }
    double mean = 0.0;
    for (int i = 0; i < d; ++i) mean += (double)h[i];
    mean /= d;
    double var = 0.0;
    for (int i = 0; i < d; ++i) {
        double c = (double)h[i] - mean;
        var += c * c;
    }
    var /= d;
    const double rstd = 1.0 / sqrt(var + (double)w->ln_eps);
    for (int i = 0; i < d; ++i) {
        float y = (float)(((double)h[i] - mean) * rstd * (double)w->ln_gamma[level][i] +
                          (double)w->ln_beta[level][i]);
        if (y_out) y_out[i] = y;
        float s = (float)(0.5 * (double)y * (1.0 + erf((double)y * 0.70710678118654752440)));
        if (w->round_state_bf16) s = bf16_to_f32(f32_to_bf16_rne(s));
        s_out[i] = s;
    }
    free(h);
    return ORACLE_OK;
}

/* "This state vector is used to predict the next set of draft tokens" (Sec. 3.1):
 * logits[r, v] = sum_c Wout_l[v, c] * S[r, c] for `rows` states at once, no bias. */
int oracle_stage_logits(const oracle_weights_t *w, int level, const float *S, int rows, float *logits) {
    if (!w || !S || !logits || rows <= 0) return ORACLE_ERR_ARG;
    if (level < 0 || level >= w->n_heads) return ORACLE_ERR_SHAPE;
    const int d = w->d_inner, V = w->V;
    const uint16_t *Wout = w->head[level];
#pragma omp parallel for schedule(static)
    for (int v = 0; v < V; ++v) {
        const uint16_t *row = Wout + (size_t)v * d;
        for (int r = 0; r < rows; ++r) {
            const float *s = S + (size_t)r * d;
            double acc = 0.0;
#pragma omp simd reduction(+ : acc)
            for (int c = 0; c < d; ++c) acc += (double)bf16_to_f32(row[c]) * (double)s[c];
            logits[(size_t)r * V + v] = (float)acc;
        }
    }
    return ORACLE_OK;
}

/* Natural-log normaliser of the softmax over the whole vocabulary, max-subtracted. */
float oracle_logsumexp(const float *x, int n) {
    float m = x[0];
    for (int i = 1; i < n; ++i)
        if (x[i] > m) m = x[i];
    double s = 0.0;
    for (int i = 0; i < n; ++i) s += exp((double)x[i] - (double)m);
    return (float)((double)m + log(s));
}

/* The k largest entries in descending order; equal values: the lower index first. */
int oracle_topk(const float *x, int n, int k, int32_t *ids, float *vals) {
    if (!x || !ids || !vals || k <= 0 || k > n) return ORACLE_ERR_SHAPE;
    for (int j = 0; j < k; ++j) {
        int best = -1;
        for (int i = 0; i < n; ++i) {
            int taken = 0;
            for (int q = 0; q < j; ++q)
                if (ids[q] == i) taken = 1;
            if (taken) continue;
            if (best < 0 || x[i] > x[best]) best = i;
        }
        ids[j] = best;
        vals[j] = x[best];
    }
    return ORACLE_OK;
}

/* ---------- draft tree (Sec. 3.1 "the model thus emits an entire tree of candidates";
 * Sec. 4.1: branch topk[l] ways at head l, then prune the product tree to the K most
 * confident leaves).  Confidence = sum over the path of log-softmax probabilities.
 *
 * Level 0 holds one node per sequence (state = ctx_state[b], token = last_tok[b],
 * score 0).  Node r of level l has children r*topk[l] + j, j = 0..topk[l]-1, ordered by
 * descending logit.  After the last head the L = prod topk leaves of a sequence are
 * ordered by (score descending, leaf index ascending) and the first K are returned with
 * the n tokens on their root-to-leaf paths (last_tok itself is not part of a candidate).
 *
 * Optional dumps (NULL to skip), for level l with N_l = B * prod_{j<l} topk[j] nodes:
 *   dump_states[l]  fp32 [N_l, d_inner]   post-GELU state of every node
 *   dump_logits[l]  fp32 [N_l, V]
 *   dump_tok[l]     int32 [N_l * topk[l]] tokens of the children (level l+1 nodes)
 *   dump_score[l]   fp32  [N_l * topk[l]] cumulative scores of the children
 */
int oracle_draft(const oracle_weights_t *w, const uint16_t *ctx_state, const int32_t *last_tok, int B,
                 const int32_t *topk, int K, int32_t *cand_tok, float *cand_logp, float **dump_states,
                 float **dump_logits, int32_t **dump_tok, float **dump_score) {
    if (!w || !ctx_state || !last_tok || !topk || !cand_tok || !cand_logp || B <= 0) return ORACLE_ERR_ARG;
    const int n = w->n_heads, d = w->d_inner, V = w->V;
    if (n <= 0 || n > ORACLE_MAX_HEADS) return ORACLE_ERR_SHAPE;
    long L = 1;
    for (int l = 0; l < n; ++l) {
        if (topk[l] <= 0 || topk[l] > V) return ORACLE_ERR_SHAPE;
        L *= topk[l];
        if (L > (1L << 24)) return ORACLE_ERR_SHAPE;
    }
    if (K <= 0 || K > L) return ORACLE_ERR_SHAPE;
    for (int b = 0; b < B; ++b)
        if (last_tok[b] < 0 || last_tok[b] >= V) return ORACLE_ERR_TOKEN;

    int rc = ORACLE_OK;
    /* per level: token of each node, cumulative score of each node */
    int32_t *tok[ORACLE_MAX_HEADS + 1] = {0};
    float *score[ORACLE_MAX_HEADS + 1] = {0};
    float *S_prev = NULL, *S_cur = NULL, *logits = NULL;
    long N = B;

    tok[0] = (int32_t *)malloc(sizeof(int32_t) * (size_t)B);
    score[0] = (float *)malloc(sizeof(float) * (size_t)B);
    S_prev = (float *)malloc(sizeof(float) * (size_t)B * w->d_base);
    if (!tok[0] || !score[0] || !S_prev) { rc = ORACLE_ERR_NOMEM; goto done; }
    for (int b = 0; b < B; ++b) {
        tok[0][b] = last_tok[b];
        score[0][b] = 0.0f;
        for (int c = 0; c < w->d_base; ++c)
            S_prev[(size_t)b * w->d_base + c] = bf16_to_f32(ctx_state[(size_t)b * w->d_base + c]);
    }

    for (int l = 0; l < n; ++l) {
        const int d_in = oracle_d_in(w, l), kl = topk[l];
        /* nodes of level l: N of them; node r has parent r / topk[l-1] in level l-1 */
        S_cur = (float *)malloc(sizeof(float) * (size_t)N * d);
        logits = (float *)malloc(sizeof(float) * (size_t)N * V);
        tok[l + 1] = (int32_t *)malloc(sizeof(int32_t) * (size_t)N * kl);
        score[l + 1] = (float *)malloc(sizeof(float) * (size_t)N * kl);
        if (!S_cur || !logits || !tok[l + 1] || !score[l + 1]) { rc = ORACLE_ERR_NOMEM; goto done; }

        int stage_rc = ORACLE_OK;
#pragma omp parallel for schedule(dynamic, 1)
        for (long r = 0; r < N; ++r) {
            const long parent = (l == 0) ? r : r / topk[l - 1];
            int e = oracle_stage_state(w, l, S_prev + (size_t)parent * d_in, tok[l][r],
                                       S_cur + (size_t)r * d, NULL, NULL, NULL);
            if (e != ORACLE_OK) {
#pragma omp critical
                stage_rc = e;
            }
        }
        if (stage_rc != ORACLE_OK) { rc = stage_rc; goto done; }
        rc = oracle_stage_logits(w, l, S_cur, (int)N, logits);
        if (rc != ORACLE_OK) goto done;

        for (long r = 0; r < N; ++r) {
            const float *x = logits + (size_t)r * V;
            const float lse = oracle_logsumexp(x, V);
            int32_t ids[64];
            float vals[64];
            int32_t *idp = ids;
            float *vp = vals;
            if (kl > 64) {
                idp = (int32_t *)malloc(sizeof(int32_t) * (size_t)kl);
                vp = (float *)malloc(sizeof(float) * (size_t)kl);
                if (!idp || !vp) { rc = ORACLE_ERR_NOMEM; goto done; }
            }
            oracle_topk(x, V, kl, idp, vp);
            for (int j = 0; j < kl; ++j) {
                tok[l + 1][r * kl + j] = idp[j];
                score[l + 1][r * kl + j] = score[l][r] + (vp[j] - lse);
            }
            if (kl > 64) { free(idp); free(vp); }
        }
        if (dump_states && dump_states[l]) memcpy(dump_states[l], S_cur, sizeof(float) * (size_t)N * d);
        if (dump_logits && dump_logits[l]) memcpy(dump_logits[l], logits, sizeof(float) * (size_t)N * V);
        if (dump_tok && dump_tok[l]) memcpy(dump_tok[l], tok[l + 1], sizeof(int32_t) * (size_t)N * kl);
        if (dump_score && dump_score[l]) memcpy(dump_score[l], score[l + 1], sizeof(float) * (size_t)N * kl);

        free(S_prev);
        S_prev = S_cur;
        S_cur = NULL;
        free(logits);
        logits = NULL;
        N *= kl;
    }

    /* prune: per sequence keep the K best leaves; ties -> lower leaf index */
    {
        char *used = (char *)malloc((size_t)L);
        if (!used) { rc = ORACLE_ERR_NOMEM; goto done; }
        for (int b = 0; b < B; ++b) {
            const float *sc = score[n] + (size_t)b * L;
            memset(used, 0, (size_t)L);
            for (int k = 0; k < K; ++k) {
                long best = -1;
                for (long i = 0; i < L; ++i) {
                    if (used[i]) continue;
                    if (best < 0 || sc[i] > sc[best]) best = i;
                }
                used[best] = 1;
                cand_logp[(size_t)b * K + k] = sc[best];
                /* walk from the leaf to the root: node index at level l+1 within sequence b */
                long idx = best; /* index among the sequence's nodes at level n */
                for (int l = n - 1; l >= 0; --l) {
                    long per_seq = 1; /* nodes of this sequence at level l+1 */
                    for (int j = 0; j <= l; ++j) per_seq *= topk[j];
                    cand_tok[((size_t)b * K + k) * n + l] = tok[l + 1][(size_t)b * per_seq + idx];
                    idx /= topk[l];
                }
            }
        }
        free(used);
    }

done:
    for (int l = 0; l <= n && l <= ORACLE_MAX_HEADS; ++l) {
        free(tok[l]);
        free(score[l]);
    }
    free(S_prev);
    free(S_cur);
    free(logits);
    return rc;
}

/* ---------- greedy multi-candidate verification (Sec. 1: accept the predicted tokens
 * that match the base model's output, reject the rest; Sec. 3.1: score all candidates,
 * keep the tokens of the best-scoring one; Sec. 5: at most n speculated + 1 base token).
 *
 * base_logits[b, k, j, :] is the base model's output at input position j of the sequence
 * [last_tok, c_0 .. c_{n-1}] of candidate k (Sec. 4.1: 1 ground-truth token + n
 * speculated), i.e. its prediction for c_j when j < n and for the token after the whole
 * candidate when j = n.
 *   g[b,k,j]     = first index of the maximum of base_logits[b,k,j,:]  (NaN never wins)
 *   m[b,k]       = number of leading positions j < n with cand_tok[b,k,j] == g[b,k,j]
 *   best_cand[b] = lowest k attaining max_k m[b,k]
 *   accept_len[b]= m[b,best];  next_tok[b] = g[b,best,accept_len[b]]
 * g_out (int32 [B,K,n+1]) is optional.
 */
static float logit_at(const void *base, int dtype, size_t i) {
    return dtype == ORACLE_BF16 ? bf16_to_f32(((const uint16_t *)base)[i]) : ((const float *)base)[i];
}

int32_t oracle_row_argmax(const void *base, int dtype, size_t offset, int V) {
    float best = -INFINITY;
    int32_t arg = 0;
    for (int v = 0; v < V; ++v) {
        float x = logit_at(base, dtype, offset + (size_t)v);
        if (x > best) {
            best = x;
            arg = v;
        }
    }
    return arg;
}

int oracle_verify(const int32_t *cand_tok, const void *base_logits, int dtype, int B, int K, int n, int V,
                  int32_t *accept_len, int32_t *best_cand, int32_t *next_tok, int32_t *g_out) {
    if (!cand_tok || !base_logits || !accept_len || !best_cand || !next_tok) return ORACLE_ERR_ARG;
    if (B <= 0 || K <= 0 || n <= 0 || V <= 0) return ORACLE_ERR_ARG;
    if (dtype != ORACLE_BF16 && dtype != ORACLE_F32) return ORACLE_ERR_ARG;
    const size_t rows = (size_t)B * K * (n + 1);
    int32_t *g = (int32_t *)malloc(sizeof(int32_t) * rows);
    if (!g) return ORACLE_ERR_NOMEM;
#pragma omp parallel for schedule(static)
    for (long r = 0; r < (long)rows; ++r) g[r] = oracle_row_argmax(base_logits, dtype, (size_t)r * V, V);

    for (int b = 0; b < B; ++b) {
        int best_k = 0, best_m = -1;
        for (int k = 0; k < K; ++k) {
            const int32_t *c = cand_tok + ((size_t)b * K + k) * n;
            const int32_t *gk = g + ((size_t)b * K + k) * (n + 1);
            int m = 0;
            while (m < n && c[m] == gk[m]) ++m;
            if (m > best_m) {
                best_m = m;
                best_k = k;
            }
        }
        accept_len[b] = best_m;
        best_cand[b] = best_k;
        next_tok[b] = g[((size_t)b * K + best_k) * (n + 1) + best_m];
    }
    if (g_out) memcpy(g_out, g, sizeof(int32_t) * rows);
    free(g);
    return ORACLE_OK;
}

int oracle_num_threads(void) {
    int t = 1;
#ifdef _OPENMP
    extern int omp_get_max_threads(void);
    t = omp_get_max_threads();
#endif
    return t;
}
