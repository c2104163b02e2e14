/*
 * CPU oracle for the rollout step of a mixture-of-experts decoder (test infrastructure).
 *
 * This file is TEST INFRASTRUCTURE.  It is the plain definition of what the rollout module of the
 * paper (Section 3.3, "the inputs to the Rollout module ...", and Section 2.3 "Segment Rollouts")
 * computes for every live trajectory: one forward pass of the policy model over the new tokens of
 * each sequence, attending over that sequence's cached keys/values, followed by sampling of the
 * next token and the log-probability of that token under the behaviour policy (the denominator of
 * the importance ratio, Eq. 3).  The paper treats the policy (a Qwen3-30B-A3B-shaped MoE
 * transformer, Section 4.1) as a black box; the layer below is the textbook pre-norm decoder layer
 * with grouped-query attention, rotary position embedding, and a softmax-top-k router.
 *
 * Conventions
 *   - weights and the KV cache are bf16 (uint16_t bit patterns), row-major [out, in];
 *   - every intermediate is a double; the only rounding the data format forces is that new keys
 *     and values are rounded to bf16 (nearest-even) when stored in the cache, and the router's
 *     logits and probabilities are rounded to fp32 before the top-k decision (the router decides
 *     in fp32);
 *   - the residual stream x, logits and log-probs cross the interface as fp32;
 *   - no blocking, fusion or reordering: loops run in the order of the definition.  OpenMP is used
 *     on outermost independent loops only.
 *
 * Nothing here is shared with, or derived from, the CUDA library.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

typedef struct {
    int32_t n_layers, hidden, n_q_heads, n_kv_heads, head_dim;
    int32_t n_experts, top_k, expert_inter, vocab, qk_norm;
    double rope_theta, rms_eps;
} orc_config;

/* One decoder layer's weights (bf16 bit patterns). */
typedef struct {
    const uint16_t *attn_norm;  /* [H]                      */
    const uint16_t *wqkv;       /* [(nq + 2 nkv) d, H]: q rows, then k rows, then v rows */
    const uint16_t *q_norm;     /* [d] (used when qk_norm)  */
    const uint16_t *k_norm;     /* [d]                      */
    const uint16_t *wo;         /* [H, nq d]                */
    const uint16_t *mlp_norm;   /* [H]                      */
    const uint16_t *router;     /* [E, H]                   */
    const uint16_t *w_gate_up;  /* [E, 2 I, H]: gate rows 0..I-1, up rows I..2I-1 */
    const uint16_t *w_down;     /* [E, H, I]                */
} orc_layer;

/* ---------------------------------------------------------------- bf16 <-> fp32 */

float orc_bf16_to_f32(uint16_t b) {
    uint32_t u = ((uint32_t)b) << 16;
    float f;
    memcpy(&f, &u, 4);
    return f;
}

/* Round to nearest, ties to even, on the upper 16 bits of the fp32 pattern. NaN stays NaN. */
uint16_t orc_f32_to_bf16(float f) {
    uint32_t u;
    memcpy(&u, &f, 4);
    if ((u & 0x7fffffffu) > 0x7f800000u) return (uint16_t)((u >> 16) | 0x0040u);
    uint32_t lsb = (u >> 16) & 1u;
    u += 0x7fffu + lsb;
    return (uint16_t)(u >> 16);
}

static inline double w2d(uint16_t b) { return (double)orc_bf16_to_f32(b); }

/* ---------------------------------------------------------------- RMSNorm
 * out_i = x_i / sqrt(mean_j x_j^2 + eps) * gain_i ; eps inside the square root. */
void orc_rmsnorm(const double *x, const uint16_t *gain, int n, double eps, double *out) {
    double ss = 0.0;
    for (int i = 0; i < n; ++i) ss += x[i] * x[i];
    double r = 1.0 / sqrt(ss / (double)n + eps);
    for (int i = 0; i < n; ++i) out[i] = x[i] * r * w2d(gain[i]);
}

/* ---------------------------------------------------------------- rotary position embedding
 * Rotate-half pairing: for i < d/2 with theta_i = base^(-2 i / d), the pair (u_i, u_{i+d/2}) is
 * rotated by the angle pos * theta_i. */
void orc_rope(double *u, int d, int64_t pos, double base) {
    int half = d / 2;
    for (int i = 0; i < half; ++i) {
        double theta = pow(base, -2.0 * (double)i / (double)d);
        double ang = (double)pos * theta;
        double c = cos(ang), s = sin(ang);
        double a = u[i], b = u[i + half];
        u[i] = a * c - b * s;
        u[i + half] = b * c + a * s;
    }
}

/* y[r] = sum_c W[r, c] x[c] */
static void matvec(const uint16_t *W, int rows, int cols, const double *x, double *y) {
    for (int r = 0; r < rows; ++r) {
        const uint16_t *w = W + (size_t)r * cols;
        double acc = 0.0;
        for (int c = 0; c < cols; ++c) acc += w2d(w[c]) * x[c];
        y[r] = acc;
    }
}

/* ---------------------------------------------------------------- softmax (in place, stable) */
void orc_softmax(double *z, int n) {
    double m = z[0];
    for (int i = 1; i < n; ++i) if (z[i] > m) m = z[i];
    double s = 0.0;
    for (int i = 0; i < n; ++i) { z[i] = exp(z[i] - m); s += z[i]; }
    for (int i = 0; i < n; ++i) z[i] /= s;
}

/* ---------------------------------------------------------------- router
 * z = W_r h (rounded to fp32), pi = softmax(z) (rounded to fp32); the k largest pi are selected,
 * larger first, equal values by lower expert index; weights = pi_sel / sum(pi_sel).
 * probs_out (optional) receives all E probabilities (fp32). */
void orc_router(const uint16_t *Wr, int E, int H, int k, const double *h,
                int32_t *idx_out, float *w_out, float *probs_out) {
    double *z = (double *)malloc(sizeof(double) * E);
    float *pi = (float *)malloc(sizeof(float) * E);
    char *taken = (char *)calloc(E, 1);
    matvec(Wr, E, H, h, z);
    for (int e = 0; e < E; ++e) z[e] = (double)(float)z[e];
    orc_softmax(z, E);
    for (int e = 0; e < E; ++e) pi[e] = (float)z[e];
    double sel_sum = 0.0;
    for (int j = 0; j < k; ++j) {
        int best = -1;
        for (int e = 0; e < E; ++e) {
            if (taken[e]) continue;
            if (best < 0 || pi[e] > pi[best]) best = e;   /* strict >: lower index wins ties */
        }
        taken[best] = 1;
        idx_out[j] = best;
        sel_sum += (double)pi[best];
    }
    for (int j = 0; j < k; ++j) w_out[j] = (float)((double)pi[idx_out[j]] / sel_sum);
    if (probs_out) for (int e = 0; e < E; ++e) probs_out[e] = pi[e];
    free(z); free(pi); free(taken);
}

/* ---------------------------------------------------------------- one expert: SwiGLU MLP
 * y = W_down ( silu(W_gate h) * (W_up h) ), silu(a) = a / (1 + exp(-a)). */
static void expert_mlp(const uint16_t *w_gate_up, const uint16_t *w_down, int H, int I,
                       const double *h, double *y, double *scratch /* 3 I */) {
    double *gate = scratch, *up = scratch + I, *act = scratch + 2 * I;
    matvec(w_gate_up, I, H, h, gate);
    matvec(w_gate_up + (size_t)I * H, I, H, h, up);
    for (int i = 0; i < I; ++i) act[i] = gate[i] / (1.0 + exp(-gate[i])) * up[i];
    matvec(w_down, H, I, act, y);
}

/* Address of cache row (page, kv head, slot) inside one layer's pool [page][kv_head][slot][d]. */
static inline size_t kv_row(int32_t page, int h, int slot, int nkv, int page_size, int d) {
    return ((((size_t)page * nkv + h) * page_size) + slot) * (size_t)d;
}

/* ---------------------------------------------------------------- one decoder layer
 * n_tok new tokens; token i belongs to sequence seq[i] (a row of block_table) and sits at
 * position pos[i] (0-based count of tokens before it in its sequence).  x [n_tok, H] is the
 * residual stream, updated in place.  k_pool / v_pool are THIS layer's pools; every new token's
 * key/value is written (bf16) at its position before any attention is evaluated, and token i
 * attends to positions 0..pos[i] of its own sequence.
 * forced_idx (optional, [n_tok, k]): use these experts instead of the router's own top-k (weights
 * are then the renormalised probabilities of the forced experts).
 * Outputs (optional): router_idx [n_tok,k], router_w [n_tok,k], router_probs [n_tok,E],
 * attn_out [n_tok, nq d] (concatenated head outputs before W_o). */
void orc_layer_forward(const orc_config *cfg, const orc_layer *L, int n_tok, float *x,
                       const int32_t *seq, const int32_t *pos,
                       uint16_t *k_pool, uint16_t *v_pool, const int32_t *block_table,
                       int max_pages_per_seq, int page_size,
                       const int32_t *forced_idx,
                       int32_t *router_idx, float *router_w, float *router_probs,
                       float *attn_out) {
    const int H = cfg->hidden, nq = cfg->n_q_heads, nkv = cfg->n_kv_heads, d = cfg->head_dim;
    const int E = cfg->n_experts, k = cfg->top_k, I = cfg->expert_inter;
    const int g = nq / nkv;
    const int qkv_rows = (nq + 2 * nkv) * d;
    double *q_all = (double *)malloc(sizeof(double) * (size_t)n_tok * nq * d);

    /* steps 1-5: norm, projections, per-head norm, RoPE, cache write */
    #pragma omp parallel for schedule(dynamic, 1)
    for (int i = 0; i < n_tok; ++i) {
        double *xi = (double *)malloc(sizeof(double) * H);
        double *h = (double *)malloc(sizeof(double) * H);
        double *qkv = (double *)malloc(sizeof(double) * qkv_rows);
        for (int c = 0; c < H; ++c) xi[c] = (double)x[(size_t)i * H + c];
        orc_rmsnorm(xi, L->attn_norm, H, cfg->rms_eps, h);
        matvec(L->wqkv, qkv_rows, H, h, qkv);
        double *qv = qkv, *kv = qkv + (size_t)nq * d, *vv = qkv + (size_t)(nq + nkv) * d;
        for (int j = 0; j < nq; ++j) {
            double *u = qv + (size_t)j * d;
            if (cfg->qk_norm) orc_rmsnorm(u, L->q_norm, d, cfg->rms_eps, u);
            orc_rope(u, d, pos[i], cfg->rope_theta);
        }
        for (int j = 0; j < nkv; ++j) {
            double *u = kv + (size_t)j * d;
            if (cfg->qk_norm) orc_rmsnorm(u, L->k_norm, d, cfg->rms_eps, u);
            orc_rope(u, d, pos[i], cfg->rope_theta);
        }
        memcpy(q_all + (size_t)i * nq * d, qv, sizeof(double) * (size_t)nq * d);
        int32_t page = block_table[(size_t)seq[i] * max_pages_per_seq + pos[i] / page_size];
        int slot = pos[i] % page_size;
        for (int j = 0; j < nkv; ++j) {
            size_t row = kv_row(page, j, slot, nkv, page_size, d);
            for (int c = 0; c < d; ++c) {
                k_pool[row + c] = orc_f32_to_bf16((float)kv[(size_t)j * d + c]);
                v_pool[row + c] = orc_f32_to_bf16((float)vv[(size_t)j * d + c]);
            }
        }
        free(xi); free(h); free(qkv);
    }

    /* step 6: attention of every (token, query head) over positions 0..pos */
    double *o_all = (double *)malloc(sizeof(double) * (size_t)n_tok * nq * d);
    #pragma omp parallel for collapse(2) schedule(dynamic, 1)
    for (int i = 0; i < n_tok; ++i) {
        for (int j = 0; j < nq; ++j) {
            const int hk = j / g;
            const int n_ctx = pos[i] + 1;
            const double *q = q_all + ((size_t)i * nq + j) * d;
            double *s = (double *)malloc(sizeof(double) * n_ctx);
            const int32_t *bt = block_table + (size_t)seq[i] * max_pages_per_seq;
            const double scale = 1.0 / sqrt((double)d);
            for (int t = 0; t < n_ctx; ++t) {
                size_t row = kv_row(bt[t / page_size], hk, t % page_size, nkv, page_size, d);
                double acc = 0.0;
                for (int c = 0; c < d; ++c) acc += q[c] * w2d(k_pool[row + c]);
                s[t] = acc * scale;
            }
            orc_softmax(s, n_ctx);
            double *o = o_all + ((size_t)i * nq + j) * d;
            for (int c = 0; c < d; ++c) o[c] = 0.0;
            for (int t = 0; t < n_ctx; ++t) {
                size_t row = kv_row(bt[t / page_size], hk, t % page_size, nkv, page_size, d);
                for (int c = 0; c < d; ++c) o[c] += s[t] * w2d(v_pool[row + c]);
            }
            free(s);
        }
    }
    if (attn_out)
        for (size_t z = 0; z < (size_t)n_tok * nq * d; ++z) attn_out[z] = (float)o_all[z];

    /* steps 7-9: output projection + residual, router, experts + residual */
    #pragma omp parallel for schedule(dynamic, 1)
    for (int i = 0; i < n_tok; ++i) {
        double *xi = (double *)malloc(sizeof(double) * H);
        double *y = (double *)malloc(sizeof(double) * H);
        double *h2 = (double *)malloc(sizeof(double) * H);
        double *scratch = (double *)malloc(sizeof(double) * 3 * I);
        int32_t *idx = (int32_t *)malloc(sizeof(int32_t) * k);
        float *w = (float *)malloc(sizeof(float) * k);
        float *probs = (float *)malloc(sizeof(float) * E);
        matvec(L->wo, H, nq * d, o_all + (size_t)i * nq * d, y);
        for (int c = 0; c < H; ++c) xi[c] = (double)x[(size_t)i * H + c] + y[c];
        orc_rmsnorm(xi, L->mlp_norm, H, cfg->rms_eps, h2);
        orc_router(L->router, E, H, k, h2, idx, w, probs);
        if (forced_idx) {
            double ssum = 0.0;
            for (int j = 0; j < k; ++j) { idx[j] = forced_idx[(size_t)i * k + j]; ssum += (double)probs[idx[j]]; }
            for (int j = 0; j < k; ++j) w[j] = (float)((double)probs[idx[j]] / ssum);
        }
        for (int j = 0; j < k; ++j) {
            const int e = idx[j];
            expert_mlp(L->w_gate_up + (size_t)e * 2 * I * H, L->w_down + (size_t)e * H * I, H, I, h2, y, scratch);
            for (int c = 0; c < H; ++c) xi[c] += (double)w[j] * y[c];
        }
        for (int c = 0; c < H; ++c) x[(size_t)i * H + c] = (float)xi[c];
        if (router_idx) for (int j = 0; j < k; ++j) router_idx[(size_t)i * k + j] = idx[j];
        if (router_w) for (int j = 0; j < k; ++j) router_w[(size_t)i * k + j] = w[j];
        if (router_probs) for (int e = 0; e < E; ++e) router_probs[(size_t)i * E + e] = probs[e];
        free(xi); free(y); free(h2); free(scratch); free(idx); free(w); free(probs);
    }
    free(q_all); free(o_all);
}

/* ---------------------------------------------------------------- embedding: x_i = embed[token_i] */
void orc_embed(const uint16_t *embed, int H, int n_tok, const int32_t *tokens, float *x) {
    for (int i = 0; i < n_tok; ++i)
        for (int c = 0; c < H; ++c) x[(size_t)i * H + c] = orc_bf16_to_f32(embed[(size_t)tokens[i] * H + c]);
}

/* ---------------------------------------------------------------- final norm + lm_head
 * logits[i, v] = sum_c W_lm[v, c] * (rms(x_i) * g_f)_c  (returned as fp32). */
void orc_lm_head(const orc_config *cfg, const uint16_t *final_norm, const uint16_t *lm_head,
                 int n_tok, const float *x, float *logits) {
    const int H = cfg->hidden, V = cfg->vocab;
    double *h = (double *)malloc(sizeof(double) * (size_t)n_tok * H);
    for (int i = 0; i < n_tok; ++i) {
        double *xi = (double *)malloc(sizeof(double) * H);
        for (int c = 0; c < H; ++c) xi[c] = (double)x[(size_t)i * H + c];
        orc_rmsnorm(xi, final_norm, H, cfg->rms_eps, h + (size_t)i * H);
        free(xi);
    }
    #pragma omp parallel for schedule(static)
    for (int v = 0; v < V; ++v) {
        const uint16_t *w = lm_head + (size_t)v * H;
        for (int i = 0; i < n_tok; ++i) {
            const double *hi = h + (size_t)i * H;
            double acc = 0.0;
            for (int c = 0; c < H; ++c) acc += w2d(w[c]) * hi[c];
            logits[(size_t)i * V + v] = (float)acc;
        }
    }
    free(h);
}

/* ---------------------------------------------------------------- Philox4x32-10
 * Counter-based generator of Salmon, Moraes, Dror and Shaw (SC'11): ten rounds of
 *   (c0,c1,c2,c3) <- (hi(M1*c2) ^ c1 ^ k0, lo(M1*c2), hi(M0*c0) ^ c3 ^ k1, lo(M0*c0))
 * with the key bumped by the Weyl constants between rounds. */
void orc_philox4x32_10(const uint32_t ctr[4], const uint32_t key[2], uint32_t out[4]) {
    const uint32_t M0 = 0xD2511F53u, M1 = 0xCD9E8D57u, W0 = 0x9E3779B9u, W1 = 0xBB67AE85u;
    uint32_t c0 = ctr[0], c1 = ctr[1], c2 = ctr[2], c3 = ctr[3], k0 = key[0], k1 = key[1];
    for (int r = 0; r < 10; ++r) {
        uint64_t p0 = (uint64_t)M0 * c0, p1 = (uint64_t)M1 * c2;
        uint32_t n0 = (uint32_t)(p1 >> 32) ^ c1 ^ k0;
        uint32_t n1 = (uint32_t)p1;
        uint32_t n2 = (uint32_t)(p0 >> 32) ^ c3 ^ k1;
        uint32_t n3 = (uint32_t)p0;
        c0 = n0; c1 = n1; c2 = n2; c3 = n3;
        k0 += W0; k1 += W1;
    }
    out[0] = c0; out[1] = c1; out[2] = c2; out[3] = c3;
}

/* One uniform per (seed, step, sequence): key = the 64-bit seed, counter = (step lo, step hi,
 * sequence id, 0); u = ((x0 >> 8) + 0.5) * 2^-24, strictly inside (0, 1). */
double orc_uniform(uint64_t seed, uint64_t step, uint32_t seq_id) {
    uint32_t ctr[4] = {(uint32_t)step, (uint32_t)(step >> 32), seq_id, 0u};
    uint32_t key[2] = {(uint32_t)seed, (uint32_t)(seed >> 32)};
    uint32_t out[4];
    orc_philox4x32_10(ctr, key, out);
    return ((double)(out[0] >> 8) + 0.5) * (1.0 / 16777216.0);
}

/* ---------------------------------------------------------------- sampling
 * greedy != 0 : token = argmax logits (lowest id on ties); logp = log_softmax(logits)[token]
 *               (temperature 1).
 * greedy == 0 : pi = softmax(logits / T).  Nucleus S = shortest prefix, in the order
 *               (pi descending, id ascending), whose mass is >= top_p (the token that crosses the
 *               threshold is inside).  The token is drawn from pi restricted to S by walking S in
 *               ASCENDING TOKEN ID and returning the first id whose cumulative pi / mass(S)
 *               exceeds u.  logp = log pi[token] over the FULL vocabulary at temperature T: the
 *               behaviour-policy probability of Eq. 3 in the paper's training setting
 *               (top_p = 1).
 * Optional outputs: nucleus_mass, in_nucleus[V] (0/1), cdf_lo / cdf_hi = the token's interval of
 * the normalised cumulative distribution. */
static const double *g_sort_pi;
static int cmp_desc(const void *a, const void *b) {
    int32_t ia = *(const int32_t *)a, ib = *(const int32_t *)b;
    if (g_sort_pi[ia] > g_sort_pi[ib]) return -1;
    if (g_sort_pi[ia] < g_sort_pi[ib]) return 1;
    return (ia > ib) - (ia < ib);
}

void orc_sample(const float *logits, int V, double temperature, double top_p, int greedy, double u,
                int32_t *token_out, float *logp_out, double *nucleus_mass, uint8_t *in_nucleus,
                double *cdf_lo, double *cdf_hi) {
    double *pi = (double *)malloc(sizeof(double) * V);
    const double T = greedy ? 1.0 : temperature;
    double m = (double)logits[0] / T;
    for (int v = 1; v < V; ++v) if ((double)logits[v] / T > m) m = (double)logits[v] / T;
    double Z = 0.0;
    for (int v = 0; v < V; ++v) Z += exp((double)logits[v] / T - m);
    const double lse = m + log(Z);
    for (int v = 0; v < V; ++v) pi[v] = exp((double)logits[v] / T - lse);

    if (greedy) {
        int best = 0;
        for (int v = 1; v < V; ++v) if (logits[v] > logits[best]) best = v;
        *token_out = best;
        *logp_out = (float)((double)logits[best] - lse);
        if (nucleus_mass) *nucleus_mass = 1.0;
        if (cdf_lo) *cdf_lo = 0.0;
        if (cdf_hi) *cdf_hi = 1.0;
        if (in_nucleus) memset(in_nucleus, 1, V);
        free(pi);
        return;
    }
    int32_t *order = (int32_t *)malloc(sizeof(int32_t) * V);
    uint8_t *in_s = (uint8_t *)calloc(V, 1);
    for (int v = 0; v < V; ++v) order[v] = v;
    #pragma omp critical(orc_sort)
    {
        g_sort_pi = pi;
        qsort(order, V, sizeof(int32_t), cmp_desc);
    }
    double mass = 0.0;
    for (int r = 0; r < V; ++r) {
        in_s[order[r]] = 1;
        mass += pi[order[r]];
        if (mass >= top_p) break;
    }
    double cum = 0.0;
    int chosen = -1, last_in = -1;
    double lo = 0.0, hi = 0.0;
    for (int v = 0; v < V; ++v) {
        if (!in_s[v]) continue;
        last_in = v;
        double next = cum + pi[v] / mass;
        if (chosen < 0 && next > u) { chosen = v; lo = cum; hi = next; }
        cum = next;
    }
    if (chosen < 0) { chosen = last_in; lo = cum - pi[last_in] / mass; hi = 1.0; } /* u beyond the rounded total */
    *token_out = chosen;
    *logp_out = (float)log(pi[chosen]);
    if (nucleus_mass) *nucleus_mass = mass;
    if (cdf_lo) *cdf_lo = lo;
    if (cdf_hi) *cdf_hi = hi;
    if (in_nucleus) memcpy(in_nucleus, in_s, V);
    free(order); free(in_s); free(pi);
}

/* log_softmax(logits / T)[token] for a given token (used when a token is teacher-forced). */
float orc_logprob_of(const float *logits, int V, double temperature, int32_t token) {
    double m = (double)logits[0] / temperature;
    for (int v = 1; v < V; ++v) if ((double)logits[v] / temperature > m) m = (double)logits[v] / temperature;
    double Z = 0.0;
    for (int v = 0; v < V; ++v) Z += exp((double)logits[v] / temperature - m);
    return (float)((double)logits[token] / temperature - m - log(Z));
}
