/*
 * CPU oracle for the review step of Cascade Speculative Drafting (arXiv 2312.11462).
 *
 * TEST INFRASTRUCTURE ONLY.  This file is the slow, plain statement of what the hot path
 * computes.  It is linked by the tests, by the smoke check and by the benchmark's CPU-baseline
 * leg, never by the product library, and it shares no code, header, table or constant generator
 * with the CUDA path.  Floating point is carried in double precision; the only narrower values
 * are the ones the data formats fix: bf16 weights (input), bf16 K/V cache entries (rounded to
 * nearest-even when a position is appended) and fp32 logits (the interface type between the
 * forward pass and the review rule).
 *
 * What each part follows:
 *   orc_spec_accept      Section 2 (proposing / reviewing stages), Section 3.1 (lenience, greedy)
 *   orc_mag_draft        Section 3.3 (the definition in words; Appendix A gives a tensor formulation)
 *   orc_review_forward   the reviewer scores every drafted position in ONE forward pass
 *                        (Sections 1 and 2); the architectures are the families named in Section 5.1
 *   orc_cascade_generate Algorithm 1 (for-loop = horizontal cascade, recursion = vertical)
 *   orc_philox4x32_10    Salmon et al., "Parallel random numbers: as easy as 1, 2, 3" (SC'11)
 *
 * Pins (tests marked "not gpu"): Philox known-answer vectors; exact joint law of the review
 * rule by enumeration on V=8, k=2; chi-square of emitted tokens against the target law; the
 * accepted-length law of Theorem 1 / Eq. 1; Max-Gram against brute-force longest-suffix search
 * and hand-worked cases; the forward pass against library models and library matmul / softmax /
 * attention in float64; greedy cascade output identical to target-only greedy decoding.
 * Parity unpinned: nothing in this file (the simulated EWIF table of Section 4 is not computed).
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

/* ------------------------------------------------------------------------------------------ */
/* bf16 helpers                                                                               */
/* ------------------------------------------------------------------------------------------ */
static inline double bf16_to_double(uint16_t h) {
    uint32_t u = (uint32_t)h << 16;
    float f;
    memcpy(&f, &u, 4);
    return (double)f;
}

/* round-to-nearest-even from double to bf16, decided in double (no float double-rounding) */
static uint16_t double_to_bf16(double x) {
    if (x != x) return 0x7FC0;
    float f = (float)x;
    uint32_t u;
    memcpy(&u, &f, 4);
    uint32_t lo_bits = u & 0xFFFF0000u;
    float lo_f;
    memcpy(&lo_f, &lo_bits, 4);
    if (isinf(lo_f)) return (uint16_t)(lo_bits >> 16);
    /* candidates around x: the truncation of f and its two neighbours in magnitude */
    uint32_t cand[3];
    cand[0] = lo_bits >> 16;
    cand[1] = cand[0] + 1;
    cand[2] = (cand[0] & 0x7FFF) ? cand[0] - 1 : cand[0];
    double best_err = 1e300;
    uint16_t best = (uint16_t)cand[0];
    for (int i = 0; i < 3; ++i) {
        uint16_t c = (uint16_t)cand[i];
        double v = bf16_to_double(c);
        if (isinf(v) || v != v) continue;
        double e = fabs(v - x);
        if (e < best_err || (e == best_err && (c & 1) == 0 && (best & 1) == 1)) {
            best_err = e;
            best = c;
        }
    }
    return best;
}

uint16_t orc_double_to_bf16(double x) { return double_to_bf16(x); }

/* Test hook: with `exact` on, cached K/V keep full precision, which lets the forward pass be
   compared with a library model that has no bf16 cache. */
static int g_kv_exact = 0;
void orc_set_kv_exact(int on) { g_kv_exact = on; }
/* the value a bf16 cache holds for x (the caches below keep that value in a double) */
static inline double kv_store(double x) { return g_kv_exact ? x : bf16_to_double(double_to_bf16(x)); }

/* ------------------------------------------------------------------------------------------ */
/* Philox4x32-10 (Salmon et al. 2011): counter (4 x u32), key (2 x u32), ten rounds.          */
/* ------------------------------------------------------------------------------------------ */
void orc_philox4x32_10(const uint32_t ctr[4], const uint32_t key[2], uint32_t out[4]) {
    uint32_t c0 = ctr[0], c1 = ctr[1], c2 = ctr[2], c3 = ctr[3];
    uint32_t k0 = key[0], k1 = key[1];
    for (int r = 0; r < 10; ++r) {
        uint64_t p0 = (uint64_t)0xD2511F53u * c0;
        uint64_t p1 = (uint64_t)0xCD9E8D57u * c2;
        uint32_t n0 = (uint32_t)(p1 >> 32) ^ c1 ^ k0;
        uint32_t n1 = (uint32_t)p1;
        uint32_t n2 = (uint32_t)(p0 >> 32) ^ c3 ^ k1;
        uint32_t n3 = (uint32_t)p0;
        c0 = n0; c1 = n1; c2 = n2; c3 = n3;
        k0 += 0x9E3779B9u;
        k1 += 0xBB67AE85u;
    }
    out[0] = c0; out[1] = c1; out[2] = c2; out[3] = c3;
}

/* u in [0,1): top 24 bits of a word */
static inline double word_to_uniform(uint32_t w) { return (double)(w >> 8) * (1.0 / 16777216.0); }

/* Draws for (seed, step, row, position): word 0 drives the accept test, word 1 the resample. */
static void review_uniforms(uint64_t seed, uint64_t step, int row, int pos, double* u, double* u2) {
    uint32_t ctr[4] = {(uint32_t)pos, (uint32_t)row, (uint32_t)step, (uint32_t)(step >> 32)};
    uint32_t key[2] = {(uint32_t)seed, (uint32_t)(seed >> 32)};
    uint32_t w[4];
    orc_philox4x32_10(ctr, key, w);
    *u = word_to_uniform(w[0]);
    *u2 = word_to_uniform(w[1]);
}

void orc_review_uniforms(uint64_t seed, uint64_t step, int row, int pos, double* u, double* u2) {
    review_uniforms(seed, step, row, pos, u, u2);
}

/* ------------------------------------------------------------------------------------------ */
/* Review rule (Section 2; lenience and greedy variant: Section 3.1)                          */
/* ------------------------------------------------------------------------------------------ */
static int argmax_f32(const float* x, int V) {
    int b = 0;
    for (int j = 1; j < V; ++j)
        if (x[j] > x[b]) b = j;
    return b;
}

/* p[j] = softmax(x / T)[j] in double */
static void softmax_T(const float* x, int V, double T, double* p) {
    double mx = (double)x[0];
    for (int j = 1; j < V; ++j)
        if ((double)x[j] > mx) mx = (double)x[j];
    double Z = 0.0;
    for (int j = 0; j < V; ++j) {
        p[j] = exp(((double)x[j] - mx) / T);
        Z += p[j];
    }
    for (int j = 0; j < V; ++j) p[j] /= Z;
}

/* inverse CDF in vocabulary order: smallest j with sum_{i<=j} r_i > u2 * S */
static int inverse_cdf(const double* r, int V, double u2, int* near_tie) {
    double S = 0.0;
    for (int j = 0; j < V; ++j) S += r[j];
    double target = u2 * S, cum = 0.0;
    int pick = -1, last_pos = -1;
    double lo = 0.0, hi = 0.0;
    for (int j = 0; j < V; ++j) {
        double prev = cum;
        cum += r[j];
        if (r[j] > 0.0) last_pos = j;
        if (pick < 0 && cum > target) {
            pick = j;
            lo = prev;
            hi = cum;
        }
    }
    if (pick < 0) {
        pick = last_pos;
        if (near_tie) *near_tie |= 2;
    } else if (near_tie) {
        double tol = 1e-11 * S;
        if (target - lo < tol || hi - target < tol) *near_tie |= 2;
    }
    return pick;
}

/*
 * target_logits [rows, k+1, V], draft_logits [rows, k, V] or NULL, onehot [rows, k] or NULL
 * (a non-zero entry, or draft_logits == NULL, means that position's draft law is the point
 * mass on its token, as for a statistical drafter), tokens [rows, k].
 * temperature == 0: greedy review (accept iff the token is the target's argmax).
 * near_tie (optional) [rows]: bit 0 = an accept test within 1e-5 relative of equality,
 * bit 1 = the resample's u*S within 1e-11*S of a boundary of the chosen interval.
 */
int orc_spec_accept(const float* target_logits, const float* draft_logits, const int32_t* onehot,
                    const int32_t* tokens, int rows, int k, int V, float temperature,
                    float lenience, uint64_t seed, uint64_t step, int32_t* n_accepted,
                    int32_t* out_token, int32_t* near_tie) {
    if (rows < 0 || k < 0 || V <= 0 || temperature < 0.0f || lenience < 1.0f) return 1;
    double* p = (double*)malloc(sizeof(double) * (size_t)V);
    double* q = (double*)malloc(sizeof(double) * (size_t)V);
    double* r = (double*)malloc(sizeof(double) * (size_t)V);
    for (int row = 0; row < rows; ++row) {
        const float* t = target_logits + (size_t)row * (k + 1) * V;
        const float* d = draft_logits ? draft_logits + (size_t)row * k * V : NULL;
        const int32_t* tok = tokens + (size_t)row * k;
        int flag = 0;
        if (temperature == 0.0f) {
            int n = 0;
            while (n < k && tok[n] == argmax_f32(t + (size_t)n * V, V)) ++n;
            n_accepted[row] = n;
            out_token[row] = argmax_f32(t + (size_t)n * V, V);
            if (near_tie) near_tie[row] = 0;
            continue;
        }
        double T = (double)temperature, l = (double)lenience;
        int n = k;
        for (int i = 0; i < k; ++i) {
            int x = tok[i];
            int point_mass = (d == NULL) || (onehot && onehot[(size_t)row * k + i]);
            softmax_T(t + (size_t)i * V, V, T, p);
            double qx = 1.0;
            if (!point_mass) {
                softmax_T(d + (size_t)i * V, V, T, q);
                qx = q[x];
            }
            double u, u2;
            review_uniforms(seed, step, row, i, &u, &u2);
            /* Appendix B: no lenience between the statistical drafter and its reviewer */
            double lhs = u * qx, rhs = (point_mass ? 1.0 : l) * p[x];
            double big = lhs > rhs ? lhs : rhs;
            if (fabs(lhs - rhs) <= 1e-5 * big) flag |= 1;
            if (lhs < rhs) continue; /* accepted */
            /* first rejection: resample position i from norm(max(0, p - q)) */
            n = i;
            double S = 0.0;
            for (int j = 0; j < V; ++j) {
                double qj = point_mass ? (j == x ? 1.0 : 0.0) : q[j];
                r[j] = p[j] - qj;
                if (r[j] < 0.0) r[j] = 0.0;
                S += r[j];
            }
            if (!(S > 0.0) || !isfinite(S)) memcpy(r, p, sizeof(double) * (size_t)V);
            out_token[row] = inverse_cdf(r, V, u2, &flag);
            break;
        }
        if (n == k) { /* every draft accepted: one more token from the target's next law */
            double u, u2;
            review_uniforms(seed, step, row, k, &u, &u2);
            softmax_T(t + (size_t)k * V, V, T, p);
            out_token[row] = inverse_cdf(p, V, u2, &flag);
        }
        n_accepted[row] = n;
        if (near_tie) near_tie[row] = flag;
    }
    free(p); free(q); free(r);
    return 0;
}

/* ------------------------------------------------------------------------------------------ */
/* Max-Gram (Section 3.3, Appendix A)                                                         */
/* ------------------------------------------------------------------------------------------ */
/*
 * One search, as Section 3.3 words it: the longest run of tokens at the end of the sequence (at
 * most max_order of them) that also occurs in the haystack, the earliest such occurrence.  An
 * occurrence counts only if at least one haystack token follows it (so the proposal is never
 * empty, and a sequence that still ends with the haystack itself does not match its own tail).
 * Returns the haystack index of the token after the occurrence, or -1 without any match.
 */
static int mag_search(const int32_t* hay, int L, const int32_t* seq, int T, int max_order) {
    int longest = T < max_order ? T : max_order;
    for (int order = longest; order >= 1; --order) {
        const int32_t* tail = seq + (T - order);
        for (int j = 0; j + order < L; ++j) {
            int same = 1;
            for (int e = 0; e < order && same; ++e) same = hay[j + e] == tail[e];
            if (same) return j + order;
        }
    }
    return -1;
}

/*
 * Propose n tokens after seq[0..T): copy the haystack tokens that follow the match; when the
 * haystack ends first, or nothing matches (then one token comes from the bigram table
 * next[last token]), search again on the extended sequence until n tokens exist.
 */
int orc_mag_draft(const int32_t* hay, int L, const int32_t* bigram_next, int V, const int32_t* seq,
                  int T, int n, int max_order, int32_t* out) {
    if (T < 1 || n < 0 || max_order < 1) return -1;
    int32_t* cur = (int32_t*)malloc(sizeof(int32_t) * (size_t)(T + n));
    memcpy(cur, seq, sizeof(int32_t) * (size_t)T);
    int len = T, made = 0;
    while (made < n) {
        int idx = mag_search(hay, L, cur, len, max_order);
        if (idx < 0) {
            int32_t last = cur[len - 1];
            int32_t nx = (last >= 0 && last < V) ? bigram_next[last] : 0;
            cur[len++] = nx;
            out[made++] = nx;
        } else {
            while (made < n && idx < L) {
                cur[len++] = hay[idx];
                out[made++] = hay[idx++];
            }
        }
    }
    free(cur);
    return made;
}

/* ------------------------------------------------------------------------------------------ */
/* Transformer forward over a block of m positions with a bf16 KV cache                       */
/* ------------------------------------------------------------------------------------------ */
typedef struct {
    int32_t arch; /* 0 = decoder-only (RMSNorm, RoPE, SwiGLU), 1 = encoder-decoder (T5 v1.1 style) */
    int32_t n_layers, n_enc_layers, d_model, n_heads, d_head, d_ff, vocab;
    int32_t max_seq, max_rows, max_enc_len, rel_buckets, rel_max_dist;
    float norm_eps, rope_theta;
} orc_model_config;

typedef struct {
    const uint16_t *norm1, *wq, *wk, *wv, *wo, *norm_x, *xq, *xk, *xv, *xo, *norm2, *wgate, *wup,
        *wdown;
} orc_layer;

typedef struct orc_model {
    orc_model_config c;
    const uint16_t* blob;
    const uint16_t *embed, *final_norm, *lm_head, *enc_rel_bias, *dec_rel_bias, *enc_final_norm;
    orc_layer* enc;
    orc_layer* dec;
    double* kcache; /* [layer][max_seq][d_inner], bf16-representable values */
    double* vcache;
    double* xk;     /* cross K [layer][max_enc_len][d_inner] */
    double* xv;
    int enc_len;
} orc_model;

static size_t align_elems(size_t n) { return (n + 127) / 128 * 128; }

static const uint16_t* take(const uint16_t* blob, size_t* off, size_t n) {
    const uint16_t* p = blob + *off;
    *off = align_elems(*off + n);
    return p;
}

size_t orc_model_weight_elems(const orc_model_config* c) {
    size_t d = c->d_model, di = (size_t)c->n_heads * c->d_head, ff = c->d_ff, V = c->vocab;
    size_t off = 0;
    off = align_elems(off + V * d);
    size_t attn = align_elems(di * d) * 3 + align_elems(d * di);
    size_t ffn = align_elems(ff * d) * 2 + align_elems(d * ff);
    if (c->arch == 0) {
        off += (size_t)c->n_layers * (2 * align_elems(d) + attn + ffn);
    } else {
        off += align_elems((size_t)c->rel_buckets * c->n_heads);
        off += (size_t)c->n_enc_layers * (2 * align_elems(d) + attn + ffn);
        off += align_elems(d);
        off += align_elems((size_t)c->rel_buckets * c->n_heads);
        off += (size_t)c->n_layers * (3 * align_elems(d) + 2 * attn + ffn);
    }
    off += align_elems(d);
    off += align_elems(V * d);
    return off;
}

static void take_attn(const uint16_t* blob, size_t* off, size_t di, size_t d, const uint16_t** q,
                      const uint16_t** k, const uint16_t** v, const uint16_t** o) {
    *q = take(blob, off, di * d);
    *k = take(blob, off, di * d);
    *v = take(blob, off, di * d);
    *o = take(blob, off, d * di);
}

orc_model* orc_model_create(const orc_model_config* c, const uint16_t* blob) {
    orc_model* m = (orc_model*)calloc(1, sizeof(orc_model));
    m->c = *c;
    m->blob = blob;
    size_t d = c->d_model, di = (size_t)c->n_heads * c->d_head, ff = c->d_ff, V = c->vocab;
    size_t off = 0;
    m->embed = take(blob, &off, V * d);
    m->dec = (orc_layer*)calloc((size_t)c->n_layers, sizeof(orc_layer));
    if (c->arch == 1) {
        m->enc = (orc_layer*)calloc((size_t)c->n_enc_layers, sizeof(orc_layer));
        m->enc_rel_bias = take(blob, &off, (size_t)c->rel_buckets * c->n_heads);
        for (int l = 0; l < c->n_enc_layers; ++l) {
            orc_layer* y = &m->enc[l];
            y->norm1 = take(blob, &off, d);
            take_attn(blob, &off, di, d, &y->wq, &y->wk, &y->wv, &y->wo);
            y->norm2 = take(blob, &off, d);
            y->wgate = take(blob, &off, ff * d);
            y->wup = take(blob, &off, ff * d);
            y->wdown = take(blob, &off, d * ff);
        }
        m->enc_final_norm = take(blob, &off, d);
        m->dec_rel_bias = take(blob, &off, (size_t)c->rel_buckets * c->n_heads);
    }
    for (int l = 0; l < c->n_layers; ++l) {
        orc_layer* y = &m->dec[l];
        y->norm1 = take(blob, &off, d);
        take_attn(blob, &off, di, d, &y->wq, &y->wk, &y->wv, &y->wo);
        if (c->arch == 1) {
            y->norm_x = take(blob, &off, d);
            take_attn(blob, &off, di, d, &y->xq, &y->xk, &y->xv, &y->xo);
        }
        y->norm2 = take(blob, &off, d);
        y->wgate = take(blob, &off, ff * d);
        y->wup = take(blob, &off, ff * d);
        y->wdown = take(blob, &off, d * ff);
    }
    m->final_norm = take(blob, &off, d);
    m->lm_head = take(blob, &off, V * d);
    size_t kv = (size_t)c->n_layers * c->max_seq * di;
    m->kcache = (double*)calloc(kv, sizeof(double));
    m->vcache = (double*)calloc(kv, sizeof(double));
    if (c->arch == 1) {
        size_t x = (size_t)c->n_layers * c->max_enc_len * di;
        m->xk = (double*)calloc(x, sizeof(double));
        m->xv = (double*)calloc(x, sizeof(double));
    }
    return m;
}

void orc_model_destroy(orc_model* m) {
    if (!m) return;
    free(m->enc); free(m->dec); free(m->kcache); free(m->vcache); free(m->xk); free(m->xv);
    free(m);
}

/* Test hook: with 1, every result of a contraction is rounded to fp32 before it is used; with 2,
   the contraction itself runs in fp32 (fp32 operands, products and running sum, in index order).
   Both are equally correct ways to carry the arithmetic; the tests use them to measure how far two
   correct implementations drift apart once both round K/V to bf16. */
static int g_linear_f32 = 0;
void orc_set_linear_f32(int on) { g_linear_f32 = on; }

/* Y[r][n] = sum_k X[r][k] * W[n][k]; W bf16 [N,K] row-major */
static void linear(const uint16_t* W, int N, int K, const double* X, int m, double* Y) {
#pragma omp parallel for schedule(static)
    for (int n = 0; n < N; ++n) {
        const uint16_t* w = W + (size_t)n * K;
        for (int r = 0; r < m; ++r) {
            const double* x = X + (size_t)r * K;
            if (g_linear_f32 == 2) {
                float acc32 = 0.f;
                for (int k = 0; k < K; ++k) acc32 += (float)bf16_to_double(w[k]) * (float)x[k];
                Y[(size_t)r * N + n] = (double)acc32;
                continue;
            }
            double acc = 0.0;
            for (int k = 0; k < K; ++k) acc += bf16_to_double(w[k]) * x[k];
            Y[(size_t)r * N + n] = g_linear_f32 ? (double)(float)acc : acc;
        }
    }
}

/* test hook: fp32 activations in, fp32 out, same contraction */
void orc_linear(const uint16_t* W, int N, int K, const float* X, int m, float* Y) {
    double* xd = (double*)malloc(sizeof(double) * (size_t)m * K);
    double* yd = (double*)malloc(sizeof(double) * (size_t)m * N);
    for (size_t i = 0; i < (size_t)m * K; ++i) xd[i] = (double)X[i];
    linear(W, N, K, xd, m, yd);
    for (size_t i = 0; i < (size_t)m * N; ++i) Y[i] = (float)yd[i];
    free(xd); free(yd);
}

/* root-mean-square norm with gain: y = x / sqrt(mean(x^2) + eps) * g  (no mean-centering) */
static void rmsnorm(const double* x, const uint16_t* g, int d, double eps, double* y) {
    double ss = 0.0;
    for (int i = 0; i < d; ++i) ss += x[i] * x[i];
    double inv = 1.0 / sqrt(ss / d + eps);
    for (int i = 0; i < d; ++i) y[i] = x[i] * inv * bf16_to_double(g[i]);
}

/* rotary embedding on one head vector at position pos: pairs (i, i + Dh/2) */
static void rope(double* v, int Dh, int pos, double theta) {
    int half = Dh / 2;
    for (int i = 0; i < half; ++i) {
        double ang = (double)pos * pow(theta, -2.0 * i / Dh);
        double c = cos(ang), s = sin(ang);
        double a = v[i], b = v[i + half];
        v[i] = a * c - b * s;
        v[i + half] = a * s + b * c;
    }
}

/*
 * Relative-position bucket of the T5 family: half the buckets hold exact small offsets, the
 * rest are spaced logarithmically up to max_dist.  rel = key position - query position.
 * The logarithmic bucket index floor(log(n/E) / log(D/E) * (B-E)) is evaluated exactly with
 * integers as the largest j with D^j * E^(B-E-j) <= n^(B-E)  (n < D <= 128 and B-E <= 16 keep
 * every product below 2^112).
 */
int orc_rel_bucket(int rel, int bidirectional, int n_buckets, int max_dist) {
    int bucket = 0, B = n_buckets, n;
    if (bidirectional) {
        B /= 2;
        if (rel > 0) bucket += B;
        n = rel < 0 ? -rel : rel;
    } else {
        n = rel < 0 ? -rel : 0;
    }
    int E = B / 2;
    if (n < E) return bucket + n;
    if (n >= max_dist) return bucket + B - 1;
    int span = B - E, j_best = 0;
    for (int j = 1; j <= span; ++j) {
        unsigned __int128 lhs = 1, rhs = 1;
        for (int t = 0; t < j; ++t) lhs *= (unsigned)max_dist;
        for (int t = 0; t < span - j; ++t) lhs *= (unsigned)E;
        for (int t = 0; t < span; ++t) rhs *= (unsigned)n;
        if (lhs <= rhs) j_best = j;
    }
    int b = E + j_best;
    if (b > B - 1) b = B - 1;
    return bucket + b;
}

static double gelu_tanh(double x) {
    return 0.5 * x * (1.0 + tanh(0.7978845608028654 * (x + 0.044715 * x * x * x)));
}
static double silu(double x) { return x / (1.0 + exp(-x)); }

/* softmax(scores) . V for one query row of one head against n_keys cached positions;
   bias may be NULL. */
static void attend(const double* q, const double* K, const double* Vv, int stride, int n_keys,
                   int Dh, double scale, const double* bias, double* out, double* scores) {
    double mx = -INFINITY;
    for (int j = 0; j < n_keys; ++j) {
        const double* kj = K + (size_t)j * stride;
        double s = 0.0;
        for (int e = 0; e < Dh; ++e) s += q[e] * kj[e];
        s = s * scale + (bias ? bias[j] : 0.0);
        scores[j] = s;
        if (s > mx) mx = s;
    }
    double Z = 0.0;
    for (int j = 0; j < n_keys; ++j) {
        scores[j] = exp(scores[j] - mx);
        Z += scores[j];
    }
    for (int e = 0; e < Dh; ++e) out[e] = 0.0;
    for (int j = 0; j < n_keys; ++j) {
        const double* vj = Vv + (size_t)j * stride;
        double pj = scores[j] / Z;
        for (int e = 0; e < Dh; ++e) out[e] += pj * vj[e];
    }
}

static void ffn_block(const orc_model* M, const orc_layer* y, double* x, int m, double* h,
                      double* g, double* u, double* tmp) {
    int d = M->c.d_model, ff = M->c.d_ff;
    for (int r = 0; r < m; ++r) rmsnorm(x + (size_t)r * d, y->norm2, d, M->c.norm_eps, h + (size_t)r * d);
    linear(y->wgate, ff, d, h, m, g);
    linear(y->wup, ff, d, h, m, u);
    for (size_t i = 0; i < (size_t)m * ff; ++i)
        g[i] = (M->c.arch == 0 ? silu(g[i]) : gelu_tanh(g[i])) * u[i];
    linear(y->wdown, d, ff, g, m, tmp);
    for (size_t i = 0; i < (size_t)m * d; ++i) x[i] += tmp[i];
}

/* Encoder pass (encoder-decoder models): fills the static cross-attention K/V of every
   decoder layer from the encoder's final hidden states. */
int orc_encoder_forward(orc_model* M, const int32_t* tokens, int n) {
    const orc_model_config* c = &M->c;
    if (c->arch != 1 || n < 1 || n > c->max_enc_len) return 1;
    int d = c->d_model, H = c->n_heads, Dh = c->d_head, di = H * Dh, ff = c->d_ff;
    double* x = (double*)malloc(sizeof(double) * (size_t)n * d);
    double* h = (double*)malloc(sizeof(double) * (size_t)n * d);
    double* q = (double*)malloc(sizeof(double) * (size_t)n * di);
    double* k = (double*)malloc(sizeof(double) * (size_t)n * di);
    double* v = (double*)malloc(sizeof(double) * (size_t)n * di);
    double* o = (double*)malloc(sizeof(double) * (size_t)n * di);
    double* tmp = (double*)malloc(sizeof(double) * (size_t)n * d);
    double* g = (double*)malloc(sizeof(double) * (size_t)n * ff);
    double* u = (double*)malloc(sizeof(double) * (size_t)n * ff);
    for (int r = 0; r < n; ++r) {
        int t = tokens[r];
        if (t < 0 || t >= c->vocab) t = 0;
        for (int i = 0; i < d; ++i) x[(size_t)r * d + i] = bf16_to_double(M->embed[(size_t)t * d + i]);
    }
    for (int l = 0; l < c->n_enc_layers; ++l) {
        const orc_layer* y = &M->enc[l];
        for (int r = 0; r < n; ++r) rmsnorm(x + (size_t)r * d, y->norm1, d, c->norm_eps, h + (size_t)r * d);
        linear(y->wq, di, d, h, n, q);
        linear(y->wk, di, d, h, n, k);
        linear(y->wv, di, d, h, n, v);
        for (size_t i = 0; i < (size_t)n * di; ++i) {
            k[i] = kv_store(k[i]);
            v[i] = kv_store(v[i]);
        }
#pragma omp parallel for schedule(static)
        for (int r = 0; r < n; ++r) {
            double* bias = (double*)malloc(sizeof(double) * (size_t)n);
            double* sc = (double*)malloc(sizeof(double) * (size_t)n);
            for (int hd = 0; hd < H; ++hd) {
                for (int j = 0; j < n; ++j) {
                    int b = orc_rel_bucket(j - r, 1, c->rel_buckets, c->rel_max_dist);
                    bias[j] = bf16_to_double(M->enc_rel_bias[(size_t)b * H + hd]);
                }
                attend(q + (size_t)r * di + (size_t)hd * Dh, k + (size_t)hd * Dh, v + (size_t)hd * Dh, di, n,
                       Dh, 1.0, bias, o + (size_t)r * di + (size_t)hd * Dh, sc);
            }
            free(bias); free(sc);
        }
        linear(y->wo, d, di, o, n, tmp);
        for (size_t i = 0; i < (size_t)n * d; ++i) x[i] += tmp[i];
        ffn_block(M, y, x, n, h, g, u, tmp);
    }
    for (int r = 0; r < n; ++r) rmsnorm(x + (size_t)r * d, M->enc_final_norm, d, c->norm_eps, h + (size_t)r * d);
    for (int l = 0; l < c->n_layers; ++l) {
        const orc_layer* y = &M->dec[l];
        linear(y->xk, di, d, h, n, k);
        linear(y->xv, di, d, h, n, v);
        double* K = M->xk + (size_t)l * c->max_enc_len * di;
        double* Vv = M->xv + (size_t)l * c->max_enc_len * di;
        for (size_t i = 0; i < (size_t)n * di; ++i) {
            K[i] = kv_store(k[i]);
            Vv[i] = kv_store(v[i]);
        }
    }
    M->enc_len = n;
    free(x); free(h); free(q); free(k); free(v); free(o); free(tmp); free(g); free(u);
    return 0;
}

/*
 * One forward pass over m new positions kv_len .. kv_len+m-1 (the drafted block preceded by the
 * last committed token).  Reads cache rows [0, kv_len), writes rows [kv_len, kv_len+m), and
 * returns fp32 logits [m, V]; row r is the model's next-token law after position kv_len+r.
 */
static int forward_rows(orc_model* M, const int32_t* tokens, int m, int kv_len, float* logits, int first_row) {
    const orc_model_config* c = &M->c;
    if (m < 1 || kv_len < 0 || kv_len + m > c->max_seq || first_row < 0 || first_row >= m) return 1;
    if (c->arch == 1 && M->enc_len < 1) return 2;
    int d = c->d_model, H = c->n_heads, Dh = c->d_head, di = H * Dh, ff = c->d_ff, V = c->vocab;
    double* x = (double*)malloc(sizeof(double) * (size_t)m * d);
    double* h = (double*)malloc(sizeof(double) * (size_t)m * d);
    double* q = (double*)malloc(sizeof(double) * (size_t)m * di);
    double* k = (double*)malloc(sizeof(double) * (size_t)m * di);
    double* v = (double*)malloc(sizeof(double) * (size_t)m * di);
    double* o = (double*)malloc(sizeof(double) * (size_t)m * di);
    double* tmp = (double*)malloc(sizeof(double) * (size_t)m * d);
    double* g = (double*)malloc(sizeof(double) * (size_t)m * ff);
    double* u = (double*)malloc(sizeof(double) * (size_t)m * ff);
    int n_out = m - first_row;      /* logits are wanted for rows first_row .. m-1 */
    double* lg = (double*)malloc(sizeof(double) * (size_t)n_out * V);
    for (int r = 0; r < m; ++r) {
        int t = tokens[r];
        if (t < 0 || t >= V) t = 0;
        for (int i = 0; i < d; ++i) x[(size_t)r * d + i] = bf16_to_double(M->embed[(size_t)t * d + i]);
    }
    double scale = c->arch == 0 ? 1.0 / sqrt((double)Dh) : 1.0;
    for (int l = 0; l < c->n_layers; ++l) {
        const orc_layer* y = &M->dec[l];
        double* K = M->kcache + (size_t)l * c->max_seq * di;
        double* Vv = M->vcache + (size_t)l * c->max_seq * di;
        /* self-attention */
        for (int r = 0; r < m; ++r) rmsnorm(x + (size_t)r * d, y->norm1, d, c->norm_eps, h + (size_t)r * d);
        linear(y->wq, di, d, h, m, q);
        linear(y->wk, di, d, h, m, k);
        linear(y->wv, di, d, h, m, v);
        for (int r = 0; r < m; ++r) {
            int pos = kv_len + r;
            if (c->arch == 0)
                for (int hd = 0; hd < H; ++hd) {
                    rope(q + (size_t)r * di + (size_t)hd * Dh, Dh, pos, c->rope_theta);
                    rope(k + (size_t)r * di + (size_t)hd * Dh, Dh, pos, c->rope_theta);
                }
            for (int i = 0; i < di; ++i) {
                K[(size_t)pos * di + i] = kv_store(k[(size_t)r * di + i]);
                Vv[(size_t)pos * di + i] = kv_store(v[(size_t)r * di + i]);
            }
        }
#pragma omp parallel for schedule(static) collapse(2)
        for (int r = 0; r < m; ++r) {
            for (int hd = 0; hd < H; ++hd) {
                int pos = kv_len + r, n_keys = pos + 1; /* causal: keys 0..pos */
                double* sc = (double*)malloc(sizeof(double) * (size_t)n_keys);
                double* bias = NULL;
                if (c->arch == 1) {
                    bias = (double*)malloc(sizeof(double) * (size_t)n_keys);
                    for (int j = 0; j < n_keys; ++j) {
                        int b = orc_rel_bucket(j - pos, 0, c->rel_buckets, c->rel_max_dist);
                        bias[j] = bf16_to_double(M->dec_rel_bias[(size_t)b * H + hd]);
                    }
                }
                attend(q + (size_t)r * di + (size_t)hd * Dh, K + (size_t)hd * Dh, Vv + (size_t)hd * Dh, di, n_keys,
                       Dh, scale, bias, o + (size_t)r * di + (size_t)hd * Dh, sc);
                free(sc); free(bias);
            }
        }
        linear(y->wo, d, di, o, m, tmp);
        for (size_t i = 0; i < (size_t)m * d; ++i) x[i] += tmp[i];
        /* cross-attention over the static encoder K/V (encoder-decoder only) */
        if (c->arch == 1) {
            const double* XK = M->xk + (size_t)l * c->max_enc_len * di;
            const double* XV = M->xv + (size_t)l * c->max_enc_len * di;
            for (int r = 0; r < m; ++r) rmsnorm(x + (size_t)r * d, y->norm_x, d, c->norm_eps, h + (size_t)r * d);
            linear(y->xq, di, d, h, m, q);
#pragma omp parallel for schedule(static) collapse(2)
            for (int r = 0; r < m; ++r) {
                for (int hd = 0; hd < H; ++hd) {
                    double* sc = (double*)malloc(sizeof(double) * (size_t)M->enc_len);
                    attend(q + (size_t)r * di + (size_t)hd * Dh, XK + (size_t)hd * Dh, XV + (size_t)hd * Dh, di,
                           M->enc_len, Dh, 1.0, NULL, o + (size_t)r * di + (size_t)hd * Dh, sc);
                    free(sc);
                }
            }
            linear(y->xo, d, di, o, m, tmp);
            for (size_t i = 0; i < (size_t)m * d; ++i) x[i] += tmp[i];
        }
        ffn_block(M, y, x, m, h, g, u, tmp);
    }
    for (int r = 0; r < m; ++r) rmsnorm(x + (size_t)r * d, M->final_norm, d, c->norm_eps, h + (size_t)r * d);
    linear(M->lm_head, V, d, h + (size_t)first_row * d, n_out, lg);
    for (size_t i = 0; i < (size_t)n_out * V; ++i) logits[i] = (float)lg[i];
    free(x); free(h); free(q); free(k); free(v); free(o); free(tmp); free(g); free(u); free(lg);
    return 0;
}

int orc_review_forward(orc_model* M, const int32_t* tokens, int m, int kv_len, float* logits) {
    return forward_rows(M, tokens, m, kv_len, logits, 0);
}

/* ------------------------------------------------------------------------------------------ */
/* Algorithm 1: CascadeSpeculativeDraftingStep, driven until max_new tokens exist             */
/* ------------------------------------------------------------------------------------------ */
/*
 * Written for checking by eye, not for speed: nothing is cached between reviews.  A review runs
 * the reviewing model over the WHOLE sequence with a fresh cache and keeps the rows it needs, and
 * the law every pending token was drawn from is kept in a plain per-position list (curProbs of
 * the algorithm).  The result does not depend on this choice: a position's K/V and logits are
 * functions of the tokens before it alone.
 */
typedef struct {
    int64_t tokens;             /* tokens generated */
    int64_t reviews[8];         /* review calls per level (0 = target) */
    int64_t forwards[8];        /* forward passes per level (one per review here) */
    int64_t drafted[8];         /* drafted tokens presented to the level's reviews */
    int64_t accepted[8];        /* of which accepted */
    int64_t mag_calls;
    int64_t mag_tokens;
    int64_t near_ties;          /* reviews whose decision lay within rounding of a threshold */
    int64_t first_near_tie;     /* index (among generated tokens) where the first such review began, -1: none */
} orc_stats;

typedef struct {
    int n_levels;               /* neural models: level 0 = target, 1.. = drafts; level n_levels = Max-Gram */
    orc_model** models;
    const int32_t* hay; int L;  /* Max-Gram haystack */
    int dynamic_hay;            /* 1: the haystack is followed by everything generated so far */
    const int32_t* bigram; int max_order;
    const int32_t* K;           /* n_levels x n_levels budget matrix */
    int max_block;              /* most drafted tokens one review takes */
    double lenience; float temperature;
    uint64_t seed, step;
    int32_t* seq; int len;      /* curGen */
    float** probs;              /* curProbs: per position the fp32 logits of the law that proposed the
                                   token, NULL = point mass (prefix and Max-Gram tokens) */
    int V, cap, init_len;
    float* margins;             /* optional: top-2 logit margin of the target at each new token */
    orc_stats* st;
} cascade;

float orc_top2_margin(const float* x, int V) {
    float a = -INFINITY, b = -INFINITY;
    for (int j = 0; j < V; ++j) {
        if (x[j] > a) { b = a; a = x[j]; }
        else if (x[j] > b) b = x[j];
    }
    return a - b;
}

static void set_prob(cascade* cs, int pos, const float* logits) {
    free(cs->probs[pos]);
    cs->probs[pos] = NULL;
    if (logits) {
        cs->probs[pos] = (float*)malloc(sizeof(float) * (size_t)cs->V);
        memcpy(cs->probs[pos], logits, sizeof(float) * (size_t)cs->V);
    }
}

/* The statistical drafter appends `want` tokens (base case of the recursion). */
static int statistical_draft(cascade* cs, int want) {
    if (want < 1) want = 1;
    if (cs->len + want > cs->cap) return 3;
    const int32_t* hay = cs->hay;
    int L = cs->L;
    int32_t* joined = NULL;
    if (cs->dynamic_hay) {      /* Section 3.3: "... the initial input (or existing generation)": both */
        int gen = cs->len - cs->init_len;
        joined = (int32_t*)malloc(sizeof(int32_t) * (size_t)(L + gen + 1));
        memcpy(joined, cs->hay, sizeof(int32_t) * (size_t)L);
        memcpy(joined + L, cs->seq + cs->init_len, sizeof(int32_t) * (size_t)gen);
        hay = joined;
        L += gen;
    }
    orc_mag_draft(hay, L, cs->bigram, cs->V, cs->seq, cs->len, want, cs->max_order, cs->seq + cs->len);
    free(joined);
    for (int i = 0; i < want; ++i) set_prob(cs, cs->len + i, NULL);
    cs->len += want;
    cs->st->mag_calls += 1;
    cs->st->mag_tokens += want;
    return 0;
}

/* review(M, curGen, curProbs, l) of Algorithm 1 for the nd pending tokens at positions P .. P+nd-1 */
static int review(cascade* cs, int r, int P, int nd) {
    int V = cs->V;
    float* law = (float*)malloc(sizeof(float) * (size_t)(nd + 1) * V);
    /* inputs 0 .. P+nd-1; output row j is the law of position j+1, so rows P-1 .. P+nd-1 are wanted */
    if (forward_rows(cs->models[r], cs->seq, P + nd, 0, law, P - 1)) { free(law); return 4; }
    cs->st->forwards[r] += 1;
    float* dl = NULL;
    int32_t* onehot = (int32_t*)calloc((size_t)(nd > 0 ? nd : 1), sizeof(int32_t));
    if (cs->temperature > 0.0f && nd > 0) {
        dl = (float*)calloc((size_t)nd * V, sizeof(float));
        for (int i = 0; i < nd; ++i) {
            if (!cs->probs[P + i]) onehot[i] = 1;
            else memcpy(dl + (size_t)i * V, cs->probs[P + i], sizeof(float) * (size_t)V);
        }
    }
    int32_t n_acc = 0, out_tok = 0, tie = 0;
    float l = (r == 0) ? 1.0f : (float)cs->lenience;   /* "if isFirstCall: l <- 1" */
    orc_spec_accept(law, dl, onehot, cs->seq + P, 1, nd, V, cs->temperature, l, cs->seed, cs->step++,
                    &n_acc, &out_tok, &tie);
    free(dl); free(onehot);
    if (tie) {
        if (cs->st->near_ties == 0) cs->st->first_near_tie = P - cs->init_len;
        cs->st->near_ties += 1;
    }
    cs->st->reviews[r] += 1;
    cs->st->drafted[r] += nd;
    cs->st->accepted[r] += n_acc;
    /* the accepted tokens and the one emitted after them now follow level r's own law */
    cs->seq[P + n_acc] = out_tok;
    for (int i = 0; i <= n_acc; ++i) {
        set_prob(cs, P + i, r > 0 ? law + (size_t)i * V : NULL);
        if (r == 0 && cs->margins) cs->margins[P + i - cs->init_len] = orc_top2_margin(law + (size_t)i * V, V);
    }
    for (int i = n_acc + 1; i < nd; ++i) set_prob(cs, P + i, NULL);   /* rejected tokens are gone */
    cs->len = P + n_acc + 1;
    free(law);
    return 0;
}

/* One call of the algorithm with level r as the reviewer ("target" of the call) and the levels
   below it as its draft list; r == n_levels is the call whose draft list is empty. */
static int cascade_step(cascade* cs, int r, int want) {
    if (r == cs->n_levels) return statistical_draft(cs, want);
    int n = cs->n_levels, P = cs->len;
    for (int i = r; i < n; ++i) {                 /* horizontal cascade: slot i belongs to level i + 1 */
        int k_i = cs->K[(size_t)r * n + i];
        if (k_i <= 0) continue;
        int slot_start = cs->len;
        while (cs->len - slot_start < k_i) {      /* vertical cascade */
            int rc = cascade_step(cs, i + 1, k_i - (cs->len - slot_start));
            if (rc) return rc;
        }
    }
    int nd = cs->len - P;
    for (int i = cs->max_block; i < nd; ++i) set_prob(cs, P + i, NULL);   /* surplus drafts are dropped */
    if (nd > cs->max_block) nd = cs->max_block;
    cs->len = P + nd;
    if (P + nd + 1 > cs->cap) return 3;
    return review(cs, r, P, nd);
}

/*
 * models[0] is the target, models[1..n_levels-1] the neural drafts (largest first); Max-Gram
 * sits below them.  K is (n_levels x n_levels) row-major, upper-triangular: K[r][c] is the
 * budget of the slot that level c+1 drafts when level r reviews.  For encoder-decoder models
 * `hay` is the encoder input (the encoder is run here) and init_seq the decoder start; for
 * decoder-only models hay and init_seq are both the prompt.
 */
int orc_cascade_generate(orc_model** models, int n_levels, const int32_t* hay, int L,
                         const int32_t* bigram_next, int max_order, const int32_t* K,
                         int max_block, float lenience, float temperature, uint64_t seed,
                         const int32_t* init_seq, int init_len, int max_new, int dynamic_hay,
                         int32_t* out_tokens, int32_t* out_len, float* margins, orc_stats* stats) {
    if (n_levels < 1 || n_levels > 7 || init_len < 1 || max_new < 0 || max_block < 0) return 1;
    cascade cs;
    memset(&cs, 0, sizeof(cs));
    orc_stats local;
    cs.st = stats ? stats : &local;
    memset(cs.st, 0, sizeof(orc_stats));
    cs.st->first_near_tie = -1;
    cs.n_levels = n_levels; cs.models = models;
    cs.hay = hay; cs.L = L; cs.dynamic_hay = dynamic_hay; cs.bigram = bigram_next; cs.max_order = max_order;
    cs.K = K; cs.max_block = max_block;
    cs.lenience = lenience; cs.temperature = temperature; cs.seed = seed; cs.step = 0;
    cs.V = models[0]->c.vocab;
    cs.cap = models[0]->c.max_seq;
    for (int r = 1; r < n_levels; ++r)
        if (models[r]->c.max_seq < cs.cap) cs.cap = models[r]->c.max_seq;
    /* the product bounds how far drafting may run ahead of the committed prefix; the same bound is
       applied here so that both sides accept and refuse the same requests */
    int window = 0;
    for (int r = 0; r < n_levels; ++r) {
        for (int c = r; c < n_levels; ++c) window += K[(size_t)r * n_levels + c] > 0 ? K[(size_t)r * n_levels + c] : 0;
        window += max_block + 1;
    }
    if (window >= 128) return 2;
    if (init_len + max_new + window > cs.cap) return 2;
    cs.seq = (int32_t*)calloc((size_t)cs.cap + 64, sizeof(int32_t));
    cs.probs = (float**)calloc((size_t)cs.cap + 64, sizeof(float*));
    memcpy(cs.seq, init_seq, sizeof(int32_t) * (size_t)init_len);
    cs.len = init_len; cs.init_len = init_len; cs.margins = margins;
    int rc = 0;
    for (int r = 0; r < n_levels && !rc; ++r)
        if (models[r]->c.arch == 1) rc = orc_encoder_forward(models[r], hay, L);
    while (!rc && cs.len - init_len < max_new) rc = cascade_step(&cs, 0, 0);
    int made = cs.len - init_len;
    if (made > max_new) made = max_new;
    memcpy(out_tokens, cs.seq + init_len, sizeof(int32_t) * (size_t)made);
    *out_len = made;
    cs.st->tokens = made;
    for (int i = 0; i < cs.cap + 64; ++i) free(cs.probs[i]);
    free(cs.probs); free(cs.seq);
    return rc;
}
