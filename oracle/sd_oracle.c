/*
 * CPU oracle for heterogeneous speculative decoding (TaskSpec).
 *
 * TEST INFRASTRUCTURE ONLY.  Plain, slow, one step after the other.  It shares
 * no code with the CUDA library and must never be linked into, imported by or
 * called from the product path; only the tests, the smoke check and the
 * benchmark's CPU-baseline leg use it.
 *
 * Precision: every floating-point quantity is a double, except the
 * probabilities p and q handed to the accept rule, which are rounded to fp32
 * because the accept comparison and the integer CDF are defined on fp32 values
 * (both sides must take that decision in the same precision).  Weights are
 * stored either as fp32 or as bf16 bit patterns (uint16) and widened exactly.
 *
 * What follows what:
 *   - loop structure (draft gamma tokens one by one, target scores them in one
 *     parallel pass): Fig. 1 (a)/(b) and Sec. 1;
 *   - accept rule: Sec. 3.1 "Parameter Settings" cites the stochastic
 *     verification of Leviathan et al.; the rule itself (accept with
 *     probability min(1, p/q), else resample from norm(max(0, p - q)), one
 *     extra token from the target when everything is accepted) is that cited
 *     rule;
 *   - routing: Sec. 2.1 (explicit task type bypasses the classifier) and
 *     Sec. 3.3.3 (MLP variant: embedding, two fully connected layers, softmax);
 *   - counters: Eq. 2 (acceptance rate) and the definition of tau in Sec. 3.1.
 *
 * Pins (see the CPU tests): Philox known-answer vectors, sampler brute force,
 * Eq. 1 closed form by Monte Carlo, q == p accepts everything, chi-square of
 * emitted tokens against p, cached forward == full recompute, greedy
 * speculative output == greedy autoregressive output, tau = 1 + gamma * AR.
 * Parity unpinned: which tokens a random-init model emits and which draft a
 * random classifier picks (the paper gives no weights); those are compared
 * GPU-vs-oracle only.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

/* ------------------------------------------------------------------------ */
/* Philox4x32-10 (Salmon et al., "Parallel random numbers: as easy as 1,2,3") */
/* ------------------------------------------------------------------------ */

void orc_philox4x32_10(const uint32_t ctr[4], const uint32_t key[2], uint32_t out[4])
{
    uint32_t c0 = ctr[0], c1 = ctr[1], c2 = ctr[2], c3 = ctr[3];
    uint32_t k0 = key[0], k1 = key[1];
    for (int round = 0; round < 10; ++round) {
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

/* Purposes of a random draw inside one iteration. */
enum { ORC_DRAW_DRAFT = 0, ORC_DRAW_ACCEPT = 1, ORC_DRAW_RESAMPLE = 2 };

/* 24-bit uniform as an integer in [1, 2^24]; u = u_int * 2^-24 lies in (0, 1]
 * and is exact in fp32.  counter = (iter, slot, seq, purpose), key = seed. */
uint32_t orc_uniform24(uint64_t seed, uint32_t iter, uint32_t slot, uint32_t seq, uint32_t purpose)
{
    uint32_t ctr[4] = { iter, slot, seq, purpose };
    uint32_t key[2] = { (uint32_t)seed, (uint32_t)(seed >> 32) };
    uint32_t out[4];
    orc_philox4x32_10(ctr, key, out);
    return (out[0] >> 8) + 1u;
}

/* ------------------------------------------------------------------------ */
/* Distribution from logits                                                  */
/* ------------------------------------------------------------------------ */

int orc_argmax(const double* v, int n)
{
    int best = 0;
    for (int k = 1; k < n; ++k)
        if (v[k] > v[best]) best = k;       /* strict: lowest index wins ties */
    return best;
}

/* p = softmax(logits / T) rounded to fp32; T == 0 gives the one-hot argmax. */
void orc_softmax_T(const double* logits, int V, double T, float* p)
{
    if (T == 0.0) {
        int a = orc_argmax(logits, V);
        for (int k = 0; k < V; ++k) p[k] = 0.0f;
        p[a] = 1.0f;
        return;
    }
    double m = logits[0];
    for (int k = 1; k < V; ++k) if (logits[k] > m) m = logits[k];
    double sum = 0.0;
    for (int k = 0; k < V; ++k) sum += exp((logits[k] - m) / T);
    for (int k = 0; k < V; ++k) p[k] = (float)(exp((logits[k] - m) / T) / sum);
}

/* ------------------------------------------------------------------------ */
/* Integer inverse-CDF sampler                                               */
/* ------------------------------------------------------------------------ */

/* Weights w[k] >= 0 (fp32, at most 1) become integers floor(w * 2^32); the
 * token returned is the first k whose running integer sum reaches
 * thr = ceil(u_int * tot / 2^24).  Integer sums are exact, so any summation
 * order gives the same token.  Returns -1 when every weight quantises to 0. */
int orc_sample_icdf(const float* w, int V, uint32_t u_int)
{
    uint64_t tot = 0;
    for (int k = 0; k < V; ++k) tot += (uint64_t)(w[k] * 4294967296.0f);
    if (tot == 0) return -1;
    uint64_t thr = ((uint64_t)u_int * tot + ((1u << 24) - 1u)) >> 24;
    uint64_t run = 0;
    for (int k = 0; k < V; ++k) {
        run += (uint64_t)(w[k] * 4294967296.0f);
        if (run >= thr) return k;
    }
    return V - 1; /* unreachable: thr <= tot */
}

static int argmax_f32(const float* v, int n)
{
    int best = 0;
    for (int k = 1; k < n; ++k) if (v[k] > v[best]) best = k;
    return best;
}

/* ------------------------------------------------------------------------ */
/* Accept / reject of one iteration of one sequence                          */
/* ------------------------------------------------------------------------ */

/* p: [gamma+1][V] target probabilities, q: [gamma][V] draft probabilities,
 * x: [gamma] draft tokens.  Writes n (number of leading accepted drafts) and
 * out_tok[0..n] = x_0..x_{n-1}, y.  Slot s is accepted iff u_s * q_s(x_s) <=
 * p_s(x_s) with one correctly rounded fp32 multiply and u_s in (0, 1]. */
void orc_accept(const float* p, const float* q, const int32_t* x, int gamma, int V,
                uint64_t seed, uint32_t iter, uint32_t seq, int32_t* n_out, int32_t* out_tok)
{
    int n = 0;
    while (n < gamma) {
        uint32_t ui = orc_uniform24(seed, iter, (uint32_t)n, seq, ORC_DRAW_ACCEPT);
        float u = (float)ui * (1.0f / 16777216.0f);
        volatile float lhs = u * q[(size_t)n * V + x[n]];
        if (!(lhs <= p[(size_t)n * V + x[n]])) break;
        ++n;
    }
    for (int s = 0; s < n; ++s) out_tok[s] = x[s];
    uint32_t ui = orc_uniform24(seed, iter, (uint32_t)n, seq, ORC_DRAW_RESAMPLE);
    const float* pn = p + (size_t)n * V;
    int y;
    if (n < gamma) {
        const float* qn = q + (size_t)n * V;
        float* r = (float*)malloc(sizeof(float) * (size_t)V);
        for (int k = 0; k < V; ++k) {
            float diff = pn[k] - qn[k];
            r[k] = diff > 0.0f ? diff : 0.0f;
        }
        y = orc_sample_icdf(r, V, ui);
        free(r);
        if (y < 0) y = orc_sample_icdf(pn, V, ui);   /* residual vanished */
    } else {
        y = orc_sample_icdf(pn, V, ui);              /* bonus token */
    }
    if (y < 0) y = argmax_f32(pn, V);
    out_tok[n] = y;
    *n_out = n;
}

/* alpha of Eq. 1 is the probability that the target agrees with one draft token.  For the
 * stochastic rule that probability, given the two distributions of a slot, is
 * sum_k min(p_s(k), q_s(k)) (the draft is drawn from q_s and kept with probability
 * min(1, p_s/q_s)).  terms[s] receives that sum, in double, for every slot s < gamma;
 * the estimate of alpha over a run is their mean over the slots that were judged
 * (slot s is judged iff all slots before it were accepted: s <= min(n, gamma - 1)). */
void orc_alpha_terms(const float* p, const float* q, int gamma, int V, double* terms)
{
    for (int s = 0; s < gamma; ++s) {
        double a = 0.0;
        for (int k = 0; k < V; ++k) {
            double pk = (double)p[(size_t)s * V + k], qk = (double)q[(size_t)s * V + k];
            a += pk < qk ? pk : qk;
        }
        terms[s] = a;
    }
}

/* ------------------------------------------------------------------------ */
/* Decoder-only transformer (RMSNorm, rotary embedding, SwiGLU, no biases)   */
/* ------------------------------------------------------------------------ */

typedef struct {
    int32_t n_layers, d_model, n_heads, n_kv_heads, head_dim, d_ffn, vocab;
    int32_t wdtype;                 /* 0: fp32 weights, 1: bf16 bit patterns */
    double rms_eps, rope_base;
    const void* embed;              /* [vocab][d_model] */
    const void* lm_head;            /* [vocab][d_model] */
    const float* final_norm;        /* [d_model] */
    const void* const* wq;          /* per layer [n_heads*head_dim][d_model] */
    const void* const* wk;          /* per layer [n_kv_heads*head_dim][d_model] */
    const void* const* wv;
    const void* const* wo;          /* per layer [d_model][n_heads*head_dim] */
    const void* const* wg;          /* per layer [d_ffn][d_model] */
    const void* const* wu;
    const void* const* wd;          /* per layer [d_model][d_ffn] */
    const float* const* norm1;      /* per layer [d_model] */
    const float* const* norm2;
} orc_model;

typedef struct {
    double* k;                      /* [n_layers][max_ctx][n_kv_heads*head_dim] */
    double* v;
    int32_t max_ctx;
} orc_cache;

static inline double wval(const void* W, int wdtype, size_t idx)
{
    if (wdtype == 0) return (double)((const float*)W)[idx];
    uint32_t bits = (uint32_t)((const uint16_t*)W)[idx] << 16;
    float f;
    memcpy(&f, &bits, 4);
    return (double)f;
}

/* Y[r][o] = sum_k X[r][k] * W[o][k] */
static void linear(const void* W, int wdtype, int n_out, int n_in,
                   const double* X, int rows, double* Y)
{
#pragma omp parallel for schedule(static)
    for (int o = 0; o < n_out; ++o) {
        for (int r = 0; r < rows; ++r) {
            double acc = 0.0;
            for (int k = 0; k < n_in; ++k)
                acc += X[(size_t)r * n_in + k] * wval(W, wdtype, (size_t)o * n_in + k);
            Y[(size_t)r * n_out + o] = acc;
        }
    }
}

static void rmsnorm(const double* x, const float* gain, int d, double eps, double* y)
{
    double ss = 0.0;
    for (int i = 0; i < d; ++i) ss += x[i] * x[i];
    double inv = 1.0 / sqrt(ss / d + eps);
    for (int i = 0; i < d; ++i) y[i] = x[i] * inv * (double)gain[i];
}

/* Rotary embedding with the half-split pairing (i, i + head_dim/2). */
static void rope(double* vec, int n_heads, int head_dim, int pos, double base)
{
    int half = head_dim / 2;
    for (int h = 0; h < n_heads; ++h) {
        double* v = vec + (size_t)h * head_dim;
        for (int i = 0; i < half; ++i) {
            double ang = (double)pos * pow(base, -2.0 * i / head_dim);
            double c = cos(ang), s = sin(ang);
            double a = v[i], b = v[i + half];
            v[i] = a * c - b * s;
            v[i + half] = a * s + b * c;
        }
    }
}

static double silu(double z) { return z / (1.0 + exp(-z)); }

/* Forward over `rows` new tokens of one sequence at positions pos0.. against
 * the cache; appends their keys/values.  logits: [rows][vocab] or NULL. */
int orc_forward_cached(const orc_model* m, orc_cache* c, const int32_t* tokens, int rows,
                       int pos0, double* logits)
{
    const int d = m->d_model, H = m->n_heads, Hkv = m->n_kv_heads, hd = m->head_dim;
    const int F = m->d_ffn, dq = H * hd, dkv = Hkv * hd, group = H / Hkv;
    if (pos0 < 0 || pos0 + rows > c->max_ctx) return 1;
    double* h = malloc(sizeof(double) * (size_t)rows * d);
    double* a = malloc(sizeof(double) * (size_t)rows * d);
    double* q = malloc(sizeof(double) * (size_t)rows * dq);
    double* k = malloc(sizeof(double) * (size_t)rows * dkv);
    double* v = malloc(sizeof(double) * (size_t)rows * dkv);
    double* o = malloc(sizeof(double) * (size_t)rows * dq);
    double* t = malloc(sizeof(double) * (size_t)rows * d);
    double* g = malloc(sizeof(double) * (size_t)rows * F);
    double* u = malloc(sizeof(double) * (size_t)rows * F);
    double* sc = malloc(sizeof(double) * (size_t)(pos0 + rows));

    for (int r = 0; r < rows; ++r)
        for (int i = 0; i < d; ++i)
            h[(size_t)r * d + i] = wval(m->embed, m->wdtype, (size_t)tokens[r] * d + i);

    for (int l = 0; l < m->n_layers; ++l) {
        double* Kc = c->k + (size_t)l * c->max_ctx * dkv;
        double* Vc = c->v + (size_t)l * c->max_ctx * dkv;
        for (int r = 0; r < rows; ++r)
            rmsnorm(h + (size_t)r * d, m->norm1[l], d, m->rms_eps, a + (size_t)r * d);
        linear(m->wq[l], m->wdtype, dq, d, a, rows, q);
        linear(m->wk[l], m->wdtype, dkv, d, a, rows, k);
        linear(m->wv[l], m->wdtype, dkv, d, a, rows, v);
        for (int r = 0; r < rows; ++r) {
            rope(q + (size_t)r * dq, H, hd, pos0 + r, m->rope_base);
            rope(k + (size_t)r * dkv, Hkv, hd, pos0 + r, m->rope_base);
            memcpy(Kc + (size_t)(pos0 + r) * dkv, k + (size_t)r * dkv, sizeof(double) * dkv);
            memcpy(Vc + (size_t)(pos0 + r) * dkv, v + (size_t)r * dkv, sizeof(double) * dkv);
        }
        for (int r = 0; r < rows; ++r) {
            int n_ctx = pos0 + r + 1;           /* attends to itself and all before */
            for (int hh = 0; hh < H; ++hh) {
                const double* qv = q + (size_t)r * dq + (size_t)hh * hd;
                int kvh = hh / group;
                double mx = -INFINITY;
                for (int p = 0; p < n_ctx; ++p) {
                    const double* kv = Kc + (size_t)p * dkv + (size_t)kvh * hd;
                    double s = 0.0;
                    for (int i = 0; i < hd; ++i) s += qv[i] * kv[i];
                    sc[p] = s / sqrt((double)hd);
                    if (sc[p] > mx) mx = sc[p];
                }
                double den = 0.0;
                for (int p = 0; p < n_ctx; ++p) { sc[p] = exp(sc[p] - mx); den += sc[p]; }
                double* ov = o + (size_t)r * dq + (size_t)hh * hd;
                for (int i = 0; i < hd; ++i) ov[i] = 0.0;
                for (int p = 0; p < n_ctx; ++p) {
                    const double* vv = Vc + (size_t)p * dkv + (size_t)kvh * hd;
                    double w = sc[p] / den;
                    for (int i = 0; i < hd; ++i) ov[i] += w * vv[i];
                }
            }
        }
        linear(m->wo[l], m->wdtype, d, dq, o, rows, t);
        for (size_t i = 0; i < (size_t)rows * d; ++i) h[i] += t[i];
        for (int r = 0; r < rows; ++r)
            rmsnorm(h + (size_t)r * d, m->norm2[l], d, m->rms_eps, a + (size_t)r * d);
        linear(m->wg[l], m->wdtype, F, d, a, rows, g);
        linear(m->wu[l], m->wdtype, F, d, a, rows, u);
        for (size_t i = 0; i < (size_t)rows * F; ++i) g[i] = silu(g[i]) * u[i];
        linear(m->wd[l], m->wdtype, d, F, g, rows, t);
        for (size_t i = 0; i < (size_t)rows * d; ++i) h[i] += t[i];
    }
    if (logits) {
        for (int r = 0; r < rows; ++r)
            rmsnorm(h + (size_t)r * d, m->final_norm, d, m->rms_eps, a + (size_t)r * d);
        linear(m->lm_head, m->wdtype, m->vocab, d, a, rows, logits);
    }
    free(h); free(a); free(q); free(k); free(v); free(o); free(t); free(g); free(u); free(sc);
    return 0;
}

/* The same network with no cache at all: every layer is evaluated for the
 * whole sequence at once and attention is a masked n x n score matrix.
 * logits: [n][vocab].  Used to pin the cached routine. */
int orc_forward_full(const orc_model* m, const int32_t* tokens, int n, double* logits)
{
    const int d = m->d_model, H = m->n_heads, Hkv = m->n_kv_heads, hd = m->head_dim;
    const int F = m->d_ffn, dq = H * hd, dkv = Hkv * hd, group = H / Hkv;
    double* h = malloc(sizeof(double) * (size_t)n * d);
    double* a = malloc(sizeof(double) * (size_t)n * d);
    double* Q = malloc(sizeof(double) * (size_t)n * dq);
    double* K = malloc(sizeof(double) * (size_t)n * dkv);
    double* Vv = malloc(sizeof(double) * (size_t)n * dkv);
    double* O = malloc(sizeof(double) * (size_t)n * dq);
    double* t = malloc(sizeof(double) * (size_t)n * d);
    double* g = malloc(sizeof(double) * (size_t)n * F);
    double* u = malloc(sizeof(double) * (size_t)n * F);
    double* S = malloc(sizeof(double) * (size_t)n * n);
    for (int r = 0; r < n; ++r)
        for (int i = 0; i < d; ++i)
            h[(size_t)r * d + i] = wval(m->embed, m->wdtype, (size_t)tokens[r] * d + i);
    for (int l = 0; l < m->n_layers; ++l) {
        for (int r = 0; r < n; ++r)
            rmsnorm(h + (size_t)r * d, m->norm1[l], d, m->rms_eps, a + (size_t)r * d);
        linear(m->wq[l], m->wdtype, dq, d, a, n, Q);
        linear(m->wk[l], m->wdtype, dkv, d, a, n, K);
        linear(m->wv[l], m->wdtype, dkv, d, a, n, Vv);
        for (int r = 0; r < n; ++r) {
            rope(Q + (size_t)r * dq, H, hd, r, m->rope_base);
            rope(K + (size_t)r * dkv, Hkv, hd, r, m->rope_base);
        }
        for (int hh = 0; hh < H; ++hh) {
            int kvh = hh / group;
            /* S = mask(Q K^T / sqrt(hd)), row-wise softmax, O = S V */
            for (int i = 0; i < n; ++i)
                for (int j = 0; j < n; ++j) {
                    if (j > i) { S[(size_t)i * n + j] = -INFINITY; continue; }
                    double s = 0.0;
                    for (int e = 0; e < hd; ++e)
                        s += Q[(size_t)i * dq + (size_t)hh * hd + e] * K[(size_t)j * dkv + (size_t)kvh * hd + e];
                    S[(size_t)i * n + j] = s / sqrt((double)hd);
                }
            for (int i = 0; i < n; ++i) {
                double mx = -INFINITY, den = 0.0;
                for (int j = 0; j < n; ++j) if (S[(size_t)i * n + j] > mx) mx = S[(size_t)i * n + j];
                for (int j = 0; j < n; ++j) { S[(size_t)i * n + j] = exp(S[(size_t)i * n + j] - mx); den += S[(size_t)i * n + j]; }
                for (int j = 0; j < n; ++j) S[(size_t)i * n + j] /= den;
                for (int e = 0; e < hd; ++e) {
                    double acc = 0.0;
                    for (int j = 0; j < n; ++j) acc += S[(size_t)i * n + j] * Vv[(size_t)j * dkv + (size_t)kvh * hd + e];
                    O[(size_t)i * dq + (size_t)hh * hd + e] = acc;
                }
            }
        }
        linear(m->wo[l], m->wdtype, d, dq, O, n, t);
        for (size_t i = 0; i < (size_t)n * d; ++i) h[i] += t[i];
        for (int r = 0; r < n; ++r)
            rmsnorm(h + (size_t)r * d, m->norm2[l], d, m->rms_eps, a + (size_t)r * d);
        linear(m->wg[l], m->wdtype, F, d, a, n, g);
        linear(m->wu[l], m->wdtype, F, d, a, n, u);
        for (size_t i = 0; i < (size_t)n * F; ++i) g[i] = silu(g[i]) * u[i];
        linear(m->wd[l], m->wdtype, d, F, g, n, t);
        for (size_t i = 0; i < (size_t)n * d; ++i) h[i] += t[i];
    }
    for (int r = 0; r < n; ++r)
        rmsnorm(h + (size_t)r * d, m->final_norm, d, m->rms_eps, a + (size_t)r * d);
    linear(m->lm_head, m->wdtype, m->vocab, d, a, n, logits);
    free(h); free(a); free(Q); free(K); free(Vv); free(O); free(t); free(g); free(u); free(S);
    return 0;
}

/* softmax(q K^T / sqrt(hd)) V for one query vector over n_ctx cached positions of one head;
 * K, V: [n_ctx][hd] with row stride `stride` doubles.  The definition, written out. */
void orc_attention_head(const double* q, const double* K, const double* V, int n_ctx, int hd, int stride, double* out)
{
    double* s = malloc(sizeof(double) * (size_t)n_ctx);
    double mx = -INFINITY, den = 0.0;
    for (int p = 0; p < n_ctx; ++p) {
        double acc = 0.0;
        for (int i = 0; i < hd; ++i) acc += q[i] * K[(size_t)p * stride + i];
        s[p] = acc / sqrt((double)hd);
        if (s[p] > mx) mx = s[p];
    }
    for (int p = 0; p < n_ctx; ++p) { s[p] = exp(s[p] - mx); den += s[p]; }
    for (int i = 0; i < hd; ++i) {
        double acc = 0.0;
        for (int p = 0; p < n_ctx; ++p) acc += s[p] / den * V[(size_t)p * stride + i];
        out[i] = acc;
    }
    free(s);
}

/* Single primitives exported so that tests can pin them one by one. */
void orc_rmsnorm(const double* x, const float* gain, int d, double eps, double* y) { rmsnorm(x, gain, d, eps, y); }
void orc_rope(double* vec, int n_heads, int head_dim, int pos, double base) { rope(vec, n_heads, head_dim, pos, base); }
double orc_silu(double z) { return silu(z); }
void orc_linear(const void* W, int wdtype, int n_out, int n_in, const double* X, int rows, double* Y)
{ linear(W, wdtype, n_out, n_in, X, rows, Y); }

/* ------------------------------------------------------------------------ */
/* Prompt classifier, MLP variant (Sec. 3.3.3): mean-pooled embedding ->      */
/* FC + ReLU -> FC -> softmax -> argmax.  Returns the class; scores optional. */
/* ------------------------------------------------------------------------ */
int orc_route_prompt(const void* embed, int wdtype, int d_in, const int32_t* tokens, int n_tok,
                     const float* w1, const float* b1, int d_hidden,
                     const float* w2, const float* b2, int n_classes,
                     int forced_task, double* probs_out)
{
    if (forced_task >= 0) return forced_task;   /* Sec. 2.1: given task type bypasses the classifier */
    double* e = calloc((size_t)d_in, sizeof(double));
    double* z = malloc(sizeof(double) * (size_t)d_hidden);
    double* o = malloc(sizeof(double) * (size_t)n_classes);
    for (int t = 0; t < n_tok; ++t)
        for (int i = 0; i < d_in; ++i) e[i] += wval(embed, wdtype, (size_t)tokens[t] * d_in + i);
    for (int i = 0; i < d_in; ++i) e[i] /= n_tok;
    for (int j = 0; j < d_hidden; ++j) {
        double acc = b1[j];
        for (int i = 0; i < d_in; ++i) acc += (double)w1[(size_t)j * d_in + i] * e[i];
        z[j] = acc > 0.0 ? acc : 0.0;
    }
    for (int c = 0; c < n_classes; ++c) {
        double acc = b2[c];
        for (int j = 0; j < d_hidden; ++j) acc += (double)w2[(size_t)c * d_hidden + j] * z[j];
        o[c] = acc;
    }
    int best = orc_argmax(o, n_classes);
    if (probs_out) {
        double mx = o[best], den = 0.0;
        for (int c = 0; c < n_classes; ++c) den += exp(o[c] - mx);
        for (int c = 0; c < n_classes; ++c) probs_out[c] = exp(o[c] - mx) / den;
    }
    free(e); free(z); free(o);
    return best;
}

/* ------------------------------------------------------------------------ */
/* The speculative decoding loop of one sequence                             */
/* ------------------------------------------------------------------------ */

typedef struct {
    int64_t iterations, drafted, accepted, emitted;   /* Eq. 2: AR = accepted / drafted; tau = emitted / iterations */
} orc_counters;

typedef struct {
    int32_t cap_iters;      /* capacity of the arrays below, in iterations */
    int32_t n_iters;        /* filled in */
    int32_t* len_before;    /* [cap] sequence length when the iteration started */
    int32_t* n_acc;         /* [cap] */
    int32_t* x;             /* [cap][gamma] draft tokens */
    int32_t* out_tok;       /* [cap][gamma+1] emitted tokens (first n_acc+1 valid) */
    float* q;               /* [cap][gamma][V] draft probabilities, or NULL */
    float* p;               /* [cap][gamma+1][V] target probabilities, or NULL */
    double* logits;         /* [cap][gamma+1][V] target logits, or NULL */
} orc_trace;

/* tokens: buffer of capacity >= n_prompt + max_new + gamma + 1 holding the
 * prompt; on return holds prompt + generated tokens, *len_out their count.
 * Caches must be empty (this routine prefills them).  draft may equal NULL
 * only when gamma == 0 (plain autoregressive decoding of the target). */
int orc_spec_decode(const orc_model* target, const orc_model* draft,
                    orc_cache* tcache, orc_cache* dcache,
                    int32_t* tokens, int n_prompt, int max_new, int gamma, double T,
                    uint64_t seed, uint32_t seq_id,
                    int32_t* len_out, orc_counters* cnt, orc_trace* tr,
                    double* alpha_sum_out, int64_t* judged_out)
{
    const int V = target->vocab;
    int L = n_prompt, tkv = 0, dkv = 0;
    uint32_t iter = 0;
    const int L_end = n_prompt + max_new;
    memset(cnt, 0, sizeof(*cnt));
    if (tr) tr->n_iters = 0;
    if (n_prompt < 1) return 1;

    double* tl = malloc(sizeof(double) * (size_t)(gamma + 1) * V);
    double* dl = malloc(sizeof(double) * (size_t)2 * V);
    float* p = malloc(sizeof(float) * (size_t)(gamma + 1) * V);
    float* q = malloc(sizeof(float) * (size_t)(gamma > 0 ? gamma : 1) * V);
    int32_t* x = malloc(sizeof(int32_t) * (size_t)(gamma + 1));
    int32_t* out = malloc(sizeof(int32_t) * (size_t)(gamma + 1));
    int32_t* rows = malloc(sizeof(int32_t) * (size_t)(gamma + 1));
    double* terms = malloc(sizeof(double) * (size_t)(gamma > 0 ? gamma : 1));
    double alpha_sum = 0.0;
    int64_t judged = 0;
    int rc = 0;

    /* prefill: everything but the last prompt token */
    if (L - 1 > 0) {
        rc |= orc_forward_cached(target, tcache, tokens, L - 1, 0, NULL);
        if (gamma > 0) rc |= orc_forward_cached(draft, dcache, tokens, L - 1, 0, NULL);
    }
    tkv = L - 1; dkv = L - 1;

    while (L < L_end && rc == 0) {
        /* (1) the draft proposes gamma tokens one after the other (Fig. 1a) */
        for (int s = 0; s < gamma; ++s) {
            int nrow;
            if (s == 0) {               /* pending tokens: 1, or 2 after a fully accepted iteration */
                nrow = L - dkv;
                rc |= orc_forward_cached(draft, dcache, tokens + dkv, nrow, dkv, dl);
                dkv = L;
            } else {
                nrow = 1;
                rc |= orc_forward_cached(draft, dcache, &x[s - 1], 1, dkv, dl);
                dkv += 1;
            }
            if (rc) break;
            orc_softmax_T(dl + (size_t)(nrow - 1) * V, V, T, q + (size_t)s * V);
            if (T == 0.0) {
                x[s] = argmax_f32(q + (size_t)s * V, V);
            } else {
                uint32_t ui = orc_uniform24(seed, iter, (uint32_t)s, seq_id, ORC_DRAW_DRAFT);
                x[s] = orc_sample_icdf(q + (size_t)s * V, V, ui);
                if (x[s] < 0) x[s] = argmax_f32(q + (size_t)s * V, V);
            }
        }
        if (rc) break;
        /* (2) the target scores last token + gamma drafts in one pass (Fig. 1b) */
        rows[0] = tokens[L - 1];
        for (int s = 0; s < gamma; ++s) rows[s + 1] = x[s];
        rc |= orc_forward_cached(target, tcache, rows, gamma + 1, tkv, tl);
        if (rc) break;
        for (int j = 0; j <= gamma; ++j) orc_softmax_T(tl + (size_t)j * V, V, T, p + (size_t)j * V);
        /* (3) accept / reject */
        int32_t n;
        orc_accept(p, q, x, gamma, V, seed, iter, seq_id, &n, out);
        orc_alpha_terms(p, q, gamma, V, terms);
        for (int s = 0; s < gamma && s <= n; ++s) { alpha_sum += terms[s]; judged += 1; }     /* the judged slots */
        if (tr && tr->n_iters < tr->cap_iters) {
            int it = tr->n_iters++;
            tr->len_before[it] = L;
            tr->n_acc[it] = n;
            for (int s = 0; s < gamma; ++s) tr->x[(size_t)it * gamma + s] = x[s];
            for (int s = 0; s <= gamma; ++s) tr->out_tok[(size_t)it * (gamma + 1) + s] = s <= n ? out[s] : -1;
            if (tr->q) memcpy(tr->q + (size_t)it * gamma * V, q, sizeof(float) * (size_t)gamma * V);
            if (tr->p) memcpy(tr->p + (size_t)it * (gamma + 1) * V, p, sizeof(float) * (size_t)(gamma + 1) * V);
            if (tr->logits) memcpy(tr->logits + (size_t)it * (gamma + 1) * V, tl, sizeof(double) * (size_t)(gamma + 1) * V);
        }
        /* (4) commit n+1 tokens; rejected positions of both caches are simply
         * forgotten: the next append overwrites them */
        for (int s = 0; s <= n; ++s) tokens[L + s] = out[s];
        tkv = L + n;
        if (gamma > 0) dkv = (L + n < L + gamma - 1) ? L + n : L + gamma - 1;
        L = L + n + 1;
        iter += 1;
        cnt->iterations += 1;
        cnt->drafted += gamma;
        cnt->accepted += n;
        cnt->emitted += n + 1;
    }
    if (L > L_end) L = L_end;       /* the last iteration may overshoot; truncate */
    *len_out = L;
    if (alpha_sum_out) *alpha_sum_out = alpha_sum;
    if (judged_out) *judged_out = judged;
    free(tl); free(dl); free(p); free(q); free(x); free(out); free(rows); free(terms);
    return rc;
}

/* ------------------------------------------------------------------------ */
/* Monte-Carlo driver for fixed distributions (used to pin Eq. 1 and the     */
/* output law): every slot of every iteration uses the same p and q.         */
/* hist_first[V] counts the first emitted token; returns total emitted.      */
/* ------------------------------------------------------------------------ */
int64_t orc_mc_fixed(const float* p1, const float* q1, int V, int gamma, int64_t iters,
                     uint64_t seed, int64_t* hist_first, int64_t* accepted_out)
{
    float* p = malloc(sizeof(float) * (size_t)(gamma + 1) * V);
    float* q = malloc(sizeof(float) * (size_t)gamma * V);
    int32_t* x = malloc(sizeof(int32_t) * (size_t)gamma);
    int32_t* out = malloc(sizeof(int32_t) * (size_t)(gamma + 1));
    for (int j = 0; j <= gamma; ++j) memcpy(p + (size_t)j * V, p1, sizeof(float) * V);
    for (int j = 0; j < gamma; ++j) memcpy(q + (size_t)j * V, q1, sizeof(float) * V);
    int64_t emitted = 0, accepted = 0;
    for (int64_t it = 0; it < iters; ++it) {
        uint32_t iter = (uint32_t)it, seq = (uint32_t)(it >> 32);
        for (int s = 0; s < gamma; ++s) {
            uint32_t ui = orc_uniform24(seed, iter, (uint32_t)s, seq, ORC_DRAW_DRAFT);
            x[s] = orc_sample_icdf(q1, V, ui);
        }
        int32_t n;
        orc_accept(p, q, x, gamma, V, seed, iter, seq, &n, out);
        emitted += n + 1;
        accepted += n;
        if (hist_first) hist_first[out[0]] += 1;
    }
    if (accepted_out) *accepted_out = accepted;
    free(p); free(q); free(x); free(out);
    return emitted;
}
