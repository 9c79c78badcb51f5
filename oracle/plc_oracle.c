/*
 * plc_oracle.c -- CPU oracle for predictive delta coding of the KV cache.
 *
 * TEST INFRASTRUCTURE ONLY.  This file is a plain, slow, single-threaded restatement of what the
 * method computes, in IEEE double unless a line says otherwise.  It shares no code, table or
 * constant with the CUDA library; only the tests, the smoke check and the benchmark's CPU-baseline
 * leg may call it.  Nothing here is tuned for speed.
 *
 * Pinned parts (see tests/test_oracle_*.py): top-K softmax, mixture, mixture variance, scale class,
 * quantise / reconstruct, frequency tables, rANS chunk coder, LCP / trie metric, dedup parents,
 * prefix clusters, adaptive step, zero-rate rule, linear-embedding predictor, rotated fixed-rate
 * quantiser.
 * Parity unpinned: the end-to-end bit rate against the paper's 3.3-4.3 bits per token position
 * (Cor. 1) -- the paper states no achieved rate for any coder; the rate is only reported.
 *
 * What follows the paper, and where:
 *   softmax over the next-token logits ................ Sec. 5.1, first display (next-token distribution)
 *   top-k renormalised prediction ..................... Sec. 7.1, "Top-k approximation" display
 *   full-vocabulary prediction ........................ Def. 5 (predicted KV vector)
 *   residual .......................................... Def. 6 (KV residual)
 *   E||R||^2 = Var[F] (scale of the coder model) ...... Thm. 2 and its proof
 *   top-k mass Z_k .................................... Thm. 4(a) and its proof
 *   reconstruction KV = R + KV^ ....................... Prop. 3, "Correctness"
 *   longest common prefix, d_T = -log2 P(s ^ s') ...... Def. 2 (trie metric)
 *   prefix costs zero bits, tail is delta coded ....... Prop. 2, proof, "Description of KV(s)"
 *   best-match lookup = deepest stored ancestor ....... Sec. 7.3 (trie-based prefix index)
 *   per-vector quantiser on the residual .............. Prop. 3, step 3 (rotated fixed-rate quantiser)
 * The paper names no entropy coder beyond "standard source coding" (Prop. 2, proof); the coder
 * below (uniform step, discretised-Laplace model, 32-lane interleaved rANS) is the
 * stated reading of this codec and is defined in full in the comments of each function.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

#define PLO_OK 0
#define PLO_E_INVALID 1
#define PLO_E_CAPACITY 4
#define PLO_E_CORRUPT 5

#define PROB_BITS 15
#define PROB_M (1u << PROB_BITS)
#define RANS_L (1u << 16)
#define NSYM 64      /* zigzag(hi) for hi in [-31,31] -> 0..62, 63 = escape */
#define ESC 63
#define HI_MAX 31
#define Q_MIN (-24)
#define Q_MAX 135
#define SYM_LIMIT (1 << 30)
#define NLANES 32

/* ---------------------------------------------------------------- number formats */

/* IEEE binary16 bit pattern -> double (exact). */
static double half_to_double(uint16_t h) {
    int sign = (h >> 15) & 1, e = (h >> 10) & 31, m = h & 1023;
    double v;
    if (e == 0) v = ldexp((double)m, -24);
    else if (e == 31) v = m ? NAN : INFINITY;
    else v = ldexp((double)(1024 + m), e - 25);
    return sign ? -v : v;
}

/* Round a double to the nearest bfloat16 (8 significant bits, ties to even), returned as double.
 * Values below the bfloat16 normal range are not produced by any caller that matters (they are
 * probabilities < 1e-38) and are rounded on the same 8-bit grid. */
static double round_bf16(double x) {
    if (x == 0.0 || !isfinite(x)) return x;
    int e;
    double m = frexp(x, &e);          /* |m| in [0.5,1) */
    double r = nearbyint(ldexp(m, 8)); /* default rounding mode: ties to even */
    return ldexp(r, e - 8);
}

double plo_half_to_double(uint16_t h) { return half_to_double(h); }
double plo_round_bf16(double x) { return round_bf16(x); }

/* ---------------------------------------------------------------- top-K softmax */

typedef struct { double v; int32_t i; } kv_pair;

static int cmp_desc(const void* a, const void* b) {
    const kv_pair* x = (const kv_pair*)a; const kv_pair* y = (const kv_pair*)b;
    if (x->v > y->v) return -1;
    if (x->v < y->v) return 1;
    return (x->i > y->i) - (x->i < y->i);   /* equal logits: smaller index first */
}

/* One position.  Sec. 5.1: P(t | t_<i) = softmax(logits)_t.  Sec. 7.1: the top-k prediction uses
 * the k most probable tokens with their probabilities renormalised over that set.
 * Order: logit descending, index ascending among equal logits (the paper is silent on ties).
 *   w_k   = exp(l_k - l_max) / sum_{j<K} exp(l_j - l_max)
 *   lse   = l_max + ln sum_v exp(l_v - l_max)
 *   Z_k   = sum_{j<K} exp(l_j - lse)                 (Thm. 4(a): acceptance rate of the top-k draft)
 *   logp2 = (l[token] - lse) / ln 2                  (log2 P(x_i | x_<i), the trie edge weight)
 */
int plo_topk_softmax_row(const uint16_t* logits, int V, int K, int token,
                         int32_t* idx, double* w, double* lse, double* zk, double* logp2) {
    if (V < 1 || K < 1 || K > V) return PLO_E_INVALID;
    kv_pair* p = (kv_pair*)malloc(sizeof(kv_pair) * (size_t)V);
    if (!p) return PLO_E_INVALID;
    for (int v = 0; v < V; ++v) { p[v].v = half_to_double(logits[v]); p[v].i = v; }
    double tok_logit = (token >= 0 && token < V) ? p[token].v : NAN;
    qsort(p, (size_t)V, sizeof(kv_pair), cmp_desc);
    double lmax = p[0].v, sum_all = 0.0, sum_k = 0.0;
    for (int v = 0; v < V; ++v) sum_all += exp(p[v].v - lmax);
    for (int k = 0; k < K; ++k) sum_k += exp(p[k].v - lmax);
    double l = lmax + log(sum_all);
    double z = 0.0;
    for (int k = 0; k < K; ++k) {
        idx[k] = p[k].i;
        w[k] = exp(p[k].v - lmax) / sum_k;
        z += exp(p[k].v - l);
    }
    *lse = l; *zk = z; *logp2 = (tok_logit - l) / log(2.0);
    free(p);
    return PLO_OK;
}

int plo_topk_softmax(const uint16_t* logits, const int32_t* tokens, int64_t N, int V, int K,
                     int32_t* idx, double* w, double* lse, double* zk, double* logp2) {
    for (int64_t n = 0; n < N; ++n) {
        int rc = plo_topk_softmax_row(logits + n * V, V, K, tokens ? tokens[n] : -1,
                                      idx + n * K, w + n * K, lse + n, zk + n, logp2 + n);
        if (rc) return rc;
    }
    return PLO_OK;
}

/* ---------------------------------------------------------------- prediction */

/* Top-K mixture for one (table, position).  Sec. 7.1 with F_M(t_<i, t) := T[t]:
 *   mu      = sum_k w_k T[idx_k]
 *   sigma2  = (1/d) sum_k w_k || T[idx_k] - mu ||^2     (Thm. 2: E||R||^2 = Var_t[F], per component)
 */
void plo_mixture(const uint16_t* table /*[V][d]*/, int d, const int32_t* idx, const double* w, int K,
                 double* mu, double* sigma2) {
    for (int j = 0; j < d; ++j) mu[j] = 0.0;
    for (int k = 0; k < K; ++k) {
        const uint16_t* row = table + (size_t)idx[k] * d;
        for (int j = 0; j < d; ++j) mu[j] += w[k] * half_to_double(row[j]);
    }
    double s = 0.0;
    for (int k = 0; k < K; ++k) {
        const uint16_t* row = table + (size_t)idx[k] * d;
        double n2 = 0.0;
        for (int j = 0; j < d; ++j) { double t = half_to_double(row[j]) - mu[j]; n2 += t * t; }
        s += w[k] * n2;
    }
    *sigma2 = s / d;
}

/* Full-vocabulary prediction for one (table, position), Def. 5, in the arithmetic of a bf16
 * contraction: p_v = exp(l_v - lse) and T[v] are each rounded to bfloat16 first, the sum over the
 * whole vocabulary is exact (double), nothing is renormalised.
 *   mu     = sum_v bf16(p_v) bf16(T[v])
 *   sigma2 = max(0, sum_v bf16(p_v) bf16(||T[v]||^2 / d) - ||mu||^2 / d)
 * where ||T[v]||^2 is taken over the bf16-rounded row.
 */
void plo_dense_mixture(const uint16_t* table /*[V][d]*/, int V, int d, const uint16_t* logits, double lse,
                       double* mu, double* sigma2) {
    for (int j = 0; j < d; ++j) mu[j] = 0.0;
    double s = 0.0;
    for (int v = 0; v < V; ++v) {
        double p = round_bf16(exp(half_to_double(logits[v]) - lse));
        const uint16_t* row = table + (size_t)v * d;
        double n2 = 0.0;
        for (int j = 0; j < d; ++j) {
            double t = round_bf16(half_to_double(row[j]));
            mu[j] += p * t;
            n2 += t * t;
        }
        s += p * round_bf16(n2 / d);
    }
    double m2 = 0.0;
    for (int j = 0; j < d; ++j) m2 += mu[j] * mu[j];
    double r = s - m2 / d;
    *sigma2 = r > 0.0 ? r : 0.0;
}

/* Linear embedding approximation (Sec. 7.1): F(t_<i, t) ~ c + A E(t), hence
 *   KV^ ~ c + A Ebar,  Ebar = E_{t ~ P}[E(t)] = sum_v p_v E(v),
 * "a single weighted sum over the vocabulary using the softmax output".  In the arithmetic of two
 * chained bf16 contractions: p_v, E and A are rounded to bfloat16, Ebar is summed exactly and then
 * rounded to bfloat16 itself (it is the input of the second contraction), mu = c + A Ebar exactly. */
void plo_expected_embedding(const uint16_t* E /*[V][dm]*/, int V, int dm, const uint16_t* logits, double lse, double* ebar) {
    for (int k = 0; k < dm; ++k) ebar[k] = 0.0;
    for (int v = 0; v < V; ++v) {
        double p = round_bf16(exp(half_to_double(logits[v]) - lse));
        const uint16_t* row = E + (size_t)v * dm;
        for (int k = 0; k < dm; ++k) ebar[k] += p * round_bf16(half_to_double(row[k]));
    }
    for (int k = 0; k < dm; ++k) ebar[k] = round_bf16(ebar[k]);
}

/* out[j] = c[j] + sum_k bf16(A[j][k]) x[k]   (x already on the bf16 grid) */
void plo_linear_apply(const uint16_t* A /*[d][dm]*/, const uint16_t* c /*[d]*/, int d, int dm, const double* x, double* out) {
    for (int j = 0; j < d; ++j) {
        double s = half_to_double(c[j]);
        for (int k = 0; k < dm; ++k) s += round_bf16(half_to_double(A[(size_t)j * dm + k])) * x[k];
        out[j] = s;
    }
}

/* n2b[v] = bf16(||c + A E(v)||^2 / d): squared norm of the linear model's own candidate vector. */
void plo_linear_rownorms(const uint16_t* E, const uint16_t* A, const uint16_t* c, int V, int d, int dm, double* n2b) {
    double* x = (double*)malloc(sizeof(double) * (size_t)dm);
    double* t = (double*)malloc(sizeof(double) * (size_t)d);
    for (int v = 0; v < V; ++v) {
        for (int k = 0; k < dm; ++k) x[k] = round_bf16(half_to_double(E[(size_t)v * dm + k]));
        plo_linear_apply(A, c, d, dm, x, t);
        double n2 = 0.0;
        for (int j = 0; j < d; ++j) n2 += t[j] * t[j];
        n2b[v] = round_bf16(n2 / d);
    }
    free(x); free(t);
}

/* Prediction and variance of one (table, position) under the linear model:
 *   sigma2 = max(0, sum_v bf16(p_v) n2b[v] - ||mu||^2 / d)   (Thm. 2 with F := c + A E) */
void plo_linear_mixture(const uint16_t* A, const uint16_t* c, int V, int d, int dm, const uint16_t* logits, double lse,
                        const double* ebar, const double* n2b, double* mu, double* sigma2) {
    plo_linear_apply(A, c, d, dm, ebar, mu);
    double s = 0.0, m2 = 0.0;
    for (int v = 0; v < V; ++v) s += round_bf16(exp(half_to_double(logits[v]) - lse)) * n2b[v];
    for (int j = 0; j < d; ++j) m2 += mu[j] * mu[j];
    double r = s - m2 / d;
    *sigma2 = r > 0.0 ? r : 0.0;
}

/* ---------------------------------------------------------------- scale class */

/* Class of the per-position scale: q = clamp(round(8 log2(sigma_tot / delta)), -24, 135) with
 * sigma_tot^2 = sigma2 + sigma_floor^2.  The rounding decision is an integer decided by floating
 * point, so it is taken in binary32 on v = sigma_tot^2 / delta^2 by exponent and mantissa
 * thresholds (no transcendental): with v = m 2^e, m in [1,2),
 *   round(4 log2 v) = 4 e + #{ i in 0..3 : m >= 2^((2i+1)/8) },
 * the four thresholds rounded to binary32.  v <= 0 gives the smallest class. */
int plo_class_from_v(float v) {
    if (!(v > 0.0f)) return Q_MIN;
    if (isinf(v)) return Q_MAX;
    int e;
    float m = 2.0f * frexpf(v, &e);   /* m in [1,2), v = m 2^(e-1) */
    e -= 1;
    int q = 4 * e;
    for (int i = 0; i < 4; ++i) {
        float thr = (float)exp2((2 * i + 1) / 8.0);
        if (m >= thr) ++q;
    }
    if (q < Q_MIN) q = Q_MIN;
    if (q > Q_MAX) q = Q_MAX;
    return q;
}

int plo_class(double sigma2, float sigma_floor, float delta) {
    double var = sigma2 + (double)sigma_floor * (double)sigma_floor;
    float v = (float)(var / ((double)delta * (double)delta));
    return plo_class_from_v(v);
}

/* Class -> (bit-plane count s, table id qp).  Classes below 16 use their own table and no planes;
 * from 16 up the scale is halved s times so that the reduced scale 2^(qp/8) stays in [2,4). */
void plo_class_params(int q, int* s, int* qp) {
    if (q < 16) { *s = 0; *qp = q; }
    else { *s = (q >> 3) - 1; *qp = 8 + (q & 7); }
}

/* ---------------------------------------------------------------- quantiser */

/* Def. 6 then a uniform mid-tread quantiser of step delta, no clamping below 2^30.
 * The rounding decision is taken in binary32: mu is rounded to float, r = kv - mu,
 * t = r * (1/delta) with the reciprocal itself rounded to binary32 once, sym = nearest integer
 * (ties to even).  (The paper fixes no quantiser arithmetic, Prop. 3: "any per-vector quantizer";
 * a scaled multiply is the usual form of a uniform quantiser and keeps |KV' - KV| <= delta/2 up
 * to one part in 2^23 of the residual.) */
void plo_quantise(const uint16_t* kv, const double* mu, int d, float delta, int32_t* sym) {
    for (int j = 0; j < d; ++j) {
        float muf = (float)mu[j];
        float r = (float)half_to_double(kv[j]) - muf;
        float inv = 1.0f / delta;
        float t = r * inv;
        float n = nearbyintf(t);
        if (n > (float)SYM_LIMIT) n = (float)SYM_LIMIT;
        if (n < -(float)SYM_LIMIT) n = -(float)SYM_LIMIT;
        sym[j] = (int32_t)n;
    }
}

/* Prop. 3, "Correctness": KV = R + KV^, with R at its quantised value; one fused binary32 step. */
void plo_reconstruct(const double* mu, const int32_t* sym, int d, float delta, float* out) {
    for (int j = 0; j < d; ++j) out[j] = fmaf((float)sym[j], delta, (float)mu[j]);
}

/* ---------------------------------------------------------------- rotated fixed-rate quantiser */

/* Prop. 3, step 3: "any per-vector quantizer" applied to R_i.  Besides the entropy-coded uniform
 * quantiser above, the codec offers the generic member of the family the paper points to (a
 * random rotation followed by a b-bit scalar quantiser; the paper gives no details of TurboQuant,
 * so nothing of it is reproduced here).  For one residual vector r of d = 2^m components:
 *   x_j = eps_j r_j                          eps_j = -1 where neg[j] != 0, else +1   (input to the method)
 *   y_k = d^(-1/2) sum_j (-1)^popcount(j & k) x_j      (Sylvester-Hadamard matrix, orthonormal, symmetric)
 *   s   = max_k |y_k|                                   (per-vector scale, stored as binary32)
 *   c_k = clamp(floor((y_k / s + 1) 2^b / 2), 0, 2^b - 1)          (mid-rise, 2^b levels on [-s, s])
 * and back:  y^_k = s ((c_k + 1/2) 2 / 2^b - 1),  x^ = H y^ (the same matrix),  r^_j = eps_j x^_j,
 * so |y^_k - y_k| <= s / 2^b and ||r^ - r||_2 = ||y^ - y||_2 <= sqrt(d) s / 2^b.
 * The transform is written out from its definition, O(d^2), in double. */
static int parity(unsigned v) { int p = 0; while (v) { p ^= 1; v &= v - 1; } return p; }

void plo_rotq_rotate(const double* r, const uint8_t* neg, int d, double* y) {
    const double norm = 1.0 / sqrt((double)d);
    for (int k = 0; k < d; ++k) {
        double acc = 0.0;
        for (int j = 0; j < d; ++j) {
            double x = neg[j] ? -r[j] : r[j];
            acc += parity((unsigned)(j & k)) ? -x : x;
        }
        y[k] = acc * norm;
    }
}

void plo_rotq_unrotate(const double* y, const uint8_t* neg, int d, double* r) {
    const double norm = 1.0 / sqrt((double)d);
    for (int j = 0; j < d; ++j) {
        double acc = 0.0;
        for (int k = 0; k < d; ++k) acc += parity((unsigned)(j & k)) ? -y[k] : y[k];
        acc *= norm;
        r[j] = neg[j] ? -acc : acc;
    }
}

/* Residual (Def. 6) of one vector, rotation, scale and codes.  The decisions (scale, codes) are taken
 * in binary32, the precision of the kernels: y is rounded to float, s = max |y| as a float,
 * c = floor(fma(y * (1/s), 2^b / 2, 2^b / 2)) with the reciprocal rounded once; s = 0 gives the middle
 * level everywhere and reconstructs to zero. */
int plo_rotq_quantise(const uint16_t* kv, const double* mu, const uint8_t* neg, int d, int b, float* scale, int32_t* code) {
    if (d < 1 || d > 4096 || (d & (d - 1)) || b < 1 || b > 8) return PLO_E_INVALID;
    double r[4096], y[4096];
    for (int j = 0; j < d; ++j) r[j] = (double)((float)half_to_double(kv[j]) - (float)mu[j]);
    plo_rotq_rotate(r, neg, d, y);
    float s = 0.0f;
    for (int k = 0; k < d; ++k) { float a = fabsf((float)y[k]); if (a > s) s = a; }
    const float inv = s > 0.0f ? 1.0f / s : 0.0f, half_levels = (float)(1 << b) * 0.5f;
    for (int k = 0; k < d; ++k) {
        float u = fmaf((float)y[k] * inv, half_levels, half_levels);
        int c = (int)floorf(u);
        if (c < 0) c = 0;
        if (c > (1 << b) - 1) c = (1 << b) - 1;
        code[k] = c;
    }
    *scale = s;
    return PLO_OK;
}

/* Prop. 3, "Correctness": KV' = KV^ + r^ with r^ rebuilt from the codes. */
int plo_rotq_reconstruct(const double* mu, const uint8_t* neg, int d, int b, float scale, const int32_t* code, float* out) {
    if (d < 1 || d > 4096 || (d & (d - 1)) || b < 1 || b > 8) return PLO_E_INVALID;
    double yq[4096], r[4096];
    for (int k = 0; k < d; ++k)
        yq[k] = (double)(scale * fmaf((float)code[k] + 0.5f, 2.0f / (float)(1 << b), -1.0f));
    plo_rotq_unrotate(yq, neg, d, r);
    for (int j = 0; j < d; ++j) out[j] = (float)mu[j] + (float)r[j];
    return PLO_OK;
}

/* Record of one vector: the scale (binary32, little endian) followed by (d/32) * b words of 32 bits.
 * Word g*b + p holds bit p of the codes of 32 components, one per lane: lane l's g-th component is
 * the one the rANS format gives to that lane (comp_index).  4 + d*b/8 bytes. */
static int comp_index(int l, int g, int d);
int plo_rotq_pack(const int32_t* code, float scale, int d, int b, uint8_t* rec) {
    if (!(d == 32 || d == 64 || d == 128 || d == 256) || b < 1 || b > 8) return PLO_E_INVALID;
    memcpy(rec, &scale, 4);
    const int G = d / NLANES;
    for (int g = 0; g < G; ++g)
        for (int p = 0; p < b; ++p) {
            uint32_t w = 0;
            for (int l = 0; l < NLANES; ++l) w |= (uint32_t)((code[comp_index(l, g, d)] >> p) & 1) << l;
            memcpy(rec + 4 + 4 * (g * b + p), &w, 4);
        }
    return PLO_OK;
}

int plo_rotq_unpack(const uint8_t* rec, int d, int b, float* scale, int32_t* code) {
    if (!(d == 32 || d == 64 || d == 128 || d == 256) || b < 1 || b > 8) return PLO_E_INVALID;
    memcpy(scale, rec, 4);
    const int G = d / NLANES;
    for (int j = 0; j < d; ++j) code[j] = 0;
    for (int g = 0; g < G; ++g)
        for (int p = 0; p < b; ++p) {
            uint32_t w;
            memcpy(&w, rec + 4 + 4 * (g * b + p), 4);
            for (int l = 0; l < NLANES; ++l) code[comp_index(l, g, d)] |= (int32_t)((w >> l) & 1u) << p;
        }
    return PLO_OK;
}

/* ---------------------------------------------------------------- frequency tables */

/* Discretised Laplace of standard deviation s' = 2^(qp/8) over the signed integer hi:
 *   P(|hi| >= k) = exp(-(k - 1/2) sqrt2 / s'),  k >= 1,  split evenly between the two signs.
 * Integer construction (so that both ends of the codec can rebuild it bit for bit):
 *   theta = round(2^32 exp(-sqrt2/s')),  rho = round(2^32 exp(-sqrt2/(2 s')))
 *   G[0] = 2^32, G[1] = rho, G[k+1] = (G[k] theta) >> 32            (k = 1..31)
 *   f(0)     = max(1, (G[0]-G[1]) >> 17)
 *   f(+-k)   = max(1, (G[k]-G[k+1]) >> 18)                           (k = 1..31)
 *   f(ESC)   = max(1, G[32] >> 17)
 *   f(0)    += 2^15 - sum f                                           (normalisation)
 * Alphabet order (zigzag): 0, +1, -1, +2, -2, ..., +31, -31, ESC.  c = exclusive prefix sums. */
int plo_table_constants(int qp, uint32_t* theta, uint32_t* rho) {
    if (qp < Q_MIN || qp > 15) return PLO_E_INVALID;
    double s = exp2(qp / 8.0);
    double x = sqrt(2.0) / s;
    *theta = (uint32_t)llround(4294967296.0 * exp(-x));
    *rho = (uint32_t)llround(4294967296.0 * exp(-x / 2.0));
    return PLO_OK;
}

int plo_build_table(int qp, uint32_t* f /*[64]*/, uint32_t* c /*[65]*/) {
    uint32_t theta, rho;
    int rc = plo_table_constants(qp, &theta, &rho);
    if (rc) return rc;
    uint64_t G[HI_MAX + 2];
    G[0] = 1ull << 32; G[1] = rho;
    for (int k = 1; k <= HI_MAX; ++k) G[k + 1] = (G[k] * (uint64_t)theta) >> 32;
    int64_t sum = 0;
    uint64_t m0 = (G[0] - G[1]) >> 17;
    f[0] = (uint32_t)(m0 < 1 ? 1 : m0);
    for (int k = 1; k <= HI_MAX; ++k) {
        uint64_t mk = (G[k] - G[k + 1]) >> 18;
        uint32_t fk = (uint32_t)(mk < 1 ? 1 : mk);
        f[2 * k - 1] = fk; f[2 * k] = fk;
    }
    uint64_t me = G[HI_MAX + 1] >> 17;
    f[ESC] = (uint32_t)(me < 1 ? 1 : me);
    for (int i = 0; i < NSYM; ++i) sum += f[i];
    int64_t f0 = (int64_t)f[0] + ((int64_t)PROB_M - sum);
    if (f0 < 1) return PLO_E_INVALID;
    f[0] = (uint32_t)f0;
    c[0] = 0;
    for (int i = 0; i < NSYM; ++i) c[i + 1] = c[i] + f[i];
    return PLO_OK;
}

/* ---------------------------------------------------------------- rANS chunk coder */

/* Split of a symbol under s bit planes (s = 0: hi = sym, no planes):
 *   u = sym + 2^(s-1),  hi = floor(u / 2^s),  lo = u mod 2^s   <=>   sym = hi 2^s + lo - 2^(s-1). */
static void split_sym(int32_t sym, int s, int32_t* hi, uint32_t* lo) {
    if (s == 0) { *hi = sym; *lo = 0; return; }
    int64_t u = (int64_t)sym + ((int64_t)1 << (s - 1));
    int64_t h = u >> s;                              /* arithmetic shift = floor */
    *hi = (int32_t)h; *lo = (uint32_t)(u - (h << s));
}
static int32_t join_sym(int32_t hi, uint32_t lo, int s) {
    if (s == 0) return hi;
    return (int32_t)(((int64_t)hi << s) + (int64_t)lo - ((int64_t)1 << (s - 1)));
}
static int comp_index(int l, int g, int d) {
    int R = d / 8, G = d / NLANES;
    return 8 * (l % R) + G * (l / R) + g;
}
static int valid_d(int d) { return d == 32 || d == 64 || d == 128 || d == 256; }
static int zigzag(int32_t hi) { return hi > 0 ? 2 * hi - 1 : -2 * hi; }
static int32_t unzigzag(int zz) { return (zz & 1) ? (zz + 1) / 2 : -(zz / 2); }

/* Class value that marks a position carrying no symbols at all (zero-rate rule, Thm. 3). */
#define PLO_Q_SKIP (-100000)
int plo_q_skip(void) { return PLO_Q_SKIP; }

/* A chunk is P consecutive positions of one stream (one d-vector per position); d = 32 G, d in
 * {32, 64, 128, 256}.  The vector is cut into R = d/8 groups of 8 components (16 bytes of f16);
 * lane l (0..31) owns, in group l mod R, the G components starting at G*(l div R):
 *   component(l, g) = 8 (l mod R) + G (l div R) + g,  g = 0..G-1,
 * and keeps one rANS state in [2^16, 2^32).
 * The chunk's bytes are: 32 little-endian uint32 decoder start states (lane 0..31), then a
 * sequence of little-endian 16-bit words in the order the decoder consumes them:
 *   for position p ascending, for g ascending:
 *     (1) s plane words: for b = 0..s-1 a 32-bit word whose bit l is bit b of lane l's lo,
 *         low half first;
 *     (2) for lanes ascending, the refill word of every lane whose state fell below 2^16 after
 *         its symbol was decoded;
 *     (3) for lanes ascending among those that decoded ESC, the raw 32-bit hi, low half first.
 * Decoder step for a lane: slot = x mod 2^15; zz = symbol with c[zz] <= slot < c[zz+1];
 *   x = f[zz] (x >> 15) + slot - c[zz]; if x < 2^16: x = (x << 16) | word.
 * Encoder step (run in exactly the reverse order, words written back to front):
 *   if x >= f << 17: emit x mod 2^16, x >>= 16;  x = ((x / f) << 15) + (x mod f) + c.
 * Encoder start state 2^16 per lane; a valid chunk decodes back to that state in every lane.
 *
 * ideal_bits (optional) = sum over coded symbols of log2(2^15 / f) + 32 per escape + s per
 * component: the code length the model assigns, which the byte count may exceed only by the
 * state flush. */
int plo_rans_encode_chunk(const int32_t* sym /*[P][d]*/, const int32_t* q /*[P]*/, int P, int d,
                          uint8_t* out, uint64_t cap, uint64_t* nbytes, double* ideal_bits,
                          uint64_t* n_escapes) {
    if (!valid_d(d) || P < 0) return PLO_E_INVALID;
    int G = d / NLANES;
    size_t wcap = (size_t)P * d * 4 + 16;
    uint16_t* words = (uint16_t*)malloc(wcap * sizeof(uint16_t));
    if (!words) return PLO_E_INVALID;
    size_t wp = wcap;
    uint32_t x[NLANES];
    for (int l = 0; l < NLANES; ++l) x[l] = RANS_L;
    double ideal = 0.0; uint64_t nesc = 0;
    uint32_t f[NSYM], c[NSYM + 1];
    int cur_qp = 1000;
    for (int p = P - 1; p >= 0; --p) {
        int s, qp;
        if (q[p] == PLO_Q_SKIP) continue;              /* zero-rate position: nothing in the stream */
        if (q[p] < Q_MIN || q[p] > Q_MAX) { free(words); return PLO_E_INVALID; }
        plo_class_params(q[p], &s, &qp);
        if (qp != cur_qp) { plo_build_table(qp, f, c); cur_qp = qp; }
        for (int g = G - 1; g >= 0; --g) {
            int32_t hi[NLANES]; uint32_t lo[NLANES];
            for (int l = 0; l < NLANES; ++l) split_sym(sym[(size_t)p * d + comp_index(l, g, d)], s, &hi[l], &lo[l]);
            /* (3) escapes, lanes descending, high half pushed first so that low half reads first */
            for (int l = NLANES - 1; l >= 0; --l) {
                if (hi[l] > HI_MAX || hi[l] < -HI_MAX) {
                    uint32_t raw = (uint32_t)hi[l];
                    words[--wp] = (uint16_t)(raw >> 16);
                    words[--wp] = (uint16_t)(raw & 0xFFFF);
                    ideal += 32.0; ++nesc;
                }
            }
            /* (2) symbols, lanes descending */
            for (int l = NLANES - 1; l >= 0; --l) {
                int zz = (hi[l] > HI_MAX || hi[l] < -HI_MAX) ? ESC : zigzag(hi[l]);
                uint32_t fs = f[zz], cs = c[zz];
                if ((uint64_t)x[l] >= ((uint64_t)fs << 17)) { words[--wp] = (uint16_t)(x[l] & 0xFFFF); x[l] >>= 16; }
                x[l] = ((x[l] / fs) << PROB_BITS) + (x[l] % fs) + cs;
                ideal += log2((double)PROB_M / fs);
            }
            /* (1) planes, b descending, high half pushed first */
            for (int b = s - 1; b >= 0; --b) {
                uint32_t plane = 0;
                for (int l = 0; l < NLANES; ++l) plane |= ((lo[l] >> b) & 1u) << l;
                words[--wp] = (uint16_t)(plane >> 16);
                words[--wp] = (uint16_t)(plane & 0xFFFF);
            }
            ideal += (double)s * NLANES;
        }
    }
    size_t nwords = wcap - wp;
    uint64_t total = 4 * NLANES + 2 * (uint64_t)nwords;
    *nbytes = total;
    if (ideal_bits) *ideal_bits = ideal;
    if (n_escapes) *n_escapes = nesc;
    if (total > cap) { free(words); return PLO_E_CAPACITY; }
    for (int l = 0; l < NLANES; ++l) {
        out[4 * l + 0] = (uint8_t)(x[l]); out[4 * l + 1] = (uint8_t)(x[l] >> 8);
        out[4 * l + 2] = (uint8_t)(x[l] >> 16); out[4 * l + 3] = (uint8_t)(x[l] >> 24);
    }
    for (size_t i = 0; i < nwords; ++i) {
        out[4 * NLANES + 2 * i] = (uint8_t)(words[wp + i]);
        out[4 * NLANES + 2 * i + 1] = (uint8_t)(words[wp + i] >> 8);
    }
    free(words);
    return PLO_OK;
}

int plo_rans_decode_chunk(const uint8_t* in, uint64_t nbytes, const int32_t* q /*[P]*/, int P, int d,
                          int32_t* sym /*[P][d]*/) {
    if (!valid_d(d) || P < 0) return PLO_E_INVALID;
    if (nbytes < 4 * NLANES || (nbytes & 1)) return PLO_E_CORRUPT;
    int G = d / NLANES;
    uint64_t nwords = (nbytes - 4 * NLANES) / 2, rp = 0;
    const uint8_t* wb = in + 4 * NLANES;
#define NEXT_WORD(dst) do { if (rp >= nwords) return PLO_E_CORRUPT; \
        (dst) = (uint32_t)wb[2 * rp] | ((uint32_t)wb[2 * rp + 1] << 8); ++rp; } while (0)
    uint32_t x[NLANES];
    for (int l = 0; l < NLANES; ++l) {
        x[l] = (uint32_t)in[4 * l] | ((uint32_t)in[4 * l + 1] << 8) | ((uint32_t)in[4 * l + 2] << 16) |
               ((uint32_t)in[4 * l + 3] << 24);
        if (x[l] < RANS_L) return PLO_E_CORRUPT;
    }
    uint32_t f[NSYM], c[NSYM + 1];
    int cur_qp = 1000;
    for (int p = 0; p < P; ++p) {
        int s, qp;
        if (q[p] == PLO_Q_SKIP) { for (int j = 0; j < d; ++j) sym[(size_t)p * d + j] = 0; continue; }
        if (q[p] < Q_MIN || q[p] > Q_MAX) return PLO_E_INVALID;
        plo_class_params(q[p], &s, &qp);
        if (qp != cur_qp) { plo_build_table(qp, f, c); cur_qp = qp; }
        for (int g = 0; g < G; ++g) {
            uint32_t lo[NLANES]; int zzs[NLANES];
            for (int l = 0; l < NLANES; ++l) lo[l] = 0;
            for (int b = 0; b < s; ++b) {
                uint32_t wlo, whi; NEXT_WORD(wlo); NEXT_WORD(whi);
                uint32_t plane = wlo | (whi << 16);
                for (int l = 0; l < NLANES; ++l) lo[l] |= ((plane >> l) & 1u) << b;
            }
            for (int l = 0; l < NLANES; ++l) {
                uint32_t slot = x[l] & (PROB_M - 1);
                int zz = 0;
                while (c[zz + 1] <= slot) ++zz;
                x[l] = f[zz] * (x[l] >> PROB_BITS) + slot - c[zz];
                if (x[l] < RANS_L) { uint32_t w; NEXT_WORD(w); x[l] = (x[l] << 16) | w; }
                zzs[l] = zz;
            }
            for (int l = 0; l < NLANES; ++l) {
                int32_t hi;
                if (zzs[l] == ESC) { uint32_t a, b2; NEXT_WORD(a); NEXT_WORD(b2); hi = (int32_t)(a | (b2 << 16)); }
                else hi = unzigzag(zzs[l]);
                sym[(size_t)p * d + comp_index(l, g, d)] = join_sym(hi, lo[l], s);
            }
        }
    }
#undef NEXT_WORD
    if (rp != nwords) return PLO_E_CORRUPT;
    for (int l = 0; l < NLANES; ++l) if (x[l] != RANS_L) return PLO_E_CORRUPT;
    return PLO_OK;
}

/* ---------------------------------------------------------------- prefix dedup */

/* Def. 2: s ^ s' is the maximal common prefix; d_T(s,s') = -log2 P(s ^ s'), with
 * P(prefix) = prod_j P(x_j | x_<j) (Def. 1: edge weights of the trie), i.e. minus the sum of the
 * first lcp values of logp2[s][.]; zero for an empty common prefix.
 * Best match (Sec. 7.3: follow the query's path and return the deepest stored ancestor), applied
 * to sessions in arrival order: parent[s] = the earlier session with the longest common prefix,
 * ties to the smallest index; shared_len[s] = that length; no earlier session or length 0 -> -1, 0. */
void plo_prefix_dedup(const int32_t* tokens, const int32_t* lens, const float* logp2, int S, int64_t stride,
                      int32_t* lcp /*[S][S]*/, double* dT /*[S][S]*/, int32_t* parent, int32_t* shared_len) {
    for (int a = 0; a < S; ++a)
        for (int b = 0; b < S; ++b) {
            int m = lens[a] < lens[b] ? lens[a] : lens[b], n = 0;
            while (n < m && tokens[a * stride + n] == tokens[b * stride + n]) ++n;
            lcp[a * S + b] = n;
            double bits = 0.0;
            for (int j = 0; j < n; ++j) bits -= (double)logp2[a * stride + j];
            dT[a * S + b] = bits;
        }
    for (int a = 0; a < S; ++a) {
        int best = -1, bl = 0;
        for (int b = 0; b < a; ++b) if (lcp[a * S + b] > bl) { bl = lcp[a * S + b]; best = b; }
        parent[a] = best; shared_len[a] = bl;
    }
}

/* Def. 3 (semantic prefix cluster at threshold delta; centroid = its most probable member) on the
 * matrices of plo_prefix_dedup.  Reading taken: with d_T = -log2 P(s ^ s') (Def. 2) a LONGER shared
 * prefix gives a LARGER d_T, and d_T(a,c) >= min(d_T(a,b), d_T(b,c)); the relation the definition
 * needs -- one whose maximal subsets are unique -- is therefore "the shared prefix carries at least
 * delta bits", d_T(s,s') >= delta, which is an equivalence by that inequality (the printed "<="
 * is not: it would separate exactly the sessions that share the most).  A session is always a member
 * of its own cluster.  cluster[s] = smallest member index; centroid[s] = member with the largest
 * P(s') = 2^-d_T(s',s') (ties: smallest index); begin[s] = first position of s that is not covered by
 * the centroid's cache (0 for the centroid itself): the tail Cor. 3 charges for. */
void plo_prefix_clusters(const int32_t* lcp /*[S][S]*/, const double* dT /*[S][S]*/, int S, double delta,
                         int32_t* cluster, int32_t* centroid, int32_t* begin) {
    for (int a = 0; a < S; ++a) {
        int first = a, best = a;
        for (int b = 0; b < S; ++b) {
            if (b != a && !(dT[(size_t)a * S + b] >= delta)) continue;
            if (b < first) first = b;
            double pb = dT[(size_t)b * S + b], pbest = dT[(size_t)best * S + best];
            if (pb < pbest || (pb == pbest && b < best)) best = b;
        }
        cluster[a] = first; centroid[a] = best;
        begin[a] = best == a ? 0 : lcp[(size_t)a * S + best];
    }
}

/* ---------------------------------------------------------------- adaptive step */

/* Def. 7 (surprisal-adaptive quantiser): at a position of surprisal h = -log2 P(x_i | x_<i) the
 * residual gets b = max(1, floor(b0 h / hbar)) bits per component.  With an entropy coder behind
 * the quantiser a bit more means half the step, so the position's step is delta 2^(b0 - b): b = b0
 * reproduces the fixed-step coder.  The paper puts no upper limit on b; the symbol range is
 * finite, so b is capped at b0 + extra.  The floor is an integer decided by floating point: it is
 * taken in binary32 on h rounded to binary32. */
int plo_adaptive_bits(float h, int b0, float hbar, int extra) {
    float r = (float)b0 * (h / hbar);
    int b = (int)floorf(r);
    if (!(r >= 1.0f)) b = 1;
    if (b > b0 + extra) b = b0 + extra;
    return b;
}

/* ---------------------------------------------------------------- zero-rate rule */

/* Thm. 3 / Cor. 6 (reverse water-filling): a position whose residual variance per component does
 * not exceed the target distortion D needs no bits; the decoder then takes KV' = KV^.  The
 * variance the coder knows is the mixture's (plus the optional floor), and its comparison with D
 * is taken on the integer scale class q = round(4 log2(sigma^2 / step^2)), so that both sides
 * decide alike: a position is skipped iff q <= floor(4 log2(D / step^2) - 1/2), which implies
 * sigma^2 <= D (the rounding of q is at most 1/2).  D <= 0 switches the rule off. */
int plo_zero_class(double D, double step) {
    if (!(D > 0.0)) return -1000000;
    return (int)floor(4.0 * log2(D / (step * step)) - 0.5);
}

/* ---------------------------------------------------------------- whole path */

/* Strides, in elements, of a KV tensor whose last dimension (d) is contiguous. */
typedef struct { int64_t layer, kv, session, head, pos; } plo_kv_strides;

typedef struct {
    int32_t L, H, d, V, K;
    float delta, sigma_floor;
    int32_t chunk_pos;
    int32_t dense;          /* 0: top-K mixture, 1: full-vocabulary bf16 mixture */
    int32_t adaptive_b0;    /* > 0: surprisal-adaptive step (Def. 7) with target depth b0 */
    int32_t adaptive_extra; /* cap: b_i <= b0 + adaptive_extra */
    float adaptive_hbar;    /* average surprisal h-bar, bits */
    /* dense == 2: linear-embedding predictor F(t) ~ c + A E(t) (Sec. 7.1); T is not used */
    int32_t lin_dm;               /* embedding width d_model */
    const uint16_t* lin_E;        /* [V][dm] f16 token embeddings */
    const uint16_t* lin_A;        /* [L][2][H][d][dm] f16 */
    const uint16_t* lin_c;        /* [L][2][H][d] f16 */
    float zero_D;                 /* > 0: zero-rate rule (Thm. 3) at target distortion D per component */
} plo_config;

typedef struct {
    double ideal_bits;      /* model code length of everything coded */
    double token_bits;      /* sum of -log2 P(x_i | x_<i) over coded positions */
    uint64_t payload_bytes; /* sum of exact chunk sizes */
    uint64_t n_chunks, n_escapes, coded_positions;
    uint64_t skipped_vectors; /* (stream, position) pairs left out by the zero-rate rule */
} plo_stats;

static int64_t chunk_slot(const plo_config* c, int S, int max_chunks, int s, int l, int kv, int h, int ch) {
    (void)S;
    return ((((int64_t)s * c->L + l) * 2 + kv) * c->H + h) * max_chunks + ch;
}

/* Encode (Sec. 7.2, integration point 1, for every position in [pos_begin[s], pos_end[s]) of
 * every session; Prop. 2: positions before pos_begin cost nothing).  The index is
 * [S][L][2][H][max_chunks]; payloads are laid out in that order, each starting on a 16-byte
 * boundary of `payload`.  Optional exports, each [S][n][L][2][H] outermost-to-innermost with
 * d innermost where it applies: sym_out (int32), q_out (int32), mu_out (float). */
int plo_encode(const plo_config* cfg, const uint16_t* T, const uint16_t* kv, const plo_kv_strides* st,
               const uint16_t* logits /*[S][n][V]*/, const int32_t* tokens /*[S][n]*/, int S, int n,
               const int32_t* pos_begin, const int32_t* pos_end, int max_chunks,
               uint8_t* payload, uint64_t cap, uint64_t* chunk_offset, uint32_t* chunk_bytes,
               plo_stats* stats, int32_t* sym_out, int32_t* q_out, float* mu_out, int32_t* bits_out /*[S][n]*/) {
    int L = cfg->L, H = cfg->H, d = cfg->d, V = cfg->V, K = cfg->K, CP = cfg->chunk_pos;
    if (!valid_d(d) || CP < 1) return PLO_E_INVALID;
    if (cfg->adaptive_b0 > 0 && !tokens) return PLO_E_INVALID;
    float* pdelta = (float*)malloc(sizeof(float) * (size_t)n);   /* step of each position of the session */
    memset(stats, 0, sizeof(*stats));
    int32_t* idx = (int32_t*)malloc(sizeof(int32_t) * (size_t)n * K);
    double* w = (double*)malloc(sizeof(double) * (size_t)n * K);
    double* lse = (double*)malloc(sizeof(double) * (size_t)n);
    double* zk = (double*)malloc(sizeof(double) * (size_t)n);
    double* lp = (double*)malloc(sizeof(double) * (size_t)n);
    int32_t* csym = (int32_t*)malloc(sizeof(int32_t) * (size_t)CP * d);
    int32_t* cq = (int32_t*)malloc(sizeof(int32_t) * (size_t)CP);
    double* mu = (double*)malloc(sizeof(double) * (size_t)d);
    uint64_t cursor = 0; int rc = PLO_OK;
    for (int64_t i = 0; i < (int64_t)S * L * 2 * H * max_chunks; ++i) { chunk_offset[i] = 0; chunk_bytes[i] = 0; }
    for (int s = 0; s < S && !rc; ++s) {
        int b = pos_begin ? pos_begin[s] : 0, e = pos_end ? pos_end[s] : n;
        if (b < 0 || e > n || b > e) { rc = PLO_E_INVALID; break; }
        for (int i = b; i < e; ++i) {
            plo_topk_softmax_row(logits + ((size_t)s * n + i) * V, V, K, tokens ? tokens[(size_t)s * n + i] : -1,
                                 idx + (size_t)i * K, w + (size_t)i * K, lse + i, zk + i, lp + i);
            if (tokens) stats->token_bits -= lp[i];
            pdelta[i] = cfg->delta;
            if (cfg->adaptive_b0 > 0) {
                int bi = plo_adaptive_bits((float)(-lp[i]), cfg->adaptive_b0, cfg->adaptive_hbar, cfg->adaptive_extra);
                pdelta[i] = ldexpf(cfg->delta, cfg->adaptive_b0 - bi);
                if (bits_out) bits_out[(size_t)s * n + i] = bi;
            }
        }
        stats->coded_positions += (uint64_t)(e - b);
        const int lin = cfg->dense == 2, dm = cfg->lin_dm;
        double* ebar = NULL; double* n2b = NULL;
        if (lin) {
            ebar = (double*)malloc(sizeof(double) * (size_t)n * dm);
            n2b = (double*)malloc(sizeof(double) * (size_t)V);
            for (int i = b; i < e; ++i)
                plo_expected_embedding(cfg->lin_E, V, dm, logits + ((size_t)s * n + i) * V, lse[i], ebar + (size_t)i * dm);
        }
        for (int l = 0; l < L && !rc; ++l) for (int a = 0; a < 2 && !rc; ++a) for (int h = 0; h < H && !rc; ++h) {
            const size_t tix = ((size_t)l * 2 + a) * H + h;
            const uint16_t* table = lin ? NULL : T + (tix * (size_t)V) * d;
            const uint16_t* At = lin ? cfg->lin_A + tix * (size_t)d * dm : NULL;
            const uint16_t* ct = lin ? cfg->lin_c + tix * (size_t)d : NULL;
            if (lin) plo_linear_rownorms(cfg->lin_E, At, ct, V, d, dm, n2b);
            for (int ch = 0; b + ch * CP < e; ++ch) {
                int p0 = b + ch * CP, P = e - p0 < CP ? e - p0 : CP;
                for (int p = 0; p < P; ++p) {
                    int i = p0 + p; double s2;
                    if (lin) plo_linear_mixture(At, ct, V, d, dm, logits + ((size_t)s * n + i) * V, lse[i], ebar + (size_t)i * dm, n2b, mu, &s2);
                    else if (cfg->dense) plo_dense_mixture(table, V, d, logits + ((size_t)s * n + i) * V, lse[i], mu, &s2);
                    else plo_mixture(table, d, idx + (size_t)i * K, w + (size_t)i * K, K, mu, &s2);
                    cq[p] = plo_class(s2, cfg->sigma_floor, pdelta[i]);
                    const int skip = cq[p] <= plo_zero_class((double)cfg->zero_D, (double)pdelta[i]);
                    const uint16_t* x = kv + l * st->layer + a * st->kv + s * st->session + h * st->head + (int64_t)i * st->pos;
                    plo_quantise(x, mu, d, pdelta[i], csym + (size_t)p * d);
                    if (skip) memset(csym + (size_t)p * d, 0, sizeof(int32_t) * (size_t)d);
                    size_t o = ((((size_t)s * n + i) * L + l) * 2 + a) * H + h;
                    if (sym_out) memcpy(sym_out + o * d, csym + (size_t)p * d, sizeof(int32_t) * d);
                    if (q_out) q_out[o] = cq[p];
                    if (skip) { cq[p] = PLO_Q_SKIP; stats->skipped_vectors++; }
                    if (mu_out) for (int j = 0; j < d; ++j) mu_out[o * d + j] = (float)mu[j];
                }
                uint64_t nb = 0, nesc = 0; double ideal = 0.0;
                cursor = (cursor + 15) & ~(uint64_t)15;
                int r = plo_rans_encode_chunk(csym, cq, P, d, payload + cursor, cursor < cap ? cap - cursor : 0, &nb, &ideal, &nesc);
                if (r) { rc = r; break; }
                int64_t slot = chunk_slot(cfg, S, max_chunks, s, l, a, h, ch);
                chunk_offset[slot] = cursor; chunk_bytes[slot] = (uint32_t)nb;
                cursor += nb;
                stats->ideal_bits += ideal; stats->payload_bytes += nb; stats->n_chunks++; stats->n_escapes += nesc;
            }
        }
        free(ebar); free(n2b);
    }
    free(idx); free(w); free(lse); free(zk); free(lp); free(csym); free(cq); free(mu); free(pdelta);
    return rc;
}

/* Decode (Sec. 7.2, integration point 2): the prediction and its class are recomputed from the
 * logits exactly as in the encoder, the symbols come from the chunk, KV' = mu + sym delta.
 * kv_out is float with the same strides; positions outside [pos_begin, pos_end) are not written. */
int plo_decode(const plo_config* cfg, const uint16_t* T, const uint16_t* logits, const int32_t* tokens, int S, int n,
               const int32_t* pos_begin, const int32_t* pos_end, int max_chunks,
               const uint8_t* payload, const uint64_t* chunk_offset, const uint32_t* chunk_bytes,
               float* kv_out, const plo_kv_strides* st, int32_t* sym_out) {
    int L = cfg->L, H = cfg->H, d = cfg->d, V = cfg->V, K = cfg->K, CP = cfg->chunk_pos;
    if (!valid_d(d) || CP < 1) return PLO_E_INVALID;
    int32_t* idx = (int32_t*)malloc(sizeof(int32_t) * (size_t)n * K);
    double* w = (double*)malloc(sizeof(double) * (size_t)n * K);
    double* lse = (double*)malloc(sizeof(double) * (size_t)n);
    double zk, lp;
    int32_t* csym = (int32_t*)malloc(sizeof(int32_t) * (size_t)CP * d);
    int32_t* cq = (int32_t*)malloc(sizeof(int32_t) * (size_t)CP);
    double* mus = (double*)malloc(sizeof(double) * (size_t)CP * d);
    float* pdelta = (float*)malloc(sizeof(float) * (size_t)n);
    int rc = PLO_OK;
    if (cfg->adaptive_b0 > 0 && !tokens) rc = PLO_E_INVALID;
    for (int s = 0; s < S && !rc; ++s) {
        int b = pos_begin ? pos_begin[s] : 0, e = pos_end ? pos_end[s] : n;
        if (b < 0 || e > n || b > e) { rc = PLO_E_INVALID; break; }
        for (int i = b; i < e; ++i) {
            plo_topk_softmax_row(logits + ((size_t)s * n + i) * V, V, K, tokens ? tokens[(size_t)s * n + i] : -1,
                                 idx + (size_t)i * K, w + (size_t)i * K, lse + i, &zk, &lp);
            pdelta[i] = cfg->delta;
            if (cfg->adaptive_b0 > 0) {
                int bi = plo_adaptive_bits((float)(-lp), cfg->adaptive_b0, cfg->adaptive_hbar, cfg->adaptive_extra);
                pdelta[i] = ldexpf(cfg->delta, cfg->adaptive_b0 - bi);
            }
        }
        const int lin = cfg->dense == 2, dm = cfg->lin_dm;
        double* ebar = NULL; double* n2b = NULL;
        if (lin) {
            ebar = (double*)malloc(sizeof(double) * (size_t)n * dm);
            n2b = (double*)malloc(sizeof(double) * (size_t)V);
            for (int i = b; i < e; ++i)
                plo_expected_embedding(cfg->lin_E, V, dm, logits + ((size_t)s * n + i) * V, lse[i], ebar + (size_t)i * dm);
        }
        for (int l = 0; l < L && !rc; ++l) for (int a = 0; a < 2 && !rc; ++a) for (int h = 0; h < H && !rc; ++h) {
            const size_t tix = ((size_t)l * 2 + a) * H + h;
            const uint16_t* table = lin ? NULL : T + (tix * (size_t)V) * d;
            const uint16_t* At = lin ? cfg->lin_A + tix * (size_t)d * dm : NULL;
            const uint16_t* ct = lin ? cfg->lin_c + tix * (size_t)d : NULL;
            if (lin) plo_linear_rownorms(cfg->lin_E, At, ct, V, d, dm, n2b);
            for (int ch = 0; b + ch * CP < e; ++ch) {
                int p0 = b + ch * CP, P = e - p0 < CP ? e - p0 : CP;
                for (int p = 0; p < P; ++p) {
                    int i = p0 + p; double s2;
                    if (lin) plo_linear_mixture(At, ct, V, d, dm, logits + ((size_t)s * n + i) * V, lse[i], ebar + (size_t)i * dm, n2b, mus + (size_t)p * d, &s2);
                    else if (cfg->dense) plo_dense_mixture(table, V, d, logits + ((size_t)s * n + i) * V, lse[i], mus + (size_t)p * d, &s2);
                    else plo_mixture(table, d, idx + (size_t)i * K, w + (size_t)i * K, K, mus + (size_t)p * d, &s2);
                    cq[p] = plo_class(s2, cfg->sigma_floor, pdelta[i]);
                    if (cq[p] <= plo_zero_class((double)cfg->zero_D, (double)pdelta[i])) cq[p] = PLO_Q_SKIP;
                }
                int64_t slot = chunk_slot(cfg, S, max_chunks, s, l, a, h, ch);
                int r = plo_rans_decode_chunk(payload + chunk_offset[slot], chunk_bytes[slot], cq, P, d, csym);
                if (r) { rc = r; break; }
                for (int p = 0; p < P; ++p) {
                    int i = p0 + p;
                    float* o = kv_out + l * st->layer + a * st->kv + s * st->session + h * st->head + (int64_t)i * st->pos;
                    plo_reconstruct(mus + (size_t)p * d, csym + (size_t)p * d, d, pdelta[i], o);
                    if (sym_out) {
                        size_t oo = ((((size_t)s * n + i) * L + l) * 2 + a) * H + h;
                        memcpy(sym_out + oo * d, csym + (size_t)p * d, sizeof(int32_t) * d);
                    }
                }
            }
        }
        free(ebar); free(n2b);
    }
    free(idx); free(w); free(lse); free(csym); free(cq); free(mus); free(pdelta);
    return rc;
}
