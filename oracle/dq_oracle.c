/*
 * dq_oracle.c -- TEST INFRASTRUCTURE, NOT THE PRODUCT.
 *
 * A plain, slow, single-pass-per-definition CPU statement of what one round of
 * double quantization computes (AsyLPG = Algorithm 1, Sparse-AsyLPG =
 * Algorithm 2, Acc-AsyLPG = Algorithm 3 of "Double Quantization for
 * Communication-Efficient Distributed Optimization").  It exists so that the
 * CUDA library can be compared against something that can be checked against
 * the paper by eye.  It shares no code with the CUDA path, is never tuned, and
 * only tests, the smoke check and the benchmark's CPU-baseline leg may call it.
 *
 * Conventions
 *   - every fp32 expression is one IEEE-754 round-to-nearest operation
 *     (compile with -ffp-contract=off); fmaf() is written where a fused
 *     multiply-add is meant;
 *   - gradients and objectives are accumulated in double and rounded once;
 *   - all random draws come from Philox4x32-10 with the counter layout below,
 *     so a (seed, round, worker, coordinate) tuple names one draw.
 *
 * Where the paper leaves a detail open the choice is stated at the function.
 *
 * Parity pins (tests/test_oracle_*.py): Philox known answers + an independent
 * big-integer restatement; Q: code range, grid points, Monte-Carlo mean and the
 * variance of Lemma 5 (appendix, first lemma); pack: brute-force bit packer;
 * gradients: finite differences; sparsifier: E[beta]=alpha and the second
 * moment in the proof of the sparsification lemma; prox: brute-force 1-D
 * minimisation of its definition; rounds: textbook ProxSVRG special case
 * (Theorem 1's setting), Algorithm 3's momentum identities, closed-form bits.
 * End-to-end convergence figures of Section 5 need the paper's datasets:
 * parity unpinned for those.
 */
#include <float.h>
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

enum { DQO_OK = 0, DQO_ERR_ARG = 1, DQO_ERR_NONFINITE = 4 };
enum { DQO_DENSE_F32 = 0, DQO_CSR_F32 = 1, DQO_DENSE_BF16 = 2 };
enum { DQO_MSG_DENSE = 0, DQO_MSG_SPARSE = 1 };
enum { DQO_STREAM_MODEL = 0, DQO_STREAM_GRAD = 1, DQO_STREAM_MASK = 2, DQO_STREAM_BATCH = 3 };
#define DQO_MASTER 0xFFFFFFFFu

/* ------------------------------------------------------------------------ */
/* Random numbers.  The paper only says "with probability" (Section 3.1,    */
/* rule (i); eq. (4)); the generator is this build's choice: Philox4x32-10  */
/* as published by Salmon, Moraes, Dror and Shaw (SC'11).                   */
/* ------------------------------------------------------------------------ */
void dqo_philox4x32_10(const uint32_t ctr[4], const uint32_t key[2], uint32_t out[4])
{
    uint32_t c0 = ctr[0], c1 = ctr[1], c2 = ctr[2], c3 = ctr[3];
    uint32_t k0 = key[0], k1 = key[1];
    for (int r = 0; r < 10; ++r) {
        if (r > 0) { k0 += 0x9E3779B9u; k1 += 0xBB67AE85u; }
        uint64_t p0 = (uint64_t)0xD2511F53u * (uint64_t)c0;
        uint64_t p1 = (uint64_t)0xCD9E8D57u * (uint64_t)c2;
        uint32_t n0 = (uint32_t)(p1 >> 32) ^ c1 ^ k0;
        uint32_t n1 = (uint32_t)p1;
        uint32_t n2 = (uint32_t)(p0 >> 32) ^ c3 ^ k1;
        uint32_t n3 = (uint32_t)p0;
        c0 = n0; c1 = n1; c2 = n2; c3 = n3;
    }
    out[0] = c0; out[1] = c1; out[2] = c2; out[3] = c3;
}

/* One Philox call serves eight consecutive coordinates: counter =
 * (i >> 3, round, worker, stream), key = seed.  Coordinate i owns half
 * (i & 1) of word ((i & 7) >> 1). */
static uint32_t word_of(uint64_t seed, uint32_t round, uint32_t worker, uint32_t stream, uint64_t i)
{
    uint32_t ctr[4] = { (uint32_t)(i >> 3), round, worker, stream };
    uint32_t key[2] = { (uint32_t)seed, (uint32_t)(seed >> 32) };
    uint32_t out[4];
    dqo_philox4x32_10(ctr, key, out);
    return out[(i & 7) >> 1];
}

/* 16 uniform bits for coordinate i: bits [0,16) of the word for even i,
 * bits [16,32) for odd i. */
uint32_t dqo_u16(uint64_t seed, uint32_t round, uint32_t worker, uint32_t stream, uint64_t i)
{
    uint32_t w = word_of(seed, round, worker, stream, i);
    return (i & 1) ? (w >> 16) : (w & 0xFFFFu);
}

/* 15 uniform bits for coordinate i: the top 15 of its 16-bit draw. */
uint32_t dqo_u15(uint64_t seed, uint32_t round, uint32_t worker, uint32_t stream, uint64_t i)
{
    return dqo_u16(seed, round, worker, stream, i) >> 1;
}

/* ------------------------------------------------------------------------ */
/* Q_(delta,b): Section 3.1.                                                */
/* ------------------------------------------------------------------------ */
static int levels(int b) { return (1 << (b - 1)) - 1; }          /* 2^(b-1) - 1 */

/* delta = ||v||_inf / (2^(b-1) - 1)  (Algorithm 1 steps 8 and 12). */
float dqo_scale_delta(float nrm, int b) { return nrm / (float)levels(b); }

/* The multiplier that maps v onto the code axis: the largest fp32 number c
 * with c * nrm <= 2^(b-1)-1 in exact arithmetic (1/delta rounded toward zero),
 * so that |v_i| <= nrm implies |v_i * c| <= 2^(b-1)-1 and every coordinate
 * lies in the convex hull of dom(delta,b) as Lemma 5's proof requires. */
float dqo_scale_inv(float nrm, int b)
{
    const double L = (double)levels(b);
    float c = (float)(L / (double)nrm);
    if (isinf(c)) c = FLT_MAX;
    while ((double)c * (double)nrm > L) c = nextafterf(c, 0.0f);       /* product exact in double */
    for (;;) {
        float up = nextafterf(c, INFINITY);
        if (isinf(up) || (double)up * (double)nrm > L) break;
        c = up;
    }
    return c;
}

/* One coordinate.  t = v*inv is the position on the code axis; z = floor(t)
 * and z+1 are the neighbouring grid points and rule (i) rounds up with
 * probability t - z.  The position is held in fixed point: with e = 8 for
 * b <= 8 and e = b for the wider codes (b = 9, 10, 11, the widths of Table 1
 * beyond a byte), r = fl(v*inv + 1.5 * 2^e) lies in [2^e, 2^(e+1)) where the
 * fp32 spacing is 2^-(23-e), so the integer F = bits(r) - bits(2^e) equals
 * (t + 2^(e-1)) * 2^(23-e) with t rounded to nearest at 2^-(23-e) (one fused
 * rounding): 15 fractional bits up to 8-bit codes, then 14, 13, 12.  Adding a
 * uniform integer of as many bits (the top bits of the coordinate's draw) and
 * dropping the fraction rounds up with probability frac(F)/2^(23-e).  Rule (ii)
 * (outside the hull: nearest end point of dom(delta,b)) is the clamp.
 * This fixed-point form IS the reading taken of rule (i)'s "with probability
 * (x - z)/delta" (the paper gives no resolution for the draw); it cannot be
 * checked against the rule by eye, so tests/test_oracle_philox_quantizer.py
 * (test_q_code_is_stochastic_rounding_with_exact_probability) counts, over all
 * 2^15 draws, how often a coordinate is rounded up and compares the count with
 * frac(t) 2^15 computed from exact rationals. */
int32_t dqo_q_code(float v, float inv, int b, uint32_t u15)
{
    const int e = b <= 8 ? 8 : b, fbits = 23 - e;
    const float off = 1.5f * (float)(1 << e);
    float r = fmaf(v, inv, off);
    float lo = off - (float)(1 << (b - 1));                      /* -2^(b-1): smallest member of dom */
    float hi = off + (float)levels(b);                           /* 2^(b-1)-1: largest member        */
    r = fminf(fmaxf(r, lo), hi);
    uint32_t bits; memcpy(&bits, &r, 4);
    uint32_t F = bits - ((uint32_t)(127 + e) << 23);             /* bits(2^e) */
    return (int32_t)((F + (u15 >> (15 - fbits))) >> fbits) - (1 << (e - 1));
}

float dqo_norm_inf(const float* v, int64_t d)
{
    float m = 0.0f;
    for (int64_t i = 0; i < d; ++i) { float a = fabsf(v[i]); if (a > m) m = a; }
    return m;
}

static int all_finite(const float* v, int64_t d)
{
    for (int64_t i = 0; i < d; ++i) if (!isfinite(v[i])) return 0;
    return 1;
}

/* Q_(delta,b)(v) for a whole vector with delta from its infinity norm.
 * ||v||_inf = 0 gives delta = 0 and all-zero codes (the paper divides by
 * zero there; reading).  Non-finite input is an error. */
int dqo_quantize(const float* v, int64_t d, int b, uint64_t seed, uint32_t round, uint32_t worker,
                 uint32_t stream, int32_t* codes, float* delta)
{
    if (b < 2 || b > 11 || d < 0) return DQO_ERR_ARG;
    if (!all_finite(v, d)) return DQO_ERR_NONFINITE;
    float nrm = dqo_norm_inf(v, d);
    if (nrm == 0.0f) { *delta = 0.0f; for (int64_t i = 0; i < d; ++i) codes[i] = 0; return DQO_OK; }
    *delta = dqo_scale_delta(nrm, b);
    float inv = dqo_scale_inv(nrm, b);
    for (int64_t i = 0; i < d; ++i)
        codes[i] = dqo_q_code(v[i], inv, b, dqo_u15(seed, round, worker, stream, (uint64_t)i));
    return DQO_OK;
}

/* ------------------------------------------------------------------------ */
/* Message encoding: Section 3.1 counts b bits per coordinate; the container */
/* is this build's choice: the codes as b-bit two's complement fields laid    */
/* end to end, coordinate j in bits [j b, (j+1) b) of the message, bit k of   */
/* the message being bit k mod 8 of byte k / 8; unused bits zero.  (For b     */
/* dividing 8: coordinate j in byte j/(8/b) at bit offset (j mod (8/b)) b.)   */
/* ------------------------------------------------------------------------ */
void dqo_pack(const int32_t* codes, int64_t count, int b, uint8_t* out, int64_t out_bytes)
{
    memset(out, 0, (size_t)out_bytes);
    uint32_t mask = (1u << b) - 1u;
    for (int64_t j = 0; j < count; ++j) {
        uint32_t field = (uint32_t)codes[j] & mask;
        for (int k = 0; k < b; ++k) {
            int64_t bit = j * b + k;
            if ((field >> k) & 1u) out[bit >> 3] |= (uint8_t)(1u << (bit & 7));
        }
    }
}

void dqo_unpack(const uint8_t* in, int64_t count, int b, int32_t* codes)
{
    for (int64_t j = 0; j < count; ++j) {
        uint32_t u = 0;
        for (int k = 0; k < b; ++k) {
            int64_t bit = j * b + k;
            u |= (uint32_t)((in[bit >> 3] >> (bit & 7)) & 1u) << k;
        }
        codes[j] = (u & (1u << (b - 1))) ? (int32_t)u - (1 << b) : (int32_t)u;   /* sign extend */
    }
}

/* ------------------------------------------------------------------------ */
/* Sparsification: eq. (4) and Lemma 2.                                      */
/* ------------------------------------------------------------------------ */

/* ||alpha||_1 on an integer grid so that the value does not depend on the
 * order of summation (the mask must be reproducible bit for bit): with
 * ||alpha||_inf in [2^(e-1), 2^e), every |alpha_i| * 2^(35-e) is truncated to
 * an integer below 2^35 and the integers are added exactly. */
float dqo_norm_l1(const float* v, int64_t d, float ninf)
{
    if (ninf == 0.0f) return 0.0f;
    int e; (void)frexpf(ninf, &e);
    uint64_t sum = 0;
    for (int64_t i = 0; i < d; ++i)
        sum += (uint64_t)ldexp((double)fabsf(v[i]), 35 - e);      /* exact scaling, then truncation */
    return (float)ldexp((double)sum, e - 35);
}

/* beta = [Z_i alpha_i / p_i], Z_i ~ Bernoulli(p_i), eq. (4), with Lemma 2's
 * p_i = |alpha_i| phi / ||alpha||_1.  The budget must satisfy
 * phi <= ||alpha||_1/||alpha||_inf (Lemma 2), so a larger request is clamped;
 * phi <= 0 asks for equality as in Section 5.1.  Each probability is rounded
 * UP to a multiple of 2^-16 (the resolution of the uniform draw) and the
 * survivor is divided by that rounded probability, so E[beta] = alpha holds
 * exactly (eq. (4) allows any 0 < p_i <= 1). */
int dqo_sparsify(const float* alpha, int64_t d, float phi, uint64_t seed, uint32_t round, uint32_t worker,
                 float* beta, uint8_t* Z, uint32_t* m_out /* p_i * 2^16, may be NULL */,
                 float* ninf_out, float* n1_out, float* phi_eff_out)
{
    if (!all_finite(alpha, d)) return DQO_ERR_NONFINITE;
    float ninf = dqo_norm_inf(alpha, d);
    float n1 = dqo_norm_l1(alpha, d, ninf);
    if (ninf_out) *ninf_out = ninf;
    if (n1_out) *n1_out = n1;
    if (ninf == 0.0f || n1 == 0.0f) {
        if (phi_eff_out) *phi_eff_out = 0.0f;
        for (int64_t i = 0; i < d; ++i) { beta[i] = 0.0f; Z[i] = 0; if (m_out) m_out[i] = 0; }
        return DQO_OK;
    }
    float cap = n1 / ninf;
    float phi_eff = (phi > 0.0f) ? fminf(phi, cap) : cap;
    float s = phi_eff / n1;
    if (phi_eff_out) *phi_eff_out = phi_eff;
    for (int64_t i = 0; i < d; ++i) {
        /* p_i * 2^16 rounded up, as an integer in 0..2^16.  A zero coordinate has p_i = 0 whatever s is and
         * never survives; this is said first because with ||alpha||_1 subnormal s = phi/||alpha||_1 overflows
         * to +inf and 0 * inf would be a NaN (no NaN may reach the integer conversion).  A nonzero coordinate
         * under an overflowed s has p_i = inf, clamped to 1 like every p_i >= 1. */
        float a = fabsf(alpha[i]);
        uint32_t m = 0;
        if (a != 0.0f) {
            float scaled = ceilf((a * s) * 65536.0f);             /* exact power-of-two scaling */
            m = (scaled >= 65536.0f) ? 65536u : (uint32_t)scaled;
        }
        uint32_t u = dqo_u16(seed, round, worker, DQO_STREAM_MASK, (uint64_t)i);
        int z = (u < m);
        Z[i] = (uint8_t)z;
        beta[i] = z ? (alpha[i] * 65536.0f) / (float)m : 0.0f;   /* alpha_i / (m / 2^16) */
        if (m_out) m_out[i] = m;
    }
    return DQO_OK;
}

/* Step 13 of Algorithm 2: quantise beta with delta from its infinity norm.
 * Only survivors (Z_i = 1) carry a code; their rounding draw is keyed by the
 * coordinate index i, not by the position in the sparse list. */
int dqo_quantize_survivors(const float* beta, const uint8_t* Z, int64_t d, int b, uint64_t seed,
                           uint32_t round, uint32_t worker, int32_t* codes, float* delta)
{
    float nrm = 0.0f;
    for (int64_t i = 0; i < d; ++i) if (Z[i]) { float a = fabsf(beta[i]); if (a > nrm) nrm = a; }
    if (!isfinite(nrm)) return DQO_ERR_NONFINITE;
    for (int64_t i = 0; i < d; ++i) codes[i] = 0;
    if (nrm == 0.0f) { *delta = 0.0f; return DQO_OK; }
    *delta = dqo_scale_delta(nrm, b);
    float inv = dqo_scale_inv(nrm, b);
    for (int64_t i = 0; i < d; ++i)
        if (Z[i]) codes[i] = dqo_q_code(beta[i], inv, b, dqo_u15(seed, round, worker, DQO_STREAM_GRAD, (uint64_t)i));
    return DQO_OK;
}

/* ------------------------------------------------------------------------ */
/* The smooth part f = 1/n sum f_i, eq. (1).  Section 5.1 says "logistic     */
/* regression" without the formula; reading: labels y in {-1,+1},            */
/* f_a(x) = log(1 + exp(-y_a <a_a, x>)).  Regularisers live in h.            */
/* ------------------------------------------------------------------------ */
typedef struct {
    int32_t format; int32_t pad_;
    int64_t n, d;
    const void* values;        /* dense: [n][d] float or bf16 bits; CSR: [nnz] float */
    const int32_t* col_idx;    /* CSR only */
    const int64_t* row_ptr;    /* CSR only, [n+1] */
    const float* labels;       /* [n], +-1 */
} dqo_data;

static double bf16_to_double(uint16_t h) { uint32_t u = (uint32_t)h << 16; float f; memcpy(&f, &u, 4); return (double)f; }

/* <a_row, x> in double. */
double dqo_margin(const dqo_data* D, int64_t row, const float* x)
{
    double s = 0.0;
    if (D->format == DQO_CSR_F32) {
        const float* val = (const float*)D->values;
        for (int64_t k = D->row_ptr[row]; k < D->row_ptr[row + 1]; ++k) s += (double)val[k] * (double)x[D->col_idx[k]];
    } else if (D->format == DQO_DENSE_F32) {
        const float* a = (const float*)D->values + row * D->d;
        for (int64_t i = 0; i < D->d; ++i) s += (double)a[i] * (double)x[i];
    } else {
        const uint16_t* a = (const uint16_t*)D->values + row * D->d;
        for (int64_t i = 0; i < D->d; ++i) s += bf16_to_double(a[i]) * (double)x[i];
    }
    return s;
}

/* out += w * a_row ; optionally mag += |w| * |a_row|. */
static void add_row(const dqo_data* D, int64_t row, double w, double* out, double* mag)
{
    if (D->format == DQO_CSR_F32) {
        const float* val = (const float*)D->values;
        for (int64_t k = D->row_ptr[row]; k < D->row_ptr[row + 1]; ++k) {
            out[D->col_idx[k]] += w * (double)val[k];
            if (mag) mag[D->col_idx[k]] += fabs(w) * fabs((double)val[k]);
        }
    } else if (D->format == DQO_DENSE_F32) {
        const float* a = (const float*)D->values + row * D->d;
        for (int64_t i = 0; i < D->d; ++i) { out[i] += w * (double)a[i]; if (mag) mag[i] += fabs(w) * fabs((double)a[i]); }
    } else {
        const uint16_t* a = (const uint16_t*)D->values + row * D->d;
        for (int64_t i = 0; i < D->d; ++i) { double v = bf16_to_double(a[i]); out[i] += w * v; if (mag) mag[i] += fabs(w) * fabs(v); }
    }
}

/* d/dz log(1+exp(-y z)) = -y / (1 + exp(y z)): the scalar factor of grad f_a. */
static double loss_slope(double y, double z) { return -y / (1.0 + exp(y * z)); }

/* Worker step 11: alpha = (1/B) sum_{a in batch} [grad f_a(xhat) - grad f_a(xsnap)].
 * The algorithm boxes show one sample; Section 5 uses minibatches (B = 200, 20).
 * S_i = (1/B) sum |slope difference| |a_{a,i}| is returned for tolerances. */
void dqo_worker_grad(const dqo_data* D, const float* xhat, const float* xsnap, const int64_t* rows, int B,
                     float* alpha, float* S)
{
    int64_t d = D->d;
    double* acc = (double*)calloc((size_t)d, sizeof(double));
    double* mag = (double*)calloc((size_t)d, sizeof(double));
    for (int j = 0; j < B; ++j) {
        int64_t a = rows[j];
        double y = (double)D->labels[a];
        double diff = loss_slope(y, dqo_margin(D, a, xhat)) - loss_slope(y, dqo_margin(D, a, xsnap));
        add_row(D, a, diff, acc, mag);
    }
    for (int64_t i = 0; i < d; ++i) { alpha[i] = (float)(acc[i] / (double)B); if (S) S[i] = (float)(mag[i] / (double)B); }
    free(acc); free(mag);
}

/* grad f(x) = (1/n) sum_i grad f_i(x), the epoch's full gradient (Algorithm 1
 * step 5); also returns the margins z_i = <a_i, x> when z != NULL. */
void dqo_full_grad(const dqo_data* D, const float* x, float* g, float* z)
{
    double* acc = (double*)calloc((size_t)D->d, sizeof(double));
    for (int64_t a = 0; a < D->n; ++a) {
        double m = dqo_margin(D, a, x);
        if (z) z[a] = (float)m;
        add_row(D, a, loss_slope((double)D->labels[a], m), acc, NULL);
    }
    for (int64_t i = 0; i < D->d; ++i) g[i] = (float)(acc[i] / (double)D->n);
    free(acc);
}

/* f(x) alone (no h), for finite-difference checks. */
double dqo_smooth_loss(const dqo_data* D, const float* x)
{
    double s = 0.0;
    for (int64_t a = 0; a < D->n; ++a) {
        double m = -(double)D->labels[a] * dqo_margin(D, a, x);    /* log(1+exp(m)) */
        s += (m > 0.0) ? m + log1p(exp(-m)) : log1p(exp(m));
    }
    return s / (double)D->n;
}

/* P(x) = f(x) + h(x), eq. (1), with h = l1 ||x||_1 + (l2/2) ||x||^2 (x assumed inside Omega). */
double dqo_objective(const dqo_data* D, const float* x, float l1, float l2)
{
    double a = 0.0, q = 0.0;
    for (int64_t i = 0; i < D->d; ++i) { a += fabs((double)x[i]); q += (double)x[i] * (double)x[i]; }
    return dqo_smooth_loss(D, x) + (double)l1 * a + 0.5 * (double)l2 * q;
}

/* ------------------------------------------------------------------------ */
/* Second smooth part (Section 5.2): a 3-layer fully connected network,      */
/* input -> hidden (ReLU) -> classes, softmax cross-entropy.  The parameter   */
/* vector is x = [W1 (hidden x in, row-major), b1 (hidden), W2 (classes x     */
/* hidden), b2 (classes)]; labels hold the class index.  The L2 regulariser   */
/* of Section 5.2 lives in h like the others.                                 */
/* ------------------------------------------------------------------------ */
int64_t dqo_mlp_params(int64_t in, int hidden, int classes) { return (int64_t)hidden * (in + 1) + (int64_t)classes * (hidden + 1); }

/* Loss of one sample; if grad != NULL adds w * d loss / d x to grad and, if mag != NULL, the absolute values of the
 * same terms to mag (for tolerances). */
static double mlp_sample(const float* a, int label, int64_t in, int hidden, int classes, const float* x,
                         double w, double* grad, double* mag)
{
    const float* W1 = x; const float* b1 = W1 + (int64_t)hidden * in;
    const float* W2 = b1 + hidden; const float* b2 = W2 + (int64_t)classes * hidden;
    double* h = (double*)malloc(sizeof(double) * (size_t)(2 * hidden + 2 * classes));
    double* z = h + hidden; double* p = z + classes; double* habs = p + classes;
    for (int j = 0; j < hidden; ++j) {
        double s = (double)b1[j], sa = fabs((double)b1[j]);
        for (int64_t i = 0; i < in; ++i) { double t = (double)W1[(int64_t)j * in + i] * (double)a[i]; s += t; sa += fabs(t); }
        h[j] = s > 0.0 ? s : 0.0;
        habs[j] = sa;             /* magnitude of the terms behind h_j: a hidden unit near its kink is a cancelling sum */
    }
    double zmax = -INFINITY;
    for (int c = 0; c < classes; ++c) {
        double s = (double)b2[c];
        for (int j = 0; j < hidden; ++j) s += (double)W2[(int64_t)c * hidden + j] * h[j];
        z[c] = s; if (s > zmax) zmax = s;
    }
    double sum = 0.0;
    for (int c = 0; c < classes; ++c) { p[c] = exp(z[c] - zmax); sum += p[c]; }
    for (int c = 0; c < classes; ++c) p[c] /= sum;
    double loss = -(z[label] - zmax - log(sum));
    if (grad) {
        double* gW1 = grad; double* gb1 = gW1 + (int64_t)hidden * in; double* gW2 = gb1 + hidden; double* gb2 = gW2 + (int64_t)classes * hidden;
        double* mW1 = mag; double* mb1 = mag ? mW1 + (int64_t)hidden * in : NULL; double* mW2 = mag ? mb1 + hidden : NULL;
        double* mb2 = mag ? mW2 + (int64_t)classes * hidden : NULL;
        double* dh = (double*)calloc((size_t)hidden, sizeof(double));
        for (int c = 0; c < classes; ++c) {
            double dz = w * (p[c] - (c == label ? 1.0 : 0.0));
            gb2[c] += dz; if (mag) mb2[c] += fabs(dz);
            for (int j = 0; j < hidden; ++j) {
                gW2[(int64_t)c * hidden + j] += dz * h[j]; if (mag) mW2[(int64_t)c * hidden + j] += fabs(dz) * habs[j];
                dh[j] += dz * (double)W2[(int64_t)c * hidden + j];
            }
        }
        for (int j = 0; j < hidden; ++j) {
            if (h[j] <= 0.0) continue;                                   /* ReLU gate */
            gb1[j] += dh[j]; if (mag) mb1[j] += fabs(dh[j]);
            for (int64_t i = 0; i < in; ++i) {
                gW1[(int64_t)j * in + i] += dh[j] * (double)a[i]; if (mag) mW1[(int64_t)j * in + i] += fabs(dh[j] * (double)a[i]);
            }
        }
        free(dh);
    }
    free(h);
    return loss;
}

/* f(x) = (1/n) sum_i loss_i(x) over the rows listed (rows == NULL: all n rows). */
double dqo_mlp_loss(const dqo_data* D, int hidden, int classes, const float* x, const int64_t* rows, int64_t count)
{
    double s = 0.0;
    for (int64_t k = 0; k < count; ++k) {
        int64_t a = rows ? rows[k] : k;
        s += mlp_sample((const float*)D->values + a * D->d, (int)D->labels[a], D->d, hidden, classes, x, 0.0, NULL, NULL);
    }
    return s / (double)count;
}

/* g = (1/count) sum grad loss_i(x) over the listed rows, rounded to fp32 once. */
void dqo_mlp_grad(const dqo_data* D, int hidden, int classes, const float* x, const int64_t* rows, int64_t count, float* g)
{
    int64_t P = dqo_mlp_params(D->d, hidden, classes);
    double* acc = (double*)calloc((size_t)P, sizeof(double));
    for (int64_t k = 0; k < count; ++k) {
        int64_t a = rows ? rows[k] : k;
        mlp_sample((const float*)D->values + a * D->d, (int)D->labels[a], D->d, hidden, classes, x, 1.0 / (double)count, acc, NULL);
    }
    for (int64_t i = 0; i < P; ++i) g[i] = (float)acc[i];
    free(acc);
}

/* Worker step 11 for the network: alpha = minibatch grad at xhat minus minibatch grad at xsnap; S = sum of the
 * absolute per-sample terms of both gradients (tolerance scale). */
void dqo_mlp_worker_grad(const dqo_data* D, int hidden, int classes, const float* xhat, const float* xsnap,
                         const int64_t* rows, int B, float* alpha, float* S)
{
    int64_t P = dqo_mlp_params(D->d, hidden, classes);
    double* acc = (double*)calloc((size_t)P, sizeof(double));
    double* mag = (double*)calloc((size_t)P, sizeof(double));
    for (int k = 0; k < B; ++k) {
        const float* a = (const float*)D->values + rows[k] * D->d; int label = (int)D->labels[rows[k]];
        mlp_sample(a, label, D->d, hidden, classes, xhat, 1.0 / (double)B, acc, mag);
        mlp_sample(a, label, D->d, hidden, classes, xsnap, -1.0 / (double)B, acc, mag);
    }
    for (int64_t i = 0; i < P; ++i) { alpha[i] = (float)acc[i]; if (S) S[i] = (float)mag[i]; }
    free(acc); free(mag);
}

/* P(x) = f(x) + h(x) for the network. */
double dqo_mlp_objective(const dqo_data* D, int hidden, int classes, const float* x, float l1, float l2)
{
    int64_t P = dqo_mlp_params(D->d, hidden, classes);
    double a = 0.0, q = 0.0;
    for (int64_t i = 0; i < P; ++i) { a += fabs((double)x[i]); q += (double)x[i] * (double)x[i]; }
    return dqo_mlp_loss(D, hidden, classes, x, NULL, D->n) + (double)l1 * a + 0.5 * (double)l2 * q;
}

/* Worker w keeps the contiguous partition [floor(w n/M), floor((w+1) n/M))
 * (Section 3.2: "keeps a disjoint partition") and draws its minibatch from it
 * with replacement: slot j takes word (j & 3) of Philox counter
 * (j >> 2, round, w, batch stream) and maps it to lo + floor(word * n_w / 2^32). */
void dqo_sample_batch(uint64_t seed, uint32_t round, int w, int M, int64_t n, int B, int64_t* rows)
{
    int64_t lo = (int64_t)(((__int128)w * n) / M), hi = (int64_t)(((__int128)(w + 1) * n) / M);
    uint64_t nw = (uint64_t)(hi - lo);
    uint32_t key[2] = { (uint32_t)seed, (uint32_t)(seed >> 32) };
    for (int j = 0; j < B; ++j) {
        uint32_t ctr[4] = { (uint32_t)(j >> 2), round, (uint32_t)w, DQO_STREAM_BATCH }, out[4];
        dqo_philox4x32_10(ctr, key, out);
        rows[j] = lo + (int64_t)(((uint64_t)out[j & 3] * nw) >> 32);
    }
}

/* ------------------------------------------------------------------------ */
/* Master: prox step (notation paragraph: prox_{eta h}(x) = argmin_y h(y) +   */
/* ||y-x||^2/(2 eta)) for h = l1|.|_1 + (l2/2)|.|^2 + indicator of the box    */
/* Omega = [lo,hi]^d.  Separable and convex, so per coordinate the minimiser  */
/* is the unconstrained one, soft(v, eta l1)/(1 + eta l2), projected on the   */
/* interval.                                                                  */
/* ------------------------------------------------------------------------ */
float dqo_prox(float v, float eta, float l1, float l2, float lo, float hi)
{
    float a = fabsf(v) - eta * l1;
    float r = (a > 0.0f) ? copysignf(a, v) : 0.0f;
    r = r / (1.0f + eta * l2);
    return fminf(fmaxf(r, lo), hi);
}

/* Master step 9 for a synchronous round of M workers (reading: the M lanes of
 * one round see the same broadcast model and the master averages their
 * dequantised messages, then takes ONE prox step):
 *   g = (1/M) sum_w k_w delta_w,  u = g + grad f(xsnap),
 *   Alg. 1/2: x <- prox(x - eta u);
 *   Alg. 3:   y <- prox(y - eta u), x <- xsnap + theta (y - xsnap), xsum += x.
 * Returns ||x||_inf of the new model through normx. */
void dqo_master_step(const int32_t* codes /*[M][d]*/, const float* delta /*[M]*/, int M, int64_t d,
                     const float* gfull, float* x, float* y, const float* xsnap, float* xsum,
                     float eta, float theta, int accelerated,
                     float l1, float l2, float lo, float hi, float* normx)
{
    float invM = 1.0f / (float)M, nx = 0.0f;
    for (int64_t i = 0; i < d; ++i) {
        float acc = 0.0f;
        for (int w = 0; w < M; ++w) acc = fmaf((float)codes[(int64_t)w * d + i], delta[w], acc);
        float u = acc * invM + gfull[i];
        if (!accelerated) {
            x[i] = dqo_prox(fmaf(-eta, u, x[i]), eta, l1, l2, lo, hi);
        } else {
            y[i] = dqo_prox(fmaf(-eta, u, y[i]), eta, l1, l2, lo, hi);
            x[i] = fmaf(theta, y[i] - xsnap[i], xsnap[i]);
            xsum[i] = xsum[i] + x[i];
        }
        float a = fabsf(x[i]); if (a > nx) nx = a;
    }
    if (normx) *normx = nx;
}

/* Master step 9 as Algorithm 1 states it, one message per master tick: the M
 * workers of a round all pulled the model broadcast at the round's start, and
 * the master applies their messages one after the other in worker order, each
 * with its own semi-stochastic gradient u = Q(alpha_w) + grad f(xsnap) and its
 * own prox step.  Message w therefore meets a model that is w ticks newer than
 * the one it was computed on: the delay t - D(t) = w <= tau = M - 1 of
 * Assumption 3.  Algorithm 3 updates y, x and the running sum at every tick. */
void dqo_master_step_sequential(const int32_t* codes, const float* delta, int M, int64_t d,
                                const float* gfull, float* x, float* y, const float* xsnap, float* xsum,
                                float eta, float theta, int accelerated,
                                float l1, float l2, float lo, float hi, float* normx)
{
    float nx = 0.0f;
    for (int64_t i = 0; i < d; ++i) {
        for (int w = 0; w < M; ++w) {
            float u = (float)codes[(int64_t)w * d + i] * delta[w] + gfull[i];
            if (!accelerated) {
                x[i] = dqo_prox(fmaf(-eta, u, x[i]), eta, l1, l2, lo, hi);
            } else {
                y[i] = dqo_prox(fmaf(-eta, u, y[i]), eta, l1, l2, lo, hi);
                x[i] = fmaf(theta, y[i] - xsnap[i], xsnap[i]);
                xsum[i] = xsum[i] + x[i];
            }
        }
        float a = fabsf(x[i]); if (a > nx) nx = a;
    }
    if (normx) *normx = nx;
}

/* ------------------------------------------------------------------------ */
/* Model precision: the master quantises x "subject to" condition (3),        */
/*   E_Q ||Q(x) - x||^2 <= mu ||x - xsnap||^2                                 */
/* (condition (6) of Algorithm 3 has theta_s mu), and Section 5.2 searches    */
/* b_x so that it holds.  Under rule (i) a coordinate between the grid points */
/* z and z + delta has expected squared error (x - z)(z + delta - x)          */
/* (proof of the appendix's first lemma), so the left side is a closed form.  */
/* The search is over the widths 2..11 of Table 1.                            */
/* ------------------------------------------------------------------------ */
double dqo_expected_sq_error(const float* x, int64_t d, int b)
{
    float nrm = dqo_norm_inf(x, d);
    if (nrm == 0.0f) return 0.0;
    double delta = (double)dqo_scale_delta(nrm, b), e = 0.0;
    for (int64_t i = 0; i < d; ++i) {
        double t = (double)x[i] / delta, frac = t - floor(t);
        e += frac * (1.0 - frac);                                  /* (x - z)(z + delta - x) / delta^2 */
    }
    return e * delta * delta;
}

double dqo_sq_distance(const float* x, const float* y, int64_t d)
{
    double s = 0.0;
    for (int64_t i = 0; i < d; ++i) { double t = (double)x[i] - (double)y[i]; s += t * t; }
    return s;
}

/* Smallest width in 2..11 (the widths of Table 1) that satisfies the condition; 11 when none does.
 * err[0..9] receive the expected errors at 2..11 bits, *dist2 the squared distance. */
int dqo_select_bx(const float* x, const float* xsnap, int64_t d, float mu, double* err, double* dist2)
{
    double D = dqo_sq_distance(x, xsnap, d);
    int chosen = 11;
    for (int b = 11; b >= 2; --b) {
        double e = dqo_expected_sq_error(x, d, b);
        if (err) err[b - 2] = e;
        if (e <= (double)mu * D) chosen = b;
    }
    if (dist2) *dist2 = D;
    return chosen;
}

/* ------------------------------------------------------------------------ */
/* Round and epoch drivers.                                                  */
/* ------------------------------------------------------------------------ */
typedef struct {
    int64_t d; int32_t M, B, bx, b;
    float l1, l2, box_lo, box_hi;
    int32_t sparsify; float phi;
    int32_t msg_format, accelerated, snapshot_flag, pad_;
    uint64_t seed;
    float mu;                       /* mu > 0: choose b_x per round by condition (3)/(6); 0: fixed b_x */
    int32_t sequential;             /* 1: one prox step per message (dqo_master_step_sequential) */
    int32_t model, hidden, classes, pad3_;   /* model 0: logistic regression; 1: the 3-layer network */
} dqo_config;

typedef struct { float *x, *xsnap, *gfull, *y, *xsum; } dqo_state;

/* Optional capture of every intermediate of a round (any pointer may be NULL). */
typedef struct {
    int32_t* codes_x;  /* [d]    */  float* delta_x;  float* xhat;   /* [d] */
    int64_t* rows;     /* [M][B] */
    float* alpha;      /* [M][d] */  float* S;        /* [M][d] */
    float* beta;       /* [M][d] */  uint8_t* Z;      /* [M][d] */
    int32_t* codes;    /* [M][d] */  float* delta;    /* [M] */
    float* ninf;       /* [M] */     float* n1;       /* [M] */   float* phi_eff; /* [M] */
    int64_t* nnz;      /* [M] */
    uint64_t bits_down, bits_up;
    float normx; int32_t flag_round;
    int32_t bx_used; int32_t pad_;
} dqo_trace;

static int ceil_log2(int64_t d) { int k = 0; while (((int64_t)1 << k) < d) ++k; return k; }

/* Epoch boundary.  Alg. 1/2 (steps 3, 5, 14): xsnap <- x, then the full
 * gradient at xsnap.  Alg. 3 (steps 3, 5, 15): xsnap <- xsum / m_prev if an
 * epoch has run, xsum <- 0, y carried over (y_0 = y_m of the previous epoch is
 * assigned before it is used), x <- xsnap + theta (y - xsnap), then the full
 * gradient at xsnap.  z_snap (may be NULL) receives the margins at xsnap. */
void dqo_epoch_begin(const dqo_config* C, const dqo_data* D, dqo_state* S, float theta, int64_t m_prev, float* z_snap)
{
    int64_t d = C->d;
    if (!C->accelerated) {
        memcpy(S->xsnap, S->x, (size_t)d * 4);
    } else {
        if (m_prev > 0) for (int64_t i = 0; i < d; ++i) S->xsnap[i] = S->xsum[i] / (float)m_prev;
        for (int64_t i = 0; i < d; ++i) { S->xsum[i] = 0.0f; S->x[i] = fmaf(theta, S->y[i] - S->xsnap[i], S->xsnap[i]); }
    }
    if (C->model == 1) dqo_mlp_grad(D, C->hidden, C->classes, S->xsnap, NULL, D->n, S->gfull);
    else dqo_full_grad(D, S->xsnap, S->gfull, z_snap);
}

/* One inner iteration (Algorithm 1 steps 6-13, with Algorithm 2's step 12-13
 * or Algorithm 3's step 9) for M workers.  flag_round: the model equals the
 * snapshot, the master sends one flag bit and workers use xsnap (end of the
 * "Model Parameter Quantization" paragraph).
 * Delays (Algorithm 1 step 11 evaluates the gradient at x_{D(t)}, Assumption 3
 * bounds t - D(t) by tau): when stale is given, worker w computes its gradient
 * at the low-precision model stale[w] (one broadcast in an earlier round of
 * the same epoch, kept by the caller) instead of this round's; stale[w] = NULL
 * means this round's.  Everything else is unchanged. */
int dqo_round_delayed(const dqo_config* C, const dqo_data* D, dqo_state* S, uint32_t round, int flag_round,
                      float eta, float theta, dqo_trace* T, const float* const* stale);

int dqo_round(const dqo_config* C, const dqo_data* D, dqo_state* S, uint32_t round, int flag_round,
              float eta, float theta, dqo_trace* T)
{
    return dqo_round_delayed(C, D, S, round, flag_round, eta, theta, T, NULL);
}

int dqo_round_delayed(const dqo_config* C, const dqo_data* D, dqo_state* S, uint32_t round, int flag_round,
                      float eta, float theta, dqo_trace* T, const float* const* stale)
{
    const int64_t d = C->d; const int M = C->M, B = C->B;
    int rc = DQO_OK;
    int32_t* codes_x = (int32_t*)malloc((size_t)d * 4);
    float* xhat = (float*)malloc((size_t)d * 4);
    int32_t* codes = (int32_t*)malloc((size_t)M * d * 4);
    float* delta = (float*)malloc((size_t)M * 4);
    float* alpha = (float*)malloc((size_t)d * 4);
    float* Sabs = (float*)malloc((size_t)d * 4);
    float* beta = (float*)malloc((size_t)d * 4);
    uint8_t* Z = (uint8_t*)malloc((size_t)d);
    int64_t* rows = (int64_t*)malloc((size_t)B * 8);
    uint64_t bits_down, bits_up = 0;
    float delta_x = 0.0f;
    int bx = C->bx;

    /* master (i): model quantisation, step 8 */
    if (flag_round) {
        memcpy(xhat, S->xsnap, (size_t)d * 4);
        for (int64_t i = 0; i < d; ++i) codes_x[i] = 0;
        bits_down = (uint64_t)M;
    } else {
        if (C->mu > 0.0f)      /* condition (3); Algorithm 3 uses theta_s mu (condition (6)) */
            bx = dqo_select_bx(S->x, S->xsnap, d, C->accelerated ? theta * C->mu : C->mu, NULL, NULL);
        rc = dqo_quantize(S->x, d, bx, C->seed, round, DQO_MASTER, DQO_STREAM_MODEL, codes_x, &delta_x);
        for (int64_t i = 0; i < d; ++i) xhat[i] = (float)codes_x[i] * delta_x;
        bits_down = (uint64_t)M * (32u + (uint64_t)bx * (uint64_t)d);
    }
    if (T) {
        if (T->codes_x) memcpy(T->codes_x, codes_x, (size_t)d * 4);
        if (T->delta_x) *T->delta_x = delta_x;
        if (T->xhat) memcpy(T->xhat, xhat, (size_t)d * 4);
        T->flag_round = flag_round;
        T->bx_used = flag_round ? 0 : bx;
    }

    /* workers, steps 11-13 */
    for (int w = 0; w < M && rc == DQO_OK; ++w) {
        int32_t* cw = codes + (int64_t)w * d;
        int64_t nnz = d;
        float ninf = 0.0f, n1 = 0.0f, phi_eff = 0.0f;
        dqo_sample_batch(C->seed, round, w, M, D->n, B, rows);
        const float* xw = (stale && stale[w]) ? stale[w] : xhat;     /* the model this worker pulled */
        if (C->model == 1) dqo_mlp_worker_grad(D, C->hidden, C->classes, xw, S->xsnap, rows, B, alpha, Sabs);
        else dqo_worker_grad(D, xw, S->xsnap, rows, B, alpha, Sabs);
        if (C->sparsify) {
            rc = dqo_sparsify(alpha, d, C->phi, C->seed, round, (uint32_t)w, beta, Z, NULL, &ninf, &n1, &phi_eff);
            if (rc == DQO_OK) rc = dqo_quantize_survivors(beta, Z, d, C->b, C->seed, round, (uint32_t)w, cw, &delta[w]);
            nnz = 0; for (int64_t i = 0; i < d; ++i) nnz += Z[i];
        } else {
            rc = dqo_quantize(alpha, d, C->b, C->seed, round, (uint32_t)w, DQO_STREAM_GRAD, cw, &delta[w]);
            ninf = dqo_norm_inf(alpha, d);
        }
        /* message size: 32 + b d bits dense (Section 3.1); sparse: 32 bits plus
         * (log d + b) bits per nonzero of beta (remark after Theorem 3) */
        if (C->sparsify && C->msg_format == DQO_MSG_SPARSE)
            bits_up += 32u + (uint64_t)nnz * (uint64_t)(ceil_log2(d) + C->b);
        else
            bits_up += 32u + (uint64_t)C->b * (uint64_t)d;
        if (T) {
            if (T->rows) memcpy(T->rows + (int64_t)w * B, rows, (size_t)B * 8);
            if (T->alpha) memcpy(T->alpha + (int64_t)w * d, alpha, (size_t)d * 4);
            if (T->S) memcpy(T->S + (int64_t)w * d, Sabs, (size_t)d * 4);
            if (C->sparsify && T->beta) memcpy(T->beta + (int64_t)w * d, beta, (size_t)d * 4);
            if (C->sparsify && T->Z) memcpy(T->Z + (int64_t)w * d, Z, (size_t)d);
            if (T->ninf) T->ninf[w] = ninf;
            if (T->n1) T->n1[w] = n1;
            if (T->phi_eff) T->phi_eff[w] = phi_eff;
            if (T->nnz) T->nnz[w] = nnz;
        }
    }

    /* master (ii), step 9 */
    float normx = 0.0f;
    if (rc == DQO_OK)
        (C->sequential ? dqo_master_step_sequential : dqo_master_step)(
            codes, delta, M, d, S->gfull, S->x, S->y, S->xsnap, S->xsum, eta, theta, C->accelerated,
            C->l1, C->l2, C->box_lo, C->box_hi, &normx);
    if (T) {
        if (T->codes) memcpy(T->codes, codes, (size_t)M * d * 4);
        if (T->delta) memcpy(T->delta, delta, (size_t)M * 4);
        T->bits_down = bits_down; T->bits_up = bits_up; T->normx = normx;
    }
    free(codes_x); free(xhat); free(codes); free(delta); free(alpha); free(Sabs); free(beta); free(Z); free(rows);
    return rc;
}
