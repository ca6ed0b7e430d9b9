/*
 * QLESS oracle: a plain, slow, single-threaded CPU statement of what the QLESS
 * hot path computes (gradient -> projected -> normalised -> quantised datastore
 * -> influence scores -> top-k).
 *
 * THIS IS TEST INFRASTRUCTURE. It exists so that the CUDA library can be
 * checked against something written straight from the paper's equations. It
 * shares no code with the CUDA path, is never tuned, and nothing in the product
 * may call it. Floating point is accumulated in double unless the paper's
 * pipeline fixes a narrower type (bf16 operands of the projection, fp32 stored
 * vectors).
 *
 * Notation follows the paper with one renaming that avoids a clash: the paper
 * projects R^d -> R^k; here the gradient dimension is P and the projected
 * dimension is d (d = 8192 in Sec. 4.1 of the paper).
 *
 * Pins (what fixes each function independently of this file) live in
 * tests/test_oracle_pins.py.
 *
 * Parity unpinned: the Adam hyper-parameters (beta1, beta2, eps) and the maps
 * from Philox output to a matrix entry (Rademacher bit, Gaussian pair) are
 * conventions of this library,
 * not statements of the paper; the paper cannot pin them. Everything else has
 * at least one pin.
 *
 * Build: gcc -O2 -ffp-contract=off -fno-fast-math -shared -fPIC
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

/* ------------------------------------------------------------------------- */
/* Philox4x32-10 (Salmon, Moraes, Dror, Shaw: "Parallel random numbers: as   */
/* easy as 1, 2, 3", SC'11, Sec. 3.3 and Table 2 constants).                  */
/* ------------------------------------------------------------------------- */

void qlo_philox4x32_10(const uint32_t ctr[4], const uint32_t key[2], uint32_t out[4])
{
    uint32_t c0 = ctr[0], c1 = ctr[1], c2 = ctr[2], c3 = ctr[3];
    uint32_t k0 = key[0], k1 = key[1];
    for (int round = 0; round < 10; ++round) {
        if (round > 0) { /* key schedule: Weyl sequence, bumped between rounds */
            k0 += 0x9E3779B9u;
            k1 += 0xBB67AE85u;
        }
        uint64_t p0 = (uint64_t)0xD2511F53u * (uint64_t)c0;
        uint64_t p1 = (uint64_t)0xCD9E8D57u * (uint64_t)c2;
        uint32_t hi0 = (uint32_t)(p0 >> 32), lo0 = (uint32_t)p0;
        uint32_t hi1 = (uint32_t)(p1 >> 32), lo1 = (uint32_t)p1;
        uint32_t n0 = hi1 ^ c1 ^ k0;
        uint32_t n1 = lo1;
        uint32_t n2 = hi0 ^ c3 ^ k1;
        uint32_t n3 = lo0;
        c0 = n0; c1 = n1; c2 = n2; c3 = n3;
    }
    out[0] = c0; out[1] = c1; out[2] = c2; out[3] = c3;
}

/* ------------------------------------------------------------------------- */
/* Rademacher projection matrix R in {+-1/sqrt(d)}^{d x P}  (paper Sec. 2.2,  */
/* Eq. 1, and Sec. 2.4: "a randomly sampled matrix ... (e.g., Gaussian or     */
/* Rademacher)"). R is never stored: entry (r, j) is a pure function of       */
/* (seed, r, j).                                                              */
/*                                                                            */
/* Entry map (library convention): the 128 entries j = 128*blk .. 128*blk+127 */
/* of row r are the 128 output bits of ONE Philox call with                   */
/*     counter = (blk, r, 0, 0),  key = (seed low 32, seed high 32).          */
/* Inside the block, t = j mod 128 selects output word t/32; with u = t mod   */
/* 32 the bit taken is   beta(u) = 15 - (u / 2) + 16 * (u mod 2).             */
/* (Even columns walk bits 15..0 downwards, odd columns walk 31..16.)         */
/* bit = 1 means the entry is -1, bit = 0 means +1.                           */
/* ------------------------------------------------------------------------- */

int qlo_rademacher_sign(uint64_t seed, uint32_t r, uint64_t j)
{
    uint32_t ctr[4] = { (uint32_t)(j >> 7), r, 0u, 0u };
    uint32_t key[2] = { (uint32_t)(seed & 0xFFFFFFFFu), (uint32_t)(seed >> 32) };
    uint32_t w[4];
    qlo_philox4x32_10(ctr, key, w);
    uint32_t t = (uint32_t)(j & 127u);
    uint32_t u = t & 31u;
    uint32_t beta = 15u - (u >> 1) + 16u * (u & 1u);
    uint32_t bit = (w[t >> 5] >> beta) & 1u;
    return bit ? -1 : +1;
}

/* Signs of row r for columns j0 .. j0+nj-1, as int8 +-1. */
void qlo_rademacher_row(uint64_t seed, uint32_t r, uint64_t j0, uint64_t nj, int8_t* out)
{
    uint32_t key[2] = { (uint32_t)(seed & 0xFFFFFFFFu), (uint32_t)(seed >> 32) };
    uint32_t w[4] = {0, 0, 0, 0};
    uint64_t have_blk = UINT64_MAX;
    for (uint64_t i = 0; i < nj; ++i) {
        uint64_t j = j0 + i;
        uint64_t blk = j >> 7;
        if (blk != have_blk) {
            uint32_t ctr[4] = { (uint32_t)blk, r, 0u, 0u };
            qlo_philox4x32_10(ctr, key, w);
            have_blk = blk;
        }
        uint32_t t = (uint32_t)(j & 127u);
        uint32_t u = t & 31u;
        uint32_t beta = 15u - (u >> 1) + 16u * (u & 1u);
        out[i] = ((w[t >> 5] >> beta) & 1u) ? (int8_t)-1 : (int8_t)1;
    }
}

/* ------------------------------------------------------------------------- */
/* bfloat16: the upper 16 bits of an IEEE binary32; round to nearest even.   */
/* ------------------------------------------------------------------------- */

float qlo_round_to_bf16(float x)
{
    uint32_t u;
    memcpy(&u, &x, 4);
    if ((u & 0x7F800000u) == 0x7F800000u) { /* inf / nan: keep class */
        if (u & 0x007FFFFFu) u |= 0x00400000u;
        u &= 0xFFFF0000u;
    } else {
        uint32_t lsb = (u >> 16) & 1u;
        u += 0x7FFFu + lsb;
        u &= 0xFFFF0000u;
    }
    float y;
    memcpy(&y, &u, 4);
    return y;
}

/* ------------------------------------------------------------------------- */
/* Adam training gradient Gamma(z; theta) of a training example z (paper      */
/* Sec. 2.2). The paper                                                        */
/* names it without a formula; the reading taken is the Adam update direction */
/* the optimiser would apply if the example's gradient g were the next one,   */
/* given the checkpoint's moments m, v:                                       */
/*    m' = b1 m + (1-b1) g,   v' = b2 v + (1-b2) g^2,                         */
/*    (step > 0: m' /= c1, v' /= c2 with c = fp32(1 - b^step), the power      */
/*     taken in double)                                                       */
/*    Gamma = m' / (sqrt(v') + eps)                                           */
/* in fp32, then rounded to bf16 because the projection contracts bf16        */
/* operands. m == NULL means the SGD (validation) gradient: Gamma = bf16(g).  */
/* ------------------------------------------------------------------------- */

void qlo_adam_gamma(const float* g, const float* m, const float* v, int64_t P,
                    float beta1, float beta2, float eps, int64_t step, float* gamma)
{
    if (m == NULL || v == NULL) {
        for (int64_t j = 0; j < P; ++j) gamma[j] = qlo_round_to_bf16(g[j]);
        return;
    }
    float c1 = 1.0f, c2 = 1.0f;
    if (step > 0) {
        c1 = (float)(1.0 - pow((double)beta1, (double)step));
        c2 = (float)(1.0 - pow((double)beta2, (double)step));
    }
    for (int64_t j = 0; j < P; ++j) {
        float gj = g[j];
        float m1 = beta1 * m[j] + (1.0f - beta1) * gj;
        float v1 = beta2 * v[j] + (1.0f - beta2) * (gj * gj);
        if (step > 0) { m1 = m1 / c1; v1 = v1 / c2; }
        float den = sqrtf(v1) + eps;
        gamma[j] = qlo_round_to_bf16(m1 / den);
    }
}

/* ------------------------------------------------------------------------- */
/* Random projection, Eq. 1:  y = R Gamma,  R_rj = s_rj / sqrt(d).            */
/* gamma: [n, P] fp32 holding bf16-representable values; y: [n, d] fp32.      */
/* Sum in double over j ascending, scale by the fp32 value of 1/sqrt(d).      */
/* ------------------------------------------------------------------------- */

void qlo_project(const float* gamma, int64_t n, int64_t P, int32_t d, uint64_t seed, float* y)
{
    int8_t* s = (int8_t*)malloc((size_t)P);
    float inv_sqrt_d = 1.0f / sqrtf((float)d);
    for (int32_t r = 0; r < d; ++r) {
        qlo_rademacher_row(seed, (uint32_t)r, 0, (uint64_t)P, s);
        for (int64_t i = 0; i < n; ++i) {
            const float* gi = gamma + i * P;
            double acc = 0.0;
            for (int64_t j = 0; j < P; ++j) acc += (double)gi[j] * (double)s[j];
            y[i * (int64_t)d + r] = (float)(acc * (double)inv_sqrt_d);
        }
    }
    free(s);
}

/* Same, for a subset of output coordinates rows[0..nr) (sampled parity at   */
/* sizes where all d coordinates would take hours). y: [n, nr].               */
void qlo_project_rows(const float* gamma, int64_t n, int64_t P, int32_t d, uint64_t seed,
                      const int32_t* rows, int32_t nr, float* y)
{
    int8_t* s = (int8_t*)malloc((size_t)P);
    float inv_sqrt_d = 1.0f / sqrtf((float)d);
    for (int32_t a = 0; a < nr; ++a) {
        qlo_rademacher_row(seed, (uint32_t)rows[a], 0, (uint64_t)P, s);
        for (int64_t i = 0; i < n; ++i) {
            const float* gi = gamma + i * P;
            double acc = 0.0;
            for (int64_t j = 0; j < P; ++j) acc += (double)gi[j] * (double)s[j];
            y[i * (int64_t)nr + a] = (float)(acc * (double)inv_sqrt_d);
        }
    }
    free(s);
}

/* ------------------------------------------------------------------------- */
/* Gaussian projection matrix (the other distribution Sec. 2.4 allows for R): */
/* R_rj = z_rj / sqrt(d), z_rj ~ N(0, 1), again a pure function of            */
/* (seed, r, j) and never stored.                                             */
/*                                                                            */
/* Entry map (library convention): the four entries j = 4q .. 4q+3 of row r   */
/* come from ONE Philox call with                                             */
/*     counter = (q mod 2^32, r, q div 2^32, 1),  key = seed as above         */
/* (the last counter word keeps this stream apart from the Rademacher one).   */
/* Output words (w0, w1) give entries 4q, 4q+1 and (w2, w3) give 4q+2, 4q+3   */
/* by the Box-Muller transform (Box and Muller, Ann. Math. Statist. 1958):    */
/*     u1 = (floor(wa / 2^9) + 1/2) / 2^23,  u2 = (floor(wb / 2^9) + 1/2) / 2^23 */
/*     z_even = sqrt(-2 ln u1) cos(2 pi u2),  z_odd = sqrt(-2 ln u1) sin(2 pi u2) */
/* (both uniforms lie strictly inside (0, 1) and are exact in binary32).      */
/* The entry that enters the contraction is z rounded to bf16, because the    */
/* projection multiplies bf16 operands.                                       */
/* ------------------------------------------------------------------------- */

/* The entry before rounding, in double. */
double qlo_gaussian_entry_exact(uint64_t seed, uint32_t r, uint64_t j)
{
    uint64_t q = j >> 2;
    uint32_t ctr[4] = { (uint32_t)(q & 0xFFFFFFFFu), r, (uint32_t)(q >> 32), 1u };
    uint32_t key[2] = { (uint32_t)(seed & 0xFFFFFFFFu), (uint32_t)(seed >> 32) };
    uint32_t w[4];
    qlo_philox4x32_10(ctr, key, w);
    uint32_t wa = (j & 2u) ? w[2] : w[0];
    uint32_t wb = (j & 2u) ? w[3] : w[1];
    double u1 = ((double)(wa >> 9) + 0.5) / 8388608.0;
    double u2 = ((double)(wb >> 9) + 0.5) / 8388608.0;
    double rho = sqrt(-2.0 * log(u1));
    double ang = 2.0 * 3.14159265358979323846 * u2;
    return (j & 1u) ? rho * sin(ang) : rho * cos(ang);
}

/* Entries of row r for columns j0 .. j0+nj-1 as they enter the contraction:  */
/* fp32 holding bf16-representable values.                                    */
void qlo_gaussian_row(uint64_t seed, uint32_t r, uint64_t j0, uint64_t nj, float* out)
{
    for (uint64_t i = 0; i < nj; ++i)
        out[i] = qlo_round_to_bf16((float)qlo_gaussian_entry_exact(seed, r, j0 + i));
}

/* Eq. 1 with the Gaussian matrix: y_r = (sum_j Gamma_j z_rj) / sqrt(d), the   */
/* sum in double over j ascending, the scale the fp32 value of 1/sqrt(d).     */
void qlo_project_gaussian(const float* gamma, int64_t n, int64_t P, int32_t d, uint64_t seed, float* y)
{
    float* z = (float*)malloc(sizeof(float) * (size_t)P);
    float inv_sqrt_d = 1.0f / sqrtf((float)d);
    for (int32_t r = 0; r < d; ++r) {
        qlo_gaussian_row(seed, (uint32_t)r, 0, (uint64_t)P, z);
        for (int64_t i = 0; i < n; ++i) {
            const float* gi = gamma + i * P;
            double acc = 0.0;
            for (int64_t j = 0; j < P; ++j) acc += (double)gi[j] * (double)z[j];
            y[i * (int64_t)d + r] = (float)(acc * (double)inv_sqrt_d);
        }
    }
    free(z);
}

/* ------------------------------------------------------------------------- */
/* L2 normalisation, Eq. 2:  yhat = y / ||y||.                                */
/* Returns the norm as fp32. A zero vector stays zero.                        */
/* ------------------------------------------------------------------------- */

float qlo_normalize(const float* y, int32_t d, float* yhat)
{
    double n2 = 0.0;
    for (int32_t m = 0; m < d; ++m) n2 += (double)y[m] * (double)y[m];
    float nrm = (float)sqrt(n2);
    if (nrm == 0.0f) {
        for (int32_t m = 0; m < d; ++m) yhat[m] = 0.0f;
        return 0.0f;
    }
    float rn = 1.0f / nrm;
    for (int32_t m = 0; m < d; ++m) yhat[m] = y[m] * rn;
    return nrm;
}

/* ------------------------------------------------------------------------- */
/* Absmax quantisation, Eq. 4-5 and Sec. 3.1:                                 */
/*    S = max_m |x_m|,  alpha = 2^(b-1) - 1,  q_m = round(alpha x_m / S).     */
/* round = IEEE round-half-to-even. b = 1: alpha would be 0, so the 1-bit     */
/* store is the sign quantiser ("Sign 1-bit" row of Table 3; Sec. 2.4 binary  */
/* QRP with levels {-1,+1}); sign(0) = +1. S = 0: all codes 0.                */
/* q: [d] int8 (unpacked); returns S; *sumsq = sum q^2.                       */
/* ------------------------------------------------------------------------- */

float qlo_quantize(const float* x, int32_t d, int32_t bits, int8_t* q, int32_t* sumsq)
{
    float S = 0.0f;
    for (int32_t m = 0; m < d; ++m) {
        float a = fabsf(x[m]);
        if (a > S) S = a;
    }
    int64_t ss = 0;
    if (S == 0.0f) {
        for (int32_t m = 0; m < d; ++m) q[m] = 0;
        *sumsq = 0;
        return 0.0f;
    }
    if (bits == 1) {
        for (int32_t m = 0; m < d; ++m) q[m] = (x[m] < 0.0f) ? (int8_t)-1 : (int8_t)1;
        *sumsq = d;
        return S;
    }
    int32_t alpha = (1 << (bits - 1)) - 1;
    float r = (float)alpha / S;
    for (int32_t m = 0; m < d; ++m) {
        float t = rintf(x[m] * r);
        int32_t qi = (int32_t)t;
        if (qi > alpha) qi = alpha;
        if (qi < -alpha) qi = -alpha;
        q[m] = (int8_t)qi;
        ss += (int64_t)qi * qi;
    }
    *sumsq = (int32_t)ss;
    return S;
}

/* ------------------------------------------------------------------------- */
/* Dense little-endian bit packing of b-bit codes ("k b-bit integers plus one */
/* float per gradient vector", Sec. 3.1; sizes of Table 1 need d*b/8 bytes).  */
/*  b=8: one int8 per code.                                                   */
/*  b=4: code m in bits [4(m&1), +4) of byte m>>1, two's complement.          */
/*  b=2: code m in bits [2(m&3), +2) of byte m>>2, two's complement.          */
/*  b=1: code m is bit (m&7) of byte m>>3 (= bit m&31 of the little-endian    */
/*       uint32 word m>>5); bit=1 <=> -1; an all-zero vector (S = 0) is       */
/*       stored as all bits 0.                                                */
/* ------------------------------------------------------------------------- */

void qlo_pack(const int8_t* q, int32_t d, int32_t bits, uint8_t* out)
{
    int64_t nbytes = (int64_t)d * bits / 8;
    memset(out, 0, (size_t)nbytes);
    for (int32_t m = 0; m < d; ++m) {
        if (bits == 8) {
            out[m] = (uint8_t)q[m];
        } else if (bits == 4) {
            out[m >> 1] |= (uint8_t)(((uint8_t)q[m] & 0xFu) << (4 * (m & 1)));
        } else if (bits == 2) {
            out[m >> 2] |= (uint8_t)(((uint8_t)q[m] & 0x3u) << (2 * (m & 3)));
        } else { /* bits == 1 */
            if (q[m] < 0) out[m >> 3] |= (uint8_t)(1u << (m & 7));
        }
    }
}

/* Inverse of qlo_pack. For b=1 a stored bit 0 reads back as +1. */
void qlo_unpack(const uint8_t* in, int32_t d, int32_t bits, int8_t* q)
{
    for (int32_t m = 0; m < d; ++m) {
        if (bits == 8) {
            q[m] = (int8_t)in[m];
        } else if (bits == 4) {
            int v = (in[m >> 1] >> (4 * (m & 1))) & 0xF;
            q[m] = (int8_t)(v >= 8 ? v - 16 : v);
        } else if (bits == 2) {
            int v = (in[m >> 2] >> (2 * (m & 3))) & 0x3;
            q[m] = (int8_t)(v >= 2 ? v - 4 : v);
        } else {
            int v = (in[m >> 3] >> (m & 7)) & 1;
            q[m] = (int8_t)(v ? -1 : 1);
        }
    }
}

/* ------------------------------------------------------------------------- */
/* Stage 2 as the datastore builder sees it: normalise (Eq. 2), quantise      */
/* (Eq. 4-5), pack. x: [n, d] fp32. normalize = 0 skips Eq. 2 (the caller     */
/* passes already-normalised rows).                                           */
/* codes: [n, d*bits/8]; scales: [n]; sumsq: [n].                             */
/* ------------------------------------------------------------------------- */

void qlo_quantize_rows(const float* x, int64_t n, int32_t d, int32_t bits, int normalize,
                       uint8_t* codes, float* scales, int32_t* sumsq)
{
    float* xh = (float*)malloc(sizeof(float) * (size_t)d);
    int8_t* q = (int8_t*)malloc((size_t)d);
    int64_t row_bytes = (int64_t)d * bits / 8;
    for (int64_t i = 0; i < n; ++i) {
        const float* xi = x + i * (int64_t)d;
        if (normalize) qlo_normalize(xi, d, xh);
        else memcpy(xh, xi, sizeof(float) * (size_t)d);
        scales[i] = qlo_quantize(xh, d, bits, q, &sumsq[i]);
        qlo_pack(q, d, bits, codes + i * row_bytes);
    }
    free(xh);
    free(q);
}

/* ------------------------------------------------------------------------- */
/* Integer inner product of two code vectors (numerator of Eq. 7).            */
/* ------------------------------------------------------------------------- */

int64_t qlo_dot(const int8_t* a, const int8_t* b, int32_t d)
{
    int64_t acc = 0;
    for (int32_t m = 0; m < d; ++m) acc += (int64_t)a[m] * (int64_t)b[m];
    return acc;
}

/* Integer dots of train rows [t0, t0+nt) against all V validation rows of    */
/* one checkpoint. dots: [nt, V] int32.                                       */
void qlo_dots(const uint8_t* train_codes, const uint8_t* val_codes, int64_t t0, int64_t nt,
              int32_t V, int32_t d, int32_t bits, int32_t* dots)
{
    int64_t row_bytes = (int64_t)d * bits / 8;
    int8_t* qt = (int8_t*)malloc((size_t)d);
    int8_t* qv = (int8_t*)malloc((size_t)d * (size_t)(V > 0 ? V : 1));
    for (int32_t v = 0; v < V; ++v) qlo_unpack(val_codes + v * row_bytes, d, bits, qv + (int64_t)v * d);
    for (int64_t t = 0; t < nt; ++t) {
        qlo_unpack(train_codes + (t0 + t) * row_bytes, d, bits, qt);
        for (int32_t v = 0; v < V; ++v)
            dots[t * V + v] = (int32_t)qlo_dot(qt, qv + (int64_t)v * d, d);
    }
    free(qt);
    free(qv);
}

/* ------------------------------------------------------------------------- */
/* Influence score, Eq. 6-7 plus the LESS aggregation:                        */
/*   qhat = q / ||q||                       (Eq. 6, norm of the integer code) */
/*   Inf(z, z') = sum_i eta_i <qhat_z',i , qhat_z,i>                 (Eq. 7)  */
/*   A[z, j]   = sum_i eta_i * mean_{z' in task j} <qhat_z',i, qhat_z,i>      */
/*   score[z]  = max_j A[z, j]                                                */
/* (influence accumulated over the validation data, Sec. 4.1; mean-per-task / max-over-tasks   */
/* is the LESS rule the paper inherits.)                                      */
/* mode 0 (cosine): as above; a vector whose stored scale S is 0 is the zero  */
/*   vector and contributes 0.                                                */
/* mode 1 (dequant): <S_z q_z/alpha, S_z' q_z'/alpha> -- the inner product of */
/*   the reconstructed vectors (alpha := 1 at b = 1), approximating Eq. 3.    */
/* train_codes: [C][N][row_bytes] with ckpt stride in bytes; val likewise.    */
/* train_scales: [C][N]; val_scales: [C][V]. eta: [C]. task_off: [T+1].       */
/* Scores for train rows [t0, t0+nt): scores [nt]; per_task [nt, T] or NULL.  */
/* ------------------------------------------------------------------------- */

void qlo_score(const uint8_t* train_codes, int64_t train_ckpt_stride,
               const uint8_t* val_codes, int64_t val_ckpt_stride,
               const float* train_scales, const float* val_scales,
               const float* eta, const int32_t* task_off,
               int64_t N, int32_t V, int32_t C, int32_t T, int32_t d, int32_t bits, int32_t mode,
               int64_t t0, int64_t nt, float* scores, float* per_task)
{
    int64_t row_bytes = (int64_t)d * bits / 8;
    int8_t* qt = (int8_t*)malloc((size_t)d);
    int8_t* qv = (int8_t*)malloc((size_t)d * (size_t)(V > 0 ? V : 1) * (size_t)C);
    double* vnorm = (double*)malloc(sizeof(double) * (size_t)(V > 0 ? V : 1) * (size_t)C);
    double* A = (double*)malloc(sizeof(double) * (size_t)(T > 0 ? T : 1));
    double alpha = (bits == 1) ? 1.0 : (double)((1 << (bits - 1)) - 1);

    for (int32_t i = 0; i < C; ++i)
        for (int32_t v = 0; v < V; ++v) {
            int8_t* dst = qv + ((int64_t)i * V + v) * d;
            qlo_unpack(val_codes + i * val_ckpt_stride + v * row_bytes, d, bits, dst);
            vnorm[(int64_t)i * V + v] = sqrt((double)qlo_dot(dst, dst, d));
        }

    for (int64_t t = 0; t < nt; ++t) {
        for (int32_t j = 0; j < T; ++j) A[j] = 0.0;
        for (int32_t i = 0; i < C; ++i) {
            float St = train_scales[(int64_t)i * N + (t0 + t)];
            qlo_unpack(train_codes + i * train_ckpt_stride + (t0 + t) * row_bytes, d, bits, qt);
            double tnorm = sqrt((double)qlo_dot(qt, qt, d));
            for (int32_t j = 0; j < T; ++j) {
                double sum = 0.0;
                for (int32_t v = task_off[j]; v < task_off[j + 1]; ++v) {
                    float Sv = val_scales[(int64_t)i * V + v];
                    double D = (double)qlo_dot(qt, qv + ((int64_t)i * V + v) * d, d);
                    double sim;
                    if (mode == 0) {
                        if (St == 0.0f || Sv == 0.0f || tnorm == 0.0 || vnorm[(int64_t)i * V + v] == 0.0)
                            sim = 0.0;
                        else
                            sim = D / (tnorm * vnorm[(int64_t)i * V + v]);
                    } else {
                        sim = ((double)St / alpha) * ((double)Sv / alpha) * D;
                    }
                    sum += sim;
                }
                int32_t cnt = task_off[j + 1] - task_off[j];
                A[j] += (double)eta[i] * (sum / (double)cnt);
            }
        }
        double best = A[0];
        for (int32_t j = 1; j < T; ++j) if (A[j] > best) best = A[j];
        scores[t] = (float)best;
        if (per_task) for (int32_t j = 0; j < T; ++j) per_task[t * T + j] = (float)A[j];
    }
    free(qt); free(qv); free(vnorm); free(A);
}

/* ------------------------------------------------------------------------- */
/* Top-k selection ("Select the top 5% of training data ... based on these    */
/* scores", Sec. 4.1).  k = floor(frac * N + 1e-6) clamped to [0, N].         */
/* Total order on fp32: by value, -0 < +0, every NaN below -inf; ties go to   */
/* the smaller index. Output: the k chosen indices in ascending order.        */
/* Done the slow way: stable sort of all N keys.                              */
/* ------------------------------------------------------------------------- */

static uint32_t qlo_order_key(float x)
{
    uint32_t u;
    memcpy(&u, &x, 4);
    if ((u & 0x7F800000u) == 0x7F800000u && (u & 0x007FFFFFu)) return 0u; /* NaN: lowest */
    return (u >> 31) ? ~u : (u | 0x80000000u);
}

typedef struct { uint32_t key; int64_t idx; } qlo_pair;

static int qlo_pair_cmp(const void* a, const void* b)
{
    const qlo_pair* x = (const qlo_pair*)a;
    const qlo_pair* y = (const qlo_pair*)b;
    if (x->key != y->key) return (x->key > y->key) ? -1 : 1; /* larger score first */
    if (x->idx != y->idx) return (x->idx < y->idx) ? -1 : 1; /* then smaller index */
    return 0;
}

static int qlo_i64_cmp(const void* a, const void* b)
{
    int64_t x = *(const int64_t*)a, y = *(const int64_t*)b;
    return (x > y) - (x < y);
}

int64_t qlo_topk_count(int64_t N, double frac)
{
    double kf = floor(frac * (double)N + 1e-6);
    if (kf < 0.0) kf = 0.0;
    if (kf > (double)N) kf = (double)N;
    return (int64_t)kf;
}

int64_t qlo_select_topk(const float* scores, int64_t N, double frac, int64_t* indices)
{
    int64_t k = qlo_topk_count(N, frac);
    if (k == 0) return 0;
    qlo_pair* p = (qlo_pair*)malloc(sizeof(qlo_pair) * (size_t)N);
    for (int64_t i = 0; i < N; ++i) { p[i].key = qlo_order_key(scores[i]); p[i].idx = i; }
    qsort(p, (size_t)N, sizeof(qlo_pair), qlo_pair_cmp); /* comparator is a total order */
    for (int64_t i = 0; i < k; ++i) indices[i] = p[i].idx;
    qsort(indices, (size_t)k, sizeof(int64_t), qlo_i64_cmp);
    free(p);
    return k;
}

/* ------------------------------------------------------------------------- */
/* Stage 1+2 end to end for rows of one checkpoint:                           */
/* gradient -> Gamma (bf16) -> projection -> normalise -> quantise -> pack.   */
/* g: [n, P] fp32 (bf16 inputs are widened by the caller, which is exact).    */
/* proj_out (optional): [n, d] un-normalised projection.                      */
/* ------------------------------------------------------------------------- */

void qlo_project_quantize(const float* g, int64_t n, int64_t P,
                          const float* m, const float* v,
                          float beta1, float beta2, float eps, int64_t step,
                          int32_t d, uint64_t seed, int32_t bits,
                          uint8_t* codes, float* scales, int32_t* sumsq, float* proj_out)
{
    float* gamma = (float*)malloc(sizeof(float) * (size_t)n * (size_t)P);
    float* y = (float*)malloc(sizeof(float) * (size_t)n * (size_t)d);
    for (int64_t i = 0; i < n; ++i)
        qlo_adam_gamma(g + i * P, m, v, P, beta1, beta2, eps, step, gamma + i * P);
    qlo_project(gamma, n, P, d, seed, y);
    if (proj_out) memcpy(proj_out, y, sizeof(float) * (size_t)n * (size_t)d);
    qlo_quantize_rows(y, n, d, bits, 1, codes, scales, sumsq);
    free(gamma);
    free(y);
}
