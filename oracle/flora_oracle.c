/*
 * Flora CPU oracle — TEST INFRASTRUCTURE, not a product path.
 *
 * A plain, slow, obviously-correct statement of what the Flora hot path
 * computes (arXiv 2402.03293): the seeded Gaussian projection A ~ N_s(0, 1/r)
 * (Algorithm 1, "A_W <- N_{s_W}(0,1/r)"), compression C += G A^T and
 * decompression C A (Algorithm 1), the compressed momentum
 * M <- beta M' + (1-beta) G A'^T and the transfer M' = M A A'^T (Algorithm 2).
 *
 * Only the test-suite, the smoke check and the CPU-baseline timing may call
 * this file.  It shares no code with the CUDA library: the generator below is
 * written a second time, from its definition, inside the CUDA sources.
 *
 * Conventions: matrices are row-major with an explicit leading dimension.
 * G, W are n x m (fp32, or bf16 held as uint16); A is an explicit r x m fp32
 * array produced by flora_oracle_materialize_A (optionally rounded to bf16
 * values by flora_oracle_round_to_bf16); C, M are n x r fp32.  Every
 * contraction is a triple loop accumulated in double and rounded once to the
 * storage type (round to nearest even).
 *
 * Pins (tests, CPU only): the Philox core against the cuRAND host generator
 * and an independent big-integer implementation plus round invertibility; the
 * normal transform against the libm double-precision Box-Muller formula and
 * moment / Kolmogorov-Smirnov tests; the contractions against brute force
 * written from the algorithms, float64 matmul on explicit A, linearity,
 * E[A^T A] = I (Theorem 2.4), row-norm preservation (Lemma 2.3) and the
 * closed forms of the momentum recursion.  The paper prints no worked
 * numeric example of the path, so no printed-value pin exists.
 *
 * Build: gcc -O2 -ffp-contract=off -fopenmp -shared -fPIC flora_oracle.c -lm
 * (-ffp-contract=off matters: every fused multiply-add below is an explicit
 * fmaf, nothing else may be fused.)
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

enum { ORACLE_F32 = 0, ORACLE_BF16 = 1 };

/* ------------------------------------------------------------------------- */
/* Philox4x32-10 (Salmon, Moraes, Dror, Shaw: "Parallel random numbers: as   */
/* easy as 1, 2, 3", SC'11).  Four 32-bit counter words, two 32-bit key      */
/* words, ten rounds; the key is bumped by the Weyl constants between rounds. */
/* ------------------------------------------------------------------------- */
void flora_oracle_philox4x32_10(const uint32_t ctr[4], const uint32_t key[2], uint32_t out[4])
{
    uint32_t c0 = ctr[0], c1 = ctr[1], c2 = ctr[2], c3 = ctr[3];
    uint32_t k0 = key[0], k1 = key[1];
    for (int round = 0; round < 10; ++round) {
        uint64_t p0 = (uint64_t)0xD2511F53u * (uint64_t)c0;
        uint64_t p1 = (uint64_t)0xCD9E8D57u * (uint64_t)c2;
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

/* ------------------------------------------------------------------------- */
/* Normal transform.  The paper fixes only the law N(0,1/r) and that every    */
/* element is addressable from the seed; the arithmetic below is this         */
/* project's definition of that draw, chosen so that it is bit-reproducible   */
/* with IEEE-754 binary32 operations alone (integer ops, exact conversions,   */
/* fmaf, multiply, add, correctly rounded sqrtf).                             */
/*                                                                            */
/*   u1 = k1 / 2^24, k1 = (xa >> 8) + 1 in [1, 2^24]      (so u1 in (0,1])    */
/*   u2 = k2 / 2^24, k2 =  xb >> 8      in [0, 2^24)                          */
/*   rho = sqrt(-2 ln u1), z_cos = rho cos(2 pi u2), z_sin = rho sin(2 pi u2) */
/* ------------------------------------------------------------------------- */
static inline uint32_t f32_bits(float f) { uint32_t u; memcpy(&u, &f, 4); return u; }
static inline float bits_f32(uint32_t u) { float f; memcpy(&f, &u, 4); return f; }

/* -2 ln(k / 2^24): split k into 2^e * mant with mant in [2/3, 4/3), then
 * ln(mant) = s - s^2/2 + s^3 Q(s), s = mant - 1, Q a fixed degree-6 polynomial. */
static float neg2_ln_u1(uint32_t k1)
{
    static const float Q[7] = {
        0x1.555528p-2f, -0x1.000b1cp-2f, 0x1.99c32p-3f, -0x1.515a6cp-3f,
        0x1.1f9622p-3f, -0x1.35b3ep-3f, 0x1.1b09e8p-3f };
    float f = (float)k1;                              /* exact: k1 <= 2^24 */
    uint32_t b = f32_bits(f);
    int32_t e = (int32_t)(b - 0x3F2AAAABu) >> 23;     /* arithmetic shift  */
    float mant = bits_f32(b - ((uint32_t)e << 23));
    float s = mant - 1.0f;                            /* exact             */
    float q = Q[6];
    for (int i = 5; i >= 0; --i) q = fmaf(q, s, Q[i]);
    float s2 = s * s;
    float p = fmaf(q, s, -0.5f);
    p = fmaf(p, s2, s);                               /* ln(mant)          */
    float steps = (float)(24 - e);                    /* exact small int   */
    return fmaf(steps, 0x1.62e43p+0f /* 2 ln 2 */, -2.0f * p);
}

/* cos and sin of 2 pi k2 / 2^24 by exact integer octant reduction: the top
 * three bits of k2 pick the octant, the low 21 bits are the position inside
 * it; odd octants are reflected so that the polynomial argument stays in
 * [0, pi/4]. */
static void cos_sin_2pi_u2(uint32_t k2, float* c_out, float* s_out)
{
    uint32_t oct = k2 >> 21;
    uint32_t frac = k2 & 0x1FFFFFu;
    if (oct & 1u) frac = 0x200000u - frac;
    float x = (float)frac * 0x1.921fb6p-22f;          /* (pi/4) 2^-21      */
    float z = x * x;
    float sp = fmaf(-0x1.9943e2p-13f, z, 0x1.11073ap-7f);
    sp = fmaf(sp, z, -0x1.555546p-3f);
    float sx = fmaf(x * z, sp, x);                    /* sin x             */
    float cp = fmaf(-0x1.644d62p-10f, z, 0x1.553e8p-5f);
    cp = fmaf(cp, z, -0x1.ffffb2p-2f);
    float cx = fmaf(z, cp, 1.0f);                     /* cos x             */
    int swap = ((oct + 1u) >> 1) & 1u;                /* octants 1,2,5,6   */
    float c = swap ? sx : cx;
    float s = swap ? cx : sx;
    if (((oct + 2u) >> 2) & 1u) c = -c;               /* octants 2..5      */
    if (oct >> 2) s = -s;                             /* octants 4..7      */
    *c_out = c; *s_out = s;
}

void flora_oracle_normal_pair(uint32_t xa, uint32_t xb, float* z_cos, float* z_sin)
{
    float rho = sqrtf(neg2_ln_u1((xa >> 8) + 1u));
    float c, s;
    cos_sin_2pi_u2(xb >> 8, &c, &s);
    *z_cos = rho * c;
    *z_sin = rho * s;
}

/* The uniforms behind a pair, in double, for checking the transform against
 * the textbook formula. */
void flora_oracle_pair_uniforms(uint32_t xa, uint32_t xb, double* u1, double* u2)
{
    *u1 = (double)((xa >> 8) + 1u) / 16777216.0;
    *u2 = (double)(xb >> 8) / 16777216.0;
}

/* A[j,k] for a whole r x m matrix (Algorithm 1: A_W <- N_{s_W}(0, 1/r)).
 * Key = the two halves of the seed.  The Philox block with counter
 * (q, j, 0, 0) yields columns 4q..4q+3 of row j: words (0,1) make columns
 * 4q (cos) and 4q+1 (sin), words (2,3) make columns 4q+2 and 4q+3.  Each
 * standard normal is scaled by fl32(1/sqrtf(r)). */
void flora_oracle_materialize_A(uint64_t seed, int r, int64_t m, float* A, int64_t lda)
{
    uint32_t key[2] = { (uint32_t)(seed & 0xFFFFFFFFu), (uint32_t)(seed >> 32) };
    float scale = 1.0f / sqrtf((float)r);
    for (int j = 0; j < r; ++j) {
        for (int64_t q = 0; 4 * q < m; ++q) {
            uint32_t ctr[4] = { (uint32_t)q, (uint32_t)j, 0u, 0u }, x[4];
            float z[4];
            flora_oracle_philox4x32_10(ctr, key, x);
            flora_oracle_normal_pair(x[0], x[1], &z[0], &z[1]);
            flora_oracle_normal_pair(x[2], x[3], &z[2], &z[3]);
            for (int t = 0; t < 4 && 4 * q + t < m; ++t)
                A[(int64_t)j * lda + 4 * q + t] = z[t] * scale;
        }
    }
}

/* fp32 -> bf16 bits, round to nearest even (no NaN handling needed here). */
static inline uint16_t bf16_bits_rne(float f)
{
    uint32_t u = f32_bits(f);
    u += 0x7FFFu + ((u >> 16) & 1u);
    return (uint16_t)(u >> 16);
}
static inline float bf16_value(uint16_t h) { return bits_f32((uint32_t)h << 16); }

void flora_oracle_round_to_bf16(const float* in, int64_t count, float* out_values, uint16_t* out_bits)
{
    for (int64_t i = 0; i < count; ++i) {
        uint16_t h = bf16_bits_rne(in[i]);
        if (out_bits) out_bits[i] = h;
        if (out_values) out_values[i] = bf16_value(h);
    }
}

static inline double load_elem(const void* base, int dtype, int64_t idx)
{
    return dtype == ORACLE_BF16 ? (double)bf16_value(((const uint16_t*)base)[idx])
                                : (double)((const float*)base)[idx];
}
/* (float)v followed by bf16 rounding would round twice; round the double to
 * bf16 directly instead. */
static inline uint16_t bf16_bits_from_double(double v)
{
    /* a bf16 value is a double with at most 8 significant bits: find the two
     * neighbours through the float truncation and pick the nearer (ties to
     * even mantissa). */
    float f = (float)v;
    uint32_t u = f32_bits(f);
    uint32_t lo = u & 0xFFFF0000u;              /* toward zero            */
    double a = (double)bits_f32(lo);
    if (a == v) return (uint16_t)(lo >> 16);
    /* f may itself have been rounded away from v: step so that a, b bracket v */
    if (fabs(a) > fabs(v)) { lo -= 0x10000u; a = (double)bits_f32(lo); }
    uint32_t hi = lo + 0x10000u;                /* away from zero         */
    double b = (double)bits_f32(hi);
    double da = fabs(v - a), db = fabs(b - v);
    if (da < db) return (uint16_t)(lo >> 16);
    if (db < da) return (uint16_t)(hi >> 16);
    return (uint16_t)(((lo >> 16) & 1u) ? (hi >> 16) : (lo >> 16));
}
uint16_t flora_oracle_double_to_bf16(double v) { return bf16_bits_from_double(v); }
static inline void store_rounded(void* base, int dtype, int64_t idx, double v)
{
    if (dtype == ORACLE_BF16) ((uint16_t*)base)[idx] = bf16_bits_from_double(v);
    else ((float*)base)[idx] = (float)v;
}

/* Algorithm 1, compression:  C <- C + G A^T.
 * Algorithm 2, momentum:     M <- beta M + (1 - beta) G A^T.
 * Both are  S[i,j] <- b * S[i,j] + a * sum_k G[i,k] A[j,k]. */
void flora_oracle_compress_axpby(const void* G, int g_dtype, int64_t n, int64_t m, int64_t ldg,
                                 const float* A, int r, int64_t lda,
                                 double a, double b, float* S, int64_t lds)
{
    #pragma omp parallel for schedule(static)
    for (int64_t i = 0; i < n; ++i)
        for (int j = 0; j < r; ++j) {
            double acc = 0.0;
            for (int64_t k = 0; k < m; ++k)
                acc += load_elem(G, g_dtype, i * ldg + k) * (double)A[(int64_t)j * lda + k];
            S[i * lds + j] = (float)(b * (double)S[i * lds + j] + a * acc);
        }
}

void flora_oracle_compress_accumulate(const void* G, int g_dtype, int64_t n, int64_t m, int64_t ldg,
                                      const float* A, int r, int64_t lda, float* C, int64_t ldc)
{
    flora_oracle_compress_axpby(G, g_dtype, n, m, ldg, A, r, lda, 1.0, 1.0, C, ldc);
}

void flora_oracle_momentum_step(const void* G, int g_dtype, int64_t n, int64_t m, int64_t ldg,
                                const float* A, int r, int64_t lda, float beta, float* M, int64_t ldm)
{
    flora_oracle_compress_axpby(G, g_dtype, n, m, ldg, A, r, lda,
                                1.0 - (double)beta, (double)beta, M, ldm);
}

/* Algorithm 1, decompression, applied as an update:
 * W <- W - lr * scale * (C A)   (scale = 1/tau for an accumulation cycle,
 * 1 for the momentum "yield M A'"). */
void flora_oracle_decompress_apply(void* W, int w_dtype, int64_t n, int64_t m, int64_t ldw,
                                   const float* C, int r, int64_t ldc,
                                   const float* A, int64_t lda, float lr, float scale)
{
    double step = (double)lr * (double)scale;
    #pragma omp parallel for schedule(static)
    for (int64_t i = 0; i < n; ++i)
        for (int64_t k = 0; k < m; ++k) {
            double acc = 0.0;
            for (int j = 0; j < r; ++j)
                acc += (double)C[i * ldc + j] * (double)A[(int64_t)j * lda + k];
            store_rounded(W, w_dtype, i * ldw + k, load_elem(W, w_dtype, i * ldw + k) - step * acc);
        }
}

/* Algorithm 2, transfer, in the printed order: first the n x m product
 * P = src A_old, then dst <- b dst + a P A_new^T.  With a = 1, b = 0 and
 * dst = src this is M' = M A A'^T. */
int flora_oracle_transfer_axpby(float* dst, int64_t ldd, const float* src, int64_t lds,
                                int64_t n, int r, int64_t m,
                                const float* A_old, int64_t lda_old,
                                const float* A_new, int64_t lda_new, double a, double b)
{
    int fail = 0;
    #pragma omp parallel for schedule(static)
    for (int64_t i = 0; i < n; ++i) {
        double* P = (double*)malloc((size_t)m * sizeof(double));
        double* out = (double*)malloc((size_t)r * sizeof(double));
        if (!P || !out) { fail = 1; free(P); free(out); continue; }
        for (int64_t k = 0; k < m; ++k) {
            double acc = 0.0;
            for (int j = 0; j < r; ++j)
                acc += (double)src[i * lds + j] * (double)A_old[(int64_t)j * lda_old + k];
            P[k] = acc;
        }
        for (int j = 0; j < r; ++j) {
            double acc = 0.0;
            for (int64_t k = 0; k < m; ++k)
                acc += P[k] * (double)A_new[(int64_t)j * lda_new + k];
            out[j] = acc;
        }
        for (int j = 0; j < r; ++j)
            dst[i * ldd + j] = (float)(b * (double)dst[i * ldd + j] + a * out[j]);
        free(P); free(out);
    }
    return fail;
}

int flora_oracle_resample_transfer(float* M, int64_t ldm, int64_t n, int r, int64_t m,
                                   const float* A_old, int64_t lda_old,
                                   const float* A_new, int64_t lda_new)
{
    return flora_oracle_transfer_axpby(M, ldm, M, ldm, n, r, m, A_old, lda_old, A_new, lda_new, 1.0, 0.0);
}

void flora_oracle_set_threads(int t)
{
#ifdef _OPENMP
    if (t > 0) omp_set_num_threads(t);
#else
    (void)t;
#endif
}
int flora_oracle_max_threads(void)
{
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}
