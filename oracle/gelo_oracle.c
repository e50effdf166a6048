/*
 * GELO oracle -- TEST INFRASTRUCTURE ONLY.
 *
 * A plain, slow, fp64 CPU statement of what the obfuscated Q/K/V offload
 * computes, written from the paper (Section 3.2 "Core Algorithm", Eq. 1-4, and
 * the two Gram-leak mitigations, Eq. 7-9).  Nothing in the product may call it;
 * only tests, the smoke check and the benchmark's CPU-baseline leg do.  It
 * shares no code with the CUDA library.
 *
 * Everything is naive loops on row-major double arrays.  The only parallelism
 * is an OpenMP "parallel for" over independent output rows.
 *
 * Where the paper is silent the readings are:
 *   - random numbers: Philox4x32 with 10 rounds (Salmon et al., SC'11), one
 *     32-bit word per matrix element, Box-Muller on word pairs (layout below);
 *   - orthogonal A: Q of the Householder QR of a Gaussian matrix, columns
 *     flipped so that diag(R) > 0 (the unique QR factor);
 *   - non-orthogonal A (Mitigation 1): A = Q0 + gamma * G1, G1 ~ N(0, 1/m),
 *     accepted when its 2-norm condition number is <= the bound;
 *   - shield rows (Mitigation 2): S = (scale * median_i ||h_i||_2 / sqrt(d)) * G_S.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

/* ------------------------------------------------------------------ */
/* Philox4x32-10 (SC'11, "Parallel Random Numbers: As Easy as 1, 2, 3") */
/* ------------------------------------------------------------------ */

static void philox_round(uint32_t c[4], uint32_t k0, uint32_t k1)
{
    const uint64_t p0 = (uint64_t)0xD2511F53u * c[0];
    const uint64_t p1 = (uint64_t)0xCD9E8D57u * c[2];
    const uint32_t n0 = (uint32_t)(p1 >> 32) ^ c[1] ^ k0;
    const uint32_t n1 = (uint32_t)p1;
    const uint32_t n2 = (uint32_t)(p0 >> 32) ^ c[3] ^ k1;
    const uint32_t n3 = (uint32_t)p0;
    c[0] = n0; c[1] = n1; c[2] = n2; c[3] = n3;
}

void oracle_philox4x32_10(const uint32_t ctr[4], const uint32_t key[2], uint32_t out[4])
{
    uint32_t c[4] = { ctr[0], ctr[1], ctr[2], ctr[3] };
    uint32_t k0 = key[0], k1 = key[1];
    for (int r = 0; r < 10; ++r) {
        philox_round(c, k0, k1);
        k0 += 0x9E3779B9u;
        k1 += 0xBB67AE85u;
    }
    memcpy(out, c, sizeof c);
}

/*
 * Word of element e of a matrix drawn from (seed, stream, attempt):
 * block q = e / 4 gives counter (lo32(q), hi32(q), stream, attempt),
 * key (lo32(seed), hi32(seed)); the element takes word e % 4 of the block.
 */
void oracle_philox_words(uint64_t seed, uint32_t stream, uint32_t attempt,
                         uint64_t first, uint64_t count, uint32_t* out)
{
    const uint32_t key[2] = { (uint32_t)seed, (uint32_t)(seed >> 32) };
    for (uint64_t i = 0; i < count; ++i) {
        const uint64_t e = first + i, q = e >> 2;
        const uint32_t ctr[4] = { (uint32_t)q, (uint32_t)(q >> 32), stream, attempt };
        uint32_t w[4];
        oracle_philox4x32_10(ctr, key, w);
        out[i] = w[e & 3];
    }
}

/* 23-bit uniform strictly inside (0,1): u = ((w >> 9) + 1/2) * 2^-23.  Every such u is
 * exactly representable in binary32, so a single-precision sampler sees the same u. */
static double uniform_from_word(uint32_t w)
{
    return ((double)(w >> 9) + 0.5) * (1.0 / 8388608.0);
}

/*
 * Standard normals, one per element.  Words (0,1) and (2,3) of a block form
 * Box-Muller pairs (u_a, u_b): the even word's element is r*cos(2 pi u_b), the
 * odd word's is r*sin(2 pi u_b), r = sqrt(-2 ln u_a).
 */
void oracle_gaussian(uint64_t seed, uint32_t stream, uint32_t attempt,
                     uint64_t first, uint64_t count, double* out)
{
    const uint32_t key[2] = { (uint32_t)seed, (uint32_t)(seed >> 32) };
    const double two_pi = 6.283185307179586476925286766559;
    for (uint64_t i = 0; i < count; ++i) {
        const uint64_t e = first + i, q = e >> 2;
        const uint32_t ctr[4] = { (uint32_t)q, (uint32_t)(q >> 32), stream, attempt };
        uint32_t w[4];
        oracle_philox4x32_10(ctr, key, w);
        const int pair = (int)((e & 3) >> 1);
        const double ua = uniform_from_word(w[2 * pair]);
        const double ub = uniform_from_word(w[2 * pair + 1]);
        const double r = sqrt(-2.0 * log(ua));
        out[i] = (e & 1) ? r * sin(two_pi * ub) : r * cos(two_pi * ub);
    }
}

/* ------------------------------------------------------------------ */
/* Dense products                                                      */
/* ------------------------------------------------------------------ */

/* C (M x N) = A (M x K) * B (K x N), all row-major with the given strides. */
void oracle_matmul(int64_t M, int64_t N, int64_t K,
                   const double* A, int64_t lda, const double* B, int64_t ldb,
                   double* C, int64_t ldc)
{
#pragma omp parallel for schedule(static)
    for (int64_t i = 0; i < M; ++i) {
        double* c = C + i * ldc;
        for (int64_t j = 0; j < N; ++j) c[j] = 0.0;
        for (int64_t l = 0; l < K; ++l) {
            const double a = A[i * lda + l];
            const double* b = B + l * ldb;
            for (int64_t j = 0; j < N; ++j) c[j] += a * b[j];
        }
    }
}

/* Selected rows of H * W: out[r, :] = H[rows[r], :] * W  (Eq. 4's right side). */
void oracle_rows_times_w(int64_t nrows, const int64_t* rows, int64_t d, int64_t p,
                         const double* H, const double* W, double* out)
{
#pragma omp parallel for schedule(static)
    for (int64_t r = 0; r < nrows; ++r) {
        const double* h = H + rows[r] * d;
        double* o = out + r * p;
        for (int64_t j = 0; j < p; ++j) o[j] = 0.0;
        for (int64_t l = 0; l < d; ++l) {
            const double a = h[l];
            const double* w = W + l * p;
            for (int64_t j = 0; j < p; ++j) o[j] += a * w[j];
        }
    }
}

/* ------------------------------------------------------------------ */
/* Householder QR:  G = Q R,  diag(R) > 0                              */
/* ------------------------------------------------------------------ */

/*
 * Unblocked Householder QR of the m x m matrix G (row-major).  Q and R are
 * m x m row-major outputs.  Column j of Q and row j of R are negated when
 * R_jj < 0, which makes the factorisation the unique one with positive
 * diagonal.  Returns 0, or -1 if memory ran out.
 */
int oracle_householder_qr(int64_t m, const double* G, double* Q, double* R)
{
    double* v = (double*)malloc((size_t)m * sizeof(double));
    double* w = (double*)malloc((size_t)m * sizeof(double));
    if (!v || !w) { free(v); free(w); return -1; }
    memcpy(R, G, (size_t)m * m * sizeof(double));
    for (int64_t i = 0; i < m; ++i)
        for (int64_t j = 0; j < m; ++j) Q[i * m + j] = (i == j) ? 1.0 : 0.0;

    for (int64_t j = 0; j < m; ++j) {
        /* reflector H_j = I - 2 v v^T / (v^T v) that maps R[j:, j] to -sign(x0) ||x|| e_0 */
        double nrm2 = 0.0;
        for (int64_t i = j; i < m; ++i) nrm2 += R[i * m + j] * R[i * m + j];
        const double nrm = sqrt(nrm2);
        if (nrm == 0.0) continue;
        const double x0 = R[j * m + j];
        const double alpha = (x0 >= 0.0) ? -nrm : nrm;
        for (int64_t i = 0; i < j; ++i) v[i] = 0.0;
        for (int64_t i = j; i < m; ++i) v[i] = R[i * m + j];
        v[j] -= alpha;
        double vtv = 0.0;
        for (int64_t i = j; i < m; ++i) vtv += v[i] * v[i];
        if (vtv == 0.0) continue;
        /* R <- H_j R */
        for (int64_t c = 0; c < m; ++c) w[c] = 0.0;
        for (int64_t i = j; i < m; ++i)
            for (int64_t c = j; c < m; ++c) w[c] += v[i] * R[i * m + c];
#pragma omp parallel for schedule(static)
        for (int64_t i = j; i < m; ++i)
            for (int64_t c = j; c < m; ++c) R[i * m + c] -= (2.0 / vtv) * v[i] * w[c];
        /* Q <- Q H_j */
#pragma omp parallel for schedule(static)
        for (int64_t r = 0; r < m; ++r) {
            double s = 0.0;
            for (int64_t i = j; i < m; ++i) s += Q[r * m + i] * v[i];
            s *= 2.0 / vtv;
            for (int64_t i = j; i < m; ++i) Q[r * m + i] -= s * v[i];
        }
    }
    for (int64_t j = 0; j < m; ++j) {
        for (int64_t i = j + 1; i < m; ++i) R[i * m + j] = 0.0;
        if (R[j * m + j] < 0.0) {
            for (int64_t c = j; c < m; ++c) R[j * m + c] = -R[j * m + c];
            for (int64_t r = 0; r < m; ++r) Q[r * m + j] = -Q[r * m + j];
        }
    }
    free(v); free(w);
    return 0;
}

/* ------------------------------------------------------------------ */
/* Inverse by Gaussian elimination with partial pivoting               */
/* ------------------------------------------------------------------ */

/*
 * Ainv = A^-1 for row-major m x m A.  Elimination is carried out on [A | I];
 * at step j the row with the largest |entry| in column j (first such row on a
 * tie) is swapped up.  Returns 0, 1 if a pivot is exactly zero, -1 on
 * allocation failure.
 */
int oracle_lu_inverse(int64_t m, const double* A, double* Ainv)
{
    double* M = (double*)malloc((size_t)m * m * sizeof(double));
    if (!M) return -1;
    memcpy(M, A, (size_t)m * m * sizeof(double));
    for (int64_t i = 0; i < m; ++i)
        for (int64_t j = 0; j < m; ++j) Ainv[i * m + j] = (i == j) ? 1.0 : 0.0;

    for (int64_t j = 0; j < m; ++j) {
        int64_t piv = j;
        double best = fabs(M[j * m + j]);
        for (int64_t i = j + 1; i < m; ++i)
            if (fabs(M[i * m + j]) > best) { best = fabs(M[i * m + j]); piv = i; }
        if (best == 0.0) { free(M); return 1; }
        if (piv != j) {
            for (int64_t c = 0; c < m; ++c) {
                double t = M[j * m + c]; M[j * m + c] = M[piv * m + c]; M[piv * m + c] = t;
                t = Ainv[j * m + c]; Ainv[j * m + c] = Ainv[piv * m + c]; Ainv[piv * m + c] = t;
            }
        }
        const double inv = 1.0 / M[j * m + j];
#pragma omp parallel for schedule(static)
        for (int64_t i = j + 1; i < m; ++i) {
            const double f = M[i * m + j] * inv;
            if (f == 0.0) continue;
            for (int64_t c = j; c < m; ++c) M[i * m + c] -= f * M[j * m + c];
            for (int64_t c = 0; c < m; ++c) Ainv[i * m + c] -= f * Ainv[j * m + c];
        }
    }
    /* back substitution: U X = (L^-1 P) */
    for (int64_t j = m - 1; j >= 0; --j) {
        const double inv = 1.0 / M[j * m + j];
        for (int64_t c = 0; c < m; ++c) Ainv[j * m + c] *= inv;
#pragma omp parallel for schedule(static)
        for (int64_t i = 0; i < j; ++i) {
            const double f = M[i * m + j];
            if (f == 0.0) continue;
            for (int64_t c = 0; c < m; ++c) Ainv[i * m + c] -= f * Ainv[j * m + c];
        }
    }
    free(M);
    return 0;
}

/* ------------------------------------------------------------------ */
/* 2-norm condition number (Mitigation 1: kappa(A) below a bound, 100)   */
/* ------------------------------------------------------------------ */

/*
 * Singular values by one-sided (Hestenes) Jacobi: columns of a copy of A are
 * rotated pairwise until mutually orthogonal; their norms are then the
 * singular values.  Writes sigma_max and sigma_min and returns the number of
 * sweeps used (negative on allocation failure).
 */
int oracle_singular_extremes(int64_t m, const double* A, double* smax, double* smin)
{
    double* B = (double*)malloc((size_t)m * m * sizeof(double));
    if (!B) return -1;
    /* work on the transpose so that "columns" are contiguous rows of B */
    for (int64_t i = 0; i < m; ++i)
        for (int64_t j = 0; j < m; ++j) B[j * m + i] = A[i * m + j];
    int sweep = 0;
    for (; sweep < 60; ++sweep) {
        double off = 0.0;
        for (int64_t p = 0; p < m - 1; ++p) {
            for (int64_t q = p + 1; q < m; ++q) {
                double* bp = B + p * m; double* bq = B + q * m;
                double app = 0.0, aqq = 0.0, apq = 0.0;
                for (int64_t i = 0; i < m; ++i) {
                    app += bp[i] * bp[i]; aqq += bq[i] * bq[i]; apq += bp[i] * bq[i];
                }
                if (apq == 0.0) continue;
                const double rel = fabs(apq) / sqrt(app * aqq);
                if (rel > off) off = rel;
                if (rel < 1e-15) continue;
                const double zeta = (aqq - app) / (2.0 * apq);
                const double t = ((zeta >= 0.0) ? 1.0 : -1.0) / (fabs(zeta) + sqrt(1.0 + zeta * zeta));
                const double c = 1.0 / sqrt(1.0 + t * t), s = c * t;
                for (int64_t i = 0; i < m; ++i) {
                    const double x = bp[i], y = bq[i];
                    bp[i] = c * x - s * y;
                    bq[i] = s * x + c * y;
                }
            }
        }
        if (off < 1e-14) { ++sweep; break; }
    }
    double hi = 0.0, lo = INFINITY;
    for (int64_t p = 0; p < m; ++p) {
        double s2 = 0.0;
        for (int64_t i = 0; i < m; ++i) s2 += B[p * m + i] * B[p * m + i];
        const double s = sqrt(s2);
        if (s > hi) hi = s;
        if (s < lo) lo = s;
    }
    *smax = hi; *smin = lo;
    free(B);
    return sweep;
}

/* ------------------------------------------------------------------ */
/* Sampling the secret mixing matrix (Section 3.2, step 1.2)           */
/* ------------------------------------------------------------------ */

/*
 * kind 0: orthogonal.  G0 ~ N(0,1)^{m x m} from stream 0; A = Q (diag R > 0);
 *         Ainv = A^T.
 * kind 1: non-orthogonal.  A = Q0 + gamma * G1 / sqrt(m), Q0 as above, G1 from
 *         stream 1; Ainv by elimination.
 * Both use the given attempt number in the Philox counter.  Returns 0 on
 * success.
 */
int oracle_sample_mixing(int64_t m, int kind, uint64_t seed, uint32_t attempt,
                         double gamma, double* A, double* Ainv)
{
    const size_t mm = (size_t)m * m;
    double* G = (double*)malloc(mm * sizeof(double));
    double* R = (double*)malloc(mm * sizeof(double));
    if (!G || !R) { free(G); free(R); return -1; }
    oracle_gaussian(seed, 0u, attempt, 0, mm, G);
    int rc = oracle_householder_qr(m, G, A, R);
    if (rc == 0 && kind == 0) {
        for (int64_t i = 0; i < m; ++i)
            for (int64_t j = 0; j < m; ++j) Ainv[i * m + j] = A[j * m + i];
    } else if (rc == 0) {
        oracle_gaussian(seed, 1u, attempt, 0, mm, G);
        const double s = gamma / sqrt((double)m);
        for (size_t i = 0; i < mm; ++i) A[i] += s * G[i];
        rc = oracle_lu_inverse(m, A, Ainv);
    }
    free(G); free(R);
    return rc;
}

/* ------------------------------------------------------------------ */
/* Shield rows (Mitigation 2, Eq. 7-8)                                 */
/* ------------------------------------------------------------------ */

static int cmp_double(const void* a, const void* b)
{
    const double x = *(const double*)a, y = *(const double*)b;
    return (x > y) - (x < y);
}

/* Median of the Euclidean norms of the n rows of H (n x d); even n: mean of the middle two. */
double oracle_median_row_norm(int64_t n, int64_t d, const double* H)
{
    if (n <= 0) return 0.0;
    double* nr = (double*)malloc((size_t)n * sizeof(double));
    if (!nr) return NAN;
    for (int64_t i = 0; i < n; ++i) {
        double s = 0.0;
        for (int64_t j = 0; j < d; ++j) s += H[i * d + j] * H[i * d + j];
        nr[i] = sqrt(s);
    }
    qsort(nr, (size_t)n, sizeof(double), cmp_double);
    const double med = (n & 1) ? nr[n / 2] : 0.5 * (nr[n / 2 - 1] + nr[n / 2]);
    free(nr);
    return med;
}

/* S (k x d) = (scale * median row norm of H / sqrt(d)) * G_S, G_S from stream 2. */
void oracle_shield_rows(int64_t n, int64_t d, int64_t k, const double* H, double scale,
                        uint64_t seed, double* S)
{
    if (k <= 0) return;
    const double f = scale * oracle_median_row_norm(n, d, H) / sqrt((double)d);
    oracle_gaussian(seed, 2u, 0u, 0, (uint64_t)k * (uint64_t)d, S);
    for (int64_t i = 0; i < k * d; ++i) S[i] *= f;
}

/*
 * Student-t shield rows (Section 4.4.1, Table 9 lists "Student-t" beside Gaussian shields without
 * degrees of freedom or scaling; reading: nu is a parameter, the draws are standardised to unit
 * variance so that the same global factor gives the same expected row energy as Gaussian shields).
 * Element e owns B = 4 * ceil((nu + 1) / 4) consecutive positions of the Gaussian stream
 * (seed, stream 2, attempt word = nu), starting at e * B:
 *     t = g_0 / sqrt((g_1^2 + ... + g_nu^2) / nu),   x = t * sqrt((nu - 2) / nu),   3 <= nu <= 63.
 */
void oracle_student_t(uint64_t seed, uint32_t nu, uint64_t first, uint64_t count, double* out)
{
    const uint64_t B = 4u * (((uint64_t)nu + 1u + 3u) / 4u);
    double g[64];
    for (uint64_t i = 0; i < count; ++i) {
        const uint64_t e = first + i;
        oracle_gaussian(seed, 2u, nu, e * B, (uint64_t)nu + 1u, g);
        double chi = 0.0;
        for (uint32_t j = 1; j <= nu; ++j) chi += g[j] * g[j];
        out[i] = g[0] / sqrt(chi / (double)nu) * sqrt(((double)nu - 2.0) / (double)nu);
    }
}

/* S (k x d) = (scale * median row norm of H / sqrt(d)) * X, X standardised Student-t draws. */
void oracle_shield_rows_t(int64_t n, int64_t d, int64_t k, const double* H, double scale,
                          uint64_t seed, uint32_t nu, double* S)
{
    if (k <= 0) return;
    const double f = scale * oracle_median_row_norm(n, d, H) / sqrt((double)d);
    oracle_student_t(seed, nu, 0, (uint64_t)k * (uint64_t)d, S);
    for (int64_t i = 0; i < k * d; ++i) S[i] *= f;
}

/*
 * FP8 operands for the offloaded product (the paper's Limitations / Future Work name FP8 beside FP16;
 * reading: the product of Eq. 2, the one the untrusted accelerator runs, takes U and W in the OCP
 * 8-bit format E4M3 -- sign, 4 exponent bits with bias 7, 3 mantissa bits, no infinities, largest
 * finite value 448, subnormals down to 2^-9 -- with ONE fp32 scale per tensor, s = max|x| / 448,
 * code = round-to-nearest-even(x / s) with the division in binary32, and Y' = (s_U s_W) (U8 W8)).
 */
double oracle_e4m3_decode(uint8_t code)
{
    const int sign = code >> 7, e = (code >> 3) & 15, f = code & 7;
    double v;
    if (e == 15 && f == 7) v = NAN;                               /* the one NaN pattern per sign */
    else if (e == 0) v = ldexp((double)f, -9);                    /* subnormal: f * 2^-3 * 2^-6 */
    else v = ldexp(1.0 + (double)f / 8.0, e - 7);
    return sign ? -v : v;
}

/* Nearest E4M3 value to x (ties to the even mantissa), saturating at +-448. */
uint8_t oracle_e4m3_encode(float x)
{
    const uint8_t sign = signbit(x) ? 0x80u : 0u;
    double a = fabs((double)x);
    if (isnan(a)) return (uint8_t)(sign | 0x7Fu);
    if (a >= 448.0) return (uint8_t)(sign | 0x7Eu);               /* 448 = 1.75 * 2^8 */
    /* spacing of the representable values around a: 2^(e-3) for normals (e >= -6), 2^-9 below 2^-6 */
    int e;
    frexp(a, &e);                                                  /* a = m * 2^e, 0.5 <= m < 1  ->  exponent e - 1 */
    int ex = e - 1;
    if (ex < -6) ex = -6;
    const double q = ldexp(1.0, ex - 3);
    double n = nearbyint(a / q);                                   /* default rounding mode: ties to even */
    double r = n * q;
    if (r >= 448.0) return (uint8_t)(sign | 0x7Eu);
    if (r == 0.0) return sign;
    int e2;
    const double m2 = frexp(r, &e2);                               /* r = m2 * 2^e2 */
    int ex2 = e2 - 1;
    if (ex2 < -6) return (uint8_t)(sign | (uint8_t)nearbyint(r / ldexp(1.0, -9)));
    const int f = (int)nearbyint((m2 * 2.0 - 1.0) * 8.0);
    return (uint8_t)(sign | ((ex2 + 7) << 3) | f);
}

/* scale = max|x| / 448 in binary32 (1 if the tensor is all zero); codes[i] = encode(x[i] / scale), binary32 division */
float oracle_quantize_e4m3(int64_t count, const float* x, uint8_t* codes)
{
    float amax = 0.0f;
    for (int64_t i = 0; i < count; ++i) { const float a = fabsf(x[i]); if (a > amax) amax = a; }
    const float scale = amax > 0.0f ? amax / 448.0f : 1.0f;
    for (int64_t i = 0; i < count; ++i) codes[i] = oracle_e4m3_encode(x[i] / scale);
    return scale;
}

/* ------------------------------------------------------------------ */
/* The chain (Eq. 1-3 with H_full = [H; S])                            */
/* ------------------------------------------------------------------ */

/*
 * Given A, Ainv (m x m, m = n + k), H (n x d), S (k x d), W (d x p):
 *   U  = A [H; S]          (m x d)   Eq. 1 / Eq. 8
 *   Yp = U W               (m x p)   Eq. 2
 *   Y  = (Ainv Yp)[0:n, :] (n x p)   Eq. 3, shield rows dropped
 * U and Yp are optional outputs (may be NULL).  Returns 0 or -1.
 */
int oracle_chain(int64_t n, int64_t k, int64_t d, int64_t p,
                 const double* A, const double* Ainv, const double* H, const double* S,
                 const double* W, double* U_out, double* Yp_out, double* Y)
{
    const int64_t m = n + k;
    double* Hf = (double*)malloc((size_t)m * d * sizeof(double));
    double* U = U_out ? U_out : (double*)malloc((size_t)m * d * sizeof(double));
    double* Yp = Yp_out ? Yp_out : (double*)malloc((size_t)m * p * sizeof(double));
    double* Yf = (double*)malloc((size_t)m * p * sizeof(double));
    int rc = -1;
    if (Hf && U && Yp && Yf) {
        memcpy(Hf, H, (size_t)n * d * sizeof(double));
        if (k > 0) memcpy(Hf + (size_t)n * d, S, (size_t)k * d * sizeof(double));
        oracle_matmul(m, d, m, A, m, Hf, d, U, d);
        oracle_matmul(m, p, d, U, d, W, p, Yp, p);
        oracle_matmul(m, p, m, Ainv, m, Yp, p, Yf, p);
        memcpy(Y, Yf, (size_t)n * p * sizeof(double));
        rc = 0;
    }
    free(Hf); free(Yf);
    if (!U_out) free(U);
    if (!Yp_out) free(Yp);
    return rc;
}
