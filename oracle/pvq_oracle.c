/*
 * CPU oracle for group-wise Pyramid Vector Quantization (arxiv 2410.16926).
 *
 * TEST INFRASTRUCTURE ONLY.  This file is the slow, plain reference that the
 * CUDA library is compared against.  It shares no code, header, table or
 * constant with the CUDA path, and the product never calls it.
 *
 * Every routine follows one passage of the paper, in the paper's order:
 *   count table        Sec. 2.4, recurrence below the closed form (with the
 *                      last term read as N(D-1,K-1)) and its boundary values
 *   pulses K           Sec. 3.3 Step 2 (largest K whose index fits the budget)
 *   direction          Sec. 2.5 "Quantizing the direction" / Algorithm 1, in
 *                      the floor + greedy single-pulse reading
 *   enumeration        Algorithm 2 (pyramid encoding)
 *   de-enumeration     Algorithm 3 (corrected pyramid decoding)
 *   amplitude          Sec. 2.3 (amplitude = ||w||_2), Sec. 3.3 Step 5 and
 *                      Sec. 3.4 (quantile quantiser on s_g^2 / ||s||^2)
 *   reconstruction     Sec. 2.4 (projection of the pyramid point on the sphere)
 *   16-bit amplitudes  Sec. 4.1 setting: the amplitude itself as IEEE binary16 (scale_bits = 16)
 *   least squares      Sec. 3.3 Step 4 read as the least-squares scale of the unit
 *                      direction, s = w_hat^T w / w_hat^T w_hat (amp_mode = 1)
 *   rotation           Sec. 2.3 "Hadamard coherence processing" / Sec. 3.3 Step 1, along
 *                      the input dimension: x <- (x * s) H_n / sqrt(n) per block of n
 *
 * Integers are multi-word unsigned numbers kept as little-endian arrays of
 * 32-bit limbs and handled one limb at a time with a 64-bit carry.
 * Floating point is IEEE binary32, one rounding per operation (compile with
 * -ffp-contract=off and without -ffast-math).  Sums over a group and over a
 * row use one fixed balanced tree, defined in tree_sum().
 *
 * Parity unpinned by the paper (it prints no value for them): the order of
 * the fp32 roundings and the bit packing of the amplitude indices.  Both are
 * conventions of this codec.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

#define PVQO_MAXW 32 /* limbs per integer: up to 1024-bit indices */

typedef struct {
    uint32_t w[PVQO_MAXW];
} big_t;

/* ---------------------------------------------------------------- big ints */

static void big_zero(big_t *a) { memset(a->w, 0, sizeof a->w); }

static void big_set_u32(big_t *a, uint32_t v) {
    big_zero(a);
    a->w[0] = v;
}

/* a += b ; returns the carry out of the top limb */
static uint32_t big_add(big_t *a, const big_t *b) {
    uint64_t carry = 0;
    for (int i = 0; i < PVQO_MAXW; ++i) {
        uint64_t s = (uint64_t)a->w[i] + b->w[i] + carry;
        a->w[i] = (uint32_t)s;
        carry = s >> 32;
    }
    return (uint32_t)carry;
}

/* a -= b ; caller guarantees a >= b */
static void big_sub(big_t *a, const big_t *b) {
    uint64_t borrow = 0;
    for (int i = 0; i < PVQO_MAXW; ++i) {
        uint64_t d = (uint64_t)a->w[i] - b->w[i] - borrow;
        a->w[i] = (uint32_t)d;
        borrow = (d >> 32) & 1u;
    }
}

/* -1, 0, +1 for a < b, a == b, a > b */
static int big_cmp(const big_t *a, const big_t *b) {
    for (int i = PVQO_MAXW - 1; i >= 0; --i) {
        if (a->w[i] != b->w[i]) return a->w[i] < b->w[i] ? -1 : 1;
    }
    return 0;
}

static int big_is_zero(const big_t *a) {
    for (int i = 0; i < PVQO_MAXW; ++i)
        if (a->w[i]) return 0;
    return 1;
}

/* number of significant bits (0 for zero) */
static int big_bitlen(const big_t *a) {
    for (int i = PVQO_MAXW - 1; i >= 0; --i) {
        if (a->w[i]) {
            int b = 0;
            uint32_t v = a->w[i];
            while (v) {
                ++b;
                v >>= 1;
            }
            return 32 * i + b;
        }
    }
    return 0;
}

/* is a an exact power of two? */
static int big_is_pow2(const big_t *a) {
    int ones = 0;
    for (int i = 0; i < PVQO_MAXW; ++i) {
        uint32_t v = a->w[i];
        while (v) {
            ones += (int)(v & 1u);
            v >>= 1;
        }
    }
    return ones == 1;
}

/* ------------------------------------------------------------- count table */

/*
 * N(n,k) = |P(n,k)| for 0 <= n <= nmax, 0 <= k <= kmax (Sec. 2.4).
 *   N(n,0) = 1 for all n >= 0;  N(0,k) = 0 for all k >= 1;
 *   N(n,k) = N(n-1,k) + N(n,k-1) + N(n-1,k-1).
 * Returns a malloc'ed array indexed [n*(kmax+1)+k], or NULL when a value does
 * not fit PVQO_MAXW limbs.
 */
static big_t *count_table(int nmax, int kmax) {
    size_t stride = (size_t)kmax + 1;
    big_t *t = (big_t *)malloc(sizeof(big_t) * (size_t)(nmax + 1) * stride);
    if (!t) return NULL;
    for (int n = 0; n <= nmax; ++n) {
        for (int k = 0; k <= kmax; ++k) {
            big_t *e = &t[(size_t)n * stride + k];
            if (k == 0) {
                big_set_u32(e, 1u);
            } else if (n == 0) {
                big_zero(e);
            } else {
                uint32_t c = 0;
                *e = t[(size_t)(n - 1) * stride + k];
                c |= big_add(e, &t[(size_t)n * stride + (k - 1)]);
                c |= big_add(e, &t[(size_t)(n - 1) * stride + (k - 1)]);
                if (c) {
                    free(t);
                    return NULL;
                }
            }
        }
    }
    return t;
}

/* Writes N(n,k), n = 0..nmax, k = 0..kmax as W little-endian limbs each.
 * Returns 0, or -1 when an entry needs more than W limbs. */
int pvqo_count_table(int nmax, int kmax, int W, uint32_t *out) {
    if (nmax < 0 || kmax < 0 || W < 1 || W > PVQO_MAXW) return -1;
    big_t *t = count_table(nmax, kmax);
    if (!t) return -1;
    size_t stride = (size_t)kmax + 1;
    int rc = 0;
    for (int n = 0; n <= nmax && rc == 0; ++n) {
        for (int k = 0; k <= kmax; ++k) {
            const big_t *e = &t[(size_t)n * stride + k];
            if (big_bitlen(e) > 32 * W) {
                rc = -1;
                break;
            }
            memcpy(out + ((size_t)n * stride + k) * (size_t)W, e->w, 4u * (size_t)W);
        }
    }
    free(t);
    return rc;
}

/* ceil(log2 N(N,K)): bits needed to hold every code in [0, N(N,K)-1]
 * (Sec. 3.3 Step 7).  -1 on overflow of the oracle's integer width. */
int pvqo_index_bits(int N, int K) {
    if (N < 1 || K < 0) return -1;
    big_t *t = count_table(N, K);
    if (!t) return -1;
    const big_t *e = &t[(size_t)N * ((size_t)K + 1) + K];
    int bl = big_bitlen(e);
    int bits = big_is_pow2(e) ? bl - 1 : bl; /* ceil(log2 v) */
    free(t);
    return bits;
}

/* Sec. 3.3 Step 2: the largest K with N(N,K) <= 2^index_bits, tested on the
 * integers themselves.  0 when not even K = 1 fits; -1 on bad arguments.
 * The search stops at 8191 pulses (N(1,K) = 2 for every K would never end it,
 * and no caller stores more: a coordinate is kept in 16 bits). */
int pvqo_max_pulses(int N, int index_bits) {
    if (N < 1 || index_bits < 1 || index_bits > 32 * (PVQO_MAXW - 1)) return -1;
    int K = 0;
    for (;;) {
        int b = pvqo_index_bits(N, K + 1);
        if (b < 0 || b > index_bits) break;
        ++K;
        if (K >= 8191) break;
    }
    return K;
}

/* --------------------------------------------------------- fp32 primitives */

static float bf16_to_f32(uint16_t h) {
    uint32_t u = (uint32_t)h << 16;
    float f;
    memcpy(&f, &u, 4);
    return f;
}

/* round to nearest, ties to even; NaN stays NaN */
static uint16_t f32_to_bf16_rne(float f) {
    uint32_t u;
    memcpy(&u, &f, 4);
    if ((u & 0x7fffffffu) > 0x7f800000u) return (uint16_t)((u >> 16) | 0x0040u);
    uint32_t lsb = (u >> 16) & 1u;
    u += 0x7fffu + lsb;
    return (uint16_t)(u >> 16);
}

/* IEEE binary16 <-> binary32; to binary16 rounds to nearest, ties to even, overflows to infinity */
static uint16_t f32_to_f16_rne(float f) {
    uint32_t u;
    memcpy(&u, &f, 4);
    uint32_t sign = (u >> 16) & 0x8000u;
    uint32_t a = u & 0x7fffffffu;
    if (a > 0x7f800000u) return (uint16_t)(sign | 0x7e00u);          /* NaN */
    if (a >= 0x47800000u) return (uint16_t)(sign | 0x7c00u);         /* >= 65536: infinity (also from 65520 up, below) */
    if (a < 0x33000000u) return (uint16_t)sign;                      /* below 2^-25: zero */
    int e = (int)(a >> 23) - 127;                                    /* unbiased exponent */
    uint32_t m = (a & 0x7fffffu) | 0x800000u;                        /* 24-bit significand */
    int shift = e >= -14 ? 13 : 13 + (-14 - e);                      /* bits dropped */
    uint32_t kept = m >> shift;
    uint32_t rem = m & ((1u << shift) - 1u);
    uint32_t half = 1u << (shift - 1);
    if (rem > half || (rem == half && (kept & 1u))) kept += 1;
    uint32_t h;
    if (e >= -14)
        h = ((uint32_t)(e + 15) << 10) + (kept - 0x400u);            /* a carry out of the significand moves into the exponent */
    else
        h = kept;                                                     /* subnormal (or the smallest normal after rounding up) */
    if (h >= 0x7c00u) h = 0x7c00u;
    return (uint16_t)(sign | h);
}

static float f16_to_f32(uint16_t h) {
    uint32_t sign = ((uint32_t)h & 0x8000u) << 16;
    uint32_t e = (h >> 10) & 0x1fu, m = h & 0x3ffu;
    float f;
    if (e == 0x1f) {
        uint32_t u = sign | 0x7f800000u | (m << 13);
        memcpy(&f, &u, 4);
        return f;
    }
    if (e == 0) {
        f = (float)m * 5.9604644775390625e-8f;                        /* m * 2^-24, exact */
        return sign ? -f : f;
    }
    uint32_t u = sign | ((e + 112u) << 23) | (m << 13);
    memcpy(&f, &u, 4);
    return f;
}

uint16_t pvqo_f32_to_f16(float f) { return f32_to_f16_rne(f); }
float pvqo_f16_to_f32(uint16_t h) { return f16_to_f32(h); }

/*
 * The one summation order of this codec: a balanced tree over contiguous
 * halves, tree(lo,hi) = tree(lo,mid) + tree(mid,hi), mid the midpoint, each
 * addition rounded to binary32.  n must be a power of two.
 */
static float tree_sum(const float *v, int lo, int hi) {
    if (hi - lo == 1) return v[lo];
    int mid = lo + (hi - lo) / 2;
    float a = tree_sum(v, lo, mid);
    float b = tree_sum(v, mid, hi);
    return a + b;
}

/* tree_sum after padding with +0.0f up to the next power of two */
float pvqo_tree_sum_padded(const float *v, int n) {
    int p = 1;
    while (p < n) p <<= 1;
    float *tmp = (float *)calloc((size_t)p, sizeof(float));
    memcpy(tmp, v, sizeof(float) * (size_t)n);
    float s = tree_sum(tmp, 0, p);
    free(tmp);
    return s;
}

/* ----------------------------------------------------- direction (Alg. 1) */

/*
 * Greedy fix-up of Sec. 2.5: while the pulses do not sum to K, add one pulse
 * where the residual e_i = a_i - m_i is largest (or remove one where it is
 * smallest among m_i > 0); on equal residuals the lowest index wins.  m and e
 * are updated in place.  The loops are bounded so that non-finite input
 * cannot spin.
 */
void pvqo_fixup(int32_t *m, float *e, int N, int K) {
    long sum = 0;
    for (int i = 0; i < N; ++i) sum += m[i];
    long guard = 4L * ((long)N + (long)K) + 16;
    while (sum < K && guard-- > 0) {
        int j = 0;
        for (int i = 1; i < N; ++i)
            if (e[i] > e[j]) j = i;
        m[j] += 1;
        e[j] = e[j] - 1.0f;
        sum += 1;
    }
    while (sum > K && guard-- > 0) {
        int j = -1;
        for (int i = 0; i < N; ++i)
            if (m[i] > 0 && (j < 0 || e[i] < e[j])) j = i;
        if (j < 0) break;
        m[j] -= 1;
        e[j] = e[j] + 1.0f;
        sum -= 1;
    }
}

/*
 * One group: x (N values) -> y on the pyramid P(N,K), sum |y_i| = K.
 * l1 is the tree sum of |x_i| computed by the caller.
 *   scale to the l1 ball of radius K, floor, greedy fix-up, restore signs.
 * A group whose l1 is zero (or so small that K/l1 is not finite) carries no
 * direction; it maps to (K,0,...,0).
 */
static void quantize_direction(const float *x, float l1, int N, int K, int32_t *y) {
    float gsc = (float)K / l1;
    if (!(l1 > 0.0f) || !isfinite(gsc)) {
        for (int i = 0; i < N; ++i) y[i] = 0;
        y[0] = K;
        return;
    }
    float *e = (float *)malloc(sizeof(float) * (size_t)N);
    for (int i = 0; i < N; ++i) {
        float a = fabsf(x[i]) * gsc;
        float f = floorf(a);
        y[i] = (int32_t)f;
        e[i] = a - f;
    }
    pvqo_fixup(y, e, N, K);
    for (int i = 0; i < N; ++i)
        if (signbit(x[i])) y[i] = -y[i];
    free(e);
}

/* the direction step alone, for tests: computes l1 with the tree itself */
void pvqo_quantize_group(const float *x, int N, int K, int32_t *y) {
    float *ax = (float *)malloc(sizeof(float) * (size_t)N);
    for (int i = 0; i < N; ++i) ax[i] = fabsf(x[i]);
    float l1 = tree_sum(ax, 0, N);
    free(ax);
    quantize_direction(x, l1, N, K, y);
}

/* ---------------------------------------------------- enumeration (Alg. 2) */

/*
 * Pyramid point -> code in [0, N(N,K)-1].  With d-1 = N-1-i dimensions left
 * after position i and k pulses left, a non-zero x_i adds
 *   N(d-1,k) + 2 * sum_{j=1}^{|x_i|-1} N(d-1,k-j) + [x_i<0] * N(d-1,k-|x_i|).
 */
static void enumerate(const int32_t *y, int N, int K, const big_t *t, big_t *c) {
    size_t stride = (size_t)K + 1;
    big_zero(c);
    int k = K;
    for (int i = 0; i < N && k != 0; ++i) {
        int d1 = N - 1 - i;
        int mag = y[i] < 0 ? -y[i] : y[i];
        if (mag >= 1) {
            big_add(c, &t[(size_t)d1 * stride + k]);
            for (int j = 1; j <= mag - 1; ++j) {
                big_add(c, &t[(size_t)d1 * stride + (k - j)]);
                big_add(c, &t[(size_t)d1 * stride + (k - j)]);
            }
            if (y[i] < 0) big_add(c, &t[(size_t)d1 * stride + (k - mag)]);
        }
        k -= mag;
    }
}

int pvqo_enumerate(const int32_t *y, int N, int K, int W, uint32_t *code) {
    long s = 0;
    for (int i = 0; i < N; ++i) s += y[i] < 0 ? -y[i] : y[i];
    if (s != K || W < 1 || W > PVQO_MAXW) return -1;
    big_t *t = count_table(N, K);
    if (!t) return -1;
    big_t c;
    enumerate(y, N, K, t, &c);
    free(t);
    if (big_bitlen(&c) > 32 * W) return -1;
    memcpy(code, c.w, 4u * (size_t)W);
    return 0;
}

/* ------------------------------------------------- de-enumeration (Alg. 3) */

/*
 * Code -> pyramid point.  r = c - z is the part of the code not yet
 * explained.  At each position: r < N(d-1,k) means x_i = 0; otherwise take
 * N(d-1,k) off, peel 2N(d-1,k-j) per further pulse, and the last comparison
 * with N(d-1,k-j) gives the sign (the negative branch also takes that count
 * off: the line the original description misses).
 * Returns 1 when the code is valid (r and k both end at zero), else 0.
 */
static int deenumerate(const big_t *c, int N, int K, const big_t *t, int32_t *y) {
    size_t stride = (size_t)K + 1;
    big_t r = *c;
    int k = K;
    for (int i = 0; i < N; ++i) y[i] = 0;
    for (int i = 0; i < N && k > 0; ++i) {
        int d1 = N - 1 - i;
        const big_t *row = &t[(size_t)d1 * stride];
        if (big_cmp(&r, &row[k]) < 0) continue; /* x_i = 0 */
        big_sub(&r, &row[k]);
        int j = 1;
        for (;;) {
            if (j >= k) break; /* only an invalid code can get here and go on */
            big_t two = row[k - j];
            big_add(&two, &row[k - j]);
            if (big_cmp(&r, &two) < 0) break;
            big_sub(&r, &two);
            ++j;
        }
        if (big_cmp(&r, &row[k - j]) < 0) {
            y[i] = j;
        } else {
            y[i] = -j;
            big_sub(&r, &row[k - j]);
        }
        k -= j;
    }
    return (k == 0 && big_is_zero(&r)) ? 1 : 0;
}

int pvqo_deenumerate(const uint32_t *code, int N, int K, int W, int32_t *y) {
    if (W < 1 || W > PVQO_MAXW) return -1;
    big_t *t = count_table(N, K);
    if (!t) return -1;
    big_t c;
    big_zero(&c);
    memcpy(c.w, code, 4u * (size_t)W);
    int ok = deenumerate(&c, N, K, t, y);
    free(t);
    return ok;
}

/* ------------------------------------------------------------ whole matrix */

static size_t scale_row_stride(int64_t G, int scale_bits) {
    size_t bytes = (size_t)((G * scale_bits + 7) / 8);
    return (bytes + 3u) & ~(size_t)3u;
}

size_t pvqo_scale_row_stride(int64_t G, int scale_bits) { return scale_row_stride(G, scale_bits); }

static void put_bits(uint8_t *row, int64_t bitpos, int nbits, uint32_t v) {
    for (int b = 0; b < nbits; ++b) {
        int64_t p = bitpos + b;
        if ((v >> b) & 1u) row[p >> 3] |= (uint8_t)(1u << (p & 7));
    }
}

static uint32_t get_bits(const uint8_t *row, int64_t bitpos, int nbits) {
    uint32_t v = 0;
    for (int b = 0; b < nbits; ++b) {
        int64_t p = bitpos + b;
        v |= (uint32_t)((row[p >> 3] >> (p & 7)) & 1u) << b;
    }
    return v;
}

/*
 * Encode a rows x cols matrix (row-major, leading dimension ld, dtype 0 =
 * fp32, 1 = bf16), groups of N contiguous elements along each row.
 *   per group   l1 = tree(|x_i|), ss = tree(x_i * x_i)
 *   per row     ss_row = padded tree over the groups' ss; row_norm = sqrt(ss_row)
 *   amplitude   u = ss / ss_row (0 when ss_row is not positive);
 *               q = #{ j : u >= edges[j] }, edges = the 2^b - 1 inner quantiles
 *               of Beta(N/2, N(G-1)/2), i.e. floor(CDF(u) 2^b) clamped
 *   direction   quantize_direction, then enumerate
 * Outputs: codes[(r*G+g)*W + w]; scale indices as an LSB-first bit stream per
 * row; row_norm[r].
 */
/*
 * amp_mode 0: the amplitude of a group is ||x_g||_2 (Sec. 2.3), so u = ss / ss_row.
 * amp_mode 1: least squares (Step 4): with y the chosen point and y_hat = y / ||y||_2,
 *             a = y_hat^T x = (sum |y_i| |x_i|) / sqrt(sum y_i^2)   (y_i has the sign of x_i)
 *             with the tree sum over i of the rounded products, and u = (a * a) / ss_row.
 * scale_bits 1..8: q from the quantile edges as above.  scale_bits 16: the amplitude itself,
 *             sqrt(ss) or a, rounded to IEEE binary16, 16 bits per group in the same stream.
 */
int pvqo_encode_amp(const void *x, int dtype, int64_t rows, int64_t cols, int64_t ld, int N, int K,
                    int scale_bits, int amp_mode, int W, const float *edges, uint32_t *codes,
                    uint8_t *scale_idx, float *row_norm, int nthreads) {
    if (N < 1 || (N & (N - 1)) || cols % N || W < 1 || W > PVQO_MAXW) return -1;
    if ((scale_bits < 1 || scale_bits > 8) && scale_bits != 16) return -1;
    if (amp_mode != 0 && amp_mode != 1) return -1;
    big_t *t = count_table(N, K);
    if (!t) return -1;
    {
        /* every code must fit W limbs: N(N,K) <= 2^(32W) */
        const big_t *top = &t[(size_t)N * ((size_t)K + 1) + K];
        int bl = big_bitlen(top);
        if (bl > 32 * W + 1 || (bl == 32 * W + 1 && !big_is_pow2(top))) {
            free(t);
            return -1;
        }
    }
    int64_t G = cols / N;
    int nedges = scale_bits <= 8 ? (1 << scale_bits) - 1 : 0;
    size_t sstride = scale_row_stride(G, scale_bits);
    memset(scale_idx, 0, sstride * (size_t)rows);
#ifdef _OPENMP
    if (nthreads > 0) omp_set_num_threads(nthreads);
#pragma omp parallel for schedule(dynamic, 4)
#endif
    for (int64_t r = 0; r < rows; ++r) {
        float *xs = (float *)malloc(sizeof(float) * (size_t)cols);
        float *tmp = (float *)malloc(sizeof(float) * (size_t)N);
        float *l1 = (float *)malloc(sizeof(float) * (size_t)G);
        float *ss = (float *)malloc(sizeof(float) * (size_t)G);
        int32_t *y = (int32_t *)malloc(sizeof(int32_t) * (size_t)N);
        for (int64_t c = 0; c < cols; ++c) {
            if (dtype == 0)
                xs[c] = ((const float *)x)[r * ld + c];
            else
                xs[c] = bf16_to_f32(((const uint16_t *)x)[r * ld + c]);
        }
        for (int64_t g = 0; g < G; ++g) {
            const float *xg = xs + g * N;
            for (int i = 0; i < N; ++i) tmp[i] = fabsf(xg[i]);
            l1[g] = tree_sum(tmp, 0, N);
            for (int i = 0; i < N; ++i) tmp[i] = xg[i] * xg[i];
            ss[g] = tree_sum(tmp, 0, N);
        }
        float ss_row = pvqo_tree_sum_padded(ss, (int)G);
        row_norm[r] = sqrtf(ss_row);
        for (int64_t g = 0; g < G; ++g) {
            quantize_direction(xs + g * N, l1[g], N, K, y);
            float amp2 = ss[g];          /* squared amplitude */
            float amp = sqrtf(ss[g]);
            if (amp_mode == 1) {
                long ssy = 0;
                for (int i = 0; i < N; ++i) {
                    int32_t m = y[i] < 0 ? -y[i] : y[i];
                    ssy += (long)m * m;
                    tmp[i] = (float)m * fabsf(xs[g * N + i]);
                }
                float dot = tree_sum(tmp, 0, N);
                amp = dot / sqrtf((float)ssy);
                amp2 = amp * amp;
            }
            uint32_t q = 0;
            if (scale_bits == 16) {
                q = f32_to_f16_rne(amp);
            } else {
                float u = ss_row > 0.0f ? amp2 / ss_row : 0.0f;
                for (int j = 0; j < nedges; ++j)
                    if (u >= edges[j]) ++q;
            }
            put_bits(scale_idx + sstride * (size_t)r, g * scale_bits, scale_bits, q);
            big_t c;
            enumerate(y, N, K, t, &c);
            memcpy(codes + ((size_t)r * (size_t)G + (size_t)g) * (size_t)W, c.w, 4u * (size_t)W);
        }
        free(xs);
        free(tmp);
        free(l1);
        free(ss);
        free(y);
    }
    free(t);
    return 0;
}

int pvqo_encode(const void *x, int dtype, int64_t rows, int64_t cols, int64_t ld, int N, int K,
                int scale_bits, int W, const float *edges, uint32_t *codes, uint8_t *scale_idx,
                float *row_norm, int nthreads) {
    return pvqo_encode_amp(x, dtype, rows, cols, ld, N, K, scale_bits, 0, W, edges, codes, scale_idx, row_norm,
                           nthreads);
}

/*
 * Decode to bf16.  Per group: de-enumerate; ssy = sum y_i^2 (exact);
 *   amp = row_norm * levels[q]           (levels = sqrt of the bin midpoints' quantiles)
 *   s   = amp / sqrt((float)ssy)         (point on the unit sphere times amplitude)
 *   out_i = bf16_rne((float)y_i * s)
 * An invalid code (>= N(N,K)) gives an all-zero group and sets bit 0 of
 * *status.
 */
int pvqo_decode(const uint32_t *codes, const uint8_t *scale_idx, const float *row_norm, int64_t rows,
                int64_t cols, int N, int K, int scale_bits, int W, const float *levels,
                uint16_t *out, int64_t ld_out, uint32_t *status, int nthreads) {
    if (N < 1 || (N & (N - 1)) || cols % N || W < 1 || W > PVQO_MAXW) return -1;
    if ((scale_bits < 1 || scale_bits > 8) && scale_bits != 16) return -1;
    big_t *t = count_table(N, K);
    if (!t) return -1;
    int64_t G = cols / N;
    size_t sstride = scale_row_stride(G, scale_bits);
    uint32_t bad = 0;
#ifdef _OPENMP
    if (nthreads > 0) omp_set_num_threads(nthreads);
#pragma omp parallel for schedule(dynamic, 4) reduction(| : bad)
#endif
    for (int64_t r = 0; r < rows; ++r) {
        int32_t *y = (int32_t *)malloc(sizeof(int32_t) * (size_t)N);
        for (int64_t g = 0; g < G; ++g) {
            big_t c;
            big_zero(&c);
            memcpy(c.w, codes + ((size_t)r * (size_t)G + (size_t)g) * (size_t)W, 4u * (size_t)W);
            int ok = deenumerate(&c, N, K, t, y);
            uint16_t *o = out + r * ld_out + g * N;
            if (!ok) {
                bad |= 1u;
                for (int i = 0; i < N; ++i) o[i] = 0;
                continue;
            }
            uint32_t q = get_bits(scale_idx + sstride * (size_t)r, g * scale_bits, scale_bits);
            long ssy = 0;
            for (int i = 0; i < N; ++i) ssy += (long)y[i] * y[i];
            /* scale_bits 16: q is the amplitude itself as binary16 */
            float amp = scale_bits == 16 ? f16_to_f32((uint16_t)q) : row_norm[r] * levels[q];
            float s = amp / sqrtf((float)ssy);
            for (int i = 0; i < N; ++i) o[i] = f32_to_bf16_rne((float)y[i] * s);
        }
        free(y);
    }
    free(t);
    if (status) *status |= bad;
    return 0;
}

/* ------------------------------------------------ rotation (Sec. 2.3, Step 1) */

/*
 * Random-sign Hadamard rotation along the columns, independently on every
 * contiguous block of `block` columns of every row (block a power of two
 * dividing cols): with s the +-1 sign vector of length `block` (shared by all
 * blocks and rows) and H the Sylvester-Walsh-Hadamard matrix,
 *     out = (x * s) H / sqrt(block).
 * H is applied as log2(block) stages of butterflies with strides 1, 2, 4, ...:
 * (a, b) -> (a + b, a - b) on elements j and j + stride, each sum rounded to
 * binary32; the scale is the binary32 nearest to 1/sqrt(block), applied last
 * with one multiplication.  That order is a convention of this codec (parity
 * unpinned by the paper); the result is pinned to H by exact cases.
 * dtype 0 = fp32 in, 1 = bf16 in; out is fp32 [rows][cols].
 */
int pvqo_rotate(const void *x, int dtype, int64_t rows, int64_t cols, int64_t ld, int block,
                const float *signs, float *out) {
    if (block < 1 || (block & (block - 1)) || cols % block) return -1;
    float scale = (float)(1.0 / sqrt((double)block));
    for (int64_t r = 0; r < rows; ++r) {
        float *o = out + r * cols;
        for (int64_t c = 0; c < cols; ++c) {
            float v = dtype == 0 ? ((const float *)x)[r * ld + c]
                                 : bf16_to_f32(((const uint16_t *)x)[r * ld + c]);
            o[c] = v * signs[c % block];
        }
        for (int64_t b0 = 0; b0 < cols; b0 += block) {
            float *v = o + b0;
            for (int h = 1; h < block; h <<= 1) {
                for (int j0 = 0; j0 < block; j0 += 2 * h) {
                    for (int j = j0; j < j0 + h; ++j) {
                        float a = v[j], b = v[j + h];
                        v[j] = a + b;
                        v[j + h] = a - b;
                    }
                }
            }
            for (int j = 0; j < block; ++j) v[j] = v[j] * scale;
        }
    }
    return 0;
}

int pvqo_threads(void) {
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}
