/*
 * ogq_oracle.c -- TEST INFRASTRUCTURE, NOT A PRODUCT PATH.
 *
 * A plain, slow, single-threaded CPU statement of what the quantization path
 * of "Optimal Gradient Quantization Condition for Communication-Efficient
 * Distributed Training" computes: per-tensor level solvers for BinGrad-b,
 * BinGrad-pb and ORQ, the three quantizers, a bit-packing format and the
 * decode-and-sum step; then gradient clipping, an entropy-dense (base-s) wire
 * format, the quantization error and refinement sweeps over the greedy ORQ
 * levels.  Arithmetic is fp64 (sums in long double) on fp32
 * inputs, except the one rounding decision that is defined in fp32 (see
 * ogq_oracle_quantize).  It shares no code with the CUDA library and is only
 * called from the tests, the smoke check and the benchmark's CPU baseline.
 *
 * Every function is pinned by tests that do not call it to produce their own
 * expected values (closed forms, brute force on tiny inputs, invariants and
 * published known-answer vectors), so there is no "parity unpinned" function
 * in this file.
 *
 * Build: gcc -O2 -std=c11 -ffp-contract=off -fexcess-precision=standard
 *            -shared -fPIC ogq_oracle.c -o libogq_oracle.so -lm
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

#define OGQ_ST_EMPTY 1
#define OGQ_ST_NONFINITE 2
#define OGQ_ST_CONSTANT 4
#define OGQ_ST_ITER_CAP 8

/* ------------------------------------------------------------------------ */
/* Statistics of one tensor: n, sum, min, max, sum of magnitudes.            */
/* Corollary 1 makes min and max the end levels of ORQ; the mean is the      */
/* BinGrad-b threshold suggested after Eq. (bingrad-b optimal condition).    */
/* out = {sum, min, max, abs_sum}; returns status bits.                      */
/* ------------------------------------------------------------------------ */
int ogq_oracle_stats(const float *v, int64_t n, double *out)
{
    long double s = 0.0L, sa = 0.0L;
    double mn = INFINITY, mx = -INFINITY;
    int st = 0;
    if (n <= 0) {
        out[0] = out[1] = out[2] = out[3] = 0.0;
        return OGQ_ST_EMPTY;
    }
    for (int64_t i = 0; i < n; ++i) {
        double x = (double)v[i];
        if (!isfinite(x)) st |= OGQ_ST_NONFINITE;
        s += x;
        sa += fabs(x);
        if (x < mn) mn = x;
        if (x > mx) mx = x;
    }
    if (mn == mx) st |= OGQ_ST_CONSTANT;
    out[0] = (double)s;
    out[1] = mn;
    out[2] = mx;
    out[3] = (double)sa;
    return st;
}

/* ------------------------------------------------------------------------ */
/* BinGrad-b levels, Eq. (bingrad-b optimal condition) and the paragraph     */
/* after it: b_{-1} and b_1 are the means of {v < b_0} and {v >= b_0}; b_0   */
/* starts at the mean of the tensor.  With lloyd_iters = I > 0 the first     */
/* equation b_0 = (b_{-1} + b_1)/2 is then applied I times, each followed by */
/* recomputing the two means, stopping early once the partition no longer    */
/* changes (then all three equations hold).  b_0 is an fp32 number at every  */
/* step because it is the threshold the quantizer compares fp32 values with. */
/* levels2 = {b_{-1}, b_1}; returns status bits.                             */
/* ------------------------------------------------------------------------ */
int ogq_oracle_levels_bingrad_b(const float *v, int64_t n, int lloyd_iters,
                                float *levels2, float *thresh)
{
    int st = 0;
    if (n <= 0) {
        levels2[0] = levels2[1] = 0.0f;
        *thresh = 0.0f;
        return OGQ_ST_EMPTY;
    }
    long double s = 0.0L;
    for (int64_t i = 0; i < n; ++i) {
        if (!isfinite((double)v[i])) st |= OGQ_ST_NONFINITE;
        s += (double)v[i];
    }
    float b0 = (float)(double)(s / (long double)n);
    double m_lo = 0.0, m_hi = 0.0;
    int64_t prev_lo = -1;
    int converged = 0;
    for (int it = 0;; ++it) {
        long double s_lo = 0.0L, s_hi = 0.0L;
        int64_t c_lo = 0, c_hi = 0;
        for (int64_t i = 0; i < n; ++i) {
            if (v[i] < b0) {
                s_lo += (double)v[i];
                ++c_lo;
            } else {
                s_hi += (double)v[i];
                ++c_hi;
            }
        }
        if (c_lo == 0 || c_hi == 0) {
            /* one side is empty: the tensor is (numerically) constant */
            double m = (double)((c_lo == 0) ? s_hi / (long double)c_hi : s_lo / (long double)c_lo);
            m_lo = m_hi = m;
            st |= OGQ_ST_CONSTANT;
            converged = 1;
            break;
        }
        m_lo = (double)(s_lo / (long double)c_lo);
        m_hi = (double)(s_hi / (long double)c_hi);
        if (c_lo == prev_lo) {
            converged = 1;
            break;
        }
        if (it >= lloyd_iters) break;
        prev_lo = c_lo;
        b0 = (float)((m_lo + m_hi) * 0.5);
    }
    if (lloyd_iters > 0 && !converged) st |= OGQ_ST_ITER_CAP;
    levels2[0] = (float)m_lo;
    levels2[1] = (float)m_hi;
    *thresh = b0;
    return st;
}

static int cmp_double_asc(const void *a, const void *b)
{
    double x = *(const double *)a, y = *(const double *)b;
    return (x > y) - (x < y);
}

static int cmp_double_desc(const void *a, const void *b)
{
    return -cmp_double_asc(a, b);
}

/* ------------------------------------------------------------------------ */
/* BinGrad-pb level, Eq. (bingrad-pb optimal condition).  The quantizer of   */
/* Eq. (bingrad-pb) with levels {-b, +b} has squared error                   */
/*   E(b) = sum_{|v|<b} (b^2 - v^2) + sum_{|v|>=b} (|v| - b)^2,              */
/* whose derivative is 2 g(b), g(b) = b n - sum_{|v|>=b} |v|.  For symmetric */
/* data g(b) = 0 is the printed condition (both sides times 2n).  g is       */
/* increasing and jumps upward at every data magnitude, so "minimise the     */
/* absolute difference of the two sides" is read as: b_1 is the point where  */
/* g changes sign, either a zero inside a piece between two consecutive      */
/* magnitudes or a jump at a magnitude.  Returns status; *b1 receives b_1.   */
/* ------------------------------------------------------------------------ */
int ogq_oracle_levels_bingrad_pb(const float *v, int64_t n, float *b1)
{
    int st = 0;
    if (n <= 0) {
        *b1 = 0.0f;
        return OGQ_ST_EMPTY;
    }
    double *a = (double *)malloc((size_t)n * sizeof(double));
    for (int64_t i = 0; i < n; ++i) {
        a[i] = fabs((double)v[i]);
        if (!isfinite(a[i])) st |= OGQ_ST_NONFINITE;
    }
    qsort(a, (size_t)n, sizeof(double), cmp_double_desc);
    if (a[0] == 0.0) st |= OGQ_ST_CONSTANT;
    long double P = 0.0L; /* sum of the j largest magnitudes */
    double ans = 0.0;
    int64_t j = 0;
    while (j < n) {
        double cur = a[j];
        /* take every copy of this magnitude: on the piece (next, cur] the set {|v| >= b} is a[0..j) */
        while (j < n && a[j] == cur) {
            P += cur;
            ++j;
        }
        double next = (j < n) ? a[j] : 0.0;
        double stat = (double)(P / (long double)n); /* zero of g on this piece */
        if (stat > cur) { /* g(cur) < 0 <= g just above cur: the jump at cur */
            ans = cur;
            break;
        }
        if (stat > next || j >= n) { /* next < stat <= cur: zero inside the piece */
            ans = stat;
            break;
        }
    }
    free(a);
    *b1 = (float)ans;
    return st;
}

/* ------------------------------------------------------------------------ */
/* Q*(L, R): the middle level between two bracket levels from the discrete   */
/* form of the simplified optimal condition:                                 */
/*   |{b <= v <= R}| = sum_{L <= v <= R} (v - L) / (R - L) =: T.             */
/* The expected random-rounding error of the segment as a function of b is   */
/* piecewise linear and convex with slope sum(v - L) - (R - L) |{v >= b}|,   */
/* so its minimiser is the (floor(T) + 1)-th largest element of the segment  */
/* (the lower end of the optimal interval when T is an integer).  L must be  */
/* a data value or below all data, as it always is in the recursion.         */
/* ------------------------------------------------------------------------ */
double ogq_oracle_qstar(const float *v, int64_t n, double L, double R)
{
    if (!(R > L)) return L;
    double *seg = (double *)malloc((size_t)(n > 0 ? n : 1) * sizeof(double));
    int64_t m = 0;
    long double A = 0.0L;
    for (int64_t i = 0; i < n; ++i) {
        double x = (double)v[i];
        if (x >= L && x <= R) {
            seg[m++] = x;
            A += (long double)(x - L);
        }
    }
    if (m == 0) {
        free(seg);
        return L;
    }
    double T = (double)(A / (long double)(R - L));
    int64_t k = (int64_t)floor(T);
    if (k < 0) k = 0;
    if (k > m - 1) k = m - 1;
    qsort(seg, (size_t)m, sizeof(double), cmp_double_asc);
    double b = seg[m - 1 - k];
    free(seg);
    return b;
}

static void orq_recurse(const float *v, int64_t n, double *b, int l, int r)
{
    if (r - l < 2) return;
    int mid = (l + r) / 2;
    b[mid] = ogq_oracle_qstar(v, n, b[l], b[r]);
    orq_recurse(v, n, b, l, mid);
    orq_recurse(v, n, b, mid, r);
}

/* ------------------------------------------------------------------------ */
/* ORQ levels, Algorithm 1 (greedy recursion) with s = 2^K + 1 levels.  The  */
/* two end levels are the minimum and maximum of the tensor (Corollary 1 and */
/* the first sentence after Eq. (scaled signsgd)); the middle index of every */
/* bracket is solved by Q* and both halves recurse with one level of depth   */
/* less, stopping when the brackets are adjacent.  Levels are stored         */
/* ascending as indices 0..s-1.  Returns status bits.                        */
/* ------------------------------------------------------------------------ */
int ogq_oracle_levels_orq(const float *v, int64_t n, int s, float *levels)
{
    int st = 0;
    if (n <= 0) {
        for (int k = 0; k < s; ++k) levels[k] = 0.0f;
        return OGQ_ST_EMPTY;
    }
    double mn = INFINITY, mx = -INFINITY;
    for (int64_t i = 0; i < n; ++i) {
        double x = (double)v[i];
        if (!isfinite(x)) st |= OGQ_ST_NONFINITE;
        if (x < mn) mn = x;
        if (x > mx) mx = x;
    }
    if (st & OGQ_ST_NONFINITE) {
        for (int k = 0; k < s; ++k) levels[k] = 0.0f;
        return st;
    }
    double *b = (double *)malloc((size_t)s * sizeof(double));
    for (int k = 0; k < s; ++k) b[k] = mn;
    b[s - 1] = mx;
    if (mn == mx) st |= OGQ_ST_CONSTANT;
    orq_recurse(v, n, b, 0, s - 1);
    for (int k = 0; k < s; ++k) levels[k] = (float)b[k];
    free(b);
    return st;
}

/* ------------------------------------------------------------------------ */
/* Philox4x32 with 10 rounds (Salmon, Moraes, Dror, Shaw: "Parallel random   */
/* numbers: as easy as 1, 2, 3", SC'11), written from that description.      */
/* ------------------------------------------------------------------------ */
void ogq_oracle_philox4x32_10(const uint32_t ctr[4], const uint32_t key[2], uint32_t out[4])
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
        c0 = n0;
        c1 = n1;
        c2 = n2;
        c3 = n3;
        k0 += 0x9E3779B9u;
        k1 += 0xBB67AE85u;
    }
    out[0] = c0;
    out[1] = c1;
    out[2] = c2;
    out[3] = c3;
}

/* ------------------------------------------------------------------------ */
/* Quantizers.  scheme 0 = BinGrad-pb (levels {-b_1, b_1}, s = 2),           */
/* 1 = BinGrad-b (code = [v >= b_0]), 2 = ORQ (s levels, ascending).         */
/*                                                                           */
/* Random rounding (first equation of the multi-level section; the middle    */
/* case of Eq. (bingrad-pb), read as b_{-1} <= v < b_1): with the segment    */
/* k = clamp(#{levels <= v}, 1, s-1), lo = b_{k-1}, hi = b_k, the value goes */
/* up to hi with probability (v - lo)/(hi - lo).  Values outside the levels  */
/* land on the nearest end level, which is the clipping of BinGrad-pb.       */
/* The draw is 24 bits u of a Philox word and the decision is taken in fp32, */
/* one correctly rounded operation at a time:                                */
/*     d = v - lo;  w = hi - lo;  up  <=>  (float)u * w  <  d * 2^24.        */
/* Element i of tensor `tensor_id` uses word (i mod 4) of Philox4x32-10 with */
/* key (seed low, seed high) and counter (i/4 low, i/4 high, tensor_id,      */
/* stream_id).  codes[i] receives the level index.                           */
/* ------------------------------------------------------------------------ */
void ogq_oracle_quantize(const float *v, int64_t n, int scheme, int s, const float *levels,
                         float thresh, uint64_t seed, uint32_t tensor_id, uint32_t stream_id,
                         uint8_t *codes)
{
    if (scheme == 1) {
        for (int64_t i = 0; i < n; ++i) codes[i] = (uint8_t)(v[i] >= thresh);
        return;
    }
    uint32_t key[2] = {(uint32_t)seed, (uint32_t)(seed >> 32)};
    uint32_t rnd[4] = {0, 0, 0, 0};
    for (int64_t i = 0; i < n; ++i) {
        if ((i & 3) == 0) {
            uint64_t g = (uint64_t)i >> 2;
            uint32_t ctr[4] = {(uint32_t)g, (uint32_t)(g >> 32), tensor_id, stream_id};
            ogq_oracle_philox4x32_10(ctr, key, rnd);
        }
        float x = v[i];
        int k = 0;
        for (int q = 0; q < s; ++q) k += (levels[q] <= x);
        if (k < 1) k = 1;
        if (k > s - 1) k = s - 1;
        float lo = levels[k - 1], hi = levels[k];
        volatile float d = x - lo;
        volatile float w = hi - lo;
        volatile float lhs = (float)(rnd[i & 3] >> 8) * w;
        volatile float rhs = d * 16777216.0f;
        int up = lhs < rhs;
        codes[i] = (uint8_t)(k - 1 + up);
    }
}

/* ------------------------------------------------------------------------ */
/* Bit packing.  The paper only says "encode"; the format here is a little-  */
/* endian bit stream of 32-bit words per tensor: the code of element i sits  */
/* in stream bits [i*bits, (i+1)*bits), stream bit j is bit (j mod 32) of    */
/* word j/32, and the tensor's region is zero padded to a multiple of four   */
/* words.  words must hold ogq_oracle_packed_words(n, bits) entries.         */
/* ------------------------------------------------------------------------ */
int64_t ogq_oracle_packed_words(int64_t n, int bits)
{
    int64_t w = (n * (int64_t)bits + 31) / 32;
    return (w + 3) / 4 * 4;
}

void ogq_oracle_pack(const uint8_t *codes, int64_t n, int bits, uint32_t *words)
{
    int64_t nw = ogq_oracle_packed_words(n, bits);
    memset(words, 0, (size_t)nw * sizeof(uint32_t));
    for (int64_t i = 0; i < n; ++i) {
        for (int q = 0; q < bits; ++q) {
            int64_t j = i * bits + q;
            if ((codes[i] >> q) & 1u) words[j >> 5] |= (uint32_t)1u << (j & 31);
        }
    }
}

void ogq_oracle_unpack(const uint32_t *words, int64_t n, int bits, uint8_t *codes)
{
    for (int64_t i = 0; i < n; ++i) {
        unsigned c = 0;
        for (int q = 0; q < bits; ++q) {
            int64_t j = i * bits + q;
            c |= ((words[j >> 5] >> (j & 31)) & 1u) << q;
        }
        codes[i] = (uint8_t)c;
    }
}

/* ------------------------------------------------------------------------ */
/* Server step of Algorithm 2: decode the K workers' codes with each         */
/* worker's own levels and add them up, out[i] = scale * sum_k b^k[code_k[i]].*/
/* scale = 1/K gives the average the algorithm broadcasts, scale = 1 the sum.*/
/* packed[k] and levels[k] (s floats) belong to worker k.                    */
/* ------------------------------------------------------------------------ */
void ogq_oracle_unpack_sum(const uint32_t *const *packed, const float *const *levels, int K,
                           int64_t n, int bits, float scale, float *out)
{
    for (int64_t i = 0; i < n; ++i) {
        double acc = 0.0;
        for (int k = 0; k < K; ++k) {
            unsigned c = 0;
            for (int q = 0; q < bits; ++q) {
                int64_t j = i * bits + q;
                c |= ((packed[k][j >> 5] >> (j & 31)) & 1u) << q;
            }
            acc += (double)levels[k][c];
        }
        out[i] = (float)((double)scale * acc);
    }
}

/* ======================================================================== */
/* Extensions beyond the per-tensor core: gradient clipping, an entropy-     */
/* dense wire format, the quantization error and a refinement of the greedy  */
/* ORQ levels.                                                                */
/* ======================================================================== */

/* ------------------------------------------------------------------------ */
/* Gradient clipping (Section "Experiments", paragraph after the list of     */
/* methods): clip(v) = sign(v) * min(|v|, c * sigma), sigma^2 the variance   */
/* of the gradient being quantized (here: of the tensor or bucket), c = 2.5  */
/* in the ImageNet runs and 1.7 or 2.5 in the clipping table.  The variance  */
/* is taken about the mean, over all n elements (1/n).  The threshold is     */
/* rounded to fp32 because clipped elements take exactly that value.         */
/* Returns status bits; tau = 0 for an empty tensor.                         */
/* ------------------------------------------------------------------------ */
int ogq_oracle_clip_threshold(const float *v, int64_t n, double c, float *tau)
{
    *tau = 0.0f;
    if (n <= 0) return OGQ_ST_EMPTY;
    long double s = 0.0L;
    for (int64_t i = 0; i < n; ++i) {
        if (!isfinite((double)v[i])) return OGQ_ST_NONFINITE;
        s += (long double)v[i];
    }
    long double mean = s / (long double)n;
    long double q = 0.0L;
    for (int64_t i = 0; i < n; ++i) {
        long double d = (long double)v[i] - mean;
        q += d * d;
    }
    double sigma = sqrt((double)(q / (long double)n));
    *tau = (float)(c * sigma);
    return 0;
}

void ogq_oracle_clip(const float *v, int64_t n, float tau, float *out)
{
    for (int64_t i = 0; i < n; ++i) {
        float a = fabsf(v[i]);
        float m = a < tau ? a : tau;
        out[i] = v[i] < 0.0f ? -m : m;
    }
}

/* ------------------------------------------------------------------------ */
/* Entropy-dense packing.  The compression ratios the paper quotes (x20.2    */
/* for 3 levels, x13.8 for 5, x10.1 for 9) are 32 / log2(s): they assume     */
/* that a code costs log2(s) bits, not ceil(log2 s).  The format here gets   */
/* close to that with whole words: m consecutive codes are the base-s digits */
/* of one 32-bit word, least significant digit first, m the largest count    */
/* with s^m <= 2^32 (s = 3: 20 codes per word, 5: 13, 9: 10, 17: 7, 2: 32).  */
/* Per tensor: word j = sum_{q<m} code[j*m + q] * s^q, missing codes of the  */
/* last word are 0, and the region is zero padded to a multiple of 4 words.  */
/* ------------------------------------------------------------------------ */
int ogq_oracle_dense_digits(int s)
{
    if (s < 2) return 0;
    int m = 0;
    uint64_t p = 1;
    while (p * (uint64_t)s <= ((uint64_t)1 << 32)) {
        p *= (uint64_t)s;
        ++m;
    }
    return m;
}

int64_t ogq_oracle_dense_words(int64_t n, int s)
{
    int m = ogq_oracle_dense_digits(s);
    int64_t w = (n + m - 1) / m;
    return (w + 3) / 4 * 4;
}

void ogq_oracle_pack_dense(const uint8_t *codes, int64_t n, int s, uint32_t *words)
{
    int m = ogq_oracle_dense_digits(s);
    int64_t nw = ogq_oracle_dense_words(n, s);
    memset(words, 0, (size_t)nw * sizeof(uint32_t));
    for (int64_t j = 0; j * m < n; ++j) {
        uint64_t w = 0, p = 1;
        for (int q = 0; q < m; ++q) {
            int64_t i = j * m + q;
            if (i < n) w += (uint64_t)codes[i] * p;
            p *= (uint64_t)s;
        }
        words[j] = (uint32_t)w;
    }
}

void ogq_oracle_unpack_dense(const uint32_t *words, int64_t n, int s, uint8_t *codes)
{
    int m = ogq_oracle_dense_digits(s);
    for (int64_t i = 0; i < n; ++i) {
        uint64_t w = words[i / m];
        for (int q = 0; q < (int)(i % m); ++q) w /= (uint64_t)s;
        codes[i] = (uint8_t)(w % (uint64_t)s);
    }
}

void ogq_oracle_unpack_sum_dense(const uint32_t *const *packed, const float *const *levels, int K,
                                 int64_t n, int s, float scale, float *out)
{
    int m = ogq_oracle_dense_digits(s);
    for (int64_t i = 0; i < n; ++i) {
        double acc = 0.0;
        for (int k = 0; k < K; ++k) {
            uint64_t w = packed[k][i / m];
            for (int q = 0; q < (int)(i % m); ++q) w /= (uint64_t)s;
            acc += (double)levels[k][w % (uint64_t)s];
        }
        out[i] = (float)((double)scale * acc);
    }
}

/* ------------------------------------------------------------------------ */
/* Quantization error (the quantity tracked in the training-curve figure,    */
/* ||Q(G) - G||^2).                                                           */
/*   ogq_oracle_quant_error:    the realised error of given codes,           */
/*       sum_i (levels[code_i] - v_i)^2.                                      */
/*   ogq_oracle_expected_error: its expectation over the random rounding,    */
/*       the functional the optimal condition minimises (proof of Theorem    */
/*       1): sum_i (v_i - lo_i)(hi_i - v_i) with lo, hi the levels around    */
/*       v_i; a value outside [b_0, b_{s-1}] is clipped to the end level and */
/*       contributes (v_i - b_end)^2.                                         */
/* ------------------------------------------------------------------------ */
double ogq_oracle_quant_error(const float *v, int64_t n, const float *levels, const uint8_t *codes)
{
    long double e = 0.0L;
    for (int64_t i = 0; i < n; ++i) {
        long double d = (long double)levels[codes[i]] - (long double)v[i];
        e += d * d;
    }
    return (double)e;
}

double ogq_oracle_expected_error(const float *v, int64_t n, int s, const float *levels)
{
    long double e = 0.0L;
    for (int64_t i = 0; i < n; ++i) {
        double x = (double)v[i];
        double b0 = (double)levels[0], bs = (double)levels[s - 1];
        if (x < b0) {
            e += (long double)((b0 - x) * (b0 - x));
            continue;
        }
        if (x > bs) {
            e += (long double)((x - bs) * (x - bs));
            continue;
        }
        int k = 0;
        for (int q = 0; q < s; ++q) k += ((double)levels[q] <= x);
        if (k < 1) k = 1;
        if (k > s - 1) k = s - 1;
        double lo = (double)levels[k - 1], hi = (double)levels[k];
        e += (long double)((x - lo) * (hi - x));
    }
    return (double)e;
}

/* ------------------------------------------------------------------------ */
/* Beyond the greedy levels (the conclusion names the greedy algorithm as    */
/* the part that may be improved).  Algorithm 1 fixes a level once it has    */
/* been solved from its two brackets, so afterwards only the deepest levels  */
/* satisfy the optimal condition against their final neighbours.  One        */
/* refinement sweep re-solves every interior level in ascending order from   */
/* its two current neighbours, b_k <- Q*(b_{k-1}, b_{k+1}), each update      */
/* using the levels already updated in this sweep.  Q* is the exact          */
/* minimiser of the expected error in b_k with the other levels held fixed,  */
/* so no sweep increases the error.  Sweeps stop when one changes nothing    */
/* (every level then satisfies the discrete condition against its final      */
/* neighbours) or after max_sweeps.  levels: s values, ascending, in and out;*/
/* the end levels stay.  Returns the number of sweeps that changed a level.  */
/* ------------------------------------------------------------------------ */
int ogq_oracle_refine_orq(const float *v, int64_t n, int s, float *levels, int max_sweeps)
{
    int changed_sweeps = 0;
    if (n <= 0) return 0;
    for (int it = 0; it < max_sweeps; ++it) {
        int changed = 0;
        for (int k = 1; k < s - 1; ++k) {
            float nb = (float)ogq_oracle_qstar(v, n, (double)levels[k - 1], (double)levels[k + 1]);
            if (nb != levels[k]) {
                levels[k] = nb;
                changed = 1;
            }
        }
        if (!changed) break;
        ++changed_sweeps;
    }
    return changed_sweeps;
}
