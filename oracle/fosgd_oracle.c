/*
 * FO-SGD compression round trip: plain CPU oracle.
 *
 * TEST INFRASTRUCTURE ONLY.  This file is the slow, by-the-definition statement of what
 * the library computes.  It shares no code with the CUDA path, and nothing on the product
 * path may call it.  Every loop is serial and every floating-point quantity is a double.
 *
 * Notation follows the paper: d true length, d' padded length, H the orthonormal
 * Walsh-Hadamard matrix (Section 3, recursion below Def. 3.4), D_eps = diag(eps),
 * lambda the dither amplitude, K the number of dithers, N the number of workers.
 *
 * Pins (see tests/test_oracle_*.py): dense Sylvester matrix brute force, H H = d I, norm
 * preservation, one-hot flatness (Def. 3.4), Lemma A.4 (mean = clip, MSE closed form),
 * Lemma A.5, Remark 5.2 (norm of the K=1 composite is exactly lambda sqrt(d')), Cor. A.8
 * variance of the N-worker average, the K-dither error bound of Lemma A.9, Theorem 5.5
 * amplitude law, and the published Philox4x32-10 known-answer vectors.  The single-entry and
 * product-grid functions (flatten_entry, decode_entry, flatten_grid, decode_grid) are pinned to
 * the dense matrix and to the full transforms.
 *
 * Parity unpinned by the paper (readings taken where it is silent): zero padding to a
 * power of two and the blocked variant; the index-to-counter mapping of the generator; the
 * per-block amplitude tables (the *_tab functions: Defs. 3.7 and 3.8 applied to every block
 * with that block's own lambda, pinned against the single-amplitude functions only).
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

#define FOSGD_ORACLE_SERVER_ID 0xFFFFFFFFu

/* ------------------------------------------------------------------------------------ */
/* Counter-based generator: Philox4x32 with 10 rounds (Salmon, Moraes, Dror, Shaw, SC'11). */
/* ------------------------------------------------------------------------------------ */

void fosgd_oracle_philox4x32_10(const uint32_t ctr[4], const uint32_t key[2], uint32_t out[4])
{
    uint32_t c0 = ctr[0], c1 = ctr[1], c2 = ctr[2], c3 = ctr[3];
    uint32_t k0 = key[0], k1 = key[1];
    for (int round = 0; round < 10; ++round) {
        if (round > 0) { /* Weyl key schedule */
            k0 += 0x9E3779B9u;
            k1 += 0xBB67AE85u;
        }
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

/* Four words W(seed, step, id, domain, c): counter (c, domain, lo32 step, id),
 * key (lo32 seed, hi32 seed xor hi32 step).  The last call is remembered per thread, since
 * neighbouring coordinates share a counter (a memo, not a change of what is computed). */
void fosgd_oracle_rng_words(uint64_t seed, uint64_t step, uint32_t id, uint32_t domain,
                            uint32_t c, uint32_t out[4])
{
    static __thread int have = 0;
    static __thread uint64_t m_seed, m_step;
    static __thread uint32_t m_id, m_domain, m_c, m_out[4];
    if (!(have && m_seed == seed && m_step == step && m_id == id && m_domain == domain && m_c == c)) {
        uint32_t ctr[4] = { c, domain, (uint32_t)step, id };
        uint32_t key[2] = { (uint32_t)seed, (uint32_t)(seed >> 32) ^ (uint32_t)(step >> 32) };
        fosgd_oracle_philox4x32_10(ctr, key, m_out);
        m_seed = seed; m_step = step; m_id = id; m_domain = domain; m_c = c; have = 1;
    }
    memcpy(out, m_out, sizeof m_out);
}

/* eps_i in {+1,-1} (Def. 3.5): domain 0; the 32 flips of indices 32j..32j+31 are word j,
 * which is output (j & 3) of counter j >> 2; eps_i = -1 iff bit (i & 31) is set. */
int fosgd_oracle_eps(uint64_t seed, uint64_t step, uint32_t id, int64_t i)
{
    uint32_t w[4];
    uint64_t j = (uint64_t)i >> 5;
    fosgd_oracle_rng_words(seed, step, id, 0u, (uint32_t)(j >> 2), w);
    return ((w[j & 3] >> (i & 31)) & 1u) ? -1 : +1;
}

/* Dither integer t (Def. 3.2, tau uniform on [-lambda, lambda]): domain 1 + k.  Index
 * i = 128 G + 32 r + l takes output r of counter 32 G + l; the top 24 bits k24 of that
 * word give the odd integer t = 2 k24 + 1 - 2^24, and tau_i = lambda * t * 2^-24. */
int32_t fosgd_oracle_dither_t(uint64_t seed, uint64_t step, uint32_t id, uint32_t k, int64_t i)
{
    uint32_t w[4];
    uint64_t G = (uint64_t)i >> 7;
    uint32_t r = (uint32_t)((uint64_t)i >> 5) & 3u;
    uint32_t l = (uint32_t)i & 31u;
    fosgd_oracle_rng_words(seed, step, id, 1u + k, (uint32_t)(32u * G + l), w);
    int64_t k24 = (int64_t)(w[r] >> 8);
    return (int32_t)(2 * k24 + 1 - (1 << 24));
}

/* ------------------------------------------------------------------------------------ */
/* Transform and sizes.                                                                   */
/* ------------------------------------------------------------------------------------ */

/* Unnormalised Sylvester-ordered Walsh-Hadamard transform, in place: the recursion
 * H_k = [[H, H], [H, -H]] unrolled into log2 n butterfly sweeps (Section 3). */
void fosgd_oracle_fwht(double* x, int64_t n)
{
    for (int64_t h = 1; h < n; h <<= 1)
        for (int64_t base = 0; base < n; base += 2 * h)
            for (int64_t j = base; j < base + h; ++j) {
                double a = x[j], b = x[j + h];
                x[j] = a + b;
                x[j + h] = a - b;
            }
}

/* d' (reading of the paper's "d = 2^k"): block_log2 = 0 pads to the next power of two
 * (at least 32, one packed word); block_log2 = b > 0 pads to a multiple of 2^b. */
int64_t fosgd_oracle_padded_dim(int64_t d, int block_log2)
{
    if (d < 1) return -1;
    if (block_log2 == 0) {
        int64_t p = 32;
        while (p < d) p <<= 1;
        return p;
    }
    int64_t blk = (int64_t)1 << block_log2;
    return ((d + blk - 1) / blk) * blk;
}

/* length of one transform: d' in global mode, 2^b in blocked mode */
static int64_t transform_len(int64_t dp, int block_log2)
{
    return block_log2 == 0 ? dp : ((int64_t)1 << block_log2);
}

/* Theorem 5.5: lambda = alpha B sqrt(log d / d), lambda^s = alpha^s lambda sqrt(log d),
 * natural logarithm (proof of Lemma 3.6). */
double fosgd_oracle_lambda(double B, double alpha, int64_t d_eff)
{
    return alpha * B * sqrt(log((double)d_eff) / (double)d_eff);
}

double fosgd_oracle_lambda_server(double lambda, double alpha_s, int64_t d_eff)
{
    return alpha_s * lambda * sqrt(log((double)d_eff));
}

/* y = H D_eps x over every block (Def. 3.5), x = g zero-padded to d'.  y has d' entries. */
void fosgd_oracle_flatten(const double* g, int64_t d, int block_log2, uint64_t seed,
                          uint64_t step, uint32_t id, double* y)
{
    int64_t dp = fosgd_oracle_padded_dim(d, block_log2);
    int64_t n = transform_len(dp, block_log2);
    for (int64_t i = 0; i < dp; ++i)
        y[i] = (i < d) ? (double)fosgd_oracle_eps(seed, step, id, i) * g[i] : 0.0;
    double s = 1.0 / sqrt((double)n);
    for (int64_t b = 0; b < dp; b += n) {
        fosgd_oracle_fwht(y + b, n);
        for (int64_t i = b; i < b + n; ++i) y[i] *= s;
    }
}

/* One entry of H D_eps x straight from the matrix definition H[k][j] = (-1)^popcount(k&j)/sqrt(n):
 * used to check single outputs of transforms too long to run in full. */
double fosgd_oracle_flatten_entry(const double* g, int64_t d, int block_log2, uint64_t seed,
                                  uint64_t step, uint32_t id, int64_t k)
{
    int64_t dp = fosgd_oracle_padded_dim(d, block_log2);
    int64_t n = transform_len(dp, block_log2);
    int64_t b0 = (k / n) * n, kk = k - b0;
    double acc = 0.0;
    for (int64_t j = 0; j < n && b0 + j < d; ++j) {
        double v = (double)fosgd_oracle_eps(seed, step, id, b0 + j) * g[b0 + j];
        acc += (__builtin_popcountll((unsigned long long)(kk & j)) & 1) ? -v : v;
    }
    return acc / sqrt((double)n);
}

static int planes_for(int K)
{
    int P = 0;
    while ((1 << P) < K + 1) ++P;
    return P;
}

int fosgd_oracle_planes(int K) { return planes_for(K); }

/* Encoder E_{eps,lambda,K} (Def. 3.7) with the storage of Remark 3.3: the count
 * c_i = #{k : y_i + tau_{k,i} >= 0} in {0..K} (so (K/lambda) Q = 2c - K), written as
 * P = ceil(log2(K+1)) bit planes, plane p holding bit p of c_i at word i>>5, bit i&31.
 * sgn(0) = +1 (proof of Lemma A.4).  zmin (nullable, d' floats) receives
 * min_k |y_i + tau_{k,i}|, the margin by which each sign decision was taken. */
void fosgd_oracle_encode(const double* g, int64_t d, int block_log2, uint64_t seed,
                         uint64_t step, uint32_t id, double lambda, int K,
                         uint32_t* planes, float* zmin)
{
    int64_t dp = fosgd_oracle_padded_dim(d, block_log2);
    int P = planes_for(K);
    int64_t words = dp / 32;
    double* y = (double*)malloc(sizeof(double) * (size_t)dp);
    fosgd_oracle_flatten(g, d, block_log2, seed, step, id, y);
    memset(planes, 0, sizeof(uint32_t) * (size_t)(words * P));
    for (int64_t i = 0; i < dp; ++i) {
        int c = 0;
        double m = INFINITY;
        for (int k = 0; k < K; ++k) {
            double tau = lambda * (double)fosgd_oracle_dither_t(seed, step, id, (uint32_t)k, i)
                         * (1.0 / 16777216.0);
            double z = y[i] + tau;
            if (z >= 0.0) ++c;
            if (fabs(z) < m) m = fabs(z);
        }
        for (int p = 0; p < P; ++p)
            if ((c >> p) & 1) planes[(int64_t)p * words + (i >> 5)] |= (1u << (i & 31));
        if (zmin) zmin[i] = (float)m;
    }
    free(y);
}

/* Decoder D_{eps,lambda,K} (Def. 3.8) on all d' coordinates:
 * out = (lambda / K) D_eps H^T q, q_i = 2 c_i - K; H^T = H for the Sylvester matrix. */
void fosgd_oracle_decode_full(const uint32_t* planes, int64_t d, int block_log2, uint64_t seed,
                              uint64_t step, uint32_t id, double lambda, int K, double* out)
{
    int64_t dp = fosgd_oracle_padded_dim(d, block_log2);
    int64_t n = transform_len(dp, block_log2);
    int P = planes_for(K);
    int64_t words = dp / 32;
    for (int64_t i = 0; i < dp; ++i) {
        int c = 0;
        for (int p = 0; p < P; ++p)
            c |= (int)((planes[(int64_t)p * words + (i >> 5)] >> (i & 31)) & 1u) << p;
        out[i] = (double)(2 * c - K);
    }
    double s = lambda / ((double)K * sqrt((double)n));
    for (int64_t b = 0; b < dp; b += n) fosgd_oracle_fwht(out + b, n);
    for (int64_t i = 0; i < dp; ++i)
        out[i] *= s * (double)fosgd_oracle_eps(seed, step, id, i);
}

/* One entry of the decoder of Def. 3.8 straight from the matrix definition
 * H[k][j] = (-1)^popcount(k&j)/sqrt(n): out_k = (lambda / K) eps_k sum_j H[k][j] (2 c_j - K), the sum
 * running over the block of k.  The twin of fosgd_oracle_flatten_entry for the decode side: it
 * checks single outputs of decoders too long to run in full. */
double fosgd_oracle_decode_entry(const uint32_t* planes, int64_t d, int block_log2, uint64_t seed,
                                 uint64_t step, uint32_t id, double lambda, int K, int64_t k)
{
    int64_t dp = fosgd_oracle_padded_dim(d, block_log2);
    int64_t n = transform_len(dp, block_log2);
    int P = planes_for(K);
    int64_t words = dp / 32;
    int64_t b0 = (k / n) * n, kk = k - b0;
    double acc = 0.0;   /* a sum of integers below 2^53: exact */
    for (int64_t j = 0; j < n; ++j) {
        int64_t i = b0 + j;
        int c = 0;
        for (int p = 0; p < P; ++p)
            c |= (int)((planes[(int64_t)p * words + (i >> 5)] >> (i & 31)) & 1u) << p;
        double q = (double)(2 * c - K);
        acc += (__builtin_popcountll((unsigned long long)(kk & j)) & 1) ? -q : q;
    }
    return lambda / ((double)K * sqrt((double)n)) * (double)fosgd_oracle_eps(seed, step, id, k) * acc;
}

/* Entries of one global transform (block_log2 = 0, length n = d') on a product grid of output
 * indices k = k_hi[a] 2^s + k_lo[b].  The recursion H_k = H_1 (x) H_{k-1} below Def. 3.4, applied
 * to the top log2(n) - s index bits, reads H_n = H_{n / 2^s} (x) H_{2^s}, i.e. with j = j_hi 2^s + j_lo
 *     (H v)[k_hi 2^s + k_lo] = n^{-1/2} sum_{j_hi} (-1)^popcount(k_hi & j_hi)
 *                                       [ sum_{j_lo} (-1)^popcount(k_lo & j_lo) v_j ],
 * so the bracket is shared by all k_hi and the whole grid costs n * n_lo multiply-adds instead of
 * n * n_hi * n_lo.  The signs (-1)^popcount(k_lo & j_lo) are tabulated once as +-1.0.  Nothing
 * else is reordered; both functions below are pinned to the single-entry functions above and to
 * the full transforms.  out: [n_hi][n_lo]. */
static double* walsh_sign_table(const int64_t* k_lo, int n_lo, int64_t lo_len)
{
    double* tab = (double*)malloc(sizeof(double) * (size_t)n_lo * (size_t)lo_len);
    for (int64_t j_lo = 0; j_lo < lo_len; ++j_lo)
        for (int b = 0; b < n_lo; ++b)
            tab[j_lo * n_lo + b] =
                (__builtin_popcountll((unsigned long long)(k_lo[b] & j_lo)) & 1) ? -1.0 : 1.0;
    return tab;
}

/* sum over j_hi of +-inner (the outer Kronecker factor), for every k_hi of the grid */
static void grid_outer(const double* inner, int64_t j_hi, const int64_t* k_hi, int n_hi, int n_lo,
                       double* out)
{
    for (int a = 0; a < n_hi; ++a) {
        int neg = __builtin_popcountll((unsigned long long)(k_hi[a] & j_hi)) & 1;
        for (int b = 0; b < n_lo; ++b) out[a * n_lo + b] += neg ? -inner[b] : inner[b];
    }
}

/* flatten_grid: v = D_eps x, x the zero-padded gradient, given as doubles (g_is_f32 = 0) or
 * floats (g_is_f32 = 1, for vectors too long to hold twice in host memory). */
void fosgd_oracle_flatten_grid(const void* g, int g_is_f32, int64_t d, uint64_t seed, uint64_t step,
                               uint32_t id, int s, const int64_t* k_hi, int n_hi,
                               const int64_t* k_lo, int n_lo, double* out)
{
    int64_t n = fosgd_oracle_padded_dim(d, 0);
    int64_t lo_len = (int64_t)1 << s, hi_len = n >> s;
    double* sgn = walsh_sign_table(k_lo, n_lo, lo_len);
    double* inner = (double*)malloc(sizeof(double) * (size_t)n_lo);
    for (int a = 0; a < n_hi * n_lo; ++a) out[a] = 0.0;
    for (int64_t j_hi = 0; j_hi < hi_len; ++j_hi) {
        for (int b = 0; b < n_lo; ++b) inner[b] = 0.0;
        for (int64_t j_lo = 0; j_lo < lo_len; ++j_lo) {
            int64_t j = j_hi * lo_len + j_lo;
            if (j >= d) break;   /* padding: zeros from here to the end of the vector */
            double x = g_is_f32 ? (double)((const float*)g)[j] : ((const double*)g)[j];
            double v = (double)fosgd_oracle_eps(seed, step, id, j) * x;
            const double* sj = sgn + j_lo * n_lo;
            for (int b = 0; b < n_lo; ++b) inner[b] += sj[b] * v;
        }
        grid_outer(inner, j_hi, k_hi, n_hi, n_lo, out);
    }
    double sc = 1.0 / sqrt((double)n);
    for (int a = 0; a < n_hi * n_lo; ++a) out[a] *= sc;
    free(inner);
    free(sgn);
}

/* decode_grid: the decoder of Def. 3.8 on the same kind of grid, v_j = 2 c_j - K read from the
 * bit planes; every entry is scaled by lambda / (K sqrt n) and flipped by eps at its own index. */
void fosgd_oracle_decode_grid(const uint32_t* planes, int64_t d, uint64_t seed, uint64_t step,
                              uint32_t id, double lambda, int K, int s, const int64_t* k_hi,
                              int n_hi, const int64_t* k_lo, int n_lo, double* out)
{
    int64_t n = fosgd_oracle_padded_dim(d, 0);
    int64_t lo_len = (int64_t)1 << s, hi_len = n >> s;
    int P = planes_for(K);
    int64_t words = n / 32;
    double* sgn = walsh_sign_table(k_lo, n_lo, lo_len);
    double* inner = (double*)malloc(sizeof(double) * (size_t)n_lo);
    for (int a = 0; a < n_hi * n_lo; ++a) out[a] = 0.0;
    for (int64_t j_hi = 0; j_hi < hi_len; ++j_hi) {
        for (int b = 0; b < n_lo; ++b) inner[b] = 0.0;
        for (int64_t j_lo = 0; j_lo < lo_len; ++j_lo) {
            int64_t j = j_hi * lo_len + j_lo;
            int c = 0;
            for (int p = 0; p < P; ++p)
                c |= (int)((planes[(int64_t)p * words + (j >> 5)] >> (j & 31)) & 1u) << p;
            double v = (double)(2 * c - K);
            const double* sj = sgn + j_lo * n_lo;
            for (int b = 0; b < n_lo; ++b) inner[b] += sj[b] * v;
        }
        grid_outer(inner, j_hi, k_hi, n_hi, n_lo, out);
    }
    double sc = lambda / ((double)K * sqrt((double)n));
    for (int a = 0; a < n_hi; ++a)
        for (int b = 0; b < n_lo; ++b)
            out[a * n_lo + b] *= sc * (double)fosgd_oracle_eps(seed, step, id, k_hi[a] * lo_len + k_lo[b]);
    free(inner);
    free(sgn);
}

/* Blocked mode with one amplitude per block: Defs. 3.7 and 3.8 hold for each block of n = 2^b
 * coordinates separately, block k using lambda_tab[k] for its dither and for its decoder
 * scale.  Everything else as in fosgd_oracle_encode / fosgd_oracle_decode_full. */
void fosgd_oracle_encode_tab(const double* g, int64_t d, int block_log2, uint64_t seed,
                             uint64_t step, uint32_t id, const double* lambda_tab, int K,
                             uint32_t* planes, float* zmin)
{
    int64_t dp = fosgd_oracle_padded_dim(d, block_log2);
    int64_t n = transform_len(dp, block_log2);
    int P = planes_for(K);
    int64_t words = dp / 32;
    double* y = (double*)malloc(sizeof(double) * (size_t)dp);
    fosgd_oracle_flatten(g, d, block_log2, seed, step, id, y);
    memset(planes, 0, sizeof(uint32_t) * (size_t)(words * P));
    for (int64_t i = 0; i < dp; ++i) {
        double lambda = lambda_tab[i / n];
        int c = 0;
        double m = INFINITY;
        for (int k = 0; k < K; ++k) {
            double tau = lambda * (double)fosgd_oracle_dither_t(seed, step, id, (uint32_t)k, i)
                         * (1.0 / 16777216.0);
            double z = y[i] + tau;
            if (z >= 0.0) ++c;
            if (fabs(z) < m) m = fabs(z);
        }
        for (int p = 0; p < P; ++p)
            if ((c >> p) & 1) planes[(int64_t)p * words + (i >> 5)] |= (1u << (i & 31));
        if (zmin) zmin[i] = (float)m;
    }
    free(y);
}

void fosgd_oracle_decode_full_tab(const uint32_t* planes, int64_t d, int block_log2,
                                  uint64_t seed, uint64_t step, uint32_t id,
                                  const double* lambda_tab, int K, double* out)
{
    int64_t dp = fosgd_oracle_padded_dim(d, block_log2);
    int64_t n = transform_len(dp, block_log2);
    int P = planes_for(K);
    int64_t words = dp / 32;
    for (int64_t i = 0; i < dp; ++i) {
        int c = 0;
        for (int p = 0; p < P; ++p)
            c |= (int)((planes[(int64_t)p * words + (i >> 5)] >> (i & 31)) & 1u) << p;
        out[i] = (double)(2 * c - K);
    }
    for (int64_t b = 0; b < dp; b += n) fosgd_oracle_fwht(out + b, n);
    for (int64_t i = 0; i < dp; ++i)
        out[i] *= lambda_tab[i / n] / ((double)K * sqrt((double)n))
                  * (double)fosgd_oracle_eps(seed, step, id, i);
}

/* Server average, eq. (4.1): gbar = (1/N) sum_n D(q_n), each worker decoded with its own
 * eps_n (worker ids worker_id0 .. worker_id0+M-1, N = M).  gbar has d' entries. */
void fosgd_oracle_aggregate(const uint32_t* bits, int64_t d, int M, uint32_t worker_id0,
                            uint64_t seed, uint64_t step, double lambda, int block_log2,
                            double* gbar)
{
    int64_t dp = fosgd_oracle_padded_dim(d, block_log2);
    int64_t words = dp / 32;
    double* tmp = (double*)malloc(sizeof(double) * (size_t)dp);
    for (int64_t i = 0; i < dp; ++i) gbar[i] = 0.0;
    for (int n = 0; n < M; ++n) {
        fosgd_oracle_decode_full(bits + (int64_t)n * words, d, block_log2, seed, step,
                                 worker_id0 + (uint32_t)n, lambda, 1, tmp);
        for (int64_t i = 0; i < dp; ++i) gbar[i] += tmp[i];
    }
    for (int64_t i = 0; i < dp; ++i) gbar[i] /= (double)M;
    free(tmp);
}

/* Downlink (Section 4, server-to-workers): the server encodes gbar (all d' entries, no new
 * padding) with eps^s, lambda^s and K dithers; every worker applies the matching decoder. */
void fosgd_oracle_downlink_encode(const double* gbar, int64_t dp, int block_log2, uint64_t seed,
                                  uint64_t step, double lambda_s, int K, uint32_t* planes,
                                  float* zmin)
{
    fosgd_oracle_encode(gbar, dp, block_log2, seed, step, FOSGD_ORACLE_SERVER_ID, lambda_s, K,
                        planes, zmin);
}

void fosgd_oracle_downlink_decode(const uint32_t* planes, int64_t dp, int block_log2,
                                  uint64_t seed, uint64_t step, double lambda_s, int K,
                                  double* out)
{
    fosgd_oracle_decode_full(planes, dp, block_log2, seed, step, FOSGD_ORACLE_SERVER_ID,
                             lambda_s, K, out);
}
