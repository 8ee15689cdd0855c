/*
 * DropIT oracle: a plain, slow, single-file CPU statement of what the DropIT
 * layer path computes (arXiv 2202.13808).  TEST INFRASTRUCTURE ONLY: it is
 * called from tests, from the smoke check and from the benchmark's CPU
 * baseline leg, never from the product path, and it shares no code with the
 * CUDA library.
 *
 * What it states, each from the paper:
 *   - keep count           Sec. 3.3 ("drop the smallest gamma fraction"), Sec. 4.1
 *                          ("proportion of 1-gamma"), Table 4 (memory falls by gamma)
 *   - min-k selection      Sec. 3.3 "Min-K Elements", Sec. 4.1 (largest |a| retained)
 *   - sparse cache a-hat   Sec. 3.2, a-hat = {a_Xr, X_r} ("coordinate format", Sec. 4.1)
 *   - recovery R(.)        Sec. 3.2 (dropped indices filled with zero)
 *   - FC weight gradient   Eq. 6,  g = sum_{n in X_r} grad_z_j^n a_k^n ; App. A.3 G' = (A o D) x Z
 *   - conv weight gradient Eq. 4-5 (retained term), element-wise mask over the input a
 *   - random dropping      Sec. 3.3 "Random Elements" (a gamma fraction dropped at random within the
 *                          mini-batch): every element draws a 15-bit rank from Philox4x32-10 (Salmon,
 *                          Moraes, Dror, Shaw, "Parallel random numbers: as easy as 1, 2, 3", SC'11) and
 *                          the k highest ranks are retained, ties to the lower flat index
 *
 *   - producer in front    Sec. 3.5 (the layers whose outputs are the conv / fc inputs: activations and
 *     of the path          normalisations keep their own caches): the element-wise producer y = act(x) of a bf16
 *                          tensor stated as a table over all 65536 bit patterns (act evaluated in double,
 *                          rounded once to bf16, ties to even), and the histogram of the ordering keys of y
 *
 *   - 8-bit retained values   Sec. 1 / Table 5 combine DropIT with 8-bit and 4-bit activation quantisers on the
 *                          other layers; here the same idea on DropIT's own payload: the retained bf16 values
 *                          as sign + 3 exponent bits + 4 mantissa bits under one exponent shared by the tensor
 *
 * Floating point: products and sums in double; results are returned as double.
 * Elements are passed as raw bits (uint16 for bf16, uint32 for fp32); the
 * ordering key of an element is its bits with the sign bit cleared, so
 * -0 == +0, Inf is above every finite value and NaN patterns are above Inf.
 *
 * Pinned by tests/test_oracle_*.py against: the literal rank definition
 * (oracle_select_rank) vs the sort (oracle_select_sort) vs numpy's stable
 * sort; closed-form keep counts; closed-form Gaussian quantiles; all-equal and
 * strictly-monotone tensors; numpy float64 matmul at gamma = 0; torch's
 * float64 conv weight gradient; 1x1 conv == FC on the transposed view; the
 * Philox test vectors printed with the generator's reference distribution; the
 * bf16 rounding against exact rational arithmetic, the GELU table against an
 * independent erf and the same exact rounding, the ReLU table in closed form.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

#define DT_BF16 0
#define DT_F32 1

/* ---- random ranks (Sec. 3.3 "Random Elements") -------------------------- */

/* Philox4x32-10 as published (SC'11, Sec. 3.3 / Table 2 of that paper): ten rounds of
 *   (c0, c1, c2, c3) <- (hi(M1*c2) ^ c1 ^ k0,  lo(M1*c2),  hi(M0*c0) ^ c3 ^ k1,  lo(M0*c0)),
 * the key (k0, k1) raised by the Weyl constants (W0, W1) between rounds. */
void oracle_philox4x32_10(const uint32_t ctr[4], const uint32_t key[2], uint32_t out[4]) {
    const uint32_t M0 = 0xD2511F53u, M1 = 0xCD9E8D57u, W0 = 0x9E3779B9u, W1 = 0xBB67AE85u;
    uint32_t c0 = ctr[0], c1 = ctr[1], c2 = ctr[2], c3 = ctr[3], k0 = key[0], k1 = key[1];
    for (int round = 0; round < 10; ++round) {
        const uint64_t p0 = (uint64_t)M0 * c0, p1 = (uint64_t)M1 * c2;
        const uint32_t n0 = (uint32_t)(p1 >> 32) ^ c1 ^ k0;
        const uint32_t n1 = (uint32_t)p1;
        const uint32_t n2 = (uint32_t)(p0 >> 32) ^ c3 ^ k1;
        const uint32_t n3 = (uint32_t)p0;
        c0 = n0; c1 = n1; c2 = n2; c3 = n3;
        k0 += W0;
        k1 += W1;
    }
    out[0] = c0; out[1] = c1; out[2] = c2; out[3] = c3;
}

/* Rank of element i under seed s: block b = i div 8 is the counter (b_lo, b_hi, 0, 0), the seed is the
 * key (s_lo, s_hi); the four output words hold eight 16-bit halves, low half first, and element i takes
 * half (i mod 8) without its top bit (15 bits). */
void oracle_random_ranks(int64_t n, uint64_t seed, uint32_t* ranks) {
    const uint32_t key[2] = {(uint32_t)seed, (uint32_t)(seed >> 32)};
    for (int64_t i = 0; i < n; ++i) {
        const uint64_t b = (uint64_t)i / 8;
        const uint32_t ctr[4] = {(uint32_t)b, (uint32_t)(b >> 32), 0u, 0u};
        uint32_t out[4];
        oracle_philox4x32_10(ctr, key, out);
        const int e = (int)(i % 8);
        ranks[i] = (out[e / 2] >> (16 * (e % 2))) & 0x7FFFu;
    }
}

/* ---- element decoding ------------------------------------------------- */

static double bf16_bits_to_double(uint16_t b) {
    uint32_t u = ((uint32_t)b) << 16;
    float f;
    memcpy(&f, &u, sizeof f);
    return (double)f;
}

static double f32_bits_to_double(uint32_t u) {
    float f;
    memcpy(&f, &u, sizeof f);
    return (double)f;
}

static double elem_to_double(const void* x, int64_t i, int dtype) {
    if (dtype == DT_BF16) return bf16_bits_to_double(((const uint16_t*)x)[i]);
    return f32_bits_to_double(((const uint32_t*)x)[i]);
}

/* Ordering key of |x|: the raw bits without the sign bit (Sec. 3.3, absolute magnitude). */
void oracle_keys(const void* x, int64_t n, int dtype, uint32_t* keys) {
    for (int64_t i = 0; i < n; ++i) {
        if (dtype == DT_BF16) keys[i] = ((const uint16_t*)x)[i] & 0x7FFFu;
        else keys[i] = ((const uint32_t*)x)[i] & 0x7FFFFFFFu;
    }
}

/* ---- keep count (Sec. 3.3 / Sec. 4.1 / Table 4) ------------------------ */

/* gamma is the DROPPED fraction.  The number dropped is the smallest integer
 * not below gamma*n (so at least a gamma fraction goes, never more kept than
 * the 1-gamma budget); the 1e-6 guard absorbs the binary rounding of gamma
 * (0.9*10 evaluates to 9.000000000000002 in double). */
int64_t oracle_keep_count(int64_t n, double gamma) {
    double d = ceil(gamma * (double)n - 1e-6);
    if (d < 0.0) d = 0.0;
    if (d > (double)n) d = (double)n;
    return n - (int64_t)d;
}

/* ---- selection --------------------------------------------------------- */

/* Literal definition: rank(i) = #{j : key_j > key_i} + #{j < i : key_j == key_i};
 * element i is retained iff rank(i) < k.  O(n^2), for small n. */
void oracle_select_rank(const uint32_t* keys, int64_t n, int64_t k, uint8_t* keep) {
    for (int64_t i = 0; i < n; ++i) {
        int64_t rank = 0;
        for (int64_t j = 0; j < n; ++j) {
            if (keys[j] > keys[i]) ++rank;
            else if (keys[j] == keys[i] && j < i) ++rank;
        }
        keep[i] = (uint8_t)(rank < k);
    }
}

typedef struct {
    uint32_t key;
    uint32_t pad;
    int64_t idx;
} keyed_t;

static int cmp_key_desc_idx_asc(const void* pa, const void* pb) {
    const keyed_t* a = (const keyed_t*)pa;
    const keyed_t* b = (const keyed_t*)pb;
    if (a->key != b->key) return (a->key > b->key) ? -1 : 1;
    if (a->idx != b->idx) return (a->idx < b->idx) ? -1 : 1;
    return 0;
}

/* Same set by sorting on (key descending, flat index ascending) and taking the
 * first k.  The comparator is a total order, so the library sort needs no
 * stability guarantee.  Returns 0, or -1 if memory could not be had. */
int oracle_select_sort(const uint32_t* keys, int64_t n, int64_t k, uint8_t* keep) {
    if (n < 0) return -1;
    keyed_t* v = (keyed_t*)malloc((size_t)(n > 0 ? n : 1) * sizeof(keyed_t));
    if (!v) return -1;
    for (int64_t i = 0; i < n; ++i) {
        v[i].key = keys[i];
        v[i].pad = 0;
        v[i].idx = i;
    }
    qsort(v, (size_t)n, sizeof(keyed_t), cmp_key_desc_idx_asc);
    memset(keep, 0, (size_t)n);
    for (int64_t r = 0; r < k && r < n; ++r) keep[v[r].idx] = 1;
    free(v);
    return 0;
}

/* D(.) with the min-k strategy on a whole tensor: keys, keep count, selection. */
int oracle_min_k(const void* x, int64_t n, double gamma, int dtype, uint8_t* keep, int64_t* k_out) {
    uint32_t* keys = (uint32_t*)malloc((size_t)(n > 0 ? n : 1) * sizeof(uint32_t));
    if (!keys) return -1;
    oracle_keys(x, n, dtype, keys);
    int64_t k = oracle_keep_count(n, gamma);
    int rc = oracle_select_sort(keys, n, k, keep);
    free(keys);
    if (k_out) *k_out = k;
    return rc;
}

/* D(.) with the random strategy (Sec. 3.3 "Random Elements"): the same number of elements is retained as
 * under min-k, chosen by rank instead of magnitude. */
int oracle_random_k(int64_t n, double gamma, uint64_t seed, uint8_t* keep, int64_t* k_out) {
    const int64_t k = oracle_keep_count(n, gamma);
    if (k_out) *k_out = k;
    if (n <= 0) return 0;
    uint32_t* ranks = (uint32_t*)malloc((size_t)n * sizeof(uint32_t));
    if (!ranks) return -1;
    oracle_random_ranks(n, seed, ranks);
    const int rc = oracle_select_sort(ranks, n, k, keep);
    free(ranks);
    return rc;
}

/* ---- encoders for a-hat = {a_Xr, X_r} (Sec. 3.2) ------------------------ */

/* Occupancy bitmask: element i <-> bit (i mod 32) of 32-bit word (i div 32);
 * the unused high bits of the last word are 0.  words has ceil(n/32) entries. */
void oracle_encode_bitmask(const uint8_t* keep, int64_t n, uint32_t* words) {
    int64_t nw = (n + 31) / 32;
    for (int64_t w = 0; w < nw; ++w) words[w] = 0;
    for (int64_t i = 0; i < n; ++i)
        if (keep[i]) words[i / 32] |= (uint32_t)1 << (i % 32);
}

/* Retained flat indices in ascending order (the coordinate format's X_r). Returns the count. */
int64_t oracle_encode_index32(const uint8_t* keep, int64_t n, int32_t* idx) {
    int64_t c = 0;
    for (int64_t i = 0; i < n; ++i)
        if (keep[i]) idx[c++] = (int32_t)i;
    return c;
}

/* Retained values a_Xr, raw bits untouched, ascending flat index. Returns the count. */
int64_t oracle_pack_values(const void* x, const uint8_t* keep, int64_t n, int dtype, void* values) {
    int64_t c = 0;
    for (int64_t i = 0; i < n; ++i) {
        if (!keep[i]) continue;
        if (dtype == DT_BF16) ((uint16_t*)values)[c] = ((const uint16_t*)x)[i];
        else ((uint32_t*)values)[c] = ((const uint32_t*)x)[i];
        ++c;
    }
    return c;
}

/* offsets[c] = number of retained elements with flat index < c*chunk, for
 * c = 0 .. ceil(n/chunk)-1 (a seek table into the packed values). */
void oracle_chunk_offsets(const uint8_t* keep, int64_t n, int64_t chunk, uint32_t* offsets) {
    int64_t seen = 0; /* retained elements with flat index < i */
    for (int64_t i = 0; i < n; ++i) {
        if (i % chunk == 0) offsets[i / chunk] = (uint32_t)seen;
        seen += keep[i];
    }
}

/* ---- recovery R(.) (Sec. 3.2): dropped positions become +0 --------------- */

void oracle_recover_from_bitmask(const void* values, const uint32_t* words, int64_t n, int dtype, void* x_out) {
    int64_t c = 0;
    for (int64_t i = 0; i < n; ++i) {
        int kept = (int)((words[i / 32] >> (i % 32)) & 1u);
        if (dtype == DT_BF16) ((uint16_t*)x_out)[i] = kept ? ((const uint16_t*)values)[c] : 0;
        else ((uint32_t*)x_out)[i] = kept ? ((const uint32_t*)values)[c] : 0;
        c += kept;
    }
}

void oracle_recover_from_index32(const void* values, const int32_t* idx, int64_t k, int64_t n, int dtype,
                                 void* x_out) {
    if (dtype == DT_BF16) memset(x_out, 0, (size_t)n * 2);
    else memset(x_out, 0, (size_t)n * 4);
    for (int64_t r = 0; r < k; ++r) {
        if (dtype == DT_BF16) ((uint16_t*)x_out)[idx[r]] = ((const uint16_t*)values)[r];
        else ((uint32_t*)x_out)[idx[r]] = ((const uint32_t*)values)[r];
    }
}

/* ---- FC weight gradient, Eq. 6 ------------------------------------------ */

/* dw[j*Ca + c] = sum over retained (n, c) of dy[n*Cz + j] * a[n*Ca + c].
 * Only retained entries are visited; each visits every output row j.
 * The j loop is the only parallel one (independent outputs). */
void oracle_fc_weight_grad(const void* dy, const void* x, const uint8_t* keep, int64_t M, int64_t Ca, int64_t Cz,
                           int dtype, double* dw) {
    for (int64_t i = 0; i < Cz * Ca; ++i) dw[i] = 0.0;
#pragma omp parallel for schedule(static)
    for (int64_t j = 0; j < Cz; ++j) {
        for (int64_t n = 0; n < M; ++n) {
            double g = elem_to_double(dy, n * Cz + j, dtype);
            for (int64_t c = 0; c < Ca; ++c) {
                if (!keep[n * Ca + c]) continue;
                dw[j * Ca + c] += g * elem_to_double(x, n * Ca + c, dtype);
            }
        }
    }
}

/* One output entry of Eq. 6 at a time, for spot checks at sizes where the full
 * gradient is too slow: out[s] = dW[js[s], cs[s]]. */
void oracle_fc_weight_grad_entries(const void* dy, const void* x, const uint8_t* keep, int64_t M, int64_t Ca,
                                   int64_t Cz, int dtype, const int64_t* js, const int64_t* cs, int64_t ns,
                                   double* out) {
#pragma omp parallel for schedule(static)
    for (int64_t s = 0; s < ns; ++s) {
        int64_t j = js[s], c = cs[s];
        double acc = 0.0;
        for (int64_t n = 0; n < M; ++n)
            if (keep[n * Ca + c]) acc += elem_to_double(dy, n * Cz + j, dtype) * elem_to_double(x, n * Ca + c, dtype);
        out[s] = acc;
    }
}

/* ---- conv weight gradient, Eq. 4-5 (retained term) ----------------------- */

/* dw[j,c,u,v] = sum_{n,y,x} dy[n,j,y,x] * R(a-hat)[n,c, y*stride+u-pad, x*stride+v-pad],
 * out-of-range input positions contribute 0; NCHW, cross-correlation, groups 1,
 * dilation 1.  keep is the element-wise mask over the input a. */
void oracle_conv_weight_grad(const void* dy, const void* x, const uint8_t* keep, int64_t B, int64_t Ca, int64_t H,
                             int64_t W, int64_t Cz, int64_t R, int64_t S, int64_t stride, int64_t pad, int dtype,
                             double* dw) {
    int64_t Ho = (H + 2 * pad - R) / stride + 1;
    int64_t Wo = (W + 2 * pad - S) / stride + 1;
#pragma omp parallel for schedule(static)
    for (int64_t j = 0; j < Cz; ++j)
        for (int64_t c = 0; c < Ca; ++c)
            for (int64_t u = 0; u < R; ++u)
                for (int64_t v = 0; v < S; ++v) {
                    double acc = 0.0;
                    for (int64_t n = 0; n < B; ++n)
                        for (int64_t y = 0; y < Ho; ++y)
                            for (int64_t xx = 0; xx < Wo; ++xx) {
                                int64_t yi = y * stride + u - pad;
                                int64_t xi = xx * stride + v - pad;
                                if (yi < 0 || yi >= H || xi < 0 || xi >= W) continue;
                                int64_t ia = ((n * Ca + c) * H + yi) * W + xi;
                                if (!keep[ia]) continue;
                                int64_t iz = ((n * Cz + j) * Ho + y) * Wo + xx;
                                acc += elem_to_double(dy, iz, dtype) * elem_to_double(x, ia, dtype);
                            }
                    dw[((j * Ca + c) * R + u) * S + v] = acc;
                }
}

/* Spot entries of the conv gradient: out[s] = dW[js[s], cs[s], us[s], vs[s]]. */
void oracle_conv_weight_grad_entries(const void* dy, const void* x, const uint8_t* keep, int64_t B, int64_t Ca,
                                     int64_t H, int64_t W, int64_t Cz, int64_t R, int64_t S, int64_t stride,
                                     int64_t pad, int dtype, const int64_t* js, const int64_t* cs, const int64_t* us,
                                     const int64_t* vs, int64_t ns, double* out) {
    int64_t Ho = (H + 2 * pad - R) / stride + 1;
    int64_t Wo = (W + 2 * pad - S) / stride + 1;
#pragma omp parallel for schedule(static)
    for (int64_t s = 0; s < ns; ++s) {
        int64_t j = js[s], c = cs[s], u = us[s], v = vs[s];
        double acc = 0.0;
        for (int64_t n = 0; n < B; ++n)
            for (int64_t y = 0; y < Ho; ++y)
                for (int64_t xx = 0; xx < Wo; ++xx) {
                    int64_t yi = y * stride + u - pad;
                    int64_t xi = xx * stride + v - pad;
                    if (yi < 0 || yi >= H || xi < 0 || xi >= W) continue;
                    int64_t ia = ((n * Ca + c) * H + yi) * W + xi;
                    if (!keep[ia]) continue;
                    int64_t iz = ((n * Cz + j) * Ho + y) * Wo + xx;
                    acc += elem_to_double(dy, iz, dtype) * elem_to_double(x, ia, dtype);
                }
        out[s] = acc;
    }
}

/* ---- the producer in front of the path (Sec. 3.5) ------------------------ */

/* A double rounded once to bf16 (8 significant bits, the exponent range of fp32), ties to even.
 * |v| = m * 2^(e-7) with 128 <= m < 256 is scaled so that rint() (ties to even in the default
 * rounding mode; the scaling by a power of two is exact) does the rounding.  Subnormal results
 * use the fixed scale 2^-133.  NaN gives the one pattern 0x7FC0. */
uint16_t oracle_round_to_bf16(double v) {
    if (v != v) return 0x7FC0;
    const uint16_t sign = signbit(v) ? 0x8000 : 0;
    const double a = fabs(v);
    if (a == 0.0) return sign;
    if (isinf(a)) return (uint16_t)(sign | 0x7F80);
    int e2;
    (void)frexp(a, &e2);              /* a = f * 2^e2, 0.5 <= f < 1  ->  floor(log2 a) = e2 - 1 */
    int e = e2 - 1;
    if (e < -126) {                   /* subnormal range of bf16: units of 2^-133 */
        const double r = rint(ldexp(a, 133));      /* 0 .. 128 */
        return (uint16_t)(sign | (uint16_t)r);     /* 128 = the smallest normal: exponent field 1, mantissa 0 */
    }
    double r = rint(ldexp(a, 7 - e)); /* 128 .. 256 */
    if (r == 256.0) {
        r = 128.0;
        e += 1;
    }
    const int E = e + 127;
    if (E >= 255) return (uint16_t)(sign | 0x7F80);
    return (uint16_t)(sign | (uint16_t)(E << 7) | ((uint16_t)r - 128));
}

#define ACT_IDENTITY 0
#define ACT_RELU 1
#define ACT_GELU 2

/* y = act(x) for every bf16 bit pattern b (table[b] = bits of y).
 *   identity: the bits themselves.
 *   ReLU: max(x, 0): x for x > 0, +0 for x <= 0 (also for -0); NaN patterns pass through unchanged.
 *   GELU: x * Phi(x) with Phi(x) = erfc(-x / sqrt 2) / 2 in double (the form that keeps its digits for
 *         negative x, where 1 + erf(x / sqrt 2) cancels), rounded once; NaN patterns pass through unchanged,
 *         and -Inf (whose product Inf * 0 is not a number) gives 0x7FC0. */
void oracle_activation_table(int act, uint16_t* table) {
    for (uint32_t b = 0; b < 65536; ++b) {
        const uint16_t key = (uint16_t)(b & 0x7FFF);
        uint16_t y;
        if (act == ACT_IDENTITY || key > 0x7F80) {
            y = (uint16_t)b;
        } else if (act == ACT_RELU) {
            y = ((b & 0x8000) || key == 0) ? 0 : (uint16_t)b;
        } else {
            const double x = bf16_bits_to_double((uint16_t)b);
            y = oracle_round_to_bf16(x * (0.5 * erfc(-x / sqrt(2.0))));
        }
        table[b] = y;
    }
}

/* y[i] = table[x[i]] */
void oracle_apply_table(const uint16_t* table, const uint16_t* x, int64_t n, uint16_t* y) {
    for (int64_t i = 0; i < n; ++i) y[i] = table[x[i]];
}

/* Histogram of the ordering keys of a bf16 tensor: hist[key] = #{i : bits_i with the sign cleared = key}. */
void oracle_key_histogram_bf16(const uint16_t* x, int64_t n, uint64_t* hist /* 32768 */) {
    memset(hist, 0, 32768 * sizeof(uint64_t));
    for (int64_t i = 0; i < n; ++i) hist[x[i] & 0x7FFF] += 1;
}

/* ---- retained values in 8 bits ------------------------------------------- */

/* Min-k retains the LARGEST magnitudes, so the retained values of a tensor span few binades: eight bits hold
 * them well.  The code is a small floating-point number, sign | e (3 bits) | m (4 bits), scaled by the tensor's
 * top exponent field E_top (the largest exponent field among its finite retained values):
 *     u = 2^(E_top - 127 - 10)                    one step of the lowest binade
 *     e = 0:       value = m * u                  (zero and the sub-binade below 16 u)
 *     e = 1 .. 7:  value = (16 + m) * 2^(e-1) * u (the top binade, e = 7, is the binade of E_top)
 * A value is rounded to the nearest code, ties to even (in code order); above the largest code it saturates,
 * and so do Inf and NaN patterns.  With E_top < 11 (everything below 2^-116) every code is zero.
 * |decode(encode(v)) - v| <= |v| / 32 for 16 u <= |v| <= the largest code, and <= u / 2 below. */
uint32_t oracle_q8_top_exponent(const uint16_t* values, int64_t k) {
    uint32_t top = 0;
    for (int64_t i = 0; i < k; ++i) {
        const uint32_t e = (values[i] >> 7) & 0xFFu;
        if (e != 0xFFu && e > top) top = e;
    }
    return top;
}

uint8_t oracle_q8_encode_one(uint16_t v, uint32_t e_top) {
    const uint8_t sign = (uint8_t)((v >> 8) & 0x80u);
    if (((v >> 7) & 0xFFu) == 0xFFu) return (uint8_t)(sign | 0x7Fu);
    if (e_top < 11) return sign;
    const double a = ldexp(fabs(bf16_bits_to_double(v)), 127 + 10 - (int)e_top);   /* |v| / u, exact */
    double code;
    if (a < 16.0) {
        code = rint(a);                                   /* 0 .. 16 (16 is the first code of e = 1) */
    } else {
        int ex;
        (void)frexp(a, &ex);                              /* a in [2^(ex-1), 2^ex): binade e = ex - 4 */
        const int e = ex - 4;
        code = (double)((e - 1) << 4) + rint(ldexp(a, -(e - 1)));   /* mantissa in 16 .. 32; 32 carries into e + 1 */
    }
    if (code > 127.0) code = 127.0;
    return (uint8_t)(sign | (uint8_t)code);
}

uint16_t oracle_q8_decode_one(uint8_t q, uint32_t e_top) {
    const uint16_t sign = (uint16_t)((q & 0x80u) << 8);
    const uint32_t c = q & 0x7Fu;
    if (c == 0 || e_top < 11) return sign;
    const uint32_t e = c >> 4, m = c & 15u;
    const double val = (e == 0) ? ldexp((double)m, (int)e_top - 137) : ldexp((double)(16 + m), (int)e_top - 137 + (int)e - 1);
    return (uint16_t)(sign | oracle_round_to_bf16(val));  /* exact: at most five significant bits */
}

void oracle_q8_encode(const uint16_t* values, int64_t k, uint32_t e_top, uint8_t* codes) {
    for (int64_t i = 0; i < k; ++i) codes[i] = oracle_q8_encode_one(values[i], e_top);
}

void oracle_q8_decode(const uint8_t* codes, int64_t k, uint32_t e_top, uint16_t* values) {
    for (int64_t i = 0; i < k; ++i) values[i] = oracle_q8_decode_one(codes[i], e_top);
}

int oracle_num_threads(void) {
#ifdef _OPENMP
    extern int omp_get_max_threads(void);
    return omp_get_max_threads();
#else
    return 1;
#endif
}
