/*
 * Scalar CPU oracle for few-bit stochastic rounding (FBSR).
 *
 * TEST INFRASTRUCTURE ONLY.  One element at a time, no blocking, no vector
 * code, no code shared with the CUDA library.  It exists so that the CUDA
 * kernels can be compared with it bit for bit; nothing in the product path
 * may call it.
 *
 * What it follows ("On Stochastic Rounding with Few Random Bits"):
 *   Section II, Eq. (1)      value of a triple (s, e, t) in format (K, P, B; M)
 *   Section II-A, Eq. (2)    exponent, clamped at 1-B so subnormals share one lsb
 *   Section II-A, Eq. (3)    scaled significand sigma~ and delta~ = frac(sigma~)
 *   Section II-A, Eq. (5)    sigma = floor(sigma~) + [R(delta~)], exponent
 *                            incremented when sigma = 2^P
 *   Section II-B             R_SRFF(d, n) = d + n 2^-N >= 1
 *                            R_SRF (d, n) = d + (n + 1/2) 2^-N >= 1
 *   Section III-F, Eq. (8)   R_SRC(d, n) = R_SRFF(Round(d 2^N) 2^-N, n), Round =
 *                            nearest, ties to even
 *   Section II-A, Eq. (4)    deterministic modes (no draw): R_TA(d) = d >= 1/2;
 *                            R_TNE = d > 1/2 or (d = 1/2 and floor(sigma~)+1 even); ties-to-odd likewise
 *
 * The input is binary32, so delta~ is the rational r / 2^s with r, s integers.
 * Each predicate is evaluated exactly by clearing denominators in 128-bit
 * integers; there is no floating-point comparison anywhere in the rounding.
 *
 * Outside the paper (its Section II sets these aside): the magnitude is
 * rounded and the sign copied; NaN -> quiet NaN with the sign kept; +-Inf ->
 * +-Inf, or +-M if the format has none; finite |y| > M -> +-M; these elements
 * are not SR-rounded and are excluded from the error sums.
 *
 * Random source (the paper leaves it open): Philox4x32-10, Salmon, Moraes,
 * Dror, Shaw, "Parallel random numbers: as easy as 1, 2, 3", SC'11.
 * Element with global index g and k bits per draw: dpw = 32 / k draws per
 * word, E = 4 dpw elements per generator call, block b = g / E, counter
 * (b lo, b hi, stream, 0), key (seed lo, seed hi), output word (g mod E) / dpw,
 * field g mod dpw counted from the low bits.
 *
 * Parity unpinned by the paper (the library's own definitions, pinned only by the means named): the policy for
 * special and out-of-range values (torch's casts); the optimizer arithmetic of the SGD / Adam / Algorithm-1 steps
 * (exact-rational replay, torch.optim); the block-scale recipe (numpy's frexp); Binary8P4's bias, M and special
 * patterns, which the paper does not print (the P3109 report's values; torch's float8_e4m3fnuz for all but 0x7F).
 *
 * Build: gcc -O2 -std=c11 -ffp-contract=off -fno-fast-math -shared -fPIC
 * (no contraction: every binary32 operation below rounds exactly once).
 */
#include <math.h>
#include <stddef.h>
#include <stdint.h>
#include <string.h>

typedef unsigned __int128 u128;

enum { FMT_BF16 = 0, FMT_FP16 = 1, FMT_E4M3 = 2, FMT_E5M2 = 3, FMT_B8P4 = 4, FMT_COUNT = 5 };
enum { VAR_SRFF = 0, VAR_SRF = 1, VAR_SRC = 2, VAR_RTNE = 3, VAR_RTA = 4, VAR_RTO = 5 };
enum { KIND_FINITE = 0, KIND_NAN = 1, KIND_INF = 2, KIND_SAT = 3 };

typedef struct {
    int K, P, B;
    double M;          /* largest finite value */
    uint32_t max_code; /* encoding of M */
    int has_inf;
    uint32_t inf_code;
    uint32_t nan_code;
    int single_zero;   /* no negative zero: the pattern 1000...0 is the one NaN, and a NaN has no sign */
} format_t;

static const format_t FORMATS[FMT_COUNT] = {
    /* bf16 */ {16, 8, 127, 0x1.FEp127, 0x7F7Fu, 1, 0x7F80u, 0x7FC0u, 0},
    /* fp16 */ {16, 11, 15, 65504.0, 0x7BFFu, 1, 0x7C00u, 0x7E00u, 0},
    /* e4m3 */ {8, 4, 7, 448.0, 0x7Eu, 0, 0u, 0x7Fu, 0},
    /* e5m2 */ {8, 3, 15, 57344.0, 0x7Bu, 1, 0x7Cu, 0x7Fu, 0},
    /* Section IV's target, IEEE WG P3109 Binary8P4: (K, P, B; M) = (8, 4, 8; 224); the all-ones magnitude is
       the infinity, 0x80 the single NaN, and there is one zero. */
    /* b8p4 */ {8, 4, 8, 224.0, 0x7Eu, 1, 0x7Fu, 0x80u, 1},
};

typedef struct {
    uint64_t n_finite, n_up, n_nan, n_inf, n_sat;
    double sum_e, sum_e2, sum_signed_e, sum_abs_e;
} oracle_stats_t;

static uint32_t bits_of(float x) { uint32_t u; memcpy(&u, &x, 4); return u; }

/* ------------------------------------------------------------------ Philox */
void fbsr_oracle_philox4x32_10(const uint32_t ctr[4], const uint32_t key[2], uint32_t out[4])
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

uint32_t fbsr_oracle_draw(uint64_t seed, uint64_t g, int k, uint32_t stream)
{
    uint64_t dpw = 32u / (unsigned)k;
    uint64_t E = 4 * dpw;
    uint64_t b = g / E;
    uint32_t ctr[4] = {(uint32_t)b, (uint32_t)(b >> 32), stream, 0u};
    uint32_t key[2] = {(uint32_t)seed, (uint32_t)(seed >> 32)};
    uint32_t out[4];
    fbsr_oracle_philox4x32_10(ctr, key, out);
    uint64_t w = (g % E) / dpw;
    uint64_t j = g % dpw;
    return (out[w] >> (j * (unsigned)k)) & ((1u << k) - 1u);
}

/* The packed word stream itself: word index W (global) is output W mod 4 of
 * block W / 4.  Element g reads field g mod dpw of word g / dpw. */
void fbsr_oracle_random_words(uint64_t seed, uint64_t first_word, size_t nwords, uint32_t stream,
                              uint32_t* out_words)
{
    for (size_t j = 0; j < nwords; ++j) {
        uint64_t W = first_word + j, b = W / 4;
        uint32_t ctr[4] = {(uint32_t)b, (uint32_t)(b >> 32), stream, 0u};
        uint32_t key[2] = {(uint32_t)seed, (uint32_t)(seed >> 32)};
        uint32_t out[4];
        fbsr_oracle_philox4x32_10(ctr, key, out);
        out_words[j] = out[W % 4];
    }
}

static uint32_t field_of_words(const uint32_t* words, size_t i, int k)
{
    size_t dpw = 32u / (unsigned)k;
    return (words[i / dpw] >> ((i % dpw) * (unsigned)k)) & ((1u << k) - 1u);
}

/* ------------------------------------------------------------- Eq. (1) */
static float decode_f(const format_t* f, uint32_t code)
{
    uint32_t s = (code >> (f->K - 1)) & 1u;
    uint32_t e = (code >> (f->P - 1)) & ((1u << (f->K - f->P)) - 1u);
    uint32_t t = code & ((1u << (f->P - 1)) - 1u);
    uint32_t mag = code & ((1u << (f->K - 1)) - 1u);
    double v;
    if (f->single_zero && code == f->nan_code) return NAN;
    if (f->has_inf && mag == f->inf_code) v = INFINITY;
    else if ((f->has_inf && mag > f->inf_code) || (!f->has_inf && mag == f->nan_code)) v = NAN;
    else if (e == 0) v = ldexp(0.0 + ldexp((double)t, 1 - f->P), 1 - f->B);
    else v = ldexp(1.0 + ldexp((double)t, 1 - f->P), (int)e - f->B);
    float r = (float)v; /* exact: every target value is a binary32 value */
    return s ? -r : r;
}

float fbsr_oracle_decode(int fmt, uint32_t code) { return decode_f(&FORMATS[fmt & 0xFF], code); }

/* ------------------------------------------------ one element, Eq. (2)-(8) */
static uint32_t round_one_f(float y, const format_t* f, int ieee_overflow, int variant, int N, uint32_t n,
                            int* kind_out, int* up_out, double* delta_out)
{
    const int P = f->P, B = f->B;
    uint32_t yb = bits_of(y);
    uint32_t sign = (yb >> 31) << (f->K - 1);
    uint32_t mag = yb & 0x7FFFFFFFu;
    int kind = KIND_FINITE, up = 0;
    double delta = 0.0;
    uint32_t code;

    if (mag > 0x7F800000u) { kind = KIND_NAN; code = f->nan_code; goto done; }
    if (mag == 0x7F800000u) { kind = KIND_INF; code = f->has_inf ? f->inf_code : f->max_code; goto done; }
    if (mag == 0u) { code = 0u; goto done; }
    if ((double)fabsf(y) > f->M) {
        kind = KIND_SAT; code = f->max_code;
        if (ieee_overflow) {
            int e2;
            frexp(f->M, &e2);                                    /* M = m 2^e2, m in [0.5, 1) */
            const double half_ulp = ldexp(1.0, (e2 - 1) - (f->P - 1) - 1);
            /* exactly M + ulp/2 is a tie: it goes to the even neighbour, which is M when M's last bit is 0 */
            const double a = (double)fabsf(y), thr = f->M + half_ulp;
            if (a > thr || (a == thr && (f->max_code & 1u))) code = f->has_inf ? f->inf_code : f->nan_code;
        }
        goto done;
    }

    {
        /* |y| = m * 2^q exactly, m the 24-bit integer significand. */
        uint32_t e32 = mag >> 23, t32 = mag & 0x7FFFFFu;
        uint64_t m = e32 ? (t32 | 0x800000u) : t32;
        int q = (e32 ? (int)e32 : 1) - 150;
        /* floor(log2 |y|) */
        int msb = 63 - __builtin_clzll(m);
        int flog = msb + q;
        int e = flog > 1 - B ? flog : 1 - B;          /* Eq. (2) */
        /* sigma~ = |y| 2^-e 2^(P-1) = m / 2^s,  s = e - q - (P-1) > 0.  Eq. (3) */
        int s = e - q - (P - 1);
        uint64_t fl, r;
        if (s >= 64) {
            /* m < 2^24 so delta~ < 2^-40: with N <= 16 no predicate can hold
               (delta~ + (n + 1/2) 2^-N <= 2^-40 + 1 - 2^-17 < 1; Round(delta~ 2^N) = 0;
               delta~ < 1/2 for the deterministic modes). */
            fl = 0; r = m; up = 0;
            delta = ldexp((double)m, -s);
        } else {
            fl = m >> s;
            r = m & (((uint64_t)1 << s) - 1u);
            delta = ldexp((double)r, -s);            /* exact */
            u128 one = (u128)1;
            if (variant == VAR_SRFF) {
                /* r/2^s + n/2^N >= 1   <=>   r 2^N + n 2^s >= 2^(s+N) */
                up = ((u128)r << N) + ((u128)n << s) >= (one << (s + N));
            } else if (variant == VAR_RTA) {
                up = ((u128)r << 1) >= (one << s);                                   /* delta >= 1/2 */
            } else if (variant == VAR_RTNE || variant == VAR_RTO) {
                u128 twice = (u128)r << 1, den = one << s;
                int next_is_even = ((fl + 1) & 1u) == 0;
                up = twice > den || (twice == den && (variant == VAR_RTNE ? next_is_even : !next_is_even));
            } else if (variant == VAR_SRF) {
                /* r/2^s + (2n+1)/2^(N+1) >= 1 */
                up = ((u128)r << (N + 1)) + ((u128)(2u * n + 1u) << s) >= (one << (s + N + 1));
            } else {
                /* qn = Round(r 2^N / 2^s), nearest, ties to even; then qn + n >= 2^N */
                u128 num = (u128)r << N;
                u128 qn = num >> s;
                u128 rem = num - (qn << s);
                u128 twice = rem << 1, den = one << s;
                if (twice > den || (twice == den && (qn & 1u))) qn += 1;
                up = qn + n >= (one << N);
            }
        }
        uint64_t sigma = fl + (uint64_t)up;            /* Eq. (5) */
        if (sigma == ((uint64_t)1 << P)) { sigma >>= 1; e += 1; }
        uint32_t be, t;
        if (sigma >= ((uint64_t)1 << (P - 1))) { be = (uint32_t)(e + B); t = (uint32_t)(sigma - ((uint64_t)1 << (P - 1))); }
        else { be = 0u; t = (uint32_t)sigma; }
        code = (be << (P - 1)) | t;
    }
done:
    if (kind_out) *kind_out = kind;
    if (up_out) *up_out = up;
    if (delta_out) *delta_out = delta;
    if (f->single_zero && (kind == KIND_NAN || code == 0u)) return code;   /* the NaN and the zero carry no sign */
    return sign | code;
}

uint32_t fbsr_oracle_round_one(float y, int fmt, int variant, int N, uint32_t n,
                               int* kind_out, int* up_out, double* delta_out)
{
    /* bit 8 of fmt selects the paper-literal treatment of finite values beyond M (Section II hands them to the
       deterministic nearest rounding of IEEE 754): below M + ulp(M)/2 they give M, from there on
       the infinity (the NaN code where the format has no infinity).  Without it they saturate to M. */
    return round_one_f(y, &FORMATS[fmt & 0xFF], (fmt >> 8) & 1, variant, N, n, kind_out, up_out, delta_out);
}

static void store_code(void* dst, size_t i, int fmt, uint32_t code)
{
    if (FORMATS[fmt & 0xFF].K == 16) ((uint16_t*)dst)[i] = (uint16_t)code;
    else ((uint8_t*)dst)[i] = (uint8_t)code;
}

static uint32_t load_code(const void* src, size_t i, int fmt)
{
    return FORMATS[fmt & 0xFF].K == 16 ? ((const uint16_t*)src)[i] : ((const uint8_t*)src)[i];
}

/* y = fl32(x * scale), one rounded binary32 multiply (scaled tensors,
 * Section I-A).  A NaN input is passed through untouched so that its sign,
 * which the output keeps, does not depend on how a platform propagates NaNs. */
static float scaled(float x, float scale) { return isnan(x) ? x : x * scale; }

/* NaNs produced by arithmetic (optimizer, accumulation) have a platform
 * dependent sign; they are written as the positive quiet NaN. */
static float arith_result(float y) { return isnan(y) ? NAN : y; }

static int bad_args(int fmt, int variant, int k)
{
    return (fmt & ~0x100) < 0 || (fmt & ~0x100) >= FMT_COUNT || variant < 0 || variant > 5 || k < 1 || k > 16;
}

/* ------------------------------------------------------------ array forms */
int fbsr_oracle_round(const float* src, void* dst, size_t n, int fmt, int variant, int k,
                      uint64_t seed, uint64_t offset, float scale)
{
    if (bad_args(fmt, variant, k)) return 1;
    for (size_t i = 0; i < n; ++i) {
        float y = scaled(src[i], scale);
        uint32_t nr = fbsr_oracle_draw(seed, offset + i, k, 0u);
        store_code(dst, i, fmt, fbsr_oracle_round_one(y, fmt, variant, k, nr, 0, 0, 0));
    }
    return 0;
}

int fbsr_oracle_round_bits(const float* src, void* dst, size_t n, int fmt, int variant, int k,
                           const uint32_t* rand_words, float scale)
{
    if (bad_args(fmt, variant, k)) return 1;
    for (size_t i = 0; i < n; ++i) {
        float y = scaled(src[i], scale);
        uint32_t nr = field_of_words(rand_words, i, k);
        store_code(dst, i, fmt, fbsr_oracle_round_one(y, fmt, variant, k, nr, 0, 0, 0));
    }
    return 0;
}

/* Low-precision source (the paper's own regime, Section III-E and Algorithm 1: BFloat16 or
 * binary16 values rounded to an 8-bit format): the stored code is widened exactly by Eq. (1),
 * scaled, and rounded like any other binary32 value.  A NaN source keeps its sign. */
int fbsr_oracle_round_lp(const void* src, int src_fmt, void* dst, size_t n, int dst_fmt, int variant, int k,
                         uint64_t seed, uint64_t offset, float scale)
{
    if (bad_args(dst_fmt, variant, k) || src_fmt < 0 || src_fmt > 3) return 1;
    for (size_t i = 0; i < n; ++i) {
        float y = scaled(fbsr_oracle_decode(src_fmt, load_code(src, i, src_fmt)), scale);
        uint32_t nr = fbsr_oracle_draw(seed, offset + i, k, 0u);
        store_code(dst, i, dst_fmt, fbsr_oracle_round_one(y, dst_fmt, variant, k, nr, 0, 0, 0));
    }
    return 0;
}

/* Block-scaled tensors (Section I-A: every block of low-precision values carries its own scale factor, here
 * a power of two).  Blocks are 32 consecutive elements of the call.  Per block:
 *   amax = largest finite |x| (0 if none);  e_blk = clamp(floor(log2 amax) - emax, -127, 127) with
 *   emax = floor(log2 M) of the target and e_blk = -127 for amax = 0 or subnormal;
 *   scale byte = e_blk + 127;  y = fl32(x 2^-e_blk);  code = FBSR(y).
 * The recipe (shared power-of-two exponent from the block maximum) is this library's definition. */
int fbsr_oracle_round_mx(const float* src, void* dst, uint8_t* scales, size_t n, int fmt, int variant, int k,
                         uint64_t seed, uint64_t offset)
{
    if (bad_args(fmt, variant, k)) return 1;
    int emax;
    frexp(FORMATS[fmt & 0xFF].M, &emax);
    emax -= 1;                                            /* M = m 2^emax, m in [1, 2) */
    for (size_t b0 = 0; b0 < n; b0 += 32) {
        size_t b1 = b0 + 32 < n ? b0 + 32 : n;
        float amax = 0.0f;
        for (size_t i = b0; i < b1; ++i)
            if (isfinite(src[i]) && fabsf(src[i]) > amax) amax = fabsf(src[i]);
        int e_blk = -127;
        if (amax >= 0x1p-126f) {
            int e2;
            frexpf(amax, &e2);                            /* amax = m 2^e2, m in [0.5, 1) */
            e_blk = (e2 - 1) - emax;
            if (e_blk < -127) e_blk = -127;
            if (e_blk > 127) e_blk = 127;
        }
        scales[b0 / 32] = (uint8_t)(e_blk + 127);
        const float s = ldexpf(1.0f, -e_blk);             /* exact, 2^-127 is a binary32 subnormal */
        for (size_t i = b0; i < b1; ++i) {
            float y = scaled(src[i], s);
            uint32_t nr = fbsr_oracle_draw(seed, offset + i, k, 0u);
            store_code(dst, i, fmt, fbsr_oracle_round_one(y, fmt, variant, k, nr, 0, 0, 0));
        }
    }
    return 0;
}

/* Error of one SR-rounded element in target ulps: e = up - delta~ (the
 * quantity whose mean Section III calls bias).  Group g holds elements
 * [g*group_size, (g+1)*group_size) of this call. */
int fbsr_oracle_round_stats(const float* src, void* dst, size_t n, int fmt, int variant, int k,
                            uint64_t seed, uint64_t offset, float scale, size_t group_size,
                            double* group_sum_e, double* group_sum_e2, oracle_stats_t* total)
{
    if (bad_args(fmt, variant, k)) return 1;
    long double se = 0, se2 = 0, sse = 0, sae = 0, ge = 0, ge2 = 0;
    oracle_stats_t st;
    memset(&st, 0, sizeof st);
    for (size_t i = 0; i < n; ++i) {
        float y = scaled(src[i], scale);
        uint32_t nr = fbsr_oracle_draw(seed, offset + i, k, 0u);
        int kind, up;
        double delta;
        store_code(dst, i, fmt, fbsr_oracle_round_one(y, fmt, variant, k, nr, &kind, &up, &delta));
        if (kind == KIND_FINITE) {
            double e = (double)up - delta;
            st.n_finite++;
            st.n_up += (uint64_t)up;
            se += e; se2 += e * e;
            sse += signbit(y) ? -e : e;
            sae += fabs(e);
            ge += e; ge2 += e * e;
        } else if (kind == KIND_NAN) st.n_nan++;
        else if (kind == KIND_INF) st.n_inf++;
        else st.n_sat++;
        if (group_size && ((i + 1) % group_size == 0 || i + 1 == n)) {
            size_t g = i / group_size;
            if (group_sum_e) group_sum_e[g] = (double)ge;
            if (group_sum_e2) group_sum_e2[g] = (double)ge2;
            ge = 0; ge2 = 0;
        }
    }
    st.sum_e = (double)se; st.sum_e2 = (double)se2;
    st.sum_signed_e = (double)sse; st.sum_abs_e = (double)sae;
    if (total) *total = st;
    return 0;
}

/* Fused optimizer steps.  Algorithm 1 only says: compute the update in the
 * wide format, then SR-round the new weight.  The binary32 operation list is
 * this library's own definition; each line is one correctly rounded operation
 * (fmaf = fused multiply-add). */
int fbsr_oracle_sgd_update(float* w, const float* g, float* m, void* dst, size_t n, int fmt,
                           int variant, int k, uint64_t seed, uint64_t offset, float lr, float mu)
{
    if (bad_args(fmt, variant, k)) return 1;
    for (size_t i = 0; i < n; ++i) {
        float m2 = fmaf(mu, m[i], g[i]);
        float w2 = fmaf(-lr, m2, w[i]);
        m[i] = m2; w[i] = w2;
        uint32_t nr = fbsr_oracle_draw(seed, offset + i, k, 0u);
        store_code(dst, i, fmt, fbsr_oracle_round_one(arith_result(w2), fmt, variant, k, nr, 0, 0, 0));
    }
    return 0;
}

void fbsr_oracle_adam_coefficients(float lr, float beta1, float beta2, int step, float out[4])
{
    double b1t = 1.0, b2t = 1.0;
    for (int t = 0; t < step; ++t) { b1t *= (double)beta1; b2t *= (double)beta2; }
    out[0] = (float)((double)lr / (1.0 - b1t));
    out[1] = (float)(1.0 / sqrt(1.0 - b2t));
    out[2] = (float)(1.0 - (double)beta1);
    out[3] = (float)(1.0 - (double)beta2);
}

int fbsr_oracle_adam_update(float* w, const float* g, float* m, float* v, void* dst, size_t n,
                            int fmt, int variant, int k, uint64_t seed, uint64_t offset,
                            float lr, float beta1, float beta2, float eps, int step)
{
    if (bad_args(fmt, variant, k) || step < 1) return 1;
    float c[4];
    fbsr_oracle_adam_coefficients(lr, beta1, beta2, step, c);
    const float c1 = c[0], c2 = c[1], a1 = c[2], a2 = c[3];
    for (size_t i = 0; i < n; ++i) {
        float a1g = a1 * g[i];
        float m2 = fmaf(beta1, m[i], a1g);
        float a2g = a2 * g[i];
        float a2gg = a2g * g[i];
        float v2 = fmaf(beta2, v[i], a2gg);
        float sq = sqrtf(v2);
        float sc = sq * c2;
        float d = sc + eps;
        float qt = m2 / d;
        float w2 = fmaf(-c1, qt, w[i]);
        m[i] = m2; v[i] = v2; w[i] = w2;
        uint32_t nr = fbsr_oracle_draw(seed, offset + i, k, 0u);
        store_code(dst, i, fmt, fbsr_oracle_round_one(arith_result(w2), fmt, variant, k, nr, 0, 0, 0));
    }
    return 0;
}

/* Algorithm 1, last line (the 8-bit weight rounded from the 16-bit sum of weight and update), with the sum
 * formed in the 16-bit format as the algorithm states: w16 = value(w8) exactly; s = fl32(w16 + u16) rounded to the 16-bit
 * format with ties to even (saturating like every other rounding here); w8' = FBSR(s).  Forming the
 * 16-bit sum by way of one binary32 addition is this library's definition. */
int fbsr_oracle_qat_update(void* w8, const void* u16, size_t n, int w_fmt, int u_fmt, int variant, int k,
                           uint64_t seed, uint64_t offset)
{
    if (bad_args(w_fmt, variant, k) || u_fmt < 0 || u_fmt > 1 || (w_fmt & 0xFF) < 2) return 1;
    for (size_t i = 0; i < n; ++i) {
        float wv = fbsr_oracle_decode(w_fmt, load_code(w8, i, w_fmt));
        float uv = fbsr_oracle_decode(u_fmt, load_code(u16, i, u_fmt));
        float s32 = arith_result(wv + uv);
        uint32_t s16 = fbsr_oracle_round_one(s32, u_fmt, VAR_RTNE, 1, 0u, 0, 0, 0);
        float y = arith_result(fbsr_oracle_decode(u_fmt, s16));
        uint32_t nr = fbsr_oracle_draw(seed, offset + i, k, 0u);
        store_code(w8, i, w_fmt, fbsr_oracle_round_one(y, w_fmt, variant, k, nr, 0, 0, 0));
    }
    return 0;
}

/* Algorithm 1, one whole iteration per parameter, from the gradient on:
 *   w16 = value(w8)  (exact);  g = value(g16);
 *   the algorithm's 16-bit AdamW update: moments in binary32, every operation rounded once, the result rounded to F16:
 *     m' = fma(b1, m, a1 g);  v' = fma(b2, v, (a2 g) g);  d = sqrt(v') c2 + eps;
 *     u32 = fma(-c1, m'/d, -(lr wd) w16);   u16 = RTNE_F16(u32)          (c1, c2, a1, a2 as for Adam)
 *   w8' = FBSR(RTNE_F16(fl32(w16 + u16)))                                 (the step above)
 * The paper gives no arithmetic for the update; this operation list is the library's definition. */
int fbsr_oracle_qat_adamw_step(void* w8, const void* g16, float* m, float* v, size_t n, int w_fmt, int g_fmt,
                               int variant, int k, uint64_t seed, uint64_t offset, float lr, float beta1,
                               float beta2, float eps, float weight_decay, int step)
{
    if (bad_args(w_fmt, variant, k) || g_fmt < 0 || g_fmt > 1 || (w_fmt & 0xFF) < 2 || step < 1) return 1;
    float c[4];
    fbsr_oracle_adam_coefficients(lr, beta1, beta2, step, c);
    const float c1 = c[0], c2 = c[1], a1 = c[2], a2 = c[3];
    const float lrwd = lr * weight_decay;
    for (size_t i = 0; i < n; ++i) {
        float wv = fbsr_oracle_decode(w_fmt, load_code(w8, i, w_fmt));
        float gv = fbsr_oracle_decode(g_fmt, load_code(g16, i, g_fmt));
        float a1g = a1 * gv;
        float m2 = fmaf(beta1, m[i], a1g);
        float a2g = a2 * gv;
        float a2gg = a2g * gv;
        float v2 = fmaf(beta2, v[i], a2gg);
        float sq = sqrtf(v2);
        float sc = sq * c2;
        float d = sc + eps;
        float qt = m2 / d;
        float decay = -lrwd * wv;
        float u32 = fmaf(-c1, qt, decay);
        m[i] = m2; v[i] = v2;
        uint32_t u16 = fbsr_oracle_round_one(arith_result(u32), g_fmt, VAR_RTNE, 1, 0u, 0, 0, 0);
        float uv = fbsr_oracle_decode(g_fmt, u16);
        float s32 = arith_result(wv + uv);
        uint32_t s16 = fbsr_oracle_round_one(s32, g_fmt, VAR_RTNE, 1, 0u, 0, 0, 0);
        float y = arith_result(fbsr_oracle_decode(g_fmt, s16));
        uint32_t nr = fbsr_oracle_draw(seed, offset + i, k, 0u);
        store_code(w8, i, w_fmt, fbsr_oracle_round_one(y, w_fmt, variant, k, nr, 0, 0, 0));
    }
    return 0;
}

/* Low-precision accumulation (last line of Algorithm 1): the stored weight is
 * widened exactly, the update added in binary32, the sum SR-rounded back. */
int fbsr_oracle_accumulate(void* w_lp, const float* update, size_t n, int fmt, int variant, int k,
                           uint64_t seed, uint64_t offset)
{
    if (bad_args(fmt, variant, k)) return 1;
    for (size_t i = 0; i < n; ++i) {
        float wv = fbsr_oracle_decode(fmt, load_code(w_lp, i, fmt));
        float y = arith_result(wv + update[i]);
        uint32_t nr = fbsr_oracle_draw(seed, offset + i, k, 0u);
        store_code(w_lp, i, fmt, fbsr_oracle_round_one(y, fmt, variant, k, nr, 0, 0, 0));
    }
    return 0;
}

/* ------------------------------------------------------------------ formats given at run time
 * Section II describes a format by (K, P, B; M).  The descriptor carries K, P, B, the code of M, and how the
 * codes above it are used: has_inf / inf_code (magnitude code of the infinity), nan_code (magnitude code written
 * for NaN, or the full pattern 1000...0 when single_zero is set), single_zero (one zero, one unsigned NaN).
 * Accepted: K in {8, 16}; 2 <= P <= min(K - 1, 13); 1 <= B <= 127; exponent of M at most 127. */
typedef struct {
    int32_t K, P, B;
    uint32_t max_code;
    int32_t has_inf;
    uint32_t inf_code, nan_code;
    int32_t single_zero;
} oracle_desc_t;

static int desc_to_format(const oracle_desc_t* d, format_t* f)
{
    if (!d || (d->K != 8 && d->K != 16)) return 1;
    if (d->P < 2 || d->P > d->K - 1 || d->P > 13) return 1;
    if (d->B < 1 || d->B > 127) return 1;
    const uint32_t mag_mask = (1u << (d->K - 1)) - 1u;
    if (d->max_code == 0u || d->max_code > mag_mask) return 1;
    if ((int)(d->max_code >> (d->P - 1)) - d->B > 127) return 1;
    if (d->has_inf && (d->inf_code <= d->max_code || d->inf_code > mag_mask)) return 1;
    if (d->single_zero) { if (d->nan_code != (1u << (d->K - 1))) return 1; }
    else if (d->nan_code <= d->max_code || d->nan_code > mag_mask || (d->has_inf && d->nan_code == d->inf_code)) return 1;
    f->K = d->K; f->P = d->P; f->B = d->B; f->max_code = d->max_code; f->has_inf = d->has_inf;
    f->inf_code = d->inf_code; f->nan_code = d->nan_code; f->single_zero = d->single_zero;
    f->M = 0.0;
    /* M is the value of max_code; decode_f only treats inf_code / nan_code specially, and those lie above it */
    f->M = (double)decode_f(f, d->max_code);
    return 0;
}

int fbsr_oracle_desc_valid(const oracle_desc_t* d) { format_t f; return desc_to_format(d, &f) == 0; }

float fbsr_oracle_decode_desc(const oracle_desc_t* d, uint32_t code)
{
    format_t f;
    if (desc_to_format(d, &f)) return NAN;
    return decode_f(&f, code);
}

uint32_t fbsr_oracle_round_one_desc(float y, const oracle_desc_t* d, int ieee_overflow, int variant, int N, uint32_t n,
                                    int* kind_out, int* up_out, double* delta_out)
{
    format_t f;
    if (desc_to_format(d, &f)) return 0xFFFFFFFFu;
    return round_one_f(y, &f, ieee_overflow, variant, N, n, kind_out, up_out, delta_out);
}

int fbsr_oracle_round_desc(const float* src, void* dst, size_t n, const oracle_desc_t* d, int ieee_overflow,
                           int variant, int k, uint64_t seed, uint64_t offset, float scale)
{
    format_t f;
    if (desc_to_format(d, &f) || variant < 0 || variant > 5 || k < 1 || k > 16) return 1;
    for (size_t i = 0; i < n; ++i) {
        float y = scaled(src[i], scale);
        uint32_t nr = fbsr_oracle_draw(seed, offset + i, k, 0u);
        uint32_t code = round_one_f(y, &f, ieee_overflow, variant, k, nr, 0, 0, 0);
        if (f.K == 16) ((uint16_t*)dst)[i] = (uint16_t)code; else ((uint8_t*)dst)[i] = (uint8_t)code;
    }
    return 0;
}
