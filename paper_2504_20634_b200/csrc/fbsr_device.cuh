// Device primitives for few-bit stochastic rounding on sm_100a:
// Philox4x32-10, k-bit field extraction, the per-format integer rounder.
//
// Rounding of one binary32 pattern y to format (K, P, B; M), Section II-A:
//   sh  = number of excess bits = (24 - P) + max(0, (1 - B) - exponent(y))   [Eq. (2)]
//   m   = 24-bit integer significand of |y|, F = m >> sh = floor(sigma~)     [Eq. (3)]
//   r   = low sh bits of m, delta~ = r / 2^sh
// and the predicates of Section II-B / Eq. (8) become integer carries:
//   SRFF  sigma = ((m >> (sh - N)) + n) >> N
//   SRF   sigma = ((m >> (sh - N - 1)) + 2n + 1) >> (N + 1)
//   SRC   sigma = (RTNE(m / 2^(sh - N)) + n) >> N
// (a right shift by a negative amount means a left shift).  The output magnitude
// is ((te - emin) << (P - 1)) + sigma, which carries sigma = 2^P into the exponent
// and subnormal -> normal by the same addition [Eq. (5)].
#pragma once
#include <cstdint>
#include <cuda_runtime.h>

namespace fbsr {

enum { BF16 = 0, FP16 = 1, E4M3 = 2, E5M2 = 3, B8P4 = 4 };
enum { SRFF = 0, SRF = 1, SRC = 2, RTNE = 3, RTA = 4, RTO = 5 };    // 3..5: Section II-A, no draw

// SINGLE_ZERO: the format has one zero and one NaN (the pattern that would be minus zero); neither has a sign.
template <int FMT> struct Format;
template <> struct Format<BF16> {
    static constexpr bool SINGLE_ZERO = false, HAS_INF = true;
    static constexpr int K = 16, P = 8, EMINB = 1;        // (1 - B) + 127: emin as a binary32 biased exponent
    static constexpr uint32_t MAXBITS = 0x7F7F0000u;       // binary32 pattern of M
    static constexpr uint32_t MAXCODE = 0x7F7Fu, INFCODE = 0x7F80u, NANCODE = 0x7FC0u;
};
template <> struct Format<FP16> {
    static constexpr bool SINGLE_ZERO = false, HAS_INF = true;
    static constexpr int K = 16, P = 11, EMINB = 113;
    static constexpr uint32_t MAXBITS = 0x477FE000u;
    static constexpr uint32_t MAXCODE = 0x7BFFu, INFCODE = 0x7C00u, NANCODE = 0x7E00u;
};
template <> struct Format<E4M3> {
    static constexpr bool SINGLE_ZERO = false, HAS_INF = false;
    static constexpr int K = 8, P = 4, EMINB = 121;
    static constexpr uint32_t MAXBITS = 0x43E00000u;
    static constexpr uint32_t MAXCODE = 0x7Eu, INFCODE = 0x7Eu /* no Inf: saturate */, NANCODE = 0x7Fu;
};
template <> struct Format<E5M2> {
    static constexpr bool SINGLE_ZERO = false, HAS_INF = true;
    static constexpr int K = 8, P = 3, EMINB = 113;
    static constexpr uint32_t MAXBITS = 0x47600000u;
    static constexpr uint32_t MAXCODE = 0x7Bu, INFCODE = 0x7Cu, NANCODE = 0x7Fu;
};
// Section IV's target, IEEE WG P3109 Binary8P4 = (8, 4, 8; 224): E4M3's grid at half the scale; the all-ones
// magnitude is the infinity and 0x80 the NaN.
template <> struct Format<B8P4> {
    static constexpr bool SINGLE_ZERO = true, HAS_INF = true;
    static constexpr int K = 8, P = 4, EMINB = 120;
    static constexpr uint32_t MAXBITS = 0x43600000u;
    static constexpr uint32_t MAXCODE = 0x7Eu, INFCODE = 0x7Fu, NANCODE = 0x80u;
};

// A format described at run time, Section II's (K, P, B; M): the members of Format<FMT> as data.
// INFCODE is the code written for an infinite input (the code of M when the format has no infinity).
struct RtFormat {
    int K, P, EMINB;
    uint32_t MAXBITS, MAXCODE, INFCODE, NANCODE;
    bool SINGLE_ZERO, HAS_INF;
};

// ----------------------------------------------------------------------------
// Philox4x32-10 (Salmon et al., SC'11).  The round keys depend only on the
// seed: the key additions are uniform across the grid.
// ----------------------------------------------------------------------------
__device__ __forceinline__ uint4 philox4x32_10(uint32_t c0, uint32_t c1, uint32_t c2, uint32_t c3,
                                               uint32_t k0, uint32_t k1)
{
#pragma unroll
    for (int r = 0; r < 10; ++r) {
        const uint64_t p0 = (uint64_t)0xD2511F53u * c0;
        const uint64_t p1 = (uint64_t)0xCD9E8D57u * c2;
        const uint32_t n0 = (uint32_t)(p1 >> 32) ^ c1 ^ k0;
        const uint32_t n2 = (uint32_t)(p0 >> 32) ^ c3 ^ k1;
        c1 = (uint32_t)p1;
        c3 = (uint32_t)p0;
        c0 = n0;
        c2 = n2;
        k0 += 0x9E3779B9u;
        k1 += 0xBB67AE85u;
    }
    return make_uint4(c0, c1, c2, c3);
}

__device__ __forceinline__ uint4 philox_block(uint64_t block, uint32_t k0, uint32_t k1)
{
    return philox4x32_10((uint32_t)block, (uint32_t)(block >> 32), 0u, 0u, k0, k1);
}

// Outcome of one element for the statistics path.
struct ElementInfo {
    int kind;      // 0 SR-rounded, 1 NaN, 2 Inf, 3 saturated
    int up;        // 1 if the magnitude was rounded up
    double delta;  // delta~ = r / 2^sh, exact in binary64
};

// ----------------------------------------------------------------------------
// One element.  ybits: the (scaled) binary32 pattern; n: the N-bit draw.
// Returns the K-bit code.  VAR and N are ordinary arguments so that the slow
// path can pass run-time values; the tiled kernels pass constants and the
// branches fold away.  The format is an object: Format<FMT> (all members compile-time
// constants, so everything folds as before) or an RtFormat filled in by the host.
// ----------------------------------------------------------------------------
template <class F, bool STATS, bool BF16_SHORTCUT>
__device__ __forceinline__ uint32_t round_core_fmt(const F f, uint32_t ybits, uint32_t n, const int VAR, const int N,
                                                   ElementInfo* info, const bool ieee_overflow)
{
    const int P = f.P;
    const uint32_t mag = ybits & 0x7FFFFFFFu;
    const uint32_t sign = (ybits >> 31) << (f.K - 1);
    uint32_t enc;

    if constexpr (BF16_SHORTCUT) {
        // bfloat16 shares binary32's exponent range: sh is always 16 and the
        // whole of Eq. (2)-(5) is one addition on the magnitude pattern.
        uint32_t t;
        if (VAR >= RTNE) {
            const uint32_t floor_lsb = (mag >> 16) & 1u;
            t = mag + (VAR == RTA ? 0x8000u : 0x7FFFu + (VAR == RTNE ? floor_lsb : floor_lsb ^ 1u));
        } else if (VAR == SRFF || N == 16) {
            t = mag + (n << (16 - N));
        } else if (VAR == SRF) {
            t = mag + (((n << 1) | 1u) << (15 - N));
        } else {
            const int s = 16 - N;                            // bits removed by the pre-round, >= 1
            const uint32_t pre = (mag + ((1u << (s - 1)) - 1u) + ((mag >> s) & 1u)) & ~((1u << s) - 1u);
            t = pre + (n << s);
        }
        enc = t >> 16;
    } else {
        const uint32_t e32 = mag >> 23;
        const uint32_t m = (mag & 0x7FFFFFu) | (e32 ? 0x800000u : 0u);
        const int eb = max((int)e32, 1);
        const int te = max(eb, (int)f.EMINB);
        const int sh = (24 - P) + (te - eb);                 // excess bits, >= 24 - P >= 13
        const uint32_t m6 = m << 6;                          // 6 guard positions keep every shift >= 0
        uint32_t sig;
        if (VAR >= RTNE) {
            const int sa = min(sh + 6, 31);                  // >= 19
            const uint32_t floor_lsb = (m6 >> sa) & 1u;
            const uint32_t inc = VAR == RTA ? (1u << (sa - 1)) : ((1u << (sa - 1)) - 1u) + (VAR == RTNE ? floor_lsb : floor_lsb ^ 1u);
            sig = (m6 + inc) >> sa;
        } else if (VAR == SRFF) {
            const int sa = min(sh - N + 6, 31);
            sig = ((m6 >> sa) + n) >> N;
        } else if (VAR == SRF) {
            const int sa = min(sh - N + 5, 31);
            sig = ((m6 >> sa) + ((n << 1) | 1u)) >> (N + 1);
        } else {
            const int sa = min(sh - N + 6, 31);              // >= 3
            const uint32_t pre = (m6 + ((1u << (sa - 1)) - 1u) + ((m6 >> sa) & 1u)) >> sa;
            sig = (pre + n) >> N;
        }
        enc = ((uint32_t)(te - f.EMINB) << (P - 1)) + sig;
        if constexpr (STATS) {
            const uint32_t fl = m >> min(sh, 31);
            const uint32_t r = sh < 32 ? (m & ((1u << sh) - 1u)) : m;
            info->up = (int)(sig - fl);
            // 2^-sh as a binary64 pattern (sh < 300 keeps it a normal double)
            info->delta = (double)r * __longlong_as_double((long long)(1023 - sh) << 52);
        }
    }
    if constexpr (STATS) info->kind = 0;
    if (mag > f.MAXBITS) {
        if (mag > 0x7F800000u) { enc = f.NANCODE; if constexpr (STATS) info->kind = 1; }
        else if (mag == 0x7F800000u) { enc = f.INFCODE; if constexpr (STATS) info->kind = 2; }
        else {
            // finite and beyond M: saturate, or (Section II read literally) round as IEEE nearest-even does:
            // M below M + ulp/2, the infinity above it (the NaN code for E4M3), the tie to the even neighbour
            enc = f.MAXCODE;
            if constexpr (STATS) info->kind = 3;
            if (ieee_overflow) {
                const uint32_t tie = f.MAXBITS + (1u << (24 - P - 1));
                if (mag > tie || (mag == tie && (f.MAXCODE & 1u))) enc = f.HAS_INF ? f.INFCODE : f.NANCODE;
            }
        }
    }
    if (f.SINGLE_ZERO) {
        if (enc == 0u || enc == f.NANCODE) return enc;        // the zero and the NaN carry no sign
    }
    return enc | sign;
}

template <int FMT, bool STATS>
__device__ __forceinline__ uint32_t round_core(uint32_t ybits, uint32_t n, const int VAR, const int N,
                                               ElementInfo* info, const bool ieee_overflow = false)
{
    return round_core_fmt<Format<FMT>, STATS, FMT == BF16 && !STATS>(Format<FMT>{}, ybits, n, VAR, N, info, ieee_overflow);
}

// ----------------------------------------------------------------------------
// Eight draws of one lane, normalised: element c's field starts at bit
// (c % G) * K of word u[c / G].  The field is never isolated on its own; it is
// shifted straight to where the rounder adds it (two integer instructions).
// ----------------------------------------------------------------------------
template <int K> struct Draws8 {
    static constexpr int DPW = 32 / K;
    static constexpr bool POW2 = (DPW & (DPW - 1)) == 0;
    // fields per normalised word: a whole group must fit in 32 bits and, when two neighbouring words are
    // joined, inside those two words for every starting field (f + G <= 2 dpw)
    static constexpr int G = POW2 ? (DPW >= 8 ? 8 : DPW)
                                  : (8 * K <= 32 && DPW >= 7) ? 8 : (4 * K <= 32 ? 4 : 2);
    static constexpr uint32_t MASK = (1u << K) - 1u;
    uint32_t u[8 / G] = {};

    // Field of element c moved so that its lowest bit lands on bit POS (0 <= POS, POS + K <= 32).
    template <int POS>
    __device__ __forceinline__ uint32_t at(const int c) const
    {
        const int b = (c % G) * K;
        const uint32_t w = u[c / G];
        return (b <= POS ? (w << (POS - b)) : (w >> (b - POS))) & (MASK << POS);
    }

    // acc + (field of element c moved to bit POS).  The field is masked where it sits; the move is written
    // as a multiply by a power of two so that the compiler may fold it with the addition (shift-add or
    // multiply-add, its choice).
    template <int POS>
    __device__ __forceinline__ uint32_t add_at(const int c, const uint32_t acc) const
    {
        const int b = (c % G) * K;
        const uint32_t f = u[c / G] & (MASK << b);
        if (b <= POS) return f * (1u << (POS - b)) + acc;
        return __umulhi(f, 1u << (32 - (b - POS))) + acc;
    }

    // Field of element c without its S lowest bits, at bit 0.
    template <int S>
    __device__ __forceinline__ uint32_t top(const int c) const
    {
        return (u[c / G] >> ((c % G) * K + S)) & (MASK >> S);
    }

    // From the tile's packed word stream; p0 = tile-relative index of the lane's first element.
    __device__ __forceinline__ void from_stream(const uint32_t* wb, const int p0)
    {
        if constexpr (POW2 && DPW >= 8) {
            u[0] = wb[p0 / DPW] >> ((p0 % DPW) * K);
        } else if constexpr (DPW == 4) {
            const uint2 w = *reinterpret_cast<const uint2*>(wb + p0 / 4);
            u[0] = w.x; u[1] = w.y;
        } else if constexpr (DPW == 2) {
            const uint4 w = *reinterpret_cast<const uint4*>(wb + p0 / 2);
            u[0] = w.x; u[1] = w.y; u[2] = w.z; u[3] = w.w;
        } else {
            // Words hold DPW fields in their low DPW*K bits.  Two consecutive words, joined
            // without the unused top bits, always cover a group of G fields.
#pragma unroll
            for (int g = 0; g < 8 / G; ++g) {
                const int p = p0 + g * G, q = p / DPW, f = p - q * DPW;
                const uint64_t joined = (uint64_t)(wb[q] & (uint32_t)((1ull << (DPW * K)) - 1ull)) |
                                        ((uint64_t)wb[q + 1] << (DPW * K));
                u[g] = (uint32_t)(joined >> (f * K));
            }
        }
    }

    // Normalised layout (used where the generator fills the buffer): for draw counts per word that are not a power
    // of two the lane that computes a call writes its E fields as E / G words of G fields each, so that an octet of
    // elements later reads 8 / G ready words instead of joining raw words itself.  Power-of-two counts keep the raw
    // layout, which is already normalised.
    static constexpr int E = 4 * DPW;
    static constexpr int WORDS_PER_CALL = POW2 ? 4 : E / G;
    static_assert(POW2 || E % G == 0, "a call splits into whole groups");

    __device__ __forceinline__ static void store_call(uint32_t* dst, const uint4& o)
    {
        if constexpr (POW2) {
            *reinterpret_cast<uint4*>(dst) = o;
        } else {
            // the call's fields as one bit sequence: each word contributes its low DPW * K bits
            constexpr int B = DPW * K;
            constexpr uint32_t PAYLOAD = (uint32_t)((1ull << B) - 1ull);
            const unsigned __int128 seq = (unsigned __int128)(o.x & PAYLOAD) | ((unsigned __int128)(o.y & PAYLOAD) << B) |
                                          ((unsigned __int128)(o.z & PAYLOAD) << (2 * B)) |
                                          ((unsigned __int128)(o.w & PAYLOAD) << (3 * B));
#pragma unroll
            for (int m = 0; m < WORDS_PER_CALL; ++m) dst[m] = (uint32_t)(seq >> (m * G * K));
        }
    }

    // From the tile's buffer in the normalised layout; p0 = tile-relative index of the lane's first element.
    __device__ __forceinline__ void from_normalised(const uint32_t* wb, const int p0)
    {
        if constexpr (POW2) {
            from_stream(wb, p0);
        } else if constexpr (G == 8) {
            u[0] = wb[p0 / 8];
        } else if constexpr (G == 4) {
            const uint2 w = *reinterpret_cast<const uint2*>(wb + p0 / 4);
            u[0] = w.x; u[1] = w.y;
        } else {
            const uint4 w = *reinterpret_cast<const uint4*>(wb + p0 / 2);
            u[0] = w.x; u[1] = w.y; u[2] = w.z; u[3] = w.w;
        }
    }

    // From one Philox call that serves exactly these 8 elements (two draws per word).
    __device__ __forceinline__ void from_call(const uint4& w)
    {
        static_assert(DPW == 2, "a call serves one lane-row only with two draws per word");
        u[0] = w.x; u[1] = w.y; u[2] = w.z; u[3] = w.w;
    }
};

// ----------------------------------------------------------------------------
// Fast row rounder.  The value is first rescaled by 2^(1 - EMINB) so that the target's
// exponent range starts where binary32's does: target subnormals become binary32
// subnormals (the hardware does the alignment shift of Eq. (2)), target normals are
// scaled exactly, and Eq. (3)-(5) reduce to bfloat16's single addition with
// sh0 = 24 - P excess bits:  code = (pattern + (n << (sh0 - N))) >> sh0.
// The multiply rounds toward zero; below the target's emin it keeps 23 - (P - 1) = sh0
// bits under the target lsb, which is all that SRFF needs for N <= sh0, SRF for
// N <= sh0 - 1, and (with a sticky bit from a second, upward-rounded multiply) the
// nearest-even pre-round of SRC for N <= sh0 - 2.
// For larger N (binary16 with N >= 12..14) the subnormal range needs more bits than the
// rescaled pattern keeps, so two candidates are formed and one selected per element:
//   |y| >= 2^emin : the pattern form; with N >= sh0 it is exact SR on the sh0 excess bits,
//                   which only the top sh0 bits of the draw can influence;
//   |y| <  2^emin : sigma~ 2^N = |y| / 2^(emin - (P-1) - N) converted to an integer (toward
//                   zero for SRFF/SRF, to nearest-even for SRC's pre-round), draw added,
//                   N bits dropped; the biased exponent is 0, so sigma is the code.
// Rows that hold Inf or NaN (or, for bfloat16, |y| > M) are flagged and redone by the caller
// with round_core: the flag comes from floating-point instructions, off the integer pipe.
// ----------------------------------------------------------------------------
template <int FMT, int VAR, int N> struct FastRow {
    using F = Format<FMT>;
    static constexpr int SH0 = 24 - F::P;
    static constexpr bool ALL_BITS = (N == SH0);             // then every variant is exact SR
    static constexpr bool deterministic = VAR >= RTNE;
    static constexpr bool one_regime =
        FMT == BF16 || deterministic ? true
                    : (VAR == SRFF ? N <= SH0 : VAR == SRF ? N <= SH0 - 1 : N <= SH0 - 2);
};

// VALUE_BITS: an upper bound on the significant bits of the values handed in (24 for arbitrary binary32 values; 8 or
// 11 when they are exactly bfloat16 or binary16 values).  A value of b bits loses bits in the rescaled pattern only
// when it lies b + 8 or more binades below the target's emin, where the pattern is below 2^(b - 1); the nearest-even
// pre-round of SRC (and the deterministic modes) looks at the lost bits only to tell a tie at bit POS - 1 from a value
// just above it, and a pattern below 2^(b - 1) is below every such tie once POS >= b: the sticky bit (a second,
// upward-rounded multiply per element) is then never needed.
template <int FMT, int VAR, int N, int VALUE_BITS = 24>
__device__ __forceinline__ bool round_row_fast(const float (&y)[8], const Draws8<N>& d, uint32_t (&t)[8])
{
    using F = Format<FMT>;
    using R = FastRow<FMT, VAR, N>;
    constexpr int SH0 = R::SH0;
    constexpr int EFF = R::deterministic ? VAR : (R::ALL_BITS || (FMT == BF16 && N == 16)) ? SRFF : VAR;
    constexpr int POS = R::deterministic ? SH0 : SH0 - N;     // where the draw (or the half step) is added
    float flag = 0.0f;
    if constexpr (!R::one_regime && N >= SH0) {
        // Draws at least as wide as the excess bits of a normal result (binary16 with N = 13..16).  Both candidates
        // are formed with the code in the top K bits, and the draw enters both as the same term
        // D = n 2^(W - N), W = 32 - K:
        //   |y| >= 2^emin: every variant is exact SR on the sh0 excess bits: (pattern << L) + D; the bits of D below
        //                  the pattern's lowest bit meet zeros and cannot carry;
        //   |y| <  2^emin: floor(sigma~ + n 2^-N) is the top K bits of floor(sigma~ 2^W) + D (SRFF); SRF adds half a
        //                  step more (at N = W one position finer, then one shift); SRC converts sigma~ 2^N to
        //                  nearest-even first.
        static_assert(FMT != BF16 && F::K == 16, "only binary16 has draws wider than its excess bits");
        constexpr int W = 32 - F::K, L = W - SH0;                                       // 16, 3
        static_assert(N <= W && L >= 0, "the draw fits under the code");
        const float rescale = __uint_as_float((uint32_t)(128 - F::EMINB) << 23);        // 2^(1 - EMINB)
        const float min_normal = __uint_as_float((uint32_t)F::EMINB << 23);             // 2^emin
        // sigma~ 2^X = |y| 2^(X + P - 1 - emin); emin = EMINB - 127
        constexpr int X = VAR == SRC ? N : (VAR == SRF && N == W) ? W + 1 : W;
        const float to_steps = __uint_as_float((uint32_t)(X + F::P - 1 + 254 - F::EMINB) << 23);
#pragma unroll
        for (int c = 0; c < 8; ++c) {
            const float a = fabsf(y[c]);
            flag = __fmaf_rn(y[c], 0.0f, flag);
            const uint32_t D = d.template at<W - N>(c);
            const uint32_t u = min(__float_as_uint(__fmul_rz(a, rescale)), F::MAXCODE << SH0);
            const uint32_t hi = u * (1u << L) + D;
            const float steps = __fmul_rn(a, to_steps);                                 // exact below 2^emin
            uint32_t lo;
            if constexpr (VAR == SRFF) lo = __float2uint_rz(steps) + D;
            else if constexpr (VAR == SRF && N < W) lo = __float2uint_rz(steps) + D + (1u << (W - N - 1));
            else if constexpr (VAR == SRF) lo = (__float2uint_rz(steps) + 2u * D + 1u) >> 1;
            else lo = __float2uint_rn(steps) * (1u << (W - N)) + D;
            t[c] = a < min_normal ? lo : hi;
        }
        return flag != flag;
    } else if constexpr (!R::one_regime) {
        static_assert(FMT != BF16 && N >= SH0 - 1, "two-regime form is for draws about as wide as the excess bits");
        const float rescale = __uint_as_float((uint32_t)(128 - F::EMINB) << 23);        // 2^(1 - EMINB)
        const float min_normal = __uint_as_float((uint32_t)F::EMINB << 23);             // 2^emin
        constexpr int EXTRA = (VAR == SRF) ? 1 : 0;                                     // SRF compares half a step finer
        const float to_steps = __uint_as_float((uint32_t)(F::P + N + EXTRA + 253 - F::EMINB) << 23);
#pragma unroll
        for (int c = 0; c < 8; ++c) {
            const float a = fabsf(y[c]);
            flag = __fmaf_rn(y[c], 0.0f, flag);
            // normal range of the target
            const uint32_t u = __float_as_uint(__fmul_rz(a, rescale));
            uint32_t sum;
            if constexpr (N >= SH0) sum = u + d.template top<N - SH0>(c);
            else sum = u + d.template at<1>(c) + ((u >> 1) & 1u);                       // SRC, N = sh0 - 1
            const uint32_t hi = min(sum >> SH0, F::MAXCODE);
            // subnormal range of the target
            const float steps = __fmul_rn(a, to_steps);                                 // exact below 2^emin
            uint32_t lo;
            if constexpr (VAR == SRFF) lo = (__float2uint_rz(steps) + d.template at<0>(c)) >> N;
            else if constexpr (VAR == SRF) lo = (__float2uint_rz(steps) + ((d.template at<0>(c) << 1) | 1u)) >> (N + 1);
            else lo = (__float2uint_rn(steps) + d.template at<0>(c)) >> N;
            t[c] = (a < min_normal ? lo : hi) << (32 - F::K);        // code in the top K bits, like the one-regime form
        }
        return flag != flag;
    } else {
#pragma unroll
    for (int c = 0; c < 8; ++c) {
        uint32_t u;
        if constexpr (FMT == BF16) {
            u = __float_as_uint(y[c]);                        // sign rides along in bit 31
            // |y| + (maxfloat - M) overflows exactly when |y| > M; Inf and NaN propagate.
            const float z = __fadd_rn(fabsf(y[c]), __uint_as_float(0x7B7FFF00u));
            flag = __fmaf_rn(z, 0.0f, flag);
        } else {
            const float rescale = __uint_as_float((uint32_t)(128 - F::EMINB) << 23);   // 2^(1 - EMINB)
            u = __float_as_uint(__fmul_rz(fabsf(y[c]), rescale));
            if constexpr ((EFF == SRC || EFF == RTNE || EFF == RTO) && POS < VALUE_BITS) {
                const uint32_t up = __float_as_uint(__fmul_ru(fabsf(y[c]), rescale));
                u |= (u ^ up) & 1u;                           // sticky: round to odd
            }
            flag = __fmaf_rn(y[c], 0.0f, flag);               // NaN iff y is Inf or NaN
        }
        // Other formats: saturate the pattern first (what is added below stays under one code step), then move
        // it left by L so that the code ends at bit 30: packing then takes whole bytes and needs no shift.
        constexpr int L = FMT == BF16 ? 0 : 31 - (F::K - 1) - SH0;
        if constexpr (FMT != BF16) u = min(u, F::MAXCODE << SH0);
        const uint32_t base = u * (1u << L);
        const uint32_t floor_lsb = ((u >> POS) & 1u) << L;     // used by the nearest-even / nearest-odd forms only
        constexpr uint32_t HALF = POS > 0 ? 1u << (POS > 0 ? POS - 1 + L : 0) : 0u;
        constexpr uint32_t BELOW_HALF = POS > 0 ? ((1u << (POS > 0 ? POS - 1 : 0)) - 1u) << L : 0u;
        uint32_t sum;
        if constexpr (EFF == RTA) {
            sum = base + HALF;                                // ties away: add half a step
        } else if constexpr (EFF == RTNE || EFF == RTO) {
            sum = base + BELOW_HALF + (EFF == RTNE ? floor_lsb : floor_lsb ^ (1u << L));
        } else if constexpr (EFF == SRFF) {
            sum = d.template add_at<POS + L>(c, base);
        } else if constexpr (EFF == SRF) {
            sum = d.template add_at<POS + L>(c, base + HALF);
        } else {
            sum = d.template add_at<POS + L>(c, base + BELOW_HALF + floor_lsb);
        }
        t[c] = sum;                                           // code in the top K bits (bf16: with its sign)
    }
    return flag != flag;
    }
}

// y = fl32(x * scale); a NaN input passes through so that its sign survives.
__device__ __forceinline__ uint32_t scaled_bits(float x, float scale)
{
    const uint32_t xb = __float_as_uint(x);
    if ((xb & 0x7FFFFFFFu) > 0x7F800000u) return xb;
    return __float_as_uint(__fmul_rn(x, scale));
}

// NaNs produced by arithmetic are written as the positive quiet NaN.
__device__ __forceinline__ uint32_t arith_bits(float y)
{
    const uint32_t yb = __float_as_uint(y);
    return (yb & 0x7FFFFFFFu) > 0x7F800000u ? 0x7FC00000u : yb;
}

// Value of a stored code, Eq. (1), widened exactly to binary32.
template <int FMT>
__device__ __forceinline__ float decode_element(uint32_t code)
{
    using F = Format<FMT>;
    constexpr int P = F::P, K = F::K;
    if constexpr (FMT == BF16) {
        return __uint_as_float((code & 0xFFFFu) << 16);
    } else {
        const uint32_t sign = ((code >> (K - 1)) & 1u) << 31;
        const uint32_t mag = code & ((1u << (K - 1)) - 1u);
        const uint32_t e = mag >> (P - 1), t = mag & ((1u << (P - 1)) - 1u);
        if constexpr (F::SINGLE_ZERO) {
            if (code == F::NANCODE) return __uint_as_float(0x7FC00000u);
            if (mag == F::INFCODE) return __uint_as_float(sign | 0x7F800000u);
        } else if constexpr (FMT == E4M3) {
            if (mag == F::NANCODE) return __uint_as_float(sign | 0x7FC00000u);
        } else {
            if (mag > F::INFCODE) return __uint_as_float(sign | 0x7FC00000u);
            if (mag == F::INFCODE) return __uint_as_float(sign | 0x7F800000u);
        }
        uint32_t bits;
        if (e == 0) {
            // subnormal: t 2^(1-P) 2^(1-B), exact in binary32
            const float v = __fmul_rn((float)t, __uint_as_float((uint32_t)(F::EMINB - (P - 1)) << 23));
            bits = __float_as_uint(v);
        } else {
            bits = ((e + (uint32_t)(F::EMINB - 1)) << 23) | (t << (24 - P));
        }
        return __uint_as_float(sign | bits);
    }
}

}  // namespace fbsr
