// Kernels for few-bit stochastic rounding on sm_100a.
//
// Kernels:
//
//  * tile_kernel: the bandwidth path.  A warp owns a tile of ROWS rows of 256
//    consecutive elements; in each row a lane owns 8 consecutive elements, so a
//    warp instruction reads 1 KiB of binary32 input (one 256-bit load per lane)
//    and writes 512 contiguous bytes of 16-bit codes (one 128-bit store per
//    lane) or 256 bytes of 8-bit codes.  The tile size is chosen per k so that a
//    tile is a whole number of Philox calls, evenly spread over the 32 lanes;
//    the words go through a per-warp shared-memory buffer laid out exactly like
//    the packed word stream of the interface, from which every lane picks the
//    fields of its own elements.  With two draws per word a Philox call serves
//    exactly one lane's 8 elements and the buffer is skipped.
//
//  * general_coalesced_kernel / generic_kernel: any pointer alignment, any offset, heads and
//    tails, scalar loads and stores, run-time k and variant.  The first (no statistics) gives a
//    warp 32 generator calls and walks their elements 32 at a time, so accesses are coalesced;
//    the second (with statistics, used for the edges of the statistics call) gives each thread
//    one call.
//
//  * staged_tile_kernel (fbsr_round with pointers of any element alignment), stats_tile_kernel
//    (rounding plus integer error sums): the tile structure of tile_kernel, described where
//    they are defined.
//
// An "Op" supplies the value to be rounded: the scaled input (fbsr_round), the
// freshly updated master weight (SGD-momentum, Adam) or the widened stored
// weight plus its update (accumulate).
#pragma once
#include <cuda_bf16.h>
#include <cuda_fp16.h>

#include "fbsr_device.cuh"

namespace fbsr {

// Launch shape and prefetch depth, as measured on B200 (2^27..2^28 elements):
constexpr int WARPS_PER_CTA = 8;
constexpr int ROW_BATCH = 4;            // rows whose loads are issued before the first row is consumed
constexpr int MIN_CTAS_ROUND = 4;       // resident CTAs the compiler must allow for the rounding ops (caps registers at 64)
constexpr int MIN_CTAS_SGD = 2;         // the optimizer ops hold three or four rows of state per row in flight
constexpr int MIN_CTAS_ADAM = 2;
// the fused Algorithm-1 step: (rows in flight, resident CTAs) = (1, 4) gave 6.4-6.6 TB/s, (2, 3) 6.3-6.7,
// (2, 2) 5.6-5.8, (1, 6) 6.0-6.1
constexpr int QATADAM_BATCH = 1;
constexpr int QATADAM_MIN_CTAS = 4;
constexpr int CTA_THREADS = WARPS_PER_CTA * 32;
constexpr int ROW_ELEMS = 256;          // 32 lanes x 8 elements

template <int K, int OCT = 1> struct Tile {
    static constexpr int DPW = 32 / K;                        // draws per word
    static constexpr int E = 4 * DPW;                         // elements per Philox call
    static constexpr bool POW2 = (DPW & (DPW - 1)) == 0;
    // Power-of-two dpw: 4 lane-rows of 256 elements (1024) always hold whole calls.  Otherwise the smallest
    // number of them that does (dpw, or dpw/2 when dpw is even), doubled while below 4; and doubled once more
    // if an op that takes OCT octets per lane could not split it into whole rows of 256 * OCT elements.
    static constexpr int R0 = (DPW % 2 == 0) ? DPW / 2 : DPW;
    static constexpr int ROWS1 = POW2 ? 4 : (R0 >= 4 ? R0 : R0 * ((4 + R0 - 1) / R0));
    static constexpr int ELEMS = ROWS1 * ROW_ELEMS * (ROWS1 % OCT == 0 ? 1 : 2);
    static constexpr int CALLS = ELEMS / E;                   // Philox calls per tile
    static constexpr int WORDS = ELEMS / DPW;                 // random words per tile
    static constexpr int BUFFER_WORDS = CALLS * Draws8<K>::WORDS_PER_CALL;   // of the generator-filled buffer
    static constexpr uint32_t MASK = (1u << K) - 1u;
    static_assert(ELEMS % E == 0, "a tile must hold whole Philox calls");
};

// ---------------------------------------------------------------------------- vector memory access
#define FBSR_STORE __stcs          // streaming store: the codes are not read again by this kernel
struct F8 { float4 a, b; };

__device__ __forceinline__ F8 load_f8_stream(const float* p)
{
    // 256-bit read-only load that does not allocate in L1: the data is used once.
    F8 v;
    asm volatile("ld.global.nc.L1::no_allocate.L2::evict_first.v8.f32 {%0,%1,%2,%3,%4,%5,%6,%7}, [%8];"
                 : "=f"(v.a.x), "=f"(v.a.y), "=f"(v.a.z), "=f"(v.a.w),
                   "=f"(v.b.x), "=f"(v.b.y), "=f"(v.b.z), "=f"(v.b.w)
                 : "l"(p));
    return v;
}

__device__ __forceinline__ F8 load_f8(const float* p)
{
    F8 v;
    asm volatile("ld.global.v8.f32 {%0,%1,%2,%3,%4,%5,%6,%7}, [%8];"
                 : "=f"(v.a.x), "=f"(v.a.y), "=f"(v.a.z), "=f"(v.a.w),
                   "=f"(v.b.x), "=f"(v.b.y), "=f"(v.b.z), "=f"(v.b.w)
                 : "l"(p));
    return v;
}

__device__ __forceinline__ void store_f8(float* p, const float (&y)[8])
{
    asm volatile("st.global.v8.f32 [%0], {%1,%2,%3,%4,%5,%6,%7,%8};"
                 :: "l"(p), "f"(y[0]), "f"(y[1]), "f"(y[2]), "f"(y[3]),
                    "f"(y[4]), "f"(y[5]), "f"(y[6]), "f"(y[7]) : "memory");
}

__device__ __forceinline__ void unpack(const F8& v, float (&x)[8])
{
    x[0] = v.a.x; x[1] = v.a.y; x[2] = v.a.z; x[3] = v.a.w;
    x[4] = v.b.x; x[5] = v.b.y; x[6] = v.b.z; x[7] = v.b.w;
}

// Words that 8 packed codes occupy.
template <int FMT> struct WordsPerOctet { static constexpr int value = Format<FMT>::K == 16 ? 4 : 2; };

// 8 plain codes -> packed words.
template <int FMT>
__device__ __forceinline__ void pack_codes8(const uint32_t (&c)[8], uint32_t* out)
{
    if constexpr (Format<FMT>::K == 16) {
        out[0] = c[0] | (c[1] << 16); out[1] = c[2] | (c[3] << 16);
        out[2] = c[4] | (c[5] << 16); out[3] = c[6] | (c[7] << 16);
    } else {
        out[0] = c[0] | (c[1] << 8) | (c[2] << 16) | (c[3] << 24);
        out[1] = c[4] | (c[5] << 8) | (c[6] << 16) | (c[7] << 24);
    }
}

// N packed words -> one streaming vector store (8, 16 or 32 bytes).
template <int NWORDS>
__device__ __forceinline__ void store_words(void* p, const uint32_t (&w)[NWORDS])
{
    static_assert(NWORDS == 2 || NWORDS == 4 || NWORDS == 8, "8-, 16- or 32-byte stores");
    if constexpr (NWORDS == 2) {
        FBSR_STORE(reinterpret_cast<uint2*>(p), make_uint2(w[0], w[1]));
    } else if constexpr (NWORDS == 4) {
        FBSR_STORE(reinterpret_cast<uint4*>(p), make_uint4(w[0], w[1], w[2], w[3]));
    } else {
        FBSR_STORE(reinterpret_cast<uint4*>(p), make_uint4(w[0], w[1], w[2], w[3]));
        FBSR_STORE(reinterpret_cast<uint4*>(p) + 1, make_uint4(w[4], w[5], w[6], w[7]));
    }
}

template <int FMT>
__device__ __forceinline__ void store_codes8(void* dst, size_t elem, const uint32_t (&c)[8])
{
    uint32_t w[WordsPerOctet<FMT>::value];
    pack_codes8<FMT>(c, w);
    store_words<WordsPerOctet<FMT>::value>(static_cast<char*>(dst) + elem * (Format<FMT>::K / 8), w);
}

template <int FMT>
__device__ __forceinline__ void store_code1(void* dst, size_t elem, uint32_t c)
{
    if constexpr (Format<FMT>::K == 16) static_cast<uint16_t*>(dst)[elem] = (uint16_t)c;
    else static_cast<uint8_t*>(dst)[elem] = (uint8_t)c;
}

// ---------------------------------------------------------------------------- Ops
// fetch(): issue the loads of 8 consecutive elements; finish(): produce the 8
// values to round (and write back whatever state the op updates);
// exact_bits(): the pattern that the element-wise rounder must see for element c
// (differs from the value's own bits only for NaN, whose sign rule depends on the op);
// scalar(): the same for one element on the slow path.

struct RoundOp {
    static constexpr int BATCH = ROW_BATCH, MIN_CTAS = MIN_CTAS_ROUND, OCTETS = 1;
    const float* src;
    float scale;
    struct Regs { F8 x; };
    __device__ __forceinline__ void fetch(size_t elem, Regs& r) const { r.x = load_f8_stream(src + elem); }
    __device__ __forceinline__ void finish(size_t, const Regs& r, float (&y)[8]) const
    {
        float x[8];
        unpack(r.x, x);
#pragma unroll
        for (int c = 0; c < 8; ++c) y[c] = __fmul_rn(x[c], scale);
    }
    __device__ __forceinline__ uint32_t exact_bits(const Regs& r, int c, float y) const
    {
        float x[8];
        unpack(r.x, x);
        return y != y ? __float_as_uint(x[c]) : __float_as_uint(y);   // a NaN keeps the input's sign
    }
    __device__ __forceinline__ uint32_t scalar(size_t i) const { return scaled_bits(src[i], scale); }
};

// Block-scaled rounding: 32 consecutive elements (4 lanes of a row) share a power-of-two scale taken from
// their largest finite magnitude; the scale byte is written by the first lane of the block.
template <int FMT>
struct MxOp {
    static constexpr int BATCH = ROW_BATCH, MIN_CTAS = MIN_CTAS_ROUND, OCTETS = 1;
    static constexpr int EMAX = (int)(Format<FMT>::MAXBITS >> 23) - 127;        // floor(log2 M)
    const float* src; uint8_t* scales; size_t n;
    struct Regs { F8 x; };
    __device__ __forceinline__ static int block_exponent(uint32_t amax_bits)
    {
        const int e = (int)(amax_bits >> 23) - 127 - EMAX;                       // subnormal or zero amax clamps to -127
        return max(-127, min(127, e));
    }
    __device__ __forceinline__ static float inverse_scale(int e_blk)
    {
        const uint32_t field = (uint32_t)(127 - e_blk);                          // 0..254; 0 means 2^-127, a subnormal
        return __uint_as_float(field ? field << 23 : 0x00400000u);
    }
    __device__ __forceinline__ static uint32_t finite_magnitude(float v)
    {
        const uint32_t m = __float_as_uint(v) & 0x7FFFFFFFu;
        return m < 0x7F800000u ? m : 0u;
    }
    __device__ __forceinline__ void fetch(size_t elem, Regs& r) const { r.x = load_f8_stream(src + elem); }
    __device__ __forceinline__ void finish(size_t elem, const Regs& r, float (&y)[8]) const
    {
        float x[8];
        unpack(r.x, x);
        // largest magnitude pattern of the block, Inf and NaN included at first: they are rare, and a block that holds
        // one (its four lanes see the same maximum, so they decide alike) repeats the reduction over finite values only
        uint32_t m = 0u;
#pragma unroll
        for (int c = 0; c < 8; ++c) m = max(m, __float_as_uint(x[c]) & 0x7FFFFFFFu);
        m = max(m, __shfl_xor_sync(0xFFFFFFFFu, m, 1));
        m = max(m, __shfl_xor_sync(0xFFFFFFFFu, m, 2));
        const bool special = m >= 0x7F800000u;
        const uint32_t redo_lanes = __ballot_sync(0xFFFFFFFFu, special);
        if (special) {
            m = 0u;
#pragma unroll
            for (int c = 0; c < 8; ++c) m = max(m, finite_magnitude(x[c]));
            m = max(m, __shfl_xor_sync(redo_lanes, m, 1));
            m = max(m, __shfl_xor_sync(redo_lanes, m, 2));
        }
        const int e_blk = block_exponent(m);
        const float s = inverse_scale(e_blk);
#pragma unroll
        for (int c = 0; c < 8; ++c) y[c] = __fmul_rn(x[c], s);
        if ((threadIdx.x & 3) == 0) scales[elem / 32] = (uint8_t)(e_blk + 127);
    }
    __device__ __forceinline__ uint32_t exact_bits(const Regs& r, int c, float y) const
    {
        float x[8];
        unpack(r.x, x);
        return y != y ? __float_as_uint(x[c]) : __float_as_uint(y);
    }
    __device__ __forceinline__ uint32_t scalar(size_t i) const
    {
        const size_t b0 = i / 32 * 32, b1 = b0 + 32 < n ? b0 + 32 : n;
        uint32_t m = 0u;
        for (size_t j = b0; j < b1; ++j) m = max(m, finite_magnitude(src[j]));
        const int e_blk = block_exponent(m);
        if (i == b0) scales[i / 32] = (uint8_t)(e_blk + 127);
        return scaled_bits(src[i], inverse_scale(e_blk));
    }
};

// Significant bits of the values an op hands to the row rounder: 24 unless the op declares VALUE_BITS.
template <class Op, class = void> struct ValueBits { static constexpr int value = 24; };
template <class Op> struct ValueBits<Op, decltype((void)Op::VALUE_BITS)> { static constexpr int value = Op::VALUE_BITS; };

// Source already in a 16-bit format: widen exactly (Eq. (1)), then scale.  POW2_SCALE (decided by the host): the
// scale is a power of two, so the scaled value still has the source's 8 or 11 significant bits.
template <int SRC, bool POW2_SCALE = false>
struct LpSrcOp {
    static_assert(SRC == BF16 || SRC == FP16, "16-bit sources");
    static constexpr int VALUE_BITS = POW2_SCALE ? (SRC == BF16 ? 8 : 11) : 24;
    // two octets per lane: one 256-bit load of 16 codes, one 128-bit store of 16 eight-bit codes
    static constexpr int BATCH = ROW_BATCH, MIN_CTAS = MIN_CTAS_ROUND, OCTETS = 2;
    const void* src;
    float scale;
    struct Regs { uint32_t c[8]; };
    __device__ __forceinline__ void fetch(size_t elem, Regs& r) const
    {
        const uint16_t* p = static_cast<const uint16_t*>(src) + elem;
        asm volatile("ld.global.nc.L1::no_allocate.L2::evict_first.v8.u32 {%0,%1,%2,%3,%4,%5,%6,%7}, [%8];"
                     : "=r"(r.c[0]), "=r"(r.c[1]), "=r"(r.c[2]), "=r"(r.c[3]),
                       "=r"(r.c[4]), "=r"(r.c[5]), "=r"(r.c[6]), "=r"(r.c[7]) : "l"(p));
    }
    __device__ __forceinline__ void finish(size_t, const Regs& r, int o, float (&y)[8]) const
    {
#pragma unroll
        for (int c = 0; c < 8; ++c) {
            const uint32_t w = r.c[4 * o + (c >> 1)];
            float v;
            if constexpr (SRC == BF16) v = __uint_as_float((c & 1) ? (w & 0xFFFF0000u) : (w << 16));
            else v = __half2float(__ushort_as_half((unsigned short)((c & 1) ? (w >> 16) : (w & 0xFFFFu))));
            y[c] = __fmul_rn(v, scale);
        }
    }
    __device__ __forceinline__ uint32_t exact_bits(const Regs& r, int o, int c, float y) const
    {
        // a NaN keeps the sign of the stored code
        const uint32_t w = r.c[4 * o + (c >> 1)];
        const uint32_t code = (c & 1) ? (w >> 16) : (w & 0xFFFFu);
        return y != y ? __float_as_uint(decode_element<SRC>(code)) : __float_as_uint(y);
    }
    __device__ __forceinline__ uint32_t scalar(size_t i) const
    {
        const float v = decode_element<SRC>(static_cast<const uint16_t*>(src)[i]);
        return scaled_bits(v, scale);
    }
};

// m' = fma(mu, m, g);  w' = fma(-lr, m', w)
struct SgdOp {
    static constexpr int BATCH = ROW_BATCH >= 2 ? ROW_BATCH / 2 : 1, MIN_CTAS = MIN_CTAS_SGD, OCTETS = 1;
    float* w; const float* g; float* m;
    float neg_lr, mu;
    struct Regs { F8 w, g, m; };
    __device__ __forceinline__ void step(float& wv, float gv, float& mv) const
    {
        mv = __fmaf_rn(mu, mv, gv);
        wv = __fmaf_rn(neg_lr, mv, wv);
    }
    __device__ __forceinline__ void fetch(size_t elem, Regs& r) const
    {
        r.w = load_f8(w + elem); r.g = load_f8_stream(g + elem); r.m = load_f8(m + elem);
    }
    __device__ __forceinline__ void finish(size_t elem, const Regs& r, float (&y)[8]) const
    {
        float gv[8], mv[8];
        unpack(r.w, y); unpack(r.g, gv); unpack(r.m, mv);
#pragma unroll
        for (int c = 0; c < 8; ++c) step(y[c], gv[c], mv[c]);
        store_f8(w + elem, y); store_f8(m + elem, mv);
    }
    __device__ __forceinline__ uint32_t exact_bits(const Regs&, int, float y) const { return arith_bits(y); }
    __device__ __forceinline__ uint32_t scalar(size_t i) const
    {
        float wv = w[i], mv = m[i];
        step(wv, g[i], mv);
        w[i] = wv; m[i] = mv;
        return arith_bits(wv);
    }
};

// m' = fma(b1, m, a1 g); v' = fma(b2, v, (a2 g) g); d = sqrt(v') c2 + eps; w' = fma(-c1, m'/d, w)
struct AdamOp {
    static constexpr int BATCH = ROW_BATCH >= 2 ? ROW_BATCH / 2 : 1, MIN_CTAS = MIN_CTAS_ADAM, OCTETS = 1;
    float* w; const float* g; float* m; float* v;
    float beta1, beta2, eps, neg_c1, c2, a1, a2;
    struct Regs { F8 w, g, m, v; };
    __device__ __forceinline__ void step(float& wv, float gv, float& mv, float& vv) const
    {
        mv = __fmaf_rn(beta1, mv, __fmul_rn(a1, gv));
        vv = __fmaf_rn(beta2, vv, __fmul_rn(__fmul_rn(a2, gv), gv));
        const float d = __fadd_rn(__fmul_rn(__fsqrt_rn(vv), c2), eps);
        wv = __fmaf_rn(neg_c1, __fdiv_rn(mv, d), wv);
    }
    __device__ __forceinline__ void fetch(size_t elem, Regs& r) const
    {
        r.w = load_f8(w + elem); r.g = load_f8_stream(g + elem);
        r.m = load_f8(m + elem); r.v = load_f8(v + elem);
    }
    __device__ __forceinline__ void finish(size_t elem, const Regs& r, float (&y)[8]) const
    {
        float gv[8], mv[8], vv[8];
        unpack(r.w, y); unpack(r.g, gv); unpack(r.m, mv); unpack(r.v, vv);
#pragma unroll
        for (int c = 0; c < 8; ++c) step(y[c], gv[c], mv[c], vv[c]);
        store_f8(w + elem, y); store_f8(m + elem, mv); store_f8(v + elem, vv);
    }
    __device__ __forceinline__ uint32_t exact_bits(const Regs&, int, float y) const { return arith_bits(y); }
    __device__ __forceinline__ uint32_t scalar(size_t i) const
    {
        float wv = w[i], mv = m[i], vv = v[i];
        step(wv, g[i], mv, vv);
        w[i] = wv; m[i] = mv; v[i] = vv;
        return arith_bits(wv);
    }
};

// Four stored 8-bit codes (one 32-bit word, low byte first) widened exactly to binary32 (Eq. (1)) by way of
// binary16, which holds every value of both 8-bit formats: E5M2 is the upper byte of a binary16 pattern,
// E4M3 has a hardware convert for pairs.  NaN codes become NaNs (the sign rule is applied by the caller).
// Binary8P4 is E4M3's grid at half the scale (exact in binary16), except for the all-ones magnitude (the
// infinity) and the pattern 0x80 (the NaN), which are patched per byte.
template <int FMT>
__device__ __forceinline__ void decode4(uint32_t w, float (&v)[4])
{
    static_assert(Format<FMT>::K == 8, "8-bit formats");
    uint32_t h01, h23;
    if constexpr (FMT == B8P4) {
        asm("cvt.rn.f16x2.e4m3x2 %0, %1;" : "=r"(h01) : "h"((unsigned short)(w & 0xFFFFu)));
        asm("cvt.rn.f16x2.e4m3x2 %0, %1;" : "=r"(h23) : "h"((unsigned short)(w >> 16)));
        // the halving is exact in binary16 as well (the smallest E4M3 value is 2^-9), and there it takes two at a time
        const __half2 half = __float2half2_rn(0.5f);
        const float2 a = __half22float2(__hmul2(*reinterpret_cast<const __half2*>(&h01), half));
        const float2 b = __half22float2(__hmul2(*reinterpret_cast<const __half2*>(&h23), half));
        v[0] = a.x; v[1] = a.y; v[2] = b.x; v[3] = b.y;
        // bit 7 of a byte: its magnitude is all ones (the infinity) / its magnitude is zero and its sign is set (the NaN)
        const uint32_t mag = w & 0x7F7F7F7Fu;
        const uint32_t special = ((mag + 0x01010101u) | (~(mag + 0x7F7F7F7Fu) & w)) & 0x80808080u;
        if (special) {
#pragma unroll
            for (int c = 0; c < 4; ++c) {
                const uint32_t code = (w >> (8 * c)) & 0xFFu;
                if ((code & 0x7Fu) == 0x7Fu) v[c] = __uint_as_float(((code & 0x80u) << 24) | 0x7F800000u);
                if (code == 0x80u) v[c] = __uint_as_float(0x7FC00000u);
            }
        }
        return;
    } else if constexpr (FMT == E5M2) {
        h01 = __byte_perm(w, 0u, 0x1404);                  // bytes [0, b0, 0, b1]
        h23 = __byte_perm(w, 0u, 0x3424);                  // bytes [0, b2, 0, b3]
    } else {
        asm("cvt.rn.f16x2.e4m3x2 %0, %1;" : "=r"(h01) : "h"((unsigned short)(w & 0xFFFFu)));
        asm("cvt.rn.f16x2.e4m3x2 %0, %1;" : "=r"(h23) : "h"((unsigned short)(w >> 16)));
    }
    const float2 a = __half22float2(*reinterpret_cast<const __half2*>(&h01));
    const float2 b = __half22float2(*reinterpret_cast<const __half2*>(&h23));
    v[0] = a.x; v[1] = a.y; v[2] = b.x; v[3] = b.y;
}

// y = fl32(value(w_lp) + u); the codes are rewritten in place by the caller of finish()
template <int FMT>
struct AccumOp {
    static constexpr int BATCH = ROW_BATCH, MIN_CTAS = MIN_CTAS_ROUND, OCTETS = 1;
    const void* w_lp; const float* u;
    struct Regs { F8 u; uint4 c; };
    __device__ __forceinline__ void fetch(size_t elem, Regs& r) const
    {
        r.u = load_f8_stream(u + elem);
        if constexpr (Format<FMT>::K == 16) {
            r.c = *reinterpret_cast<const uint4*>(static_cast<const uint16_t*>(w_lp) + elem);
        } else {
            const uint2 t = *reinterpret_cast<const uint2*>(static_cast<const uint8_t*>(w_lp) + elem);
            r.c = make_uint4(t.x, t.y, 0u, 0u);
        }
    }
    __device__ __forceinline__ uint32_t exact_bits(const Regs&, int, float y) const { return arith_bits(y); }
    __device__ __forceinline__ void finish(size_t, const Regs& r, float (&y)[8]) const
    {
        float uv[8];
        unpack(r.u, uv);
        const uint32_t cw[4] = {r.c.x, r.c.y, r.c.z, r.c.w};
        if constexpr (Format<FMT>::K == 8) {
            float lo[4], hi[4];
            decode4<FMT>(cw[0], lo);
            decode4<FMT>(cw[1], hi);
#pragma unroll
            for (int c = 0; c < 4; ++c) { y[c] = __fadd_rn(lo[c], uv[c]); y[c + 4] = __fadd_rn(hi[c], uv[c + 4]); }
        } else {
#pragma unroll
            for (int c = 0; c < 8; ++c) {
                const uint32_t code = (cw[c >> 1] >> ((c & 1) * 16)) & 0xFFFFu;
                y[c] = __fadd_rn(decode_element<FMT>(code), uv[c]);
            }
        }
    }
    __device__ __forceinline__ uint32_t scalar(size_t i) const
    {
        uint32_t code;
        if constexpr (Format<FMT>::K == 16) code = static_cast<const uint16_t*>(w_lp)[i];
        else code = static_cast<const uint8_t*>(w_lp)[i];
        return arith_bits(__fadd_rn(decode_element<FMT>(code), u[i]));
    }
};

// Algorithm 1, last line: w16 = value(w8); s = RTNE_16(fl32(w16 + u16)); the caller of finish() rounds s to 8 bits.
template <int WF, int UF>
struct QatOp {
    static_assert(Format<WF>::K == 8 && (UF == BF16 || UF == FP16), "8-bit weights, 16-bit updates");
    static constexpr int VALUE_BITS = UF == BF16 ? 8 : 11;              // the sum is a value of the 16-bit format
    // two octets per lane: 16 weight codes (128 bits) and 16 update codes (256 bits) in, 16 weight codes out
    static constexpr int BATCH = ROW_BATCH >= 2 ? ROW_BATCH / 2 : 1, MIN_CTAS = MIN_CTAS_ROUND, OCTETS = 2;
    const void* w8; const void* u16;
    struct Regs { uint32_t w[4]; uint32_t u[8]; };
    __device__ __forceinline__ static float sum16(uint32_t wcode, uint32_t ucode)
    {
        return sum16v<true>(decode_element<WF>(wcode), ucode);
    }
    // EXACT: round to the 16-bit format with ties to even, a finite sum beyond its largest value saturating.
    // !EXACT: the plain hardware conversion, which turns such a sum into an infinity instead; the row is then
    // flagged like any row holding Inf or NaN and redone through exact_bits(), so the check is paid only there.
    template <bool EXACT>
    __device__ __forceinline__ static float sum16v(float wv, uint32_t ucode)
    {
        const float uv = UF == BF16 ? __uint_as_float(ucode << 16) : __half2float(__ushort_as_half((unsigned short)ucode));
        float s = __fadd_rn(wv, uv);
        if constexpr (EXACT) {
            const float m16 = __uint_as_float(Format<UF>::MAXBITS);
            const float a = fabsf(s);
            if (a > m16 && a < __uint_as_float(0x7F800000u)) s = copysignf(m16, s);
        }
        if constexpr (UF == BF16) return __bfloat162float(__float2bfloat16_rn(s));
        else return __half2float(__float2half_rn(s));
    }
    __device__ __forceinline__ void fetch(size_t elem, Regs& r) const
    {
        const uint4 w = *reinterpret_cast<const uint4*>(static_cast<const uint8_t*>(w8) + elem);
        r.w[0] = w.x; r.w[1] = w.y; r.w[2] = w.z; r.w[3] = w.w;
        const uint16_t* p = static_cast<const uint16_t*>(u16) + elem;
        asm volatile("ld.global.nc.L1::no_allocate.L2::evict_first.v8.u32 {%0,%1,%2,%3,%4,%5,%6,%7}, [%8];"
                     : "=r"(r.u[0]), "=r"(r.u[1]), "=r"(r.u[2]), "=r"(r.u[3]),
                       "=r"(r.u[4]), "=r"(r.u[5]), "=r"(r.u[6]), "=r"(r.u[7]) : "l"(p));
    }
    __device__ __forceinline__ void finish(size_t, const Regs& r, int o, float (&y)[8]) const
    {
        float lo[4], hi[4];
        decode4<WF>(r.w[2 * o], lo);
        decode4<WF>(r.w[2 * o + 1], hi);
#pragma unroll
        for (int c = 0; c < 8; ++c) {
            const uint32_t ucode = (r.u[4 * o + (c >> 1)] >> ((c & 1) * 16)) & 0xFFFFu;
            y[c] = sum16v<false>(c < 4 ? lo[c] : hi[c - 4], ucode);
        }
    }
    __device__ __forceinline__ uint32_t exact_bits(const Regs& r, int o, int c, float) const
    {
        const uint32_t wcode = (r.w[2 * o + (c >> 2)] >> ((c & 3) * 8)) & 0xFFu;
        const uint32_t ucode = (r.u[4 * o + (c >> 1)] >> ((c & 1) * 16)) & 0xFFFFu;
        return arith_bits(sum16(wcode, ucode));
    }
    __device__ __forceinline__ uint32_t scalar(size_t i) const
    {
        return arith_bits(sum16(static_cast<const uint8_t*>(w8)[i], static_cast<const uint16_t*>(u16)[i]));
    }
};

// Algorithm 1 from the gradient on: w16 = value(w8); the AdamW update in binary32 with one rounding per operation,
// rounded to the 16-bit format (u16); s = RTNE_16(fl32(w16 + u16)); the caller of finish() rounds s to 8 bits.
//   m' = fma(b1, m, a1 g);  v' = fma(b2, v, (a2 g) g);  d = sqrt(v') c2 + eps;  u32 = fma(-c1, m'/d, -(lr wd) w16)
template <int WF, int UF>
struct QatAdamOp {
    static_assert(Format<WF>::K == 8 && (UF == BF16 || UF == FP16), "8-bit weights, 16-bit gradients and updates");
    static constexpr int VALUE_BITS = UF == BF16 ? 8 : 11;              // the sum is a value of the 16-bit format
    static constexpr int BATCH = QATADAM_BATCH, MIN_CTAS = QATADAM_MIN_CTAS, OCTETS = 1;
    const void* w8; const void* g16; float* m; float* v;
    float beta1, beta2, eps, neg_c1, c2, a1, a2, neg_lrwd;
    struct Regs { uint2 w; uint4 g; F8 m, v; };
    __device__ __forceinline__ static float widen16(uint32_t code)
    {
        return UF == BF16 ? __uint_as_float(code << 16) : __half2float(__ushort_as_half((unsigned short)code));
    }
    // EXACT: round to the 16-bit format, ties to even, a finite value beyond its largest one saturating.
    // !EXACT: the plain hardware conversion, which gives an infinity there; that infinity survives to the result
    // (w + Inf is Inf or NaN), the row is flagged and redone through exact_bits(), as for QatOp.
    template <bool EXACT>
    __device__ __forceinline__ static float round16(float s)
    {
        if constexpr (EXACT) {
            const float m16 = __uint_as_float(Format<UF>::MAXBITS);
            const float a = fabsf(s);
            if (a > m16 && a < __uint_as_float(0x7F800000u)) s = copysignf(m16, s);
        }
        if constexpr (UF == BF16) return __bfloat162float(__float2bfloat16_rn(s));
        else return __half2float(__float2half_rn(s));
    }
    template <bool EXACT>
    __device__ __forceinline__ float step(float wv, uint32_t gcode, float& mv, float& vv) const
    {
        const float gv = widen16(gcode);
        mv = __fmaf_rn(beta1, mv, __fmul_rn(a1, gv));
        vv = __fmaf_rn(beta2, vv, __fmul_rn(__fmul_rn(a2, gv), gv));
        const float d = __fadd_rn(__fmul_rn(__fsqrt_rn(vv), c2), eps);
        const float u32 = __fmaf_rn(neg_c1, __fdiv_rn(mv, d), __fmul_rn(neg_lrwd, wv));
        const float u16 = round16<EXACT>(u32);
        return round16<EXACT>(__fadd_rn(wv, u16));
    }
    __device__ __forceinline__ void fetch(size_t elem, Regs& r) const
    {
        r.w = *reinterpret_cast<const uint2*>(static_cast<const uint8_t*>(w8) + elem);
        r.g = *reinterpret_cast<const uint4*>(static_cast<const uint16_t*>(g16) + elem);
        r.m = load_f8(m + elem); r.v = load_f8(v + elem);
    }
    __device__ __forceinline__ void finish(size_t elem, const Regs& r, float (&y)[8]) const
    {
        float lo[4], hi[4], mv[8], vv[8];
        decode4<WF>(r.w.x, lo);
        decode4<WF>(r.w.y, hi);
        unpack(r.m, mv); unpack(r.v, vv);
        const uint32_t gw[4] = {r.g.x, r.g.y, r.g.z, r.g.w};
#pragma unroll
        for (int c = 0; c < 8; ++c) {
            const uint32_t gcode = (gw[c >> 1] >> ((c & 1) * 16)) & 0xFFFFu;
            y[c] = step<false>(c < 4 ? lo[c] : hi[c - 4], gcode, mv[c], vv[c]);
        }
        store_f8(m + elem, mv); store_f8(v + elem, vv);
    }
    // the element again, from the values fetched before the update, with the saturating conversions
    __device__ __forceinline__ uint32_t exact_bits(const Regs& r, int c, float) const
    {
        float mo[8], vo[8];
        unpack(r.m, mo); unpack(r.v, vo);
        const uint32_t wcode = ((c < 4 ? r.w.x : r.w.y) >> ((c & 3) * 8)) & 0xFFu;
        const uint32_t gw[4] = {r.g.x, r.g.y, r.g.z, r.g.w};
        const uint32_t gcode = (gw[c >> 1] >> ((c & 1) * 16)) & 0xFFFFu;
        float mv = mo[c], vv = vo[c];
        return arith_bits(step<true>(decode_element<WF>(wcode), gcode, mv, vv));
    }
    __device__ __forceinline__ uint32_t scalar(size_t i) const
    {
        float mv = m[i], vv = v[i];
        const float y = step<true>(decode_element<WF>(static_cast<const uint8_t*>(w8)[i]), static_cast<const uint16_t*>(g16)[i], mv, vv);
        m[i] = mv; v[i] = vv;
        return arith_bits(y);
    }
};

// ---------------------------------------------------------------------------- packing a row of codes
// Fast rows: t[] as left by round_row_fast: the code sits in the top K bits of each word (bfloat16 with its sign,
// the other formats with bit 31 clear and the sign still to be taken from y), so packing is byte selection.
template <int FMT>
__device__ __forceinline__ void pack_row_fast(const uint32_t (&t)[8], const float (&y)[8], uint32_t* out)
{
    if constexpr (FMT == BF16) {
#pragma unroll
        for (int j = 0; j < 4; ++j) out[j] = __byte_perm(t[2 * j], t[2 * j + 1], 0x7632);
    } else if constexpr (Format<FMT>::K == 16) {
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            const uint32_t codes = __byte_perm(t[2 * j], t[2 * j + 1], 0x7632);
            const uint32_t signs = __byte_perm(__float_as_uint(y[2 * j]), __float_as_uint(y[2 * j + 1]), 0x7632);
            out[j] = codes | (signs & 0x80008000u);
        }
    } else {
#pragma unroll
        for (int j = 0; j < 2; ++j) {
            const uint32_t c01 = __byte_perm(t[4 * j], t[4 * j + 1], 0x7373);
            const uint32_t c23 = __byte_perm(t[4 * j + 2], t[4 * j + 3], 0x7373);
            const uint32_t s01 = __byte_perm(__float_as_uint(y[4 * j]), __float_as_uint(y[4 * j + 1]), 0x7373);
            const uint32_t s23 = __byte_perm(__float_as_uint(y[4 * j + 2]), __float_as_uint(y[4 * j + 3]), 0x7373);
            const uint32_t codes = __byte_perm(c01, c23, 0x5410);
            uint32_t signs = __byte_perm(s01, s23, 0x5410) & 0x80808080u;
            // one zero only: a zero magnitude takes no sign (bytes are at most 0x7F, so the add carries into
            // bit 7 of exactly the non-zero ones)
            if constexpr (Format<FMT>::SINGLE_ZERO) signs &= codes + 0x7F7F7F7Fu;
            out[j] = codes | signs;
        }
    }
}

// ---------------------------------------------------------------------------- the bandwidth kernel
// Elements [0, n_tiles * ELEMS) relative to the pointers held by op/dst.  Normally launched with one
// tile per warp; the loop only matters when the grid had to be capped.
// call0: global index of the Philox call that serves element 0 (Philox source), or
// words: the packed word stream whose word 0 serves element 0 (supplied bits).
// IEEE: finite values beyond M are rounded as IEEE nearest-even does (Section II read literally) instead of
// saturating: M below the midpoint to the next power of two, the infinity (the NaN code of a format without one)
// from there on, the midpoint itself to whichever of the two has an even code.  The row rounder has already
// clamped such an element to the code of M, so one comparison and one select per element put the other code in
// place; bfloat16 rows holding such a value are redone element by element anyway.
template <int FMT> struct IeeeOverflow {
    using F = Format<FMT>;
    static constexpr uint32_t TIE_BITS = F::MAXBITS + (1u << (24 - F::P - 1));      // M + ulp(M) / 2, exact in binary32
    static constexpr bool TIE_OVERFLOWS = (F::MAXCODE & 1u) != 0;                   // the code of M is odd: the tie leaves it
    static constexpr uint32_t CODE = F::HAS_INF ? F::INFCODE : F::NANCODE;
    __device__ __forceinline__ static bool beyond(float y)
    {
        const float tie = __uint_as_float(TIE_BITS);
        return TIE_OVERFLOWS ? fabsf(y) >= tie : fabsf(y) > tie;
    }
};

template <class Op, int FMT, int VAR, int K, bool BITS, bool IEEE = false>
__global__ void __launch_bounds__(CTA_THREADS, Op::MIN_CTAS)
tile_kernel(const Op op, void* __restrict__ dst, const uint64_t n_tiles, const uint64_t call0,
            const uint32_t k0, const uint32_t k1, const uint32_t* __restrict__ words, const uint32_t tail_count)
{
    using T = Tile<K, Op::OCTETS>;
    constexpr bool DRAWS = VAR < RTNE;                     // the deterministic modes use no random bits
    // The elements after the last whole tile (fewer than one tile) are done by CTA 0, one element per
    // thread and step, each with its own generator call: it starts first and overlaps the tiles.
    const uint32_t first_tile_cta = tail_count ? 1u : 0u;
    if (tail_count && blockIdx.x == 0) {
        const size_t tail_begin = (size_t)n_tiles * T::ELEMS;
        for (uint32_t i = threadIdx.x; i < tail_count; i += CTA_THREADS) {
            const size_t p = tail_begin + i;
            const uint32_t j = (uint32_t)(p % T::E);
            uint32_t word = 0u;
            if constexpr (!DRAWS) {
            } else if constexpr (BITS) {
                word = words[p / T::DPW];
            } else {
                const uint4 o = philox_block(call0 + p / T::E, k0, k1);
                const uint32_t ws = j / T::DPW;
                word = ws == 0 ? o.x : ws == 1 ? o.y : ws == 2 ? o.z : o.w;
            }
            const uint32_t n = (word >> ((j % T::DPW) * K)) & T::MASK;
            store_code1<FMT>(dst, p, round_core<FMT, false>(op.scalar(p), n, VAR, K, nullptr, IEEE));
        }
        return;
    }
    constexpr bool OWN_CALL = (T::DPW == 2) && !BITS;      // a call serves exactly one lane-row
    // supplied words keep their packed layout (+4: the joined-word read of the last group); generated ones are
    // written in the normalised layout of Draws8
    __shared__ __align__(16) uint32_t wordbuf[WARPS_PER_CTA][OWN_CALL ? 4 : (BITS ? T::WORDS + 4 : T::BUFFER_WORDS)];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    uint32_t* wb = wordbuf[warp];

    for (uint64_t tile = (uint64_t)(blockIdx.x - first_tile_cta) * WARPS_PER_CTA + warp; tile < n_tiles;
         tile += (uint64_t)(gridDim.x - first_tile_cta) * WARPS_PER_CTA) {
        const size_t e0 = (size_t)tile * T::ELEMS;
        const uint64_t tile_call0 = call0 + tile * T::CALLS;

        // A lane takes OCT octets (8 consecutive elements each) per row, so a row is 256 * OCT elements; rows are
        // taken in equal batches of at most Op::BATCH (5 rows: 3 + 2, not 4 + 1).
        constexpr int OCT = Op::OCTETS;
        constexpr int ROW = ROW_ELEMS * OCT, ROWS = T::ELEMS / ROW;
        static_assert(T::ELEMS % ROW == 0, "whole rows per tile");
        constexpr int N_BATCHES = (ROWS + Op::BATCH - 1) / Op::BATCH;
        constexpr int BATCH = (ROWS + N_BATCHES - 1) / N_BATCHES;
        constexpr int WPO = WordsPerOctet<FMT>::value;
        // The loads of the first batch of rows are issued before the generator calls, which then run in their shadow.
        typename Op::Regs regs[BATCH];
#pragma unroll
        for (int j = 0; j < BATCH; ++j) op.fetch(e0 + j * ROW + lane * 8 * OCT, regs[j]);

        if constexpr (!DRAWS) {
        } else if constexpr (BITS) {
            const uint32_t* src_words = words + tile * T::WORDS;
#pragma unroll
            for (int j = 0; j < T::WORDS / 32; ++j) wb[j * 32 + lane] = __ldg(src_words + j * 32 + lane);
            static_assert(T::WORDS % 32 == 0, "whole warp-rows of words");
            __syncwarp();
        } else if constexpr (!OWN_CALL) {
#pragma unroll
            for (int j = 0; j < (T::CALLS + 31) / 32; ++j) {
                const int c = j * 32 + lane;
                if (T::CALLS % 32 == 0 || c < T::CALLS)
                    Draws8<K>::store_call(wb + Draws8<K>::WORDS_PER_CALL * c, philox_block(tile_call0 + c, k0, k1));
            }
            __syncwarp();
        }

#pragma unroll
        for (int rb = 0; rb < ROWS; rb += BATCH) {
            if (rb > 0) {
#pragma unroll
                for (int j = 0; j < BATCH; ++j)
                    if (rb + j < ROWS) op.fetch(e0 + (rb + j) * ROW + lane * 8 * OCT, regs[j]);
            }
#pragma unroll
            for (int j = 0; j < BATCH; ++j) {
                if (rb + j < ROWS) {
                    const int p0 = (rb + j) * ROW + lane * 8 * OCT;
                    uint32_t packed[OCT * WPO];
#pragma unroll
                    for (int o = 0; o < OCT; ++o) {
                        const int po = p0 + 8 * o;
                        float y[8];
                        if constexpr (OCT == 1) op.finish(e0 + po, regs[j], y);
                        else op.finish(e0 + po, regs[j], o, y);
                        Draws8<K> d;
                        if constexpr (!DRAWS) {
                        } else if constexpr (OWN_CALL) {
                            d.from_call(philox_block(tile_call0 + po / 8, k0, k1));
                        } else if constexpr (BITS) {
                            d.from_stream(wb, po);
                        } else {
                            d.from_normalised(wb, po);
                        }
                        uint32_t t[8];
                        const bool redo = round_row_fast<FMT, VAR, K, ValueBits<Op>::value>(y, d, t);
                        if constexpr (IEEE && FMT != BF16) {
#pragma unroll
                            for (int i = 0; i < 8; ++i)
                                t[i] = IeeeOverflow<FMT>::beyond(y[i]) ? IeeeOverflow<FMT>::CODE << (32 - Format<FMT>::K) : t[i];
                        }
                        if (!redo) {
                            pack_row_fast<FMT>(t, y, packed + o * WPO);
                        } else {
                            // a special value somewhere in this octet (rare): element-wise, exact
                            uint32_t c[8];
#pragma unroll
                            for (int i = 0; i < 8; ++i) {
                                uint32_t bits;
                                if constexpr (OCT == 1) bits = op.exact_bits(regs[j], i, y[i]);
                                else bits = op.exact_bits(regs[j], o, i, y[i]);
                                c[i] = round_core<FMT, false>(bits, d.template at<0>(i), VAR, K, nullptr, IEEE);
                            }
                            pack_codes8<FMT>(c, packed + o * WPO);
                        }
                    }
                    store_words<OCT * WPO>(static_cast<char*>(dst) + (e0 + p0) * (Format<FMT>::K / 8), packed);
                }
            }
        }
        if constexpr (DRAWS && !OWN_CALL) __syncwarp();      // the buffer is rewritten by the next tile
    }
}

// ---------------------------------------------------------------------------- the bandwidth kernel, any alignment
// fbsr_round for pointers that are only element-aligned (a slice of a tensor, a packed parameter buffer).  The
// tile grid is fixed by `offset` (a tile is a whole number of generator calls), so no peeling can also align the
// two pointers; instead a warp stages its tile through shared memory:
//   in   element j of the tile is copied to shared word j by 4-byte asynchronous copies, lane-consecutive, so a
//        warp instruction still reads 128 contiguous bytes of global memory whatever the pointer's alignment, and
//        the whole tile is in flight at once; a lane then takes its 8 consecutive values with two 128-bit reads;
//   out  the packed codes go to shared memory (over values already consumed), and are written out as
//        4-byte words aligned in GLOBAL memory: word m is funnelled out of two neighbouring shared words by a
//        byte permute whose selector is the pointer's misalignment; the few bytes before the first and after the
//        last aligned word of the tile are stored one code at a time (the neighbouring tile writes the rest of
//        that word).
// Rounding, draws and the treatment of special values are those of tile_kernel.
constexpr int STAGED_WARPS = 4;                          // keeps the static shared memory of every k under 48 KB
constexpr int STAGED_THREADS = STAGED_WARPS * 32;

__device__ __forceinline__ void copy_async_4(void* smem_dst, const void* gmem_src)
{
    asm volatile("cp.async.ca.shared.global [%0], [%1], 4;" ::"r"((uint32_t)__cvta_generic_to_shared(smem_dst)), "l"(gmem_src) : "memory");
}

template <int FMT, int VAR, int K, bool BITS>
__global__ void __launch_bounds__(STAGED_THREADS, 4)
staged_tile_kernel(const RoundOp op, void* __restrict__ dst, const uint64_t n_tiles, const uint64_t call0,
                   const uint32_t k0, const uint32_t k1, const uint32_t* __restrict__ words, const uint32_t tail_count)
{
    using T = Tile<K, 1>;
    constexpr bool DRAWS = VAR < RTNE;
    constexpr int CB = Format<FMT>::K / 8;
    const uint32_t first_tile_cta = tail_count ? 1u : 0u;
    if (tail_count && blockIdx.x == 0) {
        // the elements after the last whole tile, one per thread and step, as in tile_kernel
        const size_t tail_begin = (size_t)n_tiles * T::ELEMS;
        for (uint32_t i = threadIdx.x; i < tail_count; i += STAGED_THREADS) {
            const size_t p = tail_begin + i;
            const uint32_t j = (uint32_t)(p % T::E);
            uint32_t word = 0u;
            if constexpr (!DRAWS) {
            } else if constexpr (BITS) {
                word = words[p / T::DPW];
            } else {
                const uint4 o = philox_block(call0 + p / T::E, k0, k1);
                const uint32_t ws = j / T::DPW;
                word = ws == 0 ? o.x : ws == 1 ? o.y : ws == 2 ? o.z : o.w;
            }
            const uint32_t n = (word >> ((j % T::DPW) * K)) & T::MASK;
            store_code1<FMT>(dst, p, round_core<FMT, false>(op.scalar(p), n, VAR, K, nullptr));
        }
        return;
    }
    constexpr bool OWN_CALL = (T::DPW == 2) && !BITS;
    constexpr int OUT_WORDS = T::ELEMS * CB / 4;
    // the packed codes of row j (at most half as many bytes as its values) overwrite the front of the same buffer:
    // bytes [0, 256 (j + 1) CB) only ever held rows 0..j, which the warp has already taken into registers
    static_assert(OUT_WORDS + 1 <= T::ELEMS, "the codes and the funnel's look-ahead word fit in the input buffer");
    __shared__ __align__(16) float in_buf[STAGED_WARPS][T::ELEMS];
    __shared__ __align__(16) uint32_t wordbuf[STAGED_WARPS][OWN_CALL ? 4 : (BITS ? T::WORDS + 4 : T::BUFFER_WORDS)];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    float* in = in_buf[warp];
    uint32_t* ob = reinterpret_cast<uint32_t*>(in);
    uint32_t* wb = wordbuf[warp];
    constexpr int ROWS = T::ELEMS / ROW_ELEMS;
    constexpr int WPO = WordsPerOctet<FMT>::value;

    for (uint64_t tile = (uint64_t)(blockIdx.x - first_tile_cta) * STAGED_WARPS + warp; tile < n_tiles;
         tile += (uint64_t)(gridDim.x - first_tile_cta) * STAGED_WARPS) {
        const size_t e0 = (size_t)tile * T::ELEMS;
        const uint64_t tile_call0 = call0 + tile * T::CALLS;
        const float* src = op.src + e0;
#pragma unroll
        for (int j = 0; j < T::ELEMS / 32; ++j) copy_async_4(in + j * 32 + lane, src + j * 32 + lane);
        asm volatile("cp.async.commit_group;" ::: "memory");

        // the generator calls run while the copies are in flight
        if constexpr (!DRAWS) {
        } else if constexpr (BITS) {
            const uint32_t* src_words = words + tile * T::WORDS;
#pragma unroll
            for (int j = 0; j < T::WORDS / 32; ++j) wb[j * 32 + lane] = __ldg(src_words + j * 32 + lane);
        } else if constexpr (!OWN_CALL) {
#pragma unroll
            for (int j = 0; j < (T::CALLS + 31) / 32; ++j) {
                const int c = j * 32 + lane;
                if (T::CALLS % 32 == 0 || c < T::CALLS)
                    Draws8<K>::store_call(wb + Draws8<K>::WORDS_PER_CALL * c, philox_block(tile_call0 + c, k0, k1));
            }
        }
        asm volatile("cp.async.wait_group 0;" ::: "memory");
        __syncwarp();

#pragma unroll
        for (int j = 0; j < ROWS; ++j) {
            const int p0 = j * ROW_ELEMS + lane * 8;
            RoundOp::Regs regs;
            regs.x.a = *reinterpret_cast<const float4*>(in + p0);
            regs.x.b = *reinterpret_cast<const float4*>(in + p0 + 4);
            __syncwarp();                                    // every lane holds its values before codes are written over them
            float y[8];
            op.finish(e0 + p0, regs, y);
            Draws8<K> d;
            if constexpr (!DRAWS) {
            } else if constexpr (OWN_CALL) {
                d.from_call(philox_block(tile_call0 + p0 / 8, k0, k1));
            } else if constexpr (BITS) {
                d.from_stream(wb, p0);
            } else {
                d.from_normalised(wb, p0);
            }
            uint32_t t[8], packed[WPO];
            const bool redo = round_row_fast<FMT, VAR, K>(y, d, t);
            if (!redo) {
                pack_row_fast<FMT>(t, y, packed);
            } else {
                uint32_t c[8];
#pragma unroll
                for (int i = 0; i < 8; ++i)
                    c[i] = round_core<FMT, false>(op.exact_bits(regs, i, y[i]), d.template at<0>(i), VAR, K, nullptr);
                pack_codes8<FMT>(c, packed);
            }
            if constexpr (WPO == 4) *reinterpret_cast<uint4*>(ob + p0 / 2) = make_uint4(packed[0], packed[1], packed[2], packed[3]);
            else *reinterpret_cast<uint2*>(ob + p0 / 4) = make_uint2(packed[0], packed[1]);
        }
        __syncwarp();

        // write-out: 4-byte words aligned in global memory
        char* g = static_cast<char*>(dst) + e0 * CB;
        const uint32_t head_b = (4u - (uint32_t)(reinterpret_cast<uintptr_t>(g) & 3u)) & 3u;      // bytes before the first aligned word
        const uint32_t n_words = head_b ? OUT_WORDS - 1 : OUT_WORDS;
        const uint32_t selector = 0x3210u + 0x1111u * head_b;
        uint32_t* gw = reinterpret_cast<uint32_t*>(g + head_b);
#pragma unroll 4
        for (uint32_t m = lane; m < n_words; m += 32) FBSR_STORE(gw + m, __byte_perm(ob[m], ob[m + 1], selector));
        if (head_b) {
            // the codes before the first aligned word and after the last one
            const uint32_t head_codes = head_b / CB, tail_codes = (4u - head_b) / CB;
            const unsigned char* bytes = reinterpret_cast<const unsigned char*>(ob);
            if ((uint32_t)lane < head_codes) {
                if constexpr (CB == 2) reinterpret_cast<uint16_t*>(g)[lane] = reinterpret_cast<const uint16_t*>(bytes)[lane];
                else reinterpret_cast<uint8_t*>(g)[lane] = bytes[lane];
            } else if ((uint32_t)lane < head_codes + tail_codes) {
                const uint32_t i = T::ELEMS - tail_codes + ((uint32_t)lane - head_codes);
                if constexpr (CB == 2) reinterpret_cast<uint16_t*>(g)[i] = reinterpret_cast<const uint16_t*>(bytes)[i];
                else reinterpret_cast<uint8_t*>(g)[i] = bytes[i];
            }
        }
        __syncwarp();                                        // the buffers are rewritten by the next tile
    }
}

// ---------------------------------------------------------------------------- statistics
struct StatsAcc {
    unsigned long long n_finite, n_up, n_nan, n_inf, n_sat;
    double sum_e, sum_e2, sum_signed_e, sum_abs_e;
};

__device__ __forceinline__ void stats_zero(StatsAcc& a)
{
    a.n_finite = a.n_up = a.n_nan = a.n_inf = a.n_sat = 0ull;
    a.sum_e = a.sum_e2 = a.sum_signed_e = a.sum_abs_e = 0.0;
}

__device__ __forceinline__ void stats_add(StatsAcc& a, const StatsAcc& b)
{
    a.n_finite += b.n_finite; a.n_up += b.n_up; a.n_nan += b.n_nan; a.n_inf += b.n_inf; a.n_sat += b.n_sat;
    a.sum_e += b.sum_e; a.sum_e2 += b.sum_e2; a.sum_signed_e += b.sum_signed_e; a.sum_abs_e += b.sum_abs_e;
}

__device__ __forceinline__ StatsAcc stats_shfl_down(const StatsAcc& a, int d)
{
    StatsAcc b;
    b.n_finite = __shfl_down_sync(0xFFFFFFFFu, a.n_finite, d);
    b.n_up = __shfl_down_sync(0xFFFFFFFFu, a.n_up, d);
    b.n_nan = __shfl_down_sync(0xFFFFFFFFu, a.n_nan, d);
    b.n_inf = __shfl_down_sync(0xFFFFFFFFu, a.n_inf, d);
    b.n_sat = __shfl_down_sync(0xFFFFFFFFu, a.n_sat, d);
    b.sum_e = __shfl_down_sync(0xFFFFFFFFu, a.sum_e, d);
    b.sum_e2 = __shfl_down_sync(0xFFFFFFFFu, a.sum_e2, d);
    b.sum_signed_e = __shfl_down_sync(0xFFFFFFFFu, a.sum_signed_e, d);
    b.sum_abs_e = __shfl_down_sync(0xFFFFFFFFu, a.sum_abs_e, d);
    return b;
}

// Fixed-order reduction over the CTA; the result is valid in thread 0.
__device__ __forceinline__ void stats_cta_reduce(StatsAcc& a)
{
    __shared__ StatsAcc per_warp[WARPS_PER_CTA];
#pragma unroll
    for (int d = 16; d > 0; d >>= 1) stats_add(a, stats_shfl_down(a, d));
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    if (lane == 0) per_warp[warp] = a;
    __syncthreads();
    if (threadIdx.x == 0) {
        for (int w = 1; w < WARPS_PER_CTA; ++w) stats_add(a, per_warp[w]);
    }
}

// ---------------------------------------------------------------------------- the slow, general kernel
// Elements [i_begin, i_end) of the call.  One thread per Philox call (or per group of four supplied words).
template <class Op, int FMT, bool BITS, bool STATS>
__global__ void __launch_bounds__(CTA_THREADS)
generic_kernel(const Op op, void* __restrict__ dst, const uint64_t i_begin, const uint64_t i_end,
               const uint64_t offset, const int variant, const int k, const uint32_t k0, const uint32_t k1,
               const uint32_t* __restrict__ words, const uint64_t n_words,
               const uint64_t group_size, double* __restrict__ gsum_e, double* __restrict__ gsum_e2,
               StatsAcc* __restrict__ partials, const int ieee_overflow)
{
    const uint32_t dpw = 32u / (uint32_t)k, E = 4u * dpw, mask = (1u << k) - 1u;
    const uint64_t g_first = offset + i_begin, g_last = offset + i_end;     // [g_first, g_last)
    const uint64_t call_first = g_first / E;
    const uint64_t n_calls = g_first < g_last ? (g_last - 1) / E - call_first + 1 : 0;
    StatsAcc acc;
    if constexpr (STATS) stats_zero(acc);

    for (uint64_t b = (uint64_t)blockIdx.x * CTA_THREADS + threadIdx.x; b < n_calls;
         b += (uint64_t)gridDim.x * CTA_THREADS) {
        const uint64_t call = call_first + b;
        const uint64_t g_lo = max(call * E, g_first), g_hi = min((call + 1) * E, g_last);
        uint32_t w[4];
        if constexpr (BITS) {
#pragma unroll
            for (int j = 0; j < 4; ++j) w[j] = call * 4 + j < n_words ? words[call * 4 + j] : 0u;
        } else {
            const uint4 o = philox_block(call, k0, k1);
            w[0] = o.x; w[1] = o.y; w[2] = o.z; w[3] = o.w;
        }
        uint64_t cur_group = ~0ull;
        double ge = 0.0, ge2 = 0.0;
        for (uint64_t g = g_lo; g < g_hi; ++g) {
            const uint64_t i = g - offset;
            const uint32_t j = (uint32_t)(g - call * E);
            const uint32_t ws = j / dpw, f = j - ws * dpw;
            const uint32_t word = ws == 0 ? w[0] : ws == 1 ? w[1] : ws == 2 ? w[2] : w[3];
            const uint32_t n = (word >> (f * k)) & mask;
            const uint32_t y = op.scalar(i);
            ElementInfo info;
            const uint32_t code = round_core<FMT, STATS>(y, n, variant, k, &info, ieee_overflow != 0);
            store_code1<FMT>(dst, i, code);
            if constexpr (STATS) {
                if (info.kind == 0) {
                    const double e = (double)info.up - info.delta;
                    const double e2 = e * e;
                    acc.n_finite += 1; acc.n_up += (unsigned)info.up;
                    acc.sum_e += e; acc.sum_e2 += e2;
                    acc.sum_signed_e += (y >> 31) ? -e : e;
                    acc.sum_abs_e += fabs(e);
                    if (group_size) {
                        const uint64_t grp = i / group_size;
                        if (grp != cur_group) {
                            if (cur_group != ~0ull) { atomicAdd(gsum_e + cur_group, ge); atomicAdd(gsum_e2 + cur_group, ge2); }
                            cur_group = grp; ge = 0.0; ge2 = 0.0;
                        }
                        ge += e; ge2 += e2;
                    }
                } else if (info.kind == 1) acc.n_nan += 1;
                else if (info.kind == 2) acc.n_inf += 1;
                else acc.n_sat += 1;
            }
        }
        if constexpr (STATS) {
            if (cur_group != ~0ull) { atomicAdd(gsum_e + cur_group, ge); atomicAdd(gsum_e2 + cur_group, ge2); }
        }
    }
    if constexpr (STATS) {
        stats_cta_reduce(acc);
        if (threadIdx.x == 0) partials[blockIdx.x] = acc;
    }
}

// The general kernel without statistics, with coalesced accesses.  A warp takes 32 consecutive generator calls
// (32 E elements): lane l computes call l of the chunk into the warp's shared buffer, then the warp walks the chunk's
// elements 32 at a time, lane l taking element 32 j + l, so that a warp instruction reads and writes consecutive
// elements whatever the pointers' alignment (one thread per call, as in generic_kernel, puts E elements between
// neighbouring lanes).  Run-time k and variant; elements outside [i_begin, i_end) are skipped.
// dpw_magic = floor(2^32 / dpw) + 1: the high half of p * dpw_magic is p / dpw for every p below 4096.
template <class Op, int FMT, bool BITS>
__global__ void __launch_bounds__(CTA_THREADS)
general_coalesced_kernel(const Op op, void* __restrict__ dst, const uint64_t i_begin, const uint64_t i_end,
                         const uint64_t offset, const int variant, const int k, const uint32_t k0, const uint32_t k1,
                         const uint32_t* __restrict__ words, const uint64_t n_words, const uint32_t dpw_magic,
                         const int ieee_overflow)
{
    const uint32_t dpw = 32u / (uint32_t)k, E = 4u * dpw, mask = (1u << k) - 1u;
    const bool draws = variant < RTNE;
    const uint64_t g_first = offset + i_begin, g_last = offset + i_end;     // [g_first, g_last)
    const uint64_t call_first = g_first / E;
    const uint64_t n_calls = g_first < g_last ? (g_last - 1) / E - call_first + 1 : 0;
    const uint64_t n_chunks = (n_calls + 31) / 32;
    __shared__ __align__(16) uint32_t callbuf[WARPS_PER_CTA][128];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    uint32_t* wb = callbuf[warp];
    for (uint64_t chunk = (uint64_t)blockIdx.x * WARPS_PER_CTA + warp; chunk < n_chunks;
         chunk += (uint64_t)gridDim.x * WARPS_PER_CTA) {
        const uint64_t call = call_first + chunk * 32 + lane;
        uint4 o = make_uint4(0u, 0u, 0u, 0u);
        if (draws && call < call_first + n_calls) {
            if constexpr (BITS) {
                o.x = call * 4 + 0 < n_words ? words[call * 4 + 0] : 0u;
                o.y = call * 4 + 1 < n_words ? words[call * 4 + 1] : 0u;
                o.z = call * 4 + 2 < n_words ? words[call * 4 + 2] : 0u;
                o.w = call * 4 + 3 < n_words ? words[call * 4 + 3] : 0u;
            } else {
                o = philox_block(call, k0, k1);
            }
        }
        *reinterpret_cast<uint4*>(wb + 4 * lane) = o;
        __syncwarp();
        const uint64_t g0 = (call_first + chunk * 32) * E;                  // global index of the chunk's first element
        for (uint32_t p = lane; p < 32u * E; p += 32u) {
            const uint64_t g = g0 + p;
            if (g >= g_first && g < g_last) {
                const uint32_t w = __umulhi(p, dpw_magic), f = p - w * dpw;
                const uint32_t n = (wb[w] >> (f * (uint32_t)k)) & mask;
                const uint64_t i = g - offset;
                store_code1<FMT>(dst, i, round_core<FMT, false>(op.scalar(i), n, variant, k, nullptr, ieee_overflow != 0));
            }
        }
        __syncwarp();                                        // the buffer is rewritten by the next chunk
    }
}

// Statistics of one element from its value and the magnitude of the code it was given (the draw is not needed):
// floor(sigma~) and delta~ come from the decomposition of Eq. (2)-(3), up = code - code of the floor, e = up - delta~.
// Returns true and sets e and up for an SR-rounded element; the others are only counted.
template <int FMT>
__device__ __forceinline__ bool stats_element(const uint32_t ybits, const uint32_t code_mag, StatsAcc& acc, double& e,
                                              uint32_t& up)
{
    using F = Format<FMT>;
    constexpr int P = F::P;
    const uint32_t mag = ybits & 0x7FFFFFFFu;
    if (mag > F::MAXBITS) {
        if (mag > 0x7F800000u) acc.n_nan += 1;
        else if (mag == 0x7F800000u) acc.n_inf += 1;
        else acc.n_sat += 1;
        return false;
    }
    uint32_t r;
    int sh;
    if constexpr (FMT == BF16) {
        sh = 16;                                             // same exponent range as binary32: the low half is delta~
        r = mag & 0xFFFFu;
        up = code_mag - (mag >> 16);
    } else {
        const uint32_t e32 = mag >> 23;
        const uint32_t m = (mag & 0x7FFFFFu) | (e32 ? 0x800000u : 0u);
        const int eb = max((int)e32, 1);
        const int te = max(eb, F::EMINB);
        sh = (24 - P) + (te - eb);
        const uint32_t fl = sh < 32 ? m >> sh : 0u;
        r = sh < 32 ? (m & ((1u << sh) - 1u)) : m;
        up = code_mag - (((uint32_t)(te - F::EMINB) << (P - 1)) + fl);
    }
    const double delta = (double)r * __hiloint2double((1023 - sh) << 20, 0);     // r 2^-sh, exact
    e = (up ? 1.0 : 0.0) - delta;
    return true;
}

// ---------------------------------------------------------------------------- statistics on whole tiles
// Integer form of the error sums.  With delta~ = d / 2^U (d an integer) and up in {0, 1}, e = up - delta~ gives
//   sum e    = (n_up 2^U - sum d) / 2^U
//   sum |e|  = (sum d - 2 sum_{up} d + n_up 2^U) / 2^U
//   sum e^2  = (sum d^2 + n_up 2^(2U) - 2^(U+1) sum_{up} d) / 2^(2U)
//   sum s e  = sum e - 2 (n_{up, y<0} 2^U - sum_{y<0} d) / 2^U          (s = sign of y)
// so a thread only adds d, d^2 and a few masked copies of d per element, all exact in 64-bit integers, and turns
// them into binary64 once.  U = 16 for bfloat16 (the excess bits are always the low half of the pattern) and 23
// for the other formats, which covers every element with at most 23 excess bits: the target's normal range,
// its subnormal range and the binade below.  An element with more excess bits ("deep": a magnitude below a
// quarter of the smallest subnormal, so floor(sigma~) = 0 and delta~ = sigma~ < 1, an exact binary32 product)
// enters the integer sums with d = 0 and adds its delta~ to the same four sums kept in binary64 beside them.
// NaN and Inf send the lane's octet through stats_element() instead.
template <int FMT> struct StatsFixed {
    using F = Format<FMT>;
    static constexpr int U = FMT == BF16 ? 16 : 23;
    static constexpr int SH0 = 24 - F::P;
    // smallest pattern with at most 23 excess bits: biased exponent EMINB - P + 1
    static constexpr uint32_t DEEP_BITS = FMT == BF16 ? 0u : (uint32_t)(F::EMINB - F::P + 1) << 23;
};

struct StatsInt {                        // one lane's integer sums, units of 2^-U
    unsigned long long d, up_d, neg_d, d2;          // sum d, over rounded-up elements, over negative elements, sum d^2
    uint32_t d_tile, up_d_tile, neg_d_tile;         // the first three over the current tile (at most 48 elements: no overflow)
    uint32_t counts;                    // rounded up: low half; rounded up and negative: high half (unpacked every tile)
    uint32_t n_sat;
};

struct StatsDeep { double d, up_d, neg_d, d2; };      // the same sums of delta~ over the deep elements

__device__ __forceinline__ uint32_t shl_clamped(uint32_t x, int s)
{
    uint32_t r;
    asm("shl.b32 %0, %1, %2;" : "=r"(r) : "r"(x), "r"((uint32_t)s));   // amounts above 31 give 0
    return r;
}

// One SR-rounded (or saturated) finite element: y the value, t the word left by round_row_fast.  The masked
// sums are written as 32-bit multiply-adds (`one` is 1, unknown to the compiler) so that they run on the
// multiplier pipe: the integer pipe is what bounds this kernel.  (64-bit widening multiply-adds measured slower.)
template <int FMT>
__device__ __forceinline__ void stats_fixed_element(const float y, const uint32_t t, const uint32_t one, StatsInt& s,
                                                    StatsDeep& deep)
{
    using F = Format<FMT>;
    using X = StatsFixed<FMT>;
    const uint32_t yb = __float_as_uint(y);
    const uint32_t neg = yb >> 31;
    uint32_t d, up;
    if constexpr (FMT == BF16) {
        d = yb & 0xFFFFu;
        up = ((t ^ yb) >> 16) & 1u;                                      // the code's lowest bit flips iff a carry came in
    } else {
        const uint32_t ab = yb & 0x7FFFFFFFu;
        const bool sat = ab > F::MAXBITS;                               // counted, and never rounded up: d = 0
        s.n_sat += sat ? 1u : 0u;
        // left-align the excess bits: 32 - sh = min(32 - SH0, eb + 32 - SH0 - EMINB); a shift below 9 (more than
        // 23 excess bits) leaves exponent bits in the way, so those elements take d = 0 here
        const int s8 = min(32 - X::SH0, (int)(ab >> 23) + (32 - X::SH0 - F::EMINB));
        const bool is_deep = (ab - 1u) < (X::DEEP_BITS - 1u);           // zero is not deep: all its terms are 0
        d = (is_deep || sat) ? 0u : shl_clamped(ab, s8) >> 9;
        // floor code from the rescaled pattern, as in the row rounder
        const float rescale = __uint_as_float((uint32_t)(128 - F::EMINB) << 23);
        const uint32_t u = min(__float_as_uint(__fmul_rz(fabsf(y), rescale)), F::MAXCODE << X::SH0);
        up = ((t ^ (u << (32 - F::K - X::SH0))) >> (32 - F::K)) & 1u;    // lowest bit of the code against the floor's
        if (is_deep) {
            // sigma~ = |y| 2^(P - 1 - emin), exact
            const double dl = (double)__fmul_rn(fabsf(y), __uint_as_float((uint32_t)(F::P - 1 + 254 - F::EMINB) << 23));
            deep.d += dl;
            deep.d2 = fma(dl, dl, deep.d2);
            if (up) deep.up_d += dl;
            if (neg) deep.neg_d += dl;
        }
    }
    s.d_tile += d;
    s.d2 += (unsigned long long)d * d;
    s.up_d_tile += up * d;
    s.neg_d_tile += neg * d;
    if constexpr (F::K == 16) s.counts += up + ((up & neg) << 16);
    else s.counts += up * (neg * 65536u + one);
}

// One lane-octet element by element in binary64 (the octets that hold NaN or Inf or, with group sums, a group
// boundary): rounds and stores its 8 codes and adds their statistics to
// *sums.  Kept out of line, with the binary64 sums in local memory, so that neither takes registers from the tile
// loop; it reads its inputs again.
template <int FMT, bool GROUPS, int CALLER_VAR, int CALLER_K>         // one copy per calling kernel
__device__ __noinline__ void stats_octet_general(StatsAcc* __restrict__ sums, const float* __restrict__ src8, const float scale,
                                                 const uint4 n_lo, const uint4 n_hi, const int variant, const int k,
                                                 void* __restrict__ dst8, const uint64_t i0, const uint64_t group_size,
                                                 double* __restrict__ gsum_e, double* __restrict__ gsum_e2)
{
    const uint32_t n[8] = {n_lo.x, n_lo.y, n_lo.z, n_lo.w, n_hi.x, n_hi.y, n_hi.z, n_hi.w};
    using F = Format<FMT>;
    constexpr uint32_t MAG = (1u << (F::K - 1)) - 1u;
    StatsAcc acc = *sums;
    float x[8], y[8];
    unpack(load_f8(src8), x);
#pragma unroll
    for (int c = 0; c < 8; ++c) y[c] = __fmul_rn(x[c], scale);
    uint32_t codes[8], packed[WordsPerOctet<FMT>::value];
#pragma unroll
    for (int c = 0; c < 8; ++c) {
        const uint32_t bits = y[c] != y[c] ? __float_as_uint(x[c]) : __float_as_uint(y[c]);   // a NaN keeps the input's sign
        codes[c] = round_core<FMT, false>(bits, n[c], variant, k, nullptr);
    }
    pack_codes8<FMT>(codes, packed);
    store_words<WordsPerOctet<FMT>::value>(dst8, packed);
    // group sums are flushed where the run of 8 crosses a group boundary
    uint64_t grp = 0, grp_end = ~0ull;
    double ge = 0.0, ge2 = 0.0;
    if (GROUPS) { grp = i0 / group_size; grp_end = (grp + 1) * group_size; }
#pragma unroll
    for (int c = 0; c < 8; ++c) {
        uint32_t up = 0;
        double e = 0.0;
        if (stats_element<FMT>(__float_as_uint(y[c]), codes[c] & MAG, acc, e, up)) {
            acc.n_finite += 1; acc.n_up += up;
            acc.sum_e += e; acc.sum_e2 = fma(e, e, acc.sum_e2);
            acc.sum_signed_e += (__float_as_uint(y[c]) >> 31) ? -e : e;
            acc.sum_abs_e += fabs(e);
            if (GROUPS) {
                if (i0 + c >= grp_end) {
                    if (ge != 0.0 || ge2 != 0.0) { atomicAdd(gsum_e + grp, ge); atomicAdd(gsum_e2 + grp, ge2); }
                    ge = 0.0; ge2 = 0.0;
                    grp = (i0 + c) / group_size; grp_end = (grp + 1) * group_size;
                }
                ge += e; ge2 = fma(e, e, ge2);
            }
        }
    }
    if (GROUPS && (ge != 0.0 || ge2 != 0.0)) { atomicAdd(gsum_e + grp, ge); atomicAdd(gsum_e2 + grp, ge2); }
    *sums = acc;
}

// Statistics on whole tiles: the rounding of the bandwidth kernel (generator calls shared through the warp's
// buffer, row rounder, packed stores) followed by the integer sums above; octets holding NaN or Inf (and, with
// group sums, octets that straddle a group boundary) go through stats_element() in binary64.  A capped grid walks the tiles with a fixed stride, so each thread adds its
// elements in a fixed order and leaves one partial per CTA: the totals are reproducible bit for bit.
// first_index: index within the call of element 0 (for the group sums).
constexpr int STATS_MIN_CTAS = 3;                        // resident CTAs the compiler must allow (caps the registers at 80)
constexpr int STATS_ROWS_IN_FLIGHT = 2;                  // rows whose loads are outstanding per warp
template <int FMT, int VAR, int K, bool GROUPS>
__global__ void __launch_bounds__(CTA_THREADS, STATS_MIN_CTAS)
stats_tile_kernel(const float* __restrict__ src, const float scale, void* __restrict__ dst, const uint64_t n_tiles,
                  const uint64_t first_index, const uint64_t call0, const uint32_t k0, const uint32_t k1,
                  const uint64_t group_size, double* __restrict__ gsum_e, double* __restrict__ gsum_e2,
                  StatsAcc* __restrict__ partials)
{
    using T = Tile<K, 1>;
    using F = Format<FMT>;
    using X = StatsFixed<FMT>;
    constexpr bool DRAWS = VAR < RTNE;
    constexpr bool OWN_CALL = T::DPW == 2;
    constexpr int ROWS = T::ELEMS / ROW_ELEMS;
    constexpr int WPO = WordsPerOctet<FMT>::value;
    constexpr int U = X::U;
    __shared__ __align__(16) uint32_t wordbuf[WARPS_PER_CTA][OWN_CALL ? 4 : T::BUFFER_WORDS];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    uint32_t* wb = wordbuf[warp];
    StatsAcc acc;                                            // binary64 side: the octets done element by element
    stats_zero(acc);
    StatsInt tot = {0ull, 0ull, 0ull, 0ull, 0u, 0u, 0u, 0u, 0u};
    uint32_t n_up = 0, n_up_neg = 0, fast_octets = 0;       // a thread sees far fewer than 2^32 elements
    StatsDeep deep = {0.0, 0.0, 0.0, 0.0};
    const uint32_t one = min(blockDim.x, 1u);

    for (uint64_t tile = (uint64_t)blockIdx.x * WARPS_PER_CTA + warp; tile < n_tiles;
         tile += (uint64_t)gridDim.x * WARPS_PER_CTA) {
        const size_t e0 = (size_t)tile * T::ELEMS;
        const uint64_t tile_call0 = call0 + tile * T::CALLS;
        constexpr int BATCH = STATS_ROWS_IN_FLIGHT < ROWS ? STATS_ROWS_IN_FLIGHT : ROWS;
        F8 regs[BATCH];
#pragma unroll
        for (int j = 0; j < BATCH; ++j) regs[j] = load_f8_stream(src + e0 + j * ROW_ELEMS + lane * 8);
        if constexpr (DRAWS && !OWN_CALL) {
#pragma unroll
            for (int j = 0; j < (T::CALLS + 31) / 32; ++j) {
                const int c = j * 32 + lane;
                if (T::CALLS % 32 == 0 || c < T::CALLS)
                    Draws8<K>::store_call(wb + Draws8<K>::WORDS_PER_CALL * c, philox_block(tile_call0 + c, k0, k1));
            }
            __syncwarp();
        }
#pragma unroll
        for (int j = 0; j < ROWS; ++j) {
            const int p0 = j * ROW_ELEMS + lane * 8;
            float x[8], y[8];
            unpack(regs[j % BATCH], x);
            if (j + BATCH < ROWS) regs[j % BATCH] = load_f8_stream(src + e0 + (j + BATCH) * ROW_ELEMS + lane * 8);
#pragma unroll
            for (int c = 0; c < 8; ++c) y[c] = __fmul_rn(x[c], scale);
            Draws8<K> d;
            if constexpr (!DRAWS) {
            } else if constexpr (OWN_CALL) {
                d.from_call(philox_block(tile_call0 + p0 / 8, k0, k1));
            } else {
                d.from_normalised(wb, p0);
            }
            uint32_t t[8], packed[WPO];
            const bool redo = round_row_fast<FMT, VAR, K>(y, d, t);
            const uint64_t i0 = first_index + e0 + p0;
            bool fast = !redo;
            if constexpr (GROUPS) fast &= i0 / group_size == (i0 + 7) / group_size;
            if (fast) {
                pack_row_fast<FMT>(t, y, packed);
                StatsInt os = {0ull, 0ull, 0ull, 0ull, 0u, 0u, 0u, 0u, 0u};
                StatsInt& s = GROUPS ? os : tot;
                StatsDeep od = {0.0, 0.0, 0.0, 0.0};
                StatsDeep& dp = GROUPS ? od : deep;
#pragma unroll
                for (int c = 0; c < 8; ++c) stats_fixed_element<FMT>(y[c], t[c], one, s, dp);
                fast_octets += 1;
                if constexpr (GROUPS) {
                    // the octet lies in one group: e and e^2 summed exactly, then one pair of atomics
                    const long long oct_up = os.counts & 0xFFFFu;
                    const long long ge = (oct_up << U) - (long long)os.d_tile;
                    const long long ge2 = (long long)os.d2 + (oct_up << (2 * U)) - ((long long)os.up_d_tile << (U + 1));
                    if (ge != 0 || ge2 != 0 || od.d != 0.0) {
                        const uint64_t grp = i0 / group_size;
                        atomicAdd(gsum_e + grp, (double)ge * __hiloint2double((1023 - U) << 20, 0) - od.d);
                        atomicAdd(gsum_e2 + grp, (double)ge2 * __hiloint2double((1023 - 2 * U) << 20, 0) + (od.d2 - 2.0 * od.up_d));
                    }
                    deep.d += od.d; deep.up_d += od.up_d; deep.neg_d += od.neg_d; deep.d2 += od.d2;
                    tot.d_tile += os.d_tile; tot.up_d_tile += os.up_d_tile; tot.neg_d_tile += os.neg_d_tile; tot.d2 += os.d2;
                    tot.counts += os.counts; tot.n_sat += os.n_sat;
                }
                store_words<WPO>(static_cast<char*>(dst) + (e0 + p0) * (F::K / 8), packed);
            } else {
                uint32_t n[8];
#pragma unroll
                for (int c = 0; c < 8; ++c) n[c] = DRAWS ? d.template at<0>(c) : 0u;
                stats_octet_general<FMT, GROUPS, VAR, K>(&acc, src + e0 + p0, scale, make_uint4(n[0], n[1], n[2], n[3]),
                                                 make_uint4(n[4], n[5], n[6], n[7]), VAR, K,
                                                 static_cast<char*>(dst) + (e0 + p0) * (F::K / 8), i0, group_size, gsum_e, gsum_e2);
            }
        }
        // at most 48 elements a tile: the 32-bit sums and the packed counts are folded in before they can overflow
        tot.d += tot.d_tile; tot.up_d += tot.up_d_tile; tot.neg_d += tot.neg_d_tile;
        tot.d_tile = tot.up_d_tile = tot.neg_d_tile = 0u;
        n_up += tot.counts & 0xFFFFu; n_up_neg += tot.counts >> 16; tot.counts = 0u;
        if constexpr (DRAWS && !OWN_CALL) __syncwarp();      // the buffer is rewritten by the next tile
    }
    // the thread's integer sums, exact, turned into binary64 once
    {
        const double unit = __hiloint2double((1023 - U) << 20, 0), unit2 = __hiloint2double((1023 - 2 * U) << 20, 0);
        const unsigned long long ups = n_up, ups_neg = n_up_neg;
        const long long se = (long long)(ups << U) - (long long)tot.d;
        const long long sneg = (long long)(ups_neg << U) - (long long)tot.neg_d;
        const unsigned long long sabs = tot.d - 2ull * tot.up_d + (ups << U);
        const unsigned __int128 s2 = (unsigned __int128)tot.d2 + ((unsigned __int128)ups << (2 * U)) -
                                     ((unsigned __int128)tot.up_d << (U + 1));
        acc.n_finite += 8ull * fast_octets - tot.n_sat;
        acc.n_up += ups;
        acc.n_sat += tot.n_sat;
        // deep elements: e = up - delta~ with the integer sums holding up alone
        acc.sum_e += (double)se * unit - deep.d;
        acc.sum_signed_e += (double)(se - 2 * sneg) * unit - (deep.d - 2.0 * deep.neg_d);
        acc.sum_abs_e += (double)sabs * unit + (deep.d - 2.0 * deep.up_d);
        acc.sum_e2 += ((double)(unsigned long long)(s2 >> 64) * 18446744073709551616.0 + (double)(unsigned long long)s2) * unit2 +
                      (deep.d2 - 2.0 * deep.up_d);
    }
    stats_cta_reduce(acc);
    if (threadIdx.x == 0) partials[blockIdx.x] = acc;
}

// Sum the per-CTA partials in a fixed order into the caller's fbsr_stats (same layout as StatsAcc).
static __global__ void __launch_bounds__(CTA_THREADS)
stats_finalize_kernel(const StatsAcc* __restrict__ partials, const int n_partials, StatsAcc* __restrict__ total)
{
    StatsAcc acc;
    stats_zero(acc);
    for (int i = threadIdx.x; i < n_partials; i += CTA_THREADS) stats_add(acc, partials[i]);
    stats_cta_reduce(acc);
    if (threadIdx.x == 0) *total = acc;
}

}  // namespace fbsr
