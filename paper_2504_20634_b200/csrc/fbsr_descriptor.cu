// fbsr_round_desc: rounding to a format (K, P, B; M) that is described at run time (Section II); the format's
// constants are kernel arguments.  Two kernels: descriptor_tile_kernel for whole tiles of the draw stream (variant
// and draw width compile-time, generator calls shared through the warp's buffer), and descriptor_kernel, fully
// general (run-time variant and draw width, any alignment and offset), for the head, the ragged end and unaligned
// calls.  In the general kernel a thread takes 8 consecutive elements (vector accesses when the pointers allow) and
// computes the one or two generator calls that cover them from their global indices.
// Rounding: as in the tiled kernels, |y| is first multiplied by 2^(1 - EMINB), toward zero, so that the
// target's exponent range starts where binary32's does; then Eq. (2)-(5) are one addition on the pattern
// with sh0 = 24 - P excess bits: code = (pattern + (n << (sh0 - N))) >> sh0.  This needs N <= sh0 excess
// bits (one more for SRF's half step, two more for SRC's pre-round).  Finite values beyond M saturate by a
// min on the pattern.  Wider draws, Inf, NaN and, with the IEEE overflow option, every value beyond M go
// through the element-wise integer rounder.
#include <cmath>
#include <cstring>
#include <utility>

#include "../../include/fbsr.h"
#include "fbsr_device.cuh"
#include "fbsr_kernels.cuh"
#include "fbsr_internal.h"

namespace fbsr {
namespace {

constexpr int DESC_THREADS = 256;

__global__ void __launch_bounds__(DESC_THREADS)
descriptor_kernel(const float* __restrict__ src, void* __restrict__ dst, const uint64_t n, const uint64_t call_base,
                  const uint32_t first_field, const bool short_call, const float scale, const RtFormat f, const int variant, const int k, const uint32_t k0,
                  const uint32_t k1, const bool ieee_overflow, const bool vectors)
{
    const uint32_t dpw = 32u / (uint32_t)k, E = 4u * dpw, mask = (1u << k) - 1u;      // E >= 8
    const bool draws = variant < RTNE;
    // the one-addition form and its constants
    const int sh0 = 24 - f.P;                                                           // >= 11
    const int needed = variant == SRF ? k + 1 : variant == SRC ? k + 2 : k;
    const bool one_addition = !draws || needed <= sh0;
    const int pos = draws ? sh0 - k : sh0;                   // where the draw (or the half step) is added
    const uint32_t half = one_addition && pos > 0 ? 1u << (pos - 1) : 0u;
    const uint32_t below_half = half ? half - 1u : 0u;
    const bool sticky = variant == SRC || variant == RTNE || variant == RTO;
    const uint32_t flip = variant == RTO ? 1u : 0u;
    const float rescale = __uint_as_float((uint32_t)(128 - f.EMINB) << 23);            // 2^(1 - EMINB)
    const uint32_t max_pattern = f.MAXCODE << sh0;                                      // rescaled pattern of M
    const uint64_t n_octets = (n + 7) / 8;
    for (uint64_t o = (uint64_t)blockIdx.x * DESC_THREADS + threadIdx.x; o < n_octets;
         o += (uint64_t)gridDim.x * DESC_THREADS) {
        const uint64_t i0 = o * 8;
        const int cnt = (int)min((uint64_t)8, n - i0);
        const bool whole = vectors && cnt == 8;
        float x[8];
        if (whole) {
            const float4 lo = __ldg(reinterpret_cast<const float4*>(src + i0));
            const float4 hi = __ldg(reinterpret_cast<const float4*>(src + i0) + 1);
            x[0] = lo.x; x[1] = lo.y; x[2] = lo.z; x[3] = lo.w; x[4] = hi.x; x[5] = hi.y; x[6] = hi.z; x[7] = hi.w;
        } else {
#pragma unroll
            for (int c = 0; c < 8; ++c) x[c] = c < cnt ? src[i0 + c] : 0.0f;
        }
        // global index of element i0 = call_base * E + first_field + i0; a 32-bit division when the call is short
        const uint64_t rel = (uint64_t)first_field + i0;
        const uint64_t q = short_call ? (uint64_t)((uint32_t)rel / E) : rel / E;
        const uint64_t call = call_base + q;
        const uint32_t j0 = (uint32_t)(rel - q * E);
        uint4 a = make_uint4(0u, 0u, 0u, 0u), b = a;
        if (draws) {
            a = philox_block(call, k0, k1);
            b = (j0 + 7 >= E) ? philox_block(call + 1, k0, k1) : a;
        }
        // word and field of the first element; the following ones are reached by stepping, without divisions
        uint32_t ws = j0 / dpw, shift = (j0 - ws * dpw) * (uint32_t)k;
        const uint32_t shift_end = dpw * (uint32_t)k;
        uint4 cur = a;
        uint32_t codes[8];
#pragma unroll
        for (int c = 0; c < 8; ++c) {
            const uint32_t word = ws == 0 ? cur.x : ws == 1 ? cur.y : ws == 2 ? cur.z : cur.w;
            const uint32_t nr = (word >> shift) & mask;
            const uint32_t yb = scaled_bits(x[c], scale);
            const uint32_t mbits = yb & 0x7FFFFFFFu;
            if (one_addition && mbits <= (ieee_overflow ? f.MAXBITS : 0x7F7FFFFFu)) {
                const float mag = __uint_as_float(mbits);
                uint32_t u = __float_as_uint(__fmul_rz(mag, rescale));
                if (sticky) u |= (u ^ __float_as_uint(__fmul_ru(mag, rescale))) & 1u;   // what the truncation lost
                u = min(u, max_pattern);                     // finite values beyond M saturate: nothing added below can carry past M
                uint32_t sum;
                if (variant == SRFF) sum = u + (nr << pos);
                else if (variant == SRF) sum = u + half + (nr << pos);
                else if (variant == RTA) sum = u + half;
                else sum = u + below_half + (((u >> pos) & 1u) ^ flip) + (draws ? nr << pos : 0u);
                const uint32_t code = sum >> sh0;
                const uint32_t sign = (yb >> 31) << (f.K - 1);
                codes[c] = (f.SINGLE_ZERO && code == 0u) ? 0u : (code | sign);
            } else {
                codes[c] = round_core_fmt<RtFormat, false, false>(f, yb, nr, variant, k, nullptr, ieee_overflow);
            }
            shift += (uint32_t)k;
            if (shift == shift_end) {
                shift = 0u;
                if (++ws == 4u) { ws = 0u; cur = b; }
            }
        }
        if (whole) {
            if (f.K == 16) {
                *reinterpret_cast<uint4*>(static_cast<uint16_t*>(dst) + i0) =
                    make_uint4(codes[0] | (codes[1] << 16), codes[2] | (codes[3] << 16),
                               codes[4] | (codes[5] << 16), codes[6] | (codes[7] << 16));
            } else {
                *reinterpret_cast<uint2*>(static_cast<uint8_t*>(dst) + i0) =
                    make_uint2(codes[0] | (codes[1] << 8) | (codes[2] << 16) | (codes[3] << 24),
                               codes[4] | (codes[5] << 8) | (codes[6] << 16) | (codes[7] << 24));
            }
        } else {
#pragma unroll
            for (int c = 0; c < 8; ++c) {
                if (c < cnt) {
                    if (f.K == 16) static_cast<uint16_t*>(dst)[i0 + c] = (uint16_t)codes[c];
                    else static_cast<uint8_t*>(dst)[i0 + c] = (uint8_t)codes[c];
                }
            }
        }
    }
}

// Whole tiles with the variant and the draw width fixed at compile time and only the format left to run time:
// the generator calls of a tile are shared through the warp's buffer and the fields are taken from the packed
// word stream, as in the bandwidth kernel; a lane owns 8 consecutive elements of a 256-element row.
// one_addition: the draw fits under the format's 24 - P excess bits (decided by the host, uniform for the launch).
// ROW_FORM (decided by the host): the draw fits under the excess bits and the code fits above them, so whole
// lane-rows are rounded by the one-addition form; otherwise every element goes through the element-wise rounder.
template <int VAR, int N, int CODE_BYTES, bool ROW_FORM>
__global__ void __launch_bounds__(CTA_THREADS, 3)
descriptor_tile_kernel(const float* __restrict__ src, const float scale, void* __restrict__ dst, const uint64_t n_tiles,
                       const uint64_t call0, const uint32_t k0, const uint32_t k1, const RtFormat f,
                       const bool ieee_overflow, const bool one_addition)
{
    using T = Tile<N, 1>;
    constexpr bool DRAWS = VAR < RTNE;
    constexpr bool OWN_CALL = T::DPW == 2;
    constexpr int ROWS = T::ELEMS / ROW_ELEMS;
    __shared__ __align__(16) uint32_t wordbuf[WARPS_PER_CTA][OWN_CALL ? 4 : T::BUFFER_WORDS];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    uint32_t* wb = wordbuf[warp];
    const int sh0 = 24 - f.P;
    const int pos = DRAWS ? sh0 - N : sh0;                   // >= 0 whenever one_addition holds
    const uint32_t half = pos > 0 ? 1u << (pos - 1) : 0u;
    const uint32_t below_half = half ? half - 1u : 0u;
    constexpr bool STICKY = VAR == SRC || VAR == RTNE || VAR == RTO;
    const float rescale = __uint_as_float((uint32_t)(128 - f.EMINB) << 23);            // 2^(1 - EMINB)
    const uint32_t max_pattern = f.MAXCODE << sh0;
    const uint32_t fast_limit = ieee_overflow ? f.MAXBITS : 0x7F7FFFFFu;
    const uint32_t sign_shift = 32u - (uint32_t)(8 * CODE_BYTES);
    // Row form, as in the bandwidth kernel: the saturated pattern is moved left so that the code comes out of the
    // addition in the top K bits (packing is then byte selection), the draw is rotated to where it is added and
    // masked there, and Inf / NaN are found per lane-row by a floating-point flag and redone element by element.
    // It needs the code to fit above the excess bits (32 - K - sh0 >= 0: every format with at most 8 exponent bits).
    constexpr int KBITS = 8 * CODE_BYTES;
    const int lift = 32 - KBITS - sh0;                        // left shift of the pattern
    constexpr bool row_form = ROW_FORM;
    const uint32_t lift_mul = row_form ? 1u << lift : 1u;
    const int draw_pos = pos + (row_form ? lift : 0);         // bit where the draw's lowest bit is added
    const uint32_t draw_mask = DRAWS ? ((1u << N) - 1u) << draw_pos : 0u;
    const uint32_t half_l = half * lift_mul, below_half_l = below_half * lift_mul;
    const float tie = __uint_as_float(f.MAXBITS + (1u << (sh0 - 1)));          // M + ulp(M) / 2
    const bool tie_overflows = (f.MAXCODE & 1u) != 0u;
    const uint32_t overflow_top = (f.HAS_INF ? f.INFCODE : f.NANCODE) << (32 - KBITS);
    const uint32_t zero_mask = f.SINGLE_ZERO ? 0xFFFFFFFFu : 0u;

    for (uint64_t tile = (uint64_t)blockIdx.x * WARPS_PER_CTA + warp; tile < n_tiles;
         tile += (uint64_t)gridDim.x * WARPS_PER_CTA) {
        const size_t e0 = (size_t)tile * T::ELEMS;
        const uint64_t tile_call0 = call0 + tile * T::CALLS;
        constexpr int BATCH = ROWS < 4 ? ROWS : (ROWS % 3 == 0 ? 3 : (ROWS % 2 == 0 ? 2 : ROWS));
        F8 regs[BATCH];
#pragma unroll
        for (int j = 0; j < BATCH; ++j) regs[j] = load_f8_stream(src + e0 + j * ROW_ELEMS + lane * 8);
        if constexpr (DRAWS && !OWN_CALL) {
#pragma unroll
            for (int j = 0; j < (T::CALLS + 31) / 32; ++j) {
                const int c = j * 32 + lane;
                if (T::CALLS % 32 == 0 || c < T::CALLS)
                    Draws8<N>::store_call(wb + Draws8<N>::WORDS_PER_CALL * c, philox_block(tile_call0 + c, k0, k1));
            }
            __syncwarp();
        }
#pragma unroll
        for (int rb = 0; rb < ROWS; rb += BATCH) {
            if (rb > 0) {
#pragma unroll
                for (int j = 0; j < BATCH; ++j)
                    if (rb + j < ROWS) regs[j] = load_f8_stream(src + e0 + (rb + j) * ROW_ELEMS + lane * 8);
            }
#pragma unroll
            for (int j = 0; j < BATCH; ++j) {
                if (rb + j >= ROWS) continue;
                const int p0 = (rb + j) * ROW_ELEMS + lane * 8;
                float x[8];
                unpack(regs[j], x);
                Draws8<N> d;
                if constexpr (!DRAWS) {
                } else if constexpr (OWN_CALL) {
                    d.from_call(philox_block(tile_call0 + p0 / 8, k0, k1));
                } else {
                    d.from_normalised(wb, p0);
                }
                if constexpr (row_form) {
                    float y[8], flag = 0.0f;
                    uint32_t t[8];
#pragma unroll
                    for (int c = 0; c < 8; ++c) {
                        y[c] = __fmul_rn(x[c], scale);
                        flag = __fmaf_rn(y[c], 0.0f, flag);                      // NaN iff y is Inf or NaN
                        uint32_t u = __float_as_uint(__fmul_rz(fabsf(y[c]), rescale));
                        if constexpr (STICKY) u |= (u ^ __float_as_uint(__fmul_ru(fabsf(y[c]), rescale))) & 1u;
                        u = min(u, max_pattern);
                        const uint32_t base = u * lift_mul;
                        uint32_t draw = 0u;
                        if constexpr (DRAWS) {
                            // the field of element c sits at bit b of its word: rotate it to draw_pos and mask it there
                            constexpr int G = Draws8<N>::G;
                            const int b = (c % G) * N;
                            draw = __funnelshift_l(d.u[c / G], d.u[c / G], (uint32_t)(draw_pos - b) & 31u) & draw_mask;
                        }
                        if constexpr (VAR == SRFF) t[c] = base + draw;
                        else if constexpr (VAR == SRF) t[c] = base + half_l + draw;
                        else if constexpr (VAR == RTA) t[c] = base + half_l;
                        else t[c] = base + below_half_l + ((((u >> pos) & 1u) ^ (VAR == RTO ? 1u : 0u)) * lift_mul) + draw;
                        if (ieee_overflow) {
                            const bool beyond = tie_overflows ? fabsf(y[c]) >= tie : fabsf(y[c]) > tie;
                            t[c] = beyond ? overflow_top : t[c];
                        }
                    }
                    if (flag == flag) {
                        // codes in the top K bits, bit 31 clear: pack by byte selection, signs from y
                        if constexpr (CODE_BYTES == 2) {
                            uint32_t w[4];
#pragma unroll
                            for (int q = 0; q < 4; ++q) {
                                const uint32_t cw = __byte_perm(t[2 * q], t[2 * q + 1], 0x7632);
                                uint32_t sg = __byte_perm(__float_as_uint(y[2 * q]), __float_as_uint(y[2 * q + 1]), 0x7632) & 0x80008000u;
                                sg &= ~zero_mask | (cw + 0x7FFF7FFFu);                // one zero only: a zero magnitude takes no sign
                                w[q] = cw | sg;
                            }
                            store_words<4>(static_cast<char*>(dst) + (e0 + p0) * 2, w);
                        } else {
                            uint32_t w[2];
#pragma unroll
                            for (int q = 0; q < 2; ++q) {
                                const uint32_t c01 = __byte_perm(t[4 * q], t[4 * q + 1], 0x7373), c23 = __byte_perm(t[4 * q + 2], t[4 * q + 3], 0x7373);
                                const uint32_t s01 = __byte_perm(__float_as_uint(y[4 * q]), __float_as_uint(y[4 * q + 1]), 0x7373);
                                const uint32_t s23 = __byte_perm(__float_as_uint(y[4 * q + 2]), __float_as_uint(y[4 * q + 3]), 0x7373);
                                const uint32_t cw = __byte_perm(c01, c23, 0x5410);
                                uint32_t sg = __byte_perm(s01, s23, 0x5410) & 0x80808080u;
                                sg &= ~zero_mask | (cw + 0x7F7F7F7Fu);
                                w[q] = cw | sg;
                            }
                            store_words<2>(static_cast<char*>(dst) + (e0 + p0), w);
                        }
                        continue;
                    }
                }
                uint32_t codes[8];
#pragma unroll
                for (int c = 0; c < 8; ++c) {
                    const uint32_t yb = __float_as_uint(__fmul_rn(x[c], scale));    // a NaN takes the other branch
                    const uint32_t mbits = yb & 0x7FFFFFFFu;
                    const uint32_t nr = DRAWS ? d.template at<0>(c) : 0u;
                    if (!row_form && one_addition && mbits <= fast_limit) {
                        const float mag = __uint_as_float(mbits);
                        uint32_t u = __float_as_uint(__fmul_rz(mag, rescale));
                        if constexpr (STICKY) u |= (u ^ __float_as_uint(__fmul_ru(mag, rescale))) & 1u;
                        u = min(u, max_pattern);
                        uint32_t sum;
                        if constexpr (VAR == SRFF) sum = u + (nr << pos);
                        else if constexpr (VAR == SRF) sum = u + half + (nr << pos);
                        else if constexpr (VAR == RTA) sum = u + half;
                        else sum = u + below_half + (((u >> pos) & 1u) ^ (VAR == RTO ? 1u : 0u)) + (DRAWS ? nr << pos : 0u);
                        const uint32_t code = sum >> sh0;
                        codes[c] = (f.SINGLE_ZERO && code == 0u) ? 0u : (code | ((yb >> 31) << (31u - sign_shift)));
                    } else {
                        // scaled_bits: a NaN input keeps its own sign
                        codes[c] = round_core_fmt<RtFormat, false, false>(f, scaled_bits(x[c], scale), nr, VAR, N, nullptr,
                                                                          ieee_overflow);
                    }
                }
                if constexpr (CODE_BYTES == 2) {
                    const uint32_t w[4] = {codes[0] | (codes[1] << 16), codes[2] | (codes[3] << 16),
                                           codes[4] | (codes[5] << 16), codes[6] | (codes[7] << 16)};
                    store_words<4>(static_cast<char*>(dst) + (e0 + p0) * 2, w);
                } else {
                    const uint32_t w[2] = {codes[0] | (codes[1] << 8) | (codes[2] << 16) | (codes[3] << 24),
                                           codes[4] | (codes[5] << 8) | (codes[6] << 16) | (codes[7] << 24)};
                    store_words<2>(static_cast<char*>(dst) + (e0 + p0), w);
                }
            }
        }
        if constexpr (DRAWS && !OWN_CALL) __syncwarp();      // the buffer is rewritten by the next tile
    }
}

struct TileCall {
    const float* src; void* dst; uint64_t n_tiles, call0; float scale; uint32_t k0, k1; RtFormat f;
    bool ieee_overflow, one_addition; cudaStream_t stream;
};

template <int VAR, int N>
void launch_descriptor_tiles(const TileCall& t)
{
    const uint64_t want = (t.n_tiles + WARPS_PER_CTA - 1) / WARPS_PER_CTA;
    const unsigned grid = (unsigned)(want < 0x7FFFFFF0ull ? want : 0x7FFFFFF0ull);
    const bool row_form = t.one_addition && 32 - t.f.K - (24 - t.f.P) >= 0;
    auto kern = t.f.K == 16 ? (row_form ? descriptor_tile_kernel<VAR, N, 2, true> : descriptor_tile_kernel<VAR, N, 2, false>)
                            : (row_form ? descriptor_tile_kernel<VAR, N, 1, true> : descriptor_tile_kernel<VAR, N, 1, false>);
    kern<<<grid, CTA_THREADS, 0, t.stream>>>(t.src, t.scale, t.dst, t.n_tiles, t.call0, t.k0, t.k1, t.f, t.ieee_overflow,
                                             t.one_addition);
    count_launch();
}

template <int VAR>
void descriptor_tiles_by_k(int k, const TileCall& t)
{
    switch (k) {
    case 1: return launch_descriptor_tiles<VAR, 1>(t);
    case 2: return launch_descriptor_tiles<VAR, 2>(t);
    case 3: return launch_descriptor_tiles<VAR, 3>(t);
    case 4: return launch_descriptor_tiles<VAR, 4>(t);
    case 5: return launch_descriptor_tiles<VAR, 5>(t);
    case 6: return launch_descriptor_tiles<VAR, 6>(t);
    case 7: return launch_descriptor_tiles<VAR, 7>(t);
    case 8: return launch_descriptor_tiles<VAR, 8>(t);
    case 9: return launch_descriptor_tiles<VAR, 9>(t);
    case 10: return launch_descriptor_tiles<VAR, 10>(t);
    case 11: return launch_descriptor_tiles<VAR, 11>(t);
    case 12: return launch_descriptor_tiles<VAR, 12>(t);
    case 13: return launch_descriptor_tiles<VAR, 13>(t);
    case 14: return launch_descriptor_tiles<VAR, 14>(t);
    case 15: return launch_descriptor_tiles<VAR, 15>(t);
    default: return launch_descriptor_tiles<VAR, 16>(t);
    }
}

// Elements per tile for k bits per draw (the deterministic modes use the 1024-element tile of k = 16).
template <int... Ks>
size_t tile_elements_of(int k, std::integer_sequence<int, Ks...>)
{
    static constexpr size_t table[16] = {(size_t)Tile<Ks + 1, 1>::ELEMS...};
    return table[k - 1];
}
size_t descriptor_tile_elements(int variant, int k)
{
    return tile_elements_of(variant >= RTNE ? 16 : k, std::make_integer_sequence<int, 16>{});
}

// The general kernel on elements [begin, end) of the call.
void launch_descriptor_general(const float* src, void* dst, size_t begin, size_t end, const RtFormat& f, int variant, int k,
                               uint64_t seed, uint64_t offset, float scale, bool ieee, cudaStream_t stream)
{
    if (begin >= end) return;
    const size_t n = end - begin, cb = (size_t)f.K / 8;
    const float* s = src + begin;
    void* d = static_cast<char*>(dst) + begin * cb;
    const bool vectors = reinterpret_cast<uintptr_t>(s) % 16 == 0 && reinterpret_cast<uintptr_t>(d) % (8 * cb) == 0;
    const uint64_t n_octets = ((uint64_t)n + 7) / 8;
    const uint64_t want = (n_octets + DESC_THREADS - 1) / DESC_THREADS;
    const unsigned grid = (unsigned)(want < 0x7FFFFFF0ull ? want : 0x7FFFFFF0ull);
    const uint32_t E = 4u * (32u / (uint32_t)k);
    const uint64_t g0 = offset + begin;
    const uint32_t first_field = (uint32_t)(g0 % E);
    const bool short_call = (uint64_t)n + first_field + 8u < 0xFFFFFFFFull;
    descriptor_kernel<<<grid, DESC_THREADS, 0, stream>>>(s, d, (uint64_t)n, g0 / E, first_field, short_call, scale, f, variant, k,
                                                         (uint32_t)seed, (uint32_t)(seed >> 32), ieee, vectors);
    count_launch();
}

// Checks the descriptor and fills in the constants the rounder needs.  Returns false if it is not accepted.
bool make_rt_format(const fbsr_format_desc* d, RtFormat* f)
{
    if (d == nullptr || (d->K != 8 && d->K != 16)) return false;
    if (d->P < 2 || d->P > d->K - 1 || d->P > 13) return false;
    if (d->B < 1 || d->B > 127) return false;
    const uint32_t magnitudes = (1u << (d->K - 1)) - 1u;
    if (d->max_code == 0u || d->max_code > magnitudes) return false;
    const int e_field = (int)(d->max_code >> (d->P - 1));
    const uint32_t t_field = d->max_code & ((1u << (d->P - 1)) - 1u);
    if (e_field - d->B > 127) return false;                                  // M must be a finite binary32 value
    if (d->has_inf && (d->inf_code <= d->max_code || d->inf_code > magnitudes)) return false;
    if (d->single_zero) {
        if (d->nan_code != (1u << (d->K - 1))) return false;
    } else if (d->nan_code <= d->max_code || d->nan_code > magnitudes || (d->has_inf && d->nan_code == d->inf_code)) {
        return false;
    }
    // M by Eq. (1), exact in binary32 (P <= 13 significand bits, exponent within range)
    const float M = e_field == 0 ? std::ldexp((float)t_field, 2 - d->P - d->B)
                                 : std::ldexp((float)((1u << (d->P - 1)) | t_field), e_field - d->B - (d->P - 1));
    uint32_t mbits;
    std::memcpy(&mbits, &M, 4);
    f->K = d->K; f->P = d->P; f->EMINB = 128 - d->B;
    f->MAXBITS = mbits; f->MAXCODE = d->max_code;
    f->INFCODE = d->has_inf ? d->inf_code : d->max_code;
    f->NANCODE = d->nan_code;
    f->SINGLE_ZERO = d->single_zero != 0; f->HAS_INF = d->has_inf != 0;
    return true;
}

}  // namespace
}  // namespace fbsr

extern "C" int fbsr_format_desc_valid(const fbsr_format_desc* desc)
{
    fbsr::RtFormat f;
    return fbsr::make_rt_format(desc, &f) ? 1 : 0;
}

extern "C" int fbsr_round_desc(const float* src, void* dst, size_t n, const fbsr_format_desc* desc, int ovf_ieee,
                               int variant, int k_bits, uint64_t seed, uint64_t offset, float scale, void* cuda_stream)
{
    using namespace fbsr;
    RtFormat f;
    if (!make_rt_format(desc, &f)) return FBSR_ERR_INVALID_ARG;
    if (variant < 0 || variant > 5 || k_bits < 1 || k_bits > 16) return FBSR_ERR_INVALID_ARG;
    if (!(scale > 0.0f) || !std::isfinite(scale)) return FBSR_ERR_INVALID_ARG;
    if (n > 0 && (src == nullptr || dst == nullptr)) return FBSR_ERR_INVALID_ARG;
    const size_t code_bytes = (size_t)f.K / 8;
    if (reinterpret_cast<uintptr_t>(src) % 4 != 0 || reinterpret_cast<uintptr_t>(dst) % code_bytes != 0) return FBSR_ERR_ALIGNMENT;
    if (n == 0) return FBSR_OK;
    const cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
    const bool ieee = ovf_ieee != 0;
    // Whole tiles of the draw stream go to the tiled kernel when the pointers allow its vector accesses; the head
    // before the first tile boundary, the ragged end, and calls with unaligned pointers go to the general kernel.
    const size_t tile = descriptor_tile_elements(variant, k_bits);
    const size_t head = (size_t)((tile - offset % tile) % tile);
    size_t n_tiles = 0;
    if (head < n && reinterpret_cast<uintptr_t>(src + head) % 32 == 0 &&
        reinterpret_cast<uintptr_t>(static_cast<char*>(dst) + head * code_bytes) % (8 * code_bytes) == 0)
        n_tiles = (n - head) / tile;
    if (n_tiles == 0) {
        launch_descriptor_general(src, dst, 0, n, f, variant, k_bits, seed, offset, scale, ieee, stream);
    } else {
        const int needed = variant == SRF ? k_bits + 1 : variant == SRC ? k_bits + 2 : k_bits;
        const int k_tile = variant >= RTNE ? 16 : k_bits;
        TileCall t{src + head, static_cast<char*>(dst) + head * code_bytes, n_tiles,
                   (offset + head) / (4u * (32u / (uint32_t)k_tile)), scale, (uint32_t)seed, (uint32_t)(seed >> 32), f, ieee,
                   variant >= RTNE || needed <= 24 - f.P, stream};
        launch_descriptor_general(src, dst, 0, head, f, variant, k_bits, seed, offset, scale, ieee, stream);
        switch (variant) {
        case SRFF: descriptor_tiles_by_k<SRFF>(k_bits, t); break;
        case SRF: descriptor_tiles_by_k<SRF>(k_bits, t); break;
        case SRC: descriptor_tiles_by_k<SRC>(k_bits, t); break;
        case RTNE: launch_descriptor_tiles<RTNE, 16>(t); break;
        case RTA: launch_descriptor_tiles<RTA, 16>(t); break;
        default: launch_descriptor_tiles<RTO, 16>(t); break;
        }
        launch_descriptor_general(src, dst, head + n_tiles * tile, n, f, variant, k_bits, seed, offset, scale, ieee, stream);
    }
    return cudaGetLastError() == cudaSuccess ? FBSR_OK : FBSR_ERR_CUDA;
}
