// fbsr_round_desc: rounding to a format (K, P, B; M) that is described at run time (Section II).
// One kernel for every such format, with the format's constants as kernel arguments.  A thread takes 8
// consecutive elements (vector accesses when the pointers allow) and computes the one or two generator
// calls that cover them from their global indices.
// Rounding: as in the tiled kernels, |y| is first multiplied by 2^(1 - EMINB), toward zero, so that the
// target's exponent range starts where binary32's does; then Eq. (2)-(5) are one addition on the pattern
// with sh0 = 24 - P excess bits: code = (pattern + (n << (sh0 - N))) >> sh0.  This needs N <= sh0 excess
// bits (one more for SRF's half step, two more for SRC's pre-round).  Finite values beyond M saturate by a
// min on the pattern.  Wider draws, Inf, NaN and, with the IEEE overflow option, every value beyond M go
// through the element-wise integer rounder.
#include <cmath>
#include <cstring>

#include "../../include/fbsr.h"
#include "fbsr_device.cuh"
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
    const bool vectors = reinterpret_cast<uintptr_t>(src) % 16 == 0 && reinterpret_cast<uintptr_t>(dst) % (8 * code_bytes) == 0;
    const uint64_t n_octets = ((uint64_t)n + 7) / 8;
    const uint64_t want = (n_octets + DESC_THREADS - 1) / DESC_THREADS;
    const unsigned grid = (unsigned)(want < 0x7FFFFFF0ull ? want : 0x7FFFFFF0ull);
    const uint32_t E = 4u * (32u / (uint32_t)k_bits);
    const uint32_t first_field = (uint32_t)(offset % E);
    const bool short_call = (uint64_t)n + first_field + 8u < 0xFFFFFFFFull;
    descriptor_kernel<<<grid, DESC_THREADS, 0, static_cast<cudaStream_t>(cuda_stream)>>>(
        src, dst, (uint64_t)n, offset / E, first_field, short_call, scale, f, variant, k_bits, (uint32_t)seed, (uint32_t)(seed >> 32),
        ovf_ieee != 0, vectors);
    count_launch();
    return cudaGetLastError() == cudaSuccess ? FBSR_OK : FBSR_ERR_CUDA;
}
