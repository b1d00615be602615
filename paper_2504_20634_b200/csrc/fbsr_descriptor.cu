// fbsr_round_desc: rounding to a format (K, P, B; M) that is described at run time (Section II).
// One kernel for every such format: the element-wise integer rounder with the format's constants as
// kernel arguments.  A thread takes 8 consecutive elements (vector accesses when the pointers allow),
// and computes the one or two generator calls that cover them from their global indices.
#include <cmath>
#include <cstring>

#include "../../include/fbsr.h"
#include "fbsr_device.cuh"
#include "fbsr_internal.h"

namespace fbsr {
namespace {

constexpr int DESC_THREADS = 256;

__global__ void __launch_bounds__(DESC_THREADS)
descriptor_kernel(const float* __restrict__ src, void* __restrict__ dst, const uint64_t n, const uint64_t offset,
                  const float scale, const RtFormat f, const int variant, const int k, const uint32_t k0,
                  const uint32_t k1, const bool ieee_overflow, const bool vectors)
{
    const uint32_t dpw = 32u / (uint32_t)k, E = 4u * dpw, mask = (1u << k) - 1u;      // E >= 8
    const bool draws = variant < RTNE;
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
        const uint64_t g0 = offset + i0, call = g0 / E;
        const uint32_t j0 = (uint32_t)(g0 - call * E);
        uint4 a = make_uint4(0u, 0u, 0u, 0u), b = a;
        if (draws) {
            a = philox_block(call, k0, k1);
            b = (j0 + 7 >= E) ? philox_block(call + 1, k0, k1) : a;
        }
        uint32_t codes[8];
#pragma unroll
        for (int c = 0; c < 8; ++c) {
            uint32_t j = j0 + c;
            const uint4 w4 = j < E ? a : b;
            j = j < E ? j : j - E;
            const uint32_t ws = j / dpw;
            const uint32_t word = ws == 0 ? w4.x : ws == 1 ? w4.y : ws == 2 ? w4.z : w4.w;
            const uint32_t nr = (word >> ((j - ws * dpw) * (uint32_t)k)) & mask;
            codes[c] = round_core_fmt<RtFormat, false, false>(f, scaled_bits(x[c], scale), nr, variant, k, nullptr,
                                                              ieee_overflow);
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
    descriptor_kernel<<<grid, DESC_THREADS, 0, static_cast<cudaStream_t>(cuda_stream)>>>(
        src, dst, (uint64_t)n, offset, scale, f, variant, k_bits, (uint32_t)seed, (uint32_t)(seed >> 32),
        ovf_ieee != 0, vectors);
    count_launch();
    return cudaGetLastError() == cudaSuccess ? FBSR_OK : FBSR_ERR_CUDA;
}
