// Host-side plumbing shared by the translation units of libfbsr.so (not part of the public ABI).
#pragma once
#include <cstddef>
#include <cstdint>
#include <cuda_runtime.h>

namespace fbsr {

enum OpKind { OP_ROUND = 0, OP_ROUND_BITS, OP_ROUND_STATS, OP_SGD, OP_ADAM, OP_ACCUM, OP_ROUND_LP, OP_QAT, OP_ROUND_MX, OP_QAT_ADAMW };

// Everything an entry point hands to the per-format dispatcher.  Validated by the caller.
struct CallArgs {
    OpKind op;
    int variant, k;
    int ovf_ieee;                   // finite values beyond M: IEEE nearest-even instead of saturation
    size_t n;
    uint64_t seed, offset;
    cudaStream_t stream;
    void* dst;                      // low-precision codes (w_lp for OP_ACCUM)
    // OP_ROUND*, OP_ACCUM (src = update)
    const float* src;
    float scale;
    const uint32_t* words;          // OP_ROUND_BITS
    uint8_t* scales;                // OP_ROUND_MX: one exponent byte per block of 32
    const void* src_lp;             // OP_ROUND_LP: codes of src_fmt; OP_QAT: the 16-bit updates
    int src_fmt;
    // OP_ROUND_STATS
    size_t group_size;
    double* gsum_e;
    double* gsum_e2;
    void* total;                    // fbsr_stats*
    void* partials;                 // workspace
    // OP_SGD / OP_ADAM
    float* w; const float* g; float* m; float* v;
    float neg_lr, mu;                                   // SGD-momentum
    float beta1, beta2, eps, neg_c1, c2, a1, a2;        // Adam
    float neg_lrwd;                                     // OP_QAT_ADAMW: -(lr * weight_decay)
};

constexpr int MAX_SLOW_GRID = 148 * 8;      // CTAs of the general kernel; also the number of partial slots

// One dispatcher per (format, op group); each lives in its own translation unit
// (dispatch_lp_* and dispatch_qat_adamw_* exist for the 8-bit targets only).
#define FBSR_DECLARE_DISPATCH(fmt) \
    int dispatch_round_##fmt(const CallArgs&); \
    int dispatch_round_words_##fmt(const CallArgs&); \
    int dispatch_stats_##fmt(const CallArgs&); \
    int dispatch_optim_##fmt(const CallArgs&);\
    int dispatch_lp_##fmt(const CallArgs&); \
    int dispatch_qat_##fmt(const CallArgs&); \
    int dispatch_qat_adamw_##fmt(const CallArgs&);
FBSR_DECLARE_DISPATCH(0) FBSR_DECLARE_DISPATCH(1) FBSR_DECLARE_DISPATCH(2) FBSR_DECLARE_DISPATCH(3) FBSR_DECLARE_DISPATCH(4)
#undef FBSR_DECLARE_DISPATCH

void count_launch();                         // bumps the counter behind fbsr_launch_count()

}  // namespace fbsr
