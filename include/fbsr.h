/*
 * fbsr.h -- few-bit stochastic rounding (FBSR) on NVIDIA B200 (sm_100a).
 *
 * C-ABI of libfbsr.so.  The operations follow "On Stochastic Rounding with Few
 * Random Bits" (Fitzgibbon & Felix): a binary32 value y is rounded to a narrower
 * format (K, P, B; M) by
 *     e~     = max(floor(log2 |y|), 1 - B)                      Section II-A, Eq. (2)
 *     sigma~ = |y| 2^-e~ 2^(P-1),  delta~ = sigma~ - floor(sigma~)           Eq. (3)
 *     sigma  = floor(sigma~) + [R(delta~, n)]                                Eq. (5)
 * with n an integer of N = k_bits random bits and R one of
 *     R_SRFF(d, n) = d + n 2^-N >= 1                            Section II-B
 *     R_SRF (d, n) = d + (n + 1/2) 2^-N >= 1                    Section II-B
 *     R_SRC (d, n) = R_SRFF(Round(d 2^N) 2^-N, n)               Section III-F, Eq. (8)
 * (Round = nearest, ties to even).  sigma = 2^P increments the exponent.
 *
 * Conventions shared by every entry point unless stated otherwise
 *   - Pointers are DEVICE pointers owned by the caller.  The library allocates no
 *     memory, never synchronises, and only enqueues work on `cuda_stream`
 *     (a cudaStream_t passed as void*; NULL = the default stream) of the current
 *     device.  Buffers must stay valid until that work has run.
 *   - Results are a pure function of the arguments: the same (seed, offset)
 *     gives the same bits on every call and for every way of splitting a tensor
 *     into calls, provided `offset` is the global index of element 0.
 *   - The magnitude is rounded and the sign copied.  NaN -> quiet NaN, sign of
 *     the input kept (0x7FC0 bf16, 0x7E00 fp16, 0x7F e4m3 and e5m2).  +-Inf ->
 *     +-Inf, or +-M for e4m3, which has no infinity.  Finite |y| > M -> +-M.
 *     Binary8P4 has one zero and one NaN: a zero result is 0x00 whatever the sign
 *     of the input (-0, or a negative value rounded down to zero), NaN -> 0x80.
 *     None of these consume the paper's predicates (Section II leaves values
 *     outside the finite range to deterministic rounding).
 *   - Random draws: Philox4x32-10 with key (seed lo, seed hi).  With
 *     dpw = 32 / k_bits (integer division) draws per 32-bit word and E = 4 dpw,
 *     the element with global index g uses field (g mod dpw), low bits first, of
 *     output word ((g mod E) / dpw) of the generator call with counter
 *     (b lo, b hi, 0, 0), b = g / E.  The paper leaves the generator open
 *     (Section II-B); this indexing is the library's definition.
 *   - Any n (including 0) and any element alignment are accepted.  The fast
 *     path needs src 32-byte aligned, dst 16-byte aligned and `offset` a multiple
 *     of the tile size reported by fbsr_tile_elements(); other calls are served
 *     by a slower kernel with identical results.  fbsr_round itself has a second
 *     fast kernel that takes pointers of any element alignment (a slice of a
 *     tensor, a packed parameter buffer) at about four fifths of the speed; the
 *     part of a call before the first tile boundary of `offset` (less than one
 *     tile) always goes to the slower kernel.
 *   - Errors are reported by the return value only.  Nothing is written on error.
 */
#ifndef FBSR_H
#define FBSR_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
    FBSR_OK = 0,
    FBSR_ERR_INVALID_ARG = 1, /* null pointer with n > 0, bad enum, k_bits outside 1..16, bad scale */
    FBSR_ERR_UNSUPPORTED = 2, /* a combination this build does not implement */
    FBSR_ERR_ALIGNMENT = 3,   /* a pointer is not aligned to its element size */
    FBSR_ERR_CUDA = 4,        /* the CUDA runtime reported an error at launch */
    FBSR_ERR_WORKSPACE = 5,   /* workspace missing or too small */
    FBSR_ERR_TOO_LARGE = 6    /* n exceeds the limit of an entry point with built-in scratch */
} fbsr_status;

/* Target formats (K, P, B; M), Section II.  P counts the hidden bit. */
typedef enum {
    FBSR_BF16 = 0, /* (16,  8, 127; 0x1.FEp127) */
    FBSR_FP16 = 1, /* (16, 11,  15; 65504)      */
    FBSR_E4M3 = 2, /* ( 8,  4,   7; 448)   OCP E4M3: no Inf, S.1111.111 is NaN */
    FBSR_E5M2 = 3, /* ( 8,  3,  15; 57344) */
    FBSR_B8P4 = 4  /* ( 8,  4,   8; 224)   IEEE WG P3109 Binary8P4, the target of Section IV:
                      0x7F / 0xFF are +-Inf, 0x80 is the NaN, there is no negative zero */
} fbsr_fmt;

/* May be or-ed into any `fmt` argument.  Section II leaves values beyond the finite range to the deterministic
 * nearest rounding of IEEE 754; with this flag finite |y| > M follow that reading (M below M + ulp(M)/2, +-Inf
 * above it -- the NaN code for e4m3 -- ties to the even neighbour) instead of saturating.  fbsr_round and
 * fbsr_round_lp serve the flag at full speed on aligned calls (one comparison per element in the tiled kernel);
 * the other entry points, and calls whose pointers are off the fast path's alignment, use the general kernel. */
#define FBSR_OVF_IEEE 0x100

/* Round-up predicates: the few-bit stochastic ones of Section II-B and Eq. (8), and the deterministic
 * ones of Section II-A (ties to even, ties away from zero (Eq. (4)), ties to odd), which use no draw:
 * for those k_bits, seed and offset are ignored (k_bits must still be in 1..16). */
typedef enum {
    FBSR_SRFF = 0, FBSR_SRF = 1, FBSR_SRC = 2,
    FBSR_RTNE = 3, FBSR_RTA = 4, FBSR_RTO = 5
} fbsr_variant;

/* Error statistics over the SR-rounded elements of one call.  e = up - delta~
 * is the rounding error of the magnitude in target ulps, the quantity whose
 * mean Section III calls bias.  NaN, Inf and saturated elements are counted
 * but excluded from the sums. */
typedef struct {
    uint64_t n_finite;   /* elements that were SR-rounded (|y| <= M, zeros included) */
    uint64_t n_up;       /* of those, how many rounded up in magnitude */
    uint64_t n_nan;
    uint64_t n_inf;
    uint64_t n_sat;      /* finite |y| > M */
    double sum_e;        /* sum of e */
    double sum_e2;       /* sum of e^2 */
    double sum_signed_e; /* sum of sign(y) e: error of the signed value */
    double sum_abs_e;    /* sum of |e| */
} fbsr_stats;

/* ---------------------------------------------------------------------------
 * fbsr_round -- Section II-A/II-B/III-F: dst[i] = FBSR(fl32(src[i] * scale)).
 *   src      device, n binary32 values (read only; must not overlap dst)
 *   dst      device, n codes: uint16 for bf16/fp16, uint8 for e4m3/e5m2/b8p4
 *   fmt, variant, k_bits   fbsr_fmt, fbsr_variant, N in 1..16
 *   seed, offset           Philox key and global index of element 0
 *   scale    finite, > 0; the per-tensor factor of a scaled tensor (Section I-A),
 *            applied as one rounded binary32 multiply
 * ------------------------------------------------------------------------- */
int fbsr_round(const float* src, void* dst, size_t n, int fmt, int variant, int k_bits,
               uint64_t seed, uint64_t offset, float scale, void* cuda_stream);

/* fbsr_round_lp -- the paper's own regime (Section III-E, Fig. 2, the rounding to 8 bits that ends Algorithm 1):
 * the source is already a low-precision tensor.  dst[i] = FBSR(fl32(value(src[i]) * scale)), where
 * value() widens the stored code exactly by Eq. (1).
 *   src      device, n codes of src_fmt (FBSR_BF16 or FBSR_FP16, uint16 each); must not overlap dst
 *   dst      device, n codes of dst_fmt (FBSR_E4M3, FBSR_E5M2 or FBSR_B8P4, uint8 each)
 * Other format pairs return FBSR_ERR_UNSUPPORTED.  The fast path needs src 32-byte aligned, dst 16-byte
 * aligned (a lane reads 16 source codes and writes 16 target codes at a time) and `offset` on the tile grid;
 * other calls are served by the general kernel with identical results.  A NaN source keeps its sign. */
int fbsr_round_lp(const void* src, int src_fmt, void* dst, size_t n, int dst_fmt, int variant, int k_bits,
                  uint64_t seed, uint64_t offset, float scale, void* cuda_stream);

/* fbsr_round_desc -- fbsr_round for a format (K, P, B; M) given at run time, Section II's parametrisation
 * (width, precision, exponent bias and largest finite value); the rounding itself is Section II-A
 * Eq. (2)-(5) with the predicates of Section II-B and Eq. (8), as in fbsr_round.
 *   desc     HOST pointer, read before the call returns:
 *     K          8 or 16: width of a code (dst is uint8 or uint16)
 *     P          precision including the hidden bit, 2 <= P <= min(K - 1, 13)
 *     B          exponent bias, 1 <= B <= 127
 *     max_code   magnitude code of M, the largest finite value (exponent field of M minus B at most 127)
 *     has_inf / inf_code   whether an infinity exists, and its magnitude code (> max_code)
 *     nan_code   magnitude code written for NaN (> max_code, != inf_code); with single_zero the pattern
 *                1 << (K - 1) instead
 *     single_zero  non-zero: one zero and one unsigned NaN (the pattern that would be minus zero), as in
 *                Binary8P4; a zero result then has no sign
 *   ovf_ieee non-zero: finite |y| > M are rounded as IEEE nearest-even does (see FBSR_OVF_IEEE)
 * Special values follow the conventions at the top of this file (Inf -> the infinity, or +-M without one).
 * Whole tiles of the draw stream (src 32-byte aligned and dst 8 x code-size aligned at the first tile boundary) are
 * served by a tiled kernel at roughly half the speed of the built-in formats' kernels; the head, the ragged end and
 * unaligned calls by a general kernel (any alignment, any offset) that is several times slower.
 * The built-in formats written as descriptors give the built-in results bit for bit.
 * Returns FBSR_ERR_INVALID_ARG for a descriptor outside the ranges above. */
typedef struct {
    int32_t K, P, B;
    uint32_t max_code;
    int32_t has_inf;
    uint32_t inf_code, nan_code;
    int32_t single_zero;
} fbsr_format_desc;

int fbsr_round_desc(const float* src, void* dst, size_t n, const fbsr_format_desc* desc, int ovf_ieee,
                    int variant, int k_bits, uint64_t seed, uint64_t offset, float scale, void* cuda_stream);

/* 1 if fbsr_round_desc accepts the descriptor, else 0.  Host only, no CUDA call. */
int fbsr_format_desc_valid(const fbsr_format_desc* desc);

/* fbsr_round_mx -- block-scaled tensors (Section I-A: each block of low-precision values carries a scale
 * factor of its own, here a power of two).  Blocks are 32 consecutive elements of the call; per block
 *     amax  = largest finite |src| (0 if none)
 *     e_blk = clamp(floor(log2 amax) - emax, -127, 127), emax = floor(log2 M);  -127 if amax < 2^-126
 *     scales[block] = e_blk + 127;   dst[i] = FBSR(fl32(src[i] * 2^-e_blk))
 * so the block maximum lands in the format's top binade (values between M and 2^(emax+1) saturate).
 *   scales   device, ceil(n / 32) bytes, overwritten
 * Draws are indexed by offset + i as everywhere else.  The fast path additionally needs the first tile
 * boundary of the call to fall on a block boundary (true for offset = 0 or any multiple of the tile size). */
int fbsr_round_mx(const float* src, void* dst, uint8_t* scales, size_t n, int fmt, int variant, int k_bits,
                  uint64_t seed, uint64_t offset, void* cuda_stream);

/* fbsr_round_bits -- the same rounding with caller-supplied random bits
 * (Section II-B treats the randomness as a finite string of bits handed to the
 * rounder).  rand_words: device, ceil(n / dpw) words; element i uses field
 * (i mod dpw) of word (i / dpw), low bits first; higher bits are ignored. */
int fbsr_round_bits(const float* src, void* dst, size_t n, int fmt, int variant, int k_bits,
                    const uint32_t* rand_words, float scale, void* cuda_stream);

/* fbsr_round_stats -- fbsr_round plus the error statistics of Section III
 * (bias = mean of e) accumulated in binary64.
 *   group_size       0, or the length of the consecutive groups of this call's
 *                    elements (group j = elements [j group_size, (j+1) group_size))
 *   group_sum_e/_e2  device, ceil(n / group_size) doubles each, overwritten with
 *                    the per-group sums of e and e^2; may be NULL when group_size = 0.
 *                    Group sums are added with atomics: their last bits may vary
 *                    from run to run.
 *   total            device, one fbsr_stats, overwritten.  Totals are reduced in a
 *                    fixed order and are reproducible bit for bit.
 *   workspace        device scratch of at least fbsr_stats_workspace_bytes() bytes,
 *                    8-byte aligned; contents on entry are ignored. */
size_t fbsr_stats_workspace_bytes(void);
int fbsr_round_stats(const float* src, void* dst, size_t n, int fmt, int variant, int k_bits,
                     uint64_t seed, uint64_t offset, float scale, size_t group_size,
                     double* group_sum_e, double* group_sum_e2, fbsr_stats* total,
                     void* workspace, size_t workspace_bytes, void* cuda_stream);

/* fbsr_round_stats_noalloc -- fbsr_round_stats without a workspace argument.
 * (The paper has no counterpart; this exists for the sake of callers, see below.)
 *
 * Who it is for: code that may not allocate device memory at the point where it
 * wants rounding statistics -- a step that runs inside a memory pool whose size was
 * fixed at start-up, a plugin inside someone else's process that must not touch
 * the allocator, a monitoring hook on a device that is already full.  Such a
 * caller cannot provide the scratch that fbsr_round_stats needs for its per-CTA
 * partial sums, so this variant keeps that scratch inside the library: a
 * file-scope device array of FBSR_NOALLOC_SCRATCH_BYTES (85,248 bytes), which
 * every GPU that loads libfbsr.so holds until the process exits.  The call itself
 * performs no cudaMalloc / cudaFree and calls no allocating routine.
 *
 * Arguments and results are those of fbsr_round_stats (same kernels, same fixed
 * reduction order, so totals are bit-identical to it); src, dst, the group arrays
 * and `total` are still the caller's.
 *   - n must not exceed FBSR_NOALLOC_MAX_ELEMENTS (2^31); larger calls return
 *     FBSR_ERR_TOO_LARGE and do nothing.  The limit bounds how long one call can
 *     occupy the shared scratch.
 *   - The first call on each device looks up the device address of the scratch
 *     array (cudaGetSymbolAddress) with that device current; make that first
 *     call outside any stream capture.  The address is remembered per device
 *     ordinal for the life of the process and does not survive a
 *     cudaDeviceReset: do not call this entry point again after one.
 *   - All calls on a device share the one array.  It keeps whatever the previous
 *     call left there; nothing in it has to start at zero, because every slot a
 *     call reads is first written by that same call.  Two calls that can overlap
 *     on the GPU (different streams without an ordering between them) race on
 *     it and give undefined statistics: order them, or use fbsr_round_stats with
 *     separate workspaces. */
#define FBSR_NOALLOC_SCRATCH_BYTES 85248u
#define FBSR_NOALLOC_MAX_ELEMENTS ((size_t)1 << 31)
int fbsr_round_stats_noalloc(const float* src, void* dst, size_t n, int fmt, int variant, int k_bits,
                             uint64_t seed, uint64_t offset, float scale, size_t group_size,
                             double* group_sum_e, double* group_sum_e2, fbsr_stats* total,
                             void* cuda_stream);

/* fbsr_sgd_update -- last line of Algorithm 1 with a binary32 master copy:
 *     m' = fma(mu, m, g);  w' = fma(-lr, m', w);  dst = FBSR(w')
 * master_w and momentum are updated in place; grad is read only.  Every
 * operation is one correctly rounded binary32 operation (no flush to zero). */
int fbsr_sgd_update(float* master_w, const float* grad, float* momentum, void* dst_lp, size_t n,
                    int fmt, int variant, int k_bits, uint64_t seed, uint64_t offset,
                    float lr, float mu, void* cuda_stream);

/* fbsr_adam_update -- same, with Adam (no weight decay).  Host scalars, in
 * binary64 then rounded to binary32: b1t = beta1^step and b2t = beta2^step by
 * repeated multiplication, c1 = lr / (1 - b1t), c2 = 1 / sqrt(1 - b2t),
 * a1 = 1 - beta1, a2 = 1 - beta2.  Per element, binary32:
 *     m' = fma(beta1, m, a1 g);  v' = fma(beta2, v, (a2 g) g);
 *     d  = sqrt(v') c2 + eps;    w' = fma(-c1, m' / d, w);  dst = FBSR(w')
 * step >= 1 is the 1-based step count. */
int fbsr_adam_update(float* master_w, const float* grad, float* m, float* v, void* dst_lp, size_t n,
                     int fmt, int variant, int k_bits, uint64_t seed, uint64_t offset,
                     float lr, float beta1, float beta2, float eps, int step, void* cuda_stream);

/* The four host scalars of fbsr_adam_update and fbsr_qat_adamw_step for a given step (Algorithm 1 leaves the
 * arithmetic of its AdamW update open; this is the library's definition, stated with fbsr_adam_update):
 * out = {c1, c2, a1, a2}.  beta^step is formed by repeated multiplication in binary64; the multiplication stops
 * once the product of a |beta| < 1 has fallen below 2^-54, from where on 1 - beta^step is exactly 1, so the cost
 * on the host does not grow with the step count.  Host only, no CUDA call; out must hold 4 floats. */
void fbsr_adam_scalars(float lr, float beta1, float beta2, int step, float out[4]);

/* fbsr_accumulate -- the last step of Algorithm 1 (weight plus update, rounded to the narrow format) with the sum
 * formed in binary32:  w_lp[i] = FBSR(fl32(value(w_lp[i]) + update[i])), in place.
 * A NaN sum is written as the positive quiet NaN. */
int fbsr_accumulate(void* w_lp, const float* update, size_t n, int fmt, int variant, int k_bits,
                    uint64_t seed, uint64_t offset, void* cuda_stream);

/* fbsr_qat_adamw_step -- Algorithm 1, one whole iteration from the gradient on, fused:
 *     w16 = value(w8);  g = value(grad16);
 *     the algorithm's 16-bit AdamW update: moments in binary32, each operation rounded once, the result rounded to the 16-bit format
 *         m' = fma(beta1, m, a1 g);  v' = fma(beta2, v, (a2 g) g);  d = sqrt(v') c2 + eps;
 *         u32 = fma(-c1, m' / d, -(lr weight_decay) w16);   u16 = RTNE_16(u32)      (c1, c2, a1, a2 as in fbsr_adam_update)
 *     w8 = FBSR(RTNE_16(fl32(w16 + u16)))                                            (as in fbsr_qat_update; SR applied here)
 *   w8       device, n codes of w_fmt (FBSR_E4M3, FBSR_E5M2 or FBSR_B8P4), read and overwritten
 *   grad16   device, n codes of g_fmt (FBSR_BF16 or FBSR_FP16), the algorithm's 16-bit format
 *   m, v     device, n binary32 moments each, read and overwritten
 * 20 bytes per parameter.  The paper states the shape of the step, not its arithmetic: the operation list is this
 * library's.  A NaN result is written as the positive NaN code; m and v then hold NaNs of unspecified sign. */
int fbsr_qat_adamw_step(void* w8, const void* grad16, float* m, float* v, size_t n, int w_fmt, int g_fmt, int variant,
                        int k_bits, uint64_t seed, uint64_t offset, float lr, float beta1, float beta2, float eps,
                        float weight_decay, int step, void* cuda_stream);

/* fbsr_qat_update -- Algorithm 1, last line, with the sum formed in the 16-bit format as written there:
 *     w16 = value(w8);  s = RTNE_16(fl32(w16 + u16));  w8 = FBSR(s)          (in place on w8)
 *   w8       device, n codes of w_fmt (FBSR_E4M3, FBSR_E5M2 or FBSR_B8P4), read and overwritten
 *   update16 device, n codes of u_fmt (FBSR_BF16 or FBSR_FP16): the update computed in the 16-bit format
 * RTNE_16 rounds to u_fmt with ties to even (saturating); a NaN sum is written as the positive NaN. */
int fbsr_qat_update(void* w8, const void* update16, size_t n, int w_fmt, int u_fmt, int variant, int k_bits,
                    uint64_t seed, uint64_t offset, void* cuda_stream);

/* fbsr_round_host -- fbsr_round for HOST buffers (pinned memory gives overlap):
 * copies src to the device in chunks, rounds, copies the codes back, using
 * dev_workspace (device, >= fbsr_round_host_min_workspace() bytes, 256-byte
 * aligned) as a double buffer.  Kernels are enqueued on cuda_stream, the copies
 * on two internal streams (one per direction, so that the upload of a chunk, the
 * rounding of the previous one and the download of the one before overlap); the
 * uploads wait for what cuda_stream held at the time of the call, and everything
 * is joined back into cuda_stream before return: dst_host is valid once
 * cuda_stream has been synchronised.  Callers on different streams may call
 * concurrently with workspaces of their own. */
size_t fbsr_round_host_min_workspace(void);
int fbsr_round_host(const float* src_host, void* dst_host, size_t n, int fmt, int variant, int k_bits,
                    uint64_t seed, uint64_t offset, float scale, void* dev_workspace,
                    size_t workspace_bytes, void* cuda_stream);

/* A common multiple of the warp-tile sizes the entry points use for k_bits: `offset` values that are
 * multiples of it keep a sharded call on the fast path.  0 if k_bits is invalid. */
size_t fbsr_tile_elements(int k_bits);

/* Number of kernel launches the library has enqueued since it was loaded. */
uint64_t fbsr_launch_count(void);

const char* fbsr_status_string(int status);
int fbsr_version(void);

#ifdef __cplusplus
}
#endif
#endif /* FBSR_H */
