// C-ABI entry points of libfbsr.so: argument validation, host-side scalars, dispatch by format,
// and the chunked host-buffer pipeline.  See include/fbsr.h for the contract of each call.
#include <atomic>
#include <cmath>
#include <mutex>

#include "../../include/fbsr.h"
#include "fbsr_internal.h"

namespace fbsr {

static std::atomic<uint64_t> g_launches{0};
void count_launch() { g_launches.fetch_add(1, std::memory_order_relaxed); }

namespace {

typedef int (*dispatch_fn)(const CallArgs&);
const dispatch_fn kRound[5] = {dispatch_round_0, dispatch_round_1, dispatch_round_2, dispatch_round_3, dispatch_round_4};
const dispatch_fn kRoundWords[5] = {dispatch_round_words_0, dispatch_round_words_1, dispatch_round_words_2, dispatch_round_words_3, dispatch_round_words_4};
const dispatch_fn kStats[5] = {dispatch_stats_0, dispatch_stats_1, dispatch_stats_2, dispatch_stats_3, dispatch_stats_4};
const dispatch_fn kOptim[5] = {dispatch_optim_0, dispatch_optim_1, dispatch_optim_2, dispatch_optim_3, dispatch_optim_4};
inline bool eight_bit(int fmt) { return fmt == FBSR_E4M3 || fmt == FBSR_E5M2 || fmt == FBSR_B8P4; }
inline int dispatch_lp(int fmt, const CallArgs& a)
{
    if (a.op == OP_QAT) return fmt == FBSR_E4M3 ? dispatch_qat_2(a) : fmt == FBSR_E5M2 ? dispatch_qat_3(a) : dispatch_qat_4(a);
    return fmt == FBSR_E4M3 ? dispatch_lp_2(a) : fmt == FBSR_E5M2 ? dispatch_lp_3(a) : dispatch_lp_4(a);
}

inline bool bad_enum(int fmt, int variant, int k) { return fmt < 0 || fmt > 4 || variant < 0 || variant > 5 || k < 1 || k > 16; }
// FBSR_OVF_IEEE may be or-ed into a format argument: take it out and report it.
inline int take_overflow_flag(int& fmt)
{
    const int flag = (fmt & FBSR_OVF_IEEE) ? 1 : 0;
    fmt &= ~FBSR_OVF_IEEE;
    return flag;
}
inline size_t code_bytes(int fmt) { return fmt <= 1 ? 2 : 1; }
inline bool misaligned(const void* p, size_t a) { return (reinterpret_cast<uintptr_t>(p) % a) != 0; }

inline int finish(int rc)
{
    if (rc != 0) return FBSR_ERR_UNSUPPORTED;
    return cudaGetLastError() == cudaSuccess ? FBSR_OK : FBSR_ERR_CUDA;
}

CallArgs base_args(OpKind op, int variant, int k, size_t n, uint64_t seed, uint64_t offset, void* dst, void* stream)
{
    CallArgs a{};
    a.op = op; a.variant = variant; a.k = k; a.n = n; a.seed = seed; a.offset = offset;
    a.dst = dst; a.stream = static_cast<cudaStream_t>(stream); a.scale = 1.0f;
    return a;
}

// beta^step by repeated multiplication in binary64 (the definition shared with the oracle).  Once the running
// product of a |beta| < 1 is below 2^-54 it no longer matters: 1 - product rounds to exactly 1.0, so the loop
// stops there and a long run does not pay for its step count on the host.
double beta_power(float beta, int step)
{
    const double b = (double)beta;
    const bool shrinking = std::fabs(b) < 1.0;
    double p = 1.0;
    for (int t = 0; t < step; ++t) {
        p *= b;
        if (shrinking && std::fabs(p) < 0x1p-54) break;
    }
    return p;
}

// Host scalars of the Adam steps: out = {lr / (1 - beta1^step), 1 / sqrt(1 - beta2^step), 1 - beta1, 1 - beta2},
// each formed in binary64 and rounded once to binary32.
void adam_scalars(float lr, float beta1, float beta2, int step, float out[4])
{
    const double b1t = beta_power(beta1, step), b2t = beta_power(beta2, step);
    out[0] = (float)((double)lr / (1.0 - b1t));
    out[1] = (float)(1.0 / std::sqrt(1.0 - b2t));
    out[2] = (float)(1.0 - (double)beta1);
    out[3] = (float)(1.0 - (double)beta2);
}

int check_round(const float* src, const void* dst, size_t n, int fmt, int variant, int k, float scale)
{
    if (bad_enum(fmt, variant, k)) return FBSR_ERR_INVALID_ARG;
    if (!(scale > 0.0f) || !std::isfinite(scale)) return FBSR_ERR_INVALID_ARG;
    if (n > 0 && (src == nullptr || dst == nullptr)) return FBSR_ERR_INVALID_ARG;
    if (misaligned(src, 4) || misaligned(dst, code_bytes(fmt))) return FBSR_ERR_ALIGNMENT;
    return FBSR_OK;
}

}  // namespace
}  // namespace fbsr

using namespace fbsr;

extern "C" {

int fbsr_round(const float* src, void* dst, size_t n, int fmt, int variant, int k_bits, uint64_t seed,
               uint64_t offset, float scale, void* cuda_stream)
{
    const int ovf_ieee = take_overflow_flag(fmt);
    if (int rc = check_round(src, dst, n, fmt, variant, k_bits, scale)) return rc;
    if (n == 0) return FBSR_OK;
    CallArgs a = base_args(OP_ROUND, variant, k_bits, n, seed, offset, dst, cuda_stream);
    a.ovf_ieee = ovf_ieee;
    a.src = src; a.scale = scale;
    return finish(kRound[fmt](a));
}

int fbsr_round_lp(const void* src, int src_fmt, void* dst, size_t n, int dst_fmt, int variant, int k_bits,
                  uint64_t seed, uint64_t offset, float scale, void* cuda_stream)
{
    const int ovf_ieee = take_overflow_flag(dst_fmt);
    if (bad_enum(dst_fmt, variant, k_bits) || src_fmt < 0 || src_fmt > 4) return FBSR_ERR_INVALID_ARG;
    if (!(scale > 0.0f) || !std::isfinite(scale)) return FBSR_ERR_INVALID_ARG;
    if ((src_fmt != FBSR_BF16 && src_fmt != FBSR_FP16) || !eight_bit(dst_fmt))
        return FBSR_ERR_UNSUPPORTED;
    if (n > 0 && (src == nullptr || dst == nullptr)) return FBSR_ERR_INVALID_ARG;
    if (misaligned(src, 2)) return FBSR_ERR_ALIGNMENT;
    if (n == 0) return FBSR_OK;
    CallArgs a = base_args(OP_ROUND_LP, variant, k_bits, n, seed, offset, dst, cuda_stream);
    a.ovf_ieee = ovf_ieee;
    a.src_lp = src; a.src_fmt = src_fmt; a.scale = scale;
    return finish(dispatch_lp(dst_fmt, a));
}

int fbsr_round_mx(const float* src, void* dst, uint8_t* scales, size_t n, int fmt, int variant, int k_bits,
                  uint64_t seed, uint64_t offset, void* cuda_stream)
{
    const int ovf_ieee = take_overflow_flag(fmt);
    if (int rc = check_round(src, dst, n, fmt, variant, k_bits, 1.0f)) return rc;
    if (n > 0 && scales == nullptr) return FBSR_ERR_INVALID_ARG;
    if (n == 0) return FBSR_OK;
    CallArgs a = base_args(OP_ROUND_MX, variant, k_bits, n, seed, offset, dst, cuda_stream);
    a.ovf_ieee = ovf_ieee;
    a.src = src; a.scales = scales;
    return finish(kRoundWords[fmt](a));
}

int fbsr_round_bits(const float* src, void* dst, size_t n, int fmt, int variant, int k_bits,
                    const uint32_t* rand_words, float scale, void* cuda_stream)
{
    const int ovf_ieee = take_overflow_flag(fmt);
    if (int rc = check_round(src, dst, n, fmt, variant, k_bits, scale)) return rc;
    if (n > 0 && rand_words == nullptr) return FBSR_ERR_INVALID_ARG;
    if (misaligned(rand_words, 4)) return FBSR_ERR_ALIGNMENT;
    if (n == 0) return FBSR_OK;
    CallArgs a = base_args(OP_ROUND_BITS, variant, k_bits, n, 0, 0, dst, cuda_stream);
    a.ovf_ieee = ovf_ieee;
    a.src = src; a.scale = scale; a.words = rand_words;
    return finish(kRoundWords[fmt](a));
}

size_t fbsr_stats_workspace_bytes(void) { return (size_t)MAX_SLOW_GRID * sizeof(fbsr_stats); }

int fbsr_round_stats(const float* src, void* dst, size_t n, int fmt, int variant, int k_bits, uint64_t seed,
                     uint64_t offset, float scale, size_t group_size, double* group_sum_e, double* group_sum_e2,
                     fbsr_stats* total, void* workspace, size_t workspace_bytes, void* cuda_stream)
{
    const int ovf_ieee = take_overflow_flag(fmt);
    if (int rc = check_round(src, dst, n, fmt, variant, k_bits, scale)) return rc;
    if (total == nullptr) return FBSR_ERR_INVALID_ARG;
    if (group_size > 0 && n > 0 && (group_sum_e == nullptr || group_sum_e2 == nullptr)) return FBSR_ERR_INVALID_ARG;
    if (misaligned(total, 8) || misaligned(group_sum_e, 8) || misaligned(group_sum_e2, 8)) return FBSR_ERR_ALIGNMENT;
    if (workspace == nullptr || workspace_bytes < fbsr_stats_workspace_bytes()) return FBSR_ERR_WORKSPACE;
    if (misaligned(workspace, 8)) return FBSR_ERR_ALIGNMENT;
    CallArgs a = base_args(OP_ROUND_STATS, variant, k_bits, n, seed, offset, dst, cuda_stream);
    a.ovf_ieee = ovf_ieee;
    a.src = src; a.scale = scale; a.group_size = group_size;
    a.gsum_e = group_sum_e; a.gsum_e2 = group_sum_e2; a.total = total; a.partials = workspace;
    if (group_size > 0 && n > 0) {
        const size_t groups = (n + group_size - 1) / group_size;
        if (cudaMemsetAsync(group_sum_e, 0, groups * sizeof(double), a.stream) != cudaSuccess ||
            cudaMemsetAsync(group_sum_e2, 0, groups * sizeof(double), a.stream) != cudaSuccess)
            return FBSR_ERR_CUDA;
    }
    return finish(kStats[fmt](a));
}

}  // extern "C"

// Scratch of the no-allocation statistics entry point: one slot per CTA of the statistics kernels.
// In host code this name is only a handle for cudaGetSymbolAddress, never a device address.
static __device__ __align__(256) unsigned char g_noalloc_stats_scratch[FBSR_NOALLOC_SCRATCH_BYTES];
static_assert(FBSR_NOALLOC_SCRATCH_BYTES == MAX_SLOW_GRID * sizeof(fbsr_stats), "scratch must hold one partial per CTA");

// Device address of the scratch array on the current device, looked up once per device.
static int noalloc_scratch_address(void** out)
{
    static void* addr[64] = {nullptr};
    static std::mutex mu;
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return FBSR_ERR_CUDA;
    std::lock_guard<std::mutex> lock(mu);
    if (addr[dev] == nullptr) {
        void* p = nullptr;
        if (cudaGetSymbolAddress(&p, g_noalloc_stats_scratch) != cudaSuccess || p == nullptr) {
            cudaGetLastError();
            return FBSR_ERR_CUDA;
        }
        addr[dev] = p;
    }
    *out = addr[dev];
    return FBSR_OK;
}

extern "C" {

int fbsr_round_stats_noalloc(const float* src, void* dst, size_t n, int fmt, int variant, int k_bits, uint64_t seed,
                             uint64_t offset, float scale, size_t group_size, double* group_sum_e,
                             double* group_sum_e2, fbsr_stats* total, void* cuda_stream)
{
    if (n > FBSR_NOALLOC_MAX_ELEMENTS) return FBSR_ERR_TOO_LARGE;
    void* scratch = nullptr;
    if (int rc = noalloc_scratch_address(&scratch)) return rc;
    // Every partial slot that the final reduction reads is written by this call's own CTAs first,
    // so the array needs no clearing between calls.
    return fbsr_round_stats(src, dst, n, fmt, variant, k_bits, seed, offset, scale, group_size, group_sum_e,
                            group_sum_e2, total, scratch, FBSR_NOALLOC_SCRATCH_BYTES, cuda_stream);
}

int fbsr_sgd_update(float* master_w, const float* grad, float* momentum, void* dst_lp, size_t n, int fmt,
                    int variant, int k_bits, uint64_t seed, uint64_t offset, float lr, float mu, void* cuda_stream)
{
    const int ovf_ieee = take_overflow_flag(fmt);
    if (bad_enum(fmt, variant, k_bits)) return FBSR_ERR_INVALID_ARG;
    if (n > 0 && (!master_w || !grad || !momentum || !dst_lp)) return FBSR_ERR_INVALID_ARG;
    if (misaligned(master_w, 4) || misaligned(grad, 4) || misaligned(momentum, 4) ||
        misaligned(dst_lp, code_bytes(fmt))) return FBSR_ERR_ALIGNMENT;
    if (n == 0) return FBSR_OK;
    CallArgs a = base_args(OP_SGD, variant, k_bits, n, seed, offset, dst_lp, cuda_stream);
    a.ovf_ieee = ovf_ieee;
    a.w = master_w; a.g = grad; a.m = momentum; a.neg_lr = -lr; a.mu = mu;
    return finish(kOptim[fmt](a));
}

int fbsr_adam_update(float* master_w, const float* grad, float* m, float* v, void* dst_lp, size_t n, int fmt,
                     int variant, int k_bits, uint64_t seed, uint64_t offset, float lr, float beta1, float beta2,
                     float eps, int step, void* cuda_stream)
{
    const int ovf_ieee = take_overflow_flag(fmt);
    if (bad_enum(fmt, variant, k_bits) || step < 1) return FBSR_ERR_INVALID_ARG;
    if (n > 0 && (!master_w || !grad || !m || !v || !dst_lp)) return FBSR_ERR_INVALID_ARG;
    if (misaligned(master_w, 4) || misaligned(grad, 4) || misaligned(m, 4) || misaligned(v, 4) ||
        misaligned(dst_lp, code_bytes(fmt))) return FBSR_ERR_ALIGNMENT;
    if (n == 0) return FBSR_OK;
    float sc[4];
    adam_scalars(lr, beta1, beta2, step, sc);
    CallArgs a = base_args(OP_ADAM, variant, k_bits, n, seed, offset, dst_lp, cuda_stream);
    a.ovf_ieee = ovf_ieee;
    a.w = master_w; a.g = grad; a.m = m; a.v = v;
    a.beta1 = beta1; a.beta2 = beta2; a.eps = eps;
    a.neg_c1 = -sc[0]; a.c2 = sc[1]; a.a1 = sc[2]; a.a2 = sc[3];
    return finish(kOptim[fmt](a));
}

int fbsr_accumulate(void* w_lp, const float* update, size_t n, int fmt, int variant, int k_bits, uint64_t seed,
                    uint64_t offset, void* cuda_stream)
{
    const int ovf_ieee = take_overflow_flag(fmt);
    if (bad_enum(fmt, variant, k_bits)) return FBSR_ERR_INVALID_ARG;
    if (n > 0 && (!w_lp || !update)) return FBSR_ERR_INVALID_ARG;
    if (misaligned(update, 4) || misaligned(w_lp, code_bytes(fmt))) return FBSR_ERR_ALIGNMENT;
    if (n == 0) return FBSR_OK;
    CallArgs a = base_args(OP_ACCUM, variant, k_bits, n, seed, offset, w_lp, cuda_stream);
    a.ovf_ieee = ovf_ieee;
    a.src = update;
    return finish(kOptim[fmt](a));
}

int fbsr_qat_update(void* w8, const void* update16, size_t n, int w_fmt, int u_fmt, int variant, int k_bits,
                    uint64_t seed, uint64_t offset, void* cuda_stream)
{
    const int ovf_ieee = take_overflow_flag(w_fmt);
    if (bad_enum(w_fmt, variant, k_bits) || u_fmt < 0 || u_fmt > 4) return FBSR_ERR_INVALID_ARG;
    if (!eight_bit(w_fmt) || (u_fmt != FBSR_BF16 && u_fmt != FBSR_FP16)) return FBSR_ERR_UNSUPPORTED;
    if (n > 0 && (!w8 || !update16)) return FBSR_ERR_INVALID_ARG;
    if (misaligned(update16, 2)) return FBSR_ERR_ALIGNMENT;
    if (n == 0) return FBSR_OK;
    CallArgs a = base_args(OP_QAT, variant, k_bits, n, seed, offset, w8, cuda_stream);
    a.ovf_ieee = ovf_ieee;
    a.src_lp = update16; a.src_fmt = u_fmt;
    return finish(dispatch_lp(w_fmt, a));
}

int fbsr_qat_adamw_step(void* w8, const void* grad16, float* m, float* v, size_t n, int w_fmt, int g_fmt, int variant,
                        int k_bits, uint64_t seed, uint64_t offset, float lr, float beta1, float beta2, float eps,
                        float weight_decay, int step, void* cuda_stream)
{
    const int ovf_ieee = take_overflow_flag(w_fmt);
    if (bad_enum(w_fmt, variant, k_bits) || g_fmt < 0 || g_fmt > 4 || step < 1) return FBSR_ERR_INVALID_ARG;
    if (!eight_bit(w_fmt) || (g_fmt != FBSR_BF16 && g_fmt != FBSR_FP16)) return FBSR_ERR_UNSUPPORTED;
    if (n > 0 && (!w8 || !grad16 || !m || !v)) return FBSR_ERR_INVALID_ARG;
    if (misaligned(grad16, 2) || misaligned(m, 4) || misaligned(v, 4)) return FBSR_ERR_ALIGNMENT;
    if (n == 0) return FBSR_OK;
    float sc[4];
    adam_scalars(lr, beta1, beta2, step, sc);
    CallArgs a = base_args(OP_QAT_ADAMW, variant, k_bits, n, seed, offset, w8, cuda_stream);
    a.ovf_ieee = ovf_ieee;
    a.src_lp = grad16; a.src_fmt = g_fmt; a.m = m; a.v = v;
    a.beta1 = beta1; a.beta2 = beta2; a.eps = eps;
    a.neg_c1 = -sc[0]; a.c2 = sc[1]; a.a1 = sc[2]; a.a2 = sc[3];
    const volatile float lrwd = lr * weight_decay;           // one rounded binary32 product
    a.neg_lrwd = -lrwd;
    return finish(w_fmt == FBSR_E4M3 ? dispatch_qat_adamw_2(a) : w_fmt == FBSR_E5M2 ? dispatch_qat_adamw_3(a)
                                                                                   : dispatch_qat_adamw_4(a));
}

void fbsr_adam_scalars(float lr, float beta1, float beta2, int step, float out[4])
{
    if (out == nullptr) return;
    adam_scalars(lr, beta1, beta2, step < 1 ? 1 : step, out);
}

size_t fbsr_tile_elements(int k_bits)
{
    if (k_bits < 1 || k_bits > 16) return 0;
    const int dpw = 32 / k_bits;
    if ((dpw & (dpw - 1)) == 0) return 1024;                 // power-of-two draws per word: 4 rows
    const int r0 = (dpw % 2 == 0) ? dpw / 2 : dpw;           // rows that hold whole generator calls
    return (size_t)(r0 % 2 == 0 ? r0 : 2 * r0) * 256;        // an even number of them
}

size_t fbsr_round_host_min_workspace(void) { return (size_t)1 << 20; }

int fbsr_round_host(const float* src_host, void* dst_host, size_t n, int fmt, int variant, int k_bits,
                    uint64_t seed, uint64_t offset, float scale, void* dev_workspace, size_t workspace_bytes,
                    void* cuda_stream)
{
    const int ovf_ieee = take_overflow_flag(fmt);
    if (int rc = check_round(src_host, dst_host, n, fmt, variant, k_bits, scale)) return rc;
    if (dev_workspace == nullptr || workspace_bytes < fbsr_round_host_min_workspace()) return FBSR_ERR_WORKSPACE;
    if (misaligned(dev_workspace, 256)) return FBSR_ERR_ALIGNMENT;
    if (n == 0) return FBSR_OK;

    // Per-device copy streams (one per direction), created on first use and kept for the life of the process;
    // the lock covers only that creation.  The events are made per call, so concurrent callers on different
    // streams share nothing but the two copy streams, in which their copies simply queue.
    struct Side { cudaStream_t h2d = nullptr, d2h = nullptr; bool ok = false; };
    static Side sides[64];
    static std::mutex mu;
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return FBSR_ERR_CUDA;
    Side s;
    {
        std::lock_guard<std::mutex> lock(mu);
        Side& shared = sides[dev];
        if (!shared.ok) {
            if (cudaStreamCreateWithFlags(&shared.h2d, cudaStreamNonBlocking) != cudaSuccess ||
                cudaStreamCreateWithFlags(&shared.d2h, cudaStreamNonBlocking) != cudaSuccess) return FBSR_ERR_CUDA;
            shared.ok = true;
        }
        s = shared;
    }
    // uploaded / rounded / drained per slot, and the fork point of the caller's stream
    struct Events {
        cudaEvent_t e[7] = {nullptr, nullptr, nullptr, nullptr, nullptr, nullptr, nullptr};
        bool create() { for (auto& x : e) if (cudaEventCreateWithFlags(&x, cudaEventDisableTiming) != cudaSuccess) return false; return true; }
        ~Events() { for (auto x : e) if (x) cudaEventDestroy(x); }      // released by the runtime once the work has run
    } ev;
    if (!ev.create()) return FBSR_ERR_CUDA;
    cudaEvent_t* uploaded = ev.e; cudaEvent_t* rounded = ev.e + 2; cudaEvent_t* drained = ev.e + 4; cudaEvent_t start = ev.e[6];

    const cudaStream_t main = static_cast<cudaStream_t>(cuda_stream);
    const size_t cb = code_bytes(fmt);
    const size_t tile = fbsr_tile_elements(k_bits);
    // Two slots, each: chunk binary32 inputs then chunk codes, both 256-byte aligned.
    size_t chunk = (workspace_bytes / 2 - 512) / (4 + cb);
    chunk = chunk / tile * tile;
    const size_t max_chunk = (size_t)1 << 26;               // keeps the first copy from delaying the first kernel
    if (chunk > max_chunk) chunk = max_chunk / tile * tile;
    if (chunk == 0) return FBSR_ERR_WORKSPACE;
    // The codes of the last chunk travel back with nothing left to overlap them, so a large call is cut into at
    // least 8 chunks (of at least 2^21 elements, where a copy is still long against its fixed costs).
    size_t target = (n + 7) / 8;
    if (target < ((size_t)1 << 21)) target = (size_t)1 << 21;
    target = (target + tile - 1) / tile * tile;
    if (chunk > target) chunk = target;
    // equal chunks (rounded up to whole tiles) instead of full chunks plus a sliver
    const size_t n_chunks = (n + chunk - 1) / chunk;
    chunk = ((n + n_chunks - 1) / n_chunks + tile - 1) / tile * tile;
    char* slot_in[2]; char* slot_out[2];
    const size_t in_bytes = (chunk * 4 + 255) / 256 * 256, out_bytes = (chunk * cb + 255) / 256 * 256;
    for (int i = 0; i < 2; ++i) {
        slot_in[i] = static_cast<char*>(dev_workspace) + i * (in_bytes + out_bytes);
        slot_out[i] = slot_in[i] + in_bytes;
    }
    if (2 * (in_bytes + out_bytes) > workspace_bytes) return FBSR_ERR_WORKSPACE;

    // the uploads start after whatever the caller's stream held at the time of the call
    if (cudaEventRecord(start, main) != cudaSuccess || cudaStreamWaitEvent(s.h2d, start, 0) != cudaSuccess) return FBSR_ERR_CUDA;
    bool used[2] = {false, false};
    size_t idx = 0;
    for (size_t at = 0; at < n; at += chunk, ++idx) {
        const int sl = (int)(idx & 1);
        const size_t len = n - at < chunk ? n - at : chunk;
        // chunk idx is uploaded on the upload stream while chunk idx - 1 is being rounded: the slot's previous
        // input must have been read (its kernel done) before the copy overwrites it
        if (used[sl] && cudaStreamWaitEvent(s.h2d, rounded[sl], 0) != cudaSuccess) return FBSR_ERR_CUDA;
        if (cudaMemcpyAsync(slot_in[sl], src_host + at, len * 4, cudaMemcpyHostToDevice, s.h2d) != cudaSuccess) return FBSR_ERR_CUDA;
        if (cudaEventRecord(uploaded[sl], s.h2d) != cudaSuccess) return FBSR_ERR_CUDA;
        if (cudaStreamWaitEvent(main, uploaded[sl], 0) != cudaSuccess) return FBSR_ERR_CUDA;
        // the slot's previous codes must have left before the kernel writes new ones
        if (used[sl] && cudaStreamWaitEvent(main, drained[sl], 0) != cudaSuccess) return FBSR_ERR_CUDA;
        CallArgs a = base_args(OP_ROUND, variant, k_bits, len, seed, offset + at, slot_out[sl], main);
        a.ovf_ieee = ovf_ieee;
        a.src = reinterpret_cast<const float*>(slot_in[sl]); a.scale = scale;
        if (kRound[fmt](a) != 0) return FBSR_ERR_UNSUPPORTED;
        if (cudaEventRecord(rounded[sl], main) != cudaSuccess) return FBSR_ERR_CUDA;
        if (cudaStreamWaitEvent(s.d2h, rounded[sl], 0) != cudaSuccess) return FBSR_ERR_CUDA;
        if (cudaMemcpyAsync(static_cast<char*>(dst_host) + at * cb, slot_out[sl], len * cb, cudaMemcpyDeviceToHost, s.d2h) != cudaSuccess) return FBSR_ERR_CUDA;
        if (cudaEventRecord(drained[sl], s.d2h) != cudaSuccess) return FBSR_ERR_CUDA;
        used[sl] = true;
    }
    // join: the caller's stream finishes only after every code has reached the host
    for (int sl = 0; sl < 2; ++sl)
        if (used[sl] && cudaStreamWaitEvent(main, drained[sl], 0) != cudaSuccess) return FBSR_ERR_CUDA;
    return cudaGetLastError() == cudaSuccess ? FBSR_OK : FBSR_ERR_CUDA;
}

uint64_t fbsr_launch_count(void) { return g_launches.load(std::memory_order_relaxed); }

const char* fbsr_status_string(int status)
{
    switch (status) {
    case FBSR_OK: return "ok";
    case FBSR_ERR_INVALID_ARG: return "invalid argument";
    case FBSR_ERR_UNSUPPORTED: return "unsupported combination";
    case FBSR_ERR_ALIGNMENT: return "pointer not aligned to its element size";
    case FBSR_ERR_CUDA: return "CUDA runtime error";
    case FBSR_ERR_WORKSPACE: return "workspace missing or too small";
    case FBSR_ERR_TOO_LARGE: return "n exceeds the limit of this entry point's built-in scratch";
    default: return "unknown status";
    }
}

int fbsr_version(void) { return 100; }

}  // extern "C"
