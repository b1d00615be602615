// Kernel instantiations and launch logic for one target format and one group of
// operations.  Compiled once per (FBSR_FMT, FBSR_GROUP): FBSR_GROUP 0 = fbsr_round, 4 = supplied bits and block
// scales, 5 = rounding with statistics (three units so that they compile in parallel), 1 = fused optimizer and
// accumulation, 2 = 16-bit sources, 6 = the 16-bit-sum update, 3 = the fused Algorithm-1 step (2, 3, 6: 8-bit targets only).
#include <array>
#include <cmath>
#include <utility>

#include "fbsr_internal.h"
#include "fbsr_kernels.cuh"

#ifndef FBSR_FMT
#error "compile with -DFBSR_FMT=0..4"
#endif
#ifndef FBSR_GROUP
#error "compile with -DFBSR_GROUP=0..6"
#endif

namespace fbsr {
namespace {

constexpr int FMT = FBSR_FMT;
constexpr int CODE_BYTES = Format<FMT>::K / 8;

inline bool aligned(const void* p, size_t a) { return (reinterpret_cast<uintptr_t>(p) % a) == 0; }

// Host view of an Op: which pointers the tiled kernel reads with 256-bit accesses, and
// the same Op with every pointer moved forward by h elements.
[[maybe_unused]] inline bool op_aligned(const RoundOp& o, size_t h) { return aligned(o.src + h, 32); }
[[maybe_unused]] inline RoundOp op_advance(RoundOp o, size_t h) { o.src += h; return o; }
[[maybe_unused]] inline bool op_aligned(const SgdOp& o, size_t h) { return aligned(o.w + h, 32) && aligned(o.g + h, 32) && aligned(o.m + h, 32); }
[[maybe_unused]] inline SgdOp op_advance(SgdOp o, size_t h) { o.w += h; o.g += h; o.m += h; return o; }
[[maybe_unused]] inline bool op_aligned(const AdamOp& o, size_t h)
{
    return aligned(o.w + h, 32) && aligned(o.g + h, 32) && aligned(o.m + h, 32) && aligned(o.v + h, 32);
}
[[maybe_unused]] inline AdamOp op_advance(AdamOp o, size_t h) { o.w += h; o.g += h; o.m += h; o.v += h; return o; }
[[maybe_unused]] inline bool op_aligned(const AccumOp<FMT>& o, size_t h) { return aligned(o.u + h, 32); }
[[maybe_unused]] inline AccumOp<FMT> op_advance(AccumOp<FMT> o, size_t h)
{
    o.u += h; o.w_lp = static_cast<const char*>(o.w_lp) + h * CODE_BYTES; return o;
}

[[maybe_unused]] inline bool op_aligned(const MxOp<FMT>& o, size_t h) { return aligned(o.src + h, 32) && h % 32 == 0; }
[[maybe_unused]] inline MxOp<FMT> op_advance(MxOp<FMT> o, size_t h) { o.src += h; o.scales += h / 32; o.n -= h; return o; }
constexpr int QAT_WF = CODE_BYTES == 1 ? FMT : E4M3;                    // the weight format of the Algorithm-1 step is 8 bits wide
template <int UF> inline bool op_aligned(const QatOp<QAT_WF, UF>& o, size_t h)
{
    return aligned(static_cast<const uint16_t*>(o.u16) + h, 32);      // w8 is checked as dst
}
template <int UF> inline QatOp<QAT_WF, UF> op_advance(QatOp<QAT_WF, UF> o, size_t h)
{
    o.w8 = static_cast<const uint8_t*>(o.w8) + h; o.u16 = static_cast<const uint16_t*>(o.u16) + h; return o;
}
template <int UF> inline bool op_aligned(const QatAdamOp<QAT_WF, UF>& o, size_t h)
{
    return aligned(static_cast<const uint16_t*>(o.g16) + h, 16) && aligned(o.m + h, 32) && aligned(o.v + h, 32);   // w8 is checked as dst
}
template <int UF> inline QatAdamOp<QAT_WF, UF> op_advance(QatAdamOp<QAT_WF, UF> o, size_t h)
{
    o.w8 = static_cast<const uint8_t*>(o.w8) + h; o.g16 = static_cast<const uint16_t*>(o.g16) + h; o.m += h; o.v += h; return o;
}
template <int SRC, bool P2> inline bool op_aligned(const LpSrcOp<SRC, P2>& o, size_t h)
{
    return aligned(static_cast<const uint16_t*>(o.src) + h, 32);
}
template <int SRC, bool P2> inline LpSrcOp<SRC, P2> op_advance(LpSrcOp<SRC, P2> o, size_t h)
{
    o.src = static_cast<const uint16_t*>(o.src) + h; return o;
}

struct Plan { size_t head, n_tiles, tail_begin; bool aligned; };

// Ops that also have the staged kernel, which takes pointers of any alignment (generated draws only).
template <class Op, bool BITS> struct HasStaged { static constexpr bool value = false; };
template <> struct HasStaged<RoundOp, false> { static constexpr bool value = true; };

template <class Op, int VAR, int K, bool BITS, bool IEEE = false>
int launch_tiles(const Op& op, const CallArgs& a, const Plan& p)
{
    using T = Tile<K, Op::OCTETS>;
    const uint32_t tail_count = (uint32_t)(a.n - p.tail_begin);          // < one tile; served by an extra CTA
    const Op adv = op_advance(op, p.head);
    void* dst = static_cast<char*>(a.dst) + p.head * CODE_BYTES;
    const uint64_t call0 = BITS ? 0 : (a.offset + p.head) / T::E;
    const uint32_t* words = BITS ? a.words + p.head / T::DPW : nullptr;
    if constexpr (HasStaged<Op, BITS>::value && !IEEE) {
        if (!p.aligned) {
            const uint64_t want = (p.n_tiles + STAGED_WARPS - 1) / STAGED_WARPS;
            const unsigned grid = (unsigned)(want < 0x7FFFFFF0ull ? want : 0x7FFFFFF0ull) + (tail_count ? 1u : 0u);
            staged_tile_kernel<FMT, VAR, K, BITS><<<grid, STAGED_THREADS, 0, a.stream>>>(
                adv, dst, p.n_tiles, call0, (uint32_t)a.seed, (uint32_t)(a.seed >> 32), words, tail_count);
            count_launch();
            return 0;
        }
    }
    auto kern = tile_kernel<Op, FMT, VAR, K, BITS, IEEE>;
    // One tile per warp, CTAs handed out by the hardware scheduler.  A persistent grid with a static
    // tile stride measured 5-10 % slower here: multiprocessors do not all see the same memory
    // bandwidth, and a static split makes the whole launch wait for the slowest of them.
    const uint64_t want = (p.n_tiles + WARPS_PER_CTA - 1) / WARPS_PER_CTA;
    const unsigned grid = (unsigned)(want < 0x7FFFFFF0ull ? want : 0x7FFFFFF0ull) + (tail_count ? 1u : 0u);
    kern<<<grid, CTA_THREADS, 0, a.stream>>>(adv, dst, p.n_tiles, call0, (uint32_t)a.seed,
                                             (uint32_t)(a.seed >> 32), words, tail_count);
    count_launch();
    return 0;
}

template <class Op, bool BITS, bool STATS>
int launch_generic(const Op& op, const CallArgs& a, size_t i_begin, size_t i_end, int* n_ctas_out)
{
    if (n_ctas_out) *n_ctas_out = 0;
    if (i_begin >= i_end) return 0;
    const uint64_t E = 4u * (32u / (unsigned)a.k);
    const uint64_t off = BITS ? 0 : a.offset;
    const uint64_t n_calls = (off + i_end - 1) / E - (off + i_begin) / E + 1;
    uint64_t ctas = (n_calls + CTA_THREADS - 1) / CTA_THREADS;
    if (ctas > (uint64_t)MAX_SLOW_GRID) ctas = MAX_SLOW_GRID;
    const uint64_t dpw = 32u / (unsigned)a.k;
    if constexpr (!STATS) {
        // a warp per 32 calls, coalesced accesses
        uint64_t warps = (n_calls + 31) / 32;
        ctas = (warps + WARPS_PER_CTA - 1) / WARPS_PER_CTA;
        if (ctas > (uint64_t)MAX_SLOW_GRID) ctas = MAX_SLOW_GRID;
        general_coalesced_kernel<Op, FMT, BITS><<<(unsigned)ctas, CTA_THREADS, 0, a.stream>>>(
            op, a.dst, i_begin, i_end, off, a.variant, a.k, (uint32_t)a.seed, (uint32_t)(a.seed >> 32), a.words,
            BITS ? (a.n + dpw - 1) / dpw : 0, (uint32_t)(0x100000000ull / dpw) + 1u, a.ovf_ieee);
        count_launch();
        if (n_ctas_out) *n_ctas_out = (int)ctas;
        return 0;
    }
    generic_kernel<Op, FMT, BITS, STATS><<<(unsigned)ctas, CTA_THREADS, 0, a.stream>>>(
        op, a.dst, i_begin, i_end, off, a.variant, a.k, (uint32_t)a.seed, (uint32_t)(a.seed >> 32),
        a.words, BITS ? (a.n + dpw - 1) / dpw : 0, STATS ? a.group_size : 0, a.gsum_e, a.gsum_e2,
        static_cast<StatsAcc*>(a.partials), a.ovf_ieee);
    count_launch();
    if (n_ctas_out) *n_ctas_out = (int)ctas;
    return 0;
}

// Split a call into [0, head) on the general kernel, whole tiles, and [tail_begin, n) (less than a tile).
template <class Op, int K, bool BITS>
Plan make_plan(const Op& op, const CallArgs& a)
{
    using T = Tile<K, Op::OCTETS>;
    Plan p{0, 0, 0, false};
    const uint64_t off = BITS ? 0 : a.offset;
    const size_t head = (size_t)((T::ELEMS - off % T::ELEMS) % T::ELEMS);
    const size_t dst_align = (CODE_BYTES == 2 ? 16 : 8) * Op::OCTETS;      // one vector store per lane-row
    p.aligned = op_aligned(op, head) && aligned(static_cast<char*>(a.dst) + head * CODE_BYTES, dst_align);
    if (head < a.n && (p.aligned || HasStaged<Op, BITS>::value)) {
        p.head = head;
        p.n_tiles = (a.n - head) / T::ELEMS;
    }
    if (p.n_tiles == 0) p.head = 0;
    p.tail_begin = p.head + p.n_tiles * T::ELEMS;
    return p;
}

// The IEEE reading of overflow (finite values beyond M) is a template variant of the tiled kernel for the ops
// listed here (plain rounding with generated draws, 16-bit sources); the other calls use the general kernel.
template <class Op, bool BITS> struct HasIeee { static constexpr bool value = false; };
template <> struct HasIeee<RoundOp, false> { static constexpr bool value = true; };
template <int SRC, bool P2> struct HasIeee<LpSrcOp<SRC, P2>, false> { static constexpr bool value = true; };

template <class Op, int VAR, int K, bool BITS>
int run(const Op& op, const CallArgs& a)
{
    Plan p = make_plan<Op, K, BITS>(op, a);
    constexpr bool ieee_tiles = HasIeee<Op, BITS>::value;
    if (a.ovf_ieee && !(ieee_tiles && p.aligned)) p.n_tiles = 0;
    if (p.n_tiles == 0) return launch_generic<Op, BITS, false>(op, a, 0, a.n, nullptr);
    launch_generic<Op, BITS, false>(op, a, 0, p.head, nullptr);
    if constexpr (ieee_tiles) {
        if (a.ovf_ieee) return launch_tiles<Op, VAR, K, BITS, true>(op, a, p);
    }
    return launch_tiles<Op, VAR, K, BITS>(op, a, p);          // whole tiles and the ragged end
}

// ---- (variant, k) -> instantiation
template <class Op, bool BITS> using RunFn = int (*)(const Op&, const CallArgs&);

template <class Op, bool BITS, int VAR, int... Ks>
constexpr std::array<RunFn<Op, BITS>, 16> row_of(std::integer_sequence<int, Ks...>)
{
    return {{&run<Op, VAR, Ks + 1, BITS>...}};
}

template <class Op, bool BITS>
int by_variant_and_k(const Op& op, const CallArgs& a)
{
    using Seq = std::make_integer_sequence<int, 16>;
    static constexpr std::array<RunFn<Op, BITS>, 16> table[3] = {
        row_of<Op, BITS, SRFF>(Seq{}), row_of<Op, BITS, SRF>(Seq{}), row_of<Op, BITS, SRC>(Seq{})};
    // the deterministic modes use no draws: one instantiation each, on the 1024-element tile of k = 16
    if (a.variant == RTNE) return run<Op, RTNE, 16, false>(op, a);
    if (a.variant == RTA) return run<Op, RTA, 16, false>(op, a);
    if (a.variant == RTO) return run<Op, RTO, 16, false>(op, a);
    return table[a.variant][a.k - 1](op, a);
}

}  // namespace

#define FBSR_CAT_(a, b) a##b
#define FBSR_CAT(a, b) FBSR_CAT_(a, b)

#if FBSR_GROUP == 5
namespace {
// Statistics: the head of the call (up to the first tile boundary of the draw stream) and the ragged end go to the
// general kernel, whole tiles to the tiled statistics kernel; every CTA leaves one partial in the workspace (tiles
// first, then head, then end) and stats_finalize_kernel adds them in that order.
constexpr int STATS_EDGE_SLOTS = 8;                                    // per edge; an edge is less than one tile
constexpr int STATS_TILE_GRID = MAX_SLOW_GRID - 2 * STATS_EDGE_SLOTS;  // CTAs (and partial slots) of the tiled kernel

template <int VAR, int K>
int run_stats(const CallArgs& a)
{
    const RoundOp op{a.src, a.scale};
    StatsAcc* slots = static_cast<StatsAcc*>(a.partials);
    int n_slots = 0;
    const Plan p = a.ovf_ieee ? Plan{0, 0, 0, false} : make_plan<RoundOp, K, false>(op, a);
    if (p.n_tiles > 0 && p.aligned) {
        using T = Tile<K, 1>;
        const uint64_t want = (p.n_tiles + WARPS_PER_CTA - 1) / WARPS_PER_CTA;
        const unsigned grid = (unsigned)(want < (uint64_t)STATS_TILE_GRID ? want : (uint64_t)STATS_TILE_GRID);
        auto kern = a.group_size ? stats_tile_kernel<FMT, VAR, K, true> : stats_tile_kernel<FMT, VAR, K, false>;
        kern<<<grid, CTA_THREADS, 0, a.stream>>>(
            a.src + p.head, a.scale, static_cast<char*>(a.dst) + p.head * CODE_BYTES, p.n_tiles, p.head,
            (a.offset + p.head) / T::E, (uint32_t)a.seed, (uint32_t)(a.seed >> 32), a.group_size, a.gsum_e, a.gsum_e2,
            slots);
        count_launch();
        n_slots = (int)grid;
        CallArgs edge = a;
        int used = 0;
        edge.partials = slots + n_slots;
        launch_generic<RoundOp, false, true>(op, edge, 0, p.head, &used);
        n_slots += used;
        edge.partials = slots + n_slots;
        launch_generic<RoundOp, false, true>(op, edge, p.tail_begin, a.n, &used);
        n_slots += used;
    } else {
        launch_generic<RoundOp, false, true>(op, a, 0, a.n, &n_slots);
    }
    stats_finalize_kernel<<<1, CTA_THREADS, 0, a.stream>>>(slots, n_slots, static_cast<StatsAcc*>(a.total));
    count_launch();
    return 0;
}

template <int VAR>
int stats_by_k(const CallArgs& a)
{
    switch (a.k) {
    case 1: return run_stats<VAR, 1>(a);
    case 2: return run_stats<VAR, 2>(a);
    case 3: return run_stats<VAR, 3>(a);
    case 4: return run_stats<VAR, 4>(a);
    case 5: return run_stats<VAR, 5>(a);
    case 6: return run_stats<VAR, 6>(a);
    case 7: return run_stats<VAR, 7>(a);
    case 8: return run_stats<VAR, 8>(a);
    case 9: return run_stats<VAR, 9>(a);
    case 10: return run_stats<VAR, 10>(a);
    case 11: return run_stats<VAR, 11>(a);
    case 12: return run_stats<VAR, 12>(a);
    case 13: return run_stats<VAR, 13>(a);
    case 14: return run_stats<VAR, 14>(a);
    case 15: return run_stats<VAR, 15>(a);
    case 16: return run_stats<VAR, 16>(a);
    default: return 1;
    }
}

int stats_by_variant_and_k(const CallArgs& a)
{
    if (a.variant == RTNE) return run_stats<RTNE, 16>(a);
    if (a.variant == RTA) return run_stats<RTA, 16>(a);
    if (a.variant == RTO) return run_stats<RTO, 16>(a);
    return a.variant == SRFF ? stats_by_k<SRFF>(a) : a.variant == SRF ? stats_by_k<SRF>(a) : stats_by_k<SRC>(a);
}
}  // namespace

int FBSR_CAT(dispatch_stats_, FBSR_FMT)(const CallArgs& a) { return stats_by_variant_and_k(a); }
#elif FBSR_GROUP == 0
int FBSR_CAT(dispatch_round_, FBSR_FMT)(const CallArgs& a)
{
    return by_variant_and_k<RoundOp, false>(RoundOp{a.src, a.scale}, a);
}
#elif FBSR_GROUP == 4
int FBSR_CAT(dispatch_round_words_, FBSR_FMT)(const CallArgs& a)
{
    switch (a.op) {
    case OP_ROUND_BITS: return by_variant_and_k<RoundOp, true>(RoundOp{a.src, a.scale}, a);
    case OP_ROUND_MX: return by_variant_and_k<MxOp<FMT>, false>(MxOp<FMT>{a.src, a.scales, a.n}, a);
    default: return 1;
    }
}
#elif FBSR_GROUP == 2
int FBSR_CAT(dispatch_lp_, FBSR_FMT)(const CallArgs& a)
{
    static_assert(CODE_BYTES == 1, "16-bit sources are rounded to 8-bit targets");
    // a power-of-two scale keeps the source's 8 or 11 significant bits: the kernels that round to nearest first
    // (SRC and the deterministic modes) then need no sticky bit; the other variants have no such code to drop
    int exponent = 0;
    const bool pow2 = std::frexp(a.scale, &exponent) == 0.5f && (a.variant == SRC || a.variant >= RTNE);
    if (a.src_fmt == BF16) {
        if (pow2) return by_variant_and_k<LpSrcOp<BF16, true>, false>(LpSrcOp<BF16, true>{a.src_lp, a.scale}, a);
        return by_variant_and_k<LpSrcOp<BF16>, false>(LpSrcOp<BF16>{a.src_lp, a.scale}, a);
    }
    if (a.src_fmt == FP16) {
        if (pow2) return by_variant_and_k<LpSrcOp<FP16, true>, false>(LpSrcOp<FP16, true>{a.src_lp, a.scale}, a);
        return by_variant_and_k<LpSrcOp<FP16>, false>(LpSrcOp<FP16>{a.src_lp, a.scale}, a);
    }
    return 1;
}
#elif FBSR_GROUP == 6
int FBSR_CAT(dispatch_qat_, FBSR_FMT)(const CallArgs& a)
{
    static_assert(CODE_BYTES == 1, "the weights of Algorithm 1 are 8 bits wide");
    if (a.src_fmt == BF16) return by_variant_and_k<QatOp<FMT, BF16>, false>(QatOp<FMT, BF16>{a.dst, a.src_lp}, a);
    if (a.src_fmt == FP16) return by_variant_and_k<QatOp<FMT, FP16>, false>(QatOp<FMT, FP16>{a.dst, a.src_lp}, a);
    return 1;
}
#elif FBSR_GROUP == 3
int FBSR_CAT(dispatch_qat_adamw_, FBSR_FMT)(const CallArgs& a)
{
    static_assert(CODE_BYTES == 1, "the weights of Algorithm 1 are 8 bits wide");
    if (a.src_fmt == BF16) {
        return by_variant_and_k<QatAdamOp<FMT, BF16>, false>(
            QatAdamOp<FMT, BF16>{a.dst, a.src_lp, a.m, a.v, a.beta1, a.beta2, a.eps, a.neg_c1, a.c2, a.a1, a.a2, a.neg_lrwd}, a);
    }
    if (a.src_fmt == FP16) {
        return by_variant_and_k<QatAdamOp<FMT, FP16>, false>(
            QatAdamOp<FMT, FP16>{a.dst, a.src_lp, a.m, a.v, a.beta1, a.beta2, a.eps, a.neg_c1, a.c2, a.a1, a.a2, a.neg_lrwd}, a);
    }
    return 1;
}
#else
int FBSR_CAT(dispatch_optim_, FBSR_FMT)(const CallArgs& a)
{
    switch (a.op) {
    case OP_SGD: return by_variant_and_k<SgdOp, false>(SgdOp{a.w, a.g, a.m, a.neg_lr, a.mu}, a);
    case OP_ADAM:
        return by_variant_and_k<AdamOp, false>(
            AdamOp{a.w, a.g, a.m, a.v, a.beta1, a.beta2, a.eps, a.neg_c1, a.c2, a.a1, a.a2}, a);
    case OP_ACCUM: return by_variant_and_k<AccumOp<FMT>, false>(AccumOp<FMT>{a.dst, a.src}, a);
    default: return 1;
    }
}
#endif

}  // namespace fbsr
