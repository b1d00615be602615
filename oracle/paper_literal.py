"""Paper-literal few-bit stochastic rounding in exact rational arithmetic.

TEST INFRASTRUCTURE ONLY.  This module is the slow, exact statement of what the
rounding path computes.  It is never imported by the CUDA library or its Python
binding; only tests, the smoke check and the CPU-baseline leg of the benchmark
may use it.

Every quantity that the paper treats as a real number (the significand, its
fractional part, the noise n * 2**-N) is a ``fractions.Fraction`` here, so the
predicates are evaluated exactly as printed:

* value function F(s, e, t; P, B)            -- Section II, Eq. (1)
* exponent with subnormals                   -- Section II-A, Eq. (2)
* scaled significand                         -- Section II-A, Eq. (3)
* sigma = floor(sigma~) + [R(delta~)]        -- Section II-A, Eq. (5)
* R_SRFF, R_SRF                              -- Section II-B
* R_SRC                                      -- Section III-F, Eq. (8)
* ties-to-even pre-round inside R_SRC        -- Section II-A (R_TNE), III-F

Choices the paper leaves open (sign handling, out-of-range values, the random
source and how draws are indexed) are stated where they are made.
"""
from fractions import Fraction
from math import isqrt

# ---------------------------------------------------------------------------
# Formats (K, P, B; M) -- Section II.  P counts the hidden bit.
# ---------------------------------------------------------------------------
# name -> dict(K, P, B, M, has_inf, max_code, inf_code, nan_code)
#   M        : largest finite value (Section II), exact.
#   max_code : magnitude encoding of M.
#   inf_code : magnitude encoding of +Inf, or None when the format has none.
#   nan_code : magnitude encoding written for NaN inputs (quiet NaN).
FORMATS = {
    "bf16": dict(K=16, P=8, B=127, M=Fraction(255, 128) * Fraction(2) ** 127,
                 max_code=0x7F7F, inf_code=0x7F80, nan_code=0x7FC0),
    "fp16": dict(K=16, P=11, B=15, M=Fraction(65504),
                 max_code=0x7BFF, inf_code=0x7C00, nan_code=0x7E00),
    # OCP 8-bit E4M3 ("fn"): no infinities, the all-ones pattern is the only NaN.
    "e4m3": dict(K=8, P=4, B=7, M=Fraction(448),
                 max_code=0x7E, inf_code=None, nan_code=0x7F),
    "e5m2": dict(K=8, P=3, B=15, M=Fraction(57344),
                 max_code=0x7B, inf_code=0x7C, nan_code=0x7F),
    # Section IV's target format, IEEE WG P3109 Binary8P4 = (8, 4, 8; 224): one zero, the pattern 0x80 is
    # the single NaN (so neither zero nor NaN has a sign), the all-ones magnitude is the infinity.
    "b8p4": dict(K=8, P=4, B=8, M=Fraction(224),
                 max_code=0x7E, inf_code=0x7F, nan_code=0x80, single_zero=True),
}
FORMAT_IDS = {"bf16": 0, "fp16": 1, "e4m3": 2, "e5m2": 3, "b8p4": 4}
VARIANTS = ("srff", "srf", "src")
DETERMINISTIC = ("rtne", "rta", "rto")          # Section II-A: ties to even, ties away, ties to odd
VARIANT_IDS = {"srff": 0, "srf": 1, "src": 2, "rtne": 3, "rta": 4, "rto": 5}


def format_of(fmt):
    """A format is named (a key of FORMATS) or given outright as a dict with the same fields."""
    return fmt if isinstance(fmt, dict) else FORMATS[fmt]


def make_format(K, P, B, max_code, inf_code=None, nan_code=None, single_zero=False):
    """A format (K, P, B; M) described at run time, Section II: M is the value of max_code by Eq. (1)."""
    f = dict(K=K, P=P, B=B, M=None, max_code=max_code, inf_code=inf_code, nan_code=nan_code, single_zero=single_zero)
    e, t = max_code >> (P - 1), max_code & ((1 << (P - 1)) - 1)
    f["M"] = value_of(f, 0, e, t)
    return f


def pow2(e):
    """2**e as an exact rational for any integer e."""
    return Fraction(2) ** e


def floor_log2(x):
    """floor(log2 x) for a positive rational x, exactly."""
    assert x > 0
    e = x.numerator.bit_length() - x.denominator.bit_length()
    # 2**e may be off by one from the true floor; fix it up exactly.
    while pow2(e) > x:
        e -= 1
    while pow2(e + 1) <= x:
        e += 1
    return e


def value_of(fmt, s, e, t):
    """F(s, e, t; P, B), Eq. (1): the real value of a finite triple."""
    f = format_of(fmt)
    P, B = f["P"], f["B"]
    if e == 0:
        mag = (0 + t * pow2(1 - P)) * pow2(1 - B)
    else:
        mag = (1 + t * pow2(1 - P)) * pow2(e - B)
    return -mag if s else mag


def split_code(fmt, code):
    """Bit pattern -> (s, e, t)."""
    f = format_of(fmt)
    K, P = f["K"], f["P"]
    s = (code >> (K - 1)) & 1
    e = (code >> (P - 1)) & ((1 << (K - P)) - 1)
    t = code & ((1 << (P - 1)) - 1)
    return s, e, t


def decode(fmt, code):
    """Bit pattern -> Fraction, or the strings 'nan' / '+inf' / '-inf'."""
    f = format_of(fmt)
    mag = code & ((1 << (f["K"] - 1)) - 1)
    s, e, t = split_code(fmt, code)
    if f.get("single_zero") and code == f["nan_code"]:
        return "nan"
    if f["inf_code"] is not None:
        if mag == f["inf_code"]:
            return "-inf" if s else "+inf"
        if mag > f["inf_code"]:
            return "nan"
    elif mag == f["nan_code"]:
        return "nan"
    return value_of(fmt, s, e, t)


# ---------------------------------------------------------------------------
# binary32 <-> exact rationals
# ---------------------------------------------------------------------------
def f32_bits_to_fraction(u):
    """Finite binary32 pattern -> exact value (binary32 is (32, 24, 127))."""
    s, e, t = u >> 31, (u >> 23) & 0xFF, u & 0x7FFFFF
    assert e != 0xFF
    if e == 0:
        mag = t * pow2(1 - 24) * pow2(1 - 127)
    else:
        mag = (1 + t * pow2(1 - 24)) * pow2(e - 127)
    return -mag if s else mag


def fraction_to_f32_bits(x, negative_zero=False):
    """Round an exact rational to binary32, nearest with ties to even.

    Used for the binary32 arithmetic steps (scale multiply, optimizer update)
    so that each one is 'the exact result, rounded once'.
    """
    if x == 0:
        return 0x80000000 if negative_zero else 0
    s = 1 if x < 0 else 0
    a = -x if s else x
    e = max(floor_log2(a), -126)
    sig = a * pow2(23 - e)           # in [2**23, 2**24) or below for subnormals
    fl = sig.numerator // sig.denominator
    d = sig - fl
    if d > Fraction(1, 2) or (d == Fraction(1, 2) and (fl & 1)):
        fl += 1
    if fl == 1 << 24:
        fl >>= 1
        e += 1
    if e > 127:
        return (s << 31) | 0x7F800000
    if fl < (1 << 23):
        return (s << 31) | fl                      # subnormal or zero
    return (s << 31) | ((e + 127) << 23) | (fl - (1 << 23))


# ---------------------------------------------------------------------------
# The three few-bit predicates and the tie-to-even pre-round
# ---------------------------------------------------------------------------
def round_nearest_even(z):
    """Nearest integer to the non-negative rational z, ties to the even one."""
    fl = z.numerator // z.denominator
    d = z - fl
    if d > Fraction(1, 2) or (d == Fraction(1, 2) and (fl + 1) % 2 == 0):
        return fl + 1
    return fl


def r_srff(delta, n, N):
    """R_SRFF(delta, n) = delta + n 2^-N >= 1   (Section II-B)."""
    return delta + n * pow2(-N) >= 1


def r_srf(delta, n, N):
    """R_SRF(delta, n) = delta + (n + 1/2) 2^-N >= 1   (Section II-B)."""
    return delta + (n + Fraction(1, 2)) * pow2(-N) >= 1


def r_src(delta, n, N):
    """R_SRC(delta, n) = R_SRFF(Round(delta 2^N) 2^-N, n)   (Eq. (8)).

    Round is round-to-nearest, ties to even, one of the unbiased choices the
    paper allows.  The integer being rounded to is the trailing N bits of the
    precision-(P+N) significand, so 'even' refers to that integer.
    """
    return r_srff(round_nearest_even(delta * pow2(N)) * pow2(-N), n, N)


def r_ta(delta):
    """R_TA(delta) = delta >= 0.5   (Section II-A, Eq. (4))."""
    return delta >= Fraction(1, 2)


def r_tne(sig, delta):
    """R_TNE(sigma~, delta) = delta > 0.5 or (delta = 0.5 and IsEven(floor(sigma~) + 1))   (Section II-A)."""
    fl = sig.numerator // sig.denominator
    return delta > Fraction(1, 2) or (delta == Fraction(1, 2) and (fl + 1) % 2 == 0)


def r_tno(sig, delta):
    """Ties to odd, the analogue the paper mentions next to R_TNE."""
    fl = sig.numerator // sig.denominator
    return delta > Fraction(1, 2) or (delta == Fraction(1, 2) and (fl + 1) % 2 == 1)


PREDICATES = {"srff": r_srff, "srf": r_srf, "src": r_src}


def round_positive(xt, fmt, variant, n, N):
    """Round a strictly positive real xt <= M to the format (Section II-A).

    Returns (code_magnitude, up, delta) where up is the predicate's 0/1 value
    and delta the fractional part it was evaluated on.
    """
    f = format_of(fmt)
    P, B = f["P"], f["B"]
    assert xt > 0 and (variant in DETERMINISTIC or 0 <= n < (1 << N))
    e = max(floor_log2(xt), 1 - B)                     # Eq. (2)
    sig = xt * pow2(-e) * pow2(P - 1)                  # Eq. (3)
    fl = sig.numerator // sig.denominator
    delta = sig - fl
    if variant == "rta":
        up = 1 if r_ta(delta) else 0
    elif variant == "rtne":
        up = 1 if r_tne(sig, delta) else 0
    elif variant == "rto":
        up = 1 if r_tno(sig, delta) else 0
    else:
        up = 1 if PREDICATES[variant](delta, n, N) else 0
    sigma = fl + up                                    # Eq. (5)
    rounded_value = sigma * pow2(e - (P - 1))
    if sigma == (1 << P):                              # exponent increment
        sigma >>= 1
        e += 1
    if sigma >= (1 << (P - 1)):
        be, t = e + B, sigma - (1 << (P - 1))
    else:                                              # subnormal (or zero)
        assert e == 1 - B
        be, t = 0, sigma
    code = (be << (P - 1)) | t
    # The encoded triple must carry exactly the rounded value (Eq. (1)).
    assert value_of(fmt, 0, be, t) == rounded_value
    return code, up, delta


def round_f32_bits(ybits, fmt, variant, n, N, ieee_overflow=False):
    """Round one binary32 pattern (already scaled) to the target format.

    Policy outside the paper's scope (Section II says such values are handled
    deterministically and otherwise ignores them):
      * the magnitude is rounded and the sign copied (the paper rounds x > 0);
      * NaN  -> the format's quiet NaN, sign kept;
      * +-Inf -> +-Inf, or +-M when the format has no infinity;
      * finite |y| > M -> +-M (saturate); such values are not SR-rounded;
      * +-0 -> +-0;
      * a format with a single zero (Binary8P4) has no sign on its NaN and none on a zero result, whether
        the input was -0 or a negative value that rounded down to zero.
    Returns (code, kind, up, delta), kind in {'finite','nan','inf','sat'}.
    """
    f = format_of(fmt)
    sign = (ybits >> 31) << (f["K"] - 1)
    mag = ybits & 0x7FFFFFFF
    single_zero = f.get("single_zero", False)
    if mag > 0x7F800000:
        return (0 if single_zero else sign) | f["nan_code"], "nan", 0, Fraction(0)
    if mag == 0x7F800000:
        code = f["inf_code"] if f["inf_code"] is not None else f["max_code"]
        return sign | code, "inf", 0, Fraction(0)
    if mag == 0:
        return (0 if single_zero else sign), "finite", 0, Fraction(0)
    xt = f32_bits_to_fraction(mag)
    if xt > f["M"]:
        if ieee_overflow:
            # Section II: values beyond the finite range are rounded as IEEE round-to-nearest does:
            # M below M + ulp(M)/2, the infinity (or the NaN of a format without one) above it, ties to even.
            half_ulp = pow2(floor_log2(f["M"]) - (f["P"] - 1) - 1)
            thr = f["M"] + half_ulp          # a tie at thr goes to the even neighbour: M if its last bit is 0
            if xt > thr or (xt == thr and f["max_code"] & 1):
                return sign | (f["inf_code"] if f["inf_code"] is not None else f["nan_code"]), "sat", 0, Fraction(0)
        return sign | f["max_code"], "sat", 0, Fraction(0)
    code, up, delta = round_positive(xt, fmt, variant, n, N)
    if single_zero and code == 0:
        return 0, "finite", up, delta
    return sign | code, "finite", up, delta


# ---------------------------------------------------------------------------
# Random draws: Philox4x32-10 (Salmon et al., SC'11) keyed by seed, counted by
# element block.  The paper leaves the generator open (Section II-B).
# ---------------------------------------------------------------------------
PHILOX_M0, PHILOX_M1 = 0xD2511F53, 0xCD9E8D57
PHILOX_W0, PHILOX_W1 = 0x9E3779B9, 0xBB67AE85
MASK32 = 0xFFFFFFFF


def philox4x32_10(ctr, key):
    c0, c1, c2, c3 = ctr
    k0, k1 = key
    for _ in range(10):
        p0 = PHILOX_M0 * c0
        p1 = PHILOX_M1 * c2
        c0, c1, c2, c3 = ((p1 >> 32) ^ c1 ^ k0) & MASK32, p1 & MASK32, \
                         ((p0 >> 32) ^ c3 ^ k1) & MASK32, p0 & MASK32
        k0 = (k0 + PHILOX_W0) & MASK32
        k1 = (k1 + PHILOX_W1) & MASK32
    return c0, c1, c2, c3


def draws_per_word(k):
    return 32 // k


def draw(seed, g, k, stream=0):
    """The k-bit integer n used for global element index g.

    One generator call serves E = 4 * (32 // k) consecutive elements: block
    b = g // E has counter (b lo, b hi, stream, 0) and key (seed lo, seed hi);
    element g uses field (g mod dpw), low bits first, of output word
    ((g mod E) // dpw).  Unused high bits of each word are discarded.
    """
    dpw = draws_per_word(k)
    E = 4 * dpw
    b = g // E
    out = philox4x32_10((b & MASK32, (b >> 32) & MASK32, stream, 0),
                        (seed & MASK32, (seed >> 32) & MASK32))
    w = (g % E) // dpw
    j = g % dpw
    return (out[w] >> (j * k)) & ((1 << k) - 1)


def field_of_words(words, i, k):
    """Draw for element i from a caller-supplied packed word array."""
    dpw = draws_per_word(k)
    return (int(words[i // dpw]) >> ((i % dpw) * k)) & ((1 << k) - 1)


def scale_bits(xbits, scale_bits_):
    """y = fl32(x * scale), one correctly rounded binary32 multiply."""
    mag = xbits & 0x7FFFFFFF
    if mag >= 0x7F800000:
        return xbits                      # NaN / Inf pass through (scale > 0, finite)
    x = f32_bits_to_fraction(xbits)
    sc = f32_bits_to_fraction(scale_bits_)
    return fraction_to_f32_bits(x * sc, negative_zero=bool(xbits >> 31))


def fbsr_round(xbits_list, fmt, variant, k, seed, offset=0, scale_bits_=0x3F800000,
               words=None):
    """Round a sequence of binary32 patterns; returns (codes, stats dict).

    Statistics use the magnitude-domain error e = up - delta in target ulps
    (the quantity whose mean the paper calls bias, Section III), summed
    exactly over the elements that were SR-rounded.
    """
    codes = []
    st = dict(n_finite=0, n_up=0, n_nan=0, n_inf=0, n_sat=0,
              sum_e=Fraction(0), sum_e2=Fraction(0), sum_signed_e=Fraction(0),
              sum_abs_e=Fraction(0), e=[])
    for i, xb in enumerate(xbits_list):
        n = field_of_words(words, i, k) if words is not None else draw(seed, offset + i, k)
        yb = scale_bits(int(xb), scale_bits_)
        code, kind, up, delta = round_f32_bits(yb, fmt, variant, n, k)
        codes.append(code)
        if kind == "finite":
            e = up - delta
            st["n_finite"] += 1
            st["n_up"] += up
            st["sum_e"] += e
            st["sum_e2"] += e * e
            st["sum_signed_e"] += -e if (yb >> 31) else e
            st["sum_abs_e"] += abs(e)
            st["e"].append(e)
        else:
            st["n_" + kind] += 1
            st["e"].append(None)
    return codes, st


# ---------------------------------------------------------------------------
# Closed forms from Section III and the appendices, in target ulps
# ---------------------------------------------------------------------------
def bias_srff_continuous(N):
    return -pow2(-(N + 1))


def bias_srff_finite(N, D):
    """Mean over the 2^D residues; exact form before the bound, Appendix C."""
    tot = sum(Fraction((pow2(D - N) * n).__floor__()) * pow2(-D) for n in range(1 << N))
    return pow2(-N) * tot - (1 - pow2(-D)) / 2


def bias_srf_finite(N, D):
    """Exact form before the bound, Appendix D."""
    tot = sum(Fraction((n * pow2(D - N) + pow2(D - N - 1)).__floor__()) * pow2(-D)
              for n in range(1 << N))
    return pow2(-N) * tot - (1 - pow2(-D)) / 2


# ---------------------------------------------------------------------------
# Fused optimizer steps in binary32: every operation is the exact result
# rounded once (fused multiply-add where stated).  The paper only says the
# update is computed in a wider format and then SR-rounded (Algorithm 1), so
# the operation list below is this library's definition.
# ---------------------------------------------------------------------------
def _q(bits):
    return f32_bits_to_fraction(bits)


def _rn(x):
    return fraction_to_f32_bits(x)


def _fma(a, b, c):
    return _rn(_q(a) * _q(b) + _q(c))


def _mul(a, b):
    return _rn(_q(a) * _q(b))


def _add(a, b):
    return _rn(_q(a) + _q(b))


def _div(a, b):
    return _rn(_q(a) / _q(b))


def _neg(a):
    return a ^ 0x80000000


def _sqrt(a):
    """Correctly rounded binary32 square root of a non-negative finite value."""
    x = _q(a)
    if x == 0:
        return a
    # Scale to an integer with plenty of guard bits: x = num/den.
    shift = 200
    v = isqrt((x.numerator << (2 * shift)) // x.denominator)     # floor(sqrt(x) * 2^shift)
    lo = Fraction(v, 1 << shift)
    # sqrt of a binary32 number is never a rounding tie, and 2^-200 relative
    # resolution is far finer than half an ulp, so rounding lo (nudged up when
    # inexact) gives the correctly rounded result.
    if lo * lo != x:
        lo += Fraction(1, 1 << (shift + 1))
    return _rn(lo)


def sgd_momentum_step(w, g, m, lr, mu):
    """m' = fma(mu, m, g);  w' = fma(-lr, m', w).  All arguments binary32 patterns."""
    m2 = _fma(mu, m, g)
    w2 = _fma(_neg(lr), m2, w)
    return w2, m2


def adam_coefficients(lr_bits, beta1_bits, beta2_bits, step):
    """Host-side scalars, computed in binary64 and rounded to binary32.

    b1t = beta1^step, b2t = beta2^step by repeated binary64 multiplication;
    c1 = f32(lr / (1 - b1t)); c2 = f32(1 / sqrt(1 - b2t));
    a1 = f32(1 - beta1); a2 = f32(1 - beta2).
    Python floats are binary64, so this is the same arithmetic.
    """
    import struct
    import math

    def f(bits):
        return struct.unpack("<f", struct.pack("<I", bits))[0]

    def b(x):
        return struct.unpack("<I", struct.pack("<f", x))[0]

    lr, b1, b2 = f(lr_bits), f(beta1_bits), f(beta2_bits)
    b1t = b2t = 1.0
    for _ in range(step):
        b1t *= b1
        b2t *= b2
    return b(lr / (1.0 - b1t)), b(1.0 / math.sqrt(1.0 - b2t)), b(1.0 - b1), b(1.0 - b2)


def qat_adamw_step(w8, g16, m, v, w_fmt, g_fmt, variant, n, N, beta1, beta2, eps, c1, c2, a1, a2, lrwd):
    """One iteration of Algorithm 1 for one finite parameter, every step exact and rounded once.

    w8, g16: stored codes; m, v and the scalars: binary32 patterns (lrwd = fl32(lr * weight_decay)).
    Returns (new w8 code, m', v', u16 code).  Same operation list as the C tier:
    u32 = fma(-c1, m'/d, -(lrwd) w16), u16 = RTNE_F16(u32), s16 = RTNE_F16(fl32(w16 + u16)), w8' = FBSR(s16).
    """
    wbits = fraction_to_f32_bits(decode(w_fmt, w8), negative_zero=bool(w8 >> (format_of(w_fmt)["K"] - 1)) and decode(w_fmt, w8) == 0)
    gbits = fraction_to_f32_bits(decode(g_fmt, g16), negative_zero=bool(g16 >> 15) and decode(g_fmt, g16) == 0)
    m2 = _fma(beta1, m, _mul(a1, gbits))
    v2 = _fma(beta2, v, _mul(_mul(a2, gbits), gbits))
    d = _add(_mul(_sqrt(v2), c2), eps)
    u32 = _fma(_neg(c1), _div(m2, d), _mul(_neg(lrwd), wbits))
    u16 = round_f32_bits(u32, g_fmt, "rtne", 0, 1)[0]
    ubits = fraction_to_f32_bits(decode(g_fmt, u16), negative_zero=bool(u16 >> 15) and decode(g_fmt, u16) == 0)
    s32 = _add(wbits, ubits)
    s16 = round_f32_bits(s32, g_fmt, "rtne", 0, 1)[0]
    sbits = fraction_to_f32_bits(decode(g_fmt, s16), negative_zero=bool(s16 >> 15) and decode(g_fmt, s16) == 0)
    return round_f32_bits(sbits, w_fmt, variant, n, N)[0], m2, v2, u16


def adam_step(w, g, m, v, beta1, beta2, eps, c1, c2, a1, a2):
    """m' = fma(b1, m, a1*g); v' = fma(b2, v, (a2*g)*g);
    d = sqrt(v')*c2 + eps;  w' = fma(-c1, m'/d, w)."""
    m2 = _fma(beta1, m, _mul(a1, g))
    v2 = _fma(beta2, v, _mul(_mul(a2, g), g))
    d = _add(_mul(_sqrt(v2), c2), eps)
    w2 = _fma(_neg(c1), _div(m2, d), w)
    return w2, m2, v2
