"""ctypes loader for the scalar C oracle (``fbsr_oracle.c``).  TEST INFRASTRUCTURE ONLY.

The shared object is compiled next to its source with gcc on first use (or when
the source is newer).  Arrays are numpy arrays; the functions mirror the C-ABI of
the CUDA library argument for argument but run on host memory.
"""
import ctypes
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "fbsr_oracle.c")
_LIB = os.path.join(_HERE, "libfbsr_oracle.so")
_CFLAGS = ["-O2", "-std=gnu11", "-ffp-contract=off", "-fno-fast-math", "-shared", "-fPIC"]

FMT = {"bf16": 0, "fp16": 1, "e4m3": 2, "e5m2": 3, "b8p4": 4}
OVF_IEEE = 0x100                   # or-ed into a format id: paper-literal overflow instead of saturation
for _name in ("bf16", "fp16", "e4m3", "e5m2", "b8p4"):
    FMT[_name + "+ieee"] = FMT[_name] | OVF_IEEE
VARIANT = {"srff": 0, "srf": 1, "src": 2, "rtne": 3, "rta": 4, "rto": 5}
CODE_DTYPE = {"bf16": np.uint16, "fp16": np.uint16, "e4m3": np.uint8, "e5m2": np.uint8, "b8p4": np.uint8,
              "bf16+ieee": np.uint16, "fp16+ieee": np.uint16, "e4m3+ieee": np.uint8, "e5m2+ieee": np.uint8,
              "b8p4+ieee": np.uint8}


class OracleDesc(ctypes.Structure):
    """A format (K, P, B; M) given at run time; see the comment above oracle_desc_t in fbsr_oracle.c."""
    _fields_ = [("K", ctypes.c_int32), ("P", ctypes.c_int32), ("B", ctypes.c_int32), ("max_code", ctypes.c_uint32),
                ("has_inf", ctypes.c_int32), ("inf_code", ctypes.c_uint32), ("nan_code", ctypes.c_uint32),
                ("single_zero", ctypes.c_int32)]


def make_desc(K, P, B, max_code, inf_code=None, nan_code=None, single_zero=False):
    return OracleDesc(K, P, B, max_code, 0 if inf_code is None else 1, 0 if inf_code is None else inf_code,
                      nan_code, 1 if single_zero else 0)


class OracleStats(ctypes.Structure):
    _fields_ = [("n_finite", ctypes.c_uint64), ("n_up", ctypes.c_uint64),
                ("n_nan", ctypes.c_uint64), ("n_inf", ctypes.c_uint64),
                ("n_sat", ctypes.c_uint64), ("sum_e", ctypes.c_double),
                ("sum_e2", ctypes.c_double), ("sum_signed_e", ctypes.c_double),
                ("sum_abs_e", ctypes.c_double)]

    def as_dict(self):
        return {name: getattr(self, name) for name, _ in self._fields_}


def build(force=False):
    """Compile the C oracle into ``libfbsr_oracle.so`` beside its source."""
    stale = (not os.path.exists(_LIB)) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC)
    if force or stale:
        tmp = _LIB + ".tmp.%d" % os.getpid()
        subprocess.check_call(["gcc", *_CFLAGS, "-o", tmp, _SRC, "-lm"])
        os.replace(tmp, _LIB)
    return _LIB


_lib = None


def lib():
    global _lib
    if _lib is None:
        L = ctypes.CDLL(build())
        u32p = ctypes.POINTER(ctypes.c_uint32)
        L.fbsr_oracle_philox4x32_10.argtypes = [u32p, u32p, u32p]
        L.fbsr_oracle_philox4x32_10.restype = None
        L.fbsr_oracle_draw.argtypes = [ctypes.c_uint64, ctypes.c_uint64, ctypes.c_int, ctypes.c_uint32]
        L.fbsr_oracle_draw.restype = ctypes.c_uint32
        L.fbsr_oracle_random_words.argtypes = [ctypes.c_uint64, ctypes.c_uint64, ctypes.c_size_t,
                                               ctypes.c_uint32, ctypes.c_void_p]
        L.fbsr_oracle_random_words.restype = None
        L.fbsr_oracle_decode.argtypes = [ctypes.c_int, ctypes.c_uint32]
        L.fbsr_oracle_decode.restype = ctypes.c_float
        L.fbsr_oracle_round_one.argtypes = [ctypes.c_float, ctypes.c_int, ctypes.c_int, ctypes.c_int,
                                            ctypes.c_uint32, ctypes.POINTER(ctypes.c_int),
                                            ctypes.POINTER(ctypes.c_int), ctypes.POINTER(ctypes.c_double)]
        L.fbsr_oracle_round_one.restype = ctypes.c_uint32
        vp, sz, i, u64, f = ctypes.c_void_p, ctypes.c_size_t, ctypes.c_int, ctypes.c_uint64, ctypes.c_float
        L.fbsr_oracle_round.argtypes = [vp, vp, sz, i, i, i, u64, u64, f]
        L.fbsr_oracle_round_bits.argtypes = [vp, vp, sz, i, i, i, vp, f]
        L.fbsr_oracle_round_mx.argtypes = [vp, vp, vp, sz, i, i, i, u64, u64]
        L.fbsr_oracle_round_mx.restype = ctypes.c_int
        L.fbsr_oracle_round_lp.argtypes = [vp, i, vp, sz, i, i, i, u64, u64, f]
        L.fbsr_oracle_round_lp.restype = ctypes.c_int
        L.fbsr_oracle_round_stats.argtypes = [vp, vp, sz, i, i, i, u64, u64, f, sz, vp, vp,
                                              ctypes.POINTER(OracleStats)]
        L.fbsr_oracle_sgd_update.argtypes = [vp, vp, vp, vp, sz, i, i, i, u64, u64, f, f]
        L.fbsr_oracle_adam_update.argtypes = [vp, vp, vp, vp, vp, sz, i, i, i, u64, u64, f, f, f, f, i]
        L.fbsr_oracle_adam_coefficients.argtypes = [f, f, f, i, ctypes.POINTER(ctypes.c_float)]
        L.fbsr_oracle_adam_coefficients.restype = None
        L.fbsr_oracle_accumulate.argtypes = [vp, vp, sz, i, i, i, u64, u64]
        L.fbsr_oracle_qat_update.argtypes = [vp, vp, sz, i, i, i, i, u64, u64]
        L.fbsr_oracle_qat_update.restype = ctypes.c_int
        L.fbsr_oracle_qat_adamw_step.argtypes = [vp, vp, vp, vp, sz, i, i, i, i, u64, u64, f, f, f, f, f, i]
        L.fbsr_oracle_qat_adamw_step.restype = ctypes.c_int
        dp = ctypes.POINTER(OracleDesc)
        L.fbsr_oracle_desc_valid.argtypes = [dp]
        L.fbsr_oracle_desc_valid.restype = ctypes.c_int
        L.fbsr_oracle_decode_desc.argtypes = [dp, ctypes.c_uint32]
        L.fbsr_oracle_decode_desc.restype = ctypes.c_float
        L.fbsr_oracle_round_one_desc.argtypes = [ctypes.c_float, dp, i, i, i, ctypes.c_uint32, ctypes.POINTER(ctypes.c_int),
                                                 ctypes.POINTER(ctypes.c_int), ctypes.POINTER(ctypes.c_double)]
        L.fbsr_oracle_round_one_desc.restype = ctypes.c_uint32
        L.fbsr_oracle_round_desc.argtypes = [vp, vp, sz, dp, i, i, i, u64, u64, f]
        L.fbsr_oracle_round_desc.restype = ctypes.c_int
        for name in ("round", "round_bits", "round_stats", "sgd_update", "adam_update", "accumulate"):
            getattr(L, "fbsr_oracle_" + name).restype = ctypes.c_int
        _lib = L
    return _lib


def _ptr(a):
    return ctypes.c_void_p(a.ctypes.data)


def _f32(a):
    a = np.ascontiguousarray(a, dtype=np.float32)
    return a


def _check(rc):
    if rc != 0:
        raise ValueError("oracle rejected its arguments (rc=%d)" % rc)


def philox4x32_10(ctr, key):
    c = (ctypes.c_uint32 * 4)(*ctr)
    k = (ctypes.c_uint32 * 2)(*key)
    o = (ctypes.c_uint32 * 4)()
    lib().fbsr_oracle_philox4x32_10(c, k, o)
    return tuple(int(x) for x in o)


def draw(seed, g, k, stream=0):
    return int(lib().fbsr_oracle_draw(seed, g, k, stream))


def decode(fmt, code):
    return float(lib().fbsr_oracle_decode(FMT[fmt], int(code)))


_decode_tables = {}


def decode_array(fmt, codes):
    """Widen an array of target codes to float32 values (exact)."""
    if fmt not in _decode_tables:
        nbits = 16 if CODE_DTYPE[fmt] == np.uint16 else 8
        _decode_tables[fmt] = np.array([decode(fmt, c) for c in range(1 << nbits)], dtype=np.float32)
    return _decode_tables[fmt][np.asarray(codes).astype(np.int64)]


def round_one(y, fmt, variant, k, n):
    kind, up, delta = ctypes.c_int(), ctypes.c_int(), ctypes.c_double()
    code = lib().fbsr_oracle_round_one(np.float32(y), FMT[fmt], VARIANT[variant], k, n,
                                       ctypes.byref(kind), ctypes.byref(up), ctypes.byref(delta))
    return int(code), kind.value, up.value, delta.value


def draws(seed, offset, count, k):
    """All draws for global indices offset .. offset+count-1 as a numpy array."""
    return np.array([draw(seed, offset + i, k) for i in range(count)], dtype=np.uint32)


def random_words(seed, offset, count, k):
    """The packed word stream that serves elements offset .. offset+count-1.

    ``offset`` must be a multiple of 32 // k so that element 0 of the call sits
    in field 0 of word 0.  Word j is what the generator produces for global word
    index offset / dpw + j.
    """
    dpw = 32 // k
    assert offset % dpw == 0
    nwords = (count + dpw - 1) // dpw
    out = np.empty(max(nwords, 1), dtype=np.uint32)
    lib().fbsr_oracle_random_words(seed, offset // dpw, nwords, 0, _ptr(out))
    return out[:nwords]


def fbsr_round(src, fmt, variant, k, seed, offset=0, scale=1.0):
    src = _f32(src)
    dst = np.empty(src.size, dtype=CODE_DTYPE[fmt])
    _check(lib().fbsr_oracle_round(_ptr(src), _ptr(dst), src.size, FMT[fmt], VARIANT[variant], k,
                                   seed, offset, scale))
    return dst


def fbsr_round_lp(src_codes, src_fmt, fmt, variant, k, seed, offset=0, scale=1.0):
    """Round an array of low-precision codes (format src_fmt) to format fmt."""
    src = np.ascontiguousarray(src_codes, dtype=CODE_DTYPE[src_fmt])
    dst = np.empty(src.size, dtype=CODE_DTYPE[fmt])
    _check(lib().fbsr_oracle_round_lp(_ptr(src), FMT[src_fmt], _ptr(dst), src.size, FMT[fmt], VARIANT[variant], k,
                                      seed, offset, scale))
    return dst


def fbsr_round_bits(src, fmt, variant, k, rand_words, scale=1.0):
    src = _f32(src)
    words = np.ascontiguousarray(rand_words, dtype=np.uint32)
    dst = np.empty(src.size, dtype=CODE_DTYPE[fmt])
    _check(lib().fbsr_oracle_round_bits(_ptr(src), _ptr(dst), src.size, FMT[fmt], VARIANT[variant], k,
                                        _ptr(words), scale))
    return dst


def fbsr_round_stats(src, fmt, variant, k, seed, offset=0, scale=1.0, group_size=0):
    src = _f32(src)
    dst = np.empty(src.size, dtype=CODE_DTYPE[fmt])
    ngroups = (src.size + group_size - 1) // group_size if group_size else 0
    ge = np.zeros(max(ngroups, 1), dtype=np.float64)
    ge2 = np.zeros(max(ngroups, 1), dtype=np.float64)
    st = OracleStats()
    _check(lib().fbsr_oracle_round_stats(_ptr(src), _ptr(dst), src.size, FMT[fmt], VARIANT[variant], k,
                                         seed, offset, scale, group_size, _ptr(ge), _ptr(ge2),
                                         ctypes.byref(st)))
    return dst, st.as_dict(), ge[:ngroups], ge2[:ngroups]


def sgd_update(w, g, m, fmt, variant, k, seed, offset, lr, mu):
    """In place on w and m (float32 numpy arrays); returns the low-precision codes."""
    assert w.dtype == np.float32 and m.dtype == np.float32 and w.flags.c_contiguous and m.flags.c_contiguous
    g = _f32(g)
    dst = np.empty(w.size, dtype=CODE_DTYPE[fmt])
    _check(lib().fbsr_oracle_sgd_update(_ptr(w), _ptr(g), _ptr(m), _ptr(dst), w.size, FMT[fmt],
                                        VARIANT[variant], k, seed, offset, lr, mu))
    return dst


def adam_update(w, g, m, v, fmt, variant, k, seed, offset, lr, beta1, beta2, eps, step):
    for a in (w, m, v):
        assert a.dtype == np.float32 and a.flags.c_contiguous
    g = _f32(g)
    dst = np.empty(w.size, dtype=CODE_DTYPE[fmt])
    _check(lib().fbsr_oracle_adam_update(_ptr(w), _ptr(g), _ptr(m), _ptr(v), _ptr(dst), w.size, FMT[fmt],
                                         VARIANT[variant], k, seed, offset, lr, beta1, beta2, eps, step))
    return dst


def adam_coefficients(lr, beta1, beta2, step):
    out = (ctypes.c_float * 4)()
    lib().fbsr_oracle_adam_coefficients(lr, beta1, beta2, step, out)
    return tuple(np.float32(x) for x in out)


def accumulate(w_lp, update, fmt, variant, k, seed, offset=0):
    """In place on w_lp (array of target codes)."""
    assert w_lp.dtype == CODE_DTYPE[fmt] and w_lp.flags.c_contiguous
    update = _f32(update)
    _check(lib().fbsr_oracle_accumulate(_ptr(w_lp), _ptr(update), w_lp.size, FMT[fmt], VARIANT[variant], k,
                                        seed, offset))
    return w_lp


def qat_update(w8, u16, w_fmt, u_fmt, variant, k, seed, offset=0):
    """In place on w8 (8-bit codes): w8 <- FBSR(RTNE16(value(w8) + value(u16)))."""
    assert w8.dtype == np.uint8 and w8.flags.c_contiguous
    u16 = np.ascontiguousarray(u16, dtype=np.uint16)
    _check(lib().fbsr_oracle_qat_update(_ptr(w8), _ptr(u16), w8.size, FMT[w_fmt], FMT[u_fmt], VARIANT[variant], k,
                                        seed, offset))
    return w8


def qat_adamw_step(w8, g16, m, v, w_fmt, g_fmt, variant, k, seed, offset, lr, beta1, beta2, eps, weight_decay, step):
    """In place on w8 (uint8 codes), m and v (float32)."""
    assert w8.dtype == np.uint8 and g16.dtype == np.uint16 and m.dtype == np.float32 and v.dtype == np.float32
    _check(lib().fbsr_oracle_qat_adamw_step(_ptr(w8), _ptr(g16), _ptr(m), _ptr(v), w8.size, FMT[w_fmt], FMT[g_fmt],
                                            VARIANT[variant], k, seed, offset, lr, beta1, beta2, eps, weight_decay, step))
    return w8


def fbsr_round_mx(src, fmt, variant, k, seed, offset=0):
    """Block-scaled rounding (blocks of 32, shared power-of-two exponent); returns (codes, scale bytes)."""
    src = _f32(src)
    dst = np.empty(src.size, dtype=CODE_DTYPE[fmt])
    scales = np.empty((src.size + 31) // 32, dtype=np.uint8)
    _check(lib().fbsr_oracle_round_mx(_ptr(src), _ptr(dst), _ptr(scales), src.size, FMT[fmt], VARIANT[variant], k,
                                      seed, offset))
    return dst, scales


def desc_valid(desc):
    return bool(lib().fbsr_oracle_desc_valid(ctypes.byref(desc)))


def decode_desc(desc, code):
    return float(lib().fbsr_oracle_decode_desc(ctypes.byref(desc), int(code)))


def round_one_desc(y, desc, variant, k, n, ieee_overflow=False):
    kind, up, delta = ctypes.c_int(), ctypes.c_int(), ctypes.c_double()
    code = lib().fbsr_oracle_round_one_desc(np.float32(y), ctypes.byref(desc), int(ieee_overflow), VARIANT[variant], k, n,
                                            ctypes.byref(kind), ctypes.byref(up), ctypes.byref(delta))
    return int(code), kind.value, up.value, delta.value


def fbsr_round_desc(src, desc, variant, k, seed, offset=0, scale=1.0, ieee_overflow=False):
    src = _f32(src)
    dst = np.empty(src.size, dtype=np.uint16 if desc.K == 16 else np.uint8)
    _check(lib().fbsr_oracle_round_desc(_ptr(src), _ptr(dst), src.size, ctypes.byref(desc), int(ieee_overflow),
                                        VARIANT[variant], k, seed, offset, scale))
    return dst
