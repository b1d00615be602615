"""ctypes binding of libfbsr.so (see include/fbsr.h for the contract of each call).

Argument marshalling only.  Tensors must live on a CUDA device (except for
``fbsr_round_host``), be contiguous and have the dtype the C signature implies;
output tensors are allocated with torch when not supplied.  Calls are enqueued on
torch's current stream of the tensors' device.
"""
import ctypes
import os

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
_LIB_PATH = os.path.join(_HERE, "libfbsr.so")

FMT = {"bf16": 0, "fp16": 1, "e4m3": 2, "e5m2": 3, "b8p4": 4}
OVF_IEEE = 0x100          # or into a format id, or append "+ieee" to a format name: IEEE overflow instead of saturation
VARIANT = {"srff": 0, "srf": 1, "src": 2, "rtne": 3, "rta": 4, "rto": 5}
CODE_DTYPE = {"bf16": torch.uint16, "fp16": torch.uint16, "e4m3": torch.uint8, "e5m2": torch.uint8, "b8p4": torch.uint8}
VIEW_DTYPE = {"bf16": torch.bfloat16, "fp16": torch.float16, "e4m3": torch.float8_e4m3fn,    # b8p4: torch has no such dtype
              "e5m2": torch.float8_e5m2}


class FbsrError(RuntimeError):
    def __init__(self, status, what):
        self.status = status
        super().__init__("%s failed: %s (status %d)" % (what, fbsr_status_string(status), status))


class FbsrStats(ctypes.Structure):
    _fields_ = [("n_finite", ctypes.c_uint64), ("n_up", ctypes.c_uint64), ("n_nan", ctypes.c_uint64),
                ("n_inf", ctypes.c_uint64), ("n_sat", ctypes.c_uint64), ("sum_e", ctypes.c_double),
                ("sum_e2", ctypes.c_double), ("sum_signed_e", ctypes.c_double), ("sum_abs_e", ctypes.c_double)]


class FbsrFormatDesc(ctypes.Structure):
    """fbsr_format_desc of include/fbsr.h: a format (K, P, B; M) given at run time."""
    _fields_ = [("K", ctypes.c_int32), ("P", ctypes.c_int32), ("B", ctypes.c_int32), ("max_code", ctypes.c_uint32),
                ("has_inf", ctypes.c_int32), ("inf_code", ctypes.c_uint32), ("nan_code", ctypes.c_uint32),
                ("single_zero", ctypes.c_int32)]


def format_desc(K, P, B, max_code, inf_code=None, nan_code=0, single_zero=False):
    """Fill in an FbsrFormatDesc; inf_code=None means that the format has no infinity."""
    return FbsrFormatDesc(K, P, B, max_code, 0 if inf_code is None else 1, 0 if inf_code is None else inf_code,
                          nan_code, 1 if single_zero else 0)


def _load():
    if not os.path.exists(_LIB_PATH):
        raise ImportError("libfbsr.so is not built: run `python -m paper_2504_20634_b200.build` "
                          "(there is no fallback implementation)")
    L = ctypes.CDLL(_LIB_PATH)
    vp, sz, i, u64, f = ctypes.c_void_p, ctypes.c_size_t, ctypes.c_int, ctypes.c_uint64, ctypes.c_float
    L.fbsr_round.argtypes = [vp, vp, sz, i, i, i, u64, u64, f, vp]
    L.fbsr_round_bits.argtypes = [vp, vp, sz, i, i, i, vp, f, vp]
    L.fbsr_round_mx.argtypes = [vp, vp, vp, sz, i, i, i, u64, u64, vp]
    L.fbsr_round_mx.restype = i
    L.fbsr_round_lp.argtypes = [vp, i, vp, sz, i, i, i, u64, u64, f, vp]
    L.fbsr_round_lp.restype = i
    L.fbsr_round_desc.argtypes = [vp, vp, sz, ctypes.POINTER(FbsrFormatDesc), i, i, i, u64, u64, f, vp]
    L.fbsr_round_desc.restype = i
    L.fbsr_format_desc_valid.argtypes = [ctypes.POINTER(FbsrFormatDesc)]
    L.fbsr_format_desc_valid.restype = i
    L.fbsr_stats_workspace_bytes.argtypes = []
    L.fbsr_stats_workspace_bytes.restype = sz
    L.fbsr_round_stats.argtypes = [vp, vp, sz, i, i, i, u64, u64, f, sz, vp, vp, vp, vp, sz, vp]
    L.fbsr_round_stats_noalloc.argtypes = [vp, vp, sz, i, i, i, u64, u64, f, sz, vp, vp, vp, vp]
    L.fbsr_round_stats_noalloc.restype = i
    L.fbsr_sgd_update.argtypes = [vp, vp, vp, vp, sz, i, i, i, u64, u64, f, f, vp]
    L.fbsr_adam_update.argtypes = [vp, vp, vp, vp, vp, sz, i, i, i, u64, u64, f, f, f, f, i, vp]
    L.fbsr_accumulate.argtypes = [vp, vp, sz, i, i, i, u64, u64, vp]
    L.fbsr_qat_update.argtypes = [vp, vp, sz, i, i, i, i, u64, u64, vp]
    L.fbsr_qat_update.restype = i
    L.fbsr_qat_adamw_step.argtypes = [vp, vp, vp, vp, sz, i, i, i, i, u64, u64, f, f, f, f, f, i, vp]
    L.fbsr_qat_adamw_step.restype = i
    L.fbsr_round_host_min_workspace.argtypes = []
    L.fbsr_round_host_min_workspace.restype = sz
    L.fbsr_round_host.argtypes = [vp, vp, sz, i, i, i, u64, u64, f, vp, sz, vp]
    L.fbsr_adam_scalars.argtypes = [f, f, f, i, ctypes.POINTER(ctypes.c_float)]
    L.fbsr_adam_scalars.restype = None
    L.fbsr_tile_elements.argtypes = [i]
    L.fbsr_tile_elements.restype = sz
    L.fbsr_launch_count.argtypes = []
    L.fbsr_launch_count.restype = u64
    L.fbsr_status_string.argtypes = [i]
    L.fbsr_status_string.restype = ctypes.c_char_p
    L.fbsr_version.argtypes = []
    L.fbsr_version.restype = i
    for name in ("fbsr_round", "fbsr_round_bits", "fbsr_round_stats", "fbsr_sgd_update", "fbsr_adam_update",
                 "fbsr_accumulate", "fbsr_round_host"):
        getattr(L, name).restype = i
    return L


_L = _load()


def library_path():
    return _LIB_PATH


def fbsr_status_string(status):
    return _L.fbsr_status_string(int(status)).decode()


def fbsr_version():
    return int(_L.fbsr_version())


def fbsr_tile_elements(k_bits):
    return int(_L.fbsr_tile_elements(int(k_bits)))


def fbsr_adam_scalars(lr, beta1, beta2, step):
    """(c1, c2, a1, a2) of fbsr_adam_update / fbsr_qat_adamw_step as binary32 values (host only)."""
    out = (ctypes.c_float * 4)()
    _L.fbsr_adam_scalars(lr, beta1, beta2, step, out)
    return tuple(float(x) for x in out)


def fbsr_launch_count():
    return int(_L.fbsr_launch_count())


def fbsr_stats_workspace_bytes():
    return int(_L.fbsr_stats_workspace_bytes())


def fbsr_round_host_min_workspace():
    return int(_L.fbsr_round_host_min_workspace())


def _fmt(fmt):
    if isinstance(fmt, int):
        return fmt
    return FMT[fmt[:-5]] | OVF_IEEE if fmt.endswith("+ieee") else FMT[fmt]


def _fmt_name(fmt):
    # unknown integers fall through to the library, which rejects them with a status code
    if isinstance(fmt, str):
        return fmt[:-5] if fmt.endswith("+ieee") else fmt
    return {v: k for k, v in FMT.items()}.get(fmt & ~OVF_IEEE, "bf16")


def _var(variant):
    return variant if isinstance(variant, int) else VARIANT[variant]


def _dev(t, dtype, what):
    if not (t.is_cuda and t.is_contiguous() and t.dtype == dtype):
        raise TypeError("%s must be a contiguous CUDA tensor of dtype %s" % (what, dtype))
    return ctypes.c_void_p(t.data_ptr())


def _stream(t):
    return ctypes.c_void_p(torch.cuda.current_stream(t.device).cuda_stream)


def _check(status, what):
    if status != 0:
        raise FbsrError(status, what)


def _out(src, fmt, out):
    dt = CODE_DTYPE[_fmt_name(fmt)]
    if out is None:
        out = torch.empty(src.numel(), dtype=dt, device=src.device)
    return out, _dev(out, dt, "out")


def fbsr_round(src, fmt, variant, k_bits, seed, offset=0, scale=1.0, out=None):
    """dst = FBSR(fl32(src * scale)); returns the tensor of codes (uint16 / uint8)."""
    out, po = _out(src, fmt, out)
    with torch.cuda.device(src.device):
        _check(_L.fbsr_round(_dev(src, torch.float32, "src"), po, src.numel(), _fmt(fmt), _var(variant), k_bits,
                             seed, offset, scale, _stream(src)), "fbsr_round")
    return out


def fbsr_round_mx(src, fmt, variant, k_bits, seed, offset=0, out=None, scales=None):
    """Block-scaled rounding (blocks of 32 elements, shared power-of-two scale); returns (codes, scale bytes)."""
    out, po = _out(src, fmt, out)
    if scales is None:
        scales = torch.empty((src.numel() + 31) // 32, dtype=torch.uint8, device=src.device)
    with torch.cuda.device(src.device):
        _check(_L.fbsr_round_mx(_dev(src, torch.float32, "src"), po, _dev(scales, torch.uint8, "scales"), src.numel(),
                                _fmt(fmt), _var(variant), k_bits, seed, offset, _stream(src)), "fbsr_round_mx")
    return out, scales


def fbsr_round_desc(src, desc, variant, k_bits, seed, offset=0, scale=1.0, ovf_ieee=False, out=None):
    """fbsr_round for a format described at run time (an FbsrFormatDesc); returns uint8 or uint16 codes."""
    dt = torch.uint16 if desc.K == 16 else torch.uint8
    if out is None:
        out = torch.empty(src.numel(), dtype=dt, device=src.device)
    with torch.cuda.device(src.device):
        _check(_L.fbsr_round_desc(_dev(src, torch.float32, "src"), _dev(out, dt, "out"), src.numel(), ctypes.byref(desc),
                                  1 if ovf_ieee else 0, _var(variant), k_bits, seed, offset, scale, _stream(src)),
               "fbsr_round_desc")
    return out


def fbsr_format_desc_valid(desc):
    return bool(_L.fbsr_format_desc_valid(ctypes.byref(desc)))


def fbsr_round_lp(src_codes, src_fmt, fmt, variant, k_bits, seed, offset=0, scale=1.0, out=None):
    """Round a tensor of bf16/fp16 codes (uint16) to an 8-bit format; returns the uint8 codes."""
    out, po = _out(src_codes, fmt, out)
    with torch.cuda.device(src_codes.device):
        _check(_L.fbsr_round_lp(_dev(src_codes, torch.uint16, "src_codes"), _fmt(src_fmt), po, src_codes.numel(),
                                _fmt(fmt), _var(variant), k_bits, seed, offset, scale, _stream(src_codes)),
               "fbsr_round_lp")
    return out


def fbsr_round_bits(src, fmt, variant, k_bits, rand_words, scale=1.0, out=None):
    out, po = _out(src, fmt, out)
    with torch.cuda.device(src.device):
        _check(_L.fbsr_round_bits(_dev(src, torch.float32, "src"), po, src.numel(), _fmt(fmt), _var(variant),
                                  k_bits, _dev(rand_words, torch.uint32, "rand_words"), scale, _stream(src)),
               "fbsr_round_bits")
    return out


def fbsr_round_stats(src, fmt, variant, k_bits, seed, offset=0, scale=1.0, group_size=0, out=None,
                     workspace=None, total=None, read_back=True):
    """Returns (codes, stats dict, group_sum_e, group_sum_e2); the stats dict is read back with one
    device-to-host copy after the call.  With read_back=False nothing is copied or synchronised and the
    second item is the 72-byte device tensor holding the fbsr_stats record (decode it with
    stats_from_bytes once the stream has been synchronised); `total` and `workspace` may be supplied so
    that repeated calls allocate nothing."""
    out, po = _out(src, fmt, out)
    n = src.numel()
    groups = (n + group_size - 1) // group_size if group_size else 0
    ge = torch.empty(max(groups, 1), dtype=torch.float64, device=src.device) if groups or read_back else None
    ge2 = torch.empty(max(groups, 1), dtype=torch.float64, device=src.device) if groups or read_back else None
    if total is None:
        total = torch.empty(ctypes.sizeof(FbsrStats), dtype=torch.uint8, device=src.device)
    if workspace is None:
        workspace = torch.empty(fbsr_stats_workspace_bytes(), dtype=torch.uint8, device=src.device)
    with torch.cuda.device(src.device):
        _check(_L.fbsr_round_stats(_dev(src, torch.float32, "src"), po, n, _fmt(fmt), _var(variant), k_bits, seed,
                                   offset, scale, group_size, ctypes.c_void_p(ge.data_ptr()) if ge is not None else None,
                                   ctypes.c_void_p(ge2.data_ptr()) if ge2 is not None else None,
                                   ctypes.c_void_p(total.data_ptr()),
                                   ctypes.c_void_p(workspace.data_ptr()), workspace.numel(), _stream(src)),
               "fbsr_round_stats")
    if not read_back:
        return out, total, (ge[:groups] if ge is not None else None), (ge2[:groups] if ge2 is not None else None)
    st = FbsrStats.from_buffer_copy(total.cpu().numpy().tobytes())
    return out, {name: getattr(st, name) for name, _ in FbsrStats._fields_}, ge[:groups], ge2[:groups]


def fbsr_round_stats_noalloc(src, out, total, fmt, variant, k_bits, seed, offset=0, scale=1.0, group_size=0,
                             group_sum_e=None, group_sum_e2=None):
    """fbsr_round_stats for callers that cannot allocate: every buffer (codes `out`, the 72-byte
    `total`, the optional group arrays) is supplied by the caller and the library's own built-in
    scratch is used, so neither this wrapper nor the C call allocates anything.  Returns None;
    read `total` (uint8[72], layout of FbsrStats) after synchronising the stream."""
    pe = ctypes.c_void_p(group_sum_e.data_ptr()) if group_sum_e is not None else None
    pe2 = ctypes.c_void_p(group_sum_e2.data_ptr()) if group_sum_e2 is not None else None
    with torch.cuda.device(src.device):
        _check(_L.fbsr_round_stats_noalloc(_dev(src, torch.float32, "src"),
                                           _dev(out, CODE_DTYPE[_fmt_name(fmt)], "out"), src.numel(), _fmt(fmt),
                                           _var(variant), k_bits, seed, offset, scale, group_size, pe, pe2,
                                           _dev(total, torch.uint8, "total"), _stream(src)),
               "fbsr_round_stats_noalloc")


def stats_from_bytes(total):
    """Decode a 72-byte device or host uint8 tensor holding an fbsr_stats record."""
    st = FbsrStats.from_buffer_copy(total.cpu().numpy().tobytes())
    return {name: getattr(st, name) for name, _ in FbsrStats._fields_}


def fbsr_sgd_update(master_w, grad, momentum, fmt, variant, k_bits, seed, offset, lr, mu, out=None):
    out, po = _out(master_w, fmt, out)
    f32 = torch.float32
    with torch.cuda.device(master_w.device):
        _check(_L.fbsr_sgd_update(_dev(master_w, f32, "master_w"), _dev(grad, f32, "grad"),
                                  _dev(momentum, f32, "momentum"), po, master_w.numel(), _fmt(fmt), _var(variant),
                                  k_bits, seed, offset, lr, mu, _stream(master_w)), "fbsr_sgd_update")
    return out


def fbsr_adam_update(master_w, grad, m, v, fmt, variant, k_bits, seed, offset, lr, beta1, beta2, eps, step,
                     out=None):
    out, po = _out(master_w, fmt, out)
    f32 = torch.float32
    with torch.cuda.device(master_w.device):
        _check(_L.fbsr_adam_update(_dev(master_w, f32, "master_w"), _dev(grad, f32, "grad"), _dev(m, f32, "m"),
                                   _dev(v, f32, "v"), po, master_w.numel(), _fmt(fmt), _var(variant), k_bits, seed,
                                   offset, lr, beta1, beta2, eps, step, _stream(master_w)), "fbsr_adam_update")
    return out


def fbsr_accumulate(w_lp, update, fmt, variant, k_bits, seed, offset=0):
    """In place on w_lp (tensor of codes)."""
    with torch.cuda.device(w_lp.device):
        _check(_L.fbsr_accumulate(_dev(w_lp, CODE_DTYPE[_fmt_name(fmt)], "w_lp"), _dev(update, torch.float32, "update"),
                                  w_lp.numel(), _fmt(fmt), _var(variant), k_bits, seed, offset, _stream(w_lp)),
               "fbsr_accumulate")
    return w_lp


def fbsr_qat_update(w8, update16, w_fmt, u_fmt, variant, k_bits, seed, offset=0):
    """In place on w8 (uint8 codes): w8 <- FBSR(RTNE_16(value(w8) + value(update16)))."""
    with torch.cuda.device(w8.device):
        _check(_L.fbsr_qat_update(_dev(w8, torch.uint8, "w8"), _dev(update16, torch.uint16, "update16"), w8.numel(),
                                  _fmt(w_fmt), _fmt(u_fmt), _var(variant), k_bits, seed, offset, _stream(w8)),
               "fbsr_qat_update")
    return w8


def fbsr_qat_adamw_step(w8, grad16, m, v, w_fmt, g_fmt, variant, k_bits, seed, offset, lr, beta1, beta2, eps,
                        weight_decay, step):
    """One iteration of Algorithm 1, in place on w8 (uint8 codes), m and v (float32); grad16 holds g_fmt codes."""
    with torch.cuda.device(w8.device):
        _check(_L.fbsr_qat_adamw_step(_dev(w8, torch.uint8, "w8"), _dev(grad16, torch.uint16, "grad16"),
                                      _dev(m, torch.float32, "m"), _dev(v, torch.float32, "v"), w8.numel(), _fmt(w_fmt),
                                      _fmt(g_fmt), _var(variant), k_bits, seed, offset, lr, beta1, beta2, eps, weight_decay,
                                      step, _stream(w8)), "fbsr_qat_adamw_step")
    return w8


def fbsr_round_host(src_host, dst_host, fmt, variant, k_bits, seed, offset, scale, workspace):
    """Host tensors in and out (pinned for overlap); `workspace` is a CUDA uint8 tensor used as staging.
    Enqueues on the current stream of the workspace's device; synchronise it before reading dst_host."""
    if src_host.is_cuda or dst_host.is_cuda or src_host.dtype != torch.float32 or not src_host.is_contiguous():
        raise TypeError("src_host/dst_host must be contiguous host tensors (float32 in)")
    if dst_host.dtype != CODE_DTYPE[_fmt_name(fmt)] or not dst_host.is_contiguous():
        raise TypeError("dst_host has the wrong dtype")
    with torch.cuda.device(workspace.device):
        _check(_L.fbsr_round_host(ctypes.c_void_p(src_host.data_ptr()), ctypes.c_void_p(dst_host.data_ptr()),
                                  src_host.numel(), _fmt(fmt), _var(variant), k_bits, seed, offset, scale,
                                  _dev(workspace, torch.uint8, "workspace"), workspace.numel(), _stream(workspace)),
               "fbsr_round_host")
    return dst_host
