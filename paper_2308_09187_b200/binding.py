"""Thin ctypes binding of libqgx.so: argument marshalling only.

Every function has the name of the C entry point it calls (include/qgx.h).  Tensors are torch
CUDA tensors used as device memory; their data pointers go to the library unchanged.  Outputs
that the caller does not pass are allocated with torch.empty.  A nonzero status raises QgxError.
There is no fallback: if the library cannot be loaded the import fails.
"""
import ctypes as C
import os

import torch

from . import build as _build

QGX_OK = 0
QGX_ERR_INVALID_ARG, QGX_ERR_BAD_LEVELS, QGX_ERR_CAPACITY, QGX_ERR_CORRUPT = 1, 2, 3, 4
QGX_ERR_NONFINITE, QGX_ERR_TIMEOUT, QGX_ERR_CUDA, QGX_ERR_TOO_LARGE = 5, 6, 7, 8
QGX_NORM_L2, QGX_NORM_LINF = 0, 1
QGX_CODE_FIXED, QGX_CODE_HUFFMAN, QGX_CODE_ELIAS = 0, 1, 2
QGX_OP_DENSE_AFFINE, QGX_OP_BILINEAR, QGX_OP_DIAGONAL = 0, 1, 2
QGX_REFIT_NONE, QGX_REFIT_CONTINUE, QGX_REFIT_FIRST = 0, 1, 2
QGX_NORMS_SUPPLIED = 1
QGX_MAX_LEVELS, QGX_MAX_CODE_LEN, QGX_MAX_BUCKET = 32, 12, 16384

EXPORTS = [
    "qgx_create", "qgx_destroy", "qgx_sync_status", "qgx_status_str", "qgx_launch_count",
    "qgx_check_levels", "qgx_stream_capacity_words", "qgx_build_codebook_fixed", "qgx_build_codebook_elias",
    "qgx_build_codebook_huffman", "qgx_fit_levels", "qgx_symbol_pmf",
    "qgx_quantize", "qgx_encode", "qgx_decode", "qgx_average",
    "qgx_exchange", "qgx_exchange_streams", "qgx_update_levels", "qgx_histogram",
    "qgx_set_decode_split", "qgx_set_encode_path", "qgx_set_keep_symbols", "qgx_level_counts", "qgx_code_bits",
    "qgx_choose_code_host", "qgx_choose_code", "qgx_exchange_decode", "qgx_set_wait_limit", "qgx_debug_skip_buckets", "qgx_eg_init", "qgx_eg_step", "qgx_eg_step_two_tables", "qgx_family_step", "qgx_apply_operator", "qgx_timing_enable", "qgx_timing_read",
    "qgx_encode_noalloc", "qgx_exchange_segments",
]
QGX_KERNEL_ENCODE, QGX_KERNEL_DECODE, QGX_KERNEL_HISTOGRAM, QGX_KERNEL_OPERATOR, QGX_KERNEL_FINISH = range(5)


class qgx_codebook(C.Structure):
    _fields_ = [("nlev", C.c_int32), ("maxlen", C.c_int32), ("subblock", C.c_int32),
                ("len", C.c_uint8 * 32), ("code", C.c_uint32 * 32)]

    def lengths(self):
        return [int(self.len[j]) for j in range(self.nlev)]

    def codes(self):
        return [int(self.code[j]) for j in range(self.nlev)]


class qgx_quant_cfg(C.Structure):
    _fields_ = [("nlev", C.c_int32), ("bucket", C.c_int32), ("norm_type", C.c_int32), ("code_type", C.c_int32),
                ("nbins", C.c_int32), ("pad", C.c_int32), ("seed", C.c_uint64),
                ("levels", C.c_float * 32), ("cb", qgx_codebook)]

    def level_list(self):
        return [float(self.levels[j]) for j in range(self.nlev)]


class qgx_operator(C.Structure):
    _fields_ = [("kind", C.c_int32), ("noise_model", C.c_int32), ("d", C.c_uint64), ("mat", C.c_void_p),
                ("bias", C.c_void_p)]


class qgx_eg_state(C.Structure):
    _fields_ = [("d", C.c_uint64), ("K", C.c_int32), ("t", C.c_int32), ("X", C.c_void_p), ("Y", C.c_void_p),
                ("Xbar", C.c_void_p), ("Xhalf", C.c_void_p), ("anchor", C.c_void_p), ("scalars", C.c_void_p)]


class QgxError(RuntimeError):
    def __init__(self, status, where):
        self.status = int(status)
        super().__init__("%s: %s (status %d)" % (where, qgx_status_str(status), status))


_lib = None


def library_path():
    return _build.LIB


def lib():
    """Loads libqgx.so, building it first if the sources are newer (nvcc needed then)."""
    global _lib
    if _lib is None:
        path = _build.build() if os.path.exists(_build.NVCC) else _build.LIB
        L = C.CDLL(path)
        L.qgx_status_str.restype = C.c_char_p
        L.qgx_launch_count.restype = C.c_uint64
        L.qgx_launch_count.argtypes = [C.c_void_p]
        L.qgx_stream_capacity_words.restype = C.c_size_t
        L.qgx_stream_capacity_words.argtypes = [C.c_size_t, C.c_int, C.c_int, C.c_int]
        L.qgx_create.argtypes = [C.POINTER(C.c_void_p), C.c_int, C.c_void_p]
        L.qgx_destroy.argtypes = [C.c_void_p]
        L.qgx_destroy.restype = None
        L.qgx_sync_status.argtypes = [C.c_void_p]
        _lib = L
    return _lib


def _chk(st, where):
    if st != QGX_OK:
        raise QgxError(st, where)


def _ptr(t):
    if t is None:
        return None
    assert t.is_cuda and t.is_contiguous(), "device tensors must be contiguous CUDA tensors"
    return C.c_void_p(t.data_ptr())


def _levels(levels):
    vals = [float(x) for x in levels]
    return (C.c_float * len(vals))(*vals), len(vals)


class Context:
    """A qgx_ctx bound to a device and to the torch stream current at creation."""

    def __init__(self, device=0, stream=None):
        self.device = int(device)
        with torch.cuda.device(self.device):
            s = torch.cuda.current_stream() if stream is None else stream
        self.stream = s
        h = C.c_void_p()
        _chk(lib().qgx_create(C.byref(h), self.device, C.c_void_p(s.cuda_stream)), "qgx_create")
        self.h = h

    def close(self):
        if self.h:
            lib().qgx_destroy(self.h)
            self.h = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass


def qgx_create(device=0, stream=None):
    return Context(device, stream)


def qgx_destroy(ctx):
    ctx.close()


def qgx_status_str(status):
    return lib().qgx_status_str(int(status)).decode()


def qgx_sync_status(ctx, check=True):
    st = lib().qgx_sync_status(ctx.h)
    if check:
        _chk(st, "qgx_sync_status")
    return st


def qgx_launch_count(ctx):
    return int(lib().qgx_launch_count(ctx.h))


def qgx_timing_enable(ctx, max_records):
    _chk(lib().qgx_timing_enable(ctx.h, int(max_records)), "qgx_timing_enable")


def qgx_timing_read(ctx, kernel, reset=False):
    """(launches, total milliseconds) of one instrumented kernel since the last reset."""
    n, ms = C.c_int(0), C.c_double(0.0)
    _chk(lib().qgx_timing_read(ctx.h, int(kernel), int(reset), C.byref(n), C.byref(ms)), "qgx_timing_read")
    return n.value, ms.value


# ---------------------------------------------------------------- host helpers
def qgx_check_levels(levels):
    arr, n = _levels(levels)
    return lib().qgx_check_levels(arr, n)


def qgx_stream_capacity_words(d, bucket, subblock, maxlen):
    return int(lib().qgx_stream_capacity_words(d, bucket, subblock, maxlen))


def qgx_build_codebook_elias(nlev, subblock=0):
    cb = qgx_codebook()
    _chk(lib().qgx_build_codebook_elias(nlev, subblock, C.byref(cb)), "qgx_build_codebook_elias")
    return cb


def qgx_build_codebook_fixed(nlev, subblock=0):
    cb = qgx_codebook()
    _chk(lib().qgx_build_codebook_fixed(nlev, subblock, C.byref(cb)), "qgx_build_codebook_fixed")
    return cb


def qgx_build_codebook_huffman(p, subblock=0):
    arr = (C.c_double * len(p))(*[float(x) for x in p])
    cb = qgx_codebook()
    _chk(lib().qgx_build_codebook_huffman(arr, len(p), subblock, C.byref(cb)), "qgx_build_codebook_huffman")
    return cb


def qgx_fit_levels(hist, nlev=None, levels=None):
    """first fit (quantile start) when levels is None, otherwise continues from levels."""
    h = (C.c_double * len(hist))(*[float(x) for x in hist])
    if levels is None:
        arr, n, first = (C.c_float * nlev)(), nlev, 1
    else:
        arr, n = _levels(levels)
        first = 0
    _chk(lib().qgx_fit_levels(h, len(hist), arr, n, first), "qgx_fit_levels")
    return [float(arr[j]) for j in range(n)]


def qgx_symbol_pmf(hist, levels):
    h = (C.c_double * len(hist))(*[float(x) for x in hist])
    arr, n = _levels(levels)
    p = (C.c_double * n)()
    _chk(lib().qgx_symbol_pmf(h, len(hist), arr, n, p), "qgx_symbol_pmf")
    return [float(p[j]) for j in range(n)]


def make_quant_cfg(levels, bucket, cb, seed, norm_type=QGX_NORM_L2, code_type=QGX_CODE_FIXED, nbins=1024):
    cfg = qgx_quant_cfg()
    cfg.nlev = len(levels)
    cfg.bucket = bucket
    cfg.norm_type = norm_type
    cfg.code_type = code_type
    cfg.nbins = nbins
    cfg.seed = seed
    for j, x in enumerate(levels):
        cfg.levels[j] = float(x)
    C.memmove(C.byref(cfg.cb), C.byref(cb), C.sizeof(qgx_codebook))
    return cfg


# ---------------------------------------------------------------- the four steps
def _nb(d, bucket):
    return (d + bucket - 1) // bucket


def qgx_quantize(ctx, v, bucket, levels, norm_type, seed, exchange_id, flags=0, norms=None, sym=None):
    K, d = v.shape
    if norms is None:
        norms = torch.empty((K, _nb(d, bucket)), dtype=torch.float32, device=v.device)
    if sym is None:
        sym = torch.empty((K, d), dtype=torch.uint8, device=v.device)
    arr, n = _levels(levels)
    _chk(lib().qgx_quantize(ctx.h, _ptr(v), K, C.c_size_t(d), bucket, arr, n, norm_type, C.c_uint64(seed),
                            C.c_uint32(exchange_id), flags, _ptr(norms), _ptr(sym)), "qgx_quantize")
    return norms, sym


def qgx_encode(ctx, norms, sym, bucket, cb, cap_words=None, stream=None, bucket_bits=None, total_bits=None):
    K, d = sym.shape
    if cap_words is None:
        cap_words = qgx_stream_capacity_words(d, bucket, cb.subblock, cb.maxlen)
    if stream is None:
        stream = torch.zeros((K, cap_words), dtype=torch.int32, device=sym.device)
    if bucket_bits is None:
        bucket_bits = torch.empty((K, _nb(d, bucket)), dtype=torch.int32, device=sym.device)
    if total_bits is None:
        total_bits = torch.empty((K,), dtype=torch.int64, device=sym.device)
    _chk(lib().qgx_encode(ctx.h, _ptr(norms), _ptr(sym), K, C.c_size_t(d), bucket, C.byref(cb), _ptr(stream),
                          C.c_size_t(cap_words), _ptr(bucket_bits), _ptr(total_bits)), "qgx_encode")
    return stream, bucket_bits, total_bits


def qgx_encode_noalloc(ctx, norms, sym, bucket, cb, stream, bucket_bits, total_bits):
    """qgx_encode without any device allocation: for callers that cannot call cudaMalloc (code inside a
    stream capture, processes whose memory is handed out once at start-up).  Every buffer, outputs
    included, is the caller's; this wrapper allocates nothing either.  Limits: K <= 1024, K * nb <= 65536."""
    K, d = sym.shape
    _chk(lib().qgx_encode_noalloc(ctx.h, _ptr(norms), _ptr(sym), K, C.c_size_t(d), bucket, C.byref(cb), _ptr(stream),
                                  C.c_size_t(stream.shape[1]), _ptr(bucket_bits), _ptr(total_bits)), "qgx_encode_noalloc")
    return stream, bucket_bits, total_bits


def qgx_decode(ctx, stream, bucket_bits, d, bucket, cb, norms=None, sym=None):
    K, cap_words = stream.shape
    if norms is None:
        norms = torch.empty((K, _nb(d, bucket)), dtype=torch.float32, device=stream.device)
    if sym is None:
        sym = torch.empty((K, d), dtype=torch.uint8, device=stream.device)
    _chk(lib().qgx_decode(ctx.h, _ptr(stream), C.c_size_t(cap_words), _ptr(bucket_bits), K, C.c_size_t(d), bucket,
                          C.byref(cb), _ptr(norms), _ptr(sym)), "qgx_decode")
    return norms, sym


def qgx_average(ctx, norms, sym, bucket, levels, out=None):
    K, d = sym.shape
    if out is None:
        out = torch.empty((d,), dtype=torch.float32, device=sym.device)
    arr, n = _levels(levels)
    _chk(lib().qgx_average(ctx.h, _ptr(norms), _ptr(sym), K, C.c_size_t(d), bucket, arr, n, _ptr(out)), "qgx_average")
    return out


# ---------------------------------------------------------------- fused exchange
def qgx_exchange(ctx, v, cfg, exchange_id, slot=0, mean_out=None, total_bits=None):
    K, d = v.shape
    if mean_out is None:
        mean_out = torch.empty((d,), dtype=torch.float32, device=v.device)
    if total_bits is None:
        total_bits = torch.empty((K,), dtype=torch.int64, device=v.device)
    _chk(lib().qgx_exchange(ctx.h, _ptr(v), K, C.c_size_t(d), C.byref(cfg), C.c_uint32(exchange_id), slot,
                            _ptr(mean_out), _ptr(total_bits)), "qgx_exchange")
    return mean_out, total_bits


def qgx_exchange_decode(ctx, K, d, cfg, slot=0, mean_out=None):
    if mean_out is None:
        mean_out = torch.empty((d,), dtype=torch.float32, device="cuda:%d" % ctx.device)
    _chk(lib().qgx_exchange_decode(ctx.h, K, C.c_size_t(d), C.byref(cfg), slot, _ptr(mean_out)), "qgx_exchange_decode")
    return mean_out


def qgx_set_wait_limit(ctx, polls):
    _chk(lib().qgx_set_wait_limit(ctx.h, int(polls)), "qgx_set_wait_limit")


def qgx_debug_skip_buckets(ctx, buckets):
    _chk(lib().qgx_debug_skip_buckets(ctx.h, C.c_size_t(buckets)), "qgx_debug_skip_buckets")


class qgx_segment(C.Structure):
    _fields_ = [("offset", C.c_size_t), ("length", C.c_size_t), ("cfg", C.POINTER(qgx_quant_cfg))]


def qgx_exchange_segments(ctx, v, sizes, cfgs, exchange_id, mean_out=None, total_bits=None):
    """sizes[s] coordinates per tensor (laid back to back in v[K, sum(sizes)]), cfgs[s] its qgx_quant_cfg."""
    K, d = v.shape
    if mean_out is None:
        mean_out = torch.empty((d,), dtype=torch.float32, device=v.device)
    if total_bits is None:
        total_bits = torch.empty((K,), dtype=torch.int64, device=v.device)
    segs = (qgx_segment * len(sizes))()
    at = 0
    for s, (n, cfg) in enumerate(zip(sizes, cfgs)):
        segs[s].offset, segs[s].length, segs[s].cfg = at, n, C.pointer(cfg)
        at += n
    _chk(lib().qgx_exchange_segments(ctx.h, _ptr(v), K, C.c_size_t(d), segs, len(sizes), C.c_uint32(exchange_id),
                                     _ptr(mean_out), _ptr(total_bits)), "qgx_exchange_segments")
    return mean_out, total_bits


QGX_SPLIT_AUTO, QGX_SPLIT_NEVER, QGX_SPLIT_ALWAYS, QGX_SPLIT_SYMBOLS = 0, 1, 2, 3


def qgx_set_decode_split(ctx, mode):
    _chk(lib().qgx_set_decode_split(ctx.h, int(mode)), "qgx_set_decode_split")


QGX_ENCODE_AUTO, QGX_ENCODE_REGISTERS, QGX_ENCODE_STAGED = 0, 1, 2


def qgx_set_encode_path(ctx, mode):
    _chk(lib().qgx_set_encode_path(ctx.h, int(mode)), "qgx_set_encode_path")


def qgx_exchange_streams(ctx, slot, K, nb):
    """Views (no copy) of the streams the last exchange on `slot` left in the workspace."""
    sp, bp, tp = C.c_void_p(), C.c_void_p(), C.c_void_p()
    cap = C.c_size_t()
    _chk(lib().qgx_exchange_streams(ctx.h, slot, C.byref(sp), C.byref(cap), C.byref(bp), C.byref(tp)),
         "qgx_exchange_streams")
    return sp.value, int(cap.value), bp.value, tp.value


# ---------------------------------------------------------------- choice of the code
def qgx_set_keep_symbols(ctx, on):
    _chk(lib().qgx_set_keep_symbols(ctx.h, int(bool(on))), "qgx_set_keep_symbols")


def qgx_level_counts(ctx, counts=None):
    if counts is None:
        counts = torch.empty((32,), dtype=torch.int64, device="cuda:%d" % ctx.device)
    _chk(lib().qgx_level_counts(ctx.h, _ptr(counts)), "qgx_level_counts")
    return counts


def qgx_code_bits(counts, cb):
    arr = (C.c_uint64 * 32)(*[int(x) for x in counts])
    bits = C.c_uint64(0)
    _chk(lib().qgx_code_bits(arr, C.byref(cb), C.byref(bits)), "qgx_code_bits")
    return int(bits.value)


def qgx_choose_code_host(counts, cb, allow_rebuild=True):
    """(winner, [bits of the four candidates]); cb is replaced by the winner."""
    arr = (C.c_uint64 * 32)(*[int(x) for x in counts])
    bits, win = (C.c_uint64 * 4)(), C.c_int(0)
    _chk(lib().qgx_choose_code_host(arr, C.byref(cb), int(allow_rebuild), bits, C.byref(win)), "qgx_choose_code_host")
    return win.value, [int(b) for b in bits]


def qgx_choose_code(ctx, cfg, allow_rebuild=True, counts=None):
    """(winner, [bits of the four candidates], counts tensor); cfg.cb is replaced by the winner."""
    if counts is None:
        counts = torch.empty((32,), dtype=torch.int64, device="cuda:%d" % ctx.device)
    bits, win = (C.c_uint64 * 4)(), C.c_int(0)
    _chk(lib().qgx_choose_code(ctx.h, C.byref(cfg), int(allow_rebuild), _ptr(counts), bits, C.byref(win)), "qgx_choose_code")
    return win.value, [int(b) for b in bits], counts


# ---------------------------------------------------------------- level adaptation
def qgx_histogram(ctx, v, bucket, nbins, norm_type=QGX_NORM_L2, weighted=True, hist=None):
    K, d = v.shape
    if hist is None:
        hist = torch.empty((nbins,), dtype=torch.float64, device=v.device)
    _chk(lib().qgx_histogram(ctx.h, _ptr(v), K, C.c_size_t(d), bucket, norm_type, nbins, int(weighted), _ptr(hist)),
         "qgx_histogram")
    return hist


def qgx_update_levels(ctx, v, cfg, refit, hist=None):
    """Refits cfg.levels and cfg.cb in place; returns the histogram as a list (host copy)."""
    K, d = v.shape
    if hist is None:
        hist = torch.empty((cfg.nbins,), dtype=torch.float64, device=v.device)
    host = (C.c_double * cfg.nbins)()
    _chk(lib().qgx_update_levels(ctx.h, _ptr(v), K, C.c_size_t(d), C.byref(cfg), refit, _ptr(hist), host),
         "qgx_update_levels")
    return [float(x) for x in host]


# ---------------------------------------------------------------- the iteration
class EgState:
    """Device vectors of the iteration plus the C struct that points at them."""

    def __init__(self, z0, K):
        d = z0.numel()
        self.anchor = z0.detach().clone().contiguous()
        self.X = torch.empty_like(self.anchor)
        self.Y = torch.empty_like(self.anchor)
        self.Xbar = torch.empty_like(self.anchor)
        self.Xhalf = torch.zeros_like(self.anchor)
        self.scalars = torch.zeros(2, dtype=torch.float64, device=z0.device)
        self.c = qgx_eg_state(d, K, 1, self.X.data_ptr(), self.Y.data_ptr(), self.Xbar.data_ptr(),
                              self.Xhalf.data_ptr(), self.anchor.data_ptr(), self.scalars.data_ptr())

    @property
    def t(self):
        return self.c.t

    def read_scalars(self):
        s = self.scalars.cpu()
        return float(s[0]), float(s[1])


QGX_NOISE_ADDITIVE, QGX_NOISE_RELATIVE = 0, 1


def make_operator(kind, mat, bias=None, noise_model=QGX_NOISE_ADDITIVE):
    d = 2 * mat.shape[0] if kind == QGX_OP_BILINEAR else mat.shape[0]
    op = qgx_operator(kind, noise_model, d, mat.data_ptr(), bias.data_ptr() if bias is not None else None)
    op._keep = (mat, bias)
    return op


def qgx_eg_init(ctx, state):
    _chk(lib().qgx_eg_init(ctx.h, C.byref(state.c)), "qgx_eg_init")


def qgx_eg_step(ctx, state, op, noise_t, noise_half, cfg, refit=QGX_REFIT_NONE, bits=None):
    _chk(lib().qgx_eg_step(ctx.h, C.byref(state.c), C.byref(op), _ptr(noise_t), _ptr(noise_half), C.byref(cfg),
                           refit, _ptr(bits)), "qgx_eg_step")


def qgx_eg_step_two_tables(ctx, state, op, noise_t, noise_half, cfg_t, cfg_half, refit=QGX_REFIT_NONE, bits=None):
    _chk(lib().qgx_eg_step_two_tables(ctx.h, C.byref(state.c), C.byref(op), _ptr(noise_t), _ptr(noise_half),
                                      C.byref(cfg_t), C.byref(cfg_half), refit, _ptr(bits)), "qgx_eg_step_two_tables")


QGX_METHOD_DE, QGX_METHOD_DA, QGX_METHOD_OPTDA = 0, 1, 2


def qgx_family_step(ctx, state, method, op, noise, cfg, refit=QGX_REFIT_NONE, mean_prev=None, bits=None):
    _chk(lib().qgx_family_step(ctx.h, C.byref(state.c), int(method), C.byref(op), _ptr(noise), C.byref(cfg), refit,
                               _ptr(mean_prev), _ptr(bits)), "qgx_family_step")


def qgx_apply_operator(ctx, op, x, out=None):
    if out is None:
        out = torch.empty((int(op.d),), dtype=torch.float32, device=x.device)
    _chk(lib().qgx_apply_operator(ctx.h, C.byref(op), _ptr(x), _ptr(out)), "qgx_apply_operator")
    return out


class _DeviceView:
    """Wraps a raw device pointer so that torch.as_tensor can view it without a copy."""

    def __init__(self, ptr, n, typestr):
        self.__cuda_array_interface__ = {"shape": (n,), "typestr": typestr, "data": (int(ptr), False), "version": 2}


def device_view(ptr, n, dtype):
    typestr = {torch.int32: "<i4", torch.int64: "<i8", torch.float32: "<f4"}[dtype]
    return torch.as_tensor(_DeviceView(ptr, n, typestr), device="cuda")


def exchange_stream_tensors(ctx, slot, K, nb):
    """(stream [K, cap_words] int32, bucket_bits [K, nb] int32, total_bits [K] int64) of a slot: views into
    the context's workspace, valid until the next call that uses the slot."""
    sp, cap, bp, tp = qgx_exchange_streams(ctx, slot, K, nb)
    return (device_view(sp, K * cap, torch.int32).view(K, cap), device_view(bp, K * nb, torch.int32).view(K, nb),
            device_view(tp, K, torch.int64))
