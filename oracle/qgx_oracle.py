"""ctypes wrapper of the C++ oracle (oracle/qgx_oracle.cpp).  Test infrastructure only.

Arrays are numpy, C-contiguous: v, noise float32 [K, d]; norms float32 [K, nb];
sym uint8 [K, d]; stream uint32 [K, cap_words]; bucket_bits uint32 [K, nb].
Every function raises OracleError on a nonzero status.
"""
import ctypes as C
import numpy as np

from . import build as _build

OK, INVALID_ARG, BAD_LEVELS, CAPACITY, CORRUPT, NONFINITE = range(6)
L2, LINF = 0, 1
CODE_FIXED, CODE_HUFFMAN, CODE_ELIAS = 0, 1, 2
OP_DENSE_AFFINE, OP_BILINEAR, OP_DIAGONAL = 0, 1, 2


class OracleError(RuntimeError):
    def __init__(self, status, where):
        super().__init__(f"oracle {where}: status {status}")
        self.status = status


class Codebook(C.Structure):
    _fields_ = [("nlev", C.c_int32), ("maxlen", C.c_int32), ("subblock", C.c_int32),
                ("len", C.c_uint8 * 32), ("code", C.c_uint32 * 32)]

    def lengths(self):
        return [int(self.len[j]) for j in range(self.nlev)]

    def codes(self):
        return [int(self.code[j]) for j in range(self.nlev)]


class Operator(C.Structure):
    _fields_ = [("kind", C.c_int32), ("noise_model", C.c_int32), ("d", C.c_uint64),
                ("mat", C.c_void_p), ("bias", C.c_void_p)]


class EgStateC(C.Structure):
    _fields_ = [("d", C.c_uint64), ("K", C.c_int32), ("t", C.c_int32),
                ("X", C.c_void_p), ("Y", C.c_void_p), ("Xbar", C.c_void_p), ("Xhalf", C.c_void_p),
                ("anchor", C.c_void_p), ("sum_sq", C.c_double), ("gamma", C.c_float), ("pad", C.c_float)]


_lib = None


def lib():
    global _lib
    if _lib is None:
        _lib = C.CDLL(_build.build())
        _lib.qgxo_normalize.restype = C.c_float
        _lib.qgxo_normalize.argtypes = [C.c_float, C.c_float]
        _lib.qgxo_xi.restype = C.c_float
        _lib.qgxo_xi.argtypes = [C.c_float, C.c_void_p, C.c_int]
        _lib.qgxo_level_search.argtypes = [C.c_float, C.c_void_p, C.c_int]
        _lib.qgxo_round_up.argtypes = [C.c_float, C.c_uint32]
        _lib.qgxo_count_up.restype = C.c_uint64
        _lib.qgxo_count_up.argtypes = [C.c_float]
        _lib.qgxo_element_word.restype = C.c_uint32
        _lib.qgxo_element_word.argtypes = [C.c_uint64, C.c_uint32, C.c_uint32, C.c_uint64]
        _lib.qgxo_capacity_words.restype = C.c_uint64
        _lib.qgxo_capacity_words.argtypes = [C.c_uint64, C.c_int, C.c_int, C.c_int]
        _lib.qgxo_objective.restype = C.c_double
        _lib.qgxo_stationarity.restype = C.c_double
        _lib.qgxo_stationarity.argtypes = [C.c_void_p, C.c_int, C.c_double, C.c_double, C.c_double]
        _lib.qgxo_form_dual_vectors.restype = None
        _lib.qgxo_form_dual_vectors_relative.restype = None
    return _lib


def _p(a):
    return a.ctypes.data_as(C.c_void_p) if a is not None else None


def _f32(a):
    return np.ascontiguousarray(a, dtype=np.float32)


def _chk(st, where):
    if st != OK:
        raise OracleError(st, where)


# ------------------------------------------------------------------ RNG
def philox4x32_10(ctr, key):
    c = np.asarray(ctr, dtype=np.uint32)
    k = np.asarray(key, dtype=np.uint32)
    out = np.zeros(4, dtype=np.uint32)
    lib().qgxo_philox4x32_10(_p(c), _p(k), _p(out))
    return out


def element_word(seed, worker, xid, e):
    return int(lib().qgxo_element_word(seed, worker, xid, e))


# ------------------------------------------------------------------ scalar pieces
def normalize(v, norm):
    return float(lib().qgxo_normalize(v, norm))


def level_search(u, levels):
    lv = _f32(levels)
    return int(lib().qgxo_level_search(u, _p(lv), len(lv)))


def xi(u, levels, tau):
    lv = _f32(levels)
    return float(lib().qgxo_xi(u, _p(lv), tau))


def round_up(xi_, word):
    return int(lib().qgxo_round_up(xi_, word))


def count_up(xi_):
    return int(lib().qgxo_count_up(xi_))


def check_levels(levels):
    lv = _f32(levels)
    return int(lib().qgxo_check_levels(_p(lv), len(lv)))


# ------------------------------------------------------------------ vector calls
def nbuckets(d, bucket):
    return (d + bucket - 1) // bucket


def bucket_norms(v, bucket, norm_type=L2, allow_nonfinite=False):
    v = _f32(v)
    K, d = v.shape
    norms = np.zeros((K, nbuckets(d, bucket)), dtype=np.float32)
    st = lib().qgxo_bucket_norms(_p(v), K, C.c_uint64(d), bucket, norm_type, _p(norms))
    if not (allow_nonfinite and st == NONFINITE):
        _chk(st, "bucket_norms")
    return norms


def quantize(v, bucket, levels, norms, seed, xid, coord_base=0):
    """coord_base: index of v's first coordinate inside a longer layer-wise vector (variates only)."""
    v = _f32(v)
    lv = _f32(levels)
    norms = _f32(norms)
    K, d = v.shape
    sym = np.zeros((K, d), dtype=np.uint8)
    _chk(lib().qgxo_quantize_at(_p(v), K, C.c_uint64(d), bucket, _p(lv), len(lv), _p(norms),
                                C.c_uint64(seed), C.c_uint32(xid), C.c_uint64(coord_base), _p(sym)), "quantize")
    return sym


def quantize_words(v, bucket, levels, norms, words):
    v = _f32(v)
    lv = _f32(levels)
    norms = _f32(norms)
    words = np.ascontiguousarray(words, dtype=np.uint32)
    K, d = v.shape
    sym = np.zeros((K, d), dtype=np.uint8)
    _chk(lib().qgxo_quantize_words(_p(v), K, C.c_uint64(d), bucket, _p(lv), len(lv), _p(norms),
                                   _p(words), _p(sym)), "quantize_words")
    return sym


def dequantize(norms, sym, bucket, levels):
    lv = _f32(levels)
    norms = _f32(norms)
    sym = np.ascontiguousarray(sym, dtype=np.uint8)
    K, d = sym.shape
    out = np.zeros((K, d), dtype=np.float32)
    _chk(lib().qgxo_dequantize(_p(norms), _p(sym), K, C.c_uint64(d), bucket, _p(lv), len(lv), _p(out)),
         "dequantize")
    return out


def average(norms, sym, bucket, levels):
    lv = _f32(levels)
    norms = _f32(norms)
    sym = np.ascontiguousarray(sym, dtype=np.uint8)
    K, d = sym.shape
    out = np.zeros(d, dtype=np.float32)
    _chk(lib().qgxo_average(_p(norms), _p(sym), K, C.c_uint64(d), bucket, _p(lv), len(lv), _p(out)), "average")
    return out


# ------------------------------------------------------------------ codebooks and the codec
def codebook_fixed(nlev, subblock=0):
    cb = Codebook()
    _chk(lib().qgxo_codebook_fixed(nlev, subblock, C.byref(cb)), "codebook_fixed")
    return cb


def codebook_elias(nlev, subblock=0):
    cb = Codebook()
    _chk(lib().qgxo_codebook_elias(nlev, subblock, C.byref(cb)), "codebook_elias")
    return cb


def codebook_huffman(p, subblock=0):
    p = np.ascontiguousarray(p, dtype=np.float64)
    cb = Codebook()
    _chk(lib().qgxo_codebook_huffman(_p(p), len(p), subblock, C.byref(cb)), "codebook_huffman")
    return cb


def level_counts(sym, nlev):
    """How many coordinates carry each level index (32 counters)."""
    sym = np.ascontiguousarray(sym, dtype=np.uint8)
    K, d = sym.shape
    counts = np.zeros(32, dtype=np.uint64)
    _chk(lib().qgxo_level_counts(_p(sym), K, C.c_uint64(d), nlev, _p(counts)), "level_counts")
    return counts


def code_bits(counts, cb):
    lib().qgxo_code_bits.restype = C.c_uint64
    counts = np.ascontiguousarray(counts, dtype=np.uint64)
    return int(lib().qgxo_code_bits(_p(counts), C.byref(cb)))


def choose_code(counts, cb, allow_rebuild=True):
    """(winner 0..3, bits of the four candidates, the winner's codebook): current, Huffman from the counts, Elias, fixed."""
    counts = np.ascontiguousarray(counts, dtype=np.uint64)
    bits = np.zeros(4, dtype=np.uint64)
    out = Codebook()
    r = lib().qgxo_choose_code(_p(counts), cb.nlev, C.byref(cb), int(allow_rebuild), _p(bits), C.byref(out))
    if r < 0:
        raise OracleError(-r, "choose_code")
    return r, bits, out


def codebook_from(lengths, codes, subblock=0):
    """A hand-made prefix code (tests)."""
    cb = Codebook()
    cb.nlev = len(lengths)
    cb.maxlen = max(lengths)
    cb.subblock = subblock
    for j, (L, c) in enumerate(zip(lengths, codes)):
        cb.len[j] = L
        cb.code[j] = c
    return cb


def capacity_words(d, bucket, subblock, maxlen):
    return int(lib().qgxo_capacity_words(C.c_uint64(d), bucket, subblock, maxlen))


def encode(norms, sym, bucket, cb, cap_words=None):
    norms = _f32(norms)
    sym = np.ascontiguousarray(sym, dtype=np.uint8)
    K, d = sym.shape
    nb = nbuckets(d, bucket)
    if cap_words is None:
        cap_words = capacity_words(d, bucket, cb.subblock, cb.maxlen)
    stream = np.zeros((K, cap_words), dtype=np.uint32)
    bits = np.zeros((K, nb), dtype=np.uint32)
    total = np.zeros(K, dtype=np.uint64)
    _chk(lib().qgxo_encode(_p(norms), _p(sym), K, C.c_uint64(d), bucket, C.byref(cb), _p(stream),
                           C.c_uint64(cap_words), _p(bits), _p(total)), "encode")
    return stream, bits, total


def decode(stream, bucket_bits, d, bucket, cb):
    stream = np.ascontiguousarray(stream, dtype=np.uint32)
    bucket_bits = np.ascontiguousarray(bucket_bits, dtype=np.uint32)
    K, cap_words = stream.shape
    nb = nbuckets(d, bucket)
    norms = np.zeros((K, nb), dtype=np.float32)
    sym = np.zeros((K, d), dtype=np.uint8)
    _chk(lib().qgxo_decode(_p(stream), C.c_uint64(cap_words), _p(bucket_bits), K, C.c_uint64(d), bucket,
                           C.byref(cb), _p(norms), _p(sym)), "decode")
    return norms, sym


# ------------------------------------------------------------------ level adaptation
def histogram(v, bucket, nbins, norm_type=L2, weighted=True):
    v = _f32(v)
    K, d = v.shape
    hist = np.zeros(nbins, dtype=np.float64)
    _chk(lib().qgxo_histogram(_p(v), K, C.c_uint64(d), bucket, norm_type, nbins, int(weighted), _p(hist)),
         "histogram")
    return hist


def objective(hist, levels):
    hist = np.ascontiguousarray(hist, dtype=np.float64)
    lv = _f32(levels)
    return float(lib().qgxo_objective(_p(hist), len(hist), _p(lv), len(lv)))


def stationarity(hist, a, c, l):
    hist = np.ascontiguousarray(hist, dtype=np.float64)
    return float(lib().qgxo_stationarity(_p(hist), len(hist), a, c, l))


def fit_levels(hist, nlev=None, init=None, return_trace=False):
    """first fit (quantile start) when init is None, else coordinate descent from init."""
    hist = np.ascontiguousarray(hist, dtype=np.float64)
    if init is None:
        lv = np.zeros(nlev, dtype=np.float32)
        first = 1
    else:
        lv = _f32(init).copy()
        first = 0
    trace = np.zeros(40, dtype=np.float64)
    ns = C.c_int(0)
    _chk(lib().qgxo_fit_levels(_p(hist), len(hist), _p(lv), len(lv), first, _p(trace), C.byref(ns)), "fit_levels")
    if return_trace:
        return lv, trace[:ns.value + 1].copy()
    return lv


def symbol_pmf(hist, levels):
    hist = np.ascontiguousarray(hist, dtype=np.float64)
    lv = _f32(levels)
    p = np.zeros(len(lv), dtype=np.float64)
    _chk(lib().qgxo_symbol_pmf(_p(hist), len(hist), _p(lv), len(lv), _p(p)), "symbol_pmf")
    return p


def refit(v, bucket, nbins, levels, cb, first_fit, code_type, norm_type=L2):
    """Returns (new levels, histogram); cb is rebuilt in place."""
    v = _f32(v)
    K, d = v.shape
    lv = _f32(levels).copy()
    hist = np.zeros(nbins, dtype=np.float64)
    _chk(lib().qgxo_refit(_p(v), K, C.c_uint64(d), bucket, norm_type, nbins, int(first_fit), code_type,
                          _p(lv), len(lv), C.byref(cb), _p(hist)), "refit")
    return lv, hist


# ------------------------------------------------------------------ operator and iteration
NOISE_ADDITIVE, NOISE_RELATIVE = 0, 1


class Op:
    def __init__(self, kind, mat, bias=None, noise_model=NOISE_ADDITIVE):
        self.kind = kind
        self.mat = _f32(mat)
        self.bias = _f32(bias) if bias is not None else None
        d = 2 * self.mat.shape[0] if kind == OP_BILINEAR else self.mat.shape[0]
        self.d = d
        self.c = Operator(kind, noise_model, d, self.mat.ctypes.data, self.bias.ctypes.data if self.bias is not None else None)


def apply_operator(op, x):
    x = _f32(x)
    out = np.zeros(op.d, dtype=np.float32)
    _chk(lib().qgxo_apply_operator(C.byref(op.c), _p(x), _p(out)), "apply_operator")
    return out


def form_dual_vectors(a, noise, K):
    a = _f32(a)
    d = a.shape[0]
    n = _f32(noise) if noise is not None else None
    V = np.zeros((K, d), dtype=np.float32)
    lib().qgxo_form_dual_vectors(_p(a), _p(n), K, C.c_uint64(d), _p(V))
    return V


def form_dual_vectors_relative(a, scales, K):
    """V_k = A(x) .* S_k (relative noise)."""
    a = _f32(a)
    d = a.shape[0]
    n = _f32(scales) if scales is not None else None
    V = np.zeros((K, d), dtype=np.float32)
    lib().qgxo_form_dual_vectors_relative(_p(a), _p(n), K, C.c_uint64(d), _p(V))
    return V


class EgState:
    """State (X_t, Y_t, Xbar, gamma_t, sum of squared differences, t) of the iteration."""

    def __init__(self, z0, K):
        self.anchor = _f32(z0).copy()
        d = self.anchor.shape[0]
        self.X = self.anchor.copy()
        self.Y = np.zeros(d, dtype=np.float32)
        self.Xbar = np.zeros(d, dtype=np.float32)
        self.Xhalf = np.zeros(d, dtype=np.float32)
        self.c = EgStateC(d, K, 1, self.X.ctypes.data, self.Y.ctypes.data, self.Xbar.ctypes.data,
                          self.Xhalf.ctypes.data, self.anchor.ctypes.data, 0.0, float(K), 0.0)

    @property
    def t(self):
        return self.c.t

    @property
    def gamma(self):
        return self.c.gamma

    @property
    def sum_sq(self):
        return self.c.sum_sq

    def load(self, X, Y, Xbar, sum_sq, gamma, t):
        """Overwrite the state (teacher forcing)."""
        self.X[:] = X
        self.Y[:] = Y
        self.Xbar[:] = Xbar
        self.c.sum_sq = float(sum_sq)
        self.c.gamma = float(gamma)
        self.c.t = int(t)


def eg_step(state, op, noise_t, noise_half, bucket, levels, cb, seed, norm_type=L2, quantizer_off=False,
            refit=0, code_type=CODE_FIXED, nbins=1024):
    """One iteration; levels (float32 array) and cb are updated in place when refit != 0. Returns bits sent."""
    n1 = _f32(noise_t) if noise_t is not None else None
    n2 = _f32(noise_half) if noise_half is not None else None
    assert levels.dtype == np.float32 and levels.flags.c_contiguous
    bits = C.c_uint64(0)
    _chk(lib().qgxo_eg_step(C.byref(state.c), C.byref(op.c), _p(n1), _p(n2), bucket, norm_type,
                            _p(levels), len(levels), C.byref(cb), C.c_uint64(seed), int(quantizer_off),
                            int(refit), int(code_type), int(nbins), C.byref(bits)), "eg_step")
    return bits.value


def eg_step_two_tables(state, op, noise_t, noise_half, bucket, levels_t, cb_t, levels_h, cb_h, seed, norm_type=L2,
                       quantizer_off=False, refit=0, code_type=CODE_FIXED, nbins=1024):
    """One iteration with a level table and code of its own for each of the two exchanges; both are updated in place
    when refit != 0. Returns bits sent."""
    n1 = _f32(noise_t) if noise_t is not None else None
    n2 = _f32(noise_half) if noise_half is not None else None
    for lv in (levels_t, levels_h):
        assert lv.dtype == np.float32 and lv.flags.c_contiguous
    bits = C.c_uint64(0)
    _chk(lib().qgxo_eg_step_two_tables(C.byref(state.c), C.byref(op.c), _p(n1), _p(n2), bucket, norm_type,
                                       _p(levels_t), len(levels_t), C.byref(cb_t), _p(levels_h), len(levels_h),
                                       C.byref(cb_h), C.c_uint64(seed), int(quantizer_off), int(refit), int(code_type),
                                       int(nbins), C.byref(bits)), "eg_step_two_tables")
    return bits.value


METHOD_DE, METHOD_DA, METHOD_OPTDA = 0, 1, 2


def family_step(state, method, op, noise, bucket, levels, cb, seed, g_prev=None, mean_prev=None, norm_type=L2,
                quantizer_off=False, refit=0, code_type=CODE_FIXED, nbins=1024):
    """One iteration of quantized dual averaging (METHOD_DA) or optimistic dual averaging (METHOD_OPTDA);
    g_prev [K, d] and mean_prev [d] (float32, OptDA) are updated in place. Returns bits sent."""
    nz = _f32(noise) if noise is not None else None
    assert levels.dtype == np.float32 and levels.flags.c_contiguous
    for arr in (g_prev, mean_prev):
        assert arr is None or (arr.dtype == np.float32 and arr.flags.c_contiguous)
    bits = C.c_uint64(0)
    _chk(lib().qgxo_family_step(C.byref(state.c), int(method), C.byref(op.c), _p(nz), bucket, norm_type,
                                _p(levels), len(levels), C.byref(cb), C.c_uint64(seed), int(quantizer_off),
                                int(refit), int(code_type), int(nbins), _p(g_prev), _p(mean_prev), C.byref(bits)),
         "family_step")
    return bits.value


def exchange(v, bucket, levels, cb, seed, xid, norm_type=L2, return_vhat=False):
    """quantize -> encode -> decode -> average of v[K, d]; returns (mean, total_bits[K]) (+ vhat)."""
    v = _f32(v)
    lv = _f32(levels)
    K, d = v.shape
    mean = np.zeros(d, dtype=np.float32)
    total = np.zeros(K, dtype=np.uint64)
    vhat = np.zeros((K, d), dtype=np.float32) if return_vhat else None
    _chk(lib().qgxo_exchange_full(_p(v), K, C.c_uint64(d), bucket, norm_type, _p(lv), len(lv), C.byref(cb),
                                  C.c_uint64(seed), C.c_uint32(xid), 0, _p(vhat), _p(mean), _p(total)), "exchange")
    if return_vhat:
        return mean, total, vhat
    return mean, total
