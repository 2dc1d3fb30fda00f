"""numpy-facing wrappers around the C oracle (oracle/amq_oracle.c).

TEST INFRASTRUCTURE ONLY: imported by tests/, by the smoke check and by the CPU-baseline leg of the
benchmark.  Nothing in the CUDA library or its Python binding imports this package, and this package
imports nothing from them.  All arithmetic lives in the C file; this module only marshals arrays.

Array conventions: planes are int8 arrays of +1/-1 with shape (k, n); packed codes are uint32 arrays of
shape (rows, k, wpr) with wpr = 4 * ceil(n / 128); coefficients are float64.
"""
import ctypes

import numpy as np

from . import build as _build

_lib = ctypes.CDLL(_build.build())

_dp = ctypes.POINTER(ctypes.c_double)
_i8p = ctypes.POINTER(ctypes.c_int8)
_u32p = ctypes.POINTER(ctypes.c_uint32)
_i32p = ctypes.POINTER(ctypes.c_int32)
_ip = ctypes.POINTER(ctypes.c_int)
_int = ctypes.c_int


def _sig(name, restype, *argtypes):
    fn = getattr(_lib, name)
    fn.restype = restype
    fn.argtypes = list(argtypes)
    return fn


_greedy = _sig("amq_oracle_greedy", None, _dp, _int, _int, _dp, _i8p)
_ls = _sig("amq_oracle_ls_refit", _int, _dp, _int, _int, _i8p, _dp)
_levels = _sig("amq_oracle_levels", None, _dp, _int, _dp, _ip)
_bst = _sig("amq_oracle_bst", None, _dp, _int, _int, _dp, _i8p)
_obj = _sig("amq_oracle_objective", ctypes.c_double, _dp, _int, _int, _dp, _i8p)
_quant = _sig("amq_oracle_quantize", None, _dp, _int, _int, _int, _dp, _i8p, _dp)
_refined = _sig("amq_oracle_refined_greedy", None, _dp, _int, _int, _dp, _i8p)
_qvar = _sig("amq_oracle_quantize_variant", None, _dp, _int, _int, _int, _int, _int, _dp, _i8p)
_qrows_var = _sig("amq_oracle_quantize_rows_variant", None, _dp, _int, _int, _int, _int, _int, _int, _int, _u32p, _dp)
_wpr = _sig("amq_oracle_words_per_row", _int, _int)
_pack = _sig("amq_oracle_pack_plane", None, _i8p, _int, _u32p)
_unpack = _sig("amq_oracle_unpack_plane", None, _u32p, _int, _i8p)
_dotx = _sig("amq_oracle_dot_xnor", ctypes.c_int32, _u32p, _u32p, _int)
_dotxr = _sig("amq_oracle_dot_xnor_range", ctypes.c_int32, _u32p, _u32p, _int, _int)
_dotpm = _sig("amq_oracle_dot_pm1", ctypes.c_double, _i8p, _i8p, _int)
_qrows = _sig("amq_oracle_quantize_rows", None, _dp, _int, _int, _int, _int, _int, _u32p, _dp)
_dots = _sig("amq_oracle_binary_dots_range", None, _u32p, _int, _int, _int, _u32p, _int, _int, _int, _int, _i32p)
_gemm = _sig("amq_oracle_binary_gemm_range", None, _u32p, _dp, _int, _int, _int, _u32p, _dp, _int, _int,
             _dp, _int, _int, _dp)
_lstm = _sig("amq_oracle_lstm_step", None, _u32p, _dp, _dp, _int, _int, _int, _dp, _dp, _dp, _int, _int, _int,
             _dp, _dp)
_lstm_paper = _sig("amq_oracle_lstm_step_paper", None, _u32p, _dp, _u32p, _dp, _dp, _int, _int, _int, _u32p, _dp, _int,
                   _dp, _dp, _int, _int, _int, _dp, _dp)
_lsm = _sig("amq_oracle_log_softmax_argmax", None, _dp, _int, _int, _dp, _i32p)
_gru = _sig("amq_oracle_gru_step", None, _u32p, _dp, _dp, _int, _int, _int, _dp, _dp, _int, _int, _int, _dp)
_gru_orig = _sig("amq_oracle_gru_step_original", None, _u32p, _dp, _dp, _int, _int, _int, _dp, _dp, _int, _int, _int, _dp)
_lstm_seq = _sig("amq_oracle_lstm_sequence", None, _u32p, _dp, _dp, _int, _int, _int, _dp, _int, _dp, _dp,
                 _int, _int, _int, _dp, _dp, _dp)
_gru_seq = _sig("amq_oracle_gru_sequence", None, _u32p, _dp, _dp, _int, _int, _int, _dp, _int, _dp,
                _int, _int, _int, _dp, _dp)
_qops = _sig("amq_oracle_quantizer_ops", None, _int, _int, _int, _dp, _dp)
_gamma = _sig("amq_oracle_gamma", ctypes.c_double, _int, _int, _int, _int)


def _d(a):
    return np.ascontiguousarray(a, dtype=np.float64)


def _p(a, t):
    return None if a is None else a.ctypes.data_as(t)


def words_per_row(n):
    return int(_wpr(int(n)))


def greedy(w, k):
    w = _d(w).ravel()
    n = w.size
    alpha = np.zeros(k)
    b = np.zeros((k, n), dtype=np.int8)
    _greedy(_p(w, _dp), n, k, _p(alpha, _dp), _p(b, _i8p))
    return alpha, b


def ls_refit(w, b, alpha_prev=None):
    """Returns (alpha, solved).  When the system is singular alpha_prev comes back unchanged."""
    w = _d(w).ravel()
    b = np.ascontiguousarray(b, dtype=np.int8)
    k, n = b.shape
    alpha = np.zeros(k) if alpha_prev is None else _d(alpha_prev).copy()
    ok = _ls(_p(w, _dp), n, k, _p(b, _i8p), _p(alpha, _dp))
    return alpha, bool(ok)


def levels(alpha):
    alpha = _d(alpha).ravel()
    k = alpha.size
    v = np.zeros(1 << k)
    code = np.zeros(1 << k, dtype=np.intc)
    _levels(_p(alpha, _dp), k, _p(v, _dp), _p(code, _ip))
    return v, code


def bst(w, alpha):
    w = _d(w).ravel()
    alpha = _d(alpha).ravel()
    k, n = alpha.size, w.size
    b = np.zeros((k, n), dtype=np.int8)
    _bst(_p(w, _dp), n, k, _p(alpha, _dp), _p(b, _i8p))
    return b


def objective(w, alpha, b):
    w = _d(w).ravel()
    alpha = _d(alpha).ravel()
    b = np.ascontiguousarray(b, dtype=np.int8)
    return float(_obj(_p(w, _dp), w.size, alpha.size, _p(alpha, _dp), _p(b, _i8p)))


def quantize(w, k, T, with_trace=False):
    w = _d(w).ravel()
    n = w.size
    alpha = np.zeros(k)
    b = np.zeros((k, n), dtype=np.int8)
    trace = np.zeros(1 + 2 * T) if with_trace else None
    _quant(_p(w, _dp), n, k, T, _p(alpha, _dp), _p(b, _i8p), _p(trace, _dp))
    return (alpha, b, trace) if with_trace else (alpha, b)


def refined_greedy(w, k):
    w = _d(w).ravel()
    n = w.size
    alpha = np.zeros(k)
    b = np.zeros((k, n), dtype=np.int8)
    _refined(_p(w, _dp), n, k, _p(alpha, _dp), _p(b, _i8p))
    return alpha, b


METHOD_ALTERNATING, METHOD_REFINED_GREEDY = 0, 1


def quantize_variant(w, k, T, method=METHOD_ALTERNATING, final_refit=False):
    w = _d(w).ravel()
    n = w.size
    alpha = np.zeros(k)
    b = np.zeros((k, n), dtype=np.int8)
    _qvar(_p(w, _dp), n, k, T, method, int(final_refit), _p(alpha, _dp), _p(b, _i8p))
    return alpha, b


def quantize_rows_variant(x, k, T, method=METHOD_ALTERNATING, final_refit=False):
    """x (rows, n) -> codes (rows, k, wpr) uint32, coeffs (rows, k) float64."""
    x = _d(x)
    rows, n = x.shape
    codes = np.zeros((rows, k, words_per_row(n)), dtype=np.uint32)
    coeffs = np.zeros((rows, k))
    _qrows_var(_p(x, _dp), rows, n, n, k, T, method, int(final_refit), _p(codes, _u32p), _p(coeffs, _dp))
    return codes, coeffs


def pack_plane(b):
    b = np.ascontiguousarray(b, dtype=np.int8).ravel()
    words = np.zeros(words_per_row(b.size), dtype=np.uint32)
    _pack(_p(b, _i8p), b.size, _p(words, _u32p))
    return words


def pack_planes(b):
    """(k, n) planes -> (k, wpr) words."""
    return np.stack([pack_plane(p) for p in np.asarray(b)])


def unpack_plane(words, n):
    words = np.ascontiguousarray(words, dtype=np.uint32)
    b = np.zeros(n, dtype=np.int8)
    _unpack(_p(words, _u32p), n, _p(b, _i8p))
    return b


def dot_xnor(a_words, b_words, n, lo=None, hi=None):
    a = np.ascontiguousarray(a_words, dtype=np.uint32)
    b = np.ascontiguousarray(b_words, dtype=np.uint32)
    if lo is None:
        return int(_dotx(_p(a, _u32p), _p(b, _u32p), n))
    return int(_dotxr(_p(a, _u32p), _p(b, _u32p), lo, hi))


def dot_pm1(a, b):
    a = np.ascontiguousarray(a, dtype=np.int8).ravel()
    b = np.ascontiguousarray(b, dtype=np.int8).ravel()
    return float(_dotpm(_p(a, _i8p), _p(b, _i8p), a.size))


def quantize_rows(x, k, T):
    """x (rows, n) -> codes (rows, k, wpr) uint32, coeffs (rows, k) float64."""
    x = _d(x)
    rows, n = x.shape
    codes = np.zeros((rows, k, words_per_row(n)), dtype=np.uint32)
    coeffs = np.zeros((rows, k))
    _qrows(_p(x, _dp), rows, n, n, k, T, _p(codes, _u32p), _p(coeffs, _dp))
    return codes, coeffs


def binary_dots(Wcodes, xcodes, n, lo=0, hi=None):
    """D[batch][m][k_w][k_a] int32 over columns [lo, hi)."""
    Wc = np.ascontiguousarray(Wcodes, dtype=np.uint32)
    xc = np.ascontiguousarray(xcodes, dtype=np.uint32)
    m, k_w, _ = Wc.shape
    batch, k_a, _ = xc.shape
    hi = n if hi is None else hi
    D = np.zeros((batch, m, k_w, k_a), dtype=np.int32)
    _dots(_p(Wc, _u32p), m, n, k_w, _p(xc, _u32p), batch, k_a, lo, hi, _p(D, _i32p))
    return D


def binary_gemm(Wcodes, Walpha, xcodes, xbeta, n, bias=None, lo=0, hi=None):
    """y[batch][m] float64."""
    Wc = np.ascontiguousarray(Wcodes, dtype=np.uint32)
    xc = np.ascontiguousarray(xcodes, dtype=np.uint32)
    Wa, xb = _d(Walpha), _d(xbeta)
    m, k_w, _ = Wc.shape
    batch, k_a, _ = xc.shape
    hi = n if hi is None else hi
    bias = None if bias is None else _d(bias)
    y = np.zeros((batch, m))
    _gemm(_p(Wc, _u32p), _p(Wa, _dp), m, n, k_w, _p(xc, _u32p), _p(xb, _dp), batch, k_a,
          _p(bias, _dp), lo, hi, _p(y, _dp))
    return y


def lstm_step(Wcodes, Walpha, bias, I, H, x, h, c, k_a, T):
    Wc = np.ascontiguousarray(Wcodes, dtype=np.uint32)
    Wa = _d(Walpha)
    k_w = Wc.shape[1]
    x, h, c = _d(x), _d(h), _d(c)
    batch = x.shape[0]
    bias = None if bias is None else _d(bias)
    h_out, c_out = np.zeros((batch, H)), np.zeros((batch, H))
    _lstm(_p(Wc, _u32p), _p(Wa, _dp), _p(bias, _dp), I, H, k_w, _p(x, _dp), _p(h, _dp), _p(c, _dp),
          batch, k_a, T, _p(h_out, _dp), _p(c_out, _dp))
    return h_out, c_out


def lstm_step_paper(Wi_codes, Wi_alpha, Wh_codes, Wh_alpha, bias, I, H, xcodes, xbeta, h, c, k_a, T):
    """The step as the paper states it: separate W_i / W_h, x given as packed codes (an embedding row), h quantized on-line."""
    Wic = np.ascontiguousarray(Wi_codes, dtype=np.uint32)
    Whc = np.ascontiguousarray(Wh_codes, dtype=np.uint32)
    xc = np.ascontiguousarray(xcodes, dtype=np.uint32)
    Wia, Wha, xb, h, c = _d(Wi_alpha), _d(Wh_alpha), _d(xbeta), _d(h), _d(c)
    k_w, (batch, k_e, _) = Wic.shape[1], xc.shape
    bias = None if bias is None else _d(bias)
    h_out, c_out = np.zeros((batch, H)), np.zeros((batch, H))
    _lstm_paper(_p(Wic, _u32p), _p(Wia, _dp), _p(Whc, _u32p), _p(Wha, _dp), _p(bias, _dp), I, H, k_w,
                _p(xc, _u32p), _p(xb, _dp), k_e, _p(h, _dp), _p(c, _dp), batch, k_a, T, _p(h_out, _dp), _p(c_out, _dp))
    return h_out, c_out


def log_softmax_argmax(z):
    """(rows, n) logits -> (log-probabilities (rows, n) float64, argmax (rows,) int32)."""
    z = _d(z)
    rows, n = z.shape
    logp = np.zeros((rows, n))
    arg = np.zeros(rows, dtype=np.int32)
    _lsm(_p(z, _dp), rows, n, _p(logp, _dp), _p(arg, _i32p))
    return logp, arg


def gru_step(Wcodes, Walpha, bias, I, H, x, h, k_a, T):
    Wc = np.ascontiguousarray(Wcodes, dtype=np.uint32)
    Wa = _d(Walpha)
    k_w = Wc.shape[1]
    x, h = _d(x), _d(h)
    batch = x.shape[0]
    bias = None if bias is None else _d(bias)
    h_out = np.zeros((batch, H))
    _gru(_p(Wc, _u32p), _p(Wa, _dp), _p(bias, _dp), I, H, k_w, _p(x, _dp), _p(h, _dp),
         batch, k_a, T, _p(h_out, _dp))
    return h_out


def gru_step_original(Wcodes, Walpha, bias, I, H, x, h, k_a, T):
    """The GRU in its original form (reset gate applied to h before the candidate's product; bias (3H,) or None)."""
    Wc = np.ascontiguousarray(Wcodes, dtype=np.uint32)
    Wa, x, h = _d(Walpha), _d(x), _d(h)
    batch, k_w = x.shape[0], Wc.shape[1]
    bias = None if bias is None else _d(bias)
    h_out = np.zeros((batch, H))
    _gru_orig(_p(Wc, _u32p), _p(Wa, _dp), _p(bias, _dp), I, H, k_w, _p(x, _dp), _p(h, _dp), batch, k_a, T, _p(h_out, _dp))
    return h_out


def lstm_sequence(Wcodes, Walpha, bias, I, H, x_seq, h0, c0, k_a, T):
    Wc = np.ascontiguousarray(Wcodes, dtype=np.uint32)
    Wa = _d(Walpha)
    k_w = Wc.shape[1]
    x_seq, h0, c0 = _d(x_seq), _d(h0), _d(c0)
    steps, batch, _ = x_seq.shape
    bias = None if bias is None else _d(bias)
    h_seq = np.zeros((steps, batch, H))
    h_last, c_last = np.zeros((batch, H)), np.zeros((batch, H))
    _lstm_seq(_p(Wc, _u32p), _p(Wa, _dp), _p(bias, _dp), I, H, k_w, _p(x_seq, _dp), steps, _p(h0, _dp),
              _p(c0, _dp), batch, k_a, T, _p(h_seq, _dp), _p(h_last, _dp), _p(c_last, _dp))
    return h_seq, h_last, c_last


def gru_sequence(Wcodes, Walpha, bias, I, H, x_seq, h0, k_a, T):
    Wc = np.ascontiguousarray(Wcodes, dtype=np.uint32)
    Wa = _d(Walpha)
    k_w = Wc.shape[1]
    x_seq, h0 = _d(x_seq), _d(h0)
    steps, batch, _ = x_seq.shape
    bias = None if bias is None else _d(bias)
    h_seq = np.zeros((steps, batch, H))
    h_last = np.zeros((batch, H))
    _gru_seq(_p(Wc, _u32p), _p(Wa, _dp), _p(bias, _dp), I, H, k_w, _p(x_seq, _dp), steps, _p(h0, _dp),
             batch, k_a, T, _p(h_seq, _dp), _p(h_last, _dp))
    return h_seq, h_last


def quantizer_ops(n, k, T):
    b, nb = ctypes.c_double(), ctypes.c_double()
    _qops(n, k, T, ctypes.byref(b), ctypes.byref(nb))
    return b.value, nb.value


def gamma(m, n, k_w, k_h):
    return float(_gamma(m, n, k_w, k_h))


def reconstruct(alpha, b):
    """sum_i alpha_i b_i as float64 (marshalling helper for tests: no method arithmetic beyond Eq. 2)."""
    return (np.asarray(alpha, dtype=np.float64)[:, None] * np.asarray(b, dtype=np.float64)).sum(axis=0)
