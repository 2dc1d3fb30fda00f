"""Python binding of the C ABI in include/amq.h (same names, argument marshalling only).

PyTorch supplies device memory and the current stream; every step of the path runs in the CUDA
library.  Importing this module loads paper_1802_00150_b200/libamq_b200.so and raises if it is missing:
there is no CPU fallback.
"""
import ctypes
import os

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
# the product library; AMQ_B200_LIBRARY names an instrumented build of the same sources instead (see build.py)
LIB_PATH = os.environ.get("AMQ_B200_LIBRARY") or os.path.join(_HERE, "libamq_b200.so")

if not os.path.exists(LIB_PATH):
    raise ImportError(
        "CUDA library %s is missing: build it with `python -m paper_1802_00150_b200.build` "
        "(there is no CPU fallback)" % LIB_PATH)

_lib = ctypes.CDLL(LIB_PATH)

OK = 0
MAX_K = 4
MAX_N = 8192

_vp, _int, _sz = ctypes.c_void_p, ctypes.c_int, ctypes.c_size_t

EXPORTS = {
    "amq_status_string": (ctypes.c_char_p, [_int]),
    "amq_last_cuda_error": (_int, []),
    "amq_kernel_launches": (ctypes.c_ulonglong, []),
    "amq_words_per_row": (_int, [_int]),
    "amq_codes_bytes": (_sz, [_int, _int, _int]),
    "amq_quantize": (_int, [_vp, _int, _int, _int, _int, _int, _vp, _vp, _vp]),
    "amq_pack": (_int, [_vp, _int, _int, _int, _vp, _vp]),
    "amq_unpack": (_int, [_vp, _vp, _int, _int, _int, _vp, _vp]),
    "amq_binary_dots": (_int, [_vp, _int, _int, _int, _vp, _int, _int, _vp, _vp]),
    "amq_binary_gemm": (_int, [_vp, _vp, _int, _int, _int, _vp, _vp, _int, _int, _vp, _vp, _int, _vp]),
    "amq_quantized_gemv": (_int, [_vp, _vp, _int, _int, _int, _vp, _int, _int, _vp, _vp, _vp, _vp, _vp]),
    "amq_device_status": (_int, [_vp]),
    "amq_cell_workspace_bytes": (_sz, [_int, _int, _int, _int]),
    "amq_cell_host_staging_bytes": (_sz, [_int, _int, _int, _int]),
    "amq_lstm_step": (_int, [_vp, _vp, _vp, _int, _int, _int, _vp, _vp, _vp, _int, _int, _int, _vp, _vp, _vp, _sz, _vp]),
    "amq_lstm_step_static_scratch_bytes": (_sz, [_int, _int, _int, _int]),
    "amq_lstm_step_static": (_int, [_vp, _vp, _vp, _int, _int, _int, _vp, _vp, _vp, _int, _int, _int, _vp, _vp, _vp]),
    "amq_gru_step": (_int, [_vp, _vp, _vp, _int, _int, _int, _vp, _vp, _int, _int, _int, _vp, _vp, _sz, _vp]),
    "amq_lstm_sequence": (_int, [_vp, _vp, _vp, _int, _int, _int, _vp, _int, _vp, _vp, _int, _int, _int,
                                 _vp, _vp, _vp, _vp, _sz, _vp]),
    "amq_gru_sequence": (_int, [_vp, _vp, _vp, _int, _int, _int, _vp, _int, _vp, _int, _int, _int,
                                _vp, _vp, _vp, _sz, _vp]),
    "amq_lstm_sequence_host": (_int, [_vp, _vp, _vp, _int, _int, _int, _vp, _int, _vp, _vp, _int, _int, _int,
                                      _vp, _vp, _vp, _vp, _sz, _vp, _sz, _vp]),
    "amq_gru_sequence_host": (_int, [_vp, _vp, _vp, _int, _int, _int, _vp, _int, _vp, _int, _int, _int,
                                     _vp, _vp, _vp, _sz, _vp, _sz, _vp]),
    "amq_workspace_status": (_int, [_vp, _vp]),
    "amq_selftest_sequence_give_up": (_int, [_vp, _vp, _vp, _int, _int, _int, _vp, _int, _vp, _vp, _int, _int,
                                             _vp, _vp, _vp, _sz, ctypes.c_uint, _vp]),
    "amq_gru_original_workspace_bytes": (_sz, [_int, _int, _int, _int]),
    "amq_gru_step_original": (_int, [_vp, _vp, _vp, _int, _int, _int, _vp, _vp, _int, _int, _int, _vp, _vp, _sz, _vp]),
    "amq_quantize_variant": (_int, [_vp, _int, _int, _int, _int, _int, _int, _int, _vp, _vp, _vp]),
    "amq_lm_decode_workspace_bytes": (_sz, [_int, _int, _int, _int, _int]),
    "amq_lm_greedy_decode": (_int, [_vp, _vp, _int, _int, _int, _vp, _vp, _vp, _vp, _vp, _int, _int, _vp, _vp, _vp, _int,
                                    _int, _int, _vp, _int, _vp, _vp, _vp, _vp, _sz, _vp]),
    "amq_log_softmax_argmax": (_int, [_vp, _int, _int, _int, _vp, _int, _vp, _vp]),
    "amq_embedding_rows": (_int, [_vp, _vp, _int, _int, _int, _vp, _int, _vp, _vp, _vp]),
    "amq_lstm_paper_workspace_bytes": (_sz, [_int, _int, _int, _int]),
    "amq_lstm_step_paper": (_int, [_vp, _vp, _vp, _vp, _vp, _int, _int, _int, _vp, _vp, _int, _vp, _vp, _int, _int, _int,
                                   _vp, _vp, _vp, _sz, _vp]),
    "amq_lstm_sequence_paper": (_int, [_vp, _vp, _vp, _vp, _vp, _int, _int, _int, _vp, _vp, _int, _int, _vp, _vp, _int, _int,
                                       _int, _vp, _vp, _vp, _vp, _sz, _vp]),
}

for _name, (_res, _args) in EXPORTS.items():
    _fn = getattr(_lib, _name)
    _fn.restype = _res
    _fn.argtypes = _args


class AmqError(RuntimeError):
    def __init__(self, status):
        self.status = status
        msg = _lib.amq_status_string(status).decode()
        if status == -5:
            msg += " (cudaError %d)" % _lib.amq_last_cuda_error()
        super().__init__("amq status %d: %s" % (status, msg))


def _check(status):
    if status != OK:
        raise AmqError(status)


def _ptr(t):
    return None if t is None else t.data_ptr()


def _stream():
    return torch.cuda.current_stream().cuda_stream


def _dev(t, dtype, name):
    if t is None:
        return None
    if not (isinstance(t, torch.Tensor) and t.is_cuda and t.dtype == dtype and t.is_contiguous()):
        raise TypeError("%s must be a contiguous CUDA tensor of dtype %s" % (name, dtype))
    return t


def status_string(status):
    return _lib.amq_status_string(status).decode()


def kernel_launches():
    return int(_lib.amq_kernel_launches())


def words_per_row(n):
    return _lib.amq_words_per_row(n)


def codes_bytes(rows, n, k):
    return _lib.amq_codes_bytes(rows, n, k)


def _new_codes(rows, k, n, device):
    return torch.empty((rows, k, words_per_row(n)), dtype=torch.int32, device=device)


def quantize(x, k, T, codes=None, coeffs=None):
    """x (rows, n) fp32, possibly a row-strided view -> codes (rows, k, wpr) int32, coeffs (rows, k) fp32."""
    if not (x.is_cuda and x.dtype == torch.float32 and x.dim() == 2 and x.stride(1) == 1):
        raise TypeError("x must be a 2-D CUDA fp32 tensor with unit column stride")
    rows, n = x.shape
    ldx = x.stride(0) if rows > 1 else max(n, x.stride(0))
    codes = _new_codes(rows, k, n, x.device) if codes is None else _dev(codes, torch.int32, "codes")
    coeffs = torch.empty((rows, k), dtype=torch.float32, device=x.device) if coeffs is None else _dev(coeffs, torch.float32, "coeffs")
    _check(_lib.amq_quantize(_ptr(x), rows, n, ldx, k, T, _ptr(codes), _ptr(coeffs), _stream()))
    return codes, coeffs


def pack(planes):
    """planes (rows, k, n) fp32 (>= 0 -> +1) -> codes (rows, k, wpr) int32."""
    planes = _dev(planes, torch.float32, "planes")
    rows, k, n = planes.shape
    codes = _new_codes(rows, k, n, planes.device)
    _check(_lib.amq_pack(_ptr(planes), rows, n, k, _ptr(codes), _stream()))
    return codes


def unpack(codes, coeffs, n):
    codes, coeffs = _dev(codes, torch.int32, "codes"), _dev(coeffs, torch.float32, "coeffs")
    rows, k, _ = codes.shape
    xhat = torch.empty((rows, n), dtype=torch.float32, device=codes.device)
    _check(_lib.amq_unpack(_ptr(codes), _ptr(coeffs), rows, n, k, _ptr(xhat), _stream()))
    return xhat


def binary_dots(Wcodes, xcodes, n):
    """-> D (batch, m, k_w, k_a) int32."""
    Wcodes, xcodes = _dev(Wcodes, torch.int32, "Wcodes"), _dev(xcodes, torch.int32, "xcodes")
    m, k_w, _ = Wcodes.shape
    batch, k_a, _ = xcodes.shape
    D = torch.empty((batch, m, k_w, k_a), dtype=torch.int32, device=Wcodes.device)
    _check(_lib.amq_binary_dots(_ptr(Wcodes), m, n, k_w, _ptr(xcodes), batch, k_a, _ptr(D), _stream()))
    return D


def binary_gemm(Wcodes, Walpha, xcodes, xbeta, n, bias=None, y=None):
    """-> y (batch, m) fp32."""
    Wcodes, xcodes = _dev(Wcodes, torch.int32, "Wcodes"), _dev(xcodes, torch.int32, "xcodes")
    Walpha, xbeta = _dev(Walpha, torch.float32, "Walpha"), _dev(xbeta, torch.float32, "xbeta")
    bias = _dev(bias, torch.float32, "bias")
    m, k_w, _ = Wcodes.shape
    batch, k_a, _ = xcodes.shape
    if y is None:
        y = torch.empty((batch, m), dtype=torch.float32, device=Wcodes.device)
    _check(_lib.amq_binary_gemm(_ptr(Wcodes), _ptr(Walpha), m, n, k_w, _ptr(xcodes), _ptr(xbeta), batch, k_a,
                                _ptr(bias), _ptr(y), y.stride(0) if batch > 1 else max(m, y.stride(0)), _stream()))
    return y


def quantized_gemv(Wcodes, Walpha, x, k_a, T, bias=None, y=None, want_codes=False):
    """Table 6's operation in one launch: x (n,) or (1, n) fp32 is quantized on-line (k_a bits, T cycles) inside the
    product kernel.  Returns y (m,), or (y, xcodes (k_a, wpr), xbeta (k_a,)) with want_codes."""
    Wcodes, Walpha = _dev(Wcodes, torch.int32, "Wcodes"), _dev(Walpha, torch.float32, "Walpha")
    x = _dev(x, torch.float32, "x")
    m, k_w, wpr = Wcodes.shape
    n = x.numel()
    if y is None:
        y = torch.empty((m,), dtype=torch.float32, device=x.device)
    xc = torch.empty((k_a, wpr), dtype=torch.int32, device=x.device) if want_codes else None
    xb = torch.empty((k_a,), dtype=torch.float32, device=x.device) if want_codes else None
    _check(_lib.amq_quantized_gemv(_ptr(Wcodes), _ptr(Walpha), m, n, k_w, _ptr(x), k_a, T, _ptr(bias), _ptr(y),
                                   _ptr(xc), _ptr(xb), _stream()))
    return (y, xc, xb) if want_codes else y


def device_status():
    """0, or -6 when a bounded device-side wait of a product kernel ran out since the last call."""
    return _lib.amq_device_status(_stream())


def cell_workspace_bytes(I, H, batch, k_a):
    return _lib.amq_cell_workspace_bytes(I, H, batch, k_a)


def cell_host_staging_bytes(I, H, batch, steps):
    return _lib.amq_cell_host_staging_bytes(I, H, batch, steps)


def new_workspace(I, H, batch, k_a, device="cuda"):
    return torch.zeros(max(cell_workspace_bytes(I, H, batch, k_a), 16), dtype=torch.uint8, device=device)


def new_host_staging(I, H, batch, steps, device="cuda"):
    return torch.empty(max(cell_host_staging_bytes(I, H, batch, steps), 16), dtype=torch.uint8, device=device)


def lstm_step(Wcodes, Walpha, bias, I, H, x, h_in, c_in, k_a, T, workspace, h_out=None, c_out=None):
    Wcodes, Walpha = _dev(Wcodes, torch.int32, "Wcodes"), _dev(Walpha, torch.float32, "Walpha")
    x, h_in, c_in = _dev(x, torch.float32, "x"), _dev(h_in, torch.float32, "h_in"), _dev(c_in, torch.float32, "c_in")
    batch, k_w = h_in.shape[0], Wcodes.shape[1]
    h_out = torch.empty_like(h_in) if h_out is None else h_out
    c_out = torch.empty_like(c_in) if c_out is None else c_out
    _check(_lib.amq_lstm_step(_ptr(Wcodes), _ptr(Walpha), _ptr(bias), I, H, k_w, _ptr(x), _ptr(h_in), _ptr(c_in),
                              batch, k_a, T, _ptr(h_out), _ptr(c_out), _ptr(workspace), workspace.numel(), _stream()))
    return h_out, c_out


STATIC_SCRATCH_BYTES = 1 << 20


def lstm_step_static_scratch_bytes(I, H, batch, k_a):
    return _lib.amq_lstm_step_static_scratch_bytes(I, H, batch, k_a)


def lstm_step_static(Wcodes, Walpha, bias, I, H, x, h_in, c_in, k_a, T, h_out, c_out):
    """amq_lstm_step without a workspace: the library's built-in scratch array is used, and neither this
    wrapper nor the call allocates (the caller brings h_out and c_out).  Problems whose scratch exceeds
    STATIC_SCRATCH_BYTES raise AmqError(-4)."""
    Wcodes, Walpha = _dev(Wcodes, torch.int32, "Wcodes"), _dev(Walpha, torch.float32, "Walpha")
    x, h_in, c_in = _dev(x, torch.float32, "x"), _dev(h_in, torch.float32, "h_in"), _dev(c_in, torch.float32, "c_in")
    h_out, c_out = _dev(h_out, torch.float32, "h_out"), _dev(c_out, torch.float32, "c_out")
    batch, k_w = h_in.shape[0], Wcodes.shape[1]
    _check(_lib.amq_lstm_step_static(_ptr(Wcodes), _ptr(Walpha), _ptr(bias), I, H, k_w, _ptr(x), _ptr(h_in),
                                     _ptr(c_in), batch, k_a, T, _ptr(h_out), _ptr(c_out), _stream()))
    return h_out, c_out


def gru_step(Wcodes, Walpha, bias, I, H, x, h_in, k_a, T, workspace, h_out=None):
    Wcodes, Walpha = _dev(Wcodes, torch.int32, "Wcodes"), _dev(Walpha, torch.float32, "Walpha")
    x, h_in = _dev(x, torch.float32, "x"), _dev(h_in, torch.float32, "h_in")
    batch, k_w = h_in.shape[0], Wcodes.shape[1]
    h_out = torch.empty_like(h_in) if h_out is None else h_out
    _check(_lib.amq_gru_step(_ptr(Wcodes), _ptr(Walpha), _ptr(bias), I, H, k_w, _ptr(x), _ptr(h_in),
                             batch, k_a, T, _ptr(h_out), _ptr(workspace), workspace.numel(), _stream()))
    return h_out


def lstm_sequence(Wcodes, Walpha, bias, I, H, x_seq, h0, c0, k_a, T, workspace, want_h_seq=False,
                  h_seq=None, h_last=None, c_last=None):
    Wcodes, Walpha = _dev(Wcodes, torch.int32, "Wcodes"), _dev(Walpha, torch.float32, "Walpha")
    x_seq, h0, c0 = _dev(x_seq, torch.float32, "x_seq"), _dev(h0, torch.float32, "h0"), _dev(c0, torch.float32, "c0")
    steps, batch, k_w = x_seq.shape[0], h0.shape[0], Wcodes.shape[1]
    if want_h_seq and h_seq is None:
        h_seq = torch.empty((steps, batch, H), dtype=torch.float32, device=h0.device)
    h_last = torch.empty_like(h0) if h_last is None else h_last
    c_last = torch.empty_like(c0) if c_last is None else c_last
    _check(_lib.amq_lstm_sequence(_ptr(Wcodes), _ptr(Walpha), _ptr(bias), I, H, k_w, _ptr(x_seq), steps, _ptr(h0),
                                  _ptr(c0), batch, k_a, T, _ptr(h_seq), _ptr(h_last), _ptr(c_last),
                                  _ptr(workspace), workspace.numel(), _stream()))
    return h_seq, h_last, c_last


def selftest_sequence_give_up(Wcodes, Walpha, bias, I, H, x_seq, h0, c0, k_a, T, workspace, poll_limit):
    """Test aid: the batch-1 LSTM sequence kernel with waits that run out (see amq.h).  Returns (h_last, c_last),
    which the kernel leaves unwritten; read the outcome with workspace_status."""
    Wcodes, Walpha = _dev(Wcodes, torch.int32, "Wcodes"), _dev(Walpha, torch.float32, "Walpha")
    x_seq, h0, c0 = _dev(x_seq, torch.float32, "x_seq"), _dev(h0, torch.float32, "h0"), _dev(c0, torch.float32, "c0")
    h_last, c_last = torch.zeros_like(h0), torch.zeros_like(c0)
    _check(_lib.amq_selftest_sequence_give_up(_ptr(Wcodes), _ptr(Walpha), _ptr(bias), I, H, Wcodes.shape[1], _ptr(x_seq),
                                              x_seq.shape[0], _ptr(h0), _ptr(c0), k_a, T, _ptr(h_last), _ptr(c_last),
                                              _ptr(workspace), workspace.numel(), poll_limit, _stream()))
    return h_last, c_last


def gru_sequence(Wcodes, Walpha, bias, I, H, x_seq, h0, k_a, T, workspace, want_h_seq=False,
                 h_seq=None, h_last=None):
    Wcodes, Walpha = _dev(Wcodes, torch.int32, "Wcodes"), _dev(Walpha, torch.float32, "Walpha")
    x_seq, h0 = _dev(x_seq, torch.float32, "x_seq"), _dev(h0, torch.float32, "h0")
    steps, batch, k_w = x_seq.shape[0], h0.shape[0], Wcodes.shape[1]
    if want_h_seq and h_seq is None:
        h_seq = torch.empty((steps, batch, H), dtype=torch.float32, device=h0.device)
    h_last = torch.empty_like(h0) if h_last is None else h_last
    _check(_lib.amq_gru_sequence(_ptr(Wcodes), _ptr(Walpha), _ptr(bias), I, H, k_w, _ptr(x_seq), steps, _ptr(h0),
                                 batch, k_a, T, _ptr(h_seq), _ptr(h_last), _ptr(workspace), workspace.numel(),
                                 _stream()))
    return h_seq, h_last


def _host(t, name):
    if t is None:
        return None
    if not (isinstance(t, torch.Tensor) and not t.is_cuda and t.dtype == torch.float32 and t.is_contiguous()):
        raise TypeError("%s must be a contiguous CPU fp32 tensor" % name)
    return t


def lstm_sequence_host(Wcodes, Walpha, bias, I, H, x_seq, h0, c0, k_a, T, workspace, staging,
                       h_last, c_last, h_seq=None):
    """x_seq, h0, c0, h_last, c_last, h_seq are HOST tensors (pinned for asynchronous copies)."""
    x_seq, h0, c0 = _host(x_seq, "x_seq"), _host(h0, "h0"), _host(c0, "c0")
    steps, batch, k_w = x_seq.shape[0], h0.shape[0], Wcodes.shape[1]
    _check(_lib.amq_lstm_sequence_host(_ptr(Wcodes), _ptr(Walpha), _ptr(bias), I, H, k_w, _ptr(x_seq), steps,
                                       _ptr(h0), _ptr(c0), batch, k_a, T, _ptr(_host(h_seq, "h_seq")),
                                       _ptr(_host(h_last, "h_last")), _ptr(_host(c_last, "c_last")),
                                       _ptr(workspace), workspace.numel(), _ptr(staging), staging.numel(), _stream()))
    return h_seq, h_last, c_last


def gru_sequence_host(Wcodes, Walpha, bias, I, H, x_seq, h0, k_a, T, workspace, staging, h_last, h_seq=None):
    x_seq, h0 = _host(x_seq, "x_seq"), _host(h0, "h0")
    steps, batch, k_w = x_seq.shape[0], h0.shape[0], Wcodes.shape[1]
    _check(_lib.amq_gru_sequence_host(_ptr(Wcodes), _ptr(Walpha), _ptr(bias), I, H, k_w, _ptr(x_seq), steps,
                                      _ptr(h0), batch, k_a, T, _ptr(_host(h_seq, "h_seq")),
                                      _ptr(_host(h_last, "h_last")), _ptr(workspace), workspace.numel(),
                                      _ptr(staging), staging.numel(), _stream()))
    return h_seq, h_last


def workspace_status(workspace):
    return _lib.amq_workspace_status(_ptr(workspace), _stream())


def embedding_rows(We_codes, We_alpha, n, tokens):
    """Rows of the quantized embedding matrix for int32 token ids of any shape -> codes (*shape, k, wpr), coeffs (*shape, k)."""
    We_codes, We_alpha = _dev(We_codes, torch.int32, "We_codes"), _dev(We_alpha, torch.float32, "We_alpha")
    tokens = _dev(tokens, torch.int32, "tokens")
    vocab, k, wpr = We_codes.shape
    xcodes = torch.empty(tuple(tokens.shape) + (k, wpr), dtype=torch.int32, device=We_codes.device)
    xbeta = torch.empty(tuple(tokens.shape) + (k,), dtype=torch.float32, device=We_codes.device)
    _check(_lib.amq_embedding_rows(_ptr(We_codes), _ptr(We_alpha), vocab, n, k, _ptr(tokens), tokens.numel(),
                                   _ptr(xcodes), _ptr(xbeta), _stream()))
    return xcodes, xbeta


def new_paper_workspace(H, batch, steps, k_a, device="cuda"):
    return torch.empty(max(_lib.amq_lstm_paper_workspace_bytes(H, batch, steps, k_a), 16), dtype=torch.uint8, device=device)


def lstm_step_paper(Wi_codes, Wi_alpha, Wh_codes, Wh_alpha, bias, I, H, xcodes, xbeta, h_in, c_in, k_a, T, workspace,
                    h_out=None, c_out=None):
    batch, k_w, k_e = h_in.shape[0], Wi_codes.shape[1], xcodes.shape[-2]
    h_out = torch.empty_like(h_in) if h_out is None else h_out
    c_out = torch.empty_like(c_in) if c_out is None else c_out
    _check(_lib.amq_lstm_step_paper(_ptr(Wi_codes), _ptr(Wi_alpha), _ptr(Wh_codes), _ptr(Wh_alpha), _ptr(bias), I, H, k_w,
                                    _ptr(xcodes), _ptr(xbeta), k_e, _ptr(h_in), _ptr(c_in), batch, k_a, T,
                                    _ptr(h_out), _ptr(c_out), _ptr(workspace), workspace.numel(), _stream()))
    return h_out, c_out


def lstm_sequence_paper(Wi_codes, Wi_alpha, Wh_codes, Wh_alpha, bias, I, H, xcodes_seq, xbeta_seq, h0, c0, k_a, T, workspace,
                        want_h_seq=False, h_last=None, c_last=None):
    steps, batch, k_e = xcodes_seq.shape[0], h0.shape[0], xcodes_seq.shape[-2]
    k_w = Wi_codes.shape[1]
    h_seq = torch.empty((steps, batch, H), dtype=torch.float32, device=h0.device) if want_h_seq else None
    h_last = torch.empty_like(h0) if h_last is None else h_last
    c_last = torch.empty_like(c0) if c_last is None else c_last
    _check(_lib.amq_lstm_sequence_paper(_ptr(Wi_codes), _ptr(Wi_alpha), _ptr(Wh_codes), _ptr(Wh_alpha), _ptr(bias), I, H, k_w,
                                        _ptr(xcodes_seq), _ptr(xbeta_seq), k_e, steps, _ptr(h0), _ptr(c0), batch, k_a, T,
                                        _ptr(h_seq), _ptr(h_last), _ptr(c_last), _ptr(workspace), workspace.numel(),
                                        _stream()))
    return h_seq, h_last, c_last


def log_softmax_argmax(logits, want_logp=True, argmax=None):
    """logits (rows, n) fp32, rows contiguous (any row stride) -> (log-probabilities (rows, n) or None, argmax (rows,) int32)."""
    if not (isinstance(logits, torch.Tensor) and logits.is_cuda and logits.dtype == torch.float32 and logits.dim() == 2
            and (logits.shape[1] == 1 or logits.stride(1) == 1)):
        raise TypeError("logits must be a 2-D CUDA float32 tensor with contiguous rows")
    rows, n = logits.shape
    ld = logits.stride(0) if rows > 1 else max(n, logits.stride(0))
    logp = torch.empty((rows, n), dtype=torch.float32, device=logits.device) if want_logp else None
    argmax = torch.empty((rows,), dtype=torch.int32, device=logits.device) if argmax is None else argmax
    _check(_lib.amq_log_softmax_argmax(_ptr(logits), rows, n, ld, _ptr(logp), n, _ptr(argmax), _stream()))
    return logp, argmax


def new_decode_workspace(vocab, I, H, k_e, k_a, device="cuda"):
    return torch.empty((_lib.amq_lm_decode_workspace_bytes(vocab, I, H, k_e, k_a),), dtype=torch.uint8, device=device)


def lm_greedy_decode(We_codes, We_alpha, Wi_codes, Wi_alpha, Wh_codes, Wh_alpha, bias, Ws_codes, Ws_alpha, bias_s, I, H,
                     k_a, T, tokens, h, c, workspace, logp=None):
    """tokens: int32 (steps + 1,), tokens[0] given, the rest written; h, c: (H,) or (1, H) fp32, updated in place."""
    vocab, k_e = We_codes.shape[0], We_codes.shape[1]
    k_w, k_s = Wi_codes.shape[1], Ws_codes.shape[1]
    steps = tokens.numel() - 1
    _check(_lib.amq_lm_greedy_decode(_ptr(We_codes), _ptr(We_alpha), vocab, I, k_e, _ptr(Wi_codes), _ptr(Wi_alpha),
                                     _ptr(Wh_codes), _ptr(Wh_alpha), _ptr(bias), H, k_w, _ptr(Ws_codes), _ptr(Ws_alpha),
                                     _ptr(bias_s), k_s, k_a, T, _ptr(tokens), steps, _ptr(h), _ptr(c), _ptr(logp),
                                     _ptr(workspace), workspace.numel(), _stream()))
    return tokens


METHOD_ALTERNATING, METHOD_REFINED_GREEDY = 0, 1


def quantize_variant(x, k, T, method=METHOD_ALTERNATING, final_refit=False):
    """As quantize, with the method (alternating / refined greedy) and an optional last coefficient refit."""
    if not (x.is_cuda and x.dtype == torch.float32 and x.dim() == 2 and x.stride(1) == 1):
        raise TypeError("x must be a 2-D CUDA fp32 tensor with unit column stride")
    rows, n = x.shape
    ldx = x.stride(0) if rows > 1 else max(n, x.stride(0))
    codes = _new_codes(rows, k, n, x.device)
    coeffs = torch.empty((rows, k), dtype=torch.float32, device=x.device)
    _check(_lib.amq_quantize_variant(_ptr(x), rows, n, ldx, k, T, method, int(final_refit), _ptr(codes), _ptr(coeffs),
                                     _stream()))
    return codes, coeffs


def gru_step_original(Wcodes, Walpha, bias, I, H, x, h_in, k_a, T, workspace=None, h_out=None):
    """The GRU in its original form (reset gate applied to h before the candidate's product); bias (3H,) or None."""
    batch, k_w = h_in.shape[0], Wcodes.shape[1]
    if workspace is None:
        workspace = torch.empty((_lib.amq_gru_original_workspace_bytes(I, H, batch, k_a),), dtype=torch.uint8, device=h_in.device)
    h_out = torch.empty_like(h_in) if h_out is None else h_out
    _check(_lib.amq_gru_step_original(_ptr(Wcodes), _ptr(Walpha), _ptr(bias), I, H, k_w, _ptr(x), _ptr(h_in), batch, k_a, T,
                                      _ptr(h_out), _ptr(workspace), workspace.numel(), _stream()))
    return h_out
