"""Host-only checks of the C ABI: the library loads, exports every symbol the header declares, the
binding names them all, and argument validation answers before anything is launched."""
import ctypes
import os
import re
import shutil

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
HEADER = os.path.join(ROOT, "include", "amq.h")
LIB = os.path.join(ROOT, "paper_1802_00150_b200", "libamq_b200.so")


def declared_symbols():
    text = open(HEADER).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"AMQ_API\s+[\w\s\*]+?\b(amq_\w+)\s*\(", text)))


@pytest.fixture(scope="module")
def lib():
    if not os.path.exists(LIB):
        if shutil.which("nvcc") is None:
            pytest.skip("library not built and nvcc not available")
        from paper_1802_00150_b200 import build
        build.build()
    return ctypes.CDLL(LIB)


def test_header_declares_the_expected_entry_points():
    names = declared_symbols()
    for required in ("amq_quantize", "amq_pack", "amq_binary_gemm", "amq_binary_dots", "amq_lstm_step",
                     "amq_gru_step", "amq_lstm_sequence", "amq_gru_sequence"):
        assert required in names


def test_library_exports_every_declared_symbol(lib):
    for name in declared_symbols():
        assert hasattr(lib, name), name


def test_binding_covers_every_declared_symbol(lib):
    from paper_1802_00150_b200 import amq
    assert sorted(amq.EXPORTS) == declared_symbols()


def test_size_helpers(lib):
    lib.amq_words_per_row.restype = ctypes.c_int
    lib.amq_codes_bytes.restype = ctypes.c_size_t
    for n, wpr in ((1, 4), (128, 4), (129, 8), (600, 20), (2048, 64), (4096, 128)):
        assert lib.amq_words_per_row(n) == wpr
    assert lib.amq_words_per_row(0) == 0
    assert lib.amq_codes_bytes(4096, 2048, 2) == 2097152          # the 2 MiB of the hidden-1024 LSTM at 2 bits
    assert lib.amq_codes_bytes(32768, 1024, 3) == 12582912
    lib.amq_cell_workspace_bytes.restype = ctypes.c_size_t
    assert lib.amq_cell_workspace_bytes(1024, 1024, 1, 2) >= 256 + 2 * 64 * 4 + 3 * 4096
    assert lib.amq_cell_workspace_bytes(1024, 1024, 1, 5) == 0
    lib.amq_status_string.restype = ctypes.c_char_p
    assert lib.amq_status_string(0) == b"ok"
    assert b"timed out" in lib.amq_status_string(-6)


def test_argument_validation_happens_on_the_host(lib):
    vp = ctypes.c_void_p
    fake = vp(0x1000)          # never dereferenced: every call below must be rejected before any launch
    odd = vp(0x1004)
    q = lib.amq_quantize
    q.argtypes = [vp, ctypes.c_int, ctypes.c_int, ctypes.c_int, ctypes.c_int, ctypes.c_int, vp, vp, vp]
    assert q(None, 1, 8, 8, 2, 2, fake, fake, None) == -1
    assert q(fake, 1, 8, 4, 2, 2, fake, fake, None) == -1          # ldx < n
    assert q(fake, 1, 8, 8, 5, 2, fake, fake, None) == -2          # k
    assert q(fake, 1, 8, 8, 0, 2, fake, fake, None) == -2
    assert q(fake, 1, 8, 8, 2, -1, fake, fake, None) == -2         # T
    assert q(fake, 1, 8193, 8193, 2, 2, fake, fake, None) == -2    # n beyond the maximum
    assert q(fake, 1, 8, 8, 2, 2, odd, fake, None) == -3           # alignment
    assert q(fake, 0, 8, 8, 2, 2, fake, fake, None) == 0           # empty input: nothing to do
    assert q(None, 0, 8, 8, 2, 2, None, None, None) == 0           # ... even with NULL buffers
    g = lib.amq_binary_gemm
    g.argtypes = [vp, vp, ctypes.c_int, ctypes.c_int, ctypes.c_int, vp, vp, ctypes.c_int, ctypes.c_int, vp, vp,
                  ctypes.c_int, vp]
    assert g(fake, fake, 4, 8, 2, fake, fake, 1, 2, None, fake, 3, None) == -1     # ldy < m
    assert g(fake, fake, 4, 8, 2, odd, fake, 1, 2, None, fake, 4, None) == -3
    assert g(fake, fake, 4, 8, 2, fake, fake, 0, 2, None, fake, 4, None) == 0
    s = lib.amq_lstm_step
    s.argtypes = [vp, vp, vp] + [ctypes.c_int] * 3 + [vp, vp, vp] + [ctypes.c_int] * 3 + [vp, vp, vp, ctypes.c_size_t, vp]
    assert s(fake, fake, None, 8, 8, 2, fake, fake, fake, 1, 2, 2, fake, fake, fake, 16, None) == -4   # workspace small
    assert s(fake, fake, None, 8, 8, 2, fake, fake, fake, 1, 2, 2, fake, fake, None, 1 << 20, None) == -4
    assert s(fake, fake, None, 8, 8, 2, fake, fake, fake, 1, 2, 2, fake, fake, fake, 1 << 20, None) == -1  # h_out == h_in
