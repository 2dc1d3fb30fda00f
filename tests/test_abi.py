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


def test_argument_validation_of_the_widened_entry_points(lib):
    """Variants of the quantizer, the paper-form cell, the original-form GRU, the output layer and the decoding loop:
    every rejection below is decided on the host, before any launch (the pointers are never dereferenced)."""
    vp, ci, sz = ctypes.c_void_p, ctypes.c_int, ctypes.c_size_t
    fake, fake2, odd = vp(0x1000), vp(0x2000), vp(0x1004)
    qv = lib.amq_quantize_variant
    qv.argtypes = [vp, ci, ci, ci, ci, ci, ci, ci, vp, vp, vp]
    assert qv(fake, 1, 8, 8, 2, 2, 2, 0, fake, fake, None) == -2           # unknown method
    assert qv(fake, 1, 8, 8, 2, 2, -1, 0, fake, fake, None) == -2
    assert qv(fake, 1, 8, 8, 5, 2, 1, 0, fake, fake, None) == -2           # k
    assert qv(fake, 1, 8, 4, 2, 2, 1, 1, fake, fake, None) == -1           # ldx < n
    assert qv(fake, 1, 8, 8, 2, 2, 1, 1, odd, fake, None) == -3
    assert qv(None, 0, 8, 8, 2, 2, 1, 1, None, None, None) == 0            # empty input
    sm = lib.amq_log_softmax_argmax
    sm.argtypes = [vp, ci, ci, ci, vp, ci, vp, vp]
    assert sm(fake, 1, 0, 0, fake, 0, fake, None) == -1                    # n < 1
    assert sm(fake, 1, 8, 4, fake, 8, fake, None) == -1                    # ld < n
    assert sm(fake, 1, 8, 8, fake, 4, fake, None) == -1                    # ldp < n
    assert sm(fake, 1, 8, 8, None, 8, None, None) == -1                    # nothing to write
    assert sm(None, 0, 8, 8, None, 8, None, None) == 0
    er = lib.amq_embedding_rows
    er.argtypes = [vp, vp, ci, ci, ci, vp, ci, vp, vp, vp]
    assert er(fake, fake, 10, 8, 5, fake, 1, fake, fake, None) < 0         # k
    assert er(fake, fake, 0, 8, 2, fake, 1, fake, fake, None) < 0          # empty vocabulary
    lib.amq_gru_original_workspace_bytes.restype = sz
    lib.amq_gru_original_workspace_bytes.argtypes = [ci, ci, ci, ci]
    need = lib.amq_gru_original_workspace_bytes(8, 8, 2, 2)
    assert need > 0 and lib.amq_gru_original_workspace_bytes(8, 8, 2, 5) == 0 and lib.amq_gru_original_workspace_bytes(8, 0, 2, 2) == 0
    go = lib.amq_gru_step_original
    go.argtypes = [vp, vp, vp, ci, ci, ci, vp, vp, ci, ci, ci, vp, vp, sz, vp]
    assert go(fake, fake, None, 8, 8, 2, fake, fake, 2, 2, 2, fake2, fake, need - 1, None) == -4
    assert go(fake, fake, None, 8, 8, 2, fake, fake, 2, 2, 2, fake, fake, need, None) == -1       # h_out == h_in
    assert go(fake, fake, None, 8, 8, 0, fake, fake, 2, 2, 2, fake2, fake, need, None) == -2      # k_w
    assert go(odd, fake, None, 8, 8, 2, fake, fake, 2, 2, 2, fake2, fake, need, None) == -3
    assert go(fake, fake, None, 8, 8, 2, fake, fake, 0, 2, 2, fake2, fake, need, None) == 0       # empty batch
    lib.amq_lm_decode_workspace_bytes.restype = sz
    lib.amq_lm_decode_workspace_bytes.argtypes = [ci] * 5
    dneed = lib.amq_lm_decode_workspace_bytes(100, 8, 8, 2, 2)
    assert dneed >= 100 * 4 and lib.amq_lm_decode_workspace_bytes(0, 8, 8, 2, 2) == 0
    dec = lib.amq_lm_greedy_decode
    dec.argtypes = [vp, vp, ci, ci, ci, vp, vp, vp, vp, vp, ci, ci, vp, vp, vp, ci, ci, ci, vp, ci, vp, vp, vp, vp, sz, vp]
    args = [fake, fake, 100, 8, 2, fake, fake, fake, fake, None, 8, 2, fake, fake, None, 2, 2, 2, fake, 3, fake, fake, None,
            fake, dneed, None]
    bad = list(args); bad[24] = dneed - 1
    assert dec(*bad) == -4                                                 # workspace too small
    bad = list(args); bad[15] = 7
    assert dec(*bad) == -2                                                 # bits of the output layer
    bad = list(args); bad[12] = None
    assert dec(*bad) == -1                                                 # no output matrix
    bad = list(args); bad[0] = odd
    assert dec(*bad) == -3
    bad = list(args); bad[19] = 0
    assert dec(*bad) == 0                                                  # no steps: nothing to do
    lib.amq_lstm_paper_workspace_bytes.restype = sz
    lib.amq_lstm_paper_workspace_bytes.argtypes = [ci] * 4
    assert lib.amq_lstm_paper_workspace_bytes(8, 2, 3, 2) > lib.amq_lstm_paper_workspace_bytes(8, 2, 1, 2) > 0
    assert lib.amq_lstm_paper_workspace_bytes(8, 2, 3, 0) == 0


def test_argument_validation_of_the_give_up_selftest(lib):
    """The test aid for the give-up path is validated on the host like every other entry (no launch below)."""
    vp, ci, sz, cu = ctypes.c_void_p, ctypes.c_int, ctypes.c_size_t, ctypes.c_uint
    fake, fake2, fake3 = vp(0x1000), vp(0x2000), vp(0x3000)
    lib.amq_cell_workspace_bytes.restype = sz
    lib.amq_cell_workspace_bytes.argtypes = [ci] * 4
    need = lib.amq_cell_workspace_bytes(8, 8, 1, 2)
    st = lib.amq_selftest_sequence_give_up
    st.argtypes = [vp, vp, vp, ci, ci, ci, vp, ci, vp, vp, ci, ci, vp, vp, vp, sz, cu, vp]
    ok_args = [fake, fake, None, 8, 8, 2, fake, 3, fake, fake, 2, 2, fake2, fake3, fake, need, 100, None]
    bad = list(ok_args); bad[15] = need - 1
    assert st(*bad) == -4                                                  # workspace too small
    bad = list(ok_args); bad[7] = 1
    assert st(*bad) == -1                                                  # one step waits for nothing
    bad = list(ok_args); bad[16] = 0
    assert st(*bad) == -1                                                  # poll limit out of range
    bad = list(ok_args); bad[16] = 1 << 17
    assert st(*bad) == -1
    bad = list(ok_args); bad[12] = fake
    assert st(*bad) == -1                                                  # h_last == h0
    bad = list(ok_args); bad[10] = 5
    assert st(*bad) == -2                                                  # bits


def test_argument_validation_of_the_one_launch_matrix_vector_entry(lib):
    vp, ci = ctypes.c_void_p, ctypes.c_int
    fake, odd = vp(0x1000), vp(0x1004)
    qg = lib.amq_quantized_gemv
    qg.argtypes = [vp, vp, ci, ci, ci, vp, ci, ci, vp, vp, vp, vp, vp]
    assert qg(fake, fake, 8, 2049, 2, fake, 2, 2, None, fake, None, None, None) == -2      # vector too long for the fused form
    assert qg(fake, fake, 8, 64, 5, fake, 2, 2, None, fake, None, None, None) == -2        # bits
    assert qg(fake, fake, 8, 64, 2, fake, 2, -1, None, fake, None, None, None) == -2       # cycles
    assert qg(fake, fake, 8, 0, 2, fake, 2, 2, None, fake, None, None, None) == -1         # empty vector
    assert qg(fake, fake, 8, 64, 2, None, 2, 2, None, fake, None, None, None) == -1        # no vector
    assert qg(odd, fake, 8, 64, 2, fake, 2, 2, None, fake, None, None, None) == -3
    assert qg(fake, fake, 8, 64, 2, fake, 2, 2, None, fake, odd, None, None) == -3
    assert qg(None, None, 0, 64, 2, None, 2, 2, None, None, None, None, None) == 0         # no rows: nothing to do


def test_paper_table6_fixture_is_the_one_the_benchmark_reads():
    """bench.py quotes the paper's single-core CPU times (Appendix A, Table 6) from this fixture: the four quantized rows
    must be there with the printed totals."""
    rows = {}
    for ln in open(os.path.join(ROOT, "tests", "golden", "table6_cpu_ms.txt")):
        f = ln.split()
        if len(f) >= 6 and f[0].isdigit():
            rows[(int(f[0]), int(f[2]))] = float(f[4])
    assert rows[(4096, 2)] == 0.35 and rows[(4096, 3)] == 0.72 and rows[(42000, 2)] == 3.17 and rows[(42000, 3)] == 6.46
    assert rows[(4096, 0)] == 1.95 and rows[(42000, 0)] == 19.10       # the full-precision baseline of the same table
