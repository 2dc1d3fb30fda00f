"""Pins of the CPU oracle's packing, binary dot, quantized product and recurrent steps."""
import numpy as np
import pytest

import oracle
from paper_1802_00150_b200 import synth


def random_planes(k, n, seed, stream):
    return np.where(synth.uniform01(k * n, seed, stream).reshape(k, n) < 0.5, -1, 1).astype(np.int8)


# ---- packing ---------------------------------------------------------------------------------------------

@pytest.mark.parametrize("n", [1, 31, 32, 33, 127, 128, 129, 300, 600])
def test_pack_layout_and_roundtrip(n):
    b = random_planes(1, n, 1, n)[0]
    words = oracle.pack_plane(b)
    assert words.size == 4 * ((n + 127) // 128) == oracle.words_per_row(n)
    # bit j of word q is element 32q + j; pads are zero -- checked with numpy's own bit unpacking
    bits = np.unpackbits(words.view(np.uint8), bitorder="little")
    assert np.array_equal(bits[:n], (b > 0).astype(np.uint8))
    assert not bits[n:].any()
    assert np.array_equal(oracle.unpack_plane(words, n), b)


# ---- XNOR / bitcount dot == the dot of the +-1 vectors (Appendix A) --------------------------------------

def test_dot_xnor_equals_pm1_dot_all_lengths():
    for n in range(1, 301):
        a, b = random_planes(2, n, 2, n)
        got = oracle.dot_xnor(oracle.pack_plane(a), oracle.pack_plane(b), n)
        assert got == int(a.astype(np.int64) @ b.astype(np.int64))
        assert got == oracle.dot_pm1(a, b)


def test_dot_and_popc_identity():
    # popc(a^b) = popc(a) + popc(b) - 2 popc(a&b)  =>  dot = n - 2popc(a) - 2popc(b) + 4popc(a&b)
    for n in (17, 64, 200, 1000):
        a, b = random_planes(2, n, 3, n)
        pa, pb = oracle.pack_plane(a), oracle.pack_plane(b)
        pc = lambda x: int(np.unpackbits(x.view(np.uint8)).sum())
        assert oracle.dot_xnor(pa, pb, n) == n - 2 * pc(pa) - 2 * pc(pb) + 4 * pc(pa & pb)


@pytest.mark.parametrize("n,lo,hi", [(300, 0, 300), (300, 0, 150), (300, 150, 300), (300, 31, 33), (300, 64, 64),
                                     (257, 5, 250), (128, 32, 96)])
def test_dot_xnor_range(n, lo, hi):
    a, b = random_planes(2, n, 4, n + lo)
    got = oracle.dot_xnor(oracle.pack_plane(a), oracle.pack_plane(b), n, lo, hi)
    assert got == int(a[lo:hi].astype(np.int64) @ b[lo:hi].astype(np.int64))


# ---- the quantized product (Sec. 4) ----------------------------------------------------------------------

@pytest.mark.parametrize("m,n,kw,ka,batch", [(7, 50, 2, 2, 1), (33, 300, 3, 2, 3), (16, 129, 1, 4, 2), (5, 600, 4, 3, 2)])
def test_product_equals_dense_product_of_reconstructions(m, n, kw, ka, batch):
    W = synth.normal((m, n), 0.05, 5, 1).astype(np.float64)
    X = synth.uniform((batch, n), -1, 1, 5, 2).astype(np.float64)
    bias = synth.normal((m,), 0.1, 5, 3).astype(np.float64)
    Wc, Wa = oracle.quantize_rows(W, kw, 2)
    Xc, Xb = oracle.quantize_rows(X, ka, 2)
    # reconstruct from the UNPACKED planes of an independent quantize call, row by row
    What = np.stack([oracle.reconstruct(*oracle.quantize(W[r], kw, 2)) for r in range(m)])
    Xhat = np.stack([oracle.reconstruct(*oracle.quantize(X[b], ka, 2)) for b in range(batch)])
    y = oracle.binary_gemm(Wc, Wa, Xc, Xb, n, bias)
    assert np.allclose(y, Xhat @ What.T + bias, rtol=1e-11, atol=1e-12)
    # integer partials
    D = oracle.binary_dots(Wc, Xc, n)
    for bt in range(batch):
        for r in (0, m - 1):
            for i in range(kw):
                for j in range(ka):
                    wi = oracle.unpack_plane(Wc[r, i], n).astype(np.int64)
                    xj = oracle.unpack_plane(Xc[bt, j], n).astype(np.int64)
                    assert D[bt, r, i, j] == wi @ xj
    # y from the partials, the formula of Fig. 3 (left)
    y2 = np.einsum("ri,bj,brij->br", Wa, Xb, D.astype(np.float64)) + bias
    assert np.allclose(y, y2, rtol=1e-12, atol=1e-13)


def test_product_column_ranges_add_up():
    m, n, I = 12, 200, 72
    W = synth.normal((m, n), 0.05, 6, 1).astype(np.float64)
    X = synth.normal((2, n), 1.0, 6, 2).astype(np.float64)
    Wc, Wa = oracle.quantize_rows(W, 2, 2)
    Xc, Xb = oracle.quantize_rows(X, 3, 2)
    full = oracle.binary_gemm(Wc, Wa, Xc, Xb, n)
    left = oracle.binary_gemm(Wc, Wa, Xc, Xb, n, lo=0, hi=I)
    right = oracle.binary_gemm(Wc, Wa, Xc, Xb, n, lo=I, hi=n)
    assert np.allclose(full, left + right, rtol=1e-12, atol=1e-13)


# ---- recurrent steps -------------------------------------------------------------------------------------

def dense_hat(codes, coeffs, n):
    rows, k, _ = codes.shape
    out = np.zeros((rows, n))
    for r in range(rows):
        for i in range(k):
            out[r] += coeffs[r, i] * oracle.unpack_plane(codes[r, i], n)
    return out


def textbook_lstm(W, bias, x, h, c, H):
    """Plain fp64 LSTM step (Eq. 6, gates i, f, o logistic and g tanh) on dense operands."""
    p = np.concatenate([x, h], axis=1) @ W.T + (0 if bias is None else bias)
    sig = lambda v: 1 / (1 + np.exp(-v))
    i, f, o, g = sig(p[:, :H]), sig(p[:, H:2 * H]), sig(p[:, 2 * H:3 * H]), np.tanh(p[:, 3 * H:])
    c2 = f * c + i * g
    return o * np.tanh(c2), c2


def textbook_gru(W, bias, x, h, I, H):
    """Plain fp64 GRU step, linear-before-reset form, rows r, z, n; bias [b_r, b_z, b_nx, b_nh]."""
    sig = lambda v: 1 / (1 + np.exp(-v))
    px, ph = x @ W[:, :I].T, h @ W[:, I:].T
    b = np.zeros(4 * H) if bias is None else bias
    r = sig(px[:, :H] + ph[:, :H] + b[:H])
    z = sig(px[:, H:2 * H] + ph[:, H:2 * H] + b[H:2 * H])
    cand = np.tanh(px[:, 2 * H:] + b[2 * H:3 * H] + r * (ph[:, 2 * H:] + b[3 * H:]))
    return (1 - z) * cand + z * h


@pytest.mark.parametrize("I,H,batch,kw,ka", [(20, 12, 2, 2, 2), (33, 31, 1, 3, 3), (64, 40, 3, 2, 3)])
def test_lstm_step_equals_textbook_step_on_reconstructed_operands(I, H, batch, kw, ka):
    n = I + H
    W = synth.normal((4 * H, n), 0.2, 7, 1).astype(np.float64)
    bias = synth.normal((4 * H,), 0.1, 7, 2).astype(np.float64)
    x = synth.normal((batch, I), 1.0, 7, 3).astype(np.float64)
    h = synth.uniform((batch, H), -1, 1, 7, 4).astype(np.float64)
    c = synth.uniform((batch, H), -1, 1, 7, 5).astype(np.float64)
    Wc, Wa = oracle.quantize_rows(W, kw, 2)
    zc, zb = oracle.quantize_rows(np.concatenate([x, h], axis=1), ka, 2)
    What, zhat = dense_hat(Wc, Wa, n), dense_hat(zc, zb, n)
    h_ref, c_ref = textbook_lstm(What, bias, zhat[:, :I], zhat[:, I:], c, H)
    h_out, c_out = oracle.lstm_step(Wc, Wa, bias, I, H, x, h, c, ka, 2)
    assert np.allclose(h_out, h_ref, rtol=1e-11, atol=1e-13) and np.allclose(c_out, c_ref, rtol=1e-11, atol=1e-13)
    h_nb, _ = oracle.lstm_step(Wc, Wa, None, I, H, x, h, c, ka, 2)
    assert np.allclose(h_nb, textbook_lstm(What, None, zhat[:, :I], zhat[:, I:], c, H)[0], rtol=1e-11, atol=1e-13)


@pytest.mark.parametrize("I,H,batch,kw,ka", [(20, 12, 2, 2, 3), (32, 31, 1, 3, 3), (37, 40, 3, 2, 2)])
def test_gru_step_equals_textbook_step_on_reconstructed_operands(I, H, batch, kw, ka):
    n = I + H
    W = synth.normal((3 * H, n), 0.2, 8, 1).astype(np.float64)
    bias = synth.normal((4 * H,), 0.1, 8, 2).astype(np.float64)
    x = synth.normal((batch, I), 1.0, 8, 3).astype(np.float64)
    h = synth.uniform((batch, H), -1, 1, 8, 4).astype(np.float64)
    Wc, Wa = oracle.quantize_rows(W, kw, 2)
    zc, zb = oracle.quantize_rows(np.concatenate([x, h], axis=1), ka, 2)
    What, zhat = dense_hat(Wc, Wa, n), dense_hat(zc, zb, n)
    # the blend uses the UNQUANTIZED previous state h; the products use the quantized z
    sig = lambda v: 1 / (1 + np.exp(-v))
    px, ph = zhat[:, :I] @ What[:, :I].T, zhat[:, I:] @ What[:, I:].T
    r = sig(px[:, :H] + ph[:, :H] + bias[:H])
    z = sig(px[:, H:2 * H] + ph[:, H:2 * H] + bias[H:2 * H])
    cand = np.tanh(px[:, 2 * H:] + bias[2 * H:3 * H] + r * (ph[:, 2 * H:] + bias[3 * H:]))
    ref = (1 - z) * cand + z * h
    got = oracle.gru_step(Wc, Wa, bias, I, H, x, h, ka, 2)
    assert np.allclose(got, ref, rtol=1e-11, atol=1e-13)


def exactly_representable(shape, a, c, seed, stream):
    u = synth.uniform01(int(np.prod(shape)), seed, stream).reshape(shape)
    return np.select([u < 0.25, u < 0.5, u < 0.75], [a + c, a - c, -a + c], -a - c)


def test_cells_reduce_to_full_precision_cells_when_two_bits_are_exact():
    # every weight row and the vector [x;h] take values in {+-a +-c}: 2-bit quantization is the identity,
    # so the quantized step must equal the plain fp64 step on the unquantized operands
    I, H, batch = 24, 16, 2
    n = I + H
    z = exactly_representable((batch, n), 0.5, 0.125, 9, 1)
    x, h = z[:, :I], z[:, I:]
    c = synth.uniform((batch, H), -1, 1, 9, 2).astype(np.float64)
    Wl = exactly_representable((4 * H, n), 0.05, 0.02, 9, 3)
    Wc, Wa = oracle.quantize_rows(Wl, 2, 2)
    h_out, c_out = oracle.lstm_step(Wc, Wa, None, I, H, x, h, c, 2, 2)
    h_ref, c_ref = textbook_lstm(Wl, None, x, h, c, H)
    assert np.allclose(h_out, h_ref, atol=1e-12) and np.allclose(c_out, c_ref, atol=1e-12)
    Wg = exactly_representable((3 * H, n), 0.05, 0.02, 9, 4)
    Gc, Ga = oracle.quantize_rows(Wg, 2, 2)
    got = oracle.gru_step(Gc, Ga, None, I, H, x, h, 2, 2)
    assert np.allclose(got, textbook_gru(Wg, None, x, h, I, H), atol=1e-12)


def test_sequences_are_repeated_steps():
    I, H, batch, steps = 16, 8, 2, 4
    W = synth.normal((4 * H, I + H), 0.3, 10, 1).astype(np.float64)
    Wc, Wa = oracle.quantize_rows(W, 2, 2)
    xs = synth.normal((steps, batch, I), 1.0, 10, 2).astype(np.float64)
    h, c = np.zeros((batch, H)), np.zeros((batch, H))
    h_seq, h_last, c_last = oracle.lstm_sequence(Wc, Wa, None, I, H, xs, h, c, 2, 2)
    for s in range(steps):
        h, c = oracle.lstm_step(Wc, Wa, None, I, H, xs[s], h, c, 2, 2)
        assert np.array_equal(h_seq[s], h)
    assert np.array_equal(h_last, h) and np.array_equal(c_last, c)
    G = synth.normal((3 * H, I + H), 0.3, 10, 3).astype(np.float64)
    Gc, Ga = oracle.quantize_rows(G, 2, 2)
    h = np.zeros((batch, H))
    g_seq, g_last = oracle.gru_sequence(Gc, Ga, None, I, H, xs, h, 3, 2)
    for s in range(steps):
        h = oracle.gru_step(Gc, Ga, None, I, H, xs[s], h, 3, 2)
        assert np.array_equal(g_seq[s], h)
    assert np.array_equal(g_last, h)


def test_synth_is_reproducible_and_shaped():
    a = synth.normal((4, 5), 0.03, 0, 1)
    b = synth.normal((4, 5), 0.03, 0, 1)
    assert a.dtype == np.float32 and np.array_equal(a, b)
    assert not np.array_equal(a, synth.normal((4, 5), 0.03, 0, 2))
    big = synth.normal((200000,), 1.0, 3, 1).astype(np.float64)
    assert abs(big.mean()) < 0.01 and abs(big.std() - 1) < 0.01
    u = synth.uniform((200000,), -1, 1, 3, 2).astype(np.float64)
    assert abs(u.mean()) < 0.01 and abs(u.std() - 1 / np.sqrt(3)) < 0.01 and u.min() >= -1 and u.max() <= 1
    # a prefix of a larger draw equals the smaller draw (counter-based)
    assert np.array_equal(synth.uniform((10,), -1, 1, 5, 5), synth.uniform((20,), -1, 1, 5, 5)[:10])
    wl = synth.WORKLOADS["lstm1024_b1"]
    assert (wl.m, wl.n) == (4096, 2048)
    ins = synth.inputs(wl)
    assert ins["x_seq"].shape == (35, 1, 1024) and np.abs(ins["x_seq"]).max() <= 3.0


@pytest.mark.parametrize("I,H,batch,kw,ke,ka", [(20, 12, 2, 2, 2, 2), (33, 31, 1, 3, 2, 3), (64, 40, 3, 2, 3, 1)])
def test_paper_form_lstm_step_equals_textbook_step_on_reconstructed_operands(I, H, batch, kw, ke, ka):
    """Eq. 6 as printed: separate W_i and W_h, x an (already quantized) embedding row, only h quantized on-line."""
    Wi = synth.normal((4 * H, I), 0.2, 17, 1).astype(np.float64)
    Wh = synth.normal((4 * H, H), 0.2, 17, 2).astype(np.float64)
    bias = synth.normal((4 * H,), 0.1, 17, 3).astype(np.float64)
    emb = synth.normal((batch, I), 0.5, 17, 4).astype(np.float64)          # the embedding rows of the tokens
    h = synth.uniform((batch, H), -1, 1, 17, 5).astype(np.float64)
    c = synth.uniform((batch, H), -1, 1, 17, 6).astype(np.float64)
    Wic, Wia = oracle.quantize_rows(Wi, kw, 2)
    Whc, Wha = oracle.quantize_rows(Wh, kw, 2)
    xc, xb = oracle.quantize_rows(emb, ke, 2)                              # offline, like every row of W_e
    hc, hb = oracle.quantize_rows(h, ka, 2)
    # textbook step on the dense reconstructions, with the stacked matrix [W_i | W_h]
    What = np.concatenate([dense_hat(Wic, Wia, I), dense_hat(Whc, Wha, H)], axis=1)
    h_ref, c_ref = textbook_lstm(What, bias, dense_hat(xc, xb, I), dense_hat(hc, hb, H), c, H)
    h_out, c_out = oracle.lstm_step_paper(Wic, Wia, Whc, Wha, bias, I, H, xc, xb, h, c, ka, 2)
    assert np.allclose(h_out, h_ref, rtol=1e-11, atol=1e-13) and np.allclose(c_out, c_ref, rtol=1e-11, atol=1e-13)


def test_paper_form_lstm_step_reduces_to_full_precision_when_two_bits_are_exact():
    I, H, batch = 24, 16, 2
    x = exactly_representable((batch, I), 0.5, 0.125, 19, 1)
    h = exactly_representable((batch, H), 0.25, 0.0625, 19, 2)
    c = synth.uniform((batch, H), -1, 1, 19, 3).astype(np.float64)
    Wi = exactly_representable((4 * H, I), 0.05, 0.02, 19, 4)
    Wh = exactly_representable((4 * H, H), 0.07, 0.01, 19, 5)
    Wic, Wia = oracle.quantize_rows(Wi, 2, 2)
    Whc, Wha = oracle.quantize_rows(Wh, 2, 2)
    xc, xb = oracle.quantize_rows(x, 2, 2)
    h_out, c_out = oracle.lstm_step_paper(Wic, Wia, Whc, Wha, None, I, H, xc, xb, h, c, 2, 2)
    h_ref, c_ref = textbook_lstm(np.concatenate([Wi, Wh], axis=1), None, x, h, c, H)
    assert np.allclose(h_out, h_ref, atol=1e-12) and np.allclose(c_out, c_ref, atol=1e-12)


def test_log_softmax_argmax_against_library_routine_and_invariants():
    from scipy.special import log_softmax
    z = synth.normal((5, 1000), 3.0, 23, 1).astype(np.float64)
    z[1, 17] = z[1, 400] = z[1].max() + 1.0                     # equal maxima: the first index wins
    z[2] += 800.0                                               # large offsets must not overflow
    logp, arg = oracle.log_softmax_argmax(z)
    assert np.allclose(logp, log_softmax(z, axis=1), rtol=1e-12, atol=1e-12)
    assert np.allclose(np.exp(logp).sum(axis=1), 1.0, atol=1e-12)
    assert np.array_equal(arg, z.argmax(axis=1)) and arg[1] == 17
    shifted, _ = oracle.log_softmax_argmax(z + 5.0)             # invariant to a common shift
    assert np.allclose(shifted, logp, atol=1e-10)


def textbook_gru_original(W, b, x, h, I, H):
    """Cho et al.: r, z from [x ; h]; candidate from [x ; r * h]; W rows r, z, n; b (3H,) or None."""
    sig = lambda v: 1 / (1 + np.exp(-v))
    b = np.zeros(3 * H) if b is None else b
    zcat = np.concatenate([x, h], axis=1)
    r = sig(zcat @ W[:H].T + b[:H])
    z = sig(zcat @ W[H:2 * H].T + b[H:2 * H])
    cand = np.tanh(np.concatenate([x, r * h], axis=1) @ W[2 * H:].T + b[2 * H:])
    return (1 - z) * cand + z * h


@pytest.mark.parametrize("I,H,batch,kw,ka", [(20, 12, 2, 2, 3), (33, 31, 1, 3, 3), (37, 40, 3, 2, 2)])
def test_original_form_gru_equals_textbook_step_on_reconstructed_operands(I, H, batch, kw, ka):
    """The composition: both on-line quantizations and both products, checked against dense fp64 algebra on the
    reconstructed operands (the second vector depends on the first product through r)."""
    n = I + H
    W = synth.normal((3 * H, n), 0.2, 28, 1).astype(np.float64)
    bias = synth.normal((3 * H,), 0.1, 28, 2).astype(np.float64)
    x = synth.normal((batch, I), 1.0, 28, 3).astype(np.float64)
    h = synth.uniform((batch, H), -1, 1, 28, 4).astype(np.float64)
    Wc, Wa = oracle.quantize_rows(W, kw, 2)
    What = dense_hat(Wc, Wa, n)
    sig = lambda v: 1 / (1 + np.exp(-v))
    z1c, z1b = oracle.quantize_rows(np.concatenate([x, h], axis=1), ka, 2)
    z1 = dense_hat(z1c, z1b, n)
    r = sig(z1 @ What[:H].T + bias[:H])
    zg = sig(z1 @ What[H:2 * H].T + bias[H:2 * H])
    z2c, z2b = oracle.quantize_rows(np.concatenate([x, r * h], axis=1), ka, 2)
    cand = np.tanh(dense_hat(z2c, z2b, n) @ What[2 * H:].T + bias[2 * H:])
    ref = (1 - zg) * cand + zg * h
    got = oracle.gru_step_original(Wc, Wa, bias, I, H, x, h, ka, 2)
    assert np.allclose(got, ref, rtol=1e-11, atol=1e-13)
    assert np.array_equal(oracle.gru_step_original(Wc, Wa, None, I, H, x, h, ka, 2),
                          oracle.gru_step_original(Wc, Wa, np.zeros(3 * H), I, H, x, h, ka, 2))


def test_original_form_gru_reduces_to_the_textbook_gru_when_quantization_is_the_identity():
    # [x ; h] takes values in {+-a +-c} (2 bits exact); with W_r = 0 and b_r large the reset gate is 1 to 1e-16, so
    # [x ; r * h] is exactly representable too and the quantized step must equal the plain fp64 step of Cho et al.
    I, H, batch = 24, 16, 2
    n = I + H
    z = exactly_representable((batch, n), 0.5, 0.125, 29, 1)
    x, h = z[:, :I], z[:, I:]
    W = exactly_representable((3 * H, n), 0.05, 0.02, 29, 2)
    W[:H] = 0.0
    bias = np.concatenate([np.full(H, 40.0), synth.normal((2 * H,), 0.1, 29, 3).astype(np.float64)])
    Wc, Wa = oracle.quantize_rows(W, 2, 2)
    got = oracle.gru_step_original(Wc, Wa, bias, I, H, x, h, 2, 2)
    assert np.allclose(got, textbook_gru_original(W, bias, x, h, I, H), atol=1e-12)
    # and it differs from the linear-before-reset form as soon as r is not 1 (the two forms are different cells)
    bias2 = bias.copy(); bias2[:H] = 0.0
    a = oracle.gru_step_original(Wc, Wa, bias2, I, H, x, h, 2, 2)
    assert np.abs(a - got).max() > 1e-3
