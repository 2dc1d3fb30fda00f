"""GPU parity at the full benchmark sizes, through the same calls and launch configurations bench.py times.
The oracle computes whole steps where that takes seconds and sampled rows where it would not."""
import numpy as np
import pytest
import torch

import oracle
import parity
from paper_1802_00150_b200 import synth

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def amq():
    assert torch.cuda.is_available(), "these tests need a CUDA device"
    from paper_1802_00150_b200 import amq as binding
    return binding


def dev(a, dtype=torch.float32):
    return torch.from_numpy(np.ascontiguousarray(a)).to(dtype).cuda()


def codes_np(t):
    return t.cpu().numpy().view(np.uint32)


def quantized_model(amq, wl):
    """Weights of the workload, quantized by the library (as bench.py does); returns device and host copies."""
    W = synth.weights(wl)
    Wcodes, Walpha = amq.quantize(dev(W), wl.k_w, wl.T)
    torch.cuda.synchronize()
    return W, Wcodes, Walpha, codes_np(Wcodes), Walpha.cpu().numpy().astype(np.float64)


def state_tolerance(Wa, beta, n):
    return 3.0 * parity.output_tolerance(Wa, beta, n).max() + 1e-6


def test_lstm300_single_step_workload(amq):
    wl = synth.WORKLOADS["lstm300_step"]
    _, Wcodes, Walpha, Wc, Wa = quantized_model(amq, wl)
    ins = synth.inputs(wl)
    x, h0, c0 = ins["x_seq"][0], ins["h0"], ins["c0"]
    ws = amq.new_workspace(wl.I, wl.H, 1, wl.k_a)
    h1, c1 = amq.lstm_step(Wcodes, Walpha, None, wl.I, wl.H, dev(x), dev(h0), dev(c0), wl.k_a, wl.T, ws)
    h_ref, c_ref = oracle.lstm_step(Wc, Wa, None, wl.I, wl.H, x, h0, c0, wl.k_a, wl.T)
    _, beta = oracle.quantize_rows(np.concatenate([x, h0], axis=1).astype(np.float64), wl.k_a, wl.T)
    tol = state_tolerance(Wa, beta, wl.n)
    assert np.abs(h1.cpu().numpy() - h_ref).max() <= tol and np.abs(c1.cpu().numpy() - c_ref).max() <= tol
    assert amq.workspace_status(ws) == 0


def test_lstm1024_batch1_sequence_workload(amq):
    """The default benchmark workload: 35 steps in one launch of the persistent kernel."""
    wl = synth.WORKLOADS["lstm1024_b1"]
    _, Wcodes, Walpha, Wc, Wa = quantized_model(amq, wl)
    ins = synth.inputs(wl)
    xs, h0, c0 = ins["x_seq"], ins["h0"], ins["c0"]
    ws = amq.new_workspace(wl.I, wl.H, 1, wl.k_a)
    g_seq, g_last, g_c = amq.lstm_sequence(Wcodes, Walpha, None, wl.I, wl.H, dev(xs), dev(h0), dev(c0), wl.k_a, wl.T, ws,
                                           want_h_seq=True)
    assert amq.workspace_status(ws) == 0
    assert torch.equal(g_seq[-1], g_last)
    # oracle trajectory (teacher): states after every step
    h, c = h0.astype(np.float64), c0.astype(np.float64)
    states = []
    for s in range(wl.steps):
        states.append((h, c))
        h, c = oracle.lstm_step(Wc, Wa, None, wl.I, wl.H, xs[s], h, c, wl.k_a, wl.T)
    states.append((h, c))
    # teacher-forced: restart the library from the oracle's state before sampled steps
    for s in (0, 1, 2, 9, 17, 26, 34):
        hp, cp = states[s]
        _, beta = oracle.quantize_rows(np.concatenate([xs[s].astype(np.float64), hp], axis=1), wl.k_a, wl.T)
        tol = state_tolerance(Wa, beta, wl.n)
        h_g, c_g = amq.lstm_step(Wcodes, Walpha, None, wl.I, wl.H, dev(xs[s]), dev(hp), dev(cp), wl.k_a, wl.T, ws)
        assert np.abs(h_g.cpu().numpy() - states[s + 1][0]).max() <= tol, s
        assert np.abs(c_g.cpu().numpy() - states[s + 1][1]).max() <= tol, s
    # the first step of the free-running sequence starts from the same state as the oracle
    _, beta = oracle.quantize_rows(np.concatenate([xs[0].astype(np.float64), states[0][0]], axis=1), wl.k_a, wl.T)
    assert np.abs(g_seq[0].cpu().numpy() - states[1][0]).max() <= state_tolerance(Wa, beta, wl.n)
    # the 35-step launch (all CTAs exchanging h) equals 35 chained single-step launches bit for bit, so the
    # teacher-forced parity of the step above carries over to every step of the sequence launch
    h, c = dev(h0), dev(c0)
    for s in range(wl.steps):
        h, c = amq.lstm_step(Wcodes, Walpha, None, wl.I, wl.H, dev(xs[s]), h, c, wl.k_a, wl.T, ws)
        assert torch.equal(h, g_seq[s]), s
    assert torch.equal(c, g_c)
    # five more runs of the sequence launch: the exchange must not make results depend on timing
    for _ in range(5):
        r_seq, _, r_c = amq.lstm_sequence(Wcodes, Walpha, None, wl.I, wl.H, dev(xs), dev(h0), dev(c0), wl.k_a, wl.T, ws,
                                          want_h_seq=True)
        assert torch.equal(r_seq, g_seq) and torch.equal(r_c, g_c)
    drift = max(np.abs(g_seq[s].cpu().numpy() - states[s + 1][0]).max() for s in range(wl.steps))
    print("free-running max |dh| over 35 steps: %.3g" % drift)
    assert np.isfinite(drift)


@pytest.mark.parametrize("name", ["lstm1024_b64", "gru2048_b256"])
def test_batched_sequence_workloads(amq, name):
    """The 35-step batched sequences bench.py times: the sequence call equals the chained step calls bit for bit, and
    sampled steps of sampled sequences, restarted from the library's own state, land on the oracle's next state."""
    wl = synth.WORKLOADS[name]
    _, Wcodes, Walpha, Wc, Wa = quantized_model(amq, wl)
    ins = synth.inputs(wl)
    xs, h0 = ins["x_seq"], ins["h0"]
    c0 = ins.get("c0")
    lstm = wl.cell == "lstm"
    ws = amq.new_workspace(wl.I, wl.H, wl.batch, wl.k_a)
    if lstm:
        g_seq, g_last, g_c = amq.lstm_sequence(Wcodes, Walpha, None, wl.I, wl.H, dev(xs), dev(h0), dev(c0), wl.k_a, wl.T,
                                               ws, want_h_seq=True)
    else:
        g_seq, g_last = amq.gru_sequence(Wcodes, Walpha, None, wl.I, wl.H, dev(xs), dev(h0), wl.k_a, wl.T, ws,
                                         want_h_seq=True)
    assert amq.workspace_status(ws) == 0 and amq.device_status() == 0
    assert torch.equal(g_seq[-1], g_last)
    sample_steps = (0, 1, 16, 34)
    sample_seqs = (0, wl.batch // 2 + 1)
    h, c = dev(h0), (dev(c0) if lstm else None)
    for s in range(wl.steps):
        h_prev, c_prev = h, c
        if lstm:
            h, c = amq.lstm_step(Wcodes, Walpha, None, wl.I, wl.H, dev(xs[s]), h_prev, c_prev, wl.k_a, wl.T, ws)
        else:
            h = amq.gru_step(Wcodes, Walpha, None, wl.I, wl.H, dev(xs[s]), h_prev, wl.k_a, wl.T, ws)
        assert torch.equal(h, g_seq[s]), s
        if s in sample_steps:
            for b in sample_seqs:
                xb = xs[s][b:b + 1]
                hp = h_prev[b:b + 1].cpu().numpy()
                _, beta = oracle.quantize_rows(np.concatenate([xb, hp], axis=1).astype(np.float64), wl.k_a, wl.T)
                tol = state_tolerance(Wa, beta, wl.n)
                if lstm:
                    cp = c_prev[b:b + 1].cpu().numpy()
                    h_ref, c_ref = oracle.lstm_step(Wc, Wa, None, wl.I, wl.H, xb, hp, cp, wl.k_a, wl.T)
                    assert np.abs(c[b:b + 1].cpu().numpy() - c_ref).max() <= tol, (s, b)
                else:
                    h_ref = oracle.gru_step(Wc, Wa, None, wl.I, wl.H, xb, hp, wl.k_a, wl.T)
                assert np.abs(h[b:b + 1].cpu().numpy() - h_ref).max() <= tol, (s, b)
    if lstm:
        assert torch.equal(c, g_c)


@pytest.mark.parametrize("name", ["lstm1024_b64", "gru2048_b256"])
def test_batched_cell_step_workloads(amq, name):
    """One full-size step of the batched layers (quantizer kernel + tensor-core product with gate epilogue)."""
    wl = synth.WORKLOADS[name]
    _, Wcodes, Walpha, Wc, Wa = quantized_model(amq, wl)
    x = synth.inputs(wl)["x_seq"][3]
    h = synth.uniform((wl.batch, wl.H), -1, 1, 7, 1)
    c = synth.uniform((wl.batch, wl.H), -1, 1, 7, 2)
    bias = synth.normal((4 * wl.H,), 0.1, 7, 3)
    ws = amq.new_workspace(wl.I, wl.H, wl.batch, wl.k_a)
    _, beta = oracle.quantize_rows(np.concatenate([x, h], axis=1).astype(np.float64), wl.k_a, wl.T)
    tol = state_tolerance(Wa, beta, wl.n)
    if wl.cell == "lstm":
        h_g, c_g = amq.lstm_step(Wcodes, Walpha, dev(bias), wl.I, wl.H, dev(x), dev(h), dev(c), wl.k_a, wl.T, ws)
        h_ref, c_ref = oracle.lstm_step(Wc, Wa, bias, wl.I, wl.H, x, h, c, wl.k_a, wl.T)
        assert np.abs(c_g.cpu().numpy() - c_ref).max() <= tol
    else:
        h_g = amq.gru_step(Wcodes, Walpha, dev(bias), wl.I, wl.H, dev(x), dev(h), wl.k_a, wl.T, ws)
        h_ref = oracle.gru_step(Wc, Wa, bias, wl.I, wl.H, x, h, wl.k_a, wl.T)
    err = np.abs(h_g.cpu().numpy() - h_ref)
    assert err.max() <= tol, (err.max(), tol)
    assert amq.workspace_status(ws) == 0 and amq.device_status() == 0
    # the activation quantizer alone, at this batch, against the oracle (staged protocol, sampled vectors)
    z = np.concatenate([x, h], axis=1)[:: max(1, wl.batch // 32)]
    parity.compare_quantizer(z, wl.k_a, wl.T, lambda a, k, T: tuple(
        f(t) for f, t in zip((codes_np, lambda t: t.cpu().numpy()), amq.quantize(dev(a), k, T))))


def test_projection_workload_bulk_quantization_and_product(amq):
    wl = synth.WORKLOADS["proj32768_b512"]
    W = synth.weights(wl)
    dW = dev(W)
    sample = np.arange(0, wl.m, 61)                  # 538 of the 32768 rows

    def gpu_rows(_x, k, T):                          # full-size launch, sampled rows returned
        codes, coeffs = amq.quantize(dW, k, T)
        torch.cuda.synchronize()
        return codes_np(codes)[sample], coeffs.cpu().numpy()[sample]

    stats = parity.compare_quantizer(W[sample], wl.k_w, wl.T, gpu_rows)
    print(stats)
    Wcodes, Walpha = amq.quantize(dW, wl.k_w, wl.T)
    acts = synth.inputs(wl)["acts"]
    Xc, Xb = oracle.quantize_rows(acts.astype(np.float64), wl.k_a, wl.T)
    dXc = torch.from_numpy(Xc.view(np.int32)).cuda()
    y = amq.binary_gemm(Wcodes, Walpha, dXc, dev(Xb), wl.n).cpu().numpy().astype(np.float64)
    assert amq.device_status() == 0
    Wc, Wa = codes_np(Wcodes), Walpha.cpu().numpy().astype(np.float64)
    ref = oracle.binary_gemm(Wc[sample], Wa[sample], Xc, Xb, wl.n)
    assert np.all(np.abs(y[:, sample] - ref) <= parity.output_tolerance(Wa[sample], Xb, wl.n) + 1e-6)
    assert np.abs(y[:, sample] - ref).max() <= 1e-5 * (np.abs(ref).max() + 1)
    # integer partials, bit-exact, on a block of rows that spans tile boundaries
    rows = slice(4000, 4300)
    D = amq.binary_dots(Wcodes[rows].contiguous(), dXc, wl.n).cpu().numpy()
    assert np.array_equal(D, oracle.binary_dots(Wc[rows], Xc, wl.n))
