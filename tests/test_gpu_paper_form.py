"""GPU parity of the LSTM in the paper's own form (separate W_i / W_h, inputs = rows of the quantized embedding,
only h quantized on-line) against the oracle, teacher-forced per step, and of the embedding gather (bit-exact)."""
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


def cdev(c):
    return torch.from_numpy(np.ascontiguousarray(c).view(np.int32)).cuda()


def model(I, H, vocab, kw, ke, seed):
    Wi = synth.normal((4 * H, I), 0.05, seed, 1).astype(np.float64)
    Wh = synth.normal((4 * H, H), 0.05, seed, 2).astype(np.float64)
    We = synth.normal((vocab, I), 0.5, seed, 3).astype(np.float64)
    bias = synth.normal((4 * H,), 0.1, seed, 4)
    return oracle.quantize_rows(Wi, kw, 2), oracle.quantize_rows(Wh, kw, 2), oracle.quantize_rows(We, ke, 2), bias


def test_embedding_rows_is_a_bit_exact_gather(amq):
    vocab, n, k = 97, 300, 3
    Wec, Wea = oracle.quantize_rows(synth.normal((vocab, n), 0.5, 3, 1).astype(np.float64), k, 2)
    tokens = (synth.uniform01(5 * 7, 3, 2) * vocab).astype(np.int32).reshape(5, 7)
    tokens[0, 0], tokens[0, 1] = -4, vocab + 9                      # clamped
    xc, xb = amq.embedding_rows(cdev(Wec), dev(Wea), n, torch.from_numpy(tokens).cuda())
    t = np.clip(tokens, 0, vocab - 1)
    assert np.array_equal(xc.cpu().numpy().view(np.uint32), Wec[t])
    assert np.array_equal(xb.cpu().numpy(), Wea[t].astype(np.float32))


@pytest.mark.parametrize("I,H,kw,ke,ka,batch,steps", [(64, 40, 2, 2, 2, 1, 4), (100, 129, 3, 2, 3, 5, 3),
                                                      (256, 256, 2, 3, 2, 20, 5), (1024, 1024, 3, 3, 3, 64, 3)])
def test_paper_form_sequence_and_steps(amq, I, H, kw, ke, ka, batch, steps):
    vocab = 211
    (Wic, Wia), (Whc, Wha), (Wec, Wea), bias = model(I, H, vocab, kw, ke, 90 + H)
    tokens = (synth.uniform01(steps * batch, 91, 1) * vocab).astype(np.int32).reshape(steps, batch)
    h0 = synth.uniform((batch, H), -1, 1, 91, 2)
    c0 = synth.uniform((batch, H), -1, 1, 91, 3)
    d = dict(Wic=cdev(Wic), Wia=dev(Wia), Whc=cdev(Whc), Wha=dev(Wha), bias=dev(bias))
    xc_seq, xb_seq = amq.embedding_rows(cdev(Wec), dev(Wea), I, torch.from_numpy(tokens).cuda())
    ws = amq.new_paper_workspace(H, batch, steps, ka)
    g_seq, g_last, g_c = amq.lstm_sequence_paper(d["Wic"], d["Wia"], d["Whc"], d["Wha"], d["bias"], I, H, xc_seq, xb_seq,
                                                 dev(h0), dev(c0), ka, 2, ws, want_h_seq=True)
    assert amq.device_status() == 0
    assert torch.equal(g_seq[-1], g_last)
    # teacher-forced per step against the oracle, and the step call against the sequence call
    ws1 = amq.new_paper_workspace(H, batch, 1, ka)
    h, c = h0.astype(np.float64), c0.astype(np.float64)
    hg, cg = dev(h0), dev(c0)
    for s in range(steps):
        xc, xb = Wec[tokens[s]], Wea[tokens[s]]
        h_ref, c_ref = oracle.lstm_step_paper(Wic, Wia, Whc, Wha, bias, I, H, xc, xb, h, c, ka, 2)
        _, hbeta = oracle.quantize_rows(h, ka, 2)
        tol = 3.0 * (parity.output_tolerance(Wha, hbeta, H).max() + parity.output_tolerance(Wia, xb, I).max()) + 1e-6
        h_g, c_g = amq.lstm_step_paper(d["Wic"], d["Wia"], d["Whc"], d["Wha"], d["bias"], I, H, xc_seq[s], xb_seq[s],
                                       dev(h), dev(c), ka, 2, ws1)
        assert np.abs(h_g.cpu().numpy() - h_ref).max() <= tol and np.abs(c_g.cpu().numpy() - c_ref).max() <= tol
        # chained library steps reproduce the library's sequence bit for bit
        hg, cg = amq.lstm_step_paper(d["Wic"], d["Wia"], d["Whc"], d["Wha"], d["bias"], I, H, xc_seq[s], xb_seq[s],
                                     hg, cg, ka, 2, ws1)
        assert torch.equal(hg, g_seq[s])
        h, c = h_ref, c_ref
    assert torch.equal(cg, g_c)
    drift = np.abs(g_last.cpu().numpy() - h).max()
    print("free-running max |dh| after %d steps: %.3g" % (steps, drift))
    assert drift <= 0.05
