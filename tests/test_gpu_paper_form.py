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


@pytest.mark.parametrize("rows,n,ld", [(1, 42000, 42000), (7, 1000, 1000), (3, 33, 33), (2, 1, 1), (3, 1001, 1004),
                                       (2, 4099, 4100), (2, 50001, 50004), (2, 49152, 49152)])
def test_log_softmax_argmax(amq, rows, n, ld):
    """Rows read once into registers (aligned rows up to 49152 logits, with and without a ragged tail) and the
    three-pass kernel (longer or unaligned rows)."""
    z = synth.normal((rows, n), 3.0, 95 + n, 1)
    if n > 400:
        z[0, 17] = z[0, 400] = z[0].max() + 1.0                 # equal maxima: the first index wins
        z[-1, n - 1] = z[-1].max() + 2.0                        # the maximum in the ragged tail
    wide = torch.full((rows, ld), float("nan"), device="cuda")
    wide[:, :n] = dev(z)
    logp, arg = amq.log_softmax_argmax(wide[:, :n])
    ref, rarg = oracle.log_softmax_argmax(z.astype(np.float64))
    assert np.abs(logp.cpu().numpy() - ref).max() <= 2e-5       # fp32 sum of up to 42000 exponentials + one log
    assert np.array_equal(arg.cpu().numpy(), rarg)


def test_output_layer_at_vocabulary_scale_and_greedy_decoding(amq):
    """Text8-scale language-model step (Eq. 6 end to end): embedding row -> cell -> 42000 x 1024 output product
    -> log-softmax / arg-max, and the arg-max fed back as the next token without leaving the device."""
    I = H = 1024
    V, kw, ke, ka = 42000, 2, 2, 2
    (Wic, Wia), (Whc, Wha), _, bias = model(I, H, 8, kw, ke, 97)
    Wsc, Wsa = oracle.quantize_rows(synth.normal((V, H), 0.05, 97, 7).astype(np.float64), kw, 2)
    Wec, Wea = oracle.quantize_rows(synth.normal((V, I), 0.5, 97, 8).astype(np.float64), ke, 2)
    bs = synth.normal((V,), 0.1, 97, 9)
    d = dict(Wic=cdev(Wic), Wia=dev(Wia), Whc=cdev(Whc), Wha=dev(Wha), bias=dev(bias), Wsc=cdev(Wsc), Wsa=dev(Wsa),
             bs=dev(bs), Wec=cdev(Wec), Wea=dev(Wea))
    ws = amq.new_paper_workspace(H, 1, 1, ka)
    tokens = torch.tensor([1234], dtype=torch.int32, device="cuda")
    h, c = torch.zeros((1, H), device="cuda"), torch.zeros((1, H), device="cuda")
    ho, co = np.zeros((1, H)), np.zeros((1, H))
    tok_o = 1234
    for step in range(3):
        xc, xb = amq.embedding_rows(d["Wec"], d["Wea"], I, tokens)
        h, c = amq.lstm_step_paper(d["Wic"], d["Wia"], d["Whc"], d["Wha"], d["bias"], I, H, xc, xb, h, c, ka, 2, ws)
        hc, hb = amq.quantize(h, ka, 2)
        logits = amq.binary_gemm(d["Wsc"], d["Wsa"], hc, hb, H, bias=d["bs"])
        logp, tokens = amq.log_softmax_argmax(logits)
        # oracle, teacher-forced on the library's state of the previous step
        ho, co = oracle.lstm_step_paper(Wic, Wia, Whc, Wha, bias, I, H, Wec[[tok_o]], Wea[[tok_o]], ho, co, ka, 2)
        assert np.abs(h.cpu().numpy() - ho).max() <= 1e-3
        hc_o, hb_o = oracle.quantize_rows(ho, ka, 2)
        z_o = oracle.binary_gemm(Wsc, Wsa, hc_o, hb_o, H, bs.astype(np.float64))
        tol = parity.output_tolerance(Wsa, hb_o, H).max()
        assert np.abs(logits.cpu().numpy() - z_o).max() <= tol
        lp_o, arg_o = oracle.log_softmax_argmax(z_o)
        assert np.abs(logp.cpu().numpy() - lp_o).max() <= 2 * tol + 2e-5
        top2 = np.sort(z_o[0])[-2:]
        tok_g = int(tokens.cpu()[0])
        if top2[1] - top2[0] > 2 * tol:                         # the decision is unique within the tolerance
            assert tok_g == int(arg_o[0])
        else:
            assert z_o[0, tok_g] >= top2[1] - 2 * tol           # otherwise any near-maximal token is valid
        tok_o = tok_g                                           # follow the library's choice
        ho, co = h.cpu().numpy().astype(np.float64), c.cpu().numpy().astype(np.float64)


def test_native_greedy_decoding_equals_the_composed_calls_and_the_oracle_on_its_first_step(amq):
    """amq_lm_greedy_decode enqueues the same kernels as the call-by-call loop above (checked there against the oracle
    at every step): tokens, states and log-probabilities must agree bit for bit; the first step is also held against
    the oracle directly."""
    I, H, V, kw, ke, ka, steps = 96, 160, 3001, 3, 2, 2, 6
    (Wic, Wia), (Whc, Wha), _, bias = model(I, H, 8, kw, ke, 131)
    Wsc, Wsa = oracle.quantize_rows(synth.normal((V, H), 0.08, 131, 7).astype(np.float64), kw, 2)
    Wec, Wea = oracle.quantize_rows(synth.normal((V, I), 0.5, 131, 8).astype(np.float64), ke, 2)
    bs = synth.normal((V,), 0.1, 131, 9)
    h0 = synth.uniform((1, H), -1, 1, 131, 10)
    c0 = synth.uniform((1, H), -1, 1, 131, 11)
    d = dict(Wic=cdev(Wic), Wia=dev(Wia), Whc=cdev(Whc), Wha=dev(Wha), bias=dev(bias), Wsc=cdev(Wsc), Wsa=dev(Wsa),
             bs=dev(bs), Wec=cdev(Wec), Wea=dev(Wea))
    # native loop
    tokens = torch.zeros((steps + 1,), dtype=torch.int32, device="cuda")
    tokens[0] = 77
    h, c = dev(h0), dev(c0)
    logp = torch.empty((steps, V), device="cuda")
    ws = amq.new_decode_workspace(V, I, H, ke, ka)
    amq.lm_greedy_decode(d["Wec"], d["Wea"], d["Wic"], d["Wia"], d["Whc"], d["Wha"], d["bias"], d["Wsc"], d["Wsa"], d["bs"],
                         I, H, ka, 2, tokens, h, c, ws, logp=logp)
    assert amq.device_status() == 0
    # the same steps call by call
    pws = amq.new_paper_workspace(H, 1, 1, ka)
    tok = torch.tensor([77], dtype=torch.int32, device="cuda")
    h2, c2 = dev(h0), dev(c0)
    for t in range(steps):
        xc, xb = amq.embedding_rows(d["Wec"], d["Wea"], I, tok)
        h2, c2 = amq.lstm_step_paper(d["Wic"], d["Wia"], d["Whc"], d["Wha"], d["bias"], I, H, xc, xb, h2, c2, ka, 2, pws)
        hc, hb = amq.quantize(h2, ka, 2)
        logits = amq.binary_gemm(d["Wsc"], d["Wsa"], hc, hb, H, bias=d["bs"])
        lp, tok = amq.log_softmax_argmax(logits)
        assert int(tok[0]) == int(tokens[t + 1]), t
        assert torch.equal(lp[0], logp[t]), t
    assert torch.equal(h2, h) and torch.equal(c2, c)
    # first step against the oracle
    ho, co = oracle.lstm_step_paper(Wic, Wia, Whc, Wha, bias, I, H, Wec[[77]], Wea[[77]], h0.astype(np.float64),
                                    c0.astype(np.float64), ka, 2)
    hc_o, hb_o = oracle.quantize_rows(ho, ka, 2)
    z_o = oracle.binary_gemm(Wsc, Wsa, hc_o, hb_o, H, bs.astype(np.float64))
    lp_o, _ = oracle.log_softmax_argmax(z_o)
    tol = parity.output_tolerance(Wsa, hb_o, H).max()
    assert np.abs(logp[0].cpu().numpy() - lp_o[0]).max() <= 2 * tol + 2e-5


def test_native_greedy_decoding_repeats_bit_for_bit(amq):
    """The kernels of the decoding chain are launched as programmatic dependents of one another (each waits for its
    predecessor first thing): a read that slipped ahead of a wait would show as run-to-run differences."""
    I, H, V, k, steps = 128, 256, 5000, 2, 24
    g = torch.Generator(device="cuda")
    g.manual_seed(7)
    q = lambda shape, std: amq.quantize(torch.randn(shape, device="cuda", generator=g) * std, k, 2)
    (Wic, Wia), (Whc, Wha), (Wec, Wea), (Wsc, Wsa) = q((4 * H, I), 0.05), q((4 * H, H), 0.05), q((V, I), 0.5), q((V, H), 0.08)
    bs = torch.randn((V,), device="cuda", generator=g) * 0.1
    ws = amq.new_decode_workspace(V, I, H, k, k)
    runs = []
    for _ in range(5):
        tokens = torch.zeros((steps + 1,), dtype=torch.int32, device="cuda")
        tokens[0] = 3
        h, c = torch.zeros((1, H), device="cuda"), torch.zeros((1, H), device="cuda")
        logp = torch.empty((steps, V), device="cuda")
        amq.lm_greedy_decode(Wec, Wea, Wic, Wia, Whc, Wha, None, Wsc, Wsa, bs, I, H, k, 2, tokens, h, c, ws, logp=logp)
        runs.append((tokens.clone(), h.clone(), c.clone(), logp.clone()))
    for r in runs[1:]:
        assert all(torch.equal(a, b) for a, b in zip(r, runs[0]))
    assert torch.unique(runs[0][0]).numel() > 3
