"""The LSTM step that brings its own scratch memory (amq_lstm_step_static).

It exists for callers that may not allocate on the device: code running inside a host application's
fixed memory budget, or a serving loop that has to stay out of the driver's allocator once it is up.
The test drives it through the C ABI and checks it against the ordinary entry point, which takes a
caller-provided workspace, on two calls in a row (the second call finds the scratch array as the first
one left it, with different contents and a different size in use).

This file sorts last on purpose: a run that stops at the first failure has then already been through
every other test.  It must also pass alone in a fresh process, where its first call is the one that
looks up the scratch array's device address.
"""
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


def one_case(amq, I, H, kw, ka, batch, seed):
    n = I + H
    W = synth.normal((4 * H, n), 0.05, seed, 1).astype(np.float64)
    Wc, Wa = oracle.quantize_rows(W, kw, 2)
    bias = synth.normal((4 * H,), 0.1, seed, 2)
    x = synth.uniform((batch, I), -1, 1, seed, 3)
    h = synth.uniform((batch, H), -1, 1, seed, 4)
    c = synth.uniform((batch, H), -1, 1, seed, 5)
    dWc = torch.from_numpy(Wc.view(np.int32)).cuda()
    dWa, dbias, dx, dh, dc = dev(Wa), dev(bias), dev(x), dev(h), dev(c)

    ws = amq.new_workspace(I, H, batch, ka)
    h_ref, c_ref = amq.lstm_step(dWc, dWa, dbias, I, H, dx, dh, dc, ka, 2, ws)
    h_out, c_out = torch.full_like(dh, 7.0), torch.full_like(dc, 7.0)
    amq.lstm_step_static(dWc, dWa, dbias, I, H, dx, dh, dc, ka, 2, h_out, c_out)
    torch.cuda.synchronize()

    # same tolerance as the cell parity tests: the pre-activation tolerance carried through the gates
    _, beta = oracle.quantize_rows(np.concatenate([x, h], axis=1).astype(np.float64), ka, 2)
    tol = 3.0 * parity.output_tolerance(Wa, beta, n).max() + 1e-6
    assert (h_out - h_ref).abs().max().item() <= tol
    assert (c_out - c_ref).abs().max().item() <= tol
    # and against the oracle itself
    o_h, o_c = oracle.lstm_step(Wc, Wa, bias, I, H, x, h, c, ka, 2)
    assert np.abs(h_out.cpu().numpy() - o_h).max() <= tol
    assert np.abs(c_out.cpu().numpy() - o_c).max() <= tol


def test_static_scratch_step_matches_workspace_step_twice_in_a_row(amq):
    # first call: many sequences, long vector (fills a large part of the scratch array);
    # second call: batch 1, short ragged vector (the ordinary entry point takes its persistent kernel here)
    one_case(amq, 256, 192, 3, 3, 33, 80)
    one_case(amq, 100, 77, 2, 2, 1, 81)
    # and once more with the first shape: contents left by the small call must not matter
    one_case(amq, 256, 192, 3, 3, 33, 82)


def test_static_scratch_limit_is_enforced_before_any_launch(amq):
    I, H, ka = 4096, 4096, 4
    wpr = amq.words_per_row(I + H)
    batch = amq.STATIC_SCRATCH_BYTES // (ka * wpr * 4) + 1          # one vector too many
    assert amq.lstm_step_static_scratch_bytes(I, H, batch, ka) > amq.STATIC_SCRATCH_BYTES
    assert amq.lstm_step_static_scratch_bytes(I, H, batch - 2, ka) <= amq.STATIC_SCRATCH_BYTES
    before = amq.kernel_launches()
    fake = torch.empty(16, dtype=torch.int32, device="cuda")         # never read: the call is refused first
    f32 = torch.empty(16, dtype=torch.float32, device="cuda")
    st = amq._lib.amq_lstm_step_static(fake.data_ptr(), f32.data_ptr(), None, I, H, 2, f32.data_ptr(),
                                       f32.data_ptr(), f32.data_ptr(), batch, ka, 2,
                                       fake.data_ptr(), fake.data_ptr() + 64, None)
    assert st == -4 and "workspace" in amq.status_string(st)
    assert amq.kernel_launches() == before
