"""The give-up path of bounded device-side waits, exercised without hurting the GPU: a status word written from
the host, and the batch-1 sequence kernel run with waits that are made to run out (a smaller bound on the same
bounded polls, expecting step tags nobody publishes).  Nothing here faults, traps or spins without a limit."""
import numpy as np
import pytest
import torch

from paper_1802_00150_b200 import synth

pytestmark = pytest.mark.gpu

TIMEOUT = -6


@pytest.fixture(scope="module")
def amq():
    assert torch.cuda.is_available(), "these tests need a CUDA device"
    from paper_1802_00150_b200 import amq as binding
    return binding


def dev(a):
    return torch.from_numpy(np.ascontiguousarray(a)).cuda()


def small_model(amq, I, H, k_w=2, seed=80):
    W = synth.normal((4 * H, I + H), 0.08, seed, 1)
    return amq.quantize(dev(W), k_w, 2)


def test_status_word_written_from_the_host_is_reported_and_cleared_by_the_next_call(amq):
    I, H, ka = 64, 48, 2
    Wcodes, Walpha = small_model(amq, I, H)
    for batch in (1, 5):                       # the persistent kernel and the two-kernel chain share the status word
        ws = amq.new_workspace(I, H, batch, ka)
        assert amq.workspace_status(ws) == 0
        ws[:4] = torch.tensor([1, 0, 0, 0], dtype=torch.uint8, device="cuda")
        assert amq.workspace_status(ws) == TIMEOUT
        assert amq.status_string(TIMEOUT) != ""
        x = dev(synth.uniform((batch, I), -1, 1, 81, 1))
        h = dev(synth.uniform((batch, H), -1, 1, 81, 2))
        c = dev(synth.uniform((batch, H), -1, 1, 81, 3))
        amq.lstm_step(Wcodes, Walpha, None, I, H, x, h, c, ka, 2, ws)
        assert amq.workspace_status(ws) == 0


@pytest.mark.parametrize("I,H,steps,limit", [(64, 48, 4, 64), (256, 300, 6, 200), (1024, 1024, 35, 1000)])
def test_waits_that_run_out_set_the_status_and_leave_the_context_usable(amq, I, H, steps, limit):
    ka = 2
    Wcodes, Walpha = small_model(amq, I, H)
    xs = dev(synth.normal((steps, 1, I), 1.0, 82, 1))
    h0 = torch.zeros((1, H), device="cuda")
    c0 = torch.zeros((1, H), device="cuda")
    ws = amq.new_workspace(I, H, 1, ka)
    want = amq.lstm_sequence(Wcodes, Walpha, None, I, H, xs, h0, c0, ka, 2, amq.new_workspace(I, H, 1, ka), want_h_seq=True)
    h_last, c_last = amq.selftest_sequence_give_up(Wcodes, Walpha, None, I, H, xs, h0, c0, ka, 2, ws, limit)
    assert amq.workspace_status(ws) == TIMEOUT          # every CTA gave up in step 1 and said so
    assert torch.all(h_last == 0) and torch.all(c_last == 0)      # outputs untouched
    # the same workspace, the same stream, the next call: status cleared, results as from a fresh workspace
    got = amq.lstm_sequence(Wcodes, Walpha, None, I, H, xs, h0, c0, ka, 2, ws, want_h_seq=True)
    assert amq.workspace_status(ws) == 0
    for g, w in zip(got, want):
        assert torch.equal(g, w)


def test_give_up_selftest_rejects_what_it_cannot_run(amq):
    I, H, ka = 64, 48, 2
    Wcodes, Walpha = small_model(amq, I, H)
    xs = dev(synth.normal((3, 1, I), 1.0, 83, 1))
    h0 = torch.zeros((1, H), device="cuda")
    ws = amq.new_workspace(I, H, 1, ka)
    for bad_limit in (0, 1 << 20):
        with pytest.raises(amq.AmqError) as e:
            amq.selftest_sequence_give_up(Wcodes, Walpha, None, I, H, xs, h0, h0.clone(), ka, 2, ws, bad_limit)
        assert e.value.status == -1
    with pytest.raises(amq.AmqError) as e:      # a single step waits for nothing: refused
        amq.selftest_sequence_give_up(Wcodes, Walpha, None, I, H, xs[:1], h0, h0.clone(), ka, 2, ws, 100)
    assert e.value.status == -1
