"""Algorithm 1 end to end (M simulated clients on one GPU, communication delay n), with the oracle
run in lock-step on the CPU as the checker.

The local SGD iterations are the model's business, not the method's: the oracle is handed the same
local updates the clients computed (they are inputs of the compression path) and must then
reproduce, round after round, every client's message and residual bit for bit and the averaged
weights within the decoder's tolerance (the device adds the clients' scaled means in no fixed
order)."""
import numpy as np
import pytest
import torch

import oracle
from paper_1805_08768_b200 import binding as sbc
from paper_1805_08768_b200.dsgd import DelayedSGD, ToyRegression

pytestmark = pytest.mark.gpu

if not torch.cuda.is_available():  # pragma: no cover
    pytest.skip("needs a CUDA device", allow_module_level=True)

DEV = torch.device("cuda:0")


@pytest.mark.parametrize("delay,p", [(1, 0.01), (10, 0.01), (10, 0.05)])
def test_delayed_sgd_rounds_in_lock_step_with_the_oracle(delay, p):
    m, rounds = 4, 6
    model = ToyRegression(m, DEV, seed=delay)
    momenta = [torch.ones_like(w) for w in model.weights]          # stands in for an optimiser's momentum
    run = DelayedSGD(model.weights, m, p, delay, model.local_update, momenta=momenta)
    want_w = [w.cpu().numpy().reshape(-1).copy() for w in model.weights]
    want_r = [[np.zeros(n, dtype=np.float32) for n in run.sizes] for _ in range(m)]
    want_m = [np.ones(n, dtype=np.float32) for n in run.sizes]
    loss0 = model.loss()
    sum_mu = [0.0] * len(run.sizes)
    for rnd in range(rounds):
        run.round()
        run.check()
        for t, n in enumerate(run.sizes):
            streams = []
            for c in range(m):
                upd = run.last_updates[c][t].cpu().numpy()          # the compression path's input
                stream, mu = oracle.encode(upd, want_r[c][t], p)    # carries want_r
                got = run.messages[c][t][: stream.size].cpu().numpy()
                assert np.array_equal(got, stream), f"round {rnd}, client {c}, tensor {t}: message differs"
                assert np.float32(run.mus[c][t].item()).view(np.uint32) == mu.view(np.uint32)
                assert np.array_equal(run.residuals[c][t].cpu().numpy().view(np.uint32), want_r[c][t].view(np.uint32))
                streams.append(stream)
                sum_mu[t] += abs(float(mu)) / m
            oracle.decode_apply(streams, 1.0 / m, want_w[t], want_m[t])   # W <- W + 1/M sum_i decode(msg_i)
            got_w = run.flat[t].cpu().numpy()
            tol = 1e-6 * (np.abs(want_w[t]) + sum_mu[t]) + 1e-30
            assert np.all(np.abs(got_w.astype(np.float64) - want_w[t]) <= tol), f"round {rnd}, tensor {t}: weights differ"
    # momentum masking: zero exactly where some client transmitted in some round
    for t in range(len(run.sizes)):
        assert np.array_equal(momenta[t].view(-1).cpu().numpy(), want_m[t])
        assert 0 < np.count_nonzero(want_m[t] == 0) or run.sizes[t] < 1 / p
    # and the loop trains: the averaged sparse binary updates lower the loss
    assert model.loss() < loss0


def test_more_delay_sends_fewer_messages_for_the_same_number_of_iterations():
    """Temporal sparsity (Section 2): n local iterations per round cut the messages per iteration by n."""
    m, p, iters = 4, 0.01, 20
    bits = {}
    for delay in (1, 10):
        model = ToyRegression(m, DEV, seed=3)
        run = DelayedSGD(model.weights, m, p, delay, model.local_update)
        sent = 0
        for _ in range(iters // delay):
            run.round()
            run.check()
            for c in range(m):
                for t in range(len(run.sizes)):
                    sent += int(sbc.sbc_stream_info_get(run.messages[c][t]).nbits) + 32   # positions + one fp32 mean
        bits[delay] = sent
    assert bits[10] * 5 < bits[1]
