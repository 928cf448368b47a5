"""The exchange step on the GPU: one NCCL rank end to end (encode -> all-gather -> decode and
apply), and the aggregate over several gathered messages (slots filled by hand, which is what
the all-gather leaves behind), both against the oracle."""
import numpy as np
import pytest
import torch
import torch.distributed as dist

import oracle
from paper_1805_08768_b200 import binding as sbc
from paper_1805_08768_b200 import workloads
from paper_1805_08768_b200.exchange import StreamExchange, exchange_round

pytestmark = pytest.mark.gpu

if not torch.cuda.is_available():  # pragma: no cover
    pytest.skip("needs a CUDA device", allow_module_level=True)

DEV = torch.device("cuda:0")


@pytest.fixture(scope="module")
def one_rank_group():
    torch.cuda.set_device(DEV)
    dist.init_process_group("nccl", init_method="tcp://127.0.0.1:29641", rank=0, world_size=1)
    try:
        yield
    finally:
        dist.destroy_process_group()


def test_one_rank_round_matches_the_oracle(one_rank_group):
    n, p = 700000, 0.01
    ex = StreamExchange.for_tensor(n, p, DEV)
    assert ex.world == 1 and ex.capacity >= sbc.sbc_stream_bytes(n, p)
    w0 = workloads.normal_flat(n, 0.05, 41)
    weights = torch.from_numpy(w0).to(DEV)
    residual = torch.zeros(n, dtype=torch.float32, device=DEV)
    status = torch.zeros(1, dtype=torch.int32, device=DEV)
    want_w, want_r = w0.copy(), np.zeros(n, dtype=np.float32)
    for rnd in range(3):                                     # residual carried across rounds
        upd = workloads.normal_flat(n, 1e-3, 50 + rnd)
        exchange_round(torch.from_numpy(upd).to(DEV), residual, p, weights, ex, status=status)
        stream, _ = oracle.encode(upd, want_r, p)
        oracle.decode_apply([stream], 1.0, want_w)
        torch.cuda.synchronize()
        assert status.item() == 0
        assert np.array_equal(ex.slots[0][: stream.size].cpu().numpy(), stream)
    assert np.array_equal(weights.cpu().numpy().view(np.uint32), want_w.view(np.uint32))
    assert np.array_equal(residual.cpu().numpy().view(np.uint32), want_r.view(np.uint32))


@pytest.mark.parametrize("ordered", [False, True])
def test_aggregate_over_gathered_messages(one_rank_group, ordered):
    n, p, clients = 400000, 0.01, 5
    ex = StreamExchange.for_tensor(n, p, DEV)
    # what an all-gather among `clients` ranks leaves on every rank: one message per slot
    ex.world = clients
    ex.recv = torch.zeros(clients * ex.capacity, dtype=torch.uint8, device=DEV)
    ex.slots = [ex.recv[c * ex.capacity:(c + 1) * ex.capacity] for c in range(clients)]
    streams, mus = [], []
    for c in range(clients):
        stream, mu = oracle.encode(workloads.normal_flat(n, 1e-3, 70 + c), np.zeros(n, dtype=np.float32), p)
        ex.slots[c][: stream.size] = torch.from_numpy(stream).to(DEV)
        streams.append(stream)
        mus.append(abs(float(mu)))
    w0 = workloads.normal_flat(n, 0.05, 42)
    m0 = workloads.normal_flat(n, 1.0, 43)
    want_w, want_m = w0.copy(), m0.copy()
    if ordered:      # one client after the other: W + s*mu_0 + s*mu_1 + ..., each addition rounded
        for stream in streams:
            oracle.decode_apply([stream], 1.0 / clients, want_w, want_m)
    else:            # Algorithm 1 as written: W + s * (sum over the clients)
        oracle.decode_apply(streams, 1.0 / clients, want_w, want_m)
    weights, momentum = torch.from_numpy(w0).to(DEV), torch.from_numpy(m0).to(DEV)
    status = torch.zeros(1, dtype=torch.int32, device=DEV)
    ex.aggregate(weights, momentum=momentum, status=status, ordered=ordered)
    torch.cuda.synchronize()
    assert status.item() == 0
    got = weights.cpu().numpy()
    if ordered:      # one client per launch in slot order: the same additions in the same order
        assert np.array_equal(got.view(np.uint32), want_w.view(np.uint32))
    else:            # any order of the (at most `clients`) additions per position
        tol = 1e-6 * (np.abs(w0).astype(np.float64) + sum(mus) / clients)
        assert np.all(np.abs(got.astype(np.float64) - want_w) <= tol)
    assert np.array_equal(momentum.cpu().numpy().view(np.uint32), want_m.view(np.uint32))
