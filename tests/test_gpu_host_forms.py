"""GPU parity of the host-buffer entry points (the calls bench.py's end-to-end leg times) and of
sbc_encode_ex with timing marks, against the CPU oracle, through the C ABI.

sbc_encode_host / sbc_decode_accumulate_host take the update and the messages from host memory and
hand the container and the dense sum back to host memory; everything in between is the same
kernels as sbc_encode / sbc_decode_accumulate, so the bar is the same: container bytes, mu and
residual bit-exact, dense sum exact for one client and within 1e-6 * sum |mu_c| for several.
"""
import concurrent.futures

import numpy as np
import pytest
import torch

import oracle
from paper_1805_08768_b200 import binding as sbc
from paper_1805_08768_b200 import workloads

pytestmark = pytest.mark.gpu

if not torch.cuda.is_available():  # pragma: no cover
    pytest.skip("needs a CUDA device", allow_module_level=True)

DEV = torch.device("cuda:0")


def host_buffer(numel, dtype, pinned):
    return torch.empty(numel, dtype=dtype, pin_memory=pinned)


class HostClient:
    """Buffers of one client that encodes from host memory, and of the server that decodes to it."""

    def __init__(self, n, p, pinned):
        self.n, self.p = n, p
        cap = sbc.sbc_stream_bytes(n, p)
        self.cap = cap
        self.upd_host = host_buffer(n, torch.float32, pinned)
        self.msg_host = host_buffer(cap, torch.uint8, pinned)
        self.dense_host = host_buffer(n, torch.float32, pinned)
        self.upd_dev = torch.empty(n, dtype=torch.float32, device=DEV)
        self.res_dev = torch.zeros(n, dtype=torch.float32, device=DEV)
        self.msg_dev = torch.empty(cap, dtype=torch.uint8, device=DEV)
        self.ws = torch.empty(sbc.sbc_workspace_bytes(n, p), dtype=torch.uint8, device=DEV)
        self.dense_dev = torch.empty(n, dtype=torch.float32, device=DEV)
        self.staging = torch.empty(cap + 64, dtype=torch.uint8, device=DEV)

    def encode(self, upd, stream=None):
        self.upd_host.copy_(torch.from_numpy(upd))
        return sbc.sbc_encode_host(self.upd_host, self.upd_dev, self.res_dev, self.p, self.msg_host, self.msg_dev,
                                   self.ws, stream=stream)

    def decode(self, nbytes, stream=None):
        return sbc.sbc_decode_accumulate_host([self.msg_host], [nbytes], self.dense_host, self.dense_dev,
                                              self.staging, stream=stream)


@pytest.mark.parametrize("pinned", [True, False], ids=["pinned", "pageable"])
@pytest.mark.parametrize("n,p", [(300001, 0.01), (1 << 21, 0.001)])
def test_host_forms_three_rounds_against_the_oracle(n, p, pinned):
    cl = HostClient(n, p, pinned)
    want_res = np.zeros(n, dtype=np.float32)
    for rnd in range(3):
        upd = workloads.normal_flat(n, 1e-3, workloads.seed_for(1, rnd, 3))
        want_stream, want_mu = oracle.encode(upd, want_res, p)       # carries want_res
        nbytes, mu = cl.encode(upd)
        assert nbytes == want_stream.size
        assert np.array_equal(cl.msg_host[:nbytes].numpy(), want_stream)
        assert np.float32(mu).view(np.uint32) == want_mu.view(np.uint32)
        assert np.array_equal(cl.res_dev.cpu().numpy().view(np.uint32), want_res.view(np.uint32))
        cl.dense_host.fill_(7.0)                                      # must be overwritten, not added to
        assert cl.decode(nbytes) == 0
        want_dense = np.zeros(n, dtype=np.float32)
        oracle.decode_accumulate([want_stream], want_dense)
        assert np.array_equal(cl.dense_host.numpy().view(np.uint32), want_dense.view(np.uint32))


def test_host_decode_of_several_clients():
    n, p, n_clients = 400000, 0.001, 5
    msgs, sizes, mus, streams_np = [], [], [], []
    for c in range(n_clients):
        cl = HostClient(n, p, pinned=True)
        nbytes, mu = cl.encode(workloads.normal_flat(n, 1e-3, workloads.seed_for(4, 0, c)))
        msgs.append(cl.msg_host)
        sizes.append(nbytes)
        mus.append(abs(mu))
        streams_np.append(cl.msg_host[:nbytes].numpy().copy())
    want = np.zeros(n, dtype=np.float32)
    oracle.decode_accumulate(streams_np, want)
    dense_host = torch.empty(n, dtype=torch.float32, pin_memory=True)
    dense_dev = torch.empty(n, dtype=torch.float32, device=DEV)
    staging = torch.empty(sum((s + 15) // 16 * 16 for s in sizes) + 16, dtype=torch.uint8, device=DEV)
    assert sbc.sbc_decode_accumulate_host(msgs, sizes, dense_host, dense_dev, staging) == 0
    got = dense_host.numpy()
    assert np.array_equal(got != 0, want != 0)
    assert np.max(np.abs(got.astype(np.float64) - want)) <= 1e-6 * sum(mus)


def test_overlapped_host_forms_two_streams_two_threads():
    """The form the end-to-end timing uses: every encode (host thread A, CUDA stream A) overlaps the
    decode of the previous message (host thread B, CUDA stream B)."""
    n, ps = 1 << 20, (1e-2, 1e-3, 1e-4)
    clients = [HostClient(n, p, pinned=True) for p in ps]
    want_res = [np.zeros(n, dtype=np.float32) for _ in ps]
    enc_stream, dec_stream = torch.cuda.Stream(device=DEV), torch.cuda.Stream(device=DEV)
    pool = concurrent.futures.ThreadPoolExecutor(max_workers=1)
    pending = None  # (future, client index, expected dense)

    def settle():
        nonlocal pending
        if pending is None:
            return
        fut, i, want_dense = pending
        assert fut.result() == 0
        assert np.array_equal(clients[i].dense_host.numpy().view(np.uint32), want_dense.view(np.uint32))
        pending = None

    for rnd in range(2):
        upd = workloads.student_t_flat(n, workloads.seed_for(5, rnd))
        for i, p in enumerate(ps):
            want_stream, want_mu = oracle.encode(upd, want_res[i], p)
            nbytes, mu = clients[i].encode(upd, stream=enc_stream)
            assert np.array_equal(clients[i].msg_host[:nbytes].numpy(), want_stream)
            assert np.float32(mu).view(np.uint32) == want_mu.view(np.uint32)
            settle()
            want_dense = np.zeros(n, dtype=np.float32)
            oracle.decode_accumulate([want_stream], want_dense)
            pending = (pool.submit(clients[i].decode, nbytes, dec_stream), i, want_dense)
    settle()
    torch.cuda.synchronize()
    for i in range(len(ps)):
        assert np.array_equal(clients[i].res_dev.cpu().numpy().view(np.uint32), want_res[i].view(np.uint32))


def test_host_encode_argument_errors_enqueue_nothing():
    n, p = 100000, 0.01
    cl = HostClient(n, p, pinned=True)
    cl.upd_host.fill_(1.0)
    cl.upd_dev.fill_(-5.0)
    torch.cuda.synchronize()
    small_ws = cl.ws[:4096]
    with pytest.raises(sbc.SbcError) as e:
        sbc.sbc_encode_host(cl.upd_host, cl.upd_dev, cl.res_dev, p, cl.msg_host, cl.msg_dev, small_ws)
    assert e.value.code == sbc.SBC_ECAPACITY
    with pytest.raises(sbc.SbcError) as e:
        sbc.sbc_encode_host(cl.upd_host, cl.upd_dev, cl.res_dev, 1.5, cl.msg_host, cl.msg_dev, cl.ws)
    assert e.value.code == sbc.SBC_EINVAL
    with pytest.raises(sbc.SbcError) as e:   # message buffers below the bound for (n, p)
        sbc.sbc_encode_host(cl.upd_host, cl.upd_dev, cl.res_dev, p, cl.msg_host[:64], cl.msg_dev[:64], cl.ws)
    assert e.value.code == sbc.SBC_ECAPACITY
    with pytest.raises(sbc.SbcError) as e:   # residual aliasing the device copy of the update
        sbc.sbc_encode_host(cl.upd_host, cl.upd_dev, cl.upd_dev, p, cl.msg_host, cl.msg_dev, cl.ws)
    assert e.value.code == sbc.SBC_EINVAL
    torch.cuda.synchronize()
    assert bool((cl.upd_dev == -5.0).all()), "a refused call copied the update to the device"


def test_host_decode_checks_headers_against_the_received_length():
    n, p = 200000, 0.01
    cl = HostClient(n, p, pinned=True)
    nbytes, _ = cl.encode(workloads.normal_flat(n, 1e-3, 6))
    good = cl.msg_host[:nbytes].numpy().copy()

    def run(mutated, length):
        msg = torch.from_numpy(mutated.copy())
        cl.dense_host.fill_(3.0)
        with pytest.raises(sbc.SbcError) as e:
            sbc.sbc_decode_accumulate_host([msg], [length], cl.dense_host, cl.dense_dev, cl.staging)
        assert e.value.code == sbc.SBC_ECORRUPT
        assert bool((cl.dense_host == 3.0).all()), "a refused message changed the host result"

    run(good, nbytes - 16)                                  # a message cut short
    bad = good.copy(); bad[24:32].view("<u8")[0] += 8 * 4096     # nbits beyond the received bytes
    run(bad, nbytes)
    bad = good.copy(); bad[8:16].view("<u8")[0] = n + 1          # another tensor's message
    run(bad, nbytes)
    bad = good.copy(); bad[0] ^= 1
    run(bad, nbytes)


def test_encode_ex_with_marks_gives_the_bytes_of_sbc_encode():
    n, p = 1 << 20, 0.01
    upd = workloads.student_t_flat(n, 91)
    u = torch.from_numpy(upd).to(DEV)
    cap, wsb = sbc.sbc_stream_bytes(n, p), sbc.sbc_workspace_bytes(n, p)
    ws = torch.empty(wsb, dtype=torch.uint8, device=DEV)
    outs, ress, mus = [], [], []
    for with_marks in (False, True):
        r = torch.zeros(n, dtype=torch.float32, device=DEV)
        out = torch.zeros(cap, dtype=torch.uint8, device=DEV)
        mu = torch.zeros(1, dtype=torch.float32, device=DEV)
        if with_marks:
            marks = [torch.cuda.Event(enable_timing=True) for _ in range(sbc.MARK_COUNT)]
            for m in marks:
                m.record()
            sbc.sbc_encode_ex(u, r, p, out, mu, ws, marks)
            torch.cuda.synchronize()
            times = [marks[i].elapsed_time(marks[i + 1]) for i in range(sbc.MARK_COUNT - 1)]
            assert all(t >= 0.0 for t in times) and sum(times) > 0.0   # recorded in stage order on the stream
        else:
            sbc.sbc_encode(u, r, p, out_stream=out, out_mu=mu, workspace=ws)
        info = sbc.sbc_stream_info_get(out)
        outs.append(out[: info.total_bytes].cpu().numpy())
        ress.append(r.cpu().numpy())
        mus.append(mu.item())
    assert np.array_equal(outs[0], outs[1]) and mus[0] == mus[1]
    assert np.array_equal(ress[0].view(np.uint32), ress[1].view(np.uint32))
    want_res = np.zeros(n, dtype=np.float32)
    want_stream, _ = oracle.encode(upd, want_res, p)
    assert np.array_equal(outs[1], want_stream)
