"""GPU parity beyond the workload configurations: random shapes, the exact route at scale,
concurrent calls on two streams, and the largest tensor the interface accepts (2^31 - 1)."""
import zlib

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


def encode_on_gpu(upd, res, p, stream=None):
    u = torch.from_numpy(upd).to(DEV)
    r = torch.from_numpy(res).to(DEV)
    out, mu = sbc.sbc_encode(u, r, p, stream=stream)
    return u, r, out, mu


def fetch(out, mu, r):
    info = sbc.sbc_stream_info_get(out)
    torch.cuda.synchronize()
    return out[: info.total_bytes].cpu().numpy(), np.float32(mu.item()), r.cpu().numpy()


def assert_matches_oracle(upd, res, p, got):
    want_res = res.copy()
    want_stream, want_mu = oracle.encode(upd, want_res, p)
    stream, mu, new_res = got
    assert np.array_equal(stream, want_stream)
    assert mu.view(np.uint32) == want_mu.view(np.uint32)
    assert np.array_equal(new_res.view(np.uint32), want_res.view(np.uint32))


@pytest.mark.parametrize("case", range(40))
def test_random_sizes_sparsities_and_distributions(case):
    rng = np.random.default_rng(1000 + case)
    n = int(rng.integers(1, 400000))
    p = float(10.0 ** rng.uniform(-4.5, -0.35))
    kind = case % 5
    if kind == 0:
        upd = rng.standard_normal(n)
    elif kind == 1:
        upd = rng.standard_t(2, n)
    elif kind == 2:
        upd = np.round(rng.standard_normal(n) * 3) / 3            # heavy ties
    elif kind == 3:
        upd = rng.standard_normal(n) * (rng.random(n) < 0.05)      # mostly zeros
    else:
        upd = np.abs(rng.standard_normal(n)) * (1 if case % 2 else -1)  # one-signed
    upd = (upd * 10.0 ** rng.integers(-6, 3)).astype(np.float32)
    res = (rng.standard_normal(n) * float(np.abs(upd).mean() + 1e-12)).astype(np.float32) if case % 3 else \
        np.zeros(n, dtype=np.float32)
    _, r, out, mu = encode_on_gpu(upd, res, p)
    assert_matches_oracle(upd, res, p, fetch(out, mu, r))


@pytest.mark.parametrize("case", range(6))
def test_long_lists_with_certain_and_band_parts(case):
    # k >= 32768: the candidate lists are split at the sample's upper bound of the threshold
    rng = np.random.default_rng(5000 + case)
    n = int(rng.integers(1 << 21, 3_500_000))
    p = float(10.0 ** rng.uniform(-1.7, -0.5))
    if case == 0:
        upd = rng.standard_normal(n)
    elif case == 1:
        upd = rng.standard_t(2, n)
    elif case == 2:
        upd = np.round(rng.standard_normal(n) * 8) / 8               # heavy ties around the threshold
    elif case == 3:
        upd = rng.standard_normal(n) * (rng.random(n) < 0.3)          # mostly zeros
    elif case == 4:
        upd = -np.abs(rng.standard_normal(n))                         # one-signed
    else:
        upd = rng.standard_normal(n)
        upd[::7] = rng.choice([-3.0, 3.0, 2.5], size=upd[::7].size)   # blocks of equal large values
    upd = (upd * 10.0 ** rng.integers(-5, 2)).astype(np.float32)
    res = (rng.standard_normal(n) * float(np.abs(upd).mean())).astype(np.float32) if case % 2 else \
        np.zeros(n, dtype=np.float32)
    assert oracle.kept_count(n, p) >= 32768
    _, r, out, mu = encode_on_gpu(upd, res, p)
    assert_matches_oracle(upd, res, p, fetch(out, mu, r))


@pytest.mark.parametrize("pattern", ["all_zero", "plus_minus_one", "two_values", "sparse_spikes"])
def test_exact_route_at_scale(pattern):
    n, p = 1 << 22, 0.01
    rng = np.random.default_rng(zlib.crc32(pattern.encode()))
    if pattern == "all_zero":
        upd = np.zeros(n, dtype=np.float32)
    elif pattern == "plus_minus_one":
        upd = rng.choice(np.array([-1.0, 1.0], dtype=np.float32), n)
    elif pattern == "two_values":
        upd = rng.choice(np.array([0.25, 0.5], dtype=np.float32), n)
    else:
        upd = np.zeros(n, dtype=np.float32)
        upd[rng.choice(n, 5000, replace=False)] = rng.standard_normal(5000).astype(np.float32)
    res = np.zeros(n, dtype=np.float32)
    u, r, out, mu = encode_on_gpu(upd, res, p)
    ws_probe = torch.empty(sbc.sbc_workspace_bytes(n, p), dtype=torch.uint8, device=DEV)
    r2 = torch.from_numpy(res).to(DEV)
    out2 = torch.empty_like(out)
    sbc.sbc_encode(u, r2, p, out_stream=out2, workspace=ws_probe)
    assert sbc.sbc_encode_diag_get(ws_probe).exact_route == 1      # these inputs defeat the sampled bounds
    assert_matches_oracle(upd, res, p, fetch(out, mu, r))


def test_two_streams_with_their_own_workspaces_run_concurrently():
    n, p = 3_000_000, 0.01
    cases = [(workloads.normal_flat(n, 1e-3, 71), 0.01), (workloads.student_t_flat(n, 72), 0.001)]
    streams = [torch.cuda.Stream(device=DEV) for _ in cases]
    torch.cuda.synchronize()
    launched = []
    for (upd, pp), st in zip(cases, streams):
        with torch.cuda.stream(st):
            for _ in range(3):   # several rounds back to back on each stream
                launched.append((upd, pp, encode_on_gpu(upd, np.zeros(n, dtype=np.float32), pp, stream=st)))
    torch.cuda.synchronize()
    for upd, pp, (_, r, out, mu) in launched:
        assert_matches_oracle(upd, np.zeros(n, dtype=np.float32), pp, fetch(out, mu, r))


def test_largest_tensor_the_interface_accepts():
    # numel = 2^31 - 1: positions still fit 31 bits; expected result from torch.topk (independent of
    # the library) + the oracle's exact sum, decision and container builder
    n, p = (1 << 31) - 1, 1e-4
    assert sbc.sbc_stream_bytes(n + 1, p) == 0 and sbc.sbc_workspace_bytes(n + 1, p) == 0
    update = workloads.student_t_flat_torch(n, 99, DEV)
    update[n - 1] = 50.0              # make sure the very last position is transmitted
    update[0] = 49.0
    k = oracle.kept_count(n, p)
    top = torch.topk(update, k, largest=True, sorted=False)
    bot = torch.topk(update, k, largest=False, sorted=False)
    ar = np.arange(k, dtype=np.int64)
    side, mu, _, _ = oracle.side_and_mu(oracle.exact_sum(top.values.cpu().numpy(), ar),
                                        oracle.exact_sum(bot.values.cpu().numpy(), ar), k)
    kept = torch.sort((bot if side else top).indices).values
    del top, bot
    want_stream = oracle.container(kept.cpu().numpy(), n, p, side, mu)
    residual = torch.zeros(n, dtype=torch.float32, device=DEV)
    out, mu_dev = sbc.sbc_encode(update, residual, p)
    info = sbc.sbc_stream_info_get(out)
    assert (info.k, info.side, info.numel) == (k, side, n)
    assert np.float32(mu_dev.item()).view(np.uint32) == mu.view(np.uint32)
    assert np.array_equal(out[: info.total_bytes].cpu().numpy(), want_stream)
    assert int(kept[-1].item()) == n - 1 and int(kept[0].item()) == 0
    # residual: update everywhere, update - mu on the kept positions
    fixed = update[kept] - float(mu)
    assert torch.equal(residual[kept].view(torch.int32), fixed.view(torch.int32))
    residual[kept] = update[kept]
    assert torch.equal(residual.view(torch.int32), update.view(torch.int32))
    del residual
    dense = torch.zeros(n, dtype=torch.float32, device=DEV)
    status = torch.zeros(1, dtype=torch.int32, device=DEV)
    sbc.sbc_decode_accumulate([out], dense, status=status)
    torch.cuda.synchronize()
    assert status.item() == 0
    assert bool((dense[kept] == float(mu)).all())
    dense[kept] = 0.0
    assert not bool(dense.any())


def test_long_stream_is_decoded_in_list_order_and_rejects_damage():
    # 3.3 M positions (13 108 chunks): long enough for the decoder's in-order form, in which a warp
    # parses 32 codewords per chunk into shared memory and then adds chunk after chunk
    n, p = 1 << 25, 0.1
    rng = np.random.default_rng(4242)
    upd = (rng.standard_normal(n) * 1e-3).astype(np.float32)
    u = torch.from_numpy(upd).to(DEV)
    r = torch.zeros(n, dtype=torch.float32, device=DEV)
    out, mu = sbc.sbc_encode(u, r, p)
    info = sbc.sbc_stream_info_get(out)
    assert info.n_chunks >= 8192
    stream = out[: info.total_bytes].cpu().numpy()
    want = np.full(n, 0.25, dtype=np.float32)
    oracle.decode_accumulate([stream], want)         # Algorithm 4 on the CPU, onto existing contents
    guard = 4096

    def run(mutated: np.ndarray):
        dense = torch.zeros(n + 2 * guard, dtype=torch.float32, device=DEV)
        dense[guard:guard + n] = 0.25
        status = torch.zeros(1, dtype=torch.int32, device=DEV)
        sbc.sbc_decode_accumulate([torch.from_numpy(mutated).to(DEV)], dense[guard:guard + n], status=status)
        torch.cuda.synchronize()
        assert not bool(dense[:guard].any()) and not bool(dense[guard + n:].any()), "decoder wrote outside the tensor"
        return status.item(), dense[guard:guard + n]

    status, dense = run(stream)
    assert status == 0
    assert np.array_equal(dense.cpu().numpy().view(np.uint32), want.view(np.uint32))
    table = 64                                          # chunk table: 16 bytes per chunk after the 64-byte header
    bad = stream.copy(); bad[info.payload_offset + 100000] ^= 0x10      # one payload bit in the middle
    assert run(bad)[0] != 0
    bad = stream.copy(); bad[info.payload_offset + 5000: info.payload_offset + 5064] = 0xFF   # a long run of ones
    assert run(bad)[0] != 0
    bad = stream.copy(); bad[table + 16 * 777 + 8: table + 16 * 777 + 16].view("<i8")[0] = n + 5   # previous position beyond the tensor
    assert run(bad)[0] & sbc.STATUS_CORRUPT
    bad = stream.copy(); bad[table + 16 * 4000: table + 16 * 4000 + 8].view("<u8")[0] += 3         # chunk offset off by three bits
    assert run(bad)[0] != 0
    bad = stream.copy(); bad[table + 16 * 9000 + 8: table + 16 * 9000 + 16].view("<i8")[0] = 2**40  # absurd previous position
    assert run(bad)[0] & sbc.STATUS_CORRUPT


def test_the_bounded_wait_of_the_exact_route_gives_up_and_reports_it():
    """The exact route's steps meet at a barrier in global memory.  Its wait is bounded: a barrier
    that cannot be passed (here: one that waits for a block that does not exist) ends by itself
    after a fraction of a second and leaves a status word, and the device is as usable as before."""
    scratch = torch.zeros(2, dtype=torch.int32, device=DEV)
    sbc.sbc_debug_barrier_timeout(scratch)
    torch.cuda.synchronize()
    assert scratch[1].item() == sbc.STATUS_TIMEOUT
    # the context is intact: an ordinary encode still matches the oracle afterwards
    n, p = 100000, 0.01
    upd = workloads.normal_flat(n, 1e-3, 77)
    want_res = np.zeros(n, dtype=np.float32)
    want_stream, _ = oracle.encode(upd, want_res, p)
    r = torch.zeros(n, dtype=torch.float32, device=DEV)
    out, _ = sbc.sbc_encode(torch.from_numpy(upd).to(DEV), r, p)
    info = sbc.sbc_stream_info_get(out)
    assert np.array_equal(out[: info.total_bytes].cpu().numpy(), want_stream)
