"""GPU parity on the five workload configurations (shapes of the paper's networks, synthetic values).

Configs 1-4 run the oracle on the full tensors (one thread per tensor: the C oracle releases the
GIL).  Config 5 (2^30 elements) is too large for the oracle's full sort, so its expected result is
assembled from independent pieces: torch's own sort for the two thresholds, the oracle's exact
sum / decision / container builder for everything after the selection.
"""
from concurrent.futures import ThreadPoolExecutor

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
POOL = ThreadPoolExecutor(max_workers=16)


class Client:
    """Device-side state of one client: residuals, streams, scratch (allocated once, reused per round)."""

    def __init__(self, sizes, p, batched=True):
        self.p, self.batched = p, batched
        self.res = [torch.zeros(n, dtype=torch.float32, device=DEV) for n in sizes]
        self.out = [torch.empty(sbc.sbc_stream_bytes(n, p), dtype=torch.uint8, device=DEV) for n in sizes]
        self.mu = [torch.empty(1, dtype=torch.float32, device=DEV) for _ in sizes]
        if batched:
            ws_bytes = sbc.sbc_workspace_bytes_batch(sizes, [p] * len(sizes))
        else:
            ws_bytes = max(sbc.sbc_workspace_bytes(n, p) for n in sizes)
        self.ws = torch.full((ws_bytes + 256,), 0xCD, dtype=torch.uint8, device=DEV)
        self.ws_bytes = ws_bytes

    def encode_round(self, tensors):
        ups = [torch.from_numpy(u).to(DEV) for u in tensors]
        if self.batched:
            sbc.sbc_encode_batch(ups, self.res, [self.p] * len(ups), self.out, self.mu, self.ws[: self.ws_bytes])
        else:
            for t, u in enumerate(ups):
                sbc.sbc_encode(u, self.res[t], self.p, self.out[t], self.mu[t], self.ws[: self.ws_bytes])
        torch.cuda.synchronize()
        assert bool((self.ws[self.ws_bytes:] == 0xCD).all()), "write past the workspace"
        got = []
        for t in range(len(tensors)):
            info = sbc.sbc_stream_info_get(self.out[t])
            got.append((self.out[t][: info.total_bytes].cpu().numpy(), np.float32(self.mu[t].item())))
        return got


def oracle_round(tensors, residuals, p):
    return list(POOL.map(lambda ur: oracle.encode(ur[0], ur[1], p), zip(tensors, residuals)))


def assert_round_equal(got, want, client, residuals_cpu, label):
    for t, ((gs, gm), (ws_, wm)) in enumerate(zip(got, want)):
        assert np.array_equal(gs, ws_), f"{label}: container of tensor {t} differs"
        assert gm.view(np.uint32) == wm.view(np.uint32), f"{label}: mu of tensor {t} differs"
        assert np.array_equal(client.res[t].cpu().numpy().view(np.uint32), residuals_cpu[t].view(np.uint32)), \
            f"{label}: residual of tensor {t} differs"


def test_config2_resnet50_shapes_ten_rounds():
    shapes = workloads.resnet50_shapes()
    sizes = [int(np.prod(s)) for _, s, _ in shapes]
    assert len(sizes) == 161 and sum(sizes) == 25557032 and sum(1 for n in sizes if n < 1000) == 84
    p = 0.001
    client = Client(sizes, p)
    res_cpu = [np.zeros(n, dtype=np.float32) for n in sizes]
    for rnd in range(10):
        tensors = workloads.resnet50_update(workloads.seed_for(2, rnd))
        want = oracle_round(tensors, res_cpu, p)
        got = client.encode_round(tensors)
        assert_round_equal(got, want, client, res_cpu, f"round {rnd}")


@pytest.mark.parametrize("p", [0.01, 0.001])
def test_config3_word_lstm_shapes_four_rounds(p):
    sizes = [int(np.prod(s)) for _, s in workloads.word_lstm_shapes()]
    assert sum(sizes) == 19765200
    client = Client(sizes, p)
    res_cpu = [np.zeros(n, dtype=np.float32) for n in sizes]
    for rnd in range(4):
        tensors = workloads.word_lstm_update(workloads.seed_for(3, rnd))
        want = oracle_round(tensors, res_cpu, p)
        got = client.encode_round(tensors)
        assert_round_equal(got, want, client, res_cpu, f"p={p} round {rnd}")


def test_config4_eight_clients_decode_aggregate():
    shapes = workloads.resnet50_shapes()
    sizes = [int(np.prod(s)) for _, s, _ in shapes]
    p = 0.001
    per_client = []
    for c in range(8):
        tensors = workloads.resnet50_update(workloads.seed_for(4, 0, c))
        client = Client(sizes, p)
        res_cpu = [np.zeros(n, dtype=np.float32) for n in sizes]
        want = oracle_round(tensors, res_cpu, p)
        got = client.encode_round(tensors)
        assert_round_equal(got, want, client, res_cpu, f"client {c}")
        per_client.append((client, want))
    # one dense aggregate per tensor, the 8 streams decoded and summed on the device
    status = torch.zeros(1, dtype=torch.int32, device=DEV)
    dense = [torch.zeros(n, dtype=torch.float32, device=DEV) for n in sizes]
    dws = torch.empty(sbc.sbc_decode_workspace_bytes_batch(len(sizes)), dtype=torch.uint8, device=DEV)
    sbc.sbc_decode_accumulate_batch([[cl.out[t] for cl, _ in per_client] for t in range(len(sizes))],
                                    dense, dws, status=status)
    torch.cuda.synchronize()
    assert status.item() == 0
    # the one-tensor-per-call form gives the same sums (to the stated tolerance)
    dense1 = [torch.zeros(n, dtype=torch.float32, device=DEV) for n in sizes]
    for t in range(0, len(sizes), 7):
        sbc.sbc_decode_accumulate([cl.out[t] for cl, _ in per_client], dense1[t], status=status)
    torch.cuda.synchronize()
    assert status.item() == 0
    for t in range(0, len(sizes), 7):
        assert torch.allclose(dense[t], dense1[t], rtol=0, atol=1e-6)

    def expected(t):
        want = np.zeros(sizes[t], dtype=np.float32)
        oracle.decode_accumulate([w[t][0] for _, w in per_client], want)
        return want

    for t, want in enumerate(POOL.map(expected, range(len(sizes)))):
        got = dense[t].cpu().numpy()
        tol = 1e-6 * sum(abs(float(w[t][1])) for _, w in per_client)
        assert np.array_equal(got != 0, want != 0) or tol > 0
        assert np.max(np.abs(got.astype(np.float64) - want)) <= tol, f"aggregate of tensor {t}"


def _check_flat_round(accumulated, update, residual, p):
    """One sbc_encode + decode of a flat tensor against an independent selection.  `accumulated` is
    what A = residual + update must be (taken with torch's own fp32 add); torch's sort gives the two
    order statistics, the oracle the exact sums, the side decision and the container.  `residual`
    is updated in place by the encode and checked bit for bit."""
    n = accumulated.numel()
    k, b = oracle.kept_count(n, p), oracle.golomb_b(p)
    sorted_vals = torch.sort(accumulated).values
    t_top = sorted_vals[n - k]          # k-th largest
    t_bot = sorted_vals[k - 1]          # k-th smallest
    del sorted_vals
    top = torch.nonzero(accumulated >= t_top).flatten()
    bot = torch.nonzero(accumulated <= t_bot).flatten()
    # continuous data: no ties expected at the thresholds; if there are, keep the lowest indices
    if top.numel() > k:
        ties = torch.nonzero(accumulated[top] == t_top).flatten()
        keep = torch.ones(top.numel(), dtype=torch.bool, device=DEV)
        keep[ties[k - (top.numel() - ties.numel()):]] = False
        top = top[keep]
    if bot.numel() > k:
        ties = torch.nonzero(accumulated[bot] == t_bot).flatten()
        keep = torch.ones(bot.numel(), dtype=torch.bool, device=DEV)
        keep[ties[k - (bot.numel() - ties.numel()):]] = False
        bot = bot[keep]
    assert top.numel() == k and bot.numel() == k
    top_vals = accumulated[top].cpu().numpy()
    bot_vals = accumulated[bot].cpu().numpy()
    ar = np.arange(k, dtype=np.int64)
    side, mu, _, _ = oracle.side_and_mu(oracle.exact_sum(top_vals, ar), oracle.exact_sum(bot_vals, ar), k)
    kept = (bot if side else top)
    want_stream = oracle.container(kept.cpu().numpy(), n, p, side, mu)
    del top, bot

    out, mu_dev = sbc.sbc_encode(update, residual, p)
    info = sbc.sbc_stream_info_get(out)
    got_stream = out[: info.total_bytes].cpu().numpy()
    assert (info.k, info.b, info.side) == (k, b, side)
    assert np.float32(mu_dev.item()).view(np.uint32) == mu.view(np.uint32)
    assert np.array_equal(got_stream, want_stream), f"p={p}: container differs"
    # residual: A everywhere, A - mu (one fp32 subtraction) on the kept positions
    expect_res = accumulated.clone()
    expect_res[kept] = accumulated[kept] - float(mu)
    assert torch.equal(residual.view(torch.int32), expect_res.view(torch.int32)), f"p={p}: residual differs"
    del expect_res
    # decode into a zeroed tensor: mu on the kept positions, zero elsewhere
    dense = torch.zeros(n, dtype=torch.float32, device=DEV)
    status = torch.zeros(1, dtype=torch.int32, device=DEV)
    sbc.sbc_decode_accumulate([out], dense, status=status)
    expect = torch.zeros(n, dtype=torch.float32, device=DEV)
    expect[kept] = float(mu)
    torch.cuda.synchronize()
    assert status.item() == 0
    assert torch.equal(dense.view(torch.int32), expect.view(torch.int32)), f"p={p}: decoded tensor differs"


def test_config5_flat_2p30_sweep_against_independent_selection():
    """Config 5 at full size, as the benchmark runs it: per p a first round from a zero residual and a
    second round that carries the first round's residual (so that E1's add is not trivial)."""
    n = 1 << 30
    update = workloads.student_t_flat_torch(n, workloads.seed_for(5), DEV)
    update2 = workloads.student_t_flat_torch(n, workloads.seed_for(5, 1), DEV)
    for p in (1e-2, 1e-3, 1e-4):
        residual = torch.zeros(n, dtype=torch.float32, device=DEV)
        _check_flat_round(update, update, residual, p)              # A = 0 + update
        carried = torch.add(residual, update2)                      # what the second communication round must accumulate
        assert bool((residual != update).any())                     # the residual really carries something
        _check_flat_round(carried, update2, residual, p)
        del residual, carried


def test_batch_and_single_tensor_calls_agree_with_mixed_sparsities():
    rng = np.random.default_rng(77)
    sizes = [1, 64, 1000, 4097, 70001, 300000, 2_000_003, 5, 131072]
    ps = [0.5, 0.001, 0.01, 0.1, 0.001, 0.01, 0.001, 0.2, 0.0001]
    ups = [(rng.standard_normal(n) * 1e-3).astype(np.float32) for n in sizes]
    ups[3][:] = 0.0                                  # an all-zero tensor in the middle of the batch (exact route)
    res0 = [(rng.standard_normal(n) * 1e-3).astype(np.float32) for n in sizes]
    res0[3][:] = 0.0
    want_res = [r.copy() for r in res0]
    want = [oracle.encode(u, r, p) for u, r, p in zip(ups, want_res, ps)]
    d_up = [torch.from_numpy(u).to(DEV) for u in ups]
    d_res = [torch.from_numpy(r).to(DEV) for r in res0]
    outs = [torch.empty(sbc.sbc_stream_bytes(n, p), dtype=torch.uint8, device=DEV) for n, p in zip(sizes, ps)]
    mus = [torch.empty(1, dtype=torch.float32, device=DEV) for _ in sizes]
    ws = torch.empty(sbc.sbc_workspace_bytes_batch(sizes, ps), dtype=torch.uint8, device=DEV)
    sbc.sbc_encode_batch(d_up, d_res, ps, outs, mus, ws)
    torch.cuda.synchronize()
    for t, (ws_, wm) in enumerate(want):
        info = sbc.sbc_stream_info_get(outs[t])
        assert np.array_equal(outs[t][: info.total_bytes].cpu().numpy(), ws_), f"tensor {t}"
        assert np.float32(mus[t].item()).view(np.uint32) == wm.view(np.uint32)
        assert np.array_equal(d_res[t].cpu().numpy().view(np.uint32), want_res[t].view(np.uint32))
    # a bad descriptor anywhere in the batch: nothing runs
    with pytest.raises(sbc.SbcError):
        sbc.sbc_encode_batch(d_up, d_res, ps[:-1] + [1.5], outs, mus, ws)


def test_batch_whose_problems_take_all_three_routes():
    # one launch of the general chain in which a problem runs on the sample's bounds, one has its
    # candidates gathered again (clustered), one has its thresholds searched over the whole tensor
    # (the sample never sees its large values), one is all zeros and one is small: the exact
    # route's kernel works on three of them at once and hands each back the right way
    rng = np.random.default_rng(4711)
    n_big = 1 << 21
    plain = (rng.standard_t(3, n_big) * 1e-3).astype(np.float32)
    clustered = (rng.standard_normal(n_big) * 1e-6).astype(np.float32)
    clustered[n_big // 2 + 777: n_big // 2 + 777 + n_big // 50] *= np.float32(1e3)
    hidden = (rng.standard_normal(n_big) * 1e-3).astype(np.float32)
    k = oracle.kept_count(n_big, 0.01)
    off_sample = np.flatnonzero((np.arange(n_big) // 32) % 16 != 0)
    extra = rng.choice(off_sample, k, replace=False)
    hidden[extra[: k // 2]] = (5e-3 + 1e-3 * rng.random(k // 2)).astype(np.float32)
    hidden[extra[k // 2:]] = (-5e-3 - 1e-3 * rng.random(k - k // 2)).astype(np.float32)
    zeros = np.zeros(300_000, dtype=np.float32)
    small = (rng.standard_normal(5000) * 1e-3).astype(np.float32)
    ups = [plain, clustered, hidden, zeros, small]
    ps = [0.01, 0.01, 0.01, 0.01, 0.01]
    sizes = [u.size for u in ups]
    for rnd in range(2):                                  # second round: carried residuals
        if rnd == 0:
            res0 = [np.zeros(n, dtype=np.float32) for n in sizes]
            d_res = [torch.from_numpy(r).to(DEV) for r in res0]
            want_res = [r.copy() for r in res0]
        want = [oracle.encode(u, r, p) for u, r, p in zip(ups, want_res, ps)]
        d_up = [torch.from_numpy(u).to(DEV) for u in ups]
        outs = [torch.empty(sbc.sbc_stream_bytes(n, p), dtype=torch.uint8, device=DEV) for n, p in zip(sizes, ps)]
        mus = [torch.empty(1, dtype=torch.float32, device=DEV) for _ in sizes]
        ws = torch.empty(sbc.sbc_workspace_bytes_batch(sizes, ps), dtype=torch.uint8, device=DEV)
        sbc.sbc_encode_batch(d_up, d_res, ps, outs, mus, ws)
        torch.cuda.synchronize()
        for t, (ws_, wm) in enumerate(want):
            info = sbc.sbc_stream_info_get(outs[t])
            assert np.array_equal(outs[t][: info.total_bytes].cpu().numpy(), ws_), f"round {rnd}, tensor {t}"
            assert np.float32(mus[t].item()).view(np.uint32) == wm.view(np.uint32), f"round {rnd}, tensor {t}"
            assert np.array_equal(d_res[t].cpu().numpy().view(np.uint32), want_res[t].view(np.uint32)), f"round {rnd}, tensor {t}"
    # the same three large tensors one by one: the routes are the ones this test is about
    for u, want_route in ((plain, (0, 0)), (clustered, (1, 1)), (hidden, (1, 0))):
        d_u = torch.from_numpy(u).to(DEV)
        d_r = torch.zeros(u.size, dtype=torch.float32, device=DEV)
        ws1 = torch.empty(sbc.sbc_workspace_bytes(u.size, 0.01), dtype=torch.uint8, device=DEV)
        sbc.sbc_encode(d_u, d_r, 0.01, workspace=ws1)
        diag = sbc.sbc_encode_diag_get(ws1)
        assert (diag.exact_route, diag.regathered) == want_route


@pytest.mark.parametrize("seed", [1, 2, 3])
def test_batch_of_short_list_problems_with_ties_zeros_and_a_bad_tensor(seed):
    # every tensor keeps at most 3584 positions, so the whole batch takes the one-kernel back half;
    # it holds tie-heavy, one-signed and all-zero tensors and one tensor with a NaN, whose header must
    # carry the error while its neighbours are encoded as usual
    rng = np.random.default_rng(900 + seed)
    n_tensors = 48
    sizes, ps, ups, res0 = [], [], [], []
    for t in range(n_tensors):
        p = float(10.0 ** rng.uniform(-3.3, -0.4))
        k_max = 3584
        n = int(rng.integers(1, min(400000, int(k_max / p))))
        kind = t % 6
        if kind == 0:
            u = rng.standard_normal(n)
        elif kind == 1:
            u = np.round(rng.standard_normal(n) * 2) / 2          # few distinct values
        elif kind == 2:
            u = np.zeros(n)                                        # exact route, mu = 0
        elif kind == 3:
            u = -np.abs(rng.standard_t(3, n))                      # one-signed
        elif kind == 4:
            u = rng.standard_normal(n) * (rng.random(n) < 0.02)    # mostly zeros
        else:
            u = rng.laplace(size=n)
        sizes.append(n)
        ps.append(p)
        ups.append((u * 10.0 ** rng.integers(-5, 2)).astype(np.float32))
        res0.append((rng.standard_normal(n) * 1e-4).astype(np.float32) if t % 2 else np.zeros(n, dtype=np.float32))
    bad = 17
    ups[bad][ups[bad].size // 2] = np.nan
    want_res = [r.copy() for r in res0]
    want = [None if t == bad else oracle.encode(ups[t], want_res[t], ps[t]) for t in range(n_tensors)]
    d_up = [torch.from_numpy(u).to(DEV) for u in ups]
    d_res = [torch.from_numpy(r).to(DEV) for r in res0]
    outs = [torch.empty(sbc.sbc_stream_bytes(n, p), dtype=torch.uint8, device=DEV) for n, p in zip(sizes, ps)]
    mus = [torch.empty(1, dtype=torch.float32, device=DEV) for _ in sizes]
    ws = torch.empty(sbc.sbc_workspace_bytes_batch(sizes, ps), dtype=torch.uint8, device=DEV)
    sbc.sbc_encode_batch(d_up, d_res, ps, outs, mus, ws)
    torch.cuda.synchronize()
    for t in range(n_tensors):
        if t == bad:
            info = sbc.sbc_stream_info_get(outs[t], check=False)
            assert info.status & sbc.STATUS_NONFINITE and info.k == 0
            continue
        info = sbc.sbc_stream_info_get(outs[t])
        assert np.array_equal(outs[t][: info.total_bytes].cpu().numpy(), want[t][0]), f"tensor {t} (n={sizes[t]}, p={ps[t]})"
        assert np.float32(mus[t].item()).view(np.uint32) == want[t][1].view(np.uint32), f"tensor {t}"
        assert np.array_equal(d_res[t].cpu().numpy().view(np.uint32), want_res[t].view(np.uint32)), f"tensor {t}"
