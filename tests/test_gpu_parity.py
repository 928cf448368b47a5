"""GPU parity: the CUDA library against the CPU oracle, through the C ABI.

Bar: kept index sets, side, Golomb bit strings and the whole container
byte-exact; mu bit-identical (both sides round the exact sum once); residual
bit-identical (same fp32 operations); decoded aggregate within
1e-6 * sum_c |mu_c| per element (the order of fp32 atomic adds is free).
"""
import zlib

import numpy as np
import pytest
import torch

import oracle
from paper_1805_08768_b200 import binding as sbc
from paper_1805_08768_b200 import workloads

pytestmark = pytest.mark.gpu

if not torch.cuda.is_available():  # pragma: no cover - the CPU box deselects with -m "not gpu"
    pytest.skip("needs a CUDA device", allow_module_level=True)

DEV = torch.device("cuda:0")


def gpu_encode(upd: np.ndarray, res: np.ndarray, p: float, offset_elems: int = 0):
    """Run sbc_encode on device copies; returns (stream bytes, mu, new residual, info)."""
    n = upd.size
    if offset_elems:  # deliberately misaligned views (4-byte aligned only)
        ubuf = torch.zeros(n + offset_elems + 4, dtype=torch.float32, device=DEV)
        rbuf = torch.zeros(n + offset_elems + 4, dtype=torch.float32, device=DEV)
        u = ubuf[offset_elems:offset_elems + n]
        r = rbuf[offset_elems:offset_elems + n]
        u.copy_(torch.from_numpy(upd))
        r.copy_(torch.from_numpy(res))
    else:
        u = torch.from_numpy(upd).to(DEV)
        r = torch.from_numpy(res).to(DEV)
    cap = sbc.sbc_stream_bytes(n, p)
    out = torch.full((cap + 64,), 0xAB, dtype=torch.uint8, device=DEV)   # canary behind the capacity
    ws_bytes = sbc.sbc_workspace_bytes(n, p)
    ws = torch.full((ws_bytes + 256,), 0xCD, dtype=torch.uint8, device=DEV)
    mu = torch.full((1,), float("nan"), dtype=torch.float32, device=DEV)
    sbc.sbc_encode(u, r, p, out_stream=out[:cap], out_mu=mu, workspace=ws[:ws_bytes])
    info = sbc.sbc_stream_info_get(out)
    torch.cuda.synchronize()
    assert bool((out[cap:] == 0xAB).all()), "write past the stream capacity"
    assert bool((ws[ws_bytes:] == 0xCD).all()), "write past the workspace"
    stream = out[: info.total_bytes].cpu().numpy()
    return stream, np.float32(mu.item()), r.cpu().numpy(), info, out


def check_against_oracle(upd, res, p, offset_elems=0):
    want_res = res.copy()
    want_stream, want_mu = oracle.encode(upd, want_res, p)
    stream, mu, got_res, info, _ = gpu_encode(upd, res, p, offset_elems)
    h = oracle.parse_header(want_stream)
    assert (info.k, info.b, info.side, info.nbits) == (h.k, h.b, h.side, h.nbits)
    assert mu.view(np.uint32) == want_mu.view(np.uint32), (mu, want_mu)
    assert stream.size == want_stream.size
    assert np.array_equal(stream, want_stream)
    assert np.array_equal(got_res.view(np.uint32), want_res.view(np.uint32))
    return stream, mu


@pytest.mark.parametrize("name,upd,res,p", workloads.adversarial_cases(),
                         ids=[c[0] for c in workloads.adversarial_cases()])
def test_encode_adversarial_cases(name, upd, res, p):
    check_against_oracle(upd, res, p)


def test_config1_round_trip():
    n, p = 2**20, 0.01
    upd = workloads.normal_flat(n, 1e-3, workloads.seed_for(1))
    res = np.zeros(n, dtype=np.float32)
    stream, mu = check_against_oracle(upd, res, p)
    # decode into a zeroed dense tensor = the binarised update
    want = np.zeros(n, dtype=np.float32)
    oracle.decode_accumulate([stream], want)
    dense = torch.zeros(n, dtype=torch.float32, device=DEV)
    status = torch.zeros(1, dtype=torch.int32, device=DEV)
    sbc.sbc_decode_accumulate([torch.from_numpy(stream).to(DEV)], dense, status=status)
    torch.cuda.synchronize()
    assert status.item() == 0
    assert np.array_equal(dense.cpu().numpy(), want)      # one client: exact
    assert np.count_nonzero(want) == oracle.kept_count(n, p)


@pytest.mark.parametrize("n", [1, 2, 31, 32, 33, 255, 257, 1023, 4095, 4097, 65537, 300001, 1500007])
@pytest.mark.parametrize("p", [0.01, 0.001])
def test_encode_ragged_sizes(n, p):
    rng = np.random.default_rng(n)
    upd = (rng.standard_normal(n) * 1e-3).astype(np.float32)
    res = (rng.standard_normal(n) * 1e-3).astype(np.float32)
    check_against_oracle(upd, res, p)


# Problems whose candidate lists hold at most 8192 entries and that keep at most 4096 positions are
# finished by one kernel (two blocks per problem); the cases sit on both sides of those two limits,
# with smooth and with tie-heavy values.
@pytest.mark.parametrize("n,p", [
    (358400, 0.01),    # k = 3584, capacity 8192: the largest problem of the short-list form
    (358500, 0.01),    # k = 3585, capacity 8194: just beyond it
    (8192, 0.5),       # k = 4096 = the most positions one block orders, capacity = n
    (8192, 0.6),       # k = 4915: short lists, but too many kept positions for one block
    (8193, 0.45),      # capacity 8193 > 8192 with k below 4096
    (4096, 0.999),     # nearly everything kept
    (5000, 0.3), (70001, 0.05), (3_000_000, 0.001), (3_584_000, 0.001), (3_585_000, 0.001),
])
@pytest.mark.parametrize("kind", ["normal", "few_values"])
def test_short_list_form_and_its_limits(n, p, kind):
    rng = np.random.default_rng(zlib.crc32(f"{n}/{p}/{kind}".encode()))
    if kind == "normal":
        upd = rng.standard_normal(n).astype(np.float32) * np.float32(1e-3)
        res = rng.standard_normal(n).astype(np.float32) * np.float32(1e-3)
    else:  # a handful of distinct values: the thresholds fall inside long runs of equal entries
        upd = rng.integers(-3, 4, size=n).astype(np.float32) * np.float32(0.25)
        res = rng.integers(-1, 2, size=n).astype(np.float32) * np.float32(0.5)
    check_against_oracle(upd, res, p)


# The kept positions come out in order because the candidates are gathered span by span (1, 2, 4 or
# 8 steps of 512 elements, by tensor size) into per-warp regions and walked in span order.  Sizes
# on both sides of every span length, sparse and dense spans, and uneven ones (all kept entries in
# the first tenth of the tensor: ten times the expected candidates per span there, none elsewhere).
@pytest.mark.parametrize("n,p,clustered", [
    (1 << 23, 0.0005, False),   # k = 4194: just beyond the one-kernel form for short lists
    (1 << 22, 0.0015, False),
    (1 << 21, 0.003, False),
    (3_000_001, 0.0039, False),
    (1 << 21, 0.006, False),
    (1 << 24, 0.0004, True),
    (1 << 24, 0.00025, True),
    (7_272_960 + 17, 0.004, False),   # 14206 steps: one short of two two-step spans per warp -> one-step spans
    (7_273_472 + 17, 0.004, False),   # 14207 steps: two-step spans
    (14_546_437, 0.002, False),       # 28412 steps: still two-step spans
    (14_546_949, 0.002, False),       # 28413 steps: four-step spans
    (29_093_381, 0.001, False),       # 56824 steps: still four-step spans
    (29_093_893, 0.001, False),       # 56825 steps: eight-step spans
])
def test_span_ordering_forms(n, p, clustered):
    rng = np.random.default_rng(zlib.crc32(f"buckets/{n}/{p}/{clustered}".encode()))
    upd = rng.standard_normal(n).astype(np.float32) * np.float32(1e-3)
    if clustered:
        upd[n // 10:] *= np.float32(1e-3)   # large magnitudes only at the front
    check_against_oracle(upd, np.zeros(n, dtype=np.float32), p)


@pytest.mark.parametrize("n,p", [
    ((1 << 25) + 4321, 0.0040),   # eight-step spans, 16.4 kept entries per span: a thread walks a span, 1184 blocks
    ((1 << 25) + 4321, 0.0038),   # 15.6 per span: the warp walks its range, one resident wave of blocks
    (1 << 22, 0.032),             # one-step spans on either side of the same limit
    (1 << 22, 0.030),
])
def test_both_counting_walks_around_their_limit(n, p):
    rng = np.random.default_rng(zlib.crc32(f"walks/{n}/{p}".encode()))
    upd = (rng.standard_t(3, n) * 1e-3).astype(np.float32)
    res = (rng.standard_normal(n) * 1e-4).astype(np.float32)
    check_against_oracle(upd, res, p)


@pytest.mark.parametrize("offset", [1, 2, 3])
def test_encode_misaligned_pointers(offset):
    rng = np.random.default_rng(offset)
    n = 70001
    upd = (rng.standard_normal(n) * 1e-3).astype(np.float32)
    res = (rng.standard_normal(n) * 1e-3).astype(np.float32)
    check_against_oracle(upd, res, 0.01, offset_elems=offset)


@pytest.mark.parametrize("dist", ["student_t", "laplace", "uniform", "lognormal_signed"])
@pytest.mark.parametrize("p", [0.1, 0.01, 1e-3, 1e-4])
def test_encode_distributions(dist, p):
    rng = np.random.default_rng(zlib.crc32(f"{dist}:{p}".encode()))
    n = 1 << 21                      # above the sample size: the bounds come from a strided sample
    if dist == "student_t":
        upd = (rng.standard_t(3, n) * 1e-3).astype(np.float32)
    elif dist == "laplace":
        upd = rng.laplace(0, 1e-3, n).astype(np.float32)
    elif dist == "uniform":
        upd = rng.uniform(-1, 1, n).astype(np.float32)
    else:
        upd = (np.exp(rng.standard_normal(n) * 3) * rng.choice([-1.0, 1.0], n)).astype(np.float32)
    check_against_oracle(upd, np.zeros(n, dtype=np.float32), p)


def test_unrepresentative_sample_takes_the_exact_route():
    # large values only where the strided sample does not look, plus a block of ties
    n = (1 << 21) + 12345
    rng = np.random.default_rng(42)
    upd = (rng.standard_normal(n) * 1e-3).astype(np.float32)
    upd[5::64] = 7.0           # many equal large values: ties at the positive threshold
    upd[9::128] = -9.0
    check_against_oracle(upd, np.zeros(n, dtype=np.float32), 0.01)
    sparse = np.zeros(n, dtype=np.float32)                     # fewer non-zeros than k
    sparse[rng.choice(n, 1000, replace=False)] = rng.standard_normal(1000).astype(np.float32)
    check_against_oracle(sparse, np.zeros(n, dtype=np.float32), 0.01)


def encode_with_diag(upd, p):
    n = upd.size
    u = torch.from_numpy(upd).to(DEV)
    r = torch.zeros(n, dtype=torch.float32, device=DEV)
    ws = torch.empty(sbc.sbc_workspace_bytes(n, p), dtype=torch.uint8, device=DEV)
    out, mu = sbc.sbc_encode(u, r, p, workspace=ws)
    diag = sbc.sbc_encode_diag_get(ws)
    info = sbc.sbc_stream_info_get(out)
    return out[: info.total_bytes].cpu().numpy(), np.float32(mu.item()), r.cpu().numpy(), diag


def test_selection_looks_only_at_the_band_between_the_two_bounds():
    # long lists: candidates at or above the sample's upper bound are kept unseen by the
    # selection, which then ranks the rest; the result is the oracle's all the same
    n, p = 1 << 23, 0.01
    k = oracle.kept_count(n, p)
    for upd in (workloads.student_t_flat(n, 31), workloads.normal_flat(n, 1e-3, 32)):
        want_res = np.zeros(n, dtype=np.float32)
        want_stream, want_mu = oracle.encode(upd, want_res, p)
        stream, mu, res, diag = encode_with_diag(upd, p)
        assert diag.exact_route == 0
        for s in range(2):
            assert 0.5 * k < diag.certain[s] < k <= diag.candidates[s] <= diag.capacity
        assert np.array_equal(stream, want_stream) and mu.view(np.uint32) == want_mu.view(np.uint32)
        assert np.array_equal(res.view(np.uint32), want_res.view(np.uint32))


@pytest.mark.parametrize("ties", [5000, 40000])
def test_many_equal_values_straddle_the_threshold_inside_the_band(ties):
    # thousands of entries with exactly the value the k-th largest one has, half of them kept (the
    # ones at the lowest positions): the bucket of the first select digit that holds the threshold
    # then holds all of them, far more than one block ranks in its registers, and the selection has
    # to work through the index half of the composites digit by digit
    n, p = 1 << 23, 0.01
    k = oracle.kept_count(n, p)
    rng = np.random.default_rng(ties)
    upd = (rng.standard_normal(n) * 1e-3).astype(np.float32)
    order = np.argsort(upd)
    v_pos, v_neg = upd[order[n - (k - ties // 2)]], upd[order[k - ties // 2 - 1]]
    middle = order[n // 4: 3 * n // 4]                  # entries far from both thresholds
    planted = rng.choice(middle, 2 * ties, replace=False)
    upd[planted[:ties]] = v_pos
    upd[planted[ties:]] = v_neg
    assert np.count_nonzero(upd > v_pos) < k < np.count_nonzero(upd >= v_pos)
    assert np.count_nonzero(upd < v_neg) < k < np.count_nonzero(upd <= v_neg)
    want_res = np.zeros(n, dtype=np.float32)
    want_stream, want_mu = oracle.encode(upd, want_res, p)
    stream, mu, res, diag = encode_with_diag(upd, p)
    assert diag.exact_route == 0                          # the sample's bounds still bracket both thresholds
    assert np.array_equal(stream, want_stream) and mu.view(np.uint32) == want_mu.view(np.uint32)
    assert np.array_equal(res.view(np.uint32), want_res.view(np.uint32))
    # magnitude selection: with the negative side scaled down its k-th largest |value| is v_pos too
    check_values_mode(np.where(upd > 0, upd, upd * np.float32(0.1)).astype(np.float32), np.zeros(n, dtype=np.float32), p)


def test_upper_bound_below_the_threshold_takes_the_exact_route():
    # large entries only where the strided sample does not look: both bounds come out too low and k
    # or more candidates pass the upper one, so it says nothing about what is kept; the thresholds
    # are then searched over the whole tensor
    n, p = 1 << 23, 0.01
    k = oracle.kept_count(n, p)
    rng = np.random.default_rng(7)
    upd = (rng.standard_normal(n) * 1e-3).astype(np.float32)
    hidden = np.flatnonzero((np.arange(n) // 32) % 16 != 0)        # the sample reads one 32-element line in 16
    extra = rng.choice(hidden, k, replace=False)
    upd[extra[: k // 2]] = (5e-3 + 1e-3 * rng.random(k // 2)).astype(np.float32)
    upd[extra[k // 2:]] = (-5e-3 - 1e-3 * rng.random(k - k // 2)).astype(np.float32)
    want_res = np.zeros(n, dtype=np.float32)
    want_stream, want_mu = oracle.encode(upd, want_res, p)
    stream, mu, res, diag = encode_with_diag(upd, p)
    assert diag.exact_route == 1 and diag.regathered == 0
    assert np.array_equal(stream, want_stream) and mu.view(np.uint32) == want_mu.view(np.uint32)
    assert np.array_equal(res.view(np.uint32), want_res.view(np.uint32))


@pytest.mark.parametrize("n,p,where", [
    (1 << 23, 0.01, "front"),      # every kept entry inside the first 2 % of the tensor
    (1 << 23, 0.01, "stripe"),     # inside one stripe in the middle, not aligned to anything
    (1 << 22, 0.01, "front"),
    (3_000_001, 0.02, "tail"),     # at the ragged end
])
def test_clustered_candidates_are_gathered_again_with_the_bounds_kept(n, p, where):
    """The streaming pass gives each warp a fixed region for its candidates.  When nearly all
    candidates sit in a few neighbouring spans, a region overflows; the sample's bounds are still
    right, so only the gathering is redone (space reserved tile by tile), not the threshold search."""
    rng = np.random.default_rng(zlib.crc32(f"cluster/{n}/{p}/{where}".encode()))
    upd = (rng.standard_normal(n) * 1e-6).astype(np.float32)
    # the strided sample must still see the large values' distribution: scale a contiguous part
    width = n // 50
    start = {"front": 0, "stripe": n // 2 + 12345, "tail": n - width}[where]
    upd[start:start + width] *= np.float32(1e3)
    want_res = np.zeros(n, dtype=np.float32)
    want_stream, want_mu = oracle.encode(upd, want_res, p)
    stream, mu, res, diag = encode_with_diag(upd, p)
    assert diag.exact_route == 1 and diag.regathered == 1
    assert np.array_equal(stream, want_stream) and mu.view(np.uint32) == want_mu.view(np.uint32)
    assert np.array_equal(res.view(np.uint32), want_res.view(np.uint32))


@pytest.mark.parametrize("n,p", [(1 << 22, 0.3), (1 << 21, 0.6), (1 << 20, 0.9), (700_001, 0.45)])
def test_dense_selections(n, p):
    # more candidates in one step of a warp than its stage holds: the stage is flushed between quarters of the step
    rng = np.random.default_rng(zlib.crc32(f"dense/{n}/{p}".encode()))
    upd = (rng.standard_normal(n) * 1e-3).astype(np.float32)
    res = (rng.standard_normal(n) * 1e-3).astype(np.float32)
    check_against_oracle(upd, res, p)


def test_multi_round_residual_carry():
    n, p = 250000, 0.001
    res_gpu = np.zeros(n, dtype=np.float32)
    res_cpu = np.zeros(n, dtype=np.float32)
    for rnd in range(4):
        upd = workloads.normal_flat(n, 1e-3, workloads.seed_for(2, rnd))
        want_stream, want_mu = oracle.encode(upd, res_cpu, p)
        stream, mu, res_gpu, _, _ = gpu_encode(upd, res_gpu, p)
        assert np.array_equal(stream, want_stream) and mu == want_mu
        assert np.array_equal(res_gpu.view(np.uint32), res_cpu.view(np.uint32))


def test_encode_is_deterministic():
    n, p = 1 << 20, 0.01
    upd = workloads.student_t_flat(n, 77)
    a = gpu_encode(upd, np.zeros(n, dtype=np.float32), p)
    b = gpu_encode(upd, np.zeros(n, dtype=np.float32), p)
    assert np.array_equal(a[0], b[0]) and a[1] == b[1] and np.array_equal(a[2], b[2])


def test_decode_aggregate_eight_clients():
    n, p = 400000, 0.001
    streams_np, dev_streams, mus = [], [], []
    for c in range(8):
        upd = workloads.normal_flat(n, 1e-3, workloads.seed_for(4, 0, c))
        stream, mu, _, _, _ = gpu_encode(upd, np.zeros(n, dtype=np.float32), p)
        streams_np.append(stream)
        dev_streams.append(torch.from_numpy(stream).to(DEV))
        mus.append(abs(float(mu)))
    want = np.zeros(n, dtype=np.float32)
    oracle.decode_accumulate(streams_np, want)
    dense = torch.zeros(n, dtype=torch.float32, device=DEV)
    status = torch.zeros(1, dtype=torch.int32, device=DEV)
    sbc.sbc_decode_accumulate(dev_streams, dense, status=status)
    torch.cuda.synchronize()
    assert status.item() == 0
    got = dense.cpu().numpy()
    assert np.array_equal(got != 0, want != 0)
    assert np.max(np.abs(got.astype(np.float64) - want)) <= 1e-6 * sum(mus)
    # adds onto existing contents, and more than one launch worth of clients
    dense.fill_(1.0)
    sbc.sbc_decode_accumulate(dev_streams * 5, dense)
    torch.cuda.synchronize()
    want5 = np.ones(n, dtype=np.float64) + 5.0 * want.astype(np.float64)
    assert np.max(np.abs(dense.cpu().numpy() - want5)) <= 1e-6 * (1 + 5 * sum(mus))


def test_non_finite_input_is_reported_not_encoded():
    n = 100000
    upd = workloads.normal_flat(n, 1e-3, 5)
    upd[777] = np.inf
    u = torch.from_numpy(upd).to(DEV)
    r = torch.zeros(n, dtype=torch.float32, device=DEV)
    out, _ = sbc.sbc_encode(u, r, 0.01)
    info = sbc.sbc_stream_info_get(out, check=False)
    assert info.status & sbc.STATUS_NONFINITE
    with pytest.raises(sbc.SbcError):
        sbc.sbc_stream_info_get(out)
    assert np.array_equal(r.cpu().numpy().view(np.uint32), upd.view(np.uint32))  # residual holds A
    # the decoder refuses a stream whose header carries an error
    dense = torch.zeros(n, dtype=torch.float32, device=DEV)
    status = torch.zeros(1, dtype=torch.int32, device=DEV)
    sbc.sbc_decode_accumulate([out], dense, status=status)
    torch.cuda.synchronize()
    assert status.item() & sbc.STATUS_CORRUPT and not bool(dense.any())


def test_corrupt_streams_set_status_and_stay_in_bounds():
    n, p = 200000, 0.01
    upd = workloads.normal_flat(n, 1e-3, 6)
    stream, _, _, info, _ = gpu_encode(upd, np.zeros(n, dtype=np.float32), p)
    guard = 4096

    def run(mutated: np.ndarray):
        dense = torch.zeros(n + guard, dtype=torch.float32, device=DEV)
        status = torch.zeros(1, dtype=torch.int32, device=DEV)
        sbc.sbc_decode_accumulate([torch.from_numpy(mutated).to(DEV)], dense[:n], status=status)
        torch.cuda.synchronize()
        assert not bool(dense[n:].any()), "decoder wrote outside the tensor"
        return status.item()

    assert run(stream) == 0
    bad = stream.copy(); bad[0] ^= 1                 # magic
    assert run(bad) & sbc.STATUS_CORRUPT
    bad = stream.copy(); bad[8:16].view("<u8")[0] = n + 1   # numel mismatch
    assert run(bad) & sbc.STATUS_CORRUPT
    bad = stream.copy(); bad[info.payload_offset:] = 0xFF    # endless unary runs
    assert run(bad) != 0
    bad = stream.copy(); bad[info.payload_offset:info.payload_offset + 64] = 0xFF
    assert run(bad) != 0                                      # positions run past numel
    bad = stream.copy(); bad[64:72].view("<u8")[0] = 2**40    # chunk table offset outside the payload
    assert run(bad) & sbc.STATUS_CORRUPT


def test_inflated_size_fields_are_refused_when_the_length_is_stated():
    """A header whose k, n_chunks, payload_offset and nbits are inflated *consistently* passes every
    check the header allows on its own; told the received length, the decoder must refuse it before
    it reads a table entry or a payload word.  The message sits inside a larger zero-filled buffer
    the test owns, so that even an unchecked read would stay inside the test's memory."""
    n, p = 200000, 0.01
    upd = workloads.normal_flat(n, 1e-3, 6)
    stream, _, _, info, _ = gpu_encode(upd, np.zeros(n, dtype=np.float32), p)
    true_len = stream.size
    b = int(info.b)

    def header(k, nbits=None, n_chunks=None, payload_offset=None):
        bad = stream.copy()
        chunk = oracle.chunk_codewords(k)                  # the chunk size that goes with k positions
        bad[52:56].view("<u4")[0] = chunk
        n_chunks = -(-k // chunk) if n_chunks is None else n_chunks
        payload_offset = 64 + 16 * n_chunks if payload_offset is None else payload_offset
        nbits = k * (1 + b) + ((n - k) >> b) if nbits is None else nbits
        bad[16:24].view("<u8")[0] = k
        bad[24:32].view("<u8")[0] = nbits
        bad[32:40].view("<u8")[0] = payload_offset
        bad[56:60].view("<u4")[0] = n_chunks
        return bad

    def run(mutated, sizes):
        arena = torch.zeros(8 << 20, dtype=torch.uint8, device=DEV)      # 8 MiB >= any container for this n
        arena[: mutated.size] = torch.from_numpy(mutated).to(DEV)
        dense = torch.zeros(n, dtype=torch.float32, device=DEV)
        status = torch.zeros(1, dtype=torch.int32, device=DEV)
        sbc.sbc_decode_accumulate([arena], dense, status=status, sizes=sizes)
        torch.cuda.synchronize()
        return status.item(), bool(dense.any())

    assert run(stream, [true_len]) == (0, True)                      # the genuine message, exact length
    assert run(stream, [true_len + 4096])[0] == 0                    # a slot larger than the message
    st, touched = run(stream, [true_len - 16])                       # cut short
    assert st & sbc.STATUS_CORRUPT and not touched
    for bad in (header(10 * int(info.k)),                            # everything inflated together
                header(n),                                           # the largest k the tensor allows
                header(int(info.k)),                                 # only the payload length (the most the header's own checks allow)
                header(int(info.k) + 4096)):                         # a few more chunks
        assert 64 + 16 * int(bad[56:60].view("<u4")[0]) + (int(bad[24:32].view("<u8")[0]) + 7) // 8 <= 8 << 20
        st, touched = run(bad, [true_len])
        assert st & sbc.STATUS_CORRUPT and not touched, "an over-long header was decoded"
    with pytest.raises(sbc.SbcError) as e:                           # a length that cannot hold a header
        run(stream, [32])
    assert e.value.code == sbc.SBC_EINVAL
    # the batched form carries the lengths in its descriptors
    arena = torch.zeros(8 << 20, dtype=torch.uint8, device=DEV)
    bad = header(10 * int(info.k))
    arena[: bad.size] = torch.from_numpy(bad).to(DEV)
    dense = torch.zeros(n, dtype=torch.float32, device=DEV)
    status = torch.zeros(1, dtype=torch.int32, device=DEV)
    dws = torch.empty(sbc.sbc_decode_workspace_bytes_batch(1), dtype=torch.uint8, device=DEV)
    sbc.sbc_decode_accumulate_batch([[arena]], [dense], dws, status=status, sizes_per_tensor=[[true_len]])
    torch.cuda.synchronize()
    assert status.item() & sbc.STATUS_CORRUPT and not bool(dense.any())


def test_argument_errors_are_returned_at_once():
    n = 1000
    u = torch.zeros(n, dtype=torch.float32, device=DEV)
    r = torch.zeros(n, dtype=torch.float32, device=DEV)
    with pytest.raises(sbc.SbcError) as e:
        sbc.sbc_encode(u, r, 1.5, out_stream=torch.empty(4096, dtype=torch.uint8, device=DEV),
                       workspace=torch.empty(1 << 20, dtype=torch.uint8, device=DEV))
    assert e.value.code == sbc.SBC_EINVAL
    with pytest.raises(sbc.SbcError) as e:
        sbc.sbc_encode(u, r, 0.01, out_stream=torch.empty(16, dtype=torch.uint8, device=DEV))
    assert e.value.code == sbc.SBC_ECAPACITY
    with pytest.raises(sbc.SbcError) as e:
        sbc.sbc_encode(u, u, 0.01)                      # aliasing
    assert e.value.code == sbc.SBC_EINVAL


@pytest.mark.parametrize("exponent", [-90, -96, -98, -99, -100, -102, -120])
def test_residual_write_back_around_the_atomic_adder_s_subnormal_limit(exponent):
    # kept entries that are subnormal or zero next to a transmitted value near 2^-100: the
    # hardware adder flushes subnormals, so the write-back switches to load/subtract/store below
    # that magnitude; either way R_j = fl32(A_j - mu) exactly
    n, p = 200000, 0.01
    k = oracle.kept_count(n, p)
    rng = np.random.default_rng(300 - exponent)
    upd = (rng.integers(-(1 << 22), 1 << 22, n).astype(np.float64) * 2.0 ** -149).astype(np.float32)  # subnormals
    upd[rng.random(n) < 0.2] = 0.0
    big = rng.choice(n, k // 2, replace=False)                       # fewer than k large entries per side
    upd[big[: k // 4]] = ((1.0 + rng.random(k // 4)) * 2.0 ** exponent).astype(np.float32)
    upd[big[k // 4:]] = (-(1.0 + rng.random(k // 2 - k // 4)) * 2.0 ** exponent).astype(np.float32)
    res = (rng.integers(-(1 << 20), 1 << 20, n).astype(np.float64) * 2.0 ** -149).astype(np.float32)
    check_against_oracle(upd, res, p)


def test_decode_of_a_subnormal_mu_is_exact():
    # the transmitted value itself is subnormal: the sum must not be flushed to zero
    n = 5000
    rng = np.random.default_rng(3)
    upd = (rng.standard_normal(n) * 1e-41).astype(np.float32)
    stream, mu, _, _, _ = gpu_encode(upd, np.zeros(n, dtype=np.float32), 0.02)
    assert mu != 0 and abs(float(mu)) < 1.2e-38
    want = np.zeros(n, dtype=np.float32)
    oracle.decode_accumulate([stream, stream, stream], want)
    dense = torch.zeros(n, dtype=torch.float32, device=DEV)
    s = torch.from_numpy(stream).to(DEV)
    sbc.sbc_decode_accumulate([s, s, s], dense)
    torch.cuda.synchronize()
    assert np.array_equal(dense.cpu().numpy().view(np.uint32), want.view(np.uint32))


def test_decode_apply_scales_adds_and_masks_momentum():
    n, p, n_clients = 300000, 0.01, 4
    rng = np.random.default_rng(12)
    streams_np, dev_streams, mus = [], [], []
    for c in range(n_clients):
        upd = workloads.normal_flat(n, 1e-3, 500 + c)
        stream, mu, _, _, _ = gpu_encode(upd, np.zeros(n, dtype=np.float32), p)
        streams_np.append(stream)
        dev_streams.append(torch.from_numpy(stream).to(DEV))
        mus.append(abs(float(mu)))
    w0 = (rng.standard_normal(n) * 0.05).astype(np.float32)
    m0 = rng.standard_normal(n).astype(np.float32)
    want_w, want_m = w0.copy(), m0.copy()
    scale = 1.0 / n_clients
    oracle.decode_apply(streams_np, scale, want_w, want_m)
    w = torch.from_numpy(w0).to(DEV)
    m = torch.from_numpy(m0).to(DEV)
    status = torch.zeros(1, dtype=torch.int32, device=DEV)
    sbc.sbc_decode_apply(dev_streams, scale, w, m, status=status)
    torch.cuda.synchronize()
    assert status.item() == 0
    got_w, got_m = w.cpu().numpy(), m.cpu().numpy()
    tol = 1e-6 * (np.abs(w0).astype(np.float64) + scale * sum(mus))
    assert np.all(np.abs(got_w.astype(np.float64) - want_w) <= tol)
    untouched = want_m == m0
    assert np.array_equal(got_w[untouched & (want_w == w0)], w0[untouched & (want_w == w0)])
    assert np.array_equal(got_m.view(np.uint32), want_m.view(np.uint32))     # momentum mask is exact
    # one client, scale 1: identical to the oracle bit for bit
    w1 = torch.from_numpy(w0).to(DEV)
    sbc.sbc_decode_apply(dev_streams[:1], 1.0, w1)
    torch.cuda.synchronize()
    want1 = w0.copy()
    oracle.decode_apply(streams_np[:1], 1.0, want1)
    assert np.array_equal(w1.cpu().numpy().view(np.uint32), want1.view(np.uint32))


# ---------------------------------------------------------------- Gradient Dropping baseline

def check_values_mode(upd, res, p):
    n = upd.size
    want_res = res.copy()
    want = oracle.encode_values(upd, want_res, p)
    u = torch.from_numpy(upd).to(DEV)
    r = torch.from_numpy(res).to(DEV)
    cap = sbc.sbc_stream_bytes_values(n, p)
    assert cap == oracle.stream_bytes_values(n, p)
    out = torch.full((cap + 64,), 0xAB, dtype=torch.uint8, device=DEV)
    sbc.sbc_encode_values(u, r, p, out_stream=out[:cap])
    info = sbc.sbc_stream_info_get(out)
    torch.cuda.synchronize()
    assert bool((out[cap:] == 0xAB).all())
    assert info.side == sbc.SIDE_VALUES and info.mu == 0.0
    got = out[: info.total_bytes].cpu().numpy()
    assert got.size == want.size and np.array_equal(got, want)
    assert np.array_equal(r.cpu().numpy().view(np.uint32), want_res.view(np.uint32))
    return out, want


@pytest.mark.parametrize("name,upd,res,p", workloads.adversarial_cases(),
                         ids=[c[0] for c in workloads.adversarial_cases()])
def test_values_mode_adversarial_cases(name, upd, res, p):
    check_values_mode(upd, res, p)


@pytest.mark.parametrize("n,p", [(1 << 21, 0.01), (3_000_001, 0.001), (1 << 22, 1e-4), (70001, 0.1)])
def test_values_mode_large_and_decode(n, p):
    rng = np.random.default_rng(n)
    upd = (rng.standard_t(3, n) * 1e-3).astype(np.float32)
    res = (rng.standard_normal(n) * 1e-3).astype(np.float32)
    out, want = check_values_mode(upd, res, p)
    # decode: dW* = A on the kept set; a values stream and a binary stream can be summed together
    upd2 = workloads.normal_flat(n, 1e-3, 5)
    s2, _, _, _, out2 = gpu_encode(upd2, np.zeros(n, dtype=np.float32), p)
    want_dense = np.zeros(n, dtype=np.float32)
    oracle.decode_accumulate([want, s2], want_dense)
    dense = torch.zeros(n, dtype=torch.float32, device=DEV)
    status = torch.zeros(1, dtype=torch.int32, device=DEV)
    sbc.sbc_decode_accumulate([out, out2], dense, status=status)
    torch.cuda.synchronize()
    assert status.item() == 0
    got = dense.cpu().numpy()
    assert np.max(np.abs(got.astype(np.float64) - want_dense)) <= 1e-6 * float(np.abs(want_dense).max())
    one = torch.zeros(n, dtype=torch.float32, device=DEV)
    sbc.sbc_decode_accumulate([out], one)
    want_one = np.zeros(n, dtype=np.float32)
    oracle.decode_accumulate([want], want_one)
    torch.cuda.synchronize()
    assert np.array_equal(one.cpu().numpy().view(np.uint32), want_one.view(np.uint32))


def test_values_mode_three_rounds_with_carried_residual():
    n, p = 500000, 0.001
    res_cpu = np.zeros(n, dtype=np.float32)
    r = torch.zeros(n, dtype=torch.float32, device=DEV)
    for rnd in range(3):
        upd = workloads.normal_flat(n, 1e-3, 900 + rnd)
        want = oracle.encode_values(upd, res_cpu, p)
        out = sbc.sbc_encode_values(torch.from_numpy(upd).to(DEV), r, p)
        info = sbc.sbc_stream_info_get(out)
        assert np.array_equal(out[: info.total_bytes].cpu().numpy(), want)
        assert np.array_equal(r.cpu().numpy().view(np.uint32), res_cpu.view(np.uint32))


# ---------------------------------------------------------------- subsampled thresholds

def check_sampled(upd, res, p, idx):
    n = upd.size
    want_res = res.copy()
    want_stream, want_mu = oracle.encode_sampled(upd, want_res, p, idx)
    u = torch.from_numpy(upd).to(DEV)
    r = torch.from_numpy(res).to(DEV)
    sidx = torch.from_numpy(idx.astype(np.int32)).to(DEV)
    cap = sbc.sbc_stream_bytes_sampled(n, p)
    out = torch.full((cap + 64,), 0xAB, dtype=torch.uint8, device=DEV)
    ws_bytes = sbc.sbc_workspace_bytes_sampled(n, p, idx.size)
    ws = torch.full((ws_bytes + 256,), 0xCD, dtype=torch.uint8, device=DEV)
    mu = torch.zeros(1, dtype=torch.float32, device=DEV)
    sbc.sbc_encode_sampled(u, r, p, sidx, out_stream=out[:cap], out_mu=mu, workspace=ws[:ws_bytes])
    info = sbc.sbc_stream_info_get(out)
    torch.cuda.synchronize()
    assert bool((out[cap:] == 0xAB).all()) and bool((ws[ws_bytes:] == 0xCD).all())
    got = out[: info.total_bytes].cpu().numpy()
    assert info.k == oracle.parse_header(want_stream).k
    assert got.size == want_stream.size and np.array_equal(got, want_stream)
    assert np.float32(mu.item()).view(np.uint32) == want_mu.view(np.uint32)
    assert np.array_equal(r.cpu().numpy().view(np.uint32), want_res.view(np.uint32))
    return out, info


@pytest.mark.parametrize("n,p,m", [(1 << 21, 0.01, 20000), (3_000_001, 0.001, 100000), (1 << 22, 1e-4, 1 << 20),
                                   (70001, 0.05, 1000), (5000, 0.01, 64)])
def test_sampled_thresholds(n, p, m):
    rng = np.random.default_rng(n + m)
    upd = (rng.standard_t(3, n) * 1e-3).astype(np.float32)
    res = (rng.standard_normal(n) * 1e-3).astype(np.float32)
    idx = rng.integers(0, n, m).astype(np.uint32)
    out, info = check_sampled(upd, res, p, idx)
    k = oracle.kept_count(n, p)
    assert info.k != k or m == n                       # the amount of sparsity is noisy, as the paper says
    dense = torch.zeros(n, dtype=torch.float32, device=DEV)
    status = torch.zeros(1, dtype=torch.int32, device=DEV)
    sbc.sbc_decode_accumulate([out], dense, status=status)
    torch.cuda.synchronize()
    assert status.item() == 0 and int((dense != 0).sum().item()) == info.k


def test_sampled_thresholds_rejected_estimate_gives_the_exact_result():
    n, p = 300000, 0.01
    rng = np.random.default_rng(8)
    upd = np.zeros(n, dtype=np.float32)
    upd[rng.choice(n, 2000, replace=False)] = rng.standard_normal(2000).astype(np.float32)
    res = np.zeros(n, dtype=np.float32)
    idx = np.arange(1000, 3000, dtype=np.uint32)        # sees (almost) only zeros: threshold 0 keeps everything
    out, info = check_sampled(upd, res, p, idx)
    want_exact, _ = oracle.encode(upd, np.zeros(n, dtype=np.float32), p)
    assert np.array_equal(out[: info.total_bytes].cpu().numpy(), want_exact)


def test_sampled_thresholds_with_clustered_candidates_keep_the_oracle_s_rule():
    """The estimate is accepted when both sets hold between 1 and min(n, 2k + 1024) entries -- also
    when nearly all of them sit in one stripe of the tensor, which overflows the streaming pass's
    per-warp regions: the gathering is then redone with the same thresholds, not the selection."""
    n, p, m = 1 << 22, 0.01, 200000
    rng = np.random.default_rng(21)
    upd = (rng.standard_normal(n) * 1e-6).astype(np.float32)
    upd[n // 3: n // 3 + n // 50] *= np.float32(1e3)            # every large entry inside 2 % of the tensor
    idx = rng.integers(0, n, m).astype(np.uint32)
    out, info = check_sampled(upd, np.zeros(n, dtype=np.float32), p, idx)
    k = oracle.kept_count(n, p)
    assert info.k != k and 0.5 * k < info.k < 2 * k                # the sampled rule's count, not the exact one


def test_values_mode_with_clustered_candidates():
    n, p = 1 << 22, 0.01
    rng = np.random.default_rng(22)
    upd = (rng.standard_normal(n) * 1e-6).astype(np.float32)
    upd[n - n // 40:] *= np.float32(1e3)
    check_values_mode(upd, np.zeros(n, dtype=np.float32), p)


def test_checkpoint_and_resume_reproduces_the_streams():
    # the residual is the only state: six rounds straight == three rounds, save/restore, three more
    n, p = 200000, 0.01
    updates = [workloads.normal_flat(n, 1e-3, 300 + r) for r in range(6)]

    def run(rounds, residual):
        streams = []
        for upd in rounds:
            stream, mu, residual, _, _ = gpu_encode(upd, residual, p)
            streams.append((stream, mu))
        return streams, residual

    straight, _ = run(updates, np.zeros(n, dtype=np.float32))
    first, saved = run(updates[:3], np.zeros(n, dtype=np.float32))
    second, _ = run(updates[3:], saved.copy())            # "restore" = hand the saved tensor back
    for (s0, m0), (s1, m1) in zip(straight, first + second):
        assert np.array_equal(s0, s1) and m0 == m1
