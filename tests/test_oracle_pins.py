"""Pins for the CPU oracle: what the paper and plain mathematics fix.

Each test checks the oracle against something other than itself: values the
paper prints, closed forms, brute force, Python's exact arithmetic, hand-worked
codes (tests/golden/), invariants of Eq. (residual) and Theorem 2.1.
"""
import math
import os
from fractions import Fraction

import numpy as np
import pytest

import oracle
from paper_1805_08768_b200 import workloads

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")
PHI = (math.sqrt(5.0) + 1.0) / 2.0


def _golden_codes():
    rows = []
    with open(os.path.join(GOLDEN, "golomb_codes.txt")) as fh:
        for line in fh:
            line = line.strip()
            if not line or line.startswith("#"):
                continue
            b, pos, bits, nbits, hx = [f.strip() for f in line.split("|")]
            rows.append((int(b), [int(x) for x in pos.split()], bits.replace(" ", ""),
                         int(nbits), bytes.fromhex(hx.replace(" ", ""))))
    return rows


def _paper_values():
    vals = {}
    with open(os.path.join(GOLDEN, "paper_values.txt")) as fh:
        for line in fh:
            if line.startswith("#") or not line.strip():
                continue
            name, value, _ = [f.strip() for f in line.split("|", 2)]
            vals[name] = value
    return vals


# ---------------------------------------------------------------- scalars

def test_bstar_values_from_the_formula():
    pv = _paper_values()
    for p in (0.1, 0.01, 0.001, 0.0001):
        assert oracle.golomb_b(p) == int(pv[f"bstar_p{p:g}"])


@pytest.mark.parametrize("p", [0.3, 0.2, 0.1, 0.05, 0.02, 0.01, 0.003, 1e-3, 3e-4, 1e-4, 1e-5])
def test_bstar_is_argmin_of_mean_bits_and_threshold_form(p):
    b = oracle.golomb_b(p)
    # Eq. for b_pos, retyped here in exact-ish Python floats
    def bpos(bb):
        return bb + 1.0 / (1.0 - (1.0 - p) ** (2 ** bb))
    best = min(range(0, 31), key=bpos)
    assert b == best
    # algebraic restatement: smallest b with (1-p)^(2^b) < phi-1
    smallest = next(bb for bb in range(0, 40) if (1.0 - p) ** (2 ** bb) < PHI - 1.0)
    assert b == smallest
    assert oracle.mean_position_bits(p, b) == pytest.approx(bpos(b), rel=1e-12)


def test_bstar_clamps_at_zero_for_large_p():
    assert oracle.golomb_b(0.5) == 0
    assert oracle.golomb_b(0.9) == 0
    assert oracle.golomb_b(0.38) >= 0


def test_printed_mean_position_bits():
    pv = _paper_values()
    # the printed 8.38 is the closed form at b = 7 (b* formula gives 6 -> 8.108)
    assert round(oracle.mean_position_bits(0.01, 7), 2) == float(pv["bpos_p0.01_printed"])
    assert round(16.0 / oracle.mean_position_bits(0.01, 7), 1) == float(pv["gain_vs_16bit_p0.01"])
    assert oracle.mean_position_bits(0.01, 6) == pytest.approx(8.108, abs=5e-4)
    assert oracle.mean_position_bits(0.001, 9) == pytest.approx(11.495, abs=5e-4)
    assert oracle.mean_position_bits(0.0001, 13) == pytest.approx(14.788, abs=5e-4)


def test_kept_count():
    assert oracle.kept_count(2**20, 0.01) == 10485
    assert oracle.kept_count(1000, 0.001) == 1
    assert oracle.kept_count(64, 0.001) == 1          # never fewer than one
    assert oracle.kept_count(2**30, 1e-4) == 107374
    assert oracle.kept_count(10, 0.2) == 2
    assert oracle.kept_count(5, 0.999) == 4
    assert oracle.kept_count(1, 0.5) == 1


# ---------------------------------------------------------------- top-k

def _brute_topk(a, k, negate):
    v = -a if negate else a
    # numpy stable argsort of the negated values = descending, lower index first
    order = np.argsort(-v.astype(np.float64), kind="stable")
    return order[:k]


@pytest.mark.parametrize("seed", range(6))
def test_topk_matches_stable_sort_on_tiny_tensors(seed):
    rng = np.random.default_rng(seed)
    for n in (1, 2, 3, 7, 33, 64):
        a = np.round(rng.standard_normal(n) * 2).astype(np.float32) / 2  # many ties
        a[rng.random(n) < 0.2] = 0.0
        a[rng.random(n) < 0.1] = -0.0
        for k in {1, max(1, n // 3), n}:
            for neg in (False, True):
                got = oracle.topk(a, k, neg)
                assert np.array_equal(got, _brute_topk(a, k, neg)), (n, k, neg)


def test_topk_medium_and_special_cases():
    rng = np.random.default_rng(11)
    a = rng.standard_normal(50000).astype(np.float32)
    for neg in (False, True):
        assert np.array_equal(oracle.topk(a, 500, neg), _brute_topk(a, 500, neg))
    # k = 1 is an arg-max / arg-min
    assert oracle.topk(a, 1, False)[0] == int(np.argmax(a))
    assert oracle.topk(a, 1, True)[0] == int(np.argmin(a))
    # all equal: the first k indices, in order
    e = np.full(100, 0.5, dtype=np.float32)
    assert np.array_equal(oracle.topk(e, 7, False), np.arange(7))
    assert np.array_equal(oracle.topk(e, 7, True), np.arange(7))
    # -0 and +0 compare equal, so index order decides
    z = np.array([-0.0, 0.0, -0.0, 0.0], dtype=np.float32)
    assert np.array_equal(oracle.topk(z, 3, False), [0, 1, 2])
    assert np.array_equal(oracle.topk(z, 3, True), [0, 1, 2])


# ---------------------------------------------------------------- exact sum

def _exact_sum_python(vals):
    return float(sum(Fraction(float(v)) for v in vals))  # Fraction -> float rounds correctly


def test_exact_sum_against_python_exact_arithmetic():
    rng = np.random.default_rng(3)
    cases = [
        np.array([1e30, 1.0, -1e30], dtype=np.float32),
        np.array([3e38, 3e38, -3e38, 1e-45], dtype=np.float32),
        np.array([1e-45] * 7 + [-3e-45], dtype=np.float32),
        np.array([16777216.0, 1.0, 1.0, 1.0, -16777216.0], dtype=np.float32),
        (rng.standard_normal(4000) * 10.0 ** rng.integers(-30, 30, 4000)).astype(np.float32),
        (rng.standard_normal(100000) * 1e-3).astype(np.float32),
        np.zeros(5, dtype=np.float32),
    ]
    # a sum that needs the round-to-even rule at 53 bits: 2^60 + 2^7 + ... halfway cases
    cases.append(np.array([2.0**60, 2.0**7, 2.0**6], dtype=np.float32))
    cases.append(np.array([2.0**60, 2.0**7], dtype=np.float32))       # exactly halfway -> even
    cases.append(np.array([2.0**60, 2.0**8, 2.0**7], dtype=np.float32))  # halfway, odd -> up
    for a in cases:
        idx = np.arange(a.size, dtype=np.int64)
        got = oracle.exact_sum(a, idx)
        assert got == _exact_sum_python(a)
        assert got == math.fsum(float(v) for v in a)
    # subset / order independence
    a = cases[4]
    perm = rng.permutation(a.size)[:1234]
    assert oracle.exact_sum(a, perm) == oracle.exact_sum(a, np.sort(perm))
    assert oracle.exact_sum(a, perm) == math.fsum(float(v) for v in a[perm])


# ---------------------------------------------------------------- Golomb code

@pytest.mark.parametrize("row", _golden_codes(), ids=lambda r: f"b{r[0]}_{'-'.join(map(str, r[1]))}")
def test_golomb_hand_computed_codes(row):
    b, positions, bits, nbits, raw = row
    assert len(bits) == nbits
    payload, got_bits = oracle.golomb_encode(positions, b)
    assert got_bits == nbits
    assert bytes(payload) == raw
    # the byte string reads as the bit string, MSB first, zero padded
    as_bits = "".join(f"{byte:08b}" for byte in raw)
    assert as_bits[:nbits] == bits and set(as_bits[nbits:]) <= {"0"}
    # Algorithm 4 inverts it
    n = positions[-1] + 3
    dense = np.zeros(n, dtype=np.float32)
    assert oracle.golomb_decode(payload, nbits, b, 0.5, dense) == len(positions)
    want = np.zeros(n, dtype=np.float32)
    want[positions] = 0.5
    assert np.array_equal(dense, want)


def _python_bits(positions, b):
    """Algorithm 3 retyped with Python strings (independent of the C loop)."""
    out, prev = [], -1
    for idx in positions:
        g = idx - prev - 1
        prev = idx
        out.append("1" * (g >> b) + "0" + (format(g & ((1 << b) - 1), f"0{b}b") if b else ""))
    return "".join(out)


@pytest.mark.parametrize("b", [0, 1, 4, 6, 9, 13])
def test_golomb_random_round_trip_and_length(b):
    rng = np.random.default_rng(100 + b)
    n = 200000
    k = 1500
    pos = np.sort(rng.choice(n, size=k, replace=False)).astype(np.int64)
    payload, nbits = oracle.golomb_encode(pos, b)
    bits = _python_bits(pos.tolist(), b)
    assert nbits == len(bits)
    got = "".join(f"{byte:08b}" for byte in bytes(payload))
    assert got[:nbits] == bits and set(got[nbits:]) <= {"0"}
    gaps = np.diff(np.concatenate([[-1], pos])) - 1
    assert nbits == k * (1 + b) + int((gaps >> b).sum())
    assert nbits <= oracle.payload_bits_bound(n, k, b)
    dense = np.zeros(n, dtype=np.float32)
    assert oracle.golomb_decode(payload, nbits, b, -1.25, dense) == k
    assert np.array_equal(np.flatnonzero(dense), pos)
    assert np.all(dense[pos] == np.float32(-1.25))


def test_golomb_decode_rejects_truncated_and_out_of_range():
    payload, nbits = oracle.golomb_encode([7, 8, 40], 3)
    dense = np.zeros(64, dtype=np.float32)
    assert oracle.golomb_decode(payload, nbits - 2, 3, 1.0, dense) == -1   # ends inside a codeword
    dense = np.zeros(40, dtype=np.float32)                                   # position 40 is outside
    assert oracle.golomb_decode(payload, nbits, 3, 1.0, dense) == -1
    ones = np.array([0xFF], dtype=np.uint8)
    assert oracle.golomb_decode(ones, 8, 3, 1.0, np.zeros(512, dtype=np.float32)) == -1


# ---------------------------------------------------------------- Algorithm 2 / Algorithm 1

def test_worked_example_of_algorithm_2():
    pv = _paper_values()
    a = np.array([float(x) for x in pv["toy_A"].split()], dtype=np.float32)
    p = 0.2
    assert oracle.kept_count(a.size, p) == 2 and oracle.golomb_b(p) == 2
    res = np.zeros_like(a)
    stream, mu = oracle.encode(a.copy(), res, p)
    h = oracle.parse_header(stream)
    assert (h.k, h.b, h.side, h.nbits, h.numel) == (2, 2, 1, 8, 10)
    assert mu == np.float32(-2.75) and h.mu == np.float32(-2.75)
    want = a.copy()
    want[4], want[9] = -0.25, 0.25
    assert np.array_equal(res, want)
    assert stream[h.payload_offset] == 0x88
    # the two means
    work = a.copy()
    kept, side, mu32, mp, mn = oracle.compress(work, 2)
    assert (mp, mn, side) == (1.75, 2.75, 1) and kept.tolist() == [4, 9]


def test_side_choice_tie_goes_positive_and_signed_topk():
    a = np.array([1.0, -1.0, 0.25, -0.25], dtype=np.float32)
    kept, side, mu, mp, mn = oracle.compress(a.copy(), 1)
    assert (side, float(mu), kept.tolist()) == (0, 1.0, [0])          # mu+ == mu-: ">=" keeps +
    # fewer than k positive entries: Algorithm 2 still takes the k largest signed values
    a = np.array([-1.0, -2.0, 0.5, -3.0, -0.1], dtype=np.float32)
    kept, side, mu, mp, mn = oracle.compress(a.copy(), 2)
    assert mp == pytest.approx((0.5 - 0.1) / 2) and mn == pytest.approx(2.5)
    assert side == 1 and kept.tolist() == [1, 3] and float(mu) == -2.5


@pytest.mark.parametrize("name,upd,res,p", workloads.adversarial_cases(),
                         ids=[c[0] for c in workloads.adversarial_cases()])
def test_invariants_on_adversarial_cases(name, upd, res, p):
    n = upd.size
    k, b = oracle.kept_count(n, p), oracle.golomb_b(p)
    A = (res + upd).astype(np.float32)                     # what Algorithm 1 accumulates
    r_new = res.copy()
    stream, mu = oracle.encode(upd, r_new, p)
    h = oracle.parse_header(stream)
    assert (h.numel, h.k, h.b, h.status) == (n, k, b, 0)
    assert len(stream) == oracle.container_bytes(k, h.nbits) <= oracle.stream_bytes(n, p)
    # round trip: Algorithm 4 on the payload gives mu on exactly k positions
    dense = np.zeros(n, dtype=np.float32)
    oracle.decode_accumulate([stream], dense)
    kept = np.flatnonzero(dense) if mu != 0 else None
    changed = np.flatnonzero(r_new.view(np.uint32) != A.view(np.uint32))
    if mu != 0:
        assert kept.size == k and np.all(dense[kept] == mu)
        # Eq. (residual): A = dW* + R_new, exactly off the kept set, to rounding on it
        assert set(changed.tolist()) <= set(kept.tolist())
        assert np.array_equal(r_new[kept], (A[kept] - mu).astype(np.float32))
        # kept set = k extreme entries of the chosen side, ties by lower index
        assert np.array_equal(np.sort(_brute_topk(A, k, bool(h.side))), kept)
        # mean of the kept values, to fp32 rounding of the exactly rounded fp64 mean
        want_mu = np.float32(math.fsum(float(v) for v in A[kept]) / k)
        assert mu == want_mu
        # Theorem 2.1 with S = span(1_kept): the mean minimises ||A - c 1_kept||
        def err(c):
            return float(np.sum((A[kept].astype(np.float64) - float(c)) ** 2))
        assert err(mu) <= err(np.nextafter(mu, np.float32(np.inf))) * (1 + 1e-12)
        assert err(mu) <= err(np.nextafter(mu, np.float32(-np.inf))) * (1 + 1e-12)
    else:
        assert changed.size == 0
    # side choice: the larger of the two exactly computed means, ">=" to the positive side
    mp = math.fsum(float(v) for v in A[_brute_topk(A, k, False)]) / k
    mn = -math.fsum(float(v) for v in A[_brute_topk(A, k, True)]) / k
    assert h.side == (0 if mp >= mn else 1)


def test_mean_code_length_matches_the_closed_form_on_iid_input():
    n, p = 2**20, 0.01
    upd = workloads.normal_flat(n, 1e-3, workloads.seed_for(1))
    res = np.zeros(n, dtype=np.float32)
    stream, _ = oracle.encode(upd, res, p)
    h = oracle.parse_header(stream)
    assert h.k == 10485 and h.b == 6
    per = h.nbits / h.k
    assert abs(per - oracle.mean_position_bits(p, h.b)) < 0.1      # ~5 standard errors
    assert h.nbits <= oracle.payload_bits_bound(n, h.k, h.b) == 10485 * 7 + ((n - 10485) >> 6)


def test_chunk_size_rule():
    # convention (unpinned by the paper): 32 codewords per chunk below 2^17 positions, 64 below 2^21, 256 beyond
    assert [oracle.chunk_codewords(k) for k in (1, 32, 33, 2**17 - 1)] == [32] * 4
    assert [oracle.chunk_codewords(k) for k in (2**17, 2**20, 2**21 - 1)] == [64] * 3
    assert [oracle.chunk_codewords(k) for k in (2**21, 2**25, 2**31 - 1)] == [256] * 3


@pytest.mark.parametrize("n,p,chunk", [
    (300_000, 0.01, 32),        # k = 3000
    (70_001, 0.3, 32),          # k = 21000, b = 1
    (400_000, 0.4, 64),         # k = 160000 >= 2^17, b = 0
    (2_200_000, 0.06, 64),      # k = 132000, b = 4
    (4_300_000, 0.5, 256),      # k = 2150000 >= 2^21, b = 0
])
def test_container_chunk_table_and_padding(n, p, chunk):
    """Every chunk-table entry, at every chunk size, against an independent parse of the payload
    bit string in Python (Algorithm 4 on a character string)."""
    rng = np.random.default_rng(n)
    k, b = oracle.kept_count(n, p), oracle.golomb_b(p)
    idx = np.sort(rng.choice(n, size=k, replace=False)).astype(np.int64)
    stream = oracle.container(idx, n, p, 1, -0.5)
    h = oracle.parse_header(stream)
    assert h.magic == oracle.MAGIC and h.version == 1 and h.k == k and h.b == b
    assert h.chunk_codewords == chunk == oracle.chunk_codewords(k)
    assert h.n_chunks == -(-h.k // chunk)
    assert h.payload_offset == 64 + 16 * h.n_chunks
    assert len(stream) % 16 == 0
    payload = bytes(stream[h.payload_offset:])
    bits = "".join(f"{byte:08b}" for byte in payload)
    assert set(bits[h.nbits:]) <= {"0"}
    table = stream[64:h.payload_offset].view("<u8").reshape(-1, 2)
    assert table.shape[0] == h.n_chunks
    i, prev, count = 0, -1, 0
    decoded = np.empty(k, dtype=np.int64)
    while count < h.k:
        if count % chunk == 0:
            assert int(table[count // chunk, 0]) == i
            assert int(table[count // chunk, 1].astype(np.int64)) == prev
        j = bits.index("0", i)            # end of the unary part
        q = j - i
        r = int(bits[j + 1:j + 1 + h.b], 2) if h.b else 0
        prev = prev + (q << h.b) + r + 1
        decoded[count] = prev
        i = j + 1 + h.b
        count += 1
    assert i == h.nbits
    assert np.array_equal(decoded, idx)


def test_decode_accumulate_sums_clients_in_fp32():
    rng = np.random.default_rng(9)
    n, p = 50000, 0.01
    streams, want = [], np.zeros(n, dtype=np.float64)
    for c in range(8):
        upd = rng.standard_normal(n).astype(np.float32)
        res = np.zeros(n, dtype=np.float32)
        s, mu = oracle.encode(upd, res, p)
        streams.append(s)
        A = upd
        side = oracle.parse_header(s).side
        kept = np.sort(_brute_topk(A, oracle.kept_count(n, p), bool(side)))
        want[kept] += float(mu)
    out = np.zeros(n, dtype=np.float32)
    oracle.decode_accumulate(streams, out)
    assert np.allclose(out, want, rtol=0, atol=1e-6 * 8 * 3.0)
    # adds onto what is already there
    out2 = np.ones(n, dtype=np.float32)
    oracle.decode_accumulate(streams[:1], out2)
    d = np.zeros(n, dtype=np.float32)
    oracle.decode_accumulate(streams[:1], d)
    assert np.array_equal(out2, (np.ones(n, dtype=np.float32) + d))


def test_rejects_bad_arguments_and_non_finite_input():
    upd = np.array([1.0, np.inf, 0.0], dtype=np.float32)
    with pytest.raises(ValueError):
        oracle.encode(upd, np.zeros(3, dtype=np.float32), 0.5)
    with pytest.raises(ValueError):
        oracle.encode(np.ones(3, dtype=np.float32), np.zeros(3, dtype=np.float32), 1.5)
    good, _ = oracle.encode(np.ones(3, dtype=np.float32), np.zeros(3, dtype=np.float32), 0.5)
    bad = good.copy()
    bad[0] ^= 0xFF
    with pytest.raises(ValueError):
        oracle.decode_accumulate([bad], np.zeros(3, dtype=np.float32))


def test_side_and_mu_and_container_entry_points():
    # Algorithm 2's decision from the two sums (worked example: sums 3.5 and -5.5 over k = 2)
    assert oracle.side_and_mu(3.5, -5.5, 2) == (1, np.float32(-2.75), 1.75, 2.75)
    assert oracle.side_and_mu(2.0, -2.0, 2)[:2] == (0, np.float32(1.0))          # tie keeps the positive side
    assert oracle.side_and_mu(-1.0, -9.0, 3)[:2] == (1, np.float32(-3.0))
    # the container built from a position list is the one encode() emits
    rng = np.random.default_rng(21)
    n, p = 40000, 0.01
    upd = rng.standard_normal(n).astype(np.float32)
    res = np.zeros(n, dtype=np.float32)
    stream, mu = oracle.encode(upd, res, p)
    h = oracle.parse_header(stream)
    kept = np.sort(_brute_topk(upd, h.k, bool(h.side)))
    assert np.array_equal(oracle.container(kept, n, p, h.side, mu), stream)


def test_decode_apply_against_dense_fp64():
    # Algorithm 1's server lines, checked against a dense fp64 computation from the kept sets
    rng = np.random.default_rng(31)
    n, p, n_clients = 30000, 0.01, 4
    streams, dense64, hit = [], np.zeros(n), np.zeros(n, dtype=bool)
    for c in range(n_clients):
        upd = rng.standard_normal(n).astype(np.float32)
        s, mu = oracle.encode(upd, np.zeros(n, dtype=np.float32), p)
        streams.append(s)
        kept = np.sort(_brute_topk(upd, oracle.kept_count(n, p), bool(oracle.parse_header(s).side)))
        dense64[kept] += float(mu)
        hit[kept] = True
    w0 = rng.standard_normal(n).astype(np.float32)
    m0 = rng.standard_normal(n).astype(np.float32)
    w, m = w0.copy(), m0.copy()
    oracle.decode_apply(streams, 1.0 / n_clients, w, m)
    want = w0.astype(np.float64) + dense64 / n_clients
    assert np.max(np.abs(w - want)) <= 1e-6 * (np.max(np.abs(w0)) + np.max(np.abs(dense64)))
    assert np.array_equal(w[~hit], w0[~hit])                 # untouched where nothing was sent
    assert np.all(m[hit] == 0) and np.array_equal(m[~hit], m0[~hit])
    # scale 1, zero weights, no momentum: the plain server sum
    z = np.zeros(n, dtype=np.float32)
    oracle.decode_apply(streams, 1.0, z)
    d = np.zeros(n, dtype=np.float32)
    oracle.decode_accumulate(streams, d)
    assert np.array_equal(z, d)


# ---------------------------------------------------------------- Gradient Dropping baseline

@pytest.mark.parametrize("seed,n,p", [(1, 10, 0.2), (2, 5000, 0.01), (3, 40000, 0.001), (4, 777, 0.3)])
def test_gradient_dropping_against_brute_force(seed, n, p):
    rng = np.random.default_rng(seed)
    upd = np.round(rng.standard_normal(n) * 4).astype(np.float32) / 4     # ties in magnitude
    res0 = (rng.standard_normal(n) * 0.1).astype(np.float32)
    A = (res0 + upd).astype(np.float32)
    k, b = oracle.kept_count(n, p), oracle.golomb_b(p)
    res = res0.copy()
    stream = oracle.encode_values(upd, res, p)
    h = oracle.parse_header(stream)
    assert (h.k, h.b, h.side, h.numel) == (k, b, 2, n)
    # kept set: k largest magnitudes, equal magnitudes by lower index (stable argsort of -|A|)
    kept = np.sort(np.argsort(-np.abs(A).astype(np.float64), kind="stable")[:k])
    assert np.array_equal(np.sort(oracle.topk_abs(A, k)), kept)
    # values travel as they are, in position order, between the chunk table and the payload
    values = stream[64 + 16 * h.n_chunks: 64 + 16 * h.n_chunks + 4 * k].view("<f4")
    assert np.array_equal(values.view(np.uint32), A[kept].view(np.uint32))
    assert h.payload_offset == 64 + 16 * h.n_chunks + ((4 * k + 15) // 16) * 16
    # residual: everything that was not sent; exactly zero where it was
    want_res = A.copy()
    want_res[kept] = 0.0
    assert np.array_equal(res, want_res)
    # the position payload is Algorithm 3's, identical to what SBC would emit for the same set
    payload, nbits = oracle.golomb_encode(kept, b)
    assert h.nbits == nbits
    assert bytes(stream[h.payload_offset: h.payload_offset + len(payload)]) == bytes(payload)
    # decoding gives dW* = A on the kept set
    dense = np.zeros(n, dtype=np.float32)
    oracle.decode_accumulate([stream], dense)
    want = np.zeros(n, dtype=np.float32)
    want[kept] = A[kept]
    assert np.array_equal(dense, want)
    assert len(stream) <= oracle.stream_bytes_values(n, p)


def test_bit_accounting_of_binarisation_and_golomb_coding():
    # Fig. 2 caption of the paper: binarisation gains about x3 over sparse 32-bit values with
    # naive 16-bit positions; Golomb coding gains up to another x2 over 16-bit positions
    n, p = 2**20, 0.01
    upd = workloads.normal_flat(n, 1e-3, workloads.seed_for(1))
    sbc_stream, _ = oracle.encode(upd, np.zeros(n, dtype=np.float32), p)
    gd_stream = oracle.encode_values(upd, np.zeros(n, dtype=np.float32), p)
    hs, hg = oracle.parse_header(sbc_stream), oracle.parse_header(gd_stream)
    k = hs.k
    naive_gd_bits = k * (32 + 16)
    golomb_gd_bits = k * 32 + hg.nbits
    sbc_naive_bits = k * 16 + 32
    sbc_bits = hs.nbits + 32
    assert 2.8 < naive_gd_bits / sbc_naive_bits < 3.1          # 32 -> 0 value bits
    assert 1.8 < sbc_naive_bits / sbc_bits < 2.1               # 16 -> ~8.1 position bits
    assert abs(hg.nbits / k - oracle.mean_position_bits(p, hg.b)) < 0.1
    assert golomb_gd_bits < naive_gd_bits


# ---------------------------------------------------------------- subsampled thresholds

def test_sampled_thresholds_with_the_whole_tensor_as_sample_equal_the_exact_method():
    # sample = every position, distinct values: floor(p*n) = k and the j-th order statistics are the
    # exact thresholds, so the result must be the exact method's
    rng = np.random.default_rng(41)
    n, p = 20000, 0.01
    upd = rng.standard_normal(n).astype(np.float32)
    res = (rng.standard_normal(n) * 0.1).astype(np.float32)
    r1, r2 = res.copy(), res.copy()
    s1, m1 = oracle.encode(upd, r1, p)
    s2, m2 = oracle.encode_sampled(upd, r2, p, np.arange(n, dtype=np.uint32))
    assert np.array_equal(s1, s2) and m1 == m2 and np.array_equal(r1, r2)


@pytest.mark.parametrize("seed", [1, 2, 3])
def test_sampled_thresholds_against_a_numpy_restatement(seed):
    rng = np.random.default_rng(seed)
    n, p, m = 200000, 0.01, 5000
    upd = (rng.standard_t(3, n) * 1e-3).astype(np.float32)
    res = (rng.standard_normal(n) * 1e-3).astype(np.float32)
    A = (res + upd).astype(np.float32)
    idx = rng.integers(0, n, m).astype(np.uint32)
    r = res.copy()
    stream, mu = oracle.encode_sampled(upd, r, p, idx)
    h = oracle.parse_header(stream)
    sv = np.sort(A[idx])[::-1]
    j = max(1, int(np.floor(p * m)))
    t_pos, t_neg = sv[j - 1], sv[m - j]
    P, N = np.flatnonzero(A >= t_pos), np.flatnonzero(A <= t_neg)
    mp = math.fsum(float(v) for v in A[P]) / P.size
    mn = -math.fsum(float(v) for v in A[N]) / N.size
    side = 0 if mp >= mn else 1
    kept = N if side else P
    assert (h.side, h.k) == (side, kept.size)
    assert mu == np.float32(-mn if side else mp)
    dense = np.zeros(n, dtype=np.float32)
    oracle.decode_accumulate([stream], dense)
    assert np.array_equal(np.flatnonzero(dense), kept)
    want_r = A.copy()
    want_r[kept] = (A[kept] - mu).astype(np.float32)
    assert np.array_equal(r, want_r)
    k = oracle.kept_count(n, p)
    assert 0.5 * k < kept.size < 2 * k             # noise in the amount of sparsity, not in its scale


def test_sampled_thresholds_fall_back_to_the_exact_method_when_the_estimate_is_useless():
    n, p = 5000, 0.01
    upd = np.zeros(n, dtype=np.float32)           # threshold 0: every entry would be kept
    upd[:10] = 1.0
    r1, r2 = np.zeros(n, dtype=np.float32), np.zeros(n, dtype=np.float32)
    s1, m1 = oracle.encode(upd, r1, p)
    s2, m2 = oracle.encode_sampled(upd, r2, p, np.arange(100, 200, dtype=np.uint32))
    assert np.array_equal(s1, s2) and m1 == m2 and np.array_equal(r1, r2)
