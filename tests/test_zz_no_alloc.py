"""sbc_encode_static -- the entry point for callers that are not allowed to allocate.

Some users of this library run where device allocation is off the table: a compression hook
invoked from a framework's communication step, or a long-running service that fixes its memory
at start-up.  For them the library carries its own fixed scratch array.  This file checks, through
the C ABI, that the variant produces exactly what sbc_encode produces, on two calls in a row
(the second call reuses the scratch the first one dirtied), and that oversized problems are
refused.  It is named so that pytest collects it last.
"""
import numpy as np
import pytest
import torch

from paper_1805_08768_b200 import binding as sbc
from paper_1805_08768_b200 import workloads

pytestmark = pytest.mark.gpu

if not torch.cuda.is_available():  # pragma: no cover
    pytest.skip("needs a CUDA device", allow_module_level=True)

DEV = torch.device("cuda:0")


def _both_ways(upd_np, res_np, p):
    n = upd_np.size
    cap = sbc.sbc_stream_bytes(n, p)
    results = []
    for use_static in (False, True):
        u = torch.from_numpy(upd_np).to(DEV)
        r = torch.from_numpy(res_np).to(DEV)
        out = torch.zeros(cap, dtype=torch.uint8, device=DEV)
        mu = torch.zeros(1, dtype=torch.float32, device=DEV)
        if use_static:
            sbc.sbc_encode_static(u, r, p, out, mu)
        else:
            sbc.sbc_encode(u, r, p, out_stream=out, out_mu=mu)
        info = sbc.sbc_stream_info_get(out)
        torch.cuda.synchronize()
        results.append((out[: info.total_bytes].cpu().numpy(), mu.cpu().numpy(), r.cpu().numpy()))
    return results


def test_static_scratch_matches_sbc_encode_on_two_calls_in_a_row():
    # call 1: ~1 M elements (a little over half of the fixed scratch), call 2: a different size, p
    # and a carried residual, run over the scratch the first call dirtied
    cases = [
        (workloads.normal_flat(1 << 20, 1e-3, 901), np.zeros(1 << 20, dtype=np.float32), 0.01),
        (workloads.student_t_flat(300001, 902), workloads.normal_flat(300001, 2e-3, 903), 0.001),
    ]
    for upd, res, p in cases:
        assert sbc.sbc_workspace_bytes(upd.size, p) <= sbc.STATIC_WORKSPACE_BYTES
        (s0, m0, r0), (s1, m1, r1) = _both_ways(upd, res, p)
        assert np.array_equal(s0, s1)                                   # container byte for byte
        assert np.array_equal(m0.view(np.uint32), m1.view(np.uint32))   # mu bit for bit
        assert np.array_equal(r0.view(np.uint32), r1.view(np.uint32))   # residual bit for bit


def test_static_scratch_at_its_limit_then_a_small_call():
    # the largest problem the fixed array takes at p = 0.01 (its scratch fills all but a few KB of
    # the 8 MiB), then a small one that reuses the same bytes
    p = 0.01
    lo, hi = 1, 1 << 26                       # the largest n whose scratch fits, by bisection on the host
    while hi - lo > 1:
        mid = (lo + hi) // 2
        if sbc.sbc_workspace_bytes(mid, p) <= sbc.STATIC_WORKSPACE_BYTES:
            lo = mid
        else:
            hi = mid
    n = lo - 1000
    assert 2_000_000 < n < 4_000_000          # what the header says about the limit (about 2.6 M at p = 0.01)
    need = sbc.sbc_workspace_bytes(n, p)
    assert 0.98 * sbc.STATIC_WORKSPACE_BYTES < need <= sbc.STATIC_WORKSPACE_BYTES
    assert sbc.sbc_workspace_bytes(n + 20_000, p) > sbc.STATIC_WORKSPACE_BYTES
    for upd, res in ((workloads.student_t_flat(n, 904), workloads.normal_flat(n, 1e-3, 905)),
                     (workloads.normal_flat(5000, 1e-3, 906), np.zeros(5000, dtype=np.float32))):
        (s0, m0, r0), (s1, m1, r1) = _both_ways(upd, res, p)
        assert np.array_equal(s0, s1)
        assert np.array_equal(m0.view(np.uint32), m1.view(np.uint32))
        assert np.array_equal(r0.view(np.uint32), r1.view(np.uint32))


def test_static_scratch_refuses_what_does_not_fit():
    n, p = 1 << 24, 0.01
    assert sbc.sbc_workspace_bytes(n, p) > sbc.STATIC_WORKSPACE_BYTES
    u = torch.zeros(n, dtype=torch.float32, device=DEV)
    r = torch.zeros(n, dtype=torch.float32, device=DEV)
    out = torch.zeros(sbc.sbc_stream_bytes(n, p), dtype=torch.uint8, device=DEV)
    mu = torch.zeros(1, dtype=torch.float32, device=DEV)
    with pytest.raises(sbc.SbcError) as e:
        sbc.sbc_encode_static(u, r, p, out, mu)
    assert e.value.code == sbc.SBC_ECAPACITY
    torch.cuda.synchronize()
    assert not bool(r.any()) and not bool(out.any())                    # nothing was enqueued
