"""halos_push_noalloc against the regular push (halos_lps_push on a statistics-enabled context).

The entry point serves callers that are not allowed to allocate device memory (frozen or exhausted
pools, start-up-only allocation policies), so its reduction scratch is a fixed array inside the
library that all calls share.  The test calls it twice in a row through the C ABI -- first on a
large vector, then on a smaller, different one, so that stale partial sums of the first call would
show up in the second -- and compares Delta bit for bit and the squared norm within the tolerance
the statistics tests use: against the regular push, and against a host computation that involves
no CUDA code (fp32 subtraction in numpy, squares summed in fp64), so that a mistake shared by the
two CUDA paths cannot hide.  It also checks that a warmed-up call leaves the amount of free device
memory unchanged and that a misaligned result pointer is refused on the host.  It lives in a file of its own that sorts last, so a run that stops at the
first failure has already finished every other test; it builds its own inputs and also passes alone.
"""
from __future__ import annotations

import numpy as np
import pytest
import torch

pytestmark = pytest.mark.gpu

STATS_RTOL = 2e-6   # same bound as tests/test_gpu_parity.py::test_norm_statistics


def _pushed_context(P, seed, n_arrivals):
    from paper_2506_04531_b200 import binding as hb
    from paper_2506_04531_b200.inputs import gen, layouts
    lay = layouts.flat_layout("x", P)
    init = torch.from_numpy(gen.theta_init(lay, seed)).cuda()
    h = hb.Halos(init, [0], K=1000, flags=hb.FLAG_STATS)
    for r in range(n_arrivals):
        res = gen.worker_result(h.read(hb.BUF_THETA0, 0), lay, seed, 0, r)
        h.worker_delta(0, torch.from_numpy(res).cuda())
        h.lps_apply(0, 0)
    theta = h.peek(hb.BUF_THETA_L, 0).clone()
    anchor = h.peek(hb.BUF_ANCHOR, 0).clone()
    h.lps_push(0)                                       # the existing entry point
    want_Delta = h.read(hb.BUF_OUTBOX, 0)
    want_sq = float(h.stats(1, 0).sum())
    h.close()
    return theta, anchor, want_Delta, want_sq


def test_push_noalloc_twice_in_a_row():
    from paper_2506_04531_b200 import binding as hb, build
    build.build()
    big = _pushed_context(3_000_003, seed=11, n_arrivals=2)      # ragged tail, 367 chunks
    small = _pushed_context(70_001, seed=12, n_arrivals=3)       # 9 chunks: most slots keep the first call's sums
    warm = torch.zeros(1, dtype=torch.float64, device="cuda")
    assert hb.push_noalloc(big[0], big[1], big[0], warm, n=0) == hb.OK     # start-up call: loads kernels and scratch
    torch.cuda.synchronize()
    for theta, anchor, want_Delta, want_sq in (big, small):
        out = torch.full_like(theta, float("nan"))
        sq = torch.full((1,), float("nan"), dtype=torch.float64, device="cuda")
        torch.cuda.synchronize()
        free_before = torch.cuda.mem_get_info()[0]
        assert hb.push_noalloc(theta, anchor, out, sq) == hb.OK
        torch.cuda.synchronize()
        assert torch.cuda.mem_get_info()[0] == free_before          # nothing was allocated on the device
        assert np.array_equal(out.cpu().numpy().view(np.uint32), want_Delta.view(np.uint32))
        assert want_sq > 0
        assert abs(float(sq.item()) - want_sq) <= STATS_RTOL * want_sq
        # the same two results from the host alone
        host_Delta = theta.cpu().numpy() - anchor.cpu().numpy()     # fp32, one rounding per element
        assert np.array_equal(out.cpu().numpy().view(np.uint32), host_Delta.view(np.uint32))
        host_sq = float(np.sum(host_Delta.astype(np.float64) ** 2))
        assert abs(float(sq.item()) - host_sq) <= STATS_RTOL * host_sq
    # unaligned views take the scalar path and give the same answer
    theta, anchor, want_Delta, want_sq = small
    pad = lambda t: torch.cat([t.new_zeros(1), t])[1:]
    out = pad(torch.empty_like(theta))
    sq = torch.zeros(1, dtype=torch.float64, device="cuda")
    assert hb.push_noalloc(pad(theta), pad(anchor), out, sq) == hb.OK
    torch.cuda.synchronize()
    assert np.array_equal(out.cpu().numpy().view(np.uint32), want_Delta.view(np.uint32))
    assert abs(float(sq.item()) - want_sq) <= STATS_RTOL * want_sq
    # a result pointer that cannot hold a double is refused before anything is launched
    two = torch.full((2,), 3.0, dtype=torch.float64, device="cuda")
    assert hb.push_noalloc(theta, anchor, out, two.data_ptr() + 4) == hb.ERR_INVALID_ARG
    torch.cuda.synchronize()
    assert two.tolist() == [3.0, 3.0]
    # empty input: defined result, and sizes beyond the fixed scratch are refused up front
    assert hb.push_noalloc(theta, anchor, out, sq, n=0) == hb.OK
    torch.cuda.synchronize()
    assert float(sq.item()) == 0.0
    sq.fill_(7.0)
    assert hb.push_noalloc(theta, anchor, out, sq, n=hb.NOALLOC_MAX_ELEMS + 1) == hb.ERR_UNSUPPORTED
    torch.cuda.synchronize()
    assert float(sq.item()) == 7.0
