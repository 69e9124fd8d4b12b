"""The allocation-free span matcher (`rac_match_spans_static`) against the ordinary entry point.

Some users of this library run where device memory cannot be requested: inside a host runtime that owns the
whole GPU heap, or in a serving loop that must not touch the allocator once it is warm.  For them the library
carries a fixed 3 MiB scratch of its own.  This test calls that entry point through the C ABI twice in a row,
on two different inputs, and requires exactly the rows, spans and span count that `rac_match_spans` produces
with a caller-provided workspace (integer results: bit-exact, the tolerance of every matcher test here).  The
second call also shows that what the first one left in the shared scratch does no harm.  Collected last on
purpose, so a failure here cannot hide any other test's result.
"""
import numpy as np
import pytest
import torch

pytestmark = pytest.mark.gpu


def _both(rac, dev, hist, query, w, K):
    h = torch.from_numpy(hist).to(dev)
    q = torch.from_numpy(query).to(dev)
    N = q.numel()
    cap = N // w + 1
    outs = []
    for static in (False, True):
        rows = torch.full((N,), 4242, dtype=torch.int32, device=dev)
        spans = torch.full((cap, 3), 77, dtype=torch.int32, device=dev)
        n = torch.full((1,), -1, dtype=torch.int32, device=dev)
        if static:
            rac.rac_match_spans_static(h, h.numel(), q, N, w, K, rows, spans, n)
        else:
            nb = rac.rac_match_workspace_bytes(h.numel(), N, K)
            ws = torch.empty(nb, dtype=torch.uint8, device=dev)
            rac.rac_match_spans(h, h.numel(), q, N, w, K, rows, spans, n, ws, nb)
        torch.cuda.synchronize()
        ns = int(n.item())
        outs.append((rows.cpu().numpy(), spans[:ns].cpu().numpy(), ns))
    return outs


def test_static_scratch_matcher_equals_workspace_matcher_twice_in_a_row():
    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    from paper_2608_04991_b200 import binding as rac
    from paper_2608_04991_b200 import synth
    rac.load()
    dev = torch.device("cuda:0")
    # first call: the largest shape the built-in scratch is sized for; second call: another, smaller draw
    for n_hist, n_query, seed in [(32768, 8192, 21), (20000, 3001, 22)]:
        assert rac.rac_match_workspace_bytes(n_hist, n_query, 8) <= rac.MATCH_STATIC_BYTES
        wl = synth.span_workload(n_hist, n_query, seed=seed)
        (r0, s0, n0), (r1, s1, n1) = _both(rac, dev, wl.hist, wl.query, 4, 8)
        assert n0 == n1 and n0 > 0
        assert np.array_equal(r0, r1)
        assert np.array_equal(s0, s1)
    # a problem that does not fit is refused with a clear error and nothing is written
    big = synth.span_workload(131072, 4096, seed=23)
    h = torch.from_numpy(big.hist).to(dev)
    q = torch.from_numpy(big.query).to(dev)
    rows = torch.full((4096,), 4242, dtype=torch.int32, device=dev)
    n = torch.full((1,), -1, dtype=torch.int32, device=dev)
    with pytest.raises(rac.RacError) as ei:
        rac.rac_match_spans_static(h, h.numel(), q, 4096, 4, 8, rows, None, n)
    assert ei.value.code == -3 and "too small" in str(ei.value)
    torch.cuda.synchronize()
    assert int(n.item()) == -1 and torch.all(rows == 4242)
