"""Pins for the oracle's span matcher (Sec. IV-B.1, Eq. 3), CPU only.

The oracle indexes sorted windows; these tests restate the definition by brute
force with different machinery (a longest-common-extension table filled from the
back, plain Python scans) and check structural invariants on larger draws.
"""
import numpy as np
import pytest

from paper_2608_04991_b200 import synth


def brute_force(hist, query, w, K):
    """Greedy cover straight from the definition, O(N*H) with an LCE table."""
    H, N = len(hist), len(query)
    lce = np.zeros((N + 1, H + 1), np.int32)
    for i in range(N - 1, -1, -1):
        for j in range(H - 1, -1, -1):
            if query[i] == hist[j]:
                lce[i, j] = lce[i + 1, j + 1] + 1
    ref_row = np.full(N, -1, np.int32)
    spans = []
    i = 0
    while i < N:
        cands = [j for j in range(H) if lce[i, j] >= w]   # windows equal <=> lce >= w
        if K > 0:
            cands = sorted(cands)[-K:]                     # the K most recent (largest start)
        if not cands:
            i += 1
            continue
        L, j = max((int(lce[i, j]), j) for j in cands)     # longest, then most recent
        spans.append((i, j, L))
        ref_row[i:i + L] = np.arange(j, j + L)
        i += L
    return ref_row, np.array(spans, np.int32).reshape(-1, 3)


@pytest.mark.parametrize("seed", range(6))
@pytest.mark.parametrize("K", [0, 1, 2, 8])
def test_matches_brute_force_on_tiny_inputs(orc, seed, K):
    rng = np.random.default_rng(100 + seed)
    vocab = [2, 3, 5][seed % 3]          # tiny vocabularies: many repeated windows, long chance matches
    w = [1, 2, 3, 4][seed % 4]
    H, N = int(rng.integers(5, 70)), int(rng.integers(1, 60))
    hist = rng.integers(0, vocab, H).astype(np.int32)
    query = rng.integers(0, vocab, N).astype(np.int32)
    if seed % 2:  # plant a copy so long spans exist too
        L = min(N, H, 17)
        query[N - L:] = hist[:L]
    rr, sp = orc.match_spans(hist, query, w=w, max_hits=K)
    brr, bsp = brute_force(hist, query, w, K)
    assert np.array_equal(rr, brr)
    assert np.array_equal(sp, bsp)


def test_adversarial_cases(orc):
    w = 4
    # query shorter than w: nothing can match
    rr, sp = orc.match_spans(np.arange(20, dtype=np.int32), np.arange(3, dtype=np.int32), w=w)
    assert np.all(rr == -1) and len(sp) == 0
    # history shorter than w
    rr, sp = orc.match_spans(np.arange(3, dtype=np.int32), np.arange(3, dtype=np.int32), w=w)
    assert np.all(rr == -1) and len(sp) == 0
    # query == history: one span covering everything, start 0 (the only start that reaches full length)
    h = np.random.default_rng(1).integers(0, 1000, 300).astype(np.int32)
    rr, sp = orc.match_spans(h, h.copy(), w=w)
    assert np.array_equal(sp, [[0, 0, 300]]) and np.array_equal(rr, np.arange(300))
    # all-same token: every window matches everywhere.  Unlimited hits: starts 0..24 all reach the full
    # query length 40, the most recent of them (24) wins.  With K = 8 only the 8 most recent starts are
    # candidates: the earliest of them extends furthest.
    ones = np.ones(64, np.int32)
    rr, sp = orc.match_spans(ones, ones[:40].copy(), w=w, max_hits=0)
    assert np.array_equal(sp, [[0, 24, 40]])
    rr, sp = orc.match_spans(ones, ones[:40].copy(), w=w, max_hits=8)
    starts = 64 - w - np.arange(8)       # 60..53
    first = int(starts.min())
    assert sp[0].tolist() == [0, first, 64 - first]
    bf_rr, bf_sp = brute_force(ones, ones[:40], w, 8)
    assert np.array_equal(sp, bf_sp) and np.array_equal(rr, bf_rr)
    # a match running into the end of the history and one running into the end of the query
    hist = np.array([9, 9, 1, 2, 3, 4, 5], np.int32)
    query = np.array([1, 2, 3, 4, 5, 6, 7, 1, 2, 3, 4], np.int32)
    rr, sp = orc.match_spans(hist, query, w=w)
    assert sp.tolist() == [[0, 2, 5], [7, 2, 4]]
    assert rr.tolist() == [2, 3, 4, 5, 6, -1, -1, 2, 3, 4, 5]
    # equal length, two starts: the more recent (larger) start wins
    hist = np.array([1, 2, 3, 4, 0, 1, 2, 3, 4, 8], np.int32)
    rr, sp = orc.match_spans(hist, np.array([1, 2, 3, 4, 7], np.int32), w=w)
    assert sp.tolist() == [[0, 5, 4]]
    # longer beats more recent
    hist = np.array([1, 2, 3, 4, 7, 0, 1, 2, 3, 4, 8], np.int32)
    rr, sp = orc.match_spans(hist, np.array([1, 2, 3, 4, 7], np.int32), w=w)
    assert sp.tolist() == [[0, 0, 5]]


def check_invariants(hist, query, w, K, rr, sp):
    N, H = len(query), len(hist)
    covered = np.zeros(N, bool)
    prev_end = 0
    for (i, j, L) in sp.tolist():
        assert L >= w and i >= prev_end                      # ordered, disjoint in the query
        assert np.array_equal(query[i:i + L], hist[j:j + L])  # an exact match
        at_end = (i + L == N) or (j + L == H)
        assert at_end or query[i + L] != hist[j + L]          # maximal
        assert np.array_equal(rr[i:i + L], np.arange(j, j + L))
        covered[i:i + L] = True
        prev_end = i + L
    assert np.all(rr[~covered] == -1)
    return covered


def test_invariants_and_hit_cap_on_zipf_workload(orc):
    wl = synth.span_workload(4096, 2048, seed=1)
    w = 4
    rr8, sp8 = orc.match_spans(wl.hist, wl.query, w=w, max_hits=8)
    rr0, sp0 = orc.match_spans(wl.hist, wl.query, w=w, max_hits=0)
    cov8 = check_invariants(wl.hist, wl.query, w, 8, rr8, sp8)
    check_invariants(wl.hist, wl.query, w, 0, rr0, sp0)
    # window occurrence counts by a dictionary (independent of the oracle's sorted index)
    counts = {}
    for j in range(len(wl.hist) - w + 1):
        key = tuple(wl.hist[j:j + w])
        counts[key] = counts.get(key, 0) + 1
    # uncovered scan positions have no candidate at all
    i = 0
    spans_by_start = {s[0]: s for s in sp8.tolist()}
    while i < len(wl.query):
        if i in spans_by_start:
            i += spans_by_start[i][2]
            continue
        if i + w <= len(wl.query):
            assert tuple(wl.query[i:i + w]) not in counts
        assert not cov8[i]
        i += 1
    # when no window occurs more than 8 times, the cap cannot matter
    if max(counts.values()) <= 8:
        assert np.array_equal(sp8, sp0)
    # planted spans are found (a planted copy can only be extended or merged, never lost, except
    # where a chance match starting earlier swallowed its head)
    planted = wl.planted_row >= 0
    assert cov8[planted].mean() > 0.97
    assert 0.4 < wl.planted_coverage < 0.8  # about 60 % on long queries, noisy on a short one


def test_cap_changes_result_only_for_frequent_windows(orc):
    # one window occurs 12 times; with K = 8 the four oldest starts are not candidates, so the longest
    # continuation (planted at the oldest start) is missed, with K = 0 it is found.
    rng = np.random.default_rng(3)
    filler = lambda n: rng.integers(100, 10000, n).astype(np.int32)
    gram = np.array([1, 2, 3, 4], np.int32)
    tail = np.array([50, 51, 52, 53, 54], np.int32)
    parts = [gram, tail, filler(5)]
    for _ in range(11):
        parts += [gram, filler(6)]
    hist = np.concatenate(parts)
    query = np.concatenate([gram, tail])
    _, sp0 = orc.match_spans(hist, query, w=4, max_hits=0)
    _, sp8 = orc.match_spans(hist, query, w=4, max_hits=8)
    assert sp0.tolist() == [[0, 0, 9]]
    last = int(np.flatnonzero((hist[:-3] == 1) & (hist[1:-2] == 2) & (hist[2:-1] == 3) & (hist[3:] == 4)).max())
    assert sp8.tolist()[0] == [0, last, 4]
    b_rr, b_sp = brute_force(hist, query, 4, 8)
    assert np.array_equal(sp8, b_sp)


# ------------------------------------------------------------------ earlier requests and intra-sequence references
def brute_force_requests(reqs, query, w, K, intra, first_live=0):
    """The definition per request: candidate (r, j, L) with query[i:i+L] == reqs[r][j:j+L], L >= w maximal inside
    request r; recency = (r, j); the K most recent hits per distinct window; longest, then most recent."""
    N = len(query)
    off = np.concatenate([[0], np.cumsum([len(r) for r in reqs])]).astype(np.int64)
    ref_row = np.full(N, -1, np.int32)
    spans = []
    i = 0
    while i < N:
        hits = []   # (r, j) of every request window equal to the query window at i
        if i + w <= N:
            for r, req in enumerate(reqs):
                for j in range(len(req) - w + 1):
                    if list(req[j:j + w]) == list(query[i:i + w]) and off[r] + j >= first_live:
                        hits.append((r, j))
        if K > 0:
            hits = sorted(hits)[-K:]
        if not hits:
            i += 1
            continue
        best = None
        for r, j in hits:
            L = w
            while i + L < N and j + L < len(reqs[r]) and query[i + L] == reqs[r][j + L]:
                L += 1
            key = (L, r, j)
            if best is None or key > best:
                best = key
        L, r, j = best
        spans.append((i, int(off[r]) + j, L))
        ref_row[i:i + L] = np.arange(off[r] + j, off[r] + j + L)
        i += L
    if intra:
        first = {}
        for q in range(N):
            t = int(query[q])
            if ref_row[q] < 0 and t in first:
                ref_row[q] = off[-1] + first[t]
            first.setdefault(t, q)
    return ref_row, np.array(spans, np.int32).reshape(-1, 3), off.astype(np.int32)


@pytest.mark.parametrize("seed", range(8))
@pytest.mark.parametrize("K", [0, 1, 3])
def test_requests_match_brute_force(orc, seed, K):
    rng = np.random.default_rng(500 + seed)
    vocab = [2, 3, 6][seed % 3]
    w = [1, 2, 3, 4][seed % 4]
    reqs = [rng.integers(0, vocab, int(rng.integers(0, 25))).astype(np.int32) for _ in range(int(rng.integers(1, 6)))]
    N = int(rng.integers(1, 50))
    query = rng.integers(0, vocab, N).astype(np.int32)
    if seed % 2 and len(reqs) > 1 and len(reqs[0]) + len(reqs[1]) >= 6:
        # plant the JOIN of two requests: a match across the boundary must be cut at it
        joined = np.concatenate([reqs[0], reqs[1]])
        L = min(N, len(joined))
        query[:L] = joined[:L]
    brr, bsp, off = brute_force_requests(reqs, query, w, K, intra=bool(seed % 2))
    hist = np.concatenate(reqs + [np.zeros(0, np.int32)]).astype(np.int32)
    rr, sp = orc.match_spans_req(hist, off, query, w=w, max_hits=K, intra=bool(seed % 2))
    assert np.array_equal(rr, brr)
    assert np.array_equal(sp, bsp)


@pytest.mark.parametrize("seed", range(10))
def test_live_window_of_the_history(orc, seed):
    """A bounded history: only windows that start at or after `first_live` are candidates.  Against the brute force
    with the same filter, and against the matcher itself on the history cut at `first_live` (the request that
    contains the cut starts there; rows shifted back) -- the cut history must give the same spans."""
    rng = np.random.default_rng(900 + seed)
    vocab = [2, 3, 6][seed % 3]
    w = [1, 2, 3, 4][seed % 4]
    K = [0, 1, 3, 8][seed % 4]
    reqs = [rng.integers(0, vocab, int(rng.integers(0, 25))).astype(np.int32) for _ in range(int(rng.integers(1, 6)))]
    N = int(rng.integers(1, 50))
    query = rng.integers(0, vocab, N).astype(np.int32)
    hist = np.concatenate(reqs + [np.zeros(0, np.int32)]).astype(np.int32)
    off = np.concatenate([[0], np.cumsum([len(r) for r in reqs])]).astype(np.int32)
    for first_live in sorted({0, 1, int(rng.integers(0, hist.size + 1)), int(hist.size // 2), int(hist.size)}):
        brr, bsp, _ = brute_force_requests(reqs, query, w, K, intra=False, first_live=first_live)
        rr, sp = orc.match_spans_req(hist, off, query, w=w, max_hits=K, first_live=first_live)
        assert np.array_equal(rr, brr) and np.array_equal(sp, bsp), (first_live,)
        assert not len(sp) or sp[:, 1].min() >= first_live
        # the same through the cut history
        cut_off = np.unique(np.clip(off, first_live, None)) - first_live
        if cut_off[0] != 0:
            cut_off = np.concatenate([[0], cut_off])
        crr, csp = orc.match_spans_req(hist[first_live:].copy(), cut_off.astype(np.int32), query, w=w, max_hits=K)
        assert np.array_equal(np.where(crr >= 0, crr + first_live, -1), rr)
        assert np.array_equal(csp + np.array([0, first_live, 0], np.int32) if len(csp) else csp, sp)


def test_request_boundaries_cut_matches_and_one_request_is_the_flat_matcher(orc):
    a = np.arange(100, 120, dtype=np.int32)
    b = np.arange(120, 140, dtype=np.int32)
    hist = np.concatenate([a, b])
    query = np.arange(110, 130, dtype=np.int32)          # straddles the boundary at 120
    rr_flat, sp_flat = orc.match_spans(hist, query, w=4)
    assert sp_flat.tolist() == [[0, 10, 20]]
    rr, sp = orc.match_spans_req(hist, [0, 20, 40], query, w=4)
    assert sp.tolist() == [[0, 10, 10], [10, 20, 10]]    # cut at the end of the first request
    assert np.array_equal(rr, rr_flat)                   # the rows happen to be the same; the spans are not
    # a window that straddles the boundary is no candidate at all
    rr, sp = orc.match_spans_req(hist, [0, 20, 40], np.arange(118, 122, dtype=np.int32), w=4)
    assert len(sp) == 0 and np.all(rr == -1)
    # one request == the flat form
    rng = np.random.default_rng(9)
    h = rng.integers(0, 4, 300).astype(np.int32)
    q = rng.integers(0, 4, 200).astype(np.int32)
    r1, s1 = orc.match_spans(h, q, w=3, max_hits=2)
    r2, s2 = orc.match_spans_req(h, [0, 300], q, w=3, max_hits=2)
    r3, s3 = orc.match_spans_req(h, None, q, w=3, max_hits=2)
    assert np.array_equal(r1, r2) and np.array_equal(s1, s2) and np.array_equal(r1, r3) and np.array_equal(s1, s3)


def test_intra_sequence_references_point_at_first_occurrences_and_never_chain(orc):
    hist = np.arange(1000, 1040, dtype=np.int32)
    query = np.array([7, 8, 7, 9, 8, 7, 1000, 1001, 1002, 1003, 7, 1001], np.int32)
    rr, sp = orc.match_spans_req(hist, None, query, w=4, intra=True)
    n = hist.size
    #           7   8   7      9   8      7      span of four            7      1001 (first seen inside the span)
    want = [-1, -1, n + 0, -1, n + 1, n + 0, 0, 1, 2, 3, n + 0, n + 7]
    assert rr.tolist() == want and sp.tolist() == [[6, 0, 4]]
    intra = rr >= n
    targets = rr[intra] - n
    assert np.all(rr[targets] < n)                        # a referenced position is never itself intra-referenced
    assert np.all(query[targets] == query[intra]) and np.all(targets < np.flatnonzero(intra))
    rr0, _ = orc.match_spans_req(hist, None, query, w=4, intra=False)
    assert np.array_equal(np.where(intra, -1, rr), rr0)
