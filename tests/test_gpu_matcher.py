"""CUDA span matcher vs CPU oracle, through the C ABI (needs a B200).  Everything is integer work:
the comparison is bit-exact."""
import numpy as np
import pytest
import torch

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def env():
    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    import oracle
    from paper_2608_04991_b200 import binding as rac
    from paper_2608_04991_b200 import synth
    rac.load()
    return type("Env", (), dict(orc=oracle, rac=rac, synth=synth, dev=torch.device("cuda:0")))


def gpu_match(env, hist, query, w, K, want_spans=True):
    rac, dev = env.rac, env.dev
    h = torch.from_numpy(np.ascontiguousarray(hist, np.int32)).to(dev)
    q = torch.from_numpy(np.ascontiguousarray(query, np.int32)).to(dev)
    N = q.numel()
    nb = rac.rac_match_workspace_bytes(h.numel(), N, K)
    ws = torch.full((nb + 32,), 0x5A, dtype=torch.uint8, device=dev)  # dirty workspace: nothing may be assumed zero
    rows = torch.full((N + 8,), 12345, dtype=torch.int32, device=dev)
    cap = N // w + 1
    spans = torch.full((cap + 2, 3), 777, dtype=torch.int32, device=dev)
    n_spans = torch.full((1,), -5, dtype=torch.int32, device=dev)
    rac.rac_match_spans(h if h.numel() else None, h.numel(), q if N else None, N, w, K, rows[:N] if N else None,
                        spans[:cap] if want_spans else None, n_spans, ws[:nb], nb)
    torch.cuda.synchronize()
    assert torch.all(rows[N:] == 12345) and torch.all(spans[cap:] == 777) and torch.all(ws[nb:] == 0x5A)
    ns = int(n_spans.item())
    return rows[:N].cpu().numpy(), spans[:ns].cpu().numpy(), ns


@pytest.mark.parametrize("seed", range(8))
def test_tiny_random_inputs(env, seed):
    rng = np.random.default_rng(200 + seed)
    vocab = [2, 3, 5, 50][seed % 4]
    w = [1, 2, 3, 4, 6][seed % 5]
    K = [1, 2, 8, 16][seed % 4]
    H, N = int(rng.integers(5, 400)), int(rng.integers(1, 300))
    hist = rng.integers(0, vocab, H).astype(np.int32)
    query = rng.integers(0, vocab, N).astype(np.int32)
    if seed % 2:
        L = min(N, H, 40)
        query[N - L:] = hist[:L]
    rr, sp, ns = gpu_match(env, hist, query, w, K)
    o_rr, o_sp = env.orc.match_spans(hist, query, w, K)
    assert np.array_equal(rr, o_rr) and np.array_equal(sp, o_sp)


def test_degenerate_sizes_and_adversarial_tokens(env):
    orc = env.orc
    cases = [
        (np.arange(20), np.arange(3), 4, 8),                 # query shorter than w
        (np.arange(3), np.arange(10), 4, 8),                 # history shorter than w
        (np.arange(0), np.arange(10), 4, 8),                 # empty history
        (np.ones(300), np.ones(200), 4, 8),                  # one window everywhere
        (np.ones(300), np.ones(200), 4, 1),
        (np.arange(500) % 7, np.arange(333) % 7, 4, 8),      # periodic: long overlapping matches
        (np.arange(64), np.arange(64), 4, 8),                # query == history
    ]
    for hist, query, w, K in cases:
        hist, query = hist.astype(np.int32), query.astype(np.int32)
        rr, sp, ns = gpu_match(env, hist, query, w, K)
        o_rr, o_sp = orc.match_spans(hist, query, w, K)
        assert np.array_equal(rr, o_rr) and np.array_equal(sp, o_sp), (len(hist), len(query), w, K)
    # empty query: only n_spans is written
    rr, sp, ns = gpu_match(env, np.arange(50, dtype=np.int32), np.arange(0, dtype=np.int32), 4, 8)
    assert ns == 0 and rr.size == 0


def test_frequent_window_cap(env):
    rng = np.random.default_rng(3)
    gram = np.array([1, 2, 3, 4], np.int32)
    tail = np.array([50, 51, 52, 53, 54], np.int32)
    parts = [gram, tail, rng.integers(100, 10000, 5).astype(np.int32)]
    for _ in range(11):
        parts += [gram, rng.integers(100, 10000, 6).astype(np.int32)]
    hist = np.concatenate(parts)
    query = np.concatenate([gram, tail])
    for K in (1, 8, 12, 16):
        rr, sp, _ = gpu_match(env, hist, query, 4, K)
        o_rr, o_sp = env.orc.match_spans(hist, query, 4, K)
        assert np.array_equal(sp, o_sp) and np.array_equal(rr, o_rr)
    assert gpu_match(env, hist, query, 4, 12)[1].tolist() == [[0, 0, 9]]


def test_unlimited_hits(env):
    """max_hits = 0: every occurrence of a window is a candidate (Sec. IV-B.1's longest exact match without the
    bucket cap).  Tiny random inputs, the adversarial token streams (one token everywhere: every position of the
    history is a candidate of every query position), a window that occurs more often than any cap, and the two
    workloads against the oracle's K = 0; at the long-context size the span list differs from the K = 8 one."""
    orc = env.orc
    rng = np.random.default_rng(77)
    for trial in range(12):
        vocab = [2, 3, 5, 50][trial % 4]
        w = [1, 2, 3, 4, 6][trial % 5]
        H, N = int(rng.integers(5, 400)), int(rng.integers(1, 300))
        hist = rng.integers(0, vocab, H).astype(np.int32)
        query = rng.integers(0, vocab, N).astype(np.int32)
        rr, sp, _ = gpu_match(env, hist, query, w, 0)
        o_rr, o_sp = orc.match_spans(hist, query, w, 0)
        assert np.array_equal(rr, o_rr) and np.array_equal(sp, o_sp), (trial, H, N, w)
    for hist, query, w in [(np.ones(700), np.ones(500), 4), (np.arange(500) % 7, np.arange(333) % 7, 4),
                           (np.arange(64), np.arange(64), 4), (np.arange(3), np.arange(10), 4), (np.arange(0), np.arange(10), 4)]:
        hist, query = hist.astype(np.int32), query.astype(np.int32)
        rr, sp, _ = gpu_match(env, hist, query, w, 0)
        o_rr, o_sp = orc.match_spans(hist, query, w, 0)
        assert np.array_equal(rr, o_rr) and np.array_equal(sp, o_sp), (len(hist), len(query))
    # a window with 20 occurrences, the OLDEST of which has the longest continuation: only K = 0 finds it
    gram = np.array([1, 2, 3, 4], np.int32)
    tail = np.array([50, 51, 52, 53, 54], np.int32)
    parts = [gram, tail]
    for _ in range(19):
        parts += [rng.integers(100, 10000, 6).astype(np.int32), gram]
    hist = np.concatenate(parts)
    query = np.concatenate([gram, tail])
    assert gpu_match(env, hist, query, 4, 0)[1].tolist() == [[0, 0, 9]]
    assert gpu_match(env, hist, query, 4, 16)[1].tolist() != [[0, 0, 9]]
    # the workloads
    for n_hist, n_query, gap, seed in [(32768, 2048, 176, 1), (131072, 131072, 112, 4)]:
        wl = env.synth.span_workload(n_hist, n_query, seed=seed, gap_max=gap)
        rr, sp, ns = gpu_match(env, wl.hist, wl.query, 4, 0)
        o_rr, o_sp = orc.match_spans(wl.hist, wl.query, 4, 0)
        assert ns == len(o_sp) and np.array_equal(sp, o_sp) and np.array_equal(rr, o_rr)
        o8_rr, o8_sp = orc.match_spans(wl.hist, wl.query, 4, 8)
        print(f"{n_hist}/{n_query}: {ns} spans without a cap, {len(o8_sp)} with 8 hits, rows differ at "
              f"{int((o8_rr != o_rr).sum())} positions")


@pytest.mark.parametrize("n_hist,n_query,gap,seed", [(32768, 2048, 176, 1), (131072, 131072, 112, 4), (5000, 70001, 60, 9)])
def test_workload_sizes(env, n_hist, n_query, gap, seed):
    wl = env.synth.span_workload(n_hist, n_query, seed=seed, gap_max=gap)
    rr, sp, ns = gpu_match(env, wl.hist, wl.query, 4, 8)
    o_rr, o_sp = env.orc.match_spans(wl.hist, wl.query, 4, 8)
    assert ns == len(o_sp)
    assert np.array_equal(sp, o_sp)
    assert np.array_equal(rr, o_rr)
    # spans may be omitted
    rr2, _, ns2 = gpu_match(env, wl.hist, wl.query, 4, 8, want_spans=False)
    assert ns2 == ns and np.array_equal(rr2, rr)
    cov = (rr >= 0).mean()
    print(f"{ns} spans, coverage {cov:.3f} (planted {wl.planted_coverage:.3f})")


def test_spans_to_rows(env):
    rac, dev = env.rac, env.dev
    wl = env.synth.span_workload(8192, 4096, seed=5)
    rr, sp, ns = gpu_match(env, wl.hist, wl.query, 4, 8)
    spans = torch.from_numpy(sp).to(dev)
    n = torch.tensor([ns], dtype=torch.int32, device=dev)
    out = torch.full((4096,), 99, dtype=torch.int32, device=dev)
    rac.rac_spans_to_rows(spans, n, 4096, out)
    torch.cuda.synchronize()
    assert np.array_equal(out.cpu().numpy(), rr)
    # clipping of a span that runs past the query
    spans = torch.tensor([[4090, 10, 20]], dtype=torch.int32, device=dev)
    n = torch.tensor([1], dtype=torch.int32, device=dev)
    rac.rac_spans_to_rows(spans, n, 4096, out)
    torch.cuda.synchronize()
    o = out.cpu().numpy()
    assert np.all(o[:4090] == -1) and o[4090:].tolist() == list(range(10, 16))


# --------------------------------------------------------------------------- persistent index over earlier requests
class GpuIndex:
    """Drives rac_index_* the way a serving loop would: one append per finished request, one query per prompt."""

    def __init__(self, env, capacity, w, K):
        self.env, self.rac, self.dev = env, env.rac, env.dev
        self.cfg = env.rac.IndexCfg(capacity, w, K)
        self.nb = env.rac.rac_index_bytes(self.cfg)
        self.mem = torch.full((self.nb + 32,), 0x5A, dtype=torch.uint8, device=env.dev)   # dirty, canary behind
        self.hist = torch.zeros(capacity, dtype=torch.int32, device=env.dev)
        self.n = 0
        self.w = w
        env.rac.rac_index_reset(self.cfg, self.mem[:self.nb], self.nb)

    def append(self, req):
        req = np.ascontiguousarray(req, np.int32)
        if req.size:
            self.hist[self.n:self.n + req.size] = torch.from_numpy(req).to(self.dev)
        self.rac.rac_index_append(self.cfg, self.mem[:self.nb], self.nb, self.hist, self.n, self.n + req.size)
        self.n += req.size

    def query(self, query, intra=False, first_live=None):
        q = torch.from_numpy(np.ascontiguousarray(query, np.int32)).to(self.dev)
        N = q.numel()
        nws = self.rac.rac_index_query_workspace_bytes(N)
        ws = torch.full((nws + 32,), 0xA5, dtype=torch.uint8, device=self.dev)
        rows = torch.full((N + 8,), 12345, dtype=torch.int32, device=self.dev)
        cap = N // self.w + 1
        spans = torch.full((cap + 2, 3), 777, dtype=torch.int32, device=self.dev)
        n_spans = torch.full((1,), -5, dtype=torch.int32, device=self.dev)
        if first_live is None:
            self.rac.rac_index_query(self.cfg, self.mem[:self.nb], self.nb, self.hist, self.n, q if N else None, N, intra,
                                     rows[:N] if N else None, spans[:cap], n_spans, ws[:nws], nws)
        else:
            self.rac.rac_index_query_live(self.cfg, self.mem[:self.nb], self.nb, self.hist, self.n, first_live,
                                          q if N else None, N, intra, rows[:N] if N else None, spans[:cap], n_spans,
                                          ws[:nws], nws)
        torch.cuda.synchronize()
        assert torch.all(rows[N:] == 12345) and torch.all(spans[cap:] == 777) and torch.all(ws[nws:] == 0xA5)
        assert torch.all(self.mem[self.nb:] == 0x5A)
        ns = int(n_spans.item())
        return rows[:N].cpu().numpy(), spans[:ns].cpu().numpy()


@pytest.mark.parametrize("seed", range(8))
def test_index_appended_request_by_request_matches_oracle(env, seed):
    rng = np.random.default_rng(700 + seed)
    vocab = [2, 3, 6, 40][seed % 4]
    w = [1, 2, 3, 4, 5][seed % 5]
    K = [1, 2, 8, 0][seed % 4]          # 0: no cap on the hits (chains instead of K-lists)
    ix = GpuIndex(env, 4096, w, K)
    reqs, off = [], [0]
    for step in range(7):
        # a prompt is matched against what has been appended so far, then becomes a request itself
        N = int(rng.integers(1, 300))
        query = rng.integers(0, vocab, N).astype(np.int32)
        if reqs and step % 2:
            src = np.concatenate(reqs)                  # copy across request joins: matches must be cut there
            L = min(N, src.size, 60)
            a = int(rng.integers(0, src.size - L + 1))
            query[:L] = src[a:a + L]
        hist = np.concatenate(reqs) if reqs else np.zeros(0, np.int32)
        for intra in (False, True):
            rr, sp = ix.query(query, intra=intra)
            o_rr, o_sp = env.orc.match_spans_req(hist, np.array(off, np.int32), query, w=w, max_hits=K, intra=intra)
            assert np.array_equal(sp, o_sp), f"step {step}"
            assert np.array_equal(rr, o_rr), f"step {step} intra {intra}"
        ix.append(query)
        reqs.append(query)
        off.append(off[-1] + N)
    # short and empty requests add no window but keep the bookkeeping right
    ix.append(np.zeros(0, np.int32))
    ix.append(np.arange(max(w - 1, 0), dtype=np.int32))
    reqs.append(np.arange(max(w - 1, 0), dtype=np.int32))
    off += [off[-1], off[-1] + max(w - 1, 0)]
    query = np.concatenate(reqs)[-50:]
    rr, sp = ix.query(query)
    o_rr, o_sp = env.orc.match_spans_req(np.concatenate(reqs), np.array(off, np.int32), query, w=w, max_hits=K)
    assert np.array_equal(sp, o_sp) and np.array_equal(rr, o_rr)


@pytest.mark.parametrize("seed", range(6))
def test_index_live_window(env, seed):
    """A bounded history: old requests are dropped by raising `first_live`; nothing in the index changes.  After
    every append the prompt is matched with the cut at several places (request boundaries and inside requests)
    and compared with the oracle's live-window matcher; the cut at 0 equals the plain query."""
    rng = np.random.default_rng(1300 + seed)
    vocab = [2, 3, 6, 40][seed % 4]
    w = [1, 2, 3, 4][seed % 4]
    K = [1, 0, 8, 16][seed % 4]
    ix = GpuIndex(env, 4096, w, K)
    reqs, off = [], [0]
    for step in range(6):
        req = rng.integers(0, vocab, int(rng.integers(0, 200))).astype(np.int32)
        ix.append(req)
        reqs.append(req)
        off.append(off[-1] + req.size)
        hist = np.concatenate(reqs)
        N = int(rng.integers(1, 250))
        query = rng.integers(0, vocab, N).astype(np.int32)
        if hist.size >= 8:
            L = min(N, hist.size, 50)
            a = int(rng.integers(0, hist.size - L + 1))
            query[:L] = hist[a:a + L]
        cuts = sorted({0, off[len(off) // 2], int(rng.integers(0, hist.size + 1)), hist.size})
        for cut in cuts:
            for intra in (False, True):
                rr, sp = ix.query(query, intra=intra, first_live=cut)
                o_rr, o_sp = env.orc.match_spans_req(hist, np.array(off, np.int32), query, w=w, max_hits=K, intra=intra,
                                                     first_live=cut)
                assert np.array_equal(sp, o_sp) and np.array_equal(rr, o_rr), (step, cut, intra)
        rr0, sp0 = ix.query(query)
        rr1, sp1 = ix.query(query, first_live=0)
        assert np.array_equal(rr0, rr1) and np.array_equal(sp0, sp1)
    with pytest.raises(Exception):
        ix.query(query, first_live=ix.n + 1)


def test_index_one_request_equals_the_one_shot_matcher_and_reset(env):
    s = env.synth
    wl = s.span_workload(20000, 3000, seed=5, gap_max=120)
    hist, query = wl.hist.astype(np.int32), wl.query.astype(np.int32)
    ix = GpuIndex(env, 20000, 4, 8)
    ix.append(hist)
    rr, sp = ix.query(query)
    rr1, sp1, _ = gpu_match(env, hist, query, 4, 8)
    assert np.array_equal(rr, rr1) and np.array_equal(sp, sp1) and len(sp) > 3
    # the same history in 50 requests: only matches that cross a boundary change
    ix2 = GpuIndex(env, 20000, 4, 8)
    bounds = np.linspace(0, 20000, 51).astype(np.int32)
    for a, b in zip(bounds[:-1], bounds[1:]):
        ix2.append(hist[a:b])
    rr2, sp2 = ix2.query(query, intra=True)
    o_rr, o_sp = env.orc.match_spans_req(hist, bounds, query, w=4, max_hits=8, intra=True)
    assert np.array_equal(rr2, o_rr) and np.array_equal(sp2, o_sp)
    assert (o_rr >= 20000).sum() > 0
    # reset: nothing matches any more
    env.rac.rac_index_reset(ix2.cfg, ix2.mem[:ix2.nb], ix2.nb)
    ix2.n = 0
    rr3, sp3 = ix2.query(query)
    assert len(sp3) == 0 and np.all(rr3 == -1)


def test_index_argument_checks(env):
    rac = env.rac
    assert rac.rac_index_bytes(rac.IndexCfg(0, 4, 8)) == 0
    assert rac.rac_index_bytes(rac.IndexCfg(100, 0, 8)) == 0
    assert rac.rac_index_bytes(rac.IndexCfg(100, 4, 17)) == 0 and rac.rac_index_bytes(rac.IndexCfg(100, 4, -1)) == 0
    assert 0 < rac.rac_index_bytes(rac.IndexCfg(100, 4, 0)) <= rac.rac_index_bytes(rac.IndexCfg(100, 4, 1))
    cfg = rac.IndexCfg(100, 4, 8)
    nb = rac.rac_index_bytes(cfg)
    mem = torch.zeros(nb, dtype=torch.uint8, device=env.dev)
    tok = torch.zeros(200, dtype=torch.int32, device=env.dev)
    rac.rac_index_reset(cfg, mem, nb)
    for fn, args, code in [
        (rac.rac_index_reset, (cfg, mem, nb - 16), -3),
        (rac.rac_index_append, (cfg, mem, nb, tok, 0, 101), -3),        # beyond the capacity
        (rac.rac_index_append, (cfg, mem, nb, tok, 10, 5), -1),
        (rac.rac_index_append, (cfg, mem[1:], nb - 1, tok, 0, 5), -2),
    ]:
        with pytest.raises(rac.RacError) as e:
            fn(*args)
        assert e.value.code == code


def _random_tokens(rng, n, vocab, hist=None):
    q = rng.integers(0, vocab, n).astype(np.int32)
    if hist is not None and hist.size and n:
        for _ in range(int(rng.integers(0, 6))):       # planted copies of history spans
            L = int(rng.integers(1, min(n, hist.size, 300) + 1))
            i, j = int(rng.integers(0, n - L + 1)), int(rng.integers(0, hist.size - L + 1))
            q[i:i + L] = hist[j:j + L]
    if rng.random() < 0.1 and n:
        q[:] = q[0]                                     # one token repeated
    return q


def test_random_sweep_one_shot_and_index(env):
    """2000 seeded random cases, half through the one-shot matcher and half through the persistent index with
    random request boundaries (empty and one-token requests included) and random use of intra-sequence references:
    vocabularies from 1 to 32000 ids, windows 1..32, 1..16 hits, sizes from 0 to a few thousand."""
    rac, orc, dev = env.rac, env.orc, env.dev
    master = np.random.default_rng(4711)
    for _ in range(2000):
        rng = np.random.default_rng(int(master.integers(1 << 40)))
        if rng.random() < 0.5:
            vocab = int(rng.choice([1, 2, 3, 7, 50, 1000, 32000]))
            w, K = int(rng.choice([1, 2, 3, 4, 4, 5, 8, 16, 32])), int(rng.choice([1, 2, 3, 8, 8, 16]))
            H = int(rng.choice([0, 1, 3, int(rng.integers(0, 6000))]))
            N = int(rng.choice([0, 1, 2, int(rng.integers(0, 4000))]))
            hist = _random_tokens(rng, H, vocab)
            query = _random_tokens(rng, N, vocab, hist)
            rr, sp, ns = gpu_match(env, hist, query, w, K)
            o_rr, o_sp = orc.match_spans(hist, query, w, K)
            assert ns == len(o_sp) and np.array_equal(rr, o_rr) and np.array_equal(sp, o_sp.reshape(-1, 3)), \
                dict(vocab=vocab, w=w, K=K, H=H, N=N)
            continue
        vocab = int(rng.choice([2, 3, 7, 50, 1000, 32000]))
        w, K = int(rng.choice([1, 2, 3, 4, 4, 5, 8])), int(rng.choice([1, 2, 8, 8, 16]))
        lens = [int(rng.choice([0, 1, 2, 3, int(rng.integers(0, 1500))])) for _ in range(int(rng.integers(1, 9)))]
        H = sum(lens)
        cap = H + int(rng.integers(0, 100)) + 1
        icfg = rac.IndexCfg(cap, w, K)
        nb = rac.rac_index_bytes(icfg)
        imem = torch.full((nb,), 0x5A, dtype=torch.uint8, device=dev)
        htok = torch.zeros(cap, dtype=torch.int32, device=dev)
        rac.rac_index_reset(icfg, imem, nb)
        hist, off = np.zeros(0, np.int32), [0]
        for L in lens:
            req = _random_tokens(rng, L, vocab, hist)
            if L:
                htok[hist.size:hist.size + L] = torch.from_numpy(req).to(dev)
            rac.rac_index_append(icfg, imem, nb, htok, hist.size, hist.size + L)
            hist = np.concatenate([hist, req])
            off.append(hist.size)
        N = int(rng.choice([0, 1, int(rng.integers(0, 3000))]))
        intra = bool(rng.random() < 0.5)
        query = _random_tokens(rng, N, vocab, hist)
        q = torch.from_numpy(query).to(dev)
        rows = torch.full((N + 8,), 12345, dtype=torch.int32, device=dev)
        sp = torch.full((N // w + 3, 3), 777, dtype=torch.int32, device=dev)
        ns = torch.full((1,), -5, dtype=torch.int32, device=dev)
        nws = rac.rac_index_query_workspace_bytes(N)
        ws = torch.full((max(nws, 16),), 0x5A, dtype=torch.uint8, device=dev)
        rac.rac_index_query(icfg, imem, nb, htok, H, q if N else None, N, intra, rows[:N] if N else None,
                            sp[:N // w + 1], ns, ws, nws)
        o_rr, o_sp = orc.match_spans_req(hist, off, query, w, K, intra)
        n = int(ns.item())
        what = dict(vocab=vocab, w=w, K=K, lens=lens, N=N, intra=intra)
        assert n == len(o_sp) and torch.all(rows[N:] == 12345), what
        assert np.array_equal(rows[:N].cpu().numpy(), o_rr) and np.array_equal(sp[:n].cpu().numpy(), o_sp.reshape(-1, 3)), what


def test_two_million_token_history(env):
    """History of 2^21 tokens, prompt of 2^19: sixteen times the benchmark's history; positions need 21 bits, the most
    frequent windows occur hundreds of times (the K cap decides), the chain walk crosses its shared-memory window
    several times.  Whole result against the oracle."""
    s, orc = env.synth, env.orc
    wl = s.span_workload(1 << 21, 1 << 19, seed=5, gap_max=112)
    rr, sp, ns = gpu_match(env, wl.hist, wl.query, 4, 8)
    o_rr, o_sp = orc.match_spans(wl.hist, wl.query, 4, 8)
    assert ns == len(o_sp) > 5000
    assert np.array_equal(rr, o_rr) and np.array_equal(sp, o_sp.reshape(-1, 3))
    assert (rr >= 0).mean() > 0.7
