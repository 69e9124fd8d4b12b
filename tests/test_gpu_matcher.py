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
