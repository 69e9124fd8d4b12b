"""Intra-sequence references end to end (Sec. IV-B.1): retrieval over earlier requests, the two coding waves,
sender and receiver, against the CPU oracle (needs a B200)."""
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
    import parity
    rac.load()
    return type("Env", (), dict(orc=oracle, rac=rac, synth=synth, P=parity, dev=torch.device("cuda:0")))


def records(payload_np, rec, toks):
    return np.ascontiguousarray(payload_np.reshape(-1, rec)[toks]).reshape(-1)


@pytest.mark.parametrize("mode", ["static top-8", "Eq. 8 with one outlier per group", "static, 3-bit, no outliers"])
def test_two_wave_round_trip_matches_oracle(env, mode):
    s, rac, orc, dev = env.synth, env.rac, env.orc, env.dev
    d, g, w, K = 1024, 128, 4, 8
    n_hist, T = 3000, 700
    wl = s.span_workload(n_hist, T, seed=21, gap_max=200)
    hist, query = wl.hist.astype(np.int32), wl.query.astype(np.int32)
    bounds = np.array([0, 500, 1100, 1101, 2200, 3000], np.int32)

    # ---- retrieval: index appended request by request, prompt queried with intra-sequence references
    icfg = rac.IndexCfg(n_hist, w, K)
    nb = rac.rac_index_bytes(icfg)
    imem = torch.empty(nb, dtype=torch.uint8, device=dev)
    htok = torch.from_numpy(hist).to(dev)
    qtok = torch.from_numpy(query).to(dev)
    rac.rac_index_reset(icfg, imem, nb)
    for a, b in zip(bounds[:-1], bounds[1:]):
        rac.rac_index_append(icfg, imem, nb, htok, int(a), int(b))
    rows = torch.empty(T, dtype=torch.int32, device=dev)
    n_spans = torch.zeros(1, dtype=torch.int32, device=dev)
    nws = rac.rac_index_query_workspace_bytes(T)
    qws = torch.empty(nws, dtype=torch.uint8, device=dev)
    rac.rac_index_query(icfg, imem, nb, htok, n_hist, qtok, T, True, rows, None, n_spans, qws, nws)
    o_rr, o_sp = orc.match_spans_req(hist, bounds, query, w=w, max_hits=K, intra=True)
    assert np.array_equal(rows.cpu().numpy(), o_rr) and int(n_spans.item()) == len(o_sp)
    w1 = np.flatnonzero(o_rr < n_hist).astype(np.int32)
    w2 = np.flatnonzero(o_rr >= n_hist).astype(np.int32)
    assert len(w2) > 50 and (o_rr[w1] >= 0).sum() > 100        # all three kinds of tokens are present

    # ---- activations: history states, span-matched targets, and repeated tokens close to their first occurrence
    gen = s.generator(77, dev)
    scale = s.channel_scale(d, 77, dev)
    Hs = s.activations(n_hist, d, scale, gen)
    hist_rows = torch.from_numpy(np.where(o_rr < n_hist, o_rr, -1).astype(np.int32)).to(dev)
    X = s.affine_noisy_target(Hs, hist_rows, g, gen, scale)
    first = torch.from_numpy((o_rr[w2] - n_hist).astype(np.int64)).to(dev)
    X[torch.from_numpy(w2.astype(np.int64)).to(dev)] = (
        1.1 * X[first].float() + 0.05 * torch.randn((len(w2), d), generator=gen, device=dev)).to(torch.bfloat16)

    if mode == "static top-8":
        cfg, bits, k, mk = rac.CodecCfg(d, g, 4, 8), 4, 8, {}
    elif mode == "static, 3-bit, no outliers":
        cfg, bits, k, mk = rac.CodecCfg(d, g, 3, 0), 3, 0, {}
    else:
        cfg, bits, k, mk = rac.CodecCfg(d, g, 4, 0, scale_mode=1, topk_group=1), 4, 0, dict(scale_mode=1, topk_group=1)
    Xb, Hb = s.bf16_bits(X), s.bf16_bits(Hs)
    step = inv = step_d = inv_d = None
    if cfg.scale_mode == 0:
        step, inv = orc.calibrate(d, g, bits, Xb, ref_base=Hb, ref_row=hist_rows.cpu().numpy())
        step_d, inv_d = env.P.to_dev(step, dev), env.P.to_dev(inv, dev)
    rec = rac.rac_record_bytes(cfg)

    # ---- sender: split, wave 1, wave 2
    wave1 = torch.full((T,), -9, dtype=torch.int32, device=dev)
    wave2 = torch.full((T,), -9, dtype=torch.int32, device=dev)
    cnt = torch.zeros(2, dtype=torch.int32, device=dev)
    rac.rac_split_waves(rows, T, n_hist, wave1, wave2, cnt)
    assert cnt.tolist() == [len(w1), len(w2)]
    assert np.array_equal(wave1[:len(w1)].cpu().numpy(), w1) and np.array_equal(wave2[:len(w2)].cpu().numpy(), w2)
    assert torch.all(wave1[len(w1):] == -9) and torch.all(wave2[len(w2):] == -9)
    pay = torch.full((T * rec,), 0xA5, dtype=torch.uint8, device=dev)
    xh = torch.full((T, d), -7.0, dtype=torch.bfloat16, device=dev)
    st = torch.zeros(1, dtype=torch.int32, device=dev)
    ews_n = rac.rac_encode_workspace_bytes(cfg, T)
    ews = torch.empty(max(ews_n, 16), dtype=torch.uint8, device=dev)
    enc = lambda lst, c: rac.rac_encode_reconstruct_list(cfg, X, T, lst, c, Hs, n_hist, rows, xh, T, None, None, step_d,
                                                         inv_d, pay, T * rec, xh, ews if ews_n else None, ews_n, st)
    enc(wave1, cnt[0:1])
    torch.cuda.synchronize()
    pay1 = pay.cpu().numpy().copy()
    w2l = torch.from_numpy(w2.astype(np.int64)).to(dev)
    assert np.all(pay1.reshape(T, rec)[w2] == 0xA5) and torch.all(xh[w2l] == -7.0)      # wave 2 untouched so far
    enc(wave2, cnt[1:2])
    torch.cuda.synchronize()
    assert int(st.item()) == 0
    pay_np = pay.cpu().numpy()
    assert np.array_equal(pay_np.reshape(T, rec)[w1], pay1.reshape(T, rec)[w1])       # wave 1 records stay as they were
    xh_bits = s.bf16_bits(xh)

    # ---- oracle, wave by wave (the second wave's reference rows are the reconstructions both sides agree on)
    rep1 = env.P.compare_encode(cfg, records(pay_np, rec, w1), Xb[w1], Hb, o_rr[w1], None, None, step, inv)
    o_x1 = orc.reconstruct(d, g, bits, k, records(pay_np, rec, w1), len(w1), ref_base=Hb, ref_row=o_rr[w1], step=step, **mk)
    assert np.array_equal(o_x1, xh_bits[w1])
    joint = np.concatenate([Hb, xh_bits])                    # rows n_hist + t = reconstruction of token t
    joint[n_hist + w2] = 0x7fc0                              # NaN where nothing may be read
    rep2 = env.P.compare_encode(cfg, records(pay_np, rec, w2), Xb[w2], joint, o_rr[w2], None, None, step, inv)
    o_x2 = orc.reconstruct(d, g, bits, k, records(pay_np, rec, w2), len(w2), ref_base=joint, ref_row=o_rr[w2], step=step, **mk)
    assert np.array_equal(o_x2, xh_bits[w2])
    print(rep1, rep2)
    # the intra-sequence reference pays: those tokens are coded with a slope, not directly
    coef2 = orc.split_payload(records(pay_np, rec, w2), len(w2), d, g, bits, k, cfg.scale_mode, 0, cfg.topk_group)[0]
    assert np.mean((coef2 & 0x7fff) != 0) > 0.95

    # ---- receiver: the same two waves from the payload alone
    xd = torch.full((T, d), 3.0, dtype=torch.bfloat16, device=dev)
    dec = lambda lst, c: rac.rac_decode_reconstruct_list(cfg, pay, T, lst, c, Hs, n_hist, rows, xd, T, None, None,
                                                         step_d, xd, st)
    dec(wave1, cnt[0:1])
    dec(wave2, cnt[1:2])
    torch.cuda.synchronize()
    assert int(st.item()) == 0 and torch.equal(xd, xh)


def test_list_argument_checks_and_bad_entries(env):
    s, rac, dev = env.synth, env.rac, env.dev
    d, g, T = 256, 64, 20
    X = s.activations(T, d, s.channel_scale(d, 3, dev), s.generator(3, dev))
    cfg = rac.CodecCfg(d, g, 4, 0, scale_mode=1)
    rec = rac.rac_record_bytes(cfg)
    pay = torch.zeros(T * rec, dtype=torch.uint8, device=dev)
    xh = torch.zeros_like(X)
    st = torch.zeros(1, dtype=torch.int32, device=dev)
    lst = torch.tensor([3, -5, 99, 7], dtype=torch.int32, device=dev)      # two entries outside [0, T): clamped
    cnt = torch.tensor([4], dtype=torch.int32, device=dev)
    rows = torch.full((T,), -1, dtype=torch.int32, device=dev)
    rows[7] = 50                                                            # beyond both buffers: flagged, coded directly
    rac.rac_encode_reconstruct_list(cfg, X, T, lst, cnt, None, 0, rows, xh, T, None, None, None, None, pay, T * rec, xh,
                                    None, 0, st)
    torch.cuda.synchronize()
    assert int(st.item()) == rac.STATUS_REF_RANGE
    touched = (pay.view(T, rec) != 0).any(dim=1).nonzero().flatten().tolist()
    assert touched == [0, 3, 7, 19]
    with pytest.raises(rac.RacError) as e:
        rac.rac_encode_reconstruct_list(cfg, X, T, lst, None, None, 0, rows, xh, T, None, None, None, None, pay, T * rec,
                                        xh, None, 0, st)
    assert e.value.code == -1
    with pytest.raises(rac.RacError) as e:
        rac.rac_encode_reconstruct_list(cfg, X, T, None, None, None, 0, rows, None, 5, None, None, None, None, pay,
                                        T * rec, xh, None, 0, st)
    assert e.value.code == -1
    # a count above T is cut to T; an empty list does nothing
    cnt[0] = 0
    before = pay.clone()
    rac.rac_encode_reconstruct_list(cfg, X, T, lst, cnt, None, 0, rows, None, 0, None, None, None, None, pay, T * rec, xh,
                                    None, 0, st)
    torch.cuda.synchronize()
    assert torch.equal(pay, before)


def test_random_two_wave_cases(env):
    """300 seeded random cases of the two-wave protocol with hand-made row lists: directly coded tokens, history
    rows and references to first-wave tokens of the same prompt in random mix (no chains), both quantisers, widths
    from 64 to 5120, references uncorrelated with the tokens (tiny slopes)."""
    s, rac, orc, dev, P = env.synth, env.rac, env.orc, env.dev, env.P
    master = np.random.default_rng(9090)
    done = 0
    while done < 300:
        rng = np.random.default_rng(int(master.integers(1 << 40)))
        d, g = int(rng.choice([64, 256, 1024, 2080, 4096, 5120])), int(rng.choice([32, 64, 128, 256]))
        if d % g:
            continue
        if rng.random() < 0.5:
            bits, kg, k = int(rng.choice([2, 3, 4, 8])), int(rng.choice([0, 1, 2])), 0
            cfg, mk = rac.CodecCfg(d, g, bits, 0, scale_mode=1, topk_group=kg), dict(scale_mode=1, topk_group=kg)
        else:
            bits, k = int(rng.choice([2, 3, 4])), int(rng.choice([0, 3, 8]))
            cfg, mk = rac.CodecCfg(d, g, bits, k), {}
        if rac.rac_record_bytes(cfg) == 0:
            continue
        done += 1
        n_hist, T = int(rng.integers(1, 300)), int(rng.integers(1, 250))
        gen = s.generator(int(rng.integers(1 << 30)), dev)
        scale = s.channel_scale(d, 5, dev)
        Hs, X = s.activations(n_hist, d, scale, gen), s.activations(T, d, scale, gen)
        rows = np.full(T, -1, np.int64)
        kind = rng.random(T)
        rows[kind < 0.4] = rng.integers(0, n_hist, int((kind < 0.4).sum()))
        stay = np.flatnonzero(kind <= 0.75)                      # tokens of the first wave
        for t in np.flatnonzero(kind > 0.75):
            cand = stay[stay < t]
            if cand.size:
                rows[t] = n_hist + int(rng.choice(cand))
        rows = rows.astype(np.int32)
        w1, w2 = np.flatnonzero(rows < n_hist).astype(np.int32), np.flatnonzero(rows >= n_hist).astype(np.int32)
        rows_d = torch.from_numpy(rows).to(dev)
        Xb, Hb = s.bf16_bits(X), s.bf16_bits(Hs)
        step = inv = step_d = inv_d = None
        if cfg.scale_mode == 0:
            step, inv = orc.calibrate(d, g, bits, Xb, ref_base=Hb, ref_row=np.where(rows < n_hist, rows, -1).astype(np.int32))
            step_d, inv_d = P.to_dev(step, dev), P.to_dev(inv, dev)
        rec = rac.rac_record_bytes(cfg)
        wave1 = torch.full((T,), -9, dtype=torch.int32, device=dev)
        wave2 = torch.full((T,), -9, dtype=torch.int32, device=dev)
        cnt = torch.zeros(2, dtype=torch.int32, device=dev)
        rac.rac_split_waves(rows_d, T, n_hist, wave1, wave2, cnt)
        assert cnt.tolist() == [len(w1), len(w2)]
        assert np.array_equal(wave1[:len(w1)].cpu().numpy(), w1) and np.array_equal(wave2[:len(w2)].cpu().numpy(), w2)
        pay = torch.full((T * rec,), 0xA5, dtype=torch.uint8, device=dev)
        xh = torch.full((T, d), -7.0, dtype=torch.bfloat16, device=dev)
        st = torch.zeros(1, dtype=torch.int32, device=dev)
        nws = rac.rac_encode_workspace_bytes(cfg, T)
        ews = torch.empty(max(nws, 16), dtype=torch.uint8, device=dev)
        for lst, c in ((wave1, cnt[0:1]), (wave2, cnt[1:2])):
            rac.rac_encode_reconstruct_list(cfg, X, T, lst, c, Hs, n_hist, rows_d, xh, T, None, None, step_d, inv_d, pay,
                                            T * rec, xh, ews if nws else None, nws, st)
        torch.cuda.synchronize()
        what = f"{cfg!r} T={T} n_hist={n_hist}"
        assert int(st.item()) == 0, what
        pay_np, xh_bits = pay.cpu().numpy(), s.bf16_bits(xh)
        try:
            if len(w1):
                P.compare_encode(cfg, records(pay_np, rec, w1), Xb[w1], Hb, rows[w1], None, None, step, inv)
                o1 = orc.reconstruct(d, g, bits, k, records(pay_np, rec, w1), len(w1), ref_base=Hb, ref_row=rows[w1], step=step, **mk)
                assert np.array_equal(o1, xh_bits[w1]), "first-wave reconstruction"
            if len(w2):
                joint = np.concatenate([Hb, xh_bits])
                joint[n_hist + w2] = 0x7fc0                      # NaN where nothing may be read
                P.compare_encode(cfg, records(pay_np, rec, w2), Xb[w2], joint, rows[w2], None, None, step, inv)
                o2 = orc.reconstruct(d, g, bits, k, records(pay_np, rec, w2), len(w2), ref_base=joint, ref_row=rows[w2], step=step, **mk)
                assert np.array_equal(o2, xh_bits[w2]), "second-wave reconstruction"
        except AssertionError as e:
            raise AssertionError(f"{what}: {e}") from e
        xd = torch.full((T, d), 3.0, dtype=torch.bfloat16, device=dev)
        for lst, c in ((wave1, cnt[0:1]), (wave2, cnt[1:2])):
            rac.rac_decode_reconstruct_list(cfg, pay, T, lst, c, Hs, n_hist, rows_d, xd, T, None, None, step_d, xd, st)
        torch.cuda.synchronize()
        assert int(st.item()) == 0 and torch.equal(xd, xh), what
