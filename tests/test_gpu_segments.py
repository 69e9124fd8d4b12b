"""Eq. 6 over several fitting positions: one coefficient pair per (segment, group), shared outside the records
(needs a B200).  Device fit against the oracle's pooled binary64 fit; coding with the shared words bit-identical."""
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


def device_fit(env, cfg, X, R, rows, seg_off, gain=None, bias=None):
    rac, dev = env.rac, env.dev
    T, d = X.shape
    J = d // cfg.group
    n_seg = len(seg_off) - 1
    so = torch.from_numpy(np.asarray(seg_off, np.int32)).to(dev)
    coef = torch.full((n_seg + 1, J), -3, dtype=torch.int32, device=dev)       # one canary row behind
    seg_of = torch.full((T + 4,), -3, dtype=torch.int32, device=dev)
    nb = rac.rac_fit_segments_workspace_bytes(cfg, T)
    ws = torch.full((nb + 32,), 0x5A, dtype=torch.uint8, device=dev)
    st = torch.zeros(1, dtype=torch.int32, device=dev)
    rac.rac_fit_segments(cfg, X, T, R, 0 if R is None else R.shape[0], rows, gain, bias, so, n_seg, coef, seg_of,
                         ws[:nb], nb, st)
    torch.cuda.synchronize()
    assert int(st.item()) == 0
    assert torch.all(coef[n_seg] == -3) and torch.all(seg_of[T:] == -3) and torch.all(ws[nb:] == 0x5A)
    return coef[:n_seg], seg_of[:T], so


@pytest.mark.parametrize("d,g,T,kw", [
    (1024, 128, 300, dict(bits=4)),
    (4096, 128, 517, dict(bits=4, topk_group=1)),
    (3584, 128, 200, dict(bits=8, qgroup=3584)),
    (96, 32, 41, dict(bits=3, topk_group=2)),
])
def test_segment_fit_and_shared_coefficient_coding_match_oracle(env, d, g, T, kw):
    s, rac, orc, dev, P = env.synth, env.rac, env.orc, env.dev, env.P
    J = d // g
    gen = s.generator(900 + d, dev)
    scale = s.channel_scale(d, 9, dev)
    X = s.activations(T, d, scale, gen)
    R = s.affine_noisy_reference(X, g, gen)
    rows = np.arange(T, dtype=np.int32)
    rows[T // 2: T // 2 + 9] = -1                                        # a run of direct tokens inside a segment
    rows_d = torch.from_numpy(rows).to(dev)
    rng = np.random.default_rng(d)
    cuts = np.sort(rng.choice(np.arange(1, T), size=11, replace=False))
    seg_off = np.concatenate([[0], cuts[:5], [cuts[5], cuts[5]], cuts[6:], [T]]).astype(np.int32)   # one empty segment
    bits = kw["bits"]
    mk = dict(scale_mode=1, qgroup=kw.get("qgroup", 0), topk_group=kw.get("topk_group", 0))
    cfg = rac.CodecCfg(d, g, bits, 0, coef_fmt=1, **mk)
    coef_d, seg_of_d, so_d = device_fit(env, cfg, X, R, rows_d, seg_off)
    Xb, Rb = s.bf16_bits(X), s.bf16_bits(R)

    # ---- the fit: every device word is the oracle's, or a rounding of the exact optimum within the window
    o_coef, dg = orc.fit_segments(d, g, Xb, seg_off, ref_base=Rb, ref_row=rows, diag=True)
    g_coef = coef_d.cpu().numpy().view(np.uint32)
    ga, gb = (g_coef & 0xffff).astype(np.uint16), (g_coef >> 16).astype(np.uint16)
    oa, ob = (o_coef & 0xffff).astype(np.uint16), (o_coef >> 16).astype(np.uint16)
    ma = (ga != oa) & ~(((ga | oa) & 0x7fff) == 0)
    mb = (gb != ob) & ~(((gb | ob) & 0x7fff) == 0)
    cancel = 1e-6 * (np.abs(dg["hbar"]) + np.abs(dg["alpha"] * dg["rbar"]))
    if ma.any():
        P._check_flips("alpha", ga[ma], oa[ma], dg["alpha"][ma], 0.0)
    if mb.any():
        P._check_flips("beta", gb[mb], ob[mb], dg["beta"][mb], cancel[mb])
    print(f"{g_coef.size} words: alpha flips {int(ma.sum())}, beta flips {int(mb.sum())}")
    assert ma.sum() + mb.sum() <= max(3, g_coef.size // 100)
    empty = int(np.flatnonzero(np.diff(seg_off) == 0)[0])
    assert not g_coef[empty].any()
    seg_of = np.repeat(np.arange(len(seg_off) - 1), np.diff(seg_off)).astype(np.int32)
    assert np.array_equal(seg_of_d.cpu().numpy(), seg_of)

    # ---- coding with the device's shared words: bit-identical to the oracle given the same words
    rec = rac.rac_record_bytes(cfg)
    assert rec == orc.record_bytes(d, g, bits, 0, 1, mk["qgroup"], mk["topk_group"], 1)
    assert rec <= rac.rac_record_bytes(rac.CodecCfg(d, g, bits, 0, **mk)) - 4 * J + 15
    pay = torch.full((T * rec + 64,), 0xA5, dtype=torch.uint8, device=dev)
    xh = torch.full((T + 1, d), -7.0, dtype=torch.bfloat16, device=dev)
    st = torch.zeros(1, dtype=torch.int32, device=dev)
    rac.rac_encode_reconstruct_list(cfg, X, T, None, None, R, T, rows_d, None, 0, None, None, None, None, pay, T * rec,
                                    xh[:T], None, 0, st, coef_seg=coef_d, seg_of=seg_of_d)
    torch.cuda.synchronize()
    assert int(st.item()) == 0 and torch.all(pay[T * rec:] == 0xA5) and torch.all(xh[T] == -7.0)
    per_tok = np.ascontiguousarray(g_coef[seg_of])
    o_pay = orc.encode(d, g, bits, 0, Xb, ref_base=Rb, ref_row=rows, forced_coef=per_tok.reshape(-1).copy(), coef_fmt=1,
                       nthreads=orc.max_threads(), **mk)
    g_pay = pay[:T * rec].cpu().numpy()
    if not np.array_equal(g_pay, o_pay):
        bad = np.flatnonzero((g_pay.reshape(T, rec) != o_pay.reshape(T, rec)).any(axis=1))
        off = np.flatnonzero(g_pay.reshape(T, rec)[bad[0]] != o_pay.reshape(T, rec)[bad[0]])
        raise AssertionError(f"{bad.size} records differ; first token {bad[0]}, byte offsets {off[:8].tolist()} of {rec}")
    o_x = orc.reconstruct(d, g, bits, 0, o_pay, T, ref_base=Rb, ref_row=rows, coef_fmt=1, shared_coef=per_tok,
                          nthreads=orc.max_threads(), **mk)
    assert np.array_equal(o_x, s.bf16_bits(xh[:T]))
    xd = torch.empty((T, d), dtype=torch.bfloat16, device=dev)
    rac.rac_decode_reconstruct_list(cfg, pay[:T * rec], T, None, None, R, T, rows_d, None, 0, None, None, None, xd, st,
                                    coef_seg=coef_d, seg_of=seg_of_d)
    torch.cuda.synchronize()
    assert int(st.item()) == 0 and torch.equal(xd, xh[:T])

    # ---- argument checks: shared words and the record format go together
    plain = rac.CodecCfg(d, g, bits, 0, **mk)
    for c, cs in ((plain, coef_d), (cfg, None)):
        with pytest.raises(rac.RacError) as e:
            rac.rac_decode_reconstruct_list(c, pay[:T * rec], T, None, None, R, T, rows_d, None, 0, None, None, None, xd,
                                            st, coef_seg=cs, seg_of=seg_of_d if cs is not None else None)
        assert e.value.code == -1
    with pytest.raises(rac.RacError):
        rac.rac_decode_reconstruct(cfg, pay[:T * rec], T, R, T, rows_d, None, None, None, xd, st)
    assert rac.rac_record_bytes(rac.CodecCfg(d, g, 4, 0, coef_fmt=1)) == (d // 2 + 15) // 16 * 16   # static table: codes only


@pytest.mark.parametrize("d,g,T,bits,k,with_gain", [
    (1024, 128, 300, 4, 0, False),
    (5120, 128, 257, 4, 8, False),
    (4096, 64, 130, 3, 8, True),
    (96, 32, 41, 2, 3, False),
])
def test_shared_coefficients_with_the_static_table(env, d, g, T, bits, k, with_gain):
    """coef_fmt = 1 with scale_mode 0: records are [codes][outlier indices][outlier values]; the step table is
    calibrated on the residuals of the shared fit; everything bit-identical to the oracle given the device's words."""
    s, rac, orc, dev = env.synth, env.rac, env.orc, env.dev
    J = d // g
    gen = s.generator(1300 + d, dev)
    scale = s.channel_scale(d, 13, dev)
    X = s.activations(T, d, scale, gen)
    R = s.affine_noisy_reference(X, g, gen)
    rows = np.arange(T, dtype=np.int32)
    rows[T // 3: T // 3 + 7] = -1
    rows_d = torch.from_numpy(rows).to(dev)
    gain = bias = gb = bb = None
    if with_gain:
        gain = (1.0 + 0.1 * torch.randn(d, generator=gen, device=dev)).to(torch.float16)
        bias = (0.02 * torch.randn(d, generator=gen, device=dev)).to(torch.float16)
        gb, bb = gain.cpu().numpy().view(np.uint16), bias.cpu().numpy().view(np.uint16)
    rng = np.random.default_rng(d + k)
    cuts = np.sort(rng.choice(np.arange(1, T), size=9, replace=False))
    seg_off = np.concatenate([[0], cuts, [T]]).astype(np.int32)
    cfg = rac.CodecCfg(d, g, bits, k, coef_fmt=1)
    rec = rac.rac_record_bytes(cfg)
    assert rec == orc.record_bytes(d, g, bits, k, 0, 0, 0, 1) == (d * bits // 8 + 4 * k + 15) // 16 * 16
    coef_d, seg_of_d, _ = device_fit(env, cfg, X, R, rows_d, seg_off, gain, bias)
    g_coef = coef_d.cpu().numpy().view(np.uint32)
    seg_of = np.repeat(np.arange(len(seg_off) - 1), np.diff(seg_off)).astype(np.int32)
    per_tok = np.ascontiguousarray(g_coef[seg_of])
    Xb, Rb = s.bf16_bits(X), s.bf16_bits(R)

    # ---- step table from the residuals of the shared fit
    step = torch.empty((2, d), dtype=torch.float32, device=dev)
    inv = torch.empty_like(step)
    nb = rac.rac_calibrate_workspace_bytes(cfg)
    ws = torch.empty(nb, dtype=torch.uint8, device=dev)
    st = torch.zeros(1, dtype=torch.int32, device=dev)
    rac.rac_calibrate_steps_shared(cfg, X, T, R, T, rows_d, gain, bias, coef_d, seg_of_d, 3.0, step, inv, ws, nb, st)
    torch.cuda.synchronize()
    assert int(st.item()) == 0
    o_step, o_inv = orc.calibrate(d, g, bits, Xb, ref_base=Rb, ref_row=rows, gain=gb, bias=bb, shared_coef=per_tok)
    gs = step.cpu().numpy()
    ulp = np.spacing(o_step.astype(np.float16)).astype(np.float32)
    assert np.all(np.abs(gs - o_step) <= ulp) and (gs != o_step).mean() < 0.02
    # the residual of a shared fit is wider than that of the token's own fit
    own = orc.calibrate(d, g, bits, Xb, ref_base=Rb, ref_row=rows, gain=gb, bias=bb)[0]
    assert np.median(o_step[0] / own[0]) > 1.0
    for c, cs in ((rac.CodecCfg(d, g, bits, k), coef_d), (cfg, None)):
        with pytest.raises(rac.RacError) as e:
            if cs is None:
                rac.rac_calibrate_steps(c, X, T, R, T, rows_d, gain, bias, 3.0, step.clone(), inv.clone(), ws, nb, st)
            else:
                rac.rac_calibrate_steps_shared(c, X, T, R, T, rows_d, gain, bias, cs, seg_of_d, 3.0, step.clone(),
                                               inv.clone(), ws, nb, st)
        assert e.value.code == -1

    # ---- coding: the device's table and words on both sides
    gi = inv.cpu().numpy()
    pay = torch.full((T * rec + 64,), 0xA5, dtype=torch.uint8, device=dev)
    xh = torch.full((T + 1, d), -7.0, dtype=torch.bfloat16, device=dev)
    nws = rac.rac_encode_workspace_bytes(cfg, T)
    ews = torch.empty(max(nws, 16), dtype=torch.uint8, device=dev)
    rac.rac_encode_reconstruct_list(cfg, X, T, None, None, R, T, rows_d, None, 0, gain, bias, step, inv, pay, T * rec,
                                    xh[:T], ews if nws else None, nws, st, coef_seg=coef_d, seg_of=seg_of_d)
    torch.cuda.synchronize()
    assert int(st.item()) == 0 and torch.all(pay[T * rec:] == 0xA5) and torch.all(xh[T] == -7.0)
    o_pay = orc.encode(d, g, bits, k, Xb, ref_base=Rb, ref_row=rows, gain=gb, bias=bb, step=gs, inv_step=gi,
                       forced_coef=per_tok.reshape(-1).copy(), coef_fmt=1, nthreads=orc.max_threads())
    g_pay = pay[:T * rec].cpu().numpy()
    if not np.array_equal(g_pay, o_pay):
        bad = np.flatnonzero((g_pay.reshape(T, rec) != o_pay.reshape(T, rec)).any(axis=1))
        off = np.flatnonzero(g_pay.reshape(T, rec)[bad[0]] != o_pay.reshape(T, rec)[bad[0]])
        raise AssertionError(f"{bad.size} records differ; first token {bad[0]}, byte offsets {off[:8].tolist()} of {rec}")
    o_x = orc.reconstruct(d, g, bits, k, o_pay, T, ref_base=Rb, ref_row=rows, gain=gb, bias=bb, step=gs, coef_fmt=1,
                          shared_coef=per_tok, nthreads=orc.max_threads())
    assert np.array_equal(o_x, s.bf16_bits(xh[:T]))
    xd = torch.empty((T, d), dtype=torch.bfloat16, device=dev)
    rac.rac_decode_reconstruct_list(cfg, pay[:T * rec], T, None, None, R, T, rows_d, None, 0, gain, bias, step, xd, st,
                                    coef_seg=coef_d, seg_of=seg_of_d)
    torch.cuda.synchronize()
    assert int(st.item()) == 0 and torch.equal(xd, xh[:T])
    # a token list: only those records and rows are written
    lst = torch.from_numpy(np.arange(1, T, 3, dtype=np.int32)).to(dev)
    cnt = torch.tensor([lst.numel()], dtype=torch.int32, device=dev)
    pay2 = torch.full_like(pay, 0x3C)
    rac.rac_encode_reconstruct_list(cfg, X, T, lst, cnt, R, T, rows_d, None, 0, gain, bias, step, inv, pay2, T * rec,
                                    None, ews if nws else None, nws, st, coef_seg=coef_d, seg_of=seg_of_d)
    torch.cuda.synchronize()
    p2, p1 = pay2[:T * rec].view(T, rec), pay[:T * rec].view(T, rec)
    sel = torch.zeros(T, dtype=torch.bool, device=dev)
    sel[lst.long()] = True
    assert int(st.item()) == 0 and torch.equal(p2[sel], p1[sel]) and torch.all(p2[~sel] == 0x3C)
    # the per-token record format and the shared words do not mix
    with pytest.raises(rac.RacError):
        rac.rac_decode_reconstruct(cfg, pay[:T * rec], T, R, T, rows_d, gain, bias, step, xd, st)


def test_one_long_segment_and_single_token_segments(env):
    s, rac, orc, dev = env.synth, env.rac, env.orc, env.dev
    d, g, T = 512, 64, 5000                                              # a whole sequence as one segment
    gen = s.generator(950, dev)
    X = s.activations(T, d, s.channel_scale(d, 10, dev), gen)
    R = (0.9 * X.float() + 0.2 + 0.05 * torch.randn((T, d), generator=gen, device=dev)).to(torch.bfloat16)
    cfg = rac.CodecCfg(d, g, 4, 0, scale_mode=1, coef_fmt=1)
    coef_d, seg_of_d, _ = device_fit(env, cfg, X, R, None, [0, T])
    o_coef, dg = orc.fit_segments(d, g, s.bf16_bits(X), np.array([0, T], np.int32), ref_base=s.bf16_bits(R), diag=True)
    gc = coef_d.cpu().numpy().view(np.uint32)
    a = (gc & 0xffff).astype(np.uint16).view(np.float16).astype(np.float64)
    b = (gc >> 16).astype(np.uint16).view(np.float16).astype(np.float64)
    assert np.all(np.abs(a - dg["alpha"]) <= 1e-3 * np.abs(dg["alpha"]) + 2.0 ** -24)
    assert np.all(np.abs(b - dg["beta"]) <= 1e-3 * np.abs(dg["beta"]) + 1e-3)
    assert (gc != o_coef).sum() <= 2
    assert np.all(np.abs(a - 1 / 0.9) < 0.02)                            # the map that generated the reference
    # every token its own segment: the pooled fit is the per-token fit
    T2 = 64
    seg_off = np.arange(T2 + 1, dtype=np.int32)
    c2, so2, _ = device_fit(env, cfg, X[:T2], R[:T2], None, seg_off)
    o2 = orc.fit_segments(d, g, s.bf16_bits(X[:T2]), seg_off, ref_base=s.bf16_bits(R[:T2]))
    assert (c2.cpu().numpy().view(np.uint32) != o2).sum() <= 3
    assert np.array_equal(so2.cpu().numpy(), np.arange(T2))


def test_spans_become_segments_on_the_device(env):
    s, rac, orc, dev = env.synth, env.rac, env.orc, env.dev
    for H, T, gap, seed in [(20000, 6000, 100, 3), (4000, 5000, 0, 4), (3000, 200, 2000, 5), (50, 40, 5, 6)]:
        wl = s.span_workload(H, T, seed=seed, gap_max=gap)
        htok, qtok = torch.from_numpy(wl.hist).to(dev), torch.from_numpy(wl.query).to(dev)
        nb = rac.rac_match_workspace_bytes(H, T, 8)
        ws = torch.empty(nb, dtype=torch.uint8, device=dev)
        rows = torch.empty(T, dtype=torch.int32, device=dev)
        cap = T // 4 + 1
        spans = torch.zeros((cap, 3), dtype=torch.int32, device=dev)
        n_spans = torch.zeros(1, dtype=torch.int32, device=dev)
        rac.rac_match_spans(htok, H, qtok, T, 4, 8, rows, spans, n_spans, ws, nb)
        max_seg = 2 * cap + 1
        seg_off = torch.full((max_seg + 3,), -9, dtype=torch.int32, device=dev)
        n_seg = torch.full((1,), -9, dtype=torch.int32, device=dev)
        rac.rac_spans_to_segments(spans, n_spans, T, max_seg, seg_off, n_seg)
        torch.cuda.synchronize()
        ns = int(n_spans.item())
        want = orc.segments_from_spans(spans[:ns].cpu().numpy(), T)
        got_n = int(n_seg.item())
        assert got_n == len(want) - 1
        assert np.array_equal(seg_off[:got_n + 1].cpu().numpy(), want)
        assert torch.all(seg_off[got_n + 1:max_seg + 1] == T) and torch.all(seg_off[max_seg + 1:] == -9)
        # every segment is a whole span or a whole gap
        r = rows.cpu().numpy()
        for a, b in zip(want[:-1], want[1:]):
            assert (r[a:b] >= 0).all() or (r[a:b] < 0).all()
    # and straight into the fit, without reading the count back: the surplus segments are empty
    d, g = 256, 64
    gen = s.generator(77, dev)
    Hs = s.activations(H, d, s.channel_scale(d, 7, dev), gen)
    X = s.affine_noisy_target(Hs, rows, g, gen, s.channel_scale(d, 7, dev))
    cfg = rac.CodecCfg(d, g, 4, 0, scale_mode=1, coef_fmt=1)
    coef = torch.full((max_seg, d // g), -1, dtype=torch.int32, device=dev)
    seg_of = torch.empty(T, dtype=torch.int32, device=dev)
    nbf = rac.rac_fit_segments_workspace_bytes(cfg, T)
    wsf = torch.empty(nbf, dtype=torch.uint8, device=dev)
    st = torch.zeros(1, dtype=torch.int32, device=dev)
    rac.rac_fit_segments(cfg, X, T, Hs, H, rows, None, None, seg_off, max_seg, coef, seg_of, wsf, nbf, st)
    torch.cuda.synchronize()
    assert int(st.item()) == 0 and not coef[got_n:].any()
    o_coef = orc.fit_segments(d, g, s.bf16_bits(X), want, ref_base=s.bf16_bits(Hs), ref_row=r)
    assert (coef[:got_n].cpu().numpy().view(np.uint32) != o_coef).sum() <= 2
    assert np.array_equal(seg_of.cpu().numpy(), np.repeat(np.arange(got_n), np.diff(want)))
