"""The five benchmark configurations, end to end on the device, against the CPU oracle (needs a B200).

Each test builds the configuration's synthetic workload at its full size, runs the hot path through the C ABI
and applies the parity protocol of `parity.py`: coefficients within tolerance (flips counted), everything else
bit-exact once the coefficients are shared, reconstruction bit-exact.  Closed loops are checked teacher-forced:
at every step both sides start from the DEVICE's previous reconstruction.
"""
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


def device_tables(env, cfg, X, ref_base, ref_row, gain=None, bias=None):
    """Step tables from the device calibration kernel (host copies returned too)."""
    rac, dev = env.rac, env.dev
    step = torch.empty((2, cfg.d), dtype=torch.float32, device=dev)
    inv = torch.empty_like(step)
    nb = rac.rac_calibrate_workspace_bytes(cfg)
    ws = torch.empty(nb, dtype=torch.uint8, device=dev)
    st = torch.zeros(1, dtype=torch.int32, device=dev)
    rac.rac_calibrate_steps(cfg, X, X.shape[0], ref_base, 0 if ref_base is None else ref_base.shape[0], ref_row, gain, bias,
                            3.0, step, inv, ws, nb, st)
    torch.cuda.synchronize()
    assert int(st.item()) == 0
    return step.cpu().numpy(), inv.cpu().numpy()


def test_config0_prefill_uplink_single_sequence(env):
    """T=128, d=4096, group 128, 4-bit, no outliers; clip = 3 sigma from a 1024-token calibration draw."""
    s = env.synth
    d, g, T = 4096, 128, 128
    gen = s.generator(s.BASE_SEED + 0, env.dev)
    scale = s.channel_scale(d, 0, env.dev)
    X = s.activations(T, d, scale, gen)
    R = s.affine_noisy_reference(X, g, gen)
    cal = s.activations(1024, d, scale, gen)
    calr = s.affine_noisy_reference(cal, g, gen)
    step, inv = env.orc.calibrate(d, g, 4, s.bf16_bits(cal), ref_base=s.bf16_bits(calr))
    rep, pay, xr = env.P.round_trip_case(env.rac.CodecCfg(d, g, 4, 0), X, ref_base=R, step=step, inv_step=inv)
    print("config 0:", rep)
    env.P.assert_caps(rep)
    # the residual is coded: error about a step (3 sigma / 7), far below the activations
    err = (xr.float() - X.float()).abs()
    assert err.mean().item() < 0.02 and X.float().abs().mean().item() > 0.5
    # device calibration agrees with the oracle's table to one binary16 step
    dstep, _ = device_tables(env, env.rac.CodecCfg(d, g, 4, 0), cal, calr, None)
    assert np.all(np.abs(dstep - step) <= np.spacing(step.astype(np.float16)).astype(np.float32))


def test_config1_prefill_uplink_with_span_retrieval(env):
    """32768-token history, 2048-token query (Zipf 1.1 / 32000), ~60 % planted coverage, min n-gram 4; history
    state buffer 32768 x 4096; matched rows are the reference, unmatched rows coded directly; 4-bit, top-8."""
    s, rac, orc, dev = env.synth, env.rac, env.orc, env.dev
    d, g, bits, k, H, N = 4096, 128, 4, 8, 32768, 2048
    wl = s.span_workload(H, N, seed=1)
    hist, query = torch.from_numpy(wl.hist).to(dev), torch.from_numpy(wl.query).to(dev)
    nb = rac.rac_match_workspace_bytes(H, N, 8)
    ws = torch.empty(nb, dtype=torch.uint8, device=dev)
    ref_row = torch.empty(N, dtype=torch.int32, device=dev)
    spans = torch.empty((N // 4 + 1, 3), dtype=torch.int32, device=dev)
    n_spans = torch.zeros(1, dtype=torch.int32, device=dev)
    rac.rac_match_spans(hist, H, query, N, 4, 8, ref_row, spans, n_spans, ws, nb)
    torch.cuda.synchronize()
    o_rows, o_spans = orc.match_spans(wl.hist, wl.query, 4, 8)
    assert np.array_equal(ref_row.cpu().numpy(), o_rows)
    assert np.array_equal(spans[: int(n_spans.item())].cpu().numpy(), o_spans)
    cov = float((o_rows >= 0).mean())
    print(f"config 1: {len(o_spans)} spans, coverage {cov:.3f} (planted {wl.planted_coverage:.3f})")
    assert 0.5 < cov < 0.8
    gen = s.generator(s.BASE_SEED + 1, dev)
    scale = s.channel_scale(d, 1, dev)
    Hs = s.activations(H, d, scale, gen)
    X = s.affine_noisy_target(Hs, torch.from_numpy(wl.planted_row), g, gen, scale)
    # the oracle only needs the history rows that are referenced
    need = np.unique(o_rows[o_rows >= 0])
    compact = np.where(o_rows >= 0, np.searchsorted(need, np.maximum(o_rows, 0)), -1).astype(np.int32)
    Hc = Hs[torch.from_numpy(need).to(dev).long()].contiguous()
    cfg = rac.CodecCfg(d, g, bits, k)
    step, inv = orc.calibrate(d, g, bits, s.bf16_bits(X), ref_base=s.bf16_bits(Hc), ref_row=compact)
    assert step[0].all() and step[1].all()
    # device on the full history buffer with the matcher's rows, oracle on the compact copy: same bytes
    step_d, inv_d = env.P.to_dev(step, dev), env.P.to_dev(inv, dev)
    pay, st = env.P.gpu_encode(cfg, X, Hs, ref_row, None, None, step_d, inv_d)
    assert st == 0
    rep = env.P.compare_encode(cfg, pay, s.bf16_bits(X), s.bf16_bits(Hc), compact, None, None, step, inv)
    print("config 1:", rep)
    xh, st = env.P.gpu_decode(cfg, pay, N, Hs, ref_row, None, None, step_d, dev)
    o_x = orc.reconstruct(d, g, bits, k, pay, N, ref_base=s.bf16_bits(Hc), ref_row=compact, step=step)
    assert st == 0 and np.array_equal(o_x, s.bf16_bits(xh))
    coef = orc.split_payload(pay, N, d, g, bits, k)[0]
    assert np.all((coef[o_rows < 0] & 0x7fff) == 0)   # unmatched rows: zero reference, alpha = 0


def test_config2_decode_steps_closed_loop(env):
    """64 sequences x 1 token per step, d=3584, 3-bit, group 128, no outliers, 512 steps.  Reference of step t =
    bf16(gain * x_hat[t-1] + bias) with the sender-side x_hat fed back.  Teacher-forced comparison per step."""
    s, rac, orc, dev = env.synth, env.rac, env.orc, env.dev
    B, d, g, bits, steps = 64, 3584, 128, 3, 512
    cfg = rac.CodecCfg(d, g, bits, 0)
    gen = s.generator(s.BASE_SEED + 2, dev)
    scale = s.channel_scale(d, 2, dev)
    gain, bias = s.predictor_gain_bias(d, 2, dev)
    gb, bb = s.f16_bits(gain), s.f16_bits(bias)
    # open-loop draw across the horizon for the step table (16 steps x 64 sequences)
    state = s.activations(B, d, scale, s.generator(s.BASE_SEED + 102, dev))
    cal_x, cal_r = [], []
    walk_gen = s.generator(s.BASE_SEED + 202, dev)
    for t in range(1, steps + 1):
        nxt = s.random_walk_step(state, walk_gen)
        if t % 32 == 0:
            cal_x.append(nxt)
            cal_r.append(state)
        state = nxt
    cal_x, cal_r = torch.cat(cal_x), torch.cat(cal_r)
    step, inv = orc.calibrate(d, g, bits, s.bf16_bits(cal_x), ref_base=s.bf16_bits(cal_r), gain=gb, bias=bb)
    step_d, inv_d = env.P.to_dev(step, dev), env.P.to_dev(inv, dev)
    # the run: step 0 is sent raw, then 512 coded steps; x_hat lives in one buffer that is decoded in place
    x = s.activations(B, d, scale, gen)
    x_hat = x.clone()                       # first step transmitted directly
    o_free = s.bf16_bits(x_hat).copy()      # oracle's own (free-running) chain, for the report only
    rec = rac.rac_record_bytes(cfg)
    payload = torch.empty(B * rec, dtype=torch.uint8, device=dev)
    status = torch.zeros(1, dtype=torch.int32, device=dev)
    flips = groups = 0
    first_diverged = None
    rms_err = []
    for t in range(1, steps + 1):
        x = s.random_walk_step(x, gen)
        prev_bits = s.bf16_bits(x_hat)      # the device's previous reconstruction: both sides start here
        if t <= 64:
            # the one-launch sender (encode + x_hat, state updated in place) must give the same bytes and state
            fused_state = x_hat.clone()
            fused_pay = torch.empty_like(payload)
            rac.rac_encode_reconstruct(cfg, x, B, fused_state, B, None, gain, bias, step_d, inv_d, fused_pay,
                                       fused_pay.numel(), fused_state, None, 0, status)
        rac.rac_encode(cfg, x, B, x_hat, B, None, gain, bias, step_d, inv_d, payload, payload.numel(), None, 0, status)
        rac.rac_sender_reconstruct(cfg, payload, B, x_hat, B, None, gain, bias, step_d, x_hat, status)  # in place
        torch.cuda.synchronize()
        if t <= 64:
            assert torch.equal(fused_pay, payload) and torch.equal(fused_state, x_hat), f"step {t}: fused sender differs"
        pay = payload.cpu().numpy()
        xb = s.bf16_bits(x)
        rep = env.P.compare_encode(cfg, pay, xb, prev_bits, None, gb, bb, step, inv)
        flips += rep.alpha_flips + rep.beta_flips
        groups += rep.groups
        o_x = orc.reconstruct(d, g, bits, 0, pay, B, ref_base=prev_bits, gain=gb, bias=bb, step=step)
        assert np.array_equal(o_x, s.bf16_bits(x_hat)), f"step {t}: reconstruction differs"
        # free-running oracle chain (not gated): where does it first leave the device's chain?
        o_pay = orc.encode(d, g, bits, 0, xb, ref_base=o_free, gain=gb, bias=bb, step=step, inv_step=inv)
        o_free = orc.reconstruct(d, g, bits, 0, o_pay, B, ref_base=o_free, gain=gb, bias=bb, step=step)
        if first_diverged is None and not np.array_equal(o_free, o_x):
            first_diverged = t
        rms_err.append(float((x_hat.float() - x.float()).pow(2).mean().sqrt().item()))
    assert int(status.item()) == 0
    final_gap = float(np.sqrt(np.mean((orc.bf16_to_f32(o_free) - x_hat.float().cpu().numpy()) ** 2)))
    print(f"config 2: {steps} steps, coefficient flips {flips}/{groups}, rms error first/last {rms_err[0]:.3f}/{rms_err[-1]:.3f}, "
          f"free-running chains first differ at step {first_diverged}, final rms gap {final_gap:.4f}")
    assert flips <= groups * 5e-3
    assert rms_err[-1] < 1.0   # the loop does not blow up


@pytest.mark.parametrize("bits", [2, 3, 4])
@pytest.mark.parametrize("g", [64, 128])
def test_config3_receiver_sweep(env, bits, g):
    """T=16384, d=4096, bits x group sweep, top-8; payloads encoded by the ORACLE, decoded on the device; the
    device's own encode of the same tensors is checked too."""
    s, orc = env.synth, env.orc
    d, k, T = 4096, 8, 16384
    gen = s.generator(s.BASE_SEED + 3, env.dev)
    scale = s.channel_scale(d, 3, env.dev)
    X = s.activations(T, d, scale, gen)
    R = s.affine_noisy_reference(X, g, gen)
    cal = s.activations(1024, d, scale, gen)
    calr = s.affine_noisy_reference(cal, g, gen)
    step, inv = orc.calibrate(d, g, bits, s.bf16_bits(cal), ref_base=s.bf16_bits(calr))
    rep, _, _ = env.P.round_trip_case(env.rac.CodecCfg(d, g, bits, k), X, ref_base=R, step=step, inv_step=inv)
    print(f"config 3 b={bits} g={g}:", rep)
    env.P.assert_caps(rep)


def test_config4_long_context_round_trip(env):
    """T=131072, d=5120, group 128, 4-bit, top-8: span match (131072-token history, ~70 % coverage), uplink encode
    with the fused sender reconstruction, cloud reconstruct, downlink encode of Y = 1.05 * X_hat + N(0, 0.2)
    against X_hat, local reconstruct -- in the launch configuration of the benchmark; the oracle checks the
    matcher whole and every token of each direction against the oracle, chunk by chunk."""
    s, rac, orc, dev = env.synth, env.rac, env.orc, env.dev
    d, g, bits, k, T, H = 5120, 128, 4, 8, 131072, 131072
    cfg = rac.CodecCfg(d, g, bits, k)
    wl = s.span_workload(H, T, seed=4, gap_max=112)
    hist, query = torch.from_numpy(wl.hist).to(dev), torch.from_numpy(wl.query).to(dev)
    nb = rac.rac_match_workspace_bytes(H, T, 8)
    ws = torch.empty(nb, dtype=torch.uint8, device=dev)
    ref_row = torch.empty(T, dtype=torch.int32, device=dev)
    n_spans = torch.zeros(1, dtype=torch.int32, device=dev)
    rac.rac_match_spans(hist, H, query, T, 4, 8, ref_row, None, n_spans, ws, nb)
    torch.cuda.synchronize()
    o_rows, o_spans = orc.match_spans(wl.hist, wl.query, 4, 8)
    assert int(n_spans.item()) == len(o_spans) and np.array_equal(ref_row.cpu().numpy(), o_rows)
    print(f"config 4: {len(o_spans)} spans, coverage {(o_rows >= 0).mean():.3f}")
    gen = s.generator(s.BASE_SEED + 4, dev)
    scale = s.channel_scale(d, 4, dev)
    Hs = s.activations(H, d, scale, gen)
    X = s.affine_noisy_target(Hs, torch.from_numpy(wl.planted_row), g, gen, scale)
    rec = rac.rac_record_bytes(cfg)
    status = torch.zeros(1, dtype=torch.int32, device=dev)
    nws = rac.rac_encode_workspace_bytes(cfg, T)
    ews = torch.empty(nws, dtype=torch.uint8, device=dev)
    st_up, iv_up = device_tables(env, cfg, X[:4096], Hs, ref_row[:4096].contiguous())
    step_up, inv_up = env.P.to_dev(st_up, dev), env.P.to_dev(iv_up, dev)
    pay_up = torch.empty(T * rec, dtype=torch.uint8, device=dev)
    Xs, Xh = torch.empty_like(X), torch.empty_like(X)
    rac.rac_encode_reconstruct(cfg, X, T, Hs, H, ref_row, None, None, step_up, inv_up, pay_up, pay_up.numel(), Xs, ews, nws, status)
    rac.rac_decode_reconstruct(cfg, pay_up, T, Hs, H, ref_row, None, None, step_up, Xh, status)
    torch.cuda.synchronize()
    assert int(status.item()) == 0 and torch.equal(Xs, Xh)      # sender state == receiver state
    Y = s.drifted_state(Xh, gen)
    st_dn, iv_dn = device_tables(env, cfg, Y[:4096], Xh, None)
    step_dn, inv_dn = env.P.to_dev(st_dn, dev), env.P.to_dev(iv_dn, dev)
    pay_dn = torch.empty(T * rec, dtype=torch.uint8, device=dev)
    Yh = torch.empty_like(Y)
    rac.rac_encode(cfg, Y, T, Xh, T, None, None, None, step_dn, inv_dn, pay_dn, pay_dn.numel(), ews, nws, status)
    rac.rac_decode_reconstruct(cfg, pay_dn, T, Xh, T, None, None, None, step_dn, Yh, status)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    # every token of both directions against the oracle, in chunks
    rep_up = env.P.compare_whole(cfg, pay_up, X, Xh, ref_base=Hs, ref_row=o_rows, step=st_up, inv_step=iv_up)
    rep_dn = env.P.compare_whole(cfg, pay_dn, Y, Yh, ref_base=Xh, ref_row=None, step=st_dn, inv_step=iv_dn)
    print("config 4 uplink:", rep_up, "| downlink:", rep_dn)
    for rep in (rep_up, rep_dn):
        env.P.assert_caps(rep)
    # Eq. 10 on every element of the downlink: inside the clip range the error is half a step plus the bf16 rounding
    within = total = 0
    for t0 in range(0, T, 16384):
        sl = slice(t0, t0 + 16384)
        err = (Y[sl].float() - Yh[sl].float()).abs()
        bound = 0.5 * step_dn[0][None, :] * 1.001 + 2.0 ** -8 * Yh[sl].float().abs()
        within += int((err <= bound).sum().item())
        total += err.numel()
    assert within / total > 0.98


@pytest.mark.parametrize("member", [dict(bits=4, topk_group=1), dict(bits=8), dict(bits=4, qgroup=5120),
                                    dict(bits=4, coef_fmt=1)])
def test_config4_shape_with_the_eq8_family(env, member):
    """The benchmark's shape (131072 x 5120, groups of 128) through the per-group-scale kernels, in the launch
    configuration `bench.py` times for its `paper_family` / `shared_coefficients` extras: every token checked
    against the oracle chunk by chunk, sender x_hat == receiver x_hat on the whole tensor, and Eq. 11's
    half-step bound (nothing clips) on every element."""
    s, rac, orc, dev = env.synth, env.rac, env.orc, env.dev
    d, g, T = 5120, 128, 131072
    J = d // g
    bits = member["bits"]
    mk = dict(scale_mode=1, qgroup=member.get("qgroup", 0), topk_group=member.get("topk_group", 0))
    shared = member.get("coef_fmt", 0) == 1
    cfg = rac.CodecCfg(d, g, bits, 0, coef_fmt=int(shared), **mk)
    gen = s.generator(s.BASE_SEED + 9, dev)
    X = s.activations(T, d, s.channel_scale(d, 9, dev), gen)
    R = s.affine_noisy_reference(X, g, gen)
    rec = rac.rac_record_bytes(cfg)
    pay = torch.empty(T * rec, dtype=torch.uint8, device=dev)
    xs, xr = torch.empty_like(X), torch.empty_like(X)
    status = torch.zeros(1, dtype=torch.int32, device=dev)
    seg_tokens = 64
    coef = seg_of = None
    if shared:
        n_seg = T // seg_tokens
        seg_off = (torch.arange(n_seg + 1, dtype=torch.int32, device=dev) * seg_tokens).to(torch.int32)
        coef = torch.empty((n_seg, J), dtype=torch.int32, device=dev)
        seg_of = torch.empty(T, dtype=torch.int32, device=dev)
        nb = rac.rac_fit_segments_workspace_bytes(cfg, T)
        ws = torch.empty(nb, dtype=torch.uint8, device=dev)
        rac.rac_fit_segments(cfg, X, T, R, T, None, None, None, seg_off, n_seg, coef, seg_of, ws, nb, status)
        rac.rac_encode_reconstruct_list(cfg, X, T, None, None, R, T, None, None, 0, None, None, None, None, pay,
                                        pay.numel(), xs, None, 0, status, coef_seg=coef, seg_of=seg_of)
        rac.rac_decode_reconstruct_list(cfg, pay, T, None, None, R, T, None, None, 0, None, None, None, xr, status,
                                        coef_seg=coef, seg_of=seg_of)
    else:
        rac.rac_encode_reconstruct(cfg, X, T, R, T, None, None, None, None, None, pay, pay.numel(), xs, None, 0, status)
        rac.rac_decode_reconstruct(cfg, pay, T, R, T, None, None, None, None, xr, status)
    torch.cuda.synchronize()
    assert int(status.item()) == 0 and torch.equal(xs, xr)
    if shared:
        # every segment: the oracle redoes the pooled fit, then codes with the device's shared words, chunk by chunk
        g_coef = coef.cpu().numpy().view(np.uint32)
        flips = 0
        chunk = 256 * seg_tokens
        for t0 in range(0, T, chunk):
            t1 = min(T, t0 + chunk)
            k0, k1 = t0 // seg_tokens, t1 // seg_tokens
            Xb, Rb = s.bf16_bits(X[t0:t1]), s.bf16_bits(R[t0:t1])
            so = np.arange(k1 - k0 + 1, dtype=np.int32) * seg_tokens
            o_coef = orc.fit_segments(d, g, Xb, so, ref_base=Rb)
            flips += int((g_coef[k0:k1] != o_coef).sum())
            per_tok = np.ascontiguousarray(np.repeat(g_coef[k0:k1], seg_tokens, axis=0))
            p_s = pay.view(T, rec)[t0:t1].cpu().numpy().reshape(-1)
            o_pay = orc.encode(d, g, bits, 0, Xb, ref_base=Rb, forced_coef=per_tok.reshape(-1).copy(), coef_fmt=1,
                               nthreads=orc.max_threads(), **mk)
            assert np.array_equal(o_pay, p_s)
            o_x = orc.reconstruct(d, g, bits, 0, p_s, t1 - t0, ref_base=Rb, coef_fmt=1, shared_coef=per_tok,
                                  nthreads=orc.max_threads(), **mk)
            assert np.array_equal(o_x, s.bf16_bits(xr[t0:t1]))
        print(member, f"shared words that differ from the binary64 pooled fit: {flips} of {g_coef.size}")
        assert flips <= max(3, g_coef.size // 2000)
    else:
        rep = env.P.compare_whole(cfg, pay, X, xr, ref_base=R, ref_row=None)
        print(member, rep)
        env.P.assert_caps(rep)
    # Eq. 11 on every element: half a scale step (the record's own scale) plus the bf16 rounding; outliers: binary16
    scale_off = 0 if shared else 4 * J
    qg = mk["qgroup"] or g
    Jq = d // qg
    for t0 in range(0, T, 16384):
        sl = slice(t0, t0 + 16384)
        sc = pay.view(T, rec)[sl, scale_off:scale_off + 2 * Jq].contiguous().view(torch.float16).float()
        half_step = 0.5 * sc.repeat_interleave(qg, dim=1) * 1.00001
        err = (X[sl].float() - xr[sl].float()).abs()
        mag = torch.maximum(X[sl].float().abs(), xr[sl].float().abs())
        assert bool((err <= half_step + 2.0 ** -8 * mag + 2.0 ** -10 * mag + 1e-12).all())


def test_config4_tokens_through_the_persistent_index(env):
    """The benchmark's token workload (131072-token history, 131072-token prompt) through the persistent index,
    appended as 64 requests: spans, rows and intra-sequence references against the oracle, whole."""
    s, rac, orc, dev = env.synth, env.rac, env.orc, env.dev
    H = T = 131072
    wl = s.span_workload(H, T, seed=s.BASE_SEED + 11, gap_max=112)
    htok, qtok = torch.from_numpy(wl.hist).to(dev), torch.from_numpy(wl.query).to(dev)
    cfg = rac.IndexCfg(H, 4, 8)
    nb = rac.rac_index_bytes(cfg)
    mem = torch.empty(nb, dtype=torch.uint8, device=dev)
    rac.rac_index_reset(cfg, mem, nb)
    bounds = np.arange(0, H + 1, 2048, dtype=np.int32)
    for a, b in zip(bounds[:-1], bounds[1:]):
        rac.rac_index_append(cfg, mem, nb, htok, int(a), int(b))
    nws = rac.rac_index_query_workspace_bytes(T)
    ws = torch.empty(nws, dtype=torch.uint8, device=dev)
    rows = torch.empty(T, dtype=torch.int32, device=dev)
    spans = torch.empty((T // 4 + 1, 3), dtype=torch.int32, device=dev)
    n_spans = torch.zeros(1, dtype=torch.int32, device=dev)
    rac.rac_index_query(cfg, mem, nb, htok, H, qtok, T, True, rows, spans, n_spans, ws, nws)
    torch.cuda.synchronize()
    o_rr, o_sp = orc.match_spans_req(wl.hist, bounds, wl.query, w=4, max_hits=8, intra=True)
    ns = int(n_spans.item())
    assert ns == len(o_sp) and np.array_equal(spans[:ns].cpu().numpy(), o_sp)
    assert np.array_equal(rows.cpu().numpy(), o_rr)
    print(f"index, 64 requests: {ns} spans, covered {((o_rr >= 0) & (o_rr < H)).mean():.3f}, intra {(o_rr >= H).mean():.3f}")


def test_whole_step_replays_from_a_cuda_graph(env):
    """Nothing on the path synchronises, allocates or reads a result back, so one step (retrieval, uplink encode with
    the sender's reconstruction, receiver reconstruction, downlink encode, reconstruction) can be captured once and
    replayed: the replay leaves the same bytes as the eager calls."""
    s, rac, dev = env.synth, env.rac, env.dev
    d, g, bits, k, T, H = 1024, 128, 4, 8, 3000, 8000
    wl = s.span_workload(H, T, seed=31, gap_max=100)
    hist, query = torch.from_numpy(wl.hist).to(dev), torch.from_numpy(wl.query).to(dev)
    gen = s.generator(31, dev)
    scale = s.channel_scale(d, 31, dev)
    Hs = s.activations(H, d, scale, gen)
    X = s.affine_noisy_target(Hs, torch.from_numpy(wl.planted_row), g, gen, scale)
    Y = s.drifted_state(X, gen)
    cfg = rac.CodecCfg(d, g, bits, k)
    rec = rac.rac_record_bytes(cfg)
    nb = rac.rac_match_workspace_bytes(H, T, 8)
    ws = torch.empty(nb, dtype=torch.uint8, device=dev)
    nws = rac.rac_encode_workspace_bytes(cfg, T)
    ews = torch.empty(nws, dtype=torch.uint8, device=dev)
    step = torch.full((2, d), 0.05, dtype=torch.float32, device=dev)
    inv = 1.0 / step
    out = {n: torch.zeros(sz, dtype=dt, device=dev) for n, sz, dt in [
        ("rows", T, torch.int32), ("n_spans", 1, torch.int32), ("pay_up", T * rec, torch.uint8),
        ("pay_dn", T * rec, torch.uint8), ("status", 1, torch.int32)]}
    xs, xr, yr = torch.zeros_like(X), torch.zeros_like(X), torch.zeros_like(X)

    def one_step():
        rac.rac_match_spans(hist, H, query, T, 4, 8, out["rows"], None, out["n_spans"], ws, nb)
        rac.rac_encode_reconstruct(cfg, X, T, Hs, H, out["rows"], None, None, step, inv, out["pay_up"], T * rec, xs, ews,
                                   nws, out["status"])
        rac.rac_decode_reconstruct(cfg, out["pay_up"], T, Hs, H, out["rows"], None, None, step, xr, out["status"])
        rac.rac_encode(cfg, Y, T, xr, T, None, None, None, step, inv, out["pay_dn"], T * rec, ews, nws, out["status"])
        rac.rac_decode_reconstruct(cfg, out["pay_dn"], T, xr, T, None, None, None, step, yr, out["status"])

    one_step()
    torch.cuda.synchronize()
    want = {n: t.clone() for n, t in out.items()}
    want_x, want_y = xr.clone(), yr.clone()
    assert int(out["status"].item()) == 0 and int(out["n_spans"].item()) > 3 and torch.equal(xs, xr)
    graph = torch.cuda.CUDAGraph()
    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    with torch.cuda.stream(side):
        with torch.cuda.graph(graph, stream=side):
            one_step()
    torch.cuda.current_stream().wait_stream(side)
    for _ in range(2):
        for t in list(out.values()) + [xs, xr, yr]:
            t.fill_(7)
        graph.replay()
        torch.cuda.synchronize()
        # the status word is only ever ORed into: it was filled with 7 above
        for n in ("rows", "n_spans", "pay_up", "pay_dn"):
            assert torch.equal(out[n], want[n]), n
        assert torch.equal(xr, want_x) and torch.equal(yr, want_y) and torch.equal(xs, want_x)


@pytest.mark.parametrize("mode", ["static top-8", "Eq. 8, one outlier per group"])
def test_buffers_beyond_four_gibibytes(env, mode):
    """1.2 million tokens of 2048 channels: X, the reference and x_hat are 4.9 GB each, so token offsets pass 2^32
    bytes and 2^31 elements, and the records of the last tokens lie beyond the first GiB of the payload.  The device
    runs the whole size; the oracle checks the first, the last and 1500 random tokens one by one."""
    s, rac, orc, dev, P = env.synth, env.rac, env.orc, env.dev, env.P
    d, g, bits, T = 2048, 128, 4, 1_200_000
    assert 2 * T * d > 2 ** 32 and T * d > 2 ** 31
    gen = s.generator(91, dev)
    scale = s.channel_scale(d, 91, dev)
    X = s.activations(T, d, scale, gen)
    R = s.affine_noisy_reference(X, g, gen)
    if mode == "static top-8":
        cfg, k, mk = rac.CodecCfg(d, g, bits, 8), 8, {}
        step = torch.empty((2, d), dtype=torch.float32, device=dev)
        inv = torch.empty_like(step)
        nb = rac.rac_calibrate_workspace_bytes(cfg)
        cws = torch.empty(nb, dtype=torch.uint8, device=dev)
        st0 = torch.zeros(1, dtype=torch.int32, device=dev)
        rac.rac_calibrate_steps(cfg, X[:2048], 2048, R, T, None, None, None, 3.0, step, inv, cws, nb, st0)
        st_np, iv_np = step.cpu().numpy(), inv.cpu().numpy()
    else:
        cfg, k, mk = rac.CodecCfg(d, g, bits, 0, scale_mode=1, topk_group=1), 0, dict(scale_mode=1, topk_group=1)
        step = inv = st_np = iv_np = None
    rec = rac.rac_record_bytes(cfg)
    assert T * rec > 2 ** 30
    payload = torch.empty(T * rec, dtype=torch.uint8, device=dev)
    xs = torch.empty_like(X)
    nws = rac.rac_encode_workspace_bytes(cfg, T)
    ews = torch.empty(max(nws, 16), dtype=torch.uint8, device=dev)
    status = torch.zeros(1, dtype=torch.int32, device=dev)
    rac.rac_encode_reconstruct(cfg, X, T, R, T, None, None, None, step, inv, payload, payload.numel(), xs, ews, nws, status)
    xr = torch.empty_like(X)
    rac.rac_decode_reconstruct(cfg, payload, T, R, T, None, None, None, step, xr, status)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    for t0 in range(0, T, 200_000):                       # sender and receiver agree everywhere
        assert torch.equal(xs[t0:t0 + 200_000], xr[t0:t0 + 200_000])
    rng = np.random.default_rng(91)
    sample = np.unique(np.concatenate([np.arange(32), np.arange(T - 32, T), rng.integers(0, T, 1500),
                                       rng.integers(T - 100_000, T, 300)]))     # extra weight beyond 2^32 bytes
    idx = torch.from_numpy(sample).to(dev)
    pay_s = payload.view(T, rec)[idx].cpu().numpy().reshape(-1)
    Xs, Rs = s.bf16_bits(X[idx]), s.bf16_bits(R[idx])
    rep = P.compare_encode(cfg, pay_s, Xs, Rs, None, None, None, st_np, iv_np)
    print(rep)
    o_x = orc.reconstruct(d, g, bits, k, pay_s, sample.size, ref_base=Rs, step=st_np, nthreads=orc.max_threads(), **mk)
    assert np.array_equal(o_x, s.bf16_bits(xr[idx]))
