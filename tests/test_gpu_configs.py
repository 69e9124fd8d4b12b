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
    assert rep.alpha_flips <= rep.groups * 5e-4 and rep.beta_flips <= rep.groups * 5e-3


def test_config4_long_context_round_trip(env):
    """T=131072, d=5120, group 128, 4-bit, top-8: span match (131072-token history, ~70 % coverage), uplink encode
    with the fused sender reconstruction, cloud reconstruct, downlink encode of Y = 1.05 * X_hat + N(0, 0.2)
    against X_hat, local reconstruct -- in the launch configuration of the benchmark; the oracle checks the
    matcher whole and ~1500 sampled tokens of each direction one by one."""
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
    rng = np.random.default_rng(4)
    sample = np.unique(np.concatenate([np.arange(48), np.arange(T - 48, T), rng.integers(0, T, 1400)]))
    idx = torch.from_numpy(sample).to(dev)
    # uplink sample: gathered references made compact for the oracle
    rows = o_rows[sample]
    has = rows >= 0
    compact = np.where(has, np.cumsum(has) - 1, -1).astype(np.int32)
    Rc = Hs[torch.from_numpy(rows[has]).to(dev).long()]
    p_s = pay_up.view(T, rec)[idx].cpu().numpy().reshape(-1)
    rep_up = env.P.compare_encode(cfg, p_s, s.bf16_bits(X[idx]), s.bf16_bits(Rc), compact, None, None, st_up, iv_up)
    o_x = orc.reconstruct(d, g, bits, k, p_s, sample.size, ref_base=s.bf16_bits(Rc), ref_row=compact, step=st_up)
    assert np.array_equal(o_x, s.bf16_bits(Xh[idx]))
    # downlink sample: reference = the reconstructed uplink rows of the same tokens
    p_s = pay_dn.view(T, rec)[idx].cpu().numpy().reshape(-1)
    rep_dn = env.P.compare_encode(cfg, p_s, s.bf16_bits(Y[idx]), s.bf16_bits(Xh[idx]), None, None, None, st_dn, iv_dn)
    o_y = orc.reconstruct(d, g, bits, k, p_s, sample.size, ref_base=s.bf16_bits(Xh[idx]), step=st_dn)
    assert np.array_equal(o_y, s.bf16_bits(Yh[idx]))
    print("config 4 uplink:", rep_up, "| downlink:", rep_dn)
    # Eq. 10 on every element of the downlink: inside the clip range the error is half a step plus the bf16 rounding
    within = total = 0
    for t0 in range(0, T, 16384):
        sl = slice(t0, t0 + 16384)
        err = (Y[sl].float() - Yh[sl].float()).abs()
        bound = 0.5 * step_dn[0][None, :] * 1.001 + 2.0 ** -8 * Yh[sl].float().abs()
        within += int((err <= bound).sum().item())
        total += err.numel()
    assert within / total > 0.98
