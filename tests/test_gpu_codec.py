"""CUDA codec vs CPU oracle, through the C ABI (needs a B200)."""
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
    oracle.lib()
    return type("Env", (), dict(orc=oracle, rac=rac, synth=synth, P=parity, dev=torch.device("cuda:0")))


def prefill_inputs(env, T, d, g, seed, cal_T=256):
    s = env.synth
    gen = s.generator(seed, env.dev)
    scale = s.channel_scale(d, seed, env.dev)
    X = s.activations(T, d, scale, gen)
    R = s.affine_noisy_reference(X, g, gen)
    cal = s.activations(cal_T, d, scale, gen)
    calr = s.affine_noisy_reference(cal, g, gen)
    return X, R, cal, calr


def oracle_tables(env, d, g, bits, cal, calr=None, **kw):
    return env.orc.calibrate(d, g, bits, env.synth.bf16_bits(cal),
                             ref_base=None if calr is None else env.synth.bf16_bits(calr), **kw)


# --------------------------------------------------------------------------- shapes, widths, tails
@pytest.mark.parametrize("d,g,bits,k,T", [
    (4096, 128, 4, 0, 128),    # the small prefill configuration
    (4096, 128, 4, 8, 301),    # several waves of persistent CTAs would need T > grid: covered further down
    (4096, 64, 3, 8, 77),
    (4096, 64, 2, 8, 77),
    (4096, 128, 3, 8, 64),
    (4096, 128, 2, 0, 33),
    (3584, 128, 3, 0, 64),     # decode width: the last warp is half empty
    (5120, 128, 4, 8, 95),     # two-stage ring
    (8192, 256, 4, 16, 21),    # widest supported, 16 outliers
    (1024, 1024, 4, 8, 19),    # one group per token
    (96, 32, 4, 3, 50),        # a single partly filled warp, groups of one lane
    (32, 32, 2, 1, 7),
])
def test_round_trip_matches_oracle(env, d, g, bits, k, T):
    X, R, cal, calr = prefill_inputs(env, T, d, g, seed=1000 + d + bits + k)
    step, inv = oracle_tables(env, d, g, bits, cal, calr)
    cfg = env.rac.CodecCfg(d, g, bits, k)
    rep, _, xr = env.P.round_trip_case(cfg, X, ref_base=R, step=step, inv_step=inv)
    print(rep)
    assert rep.alpha_flips + rep.beta_flips <= max(3, rep.groups // 200)
    # the codec actually codes: error well below the signal
    err = (xr.float() - X.float()).abs().mean().item()
    assert err < 0.1 * X.float().abs().mean().item() + 0.05


def test_many_tokens_per_cta_and_ragged_tail(env):
    # more tokens than resident CTAs, not a multiple of anything: the ring wraps several times
    d, g, bits, k, T = 4096, 128, 4, 8, 2 * 148 * 4 + 37
    X, R, cal, calr = prefill_inputs(env, T, d, g, seed=7)
    step, inv = oracle_tables(env, d, g, bits, cal, calr)
    rep, _, _ = env.P.round_trip_case(env.rac.CodecCfg(d, g, bits, k), X, ref_base=R, step=step, inv_step=inv)
    print(rep)


# --------------------------------------------------------------------------- reference resolution
def test_gathered_rows_direct_tokens_and_missing_reference(env):
    d, g, bits, k, T = 4096, 128, 4, 8, 200
    s = env.synth
    gen = s.generator(11, env.dev)
    scale = s.channel_scale(d, 11, env.dev)
    Hs = s.activations(500, d, scale, gen)
    rng = np.random.default_rng(11)
    rows = rng.integers(0, 500, T).astype(np.int32)
    rows[rng.random(T) < 0.4] = -1
    rows[:3] = [-1, 499, 0]
    ref_row = torch.from_numpy(rows).to(env.dev)
    X = s.affine_noisy_target(Hs, ref_row, g, gen, scale)
    # tables: row 0 from referenced tokens, row 1 from direct tokens
    step, inv = env.orc.calibrate(d, g, bits, s.bf16_bits(X), ref_base=s.bf16_bits(Hs), ref_row=rows)
    assert step[0].all() and step[1].all()
    cfg = env.rac.CodecCfg(d, g, bits, k)
    rep, pay, xr = env.P.round_trip_case(cfg, X, ref_base=Hs, ref_row=ref_row, step=step, inv_step=inv)
    coef = env.orc.split_payload(pay, T, d, g, bits, k)[0]
    assert np.all((coef[rows < 0] & 0x7fff) == 0)  # direct tokens: alpha = 0
    # no reference buffer at all: every token direct
    rep2, pay2, _ = env.P.round_trip_case(cfg, X, ref_base=None, step=step, inv_step=inv)
    assert np.all((env.orc.split_payload(pay2, T, d, g, bits, k)[0] & 0x7fff) == 0)


def test_predictor_gain_bias_transform(env):
    d, g, bits, T = 3584, 128, 3, 64
    s = env.synth
    gen = s.generator(12, env.dev)
    scale = s.channel_scale(d, 12, env.dev)
    prev = s.activations(T, d, scale, gen)
    X = s.random_walk_step(prev, gen)
    gain, bias = s.predictor_gain_bias(d, 12, env.dev)
    step, inv = env.orc.calibrate(d, g, bits, s.bf16_bits(X), ref_base=s.bf16_bits(prev),
                                  gain=s.f16_bits(gain), bias=s.f16_bits(bias))
    rep, _, _ = env.P.round_trip_case(env.rac.CodecCfg(d, g, bits, 0), X, ref_base=prev, gain=gain, bias=bias,
                                      step=step, inv_step=inv)
    # with outliers too (the outlier path re-applies the transform to single elements)
    rep, _, _ = env.P.round_trip_case(env.rac.CodecCfg(d, g, bits, 8), X, ref_base=prev, gain=gain, bias=bias,
                                      step=step, inv_step=inv)


# --------------------------------------------------------------------------- closed forms and degenerate inputs
def test_reference_equal_to_x_and_all_equal_magnitudes(env):
    d, g, T = 4096, 128, 9
    s = env.synth
    gen = s.generator(13, env.dev)
    X = s.activations(T, d, s.channel_scale(d, 13, env.dev), gen)
    step = np.full((2, d), 0.02, np.float32)
    inv = (np.float32(1) / step).astype(np.float32)
    for bits, k in [(4, 0), (4, 8), (3, 8), (2, 16)]:
        cfg = env.rac.CodecCfg(d, g, bits, k)
        rep, pay, xr = env.P.round_trip_case(cfg, X, ref_base=X, step=step, inv_step=inv)
        coef, codes, oi, ov = env.orc.split_payload(pay, T, d, g, bits, k)
        assert np.all(coef == 0x3c00) and not codes.any()
        if k:  # every |e| ties at zero: the k lowest channels (more candidates than the short list holds)
            assert np.array_equal(oi, np.tile(np.arange(k, dtype=np.uint16), (T, 1)))
        assert torch.equal(xr, X)


def test_constant_reference_and_many_exact_ties(env):
    d, g, bits, k, T = 1024, 128, 4, 8, 40
    rng = np.random.default_rng(14)
    vals = (rng.integers(-12, 13, size=(T, d)) / 4).astype(np.float32)   # coarse grid: many equal |e|
    X = torch.from_numpy(vals).to(torch.bfloat16).to(env.dev)
    R = torch.full((T, d), 3.5, dtype=torch.bfloat16, device=env.dev)
    step = np.full((2, d), 0.25, np.float32)
    inv = (np.float32(1) / step).astype(np.float32)
    cfg = env.rac.CodecCfg(d, g, bits, k)
    rep, pay, _ = env.P.round_trip_case(cfg, X, ref_base=R, step=step, inv_step=inv)
    coef = env.orc.split_payload(pay, T, d, g, bits, k)[0]
    assert np.all((coef & 0x7fff) == 0)  # zero variance -> alpha = 0
    assert rep.alpha_flips == 0


def test_step_zero_channels_and_saturation(env):
    d, g, bits, T = 512, 64, 4, 30
    X, R, cal, calr = prefill_inputs(env, T, d, g, seed=15)
    step, inv = oracle_tables(env, d, g, bits, cal, calr, clip_sigmas=1.0)  # tight clip: plenty of saturated codes
    step[0, ::3] = 0.0
    inv[0, ::3] = 0.0
    cfg = env.rac.CodecCfg(d, g, bits, 0)
    rep, pay, _ = env.P.round_trip_case(cfg, X, ref_base=R, step=step, inv_step=inv)
    codes = env.orc.split_payload(pay, T, d, g, bits, 0)[1]
    q = np.stack([env.orc.unpack_codes(codes[t], d, bits) for t in range(T)])
    assert not q[:, ::3].any()
    assert (np.abs(q) == 7).mean() > 0.05


# --------------------------------------------------------------------------- device-detected anomalies (no traps)
def test_status_bits(env):
    d, g, bits, k, T = 256, 64, 4, 4, 12
    rac = env.rac
    X, R, cal, calr = prefill_inputs(env, T, d, g, seed=16)
    step, inv = oracle_tables(env, d, g, bits, cal, calr)
    step_d, inv_d = env.P.to_dev(step, env.dev), env.P.to_dev(inv, env.dev)
    cfg = rac.CodecCfg(d, g, bits, k)
    # ref_row beyond the buffer: flagged, token coded as direct (same bytes as ref_row = -1)
    rows = np.arange(T, dtype=np.int32)
    rows[5] = T + 3
    pay, st = env.P.gpu_encode(cfg, X, R, torch.from_numpy(rows).to(env.dev), None, None, step_d, inv_d)
    assert st == rac.STATUS_REF_RANGE
    rows[5] = -1
    pay2, st2 = env.P.gpu_encode(cfg, X, R, torch.from_numpy(rows).to(env.dev), None, None, step_d, inv_d)
    assert st2 == 0 and np.array_equal(pay, pay2)
    # reserved code and out-of-range outlier index on decode
    rec = rac.rac_record_bytes(cfg)
    bad = pay2.copy().reshape(T, rec)
    bad[2, 4 * (d // g)] = (bad[2, 4 * (d // g)] & 0xF0) | 0x08
    xh, st = env.P.gpu_decode(cfg, bad.reshape(-1), T, R, torch.from_numpy(rows).to(env.dev), None, None, step_d, env.dev)
    assert st == rac.STATUS_RESERVED_CODE
    o_x, o_st = env.orc.reconstruct(d, g, bits, k, bad.reshape(-1), T, ref_base=env.synth.bf16_bits(R), ref_row=rows,
                                    step=step, return_status=True)
    assert o_st & 2 and np.array_equal(o_x, env.synth.bf16_bits(xh))
    bad = pay2.copy().reshape(T, rec)
    off = 4 * (d // g) + d * bits // 8
    bad[3, off:off + 2] = np.frombuffer(np.uint16(d + 5).tobytes(), np.uint8)
    xh, st = env.P.gpu_decode(cfg, bad.reshape(-1), T, R, torch.from_numpy(rows).to(env.dev), None, None, step_d, env.dev)
    assert st == rac.STATUS_OUTLIER_RANGE
    # non-finite input
    Xn = X.clone()
    Xn[7, 100] = float("inf")
    _, st = env.P.gpu_encode(cfg, Xn, R, None, None, None, step_d, inv_d)
    assert st & rac.STATUS_NONFINITE


def test_in_place_identity_reconstruction(env):
    # decode-style feedback: X_hat overwrites the reference buffer it was decoded against
    d, g, bits, T = 3584, 128, 3, 64
    s = env.synth
    gen = s.generator(17, env.dev)
    prev = s.activations(T, d, s.channel_scale(d, 17, env.dev), gen)
    X = s.random_walk_step(prev, gen)
    step, inv = env.orc.calibrate(d, g, bits, s.bf16_bits(X), ref_base=s.bf16_bits(prev))
    step_d, inv_d = env.P.to_dev(step, env.dev), env.P.to_dev(inv, env.dev)
    cfg = env.rac.CodecCfg(d, g, bits, 0)
    pay, st = env.P.gpu_encode(cfg, X, prev, None, None, None, step_d, inv_d)
    out_of_place, _ = env.P.gpu_decode(cfg, pay, T, prev, None, None, None, step_d, env.dev)
    buf = prev.clone()
    status = torch.zeros(1, dtype=torch.int32, device=env.dev)
    env.rac.rac_sender_reconstruct(cfg, torch.from_numpy(pay).to(env.dev), T, buf, T, None, None, None, step_d, buf, status)
    torch.cuda.synchronize()
    assert int(status.item()) == 0 and torch.equal(buf, out_of_place)


def test_fused_sender_in_place_with_outliers_is_refused(env):
    """With per-token outliers the sender-side x_hat may not overwrite the rows it was coded against (the outlier
    launch reads them again after x_hat is written): the call is refused before anything runs, the buffers stay
    untouched, and the out-of-place call on the same inputs matches the receiver and the oracle."""
    d, g, bits, k, T = 2048, 128, 4, 8, 96
    s, rac, dev = env.synth, env.rac, env.dev
    gen = s.generator(18, dev)
    prev = s.activations(T, d, s.channel_scale(d, 18, dev), gen)
    X = s.random_walk_step(prev, gen)
    step, inv = env.orc.calibrate(d, g, bits, s.bf16_bits(X), ref_base=s.bf16_bits(prev))
    step_d, inv_d = env.P.to_dev(step, dev), env.P.to_dev(inv, dev)
    cfg = rac.CodecCfg(d, g, bits, k)
    rec = rac.rac_record_bytes(cfg)
    pay = torch.full((T * rec,), 0xA5, dtype=torch.uint8, device=dev)
    nws = rac.rac_encode_workspace_bytes(cfg, T)
    ws = torch.empty(nws, dtype=torch.uint8, device=dev)
    status = torch.zeros(1, dtype=torch.int32, device=dev)
    state = prev.clone()
    with pytest.raises(Exception) as ei:
        rac.rac_encode_reconstruct(cfg, X, T, state, T, None, None, None, step_d, inv_d, pay, pay.numel(), state, ws, nws, status)
    assert "unsupported" in str(ei.value).lower()
    xin = X.clone()
    with pytest.raises(Exception):       # x_hat over X itself
        rac.rac_encode_reconstruct(cfg, xin, T, prev, T, None, None, None, step_d, inv_d, pay, pay.numel(), xin, ws, nws, status)
    torch.cuda.synchronize()
    assert torch.equal(state, prev) and torch.equal(xin, X) and bool(torch.all(pay == 0xA5))
    # out of place: same bytes as rac_encode, x_hat equal to the receiver's and the oracle's
    pay_f, xs, st = env.P.gpu_encode_reconstruct(cfg, X, prev, None, None, None, step_d, inv_d)
    xr, st2 = env.P.gpu_decode(cfg, pay_f, T, prev, None, None, None, step_d, dev)
    assert st == 0 and st2 == 0 and torch.equal(xs, xr)
    o_x = env.orc.reconstruct(d, g, bits, k, pay_f, T, ref_base=s.bf16_bits(prev), step=step)
    assert np.array_equal(o_x, s.bf16_bits(xs))


@pytest.mark.parametrize("d,bits,k,kg", [(5120, 4, 8, -1), (4096, 3, 0, -1), (96, 2, 0, -1), (5120, 4, 0, 1), (4096, 8, 0, 0)])
def test_waits_that_cannot_complete_give_up_and_leave_the_stream_usable(env, d, bits, k, kg):
    """The give-up path of the bounded waits, run on purpose in its safe form: every stage announces more bytes than
    its copies deliver and the poll limit is lowered, so each CTA's wait runs out, the kernel sets RAC_STATUS_TIMEOUT
    and returns.  Nothing faults, nothing spins without a bound; the next ordinary calls on the same stream give the
    bits they always give."""
    g, T = 32 if d == 96 else 128, 40
    rac, P, dev = env.rac, env.P, env.dev
    X, R, cal, calr = prefill_inputs(env, T, d, g, seed=91)
    if kg < 0:      # the static table
        step, inv = oracle_tables(env, d, g, bits, cal, calr)
        step_d, inv_d = P.to_dev(step, dev), P.to_dev(inv, dev)
        cfg = rac.CodecCfg(d, g, bits, k)
    else:           # Eq. 8 as printed: scales in the record, kg outliers per group
        step_d = inv_d = None
        cfg = rac.CodecCfg(d, g, bits, 0, scale_mode=1, topk_group=kg)
    rec = rac.rac_record_bytes(cfg)
    good, st = P.gpu_encode(cfg, X, R, None, None, None, step_d, inv_d)
    assert st == 0
    good_x, st = P.gpu_decode(cfg, good, T, R, None, None, None, step_d, dev)
    assert st == 0
    nws = rac.rac_encode_workspace_bytes(cfg, T)
    ws = torch.zeros(max(nws, 16), dtype=torch.uint8, device=dev)
    for which in (0, 1):
        status = torch.zeros(1, dtype=torch.int32, device=dev)
        if which == 0:
            out = torch.zeros(T * rec, dtype=torch.uint8, device=dev)
            rac.rac_selftest_bounded_wait(cfg, 0, X, T, R, T, step_d, inv_d, out, out.numel(), ws if nws else None, nws, status)
        else:
            out = torch.zeros((T, d), dtype=torch.bfloat16, device=dev)
            rac.rac_selftest_bounded_wait(cfg, 1, torch.from_numpy(good).to(dev), T, R, T, step_d, None, out,
                                          out.numel() * 2, None, 0, status)
        torch.cuda.synchronize()
        assert int(status.item()) & rac.STATUS_TIMEOUT, f"which={which}: status {int(status.item())}"
        # the same stream, right afterwards: ordinary calls, ordinary results
        again, st = P.gpu_encode(cfg, X, R, None, None, None, step_d, inv_d)
        assert st == 0 and np.array_equal(again, good)
        again_x, st = P.gpu_decode(cfg, good, T, R, None, None, None, step_d, dev)
        assert st == 0 and torch.equal(again_x, good_x)


def test_prepared_calls_repeat_the_plain_calls(env):
    """binding.prepare marshals the arguments of a call once; the function it returns launches the same work."""
    d, g, bits, T = 3584, 128, 3, 64
    s, rac, dev = env.synth, env.rac, env.dev
    gen = s.generator(19, dev)
    prev = s.activations(T, d, s.channel_scale(d, 19, dev), gen)
    X = s.random_walk_step(prev, gen)
    step, inv = env.orc.calibrate(d, g, bits, s.bf16_bits(X), ref_base=s.bf16_bits(prev))
    step_d, inv_d = env.P.to_dev(step, dev), env.P.to_dev(inv, dev)
    cfg = rac.CodecCfg(d, g, bits, 0)
    rec = rac.rac_record_bytes(cfg)
    status = torch.zeros(1, dtype=torch.int32, device=dev)
    pay_a, pay_b = (torch.zeros(T * rec, dtype=torch.uint8, device=dev) for _ in range(2))
    xa, xb = torch.empty_like(X), torch.empty_like(X)
    rac.rac_encode_reconstruct(cfg, X, T, prev, T, None, None, None, step_d, inv_d, pay_a, pay_a.numel(), xa, None, 0, status)
    call = rac.prepare(rac.rac_encode_reconstruct, cfg, X, T, prev, T, None, None, None, step_d, inv_d, pay_b, pay_b.numel(),
                       xb, None, 0, status)
    torch.cuda.synchronize()
    assert not pay_b.any()                      # preparing launches nothing
    call()
    call()
    torch.cuda.synchronize()
    assert int(status.item()) == 0 and torch.equal(pay_a, pay_b) and torch.equal(xa, xb)
    dec = rac.prepare(rac.rac_decode_reconstruct, cfg, pay_b, T, prev, T, None, None, None, step_d, xb, status)
    xb.zero_()
    dec()
    torch.cuda.synchronize()
    assert torch.equal(xa, xb)
    with pytest.raises(ValueError):             # a wrapper that launches nothing cannot be prepared
        rac.prepare(rac.rac_record_bytes, cfg)


def test_zero_tokens_is_a_no_op(env):
    cfg = env.rac.CodecCfg(4096, 128, 4, 8)
    t = torch.zeros(16, dtype=torch.uint8, device=env.dev)
    f = torch.zeros((2, 4096), dtype=torch.float32, device=env.dev)
    x = torch.zeros((0, 4096), dtype=torch.bfloat16, device=env.dev)
    env.rac.rac_encode(cfg, x, 0, None, 0, None, None, None, f, f, t, 0, None, 0, None)
    env.rac.rac_decode_reconstruct(cfg, t, 0, None, 0, None, None, None, f, x, None)
    torch.cuda.synchronize()


# --------------------------------------------------------------------------- calibration kernel
@pytest.mark.parametrize("d,g,bits", [(4096, 128, 4), (3584, 128, 3), (5120, 128, 4), (96, 32, 2)])
def test_calibrate_steps_matches_oracle(env, d, g, bits):
    s, rac = env.synth, env.rac
    T = 700
    gen = s.generator(18, env.dev)
    scale = s.channel_scale(d, 18, env.dev)
    Hs = s.activations(300, d, scale, gen)
    rng = np.random.default_rng(18)
    rows = rng.integers(0, 300, T).astype(np.int32)
    rows[rng.random(T) < 0.3] = -1
    ref_row = torch.from_numpy(rows).to(env.dev)
    X = s.affine_noisy_target(Hs, ref_row, g, gen, scale)
    cfg = rac.CodecCfg(d, g, bits, 0)
    step = torch.empty((2, d), dtype=torch.float32, device=env.dev)
    inv = torch.empty_like(step)
    nb = rac.rac_calibrate_workspace_bytes(cfg)
    ws = torch.empty(nb, dtype=torch.uint8, device=env.dev)
    status = torch.zeros(1, dtype=torch.int32, device=env.dev)
    rac.rac_calibrate_steps(cfg, X, T, Hs, 300, ref_row, None, None, 3.0, step, inv, ws, nb, status)
    step2, inv2 = torch.empty_like(step), torch.empty_like(step)
    rac.rac_calibrate_steps(cfg, X, T, Hs, 300, ref_row, None, None, 3.0, step2, inv2, ws, nb, status)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    assert torch.equal(step, step2) and torch.equal(inv, inv2)  # deterministic
    o_step, o_inv = env.orc.calibrate(d, g, bits, s.bf16_bits(X), ref_base=s.bf16_bits(Hs), ref_row=rows)
    gs, gi = step.cpu().numpy(), inv.cpu().numpy()
    # binary16 values; the device sums e^2 in binary32 and fits in binary32, so a step may land on the
    # neighbouring binary16 value; it must never be further than that
    assert np.array_equal(gs, gs.astype(np.float16).astype(np.float32))
    ulp = np.spacing(o_step.astype(np.float16)).astype(np.float32)
    assert np.all(np.abs(gs - o_step) <= ulp)
    assert (gs != o_step).mean() < 0.02
    assert np.array_equal(gi, np.where(gs > 0, np.float32(1) / np.where(gs > 0, gs, 1), 0).astype(np.float32))
    # no direct tokens -> row 1 is all zero
    rac.rac_calibrate_steps(cfg, X, T, Hs, 300, torch.from_numpy(np.maximum(rows, 0)).to(env.dev), None, None, 3.0,
                            step, inv, ws, nb, status)
    torch.cuda.synchronize()
    assert not step[1].any() and not inv[1].any() and step[0].all()


# --------------------------------------------------------------------------- full-size configurations
@pytest.mark.parametrize("bits,g", [(4, 128), (3, 64), (2, 128)])
def test_full_size_sweep_point(env, bits, g):
    """T=16384, d=4096, top-8: the whole tensor against the oracle (the oracle needs a few seconds)."""
    d, k, T = 4096, 8, 16384
    X, R, cal, calr = prefill_inputs(env, T, d, g, seed=3, cal_T=1024)
    step, inv = oracle_tables(env, d, g, bits, cal, calr)
    rep, _, _ = env.P.round_trip_case(env.rac.CodecCfg(d, g, bits, k), X, ref_base=R, step=step, inv_step=inv)
    print(rep)
    env.P.assert_caps(rep)


def test_long_context_whole(env):
    """T=131072, d=5120, span-style gathered rows with 30 % direct tokens: the device runs the full size in
    the launch configuration of the benchmark; the oracle checks every token, chunk by chunk."""
    d, g, bits, k, T, H = 5120, 128, 4, 8, 131072, 131072
    s, rac, orc = env.synth, env.rac, env.orc
    gen = s.generator(4, env.dev)
    scale = s.channel_scale(d, 4, env.dev)
    Hs = s.activations(H, d, scale, gen)
    wl = s.span_workload(H, T, seed=4, gap_max=112)
    ref_row = torch.from_numpy(wl.planted_row).to(env.dev)
    X = s.affine_noisy_target(Hs, ref_row, g, gen, scale)
    cfg = rac.CodecCfg(d, g, bits, k)
    step = torch.empty((2, d), dtype=torch.float32, device=env.dev)
    inv = torch.empty_like(step)
    nb = rac.rac_calibrate_workspace_bytes(cfg)
    ws = torch.empty(nb, dtype=torch.uint8, device=env.dev)
    status = torch.zeros(1, dtype=torch.int32, device=env.dev)
    rac.rac_calibrate_steps(cfg, X[:4096], 4096, Hs, H, ref_row[:4096].contiguous(), None, None, 3.0, step, inv, ws, nb, status)
    rec = rac.rac_record_bytes(cfg)
    payload = torch.empty(T * rec, dtype=torch.uint8, device=env.dev)
    nws = rac.rac_encode_workspace_bytes(cfg, T)
    ews = torch.empty(nws, dtype=torch.uint8, device=env.dev)
    rac.rac_encode(cfg, X, T, Hs, H, ref_row, None, None, step, inv, payload, payload.numel(), ews, nws, status)
    xh = torch.empty_like(X)
    rac.rac_decode_reconstruct(cfg, payload, T, Hs, H, ref_row, None, None, step, xh, status)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    # every token against the oracle, in chunks (reference rows gathered into a compact buffer per chunk)
    st, iv = step.cpu().numpy(), inv.cpu().numpy()
    rep = env.P.compare_whole(cfg, payload, X, xh, ref_base=Hs, ref_row=wl.planted_row, step=st, inv_step=iv)
    print(rep)
    env.P.assert_caps(rep)
    # properties that hold at any size: Eq. 10 bound on every element of the full tensor
    within, total = 0, 0
    for t0 in range(0, T, 16384):
        sl = slice(t0, t0 + 16384)
        err = (X[sl].float() - xh[sl].float()).abs()
        tab = torch.where((ref_row[sl] >= 0)[:, None], step[0][None, :], step[1][None, :])
        bound = 0.5 * tab * 1.001 + 2.0 ** -8 * xh[sl].float().abs()
        within += int((err <= bound).sum().item())
        total += err.numel()
    frac_within = within / total
    assert frac_within > 0.98  # the rest is clipping by the static table (3 sigma) on direct and referenced tokens


# --------------------------------------------------------------------------- Eq. 8 as printed: per-group scale in the record
@pytest.mark.parametrize("d,g,bits,T", [
    (4096, 128, 4, 257), (4096, 64, 3, 64), (3584, 128, 4, 64), (5120, 128, 2, 95), (96, 32, 4, 9), (2080, 32, 4, 33),
])
def test_dynamic_group_scale_matches_oracle(env, d, g, bits, T):
    """scale_mode 1: no step table; the scale of each (token, group) travels in the record.  Same protocol as the
    static mode; on top, nothing may clip (Eq. 11): every element within half a scale step."""
    X, R, _, _ = prefill_inputs(env, T, d, g, seed=2000 + d + bits)
    cfg = env.rac.CodecCfg(d, g, bits, 0, scale_mode=1)
    assert env.rac.rac_record_bytes(cfg) == env.orc.record_bytes(d, g, bits, 0, 1)
    rep, pay, xr = env.P.round_trip_case(cfg, X, ref_base=R)
    print(rep)
    coef, codes, _, _, scale = env.orc.split_payload(pay, T, d, g, bits, 0, 1)
    s = scale.view(np.float16).astype(np.float64).repeat(g, axis=1)
    h = X.float().cpu().numpy().astype(np.float64)
    xh = xr.float().cpu().numpy().astype(np.float64)
    # half a scale step from the quantiser, plus the bf16 rounding of the reconstruction (relative to ITS magnitude)
    assert np.all(np.abs(h - xh) <= 0.5 * s * (1 + 1e-5) + 2.0 ** -8 * np.maximum(np.abs(h), np.abs(xh)) + 1e-12)
    # direct tokens and the gain/bias reference go through the same path
    rows = np.arange(T, dtype=np.int32)
    rows[::3] = -1
    env.P.round_trip_case(cfg, X, ref_base=R, ref_row=torch.from_numpy(rows).to(env.dev))


def test_dynamic_group_scale_identity_and_rejections(env):
    d, g, T = 1024, 128, 5
    s = env.synth
    X = s.activations(T, d, s.channel_scale(d, 33, env.dev), s.generator(33, env.dev))
    cfg = env.rac.CodecCfg(d, g, 4, 0, scale_mode=1)
    rep, pay, xr = env.P.round_trip_case(cfg, X, ref_base=X)
    coef, codes, _, _, scale = env.orc.split_payload(pay, T, d, g, 4, 0, 1)
    assert not scale.any() and not codes.any() and torch.equal(xr, X)        # zero-group marker everywhere
    assert env.rac.rac_record_bytes(env.rac.CodecCfg(d, g, 4, 8, scale_mode=1)) == 0   # outliers: not in this mode
    assert env.rac.rac_record_bytes(env.rac.CodecCfg(d, g, 4, 0, scale_mode=2)) == 0


# --------------------------------------------------------------------------- the rest of the quantiser family (Sec. IV-C)
@pytest.mark.parametrize("d,g,bits,qg,kg,T", [
    (4096, 128, 4, 0, 1, 150),      # one outlier per group of 128
    (4096, 128, 4, 0, 2, 65),
    (4096, 128, 8, 0, 1, 65),       # 8-bit codes
    (4096, 128, 8, 0, 0, 65),
    (4096, 64, 3, 64, 4, 40),       # four rounds, groups of two lanes
    (5120, 128, 4, 32, 1, 95),      # quantisation groups of one lane inside alignment groups of four
    (5120, 128, 2, 256, 3, 50),     # quantisation groups of eight lanes spanning two alignment groups
    (3584, 128, 4, 3584, 0, 64),    # decode mode: one scale per token, d/32 not a power of two
    (3584, 128, 8, 3584, 0, 64),
    (4096, 128, 3, 4096, 0, 33),
    (1024, 128, 4, 1024, 0, 20),    # one scale per token inside one warp
    (8192, 256, 8, 0, 2, 21),       # widest token, eight warps
    (96, 32, 4, 32, 2, 9),          # a single partly filled warp
    (96, 32, 8, 96, 0, 9),
    (2080, 32, 4, 0, 1, 33),        # odd group counts: padding after scales and after offsets
    (4096, 128, 4, 0, 8, 70),       # eight outliers per group of 128
    (5120, 128, 4, 256, 6, 41),     # six, groups of eight lanes
    (4096, 64, 8, 32, 5, 23),       # five in groups of one lane, 8-bit codes
    (4096, 128, 4, 512, 3, 40),     # groups of 16 lanes: two-byte offsets
    (5120, 128, 8, 1024, 8, 25),    # groups of a whole warp
    (1024, 128, 4, 1024, 2, 30),    # g_q = d inside one warp, with outliers
    (2048, 64, 3, 512, 5, 33),
    (5120, 128, 4, 160, 0, 40),     # groups of five lanes: neither a power of two nor the token, crossing warps
    (5120, 128, 8, 640, 0, 25),
    (3584, 128, 4, 224, 0, 33),     # seven lanes
    (3584, 64, 3, 1792, 0, 21),     # 56 lanes: half a token
    (96, 32, 2, 96, 0, 9),
])
def test_family_matches_oracle(env, d, g, bits, qg, kg, T):
    X, R, _, _ = prefill_inputs(env, T, d, g, seed=3000 + d + bits + qg + kg)
    cfg = env.rac.CodecCfg(d, g, bits, 0, scale_mode=1, qgroup=qg, topk_group=kg)
    assert env.rac.rac_record_bytes(cfg) == env.orc.record_bytes(d, g, bits, 0, 1, qg, kg)
    rep, pay, xr = env.P.round_trip_case(cfg, X, ref_base=R)
    print(rep)
    # direct tokens mixed in, and the gain/bias reference
    rows = np.arange(T, dtype=np.int32)
    rows[1::3] = -1
    env.P.round_trip_case(cfg, X, ref_base=R, ref_row=torch.from_numpy(rows).to(env.dev))
    gain, bias = env.synth.predictor_gain_bias(d, 5, env.dev)
    env.P.round_trip_case(cfg, X, ref_base=R, gain=gain, bias=bias)


def test_family_ties_zero_groups_and_bad_offsets(env):
    d, g, T = 1024, 128, 12
    s = env.synth
    X = s.activations(T, d, s.channel_scale(d, 34, env.dev), s.generator(34, env.dev))
    # reference == X: every residual is zero, every |e| ties: the outliers are the k_g lowest offsets, scales 0
    cfg = env.rac.CodecCfg(d, g, 4, 0, scale_mode=1, qgroup=64, topk_group=3)
    rep, pay, xr = env.P.round_trip_case(cfg, X, ref_base=X)
    parts = env.orc.split_payload(pay, T, d, g, 4, 0, 1, 64, 3)
    assert not parts[4].any() and not parts[1].any() and not parts[6].any()
    assert np.array_equal(parts[5], np.tile(np.arange(3, dtype=np.uint8), (T, d // 64, 1)))
    assert torch.equal(xr, X)
    # a coarse grid of values: many equal magnitudes inside every group
    rng = np.random.default_rng(35)
    vals = (rng.integers(-6, 7, size=(T, d)) / 2).astype(np.float32)
    Xg = torch.from_numpy(vals).to(torch.bfloat16).to(env.dev)
    for kg in (1, 4):
        env.P.round_trip_case(env.rac.CodecCfg(d, g, 4, 0, scale_mode=1, qgroup=128, topk_group=kg), Xg, ref_base=None)
    # an offset outside its group: flagged, ignored, nothing else disturbed
    cfg = env.rac.CodecCfg(d, g, 4, 0, scale_mode=1, qgroup=32, topk_group=1)
    pay, st = env.P.gpu_encode(cfg, X, None, None, None, None, None, None)
    good, st0 = env.P.gpu_decode(cfg, pay, T, None, None, None, None, None, env.dev)
    bad = pay.copy().reshape(T, -1)
    goff = 4 * (d // g) + 2 * (d // 32) + d // 2
    keep = bad[3, goff + 5]
    bad[3, goff + 5] = 40
    xb, st1 = env.P.gpu_decode(cfg, bad.reshape(-1), T, None, None, None, None, None, env.dev)
    assert st0 == 0 and st1 == 16
    diff = (xb != good).nonzero().cpu().numpy()
    assert len(diff) == 1 and diff[0][0] == 3 and diff[0][1] == 5 * 32 + keep   # only the outlier that was dropped
    # configurations this build has no kernel for
    for bad_cfg in [env.rac.CodecCfg(5120, g, 4, 0, scale_mode=1, qgroup=5120, topk_group=1),   # a group wider than a warp
                    env.rac.CodecCfg(d, g, 4, 0, scale_mode=1, topk_group=9),
                    env.rac.CodecCfg(d, g, 8, 0),                                           # 8 bits: Eq. 8 family only
                    env.rac.CodecCfg(d, g, 4, 0, qgroup=64),                                # static table: g_q = g_a
                    env.rac.CodecCfg(d, g, 4, 0, scale_mode=1, qgroup=96),                  # does not divide d = 1024
                    env.rac.CodecCfg(5120, g, 4, 0, scale_mode=1, qgroup=160, topk_group=1),  # outliers need groups inside a warp
                    env.rac.CodecCfg(5120, g, 4, 0, scale_mode=1, qgroup=80),
                    env.rac.CodecCfg(d, g, 5, 0, scale_mode=1)]:
        assert env.rac.rac_record_bytes(bad_cfg) == 0


def test_family_random_configurations(env):
    """Forty seeded random members of the Eq. 8 family on small shapes: widths, both groupings, outlier counts,
    direct tokens, gathered rows and the gain/bias reference in random combination."""
    rng = np.random.default_rng(4242)
    s = env.synth
    tried = 0
    while tried < 40:
        d = int(rng.choice([64, 96, 256, 512, 1024, 2080, 3584, 4096]))
        g = int(rng.choice([32, 64, 128, 256]))
        if d % g:
            continue
        bits = int(rng.choice([2, 3, 4, 8]))
        qg = int(rng.choice([0, 32, 64, 128, 256, d]))
        kg = int(rng.choice([0, 0, 1, 2, 3, 4, 6, 8]))
        cfg = env.rac.CodecCfg(d, g, bits, 0, scale_mode=1, qgroup=qg, topk_group=kg)
        if env.rac.rac_record_bytes(cfg) == 0:
            assert env.orc.record_bytes(d, g, bits, 0, 1, qg, kg) == 0 or (qg or g) > 256 or d % (qg or g) or \
                not ((qg or g) == d or ((qg or g) & ((qg or g) - 1)) == 0)
            continue
        tried += 1
        T = int(rng.integers(1, 70))
        X, R, _, _ = prefill_inputs(env, T, d, g, seed=int(rng.integers(1 << 30)))
        kw = {}
        mode = int(rng.integers(0, 4))
        if mode == 1:      # some tokens coded directly
            rows = np.arange(T, dtype=np.int32)
            rows[rng.random(T) < 0.4] = -1
            kw["ref_row"] = torch.from_numpy(rows).to(env.dev)
        elif mode == 2:    # gathered rows
            kw["ref_row"] = torch.from_numpy(rng.integers(0, T, T).astype(np.int32)).to(env.dev)
        elif mode == 3:    # the per-channel transform of the reference
            kw["gain"], kw["bias"] = s.predictor_gain_bias(d, int(rng.integers(100)), env.dev)
        try:
            env.P.round_trip_case(cfg, X, ref_base=R, **kw)
        except AssertionError as e:
            raise AssertionError(f"{cfg!r} T={T} mode={mode}: {e}") from e


def test_static_random_configurations(env):
    """Thirty seeded random configurations of the static-table quantiser with per-token outliers on small shapes."""
    rng = np.random.default_rng(2424)
    s = env.synth
    tried = 0
    while tried < 30:
        d = int(rng.choice([32, 96, 256, 512, 1024, 2080, 3584, 4096, 8192]))
        g = int(rng.choice([32, 64, 128, 256, 1024]))
        if d % g:
            continue
        bits = int(rng.choice([2, 3, 4]))
        k = int(rng.choice([0, 1, 3, 8, 16]))
        if k > d:
            continue
        tried += 1
        T = int(rng.integers(1, 60))
        X, R, cal, calr = prefill_inputs(env, T, d, g, seed=int(rng.integers(1 << 30)), cal_T=64)
        kw = {}
        mode = int(rng.integers(0, 4))
        rows = None
        if mode == 1:
            rows = np.arange(T, dtype=np.int32)
            rows[rng.random(T) < 0.4] = -1
        elif mode == 2:
            rows = rng.integers(0, T, T).astype(np.int32)
        if rows is not None:
            kw["ref_row"] = torch.from_numpy(rows).to(env.dev)
        gb = {}
        if mode == 3:
            kw["gain"], kw["bias"] = s.predictor_gain_bias(d, int(rng.integers(100)), env.dev)
            gb = dict(gain=s.f16_bits(kw["gain"]), bias=s.f16_bits(kw["bias"]))
        step, inv = env.orc.calibrate(d, g, bits, s.bf16_bits(X), ref_base=s.bf16_bits(R), ref_row=rows, **gb)
        # a table row without calibration tokens is all zero ("code 0"): legal, and part of what is being tested
        cfg = env.rac.CodecCfg(d, g, bits, k)
        try:
            env.P.round_trip_case(cfg, X, ref_base=R, step=step, inv_step=inv, **kw)
        except AssertionError as e:
            raise AssertionError(f"{cfg!r} T={T} mode={mode}: {e}") from e


@pytest.mark.parametrize("k", [0, 8])
def test_tables_that_are_not_binary16_valued(env, k, monkeypatch):
    """Steps that binary16 cannot hold make code*step inexact in binary32.  Every reconstruction in the library takes
    fma(code, step, alpha*r + beta): the sender's pass, the streaming reconstruction and the one with a CTA barrier
    give the same bits, and the two-rounding evaluation of the oracle is at most one bf16 step away, rarely."""
    d, g, bits, T = 2048, 128, 4, 600
    X, R, cal, calr = prefill_inputs(env, T, d, g, seed=61)
    rng = np.random.default_rng(61)
    step = (0.03 + 0.02 * rng.random((2, d))).astype(np.float32)        # 24 significant bits
    assert np.any(step.astype(np.float16).astype(np.float32) != step)
    inv = (np.float32(1) / step).astype(np.float32)
    cfg = env.rac.CodecCfg(d, g, bits, k)
    P, dev = env.P, env.dev
    # a third of the tokens coded directly: they take row 1 of the table, which the streaming reconstruction keeps
    # as packed binary16 only when that is exact -- here it is not, so it has to read the row from memory
    rows_np = np.arange(T, dtype=np.int32)
    rows_np[rng.random(T) < 0.33] = -1
    rows = torch.from_numpy(rows_np).to(dev)
    pay, xs, st = P.gpu_encode_reconstruct(cfg, X, R, rows, None, None, P.to_dev(step, dev), P.to_dev(inv, dev))
    assert st == 0
    xr, st = P.gpu_decode(cfg, pay, T, R, rows, None, None, P.to_dev(step, dev), dev)
    assert st == 0 and torch.equal(xs, xr)
    # the reconstruction kernel with a CTA barrier serves the token-list calls: all tokens through a list
    toks = torch.arange(T, dtype=torch.int32, device=dev)
    cnt = torch.tensor([T], dtype=torch.int32, device=dev)
    xb = torch.empty_like(xr)
    stt = torch.zeros(1, dtype=torch.int32, device=dev)
    env.rac.rac_decode_reconstruct_list(cfg, torch.from_numpy(pay).to(dev), T, toks, cnt, R, T, rows, None, 0, None, None,
                                        P.to_dev(step, dev), xb, stt)
    torch.cuda.synchronize()
    assert int(stt.item()) == 0 and torch.equal(xb, xr)
    # row 0 exact in binary16, row 1 not, and the other way round: the two rows are handled independently
    for keep in (0, 1):
        mixed = step.copy()
        mixed[keep] = mixed[keep].astype(np.float16).astype(np.float32)
        minv = (np.float32(1) / mixed).astype(np.float32)
        pm, xm, st = P.gpu_encode_reconstruct(cfg, X, R, rows, None, None, P.to_dev(mixed, dev), P.to_dev(minv, dev))
        xd, st2 = P.gpu_decode(cfg, pm, T, R, rows, None, None, P.to_dev(mixed, dev), dev)
        assert st == 0 and st2 == 0 and torch.equal(xm, xd)
        om = env.orc.reconstruct(d, g, bits, k, pm, T, ref_base=env.synth.bf16_bits(R), ref_row=rows_np, step=mixed)
        exact_tokens = (rows_np >= 0) if keep == 0 else (rows_np < 0)
        assert np.array_equal(env.synth.bf16_bits(xd)[exact_tokens], om[exact_tokens])
    o = env.orc.reconstruct(d, g, bits, k, pay, T, ref_base=env.synth.bf16_bits(R), ref_row=rows_np, step=step)
    got = env.synth.bf16_bits(xr)
    diff = got != o
    assert diff.mean() < 1e-3
    of, gf = env.orc.bf16_to_f32(o[diff]), env.orc.bf16_to_f32(got[diff])
    assert np.all(np.abs(of - gf) <= np.maximum(np.abs(of), np.abs(gf)) * 2.0 ** -7)


def test_random_configurations_on_stressed_inputs(env):
    """600 seeded random cases over both quantisers with inputs pushed off the comfortable range: magnitudes 1e-3 and
    300 times the usual, a reference equal to the token, a constant reference row, an all-zero token, values on a
    quarter grid (exact ties everywhere); identity, direct, gathered and transformed references; 1 to 400 tokens."""
    s, rac, dev = env.synth, env.rac, env.dev
    master = np.random.default_rng(777)
    done = 0
    while done < 600:
        rng = np.random.default_rng(int(master.integers(1 << 40)))
        fam = rng.random() < 0.55
        d = int(rng.choice([32, 64, 96, 256, 512, 1024, 2080, 3584, 4096, 5120, 8192]))
        g = int(rng.choice([32, 64, 128, 256, 1024]))
        if d % g:
            continue
        T = int(rng.integers(1, 400 if d <= 2080 else 120))
        if fam:
            cfg = rac.CodecCfg(d, g, int(rng.choice([2, 3, 4, 8])), 0, scale_mode=1,
                               qgroup=int(rng.choice([0, 32, 64, 128, 256, 512, 1024, d, 96, 160, 224])), topk_group=int(rng.choice([0, 0, 1, 2, 3, 4, 7, 8])))
            if rac.rac_record_bytes(cfg) == 0:
                continue
        else:
            k = int(rng.choice([0, 1, 3, 8, 16]))
            if k > d:
                continue
            cfg = rac.CodecCfg(d, g, int(rng.choice([2, 3, 4])), k)
        done += 1
        X, R, _, _ = prefill_inputs(env, T, d, g, seed=int(rng.integers(1 << 30)), cal_T=8)
        kind = int(rng.integers(0, 7))
        if kind == 1:
            X, R = (X.float() * 1e-3).to(torch.bfloat16), (R.float() * 1e-3).to(torch.bfloat16)
        elif kind == 2:
            X, R = (X.float() * 300).to(torch.bfloat16), (R.float() * 300).to(torch.bfloat16)
        elif kind == 3:
            R = X.clone()
        elif kind == 4:
            R[int(rng.integers(0, T))] = 1.5
        elif kind == 5:
            X[int(rng.integers(0, T))] = 0
        elif kind == 6:
            X = torch.round(X.float() * 4).div(4).to(torch.bfloat16)
            R = torch.round(R.float() * 4).div(4).to(torch.bfloat16)
        mode = int(rng.integers(0, 4))
        kw, gb, rows = {}, {}, None
        if mode == 1:
            rows = np.arange(T, dtype=np.int32)
            rows[rng.random(T) < 0.4] = -1
        elif mode == 2:
            rows = rng.integers(0, T, T).astype(np.int32)
        if rows is not None:
            kw["ref_row"] = torch.from_numpy(rows).to(dev)
        if mode == 3:
            kw["gain"], kw["bias"] = s.predictor_gain_bias(d, int(rng.integers(100)), dev)
            gb = dict(gain=s.f16_bits(kw["gain"]), bias=s.f16_bits(kw["bias"]))
        if not fam:
            kw["step"], kw["inv_step"] = env.orc.calibrate(d, g, cfg.bits, s.bf16_bits(X), ref_base=s.bf16_bits(R),
                                                           ref_row=rows, **gb)
        try:
            env.P.round_trip_case(cfg, X, ref_base=R, **kw)
        except AssertionError as e:
            raise AssertionError(f"{cfg!r} T={T} mode={mode} kind={kind}: {e}") from e


@pytest.mark.parametrize("bits,kg,qg", [(4, 0, 0), (4, 1, 0), (8, 2, 0), (3, 0, 1024), (2, 1, 64)])
def test_scale_that_binary16_cannot_hold(env, bits, kg, qg):
    """Eq. 8 rounds the scale up in binary16; beyond 65504 it cannot, the scale sticks there and the codes clip --
    the one case in which the clamp of the Eq. 8 encoder does something (without it the kernel skips the clamp).
    Magnitudes of 1e5..1e7 with half of the tokens coded directly put many groups there; the rest of the groups,
    in the same warps, stay below."""
    d, g, T = 1024, 128, 150
    X, R, _, _ = prefill_inputs(env, T, d, g, seed=71)
    mag = 6e4 * ((1 << (bits - 1)) - 1)            # about Qmax * 65504: the border runs through the data
    X = (X.float() * mag).to(torch.bfloat16)
    R = (R.float() * mag).to(torch.bfloat16)
    rows = np.arange(T, dtype=np.int32)
    rows[::2] = -1
    cfg = env.rac.CodecCfg(d, g, bits, 0, scale_mode=1, qgroup=qg, topk_group=kg)
    rep, pay, xh = env.P.round_trip_case(cfg, X, ref_base=R, ref_row=torch.from_numpy(rows).to(env.dev))
    scales = env.orc.split_payload(pay, T, d, g, bits, 0, 1, qg, kg)[4]
    sat = (np.asarray(scales).reshape(-1) == 0x7bff).mean()
    assert 0.02 < sat < 0.98, sat           # saturated and ordinary groups side by side
