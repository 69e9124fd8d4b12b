"""Pins for the oracle's encode / reconstruct / calibrate (CPU only).

Nothing here re-types the oracle's formulas.  The checks are: closed forms of
the affine fit (Eq. 6), agreement with numpy's least squares, the zero-variance
rule, the error identity of Eq. 10 observed from inputs and outputs only, the
half-step bound of Eq. 11 outside the clip range and exact saturation inside
it, exhaustive rounding at every half-way point, and brute-force outlier
selection with crafted ties.
"""
import numpy as np
import pytest
import torch

from paper_2608_04991_b200 import synth


def bits_of(x):  # float array -> bf16 bits via torch (independent of the oracle's own rounding)
    return synth.bf16_bits(torch.as_tensor(np.asarray(x, np.float32)).to(torch.bfloat16))


def f16(bits):
    return np.asarray(bits, np.uint16).view(np.float16).astype(np.float64)


def flat_tables(d, step_val):
    step = np.full((2, d), step_val, np.float32)
    inv = (np.float32(1.0) / step).astype(np.float32)
    return step, inv


# ------------------------------------------------------------------ Eq. 6
def test_fit_reference_equal_to_x_gives_identity_and_zero_codes(orc):
    d, g, T = 256, 64, 5
    gen = synth.generator(10)
    X = synth.activations(T, d, synth.channel_scale(d, 0), gen)
    Xb = synth.bf16_bits(X)
    step, inv = flat_tables(d, 0.02)
    for bits, k in [(4, 0), (3, 0), (2, 0), (4, 4)]:
        payload = orc.encode(d, g, bits, k, Xb, ref_base=Xb, step=step, inv_step=inv)
        coef, codes, oi, ov = orc.split_payload(payload, T, d, g, bits, k)
        assert np.all((coef & 0xffff) == 0x3c00)      # alpha == 1.0
        assert np.all(f16(coef >> 16) == 0.0)         # beta == +-0
        assert not codes.any()                         # residual identically zero
        if k:
            # all |e| tie at zero: the k lowest channels win, values are zero
            assert np.array_equal(oi, np.tile(np.arange(k, dtype=np.uint16), (T, 1)))
            assert not (ov & 0x7fff).any()
        xh = orc.reconstruct(d, g, bits, k, payload, T, ref_base=Xb, step=step)
        assert np.array_equal(xh, Xb)


def test_fit_recovers_exact_affine_map(orc):
    # small-integer references and dyadic (a, b): X = a*R + b is exact in bf16, so the fit must return
    # exactly (a, b), the residual is zero and the round trip is the identity.
    rng = np.random.default_rng(11)
    d, g, T = 256, 64, 16
    J = d // g
    R = rng.integers(-8, 9, size=(T, d)).astype(np.float32)
    R[:, ::g] = 8.0  # make sure no group is constant
    R[:, 1::g] = -8.0
    a = rng.choice([0.75, 1.0, 1.25, 1.5, -0.5], size=(T, J)).astype(np.float32)
    b = rng.choice([-0.5, 0.0, 0.25, 2.0], size=(T, J)).astype(np.float32)
    X = np.repeat(a, g, axis=1) * R + np.repeat(b, g, axis=1)
    Xb, Rb = bits_of(X), bits_of(R)
    assert np.array_equal(orc.bf16_to_f32(Xb), X)  # exact by construction
    step, inv = flat_tables(d, 0.01)
    payload = orc.encode(d, g, 4, 0, Xb, ref_base=Rb, step=step, inv_step=inv)
    coef, codes, _, _ = orc.split_payload(payload, T, d, g, 4, 0)
    assert np.array_equal(f16(coef & 0xffff), a.astype(np.float64))
    assert np.array_equal(f16(coef >> 16), b.astype(np.float64))
    assert not codes.any()
    assert np.array_equal(orc.reconstruct(d, g, 4, 0, payload, T, ref_base=Rb, step=step), Xb)


def test_fit_zero_variance_and_missing_reference(orc):
    rng = np.random.default_rng(12)
    d, g, T = 128, 64, 4
    X = rng.standard_normal((T, d)).astype(np.float32)
    Xb = bits_of(X)
    Xv = orc.bf16_to_f32(Xb).astype(np.float64)
    mean = Xv.reshape(T, d // g, g).mean(axis=2)
    step, inv = flat_tables(d, 0.05)
    const = bits_of(np.full((T, d), 3.5, np.float32))
    neg = np.full(T, -1, np.int32)
    for kwargs in (dict(ref_base=const), dict(ref_base=None), dict(ref_base=const, ref_row=neg)):
        payload, dg = orc.encode(d, g, 4, 0, Xb, step=step, inv_step=inv, diag=True, **kwargs)
        coef, _, _, _ = orc.split_payload(payload, T, d, g, 4, 0)
        assert np.all((coef & 0x7fff) == 0)  # alpha = 0
        assert np.allclose(dg["beta"], mean, rtol=0, atol=1e-12)
        assert np.all(np.abs(f16(coef >> 16) - mean) <= np.abs(mean) * 2.0 ** -11 + 2.0 ** -25)


def test_fit_matches_library_least_squares_and_normal_equations(orc):
    rng = np.random.default_rng(13)
    for g in (32, 64, 128, 256):
        for _ in range(20):
            r = orc.bf16_to_f32(bits_of(rng.standard_normal(g) * rng.uniform(0.1, 30)))
            h = orc.bf16_to_f32(bits_of(rng.uniform(-2, 2) * r + rng.uniform(-1, 1) + 0.3 * rng.standard_normal(g)))
            a, b, hbar, rbar = orc.fit_group(h, r)
            A = np.stack([r.astype(np.float64), np.ones(g)], axis=1)
            sol = np.linalg.lstsq(A, h.astype(np.float64), rcond=None)[0]
            assert np.allclose([a, b], sol, rtol=1e-9, atol=1e-11)
            res = h.astype(np.float64) - (a * r.astype(np.float64) + b)
            scale = np.abs(h).sum() + 1.0
            assert abs(res.sum()) < 1e-10 * scale            # d/d(beta) = 0
            assert abs((res * r).sum()) < 1e-9 * scale * np.abs(r).max()  # d/d(alpha) = 0
            assert hbar == pytest.approx(h.astype(np.float64).mean(), abs=1e-12)
            assert rbar == pytest.approx(r.astype(np.float64).mean(), abs=1e-12)


def test_wire_coefficients_are_nearest_binary16(orc):
    d, g, T = 512, 128, 32
    gen = synth.generator(14)
    X = synth.activations(T, d, synth.channel_scale(d, 1), gen)
    R = synth.affine_noisy_reference(X, g, gen)
    step, inv = flat_tables(d, 0.02)
    payload, dg = orc.encode(d, g, 4, 0, synth.bf16_bits(X), ref_base=synth.bf16_bits(R), step=step, inv_step=inv,
                             diag=True)
    coef, _, _, _ = orc.split_payload(payload, T, d, g, 4, 0)
    want_a = dg["alpha"].astype(np.float16).view(np.uint16)  # numpy rounds binary64 -> binary16 in one step
    want_b = dg["beta"].astype(np.float16).view(np.uint16)
    assert np.array_equal(coef & 0xffff, want_a)
    assert np.array_equal(coef >> 16, want_b)
    # the fit is attenuated by the reference noise but sits near the drawn slope range
    a = f16(coef & 0xffff)
    assert 0.75 < a.min() and a.max() < 1.3


# ------------------------------------------------------------------ Eq. 8-11
@pytest.mark.parametrize("bits,topk", [(4, 0), (3, 0), (2, 0), (4, 8), (3, 8), (2, 8)])
def test_round_trip_error_identity_and_bounds(orc, bits, topk):
    d, g, T = 1024, 128, 48
    gen = synth.generator(20 + bits)
    scale = synth.channel_scale(d, 2)
    X = synth.activations(T, d, scale, gen)
    R = synth.affine_noisy_reference(X, g, gen)
    Xb, Rb = synth.bf16_bits(X), synth.bf16_bits(R)
    cal = synth.activations(256, d, scale, gen)
    calr = synth.affine_noisy_reference(cal, g, gen)
    # a tight 1.5-sigma clip so that saturation is exercised even after the outliers are taken out
    step, inv = orc.calibrate(d, g, bits, synth.bf16_bits(cal), ref_base=synth.bf16_bits(calr), clip_sigmas=1.5)
    assert np.all(step[0] > 0) and np.all(step[1] == 0)  # no direct tokens in the draw
    payload, dg = orc.encode(d, g, bits, topk, Xb, ref_base=Rb, step=step, inv_step=inv, diag=True)
    xh = orc.reconstruct(d, g, bits, topk, payload, T, ref_base=Rb, step=step)
    coef, codes, oi, ov = orc.split_payload(payload, T, d, g, bits, topk)
    qmax = (1 << (bits - 1)) - 1
    h = orc.bf16_to_f32(Xb).astype(np.float64)
    r = orc.bf16_to_f32(Rb).astype(np.float64)
    x_hat = orc.bf16_to_f32(xh).astype(np.float64)
    alpha = np.repeat(f16(coef & 0xffff), g, axis=1)
    beta = np.repeat(f16(coef >> 16), g, axis=1)
    e = h - (alpha * r + beta)  # Eq. 7 from the WIRE coefficients, in binary64
    assert np.allclose(dg["e"], e, rtol=0, atol=np.abs(h).max() * 2.0 ** -22)
    q = np.stack([orc.unpack_codes(codes[t], d, bits) for t in range(T)])
    assert q.min() >= -qmax and q.max() <= qmax  # reserved code never produced
    is_out = np.zeros((T, d), bool)
    if topk:
        is_out[np.arange(T)[:, None], oi.astype(np.int64)] = True
        assert np.all(q[is_out] == 0)  # E^d = E - O: dense value at an outlier position is zero
    # e_hat as the receiver sees it, from the payload alone
    e_hat = q * step[0].astype(np.float64)
    if topk:
        e_hat[np.arange(T)[:, None], oi.astype(np.int64)] = f16(ov)
    # Eq. 10: H - H_hat == E - E_hat, up to the final bf16 rounding of H_hat
    lhs = h - x_hat
    rhs = e - e_hat
    assert np.all(np.abs(lhs - rhs) <= np.abs(x_hat) * 2.0 ** -8 + 1e-30)
    # Eq. 11 with a static step: half a step inside the clip range, exact saturation outside
    s = step[0].astype(np.float64)[None, :]
    v = e / s
    inside = (np.abs(v) <= qmax + 0.5) & ~is_out
    assert np.all(np.abs(e - e_hat)[inside] <= 0.5 * s.repeat(T, 0)[inside] * (1 + 1e-6))
    clipped = (np.abs(v) > qmax + 0.5 + 1e-3) & ~is_out
    assert clipped.any()
    assert np.all(q[clipped] == (np.sign(v[clipped]) * qmax).astype(np.int64))
    if topk:
        # outliers are reproduced exactly: the receiver's value IS the stored binary16, which is the
        # nearest binary16 to the residual
        eo = dg["e"][is_out].astype(np.float64)
        assert np.array_equal(f16(ov).reshape(-1), eo.astype(np.float16).astype(np.float64))
        # and they are the k largest magnitudes of the token (strictly larger than every dense value
        # except for exact ties)
        ae = np.abs(dg["e"])
        kth = np.where(is_out, ae, np.inf).min(axis=1)
        assert np.all(np.where(is_out, 0, ae).max(axis=1) <= kth)


def test_step_zero_means_code_zero_and_direct_row_is_used(orc):
    d, g, T = 128, 64, 6
    rng = np.random.default_rng(30)
    Xb = bits_of(rng.standard_normal((T, d)))
    Rb = bits_of(rng.standard_normal((T, d)))
    step = np.zeros((2, d), np.float32)
    step[0, ::2] = 0.25          # referenced tokens: every second channel coded
    step[1, :] = 0.5             # direct tokens: coarser table
    inv = np.where(step > 0, 1.0 / np.where(step > 0, step, 1), 123.0).astype(np.float32)  # garbage where step==0
    ref_row = np.array([0, -1, 2, -1, 4, 5], np.int32)
    payload = orc.encode(d, g, 4, 0, Xb, ref_base=Rb, ref_row=ref_row, step=step, inv_step=inv)
    coef, codes, _, _ = orc.split_payload(payload, T, d, g, 4, 0)
    q = np.stack([orc.unpack_codes(codes[t], d, 4) for t in range(T)])
    for t in range(T):
        if ref_row[t] >= 0:
            assert not q[t, 1::2].any() and q[t, ::2].any()
        else:
            assert np.all((coef[t] & 0x7fff) == 0)  # alpha = 0 for direct tokens
            assert np.count_nonzero(q[t]) > d // 4
    xh = orc.reconstruct(d, g, 4, 0, payload, T, ref_base=Rb, ref_row=ref_row, step=step)
    h = orc.bf16_to_f32(Xb).astype(np.float64)
    err = np.abs(h - orc.bf16_to_f32(xh))
    direct = ref_row < 0
    assert np.all(err[direct] <= 0.25 + np.abs(h[direct]) * 2.0 ** -8)  # half of the direct-row step


def test_rounding_is_half_to_even_at_every_boundary(orc):
    # reference constant -> alpha = 0, beta = mean(h); choose h so that mean is 0 and e = h exactly.
    # With step = 1 the scaled value is e itself: put every n + 0.5 in the input and read the codes.
    for bits in (2, 3, 4):
        qmax = (1 << (bits - 1)) - 1
        halves = np.arange(-qmax - 2, qmax + 2) + 0.5
        vals = np.concatenate([halves, -halves])            # symmetric -> zero mean
        d = g = 64
        row = np.zeros(d, np.float32)
        row[:vals.size] = vals
        assert row.sum() == 0 and vals.size <= d
        Xb = bits_of(row[None, :])
        step, inv = flat_tables(d, 1.0)
        payload = orc.encode(d, g, bits, 0, Xb, step=step, inv_step=inv)
        coef, codes, _, _ = orc.split_payload(payload, 1, d, g, bits, 0)
        assert coef[0, 0] & 0x7fffffff == 0
        q = orc.unpack_codes(codes[0], d, bits)
        want = np.clip(np.round(row), -qmax, qmax).astype(np.int32)  # numpy's round is half-to-even
        assert np.array_equal(q, want)


# ------------------------------------------------------------------ outliers
def test_outliers_brute_force_and_ties_to_lower_index(orc):
    rng = np.random.default_rng(40)
    d, g, T, k = 128, 64, 64, 8
    # direct coding with zero-mean groups of small integers/4 -> plenty of exact ties in |e|
    vals = rng.integers(-12, 13, size=(T, d)).astype(np.float32) / 4
    vals -= vals.reshape(T, d // g, g).mean(axis=2).repeat(g, axis=1)
    Xb = bits_of(vals)
    step, inv = flat_tables(d, 0.25)
    payload, dg = orc.encode(d, g, 4, k, Xb, step=step, inv_step=inv, diag=True)
    _, _, oi, ov = orc.split_payload(payload, T, d, g, 4, k)
    ties_seen = 0
    for t in range(T):
        e = dg["e"][t]
        # brute force: stable sort by descending magnitude keeps the lower index first among equals
        order = sorted(range(d), key=lambda c: (-abs(float(e[c])), c))[:k]
        assert list(oi[t]) == sorted(order)
        assert np.all(np.diff(oi[t].astype(int)) > 0)
        kth = abs(float(e[order[-1]]))
        ties_seen += int(np.sum(np.abs(e) == kth) > 1)
        assert np.array_equal(f16(ov[t]), e[oi[t].astype(int)].astype(np.float16).astype(np.float64))
    assert ties_seen > T // 2  # the tie rule is really exercised


def test_reconstruct_reports_reserved_code(orc):
    d, g = 64, 64
    step, _ = flat_tables(d, 0.5)
    rec = orc.record_bytes(d, g, 4, 0)
    payload = np.zeros(rec, np.uint8)
    payload[4] = 0x08  # channel 0 carries -8, which the encoder never emits
    xh, status = orc.reconstruct(d, g, 4, 0, payload, 1, step=step, return_status=True)
    assert status & 2
    assert orc.bf16_to_f32(xh)[0, 0] == -4.0 and not orc.bf16_to_f32(xh)[0, 1:].any()


# ------------------------------------------------------------------ forced coefficients, predictor stand-in
def test_forced_coefficients_and_gain_bias_transform(orc):
    d, g, T = 256, 128, 8
    gen = synth.generator(50)
    X = synth.activations(T, d, synth.channel_scale(d, 3), gen)
    prev = synth.activations(T, d, synth.channel_scale(d, 3), gen)
    gain, bias = synth.predictor_gain_bias(d, 0)
    Xb, Pb = synth.bf16_bits(X), synth.bf16_bits(prev)
    gb, bb = synth.f16_bits(gain), synth.f16_bits(bias)
    step, inv = flat_tables(d, 0.1)
    # transform applied inside == transform applied outside with torch's own bf16 rounding
    R_outside = (gain.float() * prev.float() + bias.float()).to(torch.bfloat16)
    p_in = orc.encode(d, g, 3, 0, Xb, ref_base=Pb, gain=gb, bias=bb, step=step, inv_step=inv)
    p_out = orc.encode(d, g, 3, 0, Xb, ref_base=synth.bf16_bits(R_outside), step=step, inv_step=inv)
    # float32 multiply-add without fusion can differ from fmaf by one rounding before the bf16 cast;
    # accept the rare double-rounding difference but require near-total agreement
    assert np.mean(p_in != p_out) < 0.01
    x_in = orc.reconstruct(d, g, 3, 0, p_in, T, ref_base=Pb, gain=gb, bias=bb, step=step)
    err = np.abs(orc.bf16_to_f32(x_in).astype(np.float64) - orc.bf16_to_f32(Xb))
    # forcing the coefficients the encoder chose itself changes nothing
    coef, _, _, _ = orc.split_payload(p_in, T, d, g, 3, 0)
    p_forced = orc.encode(d, g, 3, 0, Xb, ref_base=Pb, gain=gb, bias=bb, step=step, inv_step=inv,
                          forced_coef=coef.reshape(-1).copy())
    assert np.array_equal(p_forced, p_in)
    # forcing alpha=0, beta=0 codes X directly: error bounded by clip or half a step
    zero = np.zeros(T * (d // g), np.uint32)
    p_zero = orc.encode(d, g, 3, 0, Xb, ref_base=Pb, gain=gb, bias=bb, step=step, inv_step=inv, forced_coef=zero)
    x_zero = orc.bf16_to_f32(orc.reconstruct(d, g, 3, 0, p_zero, T, ref_base=Pb, gain=gb, bias=bb, step=step))
    h = orc.bf16_to_f32(Xb)
    small = np.abs(h) <= 3.5 * 0.1
    assert np.all(np.abs(h - x_zero)[small] <= 0.05 + 2.0 ** -8 * np.abs(h[small]))
    assert err.shape == (T, d)


def test_thread_count_does_not_change_the_payload(orc):
    d, g, T = 256, 64, 37
    gen = synth.generator(60)
    X = synth.activations(T, d, synth.channel_scale(d, 4), gen)
    R = synth.affine_noisy_reference(X, g, gen)
    step, inv = flat_tables(d, 0.02)
    a = orc.encode(d, g, 4, 8, synth.bf16_bits(X), ref_base=synth.bf16_bits(R), step=step, inv_step=inv, nthreads=1)
    b = orc.encode(d, g, 4, 8, synth.bf16_bits(X), ref_base=synth.bf16_bits(R), step=step, inv_step=inv, nthreads=4)
    assert np.array_equal(a, b)
    xa = orc.reconstruct(d, g, 4, 8, a, T, ref_base=synth.bf16_bits(R), step=step, nthreads=1)
    xb = orc.reconstruct(d, g, 4, 8, a, T, ref_base=synth.bf16_bits(R), step=step, nthreads=3)
    assert np.array_equal(xa, xb)


def test_calibrated_step_is_three_sigma_rounded_up(orc):
    d, g, bits, T = 256, 128, 4, 512
    gen = synth.generator(70)
    scale = synth.channel_scale(d, 5)
    X = synth.activations(T, d, scale, gen)
    R = synth.affine_noisy_reference(X, g, gen)
    step, inv = orc.calibrate(d, g, bits, synth.bf16_bits(X), ref_base=synth.bf16_bits(R))
    # independent estimate of the residual RMS with numpy least squares per (token, group)
    h = X.float().numpy().astype(np.float64).reshape(T, d // g, g)
    r = R.float().numpy().astype(np.float64).reshape(T, d // g, g)
    rc = r - r.mean(-1, keepdims=True)
    hc = h - h.mean(-1, keepdims=True)
    a = (rc * hc).sum(-1, keepdims=True) / (rc * rc).sum(-1, keepdims=True)
    b = h.mean(-1, keepdims=True) - a * r.mean(-1, keepdims=True)
    # the residual is taken with the coefficients as they travel (binary16): on a heavy channel the
    # rounding of alpha alone moves the residual by a visible amount
    a16 = a.astype(np.float16).astype(np.float64)
    b16 = b.astype(np.float16).astype(np.float64)
    e = h - (a16 * r + b16)
    sigma = np.sqrt((e ** 2).mean(axis=0)).reshape(d)
    want = 3 * sigma / 7
    # step is a binary16 value, >= the target (up to the small effect of coefficient rounding) and within one ulp
    assert np.array_equal(step[0], step[0].astype(np.float16).astype(np.float32))
    assert np.all(step[0] >= want * (1 - 2e-3))
    assert np.all(step[0] <= want * (1 + 2e-3) + np.spacing(step[0].astype(np.float16)).astype(np.float64))
    assert np.array_equal(inv[0], (np.float32(1) / step[0]).astype(np.float32))
    assert not step[1].any() and not inv[1].any()


def test_calibration_with_shared_coefficient_words(orc):
    """Residuals taken with words that come from outside (Eq. 6 over several positions): an independent numpy
    evaluation with hand-picked words, and the reduction to the per-token form when the words are the tokens' own."""
    d, g, bits, T = 128, 32, 3, 96
    J = d // g
    gen = synth.generator(71)
    X = synth.activations(T, d, synth.channel_scale(d, 6), gen)
    R = synth.affine_noisy_reference(X, g, gen)
    Xb, Rb = synth.bf16_bits(X), synth.bf16_bits(R)
    rows = np.arange(T, dtype=np.int32)
    rows[10:20] = -1                                                     # direct tokens: table row 1, r = 0
    rng = np.random.default_rng(5)
    a16 = rng.choice(np.array([0.5, 0.75, 1.0, 1.25], np.float16), (T, J))
    b16 = rng.choice(np.array([-0.25, 0.0, 0.125], np.float16), (T, J))
    words = (a16.view(np.uint16).astype(np.uint32) | (b16.view(np.uint16).astype(np.uint32) << 16))
    step, inv = orc.calibrate(d, g, bits, Xb, ref_base=Rb, ref_row=rows, shared_coef=words)
    h = X.float().numpy().astype(np.float64)
    r = R.float().numpy().astype(np.float64)
    r[rows < 0] = 0.0
    # binary32 fma and subtraction, as Eq. 7 is evaluated: emulate with float64 then round (exact for these inputs'
    # products: bf16 x binary16 has <= 19 significant bits; the sum is rounded once to binary32)
    rt = (np.repeat(a16.astype(np.float64), g, axis=1) * r + np.repeat(b16.astype(np.float64), g, axis=1)).astype(np.float32)
    e = (X.float().numpy() - rt).astype(np.float64)
    for row, mask in ((0, rows >= 0), (1, rows < 0)):
        sigma = np.sqrt((e[mask] ** 2).mean(axis=0))
        want = 3.0 * sigma / 3.0                                         # Qmax = 3 for 3-bit codes
        ulp = np.spacing(step[row].astype(np.float16)).astype(np.float64)
        assert np.all(step[row] >= want * (1 - 1e-6)) and np.all(step[row] <= want * (1 + 1e-6) + ulp)
        assert np.array_equal(inv[row], (np.float32(1) / step[row]).astype(np.float32))
    # the tokens' own wire words reproduce the per-token calibration exactly
    _, dg = orc.encode(d, g, bits, 0, Xb, ref_base=Rb, ref_row=rows, step=step, inv_step=inv, diag=True)
    pay = orc.encode(d, g, bits, 0, Xb, ref_base=Rb, ref_row=rows, step=step, inv_step=inv)
    own = pay.reshape(T, -1)[:, :4 * J].copy().view(np.uint32).reshape(T, J)
    s0, i0 = orc.calibrate(d, g, bits, Xb, ref_base=Rb, ref_row=rows)
    s1, i1 = orc.calibrate(d, g, bits, Xb, ref_base=Rb, ref_row=rows, shared_coef=own)
    assert np.array_equal(s0, s1) and np.array_equal(i0, i1)


# ------------------------------------------------------------------ Eq. 8 as printed: dynamic per-group scale
@pytest.mark.parametrize("bits,topk", [(4, 0), (3, 0), (2, 0), (4, 8)])
def test_dynamic_scale_never_clips_and_rounds_up(orc, bits, topk):
    d, g, T = 512, 64, 40
    J = d // g
    gen = synth.generator(80 + bits)
    X = synth.activations(T, d, synth.channel_scale(d, 6), gen)
    R = synth.affine_noisy_reference(X, g, gen)
    Xb, Rb = synth.bf16_bits(X), synth.bf16_bits(R)
    payload = orc.encode(d, g, bits, topk, Xb, ref_base=Rb, scale_mode=1)
    assert payload.size == T * orc.record_bytes(d, g, bits, topk, 1)
    xh = orc.reconstruct(d, g, bits, topk, payload, T, ref_base=Rb, scale_mode=1)
    coef, codes, oi, ov, scale = orc.split_payload(payload, T, d, g, bits, topk, 1)
    qmax = (1 << (bits - 1)) - 1
    h = orc.bf16_to_f32(Xb).astype(np.float64)
    r = orc.bf16_to_f32(Rb).astype(np.float64)
    alpha = np.repeat(f16(coef & 0xffff), g, axis=1)
    beta = np.repeat(f16(coef >> 16), g, axis=1)
    e = h - (alpha * r + beta)                         # Eq. 7 from the wire coefficients
    q = np.stack([orc.unpack_codes(codes[t], d, bits) for t in range(T)])
    is_out = np.zeros((T, d), bool)
    if topk:
        is_out[np.arange(T)[:, None], oi.astype(np.int64)] = True
        assert np.all(q[is_out] == 0)
    s = f16(scale)                                     # [T, J]
    s_full = np.repeat(s, g, axis=1)
    dense_max = np.where(is_out, 0, np.abs(e)).reshape(T, J, g).max(axis=2)
    # RoundUp_wire: the stored scale is >= max|E^d|/Qmax (so nothing clips) and the binary16 below it is not
    want = dense_max / qmax
    assert np.all(s >= want * (1 - 1e-6))
    below = np.nextafter(s.astype(np.float16), np.float16(-np.inf)).astype(np.float64)
    assert np.all((below < want * (1 + 1e-6)) | (s == 0))
    # Eq. 11: every dense value within half a scale step, no exceptions, and no reserved code
    e_hat = q * s_full
    assert q.min() >= -qmax and q.max() <= qmax
    assert np.all(np.abs(e - e_hat)[~is_out] <= 0.5 * s_full[~is_out] * (1 + 1e-5) + 1e-12)
    # the largest dense magnitude of every group sits at the end of the range
    amax = np.abs(q).reshape(T, J, g).max(axis=2)
    assert np.all((amax == qmax) | (dense_max == 0))
    # Eq. 10 with the receiver's view
    if topk:
        e_hat[np.arange(T)[:, None], oi.astype(np.int64)] = f16(ov)
    x_hat = orc.bf16_to_f32(xh).astype(np.float64)
    assert np.all(np.abs((h - x_hat) - (e - e_hat)) <= np.abs(x_hat) * 2.0 ** -8 + 1e-30)
    # Eq. 12: the residual range is far below the direct-coding range on this workload
    direct_max = np.abs(h - h.reshape(T, J, g).mean(axis=2).repeat(g, axis=1)).reshape(T, J, g).max(axis=2)
    assert np.median(dense_max / direct_max) < 0.5


def test_dynamic_scale_zero_group_marker_and_identity(orc):
    d, g, T = 256, 64, 6
    gen = synth.generator(90)
    X = synth.activations(T, d, synth.channel_scale(d, 7), gen)
    Xb = synth.bf16_bits(X)
    payload = orc.encode(d, g, 4, 0, Xb, ref_base=Xb, scale_mode=1)       # reference == X: residual zero everywhere
    coef, codes, _, _, scale = orc.split_payload(payload, T, d, g, 4, 0, 1)
    assert not scale.any() and not codes.any() and np.all(coef == 0x3c00)
    assert np.array_equal(orc.reconstruct(d, g, 4, 0, payload, T, ref_base=Xb, scale_mode=1), Xb)
    # 4-bit values stay 25 % of raw; scales add 2 bytes per group
    assert orc.record_bytes(4096, 128, 4, 0, 1) - orc.record_bytes(4096, 128, 4, 0, 0) == 64
    # one group with a single non-zero residual: its scale is that value / Qmax rounded up, code +-Qmax
    row = np.zeros((1, d), np.float32)
    row[0, 5] = 3.0
    row[0, 6] = -3.0                                                     # zero mean: beta = 0 with no reference
    p2 = orc.encode(d, g, 4, 0, bits_of(row), scale_mode=1)
    coef, codes, _, _, scale = orc.split_payload(p2, 1, d, g, 4, 0, 1)
    q = orc.unpack_codes(codes[0], d, 4)
    assert q[5] == 7 and q[6] == -7 and np.count_nonzero(q) == 2
    assert scale[0, 0] == np.float16(np.nextafter(np.float16(3.0 / 7), np.float16(1))).view(np.uint16) or \
        f16(scale[0, :1])[0] >= 3.0 / 7
    assert not scale[0, 1:].any()


# ------------------------------------------------------------------ the rest of the quantiser family (Sec. IV-C)
def test_family_record_by_hand(orc):
    """One token worked by hand: d = 8, one alignment group, no reference, zero-mean values (so beta = 0 and
    e = x), quantisation groups of 4, one outlier per group, 4-bit codes."""
    x = np.array([[8, -8, 1, -1, 0.5, -0.5, 0, 0]], np.float32)
    pay = orc.encode(8, 8, 4, 0, bits_of(x), scale_mode=1, qgroup=4, topk_group=1)
    # group 0: |8| ties with |-8| -> the lower channel (offset 0) is the outlier, 8.0 = 0x4800; the dense maximum
    # is still 8: scale = RoundUp16(8/7 = 1.142857..) = 1171 * 2^-10 = 0x3c93; codes 0, -7, round(1/1.1436) = 1, -1.
    # group 1: outlier offset 0, 0.5 = 0x3800; scale = RoundUp16(0.5/7) = 1171 * 2^-14 = 0x2c93; codes 0, -7, 0, 0.
    want = bytes([0, 0, 0, 0,                   # alpha = 0, beta = 0
                  0x93, 0x3c, 0x93, 0x2c,       # two scales
                  0x90, 0xf1, 0x90, 0x00,       # codes, two per byte, low nibble first
                  0, 0,                         # in-group offsets
                  0x00, 0x48, 0x00, 0x38])      # outlier values
    assert pay.size == 32 and pay.tobytes() == want + bytes(32 - len(want))
    xh = orc.reconstruct(8, 8, 4, 0, pay, 1, scale_mode=1, qgroup=4, topk_group=1)
    s0, s1 = 1171 * 2.0 ** -10, 1171 * 2.0 ** -14
    exact = np.array([8, -7 * s0, s0, -s0, 0.5, -7 * s1, 0, 0])
    assert np.array_equal(xh[0], bits_of(exact.astype(np.float32)[None])[0])


@pytest.mark.parametrize("bits,g,qg,kg", [
    (4, 64, 64, 1), (4, 64, 64, 2), (8, 64, 64, 1), (4, 128, 32, 4), (4, 32, 128, 2), (3, 64, 256, 3),
    (8, 64, 0, 0), (8, 64, 512, 0), (4, 64, 512, 0), (2, 128, 512, 0), (4, 128, 16, 1),
    (4, 64, 512, 3), (8, 128, 512, 6),     # groups of more than 256 channels: two-byte offsets
])
def test_family_outliers_per_group_and_token_scale(orc, bits, g, qg, kg):
    d, T = 512, 24
    q_g = qg or g
    Jq = d // q_g
    gen = synth.generator(300 + bits + q_g + kg)
    X = synth.activations(T, d, synth.channel_scale(d, 8), gen)
    R = synth.affine_noisy_reference(X, g, gen)
    Xb, Rb = synth.bf16_bits(X), synth.bf16_bits(R)
    kw = dict(scale_mode=1, qgroup=qg, topk_group=kg)
    pay = orc.encode(d, g, bits, 0, Xb, ref_base=Rb, **kw)
    # record size from the layout, typed out
    ng = Jq * kg
    off_bytes = 2 if q_g > 256 else 1
    raw = 4 * (d // g) + (2 * Jq + 3) // 4 * 4 + d * bits // 8 + (ng * off_bytes + 1) // 2 * 2 + 2 * ng
    assert orc.record_bytes(d, g, bits, 0, 1, qg, kg) == (raw + 15) // 16 * 16 == pay.size // T
    parts = orc.split_payload(pay, T, d, g, bits, 0, 1, qg, kg)
    coef, codes, scale = parts[0], parts[1], parts[4]
    assert scale.shape == (T, Jq)
    qmax = (1 << (bits - 1)) - 1
    h = orc.bf16_to_f32(Xb).astype(np.float64)
    r = orc.bf16_to_f32(Rb).astype(np.float64)
    e = h - (np.repeat(f16(coef & 0xffff), g, axis=1) * r + np.repeat(f16(coef >> 16), g, axis=1))
    e32 = e.astype(np.float32)   # the residual is a binary32 value: ranking uses its bits
    q = np.stack([orc.unpack_codes(codes[t], d, bits) for t in range(T)])
    is_out = np.zeros((T, d), bool)
    e_hat_out = np.zeros((T, d))
    if kg:
        goff, gval = parts[5], parts[6]
        eg = np.abs(e32).reshape(T, Jq, q_g)
        # brute force: stable sort by decreasing magnitude keeps the lower channel first among equals
        order = np.argsort(-eg, axis=2, kind="stable")[:, :, :kg]
        want_off = np.sort(order, axis=2)
        assert np.array_equal(goff.astype(np.int64), want_off)
        chan = want_off + (np.arange(Jq) * q_g)[None, :, None]
        tt = np.arange(T)[:, None, None]
        is_out[tt, chan] = True
        want_val = e32[tt, chan].astype(np.float16)      # numpy's own round-to-nearest-even conversion
        assert np.array_equal(gval, want_val.view(np.uint16))
        e_hat_out[tt, chan] = want_val.astype(np.float64)
        assert np.all(q[is_out] == 0)
    s = f16(scale)
    s_full = np.repeat(s, q_g, axis=1)
    dense_max = np.where(is_out, 0, np.abs(e)).reshape(T, Jq, q_g).max(axis=2)
    want = dense_max / qmax
    assert np.all(s >= want * (1 - 1e-6))
    below = np.nextafter(s.astype(np.float16), np.float16(-np.inf)).astype(np.float64)
    assert np.all((below < want * (1 + 1e-6)) | (s == 0))
    e_hat = q * s_full
    assert q.min() >= -qmax and q.max() <= qmax
    assert np.all(np.abs(e - e_hat)[~is_out] <= 0.5 * s_full[~is_out] * (1 + 1e-5) + 1e-12)
    assert np.all((np.abs(q).reshape(T, Jq, q_g).max(axis=2) == qmax) | (dense_max == 0))
    # Eq. 10 / Eq. 9 with the outliers restored
    e_hat = np.where(is_out, e_hat_out, e_hat)
    xh = orc.bf16_to_f32(orc.reconstruct(d, g, bits, 0, pay, T, ref_base=Rb, **kw)).astype(np.float64)
    assert np.all(np.abs((h - xh) - (e - e_hat)) <= np.abs(xh) * 2.0 ** -8 + 1e-30)
    # taking outliers out can only lower a group's scale
    if kg:
        s_plain = f16(orc.split_payload(orc.encode(d, g, bits, 0, Xb, ref_base=Rb, scale_mode=1, qgroup=qg),
                                        T, d, g, bits, 0, 1, qg, 0)[4])
        assert np.all(s <= s_plain) and np.mean(s < s_plain) > 0.5


def test_family_token_scale_is_the_token_maximum_and_rejections(orc):
    d, g, T = 256, 64, 5
    gen = synth.generator(77)
    X = synth.activations(T, d, synth.channel_scale(d, 9), gen)
    Xb = synth.bf16_bits(X)
    pay = orc.encode(d, g, 8, 0, Xb, scale_mode=1, qgroup=d)
    coef, codes, _, _, scale = orc.split_payload(pay, T, d, g, 8, 0, 1, d, 0)
    assert scale.shape == (T, 1)
    q = np.stack([orc.unpack_codes(codes[t], d, 8) for t in range(T)])
    assert np.all(np.abs(q).max(axis=1) == 127)          # one scale per token: exactly the token's largest |e| is at the end
    assert np.array_equal(codes.view(np.int8).astype(np.int32), q)   # 8-bit codes are plain signed bytes
    # offsets are one byte up to g_q = 256 and two beyond: one more byte per outlier in the record
    r256 = orc.encode(d, g, 4, 0, Xb, scale_mode=1, qgroup=d, topk_group=2).size // T
    assert r256 == (4 * (d // g) + 4 + d // 2 + 2 + 4 + 15) // 16 * 16
    r512 = orc.encode(512, g, 4, 0, np.zeros((1, 512), np.uint16), scale_mode=1, qgroup=512, topk_group=2).size
    assert r512 == (4 * (512 // g) + 4 + 512 // 2 + 4 + 4 + 15) // 16 * 16
    with pytest.raises(ValueError):
        orc.encode(d, g, 4, 0, Xb, scale_mode=1, qgroup=d, topk_group=d + 1)    # more outliers than channels in a group
    with pytest.raises(ValueError):
        orc.encode(d, g, 4, 2, Xb, scale_mode=1, topk_group=1)              # one outlier rule at a time
    with pytest.raises(ValueError):
        orc.encode(d, g, 4, 0, Xb, step=flat_tables(d, 0.1)[0], inv_step=flat_tables(d, 0.1)[1], qgroup=32)   # static table: g_q = g_a
    with pytest.raises(ValueError):
        orc.reconstruct(d, g, 4, 0, _bad_offset_payload(orc, d, g), 1, scale_mode=1, qgroup=32, topk_group=1)


def _bad_offset_payload(orc, d, g):
    pay = orc.encode(d, g, 4, 0, np.zeros((1, d), np.uint16), scale_mode=1, qgroup=32, topk_group=1)
    J, Jq = d // g, d // 32
    pay[4 * J + 2 * Jq + d // 2] = 32      # first in-group offset: 32 is outside a group of 32
    return pay


# ------------------------------------------------------------------ Eq. 6 over several fitting positions
def test_segment_fit_matches_library_least_squares_and_single_token_case(orc):
    d, g, T = 256, 64, 37
    J = d // g
    gen = synth.generator(410)
    X = synth.activations(T, d, synth.channel_scale(d, 11), gen)
    R = synth.affine_noisy_reference(X, g, gen)
    Xb, Rb = synth.bf16_bits(X), synth.bf16_bits(R)
    seg_off = np.array([0, 1, 9, 9, 30, 37], np.int32)            # a single token, an empty segment, longer ones
    coef, dg = orc.fit_segments(d, g, Xb, seg_off, ref_base=Rb, diag=True)
    h = orc.bf16_to_f32(Xb).astype(np.float64)
    r = orc.bf16_to_f32(Rb).astype(np.float64)
    for k in range(len(seg_off) - 1):
        t0, t1 = seg_off[k], seg_off[k + 1]
        for j in range(J):
            hh = h[t0:t1, j * g:(j + 1) * g].reshape(-1)
            rr = r[t0:t1, j * g:(j + 1) * g].reshape(-1)
            if hh.size == 0:
                assert coef[k, j] == 0                            # nothing to fit: alpha = 0, beta = 0
                continue
            A = np.stack([rr, np.ones_like(rr)], axis=1)          # the Frobenius problem of Eq. 6, solved by numpy
            (a, b), *_ = np.linalg.lstsq(A, hh, rcond=None)
            assert abs(dg["alpha"][k, j] - a) <= 1e-9 * max(1.0, abs(a))
            assert abs(dg["beta"][k, j] - b) <= 1e-9 * max(1.0, abs(b))
            assert coef[k, j] & 0xffff == np.float16(dg["alpha"][k, j]).view(np.uint16)
            assert coef[k, j] >> 16 == np.float16(dg["beta"][k, j]).view(np.uint16)
    # a segment of one token is the per-token fit
    per_tok = orc.split_payload(orc.encode(d, g, 4, 0, Xb[:1], ref_base=Rb[:1], scale_mode=1), 1, d, g, 4, 0, 1)[0]
    assert np.array_equal(coef[0], per_tok[0])
    # no reference at all: alpha = 0, beta = the mean over all positions of the segment
    c2, d2 = orc.fit_segments(d, g, Xb, seg_off, diag=True)
    assert not (c2 & 0x7fff).any()
    assert np.allclose(d2["beta"][3], h[9:30].reshape(21, J, g).mean(axis=(0, 2)), rtol=0, atol=1e-12)
    # a pooled fit is never better than per-token fits on its own tokens, and equal when one map generated them all
    a_true, b_true = 1.25, -0.5
    Rc = synth.activations(8, d, synth.channel_scale(d, 12), gen)
    Xc = (a_true * Rc.float() + b_true)
    cc, dc = orc.fit_segments(d, g, synth.bf16_bits(Xc.to(torch.bfloat16)), np.array([0, 8], np.int32),
                              ref_base=synth.bf16_bits(Rc), diag=True)
    assert np.allclose(dc["alpha"], a_true, atol=2e-3) and np.allclose(dc["beta"], b_true, atol=2e-2)


@pytest.mark.parametrize("mode", [dict(scale_mode=0, bits=4, topk=8), dict(scale_mode=1, bits=4, topk=0, topk_group=1),
                                  dict(scale_mode=1, bits=8, topk=0, qgroup=512)])
def test_shared_coefficients_leave_the_record_and_round_trip(orc, mode):
    d, g, T = 512, 64, 40
    J = d // g
    gen = synth.generator(420)
    X = synth.activations(T, d, synth.channel_scale(d, 13), gen)
    R = synth.affine_noisy_reference(X, g, gen)
    Xb, Rb = synth.bf16_bits(X), synth.bf16_bits(R)
    bits, topk = mode["bits"], mode["topk"]
    kw = {k: v for k, v in mode.items() if k not in ("bits", "topk")}
    seg_off = np.array([0, 8, 8, 25, 40], np.int32)
    coef = orc.fit_segments(d, g, Xb, seg_off, ref_base=Rb)
    seg_of = np.repeat(np.arange(len(seg_off) - 1), np.diff(seg_off))
    per_tok = np.ascontiguousarray(coef[seg_of])                  # uint32[T, J]
    step = inv = None
    if kw["scale_mode"] == 0:
        step, inv = orc.calibrate(d, g, bits, Xb, ref_base=Rb)
    # the record shrinks by exactly the coefficient words (up to the 16-byte padding)
    r0 = orc.record_bytes(d, g, bits, topk, kw["scale_mode"], kw.get("qgroup", 0), kw.get("topk_group", 0))
    r1 = orc.record_bytes(d, g, bits, topk, kw["scale_mode"], kw.get("qgroup", 0), kw.get("topk_group", 0), 1)
    assert r0 - 4 * J - 15 <= r1 <= r0 - 4 * J + 15 and r1 % 16 == 0
    pay1 = orc.encode(d, g, bits, topk, Xb, ref_base=Rb, step=step, inv_step=inv, forced_coef=per_tok.reshape(-1).copy(),
                      coef_fmt=1, **kw)
    pay0 = orc.encode(d, g, bits, topk, Xb, ref_base=Rb, step=step, inv_step=inv, forced_coef=per_tok.reshape(-1).copy(), **kw)
    assert pay1.size == T * r1
    # same coefficients, same everything else: the two layouts differ only by the missing words
    body0 = pay0.reshape(T, r0)[:, 4 * J:]
    body1 = pay1.reshape(T, r1)
    n = min(body0.shape[1], body1.shape[1])
    assert np.array_equal(body0[:, :n], body1[:, :n]) and not body1[:, n:].any() and not body0[:, n:].any()
    assert np.array_equal(pay0.reshape(T, r0)[:, :4 * J].copy().view(np.uint32), per_tok)
    x1 = orc.reconstruct(d, g, bits, topk, pay1, T, ref_base=Rb, step=step, coef_fmt=1, shared_coef=per_tok, **kw)
    x0 = orc.reconstruct(d, g, bits, topk, pay0, T, ref_base=Rb, step=step, **kw)
    assert np.array_equal(x0, x1)
    with pytest.raises(ValueError):
        orc.encode(d, g, bits, topk, Xb, ref_base=Rb, step=step, inv_step=inv, coef_fmt=1, **kw)   # nothing to share
