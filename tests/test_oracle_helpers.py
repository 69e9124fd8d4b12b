"""Pins for the oracle's small helpers that GPU tests use as expected values (CPU only).

`segments_from_spans` (the segmentation "spans and the gaps between them" behind the shared-coefficient fit) and
`recon_error` (the error sums of a sender-path run) are checked against results typed in by hand; the binary64
quotient `v_ideal` the encoder reports as a diagnostic is checked against the codes it does not decide.
"""
import numpy as np
import torch

from paper_2608_04991_b200 import synth


def bf16_bits(values):
    """exact bf16 values (as Python floats) -> bit patterns, through torch (not the oracle's own conversion)"""
    t = torch.tensor(values, dtype=torch.float32)
    b = t.to(torch.bfloat16)
    assert torch.equal(b.float(), t), "test values must be bf16-representable"
    return synth.bf16_bits(b)


# ------------------------------------------------------------------ segments_from_spans
def test_segments_no_spans_and_empty_prompt(orc):
    none = np.zeros((0, 3), np.int32)
    assert orc.segments_from_spans(none, 10).tolist() == [0, 10]       # one gap covering everything
    assert orc.segments_from_spans(none, 0).tolist() == [0]            # no token, no segment
    assert orc.segments_from_spans(none, 1).tolist() == [0, 1]


def test_segments_span_at_start_end_and_adjacent(orc):
    # spans are (query start, history start, length); the history start plays no part
    assert orc.segments_from_spans(np.array([[0, 7, 4]], np.int32), 10).tolist() == [0, 4, 10]      # span at 0, gap after
    assert orc.segments_from_spans(np.array([[6, 0, 4]], np.int32), 10).tolist() == [0, 6, 10]      # gap, span ending at T
    assert orc.segments_from_spans(np.array([[0, 3, 10]], np.int32), 10).tolist() == [0, 10]        # one span is everything
    # two adjacent spans keep their common boundary and produce no empty piece between them
    assert orc.segments_from_spans(np.array([[2, 50, 3], [5, 9, 4]], np.int32), 12).tolist() == [0, 2, 5, 9, 12]
    # gap - span - gap - span - gap
    assert orc.segments_from_spans(np.array([[1, 0, 2], [7, 0, 1]], np.int32), 9).tolist() == [0, 1, 3, 7, 8, 9]
    b = orc.segments_from_spans(np.array([[0, 0, 5], [5, 0, 5]], np.int32), 10)
    assert b.dtype == np.int32 and b.tolist() == [0, 5, 10]
    # boundaries strictly increase: a segment is never empty
    rng = np.random.default_rng(5)
    for _ in range(200):
        T = int(rng.integers(1, 60))
        spans, q = [], 0
        while q < T:
            q += int(rng.integers(0, 5))
            ln = int(rng.integers(1, 9))
            if q + ln > T:
                break
            spans.append((q, int(rng.integers(0, 100)), ln))
            q += ln
        b = orc.segments_from_spans(np.array(spans, np.int32).reshape(-1, 3), T)
        assert b[0] == 0 and b[-1] == T and np.all(np.diff(b) > 0)
        inside = set(b.tolist())
        for s, _, ln in spans:      # every span is exactly one segment
            assert s in inside and s + ln in inside
            assert not any(s < x < s + ln for x in inside)


# ------------------------------------------------------------------ recon_error
def test_recon_error_sums_typed_by_hand(orc):
    # (1) exact differences: x = [1, -2, 0.5, 4], x_hat = [1.5, -2, 0.25, 3]
    #     differences -0.5, 0, 0.25, 1 -> squares 0.25 + 0 + 0.0625 + 1 = 1.3125; sum x^2 = 1 + 4 + 0.25 + 16 = 21.25
    se, sx, mx = orc.recon_error(bf16_bits([1.0, -2.0, 0.5, 4.0]), bf16_bits([1.5, -2.0, 0.25, 3.0]))
    assert (se, sx, mx) == (1.3125, 21.25, 1.0)
    # (2) identical inputs, and an empty input
    se, sx, mx = orc.recon_error(bf16_bits([3.0, -7.0]), bf16_bits([3.0, -7.0]))
    assert (se, sx, mx) == (0.0, 58.0, 0.0)
    assert orc.recon_error(np.zeros(0, np.uint16), np.zeros(0, np.uint16)) == (0.0, 0.0, 0.0)
    # (3) a pair whose difference binary32 cannot hold: x = 2^20 (bf16), x_hat = 2^-8 (bf16).  The exact difference
    #     1048575.99609375 needs 28 significant bits; the difference of two bf16 values is defined as ONE binary32
    #     subtraction, which rounds it to 2^20 = 1048576.  So the squared error is 2^40 exactly, not (2^20 - 2^-8)^2.
    se, sx, mx = orc.recon_error(bf16_bits([2.0 ** 20]), bf16_bits([2.0 ** -8]))
    assert se == 2.0 ** 40 and sx == 2.0 ** 40 and mx == 2.0 ** 20
    assert se != (2.0 ** 20 - 2.0 ** -8) ** 2
    # (4) two-dimensional inputs are summed over every element; the maximum is of |difference|
    X = bf16_bits([[1.0, 2.0], [-3.0, 4.0]])
    Y = bf16_bits([[0.0, 2.0], [-3.0, 8.0]])
    assert orc.recon_error(X, Y) == (17.0, 30.0, 4.0)


# ------------------------------------------------------------------ v_ideal (Eq. 8c as printed)
def test_codes_agree_with_the_binary64_quotient_except_next_to_a_boundary(orc):
    """Eq. 8c prints q = round(clip(e / s)); the encoder multiplies by a binary32 reciprocal.  The diagnostic
    e / s (binary64 quotient of the binary32 residual) decides nothing; here the emitted codes are compared with
    its rounding: the few that differ are one level away and within 1e-4 of a rounding boundary."""
    d, g, T = 1024, 128, 512
    gen = synth.generator(321)
    X = synth.activations(T, d, synth.channel_scale(d, 3), gen)
    R = synth.affine_noisy_reference(X, g, gen)
    Xb, Rb = synth.bf16_bits(X), synth.bf16_bits(R)
    total = differing = 0
    for bits, mode in [(4, 0), (3, 0), (2, 0), (4, 1), (8, 1)]:
        qmax = (1 << (bits - 1)) - 1
        if mode == 0:
            step, inv = orc.calibrate(d, g, bits, Xb[:256], ref_base=Rb[:256])
            pay, dg = orc.encode(d, g, bits, 0, Xb, ref_base=Rb, step=step, inv_step=inv, diag=True)
            s_of = np.broadcast_to(step[0].astype(np.float64), (T, d))
        else:
            pay, dg = orc.encode(d, g, bits, 0, Xb, ref_base=Rb, diag=True, scale_mode=1)
            scale = orc.split_payload(pay, T, d, g, bits, 0, 1)[4]
            s_of = np.repeat(scale.view(np.float16).astype(np.float64), g, axis=1)
        # the diagnostic is the quotient of the reported residual and the step / scale that is on the wire
        with np.errstate(divide="ignore", invalid="ignore"):
            want = np.where(s_of != 0, dg["e"].astype(np.float64) / s_of, 0.0)
        assert np.array_equal(dg["v_ideal"], want)
        codes = orc.split_payload(pay, T, d, g, bits, 0, mode)[1]
        q = np.stack([orc.unpack_codes(codes[t], d, bits) for t in range(T)])
        q_ideal = np.rint(np.clip(dg["v_ideal"], -qmax, qmax)).astype(np.int32)
        diff = q != q_ideal
        if diff.any():
            vi = np.abs(dg["v_ideal"][diff])
            assert np.all(np.abs(q[diff] - q_ideal[diff]) == 1)
            assert np.all(np.abs(vi - np.floor(vi) - 0.5) < 1e-4)
        total += q.size
        differing += int(diff.sum())
    # binary32 reciprocal and product are each within half an ulp, i.e. |v - e/s| < 2^-22 for |v| < 8 (2^-18 at 8 bits)
    # -- so a differing code needs e/s within that of a boundary: a handful per million at most
    print(f"codes differing from round(e/s): {differing} of {total}")
    assert differing <= total * 2e-5
