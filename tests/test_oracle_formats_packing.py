"""Pins for the oracle's number formats and bit packing (CPU only).

Each check compares the oracle with something it does not compute itself:
numpy's / torch's own float16 and bfloat16 conversions, exhaustive enumeration,
or a figure the paper prints.
"""
import os

import numpy as np
import torch

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def test_f64_to_f16_matches_numpy_single_rounding(orc):
    rng = np.random.default_rng(1)
    xs = np.concatenate([
        rng.standard_normal(4000) * 10.0 ** rng.integers(-9, 5, 4000),
        np.array([0.0, -0.0, 1.0, -1.0, 65504.0, 65519.9, 2.0 ** -24, 2.0 ** -25, 1.5 * 2.0 ** -24,
                  2.0 ** -14, 2.0 ** -14 - 2.0 ** -25, 6.1e-5, 5.96e-8, 2.98e-8]),
    ])
    for x in xs:
        if abs(x) >= 65520.0:
            continue
        want = int(np.float64(x).astype(np.float16).view(np.uint16))
        got = orc.f64_to_f16(float(x))
        assert got == want, (x, hex(got), hex(want))


def test_f64_to_f16_every_midpoint_rounds_to_even(orc):
    # every pair of adjacent positive binary16 values: the exact midpoint must go to the even one,
    # and a value a hair to either side must go to the nearer one.
    for h in range(0, 0x7bff, 7):
        lo = float(np.uint16(h).view(np.float16))
        hi = float(np.uint16(h + 1).view(np.float16))
        mid = (lo + hi) / 2.0  # exact in binary64
        even = h if (h & 1) == 0 else h + 1
        assert orc.f64_to_f16(mid) == even
        assert orc.f64_to_f16(np.nextafter(mid, 0.0)) == h
        assert orc.f64_to_f16(np.nextafter(mid, 1e9)) == h + 1
        assert orc.f16_to_f64(h) == lo


def test_f16_saturates_and_rounds_up(orc):
    assert orc.f64_to_f16(1e9) == 0x7bff
    assert orc.f64_to_f16(-1e9) == 0xfbff
    assert orc.f64_to_f16(65519.0) == 0x7bff
    rng = np.random.default_rng(2)
    for x in np.abs(rng.standard_normal(2000)) * 10.0 ** rng.integers(-6, 3, 2000):
        up = orc.f16_to_f64(orc.f64_to_f16_up(float(x)))
        assert up >= x
        # and it is the smallest such value: the binary16 just below is < x
        below = float(np.nextafter(np.float16(up), np.float16(0)))
        assert below < x or up == 0.0


def test_bf16_round_matches_torch(orc):
    g = torch.Generator().manual_seed(3)
    x = torch.randn(5000, generator=g) * torch.tensor(10.0) ** torch.randint(-6, 6, (5000,), generator=g)
    # add exact ties: values half way between two bfloat16 neighbours
    base = torch.randn(512, generator=g).to(torch.bfloat16).float()
    ties = (base.view(torch.int32) | 0x8000).view(torch.float32)
    x = torch.cat([x, ties])
    want = x.to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)
    got = orc.f32_to_bf16(x.numpy())
    assert np.array_equal(got, want)
    assert np.array_equal(orc.bf16_to_f32(want), x.to(torch.bfloat16).float().numpy())


def test_pack_roundtrip_exhaustive_and_layout(orc):
    for bits in (2, 3, 4):
        lo, hi = -(1 << (bits - 1)), (1 << (bits - 1)) - 1
        vals = np.arange(lo, hi + 1, dtype=np.int32)
        d = 64
        # every code value at every channel phase (c mod 8 covers every bit offset in a byte)
        for phase in range(8):
            for v in vals:
                q = np.zeros(d, np.int32)
                q[phase::8] = v
                packed = orc.pack_codes(q, bits)
                assert packed.size == d * bits // 8
                assert np.array_equal(orc.unpack_codes(packed, d, bits), q)
                # independent statement of the layout: the stream is the little-endian bit string
                stream = np.unpackbits(packed, bitorder="little")
                for c in (phase, phase + 8):
                    field = stream[c * bits:(c + 1) * bits]
                    u = int(sum(int(b) << n for n, b in enumerate(field)))
                    assert u == (int(v) & ((1 << bits) - 1))
    # 4-bit: two values per byte, even channel in the low nibble (Sec. IV-C, "INT4 ... packs two values per byte")
    q = np.array([1, -2, 7, -7], np.int32)
    assert list(orc.pack_codes(q, 4)) == [0x1 | (0xE << 4), 0x7 | (0x9 << 4)]


def test_record_bytes_and_paper_payload_ratio(orc):
    with open(os.path.join(GOLDEN, "payload_ratio.txt")) as f:
        rows = [l.split() for l in f if l.strip() and not l.startswith("#")]
    golden = {r[0]: float(r[1]) for r in rows}
    d = 4096
    # dense 4-bit values alone are 25.0 % of the raw bf16 bytes (paper, Sec. V-B / Tab. I decode row)
    assert (d * 4 // 8) / (2 * d) * 100.0 == golden["dense_int4_percent_of_raw"]
    for (dd, g, b, k) in [(4096, 128, 4, 0), (4096, 128, 4, 8), (3584, 128, 3, 0), (5120, 128, 4, 8),
                          (4096, 64, 2, 8), (4096, 64, 3, 8)]:
        raw = 4 * (dd // g) + dd * b // 8 + 4 * k
        rec = orc.record_bytes(dd, g, b, k)
        assert rec % 16 == 0 and 0 <= rec - raw < 16
    assert orc.record_bytes(4096, 128, 4, 0) == 2176
    assert orc.record_bytes(4096, 128, 4, 8) == 2208
    assert orc.record_bytes(3584, 128, 3, 0) == 1456
    assert orc.record_bytes(5120, 128, 4, 8) == 2752
    # our whole record (values + coefficients + outliers) stays close to the paper's 27.8 % prefill figure
    ours = orc.record_bytes(4096, 128, 4, 8) / (2 * 4096) * 100
    assert abs(ours - golden["prefill_payload_percent_of_raw"]) < 1.5
