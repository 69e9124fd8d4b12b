"""Reconstruction-error kernel and the byte-cost sweep against the oracle (needs a B200)."""
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
    from paper_2608_04991_b200 import synth, sweep
    rac.load()
    return type("Env", (), dict(orc=oracle, rac=rac, synth=synth, sweep=sweep, dev=torch.device("cuda:0")))


@pytest.mark.parametrize("T,d", [(1, 8), (7, 96), (301, 1024), (2051, 4096)])
def test_recon_error_matches_float64_definition(env, T, d):
    s, rac, dev = env.synth, env.rac, env.dev
    gen = s.generator(40 + T, dev)
    X = s.activations(T, d, s.channel_scale(d, 4, dev), gen)
    Y = (X.float() + 0.1 * torch.randn((T, d), generator=gen, device=dev)).to(torch.bfloat16)
    Y[0, 0] = X[0, 0] + 37.0                                             # a known maximum
    out = torch.full((3,), -1.0, dtype=torch.float64, device=dev)
    nb = rac.rac_recon_error_workspace_bytes()
    ws = torch.full((nb,), 0x5A, dtype=torch.uint8, device=dev)
    rac.rac_recon_error(X, Y, T, d, out, ws, nb)
    a = out.tolist()
    rac.rac_recon_error(X, Y, T, d, out, ws, nb)
    assert out.tolist() == a                                             # fixed summation order: reproducible
    se, sx, mx = env.orc.recon_error(s.bf16_bits(X), s.bf16_bits(Y))
    assert abs(a[0] - se) <= 1e-12 * se and abs(a[1] - sx) <= 1e-12 * sx and a[2] == mx
    rac.rac_recon_error(X, X, T, d, out, ws, nb)
    assert out.tolist()[0] == 0.0 and out.tolist()[2] == 0.0


def test_sweep_reports_bytes_and_error_of_the_sender_path(env):
    s, rac, orc, dev = env.synth, env.rac, env.orc, env.dev
    T, d, g = 512, 1024, 128
    gen = s.generator(50, dev)
    X = s.activations(T, d, s.channel_scale(d, 5, dev), gen)
    R = s.affine_noisy_reference(X, g, gen)
    cfgs = [rac.CodecCfg(d, g, 4, 8), rac.CodecCfg(d, g, 2, 0), rac.CodecCfg(d, g, 4, 0, scale_mode=1),
            rac.CodecCfg(d, g, 4, 0, scale_mode=1, topk_group=2), rac.CodecCfg(d, g, 8, 0, scale_mode=1),
            rac.CodecCfg(d, g, 8, 0, scale_mode=1, qgroup=d)]
    rows = env.sweep.sweep(X, R, None, cfgs)
    Xb, Rb = s.bf16_bits(X), s.bf16_bits(R)
    for cfg, r in zip(cfgs, rows):
        assert r["status"] == 0
        assert r["record_bytes"] == orc.record_bytes(d, g, cfg.bits, cfg.topk, cfg.scale_mode, cfg.qgroup, cfg.topk_group)
        # the oracle's own run of the same configuration: the error agrees up to the few coefficient roundings
        kw = dict(scale_mode=cfg.scale_mode, qgroup=cfg.qgroup, topk_group=cfg.topk_group)
        step = inv = None
        if cfg.scale_mode == 0:
            step, inv = orc.calibrate(d, g, cfg.bits, Xb, ref_base=Rb)
        pay = orc.encode(d, g, cfg.bits, cfg.topk, Xb, ref_base=Rb, step=step, inv_step=inv, **kw)
        xh = orc.reconstruct(d, g, cfg.bits, cfg.topk, pay, T, ref_base=Rb, step=step, **kw)
        se, sx, mx = orc.recon_error(Xb, xh)
        assert abs(r["rel_rms_error"] - (se / sx) ** 0.5) <= 2e-3 * (se / sx) ** 0.5
    by = {(r["scale_mode"], r["bits"], r["topk"], r["topk_group"], r["qgroup"]): r for r in rows}
    # more bits, or outliers out of the way, can only help on this workload
    assert by[(1, 8, 0, 0, g)]["rel_rms_error"] < by[(1, 4, 0, 0, g)]["rel_rms_error"] / 8
    assert by[(1, 4, 0, 2, g)]["rel_rms_error"] < by[(1, 4, 0, 0, g)]["rel_rms_error"]
    assert by[(1, 8, 0, 0, d)]["rel_rms_error"] > by[(1, 8, 0, 0, g)]["rel_rms_error"]     # one scale per token is coarser
    assert by[(0, 2, 0, 0, g)]["rel_rms_error"] > by[(0, 4, 8, 0, g)]["rel_rms_error"]
