"""Byte-cost sweep over codec configurations (the measurable half of the offline calibration of Sec. IV-C).

For every candidate configuration the sender path is run on the given activations (step tables from
``rac_calibrate_steps`` where the configuration needs them, then ``rac_encode_reconstruct``) and the packed bytes per
token are reported beside the reconstruction error (``rac_recon_error``).  Members with shared coefficient pairs
(``coef_fmt = 1``) run ``rac_fit_segments`` first and count their shared words towards the bytes.  Picking a
configuration against a model-quality target needs the model and its evaluation suites and is not done here.

Every step runs in the CUDA kernels of the C-ABI library; this module only loops over configurations.

    python -m paper_2608_04991_b200.sweep [--tokens 16384] [--d 4096]
"""
from __future__ import annotations

import argparse
from typing import Iterable, List, Optional

import torch

from . import binding as rac
from . import synth


def sweep(X: torch.Tensor, ref_base: Optional[torch.Tensor], ref_row: Optional[torch.Tensor],
          configs: Iterable[rac.CodecCfg], gain=None, bias=None, clip_sigmas: float = 3.0, reps: int = 3,
          seg_off: Optional[torch.Tensor] = None) -> List[dict]:
    """X bf16[T,d] on a CUDA device; ``ref_base`` / ``ref_row`` / ``gain`` / ``bias`` as for ``rac_encode``.
    Configurations with ``coef_fmt = 1`` (one coefficient pair per segment and group, Eq. 6 over several positions) need
    ``seg_off``, int32[n_seg + 1] on the device; their shared words count towards the bytes per token."""
    dev = X.device
    T, d = X.shape
    ref_rows = 0 if ref_base is None else ref_base.shape[0]
    x_hat = torch.empty_like(X)
    status = torch.zeros(1, dtype=torch.int32, device=dev)
    err = torch.zeros(3, dtype=torch.float64, device=dev)
    ews_n = rac.rac_recon_error_workspace_bytes()
    ews = torch.empty(ews_n, dtype=torch.uint8, device=dev)
    out = []
    for cfg in configs:
        rec = rac.rac_record_bytes(cfg)
        if rec == 0:
            raise ValueError(f"unsupported configuration {cfg!r}")
        step = inv = None
        shared = cfg.coef_fmt == 1
        coef_seg = seg_of = None
        extra = 0.0
        if shared:
            if seg_off is None:
                raise ValueError("a configuration with coef_fmt = 1 needs seg_off")
            n_seg = seg_off.numel() - 1
            J = d // cfg.group
            coef_seg = torch.empty((n_seg, J), dtype=torch.int32, device=dev)
            seg_of = torch.empty(T, dtype=torch.int32, device=dev)
            nbf = rac.rac_fit_segments_workspace_bytes(cfg, T)
            wsf = torch.empty(nbf, dtype=torch.uint8, device=dev)
            rac.rac_fit_segments(cfg, X, T, ref_base, ref_rows, ref_row, gain, bias, seg_off, n_seg, coef_seg, seg_of,
                                 wsf, nbf, status)
            extra = 4.0 * J * n_seg / T
        if cfg.scale_mode == 0 and shared:
            step = torch.empty((2, d), dtype=torch.float32, device=dev)
            inv = torch.empty_like(step)
            nb = rac.rac_calibrate_workspace_bytes(cfg)
            ws = torch.empty(nb, dtype=torch.uint8, device=dev)
            rac.rac_calibrate_steps_shared(cfg, X, T, ref_base, ref_rows, ref_row, gain, bias, coef_seg, seg_of,
                                           clip_sigmas, step, inv, ws, nb, status)
        elif cfg.scale_mode == 0:
            step = torch.empty((2, d), dtype=torch.float32, device=dev)
            inv = torch.empty_like(step)
            nb = rac.rac_calibrate_workspace_bytes(cfg)
            ws = torch.empty(nb, dtype=torch.uint8, device=dev)
            rac.rac_calibrate_steps(cfg, X, T, ref_base, ref_rows, ref_row, gain, bias, clip_sigmas, step, inv, ws, nb,
                                    status)
        pay = torch.empty(T * rec, dtype=torch.uint8, device=dev)
        nws = rac.rac_encode_workspace_bytes(cfg, T)
        ws2 = torch.empty(max(nws, 16), dtype=torch.uint8, device=dev)
        if shared:
            run = lambda: rac.rac_encode_reconstruct_list(cfg, X, T, None, None, ref_base, ref_rows, ref_row, None, 0, gain,
                                                          bias, step, inv, pay, pay.numel(), x_hat, ws2 if nws else None,
                                                          nws, status, coef_seg=coef_seg, seg_of=seg_of)
        else:
            run = lambda: rac.rac_encode_reconstruct(cfg, X, T, ref_base, ref_rows, ref_row, gain, bias, step, inv, pay,
                                                     pay.numel(), x_hat, ws2 if nws else None, nws, status)
        run()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        torch.cuda.synchronize()
        e0.record()
        for _ in range(reps):
            run()
        e1.record()
        rac.rac_recon_error(X, x_hat, T, d, err, ews, ews_n)
        torch.cuda.synchronize()
        se, sx, mx = err.tolist()
        out.append({
            "group": cfg.group, "bits": cfg.bits, "topk": cfg.topk, "scale_mode": cfg.scale_mode,
            "qgroup": cfg.qgroup or cfg.group, "topk_group": cfg.topk_group,
            "coef_fmt": cfg.coef_fmt, "record_bytes": rec, "shared_bytes_per_token": extra,
            "payload_over_raw": (rec + extra) / (2.0 * d),
            "rel_rms_error": (se / sx) ** 0.5 if sx > 0 else 0.0, "max_abs_error": mx,
            "encode_reconstruct_ms": e0.elapsed_time(e1) / reps, "status": int(status.item()),
        })
        del pay
    return out


def default_grid(d: int) -> List[rac.CodecCfg]:
    """Static-table members (per-token outliers) and Eq. 8 members (per-group outliers, 8-bit, one scale per token)."""
    cfgs = []
    for g in (64, 128, 256):
        for b in (2, 3, 4):
            for k in (0, 8):
                cfgs.append(rac.CodecCfg(d, g, b, k))
        for b in (4, 8):
            for kg in (0, 1, 2):
                cfgs.append(rac.CodecCfg(d, g, b, 0, scale_mode=1, topk_group=kg))
    cfgs.append(rac.CodecCfg(d, 128, 4, 0, scale_mode=1, qgroup=d))
    cfgs.append(rac.CodecCfg(d, 128, 8, 0, scale_mode=1, qgroup=d))
    return cfgs


def shared_grid(d: int) -> List[rac.CodecCfg]:
    """Members whose coefficient pairs are shared by the tokens of a segment (they need ``seg_off``)."""
    return [rac.CodecCfg(d, 128, 4, 8, coef_fmt=1), rac.CodecCfg(d, 128, 4, 0, coef_fmt=1),
            rac.CodecCfg(d, 128, 4, 0, scale_mode=1, coef_fmt=1), rac.CodecCfg(d, 128, 4, 0, scale_mode=1, topk_group=1, coef_fmt=1)]


def main() -> int:
    ap = argparse.ArgumentParser(description=__doc__.split("\n")[0])
    ap.add_argument("--tokens", type=int, default=16384)
    ap.add_argument("--d", type=int, default=4096)
    ap.add_argument("--seed", type=int, default=1)
    ap.add_argument("--segment", type=int, default=64, help="tokens per segment for the members with shared coefficient "
                    "pairs (0 leaves them out)")
    args = ap.parse_args()
    if not torch.cuda.is_available():
        raise SystemExit("the sweep runs the CUDA kernels: no CUDA device found")
    rac.load()
    dev = torch.device("cuda:0")
    gen = synth.generator(args.seed, dev)
    X = synth.activations(args.tokens, args.d, synth.channel_scale(args.d, args.seed, dev), gen)
    R = synth.affine_noisy_reference(X, 128, gen)
    rows = sweep(X, R, None, default_grid(args.d))
    if args.segment > 0:
        # the reference of these members carries ONE affine map per (segment, group): what a shared pair can undo
        bounds = list(range(0, args.tokens, args.segment)) + [args.tokens]
        seg_off = torch.tensor(bounds, dtype=torch.int32, device=dev)
        a = torch.rand((len(bounds) - 1, args.d // 128, 1), generator=gen, device=dev) * 0.4 + 0.8
        b = torch.randn((len(bounds) - 1, args.d // 128, 1), generator=gen, device=dev) * 0.1
        seg = torch.repeat_interleave(torch.arange(len(bounds) - 1, device=dev),
                                      torch.diff(seg_off.long()))
        Rs = torch.empty_like(X)
        for t0 in range(0, args.tokens, 4096):
            t1 = min(args.tokens, t0 + 4096)
            x = X[t0:t1].float().view(t1 - t0, args.d // 128, 128)
            z = torch.randn(x.shape, generator=gen, device=dev) * 0.05
            Rs[t0:t1] = ((x - b[seg[t0:t1]]) / a[seg[t0:t1]] + z).view(t1 - t0, args.d).to(torch.bfloat16)
        more = sweep(X, Rs, None, shared_grid(args.d) + [rac.CodecCfg(args.d, 128, 4, 8), rac.CodecCfg(args.d, 128, 4, 0, scale_mode=1)],
                     seg_off=seg_off)
        for r in more:
            r["segmented"] = True
        rows += more
    rows.sort(key=lambda r: (r["record_bytes"] + r["shared_bytes_per_token"], r["rel_rms_error"]))
    print(f"synthetic prefill uplink, {args.tokens} x {args.d}; reference = noisy affine image per (token, 128 channels)")
    if args.segment > 0:
        print(f"members marked 'seg': reference with one affine map per ({args.segment} tokens, 128 channels); 'shared' = one "
              "coefficient pair per segment and group, outside the records")
    print(f"{'mode':>7} {'coef':>7} {'g_a':>4} {'g_q':>5} {'b':>2} {'k':>3} {'k_g':>3} {'bytes':>8} {'/raw':>6} {'rel rms':>9} {'max abs':>8} {'ms':>7}")
    for r in rows:
        mode = "static" if r["scale_mode"] == 0 else "Eq.8"
        coef = "shared" if r["coef_fmt"] == 1 else ("seg" if r.get("segmented") else "token")
        print(f"{mode:>7} {coef:>7} {r['group']:>4} {r['qgroup']:>5} {r['bits']:>2} {r['topk']:>3} {r['topk_group']:>3} "
              f"{r['record_bytes'] + r['shared_bytes_per_token']:>8.1f} {r['payload_over_raw']:>6.3f} {r['rel_rms_error']:>9.5f} "
              f"{r['max_abs_error']:>8.3f} {r['encode_reconstruct_ms']:>7.3f}")
    return 0


if __name__ == "__main__":
    raise SystemExit(main())
