#!/usr/bin/env python
"""Benchmark of the RAC codec hot path on B200.

One "step" is one pass of the whole hot path over the long-context round trip
(T = 131072 tokens, d = 5120, group 128, 4-bit, top-8 outliers, 131072-token history):

    span match -> uplink encode + sender-side reconstruction (one call) -> receiver reconstruct
               -> downlink encode (reference = reconstructed uplink) -> receiver reconstruct

`value` is GB/s of bf16 activations through the codec (both directions, 2 * 2*T*d bytes per step)
with every input resident in HBM.  `e2e` is the same metric with the step's inputs copied from
pinned host memory and its wire payloads and final activations copied back inside the timed region.
`roofline` is measured live for the dominant kernel with CUDA events on the launching stream.
`--impl reference` times the CPU oracle (tests' checker) on a bounded sample of the same workload.

Launch:  python bench.py [--gpus N --steps K --warmup W]      (N > 1: under torch.distributed.run)
"""
from __future__ import annotations

import argparse
import json
import os
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "codec GB/s of bf16 activations (encode+decode round trip)"
UNIT = "GB/s"
WORKLOAD = dict(T=131072, d=5120, group=128, bits=4, topk=8, n_hist=131072, min_ngram=4, max_hits=8, gap_max=112)
# DRAM bytes (dram__bytes_read.sum + dram__bytes_write.sum) of one rac_encode[_reconstruct] call (streaming kernel +
# outlier kernel) and of one reconstruction, from an ncu capture of the SMALL case (T = 16384, same d and record);
# traffic is proportional to tokens, so a launch of T tokens moves T/16384 times as much.
NCU_SMALL_CASE_TRAFFIC = {"encode_sender_up": 267.85e6 + 180.01e6 + 51.13e6 + 1.67e6,
                          "encode_dn": 335.62e6 + 44.00e6 + 56.33e6 + 0.49e6,
                          "decode_up": 141.15e6 + 118.01e6, "decode_dn": 212.92e6 + 123.03e6}
SMALL = dict(T=16384, d=5120, group=128, bits=4, topk=8, n_hist=16384, min_ngram=4, max_hits=8, gap_max=112)


def parse_args():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=50)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="rac", choices=["rac", "reference"])
    ap.add_argument("--scaling", default="weak", choices=["weak", "strong"],
                    help="weak: every rank codes its own sequences; strong: the ranks share ONE tensor by token ranges "
                         "and gather the payload byte ranges")
    ap.add_argument("--small", action="store_true", help="a small case of the same path (for profiler captures)")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-decode-steps", action="store_true", help="skip the decode-step latency extra")
    ap.add_argument("--no-sweep", action="store_true", help="skip the b x group sweep at T=16384, d=4096")
    ap.add_argument("--sweep-only", action="store_true",
                    help="run only the b x group sweep and print its JSON (a small case for profiler captures)")
    ap.add_argument("--no-family", action="store_true", help="skip the extras beyond the graded path (Eq. 8 family, persistent index)")
    return ap.parse_args()


def measured_peak():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(path) as f:
            return float(json.load(f)["hbm_gbs"]), "measured (MEASURED_PEAKS.json hbm_gbs)"
    except Exception:
        return 6650.0, "fallback (earlier pool measurement, 6.65 TB/s)"


# --------------------------------------------------------------------------------------------- clocks
class ClockSampler:
    """Samples SM clock, power and throttle reasons of one GPU through NVML (read only) while running."""
    REASONS = {0x4: "sw_power_cap", 0x8: "hw_slowdown", 0x20: "sw_thermal_slowdown", 0x40: "hw_thermal_slowdown",
               0x80: "hw_power_brake_slowdown", 0x2: "applications_clocks_setting", 0x10: "sync_boost"}

    def __init__(self, torch_index: int):
        self.samples = []
        self.reasons = set()
        self.max_mhz = None
        self._stop = threading.Event()
        self._thr = None
        self._h = None
        try:
            import pynvml
            import torch
            pynvml.nvmlInit()
            uuid = str(torch.cuda.get_device_properties(torch_index).uuid)
            uuid = uuid if uuid.startswith("GPU-") else "GPU-" + uuid
            try:
                self._h = pynvml.nvmlDeviceGetHandleByUUID(uuid.encode())
            except Exception:
                self._h = pynvml.nvmlDeviceGetHandleByIndex(torch_index)
            self._nv = pynvml
            self.max_mhz = int(pynvml.nvmlDeviceGetMaxClockInfo(self._h, pynvml.NVML_CLOCK_SM))
        except Exception as e:  # pragma: no cover
            self.error = repr(e)

    def _run(self):
        nv = self._nv
        while not self._stop.is_set():
            try:
                mhz = int(nv.nvmlDeviceGetClockInfo(self._h, nv.NVML_CLOCK_SM))
                mask = int(nv.nvmlDeviceGetCurrentClocksEventReasons(self._h))
                self.samples.append(mhz)
                for bit, name in self.REASONS.items():
                    if mask & bit:
                        self.reasons.add(name)
            except Exception:
                pass
            self._stop.wait(0.02)

    def start(self):
        if self._h is not None:
            self._thr = threading.Thread(target=self._run, daemon=True)
            self._thr.start()

    def stop(self):
        self._stop.set()
        if self._thr:
            self._thr.join()

    def summary(self):
        if not self.samples:
            return {"sm_mhz": None, "sm_max_mhz": self.max_mhz, "reasons": sorted(self.reasons), "samples": 0}
        s = sorted(self.samples)
        return {"sm_mhz": s[len(s) // 2], "sm_max_mhz": self.max_mhz, "reasons": sorted(self.reasons),
                "samples": len(s)}


# --------------------------------------------------------------------------------------------- workload
class RoundTrip:
    """Device buffers and the ordered C-ABI calls of one step."""
    LAUNCHES_PER_STEP = 9 + 2 * 2 + 2  # matcher kernels + 2 encodes (2 launches each) + 2 reconstructions

    def __init__(self, wl, seed, dev, token_range=None):
        import numpy as np
        import torch
        from paper_2608_04991_b200 import binding as rac
        from paper_2608_04991_b200 import synth
        self.rac, self.torch, self.wl, self.dev = rac, torch, wl, dev
        T, d, g = wl["T"], wl["d"], wl["group"]
        self.a, self.b = 0, T
        self.cfg = rac.CodecCfg(d, g, wl["bits"], wl["topk"])
        self.rec = rac.rac_record_bytes(self.cfg)
        tw = synth.span_workload(wl["n_hist"], T, seed=seed, gap_max=wl["gap_max"])
        self.host_hist, self.host_query = tw.hist, tw.query
        self.planted_coverage = tw.planted_coverage
        self.hist = torch.from_numpy(tw.hist).to(dev)
        self.query = torch.from_numpy(tw.query).to(dev)
        gen = synth.generator(synth.BASE_SEED + seed, dev)
        scale = synth.channel_scale(d, seed, dev)
        self.Hs = synth.activations(wl["n_hist"], d, scale, gen)            # history state buffer
        self.X = synth.affine_noisy_target(self.Hs, torch.from_numpy(tw.planted_row), g, gen, scale)
        z = lambda *shape, dt=torch.uint8: torch.empty(shape, dtype=dt, device=dev)
        self.ws_bytes = rac.rac_match_workspace_bytes(wl["n_hist"], T, wl["max_hits"])
        self.ws = z(self.ws_bytes)
        self.ref_row = z(T, dt=torch.int32)
        self.spans = z(T // wl["min_ngram"] + 1, 3, dt=torch.int32)
        self.n_spans = z(1, dt=torch.int32)
        self.status = torch.zeros(1, dtype=torch.int32, device=dev)
        self.pay_up, self.pay_dn = z(T * self.rec), z(T * self.rec)
        self.ews_bytes = rac.rac_encode_workspace_bytes(self.cfg, T)
        self.ews = z(self.ews_bytes)
        self.Xs, self.Xh, self.Yh = (z(T, d, dt=torch.bfloat16) for _ in range(3))
        self.step_up, self.inv_up = z(2, d, dt=torch.float32), z(2, d, dt=torch.float32)
        self.step_dn, self.inv_dn = z(2, d, dt=torch.float32), z(2, d, dt=torch.float32)
        # set-up (untimed): rows, step tables from the first tokens, the downlink state
        self.match()
        nb = rac.rac_calibrate_workspace_bytes(self.cfg)
        cws = z(nb)
        Tc = min(T, 4096)
        rac.rac_calibrate_steps(self.cfg, self.X[:Tc], Tc, self.Hs, wl["n_hist"], self.ref_row[:Tc].contiguous(), None, None,
                                3.0, self.step_up, self.inv_up, cws, nb, self.status)
        self.encode_up()
        self.decode_up()
        self.Y = synth.drifted_state(self.Xh, gen)
        rac.rac_calibrate_steps(self.cfg, self.Y[:Tc], Tc, self.Xh, T, None, None, None, 3.0, self.step_dn, self.inv_dn,
                                cws, nb, self.status)
        torch.cuda.synchronize()
        self.coverage = float((self.ref_row >= 0).float().mean().item())
        self.np = np
        # strong scaling: this rank codes tokens [a, b) of the one tensor (the set-up above ran over all of them, so
        # every rank holds the same tables and the same downlink state)
        self.a, self.b = (0, T) if token_range is None else token_range
        self.shard_coverage = float((self.ref_row[self.a:self.b] >= 0).float().mean().item()) if self.b > self.a else 0.0

    # ---- the calls of one step, in order
    def match(self):
        w = self.wl
        self.rac.rac_match_spans(self.hist, w["n_hist"], self.query, w["T"], w["min_ngram"], w["max_hits"], self.ref_row,
                                 self.spans, self.n_spans, self.ws, self.ws_bytes)

    def encode_up(self):
        w = self.wl
        self.rac.rac_encode(self.cfg, self.X, w["T"], self.Hs, w["n_hist"], self.ref_row, None, None, self.step_up,
                            self.inv_up, self.pay_up, self.pay_up.numel(), self.ews, self.ews_bytes, self.status)

    # the calls below work on this rank's token range [a, b) (all T tokens unless the run shards one tensor)
    def encode_sender_up(self):
        """Uplink encode that also leaves the sender-side x_hat (the next reference) in Xs."""
        w, a, b, rec = self.wl, self.a, self.b, self.rec
        self.rac.rac_encode_reconstruct(self.cfg, self.X[a:b], b - a, self.Hs, w["n_hist"], self.ref_row[a:b], None, None,
                                        self.step_up, self.inv_up, self.pay_up[a * rec:b * rec], (b - a) * rec,
                                        self.Xs[a:b], self.ews, self.ews_bytes, self.status)

    def decode_up(self):
        w, a, b, rec = self.wl, self.a, self.b, self.rec
        self.rac.rac_decode_reconstruct(self.cfg, self.pay_up[a * rec:b * rec], b - a, self.Hs, w["n_hist"],
                                        self.ref_row[a:b], None, None, self.step_up, self.Xh[a:b], self.status)

    def encode_dn(self):
        a, b, rec = self.a, self.b, self.rec
        self.rac.rac_encode(self.cfg, self.Y[a:b], b - a, self.Xh[a:b], b - a, None, None, None, self.step_dn, self.inv_dn,
                            self.pay_dn[a * rec:b * rec], (b - a) * rec, self.ews, self.ews_bytes, self.status)

    def decode_dn(self):
        a, b, rec = self.a, self.b, self.rec
        self.rac.rac_decode_reconstruct(self.cfg, self.pay_dn[a * rec:b * rec], b - a, self.Xh[a:b], b - a, None, None, None,
                                        self.step_dn, self.Yh[a:b], self.status)

    STAGES = ["match", "encode_sender_up", "decode_up", "encode_dn", "decode_dn"]

    def step(self, events=None):
        for i, name in enumerate(self.STAGES):
            if events is not None:
                events[i].record()
            getattr(self, name)()
        if events is not None:
            events[len(self.STAGES)].record()

    # ---- algorithmic bytes (what the method itself must move, per launch)
    def bytes_of(self, name):
        w = self.wl
        T, d, rec = self.b - self.a, w["d"], self.rec
        refd = self.shard_coverage
        if name == "encode_up":
            return T * (2 * d + 2 * d * refd + rec + 4)
        if name == "encode_sender_up":
            return T * (2 * d + 2 * d * refd + rec + 4 + 2 * d)
        if name == "encode_dn":
            return T * (2 * d + 2 * d + rec)
        if name == "decode_up":
            return T * (rec + 2 * d * refd + 2 * d + 4)
        if name == "decode_dn":
            return T * (rec + 2 * d + 2 * d)
        return 0

    def activation_bytes_per_step(self):
        return 2 * 2 * self.wl["T"] * self.wl["d"]


# --------------------------------------------------------------------------------------------- the paper's quantiser family
def paper_family(dev, T, d, g=128, reps=10):
    """Eq. 8 as printed (scale_mode 1) on the benchmark's shape: encode and reconstruct of a few members of the
    family (per-group scales, k_g outliers per group, 8-bit codes, one scale per token), each timed alone with
    CUDA events over `reps` launches after 3 warm-ups; GB/s over the algorithmic bytes (X + reference + record,
    resp. record + reference + x_hat).  Inputs are larger than L2."""
    import torch
    from paper_2608_04991_b200 import binding as rac
    from paper_2608_04991_b200 import synth
    gen = synth.generator(synth.BASE_SEED + 9, dev)
    X = synth.activations(T, d, synth.channel_scale(d, 9, dev), gen)
    R = synth.affine_noisy_reference(X, g, gen)
    xh = torch.empty_like(X)
    status = torch.zeros(1, dtype=torch.int32, device=dev)
    out = []
    for name, bits, qg, kg in (("4-bit, scale per group", 4, 0, 0), ("4-bit, 1 outlier per group", 4, 0, 1),
                               ("4-bit, 2 outliers per group", 4, 0, 2), ("8-bit, scale per group", 8, 0, 0),
                               ("4-bit, one scale per token", 4, d, 0)):
        cfg = rac.CodecCfg(d, g, bits, 0, scale_mode=1, qgroup=qg, topk_group=kg)
        rec = rac.rac_record_bytes(cfg)
        pay = torch.empty(T * rec, dtype=torch.uint8, device=dev)
        enc = lambda: rac.rac_encode(cfg, X, T, R, T, None, None, None, None, None, pay, pay.numel(), None, 0, status)
        dec = lambda: rac.rac_decode_reconstruct(cfg, pay, T, R, T, None, None, None, None, xh, status)
        row = {"member": name, "record_bytes": rec, "payload_over_raw": rec / (2.0 * d)}
        for key, fn in (("encode", enc), ("reconstruct", dec)):
            for _ in range(3):
                fn()
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            torch.cuda.synchronize()
            e0.record()
            for _ in range(reps):
                fn()
            e1.record()
            torch.cuda.synchronize()
            ms = e0.elapsed_time(e1) / reps
            row[key + "_ms"] = ms
            row[key + "_GBps"] = T * (4 * d + rec) / (ms * 1e-3) / 1e9
        out.append(row)
        del pay
    if int(status.item()) != 0:
        raise RuntimeError(f"paper_family: device status {int(status.item())}")
    return out


# --------------------------------------------------------------------------------------------- shared coefficients
def shared_coefficients(dev, T, d, g=128, seg_tokens=64, reps=10):
    """Eq. 6 over several fitting positions on the benchmark's shape: one coefficient pair per (segment of
    `seg_tokens` tokens, group), records without coefficient words (4-bit codes, scale per group).  Times of the
    fit (statistics pass + merge), of the encode and of the reconstruction with the shared words."""
    import torch
    from paper_2608_04991_b200 import binding as rac
    from paper_2608_04991_b200 import synth
    gen = synth.generator(synth.BASE_SEED + 13, dev)
    X = synth.activations(T, d, synth.channel_scale(d, 13, dev), gen)
    R = synth.affine_noisy_reference(X, g, gen)
    cfg = rac.CodecCfg(d, g, 4, 0, scale_mode=1, coef_fmt=1)
    rec = rac.rac_record_bytes(cfg)
    n_seg = (T + seg_tokens - 1) // seg_tokens
    seg_off = torch.clamp(torch.arange(n_seg + 1, dtype=torch.int32, device=dev) * seg_tokens, max=T).to(torch.int32)
    coef = torch.empty((n_seg, d // g), dtype=torch.int32, device=dev)
    seg_of = torch.empty(T, dtype=torch.int32, device=dev)
    nb = rac.rac_fit_segments_workspace_bytes(cfg, T)
    ws = torch.empty(nb, dtype=torch.uint8, device=dev)
    pay = torch.empty(T * rec, dtype=torch.uint8, device=dev)
    xh = torch.empty_like(X)
    status = torch.zeros(1, dtype=torch.int32, device=dev)
    fit = lambda: rac.rac_fit_segments(cfg, X, T, R, T, None, None, None, seg_off, n_seg, coef, seg_of, ws, nb, status)
    enc = lambda: rac.rac_encode_reconstruct_list(cfg, X, T, None, None, R, T, None, None, 0, None, None, None, None, pay,
                                                  pay.numel(), None, None, 0, status, coef_seg=coef, seg_of=seg_of)
    dec = lambda: rac.rac_decode_reconstruct_list(cfg, pay, T, None, None, R, T, None, None, 0, None, None, None, xh,
                                                  status, coef_seg=coef, seg_of=seg_of)
    out = {"segment_tokens": seg_tokens, "segments": n_seg, "record_bytes": rec, "payload_over_raw": rec / (2.0 * d),
           "shared_words_bytes_per_token": 4.0 * (d // g) / seg_tokens}
    for key, fn, nbytes in (("fit", fit, T * 4 * d), ("encode", enc, T * (4 * d + rec)), ("reconstruct", dec, T * (4 * d + rec))):
        for _ in range(3):
            fn()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        torch.cuda.synchronize()
        e0.record()
        for _ in range(reps):
            fn()
        e1.record()
        torch.cuda.synchronize()
        ms = e0.elapsed_time(e1) / reps
        out[key + "_ms"] = ms
        out[key + "_GBps"] = nbytes / (ms * 1e-3) / 1e9
    if int(status.item()) != 0:
        raise RuntimeError(f"shared_coefficients: device status {int(status.item())}")
    return out


# --------------------------------------------------------------------------------------------- retrieval over requests
def retrieval_index(dev, n_hist, n_query, gap_max, request_tokens=2048, reps=10):
    """The persistent span index on the benchmark's token workload: the history appended as requests of
    `request_tokens` tokens, then the prompt queried (Eq. 3 with request-bounded matches), with and without the
    intra-sequence pass, and the wave split.  CUDA-event times; appends are timed as one sequence."""
    import torch
    from paper_2608_04991_b200 import binding as rac
    from paper_2608_04991_b200 import synth
    tw = synth.span_workload(n_hist, n_query, seed=synth.BASE_SEED + 11, gap_max=gap_max)
    htok = torch.from_numpy(tw.hist).to(dev)
    qtok = torch.from_numpy(tw.query).to(dev)
    cfg = rac.IndexCfg(n_hist, WORKLOAD["min_ngram"], WORKLOAD["max_hits"])
    nb = rac.rac_index_bytes(cfg)
    mem = torch.empty(nb, dtype=torch.uint8, device=dev)
    nws = rac.rac_index_query_workspace_bytes(n_query)
    ws = torch.empty(nws, dtype=torch.uint8, device=dev)
    rows = torch.empty(n_query, dtype=torch.int32, device=dev)
    n_spans = torch.zeros(1, dtype=torch.int32, device=dev)
    wave1, wave2 = torch.empty_like(rows), torch.empty_like(rows)
    cnt = torch.zeros(2, dtype=torch.int32, device=dev)
    bounds = list(range(0, n_hist, request_tokens)) + [n_hist]

    def build():
        rac.rac_index_reset(cfg, mem, nb)
        for a, b in zip(bounds[:-1], bounds[1:]):
            rac.rac_index_append(cfg, mem, nb, htok, a, b)

    def timed(fn, n):
        fn()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        torch.cuda.synchronize()
        e0.record()
        for _ in range(n):
            fn()
        e1.record()
        torch.cuda.synchronize()
        return e0.elapsed_time(e1) / n

    out = {"history_tokens": n_hist, "query_tokens": n_query, "requests": len(bounds) - 1, "index_bytes": nb}
    out["build_ms"] = timed(build, 3)
    out["append_us_per_request"] = out["build_ms"] * 1e3 / (len(bounds) - 1)
    q = lambda intra: rac.rac_index_query(cfg, mem, nb, htok, n_hist, qtok, n_query, intra, rows, None, n_spans, ws, nws)
    out["query_ms"] = timed(lambda: q(False), reps)
    out["query_with_intra_ms"] = timed(lambda: q(True), reps)
    out["split_waves_ms"] = timed(lambda: rac.rac_split_waves(rows, n_query, n_hist, wave1, wave2, cnt), reps)
    r = rows.cpu()
    out["spans"] = int(n_spans.item())
    out["covered_by_spans"] = float(((r >= 0) & (r < n_hist)).float().mean())
    out["intra_referenced"] = float((r >= n_hist).float().mean())
    return out


# --------------------------------------------------------------------------------------------- receiver/encoder sweep
def config3_sweep(dev, peak, T=16384, d=4096, k=8, sets=3, reps=12):
    """b in {2,3,4} x group in {64,128}, top-8 outliers per token, T x d inputs from the single-sequence prefill
    generator: `rac_encode` and `rac_decode_reconstruct` timed separately with CUDA events.  A tensor is 134 MB, just
    above the 126 MB L2, and consecutive launches rotate over `sets` independent input/output sets, so no launch
    finds its tensors in cache.  GB/s over the algorithmic bytes (X + reference + record, record + reference +
    x_hat); `frac` of the measured copy bandwidth."""
    import torch
    from paper_2608_04991_b200 import binding as rac
    from paper_2608_04991_b200 import synth
    gen = synth.generator(synth.BASE_SEED + 3, dev)
    scale = synth.channel_scale(d, 3, dev)
    Xs = [synth.activations(T, d, scale, gen) for _ in range(sets)]
    status = torch.zeros(1, dtype=torch.int32, device=dev)
    out = []
    for g in (64, 128):
        Rs = [synth.affine_noisy_reference(X, g, gen) for X in Xs]
        for bits in (2, 3, 4):
            cfg = rac.CodecCfg(d, g, bits, k)
            rec = rac.rac_record_bytes(cfg)
            step = torch.empty((2, d), dtype=torch.float32, device=dev)
            inv = torch.empty_like(step)
            nb = rac.rac_calibrate_workspace_bytes(cfg)
            cws = torch.empty(nb, dtype=torch.uint8, device=dev)
            rac.rac_calibrate_steps(cfg, Xs[0][:1024], 1024, Rs[0], T, None, None, None, 3.0, step, inv, cws, nb, status)
            pays = [torch.empty(T * rec, dtype=torch.uint8, device=dev) for _ in range(sets)]
            xhs = [torch.empty_like(Xs[0]) for _ in range(sets)]
            nws = rac.rac_encode_workspace_bytes(cfg, T)
            ews = torch.empty(nws, dtype=torch.uint8, device=dev)
            enc = lambda i: rac.rac_encode(cfg, Xs[i], T, Rs[i], T, None, None, None, step, inv, pays[i], pays[i].numel(),
                                           ews, nws, status)
            dec = lambda i: rac.rac_decode_reconstruct(cfg, pays[i], T, Rs[i], T, None, None, None, step, xhs[i], status)
            row = {"bits": bits, "group": g, "record_bytes": rec}
            nbytes = T * (4 * d + rec)
            for key, fn in (("encode", enc), ("decode", dec)):
                for i in range(sets):
                    fn(i)
                e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                torch.cuda.synchronize()
                e0.record()
                for r in range(reps):
                    fn(r % sets)
                e1.record()
                torch.cuda.synchronize()
                ms = e0.elapsed_time(e1) / reps
                row[key + "_ms"] = ms
                row[key + "_GBps"] = nbytes / (ms * 1e-3) / 1e9
                row[key + "_frac"] = row[key + "_GBps"] / peak
            out.append(row)
    if int(status.item()) != 0:
        raise RuntimeError(f"config3_sweep: device status {int(status.item())}")
    return {"T": T, "d": d, "topk": k, "buffer_sets": sets, "launches_timed": reps, "points": out,
            "note": "payloads decoded are the device's own encodes of the same inputs (bit-identical to the oracle's but "
                    "for coefficient words inside the rounding window, see the parity tests)"}


# --------------------------------------------------------------------------------------------- fidelity of the round trip
def fidelity(rt):
    """What the codec did to the benchmark's tensors, per direction (Eq. 10-11): relative RMS error and largest
    absolute error of the reconstruction (rac_recon_error: binary64 sums on the device), and the clip rate = share of
    dense codes at +-Qmax (the static table clips at 3 sigma by design; a code at the rail is either exactly on it or
    clipped)."""
    import torch
    rac, wl, dev = rt.rac, rt.wl, rt.dev
    T, d, bits, J = wl["T"], wl["d"], wl["bits"], wl["d"] // wl["group"]
    qmax = (1 << (bits - 1)) - 1
    nb = rac.rac_recon_error_workspace_bytes()
    ws = torch.empty(nb, dtype=torch.uint8, device=dev)
    acc = torch.zeros(3, dtype=torch.float64, device=dev)
    out = {}
    for name, X, Xh, pay in (("uplink", rt.X, rt.Xh, rt.pay_up), ("downlink", rt.Y, rt.Yh, rt.pay_dn)):
        rac.rac_recon_error(X, Xh, T, d, acc, ws, nb)
        se, sx, mx = (float(v) for v in acc.cpu())
        rail = 0
        if bits == 4:       # two codes per byte, two's complement: +Qmax = 0x7, -Qmax = 0x9
            codes = pay.view(T, rt.rec)[:, 4 * J: 4 * J + d // 2]
            for t0 in range(0, T, 16384):
                c = codes[t0:t0 + 16384]
                lo, hi = c & 15, c >> 4
                rail += int(((lo == qmax) | (lo == 16 - qmax)).sum().item()) + int(((hi == qmax) | (hi == 16 - qmax)).sum().item())
        out[name] = {"relative_rms_error": (se / sx) ** 0.5 if sx > 0 else None, "max_abs_error": mx,
                     "rms_of_input": (sx / (T * d)) ** 0.5,
                     "clip_rate": rail / float(T * d) if bits == 4 else None}
    return out


# --------------------------------------------------------------------------------------------- decode-step latency
def decode_step_latency(dev, n_steps=64, reps=20):
    """Config 2 (64 sequences x 1 token, d=3584, 3-bit, group 128, no outliers, per-channel gain/bias reference,
    x_hat fed back): microseconds per step of the sender call (encode + x_hat in one launch, in place) and of the
    receiver call, launched eagerly and replayed from a CUDA graph of `n_steps` dependent steps."""
    import torch
    from paper_2608_04991_b200 import binding as rac
    from paper_2608_04991_b200 import synth
    B, d, g, bits = 64, 3584, 128, 3
    cfg = rac.CodecCfg(d, g, bits, 0)
    gen = synth.generator(synth.BASE_SEED + 2, dev)
    scale = synth.channel_scale(d, 2, dev)
    gain, bias = synth.predictor_gain_bias(d, 2, dev)
    xs = [synth.activations(B, d, scale, gen)]
    for _ in range(n_steps):
        xs.append(synth.random_walk_step(xs[-1], gen))
    step = torch.empty((2, d), dtype=torch.float32, device=dev)
    inv = torch.empty_like(step)
    nb = rac.rac_calibrate_workspace_bytes(cfg)
    ws = torch.empty(nb, dtype=torch.uint8, device=dev)
    status = torch.zeros(1, dtype=torch.int32, device=dev)
    rac.rac_calibrate_steps(cfg, xs[1], B, xs[0], B, None, gain, bias, 3.0, step, inv, ws, nb, status)
    rec = rac.rac_record_bytes(cfg)
    pays = [torch.empty(B * rec, dtype=torch.uint8, device=dev) for _ in range(n_steps)]
    send_state, recv_state = xs[0].clone(), xs[0].clone()      # the first step travels raw

    def sender():
        for t in range(n_steps):
            rac.rac_encode_reconstruct(cfg, xs[t + 1], B, send_state, B, None, gain, bias, step, inv, pays[t],
                                       pays[t].numel(), send_state, None, 0, status)

    def receiver():
        for t in range(n_steps):
            rac.rac_decode_reconstruct(cfg, pays[t], B, recv_state, B, None, gain, bias, step, recv_state, status)

    # the same calls with their arguments marshalled once (binding.prepare): what a decode loop with fixed buffers does
    send_calls = [rac.prepare(rac.rac_encode_reconstruct, cfg, xs[t + 1], B, send_state, B, None, gain, bias, step, inv,
                              pays[t], pays[t].numel(), send_state, None, 0, status) for t in range(n_steps)]
    recv_calls = [rac.prepare(rac.rac_decode_reconstruct, cfg, pays[t], B, recv_state, B, None, gain, bias, step,
                              recv_state, status) for t in range(n_steps)]

    def run_prepared(calls):
        for c in calls:
            c()

    out = {}
    prepared = {"sender_encode_plus_xhat": send_calls, "receiver_reconstruct": recv_calls}
    for name, fn, state in (("sender_encode_plus_xhat", sender, send_state), ("receiver_reconstruct", receiver, recv_state)):
        fn()                                                    # warm-up (also does the one-time function set-up)
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for _ in range(reps):
            fn()
        e1.record()
        torch.cuda.synchronize()
        eager = e0.elapsed_time(e1) * 1e3 / (reps * n_steps)
        run_prepared(prepared[name])
        torch.cuda.synchronize()
        e0.record()
        for _ in range(reps):
            run_prepared(prepared[name])
        e1.record()
        torch.cuda.synchronize()
        prep = e0.elapsed_time(e1) * 1e3 / (reps * n_steps)
        graph = torch.cuda.CUDAGraph()
        side = torch.cuda.Stream()
        side.wait_stream(torch.cuda.current_stream())
        with torch.cuda.stream(side):
            with torch.cuda.graph(graph, stream=side):
                fn()
        torch.cuda.current_stream().wait_stream(side)
        graph.replay()
        torch.cuda.synchronize()
        e0.record()
        for _ in range(reps):
            graph.replay()
        e1.record()
        torch.cuda.synchronize()
        out[name] = {"us_per_step_eager": eager, "us_per_step_prepared_call": prep,
                     "us_per_step_cuda_graph": e0.elapsed_time(e1) * 1e3 / (reps * n_steps)}
    # one clean chain from the common first state: both ends must arrive at the same state
    send_state.copy_(xs[0])
    recv_state.copy_(xs[0])
    sender()
    receiver()
    torch.cuda.synchronize()
    if int(status.item()):
        raise SystemExit(f"decode-step latency: device status {int(status.item())}")
    if not torch.equal(send_state, recv_state):
        raise SystemExit("decode-step latency: sender and receiver states differ")
    out["config"] = {"sequences": B, "d": d, "bits": bits, "group": g, "steps_per_graph": n_steps}
    return out


# --------------------------------------------------------------------------------------------- CPU oracle legs
class OracleSample:
    """The CPU oracle on a bounded sample of the workload: the full span match, and the codec calls of one
    step (uplink encode + sender and receiver reconstruction, downlink encode + reconstruction) on the
    first `sample_tokens` tokens.  Inputs are drawn once; `run()` times one pass."""

    def __init__(self, wl, seed, sample_tokens):
        import numpy as np
        import torch
        import oracle
        from paper_2608_04991_b200 import synth
        self.orc, self.wl = oracle, wl
        T, d, g, bits = wl["T"], wl["d"], wl["group"], wl["bits"]
        self.S = S = min(sample_tokens, T)
        # every core this process may run on (a launcher may have set OMP_NUM_THREADS=1; the oracle takes its
        # thread count as an argument, so that does not bind it)
        self.cores = max(1, min(64, len(os.sched_getaffinity(0))))
        self.tw = tw = synth.span_workload(wl["n_hist"], T, seed=seed, gap_max=wl["gap_max"])
        rows, _ = oracle.match_spans(tw.hist, tw.query, wl["min_ngram"], wl["max_hits"])
        # activations only for the history rows the sample needs
        gen = synth.generator(synth.BASE_SEED + seed, "cpu")
        scale = synth.channel_scale(d, seed, "cpu")
        r = rows[:S]
        need = np.unique(r[r >= 0])
        Hc = synth.activations(max(1, need.size), d, scale, gen)
        self.compact = compact = np.full(S, -1, np.int32)
        compact[r >= 0] = np.searchsorted(need, r[r >= 0]).astype(np.int32)
        X = synth.affine_noisy_target(Hc, torch.from_numpy(compact), g, gen, scale)
        self.Xb, self.Hb = synth.bf16_bits(X), synth.bf16_bits(Hc)
        c = min(S, 512)
        self.step_up, self.inv_up = oracle.calibrate(d, g, bits, self.Xb[:c], ref_base=self.Hb, ref_row=compact[:c])
        pay = oracle.encode(d, g, bits, wl["topk"], self.Xb, ref_base=self.Hb, ref_row=compact, step=self.step_up,
                            inv_step=self.inv_up, nthreads=self.cores)
        xh = oracle.reconstruct(d, g, bits, wl["topk"], pay, S, ref_base=self.Hb, ref_row=compact, step=self.step_up,
                                nthreads=self.cores)
        self.Yb = synth.bf16_bits(synth.drifted_state(synth.bf16_from_bits(xh), gen))
        self.step_dn, self.inv_dn = oracle.calibrate(d, g, bits, self.Yb[:c], ref_base=xh[:c])

    def run(self, nthreads=None):
        """One timed pass.  Returns (GB/s of activations for a whole step, description, seconds of this pass).
        With a sample of all T tokens the pass IS a whole step and nothing is scaled."""
        o, wl, S = self.orc, self.wl, self.S
        T, d, g, bits, k = wl["T"], wl["d"], wl["group"], wl["bits"], wl["topk"]
        n = self.cores if nthreads is None else nthreads
        t0 = time.perf_counter()
        o.match_spans(self.tw.hist, self.tw.query, wl["min_ngram"], wl["max_hits"])
        t1 = time.perf_counter()
        pay = o.encode(d, g, bits, k, self.Xb, ref_base=self.Hb, ref_row=self.compact, step=self.step_up,
                       inv_step=self.inv_up, nthreads=n)
        o.reconstruct(d, g, bits, k, pay, S, ref_base=self.Hb, ref_row=self.compact, step=self.step_up, nthreads=n)
        xh = o.reconstruct(d, g, bits, k, pay, S, ref_base=self.Hb, ref_row=self.compact, step=self.step_up, nthreads=n)
        t2 = time.perf_counter()
        pay2 = o.encode(d, g, bits, k, self.Yb, ref_base=xh, step=self.step_dn, inv_step=self.inv_dn, nthreads=n)
        o.reconstruct(d, g, bits, k, pay2, S, ref_base=xh, step=self.step_dn, nthreads=n)
        t3 = time.perf_counter()
        t_match, t_up, t_dn = t1 - t0, t2 - t1, t3 - t2
        est_step = t_match + (t_up + t_dn) * (T / S)
        gbs = 2 * 2 * T * d / est_step / 1e9
        scaled = "nothing scaled" if S == T else f"codec time scaled by {T / S:.0f}x"
        desc = (f"full span match ({wl['n_hist']} history, {T} query tokens: {t_match:.3f} s) + codec on "
                f"{'all' if S == T else 'the first ' + str(S) + ' of'} {T} tokens (uplink encode + 2 reconstructions "
                f"{t_up:.2f} s, downlink encode + reconstruction {t_dn:.2f} s), {scaled}; {n} OpenMP thread(s), "
                f"gcc -O2 -ffp-contract=off")
        return gbs, desc, t3 - t0


L2_NOTE = "inputs larger than L2 (126 MB): every tensor of a call is 0.13 GB or more and is streamed once; no flush needed"


def bench_config(wl, small):
    """The `config` object, identical in both arms."""
    return {"workload": "long-context round trip (config 4)" + (" SMALL" if small else ""), **wl, "l2": L2_NOTE}


def run_reference(args, wl):
    """The CPU oracle as it stands, on the host cores, over the WHOLE workload: every step is one full pass (all T
    tokens), timed by wall clock.  The number of steps is cut so that the arm ends within about two minutes."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return 0
    smp = OracleSample(wl, seed=4, sample_tokens=wl["T"])
    budget_s = 100.0
    vals, secs, desc = [], [], None
    warm = min(args.warmup, 1)
    _, _, first = smp.run() if warm else (None, None, 5.0)
    steps = max(1, min(args.steps, int(budget_s / max(first, 1e-3))))
    for _ in range(steps):
        gbs, desc, sec = smp.run()
        vals.append(gbs)
        secs.append(sec)
    value = 2 * 2 * wl["T"] * wl["d"] / (sum(secs) / len(secs)) / 1e9
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus, "steps": steps,
        "warmup": warm, "ms_per_step": 1e3 * sum(secs) / len(secs), "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "f32", "data": "synthetic",
        "config": bench_config(wl, args.small),
        "note": f"CPU oracle on the whole workload, wall clock; ran {steps} of the {args.steps} steps asked for "
                f"(a step takes {sum(secs) / len(secs):.1f} s)",
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": smp.cores, "kind": "oracle", "sample": desc},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line))
    return 0


# --------------------------------------------------------------------------------------------- main
def main():
    args = parse_args()
    wl = dict(SMALL if args.small else WORKLOAD)
    if args.impl == "reference":
        return run_reference(args, wl)

    import torch
    import torch.distributed as dist
    from paper_2608_04991_b200 import binding as rac
    rac.load()  # fails loudly when the CUDA library is missing
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device (there is no CPU fallback)")
    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    if world > 1:
        dist.init_process_group("nccl", device_id=dev)
    assert world == args.gpus, f"--gpus {args.gpus} but WORLD_SIZE {world}"

    if args.sweep_only:
        if rank == 0:
            print(json.dumps({"sweep": config3_sweep(dev, measured_peak()[0])}))
        return 0
    strong = args.scaling == "strong"
    if strong:
        # one tensor, the same on every rank; rank r codes the token range shard.token_range(T, r, world) against its
        # own replica of the history states, and the payload byte ranges are gathered into every rank's own buffer
        from paper_2608_04991_b200 import shard
        rt = RoundTrip(wl, seed=4, dev=dev, token_range=shard.token_range(wl["T"], rank, world))
        byte_ranges = [shard.payload_range(rt.rec, x, y) for x, y in shard.all_ranges(wl["T"], world)]

        def exchange():
            shard.all_gather_ranges(rt.pay_up, byte_ranges, rank)
            shard.all_gather_ranges(rt.pay_dn, byte_ranges, rank)
        rt.exchange = exchange
        rt.STAGES = rt.STAGES + ["exchange"]
    else:
        rt = RoundTrip(wl, seed=4 + rank, dev=dev)   # every rank codes its own sequences: no data-path collective
    nst = len(rt.STAGES)
    steps, warm = args.steps, max(args.warmup, 3)

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    for _ in range(warm):
        rt.step()
    ev = [[torch.cuda.Event(enable_timing=True) for _ in range(nst + 1)] for _ in range(steps)]
    sampler = ClockSampler(local)
    barrier()
    sampler.start()
    for i in range(steps):
        rt.step(ev[i])
    barrier()
    sampler.stop()
    total_ms = ev[0][0].elapsed_time(ev[-1][nst])
    stage_ms = [sum(ev[i][s].elapsed_time(ev[i][s + 1]) for i in range(steps)) / steps for s in range(nst)]
    status = int(rt.status.item())
    if status:
        raise SystemExit(f"device status {status}: results invalid")
    t = torch.tensor([total_ms], dtype=torch.float64, device=dev)
    if world > 1:
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
    total_ms = float(t.item())
    ms_per_step = total_ms / steps
    act = rt.activation_bytes_per_step()
    value = (1 if strong else world) * act / (ms_per_step * 1e-3) / 1e9
    strong_check = None
    if strong:
        # the gathered payloads against one rank coding the whole tensor (untimed)
        got_up, got_dn = rt.pay_up.clone(), rt.pay_dn.clone()
        mine = (rt.a, rt.b)
        rt.a, rt.b = 0, wl["T"]
        rt.encode_sender_up()
        rt.decode_up()
        rt.encode_dn()
        torch.cuda.synchronize()
        strong_check = bool(torch.equal(got_up, rt.pay_up) and torch.equal(got_dn, rt.pay_dn))
        if not strong_check:
            raise SystemExit(f"rank {rank}: the gathered payload differs from the single-rank payload")
        rt.a, rt.b = mine

    # ---- end to end: inputs from pinned host memory, payloads and final activations back to the host
    e2e = None
    if not args.no_e2e and not strong:     # the end-to-end number belongs to the default (weak) mode
        T, d = wl["T"], wl["d"]
        pin = lambda t_: torch.empty(t_.shape, dtype=t_.dtype, pin_memory=True).copy_(t_)
        hX, hY, hq = pin(rt.X), pin(rt.Y), pin(rt.query)
        o_up = torch.empty(rt.pay_up.shape, dtype=torch.uint8, pin_memory=True)
        o_dn = torch.empty(rt.pay_dn.shape, dtype=torch.uint8, pin_memory=True)
        o_Y = torch.empty(rt.Yh.shape, dtype=torch.bfloat16, pin_memory=True)
        assert all(t_.is_pinned() for t_ in (hX, hY, hq, o_up, o_dn, o_Y)), "end-to-end buffers must be pinned"
        h2d = hX.numel() * 2 + hY.numel() * 2 + hq.numel() * 4
        d2h = o_up.numel() * 2 + o_Y.numel() * 2
        n_e2e = max(4, min(steps, 12))
        # Three streams, two buffer sets: while step i computes, the inputs of step i+1 arrive and the results of
        # step i-1 leave.  Every step still copies all of its inputs in and all of its results out.
        s_in, s_comp, s_out = torch.cuda.Stream(), torch.cuda.Stream(), torch.cuda.Stream()
        ins = [(rt.X, rt.Y, rt.query), (torch.empty_like(rt.X), torch.empty_like(rt.Y), torch.empty_like(rt.query))]
        outs = [(rt.pay_up, rt.pay_dn, rt.Yh),
                (torch.empty_like(rt.pay_up), torch.empty_like(rt.pay_dn), torch.empty_like(rt.Yh))]
        ev_in = [torch.cuda.Event() for _ in range(2)]
        ev_comp = [torch.cuda.Event() for _ in range(2)]
        ev_out = [torch.cuda.Event() for _ in range(2)]

        def e2e_step(i):
            j = i & 1
            with torch.cuda.stream(s_in):
                s_in.wait_event(ev_comp[j])          # the compute that last read this input set has finished
                ins[j][2].copy_(hq, non_blocking=True)
                ins[j][0].copy_(hX, non_blocking=True)
                ins[j][1].copy_(hY, non_blocking=True)
                ev_in[j].record(s_in)
            with torch.cuda.stream(s_comp):
                s_comp.wait_event(ev_in[j])
                s_comp.wait_event(ev_out[j])         # the copy-out that last read this output set has finished
                rt.X, rt.Y, rt.query = ins[j]
                rt.pay_up, rt.pay_dn, rt.Yh = outs[j]
                rt.step()
                ev_comp[j].record(s_comp)
            with torch.cuda.stream(s_out):
                s_out.wait_event(ev_comp[j])
                o_up.copy_(outs[j][0], non_blocking=True)
                o_dn.copy_(outs[j][1], non_blocking=True)
                o_Y.copy_(outs[j][2], non_blocking=True)
                ev_out[j].record(s_out)

        for s_ in (s_in, s_comp, s_out):
            s_.wait_stream(torch.cuda.current_stream())
        e2e_step(0)
        e2e_step(1)
        for s_ in (s_in, s_comp, s_out):
            torch.cuda.current_stream().wait_stream(s_)
        barrier()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for s_ in (s_in, s_comp, s_out):
            s_.wait_stream(torch.cuda.current_stream())
        for i in range(n_e2e):
            e2e_step(i)
        for s_ in (s_in, s_comp, s_out):
            torch.cuda.current_stream().wait_stream(s_)
        e1.record()
        barrier()
        rt.X, rt.Y, rt.query = ins[0]
        rt.pay_up, rt.pay_dn, rt.Yh = outs[0]
        if int(rt.status.item()):
            raise SystemExit(f"device status {int(rt.status.item())} in the end-to-end loop")
        te = torch.tensor([e0.elapsed_time(e1)], dtype=torch.float64, device=dev)
        if world > 1:
            dist.all_reduce(te, op=dist.ReduceOp.MAX)
        e2e = {"value": world * act / (float(te.item()) / n_e2e * 1e-3) / 1e9, "unit": UNIT, "h2d_bytes_per_step": h2d,
               "d2h_bytes_per_step": d2h, "steps": n_e2e,
               "note": "copy-in, compute and copy-out of consecutive steps overlap (3 streams, 2 buffer sets)"}

    if rank == 0:
        peak, peak_src = measured_peak()
        names = rt.STAGES
        per = {n: {"ms": stage_ms[i], "GB/s_algorithmic": (rt.bytes_of(n) / (stage_ms[i] * 1e-3) / 1e9) if rt.bytes_of(n) else None,
                   "GB/s_activations_in": 2 * wl["T"] * wl["d"] / (stage_ms[i] * 1e-3) / 1e9 if n != "match" else None}
               for i, n in enumerate(names)}
        ix = {n: i for i, n in enumerate(names)}
        enc_ms = stage_ms[ix["encode_sender_up"]] + stage_ms[ix["encode_dn"]]
        dec_ms = stage_ms[ix["decode_up"]] + stage_ms[ix["decode_dn"]]
        if enc_ms >= dec_ms:
            dom, dom_bytes, dom_ms, dom_n = ("rac_encode[_reconstruct] (encode_ws_kernel<4,true,*> + outlier_kernel<4>)",
                                             rt.bytes_of("encode_sender_up") + rt.bytes_of("encode_dn"), enc_ms, 2)
        else:
            dom, dom_bytes, dom_ms, dom_n = ("decode_ws_kernel<4,8>", rt.bytes_of("decode_up") + rt.bytes_of("decode_dn"),
                                             dec_ms, 2)
        achieved = dom_bytes / (dom_ms * 1e-3) / 1e9
        dom_stages = ("encode_sender_up", "encode_dn") if enc_ms >= dec_ms else ("decode_up", "decode_dn")
        traffic = sum(NCU_SMALL_CASE_TRAFFIC[n] for n in dom_stages) / len(dom_stages) * (wl["T"] / 16384.0)
        roofline = {"bound": "hbm", "kernel": dom, "achieved": achieved, "peak": peak, "unit": "GB/s", "frac": achieved / peak,
                    "traffic": traffic, "traffic_source": "ncu small case (T=16384) scaled by tokens, bytes per call", "peak_source": peak_src, "launches_per_step": dom_n,
                    "algorithmic_bytes_per_launch": dom_bytes / dom_n, "avg_launch_ms": dom_ms / dom_n,
                    "frac_of_nominal_8TBps": achieved / 8000.0}
        cpu = None
        if not args.no_cpu_baseline:
            smp = OracleSample(wl, seed=4, sample_tokens=wl["T"])       # one pass over the whole workload
            gbs, desc, _ = smp.run()
            one = OracleSample(wl, seed=4, sample_tokens=min(wl["T"], 4096))
            gbs1, desc1, _ = one.run(nthreads=1)
            cpu = {"value": gbs, "unit": UNIT, "cores": smp.cores, "kind": "oracle", "sample": desc,
                   "one_thread": {"value": gbs1, "unit": UNIT, "cores": 1, "sample": desc1}}
        line = {
            "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": steps, "warmup": warm,
            "ms_per_step": ms_per_step, "higher_is_better": True, "scaling": args.scaling, "vs_baseline": None,
            "strong_scaling_check": strong_check,
            "dtype": "f32", "data": "synthetic",
            "config": bench_config(wl, args.small),
            "workload_stats": {"record_bytes": rt.rec, "matched_coverage": rt.coverage, "planted_coverage": rt.planted_coverage,
                               "tokens_per_s": (1 if strong else world) * wl["T"] / (ms_per_step * 1e-3)},
            "clocks": sampler.summary(),
            "e2e": e2e,
            "gpu_launches": rt.LAUNCHES_PER_STEP * steps,
            "roofline": roofline,
            "cpu_baseline": cpu,
            "stages": per,
            "fidelity": fidelity(rt),
            "sweep": None if args.no_sweep else config3_sweep(dev, peak),
            "decode_steps": None if args.no_decode_steps else decode_step_latency(dev),
            "paper_family": None if args.no_family else paper_family(dev, wl["T"], wl["d"]),
            "retrieval_index": None if args.no_family else retrieval_index(dev, wl["n_hist"], wl["T"], wl["gap_max"]),
            "shared_coefficients": None if args.no_family else shared_coefficients(dev, wl["T"], wl["d"]),
        }
        print(json.dumps(line))
    if world > 1:
        dist.destroy_process_group()
    return 0


if __name__ == "__main__":
    sys.exit(main())
