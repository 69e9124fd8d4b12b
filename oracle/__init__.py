"""CPU oracle of the RAC codec hot path -- TEST INFRASTRUCTURE ONLY.

Thin ctypes wrapper around ``rac_oracle.c`` (plain scalar C written from the
paper's Sec. IV-B.1 and IV-C).  Only the tests, the smoke check and the
``cpu_baseline`` / ``--impl reference`` legs of the benchmark may import this
package; the product (``paper_2608_04991_b200``) never does and shares no code
with it.

Arrays are numpy: bf16 and binary16 tensors travel as ``uint16`` bit patterns.
"""
from __future__ import annotations

import ctypes as C
import os
import subprocess
from typing import Optional

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "rac_oracle.c")
_LIB = os.path.join(_HERE, "liboracle.so")
CFLAGS = ["-O2", "-ffp-contract=off", "-fopenmp", "-fPIC", "-shared", "-std=c11"]


def build(force: bool = False) -> str:
    """Compile the oracle with gcc (no-op when the library is newer than its source)."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        tmp = _LIB + f".tmp{os.getpid()}"
        subprocess.check_call(["gcc", *CFLAGS, _SRC, "-o", tmp, "-lm"])
        os.replace(tmp, _LIB)
    return _LIB


_lib = None


def lib() -> C.CDLL:
    global _lib
    if _lib is None:
        _lib = C.CDLL(build())
        _declare(_lib)
    return _lib


_u16p = C.POINTER(C.c_uint16)
_u8p = C.POINTER(C.c_uint8)
_i32p = C.POINTER(C.c_int32)
_u32p = C.POINTER(C.c_uint32)
_f32p = C.POINTER(C.c_float)
_f64p = C.POINTER(C.c_double)


def _declare(l: C.CDLL) -> None:
    l.orc_bf16_to_f32.restype = C.c_float
    l.orc_bf16_to_f32.argtypes = [C.c_uint16]
    l.orc_f32_to_bf16.restype = C.c_uint16
    l.orc_f32_to_bf16.argtypes = [C.c_float]
    l.orc_f16_to_f64.restype = C.c_double
    l.orc_f16_to_f64.argtypes = [C.c_uint16]
    l.orc_f64_to_f16.restype = C.c_uint16
    l.orc_f64_to_f16.argtypes = [C.c_double]
    l.orc_f64_to_f16_up.restype = C.c_uint16
    l.orc_f64_to_f16_up.argtypes = [C.c_double]
    l.orc_record_bytes.restype = C.c_int64
    l.orc_record_bytes.argtypes = [C.c_int] * 4
    l.orc_record_bytes_mode.restype = C.c_int64
    l.orc_record_bytes_mode.argtypes = [C.c_int] * 5
    l.orc_record_bytes_ext.restype = C.c_int64
    l.orc_record_bytes_ext.argtypes = [C.c_int] * 7
    l.orc_record_bytes_full.restype = C.c_int64
    l.orc_record_bytes_full.argtypes = [C.c_int] * 8
    l.orc_fit_segments.restype = C.c_int
    l.orc_fit_segments.argtypes = [C.c_int, C.c_int, _u16p, C.c_int64, _u16p, C.c_int64, _i32p, _u16p, _u16p,
                                   _i32p, C.c_int32, _u32p, _f64p, _f64p, _f64p, _f64p]
    l.orc_pack_codes.restype = None
    l.orc_pack_codes.argtypes = [_i32p, C.c_int, C.c_int, _u8p]
    l.orc_unpack_codes.restype = None
    l.orc_unpack_codes.argtypes = [_u8p, C.c_int, C.c_int, _i32p]
    l.orc_fit_group.restype = None
    l.orc_fit_group.argtypes = [_f32p, _f32p, C.c_int, C.c_int, _f64p, _f64p, _f64p, _f64p]
    l.orc_encode.restype = C.c_int
    l.orc_encode.argtypes = [C.c_int] * 8 + [_u16p, C.c_int64, _u16p, C.c_int64, _i32p, _u16p, _u16p,
                                             _f32p, _f32p, _u32p, _u8p,
                                             _f64p, _f64p, _f64p, _f64p, _f32p, _f32p, _f64p, C.c_int]
    l.orc_reconstruct.restype = C.c_int
    l.orc_reconstruct.argtypes = [C.c_int] * 8 + [_u32p, _u8p, C.c_int64, _u16p, C.c_int64, _i32p, _u16p, _u16p,
                                                  _f32p, _u16p, _u32p, C.c_int]
    l.orc_calibrate.restype = C.c_int
    l.orc_calibrate.argtypes = [C.c_int] * 3 + [_u16p, C.c_int64, _u16p, C.c_int64, _i32p, _u16p, _u16p,
                                                C.c_double, _f32p, _f32p]
    l.orc_calibrate_shared.restype = C.c_int
    l.orc_calibrate_shared.argtypes = [C.c_int] * 3 + [_u16p, C.c_int64, _u16p, C.c_int64, _i32p, _u16p, _u16p, _u32p,
                                                       C.c_double, _f32p, _f32p]
    l.orc_match_spans.restype = C.c_int
    l.orc_match_spans.argtypes = [_i32p, C.c_int64, _i32p, C.c_int64, C.c_int, C.c_int, _i32p, _i32p, _i32p]
    l.orc_match_spans_req.restype = C.c_int
    l.orc_match_spans_req.argtypes = [_i32p, C.c_int64, _i32p, C.c_int32, _i32p, C.c_int64, C.c_int, C.c_int, C.c_int,
                                      _i32p, _i32p, _i32p]
    l.orc_match_spans_live.restype = C.c_int
    l.orc_match_spans_live.argtypes = [_i32p, C.c_int64, _i32p, C.c_int32, _i32p, C.c_int64, C.c_int, C.c_int, C.c_int,
                                       C.c_int64, _i32p, _i32p, _i32p]
    l.orc_max_threads.restype = C.c_int
    l.orc_max_threads.argtypes = []


def _p(a: Optional[np.ndarray], typ):
    if a is None:
        return typ()
    assert a.flags["C_CONTIGUOUS"], "oracle arrays must be contiguous"
    return a.ctypes.data_as(typ)


def _chk(a: Optional[np.ndarray], dtype, n: Optional[int] = None) -> Optional[np.ndarray]:
    if a is None:
        return None
    a = np.ascontiguousarray(a)
    assert a.dtype == np.dtype(dtype), f"expected {np.dtype(dtype)}, got {a.dtype}"
    if n is not None:
        assert a.size == n, f"expected {n} elements, got {a.size}"
    return a


# ---------------------------------------------------------------- formats
def bf16_to_f32(bits: np.ndarray) -> np.ndarray:
    """bfloat16 bit patterns (uint16) -> float32 values (exact)."""
    return (bits.astype(np.uint32) << 16).view(np.float32)


def f32_to_bf16(x) -> np.ndarray:
    """float32 -> bfloat16 bit patterns, round to nearest even (scalar loop through the C routine)."""
    x = np.asarray(x, dtype=np.float32)
    out = np.empty(x.shape, np.uint16)
    l = lib()
    of, xf = out.reshape(-1), x.reshape(-1)
    for i in range(xf.size):
        of[i] = l.orc_f32_to_bf16(float(xf[i]))
    return out


def f64_to_f16(x: float) -> int:
    return int(lib().orc_f64_to_f16(float(x)))


def f64_to_f16_up(x: float) -> int:
    return int(lib().orc_f64_to_f16_up(float(x)))


def f16_to_f64(h: int) -> float:
    return float(lib().orc_f16_to_f64(int(h)))


def max_threads() -> int:
    return int(lib().orc_max_threads())


# ---------------------------------------------------------------- geometry
def record_bytes(d: int, group: int, bits: int, topk: int, scale_mode: int = 0, qgroup: int = 0,
                 topk_group: int = 0, coef_fmt: int = 0) -> int:
    return int(lib().orc_record_bytes_full(d, group, bits, topk, scale_mode, qgroup, topk_group, coef_fmt))


def split_payload(payload: np.ndarray, T: int, d: int, group: int, bits: int, topk: int, scale_mode: int = 0,
                  qgroup: int = 0, topk_group: int = 0, coef_fmt: int = 0):
    """Views into a payload: coef u32[T,J], codes u8[T,d*b/8], out_idx u16[T,k], out_val u16[T,k];
    for scale_mode 1 also scale u16[T,Jq] as a fifth item, and with per-group outliers
    grp_off u8[T,Jq,kg] (u16 when the group has more than 256 channels) and grp_val u16[T,Jq,kg] as a sixth and
    seventh."""
    J = d // group
    qg = qgroup or group
    Jq = d // qg
    rec = record_bytes(d, group, bits, topk, scale_mode, qgroup, topk_group, coef_fmt)
    p = payload.reshape(T, rec)
    nb = d * bits // 8
    sb = (2 * Jq + 3) // 4 * 4 if scale_mode == 1 else 0
    cb = 0 if coef_fmt == 1 else 4 * J          # shared coefficients travel outside the record: coef comes back empty
    o = cb + sb
    coef = np.ascontiguousarray(p[:, : cb]).view(np.uint32)
    codes = np.ascontiguousarray(p[:, o: o + nb])
    oi = np.ascontiguousarray(p[:, o + nb: o + nb + 2 * topk]).view(np.uint16)
    ov = np.ascontiguousarray(p[:, o + nb + 2 * topk: o + nb + 4 * topk]).view(np.uint16)
    if scale_mode != 1:
        return coef, codes, oi, ov
    scale = np.ascontiguousarray(p[:, cb: cb + 2 * Jq]).view(np.uint16)
    if not topk_group:
        return coef, codes, oi, ov, scale
    ng = Jq * topk_group
    g0 = o + nb + 4 * topk
    wide = qg > 256                            # two-byte offsets for groups of more than 256 channels
    g1 = g0 + (ng * (2 if wide else 1) + 1) // 2 * 2
    if wide:
        goff = np.ascontiguousarray(p[:, g0: g0 + 2 * ng]).view(np.uint16).reshape(T, Jq, topk_group)
    else:
        goff = np.ascontiguousarray(p[:, g0: g0 + ng]).reshape(T, Jq, topk_group)
    gval = np.ascontiguousarray(p[:, g1: g1 + 2 * ng]).view(np.uint16).reshape(T, Jq, topk_group)
    return coef, codes, oi, ov, scale, goff, gval


def pack_codes(q: np.ndarray, bits: int) -> np.ndarray:
    q = _chk(q, np.int32)
    d = q.size
    out = np.zeros(d * bits // 8, np.uint8)
    lib().orc_pack_codes(_p(q, _i32p), d, bits, _p(out, _u8p))
    return out


def unpack_codes(codes: np.ndarray, d: int, bits: int) -> np.ndarray:
    codes = _chk(codes, np.uint8, d * bits // 8)
    out = np.empty(d, np.int32)
    lib().orc_unpack_codes(_p(codes, _u8p), d, bits, _p(out, _i32p))
    return out


# ---------------------------------------------------------------- codec
def fit_group(h: np.ndarray, r: np.ndarray, has_ref: bool = True):
    """Eq. 6 for one group: returns (alpha*, beta*, mean(h), mean(r)) unrounded, in float64."""
    h = _chk(h, np.float32)
    r = _chk(r, np.float32, h.size)
    out = [C.c_double() for _ in range(4)]
    lib().orc_fit_group(_p(h, _f32p), _p(r, _f32p), h.size, int(has_ref), *[C.byref(o) for o in out])
    return tuple(o.value for o in out)


def encode(d, group, bits, topk, X, ref_base=None, ref_row=None, gain=None, bias=None,
           step=None, inv_step=None, forced_coef=None, diag=False, nthreads=1, scale_mode=0, qgroup=0, topk_group=0,
           coef_fmt=0):
    """Encode X (uint16 bf16 bits [T,d]).  Returns payload (uint8[T*rec]) and, with
    ``diag=True``, a dict of the unrounded fit, the binary32 residual ``e``, the binary32 scaled
    value ``v`` the codes were rounded from, and ``v_ideal`` = e / s with the quotient in binary64
    (Eq. 8 as printed; decides nothing, tests count the codes that differ from its rounding)."""
    X = _chk(X, np.uint16)
    T = X.size // d
    assert X.size == T * d
    ref_base = _chk(ref_base, np.uint16)
    ref_rows = 0 if ref_base is None else ref_base.size // d
    ref_row = _chk(ref_row, np.int32, T)
    gain = _chk(gain, np.uint16, d)
    bias = _chk(bias, np.uint16, d)
    step = _chk(step, np.float32, 2 * d)
    inv_step = _chk(inv_step, np.float32, 2 * d)
    assert scale_mode == 1 or (step is not None and inv_step is not None), "scale_mode 0 needs the step tables"
    J = d // group
    forced_coef = _chk(forced_coef, np.uint32, T * J)
    rec = record_bytes(d, group, bits, topk, scale_mode, qgroup, topk_group, coef_fmt)
    payload = np.zeros(T * rec, np.uint8)
    dg = {}
    if diag:    # diag="fit": only the per-group outputs (the per-channel ones are large)
        dg = dict(alpha=np.zeros((T, J)), beta=np.zeros((T, J)), hbar=np.zeros((T, J)), rbar=np.zeros((T, J)))
        if diag != "fit":
            dg.update(e=np.zeros((T, d), np.float32), v=np.zeros((T, d), np.float32),
                      v_ideal=np.zeros((T, d), np.float64))
    rc = lib().orc_encode(d, group, bits, topk, scale_mode, qgroup, topk_group, coef_fmt, _p(X, _u16p), T, _p(ref_base, _u16p), ref_rows,
                          _p(ref_row, _i32p), _p(gain, _u16p), _p(bias, _u16p),
                          _p(step, _f32p), _p(inv_step, _f32p), _p(forced_coef, _u32p), _p(payload, _u8p),
                          _p(dg.get("alpha"), _f64p), _p(dg.get("beta"), _f64p),
                          _p(dg.get("hbar"), _f64p), _p(dg.get("rbar"), _f64p),
                          _p(dg.get("e"), _f32p), _p(dg.get("v"), _f32p), _p(dg.get("v_ideal"), _f64p),
                          int(nthreads))
    if rc != 0:
        raise ValueError(f"orc_encode failed: {rc}")
    return (payload, dg) if diag else payload


def reconstruct(d, group, bits, topk, payload, T, ref_base=None, ref_row=None, gain=None, bias=None,
                step=None, nthreads=1, return_status=False, scale_mode=0, qgroup=0, topk_group=0, coef_fmt=0,
                shared_coef=None):
    """Eq. 9.  Returns X_hat as uint16 bf16 bits [T,d].  ``coef_fmt=1``: the records hold no coefficients;
    ``shared_coef`` uint32[T,J] gives every token the words of its segment."""
    rec = record_bytes(d, group, bits, topk, scale_mode, qgroup, topk_group, coef_fmt)
    shared_coef = _chk(shared_coef, np.uint32, T * (d // group))
    payload = _chk(payload, np.uint8, T * rec)
    ref_base = _chk(ref_base, np.uint16)
    ref_rows = 0 if ref_base is None else ref_base.size // d
    ref_row = _chk(ref_row, np.int32, T)
    gain = _chk(gain, np.uint16, d)
    bias = _chk(bias, np.uint16, d)
    step = _chk(step, np.float32, 2 * d)
    out = np.zeros((T, d), np.uint16)
    st = C.c_uint32(0)
    rc = lib().orc_reconstruct(d, group, bits, topk, scale_mode, qgroup, topk_group, coef_fmt, _p(shared_coef, _u32p), _p(payload, _u8p), T, _p(ref_base, _u16p), ref_rows,
                               _p(ref_row, _i32p), _p(gain, _u16p), _p(bias, _u16p), _p(step, _f32p),
                               _p(out, _u16p), C.byref(st), int(nthreads))
    if rc != 0:
        raise ValueError(f"orc_reconstruct failed: {rc}")
    return (out, st.value) if return_status else out


def calibrate(d, group, bits, X, ref_base=None, ref_row=None, gain=None, bias=None, clip_sigmas=3.0, shared_coef=None):
    """Step tables (step, inv_step), float32[2,d] each, from a calibration draw.  ``shared_coef`` uint32[T,J]: every
    token's residual is taken with the wire words of its segment (Eq. 6 over several fitting positions)."""
    X = _chk(X, np.uint16)
    T = X.size // d
    ref_base = _chk(ref_base, np.uint16)
    ref_rows = 0 if ref_base is None else ref_base.size // d
    ref_row = _chk(ref_row, np.int32, T)
    gain = _chk(gain, np.uint16, d)
    bias = _chk(bias, np.uint16, d)
    step = np.zeros((2, d), np.float32)
    inv = np.zeros((2, d), np.float32)
    if shared_coef is not None:
        shared_coef = _chk(shared_coef, np.uint32, T * (d // group))
        rc = lib().orc_calibrate_shared(d, group, bits, _p(X, _u16p), T, _p(ref_base, _u16p), ref_rows,
                                        _p(ref_row, _i32p), _p(gain, _u16p), _p(bias, _u16p), _p(shared_coef, _u32p),
                                        float(clip_sigmas), _p(step, _f32p), _p(inv, _f32p))
    else:
        rc = lib().orc_calibrate(d, group, bits, _p(X, _u16p), T, _p(ref_base, _u16p), ref_rows, _p(ref_row, _i32p),
                                 _p(gain, _u16p), _p(bias, _u16p), float(clip_sigmas), _p(step, _f32p), _p(inv, _f32p))
    if rc != 0:
        raise ValueError(f"orc_calibrate failed: {rc}")
    return step, inv


# ---------------------------------------------------------------- matcher
def match_spans(hist: np.ndarray, query: np.ndarray, w: int = 4, max_hits: int = 8):
    """Sec. IV-B.1.  Returns (ref_row int32[N], spans int32[n,3] as (q_start,h_start,len))."""
    hist = _chk(hist, np.int32)
    query = _chk(query, np.int32)
    N = query.size
    ref_row = np.full(N, -1, np.int32)
    spans = np.zeros((N // max(w, 1) + 1, 3), np.int32)
    ns = C.c_int32(0)
    rc = lib().orc_match_spans(_p(hist, _i32p), hist.size, _p(query, _i32p), N, int(w), int(max_hits),
                               _p(ref_row, _i32p), _p(spans, _i32p), C.byref(ns))
    if rc != 0:
        raise ValueError(f"orc_match_spans failed: {rc}")
    return ref_row, spans[: ns.value].copy()


def match_spans_req(hist: np.ndarray, req_off, query: np.ndarray, w: int = 4, max_hits: int = 8, intra: bool = False,
                    first_live: int = 0):
    """Sec. IV-B.1 with the history as a list of earlier requests (``req_off`` int32[n_req+1], or None for one
    request) and, with ``intra``, the intra-sequence references (rows >= len(hist)).  ``first_live``: only windows
    that start at or after this history position are candidates.  Returns (ref_row, spans)."""
    hist = _chk(hist, np.int32)
    query = _chk(query, np.int32)
    req_off = _chk(None if req_off is None else np.asarray(req_off, np.int32), np.int32)
    N = query.size
    ref_row = np.full(N, -1, np.int32)
    spans = np.zeros((N // max(w, 1) + 1, 3), np.int32)
    ns = C.c_int32(0)
    rc = lib().orc_match_spans_live(_p(hist, _i32p), hist.size, _p(req_off, _i32p),
                                    0 if req_off is None else req_off.size - 1, _p(query, _i32p), N, int(w),
                                    int(max_hits), int(bool(intra)), int(first_live), _p(ref_row, _i32p), _p(spans, _i32p),
                                    C.byref(ns))
    if rc != 0:
        raise ValueError(f"orc_match_spans_req failed: {rc}")
    return ref_row, spans[: ns.value].copy()


def recon_error(X_bits: np.ndarray, Xhat_bits: np.ndarray):
    """Reconstruction error of a run, in float64: (sum (x - x_hat)^2, sum x^2, max |x - x_hat|)."""
    x = bf16_to_f32(np.asarray(X_bits, np.uint16)).astype(np.float64)
    y = bf16_to_f32(np.asarray(Xhat_bits, np.uint16)).astype(np.float64)
    dlt = (x.astype(np.float32) - y.astype(np.float32)).astype(np.float64)   # the difference of two bf16 as binary32
    return float((dlt * dlt).sum()), float((x * x).sum()), float(np.abs(dlt).max(initial=0.0))


def fit_segments(d, group, X, seg_off, ref_base=None, ref_row=None, gain=None, bias=None, diag=False):
    """Eq. 6 over several fitting positions: one wire coefficient word per (segment, group).
    ``seg_off`` int32[n_seg+1].  Returns coef uint32[n_seg, J] (and the unrounded fit with ``diag``)."""
    X = _chk(X, np.uint16)
    T = X.size // d
    ref_base = _chk(ref_base, np.uint16)
    ref_rows = 0 if ref_base is None else ref_base.size // d
    ref_row = _chk(ref_row, np.int32, T)
    gain = _chk(gain, np.uint16, d)
    bias = _chk(bias, np.uint16, d)
    seg_off = _chk(np.asarray(seg_off, np.int32), np.int32)
    n_seg = seg_off.size - 1
    J = d // group
    coef = np.zeros((n_seg, J), np.uint32)
    dg = {}
    if diag:
        dg = dict(alpha=np.zeros((n_seg, J)), beta=np.zeros((n_seg, J)), hbar=np.zeros((n_seg, J)), rbar=np.zeros((n_seg, J)))
    rc = lib().orc_fit_segments(d, group, _p(X, _u16p), T, _p(ref_base, _u16p), ref_rows, _p(ref_row, _i32p),
                                _p(gain, _u16p), _p(bias, _u16p), _p(seg_off, _i32p), n_seg, _p(coef, _u32p),
                                _p(dg.get("alpha"), _f64p), _p(dg.get("beta"), _f64p), _p(dg.get("hbar"), _f64p),
                                _p(dg.get("rbar"), _f64p))
    if rc != 0:
        raise ValueError(f"orc_fit_segments failed: {rc}")
    return (coef, dg) if diag else coef


def segments_from_spans(spans: np.ndarray, T: int) -> np.ndarray:
    """Boundaries of the segmentation "spans and the gaps between them": int32[n_seg+1], empty pieces dropped."""
    b = [0]
    for q, _, ln in np.asarray(spans, np.int64).reshape(-1, 3):
        for x in (q, q + ln):
            if x > b[-1]:
                b.append(int(x))
    if b[-1] < T:
        b.append(int(T))
    return np.array(b, np.int32)
