"""ctypes binding of ``librac.so`` -- argument marshalling only.

Every function has the name and the argument order of its C entry point in
``include/rac.h``.  Arguments are either raw addresses (int) or torch tensors
living where the C function expects them (device pointers for the ``rac_*``
calls); the binding checks dtype, contiguity and device, takes
``tensor.data_ptr()`` and the current CUDA stream, calls the library and raises
on a non-zero return code.  No arithmetic of the method happens here and there
is no fallback: if the library cannot be loaded, importing callers get an error.
"""
from __future__ import annotations

import ctypes as C
import os
from typing import Optional

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "librac.so")

RAC_OK = 0
STATUS_REF_RANGE = 1
STATUS_RESERVED_CODE = 2
STATUS_NONFINITE = 4
STATUS_TIMEOUT = 8
STATUS_OUTLIER_RANGE = 16

EXPORTS = [
    "rac_version", "rac_strerror", "rac_record_bytes", "rac_payload_bytes", "rac_header_write", "rac_header_parse",
    "rac_match_workspace_bytes", "rac_match_spans", "rac_spans_to_rows",
    "rac_match_spans_static",
    "rac_index_bytes", "rac_index_reset", "rac_index_append", "rac_index_query_workspace_bytes", "rac_index_query",
    "rac_index_query_live",
    "rac_encode_workspace_bytes", "rac_encode", "rac_encode_reconstruct", "rac_decode_reconstruct",
    "rac_sender_reconstruct",
    "rac_split_waves", "rac_encode_reconstruct_list", "rac_decode_reconstruct_list",
    "rac_fit_segments_workspace_bytes", "rac_fit_segments", "rac_spans_to_segments",
    "rac_calibrate_workspace_bytes", "rac_calibrate_steps", "rac_calibrate_steps_shared",
    "rac_recon_error_workspace_bytes", "rac_recon_error",
    "rac_selftest_bounded_wait",
]


class RacError(RuntimeError):
    def __init__(self, fn: str, code: int, msg: str):
        super().__init__(f"{fn} failed: {code} ({msg})")
        self.code = code


class CodecCfg(C.Structure):
    """Mirror of ``rac_codec_cfg``."""
    _fields_ = [(n, C.c_int32) for n in ("d", "group", "bits", "topk", "coef_fmt", "scale_mode", "flags",
                                         "qgroup", "topk_group")]

    def __init__(self, d: int, group: int, bits: int, topk: int = 0, scale_mode: int = 0, qgroup: int = 0,
                 topk_group: int = 0, coef_fmt: int = 0):
        super().__init__(d, group, bits, topk, coef_fmt, scale_mode, 0, qgroup, topk_group)

    def __repr__(self):
        return (f"CodecCfg(d={self.d}, group={self.group}, bits={self.bits}, topk={self.topk}, "
                f"scale_mode={self.scale_mode}, qgroup={self.qgroup}, topk_group={self.topk_group})")


class IndexCfg(C.Structure):
    """Mirror of ``rac_index_cfg``."""
    _fields_ = [("capacity", C.c_int64), ("min_ngram", C.c_int32), ("max_hits", C.c_int32)]

    def __init__(self, capacity: int, min_ngram: int = 4, max_hits: int = 8):
        super().__init__(capacity, min_ngram, max_hits)


_lib: Optional[C.CDLL] = None


class _Recorder:
    """Stands in for the library while `prepare` runs a wrapper once: launches are recorded instead of made."""

    def __init__(self, lib):
        self._lib = lib
        self.calls = []

    def __getattr__(self, name):
        real = getattr(self._lib, name)
        if real.restype is not C.c_int:      # size queries, strings: answer them
            return real

        def record(*args):
            self.calls.append((name, real, args))
            return RAC_OK
        return record


_recorder = None


def prepare(wrapper, *args, **kwargs):
    """Marshals the arguments of one call ONCE and returns a function without arguments that repeats the call.

    ``wrapper`` is one of the functions of this module that launch work (``rac_encode_reconstruct``,
    ``rac_decode_reconstruct``, ...), ``args`` what it would be given.  Tensor addresses, sizes and the stream
    (``stream=`` or the current one at the time of this call) are fixed here; the tensors must stay alive and in
    place.  For loops that issue the same small call many times (a decode step per token), where looking at a dozen
    tensors costs more than the launch.  Not thread safe while it prepares."""
    global _recorder
    lib = load()
    rec = _Recorder(lib)
    _recorder = rec
    try:
        wrapper(*args, **kwargs)
    finally:
        _recorder = None
    if len(rec.calls) != 1:
        raise ValueError("prepare() wants a wrapper that makes exactly one library call")
    name, real, cargs = rec.calls[0]
    keep = (args, kwargs)      # the tensors (and the configuration struct the pointers refer to) stay referenced

    def call():
        rc = real(*cargs)
        if rc != RAC_OK:
            _check(name, rc)
    call.keepalive = keep
    return call


def load():
    """Load the C-ABI library.  Raises if it has not been built (``__graft_entry__.build()``)."""
    global _lib
    if _recorder is not None:
        return _recorder
    if _lib is not None:
        return _lib
    if not os.path.exists(LIB_PATH):
        raise RuntimeError(f"{LIB_PATH} is missing: build it with `python -m paper_2608_04991_b200.build` "
                           "(there is no CPU fallback)")
    l = C.CDLL(LIB_PATH)
    vp, i64, i32, sz = C.c_void_p, C.c_int64, C.c_int32, C.c_size_t
    cfgp = C.POINTER(CodecCfg)
    l.rac_version.restype = C.c_char_p
    l.rac_version.argtypes = []
    l.rac_strerror.restype = C.c_char_p
    l.rac_strerror.argtypes = [C.c_int]
    l.rac_record_bytes.restype = sz
    l.rac_record_bytes.argtypes = [cfgp]
    l.rac_payload_bytes.restype = sz
    l.rac_payload_bytes.argtypes = [cfgp, i64]
    l.rac_header_write.restype = C.c_int
    l.rac_header_write.argtypes = [cfgp, i64, vp]
    l.rac_header_parse.restype = C.c_int
    l.rac_header_parse.argtypes = [vp, cfgp, C.POINTER(i64)]
    l.rac_match_workspace_bytes.restype = sz
    l.rac_match_workspace_bytes.argtypes = [i64, i64, i32]
    l.rac_match_spans.restype = C.c_int
    l.rac_match_spans.argtypes = [vp, i64, vp, i64, i32, i32, vp, vp, vp, vp, sz, vp]
    l.rac_match_spans_static.restype = C.c_int
    l.rac_match_spans_static.argtypes = [vp, i64, vp, i64, i32, i32, vp, vp, vp, vp]
    icfgp = C.POINTER(IndexCfg)
    l.rac_index_bytes.restype = sz
    l.rac_index_bytes.argtypes = [icfgp]
    l.rac_index_reset.restype = C.c_int
    l.rac_index_reset.argtypes = [icfgp, vp, sz, vp]
    l.rac_index_append.restype = C.c_int
    l.rac_index_append.argtypes = [icfgp, vp, sz, vp, i64, i64, vp]
    l.rac_index_query_workspace_bytes.restype = sz
    l.rac_index_query_workspace_bytes.argtypes = [i64]
    l.rac_index_query.restype = C.c_int
    l.rac_index_query.argtypes = [icfgp, vp, sz, vp, i64, vp, i64, i32, vp, vp, vp, vp, sz, vp]
    l.rac_index_query_live.restype = C.c_int
    l.rac_index_query_live.argtypes = [icfgp, vp, sz, vp, i64, i64, vp, i64, i32, vp, vp, vp, vp, sz, vp]
    l.rac_spans_to_rows.restype = C.c_int
    l.rac_spans_to_rows.argtypes = [vp, vp, i64, vp, vp]
    l.rac_encode.restype = C.c_int
    l.rac_encode_workspace_bytes.restype = sz
    l.rac_encode_workspace_bytes.argtypes = [cfgp, i64]
    l.rac_encode.argtypes = [cfgp, vp, i64, vp, i64, vp, vp, vp, vp, vp, vp, sz, vp, sz, vp, vp]
    l.rac_encode_reconstruct.restype = C.c_int
    l.rac_encode_reconstruct.argtypes = [cfgp, vp, i64, vp, i64, vp, vp, vp, vp, vp, vp, sz, vp, vp, sz, vp, vp]
    for name in ("rac_decode_reconstruct", "rac_sender_reconstruct"):
        f = getattr(l, name)
        f.restype = C.c_int
        f.argtypes = [cfgp, vp, i64, vp, i64, vp, vp, vp, vp, vp, vp, vp]
    l.rac_selftest_bounded_wait.restype = C.c_int
    l.rac_selftest_bounded_wait.argtypes = [cfgp, i32, vp, i64, vp, i64, vp, vp, vp, sz, vp, sz, vp, vp]
    l.rac_split_waves.restype = C.c_int
    l.rac_split_waves.argtypes = [vp, i64, i64, vp, vp, vp, vp]
    l.rac_encode_reconstruct_list.restype = C.c_int
    l.rac_encode_reconstruct_list.argtypes = [cfgp, vp, i64, vp, vp, vp, i64, vp, vp, i64, vp, vp, vp, vp, vp, vp, vp, sz,
                                              vp, vp, sz, vp, vp]
    l.rac_decode_reconstruct_list.restype = C.c_int
    l.rac_decode_reconstruct_list.argtypes = [cfgp, vp, i64, vp, vp, vp, i64, vp, vp, i64, vp, vp, vp, vp, vp, vp, vp, vp]
    l.rac_spans_to_segments.restype = C.c_int
    l.rac_spans_to_segments.argtypes = [vp, vp, i64, i64, vp, vp, vp]
    l.rac_fit_segments_workspace_bytes.restype = sz
    l.rac_fit_segments_workspace_bytes.argtypes = [cfgp, i64]
    l.rac_fit_segments.restype = C.c_int
    l.rac_fit_segments.argtypes = [cfgp, vp, i64, vp, i64, vp, vp, vp, vp, i64, vp, vp, vp, sz, vp, vp]
    l.rac_recon_error_workspace_bytes.restype = sz
    l.rac_recon_error_workspace_bytes.argtypes = []
    l.rac_recon_error.restype = C.c_int
    l.rac_recon_error.argtypes = [vp, vp, i64, i32, vp, vp, sz, vp]
    l.rac_calibrate_workspace_bytes.restype = sz
    l.rac_calibrate_workspace_bytes.argtypes = [cfgp]
    l.rac_calibrate_steps.restype = C.c_int
    l.rac_calibrate_steps.argtypes = [cfgp, vp, i64, vp, i64, vp, vp, vp, C.c_float, vp, vp, vp, sz, vp, vp]
    l.rac_calibrate_steps_shared.restype = C.c_int
    l.rac_calibrate_steps_shared.argtypes = [cfgp, vp, i64, vp, i64, vp, vp, vp, vp, vp, C.c_float, vp, vp, vp, sz, vp, vp]
    _lib = l
    return l


def _check(fn: str, rc: int) -> None:
    if rc != RAC_OK:
        raise RacError(fn, rc, load().rac_strerror(rc).decode())


def _ptr(t, dtype=None, name="tensor") -> Optional[int]:
    """Address of a tensor (or pass an int / None through)."""
    if t is None:
        return None
    if isinstance(t, int):
        return t
    if not isinstance(t, torch.Tensor):
        raise TypeError(f"{name}: expected a torch tensor, an address or None")
    if not t.is_cuda:
        raise ValueError(f"{name}: must be a CUDA tensor")
    if not t.is_contiguous():
        raise ValueError(f"{name}: must be contiguous")
    if dtype is not None and t.dtype not in (dtype if isinstance(dtype, tuple) else (dtype,)):
        raise TypeError(f"{name}: expected {dtype}, got {t.dtype}")
    return t.data_ptr()


def _stream() -> int:
    return torch.cuda.current_stream().cuda_stream


_BF16 = torch.bfloat16
_F16 = torch.float16
_I32 = torch.int32
_F32 = torch.float32
_U8 = (torch.uint8, torch.int8)


# ----------------------------------------------------------------------------- plain queries
def rac_version() -> str:
    return load().rac_version().decode()


def rac_strerror(code: int) -> str:
    return load().rac_strerror(int(code)).decode()


def rac_record_bytes(cfg: CodecCfg) -> int:
    return int(load().rac_record_bytes(C.byref(cfg)))


def rac_payload_bytes(cfg: CodecCfg, T: int) -> int:
    return int(load().rac_payload_bytes(C.byref(cfg), int(T)))


HEADER_BYTES = 64


def rac_header_write(cfg: CodecCfg, T: int) -> bytes:
    """The 64-byte header of a serialised payload of T records (host work only)."""
    buf = C.create_string_buffer(HEADER_BYTES)
    _check("rac_header_write", load().rac_header_write(C.byref(cfg), int(T), buf))
    return buf.raw


def rac_header_parse(header: bytes):
    """(CodecCfg, T) of a header written by rac_header_write; raises RacError when it does not check out."""
    if len(header) < HEADER_BYTES:
        raise ValueError("a header is 64 bytes")
    buf = C.create_string_buffer(bytes(header[:HEADER_BYTES]), HEADER_BYTES)
    cfg, T = CodecCfg(64, 32, 4, 0), C.c_int64(0)
    _check("rac_header_parse", load().rac_header_parse(buf, C.byref(cfg), C.byref(T)))
    return cfg, int(T.value)


def rac_match_workspace_bytes(n_hist: int, n_query: int, max_hits: int) -> int:
    return int(load().rac_match_workspace_bytes(int(n_hist), int(n_query), int(max_hits)))


def rac_encode_workspace_bytes(cfg: CodecCfg, T: int) -> int:
    return int(load().rac_encode_workspace_bytes(C.byref(cfg), int(T)))


def rac_split_waves(ref_row, T, first_intra_row, wave1, wave2, wave_count, stream=None) -> None:
    rc = load().rac_split_waves(_ptr(ref_row, _I32, "ref_row"), int(T), int(first_intra_row), _ptr(wave1, _I32, "wave1"),
                                _ptr(wave2, _I32, "wave2"), _ptr(wave_count, _I32, "wave_count"),
                                _stream() if stream is None else stream)
    _check("rac_split_waves", rc)


def rac_encode_reconstruct_list(cfg, X, T, tok_list, tok_count, ref_base, ref_rows, ref_row, intra_base, intra_rows,
                                ref_gain, ref_bias, step, inv_step, payload, payload_cap, X_hat, workspace,
                                workspace_bytes, dev_status, stream=None, coef_seg=None, seg_of=None) -> None:
    rc = load().rac_encode_reconstruct_list(
        C.byref(cfg), _ptr(X, _BF16, "X"), int(T), _ptr(tok_list, _I32, "tok_list"), _ptr(tok_count, _I32, "tok_count"),
        _ptr(ref_base, _BF16, "ref_base"), int(ref_rows), _ptr(ref_row, _I32, "ref_row"),
        _ptr(intra_base, _BF16, "intra_base"), int(intra_rows), _ptr(coef_seg, _I32, "coef_seg"),
        _ptr(seg_of, _I32, "seg_of"), _ptr(ref_gain, _F16, "ref_gain"),
        _ptr(ref_bias, _F16, "ref_bias"), _ptr(step, _F32, "step"), _ptr(inv_step, _F32, "inv_step"),
        _ptr(payload, _U8, "payload"), int(payload_cap), _ptr(X_hat, _BF16, "X_hat"), _ptr(workspace, None, "workspace"),
        int(workspace_bytes), _ptr(dev_status, _I32, "dev_status"), _stream() if stream is None else stream)
    _check("rac_encode_reconstruct_list", rc)


def rac_decode_reconstruct_list(cfg, payload, T, tok_list, tok_count, ref_base, ref_rows, ref_row, intra_base,
                                intra_rows, ref_gain, ref_bias, step, X_hat, dev_status, stream=None, coef_seg=None,
                                seg_of=None) -> None:
    rc = load().rac_decode_reconstruct_list(
        C.byref(cfg), _ptr(payload, _U8, "payload"), int(T), _ptr(tok_list, _I32, "tok_list"),
        _ptr(tok_count, _I32, "tok_count"), _ptr(ref_base, _BF16, "ref_base"), int(ref_rows),
        _ptr(ref_row, _I32, "ref_row"), _ptr(intra_base, _BF16, "intra_base"), int(intra_rows),
        _ptr(coef_seg, _I32, "coef_seg"), _ptr(seg_of, _I32, "seg_of"),
        _ptr(ref_gain, _F16, "ref_gain"), _ptr(ref_bias, _F16, "ref_bias"), _ptr(step, _F32, "step"),
        _ptr(X_hat, _BF16, "X_hat"), _ptr(dev_status, _I32, "dev_status"), _stream() if stream is None else stream)
    _check("rac_decode_reconstruct_list", rc)


def rac_spans_to_segments(spans, n_spans, T, max_seg, seg_off, n_seg, stream=None) -> None:
    rc = load().rac_spans_to_segments(_ptr(spans, _I32, "spans"), _ptr(n_spans, _I32, "n_spans"), int(T), int(max_seg),
                                      _ptr(seg_off, _I32, "seg_off"), _ptr(n_seg, _I32, "n_seg"),
                                      _stream() if stream is None else stream)
    _check("rac_spans_to_segments", rc)


def rac_fit_segments_workspace_bytes(cfg: CodecCfg, T: int) -> int:
    return int(load().rac_fit_segments_workspace_bytes(C.byref(cfg), int(T)))


def rac_fit_segments(cfg, X, T, ref_base, ref_rows, ref_row, ref_gain, ref_bias, seg_off, n_seg, coef_seg, seg_of,
                     workspace, workspace_bytes, dev_status, stream=None) -> None:
    """Eq. 6 over several fitting positions; ``coef_seg`` is an int32 tensor [n_seg, J] holding the u32 words."""
    rc = load().rac_fit_segments(C.byref(cfg), _ptr(X, _BF16, "X"), int(T), _ptr(ref_base, _BF16, "ref_base"),
                                 int(ref_rows), _ptr(ref_row, _I32, "ref_row"), _ptr(ref_gain, _F16, "ref_gain"),
                                 _ptr(ref_bias, _F16, "ref_bias"), _ptr(seg_off, _I32, "seg_off"), int(n_seg),
                                 _ptr(coef_seg, _I32, "coef_seg"), _ptr(seg_of, _I32, "seg_of"),
                                 _ptr(workspace, None, "workspace"), int(workspace_bytes),
                                 _ptr(dev_status, _I32, "dev_status"), _stream() if stream is None else stream)
    _check("rac_fit_segments", rc)


def rac_recon_error_workspace_bytes() -> int:
    return int(load().rac_recon_error_workspace_bytes())


def rac_recon_error(X, X_hat, T, d, out, workspace, workspace_bytes, stream=None) -> None:
    rc = load().rac_recon_error(_ptr(X, _BF16, "X"), _ptr(X_hat, _BF16, "X_hat"), int(T), int(d), _ptr(out, None, "out"),
                                _ptr(workspace, None, "workspace"), int(workspace_bytes),
                                _stream() if stream is None else stream)
    _check("rac_recon_error", rc)


def rac_calibrate_workspace_bytes(cfg: CodecCfg) -> int:
    return int(load().rac_calibrate_workspace_bytes(C.byref(cfg)))


# ----------------------------------------------------------------------------- device calls
def rac_match_spans(hist_tok, n_hist, query_tok, n_query, min_ngram, max_hits, ref_row, spans, n_spans,
                    workspace, workspace_bytes, stream=None) -> None:
    rc = load().rac_match_spans(_ptr(hist_tok, _I32, "hist_tok"), int(n_hist), _ptr(query_tok, _I32, "query_tok"),
                                int(n_query), int(min_ngram), int(max_hits), _ptr(ref_row, _I32, "ref_row"),
                                _ptr(spans, _I32, "spans"), _ptr(n_spans, _I32, "n_spans"),
                                _ptr(workspace, None, "workspace"), int(workspace_bytes),
                                _stream() if stream is None else stream)
    _check("rac_match_spans", rc)


MATCH_STATIC_BYTES = 3 << 20  # RAC_MATCH_STATIC_BYTES in rac.h


def rac_match_spans_static(hist_tok, n_hist, query_tok, n_query, min_ngram, max_hits, ref_row, spans, n_spans,
                           stream=None) -> None:
    """Span retrieval on the library's built-in 3 MiB scratch: for callers that may not allocate device memory.
    Calls on one device must not overlap on the GPU (they share the scratch)."""
    rc = load().rac_match_spans_static(_ptr(hist_tok, _I32, "hist_tok"), int(n_hist), _ptr(query_tok, _I32, "query_tok"),
                                       int(n_query), int(min_ngram), int(max_hits), _ptr(ref_row, _I32, "ref_row"),
                                       _ptr(spans, _I32, "spans"), _ptr(n_spans, _I32, "n_spans"),
                                       _stream() if stream is None else stream)
    _check("rac_match_spans_static", rc)


def rac_index_bytes(cfg: IndexCfg) -> int:
    return int(load().rac_index_bytes(C.byref(cfg)))


def rac_index_query_workspace_bytes(n_query: int) -> int:
    return int(load().rac_index_query_workspace_bytes(int(n_query)))


def rac_index_reset(cfg, index, index_bytes, stream=None) -> None:
    rc = load().rac_index_reset(C.byref(cfg), _ptr(index, None, "index"), int(index_bytes),
                                _stream() if stream is None else stream)
    _check("rac_index_reset", rc)


def rac_index_append(cfg, index, index_bytes, hist_tok, n_before, n_after, stream=None) -> None:
    rc = load().rac_index_append(C.byref(cfg), _ptr(index, None, "index"), int(index_bytes),
                                 _ptr(hist_tok, _I32, "hist_tok"), int(n_before), int(n_after),
                                 _stream() if stream is None else stream)
    _check("rac_index_append", rc)


def rac_index_query_live(cfg, index, index_bytes, hist_tok, n_hist, first_live, query_tok, n_query, intra, ref_row, spans,
                         n_spans, workspace, workspace_bytes, stream=None) -> None:
    rc = load().rac_index_query_live(C.byref(cfg), _ptr(index, None, "index"), int(index_bytes),
                                     _ptr(hist_tok, _I32, "hist_tok"), int(n_hist), int(first_live),
                                     _ptr(query_tok, _I32, "query_tok"), int(n_query), int(bool(intra)),
                                     _ptr(ref_row, _I32, "ref_row"), _ptr(spans, _I32, "spans"), _ptr(n_spans, _I32, "n_spans"),
                                     _ptr(workspace, None, "workspace"), int(workspace_bytes),
                                     _stream() if stream is None else stream)
    _check("rac_index_query_live", rc)


def rac_index_query(cfg, index, index_bytes, hist_tok, n_hist, query_tok, n_query, intra, ref_row, spans, n_spans,
                    workspace, workspace_bytes, stream=None) -> None:
    rc = load().rac_index_query(C.byref(cfg), _ptr(index, None, "index"), int(index_bytes),
                                _ptr(hist_tok, _I32, "hist_tok"), int(n_hist), _ptr(query_tok, _I32, "query_tok"),
                                int(n_query), int(bool(intra)), _ptr(ref_row, _I32, "ref_row"),
                                _ptr(spans, _I32, "spans"), _ptr(n_spans, _I32, "n_spans"),
                                _ptr(workspace, None, "workspace"), int(workspace_bytes),
                                _stream() if stream is None else stream)
    _check("rac_index_query", rc)


def rac_spans_to_rows(spans, n_spans, n_query, ref_row, stream=None) -> None:
    rc = load().rac_spans_to_rows(_ptr(spans, _I32, "spans"), _ptr(n_spans, _I32, "n_spans"), int(n_query),
                                  _ptr(ref_row, _I32, "ref_row"), _stream() if stream is None else stream)
    _check("rac_spans_to_rows", rc)


def rac_encode(cfg, X, T, ref_base, ref_rows, ref_row, ref_gain, ref_bias, step, inv_step, payload, payload_cap,
               workspace, workspace_bytes, dev_status, stream=None) -> None:
    rc = load().rac_encode(C.byref(cfg), _ptr(X, _BF16, "X"), int(T), _ptr(ref_base, _BF16, "ref_base"), int(ref_rows),
                           _ptr(ref_row, _I32, "ref_row"), _ptr(ref_gain, _F16, "ref_gain"),
                           _ptr(ref_bias, _F16, "ref_bias"), _ptr(step, _F32, "step"), _ptr(inv_step, _F32, "inv_step"),
                           _ptr(payload, _U8, "payload"), int(payload_cap), _ptr(workspace, None, "workspace"),
                           int(workspace_bytes), _ptr(dev_status, _I32, "dev_status"),
                           _stream() if stream is None else stream)
    _check("rac_encode", rc)


def rac_encode_reconstruct(cfg, X, T, ref_base, ref_rows, ref_row, ref_gain, ref_bias, step, inv_step, payload,
                           payload_cap, X_hat, workspace, workspace_bytes, dev_status, stream=None) -> None:
    rc = load().rac_encode_reconstruct(C.byref(cfg), _ptr(X, _BF16, "X"), int(T), _ptr(ref_base, _BF16, "ref_base"),
                                       int(ref_rows), _ptr(ref_row, _I32, "ref_row"), _ptr(ref_gain, _F16, "ref_gain"),
                                       _ptr(ref_bias, _F16, "ref_bias"), _ptr(step, _F32, "step"),
                                       _ptr(inv_step, _F32, "inv_step"), _ptr(payload, _U8, "payload"), int(payload_cap),
                                       _ptr(X_hat, _BF16, "X_hat"), _ptr(workspace, None, "workspace"),
                                       int(workspace_bytes), _ptr(dev_status, _I32, "dev_status"),
                                       _stream() if stream is None else stream)
    _check("rac_encode_reconstruct", rc)


def _reconstruct(fn, cfg, payload, T, ref_base, ref_rows, ref_row, ref_gain, ref_bias, step, X_hat, dev_status, stream):
    rc = getattr(load(), fn)(C.byref(cfg), _ptr(payload, _U8, "payload"), int(T), _ptr(ref_base, _BF16, "ref_base"),
                             int(ref_rows), _ptr(ref_row, _I32, "ref_row"), _ptr(ref_gain, _F16, "ref_gain"),
                             _ptr(ref_bias, _F16, "ref_bias"), _ptr(step, _F32, "step"), _ptr(X_hat, _BF16, "X_hat"),
                             _ptr(dev_status, _I32, "dev_status"), _stream() if stream is None else stream)
    _check(fn, rc)


def rac_decode_reconstruct(cfg, payload, T, ref_base, ref_rows, ref_row, ref_gain, ref_bias, step, X_hat,
                           dev_status, stream=None) -> None:
    _reconstruct("rac_decode_reconstruct", cfg, payload, T, ref_base, ref_rows, ref_row, ref_gain, ref_bias, step,
                 X_hat, dev_status, stream)


def rac_sender_reconstruct(cfg, payload, T, ref_base, ref_rows, ref_row, ref_gain, ref_bias, step, X_hat,
                           dev_status, stream=None) -> None:
    _reconstruct("rac_sender_reconstruct", cfg, payload, T, ref_base, ref_rows, ref_row, ref_gain, ref_bias, step,
                 X_hat, dev_status, stream)


def rac_selftest_bounded_wait(cfg, which, inp, T, ref_base, ref_rows, step, inv_step, out, out_cap, workspace,
                              workspace_bytes, dev_status, stream=None) -> None:
    """Runs the encode (which=0) or reconstruction (which=1) kernels with waits that cannot complete; see rac.h."""
    rc = load().rac_selftest_bounded_wait(C.byref(cfg), int(which), _ptr(inp, None, "in"), int(T),
                                          _ptr(ref_base, _BF16, "ref_base"), int(ref_rows), _ptr(step, _F32, "step"),
                                          _ptr(inv_step, _F32, "inv_step"), _ptr(out, None, "out"), int(out_cap),
                                          _ptr(workspace, None, "workspace"), int(workspace_bytes),
                                          _ptr(dev_status, _I32, "dev_status"), _stream() if stream is None else stream)
    _check("rac_selftest_bounded_wait", rc)


def rac_calibrate_steps(cfg, X, T, ref_base, ref_rows, ref_row, ref_gain, ref_bias, clip_sigmas, step, inv_step,
                        workspace, workspace_bytes, dev_status, stream=None) -> None:
    rc = load().rac_calibrate_steps(C.byref(cfg), _ptr(X, _BF16, "X"), int(T), _ptr(ref_base, _BF16, "ref_base"),
                                    int(ref_rows), _ptr(ref_row, _I32, "ref_row"), _ptr(ref_gain, _F16, "ref_gain"),
                                    _ptr(ref_bias, _F16, "ref_bias"), float(clip_sigmas), _ptr(step, _F32, "step"),
                                    _ptr(inv_step, _F32, "inv_step"), _ptr(workspace, None, "workspace"),
                                    int(workspace_bytes), _ptr(dev_status, _I32, "dev_status"),
                                    _stream() if stream is None else stream)
    _check("rac_calibrate_steps", rc)


def rac_calibrate_steps_shared(cfg, X, T, ref_base, ref_rows, ref_row, ref_gain, ref_bias, coef_seg, seg_of, clip_sigmas,
                               step, inv_step, workspace, workspace_bytes, dev_status, stream=None) -> None:
    rc = load().rac_calibrate_steps_shared(C.byref(cfg), _ptr(X, _BF16, "X"), int(T), _ptr(ref_base, _BF16, "ref_base"),
                                           int(ref_rows), _ptr(ref_row, _I32, "ref_row"),
                                           _ptr(ref_gain, _F16, "ref_gain"), _ptr(ref_bias, _F16, "ref_bias"),
                                           _ptr(coef_seg, _I32, "coef_seg"), _ptr(seg_of, _I32, "seg_of"),
                                           float(clip_sigmas), _ptr(step, _F32, "step"),
                                           _ptr(inv_step, _F32, "inv_step"), _ptr(workspace, None, "workspace"),
                                           int(workspace_bytes), _ptr(dev_status, _I32, "dev_status"),
                                           _stream() if stream is None else stream)
    _check("rac_calibrate_steps_shared", rc)
