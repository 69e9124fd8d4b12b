"""The C-ABI library loads, exports every symbol the header declares, and rejects bad
arguments on the host before anything is launched (no GPU needed)."""
import ctypes as C
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def rac():
    from paper_2608_04991_b200 import build, binding
    build.build()
    binding.load()
    return binding


def declared_symbols():
    text = open(os.path.join(ROOT, "include", "rac.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(rac_[a-z_]+)\s*\(", text)))


def test_every_declared_symbol_is_exported(rac):
    names = declared_symbols()
    assert len(names) >= 15
    lib = rac.load()
    for n in names:
        assert hasattr(lib, n), f"{n} declared in rac.h but not exported by librac.so"
    assert sorted(rac.EXPORTS) == names
    for n in names:
        assert callable(getattr(rac, n)), f"binding lacks {n}"


def test_record_geometry_matches_the_wire_format(rac, orc):
    for d, g, b, k in [(4096, 128, 4, 0), (4096, 128, 4, 8), (3584, 128, 3, 0), (5120, 128, 4, 8), (4096, 64, 2, 8),
                       (4096, 64, 3, 8), (8192, 256, 4, 16), (64, 32, 2, 0)]:
        cfg = rac.CodecCfg(d, g, b, k)
        assert rac.rac_record_bytes(cfg) == orc.record_bytes(d, g, b, k)
        assert rac.rac_payload_bytes(cfg, 1000) == 1000 * orc.record_bytes(d, g, b, k)
    for d, g, b in [(4096, 128, 4), (3584, 128, 3), (2080, 32, 4), (96, 32, 2)]:   # per-group scales in the record
        assert rac.rac_record_bytes(rac.CodecCfg(d, g, b, 0, scale_mode=1)) == orc.record_bytes(d, g, b, 0, 1)
    assert rac.rac_record_bytes(rac.CodecCfg(4096, 128, 4, 0, scale_mode=1)) == 2176 + 64
    # the quantiser family: geometry agrees with the oracle's, 8-bit and per-group outliers only with record scales
    for d, g, b, qg, kg in [(4096, 128, 8, 0, 0), (4096, 128, 4, 0, 2), (3584, 128, 4, 3584, 0), (2080, 32, 4, 0, 1),
                            (5120, 128, 2, 256, 3), (96, 32, 8, 96, 0), (5120, 128, 4, 160, 0), (3584, 64, 3, 1792, 0)]:
        assert rac.rac_record_bytes(rac.CodecCfg(d, g, b, 0, scale_mode=1, qgroup=qg, topk_group=kg)) == \
            orc.record_bytes(d, g, b, 0, 1, qg, kg)
    assert rac.rac_record_bytes(rac.CodecCfg(4096, 128, 8, 0)) == 0
    assert rac.rac_record_bytes(rac.CodecCfg(4096, 128, 4, 0, scale_mode=1, qgroup=512, topk_group=3)) == \
        orc.record_bytes(4096, 128, 4, 0, 1, 512, 3)                   # wide groups: two-byte offsets
    assert rac.rac_record_bytes(rac.CodecCfg(5120, 128, 4, 0, scale_mode=1, qgroup=5120, topk_group=1)) == 0   # group wider than a warp
    assert C.sizeof(rac.CodecCfg) == 36
    assert rac.rac_record_bytes(rac.CodecCfg(4096, 100, 4, 0)) == 0   # group does not divide d
    assert rac.rac_record_bytes(rac.CodecCfg(4096, 128, 5, 0)) == 0   # unsupported width
    assert rac.rac_record_bytes(rac.CodecCfg(4096, 128, 4, 17)) == 0
    assert "sm_100a" in rac.rac_version()


def test_host_side_rejections_happen_before_any_launch(rac):
    lib = rac.load()
    cfg = rac.CodecCfg(4096, 128, 4, 8)
    bad = rac.CodecCfg(4096, 96, 4, 8)
    A = 0x10000  # a 16-byte aligned fake address: never dereferenced because the call is rejected first
    args = dict(X=A, T=16, ref_base=A, ref_rows=16, ref_row=None, ref_gain=None, ref_bias=None, step=A, inv_step=A,
                payload=A, payload_cap=16 * 2208, workspace=A, workspace_bytes=16 * 128 * 4, dev_status=None,
                stream=0)

    def enc(c=cfg, **kw):
        a = dict(args, **kw)
        return lib.rac_encode(C.byref(c), a["X"], a["T"], a["ref_base"], a["ref_rows"], a["ref_row"], a["ref_gain"],
                              a["ref_bias"], a["step"], a["inv_step"], a["payload"], a["payload_cap"], a["workspace"],
                              a["workspace_bytes"], a["dev_status"], a["stream"])
    assert enc(c=bad) == -1                      # d % group
    assert enc(c=rac.CodecCfg(4100, 4100 // 4, 4, 0)) in (-1, -4)
    assert enc(T=-1) == -1
    assert enc(X=None) == -1
    assert enc(X=A + 2) == -2                    # misaligned
    assert enc(payload=A + 8) == -2
    assert enc(payload_cap=16 * 2208 - 1) == -3
    assert enc(workspace_bytes=16 * 128 * 4 - 1) == -3   # outliers need 4*d/32 bytes of scratch per token
    assert enc(workspace=None) == -1
    assert enc(workspace=A + 4) == -2
    assert enc(ref_rows=8) == -1                 # identity rows need ref_rows >= T
    assert enc(ref_gain=A) == -1                 # gain without bias
    assert enc(T=0, X=None, payload=None) == 0   # nothing to do
    dec = lib.rac_decode_reconstruct(C.byref(cfg), None, 4, A, 4, None, None, None, A, A, None, 0)
    assert dec == -1
    assert lib.rac_decode_reconstruct(C.byref(cfg), A, 4, A, 4, None, None, None, A, A + 4, None, 0) == -2
    # matcher
    assert rac.rac_match_workspace_bytes(1000, 100, 8) > 0
    # 0 = unlimited hits: one chain head per slot and a link per history position, less than any K-list
    assert 0 < rac.rac_match_workspace_bytes(1000, 100, 0) < rac.rac_match_workspace_bytes(1000, 100, 1) + 4 * 1000 + 16
    assert rac.rac_match_workspace_bytes(1000, 100, -1) == 0
    assert rac.rac_match_workspace_bytes(1000, 100, 17) == 0
    need = rac.rac_match_workspace_bytes(1000, 100, 8)
    m = lambda **kw: lib.rac_match_spans(kw.get("h", A), kw.get("nh", 1000), A, 100, kw.get("w", 4), kw.get("K", 8), A, None, A,
                                         kw.get("ws", A), kw.get("wsb", need), 0)
    assert m(w=0) == -4 and m(K=-1) == -4 and m(K=17) == -4 and m(wsb=need - 1) == -3 and m(ws=A + 4) == -2 and m(h=None) == -1
    # shared coefficient pairs: the record format and the words go together, in the calibration and in the list calls
    sh = rac.CodecCfg(4096, 128, 4, 8, coef_fmt=1)
    nbc = rac.rac_calibrate_workspace_bytes(sh)
    assert nbc == rac.rac_calibrate_workspace_bytes(cfg) > 0
    cal = lambda c, cs, so, wsb=nbc: lib.rac_calibrate_steps_shared(C.byref(c), A, 16, A, 16, None, None, None, cs, so, 3.0, A, A,
                                                                  A, wsb, None, 0)
    assert cal(sh, None, A) == -1 and cal(sh, A, None) == -1 and cal(cfg, A, A) == -1 and cal(sh, A, A, nbc - 1) == -3
    assert lib.rac_calibrate_steps(C.byref(sh), A, 16, A, 16, None, None, None, 3.0, A, A, A, nbc, None, 0) == -1
    assert cal(rac.CodecCfg(4096, 128, 4, 0, scale_mode=1, coef_fmt=1), A, A) == -4      # no table in that mode
    lst = lambda c, cs, so: lib.rac_encode_reconstruct_list(C.byref(c), A, 16, None, None, A, 16, None, None, 0, cs, so, None,
                                                            None, A, A, A, 16 * 4096, None, A, 16 * 128 * 4, None, 0)
    assert lst(sh, None, None) == -1 and lst(cfg, A, A) == -1 and lst(sh, A, None) == -1
    assert rac.rac_strerror(-3) == "caller buffer too small"
    with pytest.raises(rac.RacError):
        rac._check("x", -1)


def test_payload_header_round_trip_and_rejections(rac):
    cfgs = [rac.CodecCfg(4096, 128, 4, 8), rac.CodecCfg(3584, 128, 3, 0),
            rac.CodecCfg(5120, 128, 8, 0, scale_mode=1, qgroup=256, topk_group=2),
            rac.CodecCfg(4096, 128, 4, 0, scale_mode=1, coef_fmt=1)]
    for cfg in cfgs:
        for T in (0, 1, 131072, 1 << 40):
            h = rac.rac_header_write(cfg, T)
            assert len(h) == rac.HEADER_BYTES == 64 and h[:4] == b"RACP"
            got, gT = rac.rac_header_parse(h)
            assert gT == T and bytes(got) == bytes(cfg)
            assert int.from_bytes(h[52:56], "little") == rac.rac_record_bytes(cfg) and h[60:] == b"\0\0\0\0"
    h = rac.rac_header_write(cfgs[0], 77)
    for i in range(64):                                  # any single corrupted byte is noticed
        bad = bytearray(h)
        bad[i] ^= 0x10
        with pytest.raises(rac.RacError) as e:
            rac.rac_header_parse(bytes(bad))
        assert e.value.code == -1
    # a consistent checksum over an impossible configuration is still refused (record size is re-derived)
    bad = bytearray(h)
    bad[20:24] = (100).to_bytes(4, "little")             # group 100 does not divide 4096
    bad[56:60] = (sum(int.from_bytes(bad[4 * i:4 * i + 4], "little") for i in range(14)) & 0xffffffff).to_bytes(4, "little")
    with pytest.raises(rac.RacError):
        rac.rac_header_parse(bytes(bad))
    with pytest.raises(rac.RacError):
        rac.rac_header_write(rac.CodecCfg(4096, 100, 4, 0), 5)
    with pytest.raises(rac.RacError):
        rac.rac_header_write(cfgs[0], -1)


def test_prepare_marshals_once_and_launches_nothing(rac):
    """binding.prepare runs a wrapper against a recorder: the arguments are checked and marshalled, nothing is
    called; the function it returns holds the library entry point and the marshalled arguments."""
    A = 1 << 20          # a made-up, 16-byte aligned device address: never dereferenced here
    cfg = rac.CodecCfg(4096, 128, 4, 0)
    call = rac.prepare(rac.rac_decode_reconstruct, cfg, A, 16, A, 16, None, None, None, A, A, A, stream=0)
    assert callable(call) and call.keepalive[0][0] is cfg
    assert rac.load() is not None and not isinstance(rac.load(), rac._Recorder)      # the recorder is gone again
    with pytest.raises(ValueError):
        rac.prepare(rac.rac_record_bytes, cfg)                                       # a size query launches nothing
    with pytest.raises(TypeError):
        rac.prepare(rac.rac_decode_reconstruct, cfg, "not a tensor", 16, A, 16, None, None, None, A, A, A, stream=0)
    assert not isinstance(rac.load(), rac._Recorder)                                 # also after a failed prepare
