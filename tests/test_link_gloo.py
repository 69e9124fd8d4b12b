"""The sender/receiver link on CPU: the endpoints of `paper_2608_04991_b200.link` with the CPU oracle as their codec,
first joined in one process, then as two gloo ranks.  What is checked is the protocol: the receiver rebuilds the rows
from the spans alone, both ends hold the same history states after every request, later requests find earlier ones,
and the byte accounting adds up."""
import os
import socket

import numpy as np
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from paper_2608_04991_b200 import link, synth

D, G, BITS, KG, T, NREQ = 256, 64, 4, 1, 300, 3


def _traffic(r, states, ref_row, scale):
    gen = synth.generator(500 + r)
    return synth.affine_noisy_target(states, ref_row, G, gen, scale)


def test_loopback_keeps_both_ends_in_step(orc):
    from link_oracle import OracleCodec
    reqs = synth.request_stream(NREQ, T, seed=5)
    scale = synth.channel_scale(D, 5)
    a, b = link.Loopback.pair()
    cs = OracleCodec(D, G, BITS, topk_group=KG, capacity=NREQ * T)
    cr = OracleCodec(D, G, BITS, topk_group=KG, capacity=NREQ * T)
    snd, rcv = link.Sender(cs, a), link.Receiver(cr, b)
    for r, toks in enumerate(reqs):
        tokens = torch.from_numpy(toks)
        ref_row, spans = cs.query(tokens, snd.n_hist)
        X = _traffic(r, snd.states, ref_row, scale)
        snd.uplink(tokens, X)
        x_sender = snd.x_hat.clone()
        x_hat = rcv.uplink()
        assert torch.equal(x_hat, x_sender)                       # synchronised references (Sec. IV-C)
        # the codec did its job: error within half a step of the group scale, i.e. small against the signal
        err = (x_hat.float() - X.float()).pow(2).sum().sqrt() / X.float().pow(2).sum().sqrt()
        assert err < 0.2
        y_rcv = rcv.downlink(synth.drifted_state(x_hat, synth.generator(900 + r)))
        y_snd = snd.downlink()
        assert torch.equal(y_rcv, y_snd)
        assert snd.n_hist == rcv.n_hist == (r + 1) * T
        assert link.states_digest(snd.states, snd.n_hist) == link.states_digest(rcv.states, rcv.n_hist)
        assert torch.equal(snd.states[: snd.n_hist], rcv.states[: rcv.n_hist])
        if r == 0:
            assert spans.shape[0] == 0 and bool((ref_row < 0).all())
        else:
            assert spans.shape[0] > 0 and int(spans[:, 2].sum()) > T // 4     # later prompts reuse earlier ones
    st = snd.stats
    rec = cs.rec
    assert st.requests == NREQ and st.tokens == NREQ * T
    assert st.payload_bytes == 2 * NREQ * T * rec and st.raw_bytes == 2 * NREQ * T * 2 * D
    n_spans = sum(p["spans"] for p in st.per_request)
    assert st.control_bytes == NREQ * 2 * 8 * link.HEADER_WORDS + 12 * n_spans
    assert (st.payload_bytes + st.control_bytes) < 0.45 * st.raw_bytes


def test_loopback_rejects_a_malformed_frame(orc):
    from link_oracle import OracleCodec
    import pytest
    a, b = link.Loopback.pair()
    rcv = link.Receiver(OracleCodec(D, G, BITS, capacity=64), b)
    a.send(torch.tensor([link.MAGIC_DN, 4, 0, 4 * rcv.codec.rec], dtype=torch.int64))
    with pytest.raises(RuntimeError):
        rcv.uplink()                                   # wrong frame type
    a.send(torch.tensor([link.MAGIC_UP, 65, 0, 65 * rcv.codec.rec], dtype=torch.int64))
    with pytest.raises(RuntimeError):
        rcv.uplink()                                   # more tokens than the history buffer holds
    a.send(torch.tensor([link.MAGIC_UP, 4, 0, 5], dtype=torch.int64))
    with pytest.raises(RuntimeError):
        rcv.uplink()                                   # byte count that is not tokens x record


def _worker(rank, port, out_dir):
    import sys
    sys.path.insert(0, os.path.dirname(os.path.abspath(__file__)))
    from link_oracle import OracleCodec
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=2)
    codec = OracleCodec(D, G, BITS, topk_group=KG, capacity=NREQ * T)
    tr = link.DistTransport(1 - rank)
    reqs = synth.request_stream(NREQ, T, seed=5)
    scale = synth.channel_scale(D, 5)
    end = link.Sender(codec, tr) if rank == 0 else link.Receiver(codec, tr)
    for r, toks in enumerate(reqs):
        if rank == 0:
            tokens = torch.from_numpy(toks)
            ref_row, _ = codec.query(tokens, end.n_hist)
            end.uplink(tokens, _traffic(r, end.states, ref_row, scale))
            end.downlink()
        else:
            x_hat = end.uplink()
            end.downlink(synth.drifted_state(x_hat, synth.generator(900 + r)))
    np.save(os.path.join(out_dir, f"states{rank}.npy"), synth.bf16_bits(end.states[: end.n_hist]))
    digest = torch.tensor([link.states_digest(end.states, end.n_hist)], dtype=torch.int64)
    both = [torch.zeros_like(digest) for _ in range(2)]
    dist.all_gather(both, digest)
    assert int(both[0]) == int(both[1])
    dist.barrier()
    dist.destroy_process_group()


def test_two_gloo_ranks_stay_in_step(tmp_path, orc):
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        port = s.getsockname()[1]
    mp.spawn(_worker, args=(port, str(tmp_path)), nprocs=2, join=True)
    s0, s1 = np.load(tmp_path / "states0.npy"), np.load(tmp_path / "states1.npy")
    assert s0.shape == (NREQ * T, D) and np.array_equal(s0, s1)
    assert np.any(s0 != 0)
