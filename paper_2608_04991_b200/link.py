"""Two endpoints of one link: the sender of boundary states and their receiver.

What crosses the link for one request (Sec. III, problem statement; Sec. IV-B.1; Sec. IV-C):

  uplink   header, the spans of the retrieval (control metadata: the receiver never sees the tokens), one record
           per token;
  downlink header, one record per token, coded against the uplink reconstruction both ends hold (identity rows).

Both ends keep the same history state buffer -- row j is the reconstruction x_hat of history token j -- and append
the uplink reconstruction of every request to it, so the references of later requests stay in step (the sender runs
the receiver's reconstruction on what it just wrote).  The sender alone keeps the tokens and their index.

Everything numerical happens in the library's kernels; this module moves bytes and keeps the two buffers in step.
`Loopback` joins the two ends inside one process, `DistTransport` puts them on two ranks of `torch.distributed`
(NCCL between two GPUs; any backend whose send/recv take the tensors given).  Run as a module under a two-rank
launcher for the two-GPU form:

    python -m torch.distributed.run --nnodes=1 --nproc-per-node 2 --master-addr 127.0.0.1 --master-port 29511 \
        -m paper_2608_04991_b200.link --requests 4 --tokens 4096
"""
from __future__ import annotations

import collections
from dataclasses import dataclass, field
from typing import Deque, Dict, List, Optional, Tuple

import torch

MAGIC_UP = 0x52414355    # "RACU"
MAGIC_DN = 0x52414344    # "RACD"
HEADER_WORDS = 4         # magic, tokens, spans, payload bytes


# ------------------------------------------------------------------------------------------------ transports
class Transport:
    """Ordered, reliable delivery of tensors whose shapes both ends know (the header goes first)."""

    def send(self, t: torch.Tensor) -> None:
        raise NotImplementedError

    def recv(self, t: torch.Tensor) -> None:
        raise NotImplementedError


class Loopback(Transport):
    """Both ends in one process: a queue per direction."""

    def __init__(self, tx: Deque[torch.Tensor], rx: Deque[torch.Tensor]):
        self._tx, self._rx = tx, rx

    @staticmethod
    def pair() -> Tuple["Loopback", "Loopback"]:
        a: Deque[torch.Tensor] = collections.deque()
        b: Deque[torch.Tensor] = collections.deque()
        return Loopback(a, b), Loopback(b, a)

    def send(self, t: torch.Tensor) -> None:
        self._tx.append(t.clone())

    def recv(self, t: torch.Tensor) -> None:
        if not self._rx:
            raise RuntimeError("loopback: nothing was sent")
        got = self._rx.popleft()
        if got.shape != t.shape or got.dtype != t.dtype:
            raise RuntimeError(f"loopback: expected {tuple(t.shape)} {t.dtype}, got {tuple(got.shape)} {got.dtype}")
        t.copy_(got)


class DistTransport(Transport):
    """Point-to-point over `torch.distributed` to one peer rank."""

    def __init__(self, peer: int):
        import torch.distributed as dist
        self._dist, self._peer = dist, peer

    def send(self, t: torch.Tensor) -> None:
        if t.numel():
            self._dist.send(t.contiguous(), dst=self._peer)

    def recv(self, t: torch.Tensor) -> None:
        if t.numel():
            self._dist.recv(t, src=self._peer)


# ------------------------------------------------------------------------------------------------ the codec
class DeviceCodec:
    """The library calls one end needs, on tensors of one CUDA device.  Fails if the library is missing."""

    def __init__(self, cfg, device, capacity: int, min_ngram: int = 4, max_hits: int = 8, step=None, inv_step=None,
                 with_index: bool = True):
        from . import binding as rac
        self.rac, self.cfg, self.dev = rac, cfg, torch.device(device)
        self.d, self.rec = int(cfg.d), rac.rac_record_bytes(cfg)
        self.capacity, self.w = int(capacity), int(min_ngram)
        self.step, self.inv_step = step, inv_step
        self.status = torch.zeros(1, dtype=torch.int32, device=self.dev)
        self.icfg = None
        if with_index:
            self.icfg = rac.IndexCfg(self.capacity, self.w, int(max_hits))
            self.index_bytes = rac.rac_index_bytes(self.icfg)
            self.index = torch.empty(self.index_bytes, dtype=torch.uint8, device=self.dev)
            self.hist_tok = torch.zeros(self.capacity, dtype=torch.int32, device=self.dev)
            rac.rac_index_reset(self.icfg, self.index, self.index_bytes)

    def new_states(self) -> torch.Tensor:
        return torch.zeros(self.capacity, self.d, dtype=torch.bfloat16, device=self.dev)

    def to_device(self, t: torch.Tensor) -> torch.Tensor:
        return t.to(self.dev)

    def empty(self, n: int, dtype) -> torch.Tensor:
        return torch.empty(n, dtype=dtype, device=self.dev)

    # retrieval over the requests appended so far (Sec. IV-B.1)
    def query(self, tokens: torch.Tensor, n_hist: int) -> Tuple[torch.Tensor, torch.Tensor]:
        rac, T = self.rac, tokens.numel()
        ref_row = torch.empty(T, dtype=torch.int32, device=self.dev)
        spans = torch.zeros(T // self.w + 1, 3, dtype=torch.int32, device=self.dev)
        n_spans = torch.zeros(1, dtype=torch.int32, device=self.dev)
        nb = rac.rac_index_query_workspace_bytes(T)
        ws = torch.empty(nb, dtype=torch.uint8, device=self.dev)
        rac.rac_index_query(self.icfg, self.index, self.index_bytes, self.hist_tok, n_hist, tokens, T, False, ref_row,
                            spans, n_spans, ws, nb)
        return ref_row, spans[: int(n_spans.item())]

    def append(self, tokens: torch.Tensor, n_hist: int) -> None:
        T = tokens.numel()
        self.hist_tok[n_hist:n_hist + T] = tokens
        self.rac.rac_index_append(self.icfg, self.index, self.index_bytes, self.hist_tok, n_hist, n_hist + T)

    def rows_from_spans(self, spans: torch.Tensor, T: int) -> torch.Tensor:
        ref_row = torch.empty(T, dtype=torch.int32, device=self.dev)
        n = torch.tensor([spans.shape[0]], dtype=torch.int32, device=self.dev)
        if spans.shape[0] == 0:
            spans = torch.zeros(1, 3, dtype=torch.int32, device=self.dev)   # the call wants a buffer even for no spans
        self.rac.rac_spans_to_rows(spans.contiguous(), n, T, ref_row)
        return ref_row

    # Eq. 6-8 with the sender's own Eq. 9 in the same pass
    def encode_reconstruct(self, X, ref_base, ref_rows: int, ref_row) -> Tuple[torch.Tensor, torch.Tensor]:
        rac, T = self.rac, X.shape[0]
        payload = torch.empty(T * self.rec, dtype=torch.uint8, device=self.dev)
        x_hat = torch.empty_like(X)
        nws = rac.rac_encode_workspace_bytes(self.cfg, T)
        ws = torch.empty(max(nws, 16), dtype=torch.uint8, device=self.dev)
        rac.rac_encode_reconstruct(self.cfg, X, T, ref_base, ref_rows, ref_row, None, None, self.step, self.inv_step,
                                   payload, payload.numel(), x_hat, ws, nws, self.status)
        return payload, x_hat

    # Eq. 9
    def decode_reconstruct(self, payload, T: int, ref_base, ref_rows: int, ref_row) -> torch.Tensor:
        x_hat = torch.empty(T, self.d, dtype=torch.bfloat16, device=self.dev)
        self.rac.rac_decode_reconstruct(self.cfg, payload, T, ref_base, ref_rows, ref_row, None, None, self.step, x_hat,
                                        self.status)
        return x_hat

    def check(self) -> None:
        s = int(self.status.item())
        if s:
            raise RuntimeError(f"device status {s:#x}")


# ------------------------------------------------------------------------------------------------ endpoints
@dataclass
class LinkStats:
    requests: int = 0
    tokens: int = 0
    payload_bytes: int = 0      # records, both directions
    control_bytes: int = 0      # headers and spans
    raw_bytes: int = 0          # the same states as plain bf16, both directions
    matched_tokens: int = 0
    per_request: List[Dict[str, int]] = field(default_factory=list)


class _End:
    def __init__(self, codec, transport: Transport):
        self.codec, self.link = codec, transport
        self.states = codec.new_states()
        self.n_hist = 0
        self.x_hat: Optional[torch.Tensor] = None   # uplink reconstruction of the request in flight
        self.stats = LinkStats()

    def _header(self, magic: int, T: int, n_spans: int, nbytes: int) -> torch.Tensor:
        return self.codec.to_device(torch.tensor([magic, T, n_spans, nbytes], dtype=torch.int64))

    def _recv_header(self, magic: int) -> Tuple[int, int, int]:
        h = self.codec.empty(HEADER_WORDS, torch.int64)
        self.link.recv(h)
        got, T, n_spans, nbytes = (int(v) for v in h.tolist())
        if got != magic:
            raise RuntimeError(f"unexpected frame {got:#x}")
        if T < 0 or self.n_hist + T > self.states.shape[0] or nbytes != T * self.codec.rec or n_spans < 0:
            raise RuntimeError("malformed header")
        return T, n_spans, nbytes

    def _commit(self, T: int) -> None:
        """The request's uplink reconstruction becomes history rows n_hist .. n_hist + T on this end."""
        self.states[self.n_hist:self.n_hist + T] = self.x_hat
        self.n_hist += T
        self.x_hat = None


class Sender(_End):
    """Holds the tokens and their index; codes boundary states against the shared history."""

    def uplink(self, tokens: torch.Tensor, X: torch.Tensor) -> None:
        T = tokens.numel()
        if self.n_hist + T > self.states.shape[0]:
            raise RuntimeError("history buffer full")
        ref_row, spans = self.codec.query(tokens, self.n_hist)
        payload, self.x_hat = self.codec.encode_reconstruct(X, self.states, self.n_hist, ref_row)
        self.link.send(self._header(MAGIC_UP, T, spans.shape[0], payload.numel()))
        self.link.send(spans.reshape(-1))
        self.link.send(payload)
        self._tokens = tokens
        st = self.stats
        matched = int(spans[:, 2].sum().item()) if spans.shape[0] else 0
        st.requests += 1
        st.tokens += T
        st.payload_bytes += payload.numel()
        st.control_bytes += 8 * HEADER_WORDS + 12 * spans.shape[0]
        st.raw_bytes += 2 * T * self.codec.d
        st.matched_tokens += matched
        st.per_request.append({"tokens": T, "spans": int(spans.shape[0]), "matched": matched,
                               "uplink_bytes": payload.numel() + 8 * HEADER_WORDS + 12 * spans.shape[0]})

    def downlink(self) -> torch.Tensor:
        T, _, nbytes = self._recv_header(MAGIC_DN)
        payload = self.codec.empty(nbytes, torch.uint8)
        self.link.recv(payload)
        y_hat = self.codec.decode_reconstruct(payload, T, self.x_hat, T, None)
        self.stats.payload_bytes += nbytes
        self.stats.control_bytes += 8 * HEADER_WORDS
        self.stats.raw_bytes += 2 * T * self.codec.d
        self.codec.append(self._tokens, self.n_hist)
        self._commit(T)
        self.codec.check()
        return y_hat

    def finish_without_downlink(self) -> None:
        self.codec.append(self._tokens, self.n_hist)
        self._commit(self._tokens.numel())
        self.codec.check()


class Receiver(_End):
    """Never sees tokens: rows come from the spans, states from the records."""

    def uplink(self) -> torch.Tensor:
        T, n_spans, nbytes = self._recv_header(MAGIC_UP)
        spans = self.codec.empty(3 * n_spans, torch.int32)
        self.link.recv(spans)
        payload = self.codec.empty(nbytes, torch.uint8)
        self.link.recv(payload)
        ref_row = self.codec.rows_from_spans(spans.reshape(n_spans, 3), T)
        self.x_hat = self.codec.decode_reconstruct(payload, T, self.states, self.n_hist, ref_row)
        return self.x_hat

    def downlink(self, Y: torch.Tensor) -> torch.Tensor:
        """Codes Y against the uplink reconstruction (identity rows); returns what the sender will reconstruct."""
        T = Y.shape[0]
        payload, y_hat = self.codec.encode_reconstruct(Y, self.x_hat, T, None)
        self.link.send(self._header(MAGIC_DN, T, 0, payload.numel()))
        self.link.send(payload)
        self._commit(T)
        self.codec.check()
        return y_hat

    def finish_without_downlink(self) -> None:
        self._commit(self.x_hat.shape[0])
        self.codec.check()


def states_digest(states: torch.Tensor, n_hist: int) -> int:
    """Order-dependent 63-bit digest of the first n_hist rows (to compare the two ends' buffers cheaply)."""
    if n_hist == 0:
        return 0
    bits = states[:n_hist].contiguous().view(torch.int16).to(torch.int64) & 0xFFFF
    idx = torch.arange(bits.numel(), device=bits.device, dtype=torch.int64).reshape(bits.shape)
    mixed = (bits + 1) * ((idx * 2654435761) % 2147483647 + 1)
    return int((mixed % 2305843009213693951).sum().item() % 9223372036854775807)


# ------------------------------------------------------------------------------------------------ two-rank demo
def _demo(argv=None) -> None:
    import argparse
    import json
    import os

    import torch.distributed as dist

    from . import binding as rac, synth

    ap = argparse.ArgumentParser(description="sender on rank 0, receiver on rank 1")
    ap.add_argument("--requests", type=int, default=4)
    ap.add_argument("--tokens", type=int, default=4096)
    ap.add_argument("--d", type=int, default=4096)
    ap.add_argument("--bits", type=int, default=4)
    ap.add_argument("--group", type=int, default=128)
    ap.add_argument("--topk-group", type=int, default=1)
    ap.add_argument("--check", action="store_true",
                    help="fail (exit status 1) unless both ends hold the same reconstructed history at the end: their "
                         "digests travel over the process group and are compared on both ranks")
    a = ap.parse_args(argv)
    rank, world = int(os.environ.get("RANK", "0")), int(os.environ.get("WORLD_SIZE", "1"))
    if world != 2:
        raise SystemExit("the demo needs exactly two ranks (sender, receiver)")
    dev = torch.device("cuda", int(os.environ.get("LOCAL_RANK", "0")))
    torch.cuda.set_device(dev)
    dist.init_process_group("nccl", device_id=dev)
    cfg = rac.CodecCfg(a.d, a.group, a.bits, 0, scale_mode=1, topk_group=a.topk_group)
    cap = a.requests * a.tokens
    codec = DeviceCodec(cfg, dev, cap, with_index=(rank == 0))
    link = DistTransport(1 - rank)
    # both ranks draw the same synthetic traffic; only the sender uses tokens and states, the receiver the drift
    wl = synth.request_stream(a.requests, a.tokens, seed=77)
    scale = synth.channel_scale(a.d, 77, dev)
    end = Sender(codec, link) if rank == 0 else Receiver(codec, link)
    t0, t1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    t0.record()
    for r in range(a.requests):
        gen = synth.generator(1000 + r, dev)
        if rank == 0:
            tokens = torch.from_numpy(wl[r]).to(dev)
            ref_row, _ = codec.query(tokens, end.n_hist)
            X = synth.affine_noisy_target(end.states, ref_row, a.group, gen, scale)
            end.uplink(tokens, X)
            end.downlink()
        else:
            x_hat = end.uplink()
            end.downlink(synth.drifted_state(x_hat, gen))
    t1.record()
    torch.cuda.synchronize()
    digest = torch.tensor([states_digest(end.states, end.n_hist)], dtype=torch.int64, device=dev)
    both = [torch.zeros_like(digest) for _ in range(2)]
    dist.all_gather(both, digest)
    if rank == 0:
        st = end.stats
        print(json.dumps({"requests": st.requests, "tokens": st.tokens, "payload_bytes": st.payload_bytes,
                          "control_bytes": st.control_bytes, "raw_bytes": st.raw_bytes,
                          "wire_over_raw": (st.payload_bytes + st.control_bytes) / st.raw_bytes,
                          "matched_fraction": st.matched_tokens / max(st.tokens, 1),
                          "references_in_step": int(both[0].item()) == int(both[1].item()),
                          "ms_total": t0.elapsed_time(t1)}))
    in_step = int(both[0].item()) == int(both[1].item())
    dist.destroy_process_group()
    if a.check and not in_step:
        raise SystemExit(f"rank {rank}: sender and receiver histories differ")


if __name__ == "__main__":
    _demo()
