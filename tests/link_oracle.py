"""The CPU oracle behind the interface `paper_2608_04991_b200.link` expects of a codec (test infrastructure: lets the
endpoints run as CPU ranks, and gives the GPU endpoints something to be compared with)."""
import numpy as np
import torch

import oracle
from paper_2608_04991_b200 import synth


class OracleCodec:
    def __init__(self, d, group, bits, topk=0, scale_mode=1, qgroup=0, topk_group=0, capacity=4096, min_ngram=4,
                 max_hits=8, step=None, inv_step=None):
        self.d, self.g, self.bits, self.topk = d, group, bits, topk
        self.kw = dict(scale_mode=scale_mode, qgroup=qgroup, topk_group=topk_group)
        self.rec = oracle.record_bytes(d, group, bits, topk, scale_mode, qgroup, topk_group)
        self.capacity, self.w, self.K = capacity, min_ngram, max_hits
        self.step, self.inv_step = step, inv_step
        self.hist = np.zeros(0, np.int32)
        self.req_off = [0]

    def new_states(self):
        return torch.zeros(self.capacity, self.d, dtype=torch.bfloat16)

    def to_device(self, t):
        return t

    def empty(self, n, dtype):
        return torch.empty(n, dtype=dtype)

    def query(self, tokens, n_hist):
        assert n_hist == self.hist.size
        q = tokens.numpy().astype(np.int32)
        if n_hist == 0:
            return torch.full((q.size,), -1, dtype=torch.int32), torch.zeros(0, 3, dtype=torch.int32)
        ref_row, spans = oracle.match_spans_req(self.hist, self.req_off, q, self.w, self.K)
        return torch.from_numpy(ref_row), torch.from_numpy(spans.reshape(-1, 3))

    def append(self, tokens, n_hist):
        assert n_hist == self.hist.size
        self.hist = np.concatenate([self.hist, tokens.numpy().astype(np.int32)])
        self.req_off.append(self.hist.size)

    def rows_from_spans(self, spans, T):
        rows = np.full(T, -1, np.int32)
        for q, h, n in spans.numpy().reshape(-1, 3):
            rows[q:q + n] = np.arange(h, h + n, dtype=np.int32)
        return torch.from_numpy(rows)

    def _ref(self, ref_base, ref_rows, ref_row):
        base = synth.bf16_bits(ref_base[:ref_rows]) if ref_rows > 0 else None
        rows = None if ref_row is None else ref_row.numpy().astype(np.int32)
        if base is None and rows is None:
            raise ValueError("identity rows need a reference")
        return base, rows

    def encode_reconstruct(self, X, ref_base, ref_rows, ref_row):
        T = X.shape[0]
        base, rows = self._ref(ref_base, ref_rows, ref_row)
        pay = oracle.encode(self.d, self.g, self.bits, self.topk, synth.bf16_bits(X), ref_base=base, ref_row=rows,
                            step=self.step, inv_step=self.inv_step, **self.kw)
        xh = oracle.reconstruct(self.d, self.g, self.bits, self.topk, pay, T, ref_base=base, ref_row=rows, step=self.step,
                                **self.kw)
        return torch.from_numpy(pay), synth.bf16_from_bits(xh)

    def decode_reconstruct(self, payload, T, ref_base, ref_rows, ref_row):
        base, rows = self._ref(ref_base, ref_rows, ref_row)
        xh = oracle.reconstruct(self.d, self.g, self.bits, self.topk, payload.numpy(), T, ref_base=base, ref_row=rows,
                                step=self.step, **self.kw)
        return synth.bf16_from_bits(xh)

    def check(self):
        pass
