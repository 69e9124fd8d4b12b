"""Seeded synthetic workloads shaped like the paper's boundary traffic.

This module only DRAWS inputs (activations, references, token streams, step-free
side data).  It holds none of the codec's or the matcher's arithmetic, so both
the CUDA path and the CPU oracle can be fed from it without sharing method code.

The paper measures on real prompts and real model activations (Sec. V); those are
not available offline, so the draws below stand in for them:

* activations: N(0,1) per element times a per-channel scale ~ LogNormal(0, 0.5)
  with four heavy channels multiplied by 20 (a few channels of an LLM hidden
  state carry most of the magnitude);
* prefill references: an affine image of the activation per (token, group) plus
  N(0, 0.05) noise, so that an affine fit has something to recover;
* token streams: Zipf(1.1) ids over a 32000-entry vocabulary; queries are built
  from fresh Zipf stretches alternating with copies of history spans of length
  U{8..256};
* decode states: a random walk with N(0, 0.3) steps, the reference being a
  per-channel gain/bias image of the previous reconstructed state.

Everything is a pure function of its seed.  Tensors are drawn with a
``torch.Generator`` on the requested device (CPU and CUDA streams differ; a test
that needs the same values on both sides draws once and copies).
"""
from __future__ import annotations

from dataclasses import dataclass
from typing import Optional, Tuple

import numpy as np
import torch

BASE_SEED = 0x5AC0
VOCAB = 32000
ZIPF_S = 1.1
_CHUNK = 8192  # rows drawn at a time, bounds the fp32 temporaries


def generator(seed: int, device="cpu") -> torch.Generator:
    g = torch.Generator(device=device)
    g.manual_seed(int(seed))
    return g


# ----------------------------------------------------------------- activations
def channel_scale(d: int, seed: int, device="cpu", heavy: int = 4, heavy_gain: float = 20.0) -> torch.Tensor:
    """float32[d]: LogNormal(0, 0.5) with ``heavy`` seeded channels multiplied by ``heavy_gain``."""
    rng = np.random.default_rng([BASE_SEED, seed, 1])
    s = np.exp(0.5 * rng.standard_normal(d)).astype(np.float32)
    idx = rng.choice(d, size=heavy, replace=False)
    s[idx] *= heavy_gain
    return torch.from_numpy(s).to(device)


def activations(T: int, d: int, scale: torch.Tensor, gen: torch.Generator) -> torch.Tensor:
    """bf16[T,d] = bf16(N(0,1) * scale_c)."""
    dev = scale.device
    out = torch.empty((T, d), dtype=torch.bfloat16, device=dev)
    for t0 in range(0, T, _CHUNK):
        n = min(_CHUNK, T - t0)
        z = torch.randn((n, d), generator=gen, device=dev, dtype=torch.float32)
        out[t0:t0 + n] = (z * scale).to(torch.bfloat16)
    return out


def affine_noisy_reference(X: torch.Tensor, group: int, gen: torch.Generator, noise: float = 0.05,
                           a_lo: float = 0.8, a_hi: float = 1.2, b_std: float = 0.1) -> torch.Tensor:
    """R = bf16((X - b)/a + N(0, noise)), a ~ U(a_lo, a_hi), b ~ N(0, b_std) per (token, group)."""
    T, d = X.shape
    J = d // group
    dev = X.device
    R = torch.empty_like(X)
    for t0 in range(0, T, _CHUNK):
        n = min(_CHUNK, T - t0)
        a = torch.rand((n, J, 1), generator=gen, device=dev) * (a_hi - a_lo) + a_lo
        b = torch.randn((n, J, 1), generator=gen, device=dev) * b_std
        z = torch.randn((n, J, group), generator=gen, device=dev) * noise
        x = X[t0:t0 + n].float().view(n, J, group)
        R[t0:t0 + n] = ((x - b) / a + z).view(n, d).to(torch.bfloat16)
    return R


def affine_noisy_target(Hs: torch.Tensor, rows: torch.Tensor, group: int, gen: torch.Generator,
                        fresh_scale: torch.Tensor, noise: float = 0.05) -> torch.Tensor:
    """Query activations for a span-matched prefill: where ``rows[t] >= 0`` the row is
    bf16(a*Hs[rows[t]] + b + a*N(0,noise)) per (token, group); elsewhere a fresh draw."""
    T = rows.numel()
    d = Hs.shape[1]
    J = d // group
    dev = Hs.device
    X = torch.empty((T, d), dtype=torch.bfloat16, device=dev)
    for t0 in range(0, T, _CHUNK):
        n = min(_CHUNK, T - t0)
        rw = rows[t0:t0 + n].to(dev).long()
        has = rw >= 0
        a = torch.rand((n, J, 1), generator=gen, device=dev) * 0.4 + 0.8
        b = torch.randn((n, J, 1), generator=gen, device=dev) * 0.1
        z = torch.randn((n, J, group), generator=gen, device=dev) * noise
        fresh = torch.randn((n, d), generator=gen, device=dev) * fresh_scale
        src = Hs[rw.clamp(min=0)].float().view(n, J, group)
        y = (a * src + b + a * z).view(n, d)
        X[t0:t0 + n] = torch.where(has[:, None], y, fresh).to(torch.bfloat16)
    return X


def drifted_state(X_hat: torch.Tensor, gen: torch.Generator, gain: float = 1.05, noise: float = 0.2) -> torch.Tensor:
    """Downlink stand-in: Y = bf16(gain * X_hat + N(0, noise))."""
    T, d = X_hat.shape
    Y = torch.empty_like(X_hat)
    for t0 in range(0, T, _CHUNK):
        n = min(_CHUNK, T - t0)
        z = torch.randn((n, d), generator=gen, device=X_hat.device) * noise
        Y[t0:t0 + n] = (X_hat[t0:t0 + n].float() * gain + z).to(torch.bfloat16)
    return Y


def random_walk_step(state: torch.Tensor, gen: torch.Generator, drift: float = 0.3) -> torch.Tensor:
    """Next decode state: bf16(state + N(0, drift))."""
    z = torch.randn(state.shape, generator=gen, device=state.device) * drift
    return (state.float() + z).to(torch.bfloat16)


def predictor_gain_bias(d: int, seed: int, device="cpu") -> Tuple[torch.Tensor, torch.Tensor]:
    """Per-channel stand-in for the decode predictor: gain ~ U(0.9,1.1), bias ~ N(0,0.02), float16[d]."""
    rng = np.random.default_rng([BASE_SEED, seed, 2])
    g = rng.uniform(0.9, 1.1, d).astype(np.float16)
    b = (0.02 * rng.standard_normal(d)).astype(np.float16)
    return torch.from_numpy(g).to(device), torch.from_numpy(b).to(device)


# ----------------------------------------------------------------- token streams
def zipf_tokens(n: int, rng: np.random.Generator, vocab: int = VOCAB, s: float = ZIPF_S) -> np.ndarray:
    """int32[n] with p(rank r) proportional to r^-s over ``vocab`` ids."""
    p = np.arange(1, vocab + 1, dtype=np.float64) ** (-s)
    cdf = np.cumsum(p / p.sum())
    u = rng.random(n)
    return np.minimum(np.searchsorted(cdf, u), vocab - 1).astype(np.int32)


@dataclass
class TokenWorkload:
    hist: np.ndarray          # int32[n_hist]
    query: np.ndarray         # int32[n_query]
    planted_row: np.ndarray   # int32[n_query]: history position a query token was copied from, -1 = fresh
    planted_coverage: float


def span_workload(n_hist: int, n_query: int, seed: int, gap_max: int = 176,
                  len_lo: int = 8, len_hi: int = 256) -> TokenWorkload:
    """History of Zipf tokens; query = fresh gaps U{0..gap_max} alternating with copies of
    history spans of length U{len_lo..len_hi} at uniform starts (gap_max 176 gives about 60 %
    planted coverage, 112 about 70 %)."""
    rng = np.random.default_rng([BASE_SEED, seed, 3])
    hist = zipf_tokens(n_hist, rng)
    query = np.empty(n_query, np.int32)
    planted = np.full(n_query, -1, np.int32)
    i = 0
    while i < n_query:
        gap = int(rng.integers(0, gap_max + 1))
        gap = min(gap, n_query - i)
        if gap:
            query[i:i + gap] = zipf_tokens(gap, rng)
            i += gap
        if i >= n_query:
            break
        L = int(rng.integers(len_lo, len_hi + 1))
        L = min(L, n_query - i, n_hist)
        j = int(rng.integers(0, n_hist - L + 1))
        query[i:i + L] = hist[j:j + L]
        planted[i:i + L] = np.arange(j, j + L, dtype=np.int32)
        i += L
    return TokenWorkload(hist, query, planted, float((planted >= 0).mean()))


def request_stream(n_req: int, tokens: int, seed: int, gap_max: int = 112, len_lo: int = 8,
                   len_hi: int = 256) -> list:
    """``n_req`` prompts of ``tokens`` ids each: the first is fresh Zipf text, every later one alternates fresh
    gaps U{0..gap_max} with copies of spans U{len_lo..len_hi} taken from inside ONE earlier prompt (multi-turn
    traffic: shared system prompts, quoted context).  Returns a list of int32 arrays."""
    rng = np.random.default_rng([BASE_SEED, seed, 11])
    out = [zipf_tokens(tokens, rng)]
    for _ in range(1, n_req):
        q = np.empty(tokens, np.int32)
        i = 0
        while i < tokens:
            gap = min(int(rng.integers(0, gap_max + 1)), tokens - i)
            if gap:
                q[i:i + gap] = zipf_tokens(gap, rng)
                i += gap
            if i >= tokens:
                break
            src = out[int(rng.integers(0, len(out)))]
            L = min(int(rng.integers(len_lo, len_hi + 1)), tokens - i, src.size)
            j = int(rng.integers(0, src.size - L + 1))
            q[i:i + L] = src[j:j + L]
            i += L
        out.append(q)
    return out


# ----------------------------------------------------------------- bit views
def bf16_bits(x: torch.Tensor) -> np.ndarray:
    """bf16 tensor -> numpy uint16 bit patterns (host copy)."""
    return x.detach().contiguous().cpu().view(torch.int16).numpy().view(np.uint16)


def f16_bits(x: torch.Tensor) -> np.ndarray:
    return x.detach().contiguous().cpu().view(torch.int16).numpy().view(np.uint16)


def bf16_from_bits(bits: np.ndarray, device="cpu") -> torch.Tensor:
    return torch.from_numpy(np.ascontiguousarray(bits).view(np.int16)).view(torch.bfloat16).to(device)
