"""Seeded synthetic inputs shaped like the serving workloads of the xLLM report.

This module only draws lengths and bf16 values; it contains none of the attention or paging
arithmetic, so both the CPU oracle's tests and the CUDA path's tests/benchmark may use it.

The five named workloads stand in for the paper's traces (ShareGPT-like 2k/2k decode, 128K-token
long context, a 32k outlier among short requests, m+1-row speculative verification): attention
cost depends on head shapes and length mixes only, so synthetic N(0,1) values of those shapes
are used.  bf16 values are produced once here (fp32 normal -> round-to-nearest-even bf16) and the
same bit patterns (uint16) go to every consumer.
"""
from __future__ import annotations

from dataclasses import dataclass, field
from typing import Dict, Iterator, List, Optional, Sequence

import numpy as np
import torch


@dataclass(frozen=True)
class Shape:
    """Head geometry of one workload."""

    name: str
    seed: int
    batch: int
    n_q_heads: int
    n_kv_heads: int
    head_dim: int

    @property
    def group(self) -> int:
        return self.n_q_heads // self.n_kv_heads

    @property
    def scale(self) -> float:
        return 1.0 / float(np.sqrt(self.head_dim))

    @property
    def row_bytes(self) -> int:
        """Bytes of K plus V of all KV heads for one token (bf16)."""
        return 2 * self.n_kv_heads * self.head_dim * 2


SHAPES: Dict[str, Shape] = {
    "tiny": Shape("tiny", 1001, 4, 8, 2, 64),
    "decode": Shape("decode", 1002, 64, 28, 4, 128),
    "verify": Shape("verify", 1003, 128, 32, 8, 128),
    "longctx": Shape("longctx", 1004, 8, 40, 8, 128),
    "paged": Shape("paged", 1005, 256, 32, 8, 128),
}

PAGED_MAX_SEQ_LEN = 32768 + 64
PAGED_STEPS = 10


@dataclass
class Request:
    q_len: int
    kv_len: int  # cached tokens including the q_len newest ones
    q: Optional[np.ndarray] = None  # uint16 [q_len, H_q, D]   bf16 bit patterns
    k: Optional[np.ndarray] = None  # uint16 [kv_len, H_kv, D]
    v: Optional[np.ndarray] = None  # uint16 [kv_len, H_kv, D]


@dataclass
class Batch:
    shape: Shape
    requests: List[Request] = field(default_factory=list)

    @property
    def kv_lens(self) -> np.ndarray:
        return np.array([r.kv_len for r in self.requests], dtype=np.int64)

    @property
    def q_lens(self) -> np.ndarray:
        return np.array([r.q_len for r in self.requests], dtype=np.int32)

    @property
    def kv_tokens(self) -> int:
        return int(self.kv_lens.sum())

    def kv_bytes(self) -> int:
        return self.kv_tokens * self.shape.row_bytes

    def algorithmic_bytes(self) -> int:
        """K/V read once, Q read once, O written once (bf16)."""
        qo = int(self.q_lens.sum()) * self.shape.n_q_heads * self.shape.head_dim * 2
        return self.kv_bytes() + 2 * qo


def pareto_length(u: np.ndarray) -> np.ndarray:
    """Pareto(alpha = 1.2) with x_min = 64, clipped above at 32768."""
    return np.clip(np.floor(64.0 * (1.0 - u) ** (-1.0 / 1.2)), 64, 32768).astype(np.int64)


def draw_lengths(name: str, rng: Optional[np.random.Generator] = None):
    """Return (kv_lens[int64], q_lens[int32]) for a named workload, in the stated draw order."""
    s = SHAPES[name]
    rng = np.random.default_rng(s.seed) if rng is None else rng
    if name == "tiny":
        kv = rng.integers(17, 301, size=s.batch)
        ql = np.ones(s.batch, np.int32)
    elif name == "decode":
        kv = rng.integers(512, 4097, size=s.batch)
        ql = np.ones(s.batch, np.int32)
    elif name == "verify":
        z = rng.standard_normal(s.batch)
        kv = np.clip(np.rint(np.exp(np.log(2048.0) + 0.8 * z)), 128, 16384)
        ql = np.full(s.batch, 4, np.int32)
    elif name == "longctx":
        kv = rng.integers(32768, 131073, size=s.batch)
        ql = np.ones(s.batch, np.int32)
    elif name == "paged":
        kv = pareto_length(rng.random(s.batch))
        ql = np.where(rng.random(s.batch) < 0.3, 4, 1).astype(np.int32)
    else:
        raise KeyError(name)
    return kv.astype(np.int64), ql.astype(np.int32)


def bf16_bits(x: torch.Tensor) -> np.ndarray:
    """fp32 tensor -> bf16 (round to nearest even) -> uint16 bit patterns."""
    return x.to(torch.bfloat16).contiguous().view(torch.int16).numpy().view(np.uint16)


def bits_to_f64(bits: np.ndarray) -> np.ndarray:
    """Exact widening of bf16 bit patterns to float64 (value-preserving)."""
    u32 = bits.astype(np.uint32) << np.uint32(16)
    return u32.view(np.float32).astype(np.float64)


def randn_bits(gen: torch.Generator, *size: int) -> np.ndarray:
    return bf16_bits(torch.randn(*size, generator=gen, dtype=torch.float32))


def fill_request(gen: torch.Generator, s: Shape, q_len: int, kv_len: int) -> Request:
    q = randn_bits(gen, q_len, s.n_q_heads, s.head_dim)
    k = randn_bits(gen, kv_len, s.n_kv_heads, s.head_dim)
    v = randn_bits(gen, kv_len, s.n_kv_heads, s.head_dim)
    return Request(q_len, kv_len, q, k, v)


def make_batch(name: str, with_values: bool = True, max_requests: Optional[int] = None) -> Batch:
    """Named workload at its seed: lengths, then per request Q, K, V in that order."""
    s = SHAPES[name]
    kv, ql = draw_lengths(name)
    n = s.batch if max_requests is None else min(s.batch, max_requests)
    b = Batch(s)
    gen = torch.Generator().manual_seed(s.seed)
    for r in range(n):
        if with_values:
            b.requests.append(fill_request(gen, s, int(ql[r]), int(kv[r])))
        else:
            b.requests.append(Request(int(ql[r]), int(kv[r])))
    return b


def custom_batch(seed: int, n_q_heads: int, n_kv_heads: int, head_dim: int,
                 kv_lens: Sequence[int], q_lens: Optional[Sequence[int]] = None,
                 name: str = "custom") -> Batch:
    """Arbitrary small batch for edge cases (ragged tails, q_len mixes, tiny contexts)."""
    q_lens = [1] * len(kv_lens) if q_lens is None else list(q_lens)
    s = Shape(name, seed, len(kv_lens), n_q_heads, n_kv_heads, head_dim)
    gen = torch.Generator().manual_seed(seed)
    b = Batch(s)
    for kv, ql in zip(kv_lens, q_lens):
        b.requests.append(fill_request(gen, s, int(ql), int(kv)))
    return b


# --------------------------------------------------------------------------------------------
# Continuous-batching scenario: 256 slots, ten steps, drafts accepted / rejected, ~10 % of the
# requests finish per step and are replaced.  Only the *script* lives here (who does what when);
# the paging and the attention are the library's and the oracle's business.
# --------------------------------------------------------------------------------------------
@dataclass
class StepPlan:
    t: int
    q_lens: np.ndarray          # int32 [n]   rows each live request submits this step
    new_k: List[np.ndarray]     # per request uint16 [q_len, H_kv, D] rows appended this step
    new_v: List[np.ndarray]
    q: List[np.ndarray]         # per request uint16 [q_len, H_q, D]
    accepted: np.ndarray        # int32 [n]   drafts kept after verification (q_len 4 only; else 0)
    finished: List[int]         # request indices that finish after this step
    release_mode: Dict[int, int]  # index -> 0 (keep pages, reusable) / 1 (unmap)
    admitted: Dict[int, Request]  # index -> replacement request (its prefix = kv_len - q_len rows)


class PagedScenario:
    """Deterministic ten-step script from seed 1005.

    State per request index: the host copy of everything cached so far (``k``/``v`` uint16 arrays)
    and the q_len it will submit next.  ``plans()`` yields one :class:`StepPlan` per step; the
    caller applies it to the library under test and/or hands the concatenated arrays to the oracle.
    """

    def __init__(self, n_requests: Optional[int] = None, steps: int = PAGED_STEPS,
                 max_len: int = 32768):
        self.shape = SHAPES["paged"]
        self.steps = steps
        self.rng = np.random.default_rng(self.shape.seed)
        kv, ql = draw_lengths("paged", self.rng)
        n = self.shape.batch if n_requests is None else n_requests
        self.n = n
        self.max_len = max_len
        kv = np.minimum(kv, max_len)
        self.gen = torch.Generator().manual_seed(self.shape.seed)
        s = self.shape
        self.q_len = ql[:n].copy()
        # prefix already cached before step 0: kv_len - q_len tokens
        self.k = [randn_bits(self.gen, int(kv[r] - ql[r]), s.n_kv_heads, s.head_dim) for r in range(n)]
        self.v = [randn_bits(self.gen, int(kv[r] - ql[r]), s.n_kv_heads, s.head_dim) for r in range(n)]
        self._release_toggle = 0

    def cached_len(self, r: int) -> int:
        return int(self.k[r].shape[0])

    def plans(self) -> Iterator[StepPlan]:
        s = self.shape
        for t in range(self.steps):
            n = self.n
            q_lens = self.q_len.copy()
            new_k, new_v, q = [], [], []
            for r in range(n):
                ql = int(q_lens[r])
                q.append(randn_bits(self.gen, ql, s.n_q_heads, s.head_dim))
                new_k.append(randn_bits(self.gen, ql, s.n_kv_heads, s.head_dim))
                new_v.append(randn_bits(self.gen, ql, s.n_kv_heads, s.head_dim))
            accepted = np.zeros(n, np.int32)
            for r in range(n):
                if q_lens[r] == 4:
                    accepted[r] = int(self.rng.integers(0, 4))
            finished = [r for r in range(n) if (r + t) % 10 == 0]
            release_mode, admitted = {}, {}
            for r in finished:
                release_mode[r] = self._release_toggle
                self._release_toggle ^= 1
                kv_new = int(min(pareto_length(self.rng.random(1))[0], self.max_len))
                ql_new = 4 if self.rng.random() < 0.3 else 1
                pre = kv_new - ql_new
                admitted[r] = Request(ql_new, kv_new, None,
                                      randn_bits(self.gen, pre, s.n_kv_heads, s.head_dim),
                                      randn_bits(self.gen, pre, s.n_kv_heads, s.head_dim))
            yield StepPlan(t, q_lens, new_k, new_v, q, accepted, finished, release_mode, admitted)
            # advance the host copy exactly as the caller is expected to advance the library
            for r in range(n):
                ql = int(q_lens[r])
                keep = ql if ql == 1 else 1 + int(accepted[r])
                self.k[r] = np.concatenate([self.k[r], new_k[r][:keep]], axis=0)
                self.v[r] = np.concatenate([self.v[r], new_v[r][:keep]], axis=0)
            for r in finished:
                a = admitted[r]
                self.k[r], self.v[r], self.q_len[r] = a.k, a.v, a.q_len


# --------------------------------------------------------------------------------------------
# MLA (latent-attention) batches: per token one vector of d_c latent + d_r rotary dims shared by all
# heads; per (query token, head) one query of the same width.  Values only, no arithmetic.
# --------------------------------------------------------------------------------------------
MLA_D_C = 512
MLA_D_R = 64


@dataclass
class MlaBatch:
    n_heads: int
    q_lens: List[int]
    kv_lens: List[int]
    q: np.ndarray                                   # [sum q_len, n_heads, d_c + d_r] bf16 bit patterns
    c: List[np.ndarray] = field(default_factory=list)  # per request [kv_len, d_c + d_r]

    @property
    def scale(self) -> float:
        return 1.0 / float(np.sqrt(128 + MLA_D_R))  # DeepSeek-style: softmax scale of the un-absorbed 128+64-dim heads


def mla_batch(seed: int, n_heads: int, kv_lens: Sequence[int], q_lens: Optional[Sequence[int]] = None,
              latent_std: float = 1.0, q_std: float = 0.25) -> MlaBatch:
    """Seeded MLA batch.  Queries are drawn smaller than keys (absorbed queries are products of two projections;
    with N(0,1) for both, 576-dim scores would make the softmax one-hot and hide mistakes in the weights)."""
    q_lens = [1] * len(kv_lens) if q_lens is None else [int(x) for x in q_lens]
    gen = torch.Generator().manual_seed(seed)
    d = MLA_D_C + MLA_D_R
    q = bf16_bits(torch.randn(sum(q_lens), n_heads, d, generator=gen, dtype=torch.float32) * q_std)
    c = [bf16_bits(torch.randn(int(n), d, generator=gen, dtype=torch.float32) * latent_std) for n in kv_lens]
    return MlaBatch(n_heads, q_lens, [int(n) for n in kv_lens], q, c)


# Named MLA workloads (DeepSeek-style geometry: 128 heads, 512 + 64 dims): lengths only, seeded.
MLA_HEADS = 128
MLA_WORKLOADS = {
    # name: (seed, batch, q_len, low, high)  -- context lengths uniform in [low, high]
    "decode": (3001, 128, 1, 1024, 4096),    # mid-decode batch of 2k/2k-style conversations
    "verify": (3002, 64, 4, 1024, 4096),     # m + 1 = 4 query tokens per sequence (speculative verification)
    "long": (3003, 4, 1, 32768, 32768),      # few 32k-token sequences: every unit is split across CTAs
}


def mla_lengths(name: str):
    seed, batch, q_len, lo, hi = MLA_WORKLOADS[name]
    rng = np.random.default_rng(seed)
    kv = rng.integers(lo, hi + 1, batch).astype(np.int64)
    return kv, np.full(batch, q_len, dtype=np.int32)
