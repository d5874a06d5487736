"""Helpers shared by the GPU parity tests: push a seeded batch through the C ABI, compare with the oracle."""
from __future__ import annotations

import numpy as np
import torch

import oracle
from paper_2510_14686_b200 import workloads as wl

MAX_ABS, MEAN_ABS, LSE_ABS = 1e-2, 1e-3, 1e-3   # bf16 output vs fp64 oracle, V ~ N(0,1)


def dev_bits(a: np.ndarray) -> torch.Tensor:
    """uint16 bit patterns -> int16 CUDA tensor with the same bytes."""
    return torch.from_numpy(np.ascontiguousarray(a).view(np.int16)).cuda()


def host_bits(t: torch.Tensor) -> np.ndarray:
    return t.cpu().numpy().view(np.uint16)


def make_ctx(binding, shape, n_slots, max_seq_len, budget_tokens, max_q_len=4, **kw):
    page = 2 << 20
    pages = sum(-(-(-(-int(t) // 64) * 64 * shape.row_bytes) // page) for t in budget_tokens) + 2
    return binding.Context(shape.n_q_heads, shape.n_kv_heads, shape.head_dim, n_slots, max_seq_len, pages * page,
                           max_q_len=max_q_len, **kw)


def load_requests(ctx, requests, chunk_tokens: int = 1 << 16):
    """reserve + map + append every request's K/V; returns the slot ids."""
    slots = []
    for r in requests:
        s = ctx.kv_reserve(expected_tokens=r.kv_len)
        ctx.kv_map_pages(s, r.kv_len)
        for t0 in range(0, r.kv_len, chunk_tokens):
            t1 = min(r.kv_len, t0 + chunk_tokens)
            ctx.kv_append([s], [t1 - t0], dev_bits(r.k[t0:t1]), dev_bits(r.v[t0:t1]))
        slots.append(s)
    torch.cuda.synchronize()
    return slots


def run_attention(ctx, batch, slots, want_lse=True, use_decode=None):
    s = batch.shape
    q = dev_bits(np.concatenate([r.q for r in batch.requests], axis=0))
    rows = q.shape[0]
    out = torch.zeros((rows, s.n_q_heads, s.head_dim), dtype=torch.int16, device="cuda")
    lse = torch.full((rows, s.n_q_heads), float("nan"), dtype=torch.float32, device="cuda") if want_lse else None
    q_lens = batch.q_lens
    if use_decode is None:
        use_decode = bool((q_lens == 1).all())
    if use_decode:
        ctx.decode_attention(slots, q, out, lse, s.scale)
    else:
        ctx.verify_attention(slots, q_lens, q, out, lse, s.scale)
    ctx.sync_check()
    return host_bits(out), (lse.cpu().numpy() if want_lse else None)


def oracle_batch(batch):
    outs, lses = oracle.attention_batch([r.q for r in batch.requests], [r.k for r in batch.requests],
                                        [r.v for r in batch.requests], batch.shape.scale)
    return np.concatenate(outs, axis=0), np.concatenate(lses, axis=0)


def assert_parity(out_bits, lse, ref_o, ref_lse, max_abs=MAX_ABS, mean_abs=MEAN_ABS):
    got = wl.bits_to_f64(out_bits)
    assert got.shape == ref_o.shape
    assert np.isfinite(got).all()
    err = np.abs(got - ref_o)
    assert err.max() <= max_abs, f"max-abs {err.max():.3e} at {np.unravel_index(err.argmax(), err.shape)}"
    assert err.mean() <= mean_abs, f"mean-abs {err.mean():.3e}"
    if lse is not None:
        e = np.abs(lse.astype(np.float64) - ref_lse)
        assert e.max() <= LSE_ABS, f"lse max-abs {e.max():.3e}"
    return float(err.max()), float(err.mean())
