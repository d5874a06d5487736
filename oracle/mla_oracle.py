"""CPU oracle of the MLA decode / verification attention (test infrastructure only; fp64, numpy).

Only the tests, the smoke check and the benchmark's CPU legs may import this module; the product
package never does.

What it defines.  The report's attention operator for DeepSeek-style models is multi-head latent
attention over a KV cache that is contiguous in virtual address space ("Efficient Memory Management",
paragraph "Operator Adaptation"), and with speculative decoding m+1 query tokens of one sequence meet
the same K matrix ("Algorithm Optimizations", paragraph "MLA Optimization").  In the weight-absorbed
decode form every token of the cache is ONE vector c = [latent (d_c dims) | rotary key (d_r dims)]
shared by all heads; head h of query token t holds q = [q_latent | q_rope] of the same d_c + d_r dims:

    s_j   = scale * <q, c_j>                       for every key j visible to token t
    w     = softmax(s)
    out   = sum_j w_j * c_j[:d_c]                  (the latent part is also the value)
    lse   = log(sum_j exp(s_j))                    (natural log)

Query token t of q_len (the newest q_len tokens of the sequence) sees keys 0 .. L - q_len + t.
The report gives no formula of its own; this is the textbook definition the operator must reach up to
rounding order, so the oracle is that definition written out, one (token, head) row at a time.

Inputs are bf16 bit patterns (uint16); every result is float64.
"""
from __future__ import annotations

from typing import List, Sequence, Tuple

import numpy as np


def _f64(bits: np.ndarray) -> np.ndarray:
    """bf16 bit patterns -> float64 (exact)."""
    return (np.asarray(bits, dtype=np.uint16).astype(np.uint32) << 16).view(np.float32).astype(np.float64)


def mla_attention(q_bits: np.ndarray, c_bits: np.ndarray, scale: float, d_c: int,
                  all_visible: bool = False) -> Tuple[np.ndarray, np.ndarray]:
    """One request: q_bits [q_len, H, d_c + d_r], c_bits [L, d_c + d_r] -> out [q_len, H, d_c], lse [q_len, H]."""
    q = _f64(q_bits)
    c = _f64(c_bits)
    q_len, n_heads, d = q.shape
    n_keys = c.shape[0]
    assert c.shape[1] == d and 0 < d_c <= d and n_keys >= (1 if all_visible else q_len)
    out = np.zeros((q_len, n_heads, d_c))
    lse = np.zeros((q_len, n_heads))
    for t in range(q_len):
        visible = n_keys if all_visible else n_keys - q_len + t + 1
        keys = c[:visible]                       # [visible, d]
        values = c[:visible, :d_c]               # the latent part
        for h in range(n_heads):
            s = scale * (keys @ q[t, h])         # [visible]
            m = s.max()
            e = np.exp(s - m)
            z = e.sum()
            out[t, h] = (e / z) @ values
            lse[t, h] = m + np.log(z)
    return out, lse


def mla_attention_batch(q_bits: np.ndarray, c_bits: Sequence[np.ndarray], q_lens: Sequence[int], scale: float,
                        d_c: int) -> Tuple[np.ndarray, np.ndarray]:
    """Requests packed row after row: q_bits [sum q_len, H, d]; returns out [sum q_len, H, d_c], lse [sum q_len, H]."""
    outs: List[np.ndarray] = []
    lses: List[np.ndarray] = []
    row = 0
    for ql, c in zip(q_lens, c_bits):
        o, l = mla_attention(q_bits[row:row + ql], c, scale, d_c)
        outs.append(o)
        lses.append(l)
        row += ql
    return np.concatenate(outs, axis=0), np.concatenate(lses, axis=0)
