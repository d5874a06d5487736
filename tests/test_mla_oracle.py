"""Pins for the MLA oracle: brute force, a library routine, closed forms, invariants.

Chosen so that a plausible slip (value taken from all 576 dims or from the rotary part, scale dropped, mask off
by one, head or token index transposed, un-normalised weights, log base of the LSE) fails at least one of them.
No expected value comes from the oracle itself or from the CUDA path.
"""
import math

import numpy as np
import torch

from oracle import mla_oracle
from paper_2510_14686_b200 import workloads as wl


def bits(x):
    return wl.bf16_bits(torch.as_tensor(np.asarray(x, dtype=np.float32)))


def test_brute_force_python_loops_tiny():
    b = wl.mla_batch(7, 3, [5], [2])
    q, c = wl.bits_to_f64(b.q), wl.bits_to_f64(b.c[0])
    d_c = 4  # the value is the first d_c dims only: a small d_c makes "value = whole vector" fail
    out, lse = mla_oracle.mla_attention(b.q, b.c[0], 0.3, d_c)
    for t in range(2):
        visible = 5 - 2 + t + 1
        for h in range(3):
            s = [0.3 * sum(float(q[t, h, i]) * float(c[j, i]) for i in range(q.shape[2])) for j in range(visible)]
            z = sum(math.exp(x) for x in s)
            for i in range(d_c):
                want = sum(math.exp(s[j]) / z * float(c[j, i]) for j in range(visible))
                assert abs(out[t, h, i] - want) < 1e-12
            assert abs(lse[t, h] - math.log(z)) < 1e-12


def test_against_torch_sdpa_with_separate_value_width():
    b = wl.mla_batch(8, 4, [37], [3])
    scale = b.scale
    out, lse = mla_oracle.mla_attention(b.q, b.c[0], scale, wl.MLA_D_C)
    q = torch.from_numpy(wl.bits_to_f64(b.q))          # [3, 4, 576]
    c = torch.from_numpy(wl.bits_to_f64(b.c[0]))       # [37, 576]
    for t in range(3):
        vis = 37 - 3 + t + 1
        k = c[:vis].unsqueeze(0)                       # [1, vis, 576]: one KV head for all query heads
        v = c[:vis, :wl.MLA_D_C].unsqueeze(0)
        ref = torch.nn.functional.scaled_dot_product_attention(q[t].unsqueeze(1), k.expand(4, -1, -1), v.expand(4, -1, -1),
                                                               scale=scale)
        assert np.allclose(out[t], ref.squeeze(1).numpy(), rtol=0, atol=1e-12)


def test_identical_keys_closed_form():
    rng = np.random.default_rng(3)
    one = rng.standard_normal(wl.MLA_D_C + wl.MLA_D_R)
    c = bits(np.tile(one, (9, 1)))
    q = bits(rng.standard_normal((1, 2, wl.MLA_D_C + wl.MLA_D_R)) * 0.1)
    out, lse = mla_oracle.mla_attention(q, c, 0.5, wl.MLA_D_C)
    cf, qf = wl.bits_to_f64(c), wl.bits_to_f64(q)
    for h in range(2):
        assert np.allclose(out[0, h], cf[0, :wl.MLA_D_C], rtol=0, atol=1e-13)     # mean of identical values
        assert abs(lse[0, h] - (0.5 * float(cf[0] @ qf[0, h]) + math.log(9))) < 1e-12  # natural log, scale applied


def test_rotary_dims_steer_weights_but_are_not_values():
    # two keys with the same latent part and different rotary parts: output is the latent part whatever the weights,
    # while the LSE depends on the rotary dims
    d = wl.MLA_D_C + wl.MLA_D_R
    c = np.zeros((2, d), np.float32)
    c[:, :wl.MLA_D_C] = 0.5
    c[0, wl.MLA_D_C:] = 1.0
    c[1, wl.MLA_D_C:] = -1.0
    q = np.zeros((1, 1, d), np.float32)
    q[0, 0, wl.MLA_D_C:] = 0.25
    out, lse = mla_oracle.mla_attention(bits(q), bits(c), 1.0, wl.MLA_D_C)
    assert out.shape == (1, 1, wl.MLA_D_C) and np.allclose(out, 0.5, atol=1e-15)
    s = 0.25 * 64
    assert abs(lse[0, 0] - math.log(math.exp(s) + math.exp(-s))) < 1e-12


def test_causal_tail_last_token_sees_everything_first_sees_less():
    b = wl.mla_batch(9, 2, [12], [4])
    out, lse = mla_oracle.mla_attention(b.q, b.c[0], 0.2, wl.MLA_D_C)
    for t in range(4):  # token t alone over the prefix it may see
        o1, l1 = mla_oracle.mla_attention(b.q[t:t + 1], b.c[0][:12 - 4 + t + 1], 0.2, wl.MLA_D_C)
        assert np.array_equal(o1[0], out[t]) and np.array_equal(l1[0], lse[t])
    # a key beyond a token's view must not matter: change the last key, only the last token moves
    c2 = b.c[0].copy()
    c2[-1] = bits(np.full(c2.shape[1], 3.0))
    out2, _ = mla_oracle.mla_attention(b.q, c2, 0.2, wl.MLA_D_C)
    assert np.array_equal(out2[:3], out[:3]) and not np.array_equal(out2[3], out[3])


def test_split_and_merge_equals_whole():
    b = wl.mla_batch(10, 3, [50], [1])
    whole, lse = mla_oracle.mla_attention(b.q, b.c[0], 0.1, wl.MLA_D_C)
    a, la = mla_oracle.mla_attention(b.q, b.c[0][:23], 0.1, wl.MLA_D_C, all_visible=True)
    c, lc = mla_oracle.mla_attention(b.q, b.c[0][23:], 0.1, wl.MLA_D_C, all_visible=True)
    # merge written out here: weights exp(lse_i - lse) over the parts
    tot = np.log(np.exp(la) + np.exp(lc))
    merged = np.exp(la - tot)[..., None] * a + np.exp(lc - tot)[..., None] * c
    assert np.allclose(merged, whole, atol=1e-12) and np.allclose(tot, lse, atol=1e-12)


def test_reduces_to_the_pinned_gqa_oracle_when_rotary_query_is_zero():
    # with q_rope = 0 the scores use the latent dims only: multi-query attention with K = V = latent
    import oracle
    b = wl.mla_batch(11, 4, [19], [2])
    d_c = 64
    q = b.q[:, :, :d_c + 8].copy()
    q[:, :, d_c:] = 0
    c = b.c[0][:, :d_c + 8]
    out, lse = mla_oracle.mla_attention(q, c, 0.2, d_c)
    lat = np.ascontiguousarray(c[:, None, :d_c])
    o2, l2 = oracle.attention(np.ascontiguousarray(q[:, :, :d_c]), lat, lat, 0.2)
    assert np.allclose(out, o2, atol=1e-12) and np.allclose(lse, l2, atol=1e-12)


def test_batch_packs_rows_in_request_order():
    b = wl.mla_batch(12, 2, [6, 9, 4], [1, 3, 2])
    out, lse = mla_oracle.mla_attention_batch(b.q, b.c, b.q_lens, 0.2, wl.MLA_D_C)
    assert out.shape == (6, 2, wl.MLA_D_C) and lse.shape == (6, 2)
    o1, l1 = mla_oracle.mla_attention(b.q[1:4], b.c[1], 0.2, wl.MLA_D_C)
    assert np.array_equal(out[1:4], o1) and np.array_equal(lse[1:4], l1)
