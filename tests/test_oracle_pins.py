"""Pins for the CPU oracle: closed forms, invariants, special cases and brute force.

Each test is chosen so that a plausible slip in oracle.c (wrong head map, mask offset by one,
missing scale, sign of the exponent, un-normalised output, transposed index) makes it fail.
None of the expected values comes from the oracle itself or from the CUDA path.
"""
import math
from decimal import Decimal, getcontext

import numpy as np
import pytest
import torch

import oracle
from paper_2510_14686_b200 import workloads as wl


def bits(x):
    """float array -> bf16 bit patterns (round to nearest even) via torch."""
    return wl.bf16_bits(torch.as_tensor(np.asarray(x, dtype=np.float32)))


def f64(b):
    return wl.bits_to_f64(b)


def rand_bits(rng, *shape):
    return bits(rng.standard_normal(shape))


# ---- P1: one key ---------------------------------------------------------------------
def test_single_key_returns_v_exactly():
    rng = np.random.default_rng(1)
    hq, hkv, d = 8, 2, 16
    q, k, v = rand_bits(rng, 1, hq, d), rand_bits(rng, 1, hkv, d), rand_bits(rng, 1, hkv, d)
    o, lse = oracle.attention(q, k, v, 0.25)
    g = hq // hkv
    for h in range(hq):
        assert np.array_equal(o[0, h], f64(v)[0, h // g])  # bit exact, and the right KV head
        s = 0.25 * float(np.dot(f64(q)[0, h], f64(k)[0, h // g]))
        assert lse[0, h] == pytest.approx(s, abs=1e-12)


# ---- P2: identical keys -> uniform weights -------------------------------------------------
def test_identical_keys_give_mean_of_v_and_lse_shift():
    rng = np.random.default_rng(2)
    n, hq, hkv, d = 37, 4, 2, 8
    k1 = rand_bits(rng, 1, hkv, d)
    k = np.repeat(k1, n, axis=0)
    q, v = rand_bits(rng, 1, hq, d), rand_bits(rng, n, hkv, d)
    o, lse = oracle.attention(q, k, v, 0.5)
    for h in range(hq):
        g = h // 2
        assert np.allclose(o[0, h], f64(v)[:, g].mean(axis=0), atol=1e-14)
        s = 0.5 * float(np.dot(f64(q)[0, h], f64(k1)[0, g]))
        assert lse[0, h] == pytest.approx(s + math.log(n), abs=1e-12)


# ---- P3: weights sum to one; constant V is returned -----------------------------------------
def test_weights_sum_to_one_and_constant_v():
    rng = np.random.default_rng(3)
    n, hq, hkv, d = 50, 6, 3, 8
    q, k = rand_bits(rng, 3, hq, d), rand_bits(rng, n, hkv, d)
    for i in range(3):
        for h in range(hq):
            p = oracle.softmax_weights(q, k, 0.3, i, h)
            assert len(p) == n - 3 + i + 1
            assert p.sum() == pytest.approx(1.0, abs=1e-14)
            assert (p > 0).all()
    c = rand_bits(rng, 1, 1, d)
    v = np.broadcast_to(c, (n, hkv, d)).copy()
    o, _ = oracle.attention(q, k, v, 0.3)
    assert np.allclose(o, f64(c)[0, 0], atol=1e-14)


# ---- P4: split the context anywhere, merge by log-sum-exp ------------------------------------
@pytest.mark.parametrize("n", [2, 5, 12])
def test_split_and_merge_equals_unsplit(n):
    rng = np.random.default_rng(40 + n)
    hq, hkv, d = 4, 2, 8
    q, k, v = rand_bits(rng, 1, hq, d), rand_bits(rng, n, hkv, d), rand_bits(rng, n, hkv, d)
    o_ref, lse_ref = oracle.attention(q, k, v, 0.4)
    cuts2 = [(c,) for c in range(1, n)]
    cuts3 = [(a, b) for a in range(1, n) for b in range(a + 1, n)]
    for cuts in cuts2 + cuts3:
        edges = (0,) + cuts + (n,)
        parts = [oracle.attention(q, k[a:b], v[a:b], 0.4) for a, b in zip(edges[:-1], edges[1:])]
        for h in range(hq):
            o, lse = oracle.merge_lse(np.stack([p[0][0, h] for p in parts]), np.array([p[1][0, h] for p in parts]))
            assert np.allclose(o, o_ref[0, h], atol=1e-12)
            assert lse == pytest.approx(lse_ref[0, h], abs=1e-12)


def test_merge_ignores_empty_part():
    o, lse = oracle.merge_lse(np.array([[1.0, 2.0], [7.0, 7.0]]), np.array([0.5, -np.inf]))
    assert np.array_equal(o, [1.0, 2.0]) and lse == 0.5
    # two equal-weight parts average; lse gains log 2
    o, lse = oracle.merge_lse(np.array([[1.0, 3.0], [3.0, 5.0]]), np.array([0.25, 0.25]))
    assert np.allclose(o, [2.0, 4.0]) and lse == pytest.approx(0.25 + math.log(2.0))
    # weights follow exp(lse): part 0 is e times heavier
    o, _ = oracle.merge_lse(np.array([[1.0], [0.0]]), np.array([1.0, 0.0]))
    assert o[0] == pytest.approx(math.e / (math.e + 1.0))
    with pytest.raises(ValueError):
        oracle.merge_lse(np.zeros((2, 2)), np.array([-np.inf, -np.inf]))


# ---- P5: GQA == MHA with repeated KV heads ---------------------------------------------------
def test_gqa_equals_mha_with_repeated_heads():
    rng = np.random.default_rng(5)
    n, hq, hkv, d = 23, 12, 3, 8
    q, k, v = rand_bits(rng, 2, hq, d), rand_bits(rng, n, hkv, d), rand_bits(rng, n, hkv, d)
    o, lse = oracle.attention(q, k, v, 0.35)
    g = hq // hkv
    o2, lse2 = oracle.attention(q, np.repeat(k, g, axis=1), np.repeat(v, g, axis=1), 0.35)
    assert np.array_equal(o, o2) and np.array_equal(lse, lse2)
    # a wrong (interleaved) head map must differ
    perm = np.arange(hq).reshape(g, hkv).T.reshape(-1)
    o3, _ = oracle.attention(q[:, perm], k, v, 0.35)
    assert not np.allclose(o3, o)


# ---- P6: verify row i == decode on the context truncated after that row's token ----------------
def test_verify_row_equals_decode_on_truncated_context():
    rng = np.random.default_rng(6)
    n, ql, hq, hkv, d = 19, 4, 4, 2, 8
    q, k, v = rand_bits(rng, ql, hq, d), rand_bits(rng, n, hkv, d), rand_bits(rng, n, hkv, d)
    o, lse = oracle.attention(q, k, v, 0.3)
    for i in range(ql):
        vis = n - ql + i + 1
        oi, lsei = oracle.attention(q[i:i + 1], k[:vis], v[:vis], 0.3)
        assert np.array_equal(o[i], oi[0]) and np.array_equal(lse[i], lsei[0])
    # the last row sees everything, the first row does not see the 3 newest keys
    assert not np.allclose(o[0], oracle.attention(q[0:1], k, v, 0.3)[0][0])


# ---- P7: two keys, logistic closed form ----------------------------------------------------
def test_two_keys_logistic():
    rng = np.random.default_rng(7)
    d = 8
    q, k = rand_bits(rng, 1, 1, d), rand_bits(rng, 2, 1, d)
    v = bits(np.array([[[1.0] + [0.0] * (d - 1)], [[0.0] * d]]))
    scale = 0.7
    o, _ = oracle.attention(q, k, v, scale)
    x = scale * float(np.dot(f64(q)[0, 0], f64(k)[0, 0] - f64(k)[1, 0]))
    assert o[0, 0, 0] == pytest.approx(1.0 / (1.0 + math.exp(-x)), abs=1e-14)
    assert np.all(o[0, 0, 1:] == 0.0)


# ---- P8: shift and permutation invariance -----------------------------------------------------
def test_shift_and_permutation_invariance():
    rng = np.random.default_rng(8)
    n, d = 16, 4
    # small integers stay exact in bf16, so the shifted keys are exactly k + c
    q = bits(rng.integers(-3, 4, (1, 1, d)))
    k = bits(rng.integers(-3, 4, (n, 1, d)))
    v = rand_bits(rng, n, 1, d)
    c = rng.integers(-2, 3, d).astype(np.float64)
    o, lse = oracle.attention(q, k, v, 0.25)
    o2, lse2 = oracle.attention(q, bits(f64(k) + c), v, 0.25)
    assert np.allclose(o, o2, atol=1e-13)
    assert lse2[0, 0] - lse[0, 0] == pytest.approx(0.25 * float(np.dot(f64(q)[0, 0], c)), abs=1e-12)
    perm = rng.permutation(n)
    o3, lse3 = oracle.attention(q, k[perm], v[perm], 0.25)
    assert np.allclose(o, o3, atol=1e-13) and lse3[0, 0] == pytest.approx(lse[0, 0], abs=1e-12)


# ---- P9: stability with huge scores -----------------------------------------------------------
def test_huge_scores_are_stable():
    d, n = 4, 9
    q = bits(np.full((1, 1, d), 64.0))
    k = np.zeros((n, 1, d), np.float32)
    k[5] = 64.0  # score 64*64*4*scale
    v = rand_bits(np.random.default_rng(9), n, 1, d)
    o, lse = oracle.attention(q, bits(k), v, 1.0)  # one score = 16384, others 0
    assert np.array_equal(o[0, 0], f64(v)[5, 0]) and np.isfinite(lse).all()
    assert lse[0, 0] == pytest.approx(16384.0)
    o, lse = oracle.attention(q, bits(-np.abs(k) - 64.0), v, 1.0)  # all very negative, key 5 the most
    assert np.isfinite(o).all() and np.isfinite(lse).all()
    kk = bits(np.full((n, 1, d), -64.0))
    o, lse = oracle.attention(q, kk, v, 1.0)  # all equal at -16384: uniform
    assert np.allclose(o[0, 0], f64(v)[:, 0].mean(axis=0), atol=1e-14)
    assert lse[0, 0] == pytest.approx(-16384.0 + math.log(n))


# ---- P10: 50-digit brute force --------------------------------------------------------------
def test_decimal_brute_force():
    getcontext().prec = 50
    rng = np.random.default_rng(10)
    n, ql, hq, hkv, d = 8, 2, 2, 1, 4
    q, k, v = rand_bits(rng, ql, hq, d), rand_bits(rng, n, hkv, d), rand_bits(rng, n, hkv, d)
    scale = 0.5  # exact in binary
    o, lse = oracle.attention(q, k, v, scale)
    D = lambda x: Decimal(float(x))  # bf16 values convert exactly
    for i in range(ql):
        vis = n - ql + i + 1
        for h in range(hq):
            s = [Decimal(scale) * sum(D(f64(q)[i, h, t]) * D(f64(k)[j, 0, t]) for t in range(d)) for j in range(vis)]
            e = [x.exp() for x in s]
            tot = sum(e)
            for t in range(d):
                ref = sum(e[j] * D(f64(v)[j, 0, t]) for j in range(vis)) / tot
                assert abs(Decimal(float(o[i, h, t])) - ref) <= Decimal("1e-14") * max(Decimal(1), abs(ref))
            assert abs(Decimal(float(lse[i, h])) - tot.ln()) <= Decimal("1e-13")


# ---- P11: library special case (torch fp64 SDPA, explicit mask, repeated heads) ----------------------
@pytest.mark.parametrize("seed", range(12))
def test_against_torch_sdpa_fp64(seed):
    rng = np.random.default_rng(1100 + seed)
    hkv = int(rng.integers(1, 4))
    g = int(rng.integers(1, 8))
    hq = hkv * g
    d = int(rng.choice([4, 8, 16, 64]))
    ql = int(rng.integers(1, 5))
    n = int(rng.integers(ql, 70))
    scale = float(rng.uniform(0.05, 0.6))
    q, k, v = rand_bits(rng, ql, hq, d), rand_bits(rng, n, hkv, d), rand_bits(rng, n, hkv, d)
    o, lse = oracle.attention(q, k, v, scale)
    tq = torch.from_numpy(f64(q)).permute(1, 0, 2)[None]                      # [1,Hq,ql,D]
    tk = torch.from_numpy(f64(k)).permute(1, 0, 2).repeat_interleave(g, 0)[None]
    tv = torch.from_numpy(f64(v)).permute(1, 0, 2).repeat_interleave(g, 0)[None]
    pos = torch.arange(n)[None, :] <= (n - ql + torch.arange(ql))[:, None]      # visible keys per row
    ref = torch.nn.functional.scaled_dot_product_attention(tq, tk, tv, attn_mask=pos, scale=scale)
    assert np.allclose(o, ref[0].permute(1, 0, 2).numpy(), atol=1e-12)
    s = torch.einsum("hid,hjd->hij", tq[0], tk[0]) * scale
    ref_lse = torch.logsumexp(s.masked_fill(~pos, float("-inf")), dim=-1)        # [Hq,ql]
    assert np.allclose(lse, ref_lse.T.numpy(), atol=1e-12)


def test_batch_driver_equals_single_calls():
    b = wl.custom_batch(77, 4, 2, 16, [5, 33, 64, 65], [1, 4, 2, 3])
    outs, lses = oracle.attention_batch([r.q for r in b.requests], [r.k for r in b.requests],
                                        [r.v for r in b.requests], b.shape.scale, n_threads=3)
    for r, o, l in zip(b.requests, outs, lses):
        o1, l1 = oracle.attention(r.q, r.k, r.v, b.shape.scale)
        assert np.array_equal(o, o1) and np.array_equal(l, l1)


def test_rejects_bad_sizes():
    z = np.zeros((2, 2, 4), np.uint16)
    with pytest.raises(ValueError):
        oracle.attention(np.zeros((3, 2, 4), np.uint16), z, z, 1.0)  # kv_len < q_len
    with pytest.raises(ValueError):
        oracle.attention(np.zeros((1, 3, 4), np.uint16), z, z, 1.0)  # H_q not a multiple of H_kv


# ---- P12 (host part): Eq. 2 ---------------------------------------------------------------------
def test_xtensor_locate_identities():
    rng = np.random.default_rng(12)
    for page in (4096, 65536, 2 << 20, 3 * 4096):
        start = int(rng.integers(1 << 30, 1 << 40)) * 2
        for _ in range(50):
            off = int(rng.integers(0, 64 * page))
            idx, rem = oracle.xtensor_locate(start + off, start, page)
            assert idx * page + rem == off and 0 <= rem < page
        assert oracle.xtensor_locate(start, start, page) == (0, 0)
        assert oracle.xtensor_locate(start + page - 1, start, page) == (0, page - 1)
        assert oracle.xtensor_locate(start + page, start, page) == (1, 0)
        assert oracle.xtensor_locate(start + 5 * page + 7, start, page) == (5, 7)
    with pytest.raises(ValueError):
        oracle.xtensor_locate(10, 11, 4096)
