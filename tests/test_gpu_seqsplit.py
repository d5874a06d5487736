"""GPU: a sequence's KV split over several ranges -- partial attention per part, log-sum-exp merge (the report's
"aggregation operator" for KV blocks migrated to another DP group).  The parts live in separate slots of one context,
which is what two ranks holding one part each compute, one after the other."""
import os

import numpy as np
import pytest
import torch

from paper_2510_14686_b200 import workloads as wl

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def binding():
    from paper_2510_14686_b200 import binding as b

    return b


def cut_points(rng, kv_len, q_len, n_parts):
    """n_parts - 1 cuts: every part holds a token, the last one all query tokens."""
    hi = kv_len - q_len
    if hi < n_parts - 1:
        return None
    cuts = sorted(rng.choice(np.arange(1, hi + 1), size=n_parts - 1, replace=False).tolist()) if n_parts > 1 else []
    return [0] + cuts + [kv_len]


def run_split(binding, batch, n_parts, seed):
    import gpu_harness as gh
    import oracle

    s = batch.shape
    rng = np.random.default_rng(seed)
    bounds = [cut_points(rng, r.kv_len, r.q_len, n_parts) for r in batch.requests]
    assert all(b is not None for b in bounds)
    n = len(batch.requests)
    with gh.make_ctx(binding, s, n * n_parts, max(r.kv_len for r in batch.requests) + 8,
                     [b[p + 1] - b[p] for b in bounds for p in range(n_parts)], max_q_len=4) as ctx:
        slots = [[None] * n for _ in range(n_parts)]
        for i, (r, b) in enumerate(zip(batch.requests, bounds)):
            for p in range(n_parts):
                sl = ctx.kv_reserve(expected_tokens=b[p + 1] - b[p])
                ctx.kv_map_pages(sl, b[p + 1] - b[p])
                ctx.kv_append([sl], [b[p + 1] - b[p]], gh.dev_bits(r.k[b[p]:b[p + 1]]), gh.dev_bits(r.v[b[p]:b[p + 1]]))
                slots[p][i] = sl
        q = gh.dev_bits(np.concatenate([r.q for r in batch.requests], axis=0))
        rows = q.shape[0]
        outs = torch.full((n_parts, rows, s.n_q_heads, s.head_dim), float("nan"), dtype=torch.float32, device="cuda")
        lses = torch.full((n_parts, rows, s.n_q_heads), float("nan"), dtype=torch.float32, device="cuda")
        for p in range(n_parts):
            ctx.partial_attention(slots[p], batch.q_lens, [int(p == n_parts - 1)] * n, q, outs[p], lses[p], s.scale)
        out = torch.zeros((rows, s.n_q_heads, s.head_dim), dtype=torch.int16, device="cuda")
        lse = torch.full((rows, s.n_q_heads), float("nan"), dtype=torch.float32, device="cuda")
        ctx.merge_partials(outs, lses, out, lse)
        ctx.sync_check()
        # every part by itself: an older part shows all its keys to every query token (= one decode per token)
        row0 = 0
        for r, b in zip(batch.requests, bounds):
            for p in range(n_parts):
                k, v = r.k[b[p]:b[p + 1]], r.v[b[p]:b[p + 1]]
                if p == n_parts - 1:
                    ref_o, ref_l = oracle.attention(r.q, k, v, s.scale)
                else:
                    per_tok = [oracle.attention(r.q[t:t + 1], k, v, s.scale) for t in range(r.q_len)]
                    ref_o = np.concatenate([o for o, _ in per_tok]); ref_l = np.concatenate([l for _, l in per_tok])
                got_o = outs[p, row0:row0 + r.q_len].cpu().numpy().astype(np.float64)
                got_l = lses[p, row0:row0 + r.q_len].cpu().numpy().astype(np.float64)
                assert np.abs(got_l - ref_l).max() <= 1e-3
                assert np.abs(got_o - ref_o).max() <= 1e-2
            row0 += r.q_len
        return gh.host_bits(out), lse.cpu().numpy(), outs, lses, ctx_stats(ctx)


def ctx_stats(ctx):
    return ctx.get_stats().kernel_launches


@pytest.mark.parametrize("hq,hkv,d,n_parts", [(32, 8, 128, 2), (28, 4, 128, 3), (8, 2, 64, 2), (40, 8, 128, 4)])
def test_split_sequences_match_the_oracle(binding, hq, hkv, d, n_parts):
    import gpu_harness as gh

    lens = [4000, 777, 130, 64 + n_parts, 2049, 9000]
    qls = [4, 1, 2, 3, 4, 1] if hq // hkv * 4 <= 16 else [2, 1, 2, 1, 2, 1]
    batch = wl.custom_batch(500 + hq + n_parts, hq, hkv, d, lens, qls)
    out, lse, _, _, _ = run_split(binding, batch, n_parts, seed=hq * 10 + n_parts)
    gh.assert_parity(out, lse, *gh.oracle_batch(batch))


def test_a_part_without_visible_keys_is_ignored(binding):
    """lse = -inf marks a part that saw nothing: its values, whatever they are, must not reach the result."""
    import gpu_harness as gh

    batch = wl.custom_batch(611, 8, 2, 64, [300, 50], [1, 1])
    out, lse, outs, lses, _ = run_split(binding, batch, 2, seed=3)
    s = batch.shape
    with binding.Context(s.n_q_heads, s.n_kv_heads, s.head_dim, 2, 256, 8 << 20) as ctx:
        junk_o = torch.full_like(outs[:1], float("nan"))
        junk_l = torch.full_like(lses[:1], float("-inf"))
        out2 = torch.zeros((outs.shape[1], s.n_q_heads, s.head_dim), dtype=torch.int16, device="cuda")
        lse2 = torch.zeros_like(lses[0])
        ctx.merge_partials(torch.cat([outs[:1], junk_o, outs[1:]]), torch.cat([lses[:1], junk_l, lses[1:]]), out2, lse2)
        ctx.sync_check()
        assert np.array_equal(gh.host_bits(out2), out) and np.array_equal(lse2.cpu().numpy(), lse)
        # all parts empty: zeros and -inf
        ctx.merge_partials(junk_o, junk_l, out2, lse2)
        ctx.sync_check()
        assert not gh.host_bits(out2).any() and np.isneginf(lse2.cpu().numpy()).all()


def test_split_attention_helper_single_rank_nccl(binding):
    """The helper that ranks call (partial attention, all-gather, merge) on a one-rank NCCL group."""
    import torch.distributed as dist

    import gpu_harness as gh
    from paper_2510_14686_b200 import seqsplit

    batch = wl.custom_batch(612, 32, 8, 128, [1500, 90], [4, 2])
    s = batch.shape
    port = 29600 + os.getpid() % 1000
    dist.init_process_group("nccl", init_method=f"tcp://127.0.0.1:{port}", rank=0, world_size=1,
                            device_id=torch.device("cuda", 0))
    try:
        lens = [r.kv_len for r in batch.requests]
        with gh.make_ctx(binding, s, len(lens), max(lens) + 8, lens) as ctx:
            slots = gh.load_requests(ctx, batch.requests)
            q = gh.dev_bits(np.concatenate([r.q for r in batch.requests], axis=0))
            out = torch.zeros_like(q)
            lse = torch.zeros(q.shape[:2], dtype=torch.float32, device="cuda")
            seqsplit.split_attention(ctx, slots, batch.q_lens, q, out, lse, s.scale)
            ctx.sync_check()
            gh.assert_parity(gh.host_bits(out), lse.cpu().numpy(), *gh.oracle_batch(batch))
    finally:
        dist.destroy_process_group()


def test_argument_checks(binding):
    import gpu_harness as gh

    batch = wl.custom_batch(613, 8, 2, 64, [40], [4])
    s = batch.shape
    with gh.make_ctx(binding, s, 2, 256, [40, 40]) as ctx:
        slots = gh.load_requests(ctx, batch.requests)
        q = gh.dev_bits(batch.requests[0].q)
        o = torch.zeros((4, 8, 64), dtype=torch.float32, device="cuda")
        l = torch.zeros((4, 8), dtype=torch.float32, device="cuda")
        with pytest.raises(binding.XllmError):
            ctx.partial_attention(slots, [4], [1], q, o, None, s.scale)          # lse_part is required
        ctx.kv_set_len(slots[0], 3)
        with pytest.raises(binding.XllmError):
            ctx.partial_attention(slots, [4], [1], q, o, l, s.scale)             # a tail part must hold its query tokens
        ctx.partial_attention(slots, [4], [0], q, o, l, s.scale)                 # an older part of 3 tokens is fine
        ctx.sync_check()
        with pytest.raises(binding.XllmError):
            ctx.merge_partials(o[None][:0], l[None][:0], torch.zeros((4, 8, 64), dtype=torch.int16, device="cuda"))
