"""GPU: append + attention in one call (the new rows are written by the attention launch itself)."""
import numpy as np
import pytest
import torch

from paper_2510_14686_b200 import workloads as wl

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def binding():
    from paper_2510_14686_b200 import binding as b

    return b


def run_fused(binding, batch, max_q_len=4):
    """Slots hold kv_len - q_len tokens; the fused call appends the q_len newest and attends.

    Returns (output bits, lse, extra launches): how many more kernels the fused call launched than a plain attention call
    over the same ranges -- 0 when the append rode along, 1 when it fell back to a separate append launch."""
    import gpu_harness as gh

    s = batch.shape
    lens = [r.kv_len for r in batch.requests]
    with gh.make_ctx(binding, s, len(lens), max(lens) + 8, lens, max_q_len=max_q_len) as ctx:
        slots = []
        for r in batch.requests:
            sl = ctx.kv_reserve(expected_tokens=r.kv_len)
            ctx.kv_map_pages(sl, r.kv_len)
            pre = r.kv_len - r.q_len
            if pre:
                ctx.kv_append([sl], [pre], gh.dev_bits(r.k[:pre]), gh.dev_bits(r.v[:pre]))
            slots.append(sl)
        q = gh.dev_bits(np.concatenate([r.q for r in batch.requests]))
        k_new = gh.dev_bits(np.concatenate([r.k[r.kv_len - r.q_len:] for r in batch.requests]))
        v_new = gh.dev_bits(np.concatenate([r.v[r.kv_len - r.q_len:] for r in batch.requests]))
        out = torch.zeros_like(q)
        lse = torch.full(q.shape[:2], float("nan"), dtype=torch.float32, device="cuda")
        before = ctx.get_stats()
        if (batch.q_lens == 1).all():
            ctx.append_decode_attention(slots, k_new, v_new, q, out, lse, s.scale)
        else:
            ctx.append_verify_attention(slots, batch.q_lens, k_new, v_new, q, out, lse, s.scale)
        ctx.sync_check()
        after = ctx.get_stats()
        # the ranges now hold every token, bit for bit
        for r, sl in zip(batch.requests, slots):
            assert ctx.kv_slot_info(sl).kv_len == r.kv_len
            gk = torch.zeros((r.kv_len, s.n_kv_heads, s.head_dim), dtype=torch.int16, device="cuda")
            gv = torch.zeros_like(gk)
            ctx.kv_gather(sl, 0, r.kv_len, gk, gv)
            ctx.sync_check()
            assert np.array_equal(gh.host_bits(gk), r.k) and np.array_equal(gh.host_bits(gv), r.v)
        # a plain attention call over the same ranges gives the same bits (same plan, same kernel)
        out2 = torch.zeros_like(q)
        mid = ctx.get_stats()
        if (batch.q_lens == 1).all():
            ctx.decode_attention(slots, q, out2, None, s.scale)
        else:
            ctx.verify_attention(slots, batch.q_lens, q, out2, None, s.scale)
        ctx.sync_check()
        assert torch.equal(out, out2)
        plain = ctx.get_stats().kernel_launches - mid.kernel_launches    # attention (+ combine for heavily split units)
    return gh.host_bits(out), lse.cpu().numpy(), (after.kernel_launches - before.kernel_launches) - plain


@pytest.mark.parametrize("hq,hkv,d", [(8, 2, 64), (28, 4, 128), (32, 8, 128)])
def test_fused_decode_edges(binding, hq, hkv, d):
    import gpu_harness as gh
    from test_gpu_attention import check_edge

    lens = [1, 2, 63, 64, 65, 66, 127, 128, 129, 130, 700, 3000]
    batch = wl.custom_batch(300 + hq + d, hq, hkv, d, lens)
    out, lse, launches = run_fused(binding, batch)
    assert launches == 0                                     # the append rode along with the attention launch
    check_edge(out, lse, batch)


def test_many_short_items_use_a_separate_append_launch(binding):
    from test_gpu_attention import check_edge

    rng = np.random.default_rng(5)
    lens = rng.integers(1, 200, 200).tolist()            # 200 requests x 8 KV heads = 1600 items > 8 per CTA
    batch = wl.custom_batch(414, 32, 8, 128, lens)
    out, lse, launches = run_fused(binding, batch)
    assert launches == 1                                 # same result; one append launch (the wide record holds 512 requests)
    check_edge(out, lse, batch)


def test_fused_verify_mixed_q_lens(binding):
    from test_gpu_attention import check_edge

    lens, qls = [], []
    for kv in [4, 5, 63, 64, 65, 66, 67, 68, 128, 129, 130, 131, 300, 2049, 5000]:
        for ql in (1, 2, 3, 4):
            if kv >= ql:
                lens.append(kv)
                qls.append(ql)
    batch = wl.custom_batch(411, 32, 8, 128, lens, qls)
    out, lse, launches = run_fused(binding, batch)
    assert launches == 0
    check_edge(out, lse, batch)


def test_falls_back_to_two_launches_when_rows_exceed_one_group(binding):
    from test_gpu_attention import check_edge

    batch = wl.custom_batch(412, 28, 4, 128, [100, 700, 65, 2100], [4, 3, 4, 1])   # G = 7: q_len 3, 4 need two row groups
    out, lse, launches = run_fused(binding, batch)
    assert launches == 1
    check_edge(out, lse, batch)


@pytest.mark.parametrize("name", ["decode", "verify", "longctx"])
def test_named_workload_fused(binding, name):
    """Full size, through the call the benchmark times: the step's new rows ride along with the attention launch."""
    import gpu_harness as gh

    batch = wl.make_batch(name)
    out, lse, launches = run_fused(binding, batch)
    assert launches == 0
    gh.assert_parity(out, lse, *gh.oracle_batch(batch))


def test_fused_append_with_items_from_the_shared_pool(binding):
    """Small whole units are claimed at run time; in a fused launch the claiming CTA writes their new rows itself."""
    import gpu_harness as gh

    rng = np.random.default_rng(21)
    lens, qls = [], []
    for i in range(96):
        qls.append(int(rng.integers(1, 5)))
        lens.append(int(rng.integers(300, 900)) if i % 3 == 0 else int(rng.integers(2500, 4000)))
    items, cta, _, _ = binding.plan_partition(lens, qls, 32, 8, 148)
    pool = items[cta[-1]:]
    assert len(pool) >= 32 and len(items) <= 8 * 148          # the case really has a pool and still fuses the append
    batch = wl.custom_batch(415, 32, 8, 128, lens, qls)
    out, lse, launches = run_fused(binding, batch)
    assert launches == 0
    gh.assert_parity(out, lse, *gh.oracle_batch(batch))


def test_pinned_host_buffers_as_call_tensors(binding):
    """q, k_new, v_new, out and lse_out in pinned host memory: the kernels reach them over PCIe; same bits as from HBM."""
    import gpu_harness as gh

    batch = wl.custom_batch(416, 28, 4, 128, [900, 64, 2100, 5, 130, 3000], [1] * 6)
    out_dev, lse_dev, _ = run_fused(binding, batch)
    s = batch.shape
    lens = [r.kv_len for r in batch.requests]
    with gh.make_ctx(binding, s, len(lens), max(lens) + 8, lens) as ctx:
        slots = []
        for r in batch.requests:
            sl = ctx.kv_reserve(expected_tokens=r.kv_len)
            ctx.kv_map_pages(sl, r.kv_len)
            pre = r.kv_len - r.q_len
            if pre:
                ctx.kv_append([sl], [pre], gh.dev_bits(r.k[:pre]), gh.dev_bits(r.v[:pre]))
            slots.append(sl)
        pin = lambda a: torch.from_numpy(np.ascontiguousarray(a).view(np.int16)).pin_memory()
        q = pin(np.concatenate([r.q for r in batch.requests]))
        k_new = pin(np.concatenate([r.k[r.kv_len - r.q_len:] for r in batch.requests]))
        v_new = pin(np.concatenate([r.v[r.kv_len - r.q_len:] for r in batch.requests]))
        out = torch.zeros_like(q).pin_memory()
        lse = torch.zeros(q.shape[:2], dtype=torch.float32).pin_memory()
        ctx.append_decode_attention(slots, k_new, v_new, q, out, lse, s.scale)
        ctx.sync_check()
        assert np.array_equal(out.numpy().view(np.uint16), out_dev) and np.array_equal(lse.numpy(), lse_dev)


def test_not_mapped_is_refused_before_anything_runs(binding):
    import gpu_harness as gh

    batch = wl.custom_batch(413, 8, 2, 64, [4096])
    s = batch.shape
    with gh.make_ctx(binding, s, 1, 8192, [8192]) as ctx:
        sl = ctx.kv_reserve()
        ctx.kv_map_pages(sl, 4096)                       # exactly one page of 4096 tokens at RB = 512
        r = batch.requests[0]
        ctx.kv_append([sl], [4096], gh.dev_bits(r.k), gh.dev_bits(r.v))
        q = gh.dev_bits(r.q)
        out = torch.zeros_like(q)
        with pytest.raises(binding.XllmError) as e:
            ctx.append_decode_attention([sl], gh.dev_bits(r.k[:1]), gh.dev_bits(r.v[:1]), q, out, None, s.scale)
        assert e.value.status == binding.ERR_NOT_MAPPED and ctx.kv_slot_info(sl).kv_len == 4096
