"""GPU: xTensor mapping and KV writes through the C ABI (byte-exact checks)."""
import numpy as np
import pytest
import torch

import oracle
from paper_2510_14686_b200 import workloads as wl

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def binding():
    from paper_2510_14686_b200 import binding as b

    return b


def gather(ctx, slot, t0, n, hkv, d):
    from gpu_harness import host_bits

    k = torch.zeros((n, hkv, d), dtype=torch.int16, device="cuda")
    v = torch.zeros_like(k)
    ctx.kv_gather(slot, t0, n, k, v)
    ctx.sync_check()
    return host_bits(k), host_bits(v)


@pytest.mark.parametrize("hkv,d", [(2, 64), (4, 128), (8, 128)])
def test_append_then_gather_is_bit_exact_across_page_growth(binding, hkv, d):
    from gpu_harness import dev_bits

    rng = np.random.default_rng(hkv * 1000 + d)
    row_bytes = 2 * hkv * d * 2
    tokens_per_page = (2 << 20) // row_bytes
    total = 2 * tokens_per_page + 77                     # three pages, ragged tail
    k = rng.integers(0, 1 << 16, (total, hkv, d), dtype=np.uint16)
    v = rng.integers(0, 1 << 16, (total, hkv, d), dtype=np.uint16)
    with binding.Context(hkv * 4, hkv, d, 3, total + 100, 8 * (2 << 20)) as ctx:
        s = ctx.kv_reserve()
        other = ctx.kv_reserve()
        ctx.kv_map_pages(other, 10)
        done = 0
        for n in [1, 63, 64, 1, tokens_per_page - 129 + 5, 3, 4, tokens_per_page, total]:   # grow in uneven steps
            n = min(n, total - done)
            if n == 0:
                break
            if ctx.kv_slot_info(s).mapped_tokens < done + n:      # not mapped yet: refused, nothing written
                with pytest.raises(binding.XllmError) as e:
                    ctx.kv_append([s], [n], dev_bits(k[done:done + n]), dev_bits(v[done:done + n]))
                assert e.value.status == binding.ERR_NOT_MAPPED and ctx.kv_slot_info(s).kv_len == done
            ctx.kv_map_pages(s, done + n)
            ctx.kv_append([s], [n], dev_bits(k[done:done + n]), dev_bits(v[done:done + n]))
            done += n
            assert ctx.kv_slot_info(s).kv_len == done
        assert done == total and ctx.kv_slot_info(s).pages_owned == 3
        gk, gv = gather(ctx, s, 0, total, hkv, d)
        assert np.array_equal(gk, k) and np.array_equal(gv, v)
        gk, gv = gather(ctx, s, tokens_per_page - 3, 70, hkv, d)     # a window straddling a page boundary
        assert np.array_equal(gk, k[tokens_per_page - 3:tokens_per_page + 67])
        assert np.array_equal(gv, v[tokens_per_page - 3:tokens_per_page + 67])


def test_multi_request_append_and_rollback(binding):
    from gpu_harness import dev_bits

    rng = np.random.default_rng(5)
    hkv, d = 2, 64
    with binding.Context(8, hkv, d, 4, 4096, 8 * (2 << 20)) as ctx:
        slots = [ctx.kv_reserve() for _ in range(3)]
        kept = {s: (np.zeros((0, hkv, d), np.uint16), np.zeros((0, hkv, d), np.uint16)) for s in slots}
        for rnd in range(6):
            n_new = rng.integers(0, 5, 3).astype(np.int32)
            if rnd == 0:
                n_new = np.array([100, 1, 65], np.int32)
            k = rng.integers(0, 1 << 16, (int(n_new.sum()), hkv, d), dtype=np.uint16)
            v = rng.integers(0, 1 << 16, (int(n_new.sum()), hkv, d), dtype=np.uint16)
            for s, n in zip(slots, n_new):
                ctx.kv_map_pages(s, kept[s][0].shape[0] + int(n))
            if n_new.sum():
                ctx.kv_append(slots, n_new, dev_bits(k), dev_bits(v))
            off = 0
            for s, n in zip(slots, n_new):
                kept[s] = (np.concatenate([kept[s][0], k[off:off + n]]), np.concatenate([kept[s][1], v[off:off + n]]))
                off += int(n)
            if rnd % 2 == 1:                                   # reject the last two tokens of slot 0
                keep = max(0, kept[slots[0]][0].shape[0] - 2)
                ctx.kv_set_len(slots[0], keep)
                kept[slots[0]] = (kept[slots[0]][0][:keep], kept[slots[0]][1][:keep])
        for s in slots:
            n = kept[s][0].shape[0]
            assert ctx.kv_slot_info(s).kv_len == n
            gk, gv = gather(ctx, s, 0, n, hkv, d)
            assert np.array_equal(gk, kept[s][0]) and np.array_equal(gv, kept[s][1])
        with pytest.raises(binding.XllmError) as e:
            ctx.kv_append([slots[0], slots[0]], [1, 1], dev_bits(k[:2]), dev_bits(v[:2]))
        assert e.value.status == binding.ERR_INVALID


def test_page_table_matches_real_mapping(binding):
    """Eq. 2: the byte the table locates in page p at offset o is the byte seen through the slot's range."""
    from gpu_harness import dev_bits

    rng = np.random.default_rng(9)
    hkv, d = 8, 128
    page = 2 << 20
    n = 1300                                              # 3 pages of 512 tokens
    k = rng.integers(0, 1 << 16, (n, hkv, d), dtype=np.uint16)
    v = rng.integers(0, 1 << 16, (n, hkv, d), dtype=np.uint16)
    with binding.Context(32, hkv, d, 4, 4096, 12 * page) as ctx:
        a = ctx.kv_reserve()
        ctx.kv_map_pages(a, 600)                          # a: pages 0,1
        b = ctx.kv_reserve()
        ctx.kv_map_pages(b, n)                            # b: pages 2,3,4
        ctx.kv_append([b], [n], dev_bits(k), dev_bits(v))
        info = ctx.kv_slot_info(b)
        assert info.pages_owned == 3 and ctx.get_stats().page_bytes == page
        for off in [0, 1, page - 64, page, page + 4096 * 3 + 32, 2 * page + 123 * 16, 3 * page - 64]:
            pos, pid, rem = ctx.kv_page_of(b, off)
            assert (pos, rem) == oracle.xtensor_locate(info.base + off, info.base, page)
            assert pid == 2 + pos
            through_range = ctx.debug_read_slot(b, off, 64)
            through_page = ctx.debug_read_page(pid, rem, 64)
            assert np.array_equal(through_range, through_page)
        # the slot's bytes are exactly the appended values, permuted: same multiset of 16-bit words
        raw = ctx.debug_read_slot(b, 0, -(-n // 64) * 64 * info.row_bytes).view(np.uint16)
        blocks = raw.reshape(-1, 64 * info.row_bytes // 2)[: n // 64]     # full tile blocks only
        want = np.concatenate([k[: (n // 64) * 64].reshape(-1), v[: (n // 64) * 64].reshape(-1)])
        assert np.array_equal(np.sort(blocks.reshape(-1)), np.sort(want))


def test_release_reuse_and_pressure_on_device(binding):
    from gpu_harness import dev_bits

    rng = np.random.default_rng(13)
    hkv, d = 8, 128
    with binding.Context(32, hkv, d, 4, 4096, 4 * (2 << 20)) as ctx:       # only four pages
        a = ctx.kv_reserve()
        ctx.kv_map_pages(a, 1024)
        k = rng.integers(0, 1 << 16, (1024, hkv, d), dtype=np.uint16)
        ctx.kv_append([a], [1024], dev_bits(k), dev_bits(k))
        ctx.kv_release(a, 0)                              # pages stay mapped, reusable
        st = ctx.get_stats()
        assert (st.pages_reusable, st.pages_free, st.pages_mapped) == (2, 2, 0)
        a2 = ctx.kv_reserve(expected_tokens=600)          # same slot id taken over, no driver map
        assert a2 == a
        ctx.kv_map_pages(a2, 600)
        st = ctx.get_stats()
        assert (st.pages_reused_total, st.pages_mapped_total, st.pages_mapped) == (2, 2, 2)
        k2 = rng.integers(0, 1 << 16, (600, hkv, d), dtype=np.uint16)
        ctx.kv_append([a2], [600], dev_bits(k2), dev_bits(k2))
        gk, gv = gather(ctx, a2, 0, 600, hkv, d)
        assert np.array_equal(gk, k2) and np.array_equal(gv, k2)          # only the new owner's data is visible
        b = ctx.kv_reserve()
        ctx.kv_map_pages(b, 1024)                         # takes the two free pages
        with pytest.raises(binding.XllmError) as e:
            ctx.kv_map_pages(b, 1025)                     # nothing free, nothing reusable
        assert e.value.status == binding.ERR_OOM_PHYS
        ctx.kv_release(a2, 0)
        ctx.kv_map_pages(b, 1536)                         # reclaims one page from the released slot (unmap + map)
        st = ctx.get_stats()
        assert st.pages_unmapped_total == 1 and st.pages_mapped == 3 and st.pages_reusable == 1
        k3 = rng.integers(0, 1 << 16, (1536, hkv, d), dtype=np.uint16)
        ctx.kv_append([b], [1536], dev_bits(k3), dev_bits(k3))
        gk, _ = gather(ctx, b, 0, 1536, hkv, d)
        assert np.array_equal(gk, k3)
        ctx.kv_release(b, 1)
        assert ctx.get_stats().pages_free == 3


@pytest.mark.parametrize("n_req", [1, 128, 129, 512, 513, 1100])
def test_append_of_many_requests_in_one_call_is_bit_exact(binding, n_req):
    """One append call over n_req requests with 0..3 new rows each (the descriptor record of a launch holds 128 requests,
    a wider one 512, larger calls take several launches): every slot gathers back exactly its own rows, in order."""
    from gpu_harness import dev_bits

    hkv, d = 2, 64
    rng = np.random.default_rng(n_req)
    n_new = rng.integers(0, 4, n_req).astype(np.int32)
    n_new[0] = 3
    rows = int(n_new.sum())
    k = rng.integers(0, 1 << 16, (rows, hkv, d), dtype=np.uint16)
    v = rng.integers(0, 1 << 16, (rows, hkv, d), dtype=np.uint16)
    page = 2 << 20
    with binding.Context(hkv * 4, hkv, d, n_req, 4096, n_req * page) as ctx:
        slots = [ctx.kv_reserve() for _ in range(n_req)]
        for s in slots:
            ctx.kv_map_pages(s, 8)
        before = ctx.get_stats().kernel_launches
        ctx.kv_append(slots, n_new, dev_bits(k), dev_bits(v))
        ctx.sync_check()
        launches = ctx.get_stats().kernel_launches - before
        assert launches == (1 if n_req <= 128 else -(-int((n_new > 0).sum()) // 512))
        row0 = 0
        for s, n in zip(slots, n_new):
            assert ctx.kv_slot_info(s).kv_len == n
            if n:
                gk, gv = gather(ctx, s, 0, int(n), hkv, d)
                assert np.array_equal(gk, k[row0:row0 + n]) and np.array_equal(gv, v[row0:row0 + n])
            row0 += int(n)
