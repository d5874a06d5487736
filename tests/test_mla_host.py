"""Host logic of the MLA mode without a GPU: the mapper's token/page arithmetic for 1152-byte rows whose 72 KiB tile
blocks do not divide the page size, and refusal of kernel-launching calls on a host-only context."""
import numpy as np
import pytest

from paper_2510_14686_b200 import binding

D = binding.MLA_LATENT + binding.MLA_ROPE
PAGE = 2 << 20
BLOCK = 64 * D * 2          # 73,728 bytes per 64 tokens


def host_ctx(**kw):
    return binding.Context(128, 1, D, 4, 100000, 64 * PAGE, flags=binding.FLAG_MLA | binding.FLAG_HOST_ONLY, **kw)


def test_pages_needed_round_up_and_capacity_rounds_down():
    with host_ctx() as ctx:
        s = ctx.kv_reserve()
        info = ctx.kv_slot_info(s)
        assert info.row_bytes == D * 2
        for tokens in (1, 64, 1820, 1821, 5000, 40000):
            ctx.kv_map_pages(s, tokens)
            info = ctx.kv_slot_info(s)
            blocks = -(-tokens // 64)
            pages = -(-blocks * BLOCK // PAGE)                       # whole tile blocks, rounded up to pages
            assert info.pages_owned == pages
            assert info.mapped_tokens == (pages * PAGE // BLOCK) * 64   # blocks that fit entirely
            assert info.mapped_tokens >= tokens


def test_geometry_is_checked():
    for heads, kvh, d in ((100, 1, D), (128, 2, D), (128, 1, 512)):
        with pytest.raises(binding.XllmError) as e:
            binding.Context(heads, kvh, d, 1, 1000, 4 * PAGE, flags=binding.FLAG_MLA | binding.FLAG_HOST_ONLY)
        assert e.value.status == binding.ERR_UNSUPPORTED
    with pytest.raises(binding.XllmError):      # 576 without the flag is not a K/V head size
        binding.Context(128, 1, D, 1, 1000, 4 * PAGE, flags=binding.FLAG_HOST_ONLY)


def test_host_only_context_refuses_the_mla_kernels():
    z = np.zeros(16, dtype=np.int16)
    with host_ctx() as ctx:
        s = ctx.kv_reserve()
        ctx.kv_map_pages(s, 10)
        for call in (lambda: ctx.mla_append([s], [1], z.ctypes.data, stream=0),
                     lambda: ctx.mla_gather(s, 0, 1, z.ctypes.data, stream=0),
                     lambda: ctx.mla_attention([s], z.ctypes.data, z.ctypes.data, stream=0)):
            with pytest.raises(binding.XllmError) as e:
                call()
            assert e.value.status == binding.ERR_UNSUPPORTED
