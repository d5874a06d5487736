"""The shared library loads without a GPU and exports every entry point the header declares."""
import ctypes
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def binding():
    from paper_2510_14686_b200 import build

    build.build()
    from paper_2510_14686_b200 import binding as b

    return b


def declared_functions():
    text = open(os.path.join(ROOT, "include", "xllm_attn.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(xllm_[a-z_0-9]+)\s*\(", text)))


def test_every_declared_symbol_is_exported(binding):
    names = declared_functions()
    assert {"xllm_kv_reserve", "xllm_kv_map_pages", "xllm_kv_append", "xllm_decode_attention",
            "xllm_verify_attention"} <= set(names)
    lib = ctypes.CDLL(binding.LIB_PATH)
    for n in names:
        assert hasattr(lib, n), f"{n} declared in the header but not exported"
    assert set(binding.EXPORTS) == set(names)


def test_struct_sizes_match_header_layout(binding):
    assert ctypes.sizeof(binding.WorkItem) == 40
    assert ctypes.sizeof(binding.Config) == 56
    assert ctypes.sizeof(binding.SlotInfo) == 48


def test_no_cpu_fallback_without_device(binding):
    import torch

    if torch.cuda.is_available():
        pytest.skip("a GPU is present")
    with pytest.raises(binding.XllmError) as e:
        binding.Context(8, 2, 64, 4, 1024, 64 << 20)
    assert e.value.status == binding.ERR_CUDA and "no CPU fallback" in str(e.value)


def test_host_only_context_refuses_gpu_work(binding):
    with binding.Context(8, 2, 64, 4, 1024, 64 << 20, flags=binding.FLAG_HOST_ONLY) as ctx:
        s = ctx.kv_reserve()
        ctx.kv_map_pages(s, 100)
        for call in (lambda: ctx.kv_append([s], [1], 16, 16, stream=0),
                     lambda: ctx.decode_attention([s], 16, 16, None, 1.0, stream=0),
                     lambda: ctx.verify_attention([s], [1], 16, 16, None, 1.0, stream=0),
                     lambda: ctx.kv_gather(s, 0, 0, 16, 16, stream=0)):
            with pytest.raises(binding.XllmError) as e:
                call()
            assert e.value.status == binding.ERR_UNSUPPORTED


def test_init_rejects_bad_geometry(binding):
    for args, code in [((8, 3, 64, 4, 1024, 64 << 20), binding.ERR_INVALID),
                       ((8, 2, 96, 4, 1024, 64 << 20), binding.ERR_UNSUPPORTED),
                       ((8, 2, 64, 0, 1024, 64 << 20), binding.ERR_INVALID),
                       ((8, 2, 64, 4, 1024, 1000), binding.ERR_INVALID)]:
        with pytest.raises(binding.XllmError) as e:
            binding.Context(*args, flags=binding.FLAG_HOST_ONLY)
        assert e.value.status == code
    with pytest.raises(binding.XllmError):
        binding.Context(8, 2, 64, 4, 1024, 64 << 20, max_q_len=9, flags=binding.FLAG_HOST_ONLY)
