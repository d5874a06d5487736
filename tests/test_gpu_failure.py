"""GPU: the library's own failure detection.  One tile copy of one launch is never issued (a host-armed test hook);
the kernel's bounded wait for it runs out, the launch ends by itself, the host reads the error word, and the context
keeps working.  Nothing here faults, traps or waits without a limit."""
import time

import numpy as np
import pytest
import torch

from paper_2510_14686_b200 import workloads as wl

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def binding():
    from paper_2510_14686_b200 import binding as b

    return b


@pytest.mark.parametrize("lens", [[5000, 300, 64, 1], [700] * 40])
def test_wait_runs_out_and_context_recovers(binding, lens):
    import gpu_harness as gh

    shape = wl.SHAPES["tiny"]
    batch = wl.custom_batch(77, shape.n_q_heads, shape.n_kv_heads, shape.head_dim, lens)
    shape = batch.shape
    ref_o, ref_lse = gh.oracle_batch(batch)
    with gh.make_ctx(binding, shape, len(lens), max(lens) + 8, lens) as ctx:
        slots = gh.load_requests(ctx, batch.requests)
        good, lse = gh.run_attention(ctx, batch, slots)
        gh.assert_parity(good, lse, ref_o, ref_lse)

        ctx.debug_inject_timeout(1)
        q = gh.dev_bits(np.concatenate([r.q for r in batch.requests], axis=0))
        out = torch.zeros_like(q)
        t0 = time.monotonic()
        ctx.decode_attention(slots, q, out, None, shape.scale)   # the launch itself is accepted ...
        with pytest.raises(binding.XllmError) as ei:             # ... and the wait that ran out shows at the next check
            ctx.sync_check()
        took = time.monotonic() - t0
        assert ei.value.status == binding.ERR_CUDA
        assert "bounded device-side wait expired" in str(ei.value)
        assert 1.0 < took < 15.0, took                           # the 2 s limit, not a hang and not an instant failure

        ctx.sync_check()                                         # reported once; the context is clean again
        for _ in range(2):                                       # same ranges, same plan: bit-identical to before
            again, lse2 = gh.run_attention(ctx, batch, slots)
            assert np.array_equal(again, good)
            assert np.array_equal(lse2, lse)


def test_inject_argument_checks(binding):
    shape = wl.SHAPES["tiny"]
    with binding.Context(shape.n_q_heads, shape.n_kv_heads, shape.head_dim, 2, 256, 8 << 20) as ctx:
        with pytest.raises(binding.XllmError):
            ctx.debug_inject_timeout(-1)
        ctx.debug_inject_timeout(0)
