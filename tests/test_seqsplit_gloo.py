"""N > 1 path of the sequence split on CPU: two gloo ranks each hold one part of every sequence, compute their partial
result (here: with the oracle), all-gather through the package's helper and merge -- the result equals attention over
the whole sequence."""
import os
import sys

import numpy as np
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _worker(rank, world, port, out):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    sys.path.insert(0, ROOT)
    import oracle
    from paper_2510_14686_b200 import seqsplit, workloads as wl

    dist.init_process_group("gloo", rank=rank, world_size=world)
    batch = wl.custom_batch(700, 8, 2, 64, [300, 41, 1000], [4, 1, 2])
    s = batch.shape
    cuts = [170, 7, 512]
    o_rows, l_rows = [], []
    for r, c in zip(batch.requests, cuts):
        k, v = (r.k[:c], r.v[:c]) if rank == 0 else (r.k[c:], r.v[c:])
        if rank == world - 1:                                  # the tail part: causal among the query tokens
            o, l = oracle.attention(r.q, k, v, s.scale)
        else:                                                  # an older part: every key visible to every query token
            parts = [oracle.attention(r.q[t:t + 1], k, v, s.scale) for t in range(r.q_len)]
            o = np.concatenate([p[0] for p in parts]); l = np.concatenate([p[1] for p in parts])
        o_rows.append(o); l_rows.append(l)
    out_part = torch.from_numpy(np.concatenate(o_rows))        # fp64 here; fp32 on the GPU path
    lse_part = torch.from_numpy(np.concatenate(l_rows))
    outs, lses = seqsplit.gather_parts(out_part, lse_part)
    assert outs.shape == (world,) + tuple(out_part.shape) and torch.equal(outs[rank], out_part)
    outs, lses = outs.numpy(), lses.numpy()
    ref_o, ref_l = oracle.attention_batch([r.q for r in batch.requests], [r.k for r in batch.requests],
                                          [r.v for r in batch.requests], s.scale)
    ref_o, ref_l = np.concatenate(ref_o), np.concatenate(ref_l)
    err = 0.0
    for row in range(outs.shape[1]):
        for h in range(s.n_q_heads):
            o, l = oracle.merge_lse(outs[:, row, h, :], lses[:, row, h])
            err = max(err, float(np.abs(o - ref_o[row, h]).max()), abs(l - ref_l[row, h]))
    dist.barrier()
    dist.destroy_process_group()
    out.put((rank, err))


def test_two_ranks_one_part_each():
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    port = 29700 + os.getpid() % 2000
    procs = [ctx.Process(target=_worker, args=(r, 2, port, q)) for r in range(2)]
    for p in procs:
        p.start()
    res = sorted(q.get(timeout=300) for _ in procs)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    assert [r for r, _ in res] == [0, 1]
    assert all(err < 1e-12 for _, err in res), res       # fp64 partials: the merge is exact up to rounding


def test_gather_without_a_process_group_is_a_stack_of_one():
    sys.path.insert(0, ROOT)
    from paper_2510_14686_b200 import seqsplit

    o, l = torch.zeros(3, 2, 4), torch.zeros(3, 2)
    outs, lses = seqsplit.gather_parts(o, l)
    assert outs.shape == (1, 3, 2, 4) and lses.shape == (1, 3, 2)
