"""The seeded generators reproduce the length statistics fixed for the five named workloads."""
import numpy as np

from paper_2510_14686_b200 import workloads as wl


def test_realised_lengths():
    kv, ql = wl.draw_lengths("tiny")
    assert kv.tolist() == [273, 190, 249, 21] and ql.tolist() == [1, 1, 1, 1]
    kv, _ = wl.draw_lengths("decode")
    assert (kv.min(), int(np.median(kv)), kv.max(), kv.sum()) == (522, 1931, 4060, 141622)
    kv, ql = wl.draw_lengths("verify")
    assert (kv.min(), kv.max(), kv.sum()) == (371, 9531, 303086) and (ql == 4).all()
    kv, _ = wl.draw_lengths("longctx")
    assert kv.tolist() == [104240, 32854, 44531, 45562, 51809, 46381, 107395, 70188]
    kv, ql = wl.draw_lengths("paged")
    assert (kv.min(), int(np.median(kv)), kv.max(), kv.sum()) == (64, 112, 9706, 78404)
    assert int((ql == 4).sum()) == 71 and int((kv > 4096).sum()) == 3


def test_bytes_accounting():
    b = wl.make_batch("decode", with_values=False)
    assert b.shape.row_bytes == 2048 and b.kv_bytes() == 141622 * 2048
    assert b.algorithmic_bytes() == b.kv_bytes() + 2 * 64 * 28 * 128 * 2
    assert wl.SHAPES["verify"].row_bytes == 4096 and wl.SHAPES["tiny"].row_bytes == 512


def test_values_are_seeded_bf16_normal():
    a, b = wl.make_batch("tiny"), wl.make_batch("tiny")
    for x, y in zip(a.requests, b.requests):
        assert np.array_equal(x.k, y.k) and np.array_equal(x.q, y.q) and np.array_equal(x.v, y.v)
        assert x.q.shape == (1, 8, 64) and x.k.shape == (x.kv_len, 2, 64) and x.k.dtype == np.uint16
    v = wl.bits_to_f64(np.concatenate([r.v.ravel() for r in a.requests]))
    assert abs(v.mean()) < 0.02 and abs(v.std() - 1.0) < 0.02
    # bf16 bits widen exactly: low 16 bits of the fp32 pattern are zero
    assert np.all((v.astype(np.float32).view(np.uint32) & 0xFFFF) == 0)


def test_paged_scenario_script_is_deterministic_and_consistent():
    def run():
        sc = wl.PagedScenario(n_requests=24, steps=4, max_len=700)
        log = []
        for p in sc.plans():
            assert len(p.q) == 24 and all(p.q[r].shape[0] == p.q_lens[r] for r in range(24))
            assert all(0 <= p.accepted[r] <= 3 and (p.q_lens[r] == 4 or p.accepted[r] == 0) for r in range(24))
            assert p.finished == [r for r in range(24) if (r + p.t) % 10 == 0]
            for r in p.finished:
                a = p.admitted[r]
                assert a.k.shape[0] == a.kv_len - a.q_len and p.release_mode[r] in (0, 1)
            log.append((p.q_lens.tolist(), p.accepted.tolist(), [int(p.new_k[r][0, 0, 0]) for r in range(24)]))
        return log, [sc.cached_len(r) for r in range(24)]
    a, b = run(), run()
    assert a == b
