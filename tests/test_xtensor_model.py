"""The page-pool model (oracle side) obeys the state machine of the xTensor section."""
import numpy as np

from oracle import PagePoolModel
from oracle import xtensor_model as xm


def make(n_pages=8, page=2 << 20, rb=4096, tile=64, slots=4, max_len=8192):
    return PagePoolModel(n_pages, page, rb, tile, slots, max_len)


def test_pages_for_rounds_to_tile_blocks_then_pages():
    m = make()
    assert m.pages_for(0) == 0 and m.pages_for(1) == 1 and m.pages_for(512) == 1 and m.pages_for(513) == 2
    m2 = make(page=65536, rb=512, tile=64)   # a tile block is 32 KiB: two per page
    assert m2.pages_for(64) == 1 and m2.pages_for(128) == 1 and m2.pages_for(129) == 2


def test_on_demand_growth_maps_next_contiguous_page():
    m = make()
    s = m.reserve()
    assert s == 0 and m.map_pages(s, 100) == xm.OK and m.slots[s].pages == [0]
    assert m.map_pages(s, 512) == xm.OK and m.slots[s].pages == [0]          # idempotent
    assert m.map_pages(s, 1500) == xm.OK and m.slots[s].pages == [0, 1, 2]
    assert m.mapped_tokens(s) == 1536 and m.counts() == {"free": 5, "allocated": 0, "mapped": 3, "reusable": 0}
    assert m.pages_mapped_total == 3
    m.check_invariants()


def test_release_keeps_pages_reusable_and_reserve_takes_them_over():
    m = make()
    a, b = m.reserve(), m.reserve()
    m.map_pages(a, 1500), m.map_pages(b, 400)
    assert m.release(a, 0) == xm.OK
    assert m.counts() == {"free": 4, "allocated": 0, "mapped": 1, "reusable": 3}
    c = m.reserve(hint_tokens=900)            # needs 2 pages: slot a's set of 3 is the only fit
    assert c == a and m.map_pages(c, 900) == xm.OK
    assert m.pages_reused_total == 2 and m.pages_mapped_total == 4          # no new driver maps
    assert m.counts() == {"free": 4, "allocated": 0, "mapped": 3, "reusable": 1}
    assert m.map_pages(c, 2000) == xm.OK and m.pages_reused_total == 3 and m.pages_mapped_total == 5
    m.check_invariants()


def test_unmap_release_returns_pages_in_order():
    m = make()
    a = m.reserve()
    m.map_pages(a, 1500)
    assert m.release(a, 1) == xm.OK and m.counts()["free"] == 8 and m.pages_unmapped_total == 3
    b = m.reserve()
    m.map_pages(b, 1500)
    assert m.slots[b].pages == [0, 1, 2]
    m.check_invariants()


def test_pressure_reclaims_reusable_then_fails_cleanly():
    m = make(n_pages=4)
    a, b = m.reserve(), m.reserve()
    m.map_pages(a, 1024), m.map_pages(b, 1024)            # 2 + 2 pages, pool empty
    assert m.map_pages(b, 1025) == xm.ERR_OOM_PHYS and m.slots[b].n_owned == 2
    m.release(a, 0)
    assert m.map_pages(b, 1536) == xm.OK                  # reclaims one page from the tail of slot a
    assert m.slots[a].pages == [0] and m.slots[b].pages == [2, 3, 1] and m.pages_unmapped_total == 1
    assert m.map_pages(b, 4096) == xm.ERR_OOM_PHYS        # would need 8 pages; nothing changed
    assert m.slots[b].n_owned == 3 and m.counts() == {"free": 0, "allocated": 0, "mapped": 3, "reusable": 1}
    m.check_invariants()


def test_invalid_calls():
    m = make(slots=2)
    assert m.map_pages(0, 10) == xm.ERR_INVALID           # not reserved
    a, b = m.reserve(), m.reserve()
    assert m.reserve() == xm.ERR_OOM_VA
    assert m.map_pages(a, 8193) == xm.ERR_INVALID and m.release(a, 2) == xm.ERR_INVALID
    assert m.release(b, 0) == xm.OK and m.release(b, 0) == xm.ERR_INVALID


def test_random_walk_keeps_invariants():
    rng = np.random.default_rng(0)
    m = make(n_pages=16, slots=6)
    live = {}
    for _ in range(400):
        op = rng.integers(0, 3)
        if op == 0 and len(live) < 6:
            s = m.reserve(int(rng.integers(0, 3000)))
            assert s >= 0 and s not in live
            live[s] = 0
        elif op == 1 and live:
            s = int(rng.choice(list(live)))
            t = int(rng.integers(1, 4000))
            before = m.counts()
            st = m.map_pages(s, t)
            if st == xm.OK:
                assert m.mapped_tokens(s) >= t
            else:
                assert st == xm.ERR_OOM_PHYS and m.counts() == before
        elif op == 2 and live:
            s = int(rng.choice(list(live)))
            assert m.release(s, int(rng.integers(0, 2))) == xm.OK
            del live[s]
        m.check_invariants()
