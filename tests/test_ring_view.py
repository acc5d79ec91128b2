"""Geometry of the Local workspace variant (sink pages + a ring of recent pages per request): CPU only."""
from paper_2609_20734_b200 import ring_view


def test_ring_table_is_periodic_and_collision_free():
    geo = ring_view.geometry(3, [2048], [4])
    assert (geo.n_sink_pages, geo.ring_pages, geo.pages_per_request) == (1, 129, 130)
    assert geo.pages_per_request * 16 >= 4 + 2047 + 1      # the paper's 4 slots + 2,047-entry ring + the current token
    tab = ring_view.table(geo, 3, 5000)
    for t in (1, 17, 2052, 2053, 40000, 79999):
        pages = ring_view.live_pages(geo, t, 2048, 4)
        blocks = [tab[1, p] for p in pages]
        assert len(set(blocks)) == len(pages)               # the live pages of one request never share a ring page
        assert all(geo.pages_per_request <= blk < 2 * geo.pages_per_request for blk in blocks)


def test_ring_covers_every_window_for_ragged_sizes():
    for w, s in ((1, 0), (15, 3), (16, 16), (17, 33), (100, 4), (1024, 4)):
        geo = ring_view.geometry(2, [w], [s])
        tab = ring_view.table(geo, 2, 400)
        for t in list(range(1, 3 * (w + s) + 40)) + [6000]:
            pages = ring_view.live_pages(geo, t, w, s)
            assert len({int(tab[0, p]) for p in pages}) == len(pages), (w, s, t)
