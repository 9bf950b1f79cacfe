"""The work schedule of the weight-streaming GEMM, checked on the host (no GPU: the library exports the
same function the kernel runs).  The hand-over of partial sums between CTAs relies on these facts:

  * every (tile, k-block) unit is computed exactly once, and the CTAs' loads differ by at most one unit
    within the streamed part;
  * the CTAs that share a tile are consecutive, number 0 holds the tile's first k-blocks, and the
    pieces of a tile are in k order;
  * every contributor but the first keeps its part in slot 0 (the finisher reads slot 0 of CTAs
    c+1, c+2, ...), and a CTA writes each of its slots at most once per GEMM;
  * a CTA finishes a shared tile only with its LAST streamed piece, and whatever it waits for is some
    other CTA's FIRST piece: nobody waits for a CTA that is itself waiting;
  * with at least as many tiles as CTAs the GEMM ends on whole tiles.
"""
import ctypes

import numpy as np
import pytest

import paper_2311_13581_b200 as pb
from paper_2311_13581_b200.build import build_library


def pieces(lib, n_tiles, kb, G, cta):
    out = (ctypes.c_int32 * 7)()
    res = []
    it = 0
    while True:
        rc = lib.pass_debug_schedule(n_tiles, kb, G, cta, it, out)
        assert rc in (0, 1)
        if rc == 0:
            return res
        res.append(dict(zip(("tile", "kb0", "kb1", "n_pieces", "index", "slot", "first_slot"), list(out))))
        it += 1
        assert it < 10000


SHAPES = [
    (32, 64, 148), (32, 172, 148), (96, 64, 148), (172, 64, 148), (250, 64, 148),   # 7B: O, down, QKV, gate|up, head
    (40, 80, 148), (120, 80, 148), (216, 80, 148), (250, 80, 148),                  # 13B
    (2, 4, 148), (1, 1, 148), (3, 5, 7), (7, 3, 7), (8, 3, 7), (15, 2, 7), (148, 1, 148), (149, 3, 148),
    (296, 2, 148), (300, 7, 132), (5, 1000, 148),
]


@pytest.mark.parametrize("n_tiles,kb,G", SHAPES)
def test_schedule_invariants(n_tiles, kb, G):
    build_library()
    lib = pb.load_library()
    cover = np.zeros((n_tiles, kb), dtype=np.int32)
    by_tile = {}
    per_cta = []
    for c in range(G):
        ps = pieces(lib, n_tiles, kb, G, c)
        per_cta.append(ps)
        slots_written = []
        shared = [p for p in ps if p["n_pieces"] > 1]
        for j, p in enumerate(ps):
            assert 0 <= p["tile"] < n_tiles and 0 <= p["kb0"] < p["kb1"] <= kb
            cover[p["tile"], p["kb0"]:p["kb1"]] += 1
            by_tile.setdefault(p["tile"], []).append((c, p))
            if p["n_pieces"] == 1:
                assert (p["kb0"], p["kb1"], p["index"]) == (0, kb, 0)
            elif p["index"] != 0:
                slots_written.append(p["slot"])
                assert p["slot"] == 0                       # the finisher reads slot 0 of its peers
                assert p is shared[0]                       # ... and that piece is the CTA's first shared one
            else:
                assert p is shared[-1]                      # a CTA finishes a tile only with its last shared piece
        assert len(slots_written) == len(set(slots_written)) <= 1
        # shared pieces come before whole tiles (the GEMM ends on whole tiles when it can)
        kinds = [p["n_pieces"] > 1 for p in ps]
        assert kinds == sorted(kinds, reverse=True)
    assert (cover == 1).all()
    for tile, lst in by_tile.items():
        ctas = [c for c, _ in lst]
        n = lst[0][1]["n_pieces"]
        assert len(lst) == n and ctas == list(range(ctas[0], ctas[0] + n))
        assert [p["index"] for _, p in lst] == list(range(n))
        assert lst[0][1]["kb0"] == 0 and lst[-1][1]["kb1"] == kb
        for (_, a), (_, b) in zip(lst, lst[1:]):
            assert a["kb1"] == b["kb0"]
        assert all(p["first_slot"] == lst[0][1]["slot"] for _, p in lst)
    work = [sum(p["kb1"] - p["kb0"] for p in ps) for ps in per_cta]
    if n_tiles >= G:
        rounds = n_tiles // G
        streamed = [w - rounds * kb for w in work]
        assert max(streamed) - min(streamed) <= 1
        assert all(ps[-1]["n_pieces"] == 1 for ps in per_cta)          # ends on a whole tile
    else:
        busy = [w for w in work if w]
        assert max(busy) - min(busy) <= 1


def test_schedule_rejects_bad_arguments():
    build_library()
    lib = pb.load_library()
    out = (ctypes.c_int32 * 7)()
    assert lib.pass_debug_schedule(0, 4, 8, 0, 0, out) == -1
    assert lib.pass_debug_schedule(4, 4, 8, 8, 0, out) == -1
    assert lib.pass_debug_schedule(4, 4, 8, 0, 0, None) == -1
