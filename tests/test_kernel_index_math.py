"""Index arithmetic of two skeletons, replayed on the CPU: the claims their comments make about
coverage, bank conflicts and halos are small enough to check exhaustively."""
import itertools


def _tile_pair_blocks():
    """(block column, block row) of each of the 256 consumer threads of k_tile_pair_tma."""
    out = []
    for t in range(256):
        l, dg, quad = t & 7, (t >> 3) & 7, t >> 6
        out.append(((quad & 1) * 8 + l, (quad >> 1) * 8 + ((l + dg) & 7)))
    return out


def test_tile_pair_threads_cover_the_tile_once():
    assert sorted(_tile_pair_blocks()) == sorted(itertools.product(range(16), range(16)))


def test_tile_pair_reads_are_free_of_bank_conflicts():
    # a 64 x 64 tile of 4-byte words lies row by row (256 bytes per row).  A 128-bit read is served eight lanes
    # at a time; it is conflict-free when the eight 16-byte chunks fall into eight different bank groups, and the
    # bank group of a chunk is (its word offset / 4) mod 8.
    blocks = _tile_pair_blocks()
    for first in range(0, 256, 8):
        lanes = blocks[first:first + 8]
        for i in range(4):
            direct = {((4 * by + i) * 64 + 4 * bx) // 4 % 8 for bx, by in lanes}          # row 4*by+i, columns 4*bx..
            transposed = {((4 * bx + i) * 64 + 4 * by) // 4 % 8 for bx, by in lanes}      # row 4*bx+i, columns 4*by..
            assert len(direct) == 8 and len(transposed) == 8


def test_stencil_halo_covers_what_each_level_reads():
    # k_stencil, D stacked shifts: the box of an external starts D rows above and 4 columns left of a 64 x 128
    # tile.  Level k (1..D) is computed on box rows k .. BR-1-k and is exact on the columns at least k away from
    # the box edges (a value one column off the exact region of the level below is wrong).  The roots (level D)
    # need the tile itself: box rows D .. D+63, box columns 4 .. 131.
    for D in range(1, 5):
        BR, BC = 64 + 2 * D, 136
        exact = {(r, c) for r in range(BR) for c in range(BC)}            # level 0: the copied box
        for k in range(1, D + 1):
            rows = range(k, BR - k) if k < D else range(D, D + 64)
            cols = range(BC) if k < D else range(4, 132)
            computed = set()
            for r in rows:
                for c in cols:
                    if all((r + dr, c + dc) in exact for dr, dc in ((0, 0), (-1, 0), (1, 0), (0, 1), (0, -1))):
                        computed.add((r, c))
            exact = computed
            if k < D:
                # what the next level reads of this one lies inside what is exact here
                need_rows = range(k + 1, BR - k - 1) if k + 1 < D else range(D, D + 64)
                need_cols = range(4 - (D - k - 1), 132 + (D - k - 1))
                for r in need_rows:
                    for c in need_cols:
                        assert all((r + dr, c + dc) in exact for dr, dc in ((0, 0), (-1, 0), (1, 0), (0, 1), (0, -1))), (D, k, r, c)
        assert {(r, c) for r in range(D, D + 64) for c in range(4, 132)} <= exact


def test_pair_numbering_walks_the_upper_triangle():
    # pair p -> (I, J), rows of the upper triangle one after the other (the closed form of pair_of, in integers)
    for T in (1, 2, 7, 33, 128):
        first = lambda k: k * T - k * (k - 1) // 2
        seen = []
        for p in range(T * (T + 1) // 2):
            i = max(k for k in range(T) if first(k) <= p)
            seen.append((i, i + p - first(i)))
        assert seen == [(i, j) for i in range(T) for j in range(i, T)]
