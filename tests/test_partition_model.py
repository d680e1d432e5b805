"""Model of the GEMV kernels' work split, checked exhaustively on the CPU.

The kernels cut the (K slice, strip, block) space into equal contiguous ranges, one per CTA, and complete a
strip that several CTAs share by "last arriver adds the partial rows in a fixed order".  The device code
derives, per strip, how many pieces exist and which workspace slot each piece uses; this test restates those
rules and checks, for many shapes and grid sizes, that every block is owned by exactly one CTA, that the
reader's list of (slot) equals the set of slots the writers use, and that no two live pieces share a slot."""
import itertools

import pytest


def range_begin(ci, G, T):
    return (ci * T) // G


def cta_of(L, G, T):
    return ((L + 1) * G - 1) // T


def slice_len(nb, nbz, z):
    return min(nbz, nb - z * nbz)


def writer_pieces(S, nb, Z, nbz, Gz):
    """What each CTA does: list of (z, ci, strip, first block, last block + 1, slot or 'direct')."""
    out = []
    for z in range(Z):
        ln = slice_len(nb, nbz, z)
        T = S * ln
        for ci in range(Gz):
            a, e = range_begin(ci, Gz, T), range_begin(ci + 1, Gz, T)
            pa = a
            while pa < e:
                s = pa // ln
                u0, u1 = s * ln, (s + 1) * ln
                pe = min(u1, e)
                whole = pa == u0 and pe == u1
                if whole and Z == 1:
                    slot = "direct"
                elif whole:
                    slot = ("full", z, s)
                else:
                    slot = ("edge", z * Gz + ci, 0 if a >= u0 else 1)
                out.append((z, ci, s, pa - u0, pe - u0, slot))
                pa = pe
    return out


def reader_slots(S, nb, Z, nbz, Gz, s):
    """What the last arriver of strip s reads, in order."""
    slots = []
    for z in range(Z):
        ln = slice_len(nb, nbz, z)
        T = S * ln
        u0 = s * ln
        cf, cl = cta_of(u0, Gz, T), cta_of(u0 + ln - 1, Gz, T)
        for c in range(cf, cl + 1):
            if cf == cl:
                slots.append(("full", z, s))
            else:
                slots.append(("edge", z * Gz + c, 0 if range_begin(c, Gz, T) >= u0 else 1))
    return slots


SHAPES = [(1, 1), (1, 5), (3, 1), (7, 10), (32, 10), (65, 17), (168, 84), (216, 5), (13, 3), (2, 40)]


@pytest.mark.parametrize("S,nb", SHAPES)
def test_every_block_once_and_reader_matches_writers(S, nb):
    for Z, grid in itertools.product((1, 2, 4), (1, 2, 3, 7, 16, 37, 148, 296)):
        Z = min(Z, nb)
        nbz = -(-nb // Z)
        Z = -(-nb // nbz)
        grid = min(grid, S * nb)
        Gz = max(1, grid // Z)
        pieces = writer_pieces(S, nb, Z, nbz, Gz)
        owned = {}
        for z, ci, s, b0, b1, slot in pieces:
            for b in range(b0, b1):
                key = (s, z * nbz + b)
                assert key not in owned
                owned[key] = (z, ci)
        assert len(owned) == S * nb
        for s in range(S):
            mine = [p for p in pieces if p[2] == s]
            direct = [p for p in mine if p[5] == "direct"]
            if direct:
                assert len(mine) == 1 and Z == 1
                assert len(reader_slots(S, nb, Z, nbz, Gz, s)) == 1
                continue
            want = reader_slots(S, nb, Z, nbz, Gz, s)
            got = sorted((p[0], p[1], p[5]) for p in mine)
            assert [g[2] for g in got] == want, (S, nb, Z, Gz, s)
            assert len(set(want)) == len(want)
        # a slot is never shared by two strips' live pieces
        edge = [p[5] for p in pieces if p[5] != "direct"]
        assert len(edge) == len(set(edge))
