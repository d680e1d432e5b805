"""Model of the chained kernel's work split (fdqp_run_chain), checked on the CPU.

Every step of a chain is cut like a single call -- K slices so that a slice's prepared activations fit shared memory,
contiguous block ranges per CTA inside a slice (or whole strips when that balances within 3 %), strips shared between
CTAs or slices finished through an arrival counter -- but the grid is the same for all steps, the counters and the
partial-row slots of different steps must not collide, and a step with a dependency must see every strip of the
previous step counted exactly once.  This test restates the host planner and the device rules and checks them on the
workload shapes."""
import pytest

from test_partition_model import cta_of, range_begin, slice_len

GRID = 148
XS_CAP = 64 << 10
PREP_ITEMS = 8 * 16 * 32


def plan_step(M, K, N, grid=GRID):
    rec = 136 if M <= 2 else 64
    cap = min(XS_CAP // (8 * rec * M), PREP_ITEMS // (8 * M * 4))
    assert cap >= 1
    S, nb = N // 32, -(-K // 256)
    Z = -(-nb // cap)
    nbz = -(-nb // Z)
    Z = -(-nb // nbz)
    len_last = nb - (Z - 1) * nbz
    Gz = max(1, min(grid // Z, S * len_last))
    aligned = S >= Gz and (-(-S // Gz)) * Gz <= 1.03 * S
    return dict(S=S, nb=nb, Z=Z, nbz=nbz, Gz=Gz, aligned=aligned)


def cta_range(p, z, ci):
    ln = slice_len(p["nb"], p["nbz"], z)
    if p["aligned"]:
        return range_begin(ci, p["Gz"], p["S"]) * ln, range_begin(ci + 1, p["Gz"], p["S"]) * ln, ln
    T = p["S"] * ln
    return range_begin(ci, p["Gz"], T), range_begin(ci + 1, p["Gz"], T), ln


def pieces_of(p):
    """(z, ci, strip, how the piece leaves the CTA) for every CTA of the grid."""
    out = []
    for cta in range(GRID):
        z, ci = cta // p["Gz"], cta % p["Gz"]
        if z >= p["Z"]:
            continue
        a, e, ln = cta_range(p, z, ci)
        assert e > a, "a CTA of a slice has no block"
        pa = a
        while pa < e:
            s = pa // ln
            u0, u1 = s * ln, (s + 1) * ln
            pe = min(u1, e)
            whole = pa == u0 and pe == u1
            if whole and p["Z"] == 1:
                how = "direct"
            elif whole:
                how = ("full", z * p["S"] + s)
            else:
                how = ("edge", (z * p["Gz"] + ci) * 2 + (0 if a >= u0 else 1))
            out.append((z, ci, s, pa - u0, pe - u0, how))
            pa = pe
    return out


def ticket_total(p, s):
    if p["aligned"]:
        return p["Z"]
    total = 0
    for z in range(p["Z"]):
        ln = slice_len(p["nb"], p["nbz"], z)
        T = p["S"] * ln
        total += cta_of(s * ln + ln - 1, p["Gz"], T) - cta_of(s * ln, p["Gz"], T) + 1
    return total


SHAPES = [(2560, 4096), (2048, 2560), (2560, 20480), (10240, 2560), (1152, 6912), (3840, 30720), (21504, 5376),
          (2560, 262144), (32, 32), (256, 64), (4352, 1056)]


@pytest.mark.parametrize("M", [1, 2, 3, 8])
@pytest.mark.parametrize("K,N", SHAPES)
def test_chain_step_split(M, K, N):
    p = plan_step(M, K, N)
    rec = 136 if M <= 2 else 64
    assert p["nbz"] * 8 * rec * M <= XS_CAP and p["nbz"] * 8 * M * 4 <= PREP_ITEMS
    assert p["Z"] * p["Gz"] <= GRID
    pieces = pieces_of(p)
    owned = set()
    for z, ci, s, b0, b1, how in pieces:
        for b in range(b0, b1):
            key = (s, z * p["nbz"] + b)
            assert key not in owned
            owned.add(key)
    assert len(owned) == p["S"] * p["nb"]
    stored = 0
    slots = [how for *_, how in pieces if how != "direct"]
    assert len(slots) == len(set(slots)), "two live pieces share a partial-row slot"
    for s in range(p["S"]):
        mine = [q for q in pieces if q[2] == s]
        if any(q[5] == "direct" for q in mine):
            assert len(mine) == 1
        else:
            assert len(mine) == ticket_total(p, s), (M, K, N, s)   # the last arriver is well defined
        stored += 1
    assert stored == p["S"]                                        # what a dependent step waits for


def test_chain_workspace_of_a_decoder_layer_fits():
    """Four steps of a Gemma3-4B layer, 16 at most per launch: counters and slots stay inside what a context allocates
    (arrival counters 16 x max_N / 32, edge slots 2 x 148 x 16, full slots 16384)."""
    for M in (1, 2, 8):
        steps = [plan_step(M, K, N) for K, N in SHAPES[:4]] * 4
        assert sum(p["S"] for p in steps) <= 16 * (262144 // 32)
        assert sum(2 * p["Z"] * p["Gz"] for p in steps) <= 2 * GRID * 16
        assert sum(p["Z"] * p["S"] for p in steps if p["Z"] > 1) <= 16384
