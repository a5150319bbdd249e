"""Model of how the persistent prefill GEMM deals its work out (no GPU needed).

The kernel numbers the (tile, step) pairs of a GEMM tile by tile, cuts that sequence into `C` equal contiguous ranges
of `units` (a unit = `unit_steps` steps) and lets CTA c take range c.  A tile that several CTAs share is completed
by the CTA that holds the tile's first unit; the others write their part to a slot of the workspace.  This file
restates that arithmetic (`range_begin`, `cta_of_unit`, the walk over segments, the slot rule, who completes a tile)
and checks, on random shapes, what the kernel relies on:
  * every step of every tile belongs to exactly one segment of exactly one CTA;
  * `cta_of_unit` is the inverse of `range_begin`;
  * a CTA's segments after its first begin at a tile boundary, so only its first and last segment can be partial;
  * each shared tile has exactly one completing CTA, and for that CTA the tile is its last segment;
  * every other CTA of the tile meets it as its FIRST segment (so it never waits for anybody before writing its
    part, which is what rules out a cycle of waits), and writes to slot 2 c, which nobody else writes;
  * in the mode where every part is written (slot 2 c for a first segment, 2 c + 1 otherwise), the reader's rule
    for finding the slot of CTA c's part of a tile names the slot that CTA wrote.
"""
import random


def range_begin(units, C, c):
    return units * c // C


def cta_of_unit(units, C, u):
    return ((u + 1) * C - 1) // units


def segments(units, C, c, unit_steps, S):
    """(tile, s0, s1, first) of CTA c, in the order the kernel walks them."""
    g, g_end = range_begin(units, C, c) * unit_steps, range_begin(units, C, c + 1) * unit_steps
    g_begin = g
    out = []
    while g < g_end:
        tile = g // S
        s0 = g - tile * S
        n = min(S - s0, g_end - g)
        out.append((tile, s0, s0 + n, g == g_begin))
        g += n
    return out


def check(tiles, S, unit_steps, C):
    assert S % unit_steps == 0
    su = S // unit_steps
    units = tiles * su
    C = max(1, min(C, units))
    # inverse
    for u in range(units):
        c = cta_of_unit(units, C, u)
        assert range_begin(units, C, c) <= u < range_begin(units, C, c + 1)
    covered = {}
    writers = {}       # slot -> (cta, tile), all-parts mode
    fix_slots = {}     # slot -> (cta, tile), completing mode
    completing = {}    # tile -> cta
    for c in range(C):
        segs = segments(units, C, c, unit_steps, S)
        for i, (tile, s0, s1, first) in enumerate(segs):
            assert first == (i == 0)
            if i > 0:
                assert s0 == 0, "later segments begin at a tile boundary"
            for st in range(s0, s1):
                assert (tile, st) not in covered
                covered[(tile, st)] = c
            whole = s0 == 0 and s1 == S
            if whole:
                continue
            assert i == 0 or i == len(segs) - 1, "only the first and the last segment can be partial"
            c_first, c_last = cta_of_unit(units, C, tile * su), cta_of_unit(units, C, tile * su + su - 1)
            assert c_first < c_last and c_first <= c <= c_last
            # all-parts mode
            slot = 2 * c + (0 if first else 1)
            assert slot not in writers
            writers[slot] = (c, tile)
            # completing mode
            if c == c_first:
                assert tile not in completing
                completing[tile] = c
                assert i == len(segs) - 1, "the completing CTA meets the tile last"
            else:
                assert first, "the other CTAs of a tile meet it first"
                assert 2 * c not in fix_slots
                fix_slots[2 * c] = (c, tile)
    assert len(covered) == tiles * S
    # the reader's slot rule
    for tile in range(tiles):
        c_first, c_last = cta_of_unit(units, C, tile * su), cta_of_unit(units, C, tile * su + su - 1)
        if c_first == c_last:
            assert tile not in completing
            continue
        assert completing[tile] == c_first
        for cc in range(c_first, c_last + 1):
            slot = 2 * cc + (0 if range_begin(units, C, cc) * unit_steps >= tile * S else 1)
            assert writers[slot] == (cc, tile)
            if cc > c_first:
                assert fix_slots[2 * cc] == (cc, tile)
        # the end-of-kernel rule that puts the tile's counter back to zero names the completing CTA's last tile
        g_end = range_begin(units, C, c_first + 1) * unit_steps
        assert (g_end - 1) // S == tile


def test_llama_shapes_at_280_tokens():
    # (feature tiles of 128, steps of 64 input features, units of 4 steps, 148 CTAs)
    for N, K in ((4096, 4096), (11008, 4096), (4096, 11008), (12288, 4096), (22016, 4096)):
        check((N + 127) // 128, K // 64, 4, 148)


def test_random_shapes():
    rnd = random.Random(7)
    for _ in range(300):
        unit_steps = rnd.choice([1, 1, 2, 4])
        S = unit_steps * rnd.randint(1, 40)
        tiles = rnd.randint(1, 60)
        C = rnd.randint(1, 148)
        check(tiles, S, unit_steps, C)


def test_whole_tiles_when_no_workspace():
    # without a workspace the unit is a whole tile: nobody shares anything
    for tiles, C in ((86, 148), (300, 148), (5, 148)):
        S = 64
        units = tiles
        Cc = min(C, units)
        for c in range(Cc):
            for (tile, s0, s1, first) in segments(units, Cc, c, S, S):
                assert s0 == 0 and s1 == S
