"""Host-side model of how the list kernel deals the units of a list out to its CTAs (no GPU needed).

The kernel cuts the unit stream of every phase (a run of entries that do not wait for each other) into one contiguous
slice per CTA.  A row tile whose units lie in several CTAs is finished by the CTA that holds its last unit: the others
publish their partial sums into slot (CTA, first-or-last tile of its slice, entry % 4), and the finishing CTA works out
from the slice arithmetic alone which CTAs and which slots those are.  This model restates both sides of that
arithmetic as the kernel has it and checks, on the benchmark's lists and on random ones, that every row tile of
every entry is written exactly once, that every published part is collected by exactly one CTA from the slot it was
published to, and that the collected parts add up to the whole tile.
"""
import random

C = 148
def slice_of(q, rem, c):
    u0 = c*q + min(c, rem); return u0, u0 + q + (1 if c < rem else 0)
def deal(entries, merged):
    # entries: list of (N, K, dep)
    n = len(entries); out = [None]*n; i = 0
    while i < n:
        j = i+1
        while merged and j < n and not entries[j][2]: j += 1
        units = [((N+127)//128)*(K//128) for (N,K,_) in entries[i:j]]
        tot = sum(units); q, rem = tot//C, tot % C; base = 0
        for k in range(i, j):
            out[k] = (q, rem, base, units[k-i]); base += units[k-i]
        i = j
    return out
def check(entries, merged):
    info = deal(entries, merged)
    for ei, ((N,K,_), (q,rem,base,units)) in enumerate(zip(entries, info)):
        KB = K//128; RT = (N+127)//128
        written = {}   # tile -> cta
        published = {} # (cta, which) -> tile
        plans = {}
        for c in range(C):
            ph0, ph1 = slice_of(q, rem, c)
            lo, hi = max(ph0, base), min(ph1, base+units)
            if hi <= lo: continue
            u0, u1 = lo-base, hi-base
            t_first = u0//KB; t_last = (u1-1)//KB
            plans[c] = (u0,u1,t_first,t_last)
            # epilogue: full tiles
            for t in range(t_first, t_last+1):
                if u0 <= t*KB and (t+1)*KB <= u1:
                    assert t not in written; written[t] = c
            have_last = (t_last+1)*KB > u1
            have_first = t_first*KB < u0 and (t_first+1)*KB <= u1
            if have_last:
                which = 0 if t_last == t_first else 1
                published[(c, which)] = t_last
            if have_first:
                assert t_first not in written; written[t_first] = ('fix', c)
        # completer side
        for c, (u0,u1,t_first,t_last) in plans.items():
            have_first = t_first*KB < u0 and (t_first+1)*KB <= u1
            if not have_first: continue
            tile0 = base + t_first*KB
            c_lo = c
            while c_lo > 0:
                a0, a1 = slice_of(q, rem, c_lo-1)
                if a1 <= tile0: break
                c_lo -= 1
            got_units = 0
            for cc in range(c_lo, c):
                cu0, cu1 = slice_of(q, rem, cc)
                if cu0 == cu1: continue
                which = 0 if max(cu0, base) >= tile0 else 1
                assert published.get((cc, which)) == t_first, (ei, c, cc, which, published.get((cc,which)), t_first)
                pu0, pu1, _, _ = plans[cc]
                got_units += pu1 - max(pu0, t_first*KB)
                del published[(cc, which)]
            assert got_units + (min(u1,(t_first+1)*KB) - u0) == KB, (ei, c)
        assert not published, published
        assert sorted(written) == list(range(RT)), (ei, len(written), RT)


LAYER = [(4096, 4096), (4096, 4096), (4096, 4096), (4096, 4096), (11008, 4096), (11008, 4096), (4096, 11008)]


def test_llama_lists_in_every_dependency_mode():
    for deps in ("none", "layer", "all"):
        ent = []
        for _ in range(32):
            for j, (N, K) in enumerate(LAYER):
                d = (deps == "all") or (deps == "layer" and j in (0, 3, 4, 6))
                ent.append((N, K, d and len(ent) > 0))
        for merged in (True, False):
            check(ent, merged)


def test_random_lists():
    rnd = random.Random(1)
    for _ in range(200):
        ent = [(rnd.choice([1, 37, 128, 129, 200, 1000, 4096, 11008, 37008]), 128 * rnd.choice([1, 2, 3, 8, 17, 32, 86]),
                rnd.random() < 0.3) for _ in range(rnd.randint(1, 12))]
        check(ent, True)
        check(ent, False)
