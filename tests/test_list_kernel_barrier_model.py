"""Model of the barrier protocol inside one CTA of the tcgen05 list kernel (no GPU needed).

The kernel's roles hand work to each other through mbarriers whose waits can only tell neighbouring phases apart,
through monotonic read-out counters where a role may skip a use of a buffer, and never through named barriers.
This model restates, role by role, the waits and arrivals of `w4a16_tc_kernel` with its constants (ring of S
stages, 2 unpack warpgroups, groups of 3 units, 4 groups in flight in tensor memory, 2 activation buffers) and runs
them under a random scheduler on random lists of entries (units per entry from 1 upwards, so that groups end short
and warpgroups skip uses).  It asserts what the hardware punishes or what would hang:
  * no mbarrier ever receives more arrivals than its phase expects;
  * every arrival happens in the phase the arriving role believes it is in;
  * the run ends: whenever roles are left, at least one of them can proceed (no deadlock).
An earlier form of this model found the flaw that made the first kernel fail on long lists: a warpgroup that skips
a use of a slot cannot rely on barrier parity to know that the slot was read out.
"""
import random

S, NW, KG, NG, XB = 18, 2, 3, 4, 2   # ring stages, unpack warpgroups, units per group, groups in flight, activation buffers


class Bar:
    def __init__(self, count):
        self.count, self.pending, self.phase = count, count, 0

    def arrive(self, n=1):
        self.pending -= n
        assert self.pending >= 0, "more arrivals than the phase expects"
        if self.pending == 0:
            self.phase ^= 1
            self.pending = self.count

    def done(self, parity):          # mbarrier.try_wait.parity: has the phase of that parity completed?
        return self.phase != parity


def run(entries, seed):
    """entries: units this CTA owns of each entry of the list.  Returns None, or the roles that are stuck."""
    rnd = random.Random(seed)
    full = [Bar(1) for _ in range(S)]
    empty = [Bar(5) for _ in range(S)]            # 4 unpack warps + the commit of the MMAs that read the raw bytes
    afull = [Bar(4) for _ in range(KG * NG)]
    dfull = [Bar(KG) for _ in range(NG)]
    dempty = [Bar(4) for _ in range(NG)]
    xfull = [Bar(4) for _ in range(XB)]
    xempty = [Bar(4) for _ in range(XB)]
    rd = [0] * NG                                 # groups of slot group gs that have been read out

    def producer():
        idx = ph = 0
        for n in entries:
            for _ in range(n):
                yield ("empty", lambda i=idx, p=ph: empty[i].done(p ^ 1))
                full[idx].arrive()
                idx += 1
                if idx == S:
                    idx, ph = 0, ph ^ 1

    def unpack(wg):
        stage0 = ph0 = turn0 = G = 0
        for n in entries:
            j = wg - turn0 if wg >= turn0 else wg + NW - turn0
            st, sp = stage0 + j, ph0
            if st >= S:
                st, sp = st - S, sp ^ 1
            while j < n:
                g = G + j // KG
                a = (g % NG) * KG + j % KG
                yield ("read out", lambda q=g % NG, need=g // NG: rd[q] >= need)
                yield ("full", lambda i=st, p=sp: full[i].done(p))
                assert afull[a].phase == (g // NG) & 1, "unpack arrives in the wrong phase of afull"
                afull[a].arrive(4)
                empty[st].arrive(4)
                st += NW
                if st >= S:
                    st, sp = st - S, sp ^ 1
                j += NW
            G += (n + KG - 1) // KG
            turn0 = (turn0 + n) % NW
            adv = stage0 + n
            ph0 ^= (adv // S) & 1
            stage0 = adv % S

    def issuer(w):
        G = xe = stage0 = 0
        for n in entries:
            xb, xp = xe % XB, (xe // XB) & 1
            yield ("xfull", lambda b=xb, p=xp: xfull[b].done(p))
            xe += 1
            st = (stage0 + w) % S
            j = w
            while j < (n + KG - 1) // KG * KG:
                gs, gph = G % NG, (G // NG) & 1
                if j < n:
                    a = gs * KG + w
                    yield ("afull", lambda i=a, p=gph: afull[i].done(p))
                    assert dfull[gs].phase == gph, "commit arrives in the wrong phase of dfull"
                    dfull[gs].arrive()
                    empty[st].arrive()
                else:
                    yield ("read out (empty slot)", lambda q=gs, need=G // NG: rd[q] >= need)
                    assert afull[gs * KG + w].phase == gph and dfull[gs].phase == gph, "empty slot arrives in the wrong phase"
                    afull[gs * KG + w].arrive(4)
                    dfull[gs].arrive()
                j += KG
                G += 1
                st = (st + KG) % S
            stage0 = (stage0 + n) % S

    def epilogue():
        G = xe = 0
        for n in entries:
            xb, xp = xe % XB, (xe // XB) & 1
            yield ("xfull", lambda b=xb, p=xp: xfull[b].done(p))
            xe += 1
            for _ in range((n + KG - 1) // KG):
                gs = G % NG
                yield ("dfull", lambda q=gs, p=(G // NG) & 1: dfull[q].done(p))
                assert dempty[gs].phase == (G // NG) & 1, "read-out arrives in the wrong phase of dempty"
                dempty[gs].arrive(4)
                rd[gs] = G // NG + 1
                G += 1
            xempty[xb].arrive(4)

    def stager():
        xe = 0
        for _ in entries:
            xb, xp = xe % XB, (xe // XB) & 1
            yield ("xempty", lambda b=xb, p=xp ^ 1: xempty[b].done(p))
            xfull[xb].arrive(4)
            xe += 1

    agents = {"producer": producer(), "stager": stager(), "epilogue": epilogue()}
    for w in range(NW):
        agents[f"unpack{w}"] = unpack(w)
    for w in range(KG):
        agents[f"mma{w}"] = issuer(w)
    waiting = {}
    for k, g in list(agents.items()):
        try:
            waiting[k] = next(g)
        except StopIteration:
            del agents[k]
    while agents:
        ready = [k for k in agents if waiting[k][1]()]
        if not ready:
            return {k: waiting[k][0] for k in agents}
        k = rnd.choice(ready)
        try:
            waiting[k] = next(agents[k])
        except StopIteration:
            del agents[k]
            del waiting[k]
    return None


def test_llama_like_slices_under_random_schedules():
    # units a CTA owns of the seven linears of a decoder layer when every CTA takes part in every linear
    layer = [7, 7, 6, 7, 19, 18, 19]
    for seed in range(150):
        r = random.Random(seed)
        ents = []
        for _ in range(4):
            for n in layer:
                ents.append(r.choice([1, 2, 3, 5]) if r.random() < 0.3 else max(1, n + r.randint(-1, 1)))
        assert run(ents, seed) is None


def test_long_slices_and_single_units():
    # a list without dependencies gives a CTA two or three long slices; single-unit entries end every group short
    assert run([1351, 1024, 296], 1) is None
    assert run([1] * 60, 2) is None
    assert run([2, 1, 4, 3, 40, 1, 1, 7], 3) is None
