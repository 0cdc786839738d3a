"""A CPU model of the barrier protocol of the expanded-operand kernel's main loop with TWO MMA issuer threads (host logic,
no GPU): a producer fills ring slots in order, each issuer waits on a slot's "full" barrier by phase parity, releases it
with a commit that lands some time later, and both hand the accumulators to the epilogue.  The model counts barrier
phases in full but lets a waiter see only the phase's parity, as the hardware does, and fails on

  * a wait that passes on a slot that does not hold the stage the waiter expects (a stale phase of the same parity),
  * more arrivals on a barrier than its phase expects,
  * a state in which nobody can move.

It pins the rule the kernel follows: the issuers own ring SLOTS (even / odd, an even number of slots), so that each sees
every use of the barriers it waits on.  Ownership by position inside the work item, which looks equivalent, lets a thread
skip a use of a slot at the seams between items and then pass a wait one phase early; the model reproduces that."""
import random

import pytest


class Bar:
    def __init__(self, name, count):
        self.name, self.count, self.pending, self.phase = name, count, count, 0

    def arrive(self, who):
        if self.pending == 0:
            raise RuntimeError(f"over-arrival on {self.name} by {who}")
        self.pending -= 1
        if self.pending == 0:
            self.phase += 1
            self.pending = self.count

    def passed(self, parity):
        return (self.phase & 1) != parity       # all a waiter can see


class Ring:
    def __init__(self):
        self.s, self.par, self.wrapped = 0, 0, False

    def adv(self, n):
        self.s += 1
        if self.s == n:
            self.s, self.par, self.wrapped = 0, self.par ^ 1, True


def simulate(pieces, n_slots, n_acc, by_slot, seed):
    rnd = random.Random(seed)
    full = [Bar(f"full{i}", 1) for i in range(n_slots)]
    free = [Bar(f"free{i}", 1) for i in range(n_slots)]
    accfull = [Bar(f"accfull{i}", 2) for i in range(2)]
    accfree = [Bar(f"accfree{i}", 1) for i in range(2)]
    holds = [None] * n_slots         # the stage whose load landed in the slot last
    commits = []                     # (issuer, barrier): tcgen05.commit arrivals still in flight, in order per issuer

    def producer():
        rp, g = Ring(), 0
        for length in pieces:
            for _ in range(length):
                if rp.wrapped:
                    while not free[rp.s].passed(rp.par ^ 1):
                        yield
                holds[rp.s] = g
                full[rp.s].arrive("producer")
                g += 1
                rp.adv(n_slots)
                yield

    def issuer(i):
        rp, g = Ring(), 0
        ab, par, wrapped = 0, 0, False
        for length in pieces:
            if wrapped:
                while not accfree[ab].passed(par ^ 1):
                    yield
            for c in range(length):
                mine = (rp.s & 1) == i if by_slot else (c & 1) == i
                if mine:
                    while not full[rp.s].passed(rp.par):
                        yield
                    if holds[rp.s] != g:
                        raise RuntimeError(f"issuer {i} passed a stale phase: slot {rp.s} holds stage {holds[rp.s]}, not {g}")
                    commits.append((i, free[rp.s]))
                g += 1
                rp.adv(n_slots)
                yield
            commits.append((i, accfull[ab]))
            if n_acc == 2:
                if ab == 1:
                    par ^= 1
                    wrapped = True
                ab ^= 1
            else:
                par ^= 1
                wrapped = True
            yield

    def epilogue():
        for t in range(len(pieces)):
            ab = t & 1 if n_acc == 2 else 0
            parity = ((t >> 1) if n_acc == 2 else t) & 1
            while not accfull[ab].passed(parity):
                yield
            yield
            accfree[ab].arrive("epilogue")

    agents = {"producer": producer(), "epilogue": epilogue(), "issuer0": issuer(0), "issuer1": issuer(1)}
    bars = full + free + accfull + accfree
    idle = 0
    while agents:
        before = tuple((b.phase, b.pending) for b in bars)
        moved = False
        for who in {a for a, _ in commits}:
            if rnd.random() < 0.5:
                k = next(j for j, (a, _) in enumerate(commits) if a == who)
                a, bar = commits.pop(k)
                bar.arrive(f"issuer{a}")
                moved = True
        names = list(agents)
        rnd.shuffle(names)
        for n in names:
            try:
                next(agents[n])
            except StopIteration:
                del agents[n]
                moved = True
        moved = moved or tuple((b.phase, b.pending) for b in bars) != before
        idle = 0 if moved or commits else idle + 1
        if idle > 200:
            raise RuntimeError(f"deadlock: {sorted(agents)} cannot move")


def _cases():
    for seed in range(250):
        r = random.Random(seed)
        yield seed, [r.choice([1, 1, 2, 3, 4, 5, 9]) for _ in range(r.randint(1, 6))]


@pytest.mark.parametrize("n_acc", [1, 2])
@pytest.mark.parametrize("n_slots", [2, 4, 6, 10])
def test_slot_ownership_is_safe(n_slots, n_acc):
    for seed, pieces in _cases():
        simulate(pieces, n_slots, n_acc, True, seed)


def test_ownership_by_position_in_the_item_is_not():
    failures = 0
    for seed, pieces in _cases():
        try:
            simulate(pieces, 2, 2, False, seed)
        except RuntimeError as e:
            assert "stale phase" in str(e) or "over-arrival" in str(e) or "deadlock" in str(e)
            failures += 1
    assert failures > 0
