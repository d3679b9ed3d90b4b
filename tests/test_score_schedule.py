"""Liveness of the two-pass score kernel's static schedule, checked on the CPU.

The persistent kernel deals chunks of tiles round-robin to its CTAs; inside a CTA two consumer
groups take the tiles of both passes in a fixed interleaved order, and a pass-2 chunk may only
start once every pass-1 chunk of its head (owned by other CTAs) has been published.  Whether that
order can always run to the end depends on how far pass 1 leads pass 2 (`lead_tiles`).  This file
restates the schedule (chunk enumeration, balanced chunk lengths, the lead formula, the order
rule) and runs it as a set of sequential actors with monotone dependencies; because conditions
only ever become true, "some actor can always move until all are done" does not depend on timing.
A schedule that stalls here would end in the kernel as an expired bounded wait.
"""
import math
import random

import pytest

KTILE = 128


def ceil_div(a, b):
    return -(-a // b)


class Schedule:
    def __init__(self, seq_lens, n_layers, units, window, pool_radius, chunk_tiles, grid, lead_extra=None):
        self.seq, self.L, self.units, self.R, self.grid = list(seq_lens), n_layers, units, chunk_tiles, grid
        self.out_keys = KTILE - 2 * pool_radius
        self.tiles = {1: [ceil_div(n, KTILE) for n in self.seq],
                      2: [ceil_div(max(n - window, 0), self.out_keys) for n in self.seq]}
        self.cph = {p: [ceil_div(t, self.R) for t in self.tiles[p]] for p in (1, 2)}
        self.pref = {}
        for p in (1, 2):
            acc, pre = 0, [0]
            for c in self.cph[p]:
                acc += c
                pre.append(acc)
            self.pref[p] = pre
        self.S = {p: units * self.pref[p][-1] for p in (1, 2)}
        self.total = {p: n_layers * self.S[p] for p in (1, 2)}
        # the lead, as the kernel's prologue computes it
        rho = self.S[2] / self.S[1] if self.S[1] > 0 else 1.0
        drift = longest = 0.0
        for b in range(len(self.seq)):
            c1, c2 = self.cph[1][b], self.cph[2][b]
            at = abs(units * (self.pref[1][b] * rho - self.pref[2][b]))
            drift = max(drift, at + units * abs(c1 * rho - c2))
            longest = max(longest, c1)
        extra = (self.R + 1) // 2 if lead_extra is None else lead_extra
        self.lead = math.ceil(self.R * rho * (1.0 + (longest + drift) / grid)) + extra

    def chunk(self, c, p):
        layer, r = divmod(c, self.S[p])
        pre = self.pref[p]
        b = next(i for i in range(len(self.seq)) if self.units * pre[i] <= r < self.units * pre[i + 1])
        cph = self.cph[p][b]
        unit, index = divmod(r - self.units * pre[b], cph)
        head = (layer * len(self.seq) + b) * self.units + unit
        tiles = self.tiles[p][b]
        tile0 = index * tiles // cph
        return head, b, (index + 1) * tiles // cph - tile0

    def group_events(self, cta, grp):
        """Static order of one consumer group: ('t', pass, n) tiles and ('end', pass, j) chunk ends."""
        S1, S2, R = self.S[1], self.S[2], self.R
        ord_ = {1: grp * S2, 2: self.lead * S1 + grp * S1}
        step = {1: S2, 2: S1}
        c = {1: cta, 2: cta}
        t = {1: grp, 2: grp}
        n = {1: grp, 2: grp}
        j = {1: 0, 2: 0}
        nt = {}
        for p in (1, 2):
            nt[p] = self.chunk(c[p], p)[2] if c[p] < self.total[p] else None
        out = []
        while True:
            for p in (1, 2):
                while nt[p] is not None and t[p] >= nt[p]:
                    out.append(("end", p, j[p]))
                    ord_[p] += (R - nt[p]) * step[p]
                    t[p] -= nt[p]
                    j[p] += 1
                    c[p] += self.grid
                    nt[p] = self.chunk(c[p], p)[2] if c[p] < self.total[p] else None
            if nt[1] is None and nt[2] is None:
                return out
            p = 1 if nt[1] is not None and (nt[2] is None or ord_[1] <= ord_[2]) else 2
            out.append(("t", p, n[p]))
            t[p] += 2
            n[p] += 2
            ord_[p] += 2 * step[p]


def runs_to_completion(s: Schedule):
    grid = s.grid
    chunks = {p: [[s.chunk(c, p) for c in range(cta, s.total[p], grid)] for cta in range(grid)] for p in (1, 2)}
    # tile number -> chunk ordinal, per CTA and pass
    tile_chunk = {p: [[j for j, ck in enumerate(chunks[p][cta]) for _ in range(ck[2])] for cta in range(grid)]
                  for p in (1, 2)}
    need = {}
    for cta in range(grid):
        for head, b, _ in chunks[1][cta]:
            need[head] = s.cph[1][b]
    published = {h: 0 for h in need}
    events = [[s.group_events(cta, g) for g in (0, 1)] for cta in range(grid)]
    pos = [[0, 0] for _ in range(grid)]
    issued = [{1: 0, 2: 0} for _ in range(grid)]
    done = [{1: set(), 2: set()} for _ in range(grid)]          # consumed tiles
    ends = [{1: {}, 2: {}} for _ in range(grid)]                # chunk ordinal -> groups past its end
    prepared = [0] * grid                                        # pass-2 chunks prepared, in order
    progress = True
    while progress:
        progress = False
        for cta in range(grid):
            # the pass-2 producer: next chunk once its head is complete and the slot is free
            while prepared[cta] < len(chunks[2][cta]):
                jn = prepared[cta]
                head = chunks[2][cta][jn][0]
                if published.get(head, 0) < need.get(head, 0):
                    break
                if jn >= 2 and ends[cta][2].get(jn - 2, 0) < 2:
                    break
                prepared[cta] += 1
                progress = True
            # the MMA issuers: tiles in order, buffer of group n & 1 must be free
            for p in (1, 2):
                while issued[cta][p] < len(tile_chunk[p][cta]):
                    nn = issued[cta][p]
                    if nn >= 2 and (nn - 2) not in done[cta][p]:
                        break
                    if p == 2 and tile_chunk[2][cta][nn] >= prepared[cta]:
                        break
                    issued[cta][p] += 1
                    progress = True
            for g in (0, 1):
                ev = events[cta][g]
                while pos[cta][g] < len(ev):
                    kind, p, x = ev[pos[cta][g]]
                    if kind == "t":
                        if issued[cta][p] <= x:
                            break
                        done[cta][p].add(x)
                    else:
                        ends[cta][p][x] = ends[cta][p].get(x, 0) + 1
                        if p == 1 and ends[cta][p][x] == 2:
                            published[chunks[1][cta][x][0]] += 1
                    pos[cta][g] += 1
                    progress = True
    return all(pos[cta][g] == len(events[cta][g]) for cta in range(grid) for g in (0, 1))


def test_group_orders_cover_every_tile_exactly_once():
    s = Schedule([1000, 300, 2100], n_layers=2, units=2, window=32, pool_radius=3, chunk_tiles=4, grid=5)
    for cta in range(s.grid):
        for p in (1, 2):
            tiles = sum(s.chunk(c, p)[2] for c in range(cta, s.total[p], s.grid))
            got = sorted(x for g in (0, 1) for k, pp, x in s.group_events(cta, g) if k == "t" and pp == p)
            assert got == list(range(tiles))
            for g in (0, 1):
                assert all(x % 2 == g for k, pp, x in s.group_events(cta, g) if k == "t" and pp == p)


def test_a_lead_of_zero_is_caught_by_the_model():
    """The check can fail: without any lead a CTA reaches a pass-2 tile whose head still needs one
    of the CTA's own later pass-1 chunks."""
    s = Schedule([4000], n_layers=1, units=2, window=32, pool_radius=3, chunk_tiles=4, grid=3, lead_extra=0)
    s.lead = -10 ** 6                                  # pass 2 first, always
    assert not runs_to_completion(s)


@pytest.mark.parametrize("seed", range(40))
def test_static_schedule_always_runs_to_completion(seed):
    rng = random.Random(seed)
    batch = rng.randint(1, 5)
    window = rng.choice([16, 32, 64])
    seq = [rng.randint(window, 45 * KTILE) for _ in range(batch)]
    if rng.random() < 0.3:
        seq[rng.randrange(batch)] = rng.randint(1, window)       # nothing to score for this one
    s = Schedule(seq, n_layers=rng.randint(1, 3), units=rng.choice([1, 2, 4, 8, 16]), window=window,
                 pool_radius=rng.choice([0, 2, 3]), chunk_tiles=rng.randint(1, 12),
                 grid=rng.randint(1, 24))
    assert runs_to_completion(s), (seq, s.L, s.units, s.R, s.grid, s.lead)
