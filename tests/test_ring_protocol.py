"""Host model of the GEMM kernels' ring protocol (TMA producer -> dequantiser groups -> UMMA issuer).

An mbarrier parity wait only tells two consecutive phases apart.  The kernels therefore lay the
barriers of a ring of n buffers served by d dequantiser groups over lcm(n, d) slots, so that every
barrier is always the business of the same group.  This file re-states that protocol on the host
(barriers with phase counters, actors as coroutines, TMA completions landing out of order, a random
scheduler) and checks that for every ring plan the library hands out, and for many more, every slab
reaches the UMMA issuer intact and in order, and nothing deadlocks.  It also checks that the model
has teeth: the same actors with one barrier per buffer lose data for depths that are not multiples
of the group count.
"""
import math
import random

import pytest

import paper_2511_16041_b200 as atb


class Barrier:
    """mbarrier: `count` arrivals complete the current phase."""

    def __init__(self, count):
        self.count = count
        self.pending = count
        self.phase = 0          # number of completed phases

    def arrive(self):
        self.pending -= 1
        assert self.pending >= 0
        if self.pending == 0:
            self.phase += 1
            self.pending = self.count

    def test(self, parity):
        """try_wait.parity: true when the phase of that parity is not the one in progress."""
        return (self.phase & 1) != parity


class Cursor:
    def __init__(self, buf=0, bar=0):
        self.buf, self.bar, self.phase = buf, bar, 0

    def advance(self, step, n, n_bars):
        self.buf = (self.buf + step) % n
        self.bar += step
        if self.bar >= n_bars:
            self.bar -= n_bars
            self.phase ^= 1


def lcm(a, b):
    return a * b // math.gcd(a, b)


def simulate(n_raw, n_deq, groups, run, n_slabs, seed, lcm_bars=True, group_warps=2, land_prob=0.5, newest_first=False,
             bundle=1):
    """Runs the protocol; returns the list of slab ids the issuer consumed.  `bundle` = raw slabs a
    dequantiser group converts per barrier round trip into ONE dequantised stage (thin slabs are
    bundled up to a 128-row operand group); `run` = dequantised stages the issuer takes per UMMA group.
    n_deq counts dequantised stages."""
    rng = random.Random(seed)
    raw_bars = lcm(n_raw, groups * bundle) if lcm_bars else n_raw
    deq_bars = lcm(n_deq, groups) if lcm_bars else n_deq
    raw_full = [Barrier(1) for _ in range(raw_bars)]
    raw_empty = [Barrier(group_warps) for _ in range(raw_bars)]
    deq_full = [Barrier(group_warps) for _ in range(deq_bars)]
    deq_empty = [Barrier(1) for _ in range(deq_bars)]
    raw_buf = [None] * n_raw
    deq_buf = [None] * n_deq
    in_flight = []              # TMA copies issued and not landed: (buffer, barrier, slab)
    consumed = []
    errors = []

    def producer():
        cur, freed, filled = Cursor(), Cursor(), 0
        for c in range(n_slabs):
            if filled < n_raw:
                filled += 1
            else:
                while not raw_empty[freed.bar].test(freed.phase):
                    yield
                freed.advance(1, n_raw, raw_bars)
            in_flight.append((cur.buf, cur.bar, c))
            cur.advance(1, n_raw, raw_bars)
            yield

    def dequantiser(g, w):
        rr, rd = Cursor((g * bundle) % n_raw, g * bundle), Cursor(g % n_deq, g)
        first_reuse = g
        while first_reuse < n_deq:
            first_reuse += groups
        freed = Cursor(0, first_reuse - n_deq)
        for st in range(g, n_slabs // bundle, groups):          # st = index of the bundle / dequantised stage
            for i in range(bundle):
                while not raw_full[rr.bar + i].test(rr.phase):
                    yield
            if st >= first_reuse:
                while not deq_empty[freed.bar].test(freed.phase):
                    yield
                freed.advance(groups, n_deq, deq_bars)
            got = [raw_buf[(rr.buf + i) % n_raw] for i in range(bundle)]
            if got != list(range(st * bundle, (st + 1) * bundle)):
                errors.append(("raw", st, got))
            yield                                   # the warps of a group run at their own pace
            deq_buf[rd.buf] = got
            yield
            deq_full[rd.bar].arrive()
            for i in range(bundle):
                raw_empty[rr.bar + i].arrive()
            rr.advance(groups * bundle, n_raw, raw_bars)
            rd.advance(groups, n_deq, deq_bars)
            yield

    def issuer():
        rd = Cursor()
        for c in range(0, n_slabs // bundle, run):
            for i in range(run):
                while not deq_full[rd.bar + i].test(rd.phase):
                    yield
            for i in range(run):
                consumed.extend(deq_buf[(rd.buf + i) % n_deq])
            yield                                   # the UMMAs execute
            for i in range(run):
                deq_empty[rd.bar + i].arrive()      # tcgen05.commit
            rd.advance(run, n_deq, deq_bars)
            yield

    actors = [producer(), issuer()] + [dequantiser(g, w) for g in range(groups) for w in range(group_warps)]
    live = list(actors)
    idle_rounds = 0
    while live:
        progressed = False
        # land a random copy now and then (completion order is not issue order)
        if in_flight and rng.random() < land_prob:
            buf, bar, slab = in_flight.pop(len(in_flight) - 1 if newest_first else rng.randrange(len(in_flight)))
            raw_buf[buf] = slab
            raw_full[bar].arrive()
            progressed = True
        a = rng.choice(live)
        before = (len(consumed), len(in_flight), [b.phase for b in raw_empty], [b.pending for b in deq_full],
                  [b.pending for b in raw_empty], [b.phase for b in deq_empty])
        try:
            next(a)
        except StopIteration:
            live.remove(a)
            progressed = True
        after = (len(consumed), len(in_flight), [b.phase for b in raw_empty], [b.pending for b in deq_full],
                 [b.pending for b in raw_empty], [b.phase for b in deq_empty])
        progressed |= before != after
        idle_rounds = 0 if progressed else idle_rounds + 1
        if idle_rounds > 20000:
            errors.append(("deadlock", len(consumed)))
            break
    return consumed, errors


def slab_bundle(spg, n_raw, groups):
    b = spg
    while b > 1 and n_raw % (b * groups):
        b //= 2
    return b


def all_plans():
    """(tiling, raw depth, dequantised stages, groups, stages per UMMA group, bundle) of every supported tiling."""
    for mc in (128, 256, 384):
        for tn in (64, 128, 256, 512):
            for tk in (64, 128):
                for ma in (32, 64, 128, 256):
                    if ma > mc or mc % ma or not atb.atb_tiling_supported(ma, mc, tk, tn):
                        continue
                    p = atb.atb_tiling_plan(ma, mc, tk, tn)
                    pair = (mc, tk, tn) == (256, 64, 512)
                    slab = min(ma, 128) if pair else ma
                    if slab <= 128:
                        spg = 128 // slab
                        bundle = slab_bundle(spg, p.n_raw_stages, p.dequant_groups)
                        spb = spg // bundle
                        yield (ma, mc, tk, tn), p.n_raw_stages, p.n_a_groups * spb, p.dequant_groups, spb, bundle
                    else:
                        yield (ma, mc, tk, tn), p.n_raw_stages, p.n_a_groups // (slab // 128), p.dequant_groups, 1, 1


def test_library_ring_plans_deliver_every_slab_in_order():
    seen = set()
    for tiling, n_raw, n_deq, groups, run, bundle in all_plans():
        key = (n_raw, n_deq, groups, run, bundle)
        if key in seen:
            continue
        seen.add(key)
        n_slabs = 12 * lcm(lcm(n_raw, n_deq * bundle), groups * run * bundle)
        for seed, kw in enumerate([{}, {"land_prob": 0.05}, {"land_prob": 0.03, "newest_first": True}]):
            consumed, errors = simulate(n_raw, n_deq, groups, run, n_slabs, seed, bundle=bundle, **kw)
            assert not errors, (tiling, key, errors[:3])
            assert consumed == list(range(n_slabs)), (tiling, key)
    assert len(seen) >= 4 and any(k[4] > 1 for k in seen)


@pytest.mark.parametrize("groups", [1, 2, 4])
def test_any_depth_is_safe_with_lcm_barriers(groups):
    for n_raw in range(max(1, groups), 10):
        for n_deq in range(2, 8):
            for run in (1, 2, 4):
                if n_deq % run:
                    continue
                n_slabs = 4 * lcm(lcm(n_raw, n_deq), groups * run)
                slow = {"land_prob": 0.05, "newest_first": bool(n_raw & 1)} if (n_raw + n_deq) & 1 else {}
                consumed, errors = simulate(n_raw, n_deq, groups, run, n_slabs, seed=n_raw * 100 + n_deq, **slow)
                assert not errors, (n_raw, n_deq, groups, run, errors[:3])
                assert consumed == list(range(n_slabs))


def test_bundles_of_thin_slabs_are_safe_for_any_depth():
    for groups in (2, 4):
        for bundle in (2, 4):
            for k in range(1, 4):
                n_raw = k * bundle * groups // 2 if (k * bundle * groups // 2) % bundle == 0 else k * bundle * groups
                for n_deq in (2, 3, 4, 6):
                    n_slabs = 6 * lcm(lcm(n_raw, n_deq * bundle), groups * bundle)
                    consumed, errors = simulate(n_raw, n_deq, groups, 1, n_slabs, seed=n_raw + n_deq, bundle=bundle,
                                                land_prob=0.05 if n_deq & 1 else 0.5)
                    assert not errors, (n_raw, n_deq, groups, bundle, errors[:3])
                    assert consumed == list(range(n_slabs))


def test_model_detects_phase_aliasing_with_one_barrier_per_buffer():
    """Depths that are not multiples of the group count fail when each buffer has a single barrier
    pair and copies land late and out of order: a group's parity wait passes on the phase that
    belongs to another group's slab."""
    failures = 0
    for seed in range(10):
        consumed, errors = simulate(6, 6, 4, 1, 240, seed, lcm_bars=False, land_prob=0.05)
        failures += bool(errors) or consumed != list(range(240))
    assert failures >= 5
    for seed in range(5):      # the same depths with lcm(n, d) barriers are fine
        consumed, errors = simulate(6, 6, 4, 1, 240, seed, land_prob=0.05)
        assert not errors and consumed == list(range(240))
