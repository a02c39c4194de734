"""Host model of how the precision-configuration kernels deal conversion work to their dequantiser groups.

Per K-step a CTA has UB units of the BFP16 B tile to convert (2 on one SM, 1 on a CTA pair) and, where A is
BFP16 as well, HA hand-overs of A (2 of 128 rows, or 1 of 256).  The jobs of all K-steps form ONE sequence
- B first, because the UMMA issuer waits for the B tile first - and the four dequantiser groups take its
jobs in turn: group g takes jobs g, g + 4, g + 8, ...  A group therefore jumps around in both streams, and
an mbarrier only tells two consecutive phases apart, so every barrier of a ring must always fall to the
same group: the kernels size the barrier set of each ring with stream_bars().  This file restates that
rule and the protocol on the host (barriers with phase counters, actors as coroutines, a random
scheduler, copies landing late) and checks that every hand-over reaches the issuer intact and in order
for every mix the kernels use - and that the model has teeth: with one barrier per buffer the same actors
lose data.
"""
import random

import pytest

from tests.test_ring_protocol import Barrier

GROUPS = 4


def stream_bars(n, h, ipk):
    """Smallest multiple of n (buffers) and h (hand-overs of the stream per K-step) for which hand-over x and
    hand-over x + L fall to the same group when the ipk jobs of a K-step are dealt to GROUPS groups in turn."""
    l = n
    while l % h or ((l // h) * ipk) % GROUPS:
        l += n
    return l


# (what, UB, JA = hand-overs of A that are conversion jobs, operand buffers of A / B, raw buffers of A / B)
MIXES = [
    ("config 1, one SM", 2, 0, 0, 6, 0, 4),
    ("config 1, CTA pair", 1, 0, 0, 4, 0, 4),
    ("config 2, one SM, slabs <= 128 rows", 2, 2, 4, 4, 4, 4),
    ("config 2, one SM, 256-row slabs", 2, 1, 2, 4, 2, 4),
    ("config 2, CTA pair, slabs <= 128 rows", 1, 2, 4, 4, 4, 4),
    ("config 2, CTA pair, 256-row slabs", 1, 1, 2, 4, 2, 4),
]


def job_of(n, ub, ja):
    """Job n of the sequence -> (stream, index in that stream): per K-step the UB units of B, then A's hand-overs."""
    ipk = ub + ja
    ks, j = divmod(n, ipk)
    return ("B", ks * ub + j) if j < ub else ("A", ks * ja + (j - ub))


@pytest.mark.parametrize("mix", MIXES, ids=[m[0] for m in MIXES])
def test_every_barrier_falls_to_one_group(mix):
    _, ub, ja, na, nb, nar, nbr = mix
    ipk = ub + ja
    owner = {}
    for n in range(40 * ipk * GROUPS):
        stream, x = job_of(n, ub, ja)
        h, rings = (ub, (nb, nbr)) if stream == "B" else (ja, (na, nar))
        for ring, depth in zip(("operand", "raw"), rings):
            bar = x % stream_bars(depth, h, ipk)
            assert owner.setdefault((stream, ring, bar), n % GROUPS) == n % GROUPS, (stream, ring, bar)
            assert stream_bars(depth, h, ipk) % depth == 0 and stream_bars(depth, h, ipk) <= 32


def simulate(ub, ja, na, nb, nar, nbr, k_steps, seed, sized=True, land_prob=0.3):
    """Runs producers, four dequantiser groups (two warps each) and the issuer; returns what the issuer consumed
    per stream and the list of protocol errors.  sized = False gives every ring one barrier per buffer."""
    rng = random.Random(seed)
    ipk = ub + ja
    depth = {("A", "op"): na, ("B", "op"): nb, ("A", "raw"): nar, ("B", "raw"): nbr}
    per_k = {"A": ja, "B": ub}
    nbars = {k: (stream_bars(v, per_k[k[0]], ipk) if sized else v) for k, v in depth.items() if v}
    warps = 2
    full = {k: [Barrier(1 if k[1] == "raw" else warps) for _ in range(n)] for k, n in nbars.items()}
    empty = {k: [Barrier(warps if k[1] == "raw" else 1) for _ in range(n)] for k, n in nbars.items()}
    buf = {k: [None] * v for k, v in depth.items() if v}
    in_flight, errors = [], []
    consumed = {"A": [], "B": []}

    def pos(key, x):
        """buffer, barrier and parity of hand-over x; barrier and parity of the last user of its buffer (or None)."""
        n, l = depth[key], nbars[key]
        prev = None if x < n else ((x - n) % l, ((x - n) // l) & 1)
        return x % n, x % l, (x // l) & 1, prev

    def producer(stream):
        key = (stream, "raw")
        for x in range(k_steps * per_k[stream]):
            b, bar, _, prev = pos(key, x)
            if prev is not None:
                while not empty[key][prev[0]].test(prev[1]):
                    yield
            in_flight.append((key, b, bar, x))
            yield

    def dequantiser(g):
        for n in range(g, k_steps * ipk, GROUPS):
            stream, x = job_of(n, ub, ja)
            rk, ok = (stream, "raw"), (stream, "op")
            rb, rbar, rpar, _ = pos(rk, x)
            ob, obar, _, oprev = pos(ok, x)
            while not full[rk][rbar].test(rpar):
                yield
            if oprev is not None:
                while not empty[ok][oprev[0]].test(oprev[1]):
                    yield
            got = buf[rk][rb]
            if got != x:
                errors.append(("raw", stream, x, got))
            yield
            buf[ok][ob] = got
            yield
            full[ok][obar].arrive()
            empty[rk][rbar].arrive()
            yield

    def issuer():
        for ks in range(k_steps):
            for stream in ("B", "A"):               # the issuer waits for the B tile first
                for i in range(per_k[stream]):
                    x = ks * per_k[stream] + i
                    ob, obar, opar, _ = pos((stream, "op"), x)
                    while not full[(stream, "op")][obar].test(opar):
                        yield
                    consumed[stream].append(buf[(stream, "op")][ob])
            yield                                   # the UMMAs of the K-step execute
            for stream in ("A", "B"):
                for i in range(per_k[stream]):
                    empty[(stream, "op")][(ks * per_k[stream] + i) % nbars[(stream, "op")]].arrive()   # tcgen05.commit
            yield

    actors = [producer("B"), issuer()] + ([producer("A")] if ja else [])
    actors += [dequantiser(g) for g in range(GROUPS) for _ in range(warps)]
    live, idle = list(actors), 0
    while live:
        progressed = False
        if in_flight and rng.random() < land_prob:          # copies land late and out of order
            key, b, bar, x = in_flight.pop(rng.randrange(len(in_flight)))
            buf[key][b] = x
            full[key][bar].arrive()
            progressed = True
        a = rng.choice(live)
        before = (len(consumed["A"]), len(consumed["B"]), len(in_flight),
                  [[(q.phase, q.pending) for q in v] for v in list(full.values()) + list(empty.values())])
        try:
            next(a)
        except StopIteration:
            live.remove(a)
            progressed = True
        after = (len(consumed["A"]), len(consumed["B"]), len(in_flight),
                 [[(q.phase, q.pending) for q in v] for v in list(full.values()) + list(empty.values())])
        idle = 0 if (progressed or before != after) else idle + 1
        if idle > 20000:
            errors.append(("deadlock", len(consumed["A"]), len(consumed["B"])))
            break
    return consumed, errors


@pytest.mark.parametrize("mix", MIXES, ids=[m[0] for m in MIXES])
def test_every_hand_over_reaches_the_issuer_in_order(mix):
    _, ub, ja, na, nb, nar, nbr = mix
    k_steps = 96
    for seed, land in enumerate([0.5, 0.05, 0.02]):
        consumed, errors = simulate(ub, ja, na, nb, nar, nbr, k_steps, seed, land_prob=land)
        assert not errors, errors[:3]
        assert consumed["B"] == list(range(k_steps * ub))
        assert consumed["A"] == list(range(k_steps * ja))


def test_model_detects_too_few_barriers():
    """Config 2 on the CTA pair deals three jobs per K-step to four groups: with one barrier per buffer (4 for a
    ring of 4) a barrier changes hands between groups and a parity wait passes on another group's phase."""
    failures = 0
    for seed in range(8):
        consumed, errors = simulate(1, 2, 4, 4, 4, 4, 96, seed, sized=False, land_prob=0.05)
        failures += bool(errors) or consumed["A"] != list(range(192)) or consumed["B"] != list(range(96))
    assert failures >= 4
    assert stream_bars(4, 2, 3) == 8 and stream_bars(4, 1, 3) == 4 and stream_bars(6, 2, 2) == 12
