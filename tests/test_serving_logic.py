"""Host-side mechanisms around the encoder (Sections 3.2-3.4): the oracle against what the paper prints and what the
mathematics fixes, and the C++ library against the oracle.  CPU only."""
import math
import os
from fractions import Fraction

import numpy as np
import pytest

from oracle import serving_oracle as SO

GOLDEN = os.path.join(os.path.dirname(__file__), "golden", "serving_examples.txt")


def _golden():
    g = {"kappa": [], "sm_lookup": []}
    for line in open(GOLDEN):
        if line.startswith("#") or not line.strip():
            continue
        k, *v = line.split()
        if k in ("kappa", "sm_lookup"):
            g[k].append(v)
        else:
            g[k] = v
    return g


@pytest.fixture(scope="module")
def sv():
    from paper_2609_31551_b200.build import build_library
    build_library()
    from paper_2609_31551_b200 import serving
    return serving


# ------------------------------------------------------------------ oracle pins
def test_oracle_kappa_closed_form_and_fill_probability():
    g = _golden()
    for B, val in g["kappa"]:
        assert abs(SO.kappa(int(B), 0.6) - float(val)) < 1e-6
    # B = 2: one gap, kappa = -ln(1 - p)
    assert abs(SO.kappa(2, 0.3) + math.log(0.7)) < 1e-15
    # definition: (1 - exp(-kappa))^(B-1) = p
    for B in (2, 3, 8, 64):
        for p in (0.5, 0.6, 0.7):
            assert abs((1 - math.exp(-SO.kappa(B, p))) ** (B - 1) - p) < 1e-12
    # Monte Carlo on Poisson arrivals: a batch fills to B before its idle gap expires with probability p
    rng = np.random.Generator(np.random.PCG64(7))
    lam, B, p = 3.0, 6, 0.6
    arrivals = np.cumsum(rng.exponential(1 / lam, size=300000))
    batches = SO.run_batcher(arrivals.tolist(), B, lam, p, max_age=1e9)
    full = sum(1 for _, reqs in batches if len(reqs) == B)
    assert abs(full / len(batches) - p) < 0.01


def test_oracle_batcher_invariants():
    rng = np.random.Generator(np.random.PCG64(11))
    lam, B, p, A = 5.0, 8, 0.6, 1.0
    arrivals = np.cumsum(rng.exponential(1 / lam, size=5000)).tolist()
    g = SO.kappa(B, p) / lam
    batches = SO.run_batcher(arrivals, B, lam, p, A)
    seen = [i for _, reqs in batches for i in reqs]
    assert seen == list(range(len(arrivals)))                      # every request dispatched once, in order
    for when, reqs in batches:
        t = [arrivals[i] for i in reqs]
        assert 1 <= len(reqs) <= B
        assert all(b - a <= g + 1e-12 for a, b in zip(t, t[1:]))   # no idle gap above g inside a batch
        assert when - t[0] <= A + 1e-12                            # age cap
        assert when >= t[-1]
        if len(reqs) < B:
            assert abs(when - min(t[-1] + g, t[0] + A)) < 1e-12
    assert SO.run_batcher([0.0, 0.1, 5.0], 1, lam) == [(0.0, [0]), (0.1, [1]), (5.0, [2])]   # B = 1: immediately
    # the age cap fires on a trickle that never leaves a gap above g
    trickle = [0.99 * g * i for i in range(400)]
    capped = SO.run_batcher(trickle, 1000, lam, p, A)
    assert all(when - trickle[reqs[0]] <= A + 1e-12 for when, reqs in capped) and len(capped) > 1


def test_oracle_router_reproduces_figure_6_and_bounds():
    g = _golden()
    num, den = (int(x) for x in g["router_s"][0].split("/"))
    dec = SO.route(Fraction(num, den), int(g["router_n"][0]))
    local = [i + 1 for i, d in enumerate(dec) if d == 0]
    assert local == [int(x) for x in g["router_local"]]
    assert sum(dec) == 14                                          # about seven remote per three local
    for s in (Fraction(1, 3), Fraction(7, 10), Fraction(9, 10), Fraction(1, 20), Fraction(13, 17)):
        d = SO.route(s, 2000)
        for n in range(1, 2001, 37):
            assert sum(d[:n]) == math.floor(n * s)                 # d0 = 0: remote count = floor(n s)
        runs = "".join(map(str, d))
        assert "1" * (math.ceil(1 / (1 - s)) + 1) not in runs      # bounded consecutive remote decisions
        assert "0" * (math.ceil(1 / s) + 1) not in runs            # bounded consecutive local decisions
    assert SO.route(Fraction(0), 10) == [0] * 10 and SO.route(Fraction(1), 10) == [1] * 10


def test_oracle_sm_table_reproduces_figure_8():
    g = _golden()
    levels = [int(x) for x in g["sm_levels"]]
    maxb = [int(x) for x in g["sm_max_batch"]]
    table = list(zip(levels, maxb))
    for batch, level in g["sm_lookup"]:
        assert SO.sm_table_lookup(table, int(batch)) == int(level)
    assert SO.sm_table_lookup(table, 9) == 90                      # nothing covers it: the largest share
    # build: latencies shaped like Figure 7 (steep, then flat), threshold 20 % over exclusive access
    batches = [2, 4, 6, 8]
    excl = [100.0, 180.0, 260.0, 340.0]
    lat = [[e * f for e in excl] for f in (1.15, 1.1, 1.05, 1.02, 1.0)]
    lat[0][1:] = [400.0, 600.0, 900.0]         # 10 %: only batch 2 holds
    lat[1][2:] = [330.0, 450.0]                # 30 %: up to 4
    lat[2][3] = 420.0                          # 50 %: up to 6
    assert SO.sm_table_build(levels, batches, lat, excl, 0.2) == table


# ------------------------------------------------------------------ the C++ library against the oracle
def test_library_kappa_and_batcher_match_oracle(sv):
    for B in (1, 2, 3, 8, 33):
        for p in (0.5, 0.6, 0.9):
            assert abs(sv.kappa(B, p) - SO.kappa(B, p)) < 1e-14
    assert math.isnan(sv.kappa(4, 1.5))
    rng = np.random.Generator(np.random.PCG64(3))
    for lam, B, A in ((2.0, 4, 1.0), (20.0, 16, 0.3), (0.5, 8, 1.0), (3.0, 1, 1.0)):
        arrivals = np.cumsum(rng.gamma(0.5, 2.0 / lam, size=3000)).tolist()      # bursty (CV about 1.4)
        ref = [(t, len(r)) for t, r in SO.run_batcher(arrivals, B, lam, 0.6, A)]
        got = sv.run_batcher(arrivals, B, lam, 0.6, A)
        assert [s for _, s in got] == [s for _, s in ref]
        assert np.allclose([t for t, _ in got], [t for t, _ in ref], rtol=0, atol=1e-9)
    with pytest.raises(ValueError):
        sv.run_batcher([0.0], 0, 1.0)


def test_library_router_envelopes_and_table_match_oracle(sv):
    for num, den in ((7, 10), (1, 3), (0, 1), (1, 1), (13, 17)):
        assert sv.route(num, den, 500) == SO.route(Fraction(num, den), 500)
    assert sv.router_fraction(0.7) == (7, 10)
    assert sv.router_fraction(1 / 3, 100) == (1, 3)
    assert sv.route(*sv.router_fraction(0.7), 20) == SO.route(Fraction(7, 10), 20)
    rng = np.random.Generator(np.random.PCG64(5))
    dest = rng.integers(0, 3, size=40).tolist()
    rows = rng.integers(1, 600, size=40).tolist()
    assert sv.envelope_plan(dest, rows, 3) == tuple(SO.envelope_plan(dest, rows, 3))
    with pytest.raises(ValueError):
        sv.envelope_plan([0, 5], [1, 1], 3)
    assert sv.envelope_order(dest, rows, 3) == tuple(SO.envelope_order(dest, rows, 3))
    assert sv.envelope_order([], [], 2) == ([], [0, 0])
    with pytest.raises(ValueError):
        sv.envelope_order([0, 3], [1, 1], 3)
    levels, batches = [15, 44, 74, 104, 133], [1, 2, 4, 8, 16]
    lat = rng.uniform(1.0, 2.0, size=(5, 5)) * np.array([[1, 2, 4, 8, 16]])
    excl = np.array([1.0, 2.0, 4.0, 8.0, 16.0]) * 1.1
    t = sv.sm_table_build(levels, batches, lat, excl, 0.2)
    ref = SO.sm_table_build(levels, batches, lat.tolist(), excl.tolist(), 0.2)
    assert [(t.sm_count[i], t.max_batch[i]) for i in range(t.n_levels)] == ref
    for b in range(1, 20):
        assert sv.sm_table_lookup(t, b) == SO.sm_table_lookup(ref, b)


def test_has_stage1_oracle_properties_and_library(sv):
    # 8 GPUs, encode workers on 1 GPU, prefill/decode workers on 2 GPUs each, one local prefill worker per encode GPU
    cands = [(nE, P // 2, D // 2, nE) for nE in range(1, 7) for P in (0, 2, 4) for D in (2, 4) if nE + P + D == 8]
    rate, cE, cP, cD, alpha = 2.5, 2.1, 2.0, 3.4, 0.5
    rows, kept = SO.has_stage1(cands, rate, cE, cP, cD, alpha)
    for (nE, nP, nD, nL), (rE, rP, rD, score, bmax, s_star) in zip(cands, rows):
        assert abs(rE - rate / nE / cE) < 1e-15 and abs(rD - rate / nD / cD) < 1e-15            # Eq. 3
        assert abs(rP - rate / (cP * (nP + nL * alpha))) < 1e-15                                   # prefill with the local term
        assert score == max(rE, rP, rD) and bmax == math.ceil(rate / nE)                           # Eq. 4, B_max
        assert abs(s_star - nP * cP / (nP * cP + nL * alpha * cP)) < 1e-15                         # C_remote / (C_remote + C_local)
    assert 1 <= len(kept) <= 3
    best = min(r[3] for r in rows if r[3] < 1)
    assert all(rows[i][3] < 1 and rows[i][3] <= 1.2 * best for i in kept)
    dropped = [i for i in range(len(cands)) if i not in kept and rows[i][3] < 1 and rows[i][3] <= 1.2 * best]
    assert all(rows[i][3] >= max(rows[k][3] for k in kept) for i in dropped)                       # only the top K stay
    # every stage overloaded -> nothing survives
    assert SO.has_stage1(cands, 500.0, cE, cP, cD, alpha)[1] == []
    lrows, lkept = sv.has_stage1(cands, rate, cE, cP, cD, alpha)
    assert lkept == kept
    assert np.allclose(np.asarray(lrows, dtype=float), np.asarray(rows, dtype=float), rtol=0, atol=1e-14)
    assert sv.has_stage1(cands, 500.0, cE, cP, cD, alpha)[1] == []
    with pytest.raises(ValueError):
        sv.has_stage1([(0, 1, 1, 0)], rate, cE, cP, cD, alpha)


def test_envelope_order_lays_envelopes_out_back_to_back():
    """Pin of the oracle by construction: write each request's rows in the returned order into one buffer and check
    that every destination's rows form one contiguous block, in arrival order, at the offsets of the envelope plan."""
    rng = np.random.Generator(np.random.PCG64(11))
    for n, n_dest in ((1, 1), (7, 3), (40, 4), (64, 2)):
        dest = rng.integers(0, n_dest, size=n).tolist()
        rows = rng.integers(1, 50, size=n).tolist()
        order, first = SO.envelope_order(dest, rows, n_dest)
        offs, totals = SO.envelope_plan(dest, rows, n_dest)
        assert sorted(order) == list(range(n))
        owner = []                                   # request id of every output row, in encode order
        for i in order:
            owner += [i] * rows[i]
        for d in range(n_dest):
            block = owner[first[d]: first[d] + totals[d]]
            expect = []
            for i in range(n):
                if dest[i] == d:
                    assert owner.index(i) == first[d] + offs[i] if rows[i] else True
                    expect += [i] * rows[i]
            assert block == expect
        assert first[0] == 0 and all(first[d + 1] == first[d] + totals[d] for d in range(n_dest - 1))
