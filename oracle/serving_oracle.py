"""Plain reference of the host-side control logic around the Encode stage.  TEST INFRASTRUCTURE ONLY.

Follows the paper's statements step by step: the Poisson-gap dispatch rule (Section 3.2, Eq. 5 and the
three-way dispatch condition), deficit-counter routing (Section 3.3), the SM lookup table (Section 3.4).  Exact
rational arithmetic for the router (the worked example of Figure 6 needs it).  Shares no code with the C++ library."""
from __future__ import annotations
import math
from fractions import Fraction


def kappa(B: int, p: float) -> float:
    """Eq. 5: kappa = -ln(1 - p^(1/(B-1))).  Reading: B = 1 has no gap to wait for (dispatch at once) -> 0."""
    if B <= 1:
        return 0.0
    return -math.log(1.0 - p ** (1.0 / (B - 1)))


def run_batcher(arrivals, B: int, lam: float, p: float = 0.6, max_age: float = 1.0):
    """Dispatch when |batch| = B, or idle > g, or age > A (Section 3.2).  arrivals: sorted times.
    Returns [(dispatch_time, [request indices])]."""
    g = kappa(B, p) / lam
    out, cur, first, last = [], [], None, None
    for i, t in enumerate(arrivals):
        if cur:
            deadline = min(last + g, first + max_age)
            if t > deadline:                       # the timer fired before this arrival
                out.append((deadline, cur))
                cur = []
        if not cur:
            first = t
        cur = cur + [i]
        last = t
        if len(cur) == B:
            out.append((t, cur))
            cur = []
    if cur:
        out.append((min(last + g, first + max_age), cur))
    return out


def route(s: Fraction, n: int):
    """Section 3.3: d starts at 0; every request adds s; d >= 1 -> remote and d -= 1.  Returns a list of 0/1."""
    d = Fraction(0)
    out = []
    for _ in range(n):
        d += s
        if d >= 1:
            d -= 1
            out.append(1)
        else:
            out.append(0)
    return out


def envelope_plan(dest, rows, n_dest):
    """Group requests per destination, keeping arrival order: (row offset of each request, rows per destination)."""
    totals = [0] * n_dest
    offs = []
    for d, r in zip(dest, rows):
        offs.append(totals[d])
        totals[d] += r
    return offs, totals


def envelope_order(dest, rows, n_dest):
    """Section 3.3: the order of requests that makes each destination's envelope one contiguous block of the output
    (stable by destination), and the first output row of each envelope."""
    order = sorted(range(len(dest)), key=lambda i: dest[i])          # Python's sort is stable
    first, acc = [], 0
    for d in range(n_dest):
        first.append(acc)
        acc += sum(r for dd, r in zip(dest, rows) if dd == d)
    return order, first


def sm_table_build(sm_counts, batches, latency, exclusive, tol=0.2):
    """Section 3.4: per SM level, the largest profiled batch size whose latency stays within (1 + tol) of exclusive
    access (reading: all smaller profiled sizes must hold too)."""
    table = []
    for l, sm in enumerate(sm_counts):
        best = 0
        for b, bs in enumerate(batches):
            if latency[l][b] <= (1 + tol) * exclusive[b]:
                best = bs
            else:
                break
        table.append((sm, best))
    return table


def sm_table_lookup(table, batch):
    """Smallest SM share whose supported batch size covers the micro-batch (largest level if none does)."""
    for sm, mb in table:
        if mb >= batch:
            return sm
    return table[-1][0]


def has_stage1(cands, rate, c_e, c_p, c_d, alpha, prune=1.2, top_k=3):
    """Algorithm 1, lines 1-12 (Eq. 3, Eq. 4).  cands: [(n_E, n_P, n_D, n_L)].  Returns (rows, kept indices) with
    rows = (rho_E, rho_P, rho_D, score, B_max, s*)."""
    rows = []
    for nE, nP, nD, nL in cands:
        pw = nP + nL * alpha
        rE, rP, rD = (rate / nE) / c_e, (rate / (c_p * pw) if pw > 0 else math.inf), (rate / nD) / c_d
        rows.append((rE, rP, rD, max(rE, rP, rD), math.ceil(rate / nE), (nP / pw if pw > 0 else 0.0)))
    alive = [i for i, r in enumerate(rows) if r[3] < 1.0]
    if not alive:
        return rows, []
    best = min(rows[i][3] for i in alive)
    alive = [i for i in alive if rows[i][3] <= prune * best]
    alive.sort(key=lambda i: rows[i][3])          # stable: ties keep the earlier candidate
    return rows, sorted(alive[:top_k])
