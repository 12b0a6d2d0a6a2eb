"""CPU checker for the two selection rules beside the MLA-Online step (test infrastructure, not
product code): the protected token-row set of Eq. (protected) and the retained expert fan-out of
Eq. (moe).  Plain loops and sets, written so that a reader can compare them with the paper by eye.
Shares no code with the CUDA library and imports nothing from it.

Both rules end in integers.  `protected_rows` is integer work except for the order of the Indexer
scores, which are compared as the float32 values they are given as.  `moe_fanout` decides with
float32 arithmetic in a fixed order (stated in its docstring) because a float decides an integer
there; `moe_fanout_exact` is the same rule in exact rational arithmetic, used to pin the float32
rule wherever the margin to the threshold is not a rounding question.

Pins (tests/test_oracle_policy_pins.py): a hand-worked request (tests/golden/protected_rows_example.txt),
closed-form set sizes, set-algebra invariants (monotone in every argument, union of single-cause
sets), the budget identity |A & candidates| = max(budget, structural), the top-up order property,
geometric and uniform router weights in closed form, exact rational arithmetic on random weights.
"""
from fractions import Fraction

import numpy as np


def protected_rows(seg_off, seg_delta, seg_has_artifact, dirty_rows=(), scores=None, *,
                   edge_rows=128, tail_rows=32768, budget_bp=0):
    """Eq. (protected): A = Q u N u D u B_edge u I_top u T_tail as ascending packed rows.

    Packed row t lies in segment i (seg_off[i] <= t < seg_off[i+1]) at canonical index
    j = t - seg_off[i] and request position seg_delta[i] + j.

    * Q u N: every row of a segment without offline artifact (query and new rows).
    * D: the dirty rows handed in.
    * B_edge: the first and the last `edge_rows` rows of every relocated segment, i.e. every
      segment with an artifact whose request offset differs from the offset it was built at (0).
    * T_tail: the rows whose request position is among the last `tail_rows` positions of the
      request (positions >= end - tail_rows, end = largest position + 1).
    * I_top: the controller's budget is a share of the candidate rows (rows of segments with an
      artifact), `budget_bp` basis points, rounded down.  If the sets above protect fewer
      candidate rows than that, the candidate rows with the largest Indexer scores are added
      until the budget is met (ties: lower packed row first).  The sets above are never cut.
    """
    seg_off = [int(x) for x in seg_off]
    n_segs = len(seg_off) - 1
    end = max(int(seg_delta[i]) + seg_off[i + 1] - seg_off[i] for i in range(n_segs))
    chosen = set(int(t) for t in dirty_rows)
    candidates = []
    for i in range(n_segs):
        n_i = seg_off[i + 1] - seg_off[i]
        for j in range(n_i):
            t = seg_off[i] + j
            if not seg_has_artifact[i]:
                chosen.add(t)
                continue
            candidates.append(t)
            if int(seg_delta[i]) != 0 and (j < edge_rows or j >= n_i - edge_rows):
                chosen.add(t)
            if int(seg_delta[i]) + j >= end - tail_rows:
                chosen.add(t)
    budget = (int(budget_bp) * len(candidates)) // 10000
    have = sum(1 for t in candidates if t in chosen)
    if scores is not None and budget > have:
        sc = np.asarray(scores, dtype=np.float32)
        rest = [t for t in candidates if t not in chosen]
        rest.sort(key=lambda t: (-float(sc[t]), t))
        chosen.update(rest[:budget - have])
    return np.array(sorted(chosen), dtype=np.int32)


def moe_fanout(p, tau, fence=False):
    """Eq. (moe) for a batch of tokens: p [n, 6] are the Top-6 router weights in any slot order.

    Returns (k [n], keep [n]): K_t and a bit mask over the six input slots of the K_t experts
    that stay (bit s = slot s).  The weights themselves are not touched (no renormalisation).

    Decision arithmetic, float32 throughout: sort the six weights descending (ties: lower slot
    first); c_1 = p_(1), c_k = c_{k-1} + p_(k); K_t is the smallest k in {3,4,5,6} with
    c_k >= tau * c_6 (one float32 product), and 6 if there is none.  Dividing both sides of the
    paper's condition by the same positive sum gives this form without a division per weight.
    A fence layer keeps all six.
    """
    p = np.asarray(p, dtype=np.float32)
    n = p.shape[0]
    k_out = np.zeros(n, dtype=np.uint8)
    keep = np.zeros(n, dtype=np.uint8)
    tau32 = np.float32(tau)
    for t in range(n):
        order = sorted(range(6), key=lambda s: (-float(p[t, s]), s))
        c = []
        acc = np.float32(0.0)
        for r, s in enumerate(order):
            acc = np.float32(p[t, s]) if r == 0 else np.float32(acc + p[t, s])
            c.append(acc)
        k = 6
        if not fence:
            thr = np.float32(tau32 * c[5])
            for cand in (3, 4, 5):
                if c[cand - 1] >= thr:
                    k = cand
                    break
        k_out[t] = k
        keep[t] = sum(1 << s for s in order[:k])
    return k_out, keep


def moe_fanout_exact(p_row, tau):
    """Eq. (moe) for one token in exact rational arithmetic: returns (K_t, margin) where margin is
    the smallest |sum_{j<=k} p^_j - tau| over k = 3..5 (how close any decision is to a tie)."""
    w = sorted((Fraction(float(x)) for x in p_row), reverse=True)
    total = sum(w)
    tau = Fraction(float(tau))
    k_t, margin = 6, None
    for k in (3, 4, 5):
        share = sum(w[:k]) / total
        d = abs(share - tau)
        margin = d if margin is None else min(margin, d)
        if k_t == 6 and share >= tau:
            k_t = k
    return k_t, float(margin)
