"""Pins of the CPU checker for the selection rules (Eq. protected, Eq. moe) against things other than
itself: a hand-worked request, closed-form set sizes, set algebra, the budget identity, the order
property of the top-up, closed-form router weights and exact rational arithmetic."""
import os

import numpy as np
import pytest

from oracle import policy

GOLDEN = os.path.join(os.path.dirname(__file__), "golden", "protected_rows_example.txt")
GOLDEN_MOE = os.path.join(os.path.dirname(__file__), "golden", "moe_fanout_example.txt")


def read_moe_examples():
    cases = []
    for line in open(GOLDEN_MOE):
        line = line.strip()
        if not line or line.startswith("#"):
            continue
        w, tau, k, kept = [f.strip() for f in line.split("|")]
        cases.append(([float(x) for x in w.split()], float(tau), int(k), [int(x) for x in kept.split()]))
    return cases


def read_example():
    lines = [l.strip() for l in open(GOLDEN) if l.strip() and not l.startswith("#")]
    ints = lambda s: [int(x) for x in s.split()]
    seg_off, seg_delta, has = ints(lines[0]), ints(lines[1]), ints(lines[2])
    edge, tail = ints(lines[3])
    dirty = ints(lines[4])
    cases = {}
    for l in lines[5:]:
        bp, rows = l.split(":")
        cases[int(bp)] = ints(rows)
    return seg_off, seg_delta, has, edge, tail, dirty, cases


def test_hand_worked_request():
    seg_off, seg_delta, has, edge, tail, dirty, cases = read_example()
    scores = np.array([(7 * t) % 11 for t in range(seg_off[-1])], dtype=np.float32)
    assert len(cases) == 5
    for bp, want in cases.items():
        got = policy.protected_rows(seg_off, seg_delta, has, dirty, scores, edge_rows=edge, tail_rows=tail, budget_bp=bp)
        assert got.tolist() == want, bp


def regular_layout(n_docs, n, n_q, first_at_zero=True):
    seg_off = [0]
    seg_delta = []
    pos = 0 if first_at_zero else 5
    for _ in range(n_docs):
        seg_off.append(seg_off[-1] + n)
        seg_delta.append(pos)
        pos += n
    seg_off.append(seg_off[-1] + n_q)
    seg_delta.append(pos)
    return seg_off, seg_delta, [1] * n_docs + [0]


@pytest.mark.parametrize("n_docs,n,n_q,edge,tail", [(4, 100, 7, 8, 0), (3, 10, 1, 8, 0), (5, 64, 16, 4, 40), (2, 50, 3, 0, 0),
                                                     (3, 30, 2, 5, 1000)])
def test_closed_form_sizes(n_docs, n, n_q, edge, tail):
    """Documents of equal length back to back, the first at offset 0: the first has no edge rows, the
    others min(n, 2 edge) each; the tail is the last `tail` positions; the query rows are all in."""
    seg_off, seg_delta, has = regular_layout(n_docs, n, n_q)
    got = policy.protected_rows(seg_off, seg_delta, has, edge_rows=edge, tail_rows=tail)
    T = n_docs * n + n_q
    # count by position instead of by segment: layout is the identity map row <-> position here
    want = set(range(n_docs * n, T))
    want |= set(range(max(0, T - tail), T))
    for d in range(1, n_docs):
        want |= set(range(d * n, d * n + min(edge, n))) | set(range((d + 1) * n - min(edge, n), (d + 1) * n))
    assert got.tolist() == sorted(want)
    if tail == 0 and 2 * edge <= n:
        assert len(got) == n_q + (n_docs - 1) * 2 * edge


def test_relocation_decides_edges_and_positions_decide_the_tail():
    """Packed order differs from request order: the tail follows request positions, and a document
    moved off offset 0 gains edge rows."""
    seg_off = [0, 20, 40, 44]
    seg_delta = [24, 0, 44]           # packed doc 0 sits second in the request, packed doc 1 first
    has = [1, 1, 0]
    got = policy.protected_rows(seg_off, seg_delta, has, edge_rows=3, tail_rows=10)
    # doc 0: relocated -> rows 0,1,2 and 17,18,19; tail = positions 38..47 -> doc 0 canonical 14..19 = rows 14..19
    assert got.tolist() == [0, 1, 2, 14, 15, 16, 17, 18, 19, 40, 41, 42, 43]
    moved = policy.protected_rows(seg_off, [24, 1, 44], has, edge_rows=3, tail_rows=10)
    assert set(moved) - set(got) == {20, 21, 22, 37, 38, 39}


def test_union_of_single_cause_sets_and_monotonicity():
    rng = np.random.default_rng(5)
    seg_off, seg_delta, has = regular_layout(6, 37, 9, first_at_zero=False)
    perm_delta = list(seg_delta)
    T = seg_off[-1]
    dirty = rng.choice(T, size=11, replace=False)
    full = set(policy.protected_rows(seg_off, perm_delta, has, dirty, edge_rows=4, tail_rows=50))
    only_q = set(policy.protected_rows(seg_off, perm_delta, has, edge_rows=0, tail_rows=0))
    only_d = set(policy.protected_rows(seg_off, perm_delta, has, dirty, edge_rows=0, tail_rows=0))
    only_b = set(policy.protected_rows(seg_off, perm_delta, has, edge_rows=4, tail_rows=0))
    only_t = set(policy.protected_rows(seg_off, perm_delta, has, edge_rows=0, tail_rows=50))
    assert only_q == set(range(6 * 37, T))
    assert only_d == only_q | set(int(x) for x in dirty)
    assert full == only_d | only_b | only_t
    assert len(only_b - only_q) == 6 * 8              # first document sits at offset 5: relocated too
    assert len(only_t) == 50
    bigger = set(policy.protected_rows(seg_off, perm_delta, has, dirty, edge_rows=5, tail_rows=60))
    assert full <= bigger


@pytest.mark.parametrize("bp", [0, 1000, 2000, 2500, 7000])
def test_budget_identity_and_top_up_order(bp):
    rng = np.random.default_rng(bp + 1)
    seg_off, seg_delta, has = regular_layout(5, 200, 30)
    T = seg_off[-1]
    scores = rng.standard_normal(T).astype(np.float32)
    scores[rng.choice(T, size=100, replace=False)] = 0.25      # ties
    dirty = rng.choice(T, size=17, replace=False)
    base = set(policy.protected_rows(seg_off, seg_delta, has, dirty, None, edge_rows=16, tail_rows=64, budget_bp=bp))
    got = set(policy.protected_rows(seg_off, seg_delta, has, dirty, scores, edge_rows=16, tail_rows=64, budget_bp=bp))
    cand = set(range(5 * 200))
    budget = bp * len(cand) // 10000
    assert base <= got
    assert len(got & cand) == max(budget, len(base & cand))
    added, left = got - base, cand - got
    if added and left:
        worst_in = min((float(scores[t]), -t) for t in added)
        best_out = max((float(scores[t]), -t) for t in left)
        assert worst_in > best_out


def test_moe_hand_worked_examples():
    cases = read_moe_examples()
    assert len(cases) == 12
    for w, tau, k_want, kept in cases:
        k, keep = policy.moe_fanout(np.array([w], dtype=np.float32), tau)
        assert int(k[0]) == k_want, (w, tau)
        assert [s for s in range(6) if (int(keep[0]) >> s) & 1] == kept, (w, tau)


def test_moe_geometric_weights_closed_form():
    """p = 32,16,8,4,2,1 (exact in float32): cumulative shares 56/63, 60/63, 62/63."""
    p = np.array([[4, 32, 1, 8, 16, 2]], dtype=np.float32)
    for tau, k_want in [(0.5, 3), (0.85, 3), (0.9, 4), (0.96, 5), (0.99, 6), (1.0, 6)]:
        k, keep = policy.moe_fanout(p, tau)
        assert int(k[0]) == k_want, tau
        order = [1, 4, 3, 0, 5, 2]                     # slots by descending weight
        assert int(keep[0]) == sum(1 << s for s in order[:k_want])
    k, keep = policy.moe_fanout(p, 0.5, fence=True)
    assert int(k[0]) == 6 and int(keep[0]) == 63


def test_moe_uniform_weights_closed_form():
    p = np.full((1, 6), 0.125, dtype=np.float32)      # shares k/6
    for tau, k_want in [(0.45, 3), (0.6, 4), (0.8, 5), (0.9, 6)]:
        k, keep = policy.moe_fanout(p, tau)
        assert int(k[0]) == k_want
        assert int(keep[0]) == (1 << k_want) - 1      # ties keep the lower slots


def test_moe_float32_rule_equals_exact_rule_away_from_ties():
    rng = np.random.default_rng(11)
    logits = rng.standard_normal((4000, 6)) * 1.5
    p = (np.exp(logits) / np.exp(logits).sum(1, keepdims=True) * rng.uniform(0.2, 0.9, size=(4000, 1))).astype(np.float32)
    checked = 0
    for tau in (0.7, 0.85, 0.95):
        k, keep = policy.moe_fanout(p, tau)
        for t in range(0, 4000, 7):
            k_exact, margin = policy.moe_fanout_exact(p[t], np.float32(tau))
            if margin > 1e-5:
                assert int(k[t]) == k_exact
                checked += 1
            kept = [s for s in range(6) if (int(keep[t]) >> s) & 1]
            assert len(kept) == int(k[t])
            assert min(p[t, kept]) >= max([p[t, s] for s in range(6) if s not in kept], default=0.0)
    assert checked > 1500
    ks = policy.moe_fanout(p, 0.85)[0]
    assert set(np.unique(ks)) <= {3, 4, 5, 6} and len(np.unique(ks)) >= 3
