"""Pins for the CPU oracle: what the paper and the mathematics fix, checked on the CPU.

Every pin is a function of the oracle *module*, so the same pins are also run
against deliberately broken copies of the oracle (test_planted_mistakes): a pin
set that lets a dropped term, a swapped operand or a wrong order through is
itself a failure.
"""

import importlib.util
import itertools
import math
import os
import re

import numpy as np
import pytest
import scipy.special

from oracle import csd_oracle as ORACLE

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


# ----------------------------------------------------------------------------
# a second, deliberately different statement of Algorithm 1 (greedy) used as a
# brute-force cross-check: strictly sequential, memory updated in place right
# after each look-up (the printed order), the gate taken on the explicit
# soft-max probability ratio instead of the logit difference.
# ----------------------------------------------------------------------------
def algorithm1_sequential(z_row_block, draft_row, table, lam, tau):
    K = len(draft_row)
    n = 0
    mask = [0] * K
    for i in range(K):
        x = np.asarray(z_row_block[i], dtype=np.float64)
        e = np.exp(x - x.max())
        p = e / e.sum()
        t_star = int(np.argmax(p))                 # numpy: first occurrence
        d = int(draft_row[i])
        if d == t_star:
            n += 1
            continue
        is_freq = table.get((d, t_star), 0) >= lam
        is_safe = (p[d] / p[t_star]) >= tau
        table[(d, t_star)] = table.get((d, t_star), 0) + 1
        if is_freq and is_safe:
            n += 1
            mask[i] = 1
        else:
            return n, t_star, mask
    x = np.asarray(z_row_block[K], dtype=np.float64)
    return n, int(np.argmax(x)), mask


# ----------------------------------------------------------------------------
# pins (each takes the oracle module)
# ----------------------------------------------------------------------------
def pin_row_stats_closed_forms(o):
    V = 1000
    m, t, s, lse = o.row_stats(np.full(V, 2.5, dtype=np.float32))
    assert (m, t) == (2.5, 0)
    assert s == pytest.approx(V, rel=1e-13)
    assert lse == pytest.approx(2.5 + math.log(V), rel=1e-13)
    # one raised token over a flat floor: s = 1 + (V-1) e^-delta
    x = np.zeros(V, dtype=np.float32)
    x[617] = 7.0
    m, t, s, lse = o.row_stats(x)
    assert (m, t) == (7.0, 617)
    assert s == pytest.approx(1 + (V - 1) * math.exp(-7.0), rel=1e-13)
    assert lse == pytest.approx(7.0 + math.log(1 + (V - 1) * math.exp(-7.0)), rel=1e-13)
    # invariance: shifting every logit shifts m and lse and leaves s alone
    rng = np.random.default_rng(1)
    y = rng.normal(size=V)
    a = o.row_stats(y)
    b = o.row_stats(y + 64.0)
    assert b[0] == pytest.approx(a[0] + 64.0, rel=1e-13) and b[1] == a[1]
    assert b[2] == pytest.approx(a[2], rel=1e-12) and b[3] == pytest.approx(a[3] + 64.0, rel=1e-12)


def pin_row_stats_library(o):
    rng = np.random.default_rng(2)
    for V in (1, 2, 17, 4096, 32000):
        x = (rng.normal(size=V) * 3).astype(np.float32)
        m, t, s, lse = o.row_stats(x)
        x64 = x.astype(np.float64)
        assert m == x64.max() and t == int(np.argmax(x64))
        assert lse == pytest.approx(float(scipy.special.logsumexp(x64)), rel=1e-13)
        assert s == pytest.approx(float(np.exp(scipy.special.logsumexp(x64) - m)), rel=1e-12)


def pin_lowest_index_on_ties(o):
    x = np.array([0.0, 3.0, 1.0, 3.0, 3.0, -1.0], dtype=np.float32)
    assert o.row_stats(x)[1] == 1
    x = np.array([5.0, 5.0], dtype=np.float32)
    assert o.row_stats(x)[1] == 0


def pin_eq3_identity(o):
    """exp(z_d - z_t) equals the ratio of full soft-max probabilities (Eq. 3)."""
    rng = np.random.default_rng(3)
    V = 257
    z = rng.normal(size=(2, 4, V)).astype(np.float32) * 2
    draft = rng.integers(0, V, size=(2, 3))
    out = o.verify(z, draft, o.OCM(64, 6), 0.3)
    for b in range(2):
        for i in range(3):
            p = scipy.special.softmax(z[b, i].astype(np.float64))
            t = int(np.argmax(p))
            d = int(draft[b, i])
            assert out["score"][b, i] == pytest.approx(p[d] / p[t], rel=1e-12)
            assert out["p_d"][b, i] == pytest.approx(p[d], rel=1e-12)
            assert out["p_t"][b, i] == pytest.approx(p[t], rel=1e-12)
            assert out["zd"][b, i] == float(z[b, i, d])


def pin_threshold(o):
    assert o.scg_threshold(1.0) == 0.0
    assert o.scg_threshold(0.0) == float("-inf")
    assert o.scg_threshold(0.5) == float(np.float32(-math.log(2.0)))
    assert o.scg_threshold(0.01) == float(np.float32(math.log(float(np.float32(0.01)))))
    # equality passes the gate (Score >= tau): z_d - z_t equal to the threshold itself
    lf = o.scg_threshold(0.25)
    V = 8
    z = np.full((1, 2, V), -50.0, dtype=np.float64)
    z[0, 0, 0] = 0.0            # the target's top token, logit 0: the difference is z_d itself
    z[0, 0, 5] = lf             # draft token sits exactly at the threshold
    mem = o.OCM(64, 0)
    assert o.verify(z, np.array([[5]]), mem, 0.25)["accept_len"][0] == 1
    z[0, 0, 5] = np.nextafter(lf, -np.inf)
    assert o.verify(z, np.array([[5]]), mem, 0.25)["accept_len"][0] == 0


def _random_case(rng, B, K, V, match_p=0.5):
    z = rng.normal(size=(B, K + 1, V)).astype(np.float32)
    top = rng.integers(0, V, size=(B, K + 1))
    for b in range(B):
        for i in range(K + 1):
            z[b, i, top[b, i]] += 4.0
    arg = z.argmax(axis=2)[:, :K]
    draft = np.where(rng.random((B, K)) < match_p, arg, rng.integers(0, V, size=(B, K)))
    return z, draft


def pin_empty_memory_is_strict_matching(o):
    """No pair reaches lambda >= 1 in an empty memory: CSD is plain exact matching."""
    rng = np.random.default_rng(4)
    for tau in (0.0, 0.01, 0.3, 1.0):
        z, draft = _random_case(rng, 6, 5, 50, match_p=0.7)
        out = o.verify(z, draft, o.OCM(1024, 6), tau)
        arg = z.argmax(axis=2)
        for b in range(6):
            lead = 0
            while lead < 5 and draft[b, lead] == arg[b, lead]:
                lead += 1
            assert out["accept_len"][b] == lead
            assert out["next_token"][b] == arg[b, lead]
        assert out["rescued_mask"].sum() == 0


def pin_ablation_reductions(o):
    """lambda = 0 is gating only (Lossy SD); tau = 0 is memory only (SD w/ OCM)."""
    rng = np.random.default_rng(5)
    B, K, V = 8, 4, 12
    z, draft = _random_case(rng, B, K, V, match_p=0.4)
    arg = z.argmax(axis=2)
    z64 = z.astype(np.float64)
    # gating only
    tau = 0.05
    out = o.verify(z, draft, o.OCM(1024, 0), tau)
    for b in range(B):
        n = 0
        for i in range(K):
            d, t = draft[b, i], arg[b, i]
            p = scipy.special.softmax(z64[b, i])
            if d == t or p[d] / p[t] >= tau:
                n += 1
            else:
                break
        assert out["accept_len"][b] == n
    # memory only
    mem = o.OCM(1024, 2)
    pairs = [(int(draft[b, i]), int(arg[b, i])) for b in range(B) for i in range(K) if (b + i) % 2 == 0]
    mem.update(pairs)
    mem.update(pairs)
    out = o.verify(z, draft, mem, 0.0)
    for b in range(B):
        n = 0
        for i in range(K):
            d, t = int(draft[b, i]), int(arg[b, i])
            if d == t or mem.count(d, t) >= 2:
                n += 1
            else:
                break
        assert out["accept_len"][b] == n


def pin_monotone(o):
    """For a fixed memory the accepted length never grows with tau or with lambda."""
    rng = np.random.default_rng(6)
    B, K, V = 16, 6, 10
    z, draft = _random_case(rng, B, K, V, match_p=0.3)
    arg = z.argmax(axis=2)
    mem = o.OCM(4096, 3)
    for rep in range(1, 7):
        mem.update([(int(draft[b, i]), int(arg[b, i])) for b in range(B) for i in range(K)
                    if draft[b, i] != arg[b, i] and (b * K + i) % rep == 0])
    prev = None
    for tau in (0.0, 0.001, 0.01, 0.1, 0.3, 0.6, 1.0, 1.5):
        n = o.verify(z, draft, mem, tau)["accept_len"]
        if prev is not None:
            assert np.all(n <= prev)
        prev = n
    assert prev.tolist() == o.verify(z, draft, o.OCM(64, 6), 0.3)["accept_len"].tolist()  # tau > 1: never safe
    prev = None
    for lam in (0, 1, 2, 3, 4, 6, 100):
        mem.lam = lam
        n = o.verify(z, draft, mem, 0.05)["accept_len"]
        if prev is not None:
            assert np.all(n <= prev)
        prev = n


def _load_fig1():
    spec = {}
    with open(os.path.join(GOLDEN, "fig1_false_rejection.txt")) as f:
        for line in f:
            line = line.strip()
            if not line or line.startswith("#"):
                continue
            k, v = line.split(":", 1)
            spec[k.strip()] = v.strip()
    return spec


def pin_fig1_worked_example(o):
    g = _load_fig1()
    vocab = g["vocab"].split()
    tok = {w: i for i, w in enumerate(vocab)}
    draft = [tok[w] for w in g["draft"].split()]
    top = [tok[w] for w in g["target_top"].split()]
    K, V = len(draft), len(vocab)
    pos = int(g["divergent_position"])
    pd, pt = (tok[w] for w in g["pair"].split())
    z = np.full((1, K + 1, V), -4.0, dtype=np.float32)
    for i, t in enumerate(top):
        z[0, i, t] = 6.0
    z[0, pos, pd] = 6.0 - 1.0                      # Score = e^-1 = 0.37

    def expect(key, out):
        m = re.match(r"accept_len=(\d+) mask=(\d+) next=(\S+)", g[key])
        assert out["accept_len"][0] == int(m.group(1))
        assert "".join(str(int(v)) for v in out["rescued_mask"][0]) == m.group(2)
        assert out["next_token"][0] == tok[m.group(3)]

    mem = o.OCM(64, 6)
    mem.update([(pd, pt)] * 6)
    expect("rescued", o.verify(z, np.array([draft]), mem, 0.3))        # frequent and 0.37 >= 0.3
    mem5 = o.OCM(64, 6)
    mem5.update([(pd, pt)] * 5)
    expect("not_frequent", o.verify(z, np.array([draft]), mem5, 0.3))
    expect("score_below_tau", o.verify(z, np.array([draft]), mem, 0.5))  # 0.37 < 0.5
    # the pair is ordered: (draft, target), not (target, draft)
    swapped = o.OCM(64, 6)
    swapped.update([(pt, pd)] * 6)
    expect("not_frequent", o.verify(z, np.array([draft]), swapped, 0.3))


def pin_update_traces(o):
    """Hand traces of the verification loop of Algorithm 1 on a 6-token vocabulary."""
    V, K = 6, 4
    z = np.zeros((1, K + 1, V), dtype=np.float32)
    tops = [0, 1, 2, 3, 4]
    for i, t in enumerate(tops):
        z[0, i, t] = 5.0
    z[0, 1, 5] = 4.5      # draft 5 at position 1: Score e^-0.5 = 0.61
    z[0, 3, 5] = 4.0      # draft 5 at position 3: Score e^-1 = 0.37
    draft = np.array([[0, 5, 2, 5]])
    mem = o.OCM(64, 2)
    # step 1: position 1 is a divergence (5, 1), not yet frequent -> the row ends there;
    # the terminal rejection IS recorded, nothing after it is.
    out = o.step(z, draft, mem, 0.3)
    assert out["accept_len"][0] == 1 and out["next_token"][0] == 1
    assert dict(mem.table) == {(5, 1): 1}
    assert out["rej_draft"].tolist() == [[-1, 5, -1, -1]] and out["rej_target"].tolist() == [[-1, 1, -1, -1]]
    # step 2: count 1 < 2 still (the look-up precedes the update) -> same outcome, count 2
    out = o.step(z, draft, mem, 0.3)
    assert out["accept_len"][0] == 1 and dict(mem.table) == {(5, 1): 2}
    # step 3: (5, 1) is frequent and safe -> rescued, and a rescued pair still increments;
    # position 3's divergence (5, 3) is reached, not frequent -> terminal, recorded.
    out = o.step(z, draft, mem, 0.3)
    assert out["accept_len"][0] == 3 and out["next_token"][0] == 3
    assert out["rescued_mask"].tolist() == [[0, 1, 0, 0]]
    assert dict(mem.table) == {(5, 1): 3, (5, 3): 1}
    # make (5, 3) frequent: all four accepted, bonus token from the last row
    mem.update([(5, 3)])
    out = o.step(z, draft, mem, 0.3)
    assert out["accept_len"][0] == 4 and out["next_token"][0] == 4
    assert out["rescued_mask"].tolist() == [[0, 1, 0, 1]]
    assert dict(mem.table) == {(5, 1): 4, (5, 3): 3}
    # a stricter gate rejects position 3 (0.37 < 0.5) although it is frequent; still recorded
    out = o.step(z, draft, mem, 0.5)
    assert out["accept_len"][0] == 3 and out["rescued_mask"].tolist() == [[0, 1, 0, 0]]
    assert dict(mem.table) == {(5, 1): 5, (5, 3): 4}
    # duplicates inside one step each count
    mem2 = o.OCM(64, 6)
    mem2.update([(1, 2), (1, 2), (2, 1), (-1, -1), (1, 2)])
    assert dict(mem2.table) == {(1, 2): 3, (2, 1): 1}


def pin_bruteforce_vs_sequential(o):
    """All draft sequences on tiny vocabularies against the strictly sequential
    Algorithm 1 with an explicit soft-max ratio, over several steps of one evolving
    memory (B = 1, where the snapshot reading must agree with the printed order)."""
    rng = np.random.default_rng(7)
    for (V, K, lam, tau) in ((4, 3, 1, 0.2), (5, 2, 2, 0.5), (3, 3, 0, 0.1), (6, 2, 1, 0.0)):
        zs = [np.round(rng.normal(size=(1, K + 1, V)) * 1.5, 1).astype(np.float32) for _ in range(2)]
        for seq in itertools.product(range(V), repeat=K):
            mem = o.OCM(1 << 12, lam)
            ref = {}
            for rep in range(2 * lam + 2):
                z = zs[rep % 2]
                out = o.step(z, np.array([seq]), mem, tau)
                n, nxt, mask = algorithm1_sequential(z[0], seq, ref, lam, tau)
                assert out["accept_len"][0] == n
                assert out["next_token"][0] == nxt
                assert out["rescued_mask"][0].tolist() == mask
                assert dict(mem.table) == ref


def pin_repeated_pair_in_one_row(o):
    """The same pair twice in one row: the second look-up sees the step-start count.
    It is only reached if the first was rescued, i.e. the count was already >= lambda,
    so the snapshot gives the sequential answer."""
    V, K = 4, 3
    z = np.zeros((1, K + 1, V), dtype=np.float32)
    z[0, :, 0] = 3.0
    z[0, :, 1] = 2.5
    draft = np.array([[1, 1, 1]])
    for lam in (0, 1, 2, 3):
        mem = o.OCM(64, lam)
        ref = {}
        for _ in range(5):
            out = o.step(z, draft, mem, 0.5)
            n, nxt, mask = algorithm1_sequential(z[0], draft[0], ref, lam, 0.5)
            assert (out["accept_len"][0], out["next_token"][0]) == (n, nxt)
            assert dict(mem.table) == ref


def pin_capacity_policy(o):
    """Reading R3 (not fixed by the paper): present pairs always count, new pairs are
    admitted in order while there is room, dropped occurrences are counted."""
    mem = o.OCM(8, 1)                     # limit 4
    assert mem.limit == 4
    mem.update([(1, 2), (3, 4), (1, 2), (5, 6), (7, 8), (9, 10), (3, 4), (9, 10), (11, 12)])
    assert dict(mem.table) == {(1, 2): 2, (3, 4): 2, (5, 6): 1, (7, 8): 1}
    assert mem.n_dropped == 3
    mem.update([(9, 10), (1, 2)])
    assert mem.count(1, 2) == 3 and mem.count(9, 10) == 0 and mem.n_dropped == 4
    # while there is room for every new pair of a batch, the order inside it is irrelevant
    rng = np.random.default_rng(8)
    pairs = [(int(a), int(b)) for a, b in rng.integers(0, 6, size=(40, 2))]
    a = o.OCM(256, 1); a.update(pairs)
    b = o.OCM(256, 1); b.update([pairs[j] for j in rng.permutation(len(pairs))])
    assert a.table == b.table
    # saturation
    c = o.OCM(8, 1)
    c.update([(1, 1)], weights=[2**32 - 2])
    c.update([(1, 1), (1, 1), (1, 1)])
    assert c.count(1, 1) == 2**32 - 1
    d, t, n = mem.export()
    assert list(zip(d.tolist(), t.tolist(), n.tolist())) == [(1, 2, 3), (3, 4, 2), (5, 6, 1), (7, 8, 1)]


def pin_bad_draft(o):
    V, K = 5, 3
    z = np.zeros((1, K + 1, V), dtype=np.float32)
    z[0, :, 2] = 1.0
    mem = o.OCM(64, 0)
    out = o.step(z, np.array([[2, 7, 2]]), mem, 0.0)
    assert out["accept_len"][0] == 1 and out["next_token"][0] == 2
    assert out["bad_draft"] == 1 and mem.n_keys == 0
    out = o.step(z, np.array([[-3, 2, 2]]), mem, 0.0)
    assert out["accept_len"][0] == 0 and mem.n_keys == 0


def pin_cross_row_snapshot(o):
    """R2 across rows (not fixed by the paper): row 1 does not see row 0's update of the same step."""
    V, K = 4, 1
    z = np.zeros((2, K + 1, V), dtype=np.float32)
    z[:, :, 0] = 2.0
    z[:, :, 1] = 1.9
    mem = o.OCM(64, 1)
    out = o.step(z, np.array([[1], [1]]), mem, 0.5)
    assert out["accept_len"].tolist() == [0, 0] and mem.count(1, 0) == 2
    out = o.step(z, np.array([[1], [1]]), mem, 0.5)
    assert out["accept_len"].tolist() == [1, 1] and mem.count(1, 0) == 4


def pin_near_tie_flag(o):
    V = 4
    z = np.zeros((1, 2, V), dtype=np.float64)
    z[0, 0, 0] = 1.0
    z[0, 0, 1] = 1.0 + math.log(0.3) + 2e-6
    out = o.verify(z, np.array([[1]]), o.OCM(64, 0), 0.3)
    assert out["near_tie"][0, 0]
    z[0, 0, 1] = 1.0 + math.log(0.3) + 1e-3
    assert not o.verify(z, np.array([[1]]), o.OCM(64, 0), 0.3)["near_tie"][0, 0]


def pin_ageing_and_merge(o):
    """R7 and the weighted merge: hand traces and the properties that make them order-independent."""
    mem = o.OCM(8, 2)                                   # limit: 4 pairs
    mem.update([(1, 2)] * 5 + [(3, 4)] * 2 + [(5, 6)] + [(7, 8)] * 4)
    assert mem.table == {(1, 2): 5, (3, 4): 2, (5, 6): 1, (7, 8): 4}
    mem.update([(9, 9)])                                # full: dropped
    assert mem.n_dropped == 1 and (9, 9) not in mem.table
    mem.age()
    assert mem.table == {(1, 2): 2, (3, 4): 1, (7, 8): 2}          # floor halves; the single occurrence is forgotten
    assert mem.n_dropped == 1                            # ageing is not dropping
    mem.update([(9, 9)])                                # the freed room admits a new pair
    assert mem.table[(9, 9)] == 1 and mem.n_keys == 4
    mem.age(); mem.age()
    assert mem.table == {} and mem.n_keys == 0
    # ageing a saturated count, and twice halving = quartering (floor of floor = floor)
    mem.update([(1, 1)], weights=[o.COUNT_MAX]); mem.update([(1, 1)], weights=[5])
    assert mem.table[(1, 1)] == o.COUNT_MAX
    mem.age()
    assert mem.table[(1, 1)] == (2 ** 32 - 1) // 2
    rng = np.random.default_rng(4)
    a = o.OCM(128, 1); b = o.OCM(128, 1)
    pairs = [(int(x), int(y)) for x, y in rng.integers(0, 6, size=(300, 2))]
    a.update(pairs)
    b.update(pairs[::-1])                               # another arrival order, same multiset, room for all
    a.age(); b.age()
    assert a.table == b.table and all(c == pairs.count(k) // 2 for k, c in a.table.items())
    assert all(pairs.count(k) < 2 for k in set(pairs) - set(a.table))
    # merge: counts of common pairs add, new pairs enter in sorted order while there is room
    x = o.OCM(8, 1); y = o.OCM(64, 1)
    x.update([(1, 1)] * 3 + [(2, 2)] * 2)
    y.update([(2, 2)] * 4 + [(0, 5)] + [(3, 3)] * 2 + [(9, 9)] * 7 + [(8, 8)])
    x.merge(y)
    assert x.table == {(1, 1): 3, (2, 2): 6, (0, 5): 1, (3, 3): 2} and x.n_dropped == 2    # the entries (8,8) and (9,9) found no room: one dropped occurrence each
    assert y.table[(9, 9)] == 7                          # the source is left alone
    big = o.OCM(64, 1); big.update([(1, 1)] * 3 + [(2, 2)] * 2); big.merge(y)
    assert big.table == {(1, 1): 3, (2, 2): 6, (0, 5): 1, (3, 3): 2, (9, 9): 7, (8, 8): 1} and big.n_dropped == 0
    z = o.OCM(64, 1); z.update([(4, 4)], weights=[o.COUNT_MAX - 1]); w = o.OCM(64, 1); w.update([(4, 4)] * 3)
    z.merge(w)
    assert z.table[(4, 4)] == o.COUNT_MAX                # saturates


PINS = [pin_ageing_and_merge, pin_row_stats_closed_forms, pin_row_stats_library, pin_lowest_index_on_ties, pin_eq3_identity,
        pin_threshold, pin_empty_memory_is_strict_matching, pin_ablation_reductions, pin_monotone,
        pin_fig1_worked_example, pin_update_traces, pin_bruteforce_vs_sequential,
        pin_repeated_pair_in_one_row, pin_capacity_policy, pin_bad_draft, pin_cross_row_snapshot,
        pin_near_tie_flag]


@pytest.mark.parametrize("pin", PINS, ids=lambda f: f.__name__)
def test_pin(pin):
    pin(ORACLE)


# ----------------------------------------------------------------------------
# planted mistakes: each edit of the oracle's source must be caught by some pin
# ----------------------------------------------------------------------------
MUTANTS = [
    ("tie -> highest index", "np.flatnonzero(x == m)[0]", "np.flatnonzero(x == m)[-1]"),
    ("sum without the max shift dropped term", "np.sum(np.exp(x - m))", "np.sum(np.exp(x - m)[1:])"),
    ("lse sign", "float(m + np.log(s))", "float(m - np.log(s))"),
    ("lambda strict", "cnt[b, i] >= ocm.lam", "cnt[b, i] > ocm.lam"),
    ("gate strict", "(zd[b, i] - m[b, i]) >= lf", "(zd[b, i] - m[b, i]) > lf"),
    ("gate sign", "(zd[b, i] - m[b, i]) >= lf", "(m[b, i] - zd[b, i]) >= lf"),
    ("gate or instead of and", "if is_freq and is_safe:", "if is_freq or is_safe:"),
    ("key transposed on look-up", "cnt[b, i] = ocm.count(d, t[b, i])", "cnt[b, i] = ocm.count(t[b, i], d)"),
    ("terminal rejection not recorded", "            rej_d[b, i] = d                      # UpdateMemory is unconditional\n            rej_t[b, i] = tt\n            if is_freq and is_safe:              # rescued\n                rescued[b, i] = 1\n",
     "            if is_freq and is_safe:              # rescued\n                rej_d[b, i] = d\n                rej_t[b, i] = tt\n                rescued[b, i] = 1\n"),
    ("continues past an un-rescued rejection", "            n = i                                # un-rescued rejection ends the row\n            break",
     "            n = min(n, i)\n            continue"),
    ("next token from the first row", "next_token[b] = t[b, n]", "next_token[b] = t[b, 0]"),
    ("threshold in natural units", "float(np.float32(np.log(np.float64(tau32))))", "float(np.float32(np.log10(np.float64(tau32))))"),
    ("score without max", "np.exp(zd[b, i] - m[b, i])       # ratio", "np.exp(zd[b, i])       # ratio"),
    ("p_d not normalised", "p_d[b, i] = score[b, i] / s[b, i]", "p_d[b, i] = score[b, i]"),
    ("capacity ignores limit", "elif len(self.table) < self.limit:", "elif True:"),
    ("present pair blocked when full", "            if key in self.table:\n", "            if key in self.table and len(self.table) < self.limit:\n"),
    ("duplicates collapse", "self.table[key] = min(self.table[key] + w, COUNT_MAX)", "self.table[key] = min(self.table[key], COUNT_MAX)"),
    ("no saturation", "min(self.table[key] + w, COUNT_MAX)", "(self.table[key] + w)"),
    ("bad draft recorded", "            if not (0 <= d < V):                 # R5\n                bad += 1\n                n = i\n                break\n",
     "            if not (0 <= d < V):                 # R5\n                bad += 1\n                rej_d[b, i] = d\n                rej_t[b, i] = tt\n                n = i\n                break\n"),
    ("ageing rounds up", "self.table = {k: c // 2 for k, c in self.table.items() if c // 2 > 0}", "self.table = {k: (c + 1) // 2 for k, c in self.table.items() if (c + 1) // 2 > 0}"),
    ("ageing keeps the zeros", "self.table = {k: c // 2 for k, c in self.table.items() if c // 2 > 0}", "self.table = {k: c // 2 for k, c in self.table.items()}"),
    ("ageing forgets the ones but does not halve", "self.table = {k: c // 2 for k, c in self.table.items() if c // 2 > 0}", "self.table = {k: c for k, c in self.table.items() if c // 2 > 0}"),
    ("merge ignores the counts", "self.update(zip(d.tolist(), t.tolist()), weights=c.tolist())", "self.update(zip(d.tolist(), t.tolist()))"),
    ("merge swaps draft and target", "self.update(zip(d.tolist(), t.tolist()), weights=c.tolist())", "self.update(zip(t.tolist(), d.tolist()), weights=c.tolist())"),
    ("rescue mask set on match", "            if d == tt:                          # exact match: accepted\n                continue",
     "            if d == tt:                          # exact match: accepted\n                rescued[b, i] = 1\n                continue"),
]


def _mutant(old, new):
    path = ORACLE.__file__
    src = open(path).read()
    assert src.count(old) >= 1, f"mutation anchor not found: {old[:40]!r}"
    src = src.replace(old, new)
    spec = importlib.util.spec_from_loader("csd_oracle_mutant", loader=None)
    mod = importlib.util.module_from_spec(spec)
    exec(compile(src, path + "<mutant>", "exec"), mod.__dict__)
    return mod


@pytest.mark.parametrize("name,old,new", MUTANTS, ids=[m[0] for m in MUTANTS])
def test_planted_mistakes(name, old, new):
    mod = _mutant(old, new)
    caught = []
    for pin in PINS:
        try:
            pin(mod)
        except Exception:
            caught.append(pin.__name__)
    assert caught, f"no pin notices the planted mistake: {name}"


# ----------------------------------------------------------------------------
# the C restatement of the row statistics is pinned to the numpy statement
# ----------------------------------------------------------------------------
def test_c_row_stats_matches_numpy():
    from oracle import row_stats_c
    rng = np.random.default_rng(9)
    z = (rng.normal(size=(3, 4, 5001)) * 2).astype(np.float32)
    z[1, 2, 77] = z[1, 2].max() + 0.0      # plant an exact tie lower than the arg-max if above it
    z[1, 2, 4000] = z[1, 2, 77]
    m, t, s = row_stats_c.row_stats_batch(z)
    for b in range(3):
        for i in range(4):
            mm, tt, ss, _ = ORACLE.row_stats(z[b, i])
            assert m[b, i] == mm and t[b, i] == tt
            assert s[b, i] == pytest.approx(ss, rel=1e-12)
    # closed form through the C path too
    x = np.zeros((1, 1000), dtype=np.float32)
    x[0, 617] = 7.0
    m, t, s = row_stats_c.row_stats_batch(x)
    assert (m[0], t[0]) == (7.0, 617) and s[0] == pytest.approx(1 + 999 * math.exp(-7.0), rel=1e-13)


def test_c_row_stats_bf16_bits():
    import torch
    from oracle import row_stats_c
    g = torch.Generator().manual_seed(3)
    zb = (torch.randn(2, 3, 3000, generator=g) * 2).to(torch.bfloat16)
    bits = zb.view(torch.int16).numpy().view(np.uint16)
    wide = ORACLE.bf16_bits_to_f64(bits)
    assert np.array_equal(wide, zb.to(torch.float64).numpy())        # decode against torch's own widening
    m, t, s = row_stats_c.row_stats_batch(bits, is_bf16_bits=True)
    for b in range(2):
        for i in range(3):
            mm, tt, ss, _ = ORACLE.row_stats(wide[b, i])
            assert m[b, i] == mm and t[b, i] == tt and s[b, i] == pytest.approx(ss, rel=1e-12)


def test_verify_accepts_precomputed_stats():
    from oracle import row_stats_c
    rng = np.random.default_rng(10)
    z, draft = _random_case(rng, 4, 3, 300)
    mem = ORACLE.OCM(256, 0)
    a = ORACLE.verify(z, draft, mem, 0.2)
    b = ORACLE.verify(z, draft, mem, 0.2, stats=row_stats_c.row_stats_batch(z))
    for k in ("accept_len", "next_token", "rescued_mask", "rej_draft", "rej_target", "t", "cnt"):
        assert np.array_equal(a[k], b[k])
    for k in ("m", "s", "lse", "score", "p_d", "p_t"):
        np.testing.assert_allclose(a[k], b[k], rtol=1e-12)
