"""Pins the oracle's Max-Gram drafter (Section 3.3, Appendix A) to hand-worked cases and to a
brute-force longest-suffix search written straight from the definition."""
import os

import numpy as np

import workloads

GOLD = os.path.join(os.path.dirname(__file__), "golden", "mag_cases.txt")


def brute_search(hay, seq, max_order):
    """Index of the token after the longest, earliest suffix match that is followed by a
    haystack token; None without a match."""
    L, T = len(hay), len(seq)
    for order in range(min(T, max_order), 0, -1):
        needle = list(seq[T - order:])
        for j in range(0, L - order):          # j + order <= L - 1: a following token exists
            if list(hay[j:j + order]) == needle:
                return j + order
    return None


def brute_draft(hay, nxt, seq, n, max_order):
    cur, out = list(seq), []
    while len(out) < n:
        idx = brute_search(hay, cur, max_order)
        if idx is None:
            out.append(int(nxt[cur[-1]]))
            cur.append(out[-1])
        else:
            while len(out) < n and idx < len(hay):
                out.append(int(hay[idx]))
                cur.append(out[-1])
                idx += 1
    return out


def test_hand_worked_cases(orc):
    cases = 0
    for line in open(GOLD):
        line = line.split("#")[0].strip()
        if not line:
            continue
        hay, seq, n, order, over, want = [f.strip() for f in line.split(";")]
        nxt = np.array([(a + 3) % 10 for a in range(10)], dtype=np.int32)
        for pair in over.split():
            a, b = pair.split(":")
            nxt[int(a)] = int(b)
        got = orc.mag_draft([int(x) for x in hay.split()], nxt, [int(x) for x in seq.split()],
                            int(n), int(order))
        assert got.tolist() == [int(x) for x in want.split()], line
        cases += 1
    assert cases == 10


def test_against_brute_force(orc):
    rng = np.random.default_rng(0)
    for trial in range(400):
        V = int(rng.choice([3, 5, 50]))
        L = int(rng.integers(1, 40))
        T = int(rng.integers(1, 30))
        n = int(rng.integers(1, 12))
        order = int(rng.choice([1, 2, 3, 16, 64]))
        hay = rng.integers(0, V, size=L)
        seq = rng.integers(0, V, size=T)
        if trial % 3 == 0 and T >= L:      # decoder-only start: the sequence ends with the haystack
            seq[T - L:] = hay
        nxt = rng.integers(0, V, size=V).astype(np.int32)
        got = orc.mag_draft(hay, nxt, seq, n, order)
        assert got.tolist() == brute_draft(hay, nxt, seq, n, order), (trial, hay, seq, n, order)


def test_n_at_once_equals_one_at_a_time_inside_haystack(orc):
    # uncapped order: extending the sequence by the copied token keeps the same earliest maximal
    # match, so proposing n tokens at once equals n single proposals while tokens remain
    rng = np.random.default_rng(5)
    hits = 0
    for _ in range(200):
        hay = workloads.make_repetitive_prompt(20, 60, int(rng.integers(1 << 30)))
        T = int(rng.integers(2, 12))
        start = int(rng.integers(0, 40))
        seq = np.concatenate([rng.integers(0, 20, size=3), hay[start:start + T]])
        nxt = rng.integers(0, 20, size=20).astype(np.int32)
        idx = brute_search(hay, seq, 10 ** 6)
        if idx is None:
            continue
        n = min(6, len(hay) - idx)
        at_once = orc.mag_draft(hay, nxt, seq, n, 10 ** 6).tolist()
        cur, single = list(seq), []
        for _ in range(n):
            tok = orc.mag_draft(hay, nxt, cur, 1, 10 ** 6).tolist()
            single += tok
            cur += tok
        assert at_once == single
        hits += 1
    assert hits > 50


def test_bigram_table_generator():
    prompt = np.array([4, 7, 4, 7, 4, 9, 2], dtype=np.int32)
    nxt = workloads.bigram_table(prompt, 16, seed=1)
    assert nxt[4] == 7 and nxt[7] == 4 and nxt[9] == 2
    assert ((nxt >= 0) & (nxt < 16)).all()
