"""Pins the oracle's Max-Gram drafter (Section 3.3, Appendix A) to hand-worked cases and to the
tensor formulation of Appendix A (boolean match vectors that are extended one token at a time),
written here with numpy; the oracle itself searches order by order, start by start."""
import os

import numpy as np

import workloads

GOLD = os.path.join(os.path.dirname(__file__), "golden", "mag_cases.txt")


def brute_search(hay, seq, max_order):
    """Index of the token after the longest, earliest suffix match that is followed by a haystack
    token; None without a match.  alive[j] says that a match of `order` tokens ENDS at haystack
    index j; a longer match ending there needs one more equal token on its left."""
    hay, seq = np.asarray(hay), np.asarray(seq)
    L = len(hay)
    alive = hay == seq[-1]
    alive[L - 1:] = False                      # the last haystack token has nothing after it
    if not alive.any():
        return None
    for order in range(2, min(len(seq), max_order) + 1):
        longer = np.zeros(L, dtype=bool)
        longer[order - 1:] = alive[order - 1:] & (hay[:L - order + 1] == seq[-order])
        if not longer.any():
            break
        alive = longer
    return int(np.flatnonzero(alive)[0]) + 1   # earliest end = earliest start, the length being fixed


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


def test_dynamic_haystack_is_the_static_search_over_prompt_plus_generation(orc):
    # Section 3.3 lets the match come from the initial input or from what has been generated.  With a
    # target that soon repeats itself, a drafter that also searches the generation gets more of its
    # tokens accepted than one that searches the prompt alone, and the output stays the target's own.
    from workloads import llama_shape
    shape = llama_shape(1, 16, 2, 32, 12, 200)
    blob = orc.blob_to_u16(workloads.make_weights(shape, seed=3, std=1.5))
    prompt = workloads.make_prompt(shape.vocab, 6, seed=1)
    nxt = workloads.bigram_table(prompt, shape.vocab, seed=1)
    outs, accepted = [], []
    for dyn in (False, True):
        got, _, st = orc.cascade_generate([orc.Model(shape, blob)], prompt, nxt, [[6]], 6, prompt, 120,
                                          dynamic_haystack=dyn)
        outs.append(got.tolist())
        accepted.append(st["accepted"][0])
    assert outs[0] == outs[1]                  # greedy: the drafter cannot change the output
    assert accepted[1] > accepted[0] + 10
