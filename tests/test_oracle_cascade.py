"""Pins the oracle's Algorithm 1 driver: whatever the drafts propose, the output must be the
target model's own (greedy: token for token; sampling: in distribution), and the call pattern
must follow the budget matrix K."""
import numpy as np
import pytest
from scipy import stats

import workloads
from workloads import llama_shape, t5_shape


MICRO_T = llama_shape(2, 32, 2, 64, 48, 200)
MICRO_D = llama_shape(1, 16, 2, 32, 48, 200)


def models(orc, shapes, seeds, std=0.6):
    return [orc.Model(s, orc.blob_to_u16(workloads.make_weights(s, seed=sd, std=std, gain_std=0.1)))
            for s, sd in zip(shapes, seeds)]


def target_only_greedy(orc, shape, seed, prompt, n_new, std=0.6, enc=None):
    m = models(orc, [shape], [seed], std)[0]
    if enc is not None:
        m.encoder_forward(enc)
    logits = m.review_forward(prompt, 0)[-1]
    out = []
    pos = len(prompt)
    for _ in range(n_new):
        t = int(np.argmax(logits))
        out.append(t)
        logits = m.review_forward([t], pos)[0]
        pos += 1
    return out


@pytest.mark.parametrize("K,max_block", [
    ([[4, 0], [0, 4]], 4),        # vertical cascade: draft reviews Max-Gram, target reviews draft
    ([[2, 10], [0, 10]], 16),     # the decoder-only setting of Appendix B
    ([[2, 10], [0, 10]], 5),      # same, surplus drafts dropped before the review
    ([[0, 6], [0, 0]], 6),        # Max-Gram drafts straight for the target
    ([[1, 3], [0, 1]], 3),
    ([[3, 0], [0, 1]], 8),
])
def test_greedy_output_equals_target_only_greedy(orc, K, max_block):
    prompt = workloads.make_repetitive_prompt(MICRO_T.vocab, 40, seed=3)
    nxt = workloads.bigram_table(prompt, MICRO_T.vocab, seed=1)
    want = target_only_greedy(orc, MICRO_T, 11, prompt, 48)
    for draft_seed, draft_shape in ((12, MICRO_D), (11, MICRO_T)):   # a poor draft, and a perfect one
        ms = models(orc, [MICRO_T, draft_shape], [11, draft_seed])
        got, margins, st = orc.cascade_generate(ms, prompt, nxt, K, max_block, prompt, 48)
        assert got.tolist() == want
        assert st["tokens"] == 48
        assert st["drafted"][0] <= max_block * st["reviews"][0]
        assert st["accepted"][0] + st["reviews"][0] >= 48      # each review emits n_acc + 1 tokens
        assert len(margins) == 48 and np.isfinite(margins).all() and (margins >= 0).all()
    # the perfect draft is accepted whenever the target reviews its tokens
    if K[0][0] > 0:
        assert st["accepted"][0] > 0


def test_margins_are_the_top_two_gap_of_the_target_logits(orc):
    # the margin decides which generated positions an end-to-end comparison may trust, so it is
    # pinned on its own: recompute the target's logits teacher-forced and take the gap of the two
    # largest with numpy
    prompt = workloads.make_repetitive_prompt(MICRO_T.vocab, 40, seed=3)
    nxt = workloads.bigram_table(prompt, MICRO_T.vocab, seed=1)
    ms = models(orc, [MICRO_T, MICRO_D], [11, 12])
    got, margins, st = orc.cascade_generate(ms, prompt, nxt, [[2, 3], [0, 3]], 4, prompt, 30)
    seq = np.concatenate([prompt, got]).astype(np.int32)
    logits = models(orc, [MICRO_T], [11])[0].review_forward(seq[:-1], 0)
    for i in range(30):
        top = np.sort(logits[len(prompt) - 1 + i])[-2:]
        assert margins[i] == np.float32(top[1] - top[0])
    assert orc.top2_margin([3.0, -1.0, 2.5, 2.5]) == 0.5 and orc.top2_margin([1.0, 1.0]) == 0.0
    assert st["near_ties"] == 0 and st["first_near_tie"] == -1       # greedy reviews flag nothing


def test_target_alone_and_three_levels(orc):
    prompt = workloads.make_repetitive_prompt(MICRO_T.vocab, 30, seed=8)
    nxt = workloads.bigram_table(prompt, MICRO_T.vocab, seed=2)
    want = target_only_greedy(orc, MICRO_T, 21, prompt, 30)
    # no neural draft at all: Max-Gram proposes, the target reviews
    got, _, st = orc.cascade_generate(models(orc, [MICRO_T], [21]), prompt, nxt, [[5]], 5, prompt, 30)
    assert got.tolist() == want and st["mag_calls"] == st["reviews"][0]
    # two neural drafts + Max-Gram: horizontal cascade over three slots
    ms = models(orc, [MICRO_T, MICRO_T, MICRO_D], [21, 21, 5])
    K = [[2, 2, 3], [0, 1, 4], [0, 0, 4]]
    got, _, st = orc.cascade_generate(ms, prompt, nxt, K, 7, prompt, 30)
    assert got.tolist() == want
    assert st["reviews"][1] > 0 and st["reviews"][2] > 0


def test_call_pattern_follows_budget_matrix(orc):
    # K = [[2, 10], [0, 10]]: in the first slot the draft reviews 10-token Max-Gram blocks until
    # two tokens exist; the second slot is one Max-Gram call of 10; then the target reviews.
    prompt = workloads.make_repetitive_prompt(MICRO_T.vocab, 40, seed=4)
    nxt = workloads.bigram_table(prompt, MICRO_T.vocab, seed=1)
    ms = models(orc, [MICRO_T, MICRO_D], [31, 32])
    _, _, st = orc.cascade_generate(ms, prompt, nxt, [[2, 10], [0, 10]], 16, prompt, 40)
    assert st["mag_tokens"] == 10 * st["mag_calls"]
    assert st["mag_calls"] == st["reviews"][0] + st["reviews"][1]
    assert st["reviews"][1] >= st["reviews"][0]            # at least one draft review per step
    assert st["reviews"][1] <= 2 * st["reviews"][0]        # and at most k = 2 of them
    assert st["drafted"][1] == 10 * st["reviews"][1]
    # the oracle carries no cache between reviews: one forward over the whole sequence per review
    assert st["forwards"] == st["reviews"]


def test_sampling_cascade_is_distributed_as_the_target(orc):
    V = 6
    tshape = llama_shape(1, 16, 2, 32, V, 64)
    dshape = llama_shape(1, 8, 1, 16, V, 64)
    prompt = np.array([1, 2, 3, 1, 2, 4, 1, 2], dtype=np.int32)
    nxt = workloads.bigram_table(prompt, V, seed=0)
    t_blob = orc.blob_to_u16(workloads.make_weights(tshape, seed=1, std=1.0))
    d_blob = orc.blob_to_u16(workloads.make_weights(dshape, seed=2, std=1.0))
    tm = orc.Model(tshape, t_blob)

    def law(x):
        x = x.astype(np.float64)
        e = np.exp(x - x.max())
        return e / e.sum()

    p1 = law(tm.review_forward(prompt, 0)[-1])
    joint = np.zeros((V, V))
    for y in range(V):
        joint[y] = p1[y] * law(tm.review_forward([y], len(prompt))[0])
    ms = [orc.Model(tshape, t_blob), orc.Model(dshape, d_blob)]
    counts = np.zeros((V, V))
    N = 12000
    for s in range(N):
        got, _, _ = orc.cascade_generate(ms, prompt, nxt, [[2, 2], [0, 3]], 4, prompt, 2,
                                         temperature=1.0, seed=1000 + s)
        counts[got[0], got[1]] += 1
    keep = joint.ravel() * N > 5
    obs = np.concatenate([counts.ravel()[keep], [counts.ravel()[~keep].sum()]])
    exp = np.concatenate([joint.ravel()[keep], [joint.ravel()[~keep].sum()]]) * N
    if exp[-1] == 0:
        obs, exp = obs[:-1], exp[:-1]
    assert stats.chisquare(obs, exp).pvalue > 0.01


def test_encoder_decoder_cascade_greedy(orc):
    ts = t5_shape(1, 1, 32, 2, 16, 64, 40, 96, 32)
    ds = t5_shape(1, 1, 16, 2, 8, 32, 40, 96, 32)
    enc = workloads.make_repetitive_prompt(40, 24, seed=6)
    nxt = workloads.bigram_table(enc, 40, seed=3)
    start = np.array([0], dtype=np.int32)
    want = target_only_greedy(orc, ts, 41, start, 24, enc=enc)
    ms = models(orc, [ts, ds, ds], [41, 42, 43])
    K = [[2, 2, 0], [0, 1, 4], [0, 0, 4]]      # two neural drafts share the block, Max-Gram below
    got, _, st = orc.cascade_generate(ms, enc, nxt, K, 4, start, 24)
    assert got.tolist() == want
    assert st["reviews"][1] > 0 and st["reviews"][2] > 0 and st["mag_calls"] > 0


def test_capacity_is_checked(orc):
    prompt = workloads.make_prompt(MICRO_T.vocab, 150, seed=1)
    nxt = workloads.bigram_table(prompt, MICRO_T.vocab, seed=1)
    with pytest.raises(ValueError):
        orc.cascade_generate(models(orc, [MICRO_T], [1]), prompt, nxt, [[4]], 4, prompt, 100)


def test_lenience_applies_only_where_a_draft_reviews_a_draft(orc):
    # Section 3.1 / Appendix B: lenience loosens the accept test when a neural draft reviews another
    # neural draft's tokens; never when the target reviews, never for Max-Gram tokens
    V = 48
    prompt = workloads.make_repetitive_prompt(V, 24, seed=2)
    nxt = workloads.bigram_table(prompt, V, seed=2)
    # target + Max-Gram, and target + one draft + Max-Gram: no draft reviews a draft, so lenience
    # cannot change a single token
    for shapes, seeds, K in (([MICRO_T], [7], [[4]]), ([MICRO_T, MICRO_D], [7, 8], [[2, 2], [0, 4]])):
        for seed in range(3):
            a, _, _ = orc.cascade_generate(models(orc, shapes, seeds), prompt, nxt, K, 4, prompt, 16,
                                           temperature=1.0, lenience=1.0, seed=seed)
            b, _, _ = orc.cascade_generate(models(orc, shapes, seeds), prompt, nxt, K, 4, prompt, 16,
                                           temperature=1.0, lenience=6.0, seed=seed)
            assert a.tolist() == b.tolist()
    # two neural drafts: the upper draft reviews the lower one's tokens and accepts more of them under lenience
    K3 = [[3, 0, 0], [0, 3, 0], [0, 0, 3]]
    acc1 = acc6 = 0.0
    for seed in range(12):
        ms = models(orc, [MICRO_T, MICRO_D, MICRO_D], [7, 8, 9])
        _, _, s1 = orc.cascade_generate(ms, prompt, nxt, K3, 4, prompt, 16, temperature=1.0, lenience=1.0, seed=seed)
        ms = models(orc, [MICRO_T, MICRO_D, MICRO_D], [7, 8, 9])
        _, _, s6 = orc.cascade_generate(ms, prompt, nxt, K3, 4, prompt, 16, temperature=1.0, lenience=6.0, seed=seed)
        acc1 += s1["accepted"][1] / max(s1["drafted"][1], 1)
        acc6 += s6["accepted"][1] / max(s6["drafted"][1], 1)
    assert acc6 > acc1
