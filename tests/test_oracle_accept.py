"""Pins the oracle's review rule (Section 2, Section 3.1) to what the mathematics fixes.

The exact laws used below are derived here from the statement of the rule, not from the
oracle: with draft law q_i and target law p_i at position i,
  P(x_i accepted | reached) = alpha_i = sum_x min(q_i(x), l * p_i(x)),
  the token emitted at the first rejection follows norm(max(0, p_i - q_i)),
  and after k acceptances one more token follows p_{k+1}.
"""
import numpy as np
import pytest
from scipy import stats

import workloads


def softmax(x):
    x = np.asarray(x, dtype=np.float64)
    e = np.exp(x - x.max(axis=-1, keepdims=True))
    return e / e.sum(axis=-1, keepdims=True)


def chi2_p(counts, probs):
    counts = np.asarray(counts, dtype=np.float64).ravel()
    probs = np.asarray(probs, dtype=np.float64).ravel()
    keep = probs > 0
    assert counts[~keep].sum() == 0, "mass observed where the exact law has none"
    exp = probs[keep] / probs[keep].sum() * counts.sum()
    return stats.chisquare(counts[keep], exp).pvalue


def run_trials(orc, t, d, n_trials, seed, lenience=1.0, onehot_tokens=None, temperature=1.0):
    """Same logits in every row; tokens drawn from the draft law by this harness."""
    k = t.shape[0] - 1
    V = t.shape[1]
    rng = np.random.default_rng(seed)
    if onehot_tokens is None:
        q = softmax(d / temperature)
        tok = np.stack([rng.choice(V, size=n_trials, p=q[i]) for i in range(k)], axis=1)
        dl = np.broadcast_to(d, (n_trials, k, V))
    else:
        tok = np.broadcast_to(np.asarray(onehot_tokens), (n_trials, k))
        dl = None
    tl = np.broadcast_to(t, (n_trials, k + 1, V))
    n, o, f = orc.spec_accept(tl, dl, tok, temperature, lenience, seed=seed, step=5)
    return tok.astype(np.int64), n.astype(np.int64), o.astype(np.int64), f


def exact_joint(p, q, lenience=1.0):
    """P(n_acc = i, out = y) for independent positions; p [k+1,V], q [k,V]."""
    k, V = q.shape
    out = np.zeros((k + 1, V))
    reach = 1.0
    for i in range(k):
        alpha = np.minimum(q[i], lenience * p[i]).sum()
        r = np.maximum(p[i] - q[i], 0.0)
        r = r / r.sum() if r.sum() > 0 else p[i]
        out[i] = reach * (1.0 - alpha) * r
        reach *= alpha
    out[k] = reach * p[k]
    return out


def test_bruteforce_joint_law_v8_k2(orc):
    V, k, N = 8, 2, 400_000
    t, d = workloads.small_logits(1, k, V, seed=11, scale=1.5)
    t, d = t[0], d[0]
    p, q = softmax(t), softmax(d)
    tok, n, o, _ = run_trials(orc, t, d, N, seed=3)
    joint = np.zeros((k + 1, V))
    np.add.at(joint, (n, o), 1)
    assert chi2_p(joint, exact_joint(p, q)) > 0.01
    # accepted first token: P(n >= 1, x_1 = x) = min(p_1, q_1)(x)
    acc1 = np.bincount(tok[n >= 1, 0], minlength=V)
    cells = np.concatenate([acc1, [N - acc1.sum()]])
    law = np.concatenate([np.minimum(p[0], q[0]), [1 - np.minimum(p[0], q[0]).sum()]])
    assert chi2_p(cells, law) > 0.01
    # losslessness: the first emitted token follows p_1, the second p_2 (positions independent)
    y1 = np.where(n >= 1, tok[:, 0], o)
    assert chi2_p(np.bincount(y1, minlength=V), p[0]) > 0.01
    y2 = np.where(n >= 2, tok[:, 1], o)[n >= 1]
    assert chi2_p(np.bincount(y2, minlength=V), p[1]) > 0.01
    # the third emitted token exists only after two acceptances and follows p_3
    y3 = o[n == 2]
    assert chi2_p(np.bincount(y3, minlength=V), p[2]) > 0.01


def test_accept_and_resample_draws_are_independent(orc):
    # if one uniform drove both the accept test and the resample, the resampled token would be
    # skewed toward the top of the vocabulary order after a rejection; check within strata of x_1
    V, k, N = 8, 1, 300_000
    t, d = workloads.small_logits(1, k, V, seed=5, scale=2.0)
    p, q = softmax(t[0]), softmax(d[0])
    tok, n, o, _ = run_trials(orc, t[0], d[0], N, seed=9)
    r = np.maximum(p[0] - q[0], 0)
    r /= r.sum()
    for x in range(V):
        sel = (tok[:, 0] == x) & (n == 0)
        if sel.sum() > 2000:
            assert chi2_p(np.bincount(o[sel], minlength=V), r) > 0.001


def test_accepted_length_law_eq1(orc):
    # Theorem 1: with a constant acceptance rate alpha, P(i tokens emitted) = alpha^(i-1)(1-alpha)
    # for i <= k and alpha^k for i = k+1; mean (1 - alpha^(k+1)) / (1 - alpha).
    V, k, N = 16, 4, 300_000
    t1, d1 = workloads.small_logits(1, 1, V, seed=21, scale=1.0)
    t = np.repeat(t1[0][:1], k + 1, axis=0)
    d = np.repeat(d1[0][:1], k, axis=0)
    alpha = np.minimum(softmax(t[0]), softmax(d[0])).sum()
    _, n, _, _ = run_trials(orc, t, d, N, seed=2)
    law = np.array([alpha ** i * (1 - alpha) for i in range(k)] + [alpha ** k])
    assert chi2_p(np.bincount(n, minlength=k + 1), law) > 0.01
    mean_emitted = (n + 1).mean()
    closed = (1 - alpha ** (k + 1)) / (1 - alpha)
    assert abs(mean_emitted - closed) < 4 * np.sqrt((n + 1).var() / N)
    # the probability generating function of Eq. 1 at a test point
    x = 0.7
    phi = 1 + (x - 1) * (1 - alpha ** (k + 1) * x ** (k + 1)) / (1 - alpha * x)
    assert abs(np.mean(x ** (n + 1)) - phi) < 5e-3


def test_per_position_acceptance_product(orc):
    # Corollary of Theorem 3: the i-th drafted token survives with probability prod_{j<=i} alpha_j
    V, k, N = 12, 3, 300_000
    t, d = workloads.small_logits(1, k, V, seed=33, scale=1.2)
    p, q = softmax(t[0]), softmax(d[0])
    alphas = np.minimum(p[:k], q).sum(axis=1)
    _, n, _, _ = run_trials(orc, t[0], d[0], N, seed=4)
    for i in range(1, k + 1):
        want = np.prod(alphas[:i])
        got = (n >= i).mean()
        assert abs(got - want) < 4 * np.sqrt(want * (1 - want) / N)


def test_lenience_accept_rate(orc):
    V, k, N = 8, 1, 200_000
    t, d = workloads.small_logits(1, k, V, seed=8, scale=2.0)
    p, q = softmax(t[0]), softmax(d[0])
    for l in (1.0, 2.0, 5.0):
        _, n, _, _ = run_trials(orc, t[0], d[0], N, seed=6, lenience=l)
        want = np.minimum(q[0], l * p[0]).sum()
        assert abs((n == 1).mean() - want) < 4 * np.sqrt(want * (1 - want) / N + 1e-12) + 1e-9


def test_temperature(orc):
    V, k, N = 8, 1, 200_000
    t, d = workloads.small_logits(1, k, V, seed=13, scale=2.0)
    T = 0.5
    p, q = softmax(t[0] / T), softmax(d[0] / T)
    tok, n, o, _ = run_trials(orc, t[0], d[0], N, seed=7, temperature=T)
    y1 = np.where(n >= 1, tok[:, 0], o)
    assert chi2_p(np.bincount(y1, minlength=V), p[0]) > 0.01
    want = np.minimum(p[0], q[0]).sum()
    assert abs((n == 1).mean() - want) < 4 * np.sqrt(want * (1 - want) / N)


def test_point_mass_draft(orc):
    # statistical drafter: q is the point mass on x, so x is accepted with probability p(x) and
    # the resample follows p with x removed
    V, N, x = 8, 200_000, 3
    t, _ = workloads.small_logits(1, 1, V, seed=17, scale=1.0)
    p = softmax(t[0])
    _, n, o, _ = run_trials(orc, t[0], None, N, seed=12, onehot_tokens=[x])
    assert abs((n == 1).mean() - p[0][x]) < 4 * np.sqrt(p[0][x] * (1 - p[0][x]) / N)
    res = p[0].copy()
    res[x] = 0
    res /= res.sum()
    assert chi2_p(np.bincount(o[n == 0], minlength=V), res) > 0.01
    y1 = np.where(n >= 1, x, o)
    assert chi2_p(np.bincount(y1, minlength=V), p[0]) > 0.01
    # the explicit per-position flag is the same thing as passing no draft logits
    tl = np.broadcast_to(t[0], (1000, 2, V))
    dl = np.zeros((1000, 1, V), dtype=np.float32)
    tok = np.full((1000, 1), x)
    a = orc.spec_accept(tl, None, tok, 1.0, seed=1)
    b = orc.spec_accept(tl, dl, tok, 1.0, seed=1, onehot=np.ones((1000, 1)))
    assert (a[0] == b[0]).all() and (a[1] == b[1]).all()


def test_special_cases(orc):
    V, k = 32, 4
    rng = np.random.default_rng(0)
    t = rng.standard_normal((50, k + 1, V)).astype(np.float32)
    # q == p: every draft is accepted whatever the uniform
    tok = rng.integers(0, V, size=(50, k))
    n, o, _ = orc.spec_accept(t, t[:, :k], tok, 1.0, seed=4)
    assert (n == k).all() and ((o >= 0) & (o < V)).all()
    # k = 0: plain sampling from the target law
    t0 = np.broadcast_to(t[0, :1], (100_000, 1, V))
    n0, o0, _ = orc.spec_accept(t0, np.zeros((100_000, 0, V), np.float32), np.zeros((100_000, 0)), 1.0, seed=2)
    assert (n0 == 0).all()
    assert chi2_p(np.bincount(o0, minlength=V), softmax(t[0, 0])) > 0.01
    # a token the target gives zero mass is never accepted
    tz = t.copy()
    tz[:, 0, 5] = -np.inf
    nz, oz, _ = orc.spec_accept(tz, None, np.full((50, k), 5), 1.0, seed=4)
    assert (nz == 0).all() and (oz != 5).all()
    # draws are a pure function of (seed, step, row, position)
    b1 = orc.spec_accept(t[10:11], None, tok[10:11], 1.0, seed=4, step=9)
    b2 = orc.spec_accept(t[10:11], None, tok[10:11], 1.0, seed=4, step=9)
    assert (b1[0] == b2[0]).all() and (b1[1] == b2[1]).all()


def test_greedy(orc):
    V, k = 64, 5
    rng = np.random.default_rng(1)
    t = rng.standard_normal((200, k + 1, V)).astype(np.float32)
    am = t.argmax(axis=-1)
    tok = am[:, :k].copy()
    cut = rng.integers(0, k + 1, size=200)
    for r in range(200):
        if cut[r] < k:
            tok[r, cut[r]] = (tok[r, cut[r]] + 1) % V
    n, o, _ = orc.spec_accept(t, None, tok, 0.0)
    assert (n == cut).all()
    assert (o == am[np.arange(200), cut]).all()
    # ties resolve to the smallest index
    tt = np.zeros((1, 2, V), dtype=np.float32)
    n, o, _ = orc.spec_accept(tt, None, np.array([[0]]), 0.0)
    assert n[0] == 1 and o[0] == 0


def test_bad_arguments(orc):
    t = np.zeros((1, 2, 4), dtype=np.float32)
    with pytest.raises(ValueError):
        orc.spec_accept(t, None, np.zeros((1, 1)), 1.0, lenience=0.5)
    with pytest.raises(ValueError):
        orc.spec_accept(t, None, np.zeros((1, 1)), -1.0)


def test_no_lenience_for_point_mass_positions(orc):
    # Appendix B: lenience is not used between the statistical drafter and its reviewer
    V, N, x = 8, 50_000, 2
    t, d = workloads.small_logits(1, 2, V, seed=23, scale=1.5)
    tl = np.broadcast_to(t[0], (N, 3, V))
    dl = np.broadcast_to(d[0], (N, 2, V))
    tok = np.broadcast_to(np.array([x, x]), (N, 2))
    # all point mass: any lenience gives the very same outcome as lenience 1
    a = orc.spec_accept(tl, None, tok, 1.0, lenience=1.0, seed=3)
    b = orc.spec_accept(tl, None, tok, 1.0, lenience=7.0, seed=3)
    assert (a[0] == b[0]).all() and (a[1] == b[1]).all()
    # mixed block: position 0 carries a law (lenience applies), position 1 is a point mass (it does not)
    p, q = softmax(t[0]), softmax(d[0])
    oh = np.broadcast_to(np.array([0, 1]), (N, 2))
    l = 3.0
    n, _, _ = orc.spec_accept(tl, dl, tok, 1.0, lenience=l, seed=4, onehot=oh)
    a0 = min(1.0, l * p[0][x] / q[0][x])        # P(position 0 accepted | x drawn) under lenience
    a1 = p[1][x]                                 # point mass: accepted with probability p(x), no lenience
    assert abs((n >= 1).mean() - a0) < 4 * np.sqrt(a0 * (1 - a0) / N + 1e-12) + 1e-9
    assert abs((n == 2).mean() - a0 * a1) < 4 * np.sqrt(a0 * a1 * (1 - a0 * a1) / N)
