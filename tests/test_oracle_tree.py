"""Pins of the tree-shaped review (tree attention, Section 5.1 / Appendix B): whatever the tree, the
greedy walk emits exactly the target's own greedy continuation; a chain-shaped tree is the ordinary
review; a node's law does not depend on its siblings."""
import numpy as np
import pytest

import workloads
from workloads import SHAPES


def random_tree(rng, m, lead_children=0):
    parent = [-1]
    for r in range(1, m):
        parent.append(int(rng.integers(0, r)))
    return parent


def lead_tree(levels, children, chain):
    """The shape the paper uses with its decoder-only model: at every level only the lead node has
    children (`children` of them, the first being the next lead), then a chain under the last lead."""
    parent, lead = [-1], 0
    for _ in range(levels):
        first = len(parent)
        parent += [lead] * children
        lead = first
    for _ in range(chain):
        parent.append(lead)
        lead = len(parent) - 1
    return parent


def target_greedy(orc, shape, blob, prompt, n):
    m = orc.Model(shape, blob)
    logits = m.review_forward(prompt, 0)
    out, pos = [], len(prompt)
    tok = int(np.argmax(logits[-1]))
    for _ in range(n):
        out.append(tok)
        logits = m.review_forward([tok], pos)
        pos += 1
        tok = int(np.argmax(logits[0]))
    return out


def test_greedy_walk_is_lossless_on_random_and_lead_trees(orc):
    shape = SHAPES["tiny_draft"]
    blob = orc.blob_to_u16(workloads.make_weights(shape, seed=2, std=0.6))
    prompt = workloads.make_prompt(shape.vocab, 9, seed=1)
    truth = target_greedy(orc, shape, blob, prompt, 12)
    rng = np.random.default_rng(0)
    model = orc.Model(shape, blob)
    model.review_forward(prompt[:-1], 0)
    kv = len(prompt) - 1
    longest = 0
    for trial in range(40):
        parent = random_tree(rng, int(rng.integers(1, 18))) if trial % 2 else lead_tree(2, 4, int(rng.integers(0, 4)))
        paths = orc.tree_paths(parent)
        tokens = np.zeros(len(parent), dtype=np.int32)
        tokens[0] = prompt[-1]
        for r in range(1, len(parent)):
            depth = len(paths[r]) - 1
            # half of the nodes carry the true continuation at their depth, the others noise
            tokens[r] = truth[depth - 1] if rng.random() < 0.6 else int(rng.integers(0, shape.vocab))
        logits = orc.tree_review_forward(model, tokens, parent, kv)
        out, path = orc.tree_accept_greedy(logits, tokens, parent)
        assert list(out) == truth[:len(out)]                     # lossless
        assert len(out) == len(path) and path[0] == 0
        for a, b_ in zip(path, path[1:]):
            assert parent[b_] == a and tokens[b_] == out[path.index(b_) - 1]
        # maximal: the walk stopped because no child of the last node holds the next true token
        last = path[-1]
        assert not any(parent[c] == last and tokens[c] == out[-1] for c in range(len(parent)))
        longest = max(longest, len(out))
    assert longest >= 3


def test_chain_is_the_ordinary_review_and_siblings_do_not_matter(orc):
    shape = SHAPES["tiny_draft"]
    blob = orc.blob_to_u16(workloads.make_weights(shape, seed=3, std=0.3))
    seq = workloads.make_prompt(shape.vocab, 14, seed=4)
    model = orc.Model(shape, blob)
    model.review_forward(seq[:6], 0)
    plain = model.review_forward(seq[6:12], 6)
    chain = orc.tree_review_forward(model, seq[6:12], [-1, 0, 1, 2, 3, 4], 6)
    assert np.allclose(plain, chain, atol=1e-5)
    # the same chain with two extra leaves hanging off it: the chain's rows are unchanged
    tokens = np.concatenate([seq[6:12], seq[12:14]])
    tree = orc.tree_review_forward(model, tokens, [-1, 0, 1, 2, 3, 4, 1, 3], 6)
    assert np.allclose(tree[:6], plain, atol=1e-5)
    # a leaf's law is the law of its own path
    leaf = model.review_forward(np.array([seq[6], seq[7], seq[12]]), 6)[-1]
    assert np.allclose(tree[6], leaf, atol=1e-5)
