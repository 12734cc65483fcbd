"""Tree-shaped review on the GPU (tree attention, Section 5.1 / Appendix B): csd_review_forward_tree
against the oracle's one-forward-per-path definition, csd_tree_accept_greedy against the oracle's
walk on the same logits, and the greedy walk's losslessness on the GPU path itself."""
import numpy as np
import pytest
import torch

import workloads
from workloads import SHAPES, llama_shape
from gpu_util import LOGIT_MAX_ABS, LOGIT_REL_L2, rel_l2, require_gpu, to_dev_i32
from test_oracle_tree import lead_tree, random_tree

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module", params=[0, 1], ids=["tensor-core-attention", "cuda-core-attention"])
def b(request):
    require_gpu()
    from paper_2312_11462_b200 import binding
    binding.csd_set_attention_path(request.param)
    yield binding
    binding.csd_set_attention_path(0)


@pytest.mark.parametrize("shape_name", ["tiny_target", "tiny_draft", "dh128"])
def test_tree_forward_matches_the_per_path_definition(b, orc, shape_name):
    shape = llama_shape(2, 256, 2, 512, 1000, 200) if shape_name == "dh128" else SHAPES[shape_name]
    blob = workloads.make_weights(shape, seed=11, device="cuda", std=0.05, gain_std=0.1)
    toks = workloads.make_prompt(shape.vocab, 160, seed=2)
    rng = np.random.default_rng(5)
    gm, om = b.Model(shape, blob), orc.Model(shape, orc.blob_to_u16(blob))
    for kv in (0, 3, 61, 64, 70, 130):            # empty cache, and caches that end before, on and after a key tile
        if kv:
            gm.csd_prefill(to_dev_i32(toks[:kv]), 0)
            pos = 0
            while pos < kv:
                n = min(17, kv - pos)
                om.review_forward(toks[pos:pos + n], pos)
                pos += n
        for parent in (lead_tree(1, 8, 3), random_tree(rng, 17), random_tree(rng, 6), [-1], lead_tree(2, 4, 2)):
            m = len(parent)
            tokens = rng.integers(0, shape.vocab, size=m).astype(np.int32)
            got = gm.csd_review_forward_tree(to_dev_i32(tokens), parent, kv).cpu().numpy()
            ref = orc.tree_review_forward(om, tokens, parent, kv)
            assert rel_l2(got, ref) <= LOGIT_REL_L2, (kv, parent, rel_l2(got, ref))
            assert np.abs(got - ref).max() <= LOGIT_MAX_ABS
    # a chain is the ordinary review, bit for bit
    blk = to_dev_i32(toks[130:139])
    assert torch.equal(gm.csd_review_forward_tree(blk, [-1, 0, 1, 2, 3, 4, 5, 6, 7], 130), gm.csd_review_forward(blk, 130))
    assert b.csd_device_status() == 0


def test_tree_accept_walk_and_losslessness(b, orc):
    shape = SHAPES["tiny_target"]
    blob = workloads.make_weights(shape, seed=2, device="cpu", std=0.6)
    prompt = workloads.make_prompt(shape.vocab, 20, seed=1)
    gm = b.Model(shape, blob.cuda())
    # the GPU path's own greedy continuation
    gm.csd_prefill(to_dev_i32(prompt[:-1]), 0)
    truth, pos, tok = [], len(prompt) - 1, int(prompt[-1])
    for _ in range(14):
        tok_next = int(gm.csd_review_forward(to_dev_i32([tok]), pos)[0].argmax())
        truth.append(tok_next)
        tok, pos = tok_next, pos + 1
    rng = np.random.default_rng(3)
    kv = len(prompt) - 1
    best = 0
    for trial in range(30):
        parent = lead_tree(2, 8, 0) if trial % 3 == 0 else (lead_tree(1, 8, 3) if trial % 3 == 1 else random_tree(rng, 17))
        paths = orc.tree_paths(parent)
        tokens = np.zeros(len(parent), dtype=np.int32)
        tokens[0] = prompt[-1]
        for r in range(1, len(parent)):
            d = len(paths[r]) - 1
            tokens[r] = truth[d - 1] if rng.random() < 0.6 else int(rng.integers(0, shape.vocab))
        logits = gm.csd_review_forward_tree(to_dev_i32(tokens), parent, kv)
        out, path, n_valid = b.csd_tree_accept_greedy(logits, to_dev_i32(tokens), parent)
        want_out, want_path = orc.tree_accept_greedy(logits.cpu().numpy(), tokens, parent)   # same logits: exact
        assert out.tolist() == want_out.tolist() and path.tolist() == list(want_path)
        assert out.tolist() == truth[:len(out)]                                              # lossless
        chain = 0
        while chain < len(path) and path[chain] == chain:
            chain += 1
        assert n_valid == chain >= 1
        best = max(best, len(out))
    assert best >= 3
    # arguments: a parent that does not precede its child, a root with a parent
    from paper_2312_11462_b200.binding import CsdError
    with pytest.raises(CsdError):
        gm.csd_review_forward_tree(to_dev_i32([1, 2, 3]), [-1, 2, 0], kv)
    with pytest.raises(CsdError):
        gm.csd_review_forward_tree(to_dev_i32([1, 2]), [0, 0], kv)
    assert b.csd_device_status() == 0
