"""Batched review: the blocks of several sequences in one pass over the weights, each sequence with
its own cache, ragged block sizes and cache lengths.  Every sequence's logits must match the oracle
run on that sequence alone."""
import numpy as np
import pytest
import torch

import workloads
from workloads import SHAPES, llama_shape
from gpu_util import LOGIT_MAX_ABS, LOGIT_REL_L2, rel_l2, require_gpu, to_dev_i32

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module", params=[0, 1, 2], ids=["automatic", "cuda-core", "tensor-core"])
def b(request):
    require_gpu()
    from paper_2312_11462_b200 import binding
    binding.csd_set_gemm_path(request.param)
    binding.csd_set_attention_path(1 if request.param == 1 else 0)
    yield binding
    binding.csd_set_gemm_path(0)
    binding.csd_set_attention_path(0)


@pytest.mark.parametrize("name", ["tiny_target", "wide", "t5tiny_target"])
def test_ragged_batches_match_per_sequence_oracle(b, orc, name):
    shape = llama_shape(2, 4096, 32, 11008, 2000, 128) if name == "wide" else SHAPES[name]
    blob = workloads.make_weights(shape, seed=21, device="cuda", std=0.02 if name == "wide" else 0.05, gain_std=0.1)
    n_seq = 3
    seqs = [workloads.make_prompt(shape.vocab, 90, seed=40 + i) for i in range(n_seq)]
    gms = [b.Model(shape, blob) for _ in range(n_seq)]
    oms = [orc.Model(shape, orc.blob_to_u16(blob)) for _ in range(n_seq)]
    if shape.arch == 1:
        for i in range(n_seq):
            enc = workloads.make_prompt(shape.vocab, 20 + 7 * i, seed=60 + i)
            gms[i].csd_encoder_forward(to_dev_i32(enc))
            oms[i].encoder_forward(enc)
            seqs[i][0] = 0
    kv = [0, 0, 0]
    # steps with ragged block sizes (5 + 4 + 6, then 1 + 9 + 7, ...), ragged advances (as after acceptances)
    for rows, adv in (((5, 4, 6), (3, 4, 1)), ((1, 9, 7), (1, 2, 7)), ((6, 6, 5), (6, 1, 5)), ((17,), (17,)), ((2, 15), (2, 9))):
        idx = list(range(len(rows)))
        blocks = [to_dev_i32(seqs[i][kv[i]:kv[i] + rows[i]]) for i in idx]
        got = b.csd_review_forward_batch([gms[i] for i in idx], blocks, [kv[i] for i in idx])
        for i in idx:
            ref = oms[i].review_forward(seqs[i][kv[i]:kv[i] + rows[i]], kv[i])
            g = got[i].cpu().numpy()
            assert rel_l2(g, ref) <= LOGIT_REL_L2, (name, rows, i, rel_l2(g, ref))
            assert np.abs(g - ref).max() <= LOGIT_MAX_ABS
            kv[i] += adv[i]                         # the rest of the block is rolled back
    # the batched call and the one-sequence call agree on a sequence
    one = gms[0].csd_review_forward(to_dev_i32(seqs[0][kv[0]:kv[0] + 5]), kv[0]).cpu().numpy()
    both = b.csd_review_forward_batch(gms[:2], [to_dev_i32(seqs[0][kv[0]:kv[0] + 5]), to_dev_i32(seqs[1][kv[1]:kv[1] + 3])],
                                      kv[:2])[0].cpu().numpy()
    assert rel_l2(both, one) <= 1e-4
    assert b.csd_device_status() == 0


def test_batch_argument_errors(b):
    shape = SHAPES["tiny_draft"]
    blob = workloads.make_weights(shape, seed=1, device="cuda")
    other = workloads.make_weights(shape, seed=2, device="cuda")
    m1, m2, m3 = b.Model(shape, blob), b.Model(shape, blob), b.Model(shape, other)
    t = to_dev_i32(np.arange(9))
    with pytest.raises(b.CsdError):
        b.csd_review_forward_batch([m1, m3], [t[:4], t[:4]], [0, 0])        # different weights
    with pytest.raises(b.CsdError):
        b.csd_review_forward_batch([m1, m1], [t[:4], t[:4]], [0, 0])        # the same cache twice
    with pytest.raises(b.CsdError):
        b.csd_review_forward_batch([m1, m2], [t[:9], t[:9]], [0, 0])        # 18 rows
    out = b.csd_review_forward_batch([m1, m2], [t[:8], t[:9]], [0, 0])
    assert out[0].shape[0] == 8 and out[1].shape[0] == 9
