"""End-to-end parity of csd_cascade_generate with the oracle's Algorithm 1.

Tokens are compared up to the first generated position where the oracle's top-2 logit margin
drops below 0.05 (there a rounding-level logit difference may legitimately flip the arg-max);
beyond that point the GPU path is checked teacher-forced on the oracle's tokens, and in any
case its greedy output must equal its own target-only greedy decoding (losslessness)."""
import numpy as np
import pytest
import torch

import workloads
from workloads import SHAPES
from gpu_util import LOGIT_MAX_ABS, LOGIT_REL_L2, rel_l2, require_gpu, to_dev_i32

pytestmark = pytest.mark.gpu
MARGIN = 0.05


@pytest.fixture(scope="module")
def b():
    require_gpu()
    from paper_2312_11462_b200 import binding
    return binding


def gpu_target_only_greedy(b, shape, blob, prompt, n_new):
    m = b.Model(shape, blob)
    pos = 0
    logits = None
    while pos < len(prompt):
        blk = prompt[pos:pos + 16]
        logits = m.csd_review_forward(to_dev_i32(blk), pos)
        pos += len(blk)
    out = []
    tok = int(logits[-1].argmax())
    for _ in range(n_new):
        out.append(tok)
        logits = m.csd_review_forward(to_dev_i32([tok]), pos)
        pos += 1
        tok = int(logits[0].argmax())
    return out


def agreed_prefix(got, want, margins):
    safe = len(want)
    low = np.nonzero(margins < MARGIN)[0]
    if low.size:
        safe = int(low[0])
    assert list(got[:safe]) == list(want[:safe]), (safe, got[:safe + 2], want[:safe + 2])
    return safe


@pytest.mark.parametrize("K,max_block", [([[4, 0], [0, 4]], 4), ([[2, 10], [0, 10]], 16), ([[0, 6], [0, 0]], 6)])
def test_tiny_cascade_greedy(b, orc, K, max_block):
    ts, ds = SHAPES["tiny_target"], SHAPES["tiny_draft"]
    tb = workloads.make_weights(ts, seed=0, device="cuda")
    db = workloads.make_weights(ds, seed=1, device="cuda")
    prompt = workloads.make_prompt(ts.vocab, 32, seed=0)
    nxt = workloads.bigram_table(prompt, ts.vocab, seed=0)
    oms = [orc.Model(ts, orc.blob_to_u16(tb)), orc.Model(ds, orc.blob_to_u16(db))]
    want, margins, ost = orc.cascade_generate(oms, prompt, nxt, K, max_block, prompt, 64)
    gms = [b.Model(ts, tb), b.Model(ds, db)]
    casc = b.Cascade(gms, K, max_block, to_dev_i32(nxt), 64)
    got, st = casc.csd_cascade_generate(prompt, prompt, 64)
    assert len(got) == 64 and st["tokens"] == 64
    safe = agreed_prefix(got, want, margins)
    assert safe >= 1
    # losslessness on the GPU path itself, whatever the margins
    assert list(got) == gpu_target_only_greedy(b, ts, tb, prompt, 64)
    # a second run is bit-identical
    got2, _ = casc.csd_cascade_generate(prompt, prompt, 64)
    assert np.array_equal(got, got2)
    if safe == 64:
        assert st["reviews"][0] == ost["reviews"][0] and st["mag_calls"] == ost["mag_calls"]
    assert st["kernel_launches"] > 0 and st["decode_ms"] > 0


@pytest.mark.parametrize("seed", [0, 1])
@pytest.mark.parametrize("K,max_block", [([[4, 0], [0, 4]], 4), ([[2, 10], [0, 10]], 16)])
def test_tiny_cascade_greedy_with_wide_margins(b, orc, seed, K, max_block):
    # Weights drawn on the host with a wide spread (std 0.6), seeds for which the oracle's top-2
    # margin stays above 0.05 on all 64 steps (found with the oracle alone): here the whole
    # generation, not a short prefix, must equal the oracle's token for token.
    ts, ds = SHAPES["tiny_target"], SHAPES["tiny_draft"]
    tb = workloads.make_weights(ts, seed=seed, device="cpu", std=0.6)
    db = workloads.make_weights(ds, seed=seed + 100, device="cpu", std=0.6)
    prompt = workloads.make_prompt(ts.vocab, 32, seed=seed)
    nxt = workloads.bigram_table(prompt, ts.vocab, seed=0)
    oms = [orc.Model(ts, orc.blob_to_u16(tb)), orc.Model(ds, orc.blob_to_u16(db))]
    want, margins, ost = orc.cascade_generate(oms, prompt, nxt, K, max_block, prompt, 64)
    gms = [b.Model(ts, tb.cuda()), b.Model(ds, db.cuda())]
    got, st = b.Cascade(gms, K, max_block, to_dev_i32(nxt), 64).csd_cascade_generate(prompt, prompt, 64)
    safe = agreed_prefix(got, want, margins)
    assert safe >= 32, (safe, float(margins.min()))
    if safe == 64:
        assert st["reviews"] == ost["reviews"] and st["accepted"] == ost["accepted"]
        assert st["mag_calls"] == ost["mag_calls"]


def test_accepting_cascade_and_repetitive_prompt(b, orc):
    # draft == target: every drafted token the target sees is accepted, so blocks really commit
    ts = SHAPES["tiny_target"]
    tb = workloads.make_weights(ts, seed=4, device="cuda", std=0.05)
    prompt = workloads.make_repetitive_prompt(ts.vocab, 48, seed=2)
    nxt = workloads.bigram_table(prompt, ts.vocab, seed=0)
    K = [[3, 2], [0, 5]]
    oms = [orc.Model(ts, orc.blob_to_u16(tb)) for _ in range(2)]
    want, margins, ost = orc.cascade_generate(oms, prompt, nxt, K, 5, prompt, 48)
    gms = [b.Model(ts, tb), b.Model(ts, tb)]
    got, st = b.Cascade(gms, K, 5, to_dev_i32(nxt), 64).csd_cascade_generate(prompt, prompt, 48)
    agreed_prefix(got, want, margins)
    assert list(got) == gpu_target_only_greedy(b, ts, tb, prompt, 48)
    assert st["accepted"][0] > 0


def test_dynamic_haystack_cascade(b, orc):
    # Max-Gram may match inside the generation (Section 3.3).  A 24-token vocabulary makes the
    # generated text repeat itself, and a draft equal to the target accepts what the matches propose:
    # with the dynamic haystack more Max-Gram tokens survive the draft's review than with the static one.
    from workloads import llama_shape
    ts = llama_shape(2, 64, 2, 128, 24, 200)
    tb = workloads.make_weights(ts, seed=3, device="cpu", std=0.6)    # seed with wide margins on all 80 steps
    prompt = workloads.make_prompt(ts.vocab, 12, seed=3)
    nxt = workloads.bigram_table(prompt, ts.vocab, seed=0)
    K = [[3, 3], [0, 6]]
    accepted = {}
    for dyn in (False, True):
        oms = [orc.Model(ts, orc.blob_to_u16(tb)) for _ in range(2)]
        want, margins, ost = orc.cascade_generate(oms, prompt, nxt, K, 6, prompt, 80, dynamic_haystack=dyn)
        gms = [b.Model(ts, tb.cuda()), b.Model(ts, tb.cuda())]
        got, st = b.Cascade(gms, K, 6, to_dev_i32(nxt), 64).csd_cascade_generate(prompt, prompt, 80, dynamic_haystack=dyn)
        assert agreed_prefix(got, want, margins) == 80
        assert st["reviews"] == ost["reviews"] and st["accepted"] == ost["accepted"] and st["mag_calls"] == ost["mag_calls"]
        assert list(got) == gpu_target_only_greedy(b, ts, tb.cuda(), prompt, 80)      # lossless either way
        accepted[dyn] = st["accepted"][1]
    assert accepted[True] > accepted[False]
    assert b.csd_device_status() == 0


def test_teacher_forced_logits_follow_the_oracle(b, orc):
    ts = SHAPES["tiny_target"]
    tb = workloads.make_weights(ts, seed=0, device="cuda")
    prompt = workloads.make_prompt(ts.vocab, 32, seed=0)
    nxt = workloads.bigram_table(prompt, ts.vocab, seed=0)
    om = orc.Model(ts, orc.blob_to_u16(tb))
    want, _, _ = orc.cascade_generate([om], prompt, nxt, [[4]], 4, prompt, 64)
    seq = np.concatenate([prompt, want]).astype(np.int32)
    gm = b.Model(ts, tb)
    om2 = orc.Model(ts, orc.blob_to_u16(tb))
    pos = 0
    while pos < len(seq):
        blk = seq[pos:pos + 5]
        got = gm.csd_review_forward(to_dev_i32(blk), pos).cpu().numpy()
        ref = om2.review_forward(blk, pos)
        assert rel_l2(got, ref) <= LOGIT_REL_L2 and np.abs(got - ref).max() <= LOGIT_MAX_ABS
        pos += len(blk)


@pytest.mark.parametrize("lenience", [1.0, 3.0])
def test_sampling_cascade_matches_oracle_decisions(b, orc, lenience):
    # same Philox stream, same laws => same accepted counts and tokens while logits agree.
    # With lenience > 1 (Section 3.1) a second neural draft sits below the first, so that a draft
    # reviews a draft's tokens, the one place where lenience applies (Appendix B).
    ts, ds = SHAPES["tiny_target"], SHAPES["tiny_draft"]
    blobs = [workloads.make_weights(ts, seed=0, device="cuda", std=0.05),
             workloads.make_weights(ds, seed=1, device="cuda", std=0.05)]
    shapes = [ts, ds]
    K = [[2, 2], [0, 3]]
    if lenience > 1.0:
        blobs.append(workloads.make_weights(ds, seed=2, device="cuda", std=0.05))
        shapes.append(ds)
        K = [[2, 1, 1], [0, 2, 2], [0, 0, 3]]
    prompt = workloads.make_repetitive_prompt(ts.vocab, 32, seed=5)
    nxt = workloads.bigram_table(prompt, ts.vocab, seed=0)
    agree = 0
    for seed in range(6):
        oms = [orc.Model(sh, orc.blob_to_u16(w)) for sh, w in zip(shapes, blobs)]
        want, _, ost = orc.cascade_generate(oms, prompt, nxt, K, 4, prompt, 24, temperature=1.0, lenience=lenience,
                                             seed=seed)
        gms = [b.Model(sh, w) for sh, w in zip(shapes, blobs)]
        got, st = b.Cascade(gms, K, 4, to_dev_i32(nxt), 64).csd_cascade_generate(prompt, prompt, 24, 1.0, lenience, seed)
        assert len(got) == 24 and ((got >= 0) & (got < ts.vocab)).all()
        if np.array_equal(got, want):
            agree += 1
        else:
            # a sampled token can differ only where a uniform falls within fp32 logit noise of a
            # threshold: the oracle must have flagged such a decision at or before the first difference
            first = int(np.nonzero(got != want)[0][0])
            assert ost["near_ties"] > 0 and ost["first_near_tie"] <= first, (seed, first, ost)
    assert agree >= 4


def test_encoder_decoder_cascade(b, orc):
    ts, ds = SHAPES["t5tiny_target"], SHAPES["t5tiny_draft"]
    tb = workloads.make_weights(ts, seed=3, device="cuda", std=0.06)
    db = workloads.make_weights(ds, seed=4, device="cuda", std=0.06)
    enc = workloads.make_repetitive_prompt(ts.vocab, 40, seed=1)
    nxt = workloads.bigram_table(enc, ts.vocab, seed=0)
    K = [[2, 2, 0], [0, 1, 4], [0, 0, 4]]
    start = np.array([0], dtype=np.int32)
    oms = [orc.Model(ts, orc.blob_to_u16(tb)), orc.Model(ds, orc.blob_to_u16(db)), orc.Model(ds, orc.blob_to_u16(db))]
    want, margins, _ = orc.cascade_generate(oms, enc, nxt, K, 4, start, 40)
    gms = [b.Model(ts, tb), b.Model(ds, db), b.Model(ds, db)]
    got, st = b.Cascade(gms, K, 4, to_dev_i32(nxt), 48).csd_cascade_generate(enc, start, 40)
    agreed_prefix(got, want, margins)
    assert st["reviews"][1] > 0 and st["reviews"][2] > 0


def test_capacity_errors(b):
    ts = SHAPES["tiny_target"]
    tb = workloads.make_weights(ts, seed=0, device="cuda")
    prompt = workloads.make_prompt(ts.vocab, 100, seed=0)
    nxt = to_dev_i32(workloads.bigram_table(prompt, ts.vocab, seed=0))
    casc = b.Cascade([b.Model(ts, tb)], [[4]], 4, nxt, 128)
    with pytest.raises(b.CsdError) as e:
        casc.csd_cascade_generate(prompt, prompt, 100)
    assert e.value.code == 3
