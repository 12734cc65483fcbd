"""Parity of csd_review_forward / csd_encoder_forward with the oracle: logits within
rel-L2 2e-3 and max-abs 5e-2, over blocks of several sizes, rollback and long caches."""
import numpy as np
import pytest
import torch

import workloads
from workloads import SHAPES, llama_shape, t5_shape
from gpu_util import LOGIT_MAX_ABS, LOGIT_REL_L2, rel_l2, require_gpu, to_dev_i32

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module", params=[0, 1, 2, 3], ids=["automatic", "cuda-core", "tensor-core", "tensor-core-row-ranges"])
def b(request):
    """Every test here runs once per kernel family: the automatic choice (small matrices go through the
    CUDA-core kernel), CUDA-core GEMM (128-bit loads + fp32 FMA) with the CUDA-core attention, and
    the two tensor-core GEMMs (TMA + tcgen05) with the tensor-core attention."""
    require_gpu()
    from paper_2312_11462_b200 import binding
    binding.csd_set_gemm_path(request.param)
    binding.csd_set_attention_path(1 if request.param == 1 else 0)
    yield binding
    binding.csd_set_gemm_path(0)
    binding.csd_set_attention_path(0)


def check(got, ref, what):
    got = got.cpu().numpy()
    assert np.isfinite(got).all(), what
    assert rel_l2(got, ref) <= LOGIT_REL_L2, (what, rel_l2(got, ref))
    assert np.abs(got - ref).max() <= LOGIT_MAX_ABS, (what, np.abs(got - ref).max())


def run_blocks(b, orc, shape, blob, toks, blocks, enc=None):
    gm = b.Model(shape, blob)
    om = orc.Model(shape, orc.blob_to_u16(blob))
    if enc is not None:
        gm.csd_encoder_forward(to_dev_i32(enc))
        om.encoder_forward(enc)
    pos = 0
    for m in blocks:
        blk = toks[pos:pos + m]
        got = gm.csd_review_forward(to_dev_i32(blk), pos)
        check(got, om.review_forward(blk, pos), (shape.d_model, pos, m))
        pos += m
    assert b.csd_device_status() == 0
    return gm, om, pos


@pytest.mark.parametrize("name,std", [("tiny_target", 0.02), ("tiny_draft", 0.02), ("tiny_target", 0.08)])
def test_tiny_models(b, orc, name, std):
    shape = SHAPES[name]
    blob = workloads.make_weights(shape, seed=3, device="cuda", std=std, gain_std=0.2)
    toks = workloads.make_prompt(shape.vocab, 120, seed=1)
    gm, om, pos = run_blocks(b, orc, shape, blob, toks, [17, 16, 1, 5, 5, 2, 9, 17, 3])
    # rollback: a rejected block is overwritten by the next call at the same kv_len
    junk = (toks[pos:pos + 5] + 7) % shape.vocab
    gm.csd_review_forward(to_dev_i32(junk), pos)
    om.review_forward(junk, pos)
    blk = toks[pos:pos + 4]
    check(gm.csd_review_forward(to_dev_i32(blk), pos), om.review_forward(blk, pos), "after rollback")


def test_68m_shape_and_long_cache(b, orc):
    shape = workloads.with_max_seq(SHAPES["draft68m"], 700)
    blob = workloads.make_weights(shape, seed=5, device="cuda")
    toks = workloads.make_prompt(shape.vocab, 700, seed=2)
    # a cache long enough for several key tiles and several splits per head
    blocks = [17] * 38 + [5, 9, 2, 17, 1]
    run_blocks(b, orc, shape, blob, toks, blocks)


def test_head_dim_128_and_odd_vocab(b, orc):
    shape = llama_shape(2, 512, 4, 1032, 5003, 300)
    blob = workloads.make_weights(shape, seed=8, device="cuda", std=0.05, gain_std=0.1)
    toks = workloads.make_prompt(shape.vocab, 290, seed=4)
    run_blocks(b, orc, shape, blob, toks, [17] * 16 + [5, 3, 1, 9])


def test_encoder_decoder(b, orc):
    # Unscaled attention scores make random-init encoder-decoder stacks very sensitive: one K/V
    # element whose fp32 and fp64 values fall on different sides of a bf16 rounding boundary moves
    # a head's output by about 1e-2.  Deep stacks are therefore checked with the workload's init
    # (std 0.02), and a one-layer stack with large weights pins the kernels tightly.
    for shape, n_enc, std in ((t5_shape(2, 2, 128, 4, 32, 256, 512, 96, 48), 37, 0.06),
                              (t5_shape(2, 3, 256, 4, 64, 520, 1000, 200, 160), 150, 0.02)):
        blob = workloads.make_weights(shape, seed=9, device="cuda", std=std, gain_std=0.2)
        enc = workloads.make_prompt(shape.vocab, n_enc, seed=6)
        dec = np.concatenate([[0], workloads.make_prompt(shape.vocab, 60, seed=7)]).astype(np.int32)
        run_blocks(b, orc, shape, blob, dec, [1, 5, 17, 2, 9, 17], enc=enc)
    shape = t5_shape(1, 1, 256, 4, 64, 520, 1000, 200, 160)
    blob = workloads.make_weights(shape, seed=9, device="cuda", std=0.06, gain_std=0.2)
    enc = workloads.make_prompt(shape.vocab, 150, seed=6)
    dec = np.concatenate([[0], workloads.make_prompt(shape.vocab, 40, seed=7)]).astype(np.int32)
    gm, om = b.Model(shape, blob), orc.Model(shape, orc.blob_to_u16(blob))
    gm.csd_encoder_forward(to_dev_i32(enc))
    om.encoder_forward(enc)
    pos = 0
    for m in (1, 17, 5, 17):
        got = gm.csd_review_forward(to_dev_i32(dec[pos:pos + m]), pos).cpu().numpy()
        assert rel_l2(got, om.review_forward(dec[pos:pos + m], pos)) < 2e-3
        pos += m


def test_argument_and_token_errors(b):
    shape = SHAPES["tiny_draft"]
    blob = workloads.make_weights(shape, seed=1, device="cuda")
    gm = b.Model(shape, blob)
    toks = to_dev_i32(np.arange(18))
    with pytest.raises(b.CsdError) as e:
        gm.csd_review_forward(toks, 0)                      # 18 rows
    assert e.value.code == 1
    with pytest.raises(b.CsdError) as e:
        gm.csd_review_forward(toks[:5], shape.max_seq - 2)  # would run past the cache
    assert e.value.code == 3
    bad = to_dev_i32([1, 2, shape.vocab, 3])
    out = gm.csd_review_forward(bad, 0)
    assert b.csd_device_status() == 6 and torch.isfinite(out).all()
    with pytest.raises(b.CsdError):
        b.Model(shape, blob[:-128])                         # blob too small


@pytest.mark.parametrize("d_head", [32, 64, 128])
def test_tile_edges_of_the_attention(b, orc, d_head):
    # One layer, so that the logits follow the attention closely; block sizes chosen so that the
    # cache length before a block, and the end of the block, fall before, on and after the 64-key
    # tile edges and the split boundaries (1, 2, 3 ... tiles, odd remainders, a 17-row block that
    # straddles a tile edge, a block that starts exactly on one).
    shape = llama_shape(1, 2 * d_head, 2, 4 * d_head, 512, 600)
    blob = workloads.make_weights(shape, seed=17, device="cuda", std=0.08, gain_std=0.2)
    toks = workloads.make_prompt(shape.vocab, 600, seed=4)
    blocks = [1, 17, 17, 17, 11, 1, 1, 16, 17, 14, 1, 2, 17, 17, 17, 13, 1, 5, 17, 17, 17, 17, 9, 17,
              17, 17, 17, 17, 17, 16, 1, 3, 17, 17, 17, 17, 5]
    assert sum(blocks) <= 600
    run_blocks(b, orc, shape, blob, toks, blocks)
