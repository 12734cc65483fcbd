"""Parity at the workloads' own sizes: the 7B-shaped target with its 68M-shaped draft (cascade
on a short prompt, because the oracle needs ~6 s of host time per target row block), and the
long-cache review (2048+ cached positions, head dimension 128, blocks of 2/5/9/17 rows) on a
narrower model that the oracle can prefill in seconds."""
import numpy as np
import pytest
import torch

import workloads
from workloads import SHAPES, llama_shape, t5_shape
from gpu_util import LOGIT_MAX_ABS, LOGIT_REL_L2, rel_l2, require_gpu, to_dev_i32

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def b():
    require_gpu()
    from paper_2312_11462_b200 import binding
    return binding


def test_7b_shaped_cascade_and_logits(b, orc):
    ts, ds = SHAPES["llama7b"], SHAPES["draft68m"]
    tb = workloads.make_weights(ts, seed=100, device="cuda")
    db = workloads.make_weights(ds, seed=101, device="cuda")
    prompt = workloads.make_prompt(ts.vocab, 12, seed=1000)
    nxt = workloads.bigram_table(prompt, ts.vocab, seed=7)
    K, max_block, n_new = [[4, 0], [0, 4]], 4, 6
    oms = [orc.Model(ts, orc.blob_to_u16(tb)), orc.Model(ds, orc.blob_to_u16(db))]
    want, margins, ost = orc.cascade_generate(oms, prompt, nxt, K, max_block, prompt, n_new)
    gms = [b.Model(ts, tb), b.Model(ds, db)]
    got, st = b.Cascade(gms, K, max_block, to_dev_i32(nxt), 128).csd_cascade_generate(prompt, prompt, n_new)
    low = np.nonzero(margins < 0.05)[0]
    safe = int(low[0]) if low.size else n_new
    assert list(got[:safe]) == list(want[:safe])
    assert b.csd_device_status() == 0
    # (the 32-layer stack's logits are compared in test_7b_width_depth_sweep)


@pytest.mark.parametrize("path", [1, 2, 3], ids=["cuda-core", "tensor-core", "tensor-core-row-ranges"])
def test_7b_width_shallow_stack(b, orc, path):
    # the 7B layer shapes (d 4096, 32 heads x 128, ffn 11008, vocabulary 32000) in a 3-layer stack
    shape = llama_shape(3, 4096, 32, 11008, 32000, 64)
    blob = workloads.make_weights(shape, seed=100, device="cuda")
    seq = workloads.make_prompt(shape.vocab, 24, seed=1000)
    b.csd_set_gemm_path(path)
    b.csd_set_attention_path(1 if path == 1 else 0)
    try:
        gm, om = b.Model(shape, blob), orc.Model(shape, orc.blob_to_u16(blob))
        for pos, m in ((0, 17), (17, 5), (22, 1)):
            blk = seq[pos:pos + m]
            g = gm.csd_review_forward(to_dev_i32(blk), pos).cpu().numpy()
            r = om.review_forward(blk, pos)
            assert rel_l2(g, r) <= LOGIT_REL_L2, (pos, rel_l2(g, r))
            assert np.abs(g - r).max() <= LOGIT_MAX_ABS
        assert b.csd_device_status() == 0
    finally:
        b.csd_set_gemm_path(0)
        b.csd_set_attention_path(0)


@pytest.mark.parametrize("attn_path", [0, 1], ids=["tensor-core-attention", "cuda-core-attention"])
def test_long_cache_review_blocks(b, orc, attn_path):
    b.csd_set_attention_path(attn_path)
    try:
        long_cache_review_blocks(b, orc)
    finally:
        b.csd_set_attention_path(0)


def long_cache_review_blocks(b, orc):
    shape = llama_shape(2, 1024, 8, 2752, 8000, 2624)
    blob = workloads.make_weights(shape, seed=21, device="cuda")
    toks = workloads.make_prompt(shape.vocab, 2100, seed=3)
    gm, om = b.Model(shape, blob), orc.Model(shape, orc.blob_to_u16(blob))
    S = 2048
    for pos in range(0, S, 512):
        om.review_forward(toks[pos:pos + 512], pos)
    pos = 0
    while pos < S:
        n = min(16, S - pos)
        gm.csd_review_forward(to_dev_i32(toks[pos:pos + n]), pos)
        pos += n
    for m in (2, 5, 9, 17):
        blk = toks[S:S + m]
        g = gm.csd_review_forward(to_dev_i32(blk), S).cpu().numpy()
        r = om.review_forward(blk, S)
        assert rel_l2(g, r) <= LOGIT_REL_L2, (m, rel_l2(g, r))
        assert np.abs(g - r).max() <= LOGIT_MAX_ABS
    assert b.csd_device_status() == 0


@pytest.mark.parametrize("d_head,n_heads", [(64, 48), (128, 40)])
def test_long_cache_many_heads(b, orc, d_head, n_heads):
    """Long caches at both tensor-core head dimensions with 40 and 48 heads: every CTA walks more
    tiles than its ring holds, so ring slots are refilled; cache lengths before, on and after a
    tile edge, blocks of one and two row tiles; the cache comes from a wide-block prefill."""
    shape = llama_shape(1, d_head * n_heads, n_heads, 1024, 1000, 2300)
    blob = workloads.make_weights(shape, seed=33, device="cuda", std=0.03, gain_std=0.2)
    toks = workloads.make_prompt(shape.vocab, 2300, seed=8)
    gm, om = b.Model(shape, blob), orc.Model(shape, orc.blob_to_u16(blob))
    S = 2040
    for pos in range(0, S, 510):
        om.review_forward(toks[pos:pos + 510], pos)
    gm.csd_prefill(to_dev_i32(toks[:S]), 0)
    pos = S
    for m in (5, 3, 17, 9, 16, 17, 1, 12):      # 2040, 2045, 2048, 2065, 2074, 2090, 2107, 2108
        blk = toks[pos:pos + m]
        g = gm.csd_review_forward(to_dev_i32(blk), pos).cpu().numpy()
        r = om.review_forward(blk, pos)
        assert rel_l2(g, r) <= LOGIT_REL_L2, (pos, m, rel_l2(g, r))
        assert np.abs(g - r).max() <= LOGIT_MAX_ABS
        pos += m
    assert b.csd_device_status() == 0


def sub_stack(shape, blob, n_layers):
    """The first n_layers decoder layers of a blob (with its embedding, final norm and head)."""
    from dataclasses import replace
    small = replace(shape, n_layers=n_layers)
    src = {name: (off, shp) for name, off, shp in workloads.blob_layout(shape)[0]}
    layout, total = workloads.blob_layout(small)
    out = torch.zeros(total, dtype=blob.dtype, device=blob.device)
    for name, off, shp in layout:
        n = int(np.prod(shp))
        out[off:off + n] = blob[src[name][0]:src[name][0] + n]
    return small, out


def test_7b_width_depth_sweep(b, orc):
    """How the logit error of a 7B-wide stack depends on its depth, on both GEMM kernels, next to
    the distance between two CPU forwards that differ only in how they carry the sums (fp64, and
    fp32 throughout).  Both sides round K/V to bf16 before the cache; a difference of 1e-6 upstream
    moves some cache entries to the neighbouring bf16 value (2^-9 relative), which is what the
    layers above see.  The stated 2e-3 is asserted at every depth where two correct CPU forwards
    themselves stay within it; beyond, the GPU must stay within a small factor of their distance
    and must not compound with depth."""
    full = SHAPES["llama7b"]
    blob = workloads.make_weights(full, seed=100, device="cuda")
    seq = workloads.make_prompt(full.vocab, 22, seed=1000)
    depths = (1, 2, 4, 8, 16, 32)
    err = {1: {}, 2: {}}
    yard = {}
    for L in depths:
        shape, sub = (full, blob) if L == full.n_layers else sub_stack(full, blob, L)
        u16 = orc.blob_to_u16(sub)
        refs = []
        for mode in (0, 2):
            orc.set_linear_f32(mode)
            try:
                om = orc.Model(shape, u16)
                om.review_forward(seq[:17], 0)
                refs.append(om.review_forward(seq[17:], 17))
                om.close()
            finally:
                orc.set_linear_f32(0)
        yard[L] = rel_l2(refs[1], refs[0])
        for path in (1, 2):
            b.csd_set_gemm_path(path)
            b.csd_set_attention_path(1 if path == 1 else 0)
            try:
                gm = b.Model(shape, sub)
                gm.csd_review_forward(to_dev_i32(seq[:17]), 0)
                g = gm.csd_review_forward(to_dev_i32(seq[17:]), 17).cpu().numpy()
                gm.close()
            finally:
                b.csd_set_gemm_path(0)
                b.csd_set_attention_path(0)
            err[path][L] = rel_l2(g, refs[0])
            assert np.abs(g - refs[0]).max() <= LOGIT_MAX_ABS, (path, L)
        del sub
    print("\ndepth  cpu-fp32-vs-fp64  cuda-core  tensor-core")
    for L in depths:
        print(f"{L:5d}  {yard[L]:.3e}         {err[1][L]:.3e}  {err[2][L]:.3e}")
    assert b.csd_device_status() == 0
    for path in (1, 2):
        for L in depths:
            if yard[L] <= LOGIT_REL_L2 / 2:
                assert err[path][L] <= LOGIT_REL_L2, (path, L, err[path][L])
            assert err[path][L] <= max(LOGIT_REL_L2, 2.0 * yard[L]), (path, L, err[path][L], yard[L])
        assert err[path][32] <= 2.0 * err[path][16] + 1e-4, (path, err[path][16], err[path][32])


def t5xxl_width(n_enc, n_dec, max_seq=64):
    # the xxl layer shapes (d 4096, 64 heads x 64, ff 10240, vocabulary 32128, 256 encoder positions)
    return t5_shape(n_enc, n_dec, 4096, 64, 64, 10240, 32128, max_seq, 256)


@pytest.mark.parametrize("std", [0.005, 0.02], ids=["unit-scores", "workload-init"])
@pytest.mark.parametrize("path", [1, 2], ids=["cuda-core", "tensor-core"])
def test_t5xxl_width_shallow_stack(b, orc, path, std):
    """Encoder-decoder review forward at the xxl width in a 2 + 2 layer stack: 64 heads of 64, the
    gated-GELU pair at d_ff 10240, a 256-key cross-attention, bias tables of the full length.
    This family does not scale its attention scores.  With the workload's init (std 0.02) a score
    has a standard deviation of about 13, the soft-max is close to an arg-max, and two correct CPU
    forwards (fp64 sums, fp32 throughout) already differ by percents: there the GPU is held to
    twice their distance.  With std 0.005 the scores are of order one, as in a trained model of
    the family, and the stated tolerance applies as it stands."""
    shape = t5xxl_width(2, 2)
    blob = workloads.make_weights(shape, seed=300, device="cuda", std=std)
    enc = workloads.make_prompt(shape.vocab, 256, seed=9)
    dec = np.concatenate([[0], workloads.make_prompt(shape.vocab, 22, seed=10)]).astype(np.int32)
    u16 = orc.blob_to_u16(blob)
    refs = {}
    for mode in (0, 2):                       # fp64 sums, and the all-fp32 forward as the yardstick
        orc.set_linear_f32(mode)
        try:
            om = orc.Model(shape, u16)
            om.encoder_forward(enc)
            refs[mode] = [om.review_forward(dec[pos:pos + m], pos) for pos, m in ((0, 17), (17, 5), (22, 1))]
            om.close()
        finally:
            orc.set_linear_f32(0)
    b.csd_set_gemm_path(path)
    b.csd_set_attention_path(1 if path == 1 else 0)
    try:
        gm = b.Model(shape, blob)
        gm.csd_encoder_forward(to_dev_i32(enc))
        for i, (pos, m) in enumerate(((0, 17), (17, 5), (22, 1))):
            g = gm.csd_review_forward(to_dev_i32(dec[pos:pos + m]), pos).cpu().numpy()
            e, yard = rel_l2(g, refs[0][i]), rel_l2(refs[2][i], refs[0][i])
            print(f"\nt5-xxl width, path {path}, rows {m}: gpu {e:.3e}, cpu fp32-vs-fp64 {yard:.3e}")
            yard_abs = float(np.abs(refs[2][i] - refs[0][i]).max())
            if std < 0.01:
                assert yard <= LOGIT_REL_L2 / 2          # the conditioned case must be a meaningful one
                assert e <= LOGIT_REL_L2, (pos, m, e)
            assert e <= max(LOGIT_REL_L2, 2.0 * yard), (pos, m, e, yard)
            assert np.abs(g - refs[0][i]).max() <= max(LOGIT_MAX_ABS, 2.0 * yard_abs)
        assert b.csd_device_status() == 0
    finally:
        b.csd_set_gemm_path(0)
        b.csd_set_attention_path(0)


def test_t5xxl_width_sampled_horizontal_cascade(b, orc):
    """Temperature-1 horizontal cascade (two neural drafts, Max-Gram below) under an xxl-wide target:
    the same Philox stream must give the same tokens and the same accept counts as the oracle unless
    the oracle saw a decision within rounding of its threshold."""
    ts = t5xxl_width(2, 2)
    ds = t5_shape(1, 1, 512, 8, 64, 1024, 32128, 64, 256)
    # (weights scaled so that attention scores are of order one: see the test above)
    tb = workloads.make_weights(ts, seed=300, device="cuda", std=0.005)
    dbs = [workloads.make_weights(ds, seed=301 + i, device="cuda", std=0.02) for i in range(2)]
    enc = workloads.make_repetitive_prompt(ts.vocab, 256, seed=4)
    nxt = workloads.bigram_table(enc, ts.vocab, seed=0)
    K = [[2, 2, 0], [0, 1, 4], [0, 0, 4]]
    start = np.array([0], dtype=np.int32)
    n_new, exact = 12, 0
    for seed in (1, 2):
        oms = [orc.Model(ts, orc.blob_to_u16(tb))] + [orc.Model(ds, orc.blob_to_u16(w)) for w in dbs]
        want, _, ost = orc.cascade_generate(oms, enc, nxt, K, 4, start, n_new, temperature=1.0, seed=seed)
        gms = [b.Model(ts, tb)] + [b.Model(ds, w) for w in dbs]
        got, st = b.Cascade(gms, K, 4, to_dev_i32(nxt), 256).csd_cascade_generate(enc, start, n_new, 1.0, 1.0, seed)
        assert len(got) == n_new and b.csd_device_status() == 0
        if np.array_equal(got, want):
            exact += 1
            assert st["reviews"] == ost["reviews"] and st["accepted"] == ost["accepted"]
        else:
            first = int(np.nonzero(got != want)[0][0])
            assert ost["near_ties"] > 0 and ost["first_near_tie"] <= first, (seed, first, ost)
    assert exact >= 1


def test_wide_prefill_leaves_the_cache_a_review_needs(b, orc):
    """csd_prefill at the 7B width (wide blocks of up to 128 rows, two-term activations): the review
    block that follows must meet the stated tolerance against the oracle, which forwards every
    token the plain way; so must a second block after a second prefill that starts mid-cache, and
    the result must not depend on how the prompt was cut into prefill calls beyond that tolerance."""
    shape = llama_shape(3, 4096, 32, 11008, 32000, 320)
    blob = workloads.make_weights(shape, seed=100, device="cuda")
    seq = workloads.make_prompt(shape.vocab, 300, seed=1000)
    # the oracle takes the prompt in blocks of its own choice (block partition does not change its result)
    om2 = orc.Model(shape, orc.blob_to_u16(blob))
    refs = {}
    pos = 0
    for cut in (150, 155, 290, 295):
        while pos < cut:
            n = min(17, cut - pos)
            out = om2.review_forward(seq[pos:pos + n], pos)
            pos += n
        refs[cut] = out
    gm = b.Model(shape, blob)
    dev = to_dev_i32(seq)
    gm.csd_prefill(dev[:150].contiguous(), 0)                        # 128 wide + 22 (17 + 5 review-sized)
    g = gm.csd_review_forward(dev[150:155].contiguous(), 150).cpu().numpy()
    assert rel_l2(g, refs[155]) <= LOGIT_REL_L2, rel_l2(g, refs[155])
    assert np.abs(g - refs[155]).max() <= LOGIT_MAX_ABS
    gm.csd_prefill(dev[155:290].contiguous(), 155)                   # starts mid-cache: 128 wide + 7
    g = gm.csd_review_forward(dev[290:295].contiguous(), 290).cpu().numpy()
    assert rel_l2(g, refs[295]) <= LOGIT_REL_L2, rel_l2(g, refs[295])
    # the same prompt through the review kernels only
    gm2 = b.Model(shape, blob)
    p = 0
    while p < 150:
        n = min(17, 150 - p)
        gm2.csd_review_forward(dev[p:p + n].contiguous(), p, append_only=True)
        p += n
    g2 = gm2.csd_review_forward(dev[150:155].contiguous(), 150).cpu().numpy()
    g1 = b.Model(shape, blob)
    g1.csd_prefill(dev[:150].contiguous(), 0)
    g1o = g1.csd_review_forward(dev[150:155].contiguous(), 150).cpu().numpy()
    assert rel_l2(g1o, g2) <= LOGIT_REL_L2
    assert b.csd_device_status() == 0
