"""Pins the oracle's block forward pass to library implementations in float64.

(1) With cache rounding switched off, the decoder-only oracle must agree with the `transformers`
    LLaMA model and the encoder-decoder oracle with the `transformers` T5 (v1.1, gated-GELU)
    model loaded with the same weights: embedding, RMS norm, rotary pairs, relative-position
    buckets, attention scaling, masks, gated feed-forward, untied head.
(2) With rounding on (the product's data format: bf16 K/V), a forward written with torch
    library routines (matmul, softmax, scaled_dot_product_attention) that rounds K/V the same
    way must agree; and feeding a sequence block by block must equal feeding it at once.
"""
import numpy as np
import pytest
import torch

import workloads
from workloads import SHAPES, blob_layout


def tensors(shape, blob):
    layout, _ = blob_layout(shape)
    return {name: blob[off:off + int(np.prod(shp))].reshape(shp).double() for name, off, shp in layout}


def rel_l2(a, b):
    a = np.asarray(a, dtype=np.float64)
    b = np.asarray(b, dtype=np.float64)
    return np.linalg.norm(a - b) / np.linalg.norm(b)


@pytest.fixture(scope="module")
def tiny():
    shape = SHAPES["tiny_target"]
    blob = workloads.make_weights(shape, seed=7, gain_std=0.2, std=0.08)
    return shape, blob


def test_llama_against_transformers(orc, tiny):
    from transformers import LlamaConfig, LlamaForCausalLM
    shape, blob = tiny
    w = tensors(shape, blob)
    cfg = LlamaConfig(vocab_size=shape.vocab, hidden_size=shape.d_model, intermediate_size=shape.d_ff,
                      num_hidden_layers=shape.n_layers, num_attention_heads=shape.n_heads,
                      num_key_value_heads=shape.n_heads, hidden_act="silu", max_position_embeddings=512,
                      rms_norm_eps=shape.norm_eps, tie_word_embeddings=False, attention_bias=False,
                      mlp_bias=False, rope_parameters={"rope_type": "default", "rope_theta": shape.rope_theta})
    cfg._attn_implementation = "eager"
    hf = LlamaForCausalLM(cfg).double().eval()
    sd = {"model.embed_tokens.weight": w["embed"], "model.norm.weight": w["final_norm"],
          "lm_head.weight": w["lm_head"]}
    for l in range(shape.n_layers):
        p = f"model.layers.{l}."
        sd[p + "input_layernorm.weight"] = w[f"l{l}.norm1"]
        sd[p + "post_attention_layernorm.weight"] = w[f"l{l}.norm2"]
        for a, b in (("q", "wq"), ("k", "wk"), ("v", "wv"), ("o", "wo")):
            sd[p + f"self_attn.{a}_proj.weight"] = w[f"l{l}.{b}"]
        for a, b in (("gate", "wgate"), ("up", "wup"), ("down", "wdown")):
            sd[p + f"mlp.{a}_proj.weight"] = w[f"l{l}.{b}"]
    missing, unexpected = hf.load_state_dict(sd, strict=False)
    assert not [m for m in missing if "rotary" not in m] and not unexpected
    toks = workloads.make_prompt(shape.vocab, 23, seed=3)
    with torch.no_grad():
        ref = hf(torch.from_numpy(toks.astype(np.int64))[None]).logits[0].numpy()
    orc.set_kv_exact(True)
    try:
        m = orc.Model(shape, orc.blob_to_u16(blob))
        got = np.concatenate([m.review_forward(toks[:9], 0), m.review_forward(toks[9:10], 9),
                              m.review_forward(toks[10:], 10)])
    finally:
        orc.set_kv_exact(False)
    assert rel_l2(got, ref) < 1e-6
    assert np.abs(got - ref).max() < 1e-5


def torch_llama_forward(shape, w, toks, round_kv=True):
    """Whole-sequence forward from library routines; K/V rounded to bf16 as the cache stores them."""
    T = len(toks)
    H, Dh = shape.n_heads, shape.d_head
    x = w["embed"][torch.from_numpy(toks.astype(np.int64))]
    pos = torch.arange(T, dtype=torch.float64)
    inv = shape.rope_theta ** (-torch.arange(0, Dh, 2, dtype=torch.float64) / Dh)
    rot = torch.polar(torch.ones(T, Dh // 2, dtype=torch.float64), pos[:, None] * inv[None, :])

    def rope(v):  # v [T, H, Dh]; pair (i, i + Dh/2) rotated as one complex number
        z = torch.complex(v[..., :Dh // 2], v[..., Dh // 2:]) * rot[:, None, :]
        return torch.cat([z.real, z.imag], dim=-1)

    def norm(v, g):
        return v * torch.rsqrt(v.pow(2).mean(-1, keepdim=True) + shape.norm_eps) * g

    def kvr(v):  # nearest-even to 8 significant bits, decided in float64
        if not round_kv:
            return v
        mant, expo = torch.frexp(v)
        return torch.ldexp(torch.round(mant * 256.0), expo - 8)

    for l in range(shape.n_layers):
        h = norm(x, w[f"l{l}.norm1"])
        q = rope((h @ w[f"l{l}.wq"].T).view(T, H, Dh))
        k = kvr(rope((h @ w[f"l{l}.wk"].T).view(T, H, Dh)))
        v = kvr((h @ w[f"l{l}.wv"].T).view(T, H, Dh))
        o = torch.nn.functional.scaled_dot_product_attention(
            q.transpose(0, 1)[None], k.transpose(0, 1)[None], v.transpose(0, 1)[None], is_causal=True)
        x = x + o[0].transpose(0, 1).reshape(T, H * Dh) @ w[f"l{l}.wo"].T
        h = norm(x, w[f"l{l}.norm2"])
        x = x + (torch.nn.functional.silu(h @ w[f"l{l}.wgate"].T) * (h @ w[f"l{l}.wup"].T)) @ w[f"l{l}.wdown"].T
    return (norm(x, w["final_norm"]) @ w["lm_head"].T).numpy()


def test_llama_with_bf16_cache_against_torch_routines(orc, tiny):
    shape, blob = tiny
    w = tensors(shape, blob)
    toks = workloads.make_prompt(shape.vocab, 40, seed=5)
    ref = torch_llama_forward(shape, w, toks)
    m = orc.Model(shape, orc.blob_to_u16(blob))
    got = np.concatenate([m.review_forward(toks[:17], 0), m.review_forward(toks[17:22], 17),
                          m.review_forward(toks[22:], 22)])
    # float32 output rounding only (a K/V element within 1e-16 of a bf16 tie could flip; none here)
    assert rel_l2(got, ref) < 1e-6
    # rounding the cache must matter at the 1e-3 level, or the test above proves nothing about it
    exact = torch_llama_forward(shape, w, toks, round_kv=False)
    assert 1e-5 < rel_l2(exact, ref) < 5e-2


def test_block_partition_and_rollback_invariance(orc, tiny):
    shape, blob = tiny
    toks = workloads.make_prompt(shape.vocab, 30, seed=9)
    u16 = orc.blob_to_u16(blob)
    a = orc.Model(shape, u16)
    whole = a.review_forward(toks, 0)
    b = orc.Model(shape, u16)
    parts = [b.review_forward(toks[:5], 0)]
    # a rejected block: positions 5..9 are written with other tokens, then overwritten
    b.review_forward((toks[5:10] + 1) % shape.vocab, 5)
    parts.append(b.review_forward(toks[5:6], 5))
    parts.append(b.review_forward(toks[6:30], 6))
    assert np.array_equal(np.concatenate(parts), whole)


def test_rel_bucket_against_transformers(orc):
    from transformers.models.t5.modeling_t5 import T5Attention
    rel = torch.arange(-300, 301)
    for bidir in (True, False):
        ref = T5Attention._relative_position_bucket(rel, bidirectional=bidir, num_buckets=32, max_distance=128)
        got = [orc.rel_bucket(int(r), bidir, 32, 128) for r in rel]
        assert got == ref.tolist()


def test_t5_against_transformers(orc):
    from transformers import T5Config, T5ForConditionalGeneration
    shape = SHAPES["t5tiny_target"]
    blob = workloads.make_weights(shape, seed=2, gain_std=0.2, std=0.08)
    w = tensors(shape, blob)
    cfg = T5Config(vocab_size=shape.vocab, d_model=shape.d_model, d_kv=shape.d_head, d_ff=shape.d_ff,
                   num_layers=shape.n_enc_layers, num_decoder_layers=shape.n_layers, num_heads=shape.n_heads,
                   relative_attention_num_buckets=shape.rel_buckets,
                   relative_attention_max_distance=shape.rel_max_dist, dropout_rate=0.0,
                   layer_norm_epsilon=shape.norm_eps, feed_forward_proj="gated-gelu",
                   tie_word_embeddings=False, decoder_start_token_id=0, pad_token_id=0)
    cfg._attn_implementation = "eager"
    cfg.tie_word_embeddings = False      # v1.1 layout: separate output head, no d_model**-0.5 factor
    hf = T5ForConditionalGeneration(cfg).double().eval()
    hf.lm_head.weight = torch.nn.Parameter(hf.lm_head.weight.detach().clone())
    assert not hf.config.tie_word_embeddings
    sd = {"shared.weight": w["embed"], "encoder.embed_tokens.weight": w["embed"],
          "decoder.embed_tokens.weight": w["embed"], "lm_head.weight": w["lm_head"],
          "encoder.final_layer_norm.weight": w["enc.final_norm"],
          "decoder.final_layer_norm.weight": w["final_norm"],
          "encoder.block.0.layer.0.SelfAttention.relative_attention_bias.weight": w["enc.rel_bias"],
          "decoder.block.0.layer.0.SelfAttention.relative_attention_bias.weight": w["dec.rel_bias"]}

    def ffn(dst, src):
        sd[dst + "layer_norm.weight"] = w[src + ".norm2"]
        sd[dst + "DenseReluDense.wi_0.weight"] = w[src + ".wgate"]
        sd[dst + "DenseReluDense.wi_1.weight"] = w[src + ".wup"]
        sd[dst + "DenseReluDense.wo.weight"] = w[src + ".wdown"]

    for l in range(shape.n_enc_layers):
        p = f"encoder.block.{l}."
        sd[p + "layer.0.layer_norm.weight"] = w[f"e{l}.norm1"]
        for a in "qkvo":
            sd[p + f"layer.0.SelfAttention.{a}.weight"] = w[f"e{l}.w{a}"]
        ffn(p + "layer.1.", f"e{l}")
    for l in range(shape.n_layers):
        p = f"decoder.block.{l}."
        sd[p + "layer.0.layer_norm.weight"] = w[f"l{l}.norm1"]
        sd[p + "layer.1.layer_norm.weight"] = w[f"l{l}.norm_x"]
        for a in "qkvo":
            sd[p + f"layer.0.SelfAttention.{a}.weight"] = w[f"l{l}.w{a}"]
            sd[p + f"layer.1.EncDecAttention.{a}.weight"] = w[f"l{l}.x{a}"]
        ffn(p + "layer.2.", f"l{l}")
    missing, unexpected = hf.load_state_dict(sd, strict=False)
    assert not missing and not unexpected
    enc = workloads.make_prompt(shape.vocab, 37, seed=4)
    dec = np.concatenate([[0], workloads.make_prompt(shape.vocab, 20, seed=6)]).astype(np.int32)
    with torch.no_grad():
        ref = hf(input_ids=torch.from_numpy(enc.astype(np.int64))[None],
                 decoder_input_ids=torch.from_numpy(dec.astype(np.int64))[None]).logits[0].numpy()
    orc.set_kv_exact(True)
    try:
        m = orc.Model(shape, orc.blob_to_u16(blob))
        m.encoder_forward(enc)
        got = np.concatenate([m.review_forward(dec[:1], 0), m.review_forward(dec[1:8], 1),
                              m.review_forward(dec[8:], 8)])
    finally:
        orc.set_kv_exact(False)
    # the library's norm layer squares in float32 even for a float64 model, hence 1e-5 not 1e-7
    assert rel_l2(got, ref) < 1e-5
    assert np.abs(got - ref).max() < 1e-4
    # with the bf16 cache the result moves, but only at the level bf16 rounding allows
    m2 = orc.Model(shape, orc.blob_to_u16(blob))
    m2.encoder_forward(enc)
    rounded = m2.review_forward(dec, 0)
    assert 1e-5 < rel_l2(rounded, ref) < 5e-2


def torch_t5_forward(shape, w, enc, dec, round_kv=True):
    """Encoder-decoder forward from library routines (matmul, softmax, gelu, the library's bucket
    function); every K and V that the product keeps in a bf16 cache (encoder self-attention, decoder
    self-attention, cross-attention) is rounded to 8 significant bits right after its projection."""
    from transformers.models.t5.modeling_t5 import T5Attention
    H, Dh, d = shape.n_heads, shape.d_head, shape.d_model

    def norm(v, g):
        return v * torch.rsqrt(v.pow(2).mean(-1, keepdim=True) + shape.norm_eps) * g

    def kvr(v):
        if not round_kv:
            return v
        mant, expo = torch.frexp(v)
        return torch.ldexp(torch.round(mant * 256.0), expo - 8)

    def heads(v):
        return v.view(v.shape[0], H, Dh).transpose(0, 1)          # [H, T, Dh]

    def bias(table, nq, nk, bidir):
        rel = torch.arange(nk)[None, :] - torch.arange(nq)[:, None]
        bucket = T5Attention._relative_position_bucket(rel, bidirectional=bidir, num_buckets=shape.rel_buckets,
                                                       max_distance=shape.rel_max_dist)
        return table[bucket].permute(2, 0, 1)                      # [H, nq, nk]

    def attend(q, k, v, extra):
        sc = heads(q) @ heads(k).transpose(1, 2)                   # no 1/sqrt(Dh): the family does not scale
        if extra is not None:
            sc = sc + extra
        return (torch.softmax(sc, dim=-1) @ heads(v)).transpose(0, 1).reshape(q.shape[0], H * Dh)

    def ffn(x, p):
        h = norm(x, w[p + ".norm2"])
        g = torch.nn.functional.gelu(h @ w[p + ".wgate"].T, approximate="tanh") * (h @ w[p + ".wup"].T)
        return x + g @ w[p + ".wdown"].T

    E, T = len(enc), len(dec)
    x = w["embed"][torch.from_numpy(enc.astype(np.int64))]
    eb = bias(w["enc.rel_bias"], E, E, True)
    for l in range(shape.n_enc_layers):
        h = norm(x, w[f"e{l}.norm1"])
        x = x + attend(h @ w[f"e{l}.wq"].T, kvr(h @ w[f"e{l}.wk"].T), kvr(h @ w[f"e{l}.wv"].T), eb) @ w[f"e{l}.wo"].T
        x = ffn(x, f"e{l}")
    mem = norm(x, w["enc.final_norm"])
    y = w["embed"][torch.from_numpy(dec.astype(np.int64))]
    causal = torch.full((T, T), float("-inf"), dtype=torch.float64).triu(1)
    db = bias(w["dec.rel_bias"], T, T, False) + causal
    for l in range(shape.n_layers):
        h = norm(y, w[f"l{l}.norm1"])
        y = y + attend(h @ w[f"l{l}.wq"].T, kvr(h @ w[f"l{l}.wk"].T), kvr(h @ w[f"l{l}.wv"].T), db) @ w[f"l{l}.wo"].T
        h = norm(y, w[f"l{l}.norm_x"])
        y = y + attend(h @ w[f"l{l}.xq"].T, kvr(mem @ w[f"l{l}.xk"].T), kvr(mem @ w[f"l{l}.xv"].T), None) @ w[f"l{l}.xo"].T
        y = ffn(y, f"l{l}")
    return (norm(y, w["final_norm"]) @ w["lm_head"].T).numpy()


def test_t5_with_bf16_caches_against_torch_routines(orc):
    # pins WHERE the encoder-decoder path rounds: all three K/V kinds, right after their projections
    shape = SHAPES["t5tiny_target"]
    blob = workloads.make_weights(shape, seed=2, gain_std=0.2, std=0.08)
    w = tensors(shape, blob)
    enc = workloads.make_prompt(shape.vocab, 37, seed=4)
    dec = np.concatenate([[0], workloads.make_prompt(shape.vocab, 20, seed=6)]).astype(np.int32)
    ref = torch_t5_forward(shape, w, enc, dec)
    m = orc.Model(shape, orc.blob_to_u16(blob))
    m.encoder_forward(enc)
    got = np.concatenate([m.review_forward(dec[:1], 0), m.review_forward(dec[1:8], 1), m.review_forward(dec[8:], 8)])
    assert rel_l2(got, ref) < 1e-6
    # each of the three roundings matters on its own at a level far above that bound, so a rounding
    # moved, dropped or doubled in the oracle would fail the comparison above
    exact = torch_t5_forward(shape, w, enc, dec, round_kv=False)
    assert 1e-5 < rel_l2(exact, ref) < 5e-2
    orc.set_kv_exact(True)
    try:
        m2 = orc.Model(shape, orc.blob_to_u16(blob))
        m2.encoder_forward(enc)
        unrounded = m2.review_forward(dec, 0)
    finally:
        orc.set_kv_exact(False)
    assert rel_l2(unrounded, exact) < 1e-6


def test_two_correct_forwards_drift_apart_only_through_the_bf16_cache(orc):
    # The same forward carried two equally valid ways (float64 throughout; contraction results
    # rounded to float32).  With an unrounded cache the two stay within float32 rounding at any
    # depth.  With the bf16 cache a difference of 1e-7 upstream moves some K/V entries across a
    # rounding boundary, each worth 2^-9, and the gap grows by orders of magnitude with depth:
    # a deep stack compared against ANY second implementation sees this gap, whatever the
    # accuracy of that implementation's own arithmetic.
    from workloads import llama_shape
    gaps = {}
    for depth in (1, 4, 32):
        shape = llama_shape(depth, 256, 4, 688, 1000, 64)
        blob = orc.blob_to_u16(workloads.make_weights(shape, seed=5, std=0.05))
        toks = workloads.make_prompt(shape.vocab, 40, seed=3)
        for exact in (False, True):
            outs = []
            for f32 in (False, True):
                orc.set_kv_exact(exact)
                orc.set_linear_f32(f32)
                try:
                    m = orc.Model(shape, blob)
                    outs.append(np.concatenate([m.review_forward(toks[:17], 0), m.review_forward(toks[17:22], 17),
                                                m.review_forward(toks[22:], 22)]))
                finally:
                    orc.set_kv_exact(False)
                    orc.set_linear_f32(False)
            gaps[depth, exact] = rel_l2(outs[1], outs[0])
    for depth in (1, 4, 32):
        assert gaps[depth, True] < 1e-6                      # unrounded cache: float32 rounding only
    assert gaps[1, False] < 1e-6                             # one layer: its own K/V see identical inputs
    assert gaps[4, False] > 50 * gaps[4, True]
    assert gaps[32, False] > 1000 * gaps[32, True]           # measured: 6.7e-4 against 1.3e-7
    assert gaps[32, False] < 5e-3


def test_an_all_fp32_forward_drifts_further_and_levels_off(orc):
    # The same comparison with the second forward carried in fp32 throughout (fp32 operands,
    # products and running sums): the kind of implementation a GPU path with fp32 accumulation is.
    # Its own arithmetic differs from the fp64 sums by a few 1e-7 per contraction, yet behind the
    # bf16 cache the logits end up 1e-3 apart in a deep stack, and the gap levels off with depth
    # instead of compounding.
    from workloads import llama_shape
    gap, exact_gap = {}, {}
    for depth in (2, 8, 32):
        shape = llama_shape(depth, 256, 4, 688, 1000, 64)
        blob = orc.blob_to_u16(workloads.make_weights(shape, seed=5, std=0.05))
        toks = workloads.make_prompt(shape.vocab, 40, seed=3)
        for exact in (False, True):
            outs = []
            for mode in (0, 2):
                orc.set_kv_exact(exact)
                orc.set_linear_f32(mode)
                try:
                    m = orc.Model(shape, blob)
                    outs.append(np.concatenate([m.review_forward(toks[:17], 0), m.review_forward(toks[17:22], 17),
                                                m.review_forward(toks[22:], 22)]))
                finally:
                    orc.set_kv_exact(False)
                    orc.set_linear_f32(0)
            (exact_gap if exact else gap)[depth] = rel_l2(outs[1], outs[0])
    for depth in (2, 8, 32):
        assert exact_gap[depth] < 2e-6                       # fp32 sums alone: rounding level
        assert gap[depth] > 20 * exact_gap[depth]            # the bf16 cache multiplies the difference
    assert gap[32] < 5e-3
    assert gap[32] < 4 * gap[8]                              # levels off: no compounding with depth


def test_bf16_rounding_is_nearest_even(orc):
    rng = np.random.default_rng(0)
    xs = np.concatenate([rng.standard_normal(2000) * 10.0 ** rng.integers(-6, 6, 2000), [0.0, 1.0, -1.0]])
    ref = torch.from_numpy(xs.astype(np.float32)).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)
    got = np.array([orc.double_to_bf16(float(np.float32(x))) for x in xs], dtype=np.uint16)
    assert np.array_equal(got, ref)
    # exact ties go to the even mantissa: 1 + 2^-8 lies halfway between 1.0 and 1 + 2^-7
    assert orc.double_to_bf16(1.0 + 2.0 ** -8) == 0x3F80
    assert orc.double_to_bf16(1.0 + 2.0 ** -7 + 2.0 ** -8) == 0x3F82
    assert orc.double_to_bf16(1.0 + 2.0 ** -8 + 2.0 ** -30) == 0x3F81


def test_linear_hook(orc):
    rng = np.random.default_rng(3)
    W = torch.from_numpy(rng.standard_normal((37, 129)).astype(np.float32)).to(torch.bfloat16)
    X = rng.standard_normal((5, 129)).astype(np.float32)
    got = orc.linear(W.view(torch.int16).numpy().view(np.uint16), X)
    ref = (torch.from_numpy(X).double() @ W.double().T).numpy()
    assert np.abs(got - ref).max() < 1e-5
