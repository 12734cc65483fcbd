"""Seeded synthetic inputs for the review-step hot path of Cascade Speculative Drafting.

This module produces DATA only: model shapes, random-init bf16 weight blobs in the packed
interchange layout, prompts, bigram successor tables and logit tensors.  It holds none of the
method's arithmetic (no softmax / accept rule / n-gram search / transformer math), imports
neither the CUDA package nor the CPU oracle, and is the only code both of them are fed from.

Shapes follow the model families the paper names in Section 5.1 (a LLaMA-family 7B target with a
68M draft; a FLAN-T5 xxl target with base and small drafts); weights are random because trained
checkpoints are not part of this repository.
"""
from __future__ import annotations

from dataclasses import dataclass, replace
from typing import Dict, List, Tuple

import numpy as np
import torch

ARCH_LLAMA = 0
ARCH_T5 = 1

ALIGN_ELEMS = 128  # every tensor in the blob starts on a 256-byte boundary (128 bf16 elements)


@dataclass(frozen=True)
class ModelShape:
    """Plain description of a model; each side converts it to its own C struct."""
    arch: int
    n_layers: int          # decoder layers
    n_enc_layers: int      # encoder layers (T5-style only)
    d_model: int
    n_heads: int
    d_head: int
    d_ff: int
    vocab: int
    max_seq: int           # decoder KV capacity (positions)
    max_rows: int = 17     # rows per review forward
    max_enc_len: int = 0
    rel_buckets: int = 32
    rel_max_dist: int = 128
    norm_eps: float = 1e-5
    rope_theta: float = 10000.0

    @property
    def d_inner(self) -> int:
        return self.n_heads * self.d_head


def llama_shape(n_layers, d, heads, ff, vocab, max_seq, **kw) -> ModelShape:
    return ModelShape(ARCH_LLAMA, n_layers, 0, d, heads, d // heads, ff, vocab, max_seq, **kw)


def t5_shape(n_enc, n_dec, d, heads, d_kv, ff, vocab, max_seq, max_enc_len, **kw) -> ModelShape:
    return ModelShape(ARCH_T5, n_dec, n_enc, d, heads, d_kv, ff, vocab, max_seq,
                      max_enc_len=max_enc_len, norm_eps=1e-6, **kw)


SHAPES: Dict[str, ModelShape] = {
    # tiny cascade (seconds on a CPU)
    "tiny_target": llama_shape(2, 256, 4, 1024, 4096, 160),
    "tiny_draft": llama_shape(1, 64, 2, 256, 4096, 160),
    # decoder-only workload: 7B-shaped target, 68M-shaped draft
    "llama7b": llama_shape(32, 4096, 32, 11008, 32000, 448),
    "llama7b_long": llama_shape(32, 4096, 32, 11008, 32000, 2624),
    "draft68m": llama_shape(2, 768, 12, 3072, 32000, 448),
    # encoder-decoder workload: xxl-shaped target, base- and small-shaped drafts
    "t5xxl": t5_shape(24, 24, 4096, 64, 64, 10240, 32128, 192, 256),
    "t5base": t5_shape(12, 12, 768, 12, 64, 2048, 32128, 192, 256),
    "t5small": t5_shape(8, 8, 512, 8, 64, 1024, 32128, 192, 256),
    # miniature encoder-decoder shapes for CPU tests
    "t5tiny_target": t5_shape(2, 2, 128, 4, 32, 256, 512, 96, 48),
    "t5tiny_draft": t5_shape(1, 1, 64, 2, 32, 128, 512, 96, 48),
}


def with_max_seq(shape: ModelShape, max_seq: int) -> ModelShape:
    return replace(shape, max_seq=max_seq)


# --------------------------------------------------------------------------------------------
# Packed weight blob: an interchange FORMAT (like a file format), all bf16, each tensor [out, in]
# row-major and starting on a 256-byte boundary.
# --------------------------------------------------------------------------------------------

def _align(n: int) -> int:
    return (n + ALIGN_ELEMS - 1) // ALIGN_ELEMS * ALIGN_ELEMS


def blob_layout(s: ModelShape) -> Tuple[List[Tuple[str, int, Tuple[int, ...]]], int]:
    """Return ([(name, element offset, shape)], total elements) of the packed blob."""
    out: List[Tuple[str, int, Tuple[int, ...]]] = []
    off = 0

    def add(name, *shape):
        nonlocal off
        out.append((name, off, tuple(shape)))
        off = _align(off + int(np.prod(shape)))

    d, di, ff, V = s.d_model, s.d_inner, s.d_ff, s.vocab

    def attn(prefix, q="wq", k="wk", v="wv", o="wo"):
        add(f"{prefix}.{q}", di, d)
        add(f"{prefix}.{k}", di, d)
        add(f"{prefix}.{v}", di, d)
        add(f"{prefix}.{o}", d, di)

    def ffn(prefix):
        add(f"{prefix}.norm2", d)
        add(f"{prefix}.wgate", ff, d)
        add(f"{prefix}.wup", ff, d)
        add(f"{prefix}.wdown", d, ff)

    add("embed", V, d)
    if s.arch == ARCH_T5:
        add("enc.rel_bias", s.rel_buckets, s.n_heads)
        for l in range(s.n_enc_layers):
            add(f"e{l}.norm1", d)
            attn(f"e{l}")
            ffn(f"e{l}")
        add("enc.final_norm", d)
        add("dec.rel_bias", s.rel_buckets, s.n_heads)
    for l in range(s.n_layers):
        add(f"l{l}.norm1", d)
        attn(f"l{l}")
        if s.arch == ARCH_T5:
            add(f"l{l}.norm_x", d)
            attn(f"l{l}", "xq", "xk", "xv", "xo")
        ffn(f"l{l}")
    add("final_norm", d)
    add("lm_head", V, d)
    return out, off


def make_weights(s: ModelShape, seed: int, device: str = "cpu", std: float = 0.02,
                 gain_std: float = 0.0, bias_std: float = 0.5) -> torch.Tensor:
    """Random-init blob: matrices N(0, std), norm gains 1 (+ N(0, gain_std)), relative-position
    bias tables N(0, bias_std); rounded to bf16.  `gain_std > 0` is for tests that must notice a
    dropped gain; the benchmark workloads use the plain init (gains exactly 1)."""
    layout, total = blob_layout(s)
    blob = torch.zeros(total, dtype=torch.bfloat16, device=device)
    g = torch.Generator(device=device)
    g.manual_seed(seed)
    for name, off, shape in layout:
        n = int(np.prod(shape))
        if "norm" in name:
            t = torch.ones(n, device=device)
            if gain_std > 0:
                t = t + gain_std * torch.randn(n, generator=g, device=device)
            blob[off:off + n] = t.to(torch.bfloat16)
        elif "rel_bias" in name:
            blob[off:off + n] = (bias_std * torch.randn(n, generator=g, device=device)).to(torch.bfloat16)
        else:
            step = 1 << 26
            for a in range(0, n, step):
                b = min(n, a + step)
                blob[off + a:off + b] = (std * torch.randn(b - a, generator=g, device=device)).to(torch.bfloat16)
    return blob


# --------------------------------------------------------------------------------------------
# Token-level inputs
# --------------------------------------------------------------------------------------------

def make_prompt(vocab: int, length: int, seed: int) -> np.ndarray:
    """Uniform-random token ids (stand-in for the benchmark prompts the paper uses)."""
    rng = np.random.default_rng(seed)
    return rng.integers(0, vocab, size=length, dtype=np.int64).astype(np.int32)


def make_repetitive_prompt(vocab: int, length: int, seed: int, phrase: int = 6) -> np.ndarray:
    """Prompt with repeated phrases, so that suffix matches of several orders exist."""
    rng = np.random.default_rng(seed)
    phrases = [rng.integers(0, vocab, size=phrase) for _ in range(4)]
    out: List[int] = []
    while len(out) < length:
        if rng.random() < 0.6:
            out.extend(phrases[int(rng.integers(0, len(phrases)))].tolist())
        else:
            out.append(int(rng.integers(0, vocab)))
    return np.asarray(out[:length], dtype=np.int32)


def bigram_table(prompt: np.ndarray, vocab: int, seed: int) -> np.ndarray:
    """Stand-in for the paper's corpus-derived bigram model: one successor per vocabulary entry.

    next[a] = most frequent successor of a in the prompt (ties: the successor seen first);
    ids that never occur with a successor get a seeded pseudo-random successor."""
    rng = np.random.default_rng(seed ^ 0x5EED)
    nxt = rng.integers(0, vocab, size=vocab, dtype=np.int64).astype(np.int32)
    succ: Dict[int, Dict[int, List[int]]] = {}
    for i in range(len(prompt) - 1):
        a, b = int(prompt[i]), int(prompt[i + 1])
        d = succ.setdefault(a, {})
        if b in d:
            d[b][0] += 1
        else:
            d[b] = [1, i]
    for a, d in succ.items():
        best = min(d.items(), key=lambda kv: (-kv[1][0], kv[1][1]))
        nxt[a] = best[0]
    return nxt


def accept_case(rows: int, k: int, vocab: int, sigma: float, seed: int,
                target_std: float = 3.0, device: str = "cpu"):
    """Standalone accept/residual workload: target logits N(0, target_std) for k+1 positions,
    draft logits = target logits + N(0, sigma) for the first k, tokens sampled from the draft
    distribution with this harness's own generator.  Returns fp32 [rows,k+1,V], fp32 [rows,k,V],
    int32 [rows,k]."""
    g = torch.Generator(device=device)
    g.manual_seed(seed)
    t = target_std * torch.randn(rows, k + 1, vocab, generator=g, device=device)
    d = (t[:, :k, :] + sigma * torch.randn(rows, k, vocab, generator=g, device=device)).contiguous()
    if k > 0:
        probs = torch.softmax(d.double().reshape(rows * k, vocab), dim=-1)
        tok = torch.multinomial(probs, 1, generator=g).reshape(rows, k).to(torch.int32)
    else:
        tok = torch.zeros(rows, 0, dtype=torch.int32, device=device)
    return t.contiguous(), d, tok


def small_logits(rows: int, k: int, vocab: int, seed: int, scale: float = 1.0):
    """Small dense logits for statistical tests on tiny vocabularies."""
    rng = np.random.default_rng(seed)
    t = (scale * rng.standard_normal((rows, k + 1, vocab))).astype(np.float32)
    d = (scale * rng.standard_normal((rows, k, vocab))).astype(np.float32)
    return t, d
