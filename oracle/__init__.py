"""ctypes front-end of the CPU oracle (test infrastructure only).

Only the tests, the smoke check and the benchmark's CPU-baseline leg import this module; the
product package never does.  `build()` compiles `csd_oracle.c` with gcc into this folder.
"""
from __future__ import annotations

import ctypes as C
import os
import subprocess
from typing import List, Optional, Sequence

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "csd_oracle.c")
_LIB = os.path.join(_HERE, "liborc.so")
_lib = None


def build(force: bool = False) -> str:
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        tmp = _LIB + f".{os.getpid()}.tmp"
        subprocess.check_call(["gcc", "-O2", "-march=native", "-fopenmp", "-shared", "-fPIC",
                               "-o", tmp, _SRC, "-lm"])
        os.replace(tmp, _LIB)
    return _LIB


class ModelConfig(C.Structure):
    _fields_ = [(n, C.c_int32) for n in
                ("arch", "n_layers", "n_enc_layers", "d_model", "n_heads", "d_head", "d_ff", "vocab",
                 "max_seq", "max_rows", "max_enc_len", "rel_buckets", "rel_max_dist")] + \
               [("norm_eps", C.c_float), ("rope_theta", C.c_float)]


class Stats(C.Structure):
    _fields_ = [("tokens", C.c_int64), ("reviews", C.c_int64 * 8), ("forwards", C.c_int64 * 8),
                ("drafted", C.c_int64 * 8), ("accepted", C.c_int64 * 8), ("mag_calls", C.c_int64),
                ("mag_tokens", C.c_int64), ("near_ties", C.c_int64), ("first_near_tie", C.c_int64)]

    def as_dict(self, n_levels: int):
        return dict(tokens=self.tokens, reviews=list(self.reviews)[:n_levels],
                    forwards=list(self.forwards)[:n_levels], drafted=list(self.drafted)[:n_levels],
                    accepted=list(self.accepted)[:n_levels], mag_calls=self.mag_calls,
                    mag_tokens=self.mag_tokens, near_ties=self.near_ties, first_near_tie=self.first_near_tie)


def lib():
    global _lib
    if _lib is None:
        _lib = C.CDLL(build())
        L = _lib
        L.orc_philox4x32_10.argtypes = [C.c_void_p, C.c_void_p, C.c_void_p]
        L.orc_review_uniforms.argtypes = [C.c_uint64, C.c_uint64, C.c_int, C.c_int, C.c_void_p, C.c_void_p]
        L.orc_double_to_bf16.argtypes = [C.c_double]
        L.orc_double_to_bf16.restype = C.c_uint16
        L.orc_set_kv_exact.argtypes = [C.c_int]
        L.orc_set_linear_f32.argtypes = [C.c_int]
        L.orc_top2_margin.argtypes = [C.c_void_p, C.c_int]
        L.orc_top2_margin.restype = C.c_float
        L.orc_spec_accept.argtypes = [C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_int, C.c_int,
                                      C.c_int, C.c_float, C.c_float, C.c_uint64, C.c_uint64,
                                      C.c_void_p, C.c_void_p, C.c_void_p]
        L.orc_mag_draft.argtypes = [C.c_void_p, C.c_int, C.c_void_p, C.c_int, C.c_void_p, C.c_int,
                                    C.c_int, C.c_int, C.c_void_p]
        L.orc_model_weight_elems.argtypes = [C.c_void_p]
        L.orc_model_weight_elems.restype = C.c_size_t
        L.orc_model_create.argtypes = [C.c_void_p, C.c_void_p]
        L.orc_model_create.restype = C.c_void_p
        L.orc_model_destroy.argtypes = [C.c_void_p]
        L.orc_linear.argtypes = [C.c_void_p, C.c_int, C.c_int, C.c_void_p, C.c_int, C.c_void_p]
        L.orc_rel_bucket.argtypes = [C.c_int, C.c_int, C.c_int, C.c_int]
        L.orc_encoder_forward.argtypes = [C.c_void_p, C.c_void_p, C.c_int]
        L.orc_review_forward.argtypes = [C.c_void_p, C.c_void_p, C.c_int, C.c_int, C.c_void_p]
        L.orc_cascade_generate.argtypes = [C.c_void_p, C.c_int, C.c_void_p, C.c_int, C.c_void_p, C.c_int,
                                           C.c_void_p, C.c_int, C.c_float, C.c_float, C.c_uint64,
                                           C.c_void_p, C.c_int, C.c_int, C.c_int, C.c_void_p, C.c_void_p,
                                           C.c_void_p, C.c_void_p]
    return _lib


def _p(a: Optional[np.ndarray]):
    return None if a is None else a.ctypes.data_as(C.c_void_p)


def _i32(a) -> np.ndarray:
    return np.ascontiguousarray(np.asarray(a, dtype=np.int32))


def _f32(a) -> np.ndarray:
    return np.ascontiguousarray(np.asarray(a, dtype=np.float32))


def philox4x32_10(ctr: Sequence[int], key: Sequence[int]) -> List[int]:
    c = np.asarray(ctr, dtype=np.uint32)
    k = np.asarray(key, dtype=np.uint32)
    o = np.zeros(4, dtype=np.uint32)
    lib().orc_philox4x32_10(_p(c), _p(k), _p(o))
    return [int(x) for x in o]


def review_uniforms(seed: int, step: int, row: int, pos: int):
    u = C.c_double()
    u2 = C.c_double()
    lib().orc_review_uniforms(seed, step, row, pos, C.byref(u), C.byref(u2))
    return u.value, u2.value


def double_to_bf16(x: float) -> int:
    return int(lib().orc_double_to_bf16(float(x)))


def set_kv_exact(on: bool) -> None:
    """Test hook: keep cached K/V unrounded (for comparison with library models)."""
    lib().orc_set_kv_exact(int(on))


def set_linear_f32(mode) -> None:
    """Test hook: 1/True rounds every contraction result to fp32, 2 runs the contractions in fp32
    throughout (two more correct ways to do the sums), 0/False restores the fp64 sums."""
    lib().orc_set_linear_f32(int(mode))


def top2_margin(logits) -> float:
    x = _f32(logits).ravel()
    return float(lib().orc_top2_margin(_p(x), len(x)))


def spec_accept(target_logits, draft_logits, tokens, temperature: float, lenience: float = 1.0,
                seed: int = 0, step: int = 0, onehot=None):
    """Returns (n_accepted [rows], out_token [rows], near_tie [rows])."""
    t = _f32(target_logits)
    rows, k1, V = t.shape
    k = k1 - 1
    d = None if draft_logits is None else _f32(draft_logits)
    if d is not None:
        assert d.shape == (rows, k, V)
    tok = _i32(tokens).reshape(rows, k)
    oh = None if onehot is None else _i32(onehot).reshape(rows, k)
    n = np.zeros(rows, dtype=np.int32)
    o = np.zeros(rows, dtype=np.int32)
    f = np.zeros(rows, dtype=np.int32)
    rc = lib().orc_spec_accept(_p(t), _p(d), _p(oh), _p(tok), rows, k, V, temperature, lenience,
                               seed, step, _p(n), _p(o), _p(f))
    if rc:
        raise ValueError(f"orc_spec_accept: bad arguments ({rc})")
    return n, o, f


def mag_draft(haystack, bigram_next, seq, n: int, max_order: int = 16) -> np.ndarray:
    h = _i32(haystack)
    b = _i32(bigram_next)
    s = _i32(seq)
    out = np.zeros(max(n, 1), dtype=np.int32)
    made = lib().orc_mag_draft(_p(h), len(h), _p(b), len(b), _p(s), len(s), n, max_order, _p(out))
    if made < 0:
        raise ValueError("orc_mag_draft: bad arguments")
    return out[:made]


def linear(w_bf16_u16: np.ndarray, x: np.ndarray) -> np.ndarray:
    """Y = X . W^T with W a uint16 view of bf16 [N, K], X fp32 [m, K]."""
    w = np.ascontiguousarray(w_bf16_u16, dtype=np.uint16)
    N, K = w.shape
    x = _f32(x)
    m = x.shape[0]
    y = np.zeros((m, N), dtype=np.float32)
    lib().orc_linear(_p(w), N, K, _p(x), m, _p(y))
    return y


def rel_bucket(rel: int, bidirectional: bool, n_buckets: int = 32, max_dist: int = 128) -> int:
    return int(lib().orc_rel_bucket(rel, int(bidirectional), n_buckets, max_dist))


def config_from_shape(s) -> ModelConfig:
    return ModelConfig(s.arch, s.n_layers, s.n_enc_layers, s.d_model, s.n_heads, s.d_head, s.d_ff,
                       s.vocab, s.max_seq, s.max_rows, s.max_enc_len, s.rel_buckets, s.rel_max_dist,
                       s.norm_eps, s.rope_theta)


class Model:
    """Oracle model over a host bf16 blob (uint16 numpy view, kept alive here)."""

    def __init__(self, shape, blob_u16: np.ndarray):
        self.shape = shape
        self.cfg = config_from_shape(shape)
        self.blob = np.ascontiguousarray(blob_u16, dtype=np.uint16)
        need = lib().orc_model_weight_elems(C.byref(self.cfg))
        if self.blob.size != need:
            raise ValueError(f"blob has {self.blob.size} elements, layout needs {need}")
        self.h = lib().orc_model_create(C.byref(self.cfg), _p(self.blob))

    def encoder_forward(self, tokens) -> None:
        t = _i32(tokens)
        rc = lib().orc_encoder_forward(self.h, _p(t), len(t))
        if rc:
            raise ValueError(f"orc_encoder_forward failed ({rc})")

    def review_forward(self, tokens, kv_len: int) -> np.ndarray:
        t = _i32(tokens)
        out = np.zeros((len(t), self.shape.vocab), dtype=np.float32)
        rc = lib().orc_review_forward(self.h, _p(t), len(t), kv_len, _p(out))
        if rc:
            raise ValueError(f"orc_review_forward failed ({rc})")
        return out

    def close(self):
        if self.h:
            lib().orc_model_destroy(self.h)
            self.h = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass


def blob_to_u16(blob) -> np.ndarray:
    """torch bf16 tensor (any device) -> host uint16 numpy array."""
    import torch
    return blob.detach().to("cpu").contiguous().view(torch.int16).numpy().view(np.uint16)


def cascade_generate(models: Sequence[Model], haystack, bigram_next, K, max_block: int,
                     init_seq, max_new: int, temperature: float = 0.0, lenience: float = 1.0,
                     seed: int = 0, max_order: int = 16, dynamic_haystack: bool = False):
    """Returns (tokens, margins, stats dict).  models[0] is the target."""
    n = len(models)
    arr = (C.c_void_p * n)(*[m.h for m in models])
    hay = _i32(haystack)
    big = _i32(bigram_next)
    Km = _i32(K).reshape(n, n)
    init = _i32(init_seq)
    out = np.zeros(max_new + 1, dtype=np.int32)
    margins = np.full(max_new + max_block + 2, np.inf, dtype=np.float32)
    out_len = C.c_int32(0)
    st = Stats()
    rc = lib().orc_cascade_generate(arr, n, _p(hay), len(hay), _p(big), max_order, _p(Km), max_block,
                                    lenience, temperature, seed, _p(init), len(init), max_new,
                                    int(dynamic_haystack), _p(out), C.byref(out_len), _p(margins), C.byref(st))
    if rc:
        raise ValueError(f"orc_cascade_generate failed ({rc})")
    return out[:out_len.value].copy(), margins[:out_len.value].copy(), st.as_dict(n)


# --------------------------------------------------------------------------------------------
# Tree-shaped review (Section 5.1 and Appendix B combine CS Drafting with tree attention: several
# candidate continuations are reviewed in one pass and the longest accepted path wins).  The plain
# definition: a node's law is the model's next-token law after the prefix followed by the tokens
# on the path from the root to that node; greedy acceptance walks down from the root as long as
# the target's arg-max is among the current node's children.
# --------------------------------------------------------------------------------------------

def tree_paths(parent: Sequence[int]) -> List[List[int]]:
    """Row indices from the root (row 0, parent -1) to every node; parents precede children."""
    paths: List[List[int]] = []
    for r, p in enumerate(parent):
        if r == 0:
            if p != -1:
                raise ValueError("row 0 is the root (parent -1)")
            paths.append([0])
        else:
            if not (0 <= p < r):
                raise ValueError("a parent must precede its child")
            paths.append(paths[p] + [r])
    return paths


def tree_review_forward(model: Model, tokens, parent: Sequence[int], kv_len: int) -> np.ndarray:
    """Logits [m, vocab]: row r = the model's law after cache[0:kv_len] + the tokens on the path to node r.
    One plain forward per node (the cache rows from kv_len on are overwritten every time)."""
    t = _i32(tokens)
    out = np.zeros((len(t), model.shape.vocab), dtype=np.float32)
    for r, path in enumerate(tree_paths(parent)):
        out[r] = model.review_forward(t[path], kv_len)[-1]
    return out


def tree_accept_greedy(logits, tokens, parent: Sequence[int]):
    """Greedy walk: returns (emitted tokens, rows of the accepted path starting with the root).
    At the current node the target's arg-max (smallest index on ties) is emitted; if a child holds
    that token (the child with the smallest row index if several do) the walk moves there."""
    lg = _f32(logits)
    t = _i32(tokens)
    cur, out, path = 0, [], [0]
    while True:
        y = int(np.argmax(lg[cur]))
        out.append(y)
        nxt = [c for c in range(cur + 1, len(t)) if parent[c] == cur and int(t[c]) == y]
        if not nxt:
            return np.asarray(out, dtype=np.int32), path
        cur = nxt[0]
        path.append(cur)
