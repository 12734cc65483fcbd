"""Thin Python binding of the C ABI in include/csd.h: argument marshalling only.

PyTorch provides device memory and the CUDA stream; every step of the path runs in the library's
own kernels.  There is no CPU fallback: if `libcsd.so` has not been built, importing this
module raises.
"""
from __future__ import annotations

import ctypes as C
import os
from typing import Optional, Sequence

import numpy as np
import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libcsd.so")

if not os.path.exists(LIB_PATH):
    raise ImportError(f"{LIB_PATH} is missing: build it with `python -m paper_2312_11462_b200.build` "
                      "(nvcc, sm_100a); this package has no fallback path")

lib = C.CDLL(LIB_PATH)

CSD_OK = 0
STATUS_NAMES = {0: "CSD_OK", 1: "CSD_ERR_INVALID_ARG", 2: "CSD_ERR_SHAPE", 3: "CSD_ERR_CAPACITY", 4: "CSD_ERR_OOM",
                5: "CSD_ERR_CUDA", 6: "CSD_ERR_BAD_TOKEN", 7: "CSD_ERR_TIMEOUT", 8: "CSD_ERR_UNSUPPORTED"}


class CsdError(RuntimeError):
    def __init__(self, call: str, code: int):
        self.code = code
        detail = lib.csd_status_string(code).decode()
        if code == 5:
            detail += ": " + lib.csd_last_cuda_error().decode()
        super().__init__(f"{call} -> {STATUS_NAMES.get(code, code)} ({detail})")


class ModelConfig(C.Structure):
    _fields_ = [(n, C.c_int32) for n in
                ("arch", "n_layers", "n_enc_layers", "d_model", "n_heads", "d_head", "d_ff", "vocab",
                 "max_seq", "max_rows", "max_enc_len", "rel_buckets", "rel_max_dist")] + \
               [("norm_eps", C.c_float), ("rope_theta", C.c_float)]


class CascadeStats(C.Structure):
    _fields_ = [("tokens", C.c_int64), ("reviews", C.c_int64 * 8), ("forwards", C.c_int64 * 8),
                ("drafted", C.c_int64 * 8), ("accepted", C.c_int64 * 8), ("mag_calls", C.c_int64),
                ("mag_tokens", C.c_int64), ("kernel_launches", C.c_int64), ("prefill_ms", C.c_double),
                ("decode_ms", C.c_double), ("total_ms", C.c_double)]

    def as_dict(self, n_levels: int):
        return dict(tokens=self.tokens, reviews=list(self.reviews)[:n_levels],
                    forwards=list(self.forwards)[:n_levels], drafted=list(self.drafted)[:n_levels],
                    accepted=list(self.accepted)[:n_levels], mag_calls=self.mag_calls, mag_tokens=self.mag_tokens,
                    kernel_launches=self.kernel_launches, prefill_ms=self.prefill_ms, decode_ms=self.decode_ms,
                    total_ms=self.total_ms)


class Profile(C.Structure):
    _fields_ = [("gemm_ms", C.c_double), ("gemm_launches", C.c_int64), ("gemm_weight_bytes", C.c_double),
                ("attn_ms", C.c_double), ("attn_launches", C.c_int64), ("other_ms", C.c_double),
                ("other_launches", C.c_int64)]


_vp, _i, _sz, _f, _u64 = C.c_void_p, C.c_int, C.c_size_t, C.c_float, C.c_uint64
lib.csd_status_string.restype = C.c_char_p
lib.csd_status_string.argtypes = [_i]
lib.csd_last_cuda_error.restype = C.c_char_p
lib.csd_device_status.argtypes = [_vp, _vp]
lib.csd_model_weight_bytes.restype = _sz
lib.csd_model_weight_bytes.argtypes = [_vp]
lib.csd_model_workspace_bytes.restype = _sz
lib.csd_model_workspace_bytes.argtypes = [_vp]
lib.csd_model_create.argtypes = [_vp, _vp, _sz, _vp, _sz, _vp, _vp]
lib.csd_model_destroy.argtypes = [_vp]
lib.csd_encoder_forward.argtypes = [_vp, _vp, _i, _vp]
lib.csd_review_forward.argtypes = [_vp, _vp, _i, _i, _vp, _vp]
lib.csd_prefill.argtypes = [_vp, _vp, _i, _i, _vp]
lib.csd_review_forward_tree.argtypes = [_vp, _vp, _vp, _i, _i, _vp, _vp]
lib.csd_review_forward_batch.argtypes = [_vp, _i, _vp, _vp, _vp, _vp, _vp]
lib.csd_tree_accept_greedy.argtypes = [_vp, _vp, _vp, _i, _i, _vp, _vp]
lib.csd_model_profile.argtypes = [_vp, _i]
lib.csd_model_profile_read.argtypes = [_vp, _vp, _vp]
lib.csd_set_gemm_path.argtypes = [_i]
lib.csd_set_attention_path.argtypes = [_i]
lib.csd_linear_workspace_bytes.restype = _sz
lib.csd_linear_workspace_bytes.argtypes = [_i, _i, _i]
lib.csd_linear.argtypes = [_vp, _i, _i, _vp, _i, _vp, _vp, _sz, _vp]
lib.csd_spec_accept_workspace_bytes.restype = _sz
lib.csd_spec_accept_workspace_bytes.argtypes = [_i, _i, _i]
lib.csd_spec_accept.argtypes = [_vp, _vp, _vp, _vp, _i, _i, _i, _f, _f, _u64, _u64, _vp, _vp, _vp, _sz, _vp]
lib.csd_spec_accept_static_capacity.restype = _sz
lib.csd_spec_accept_static.argtypes = [_vp, _vp, _vp, _vp, _i, _i, _i, _f, _f, _u64, _u64, _vp, _vp, _vp]
lib.csd_mag_workspace_bytes.restype = _sz
lib.csd_mag_workspace_bytes.argtypes = [_i, _i, _i]
lib.csd_mag_create.argtypes = [_vp, _i, _i, _vp, _i, _i, _vp, _sz, _vp, _vp]
lib.csd_mag_destroy.argtypes = [_vp]
lib.csd_mag_draft.argtypes = [_vp, _vp, _i, _i, _vp, _vp]
lib.csd_mag_draft_dynamic.argtypes = [_vp, _vp, _i, _i, _i, _vp, _vp]
lib.csd_cascade_workspace_bytes.restype = _sz
lib.csd_cascade_workspace_bytes.argtypes = [_i, _i, _i, _i, _i]
lib.csd_cascade_generate.argtypes = [_vp, _i, _vp, _i, _f, _f, _u64, _i, _i, _vp, _i, _vp, _vp, _i, _i, _vp, _vp, _vp,
                                     _vp, _sz, _vp]
lib.csd_rel_bucket.argtypes = [_i, _i, _i, _i]


def _check(call: str, code: int) -> None:
    if code != CSD_OK:
        raise CsdError(call, code)


def _stream() -> int:
    return torch.cuda.current_stream().cuda_stream


def _ptr(t: Optional[torch.Tensor]):
    return None if t is None else t.data_ptr()


def _ws(nbytes: int, device) -> torch.Tensor:
    """Zero-filled, 256-byte aligned device scratch."""
    return torch.zeros(max(int(nbytes), 256), dtype=torch.uint8, device=device)


def config_from_shape(s) -> ModelConfig:
    return ModelConfig(s.arch, s.n_layers, s.n_enc_layers, s.d_model, s.n_heads, s.d_head, s.d_ff, s.vocab,
                       s.max_seq, s.max_rows, s.max_enc_len, s.rel_buckets, s.rel_max_dist, s.norm_eps,
                       s.rope_theta)


def csd_device_status() -> int:
    code = C.c_int(0)
    _check("csd_device_status", lib.csd_device_status(_stream(), C.byref(code)))
    return code.value


def csd_rel_bucket(rel: int, bidirectional: bool, n_buckets: int = 32, max_dist: int = 128) -> int:
    return int(lib.csd_rel_bucket(rel, int(bidirectional), n_buckets, max_dist))


class Model:
    """csd_model bound to a bf16 weight blob (torch tensor on the GPU) and its workspace."""

    def __init__(self, shape, weights: torch.Tensor):
        assert weights.dtype == torch.bfloat16 and weights.is_cuda and weights.is_contiguous()
        self.shape = shape
        self.cfg = config_from_shape(shape)
        self.weights = weights
        need = lib.csd_model_weight_bytes(C.byref(self.cfg))
        if need == 0:
            raise CsdError("csd_model_weight_bytes", 2)
        self.workspace = _ws(lib.csd_model_workspace_bytes(C.byref(self.cfg)), weights.device)
        h = C.c_void_p()
        _check("csd_model_create",
               lib.csd_model_create(C.byref(self.cfg), _ptr(weights), weights.numel() * 2, _ptr(self.workspace),
                                    self.workspace.numel(), _stream(), C.byref(h)))
        self.h = h

    def csd_encoder_forward(self, enc_tokens: torch.Tensor) -> None:
        assert enc_tokens.dtype == torch.int32 and enc_tokens.is_cuda
        _check("csd_encoder_forward", lib.csd_encoder_forward(self.h, _ptr(enc_tokens), enc_tokens.numel(), _stream()))

    def csd_review_forward(self, block_tokens: torch.Tensor, kv_len: int,
                           logits_out: Optional[torch.Tensor] = None, append_only: bool = False):
        """Returns the logits [m, vocab]; with append_only the block only enters the cache (no logits)."""
        assert block_tokens.dtype == torch.int32 and block_tokens.is_cuda
        m = block_tokens.numel()
        if append_only:
            _check("csd_review_forward", lib.csd_review_forward(self.h, _ptr(block_tokens), m, kv_len, None, _stream()))
            return None
        if logits_out is None:
            logits_out = torch.empty(m, self.shape.vocab, dtype=torch.float32, device=block_tokens.device)
        _check("csd_review_forward",
               lib.csd_review_forward(self.h, _ptr(block_tokens), m, kv_len, _ptr(logits_out), _stream()))
        return logits_out

    def csd_review_forward_tree(self, block_tokens: torch.Tensor, parent, kv_len: int) -> torch.Tensor:
        """Logits [m, vocab] of a tree-shaped block; parent[r] < r is the row of r's parent, parent[0] = -1."""
        assert block_tokens.dtype == torch.int32 and block_tokens.is_cuda
        m = block_tokens.numel()
        par = np.ascontiguousarray(np.asarray(parent, dtype=np.int32))
        assert par.size == m
        out = torch.empty(m, self.shape.vocab, dtype=torch.float32, device=block_tokens.device)
        _check("csd_review_forward_tree",
               lib.csd_review_forward_tree(self.h, _ptr(block_tokens), par.ctypes.data_as(_vp), m, kv_len, _ptr(out), _stream()))
        return out

    def csd_prefill(self, tokens: torch.Tensor, kv_len: int) -> None:
        """Appends the tokens to the cache (wide blocks where the model allows them); no logits."""
        assert tokens.dtype == torch.int32 and tokens.is_cuda and tokens.is_contiguous()
        _check("csd_prefill", lib.csd_prefill(self.h, _ptr(tokens), tokens.numel(), kv_len, _stream()))

    def csd_model_profile(self, enable: bool) -> None:
        _check("csd_model_profile", lib.csd_model_profile(self.h, int(enable)))

    def csd_model_profile_read(self) -> dict:
        p = Profile()
        _check("csd_model_profile_read", lib.csd_model_profile_read(self.h, _stream(), C.byref(p)))
        return {n: getattr(p, n) for n, _ in Profile._fields_}

    def close(self) -> None:
        if getattr(self, "h", None):
            lib.csd_model_destroy(self.h)
            self.h = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass


def csd_linear(W: torch.Tensor, X: torch.Tensor, workspace: Optional[torch.Tensor] = None,
               out: Optional[torch.Tensor] = None) -> torch.Tensor:
    """Y = X . W^T; W bf16 [N, K], X fp32 [m, K] (both on the GPU)."""
    assert W.dtype == torch.bfloat16 and X.dtype == torch.float32 and W.is_contiguous() and X.is_contiguous()
    N, K = W.shape
    m = X.shape[0]
    if workspace is None:
        workspace = _ws(lib.csd_linear_workspace_bytes(m, N, K), W.device)
    if out is None:
        out = torch.empty(m, N, dtype=torch.float32, device=W.device)
    _check("csd_linear", lib.csd_linear(_ptr(W), N, K, _ptr(X), m, _ptr(out), _ptr(workspace), workspace.numel(),
                                        _stream()))
    return out


def csd_review_forward_batch(models: Sequence["Model"], blocks: Sequence[torch.Tensor], kv_lens: Sequence[int],
                             append_only: bool = False):
    """One pass over the weights for the blocks of several sequences (models share weights and shape,
    each has its own cache).  Returns the list of logits tensors, one per sequence."""
    n = len(models)
    rows = np.asarray([b_.numel() for b_ in blocks], dtype=np.int32)
    kv = np.asarray(kv_lens, dtype=np.int32)
    toks = torch.cat([b_.reshape(-1) for b_ in blocks]).contiguous()
    assert toks.dtype == torch.int32 and toks.is_cuda
    handles = (C.c_void_p * n)(*[m.h for m in models])
    out = None if append_only else torch.empty(int(rows.sum()), models[0].shape.vocab, dtype=torch.float32, device=toks.device)
    _check("csd_review_forward_batch",
           lib.csd_review_forward_batch(handles, n, _ptr(toks), rows.ctypes.data_as(_vp), kv.ctypes.data_as(_vp),
                                        _ptr(out), _stream()))
    if out is None:
        return None
    return list(torch.split(out, [int(r) for r in rows]))


def csd_tree_accept_greedy(target_logits: torch.Tensor, tokens: torch.Tensor, parent):
    """Returns (emitted tokens, rows of the accepted path, number of leading path rows valid in the cache)."""
    m, V = target_logits.shape
    assert target_logits.dtype == torch.float32 and target_logits.is_contiguous() and tokens.dtype == torch.int32
    par = np.ascontiguousarray(np.asarray(parent, dtype=np.int32))
    out = torch.zeros(2 + 3 * m, dtype=torch.int32, device=target_logits.device)
    _check("csd_tree_accept_greedy",
           lib.csd_tree_accept_greedy(_ptr(target_logits), _ptr(tokens), par.ctypes.data_as(_vp), m, V, _ptr(out), _stream()))
    o = out.cpu().numpy()
    n = int(o[0])
    return o[2:2 + n].copy(), o[2 + m:2 + m + n].copy(), int(o[1])


def csd_set_gemm_path(path: int) -> None:
    _check("csd_set_gemm_path", lib.csd_set_gemm_path(path))


def csd_set_attention_path(path: int) -> None:
    _check("csd_set_attention_path", lib.csd_set_attention_path(path))


def csd_linear_workspace(m: int, N: int, K: int, device) -> torch.Tensor:
    return _ws(lib.csd_linear_workspace_bytes(m, N, K), device)


def csd_spec_accept_workspace(rows: int, k: int, V: int, device) -> torch.Tensor:
    return _ws(lib.csd_spec_accept_workspace_bytes(rows, k, V), device)


def csd_spec_accept(target_logits: torch.Tensor, draft_logits: Optional[torch.Tensor], draft_tokens: torch.Tensor,
                    temperature: float, lenience: float = 1.0, seed: int = 0, step: int = 0,
                    onehot: Optional[torch.Tensor] = None, workspace: Optional[torch.Tensor] = None,
                    out: Optional[Sequence[torch.Tensor]] = None):
    """Returns (n_accepted [rows] int32, out_token [rows] int32), both on the GPU."""
    rows, k1, V = target_logits.shape
    k = k1 - 1
    assert target_logits.dtype == torch.float32 and target_logits.is_contiguous()
    assert draft_tokens.dtype == torch.int32 and draft_tokens.is_contiguous()
    if draft_logits is not None:
        assert draft_logits.dtype == torch.float32 and draft_logits.is_contiguous()
        assert tuple(draft_logits.shape) == (rows, k, V)
    if onehot is not None:
        assert onehot.dtype == torch.int32 and onehot.is_contiguous()
    dev = target_logits.device
    if workspace is None:
        workspace = csd_spec_accept_workspace(rows, k, V, dev)
    if out is None:
        out = (torch.empty(rows, dtype=torch.int32, device=dev), torch.empty(rows, dtype=torch.int32, device=dev))
    _check("csd_spec_accept",
           lib.csd_spec_accept(_ptr(target_logits), _ptr(draft_logits), _ptr(onehot), _ptr(draft_tokens), rows, k, V,
                               temperature, lenience, seed, step, _ptr(out[0]), _ptr(out[1]), _ptr(workspace),
                               workspace.numel(), _stream()))
    return out


def csd_spec_accept_static(target_logits: torch.Tensor, draft_logits: Optional[torch.Tensor],
                           draft_tokens: torch.Tensor, temperature: float, lenience: float = 1.0, seed: int = 0,
                           step: int = 0, onehot: Optional[torch.Tensor] = None, out: Sequence[torch.Tensor] = None):
    """The review rule through the entry point that allocates nothing: the caller supplies every
    buffer, outputs included (`out` = (n_accepted, out_token), int32 [rows] each)."""
    rows, k1, V = target_logits.shape
    assert out is not None and out[0].dtype == torch.int32 and out[1].dtype == torch.int32
    _check("csd_spec_accept_static",
           lib.csd_spec_accept_static(_ptr(target_logits), _ptr(draft_logits), _ptr(onehot), _ptr(draft_tokens), rows,
                                      k1 - 1, V, temperature, lenience, seed, step, _ptr(out[0]), _ptr(out[1]),
                                      _stream()))
    return out


class Mag:
    """csd_mag over a haystack and a bigram successor table (int32 tensors on the GPU)."""

    def __init__(self, haystack: torch.Tensor, bigram_next: torch.Tensor, max_order: int = 16, table_slots: int = 0):
        assert haystack.dtype == torch.int32 and bigram_next.dtype == torch.int32
        self.haystack, self.bigram = haystack.contiguous(), bigram_next.contiguous()
        nbytes = lib.csd_mag_workspace_bytes(haystack.numel(), max_order, table_slots)
        self.workspace = _ws(nbytes, bigram_next.device)
        h = C.c_void_p()
        _check("csd_mag_create",
               lib.csd_mag_create(_ptr(self.haystack), haystack.numel(), bigram_next.numel(), _ptr(self.bigram),
                                  max_order, table_slots, _ptr(self.workspace), self.workspace.numel(), _stream(),
                                  C.byref(h)))
        self.h = h

    def csd_mag_draft(self, seq: torch.Tensor, n: int) -> torch.Tensor:
        assert seq.dtype == torch.int32 and seq.is_cuda and seq.is_contiguous()
        out = torch.empty(n, dtype=torch.int32, device=seq.device)
        _check("csd_mag_draft", lib.csd_mag_draft(self.h, _ptr(seq), seq.numel(), n, _ptr(out), _stream()))
        return out

    def csd_mag_draft_dynamic(self, seq: torch.Tensor, gen_from: int, n: int) -> torch.Tensor:
        """Haystack = the handle's haystack followed by seq[gen_from:]."""
        assert seq.dtype == torch.int32 and seq.is_cuda and seq.is_contiguous()
        out = torch.empty(n, dtype=torch.int32, device=seq.device)
        _check("csd_mag_draft_dynamic",
               lib.csd_mag_draft_dynamic(self.h, _ptr(seq), seq.numel(), gen_from, n, _ptr(out), _stream()))
        return out

    def close(self) -> None:
        if getattr(self, "h", None):
            lib.csd_mag_destroy(self.h)
            self.h = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass


class Cascade:
    """Holds the workspace of csd_cascade_generate for a fixed set of models."""

    def __init__(self, models: Sequence[Model], K, max_block: int, bigram_next: torch.Tensor, max_haystack: int,
                 max_order: int = 16):
        self.models = list(models)
        n = len(self.models)
        self.K = np.ascontiguousarray(np.asarray(K, dtype=np.int32).reshape(n, n))
        self.max_block, self.max_order = max_block, max_order
        self.bigram = bigram_next.contiguous()
        assert self.bigram.dtype == torch.int32 and self.bigram.is_cuda
        cap = min(m.shape.max_seq for m in self.models)
        nbytes = lib.csd_cascade_workspace_bytes(self.models[0].shape.vocab, max_block, cap, max_haystack, max_order)
        if nbytes == 0:
            raise CsdError("csd_cascade_workspace_bytes", 1)
        self.max_haystack = max_haystack
        self.workspace = _ws(nbytes, self.bigram.device)
        self.handles = (C.c_void_p * n)(*[m.h for m in self.models])

    def csd_cascade_generate(self, haystack: np.ndarray, init_seq: np.ndarray, max_new: int,
                             temperature: float = 0.0, lenience: float = 1.0, seed: int = 0,
                             dynamic_haystack: bool = False):
        """Host in, host out.  Returns (tokens int32 numpy, stats dict)."""
        hay = np.ascontiguousarray(haystack, dtype=np.int32)
        init = np.ascontiguousarray(init_seq, dtype=np.int32)
        assert len(hay) <= self.max_haystack
        out = np.zeros(max(max_new, 1), dtype=np.int32)
        out_len = C.c_int32(0)
        st = CascadeStats()
        code = lib.csd_cascade_generate(self.handles, len(self.models), self.K.ctypes.data_as(_vp), self.max_block,
                                        lenience, temperature, seed, self.max_order, int(dynamic_haystack),
                                        hay.ctypes.data_as(_vp),
                                        len(hay), _ptr(self.bigram), init.ctypes.data_as(_vp), len(init), max_new,
                                        out.ctypes.data_as(_vp), C.byref(out_len), C.byref(st), _ptr(self.workspace),
                                        self.workspace.numel(), _stream())
        _check("csd_cascade_generate", code)
        return out[:out_len.value].copy(), st.as_dict(len(self.models))
