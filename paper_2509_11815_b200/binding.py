"""Thin ctypes binding of libspecvlm.so (argument marshalling only).

Every function has the name of the C entry point it calls (include/specvlm.h) and takes
torch CUDA tensors; torch is used for device memory and streams only. All work runs in
the library's CUDA kernels on the current torch stream. There is no CPU fallback: if the
shared library is missing, loading raises.
"""

from __future__ import annotations

import ctypes
import os
from typing import Optional

import torch

_PKG_DIR = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_PKG_DIR, "lib", "libspecvlm.so")

SPECVLM_OK = 0
STATUS_BAD_PREFIX, STATUS_BAD_TREE, STATUS_BAD_ACCEPT, STATUS_TIMEOUT = 1, 2, 4, 8

EXPORTS = (
    "specvlm_version",
    "specvlm_last_error_string",
    "specvlm_attn_workspace_bytes",
    "specvlm_workspace_init",
    "specvlm_tree_build",
    "specvlm_tree_validate_host",
    "specvlm_tree_verify_attn",
    "specvlm_tree_verify_attn_static",
    "specvlm_visual_pool",
    "specvlm_visual_prune",
    "specvlm_topk_logprob",
    "specvlm_tree_rerank",
    "specvlm_rope_append",
    "specvlm_argmax",
    "specvlm_accept",
    "specvlm_accept_sample",
    "specvlm_kv_compact",
    "specvlm_accept_compact",
    "specvlm_verify_step",
    "specvlm_verify_step_sample",
)


class SpecvlmError(RuntimeError):
    pass


class AttnDesc(ctypes.Structure):
    _fields_ = [
        ("B", ctypes.c_int32), ("H", ctypes.c_int32), ("T", ctypes.c_int32), ("D", ctypes.c_int32),
        ("S_cap", ctypes.c_int32), ("num_splits", ctypes.c_int32),
        ("softmax_scale", ctypes.c_float), ("flags", ctypes.c_int32),
        ("q_stride_b", ctypes.c_int64), ("q_stride_h", ctypes.c_int64), ("q_stride_t", ctypes.c_int64),
        ("k_stride_b", ctypes.c_int64), ("k_stride_h", ctypes.c_int64), ("k_stride_s", ctypes.c_int64),
        ("v_stride_b", ctypes.c_int64), ("v_stride_h", ctypes.c_int64), ("v_stride_s", ctypes.c_int64),
        ("o_stride_b", ctypes.c_int64), ("o_stride_h", ctypes.c_int64), ("o_stride_t", ctypes.c_int64),
    ]


class KvDesc(ctypes.Structure):
    _fields_ = [
        ("L", ctypes.c_int32), ("B", ctypes.c_int32), ("H", ctypes.c_int32), ("S_cap", ctypes.c_int32),
        ("D", ctypes.c_int32), ("reserved", ctypes.c_int32),
        ("stride_l", ctypes.c_int64), ("stride_b", ctypes.c_int64), ("stride_h", ctypes.c_int64),
        ("stride_s", ctypes.c_int64),
    ]


class RopeDesc(ctypes.Structure):
    _fields_ = ([("B", ctypes.c_int32), ("H", ctypes.c_int32), ("T", ctypes.c_int32), ("D", ctypes.c_int32),
                 ("S_cap", ctypes.c_int32), ("rope_base", ctypes.c_float)] +
                [(f"{n}_stride_{a}", ctypes.c_int64) for n, axes in (("qi", "bht"), ("kn", "bht"), ("vn", "bht"),
                                                                      ("qo", "bht"), ("kc", "bhs"), ("vc", "bhs"))
                 for a in axes])


_lib = None


def load_library(path: Optional[str] = None) -> ctypes.CDLL:
    """Load libspecvlm.so (built by `python -m paper_2509_11815_b200.build`). Raises if absent."""
    global _lib
    if _lib is not None and path is None:
        return _lib
    p = path or LIB_PATH
    if not os.path.exists(p):
        raise SpecvlmError(
            f"CUDA library not found at {p}; build it with `python -m paper_2509_11815_b200.build` "
            "(there is no CPU fallback)")
    lib = ctypes.CDLL(p)
    vp, i32, i64 = ctypes.c_void_p, ctypes.c_int, ctypes.c_int64
    lib.specvlm_version.restype = i32
    lib.specvlm_version.argtypes = []
    lib.specvlm_last_error_string.restype = ctypes.c_char_p
    lib.specvlm_last_error_string.argtypes = []
    lib.specvlm_attn_workspace_bytes.restype = i32
    lib.specvlm_attn_workspace_bytes.argtypes = [ctypes.POINTER(AttnDesc), ctypes.POINTER(ctypes.c_size_t)]
    lib.specvlm_workspace_init.restype = i32
    lib.specvlm_workspace_init.argtypes = [vp, ctypes.c_size_t, vp]
    lib.specvlm_tree_build.restype = i32
    lib.specvlm_tree_build.argtypes = [vp, vp, i32, i32, vp, vp, vp, vp, vp]
    lib.specvlm_tree_validate_host.restype = i32
    lib.specvlm_tree_validate_host.argtypes = [vp, vp, i32]
    lib.specvlm_tree_verify_attn.restype = i32
    lib.specvlm_tree_verify_attn.argtypes = [vp, vp, vp, vp, vp, vp, vp, ctypes.POINTER(AttnDesc), vp, vp, vp]
    lib.specvlm_tree_verify_attn_static.restype = i32
    lib.specvlm_tree_verify_attn_static.argtypes = [vp, vp, vp, vp, vp, vp, vp, ctypes.POINTER(AttnDesc), vp, vp]
    lib.specvlm_visual_pool.restype = i32
    lib.specvlm_visual_pool.argtypes = [vp, i32, i32, i32, i32, vp, vp]
    lib.specvlm_visual_prune.restype = i32
    lib.specvlm_visual_prune.argtypes = [vp, vp, i32, i32, i32, i32, vp, vp, vp]
    lib.specvlm_topk_logprob.restype = i32
    lib.specvlm_topk_logprob.argtypes = [vp, i32, i32, i64, i32, vp, vp, vp]
    lib.specvlm_tree_rerank.restype = i32
    lib.specvlm_tree_rerank.argtypes = [vp, vp, vp, vp, i32, i32, i32, vp, vp, vp, vp, vp, vp, vp, vp]
    lib.specvlm_rope_append.restype = i32
    lib.specvlm_rope_append.argtypes = [vp, vp, vp, vp, vp, vp, vp, vp, ctypes.POINTER(RopeDesc), vp, vp, vp]
    lib.specvlm_argmax.restype = i32
    lib.specvlm_argmax.argtypes = [vp, i32, i32, i32, i64, vp, vp]
    lib.specvlm_accept.restype = i32
    lib.specvlm_accept.argtypes = [vp, vp, vp, vp, i32, i32, i32, vp, i32, vp, vp, vp, vp]
    lib.specvlm_accept_sample.restype = i32
    lib.specvlm_accept_sample.argtypes = [vp, vp, vp, vp, vp, ctypes.c_float, i32, i32, i32, vp, i32, vp, vp, vp, vp,
                                          vp]
    lib.specvlm_kv_compact.restype = i32
    lib.specvlm_kv_compact.argtypes = [vp, vp, ctypes.POINTER(KvDesc), vp, vp, i32, vp, vp, vp, vp]
    lib.specvlm_accept_compact.restype = i32
    lib.specvlm_accept_compact.argtypes = [vp, vp, vp, i32, vp, vp, ctypes.POINTER(KvDesc), vp, vp, i32,
                                           vp, vp, vp, vp, vp]
    lib.specvlm_verify_step_sample.restype = i32
    lib.specvlm_verify_step_sample.argtypes = [vp, i64, vp, vp, ctypes.POINTER(KvDesc), vp, vp, vp, vp, vp, vp, vp,
                                               ctypes.c_float, i32, i32, vp, i64, vp, vp, i32, vp, vp, vp, i32, vp, vp,
                                               vp]
    lib.specvlm_verify_step.restype = i32
    lib.specvlm_verify_step.argtypes = [vp, i64, vp, vp, ctypes.POINTER(KvDesc), vp, vp, vp, vp, vp, i32, i32, vp, i64,
                                        vp, vp, i32, vp, vp, vp, i32, vp, vp, vp]
    if path is None:
        _lib = lib
    return lib


def _check(rc: int) -> None:
    if rc != SPECVLM_OK:
        msg = load_library().specvlm_last_error_string().decode("utf-8", "replace")
        raise SpecvlmError(f"specvlm error {rc}: {msg}")


def _ptr(t: Optional[torch.Tensor]) -> Optional[int]:
    return None if t is None else t.data_ptr()


def _stream() -> int:
    return torch.cuda.current_stream().cuda_stream


def _need(t: torch.Tensor, dtype, name: str) -> None:
    if not t.is_cuda:
        raise SpecvlmError(f"{name} must be a CUDA tensor")
    ok = t.dtype in dtype if isinstance(dtype, tuple) else t.dtype == dtype
    if not ok:
        raise SpecvlmError(f"{name} has dtype {t.dtype}, expected {dtype}")


_MASK_DTYPES = (torch.int64, torch.uint64)


def specvlm_version() -> int:
    return load_library().specvlm_version()


ATTN_FLAG_LEGACY_MMA = 1
ATTN_FLAG_PREFIX_STABLE = 2
ATTN_FLAG_INPUTS_STABLE = 4
ATTN_FLAG_HALF_SM = 8


def make_attn_desc(q: torch.Tensor, k_cache: torch.Tensor, v_cache: torch.Tensor, out: torch.Tensor,
                   num_splits: int = 0, softmax_scale: float = 0.0, flags: int = 0) -> AttnDesc:
    """q/out: [B][H][T][D] views, k/v: [B][H][S_cap][D] views (any strides, D contiguous)."""
    B, H, T, D = q.shape
    for name, t in (("q", q), ("k_cache", k_cache), ("v_cache", v_cache), ("out", out)):
        _need(t, torch.bfloat16, name)
        if t.dim() != 4 or t.stride(3) != 1:
            raise SpecvlmError(f"{name} must be 4-D with a contiguous last dimension")
    if k_cache.shape != v_cache.shape or k_cache.shape[:2] != (B, H) or k_cache.shape[3] != D:
        raise SpecvlmError("k_cache / v_cache must be [B][H][S_cap][D]")
    if out.shape != q.shape:
        raise SpecvlmError("out must have q's shape")
    d = AttnDesc()
    d.B, d.H, d.T, d.D, d.S_cap = B, H, T, D, k_cache.shape[2]
    d.num_splits, d.softmax_scale, d.flags = num_splits, softmax_scale, flags
    d.q_stride_b, d.q_stride_h, d.q_stride_t = q.stride(0), q.stride(1), q.stride(2)
    d.k_stride_b, d.k_stride_h, d.k_stride_s = k_cache.stride(0), k_cache.stride(1), k_cache.stride(2)
    d.v_stride_b, d.v_stride_h, d.v_stride_s = v_cache.stride(0), v_cache.stride(1), v_cache.stride(2)
    d.o_stride_b, d.o_stride_h, d.o_stride_t = out.stride(0), out.stride(1), out.stride(2)
    return d


def specvlm_attn_workspace_bytes(desc: AttnDesc) -> int:
    n = ctypes.c_size_t(0)
    _check(load_library().specvlm_attn_workspace_bytes(ctypes.byref(desc), ctypes.byref(n)))
    return int(n.value)


def specvlm_workspace_init(workspace: torch.Tensor) -> None:
    _check(load_library().specvlm_workspace_init(workspace.data_ptr(), workspace.numel() * workspace.element_size(),
                                                 _stream()))


def alloc_attn_workspace(desc: AttnDesc, device) -> torch.Tensor:
    """Allocate and zero a workspace for this descriptor (torch owns the memory)."""
    n = max(specvlm_attn_workspace_bytes(desc), 256)
    ws = torch.empty(n, dtype=torch.uint8, device=device)
    specvlm_workspace_init(ws)
    return ws


def specvlm_tree_build(tree_parent: torch.Tensor, prefix_len: Optional[torch.Tensor], mask_bits: torch.Tensor,
                       depth: Optional[torch.Tensor] = None, pos: Optional[torch.Tensor] = None,
                       status: Optional[torch.Tensor] = None) -> None:
    _need(tree_parent, torch.int32, "tree_parent")
    _need(mask_bits, _MASK_DTYPES, "mask_bits")
    B, T = tree_parent.shape
    _check(load_library().specvlm_tree_build(_ptr(tree_parent), _ptr(prefix_len), B, T, _ptr(mask_bits),
                                             _ptr(depth), _ptr(pos), _ptr(status), _stream()))


def specvlm_tree_validate_host(tree_parent, draft_tokens=None) -> int:
    """Host arrays (sequences of int). Returns the C return code (0 = valid)."""
    T = len(tree_parent)
    par = (ctypes.c_int32 * max(T, 1))(*[int(x) for x in tree_parent])
    tok = None
    if draft_tokens is not None:
        tok = (ctypes.c_int32 * max(T, 1))(*[int(x) for x in draft_tokens])
    return load_library().specvlm_tree_validate_host(ctypes.cast(par, ctypes.c_void_p),
                                                     ctypes.cast(tok, ctypes.c_void_p) if tok is not None else None,
                                                     T)


def specvlm_tree_verify_attn(q: torch.Tensor, k_cache: torch.Tensor, v_cache: torch.Tensor,
                             prefix_len: torch.Tensor, tree_parent: Optional[torch.Tensor],
                             tree_mask_bits: Optional[torch.Tensor], out: torch.Tensor,
                             workspace: Optional[torch.Tensor] = None, status: Optional[torch.Tensor] = None,
                             num_splits: int = 0, softmax_scale: float = 0.0,
                             desc: Optional[AttnDesc] = None) -> None:
    """One layer of tree-verification attention; see include/specvlm.h."""
    if desc is None:
        desc = make_attn_desc(q, k_cache, v_cache, out, num_splits, softmax_scale)
    _need(prefix_len, torch.int32, "prefix_len")
    if tree_mask_bits is not None:
        _need(tree_mask_bits, _MASK_DTYPES, "tree_mask_bits")
    if tree_parent is not None:
        _need(tree_parent, torch.int32, "tree_parent")
    _check(load_library().specvlm_tree_verify_attn(
        _ptr(q), _ptr(k_cache), _ptr(v_cache), _ptr(prefix_len), _ptr(tree_parent), _ptr(tree_mask_bits),
        _ptr(out), ctypes.byref(desc), _ptr(workspace), _ptr(status), _stream()))


def specvlm_tree_verify_attn_static(q: torch.Tensor, k_cache: torch.Tensor, v_cache: torch.Tensor,
                                    prefix_len: torch.Tensor, tree_parent: Optional[torch.Tensor],
                                    tree_mask_bits: Optional[torch.Tensor], out: torch.Tensor,
                                    status: Optional[torch.Tensor] = None, num_splits: int = 0,
                                    softmax_scale: float = 0.0, desc: Optional[AttnDesc] = None) -> None:
    """Attention for callers that have no device memory to spare for a workspace (a memory pool
    that already owns the GPU, a decode loop that must not stall on an allocation): the split-KV
    scratch is a fixed array inside the library. Same results as specvlm_tree_verify_attn. Shapes
    beyond the built-in limits (B*H <= 1024, B*H*splits <= 512) raise SpecvlmError. Calls share
    the array, so calls that overlap on the GPU must be ordered by the caller."""
    if desc is None:
        desc = make_attn_desc(q, k_cache, v_cache, out, num_splits, softmax_scale)
    _need(prefix_len, torch.int32, "prefix_len")
    if tree_mask_bits is not None:
        _need(tree_mask_bits, _MASK_DTYPES, "tree_mask_bits")
    if tree_parent is not None:
        _need(tree_parent, torch.int32, "tree_parent")
    _check(load_library().specvlm_tree_verify_attn_static(
        _ptr(q), _ptr(k_cache), _ptr(v_cache), _ptr(prefix_len), _ptr(tree_parent), _ptr(tree_mask_bits),
        _ptr(out), ctypes.byref(desc), _ptr(status), _stream()))


def specvlm_visual_pool(x: torch.Tensor, ratio: int, y: torch.Tensor) -> None:
    """x bf16 [B][N][C] contiguous -> y bf16 [B][ceil(N/ratio)][C]: window means over the token axis."""
    _need(x, torch.bfloat16, "x")
    _need(y, torch.bfloat16, "y")
    if not (x.is_contiguous() and y.is_contiguous()):
        raise SpecvlmError("x and y must be contiguous")
    B, N, C = x.shape
    if tuple(y.shape) != (B, (N + ratio - 1) // max(ratio, 1), C):
        raise SpecvlmError("y must be [B][ceil(N/ratio)][C]")
    _check(load_library().specvlm_visual_pool(_ptr(x), B, N, C, ratio, _ptr(y), _stream()))


def specvlm_visual_prune(x: torch.Tensor, keep_idx: torch.Tensor, y: torch.Tensor,
                         status: Optional[torch.Tensor] = None) -> None:
    """x bf16 [B][N][C], keep_idx int32 [B][M] -> y bf16 [B][M][C]: the kept token rows."""
    _need(x, torch.bfloat16, "x")
    _need(y, torch.bfloat16, "y")
    _need(keep_idx, torch.int32, "keep_idx")
    if not (x.is_contiguous() and y.is_contiguous() and keep_idx.is_contiguous()):
        raise SpecvlmError("x, y and keep_idx must be contiguous")
    B, N, C = x.shape
    M = keep_idx.shape[1]
    _check(load_library().specvlm_visual_prune(_ptr(x), _ptr(keep_idx), B, N, C, M, _ptr(y), _ptr(status), _stream()))


def specvlm_topk_logprob(logits: torch.Tensor, k: int, tokens: torch.Tensor, logprob: torch.Tensor) -> None:
    """logits fp32 [rows][V] (row-strided), tokens int32 [rows][k], logprob fp32 [rows][k]."""
    _need(logits, torch.float32, "logits")
    _need(tokens, torch.int32, "tokens")
    _need(logprob, torch.float32, "logprob")
    if logits.dim() != 2 or logits.stride(1) != 1:
        raise SpecvlmError("logits must be [rows][V] with a contiguous last dimension")
    _check(load_library().specvlm_topk_logprob(_ptr(logits), logits.shape[0], logits.shape[1], logits.stride(0), k,
                                               _ptr(tokens), _ptr(logprob), _stream()))


def specvlm_tree_rerank(cand_parent: torch.Tensor, cand_score: torch.Tensor, cand_token: torch.Tensor, T: int,
                        tree_parent: torch.Tensor, draft_tokens: torch.Tensor,
                        kept_candidates: Optional[torch.Tensor] = None, mask_bits: Optional[torch.Tensor] = None,
                        depth: Optional[torch.Tensor] = None, pos: Optional[torch.Tensor] = None,
                        prefix_len: Optional[torch.Tensor] = None, status: Optional[torch.Tensor] = None) -> None:
    """Rerank [B][C] candidates into [B][T] trees; see include/specvlm.h."""
    _need(cand_parent, torch.int32, "cand_parent")
    _need(cand_score, torch.float32, "cand_score")
    _need(cand_token, torch.int32, "cand_token")
    B, C = cand_parent.shape
    _check(load_library().specvlm_tree_rerank(_ptr(cand_parent), _ptr(cand_score), _ptr(cand_token), _ptr(prefix_len),
                                              B, C, T, _ptr(tree_parent), _ptr(draft_tokens), _ptr(kept_candidates),
                                              _ptr(mask_bits), _ptr(depth), _ptr(pos), _ptr(status), _stream()))


def specvlm_rope_append(q_in: torch.Tensor, k_new: torch.Tensor, v_new: torch.Tensor, prefix_len: torch.Tensor,
                        tree_parent: torch.Tensor, q_out: torch.Tensor, k_cache: torch.Tensor, v_cache: torch.Tensor,
                        pos_out: Optional[torch.Tensor] = None, status: Optional[torch.Tensor] = None,
                        rope_base: float = 0.0) -> None:
    """RoPE of q and the tree's new K rows at prefix_len + depth, and append of the tree's K/V rows
    to one layer's cache. q_in/k_new/v_new/q_out: [B][H][T][D]; k_cache/v_cache: [B][H][S_cap][D]."""
    for name, t in (("q_in", q_in), ("k_new", k_new), ("v_new", v_new), ("q_out", q_out), ("k_cache", k_cache),
                    ("v_cache", v_cache)):
        _need(t, torch.bfloat16, name)
        if t.dim() != 4 or t.stride(3) != 1:
            raise SpecvlmError(f"{name} must be 4-D with a contiguous last dimension")
    _need(prefix_len, torch.int32, "prefix_len")
    _need(tree_parent, torch.int32, "tree_parent")
    B, H, T, D = q_in.shape
    d = RopeDesc()
    d.B, d.H, d.T, d.D, d.S_cap, d.rope_base = B, H, T, D, k_cache.shape[2], rope_base
    for n, t in (("qi", q_in), ("kn", k_new), ("vn", v_new), ("qo", q_out)):
        for a, i in (("b", 0), ("h", 1), ("t", 2)):
            setattr(d, f"{n}_stride_{a}", t.stride(i))
    for n, t in (("kc", k_cache), ("vc", v_cache)):
        for a, i in (("b", 0), ("h", 1), ("s", 2)):
            setattr(d, f"{n}_stride_{a}", t.stride(i))
    _check(load_library().specvlm_rope_append(_ptr(q_in), _ptr(k_new), _ptr(v_new), _ptr(prefix_len),
                                              _ptr(tree_parent), _ptr(q_out), _ptr(k_cache), _ptr(v_cache),
                                              ctypes.byref(d), _ptr(pos_out), _ptr(status), _stream()))


def specvlm_argmax(target_logits: torch.Tensor, argmax_tokens: torch.Tensor) -> None:
    """target_logits fp32 [B][T][V] (rows may be strided), argmax_tokens int32 [B][T]."""
    _need(target_logits, torch.float32, "target_logits")
    _need(argmax_tokens, torch.int32, "argmax_tokens")
    B, T, V = target_logits.shape
    if target_logits.stride(2) != 1 or (B > 1 and target_logits.stride(0) != T * target_logits.stride(1)):
        raise SpecvlmError("target_logits rows must be evenly strided with a contiguous last dimension")
    _check(load_library().specvlm_argmax(_ptr(target_logits), B, T, V, target_logits.stride(1),
                                         _ptr(argmax_tokens), _stream()))


def specvlm_accept(draft_tokens: torch.Tensor, tree_parent: torch.Tensor, target_logits: Optional[torch.Tensor],
                   argmax_tokens: torch.Tensor, accepted_idx: torch.Tensor, accept_len: torch.Tensor,
                   next_token: torch.Tensor, status: Optional[torch.Tensor] = None) -> None:
    for name, t in (("draft_tokens", draft_tokens), ("tree_parent", tree_parent), ("argmax_tokens", argmax_tokens),
                    ("accepted_idx", accepted_idx), ("accept_len", accept_len), ("next_token", next_token)):
        _need(t, torch.int32, name)
    B, T = draft_tokens.shape
    V = 0
    if target_logits is not None:
        _need(target_logits, torch.float32, "target_logits")
        if not target_logits.is_contiguous():
            raise SpecvlmError("target_logits must be contiguous for specvlm_accept")
        V = target_logits.shape[-1]
    _check(load_library().specvlm_accept(_ptr(draft_tokens), _ptr(tree_parent), _ptr(target_logits),
                                         _ptr(argmax_tokens), B, T, V, _ptr(accepted_idx), accepted_idx.shape[1],
                                         _ptr(accept_len), _ptr(next_token), _ptr(status), _stream()))


def specvlm_accept_sample(draft_tokens: torch.Tensor, tree_parent: torch.Tensor, target_logits: torch.Tensor,
                          uniforms_accept: torch.Tensor, uniforms_sample: torch.Tensor, temperature: float,
                          accepted_idx: torch.Tensor, accept_len: torch.Tensor, next_token: torch.Tensor,
                          row_stats: torch.Tensor, status: Optional[torch.Tensor] = None) -> None:
    """Temperature > 0 tree acceptance by speculative sampling; see include/specvlm.h.

    row_stats: float32 [B][T][2] output (row max, sum of exp((logit - max) / temperature))."""
    for name, t in (("draft_tokens", draft_tokens), ("tree_parent", tree_parent), ("accepted_idx", accepted_idx),
                    ("accept_len", accept_len), ("next_token", next_token)):
        _need(t, torch.int32, name)
    for name, t in (("target_logits", target_logits), ("uniforms_accept", uniforms_accept),
                    ("uniforms_sample", uniforms_sample)):
        _need(t, torch.float32, name)
        if not t.is_contiguous():
            raise SpecvlmError(f"{name} must be contiguous")
    B, T = draft_tokens.shape
    _need(row_stats, torch.float32, "row_stats")
    if not row_stats.is_contiguous() or row_stats.numel() != B * T * 2:
        raise SpecvlmError("row_stats must be a contiguous float32 tensor of B * T * 2 elements")
    _check(load_library().specvlm_accept_sample(
        _ptr(draft_tokens), _ptr(tree_parent), _ptr(target_logits), _ptr(uniforms_accept), _ptr(uniforms_sample),
        float(temperature), B, T, target_logits.shape[-1], _ptr(accepted_idx), accepted_idx.shape[1],
        _ptr(accept_len), _ptr(next_token), _ptr(row_stats), _ptr(status), _stream()))


def make_kv_desc(cache: torch.Tensor) -> KvDesc:
    """cache: [L][B][H][S_cap][D] view with a contiguous last dimension."""
    _need(cache, torch.bfloat16, "kv cache")
    if cache.dim() != 5 or cache.stride(4) != 1:
        raise SpecvlmError("kv cache must be [L][B][H][S_cap][D] with contiguous D")
    d = KvDesc()
    d.L, d.B, d.H, d.S_cap, d.D = cache.shape
    d.stride_l, d.stride_b, d.stride_h, d.stride_s = cache.stride(0), cache.stride(1), cache.stride(2), cache.stride(3)
    return d


def specvlm_kv_compact(k_cache: torch.Tensor, v_cache: torch.Tensor, prefix_len: torch.Tensor,
                       accepted_idx: torch.Tensor, accept_len: torch.Tensor, new_prefix_len: torch.Tensor,
                       status: Optional[torch.Tensor] = None) -> None:
    desc = make_kv_desc(k_cache)
    if tuple(v_cache.shape) != tuple(k_cache.shape) or v_cache.stride() != k_cache.stride():
        raise SpecvlmError("k_cache and v_cache must share shape and strides")
    _check(load_library().specvlm_kv_compact(_ptr(k_cache), _ptr(v_cache), ctypes.byref(desc), _ptr(prefix_len),
                                             _ptr(accepted_idx), accepted_idx.shape[1], _ptr(accept_len),
                                             _ptr(new_prefix_len), _ptr(status), _stream()))


def specvlm_accept_compact(draft_tokens: torch.Tensor, tree_parent: torch.Tensor, argmax_tokens: torch.Tensor,
                           k_cache: torch.Tensor, v_cache: torch.Tensor, prefix_len: torch.Tensor,
                           accepted_idx: torch.Tensor, accept_len: torch.Tensor, next_token: torch.Tensor,
                           new_prefix_len: torch.Tensor, status: Optional[torch.Tensor] = None) -> None:
    desc = make_kv_desc(k_cache)
    if tuple(v_cache.shape) != tuple(k_cache.shape) or v_cache.stride() != k_cache.stride():
        raise SpecvlmError("k_cache and v_cache must share shape and strides")
    B, T = draft_tokens.shape
    _check(load_library().specvlm_accept_compact(
        _ptr(draft_tokens), _ptr(tree_parent), _ptr(argmax_tokens), T, _ptr(k_cache), _ptr(v_cache),
        ctypes.byref(desc), _ptr(prefix_len), _ptr(accepted_idx), accepted_idx.shape[1], _ptr(accept_len),
        _ptr(next_token), _ptr(new_prefix_len), _ptr(status), _stream()))


def specvlm_verify_step(q: torch.Tensor, k_cache: torch.Tensor, v_cache: torch.Tensor, prefix_len: torch.Tensor,
                        tree_parent: torch.Tensor, tree_mask_bits: Optional[torch.Tensor], draft_tokens: torch.Tensor,
                        target_logits: torch.Tensor, out: torch.Tensor, argmax_tokens: torch.Tensor,
                        accepted_idx: torch.Tensor, accept_len: torch.Tensor, next_token: torch.Tensor,
                        new_prefix_len: torch.Tensor, layers_independent: bool = False,
                        workspace: Optional[torch.Tensor] = None, status: Optional[torch.Tensor] = None) -> None:
    """Whole verify step in one call: q/out [L][B][H][T][D] (contiguous per layer), caches
    [L][B][H][S_cap][D], target_logits fp32 [B][T][V] contiguous."""
    desc = make_kv_desc(k_cache)
    if tuple(v_cache.shape) != tuple(k_cache.shape) or v_cache.stride() != k_cache.stride():
        raise SpecvlmError("k_cache and v_cache must share shape and strides")
    _need(q, torch.bfloat16, "q")
    _need(out, torch.bfloat16, "out")
    if q.dim() != 5 or not q[0].is_contiguous() or not out[0].is_contiguous() or out.shape != q.shape:
        raise SpecvlmError("q and out must be [L][B][H][T][D] with contiguous layers")
    _need(target_logits, torch.float32, "target_logits")
    if not target_logits.is_contiguous():
        raise SpecvlmError("target_logits must be contiguous")
    T, V = q.shape[3], target_logits.shape[-1]
    _check(load_library().specvlm_verify_step(
        _ptr(q), q.stride(0), _ptr(k_cache), _ptr(v_cache), ctypes.byref(desc), _ptr(prefix_len), _ptr(tree_parent),
        _ptr(tree_mask_bits), _ptr(draft_tokens), _ptr(target_logits), T, V, _ptr(out), out.stride(0),
        _ptr(argmax_tokens), _ptr(accepted_idx), accepted_idx.shape[1], _ptr(accept_len), _ptr(next_token),
        _ptr(new_prefix_len), 1 if layers_independent else 0, _ptr(workspace), _ptr(status), _stream()))


def specvlm_verify_step_sample(q: torch.Tensor, k_cache: torch.Tensor, v_cache: torch.Tensor, prefix_len: torch.Tensor,
                               tree_parent: torch.Tensor, tree_mask_bits: Optional[torch.Tensor],
                               draft_tokens: torch.Tensor, target_logits: torch.Tensor, uniforms_accept: torch.Tensor,
                               uniforms_sample: torch.Tensor, temperature: float, out: torch.Tensor,
                               row_stats: torch.Tensor, accepted_idx: torch.Tensor, accept_len: torch.Tensor,
                               next_token: torch.Tensor, new_prefix_len: torch.Tensor,
                               layers_independent: bool = False, workspace: Optional[torch.Tensor] = None,
                               status: Optional[torch.Tensor] = None) -> None:
    """Whole verify step at temperature > 0 in one call; tensors as in specvlm_verify_step and
    specvlm_accept_sample."""
    desc = make_kv_desc(k_cache)
    if tuple(v_cache.shape) != tuple(k_cache.shape) or v_cache.stride() != k_cache.stride():
        raise SpecvlmError("k_cache and v_cache must share shape and strides")
    _need(q, torch.bfloat16, "q")
    _need(out, torch.bfloat16, "out")
    if q.dim() != 5 or not q[0].is_contiguous() or not out[0].is_contiguous() or out.shape != q.shape:
        raise SpecvlmError("q and out must be [L][B][H][T][D] with contiguous layers")
    for name, t in (("target_logits", target_logits), ("uniforms_accept", uniforms_accept),
                    ("uniforms_sample", uniforms_sample), ("row_stats", row_stats)):
        _need(t, torch.float32, name)
        if not t.is_contiguous():
            raise SpecvlmError(f"{name} must be contiguous")
    B, T, V = q.shape[1], q.shape[3], target_logits.shape[-1]
    if row_stats.numel() != B * T * 2:
        raise SpecvlmError("row_stats must hold B * T * 2 floats")
    _check(load_library().specvlm_verify_step_sample(
        _ptr(q), q.stride(0), _ptr(k_cache), _ptr(v_cache), ctypes.byref(desc), _ptr(prefix_len), _ptr(tree_parent),
        _ptr(tree_mask_bits), _ptr(draft_tokens), _ptr(target_logits), _ptr(uniforms_accept), _ptr(uniforms_sample),
        float(temperature), T, V, _ptr(out), out.stride(0), _ptr(row_stats), _ptr(accepted_idx),
        accepted_idx.shape[1], _ptr(accept_len), _ptr(next_token), _ptr(new_prefix_len),
        1 if layers_independent else 0, _ptr(workspace), _ptr(status), _stream()))
