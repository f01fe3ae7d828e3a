"""Thin ctypes binding over libspecvlm.so: argument marshalling only.

Every function has the name and the meaning of the C entry point declared in
``include/specvlm.h``; tensors are torch CUDA tensors whose ``data_ptr()`` is passed straight
through.  There is no CPU fallback: a missing library or a non-zero status raises.
"""
from __future__ import annotations

import ctypes
import os
from ctypes import POINTER, byref, c_float, c_int32, c_int64, c_size_t, c_void_p

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libspecvlm.so")

OK = 0
ERR_INVALID_ARG = -1
ERR_UNSUPPORTED_SHAPE = -2
ERR_WORKSPACE_TOO_SMALL = -3
ERR_CUDA = -4
ERR_TIMEOUT = -5
ERR_TOO_LARGE = -6


class SpecvlmError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        super().__init__(f"{where}: {status_string(status)} ({status})")


class KvStruct(ctypes.Structure):
    """Mirror of specvlm_kv_t."""
    _fields_ = [
        ("k", c_void_p), ("v", c_void_p),
        ("stride_layer", c_int64), ("stride_block", c_int64), ("stride_head", c_int64),
        ("stride_token", c_int64),
        ("n_layers", c_int32), ("n_kv_heads", c_int32), ("head_dim", c_int32),
        ("block_tokens", c_int32), ("n_blocks", c_int32), ("max_blocks", c_int32),
        ("block_table", c_void_p), ("seq_lens", c_void_p),
        ("max_seq_len", c_int32),
    ]


_lib = None

EXPORTS = [
    "specvlm_version", "specvlm_status_string",
    "specvlm_stage1_scores_workspace_bytes", "specvlm_stage1_row_lse", "specvlm_stage1_scores",
    "specvlm_stage1_scores_layers", "specvlm_stage1_scores_layer_sums_offset",
    "specvlm_select", "specvlm_select_top_p", "specvlm_select_baseline", "specvlm_gather_kv",
    "specvlm_attn_workspace_bytes", "specvlm_draft_decode_attn", "specvlm_verify_attn",
    "specvlm_accept_workspace_bytes", "specvlm_accept", "specvlm_accept_noalloc",
    "specvlm_append_kv", "specvlm_rollback_kv",
    "specvlm_verify_tree_workspace_bytes", "specvlm_verify_tree_attn", "specvlm_accept_tree",
    "specvlm_compact_tree_kv", "specvlm_debug_poison_shared_memory", "specvlm_debug_wait_timeout",
    "specvlm_debug_set_attn_splits", "specvlm_debug_window_parts",
]


def lib():
    """Load libspecvlm.so (built in-tree by ``build.py``).  Raises if it is missing."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise RuntimeError(f"{LIB_PATH} is missing: build it with "
                               f"`python -m paper_2508_16201_b200.build` (there is no fallback path)")
        L = ctypes.CDLL(LIB_PATH)
        i32p = POINTER(c_int32)
        kvp = POINTER(KvStruct)
        L.specvlm_version.restype = ctypes.c_char_p
        L.specvlm_status_string.restype = ctypes.c_char_p
        L.specvlm_status_string.argtypes = [c_int32]
        L.specvlm_stage1_scores_workspace_bytes.restype = c_size_t
        L.specvlm_stage1_scores_workspace_bytes.argtypes = [kvp, i32p, i32p, c_int32, c_int32]
        L.specvlm_stage1_scores_layer_sums_offset.restype = c_size_t
        L.specvlm_stage1_scores_layer_sums_offset.argtypes = [kvp, i32p, c_int32, c_int32]
        L.specvlm_stage1_scores.restype = c_int32
        L.specvlm_stage1_scores.argtypes = [kvp, c_void_p, i32p, i32p, i32p, i32p, i32p, c_int32, c_int32,
                                            c_float, c_void_p, c_void_p, c_void_p, c_size_t, c_void_p,
                                            c_void_p]
        L.specvlm_stage1_scores_layers.restype = c_int32
        L.specvlm_stage1_scores_layers.argtypes = [kvp, c_void_p, i32p, i32p, i32p, i32p, i32p, c_int32, c_int32,
                                                   c_float, c_void_p, c_void_p, c_void_p, c_size_t, c_int32,
                                                   c_int32, c_int32, c_void_p, c_void_p]
        L.specvlm_stage1_row_lse.restype = c_int32
        L.specvlm_stage1_row_lse.argtypes = [kvp, c_void_p, i32p, i32p, c_int32, c_int32, c_float, c_void_p,
                                             c_void_p, c_void_p]
        L.specvlm_select.restype = c_int32
        L.specvlm_select.argtypes = [c_void_p, i32p, i32p, c_int32, i32p, i32p, i32p, c_int32, c_void_p,
                                     c_void_p, c_void_p]
        L.specvlm_select_baseline.restype = c_int32
        L.specvlm_select_baseline.argtypes = [c_int32, ctypes.c_uint64, i32p, c_int32, i32p, i32p, c_int32, c_void_p,
                                              c_void_p, c_void_p]
        L.specvlm_select_top_p.restype = c_int32
        L.specvlm_select_top_p.argtypes = [c_void_p, i32p, i32p, c_int32, i32p, i32p, i32p, c_int32, c_void_p,
                                           c_void_p, c_void_p, c_void_p]
        L.specvlm_debug_poison_shared_memory.restype = c_int32
        L.specvlm_debug_poison_shared_memory.argtypes = [c_void_p]
        L.specvlm_debug_wait_timeout.restype = c_int32
        L.specvlm_debug_wait_timeout.argtypes = [c_int32, c_void_p, c_void_p, c_void_p]
        L.specvlm_debug_window_parts.restype = c_int32
        L.specvlm_debug_window_parts.argtypes = [c_int32, c_int32, i32p, i32p]
        L.specvlm_debug_set_attn_splits.restype = None
        L.specvlm_debug_set_attn_splits.argtypes = [c_int32]
        L.specvlm_verify_tree_workspace_bytes.restype = c_size_t
        L.specvlm_verify_tree_workspace_bytes.argtypes = [kvp, c_int32, c_int32, c_int32]
        L.specvlm_verify_tree_attn.restype = c_int32
        L.specvlm_verify_tree_attn.argtypes = [kvp, c_void_p, c_void_p, c_int32, c_int32, c_int32, c_float, c_void_p,
                                               c_void_p, c_void_p, c_size_t, c_void_p, c_void_p]
        L.specvlm_accept_tree.restype = c_int32
        L.specvlm_accept_tree.argtypes = [c_void_p, c_void_p, c_void_p, c_int32, c_int32, c_int32, c_void_p, c_void_p,
                                          c_void_p, c_void_p, c_void_p, c_size_t, c_void_p]
        L.specvlm_compact_tree_kv.restype = c_int32
        L.specvlm_compact_tree_kv.argtypes = [kvp, c_void_p, c_void_p, c_int32, c_int32, c_void_p, c_void_p, c_void_p]
        L.specvlm_append_kv.restype = c_int32
        L.specvlm_append_kv.argtypes = [kvp, c_void_p, c_void_p, c_int32, c_int32, c_void_p, c_void_p, c_void_p]
        L.specvlm_rollback_kv.restype = c_int32
        L.specvlm_rollback_kv.argtypes = [c_void_p, c_void_p, c_int32, c_int32, c_void_p, c_void_p]
        L.specvlm_gather_kv.restype = c_int32
        L.specvlm_gather_kv.argtypes = [kvp, c_void_p, i32p, i32p, i32p, i32p, c_int32, kvp, c_void_p,
                                        c_void_p]
        L.specvlm_attn_workspace_bytes.restype = c_size_t
        L.specvlm_attn_workspace_bytes.argtypes = [kvp, c_int32, c_int32, c_int32]
        L.specvlm_draft_decode_attn.restype = c_int32
        L.specvlm_draft_decode_attn.argtypes = [kvp, c_void_p, c_int32, c_int32, c_float, c_void_p,
                                                c_void_p, c_void_p, c_size_t, c_void_p, c_void_p]
        L.specvlm_verify_attn.restype = c_int32
        L.specvlm_verify_attn.argtypes = [kvp, c_void_p, c_int32, c_int32, c_int32, c_float, c_void_p,
                                          c_void_p, c_void_p, c_size_t, c_void_p, c_void_p]
        L.specvlm_accept_workspace_bytes.restype = c_size_t
        L.specvlm_accept_workspace_bytes.argtypes = [c_int32, c_int32, c_int32]
        L.specvlm_accept.restype = c_int32
        L.specvlm_accept.argtypes = [c_void_p, c_void_p, c_int32, c_int32, c_int32, c_void_p, c_void_p,
                                     c_void_p, c_void_p, c_size_t, c_void_p]
        L.specvlm_accept_noalloc.restype = c_int32
        L.specvlm_accept_noalloc.argtypes = [c_void_p, c_void_p, c_int32, c_int32, c_int32, c_void_p, c_void_p,
                                             c_void_p, c_void_p]
        _lib = L
    return _lib


def version() -> str:
    return lib().specvlm_version().decode()


def status_string(status: int) -> str:
    return lib().specvlm_status_string(int(status)).decode()


def _check(status: int, where: str):
    if status != OK:
        raise SpecvlmError(status, where)


def _ptr(t):
    return c_void_p(t.data_ptr()) if t is not None else c_void_p(0)


def _stream():
    return c_void_p(torch.cuda.current_stream().cuda_stream)


def _i32(seq):
    arr = (c_int32 * len(seq))(*[int(x) for x in seq])
    return arr


class KvCache:
    """A bf16 K/V cache in device memory plus its specvlm_kv_t descriptor.

    ``k``/``v``: tensors of shape [n_layers][n_blocks][n_kv_heads][block_tokens][head_dim]
    (any strides with a unit channel stride).  ``block_table`` None = contiguous: sequence b
    is block b.
    """

    def __init__(self, k: torch.Tensor, v: torch.Tensor, seq_lens: torch.Tensor, max_seq_len: int,
                 block_table: torch.Tensor | None = None):
        assert k.dtype == torch.bfloat16 and v.dtype == torch.bfloat16 and k.dim() == 5
        assert k.shape == v.shape and k.stride() == v.stride() and k.stride(4) == 1
        assert seq_lens.dtype == torch.int32
        self.k, self.v, self.seq_lens, self.block_table = k, v, seq_lens, block_table
        self.max_seq_len = int(max_seq_len)
        L, NB, H, BT, D = k.shape
        s = KvStruct()
        s.k, s.v = k.data_ptr(), v.data_ptr()
        s.stride_layer, s.stride_block, s.stride_head, s.stride_token = (k.stride(0), k.stride(1),
                                                                         k.stride(2), k.stride(3))
        s.n_layers, s.n_kv_heads, s.head_dim, s.block_tokens, s.n_blocks = L, H, D, BT, NB
        if block_table is not None:
            assert block_table.dtype == torch.int32 and block_table.dim() == 2 and block_table.is_contiguous()
            s.max_blocks = block_table.shape[1]
            s.block_table = block_table.data_ptr()
        else:
            s.max_blocks = 1
            s.block_table = None
        s.seq_lens = seq_lens.data_ptr()
        s.max_seq_len = self.max_seq_len
        self.struct = s

    @property
    def n_layers(self):
        return self.k.shape[0]

    @property
    def n_kv_heads(self):
        return self.k.shape[2]

    @property
    def head_dim(self):
        return self.k.shape[4]


# When set (the GPU tests set it), scratch buffers that this binding allocates are filled with 0xff
# bytes (NaN as fp32, -1 as int32) first: no call may depend on what its workspace held before.
debug_fill_workspaces = False


def _ws(nbytes: int, device) -> torch.Tensor:
    ws = torch.empty(max(int(nbytes), 256), dtype=torch.uint8, device=device)
    if debug_fill_workspaces:
        ws.fill_(0xFF)
    return ws


# ---------------------------------------------------------------------------------- attention
def attn_workspace_bytes(kv: KvCache, batch: int, n_q_heads: int, gamma: int) -> int:
    return int(lib().specvlm_attn_workspace_bytes(byref(kv.struct), batch, n_q_heads, gamma))


def draft_decode_attn(kv: KvCache, q: torch.Tensor, sm_scale: float, out: torch.Tensor | None = None,
                      lse: torch.Tensor | None = None, ws: torch.Tensor | None = None,
                      d_status: torch.Tensor | None = None) -> torch.Tensor:
    """q, out: bf16 [n_layers][batch][n_q_heads][head_dim]."""
    L, B, Hq, D = q.shape
    assert q.is_contiguous() and q.dtype == torch.bfloat16
    if out is None:
        out = torch.empty_like(q)
    if ws is None:
        ws = _ws(attn_workspace_bytes(kv, B, Hq, 0), q.device)
    rc = lib().specvlm_draft_decode_attn(byref(kv.struct), _ptr(q), B, Hq, float(sm_scale), _ptr(out),
                                         _ptr(lse), _ptr(ws), ws.numel(), _ptr(d_status), _stream())
    _check(rc, "specvlm_draft_decode_attn")
    return out


def verify_attn(kv: KvCache, q: torch.Tensor, gamma: int, sm_scale: float,
                out: torch.Tensor | None = None, lse: torch.Tensor | None = None,
                ws: torch.Tensor | None = None, d_status: torch.Tensor | None = None) -> torch.Tensor:
    """q, out: bf16 [n_layers][batch][gamma+1][n_q_heads][head_dim]."""
    L, B, NQ, Hq, D = q.shape
    assert NQ == gamma + 1 and q.is_contiguous() and q.dtype == torch.bfloat16
    if out is None:
        out = torch.empty_like(q)
    if ws is None:
        ws = _ws(attn_workspace_bytes(kv, B, Hq, gamma), q.device)
    rc = lib().specvlm_verify_attn(byref(kv.struct), _ptr(q), B, Hq, gamma, float(sm_scale), _ptr(out),
                                   _ptr(lse), _ptr(ws), ws.numel(), _ptr(d_status), _stream())
    _check(rc, "specvlm_verify_attn")
    return out


# ---------------------------------------------------------------------------------- scores
def stage1_scores_workspace_bytes(kv: KvCache, text_cu, video_len, n_q_heads: int) -> int:
    batch = len(video_len)
    return int(lib().specvlm_stage1_scores_workspace_bytes(byref(kv.struct), _i32(text_cu), _i32(video_len),
                                                           batch, n_q_heads))


def stage1_scores_layer_sums_offset(kv: KvCache, text_cu, n_q_heads: int) -> int:
    """Byte offset, inside a rating call's workspace, of the per-layer sums fp32 [n_layers][sum_video]."""
    return int(lib().specvlm_stage1_scores_layer_sums_offset(byref(kv.struct), _i32(text_cu), len(text_cu) - 1,
                                                             n_q_heads))


def stage1_row_lse(kv: KvCache, q_text: torch.Tensor, text_cu, text_start, sm_scale: float,
                   row_lse: torch.Tensor | None = None, d_status: torch.Tensor | None = None) -> torch.Tensor:
    """q_text: bf16 [n_layers][sum_text][n_q_heads][head_dim]; returns fp32 [n_layers][sum_text][n_q_heads]."""
    L, n_text_all, Hq, D = q_text.shape
    assert q_text.is_contiguous() and q_text.dtype == torch.bfloat16 and n_text_all == text_cu[-1]
    if row_lse is None:
        row_lse = torch.empty((L, n_text_all, Hq), dtype=torch.float32, device=q_text.device)
    rc = lib().specvlm_stage1_row_lse(byref(kv.struct), _ptr(q_text), _i32(text_cu), _i32(text_start),
                                      len(text_start), Hq, float(sm_scale), _ptr(row_lse), _ptr(d_status),
                                      _stream())
    _check(rc, "specvlm_stage1_row_lse")
    return row_lse


def stage1_scores(kv: KvCache, q_text: torch.Tensor, text_cu, text_start, video_start, video_len,
                  video_cu, sm_scale: float, scores: torch.Tensor | None = None,
                  ws: torch.Tensor | None = None, d_status: torch.Tensor | None = None,
                  row_lse: torch.Tensor | None = None) -> torch.Tensor:
    """q_text: bf16 [n_layers][sum_text][n_q_heads][head_dim]; returns fp32 [sum_video]."""
    L, n_text_all, Hq, D = q_text.shape
    batch = len(video_len)
    assert q_text.is_contiguous() and q_text.dtype == torch.bfloat16 and n_text_all == text_cu[-1]
    if scores is None:
        scores = torch.empty(int(video_cu[-1]), dtype=torch.float32, device=q_text.device)
    if ws is None:
        ws = _ws(stage1_scores_workspace_bytes(kv, text_cu, video_len, Hq), q_text.device)
    rc = lib().specvlm_stage1_scores(byref(kv.struct), _ptr(q_text), _i32(text_cu), _i32(text_start),
                                     _i32(video_start), _i32(video_len), _i32(video_cu), batch, Hq,
                                     float(sm_scale), _ptr(row_lse), _ptr(scores), _ptr(ws), ws.numel(),
                                     _ptr(d_status), _stream())
    _check(rc, "specvlm_stage1_scores")
    return scores


def stage1_scores_layers(kv: KvCache, q_text: torch.Tensor, text_cu, text_start, video_start, video_len,
                         video_cu, sm_scale: float, scores: torch.Tensor, ws: torch.Tensor, layer_begin: int,
                         layer_end: int, finish: bool, d_status: torch.Tensor | None = None,
                         row_lse: torch.Tensor | None = None) -> torch.Tensor:
    """Rates layers [layer_begin, layer_end) of the problem that ``kv`` and ``q_text`` describe as a
    whole; with ``finish`` the sums of all layers (left in ``ws`` by this and earlier calls) become
    ``scores``.  ``ws`` and ``scores`` are the caller's, kept across the calls."""
    L, n_text_all, Hq, D = q_text.shape
    batch = len(video_len)
    assert q_text.is_contiguous() and q_text.dtype == torch.bfloat16 and n_text_all == text_cu[-1]
    rc = lib().specvlm_stage1_scores_layers(byref(kv.struct), _ptr(q_text), _i32(text_cu), _i32(text_start),
                                            _i32(video_start), _i32(video_len), _i32(video_cu), batch, Hq,
                                            float(sm_scale), _ptr(row_lse), _ptr(scores), _ptr(ws), ws.numel(),
                                            int(layer_begin), int(layer_end), 1 if finish else 0,
                                            _ptr(d_status), _stream())
    _check(rc, "specvlm_stage1_scores_layers")
    return scores


# ---------------------------------------------------------------------------------- select
def select(scores: torch.Tensor, video_cu, n_frames, tokens_per_frame: int, k_stage1, k_total, kept_cu,
           kept_idx: torch.Tensor | None = None, d_status: torch.Tensor | None = None) -> torch.Tensor:
    batch = len(n_frames)
    assert scores.dtype == torch.float32 and scores.is_contiguous()
    if kept_idx is None:
        kept_idx = torch.empty(max(int(kept_cu[-1]), 1), dtype=torch.int32, device=scores.device)
    rc = lib().specvlm_select(_ptr(scores), _i32(video_cu), _i32(n_frames), int(tokens_per_frame),
                              _i32(k_stage1), _i32(k_total), _i32(kept_cu), batch, _ptr(kept_idx),
                              _ptr(d_status), _stream())
    _check(rc, "specvlm_select")
    return kept_idx


def select_top_p(scores: torch.Tensor, video_cu, n_frames, tokens_per_frame: int, lambda_permille, k_total,
                 kept_cu, kept_idx: torch.Tensor | None = None, k_stage1_out: torch.Tensor | None = None,
                 d_status: torch.Tensor | None = None):
    """Returns (kept_idx, k_stage1_out): the retention sets and the Stage-I counts Eq. 6 chose."""
    batch = len(n_frames)
    assert scores.dtype == torch.float32 and scores.is_contiguous()
    if kept_idx is None:
        kept_idx = torch.empty(max(int(kept_cu[-1]), 1), dtype=torch.int32, device=scores.device)
    if k_stage1_out is None:
        k_stage1_out = torch.empty(batch, dtype=torch.int32, device=scores.device)
    rc = lib().specvlm_select_top_p(_ptr(scores), _i32(video_cu), _i32(n_frames), int(tokens_per_frame),
                                    _i32(lambda_permille), _i32(k_total), _i32(kept_cu), batch, _ptr(kept_idx),
                                    _ptr(k_stage1_out), _ptr(d_status), _stream())
    _check(rc, "specvlm_select_top_p")
    return kept_idx, k_stage1_out


SEL_WINDOW_FRONT, SEL_WINDOW_MIDDLE, SEL_WINDOW_END, SEL_FRAMES, SEL_RANDOM = 0, 1, 2, 3, 4


def select_baseline(mode: int, n_frames, tokens_per_frame: int, k_total, kept_cu, seed: int = 0,
                    device="cuda", kept_idx: torch.Tensor | None = None, want_counts: bool = True):
    """Returns (kept_idx, kept_n): the index lists of an attention-agnostic selector (kept_n None
    when the counts are not asked for)."""
    batch = len(n_frames)
    if kept_idx is None:
        kept_idx = torch.empty(max(int(kept_cu[-1]), 1), dtype=torch.int32, device=device)
    kept_n = torch.empty(batch, dtype=torch.int32, device=device) if want_counts else None
    rc = lib().specvlm_select_baseline(int(mode), int(seed), _i32(n_frames), int(tokens_per_frame), _i32(k_total),
                                       _i32(kept_cu), batch, _ptr(kept_idx), _ptr(kept_n), _stream())
    _check(rc, "specvlm_select_baseline")
    return kept_idx, kept_n


# ---------------------------------------------------------------------------------- gather
def gather_kv(src: KvCache, kept_idx: torch.Tensor, kept_cu, video_start, video_len, src_len,
              dst: KvCache, d_status: torch.Tensor | None = None) -> None:
    batch = len(video_len)
    assert kept_idx.dtype == torch.int32
    rc = lib().specvlm_gather_kv(byref(src.struct), _ptr(kept_idx), _i32(kept_cu), _i32(video_start),
                                 _i32(video_len), _i32(src_len), batch, byref(dst.struct), _ptr(d_status),
                                 _stream())
    _check(rc, "specvlm_gather_kv")


# ---------------------------------------------------------------------------------- cache maintenance
def append_kv(kv: KvCache, new_k: torch.Tensor, new_v: torch.Tensor, d_status: torch.Tensor | None = None) -> None:
    """new_k / new_v: bf16 [n_layers][batch][n_new][n_kv_heads][head_dim]; kv.seq_lens is updated."""
    assert new_k.dtype == torch.bfloat16 and new_k.is_contiguous() and new_v.is_contiguous()
    assert new_k.shape == new_v.shape and new_k.dim() == 5
    rc = lib().specvlm_append_kv(byref(kv.struct), _ptr(new_k), _ptr(new_v), new_k.shape[1], new_k.shape[2],
                                 _ptr(kv.seq_lens), _ptr(d_status), _stream())
    _check(rc, "specvlm_append_kv")


def rollback_kv(seq_lens: torch.Tensor, accept_len: torch.Tensor, gamma: int,
                d_status: torch.Tensor | None = None) -> None:
    assert seq_lens.dtype == torch.int32 and accept_len.dtype == torch.int32
    rc = lib().specvlm_rollback_kv(_ptr(seq_lens), _ptr(accept_len), seq_lens.numel(), int(gamma), _ptr(d_status),
                                   _stream())
    _check(rc, "specvlm_rollback_kv")


# ---------------------------------------------------------------------------------- tree drafting
def verify_tree_attn(kv: KvCache, q: torch.Tensor, parents: torch.Tensor, sm_scale: float,
                     out: torch.Tensor | None = None, lse: torch.Tensor | None = None,
                     ws: torch.Tensor | None = None, d_status: torch.Tensor | None = None) -> torch.Tensor:
    """q: bf16 [n_layers][batch][n_nodes][n_q_heads][head_dim]; parents: int32 [batch][n_nodes]."""
    L, B, N, Hq, D = q.shape
    assert q.dtype == torch.bfloat16 and q.is_contiguous()
    assert parents.dtype == torch.int32 and parents.is_contiguous() and tuple(parents.shape) == (B, N)
    if out is None:
        out = torch.empty_like(q)
    if ws is None:
        ws = _ws(int(lib().specvlm_verify_tree_workspace_bytes(byref(kv.struct), B, Hq, N)), q.device)
    rc = lib().specvlm_verify_tree_attn(byref(kv.struct), _ptr(q), _ptr(parents), B, Hq, N, float(sm_scale),
                                        _ptr(out), _ptr(lse), _ptr(ws), ws.numel(), _ptr(d_status), _stream())
    _check(rc, "specvlm_verify_tree_attn")
    return out


def accept_tree_buffers(batch: int, n_nodes: int, vocab: int, device, want_argmax: bool = False):
    """Output tensors and scratch of accept_tree, for callers that reuse them across calls:
    (accept_len, next_token, path, argmax or None, ws)."""
    n = torch.empty(batch, dtype=torch.int32, device=device)
    nxt = torch.empty(batch, dtype=torch.int32, device=device)
    path = torch.empty((batch, n_nodes), dtype=torch.int32, device=device)
    g = torch.empty((batch, n_nodes), dtype=torch.int32, device=device) if want_argmax else None
    return n, nxt, path, g, _ws(accept_workspace_bytes(batch, n_nodes - 1, vocab), device)


def accept_tree(target_logits: torch.Tensor, node_tokens: torch.Tensor, parents: torch.Tensor,
                want_argmax: bool = False, out=None):
    """Returns (accept_len [B], next_token [B], path [B][n_nodes], argmax [B][n_nodes] or None)."""
    B, N, V = target_logits.shape
    assert target_logits.dtype == torch.float32 and target_logits.is_contiguous()
    assert node_tokens.dtype == torch.int32 and parents.dtype == torch.int32
    dev = target_logits.device
    n, nxt, path, g, ws = out if out is not None else accept_tree_buffers(B, N, V, dev, want_argmax)
    rc = lib().specvlm_accept_tree(_ptr(target_logits), _ptr(node_tokens), _ptr(parents), B, N, V, _ptr(n), _ptr(nxt),
                                   _ptr(path), _ptr(g), _ptr(ws), ws.numel(), _stream())
    _check(rc, "specvlm_accept_tree")
    return n, nxt, path, g


def debug_poison_shared_memory() -> None:
    """Fills the SMs' shared memory with NaN bit patterns (test diagnostic)."""
    _check(lib().specvlm_debug_poison_shared_memory(_stream()), "specvlm_debug_poison_shared_memory")


def debug_wait_timeout(limit_ms: int, d_status: torch.Tensor, d_abort_flag: torch.Tensor | None = None) -> None:
    """Runs the bounded barrier wait on a barrier nobody arrives at (test diagnostic)."""
    _check(lib().specvlm_debug_wait_timeout(int(limit_ms), _ptr(d_status), _ptr(d_abort_flag), _stream()),
           "specvlm_debug_wait_timeout")


def debug_set_attn_splits(n_splits: int) -> None:
    """Forces the split count of the 16-row attention kernel (0 = built-in choice; test hook)."""
    lib().specvlm_debug_set_attn_splits(int(n_splits))


def compact_tree_kv(kv: KvCache, path: torch.Tensor, accept_len: torch.Tensor,
                    d_status: torch.Tensor | None = None) -> None:
    """Moves the accepted nodes' rows behind the root and shortens kv.seq_lens accordingly."""
    B, N = path.shape
    rc = lib().specvlm_compact_tree_kv(byref(kv.struct), _ptr(path), _ptr(accept_len), B, N, _ptr(kv.seq_lens),
                                       _ptr(d_status), _stream())
    _check(rc, "specvlm_compact_tree_kv")


# ---------------------------------------------------------------------------------- accept
def accept_workspace_bytes(batch: int, gamma: int, vocab: int) -> int:
    return int(lib().specvlm_accept_workspace_bytes(batch, gamma, vocab))


def accept(target_logits: torch.Tensor, draft_tokens: torch.Tensor, want_argmax: bool = False,
           ws: torch.Tensor | None = None, out=None):
    """target_logits fp32 [B][gamma+1][vocab], draft_tokens int32 [B][gamma].
    Returns (accept_len int32 [B], next_token int32 [B], target_argmax or None)."""
    B, G1, V = target_logits.shape
    gamma = G1 - 1
    assert target_logits.dtype == torch.float32 and target_logits.is_contiguous()
    assert draft_tokens.dtype == torch.int32 and draft_tokens.is_contiguous()
    dev = target_logits.device
    if out is None:
        accept_len = torch.empty(B, dtype=torch.int32, device=dev)
        next_token = torch.empty(B, dtype=torch.int32, device=dev)
        g = torch.empty((B, G1), dtype=torch.int32, device=dev) if want_argmax else None
    else:
        accept_len, next_token, g = out
    if ws is None:
        ws = _ws(accept_workspace_bytes(B, gamma, V), dev)
    rc = lib().specvlm_accept(_ptr(target_logits), _ptr(draft_tokens), B, gamma, V, _ptr(accept_len),
                              _ptr(next_token), _ptr(g), _ptr(ws), ws.numel(), _stream())
    _check(rc, "specvlm_accept")
    return accept_len, next_token, g


def accept_noalloc(target_logits: torch.Tensor, draft_tokens: torch.Tensor, out, want_argmax_into=None):
    """specvlm_accept_noalloc: like ``accept`` but the library's built-in scratch is used, and this
    wrapper allocates nothing either: ``out`` = (accept_len, next_token) int32 [B] tensors made by
    the caller beforehand; ``want_argmax_into`` an optional int32 [B][gamma+1] tensor.
    Raises SpecvlmError(ERR_TOO_LARGE) beyond the built-in capacity."""
    B, G1, V = target_logits.shape
    assert target_logits.dtype == torch.float32 and target_logits.is_contiguous()
    assert draft_tokens.dtype == torch.int32 and draft_tokens.is_contiguous()
    accept_len, next_token = out
    rc = lib().specvlm_accept_noalloc(_ptr(target_logits), _ptr(draft_tokens), B, G1 - 1, V, _ptr(accept_len),
                                      _ptr(next_token), _ptr(want_argmax_into), _stream())
    _check(rc, "specvlm_accept_noalloc")
    return accept_len, next_token
