"""CPU oracle for the SpecVLM pruned-draft speculative-decoding hot path.

TEST INFRASTRUCTURE ONLY: a plain, slow, obviously-correct statement of what the CUDA
library computes, written from the paper.  It imports nothing from the CUDA package and
the CUDA package imports nothing from here.  Only the tests, the smoke check and the
benchmark's cpu_baseline / reference legs may call it.

Heavy floating-point parts (token rating, softmax attention) are fp64 C in
``specvlm_oracle.c``; the integer parts (ranking, Stage II, gather, acceptance) are
written out in Python / numpy below so they can be checked against the paper by eye.

bf16 tensors are passed as numpy ``uint16`` bit patterns.

Readings taken where the paper is silent or inconsistent ("parity unpinned" against the
authors' code, pinned only against the mathematics):
  * Eq. 4: G is a block of the full causal softmax (``stage1_scores``).
  * Eq. 7: the Stage-II budget is (1-r)|V| - |V_R| so that the final set has exactly
    (1-r)|V| tokens, as the text after Eq. 7 states, and the interval is realised per
    frame in raster order (``stage2_uniform``).
"""
from __future__ import annotations

import ctypes
import math
import os

import numpy as np

from . import build as _build

_lib = None


def _load():
    global _lib
    if _lib is None:
        path = _build.build()
        lib = ctypes.CDLL(path)
        u16p = ctypes.POINTER(ctypes.c_uint16)
        f64p = ctypes.POINTER(ctypes.c_double)
        ci, cd = ctypes.c_int, ctypes.c_double
        lib.oracle_stage1_scores.argtypes = [u16p, u16p, ci, ci, ci, ci, ci, ci, ci, ci, ci, cd, ci,
                                             f64p, f64p, f64p]
        lib.oracle_stage1_scores.restype = ci
        lib.oracle_attention.argtypes = [u16p, u16p, u16p, ci, ci, ci, ci, ci, ci, cd, f64p, f64p]
        lib.oracle_attention.restype = ci
        lib.oracle_attention_probs.argtypes = [u16p, u16p, ci, ci, cd, f64p]
        lib.oracle_attention_probs.restype = ci
        lib.oracle_num_threads.restype = ci
        _lib = lib
    return _lib


def num_threads() -> int:
    """OpenMP threads the C part uses."""
    return int(_load().oracle_num_threads())


def _u16(a) -> np.ndarray:
    a = np.ascontiguousarray(a)
    assert a.dtype == np.uint16, "bf16 inputs are passed as uint16 bit patterns"
    return a


def _p16(a):
    return a.ctypes.data_as(ctypes.POINTER(ctypes.c_uint16))


def _p64(a):
    return a.ctypes.data_as(ctypes.POINTER(ctypes.c_double)) if a is not None else None


def bf16_bits_to_f64(a: np.ndarray) -> np.ndarray:
    """Exact widening of bf16 bit patterns to float64."""
    return (a.astype(np.uint32) << 16).view(np.float32).astype(np.float64)


# --------------------------------------------------------------------------------------
# Step 1a: token rating (Eq. 4-5)
# --------------------------------------------------------------------------------------
def stage1_scores(q_text: np.ndarray, k: np.ndarray, video_start: int, n_video: int,
                  text_start: int, sm_scale: float, video_only: bool = False,
                  want_rows: bool = False):
    """a_j of Eq. 5, averaged over layers and heads.

    q_text: uint16 [n_layers][n_text][Hq][d]; k: uint16 [n_layers][Hkv][n_tokens][d].
    Returns fp64 [n_video] (and, if want_rows, the per-row video mass and row LSE,
    each [n_layers][Hq][n_text]).
    """
    q_text, k = _u16(q_text), _u16(k)
    n_layers, n_text, Hq, d = q_text.shape
    n_layers2, Hkv, n_tokens, d2 = k.shape
    assert n_layers == n_layers2 and d == d2
    a = np.zeros(n_video, dtype=np.float64)
    mass = np.zeros((n_layers, Hq, n_text), dtype=np.float64) if want_rows else None
    lse = np.zeros((n_layers, Hq, n_text), dtype=np.float64) if want_rows else None
    rc = _load().oracle_stage1_scores(_p16(q_text), _p16(k), n_layers, Hq, Hkv, d, n_tokens,
                                      video_start, n_video, text_start, n_text, float(sm_scale),
                                      int(video_only), _p64(a), _p64(mass), _p64(lse))
    if rc != 0:
        raise ValueError(f"oracle_stage1_scores: bad arguments ({rc})")
    return (a, mass, lse) if want_rows else a


# --------------------------------------------------------------------------------------
# Step 1b: Stage I ranking.  The paper sorts A and adds tokens in that order (text before
# Eq. 6); the hot path keeps a fixed count k1.  Ties: lower index first.
# --------------------------------------------------------------------------------------
def stage1_topk(scores_f32: np.ndarray, k1: int) -> list[int]:
    """Indices of the k1 highest-scored tokens under the order (score desc, index asc).

    The comparison is on the fp32 values handed in (the same bits the GPU select sees).
    """
    s = np.asarray(scores_f32, dtype=np.float32)
    assert 0 <= k1 <= s.shape[0]
    order = sorted(range(s.shape[0]), key=lambda j: (-float(s[j]), j))
    return sorted(order[:k1])


def stage1_top_p(scores_f32: np.ndarray, lambda_r: float, k_cap: int | None = None) -> int:
    """Count c of Eq. 6: the smallest prefix of the descending ranking whose cumulative
    score reaches lambda_r times the total.  The sums run in ranking order, in fp64 over
    the fp32 values.  k_cap (the whole retention budget) bounds c when given."""
    s = np.asarray(scores_f32, dtype=np.float32)
    order = sorted(range(s.shape[0]), key=lambda j: (-float(s[j]), j))
    total = 0.0
    for j in order:
        total += float(s[j])
    target = float(lambda_r) * total
    c, run = 0, 0.0
    while c < len(order) and not (run >= target):
        run += float(s[order[c]])
        c += 1
    if k_cap is not None:
        c = min(c, k_cap)
    return c


TOP_P_FRAC_BITS = 36


def stage1_top_p_fixed(scores_f32: np.ndarray, lambda_permille: int, k_cap: int | None = None) -> int:
    """Count c of Eq. 6 in the arithmetic the GPU library takes the decision in.

    Eq. 6 compares a cumulative score with lambda_r times the total; in floating point the
    result of that comparison can depend on the order of the additions.  So that the count is
    a function of the scores alone, each fp32 score is first truncated to a multiple of
    2^-36 (and capped at 1, the largest value a mean probability can take), lambda_r is given
    in thousandths, and the comparison  1000 * sum_{i<c} q_(i) >= lambda * sum q  runs in
    exact integers.  `stage1_top_p` above is the same rule in fp64; a test checks that the
    two agree on long-tailed scores.
    """
    s = np.asarray(scores_f32, dtype=np.float32)
    one = 1 << TOP_P_FRAC_BITS
    q = [min(int(float(x) * one), one) for x in s]        # float(x) * 2^36 is exact in fp64
    order = sorted(range(s.shape[0]), key=lambda j: (-float(s[j]), j))
    target = int(lambda_permille) * sum(q)
    c, run = 0, 0
    while c < len(order) and not (1000 * run >= target):
        run += q[order[c]]
        c += 1
    if k_cap is not None:
        c = min(c, k_cap)
    return c


# --------------------------------------------------------------------------------------
# Step 2: Stage II spatially uniform reduction (Eq. 7 and the text after it)
# --------------------------------------------------------------------------------------
def stage2_uniform(v_r: list[int], n_frames: int, tokens_per_frame: int, k_total: int) -> list[int]:
    """V_U: tokens of V \\ V_R kept at a fixed interval, frame by frame.

    Budget n_U = k_total - |V_R| (so that |V_R u V_U| = (1-r)|V| exactly, as the text after
    Eq. 7 says); interval I = (|V| - |V_R|) / n_U (Eq. 7 with that budget).  Realisation on
    the patch grids: frame f's remaining tokens R_f (raster order, c_f of them) receive the
    quota  n_f = floor(C_{f+1} n_U / m) - floor(C_f n_U / m)  with C_f = sum_{f'<f} c_{f'}
    and m = |V| - |V_R|, and the picks inside the frame are R_f[floor(t c_f / n_f)],
    t = 0..n_f-1: a rank stride of c_f / n_f ~= I that restarts at each frame.
    """
    n_v = n_frames * tokens_per_frame
    in_r = [False] * n_v
    for j in v_r:
        in_r[j] = True
    k1 = len(v_r)
    n_u = k_total - k1
    m = n_v - k1
    assert 0 <= n_u <= m
    picks: list[int] = []
    c_before = 0
    for f in range(n_frames):
        r_f = [j for j in range(f * tokens_per_frame, (f + 1) * tokens_per_frame) if not in_r[j]]
        c_f = len(r_f)
        if m > 0:
            n_f = ((c_before + c_f) * n_u) // m - (c_before * n_u) // m
        else:
            n_f = 0
        for t in range(n_f):
            picks.append(r_f[(t * c_f) // n_f])
        c_before += c_f
    return picks


def select(scores_f32: np.ndarray, n_frames: int, tokens_per_frame: int, k1: int, k_total: int
           ) -> np.ndarray:
    """Final retention set V_R u V_U in ascending index order (int32)."""
    v_r = stage1_topk(scores_f32, k1)
    v_u = stage2_uniform(v_r, n_frames, tokens_per_frame, k_total)
    kept = sorted(set(v_r) | set(v_u))
    assert len(kept) == len(v_r) + len(v_u) == k_total
    return np.asarray(kept, dtype=np.int32)


def select_top_p(scores_f32: np.ndarray, n_frames: int, tokens_per_frame: int, lambda_permille: int,
                 k_total: int) -> tuple[np.ndarray, int]:
    """Retention set with the Stage-I count chosen by Eq. 6 (Top-P), bounded by the whole
    budget k_total (then Stage II adds nothing).  Returns (kept indices, Stage-I count)."""
    k1 = stage1_top_p_fixed(scores_f32, lambda_permille, k_cap=k_total)
    return select(scores_f32, n_frames, tokens_per_frame, k1, k_total), k1


# --------------------------------------------------------------------------------------
# Step 3: build the pruned draft context (text after Eq. 7: the draft sees V_R u V_U plus
# the language prompt)
# --------------------------------------------------------------------------------------
def gather_kv(src: np.ndarray, kept_idx: np.ndarray, video_start: int, n_video: int,
              seq_len: int) -> np.ndarray:
    """src: [..., n_tokens, d] (any leading dims, token axis = -2).  Returns the rows
    [tokens before the video] + [kept video tokens, ascending] + [tokens after the video]."""
    rows = list(range(0, video_start))
    rows += [video_start + int(j) for j in kept_idx]
    rows += list(range(video_start + n_video, seq_len))
    return np.ascontiguousarray(np.take(src, rows, axis=-2))


# --------------------------------------------------------------------------------------
# Cache maintenance around a step (Section 3.1: drafted tokens enter the caches before the
# attention over them; rejected ones are discarded after verification)
# --------------------------------------------------------------------------------------
def append_kv(cache: np.ndarray, new: np.ndarray, seq_len: int) -> tuple[np.ndarray, int]:
    """cache: [n_layers][Hkv][capacity][d] of one sequence, new: [n_layers][n_new][Hkv][d].
    Returns (cache with the new rows at positions seq_len .. seq_len + n_new - 1, new length)."""
    out = cache.copy()
    n_new = new.shape[1]
    assert seq_len + n_new <= cache.shape[2]
    for t in range(n_new):
        out[:, :, seq_len + t, :] = new[:, t, :, :]
    return out, seq_len + n_new


def rollback_len(seq_len: int, gamma: int, accept_len: int) -> int:
    """Of the gamma + 1 tokens of the verification window, accept_len + 1 stay in the cache."""
    assert 0 <= accept_len <= gamma <= seq_len - 1
    return seq_len - (gamma + 1) + (accept_len + 1)


# --------------------------------------------------------------------------------------
# Step 4a/4b: attention
# --------------------------------------------------------------------------------------
def attention(q: np.ndarray, k: np.ndarray, v: np.ndarray, kv_len: int, sm_scale: float):
    """q: uint16 [n_q][Hq][d]; k, v: uint16 [Hkv][kv_stride][d].  Query t sees keys
    [0, kv_len - n_q + t].  Returns (out fp64 [n_q][Hq][d], lse fp64 [n_q][Hq])."""
    q, k, v = _u16(q), _u16(k), _u16(v)
    n_q, Hq, d = q.shape
    Hkv, kv_stride, d2 = k.shape
    assert d == d2 and v.shape == k.shape
    out = np.zeros((n_q, Hq, d), dtype=np.float64)
    lse = np.zeros((n_q, Hq), dtype=np.float64)
    rc = _load().oracle_attention(_p16(q), _p16(k), _p16(v), n_q, Hq, Hkv, d, int(kv_len),
                                  kv_stride, float(sm_scale), _p64(out), _p64(lse))
    if rc != 0:
        raise ValueError(f"oracle_attention: bad arguments ({rc})")
    return out, lse


def attention_probs(q_row: np.ndarray, k_head: np.ndarray, n_keys: int, sm_scale: float) -> np.ndarray:
    q_row, k_head = _u16(q_row), _u16(k_head)
    probs = np.zeros(n_keys, dtype=np.float64)
    _load().oracle_attention_probs(_p16(q_row), _p16(k_head), q_row.shape[-1], int(n_keys),
                                   float(sm_scale), _p64(probs))
    return probs


def merge_partials(outs: list[np.ndarray], lses: list[np.ndarray]):
    """Combine attention results computed over disjoint key chunks (used only by the
    split-invariance pin): o = sum_c e^{lse_c - lse} o_c,  lse = log sum_c e^{lse_c}."""
    lse_all = np.stack(lses)                      # [chunks][...]
    m = lse_all.max(axis=0)
    w = np.exp(lse_all - m)
    tot = w.sum(axis=0)
    o = sum(wc[..., None] * oc for wc, oc in zip(w, outs)) / tot[..., None]
    return o, m + np.log(tot)


# --------------------------------------------------------------------------------------
# Step 4c: greedy acceptance (the target decodes greedily; speculative decoding is lossless)
# --------------------------------------------------------------------------------------
def accept(target_logits: np.ndarray, draft_tokens: np.ndarray):
    """target_logits: fp32 [gamma+1][vocab]; draft_tokens: int [gamma].

    g_t = argmax_v logits[t][v] (lowest index on ties);  n = number of leading positions
    with draft[t] == g_t;  next = g_n (the correction, or the bonus token when n = gamma).
    Returns (n, next, g)."""
    logits = np.asarray(target_logits, dtype=np.float32)
    gamma = logits.shape[0] - 1
    g = []
    for t in range(gamma + 1):
        best, best_v = 0, logits[t, 0]
        for vtok in range(1, logits.shape[1]):
            if logits[t, vtok] > best_v:          # strict: lowest index wins ties
                best, best_v = vtok, logits[t, vtok]
        g.append(best)
    n = 0
    while n < gamma and int(draft_tokens[n]) == g[n]:
        n += 1
    return n, g[n], np.asarray(g, dtype=np.int32)


def accept_fast(target_logits: np.ndarray, draft_tokens: np.ndarray):
    """Same as ``accept`` with the argmax done by numpy (first occurrence of the maximum),
    for vocabularies too large for the Python loop."""
    logits = np.asarray(target_logits, dtype=np.float32)
    gamma = logits.shape[0] - 1
    g = np.argmax(logits, axis=1).astype(np.int32)
    n = 0
    while n < gamma and int(draft_tokens[n]) == int(g[n]):
        n += 1
    return n, int(g[n]), g


def sd_speedup(tau: float, gamma: int, t_draft: float, t_target: float, t_verify: float) -> float:
    """Eq. 3: speedup = tau / (gamma * T_d / T_t + T_t^gamma / T_t)."""
    return tau / (gamma * t_draft / t_target + t_verify / t_target)


# --------------------------------------------------------------------------------------
# Tree drafting (the paper's default draft shape, experimental set-up): the window holds a tree
# of drafted tokens instead of a chain.  Node 0 is the root (the last committed token);
# parents[t] < t is node t's parent, -1 for a root.
# --------------------------------------------------------------------------------------
def tree_ancestors(parents) -> list[list[int]]:
    """For every node the window positions it attends: its ancestors and itself, ascending."""
    out = []
    for t in range(len(parents)):
        chain, cur = [t], int(parents[t])
        while cur >= 0:
            assert cur < chain[-1], "parents must point to earlier nodes"
            chain.append(cur)
            cur = int(parents[cur])
        out.append(sorted(chain))
    return out


def attention_tree(q: np.ndarray, k: np.ndarray, v: np.ndarray, kv_len: int, parents, sm_scale: float):
    """Verification attention over a drafted tree.  q: uint16 [n_nodes][Hq][d]; k, v: uint16
    [Hkv][>= kv_len][d], whose last n_nodes valid rows are the tree's nodes in node order.  Node t
    sees every key before the window and the window rows of its ancestors and itself.
    Plain two-pass softmax in fp64.  Returns (out [n_nodes][Hq][d], lse [n_nodes][Hq])."""
    qf, kf, vf = bf16_bits_to_f64(_u16(q)), bf16_bits_to_f64(_u16(k)), bf16_bits_to_f64(_u16(v))
    n_nodes, hq, d = qf.shape
    hkv = kf.shape[0]
    group = hq // hkv
    old = kv_len - n_nodes
    anc = tree_ancestors(parents)
    out = np.zeros((n_nodes, hq, d))
    lse = np.zeros((n_nodes, hq))
    for t in range(n_nodes):
        keys = list(range(old)) + [old + a for a in anc[t]]
        for h in range(hq):
            g = h // group
            s = (kf[g, keys, :] @ qf[t, h, :]) * sm_scale
            m = s.max()
            e = np.exp(s - m)
            z = e.sum()
            out[t, h] = (e / z) @ vf[g, keys, :]
            lse[t, h] = m + math.log(z)
    return out, lse


def accept_tree(logits: np.ndarray, node_tokens, parents) -> tuple[int, int, list[int]]:
    """Greedy acceptance along the tree: starting at the root, step to the child whose token is
    the target's arg-max at the current node (lowest node index among equal children) until no
    child matches.  Returns (accepted drafts, the target's token after the last accepted node,
    accepted node indices in order)."""
    n_nodes = logits.shape[0]
    g = []
    for t in range(n_nodes):
        best, arg = -math.inf, 0
        for i, x in enumerate(logits[t].tolist()):
            if x > best:
                best, arg = x, i
        g.append(arg)
    cur, path = 0, []
    while True:
        nxt = -1
        for c in range(cur + 1, n_nodes):
            if int(parents[c]) == cur and int(node_tokens[c]) == g[cur]:
                nxt = c
                break
        if nxt < 0:
            break
        path.append(nxt)
        cur = nxt
    return len(path), g[cur], path


def compact_tree_kv(cache: np.ndarray, seq_len: int, n_nodes: int, path) -> tuple[np.ndarray, int]:
    """After tree acceptance: the accepted nodes' rows move up behind the root so that the cache is
    a plain sequence again.  cache: [..., tokens, d].  Returns (cache, new length = old + 1 + len(path))."""
    out = cache.copy()
    old = seq_len - n_nodes
    for i, node in enumerate(path):
        out[..., old + 1 + i, :] = cache[..., old + node, :]
    return out, old + 1 + len(path)


# --------------------------------------------------------------------------------------
# Attention-agnostic selectors the paper compares against (random pruning in its sensitivity
# study; a window over the front / middle / end of the video tokens and full-frame dropping at
# regular temporal intervals in its ablations).  Uniform-only and attention-only are `select`
# with k1 = 0 and k1 = k_total.
# --------------------------------------------------------------------------------------
SEL_WINDOW_FRONT, SEL_WINDOW_MIDDLE, SEL_WINDOW_END, SEL_FRAMES, SEL_RANDOM = 0, 1, 2, 3, 4


def philox4x32_10(counter, key) -> list[int]:
    """Philox-4x32 with 10 rounds (Salmon, Moraes, Dror, Shaw: "Parallel random numbers: as easy
    as 1, 2, 3", SC'11): the counter-based generator both sides implement for random pruning."""
    m0, m1, w0, w1 = 0xD2511F53, 0xCD9E8D57, 0x9E3779B9, 0xBB67AE85
    c, k = [int(x) & 0xFFFFFFFF for x in counter], [int(x) & 0xFFFFFFFF for x in key]
    for _ in range(10):
        p0, p1 = m0 * c[0], m1 * c[2]
        c = [(p1 >> 32) ^ c[1] ^ k[0], p1 & 0xFFFFFFFF, (p0 >> 32) ^ c[3] ^ k[1], p0 & 0xFFFFFFFF]
        k = [(k[0] + w0) & 0xFFFFFFFF, (k[1] + w1) & 0xFFFFFFFF]
    return c


def random_scores(n_video: int, seed: int, b: int = 0) -> np.ndarray:
    """One fp32 key per video token: the top 24 bits of the first Philox word at counter
    (token, sequence, 0, 0) under the 64-bit seed.  The largest keys are kept."""
    key = [seed & 0xFFFFFFFF, (seed >> 32) & 0xFFFFFFFF]
    return np.array([philox4x32_10([j, b, 0, 0], key)[0] >> 8 for j in range(n_video)], dtype=np.float32)


def select_baseline(mode: int, n_frames: int, tokens_per_frame: int, k_total: int, seed: int = 0, b: int = 0
                    ) -> np.ndarray:
    """Kept video indices (ascending) of an attention-agnostic selector under the budget k_total.
    Frame dropping keeps floor(k_total / T) whole frames, frame i of them being floor(i F / n)."""
    n_v = n_frames * tokens_per_frame
    assert 0 <= k_total <= n_v
    if mode == SEL_WINDOW_FRONT:
        kept = range(0, k_total)
    elif mode == SEL_WINDOW_MIDDLE:
        start = (n_v - k_total) // 2
        kept = range(start, start + k_total)
    elif mode == SEL_WINDOW_END:
        kept = range(n_v - k_total, n_v)
    elif mode == SEL_FRAMES:
        nf = k_total // tokens_per_frame
        kept = [((i * n_frames) // nf) * tokens_per_frame + t for i in range(nf) for t in range(tokens_per_frame)]
    elif mode == SEL_RANDOM:
        kept = stage1_topk(random_scores(n_v, seed, b), k_total)
    else:
        raise ValueError("unknown selector")
    return np.asarray(list(kept), dtype=np.int32)
