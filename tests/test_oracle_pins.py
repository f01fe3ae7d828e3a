"""Pins for the CPU oracle: closed forms, hand-worked fixtures, brute force on tiny inputs,
invariants, and special cases that reduce to a library routine.  No GPU."""
import math
import os

import numpy as np
import pytest
import scipy.special
import torch

import oracle
from helpers import bits, from_f64, f64

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def _rand_bf16(shape, seed):
    g = torch.Generator().manual_seed(seed)
    return torch.randn(shape, generator=g).to(torch.bfloat16)


# ----------------------------------------------------------------------------- scores
def _scores_bruteforce(q, k, video_start, n_video, text_start, scale):
    """Literal transcription of Eq. 4-5 with python floats: full causal softmax matrix M,
    G = M[text rows, video cols], column mean, then mean over layers and heads."""
    L, n_text, Hq, d = q.shape
    Hkv = k.shape[1]
    qf, kf = f64(q), f64(k)
    a = [0.0] * n_video
    for l in range(L):
        for h in range(Hq):
            g = h // (Hq // Hkv)
            for i in range(n_text):
                p = text_start + i
                s = [scale * sum(qf[l, i, h, c] * kf[l, g, kk, c] for c in range(d)) for kk in range(p + 1)]
                mx = max(s)
                e = [math.exp(x - mx) for x in s]
                z = sum(e)
                for j in range(n_video):
                    a[j] += e[video_start + j] / z
    return [x / (L * Hq * n_text) for x in a]


def test_scores_bruteforce_tiny():
    # 1 layer, 1 head, |L| = 2, N_v = 3 (hand-sized), plus a GQA case with a text prefix
    for (L, Hq, Hkv, d, vs, nv, nt, seed) in [(1, 1, 1, 4, 0, 3, 2, 1), (2, 4, 2, 8, 2, 5, 3, 2)]:
        n_tok = vs + nv + nt
        q = _rand_bf16((L, nt, Hq, d), seed)
        k = _rand_bf16((L, Hkv, n_tok, d), seed + 100)
        ref = _scores_bruteforce(q, k, vs, nv, vs + nv, 0.5)
        got = oracle.stage1_scores(bits(q), bits(k), vs, nv, vs + nv, 0.5)
        np.testing.assert_allclose(got, ref, rtol=1e-12, atol=0)


def test_scores_closed_form_identical_keys():
    for line in open(os.path.join(GOLDEN, "scores_closed_form.txt")):
        if line.startswith("#") or not line.strip():
            continue
        nv, nt, expect = [x.strip() for x in line.split("|")]
        nv, nt, expect = int(nv), int(nt), float(expect)
        d, L, Hq, Hkv = 8, 2, 4, 2
        q = _rand_bf16((L, nt, Hq, d), 3)
        krow = _rand_bf16((d,), 4)
        k = krow.expand(L, Hkv, nv + nt, d).contiguous()
        got = oracle.stage1_scores(bits(q), bits(k), 0, nv, nv, 0.37)
        np.testing.assert_allclose(got, np.full(nv, expect), rtol=1e-13)
        # and the formula itself
        assert abs(expect - sum(1.0 / (nv + i + 1) for i in range(nt)) / nt) < 1e-15


def test_scores_invariants_and_library():
    L, Hq, Hkv, d, vs, nv, nt = 2, 8, 2, 16, 3, 40, 6
    n_tok = vs + nv + nt
    q = _rand_bf16((L, nt, Hq, d), 5)
    k = _rand_bf16((L, Hkv, n_tok, d), 6)
    scale = 1.0 / math.sqrt(d)
    a, mass, lse = oracle.stage1_scores(bits(q), bits(k), vs, nv, vs + nv, scale, want_rows=True)
    assert (a >= 0).all()
    assert a.sum() <= 1.0
    np.testing.assert_allclose(a.sum(), mass.mean(), rtol=1e-12)      # sum_j a_j = mean video mass
    assert (mass < 1.0).all() and (mass > 0).all()
    # library special case: fp64 softmax(QK^T/sqrt(d) + causal mask) with torch
    qd = q.double().permute(0, 2, 1, 3)                                # [L][Hq][nt][d]
    kd = k.double().repeat_interleave(Hq // Hkv, dim=1)                # [L][Hq][n_tok][d]
    s = torch.einsum("lhid,lhkd->lhik", qd, kd) * scale
    pos = torch.arange(nt)[:, None] + vs + nv
    mask = torch.arange(n_tok)[None, :] > pos
    s = s.masked_fill(mask, float("-inf"))
    M = torch.softmax(s, dim=-1)
    np.testing.assert_allclose(M.sum(-1).numpy(), 1.0, rtol=1e-12)     # rows of M sum to 1
    G = M[..., vs:vs + nv]
    ref = G.mean(dim=(0, 1, 2)).numpy()
    np.testing.assert_allclose(a, ref, rtol=1e-11)
    # (scipy's routine: torch.logsumexp's first call in a process now and then returns one thread's
    # block of rows 4e-10 off, and the exact values when called again)
    np.testing.assert_allclose(lse, scipy.special.logsumexp(s.numpy(), axis=-1), rtol=1e-12)
    # the other reading (softmax over video keys only) is a different function
    a2 = oracle.stage1_scores(bits(q), bits(k), vs, nv, vs + nv, scale, video_only=True)
    np.testing.assert_allclose(a2.sum(), 1.0, rtol=1e-12)
    assert np.abs(a2 - a).max() > 1e-4


def test_scores_symmetries():
    L, Hq, Hkv, d, nv, nt = 1, 4, 2, 8, 12, 3
    q = _rand_bf16((L, nt, Hq, d), 7)
    k = _rand_bf16((L, Hkv, nv + nt, d), 8)
    a = oracle.stage1_scores(bits(q), bits(k), 0, nv, nv, 0.3)
    # permuting the video keys permutes A
    perm = torch.randperm(nv, generator=torch.Generator().manual_seed(9))
    k2 = k.clone()
    k2[:, :, :nv] = k[:, :, perm]
    a2 = oracle.stage1_scores(bits(q), bits(k2), 0, nv, nv, 0.3)
    np.testing.assert_allclose(a2, a[perm.numpy()], rtol=1e-12)
    # duplicating the layer leaves A unchanged
    a3 = oracle.stage1_scores(bits(torch.cat([q, q])), bits(torch.cat([k, k])), 0, nv, nv, 0.3)
    np.testing.assert_allclose(a3, a, rtol=1e-12)
    # the head -> KV-head map is h // group: swapping the two KV heads while swapping the
    # query-head groups leaves A unchanged; swapping only the KV heads does not
    k4 = k.flip(1)
    q4 = torch.cat([q[:, :, 2:], q[:, :, :2]], dim=2)
    np.testing.assert_allclose(oracle.stage1_scores(bits(q4), bits(k4), 0, nv, nv, 0.3), a, rtol=1e-12)
    assert np.abs(oracle.stage1_scores(bits(q), bits(k4), 0, nv, nv, 0.3) - a).max() > 1e-6


# ----------------------------------------------------------------------------- selection
def _golden_select_cases():
    for line in open(os.path.join(GOLDEN, "stage2_handworked.txt")):
        if line.startswith("#") or not line.strip():
            continue
        name, F, T, k1, kt, scores, kept = [x.strip() for x in line.split("|")]
        yield (name, int(F), int(T), int(k1), int(kt),
               np.array(scores.split(), dtype=np.float32), [int(x) for x in kept.split()])


def test_select_handworked():
    n = 0
    for name, F, T, k1, kt, scores, kept in _golden_select_cases():
        got = oracle.select(scores, F, T, k1, kt)
        assert got.tolist() == kept, name
        n += 1
    assert n == 4


def test_topk_against_stable_sort_and_ties():
    rng = np.random.default_rng(0)
    for n, k1 in [(50, 7), (64, 64), (33, 0), (200, 100)]:
        s = rng.integers(0, 6, size=n).astype(np.float32)       # many ties
        got = oracle.stage1_topk(s, k1)
        order = np.argsort(-s, kind="stable")                    # library: stable => lower index first
        assert sorted(order[:k1].tolist()) == got
        rest = sorted(set(range(n)) - set(got))
        if got and rest:
            # every kept element precedes every dropped one in (score desc, index asc)
            worst_kept = max(got, key=lambda j: (-s[j], j))
            best_rest = min(rest, key=lambda j: (-s[j], j))
            assert (-s[worst_kept], worst_kept) < (-s[best_rest], best_rest)


def test_stage2_invariants():
    rng = np.random.default_rng(1)
    for (F, T, perm_keep) in [(4, 196, 100), (32, 196, 100), (3, 50, 500), (5, 36, 50), (7, 11, 900)]:
        nv = F * T
        s = rng.random(nv).astype(np.float32)
        kt = nv * perm_keep // 1000
        k1 = kt // 2
        v_r = oracle.stage1_topk(s, k1)
        v_u = oracle.stage2_uniform(v_r, F, T, kt)
        kept = oracle.select(s, F, T, k1, kt)
        assert len(kept) == kt and len(v_u) == kt - k1
        assert not (set(v_r) & set(v_u))
        assert (np.diff(kept) > 0).all()
        m, n_u = nv - k1, kt - k1
        in_r = set(v_r)
        for f in range(F):
            r_f = [j for j in range(f * T, (f + 1) * T) if j not in in_r]
            picks = [j for j in v_u if f * T <= j < (f + 1) * T]
            c_f, n_f = len(r_f), len(picks)
            assert abs(n_f - c_f * n_u / m) < 1.0                 # quota proportional to c_f
            if n_f:
                ranks = [r_f.index(j) for j in picks]
                assert ranks[0] == 0                              # phase restarts at the frame start
                gaps = set(np.diff(ranks).tolist())
                assert gaps <= {c_f // n_f, -(-c_f // n_f)}       # even spacing: floor or ceil of c_f/n_f


def test_stage2_textbook_stride():
    # k1 = 0, one frame, N_v divisible by n_U: indices 0, I, 2I, ...
    s = np.arange(60, 0, -1, dtype=np.float32)
    assert oracle.select(s, 1, 60, 0, 12).tolist() == list(range(0, 60, 5))
    # two frames, divisible per frame
    assert oracle.select(s, 2, 30, 0, 12).tolist() == list(range(0, 60, 5))


def test_top_p_count():
    s = np.array([4, 3, 2, 1], dtype=np.float32)     # exact in fp32; total 10
    assert oracle.stage1_top_p(s, 0.4) == 1
    assert oracle.stage1_top_p(s, 0.41) == 2
    assert oracle.stage1_top_p(s, 0.95) == 4
    assert oracle.stage1_top_p(s, 0.95, k_cap=3) == 3
    assert oracle.stage1_top_p(s[::-1].copy(), 0.41) == 2        # order of the input is irrelevant


def test_top_p_fixed_point_count():
    """The integer form of Eq. 6 that the GPU decision uses: hand-worked dyadic cases (every value
    exact in 2^-36 units), ties, the budget cap, and agreement with the fp64 form on long-tailed
    random scores, where no cumulative sum sits within rounding of the threshold."""
    s = np.array([0.125, 0.5, 0.125, 0.25], dtype=np.float32)       # ranking: 1, 3, 0, 2; total 1
    assert oracle.stage1_top_p_fixed(s, 500) == 1                    # 0.5 >= 0.5
    assert oracle.stage1_top_p_fixed(s, 501) == 2
    assert oracle.stage1_top_p_fixed(s, 750) == 2
    assert oracle.stage1_top_p_fixed(s, 751) == 3
    assert oracle.stage1_top_p_fixed(s, 876) == 4
    assert oracle.stage1_top_p_fixed(s, 1000) == 4
    assert oracle.stage1_top_p_fixed(s, 0) == 0
    assert oracle.stage1_top_p_fixed(s, 1000, k_cap=3) == 3
    kept, k1 = oracle.select_top_p(s, 1, 4, 751, 3)
    assert k1 == 3 and kept.tolist() == [0, 1, 3]                    # the tie 0.125 goes to the lower index
    kept, k1 = oracle.select_top_p(s, 1, 4, 500, 3)                  # Stage I keeps 1, Stage II adds 2 of the rest
    assert k1 == 1 and len(kept) == 3 and 1 in kept.tolist()
    assert oracle.stage1_top_p_fixed(np.zeros(5, dtype=np.float32), 400) == 0   # no mass: nothing to reach
    rng = np.random.default_rng(11)
    for lam in (400, 500, 900):
        for _ in range(5):
            a = rng.pareto(1.5, size=3000).astype(np.float32)
            a = (a / a.sum()).astype(np.float32)                     # long-tailed, sums to ~1 like a rating
            assert oracle.stage1_top_p_fixed(a, lam) == oracle.stage1_top_p(a, lam / 1000.0)


# ----------------------------------------------------------------------------- gather
def test_gather_is_fancy_index():
    g = torch.Generator().manual_seed(3)
    src = torch.randint(0, 65535, (2, 3, 20, 4), generator=g).numpy().astype(np.uint16)
    kept = np.array([1, 4, 5, 9], dtype=np.int32)
    out = oracle.gather_kv(src, kept, video_start=2, n_video=12, seq_len=18)
    rows = [0, 1, 3, 6, 7, 11, 14, 15, 16, 17]
    assert np.array_equal(out, src[:, :, rows, :])


# ----------------------------------------------------------------------------- attention
def test_attention_special_cases():
    d, Hq, Hkv = 16, 4, 2
    q = _rand_bf16((1, Hq, d), 10)
    k = _rand_bf16((Hkv, 9, d), 11)
    v = _rand_bf16((Hkv, 9, d), 12)
    # single key: o = V
    o, lse = oracle.attention(bits(q), bits(k), bits(v), 1, 0.25)
    for h in range(Hq):
        np.testing.assert_array_equal(o[0, h], f64(v)[h // 2, 0])
    # identical keys: o = mean(V)
    k_same = k[:, :1].expand(Hkv, 9, d).contiguous()
    o, _ = oracle.attention(bits(q), bits(k_same), bits(v), 9, 0.25)
    for h in range(Hq):
        np.testing.assert_allclose(o[0, h], f64(v)[h // 2].mean(axis=0), rtol=1e-13)
    # rows of P sum to one
    p = oracle.attention_probs(bits(q)[0, 0], bits(k)[0], 9, 0.25)
    assert abs(p.sum() - 1.0) < 1e-14 and (p > 0).all()


@pytest.mark.parametrize("n_q", [1, 5])
def test_attention_against_library_sdpa(n_q):
    d, Hq, Hkv, n = 64, 8, 2, 197
    q = _rand_bf16((n_q, Hq, d), 20)
    k = _rand_bf16((Hkv, n + 3, d), 21)       # kv_stride > kv_len
    v = _rand_bf16((Hkv, n + 3, d), 22)
    scale = 1.0 / math.sqrt(d)
    o, lse = oracle.attention(bits(q), bits(k), bits(v), n, scale)
    qd = q.double().permute(1, 0, 2)[None]                                   # [1][Hq][n_q][d]
    kd = k[:, :n].double().repeat_interleave(Hq // Hkv, dim=0)[None]
    vd = v[:, :n].double().repeat_interleave(Hq // Hkv, dim=0)[None]
    # query t sees keys [0, n - n_q + t]
    mask = torch.arange(n)[None, :] <= (torch.arange(n_q)[:, None] + n - n_q)
    ref = torch.nn.functional.scaled_dot_product_attention(qd, kd, vd, attn_mask=mask, scale=scale)
    np.testing.assert_allclose(o, ref[0].permute(1, 0, 2).numpy(), rtol=1e-10, atol=1e-13)
    # the second output, the natural-log sum-exp of each row's scaled visible logits, against a
    # library log-sum-exp of the masked logit matrix
    logits = torch.einsum("hqd,hkd->qhk", qd[0], kd[0]).numpy() * scale              # [n_q][Hq][n]
    logits = np.where(mask.numpy()[:, None, :], logits, -np.inf)
    np.testing.assert_allclose(lse, scipy.special.logsumexp(logits, axis=-1), rtol=1e-12)


def test_verify_rows_equal_truncated_decode_and_split_invariance():
    d, Hq, Hkv, n, gamma = 32, 4, 1, 150, 4
    q = _rand_bf16((gamma + 1, Hq, d), 30)
    k = _rand_bf16((Hkv, n, d), 31)
    v = _rand_bf16((Hkv, n, d), 32)
    o, lse = oracle.attention(bits(q), bits(k), bits(v), n, 0.2)
    for t in range(gamma + 1):
        od, ld = oracle.attention(bits(q[t:t + 1]), bits(k), bits(v), n - gamma + t, 0.2)
        np.testing.assert_allclose(o[t], od[0], rtol=1e-13)
        np.testing.assert_allclose(lse[t], ld[0], rtol=1e-13)
    # gamma = 0 verify == decode by construction; chunked evaluation + LSE merge == one pass
    q1 = q[:1]
    full, lfull = oracle.attention(bits(q1), bits(k), bits(v), n, 0.2)
    outs, lses = [], []
    for lo, hi in [(0, 64), (64, 128), (128, 150)]:
        oc, lc = oracle.attention(bits(q1), bits(k[:, lo:hi].contiguous()), bits(v[:, lo:hi].contiguous()),
                                  hi - lo, 0.2)
        outs.append(oc)
        lses.append(lc)
    om, lm = oracle.merge_partials(outs, lses)
    np.testing.assert_allclose(om, full, rtol=1e-12, atol=1e-15)
    np.testing.assert_allclose(lm, lfull, rtol=1e-12)


# ----------------------------------------------------------------------------- accept
def test_accept_cases():
    rng = np.random.default_rng(5)
    gamma, vocab = 4, 50
    logits = rng.standard_normal((gamma + 1, vocab)).astype(np.float32)
    g = logits.argmax(axis=1)
    # drafts equal the target's greedy tokens: everything accepted, bonus token = g_gamma
    n, nxt, gg = oracle.accept(logits, g[:gamma])
    assert (n, nxt) == (gamma, g[gamma]) and gg.tolist() == g.tolist()
    # first draft wrong: nothing accepted, correction = g_0
    bad = g[:gamma].copy()
    bad[0] = (bad[0] + 1) % vocab
    assert oracle.accept(logits, bad)[:2] == (0, g[0])
    # wrong in the middle; later matches do not count
    bad = g[:gamma].copy()
    bad[2] = (bad[2] + 1) % vocab
    assert oracle.accept(logits, bad)[:2] == (2, g[2])
    # losslessness: emitted tokens = draft[0..n) ++ next always equal the target's own g_0..g_n
    for _ in range(20):
        dr = np.where(rng.random(gamma) < 0.6, g[:gamma], rng.integers(0, vocab, gamma))
        n, nxt, _ = oracle.accept(logits, dr)
        assert list(dr[:n]) + [nxt] == g[:n + 1].tolist()
        assert oracle.accept_fast(logits, dr)[:2] == (n, nxt)
    # ties resolve to the lowest index
    tie = np.zeros((1, 8), dtype=np.float32)
    tie[0, [3, 5]] = 2.0
    assert oracle.accept(tie, np.zeros(0, dtype=np.int32))[:2] == (0, 3)
    assert oracle.accept_fast(tie, np.zeros(0, dtype=np.int32))[:2] == (0, 3)


def test_speedup_formula():
    # Eq. 3 special cases: a free draft and memory-bound verification give speedup = tau
    assert oracle.sd_speedup(3.0, 5, 0.0, 1.0, 1.0) == 3.0
    assert abs(oracle.sd_speedup(3.48, 5, 0.1, 1.0, 1.0) - 3.48 / 1.5) < 1e-12


# ----------------------------------------------------------------------------- cache maintenance
def test_append_and_rollback():
    rng = np.random.default_rng(8)
    cache = rng.integers(0, 65535, (2, 3, 10, 4)).astype(np.uint16)
    new = rng.integers(0, 65535, (2, 2, 3, 4)).astype(np.uint16)
    out, n = oracle.append_kv(cache, new, 5)
    assert n == 7
    assert np.array_equal(out[:, :, :5], cache[:, :, :5]) and np.array_equal(out[:, :, 7:], cache[:, :, 7:])
    assert np.array_equal(out[1, 2, 6], new[1, 1, 2]) and np.array_equal(out[0, 0, 5], new[0, 0, 0])
    # window of gamma + 1 = 5 tokens at the end of 20: all drafts accepted keeps them all, none keeps one
    assert oracle.rollback_len(20, 4, 4) == 20 and oracle.rollback_len(20, 4, 0) == 16
    assert oracle.rollback_len(20, 4, 2) == 18
    # appending gamma + 1 tokens then rolling back with n accepted leaves old + n + 1 tokens
    assert oracle.rollback_len(13 + 6, 5, 3) == 13 + 3 + 1


# ----------------------------------------------------------------------------- tree drafting
def test_tree_attention_reduces_to_chain_and_is_path_local():
    rng = np.random.default_rng(12)
    hq, hkv, d, old = 4, 2, 16, 9
    bf = lambda shape: (rng.standard_normal(shape).astype(np.float32).view(np.uint32) >> 16).astype(np.uint16)
    # a chain is the tree parents[t] = t - 1: must equal the chain attention (C routine) exactly
    n = 5
    q, k, v = bf((n, hq, d)), bf((hkv, old + n, d)), bf((hkv, old + n, d))
    o_tree, l_tree = oracle.attention_tree(q, k, v, old + n, [-1, 0, 1, 2, 3], 0.25)
    o_chain, l_chain = oracle.attention(q, k, v, old + n, 0.25)
    np.testing.assert_allclose(o_tree, o_chain, rtol=0, atol=1e-12)
    np.testing.assert_allclose(l_tree, l_chain, rtol=0, atol=1e-12)
    # a node's output depends on its own root path only: node 3 (path 0-1-3) must equal the last
    # row of the chain attention over the cache with rows (0, 1, 3) of the window kept
    parents = [-1, 0, 0, 1, 2]
    assert oracle.tree_ancestors(parents) == [[0], [0, 1], [0, 2], [0, 1, 3], [0, 2, 4]]
    o_tree, _ = oracle.attention_tree(q, k, v, old + n, parents, 0.25)
    keep = list(range(old)) + [old + 0, old + 1, old + 3]
    o_path, _ = oracle.attention(q[[0, 1, 3]], k[:, keep], v[:, keep], len(keep), 0.25)
    np.testing.assert_allclose(o_tree[3], o_path[2], rtol=0, atol=1e-12)
    np.testing.assert_allclose(o_tree[1], o_path[1], rtol=0, atol=1e-12)


def test_tree_acceptance_and_compaction():
    # logits rows put all mass on one token: g = [7, 3, 9, 5, 1]
    g = [7, 3, 9, 5, 1]
    logits = np.full((5, 12), -1.0, dtype=np.float32)
    for t, a in enumerate(g):
        logits[t, a] = 2.0
    parents = [-1, 0, 0, 1, 1]
    # children of the root carry tokens 4 and 7 -> node 2 accepted; node 2 has no children
    assert oracle.accept_tree(logits, [0, 4, 7, 5, 3], parents) == (1, 9, [2])
    # root -> node 1 (token 7) -> node 4 (token 3 = g[1]) ; next token g[4]
    assert oracle.accept_tree(logits, [0, 7, 8, 5, 3], parents) == (2, 1, [1, 4])
    # nothing matches
    assert oracle.accept_tree(logits, [0, 1, 2, 3, 4], parents) == (0, 7, [])
    # a chain tree gives the chain rule
    rng = np.random.default_rng(13)
    for _ in range(20):
        lg = rng.standard_normal((5, 30)).astype(np.float32)
        am = lg.argmax(1)
        drafts = np.where(rng.random(4) < 0.6, am[:4], rng.integers(0, 30, 4))
        n, nxt, _ = oracle.accept(lg, drafts)
        tn, tnxt, path = oracle.accept_tree(lg, [0] + drafts.tolist(), [-1, 0, 1, 2, 3])
        assert (tn, tnxt) == (n, nxt) and path == list(range(1, n + 1))
    # compaction: rows old+path[i] move to old+1+i
    cache = np.arange(2 * 12 * 3, dtype=np.uint16).reshape(2, 12, 3)
    out, n = oracle.compact_tree_kv(cache, 12, 5, [2, 4])
    assert n == 7 + 1 + 2
    assert np.array_equal(out[:, :8], cache[:, :8]) and np.array_equal(out[:, 8], cache[:, 9])
    assert np.array_equal(out[:, 9], cache[:, 11])


# ----------------------------------------------------------------------------- baseline selectors
def test_philox_known_answers_and_baseline_selectors():
    for line in open(os.path.join(GOLDEN, "philox4x32_10_kat.txt")):
        if line.startswith("#") or not line.strip():
            continue
        w = [int(x, 16) for x in line.split()]
        assert oracle.philox4x32_10(w[0:4], w[4:6]) == w[6:10]
    F, T, K = 5, 6, 13
    assert oracle.select_baseline(oracle.SEL_WINDOW_FRONT, F, T, K).tolist() == list(range(13))
    assert oracle.select_baseline(oracle.SEL_WINDOW_MIDDLE, F, T, K).tolist() == list(range(8, 21))
    assert oracle.select_baseline(oracle.SEL_WINDOW_END, F, T, K).tolist() == list(range(17, 30))
    # 13 // 6 = 2 whole frames at regular intervals: frames 0 and 2 of 5
    assert oracle.select_baseline(oracle.SEL_FRAMES, F, T, K).tolist() == list(range(0, 6)) + list(range(12, 18))
    r = oracle.select_baseline(oracle.SEL_RANDOM, 32, 196, 627, seed=7)
    assert len(r) == 627 and len(set(r.tolist())) == 627 and (np.diff(r) > 0).all()
    assert not np.array_equal(r, oracle.select_baseline(oracle.SEL_RANDOM, 32, 196, 627, seed=8))
    # roughly uniform over the frames: every frame keeps between 5 and 40 of its 196 tokens (mean 19.6)
    per_frame = np.bincount(r // 196, minlength=32)
    assert per_frame.min() >= 5 and per_frame.max() <= 40
