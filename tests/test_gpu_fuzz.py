"""Seeded random shapes through the attention, rating and selection entry points, against the
oracle.  The hand-picked cases of the other GPU tests aim at known edges; these sweep combinations
nobody thought of (group size x window rows x ragged lengths x paging x layer count), which is
where a flat work partition or a tile-edge mask would break.  Every case is small enough for the
fp64 oracle; the draws are fixed by the seed in the test id."""
import math
import os

import numpy as np
import pytest
import torch

import oracle
from gpu_util import make_cache
from helpers import bits, f64, row_rel_err
from paper_2508_16201_b200 import specvlm, synth
from test_gpu_parity import ATTN_TOL, _run_attn, _scores_case

pytestmark = pytest.mark.gpu

# SPECVLM_FUZZ_SCALE=10 runs ten times as many draws (a bug hunt, not the regular suite)
SCALE = int(os.environ.get("SPECVLM_FUZZ_SCALE", "1"))
# SPECVLM_FUZZ_FIRST=100000 starts the seeds elsewhere: another set of draws
FIRST = int(os.environ.get("SPECVLM_FUZZ_FIRST", "0"))


def _seeds(n):
    return range(FIRST, FIRST + n * SCALE)


GROUPS = [(4, 4), (8, 2), (28, 4), (40, 8), (64, 8), (16, 1), (12, 2),     # (query heads, KV heads)
          (6, 3), (6, 2), (18, 2), (11, 1), (26, 2), (30, 2)]              # groups of 2, 3, 9, 11, 13, 15 heads


def _lens(rng, batch, lo, hi, n_q):
    """ragged lengths; now and then a sequence that holds the window only, or sits on a tile edge"""
    out = []
    for _ in range(batch):
        r = rng.random()
        if r < 0.1:
            out.append(n_q)
        elif r < 0.25:
            out.append(int(rng.integers(1, 5)) * 64 + int(rng.integers(0, 2)) * n_q)
        else:
            out.append(int(rng.integers(max(lo, n_q), hi)))
    return out


@pytest.mark.parametrize("seed", _seeds(24))
def test_fuzz_chain_attention(seed):
    rng = np.random.default_rng(1000 + seed)
    Hq, Hkv = GROUPS[int(rng.integers(0, len(GROUPS)))]
    D = 64 if rng.random() < 0.3 else 128
    gamma = int(rng.integers(0, 9))
    L = int(rng.integers(1, 4))
    batch = int(rng.integers(1, 6))
    hi = 700
    if rng.random() < 0.2:                 # a few long sequences: items cut across several CTAs
        L, batch, hi = 1, int(rng.integers(1, 3)), 6000
    lens = _lens(rng, batch, 1, hi, gamma + 1)
    _run_attn(L, Hq, Hkv, D, lens, gamma, paged=bool(rng.integers(0, 2)), seed=2000 + seed, poison=True)


@pytest.mark.parametrize("seed", _seeds(16))
def test_fuzz_tree_attention(seed):
    rng = np.random.default_rng(3000 + seed)
    Hq, Hkv = GROUPS[int(rng.integers(0, len(GROUPS)))]
    D = 64 if rng.random() < 0.3 else 128
    n_nodes = int(rng.integers(1, 65)) if rng.random() < 0.3 else int(rng.integers(1, 33))
    L = int(rng.integers(1, 3))
    batch = int(rng.integers(1, 5))
    lens = _lens(rng, batch, 1, 500, n_nodes)
    paged = bool(rng.integers(0, 2))
    cache, k_host, v_host = make_cache(L, Hkv, D, lens, paged=paged, seed=4000 + seed, poison_tail=True)
    parents = [[-1] + [int(rng.integers(0, t)) for t in range(1, n_nodes)] for _ in range(batch)]
    par = torch.tensor(parents, dtype=torch.int32, device="cuda")
    q = synth.randn_bf16((L, batch, n_nodes, Hq, D), "cuda", 4000 + seed, "Qt")
    scale = 1.0 / math.sqrt(D)
    lse = torch.empty((L, batch, n_nodes, Hq), dtype=torch.float32, device="cuda")
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    out = specvlm.verify_tree_attn(cache, q, par, scale, lse=lse, d_status=status)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    got, qh = f64(out), bits(q)
    assert np.isfinite(got).all()
    worst = 0.0
    for l in range(L):
        for b in range(batch):
            ref, ref_lse = oracle.attention_tree(qh[l, b], k_host[b][l], v_host[b][l], lens[b], parents[b], scale)
            worst = max(worst, row_rel_err(got[l, b], ref))
            np.testing.assert_allclose(lse[l, b].cpu().numpy(), ref_lse, rtol=0, atol=2e-3)
    assert worst <= ATTN_TOL, f"row rel err {worst}"


@pytest.mark.parametrize("seed", _seeds(6))
def test_fuzz_scores(seed):
    rng = np.random.default_rng(5000 + seed)
    Hq, Hkv = GROUPS[int(rng.integers(0, len(GROUPS)))]
    D = 64 if rng.random() < 0.3 else 128
    batch = int(rng.integers(1, 4))
    T = int(rng.integers(20, 200))
    n_frames = [int(rng.integers(1, 5)) for _ in range(batch)]
    n_text = [int(rng.integers(1, 150)) for _ in range(batch)]
    prefix = [int(rng.integers(0, 80)) for _ in range(batch)]
    paged = bool(rng.integers(0, 2))
    _scores_case(int(rng.integers(1, 3)), Hq, Hkv, D, n_frames, T, n_text, paged=paged, seed=6000 + seed,
                 prefix=prefix)


@pytest.mark.parametrize("seed", _seeds(4))
def test_fuzz_scores_by_layer_ranges(seed):
    """random cuts of the layers (empty ranges included) give the bits of the single call"""
    rng = np.random.default_rng(5500 + seed)
    Hq, Hkv = GROUPS[int(rng.integers(0, len(GROUPS)))]
    D = 64 if rng.random() < 0.3 else 128
    L = int(rng.integers(2, 7))
    batch = int(rng.integers(1, 4))
    nv = [int(rng.integers(20, 400)) for _ in range(batch)]
    nt = [int(rng.integers(1, 100)) for _ in range(batch)]
    prefix = [int(rng.integers(0, 40)) for _ in range(batch)]
    cache, _, _ = make_cache(L, Hkv, D, [p + v + t for p, v, t in zip(prefix, nv, nt)],
                             paged=bool(rng.integers(0, 2)), seed=5600 + seed)
    text_cu = [0] + np.cumsum(nt).tolist()
    video_cu = [0] + np.cumsum(nv).tolist()
    q = synth.randn_bf16((L, text_cu[-1], Hq, D), "cuda", 5600 + seed, "Qtext")
    args = (text_cu, [p + v for p, v in zip(prefix, nv)], prefix, nv, video_cu, 1.0 / math.sqrt(D))
    whole = specvlm.stage1_scores(cache, q, *args)
    cuts = [0] + sorted(int(c) for c in rng.integers(0, L + 1, size=int(rng.integers(0, 4)))) + [L]
    ws = torch.full((specvlm.stage1_scores_workspace_bytes(cache, text_cu, nv, Hq),), 0xFF, dtype=torch.uint8,
                    device="cuda")
    out = torch.full((video_cu[-1],), float("nan"), device="cuda")
    for i, (a, b) in enumerate(zip(cuts[:-1], cuts[1:])):
        specvlm.stage1_scores_layers(cache, q, *args, out, ws, a, b, finish=(i == len(cuts) - 2))
    torch.cuda.synchronize()
    assert torch.equal(out, whole), cuts


@pytest.mark.parametrize("seed", _seeds(6))
def test_fuzz_select(seed):
    """Stage I + II on random score vectors with planted ties; fixed count and Top-P count."""
    rng = np.random.default_rng(7000 + seed)
    batch = int(rng.integers(1, 5))
    T = int(rng.integers(3, 300))
    frames = [int(rng.integers(1, 12)) for _ in range(batch)]
    nv = [f * T for f in frames]
    cu = np.concatenate([[0], np.cumsum(nv)]).astype(int).tolist()
    scores = rng.random(cu[-1]).astype(np.float32) ** 6          # long-tailed
    scores[rng.integers(0, cu[-1], size=cu[-1] // 5)] = scores[rng.integers(0, cu[-1])]   # ties
    kt = [int(rng.integers(0, n + 1)) for n in nv]
    k1 = [int(rng.integers(0, k + 1)) for k in kt]
    kept_cu = np.concatenate([[0], np.cumsum(kt)]).astype(int).tolist()
    sc_d = torch.from_numpy(scores).cuda()
    got = specvlm.select(sc_d, cu, frames, T, k1, kt, kept_cu).cpu().numpy()
    for b in range(batch):
        ref = oracle.select(scores[cu[b]:cu[b + 1]], frames[b], T, k1[b], kt[b])
        assert np.array_equal(got[kept_cu[b]:kept_cu[b + 1]], ref), f"sequence {b}"
    lam = [int(rng.integers(0, 1001)) for _ in range(batch)]
    got_p, k1_p = specvlm.select_top_p(sc_d, cu, frames, T, lam, kt, kept_cu)
    got_p, k1_p = got_p.cpu().numpy(), k1_p.cpu().numpy()
    for b in range(batch):
        ref, ref_k1 = oracle.select_top_p(scores[cu[b]:cu[b + 1]], frames[b], T, lam[b], kt[b])
        assert int(k1_p[b]) == ref_k1
        assert np.array_equal(got_p[kept_cu[b]:kept_cu[b + 1]], ref), f"top-p sequence {b}"


@pytest.mark.parametrize("seed", _seeds(6))
def test_fuzz_gather(seed):
    from gpu_util import host_view
    rng = np.random.default_rng(8000 + seed)
    L, H = int(rng.integers(1, 4)), int(rng.integers(1, 5))
    D = 64 if rng.random() < 0.3 else 128
    batch = int(rng.integers(1, 5))
    video_start = [int(rng.integers(0, 40)) for _ in range(batch)]
    video_len = [int(rng.integers(1, 600)) for _ in range(batch)]
    n_text = [int(rng.integers(1, 90)) for _ in range(batch)]
    src_len = [a + b + c for a, b, c in zip(video_start, video_len, n_text)]
    kept, kept_cu = [], [0]
    for nv in video_len:
        kk = np.sort(rng.choice(nv, int(rng.integers(0, nv + 1)), replace=False)).astype(np.int32)
        kept.append(kk)
        kept_cu.append(kept_cu[-1] + len(kk))
    dst_len = [s - v + len(k) for s, v, k in zip(src_len, video_len, kept)]
    src, sk, sv = make_cache(L, H, D, src_len, paged=bool(rng.integers(0, 2)), seed=8100 + seed)
    dst, _, _ = make_cache(L, H, D, dst_len, paged=bool(rng.integers(0, 2)), seed=8200 + seed)
    kept_all = np.concatenate(kept) if kept_cu[-1] else np.zeros(1, dtype=np.int32)
    specvlm.gather_kv(src, torch.from_numpy(kept_all).cuda(), kept_cu, video_start, video_len, src_len, dst)
    torch.cuda.synchronize()
    dk = host_view(dst.k, dst.block_table, dst_len)
    dv = host_view(dst.v, dst.block_table, dst_len)
    for b in range(batch):
        rk = oracle.gather_kv(sk[b], kept[b], video_start[b], video_len[b], src_len[b])
        rv = oracle.gather_kv(sv[b], kept[b], video_start[b], video_len[b], src_len[b])
        n = rk.shape[2]
        assert np.array_equal(dk[b][:, :, :n], rk) and np.array_equal(dv[b][:, :, :n], rv), f"sequence {b}"


@pytest.mark.parametrize("seed", _seeds(6))
def test_fuzz_accept_chain_and_tree(seed):
    rng = np.random.default_rng(9000 + seed)
    batch, gamma = int(rng.integers(1, 9)), int(rng.integers(0, 9))
    vocab = int(rng.choice([7, 1000, 4099, 32000, 152064]))
    g = torch.Generator().manual_seed(9000 + seed)
    logits = torch.randn((batch, gamma + 1, vocab), generator=g)
    if rng.random() < 0.5:                                   # exact ties: the lowest index wins
        logits = torch.round(logits * 2) / 2
    lg = logits.numpy()
    am = lg.argmax(2)
    drafts = np.where(rng.random((batch, gamma)) < 0.7, am[:, :gamma], rng.integers(0, vocab, (batch, gamma))).astype(np.int32)
    n, nxt, gmax = specvlm.accept(logits.cuda(), torch.from_numpy(drafts).cuda().contiguous(), want_argmax=True)
    torch.cuda.synchronize()
    for b in range(batch):
        rn, rnext = oracle.accept_fast(lg[b], drafts[b])[:2]
        assert (int(n[b]), int(nxt[b])) == (int(rn), int(rnext)), f"sequence {b}"
    assert np.array_equal(gmax.cpu().numpy(), am)
    # the same logits as a tree: node t's parent is a random earlier node
    n_nodes = gamma + 1
    parents = [[-1] + [int(rng.integers(0, t)) for t in range(1, n_nodes)] for _ in range(batch)]
    tokens = [[0] + [int(am[b, parents[b][t]]) if rng.random() < 0.7 else int(rng.integers(0, vocab))
                     for t in range(1, n_nodes)] for b in range(batch)]
    tn, tnxt, path, _ = specvlm.accept_tree(logits.cuda(), torch.tensor(tokens, dtype=torch.int32, device="cuda"),
                                            torch.tensor(parents, dtype=torch.int32, device="cuda"))
    torch.cuda.synchronize()
    for b in range(batch):
        rn, rnext, rpath = oracle.accept_tree(lg[b], tokens[b], parents[b])
        assert (int(tn[b]), int(tnxt[b])) == (rn, rnext), f"tree sequence {b}"
        assert path[b].cpu().tolist() == rpath + [-1] * (n_nodes - rn)


@pytest.mark.parametrize("seed", _seeds(4))
def test_fuzz_baseline_selectors(seed):
    rng = np.random.default_rng(9500 + seed)
    batch = int(rng.integers(1, 5))
    T = int(rng.integers(1, 300))
    frames = [int(rng.integers(1, 40)) for _ in range(batch)]
    kts = [int(rng.integers(0, f * T + 1)) for f in frames]
    kept_cu = np.concatenate([[0], np.cumsum(kts)]).astype(int).tolist()
    sd = int(rng.integers(0, 2**62))
    for mode in (specvlm.SEL_WINDOW_FRONT, specvlm.SEL_WINDOW_MIDDLE, specvlm.SEL_WINDOW_END, specvlm.SEL_FRAMES,
                 specvlm.SEL_RANDOM):
        kept, kept_n = specvlm.select_baseline(mode, frames, T, kts, kept_cu, seed=sd)
        kept, kept_n = kept.cpu().numpy(), kept_n.cpu().numpy()
        for b, F in enumerate(frames):
            ref = oracle.select_baseline(mode, F, T, kts[b], seed=sd, b=b)
            assert int(kept_n[b]) == len(ref), f"mode {mode} sequence {b}"
            assert np.array_equal(kept[kept_cu[b]:kept_cu[b] + len(ref)], ref), f"mode {mode} sequence {b}"


@pytest.mark.parametrize("seed", _seeds(6))
def test_fuzz_cache_append_rollback_compact(seed):
    """append -> rollback lengths, and tree compaction along a random accepted path, bit for bit."""
    from gpu_util import host_view
    rng = np.random.default_rng(9800 + seed)
    L, H = int(rng.integers(1, 4)), int(rng.integers(1, 5))
    D = 64 if rng.random() < 0.3 else 128
    batch = int(rng.integers(1, 5))
    paged = bool(rng.integers(0, 2))
    n_new = int(rng.integers(1, 10))
    lens = [int(rng.integers(0, 300)) for _ in range(batch)]
    cap = [n + n_new for n in lens]
    cache, k_host, v_host = make_cache(L, H, D, cap, paged=paged, seed=9900 + seed)
    cache.seq_lens.copy_(torch.tensor(lens, dtype=torch.int32))
    new_k = synth.randn_bf16((L, batch, n_new, H, D), "cuda", 9900 + seed, "nk")
    new_v = synth.randn_bf16((L, batch, n_new, H, D), "cuda", 9900 + seed, "nv")
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    specvlm.append_kv(cache, new_k, new_v, d_status=status)
    torch.cuda.synchronize()
    assert int(status.item()) == 0 and cache.seq_lens.cpu().tolist() == cap
    gk = host_view(cache.k, cache.block_table, cap)
    gv = host_view(cache.v, cache.block_table, cap)
    for b in range(batch):
        rk, _ = oracle.append_kv(k_host[b], bits(new_k[:, b]), lens[b])
        rv, _ = oracle.append_kv(v_host[b], bits(new_v[:, b]), lens[b])
        assert np.array_equal(gk[b], rk) and np.array_equal(gv[b], rv), f"append, sequence {b}"
        k_host[b], v_host[b] = rk, rv
    # the n_new rows as a draft tree's window: keep a random root-to-node path
    n_nodes = n_new
    paths = []
    for b in range(batch):
        parents = [-1] + [int(rng.integers(0, t)) for t in range(1, n_nodes)]
        node = int(rng.integers(0, n_nodes))
        chain = []
        while node > 0:
            chain.append(node)
            node = parents[node]
        paths.append(chain[::-1])
    path_d = torch.tensor([p + [-1] * (n_nodes - len(p)) for p in paths], dtype=torch.int32, device="cuda")
    n_acc = torch.tensor([len(p) for p in paths], dtype=torch.int32, device="cuda")
    specvlm.compact_tree_kv(cache, path_d, n_acc, d_status=status)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    new_lens = cache.seq_lens.cpu().tolist()
    gk = host_view(cache.k, cache.block_table, new_lens)
    gv = host_view(cache.v, cache.block_table, new_lens)
    for b in range(batch):
        rk, nl = oracle.compact_tree_kv(k_host[b], cap[b], n_nodes, paths[b])
        rv, _ = oracle.compact_tree_kv(v_host[b], cap[b], n_nodes, paths[b])
        assert new_lens[b] == nl
        assert np.array_equal(gk[b], rk[:, :, :nl]) and np.array_equal(gv[b], rv[:, :, :nl]), f"compaction, sequence {b}"
    # chain rollback arithmetic on fresh lengths
    gamma = n_new - 1
    acc = [int(rng.integers(0, gamma + 1)) for _ in range(batch)]
    lens_d = torch.tensor(cap, dtype=torch.int32, device="cuda")
    specvlm.rollback_kv(lens_d, torch.tensor(acc, dtype=torch.int32, device="cuda"), gamma)
    torch.cuda.synchronize()
    assert lens_d.cpu().tolist() == [oracle.rollback_len(cap[b], gamma, acc[b]) for b in range(batch)]
