"""GPU parity: every entry point of the C ABI against the CPU oracle on the same seeded inputs.

Tolerances (stated by the benchmark's target): selected indices and acceptance results bit-exact;
bf16 attention outputs within 1e-2 max relative error per output row (max |diff| over the row
divided by max |ref| over the row); fp32 scores within 1e-4 relative.
"""
import math
import os

import numpy as np
import pytest
import torch

import oracle
from helpers import bits, f64, row_rel_err
from paper_2508_16201_b200 import specvlm, synth

pytestmark = pytest.mark.gpu

ATTN_TOL = 1e-2
SCORE_TOL = 1e-4


@pytest.fixture(autouse=True)
def _sync():
    yield
    torch.cuda.synchronize()


def _oracle_attn(q_host, k_host, v_host, seq_lens, scale):
    """q_host: uint16 [L][B][n_q][Hq][D]; returns fp64 out [L][B][n_q][Hq][D], lse [L][B][n_q][Hq]."""
    L, B, NQ, Hq, D = q_host.shape
    out = np.zeros((L, B, NQ, Hq, D))
    lse = np.zeros((L, B, NQ, Hq))
    for l in range(L):
        for b in range(B):
            o, s = oracle.attention(q_host[l, b], k_host[b][l], v_host[b][l], seq_lens[b], scale)
            out[l, b], lse[l, b] = o, s
    return out, lse


def _run_attn(L, Hq, Hkv, D, seq_lens, gamma, *, paged, seed, decode_api=False, splits=None,
              poison=False, extra_capacity=0):
    from gpu_util import make_cache
    B = len(seq_lens)
    cache, k_host, v_host = make_cache(L, Hkv, D, seq_lens, paged=paged, seed=seed, poison_tail=poison,
                                       extra_capacity=extra_capacity)
    nq = gamma + 1
    q = synth.randn_bf16((L, B, nq, Hq, D), "cuda", seed, "Q")
    scale = 1.0 / math.sqrt(D)
    lse = torch.empty((L, B, nq, Hq), dtype=torch.float32, device="cuda")
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    if splits is not None:
        specvlm.debug_set_attn_splits(splits)
    try:
        if decode_api:
            assert gamma == 0
            out = specvlm.draft_decode_attn(cache, q[:, :, 0].contiguous(), scale, lse=lse, d_status=status)
            out = out[:, :, None]
        else:
            out = specvlm.verify_attn(cache, q, gamma, scale, lse=lse, d_status=status)
    finally:
        specvlm.debug_set_attn_splits(0)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    ref, ref_lse = _oracle_attn(bits(q), k_host, v_host, seq_lens, scale)
    got = f64(out)
    assert np.isfinite(got).all()
    err = row_rel_err(got, ref)
    assert err <= ATTN_TOL, f"row rel err {err}"
    np.testing.assert_allclose(lse.cpu().numpy(), ref_lse, rtol=0, atol=2e-3)
    return err


# ------------------------------------------------------------------------------- decode attention
@pytest.mark.parametrize("splits", [None, 1, 3])
def test_decode_cfg1_shapes(splits):
    # draft of the tiny config: 4 q heads / 1 kv head, d = 64, pruned cache 78 + 64 = 142 tokens
    _run_attn(1, 4, 1, 64, [142], 0, paged=False, seed=0, decode_api=True, splits=splits)


@pytest.mark.parametrize("paged", [False, True])
@pytest.mark.parametrize("splits", [None, 1, 5])
def test_decode_llava7b_shapes(paged, splits):
    # 28 q / 4 kv heads (group 7), d = 128; 755 tokens = 11 full tiles + a ragged one; 2 layers
    _run_attn(2, 28, 4, 128, [755], 0, paged=paged, seed=1, decode_api=True, splits=splits)


@pytest.mark.parametrize("n", [1, 2, 15, 16, 17, 63, 64, 65, 128, 129])
def test_decode_edge_lengths(n):
    _run_attn(1, 8, 2, 128, [n], 0, paged=(n % 2 == 0), seed=2 + n, decode_api=True, poison=True)


def test_decode_ragged_batch_paged_poisoned():
    _run_attn(2, 28, 4, 128, [300, 64, 1, 777, 130], 0, paged=True, seed=3, decode_api=True, poison=True)
    _run_attn(2, 28, 4, 128, [300, 64, 1, 777, 130], 0, paged=False, seed=3, decode_api=True, poison=True,
              splits=4, extra_capacity=5)


def test_decode_group_sizes():
    for Hq, Hkv in [(4, 4), (16, 1), (10, 2), (32, 4)]:
        _run_attn(1, Hq, Hkv, 128, [200], 0, paged=False, seed=4, decode_api=True)
        _run_attn(1, Hq, Hkv, 64, [200], 0, paged=True, seed=4, decode_api=True)


# ------------------------------------------------------------------------------- verify attention
def test_verify_gamma0_equals_decode():
    from gpu_util import make_cache
    cache, _, _ = make_cache(2, 4, 128, [333, 70], paged=True, seed=5)
    q = synth.randn_bf16((2, 2, 1, 28, 128), "cuda", 5, "Q")
    a = specvlm.verify_attn(cache, q, 0, 0.09)
    b = specvlm.draft_decode_attn(cache, q[:, :, 0].contiguous(), 0.09)
    assert torch.equal(a[:, :, 0], b)


@pytest.mark.parametrize("splits", [None, 1, 4])
def test_verify_cfg1(splits):
    # verifier of the tiny config: 8 q / 2 kv heads, d = 64, 784 + 64 tokens + gamma+1 new ones
    _run_attn(1, 8, 2, 64, [784 + 64 + 5], 4, paged=False, seed=6, splits=splits)


@pytest.mark.parametrize("Hq,Hkv,gamma,D", [
    (64, 8, 5, 128),    # 48 rows: LLaVA-OV-72B shape
    (40, 8, 5, 128),    # 30 rows: Qwen2.5-VL-32B shape
    (64, 8, 6, 128),    # 56 rows
    (64, 8, 8, 128),    # 72 rows
    (64, 8, 3, 128),    # 32 rows
    (28, 4, 1, 128),    # 14 rows -> single m-tile kernel
    (16, 2, 8, 64),     # 72 rows, d = 64
    (12, 1, 7, 64),     # 96 rows
])
@pytest.mark.parametrize("paged", [False, True])
def test_verify_row_counts(Hq, Hkv, gamma, D, paged):
    _run_attn(1, Hq, Hkv, D, [421, 64 + gamma, 9 + gamma], gamma, paged=paged, seed=7, poison=True)
    _run_attn(1, Hq, Hkv, D, [421], gamma, paged=paged, seed=8, splits=3)


@pytest.mark.parametrize("paged", [False, True])
def test_verify_window_wider_than_one_launch(paged):
    # group 16 with gamma 8: 144 rows, cut into two parts of 5 and 4 query tokens
    _run_attn(2, 32, 2, 128, [300, 64 + 9, 9], 8, paged=paged, seed=11, poison=True)
    _run_attn(1, 16, 1, 64, [200], 8, paged=paged, seed=12)


def test_verify_window_crossing_tile_boundary():
    # the gamma+1 new tokens straddle a 64-token tile edge, and sit alone in the last tile
    for n in [64 + 3, 128, 128 + 6, 6]:
        _run_attn(1, 64, 8, 128, [n], 5, paged=True, seed=9, poison=True)


def test_attention_is_deterministic():
    from gpu_util import make_cache
    cache, _, _ = make_cache(2, 8, 128, [1000, 500], paged=True, seed=10)
    q = synth.randn_bf16((2, 2, 6, 64, 128), "cuda", 10, "Q")
    a = specvlm.verify_attn(cache, q, 5, 0.09)
    b = specvlm.verify_attn(cache, q, 5, 0.09)
    assert torch.equal(a, b)


# ------------------------------------------------------------------------------- accept
@pytest.mark.parametrize("batch,gamma,vocab", [(1, 4, 1024), (3, 5, 152064), (16, 8, 152064), (2, 0, 1000),
                                               (2, 3, 4099), (1, 6, 7)])
def test_accept_bit_exact(batch, gamma, vocab):
    logits, drafts = synth.logits_and_drafts(batch, gamma, vocab, "cuda", 11)
    n, nxt, g = specvlm.accept(logits, drafts, want_argmax=True)
    lh, dh = logits.cpu().numpy(), drafts.cpu().numpy()
    seen = set()
    for b in range(batch):
        rn, rnext, rg = oracle.accept_fast(lh[b], dh[b])
        assert int(n[b]) == rn and int(nxt[b]) == rnext
        assert g[b].cpu().numpy().tolist() == rg.tolist()
        seen.add(rn)
    if batch >= 16:
        assert len(seen) >= 3          # acceptance lengths cover several values


def test_accept_small_exact_loop_and_ties():
    # python-loop oracle on a small vocabulary, with planted exact ties (lowest index must win)
    logits, drafts = synth.logits_and_drafts(2, 4, 257, "cuda", 12)
    logits[0, 1, 200] = logits[0, 1].max()
    logits[0, 1, 13] = logits[0, 1].max()
    logits[1, 0, :] = 0.5                       # a whole row of ties -> index 0
    logits[1, 3, 255] = 9.0
    logits[1, 3, 256] = 9.0
    n, nxt, g = specvlm.accept(logits, drafts, want_argmax=True)
    for b in range(2):
        rn, rnext, rg = oracle.accept(logits[b].cpu().numpy(), drafts[b].cpu().numpy())
        assert (int(n[b]), int(nxt[b])) == (rn, rnext)
        assert g[b].cpu().tolist() == rg.tolist()
    assert int(g[0, 1]) == 13 and int(g[1, 0]) == 0 and int(g[1, 3]) == 255


# ------------------------------------------------------------------------------- select
def _select_case(n_frames_list, T, perm, seed, ties=False):
    rng = np.random.default_rng(seed)
    scores, video_cu, k1s, kts, kept_cu = [], [0], [], [], [0]
    for F in n_frames_list:
        nv = F * T
        s = rng.random(nv).astype(np.float32) * 1e-3
        if ties:
            s = (rng.integers(0, 5, nv) * 0.125).astype(np.float32)
        scores.append(s)
        video_cu.append(video_cu[-1] + nv)
        kt = nv * perm // 1000
        kts.append(kt)
        k1s.append(kt // 2)
        kept_cu.append(kept_cu[-1] + kt)
    dev = torch.from_numpy(np.concatenate(scores)).cuda()
    kept = specvlm.select(dev, video_cu, n_frames_list, T, k1s, kts, kept_cu).cpu().numpy()
    for b, F in enumerate(n_frames_list):
        ref = oracle.select(scores[b], F, T, k1s[b], kts[b])
        got = kept[kept_cu[b]:kept_cu[b + 1]]
        assert np.array_equal(got, ref), f"sequence {b}"


def test_select_cfg1_and_ties():
    _select_case([4], 196, 100, 0)
    _select_case([4], 196, 100, 1, ties=True)


@pytest.mark.parametrize("F,T,perm", [(32, 196, 100), (32, 720, 100), (256, 196, 50), (256, 196, 100),
                                      (256, 196, 200), (256, 196, 500), (1, 7, 500), (3, 5, 1000), (2, 9, 0)])
def test_select_workload_sizes(F, T, perm):
    _select_case([F], T, perm, 2)


def test_select_ragged_batch_and_ties():
    _select_case([32, 128, 64, 96, 32], 196, 100, 3)
    _select_case([32, 128, 64], 196, 100, 4, ties=True)


def test_select_stage_split_extremes():
    # k1 = 0 (Stage II only), k1 = k_total (Stage I only)
    rng = np.random.default_rng(5)
    s = rng.random(4 * 196).astype(np.float32)
    dev = torch.from_numpy(s).cuda()
    for k1, kt in [(0, 78), (78, 78), (1, 784), (784, 784), (0, 0)]:
        got = specvlm.select(dev, [0, 784], [4], 196, [k1], [kt], [0, kt]).cpu().numpy()[:kt]
        assert np.array_equal(got, oracle.select(s, 4, 196, k1, kt))


def _long_tailed(rng, n):
    a = rng.pareto(1.5, size=n).astype(np.float64)
    return (a / a.sum()).astype(np.float32)


@pytest.mark.parametrize("lam", [0, 400, 500, 900, 1000])
def test_select_top_p_bit_exact(lam):
    """Eq. 6 as a mode of the selection: Stage-I counts and kept sets equal the oracle's, on
    long-tailed scores, on scores full of ties, and on a ragged batch with per-sequence lambda."""
    rng = np.random.default_rng(40 + lam)
    frames, T = [32, 4, 128, 1], 196
    scores, video_cu, kts, kept_cu = [], [0], [], [0]
    for i, F in enumerate(frames):
        nv = F * T
        s = _long_tailed(rng, nv) if i != 1 else (rng.integers(0, 4, nv) * 0.0078125).astype(np.float32)
        scores.append(s)
        video_cu.append(video_cu[-1] + nv)
        kts.append(nv // 10 if i != 3 else nv)          # last sequence: budget = everything
        kept_cu.append(kept_cu[-1] + kts[-1])
    lams = [lam, lam, max(lam - 100, 0), lam]
    dev = torch.from_numpy(np.concatenate(scores)).cuda()
    kept, k1 = specvlm.select_top_p(dev, video_cu, frames, T, lams, kts, kept_cu)
    kept, k1 = kept.cpu().numpy(), k1.cpu().numpy()
    for b, F in enumerate(frames):
        ref, ref_k1 = oracle.select_top_p(scores[b], F, T, lams[b], kts[b])
        assert int(k1[b]) == ref_k1, f"sequence {b}: Stage-I count {int(k1[b])} vs {ref_k1}"
        assert np.array_equal(kept[kept_cu[b]:kept_cu[b + 1]], ref), f"sequence {b}"


def test_select_top_p_on_rated_scores_cfg1():
    """Top-P on real ratings of the tiny workload: the oracle's fp32 scores through both sides."""
    from gpu_util import make_cache, host_view
    w = synth.workload(1)
    nv, nt = w.n_video(), w.n_text[0]
    cache, _, _ = make_cache(w.t_layers, w.t_kv_heads, w.head_dim, [nv + nt], paged=False, seed=0)
    q = synth.randn_bf16((w.t_layers, nt, w.t_q_heads, w.head_dim), "cuda", 0, "Qtext")
    synth.plant_salient_(cache.k[:, 0, :, :nv, :], q, synth.salient_set(nv, w.planted_permille, 0))
    k_host = host_view(cache.k, None, [nv + nt])
    a = oracle.stage1_scores(bits(q), k_host[0], 0, nv, nv, 1.0 / math.sqrt(w.head_dim)).astype(np.float32)
    for lam in (400, 500):
        kept, k1 = specvlm.select_top_p(torch.from_numpy(a).cuda(), [0, nv], [w.n_frames[0]], w.tokens_per_frame,
                                        [lam], [nv // 2], [0, nv // 2])
        ref, ref_k1 = oracle.select_top_p(a, w.n_frames[0], w.tokens_per_frame, lam, nv // 2)
        assert int(k1[0]) == ref_k1 and np.array_equal(kept.cpu().numpy(), ref)


@pytest.mark.parametrize("mode", [0, 1, 2, 3, 4])
def test_select_baselines_bit_exact(mode):
    """Window / frame-dropping / random (Philox) selectors equal the oracle's index lists."""
    frames, T = [32, 5, 256, 1], 196
    kts = [627, 400, 2508, 196]
    kept_cu = [0]
    for k in kts:
        kept_cu.append(kept_cu[-1] + k)
    kept, kept_n = specvlm.select_baseline(mode, frames, T, kts, kept_cu, seed=0x1234567890ABCDEF)
    kept, kept_n = kept.cpu().numpy(), kept_n.cpu().numpy()
    for b, F in enumerate(frames):
        ref = oracle.select_baseline(mode, F, T, kts[b], seed=0x1234567890ABCDEF, b=b)
        assert int(kept_n[b]) == len(ref), f"sequence {b}"
        assert np.array_equal(kept[kept_cu[b]:kept_cu[b] + len(ref)], ref), f"sequence {b}"


# ------------------------------------------------------------------------------- gather
@pytest.mark.parametrize("src_paged,dst_paged", [(False, False), (True, True), (True, False)])
def test_gather_bit_exact(src_paged, dst_paged):
    from gpu_util import make_cache, host_view
    L, H, D = 3, 4, 128
    video_start, video_len = [0, 5, 0], [784, 392, 196]
    src_len = [784 + 64, 5 + 392 + 70, 196 + 1]
    rng = np.random.default_rng(6)
    kept, kept_cu = [], [0]
    for nv in video_len:
        kk = np.sort(rng.choice(nv, nv // 10, replace=False)).astype(np.int32)
        kept.append(kk)
        kept_cu.append(kept_cu[-1] + len(kk))
    dst_len = [s - v + len(k) for s, v, k in zip(src_len, video_len, kept)]
    src, sk, sv = make_cache(L, H, D, src_len, paged=src_paged, seed=13)
    dst, _, _ = make_cache(L, H, D, dst_len, paged=dst_paged, seed=14)
    kept_dev = torch.from_numpy(np.concatenate(kept)).cuda()
    specvlm.gather_kv(src, kept_dev, kept_cu, video_start, video_len, src_len, dst)
    torch.cuda.synchronize()
    dk = host_view(dst.k, dst.block_table, dst_len)
    dv = host_view(dst.v, dst.block_table, dst_len)
    for b in range(3):
        rk = oracle.gather_kv(sk[b], kept[b], video_start[b], video_len[b], src_len[b])
        rv = oracle.gather_kv(sv[b], kept[b], video_start[b], video_len[b], src_len[b])
        assert np.array_equal(dk[b], rk) and np.array_equal(dv[b], rv)


# ------------------------------------------------------------------------------- scores
def _scores_case(L, Hq, Hkv, D, n_frames, T, n_text, *, paged, seed, prefix=None, planted=50, scale_mul=1.0):
    from gpu_util import make_cache
    B = len(n_frames)
    prefix = prefix or [0] * B
    nv = [f * T for f in n_frames]
    seq_lens = [p + v + t for p, v, t in zip(prefix, nv, n_text)]
    cache, k_host, _ = make_cache(L, Hkv, D, seq_lens, paged=paged, seed=seed)
    text_cu = [0]
    for t in n_text:
        text_cu.append(text_cu[-1] + t)
    video_cu = [0]
    for v in nv:
        video_cu.append(video_cu[-1] + v)
    q = synth.randn_bf16((L, text_cu[-1], Hq, D), "cuda", seed, "Qtext")
    # plant salient keys (contiguous caches only: a view of the video rows is needed)
    if not paged and planted:
        for b in range(B):
            sal = synth.salient_set(nv[b], planted, seed, b)
            kview = cache.k[:, b, :, prefix[b]:prefix[b] + nv[b], :]
            synth.plant_salient_(kview, q[:, text_cu[b]:text_cu[b + 1]], sal)
        from gpu_util import host_view
        k_host = host_view(cache.k, None, seq_lens)
    scale = scale_mul / math.sqrt(D)
    text_start = [p + v for p, v in zip(prefix, nv)]
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    got = specvlm.stage1_scores(cache, q, text_cu, text_start, prefix, nv, video_cu, scale, d_status=status)
    got2 = specvlm.stage1_scores(cache, q, text_cu, text_start, prefix, nv, video_cu, scale)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    assert torch.equal(got, got2)                      # fixed reduction order
    got = got.cpu().numpy().astype(np.float64)
    qh = bits(q)
    worst = 0.0
    for b in range(B):
        ref = oracle.stage1_scores(qh[:, text_cu[b]:text_cu[b + 1]], k_host[b], prefix[b], nv[b],
                                   text_start[b], scale)
        g = got[video_cu[b]:video_cu[b + 1]]
        rel = np.abs(g - ref) / np.maximum(ref, 1e-30)     # scores below fp32's range compare absolutely
        worst = max(worst, float(rel.max()))
    assert worst <= SCORE_TOL, f"scores rel err {worst}"
    return got


def test_scores_cfg1():
    got = _scores_case(1, 8, 2, 64, [4], 196, [64], paged=False, seed=0)
    assert (got >= 0).all() and got.sum() <= 1.0


@pytest.mark.parametrize("Hq,Hkv,D", [(64, 8, 128), (40, 8, 128), (28, 4, 128), (8, 8, 64), (16, 1, 128)])
def test_scores_group_sizes(Hq, Hkv, D):
    _scores_case(2, Hq, Hkv, D, [3], 100, [37], paged=False, seed=1)
    _scores_case(1, Hq, Hkv, D, [2], 77, [130], paged=True, seed=2, prefix=[9])


def test_scores_sharp_softmax():
    """Logits 12 times wider than usual: the smallest exponentials of a row lie more than 2^125 below
    its maximum, where the polynomial exponential saturates and the special-function one flushes to
    zero; neither may disturb a row's sum or a column's score."""
    got = _scores_case(2, 16, 4, 128, [3], 100, [37], paged=False, seed=7, scale_mul=12.0)
    assert np.isfinite(got).all() and (got >= 0).all() and got.sum() <= 1.0 + 1e-6
    _scores_case(1, 8, 8, 64, [2], 130, [5], paged=True, seed=8, scale_mul=12.0)


def test_scores_by_layer_ranges_equal_one_call():
    """Rating the layers in ranges (uneven ones, an empty one, the reduction on its own) gives the
    bits of the single call: each layer's sums land in the workspace, the last call adds them in
    layer order."""
    from gpu_util import make_cache
    L, Hq, Hkv, D, nv, nt, prefix = 5, 40, 8, 128, 300, 37, 3
    cache, _, _ = make_cache(L, Hkv, D, [prefix + nv + nt], paged=True, seed=20)
    q = synth.randn_bf16((L, nt, Hq, D), "cuda", 20, "Qtext")
    args = ([0, nt], [prefix + nv], [prefix], [nv], [0, nv], 1.0 / math.sqrt(D))
    whole = specvlm.stage1_scores(cache, q, *args)
    for cuts in ([0, 2, 2, 3, 5], [0, 5], [0, 1, 2, 3, 4, 5]):
        ws = torch.full((specvlm.stage1_scores_workspace_bytes(cache, [0, nt], [nv], Hq),), 0xFF, dtype=torch.uint8,
                        device="cuda")
        out = torch.full((nv,), float("nan"), device="cuda")
        for a, b in zip(cuts[:-1], cuts[1:]):
            specvlm.stage1_scores_layers(cache, q, *args, out, ws, a, b, finish=False)
        specvlm.stage1_scores_layers(cache, q, *args, out, ws, L, L, finish=True)
        torch.cuda.synchronize()
        assert torch.equal(out, whole), cuts
    # the last range may finish by itself
    ws = torch.zeros((specvlm.stage1_scores_workspace_bytes(cache, [0, nt], [nv], Hq),), dtype=torch.uint8, device="cuda")
    out = torch.empty((nv,), device="cuda")
    specvlm.stage1_scores_layers(cache, q, *args, out, ws, 0, 3, finish=False)
    specvlm.stage1_scores_layers(cache, q, *args, out, ws, 3, 5, finish=True)
    torch.cuda.synchronize()
    assert torch.equal(out, whole)
    with pytest.raises(specvlm.SpecvlmError):
        specvlm.stage1_scores_layers(cache, q, *args, out, ws, 4, 6, finish=False)


def test_scores_ragged_batch():
    _scores_case(2, 16, 4, 128, [2, 5, 1], 64, [64, 17, 200], paged=True, seed=3)
    _scores_case(2, 16, 4, 128, [2, 5, 1], 50, [64, 17, 200], paged=False, seed=4, prefix=[0, 3, 70])


def test_pipeline_cfg1_end_to_end():
    """scores -> select -> gather -> decode on the tiny config; selection compared on oracle scores
    (bit-exact) and on GPU scores (overlap reported through the assertion message only)."""
    from gpu_util import make_cache, host_view
    w = synth.workload(1)
    nv, nt = w.n_video(), w.n_text[0]
    cache, k_host, v_host = make_cache(w.t_layers, w.t_kv_heads, w.head_dim, [nv + nt], paged=False, seed=0)
    q = synth.randn_bf16((w.t_layers, nt, w.t_q_heads, w.head_dim), "cuda", 0, "Qtext")
    sal = synth.salient_set(nv, w.planted_permille, 0)
    synth.plant_salient_(cache.k[:, 0, :, :nv, :], q, sal)
    k_host = host_view(cache.k, None, [nv + nt])
    scale = 1.0 / math.sqrt(w.head_dim)
    a_gpu = specvlm.stage1_scores(cache, q, [0, nt], [nv], [0], [nv], [0, nv], scale)
    a_ref = oracle.stage1_scores(bits(q), k_host[0], 0, nv, nv, scale)
    a_ref32 = a_ref.astype(np.float32)
    kt, k1 = w.k_total(), w.k_stage1()
    kept_ref = oracle.select(a_ref32, w.n_frames[0], w.tokens_per_frame, k1, kt)
    kept_on_ref = specvlm.select(torch.from_numpy(a_ref32).cuda(), [0, nv], [w.n_frames[0]],
                                 w.tokens_per_frame, [k1], [kt], [0, kt]).cpu().numpy()
    assert np.array_equal(kept_on_ref, kept_ref)
    kept_gpu = specvlm.select(a_gpu, [0, nv], [w.n_frames[0]], w.tokens_per_frame, [k1], [kt],
                              [0, kt]).cpu().numpy()
    inter = len(set(kept_gpu.tolist()) & set(kept_ref.tolist()))
    assert inter >= 0.9 * kt, f"GPU-score selection overlaps the oracle's in {inter}/{kt}"
    # planted tokens should be over-represented in Stage I (sanity statistic, not a gate)
    assert len(kept_ref) == kt


def test_scores_row_lse_entry():
    from gpu_util import make_cache
    L, Hq, Hkv, D, nv, nt = 2, 28, 4, 128, 200, 45
    cache, k_host, _ = make_cache(L, Hkv, D, [nv + nt], paged=True, seed=21)
    q = synth.randn_bf16((L, nt, Hq, D), "cuda", 21, "Qtext")
    scale = 1.0 / math.sqrt(D)
    lse = specvlm.stage1_row_lse(cache, q, [0, nt], [nv], scale)
    _, _, ref_lse = oracle.stage1_scores(bits(q), k_host[0], 0, nv, nv, scale, want_rows=True)
    np.testing.assert_allclose(lse.cpu().numpy(), ref_lse.transpose(0, 2, 1), rtol=0, atol=1e-4)
    a = specvlm.stage1_scores(cache, q, [0, nt], [nv], [0], [nv], [0, nv], scale)
    b = specvlm.stage1_scores(cache, q, [0, nt], [nv], [0], [nv], [0, nv], scale, row_lse=lse)
    assert torch.equal(a, b)


# ------------------------------------------------------------------------------- rising maxima
@pytest.mark.parametrize("Hq,Hkv,gamma,D", [(64, 8, 8, 128),    # 72 rows: the 128-row tiles
                                            (64, 8, 5, 128),    # 48 rows: the 64-row tiles
                                            (28, 4, 0, 128),    # 7 rows: the decode kernel
                                            (16, 2, 8, 64)])    # 72 rows, d = 64
def test_attention_with_maxima_rising_along_the_sequence(Hq, Hkv, gamma, D):
    """Random N(0,1) logits never move a row's running maximum by much after the first tile, so the
    kernels' rescaling of the running sums and of the O accumulator would go untested.  Here the
    keys carry a ramp along a direction u and the query rows carry +a u, +a u / 2, 0 or -a u: the
    logits of a row rise (or fall) by about 12 log2 units per 128 tokens, with a drop half way, so
    that the reference maximum must be raised again and again for some rows of a warp and never
    for others."""
    from gpu_util import make_cache
    L, n = 2, 1500 + gamma + 1
    cache, _, _ = make_cache(L, Hkv, D, [n, 700], paged=False, seed=90)
    g = torch.Generator(device="cuda").manual_seed(91)
    u = torch.randn(D, generator=g, device="cuda")
    u = u / u.norm()
    scale = 1.0 / math.sqrt(D)
    a = 10.0
    b = 12.0 / (scale * a * math.log2(math.e))                    # ramp height per 128 tokens
    pos = torch.arange(cache.k.shape[3], device="cuda", dtype=torch.float32)
    ramp = torch.where(pos < 800, pos, pos - 640.0) / 128.0       # rises, drops by 5 tiles' worth, rises again
    cache.k.copy_((cache.k.float() + (b * ramp)[None, None, None, :, None] * u).to(torch.bfloat16))
    nq = gamma + 1
    q = synth.randn_bf16((L, 2, nq, Hq, D), "cuda", 92, "Q").float()
    slope = torch.tensor([1.0, 0.5, 0.0, -1.0], device="cuda")[torch.arange(Hq, device="cuda") % 4]
    q = (q + a * slope[None, None, None, :, None] * u).to(torch.bfloat16)
    from gpu_util import host_view
    k_host = host_view(cache.k, None, [n, 700])
    v_host = host_view(cache.v, None, [n, 700])
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    lse = torch.empty((L, 2, nq, Hq), dtype=torch.float32, device="cuda")
    if gamma == 0:
        out = specvlm.draft_decode_attn(cache, q[:, :, 0].contiguous(), scale, lse=lse, d_status=status)[:, :, None]
    else:
        out = specvlm.verify_attn(cache, q, gamma, scale, lse=lse, d_status=status)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    ref, ref_lse = _oracle_attn(bits(q), k_host, v_host, [n, 700], scale)
    got = f64(out)
    assert np.isfinite(got).all()
    err = row_rel_err(got, ref)
    assert err <= ATTN_TOL, f"row rel err {err}"
    np.testing.assert_allclose(lse.cpu().numpy(), ref_lse, rtol=0, atol=2e-3 + 1e-4 * np.abs(ref_lse).max())
