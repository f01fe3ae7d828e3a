"""Parity at the benchmark's full sizes, through the C ABI, in the launch configuration bench.py
times.  The CUDA side runs the whole workload; the fp64 oracle is run on sampled layers (each layer
is an independent problem for every call on the path), on the very same tensors copied to the host.

Workloads 3-5 keep their per-layer shapes (tokens, heads, rows, paging) and run a stated subset of
layers, since a layer count only repeats the same problem."""
import math

import numpy as np
import pytest
import torch

import oracle
from helpers import bits, f64, row_rel_err
from paper_2508_16201_b200 import specvlm, synth

pytestmark = pytest.mark.gpu

ATTN_TOL = 1e-2
SCORE_TOL = 1e-4


def _contig_cache(L, Hkv, n, D, seed, tag):
    k = synth.randn_bf16((L, 1, Hkv, n, D), "cuda", seed, tag + "K")
    v = synth.randn_bf16((L, 1, Hkv, n, D), "cuda", seed, tag + "V")
    lens = torch.tensor([n], dtype=torch.int32, device="cuda")
    return specvlm.KvCache(k, v, lens, n), k, v


def _check_layers(out, lse, q, k, v, n, scale, layers):
    """oracle attention on the sampled layers of a batch-1 contiguous cache"""
    worst = 0.0
    for l in layers:
        ref, ref_lse = oracle.attention(bits(q[l, 0]), bits(k[l, 0]), bits(v[l, 0]), n, scale)
        got = f64(out[l, 0])
        assert np.isfinite(got).all()
        worst = max(worst, row_rel_err(got, ref))
        np.testing.assert_allclose(lse[l, 0].cpu().numpy(), ref_lse, rtol=0, atol=2e-3)
    assert worst <= ATTN_TOL, f"row rel err {worst}"


def _verify_full(i, layers_run, sample, seed):
    w = synth.workload(i)
    D, g1 = w.head_dim, w.gamma + 1
    n = w.seq_len() + g1                         # the cache already holds the gamma+1 new tokens
    cache, k, v = _contig_cache(layers_run, w.t_kv_heads, n, D, seed, "t")
    q = synth.randn_bf16((layers_run, 1, g1, w.t_q_heads, D), "cuda", seed, "Qv")
    scale = 1.0 / math.sqrt(D)
    lse = torch.empty((layers_run, 1, g1, w.t_q_heads), dtype=torch.float32, device="cuda")
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    out = specvlm.verify_attn(cache, q, w.gamma, scale, lse=lse, d_status=status)
    out2 = specvlm.verify_attn(cache, q, w.gamma, scale)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    assert torch.equal(out, out2)                # the merge order of cut items is fixed
    _check_layers(out, lse, q, k, v, n, scale, sample)


def test_verify_cfg2_all_80_layers_sampled():
    _verify_full(2, 80, [0, 41, 79], seed=100)


def test_verify_cfg3_all_64_layers_sampled():
    _verify_full(3, 64, [0, 63], seed=101)       # 40 q / 8 kv heads: 30 rows, 23302 tokens


def test_verify_cfg4_8_of_80_layers_sampled():
    _verify_full(4, 8, [7], seed=102)            # 50311 tokens, gamma 6: 56 rows


@pytest.mark.parametrize("pruned", [True, False])
def test_decode_cfg2_all_28_layers(pruned):
    w = synth.workload(2)
    D = w.head_dim
    n = (w.k_total() + w.n_text[0]) if pruned else w.seq_len()
    cache, k, v = _contig_cache(w.d_layers, w.d_kv_heads, n, D, 103, "d")
    q = synth.randn_bf16((w.d_layers, 1, 1, w.d_q_heads, D), "cuda", 103, "Qd")
    scale = 1.0 / math.sqrt(D)
    lse = torch.empty((w.d_layers, 1, w.d_q_heads), dtype=torch.float32, device="cuda")
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    out = specvlm.draft_decode_attn(cache, q[:, :, 0].contiguous(), scale, lse=lse, d_status=status)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    layers = range(w.d_layers) if pruned else [0, 13, 27]
    _check_layers(out[:, :, None], lse[:, :, None], q, k, v, n, scale, layers)


@pytest.mark.parametrize("gamma", [3, 8])
def test_cfg5_batched_paged_verify_and_decode(gamma):
    """Workload 5: 16 ragged sequences, 64-token pages scattered over the pool; 2 of 80 verifier
    layers and 2 of 28 draft layers.  gamma 3 gives 32 rows per KV head, gamma 8 gives 72."""
    from gpu_util import make_cache
    w = synth.workload(5, gamma=gamma)
    D, g1, B, L = w.head_dim, gamma + 1, w.batch, 2
    scale = 1.0 / math.sqrt(D)
    # verification over the full target cache
    lens = [w.seq_len(b) + g1 for b in range(B)]
    cache, k_host, v_host = make_cache(L, w.t_kv_heads, D, lens, paged=True, seed=110 + gamma)
    q = synth.randn_bf16((L, B, g1, w.t_q_heads, D), "cuda", 110 + gamma, "Qv")
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    out = specvlm.verify_attn(cache, q, gamma, scale, d_status=status)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    qh, got = bits(q), f64(out)
    assert np.isfinite(got).all()
    worst = 0.0
    for b in range(B):
        ref, _ = oracle.attention(qh[1, b], k_host[b][1], v_host[b][1], lens[b], scale)
        worst = max(worst, row_rel_err(got[1, b], ref))
    assert worst <= ATTN_TOL, f"verify row rel err {worst}"
    del cache, k_host, v_host
    # draft decode over the pruned caches (10 % of the video tokens + the text)
    plens = [w.k_total(b) + w.n_text[b] for b in range(B)]
    dcache, dk, dv = make_cache(L, w.d_kv_heads, D, plens, paged=True, seed=120 + gamma)
    qd = synth.randn_bf16((L, B, 1, w.d_q_heads, D), "cuda", 120 + gamma, "Qd")
    od = specvlm.draft_decode_attn(dcache, qd[:, :, 0].contiguous(), scale, d_status=status)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    qh, got = bits(qd), f64(od)
    worst = 0.0
    for l in range(L):
        for b in range(B):
            ref, _ = oracle.attention(qh[l, b], dk[b][l], dv[b][l], plens[b], scale)
            worst = max(worst, row_rel_err(got[l, b][None], ref))
    assert worst <= ATTN_TOL, f"decode row rel err {worst}"


def test_scores_cfg2_80_layer_call_against_the_oracle():
    """Token rating at workload 2's size, one call over all 80 layers.  The call leaves every layer's
    column sums in its workspace: four sampled layers of THAT output are compared with the oracle's
    rating of the same layer, element by element; the final scores must be the ordered sum of the
    80 layers' sums divided by the number of (layer, head, query) rows, which ties the remaining
    layers' contribution to the identity Eq. 5's average obeys at any size."""
    w = synth.workload(2)
    D, nv, nt, L = w.head_dim, w.n_video(), w.n_text[0], w.t_layers
    scale = 1.0 / math.sqrt(D)
    k = synth.randn_bf16((L, 1, w.t_kv_heads, nv + nt, D), "cuda", 130, "tK")
    q = synth.randn_bf16((L, nt, w.t_q_heads, D), "cuda", 130, "Qtext")
    synth.plant_salient_(k[:, 0, :, :nv, :], q, synth.salient_set(nv, w.planted_permille, 130))
    lens = torch.tensor([nv + nt], dtype=torch.int32, device="cuda")
    cache = specvlm.KvCache(k, k, lens, nv + nt)
    args = ([0, nt], [nv], [0], [nv], [0, nv], scale)
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    ws = torch.full((specvlm.stage1_scores_workspace_bytes(cache, [0, nt], [nv], w.t_q_heads),), 0xFF,
                    dtype=torch.uint8, device="cuda")
    full = specvlm.stage1_scores(cache, q, *args, ws=ws, d_status=status)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    off = specvlm.stage1_scores_layer_sums_offset(cache, [0, nt], w.t_q_heads)
    sums = ws[off:off + L * nv * 4].view(torch.float32).view(L, nv).cpu().numpy().astype(np.float64)
    rows = w.t_q_heads * nt
    for l in (3, 29, 52, 77):
        ref = oracle.stage1_scores(bits(q[l:l + 1]), bits(k[l:l + 1, 0]), 0, nv, nv, scale)
        rel = float((np.abs(sums[l] / rows - ref) / ref).max())
        assert rel <= SCORE_TOL, f"layer {l} of the 80-layer call: scores rel err {rel}"
    got = full.cpu().numpy().astype(np.float64)
    mean = sums.sum(axis=0) / (L * rows)
    assert float((np.abs(got - mean) / mean).max()) <= 1e-5
    assert float(got.sum()) <= 1.0 and float(got.min()) >= 0.0


def test_gather_cfg2_all_28_layers():
    w = synth.workload(2)
    D, nv, nt, L, H = w.head_dim, w.n_video(), w.n_text[0], w.d_layers, w.d_kv_heads
    kt = w.k_total()
    src, sk, sv = _contig_cache(L, H, nv + nt, D, 140, "src")
    dst, dk, dv = _contig_cache(L, H, kt + nt, D, 141, "dst")
    g = torch.Generator().manual_seed(140)
    kept = torch.sort(torch.randperm(nv, generator=g)[:kt]).values.to(torch.int32)
    specvlm.gather_kv(src, kept.cuda(), [0, kt], [0], [nv], [nv + nt], dst)
    torch.cuda.synchronize()
    kept_np = kept.numpy()
    for name, s_t, d_t in (("K", sk, dk), ("V", sv, dv)):
        ref = oracle.gather_kv(bits(s_t[:, 0]), kept_np, 0, nv, nv + nt)
        assert np.array_equal(bits(d_t[:, 0]), ref), name


def test_scores_cfg3_shapes_sampled_layer():
    """Token rating at workload 3's per-layer size (5 query heads per KV head: 25 queries x 5 heads
    fill 125 of a tile's 128 rows; 23 040 video + 256 text tokens), 3 of 64 layers, one of them
    rated by the oracle."""
    w = synth.workload(3)
    D, nv, nt, L = w.head_dim, w.n_video(), w.n_text[0], 3
    scale = 1.0 / math.sqrt(D)
    k = synth.randn_bf16((L, 1, w.t_kv_heads, nv + nt, D), "cuda", 131, "tK")
    q = synth.randn_bf16((L, nt, w.t_q_heads, D), "cuda", 131, "Qtext")
    synth.plant_salient_(k[:, 0, :, :nv, :], q, synth.salient_set(nv, w.planted_permille, 131))
    lens = torch.tensor([nv + nt], dtype=torch.int32, device="cuda")
    args = ([0, nt], [nv], [0], [nv], [0, nv], scale)
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    full = specvlm.stage1_scores(specvlm.KvCache(k, k, lens, nv + nt), q, *args, d_status=status).double()
    one = specvlm.stage1_scores(specvlm.KvCache(k[1:2], k[1:2], lens, nv + nt), q[1:2], *args, d_status=status)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    ref = oracle.stage1_scores(bits(q[1:2]), bits(k[1:2, 0]), 0, nv, nv, scale)
    got = one.cpu().numpy().astype(np.float64)
    rel = float((np.abs(got - ref) / ref).max())
    assert rel <= SCORE_TOL, f"scores rel err {rel}"
    assert np.isfinite(full.cpu().numpy()).all() and float(full.sum()) <= 1.0 and float(full.min()) >= 0.0


# ------------------------------------------------------------------------------------------------
# Workloads 3-5 at their own per-layer sizes, every remaining call of the path.
# ------------------------------------------------------------------------------------------------
def test_scores_cfg4_shape_2_layers_one_by_the_oracle():
    """Token rating at workload 4's per-layer size: 50 176 video + 128 text tokens, 64 query / 8 KV
    heads (392 key blocks per layer, 3 % planted tokens); 2 of 80 layers run, one rated by the oracle."""
    w = synth.workload(4)
    D, nv, nt, L = w.head_dim, w.n_video(), w.n_text[0], 2
    scale = 1.0 / math.sqrt(D)
    k = synth.randn_bf16((L, 1, w.t_kv_heads, nv + nt, D), "cuda", 132, "tK")
    q = synth.randn_bf16((L, nt, w.t_q_heads, D), "cuda", 132, "Qtext")
    synth.plant_salient_(k[:, 0, :, :nv, :], q, synth.salient_set(nv, w.planted_permille, 132))
    lens = torch.tensor([nv + nt], dtype=torch.int32, device="cuda")
    args = ([0, nt], [nv], [0], [nv], [0, nv], scale)
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    both = specvlm.stage1_scores(specvlm.KvCache(k, k, lens, nv + nt), q, *args, d_status=status).double()
    one = specvlm.stage1_scores(specvlm.KvCache(k[1:2], k[1:2], lens, nv + nt), q[1:2], *args, d_status=status)
    zero = specvlm.stage1_scores(specvlm.KvCache(k[0:1], k[0:1], lens, nv + nt), q[0:1], *args, d_status=status)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    ref = oracle.stage1_scores(bits(q[1:2]), bits(k[1:2, 0]), 0, nv, nv, scale)
    got = one.cpu().numpy().astype(np.float64)
    rel = float((np.abs(got - ref) / ref).max())
    assert rel <= SCORE_TOL, f"scores rel err {rel}"
    mean = (one.double() + zero.double()) / 2
    assert float(((both - mean).abs() / mean).max()) <= 1e-5
    assert float(both.sum()) <= 1.0 and float(both.min()) >= 0.0


def test_scores_cfg5_ragged_paged_batch_of_16():
    """Token rating on workload 5: 16 sequences of 32-128 frames and 64-227 language queries in
    64-token pages scattered over the pool, one call for the batch; 2 of 80 layers run, the oracle
    rates layer 1 of every sequence."""
    from gpu_util import make_cache
    w = synth.workload(5)
    D, B, L = w.head_dim, w.batch, 2
    scale = 1.0 / math.sqrt(D)
    nv = [w.n_video(b) for b in range(B)]
    lens = [w.seq_len(b) for b in range(B)]
    cache, _, _ = make_cache(L, w.t_kv_heads, D, lens, paged=True, seed=133)
    text_cu, video_cu = [0], [0]
    for b in range(B):
        text_cu.append(text_cu[-1] + w.n_text[b])
        video_cu.append(video_cu[-1] + nv[b])
    q = synth.randn_bf16((L, text_cu[-1], w.t_q_heads, D), "cuda", 133, "Qtext")
    for b in range(B):
        synth.plant_salient_paged_(cache.k, cache.block_table[b], 0, nv[b], q[:, text_cu[b]:text_cu[b + 1]],
                                   synth.salient_set(nv[b], w.planted_permille, 133, b))
    from gpu_util import host_view
    k_host = host_view(cache.k[1:2], cache.block_table, lens)
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    both = specvlm.stage1_scores(cache, q, text_cu, nv, [0] * B, nv, video_cu, scale, d_status=status)
    c1 = specvlm.KvCache(cache.k[1:2], cache.v[1:2], cache.seq_lens, cache.max_seq_len, cache.block_table)
    one = specvlm.stage1_scores(c1, q[1:2], text_cu, nv, [0] * B, nv, video_cu, scale, d_status=status)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    got = one.cpu().numpy().astype(np.float64)
    qh = bits(q[1:2])
    worst = 0.0
    for b in range(B):
        ref = oracle.stage1_scores(qh[:, text_cu[b]:text_cu[b + 1]], k_host[b], 0, nv[b], nv[b], scale)
        g = got[video_cu[b]:video_cu[b + 1]]
        worst = max(worst, float((np.abs(g - ref) / ref).max()))
        assert g.sum() <= 1.0
    assert worst <= SCORE_TOL, f"scores rel err {worst}"
    assert np.isfinite(both.cpu().numpy()).all() and float(both.min()) >= 0.0


def _gather_contig(i, retention_permille, layers, seed):
    w = synth.workload(i, retention_permille=retention_permille)
    D, nv, nt, H = w.head_dim, w.n_video(), w.n_text[0], w.d_kv_heads
    kt = w.k_total()
    src, sk, sv = _contig_cache(layers, H, nv + nt, D, seed, "src")
    dst, dk, dv = _contig_cache(layers, H, kt + nt, D, seed + 1, "dst")
    g = torch.Generator().manual_seed(seed)
    kept = torch.sort(torch.randperm(nv, generator=g)[:kt]).values.to(torch.int32)
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    specvlm.gather_kv(src, kept.cuda(), [0, kt], [0], [nv], [nv + nt], dst, d_status=status)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    kept_np = kept.numpy()
    for name, s_t, d_t in (("K", sk, dk), ("V", sv, dv)):
        ref = oracle.gather_kv(bits(s_t[:, 0]), kept_np, 0, nv, nv + nt)
        assert np.array_equal(bits(d_t[:, 0]), ref), name


def test_gather_cfg3_all_28_layers():
    _gather_contig(3, None, 28, 142)              # 23 040 video tokens -> 2304 kept + 256 text rows


def test_gather_cfg4_half_retention_8_of_28_layers():
    _gather_contig(4, 500, 8, 144)                # 50 176 video tokens -> 25 088 kept + 128 text rows


def test_gather_cfg5_paged_to_paged():
    """Workload 5: the 16 sequences' kept rows go from the scattered pages of the full draft-shaped
    cache to the scattered pages of the pruned one; 2 of 28 layers, byte for byte."""
    from gpu_util import host_view, make_cache
    w = synth.workload(5)
    D, B, L, H = w.head_dim, w.batch, 2, w.d_kv_heads
    nv = [w.n_video(b) for b in range(B)]
    src_len = [w.seq_len(b) for b in range(B)]
    rng = np.random.default_rng(146)
    kept, kept_cu = [], [0]
    for b in range(B):
        kk = np.sort(rng.choice(nv[b], w.k_total(b), replace=False)).astype(np.int32)
        kept.append(kk)
        kept_cu.append(kept_cu[-1] + len(kk))
    dst_len = [w.k_total(b) + w.n_text[b] for b in range(B)]
    src, sk, sv = make_cache(L, H, D, src_len, paged=True, seed=146)
    dst, _, _ = make_cache(L, H, D, dst_len, paged=True, seed=147)
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    specvlm.gather_kv(src, torch.from_numpy(np.concatenate(kept)).cuda(), kept_cu, [0] * B, nv, src_len, dst,
                      d_status=status)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    dk = host_view(dst.k, dst.block_table, dst_len)
    dv = host_view(dst.v, dst.block_table, dst_len)
    for b in range(B):
        assert np.array_equal(dk[b], oracle.gather_kv(sk[b], kept[b], 0, nv[b], src_len[b]))
        assert np.array_equal(dv[b], oracle.gather_kv(sv[b], kept[b], 0, nv[b], src_len[b]))


@pytest.mark.parametrize("i,retention", [(3, 100), (4, 50), (4, 100), (4, 200), (4, 500)])
def test_decode_pruned_cfg3_and_cfg4_retention_sweep(i, retention):
    """Draft decode over the pruned caches of workloads 3 and 4: 2560 tokens (workload 3) and
    2636 / 5145 / 10 163 / 25 216 tokens (workload 4 at 5 / 10 / 20 / 50 % retention); all 28 draft
    layers run, two sampled by the oracle."""
    w = synth.workload(i, retention_permille=retention)
    D = w.head_dim
    n = w.k_total() + w.n_text[0]
    cache, k, v = _contig_cache(w.d_layers, w.d_kv_heads, n, D, 150 + retention // 10 + i, "d")
    q = synth.randn_bf16((w.d_layers, 1, 1, w.d_q_heads, D), "cuda", 150 + i, "Qd")
    scale = 1.0 / math.sqrt(D)
    lse = torch.empty((w.d_layers, 1, w.d_q_heads), dtype=torch.float32, device="cuda")
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    out = specvlm.draft_decode_attn(cache, q[:, :, 0].contiguous(), scale, lse=lse, d_status=status)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    _check_layers(out[:, :, None], lse[:, :, None], q, k, v, n, scale, [0, 27])
