"""Tree drafting on the GPU against the oracle: tree-masked verification attention (<= 1e-2 row
relative), tree acceptance (bit-exact) and cache compaction (bit-exact), on contiguous and paged
caches, including windows that straddle tile edges and a chained verify -> accept -> compact step."""
import math

import numpy as np
import pytest
import torch

import oracle
from gpu_util import host_view, make_cache
from helpers import bits, f64, row_rel_err
from paper_2508_16201_b200 import specvlm, synth

pytestmark = pytest.mark.gpu


def _random_tree(rng, n):
    return [-1] + [int(rng.integers(0, t)) for t in range(1, n)]


def _tree_case(L, Hq, Hkv, D, lens, n_nodes, *, paged, seed, chain=False):
    rng = np.random.default_rng(seed)
    B = len(lens)
    cache, k_host, v_host = make_cache(L, Hkv, D, lens, paged=paged, seed=seed, poison_tail=True)
    parents = [list(range(-1, n_nodes - 1)) if chain else _random_tree(rng, n_nodes) for _ in range(B)]
    par = torch.tensor(parents, dtype=torch.int32, device="cuda")
    q = synth.randn_bf16((L, B, n_nodes, Hq, D), "cuda", seed, "Qt")
    scale = 1.0 / math.sqrt(D)
    lse = torch.empty((L, B, n_nodes, Hq), dtype=torch.float32, device="cuda")
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    out = specvlm.verify_tree_attn(cache, q, par, scale, lse=lse, d_status=status)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    got, qh = f64(out), bits(q)
    assert np.isfinite(got).all()
    worst = 0.0
    for l in range(L):
        for b in range(B):
            ref, ref_lse = oracle.attention_tree(qh[l, b], k_host[b][l], v_host[b][l], lens[b], parents[b], scale)
            worst = max(worst, row_rel_err(got[l, b], ref))
            np.testing.assert_allclose(lse[l, b].cpu().numpy(), ref_lse, rtol=0, atol=2e-3)
    assert worst <= 1e-2, f"row rel err {worst}"
    return out, cache, q


@pytest.mark.parametrize("paged", [False, True])
@pytest.mark.parametrize("Hq,Hkv,n_nodes,D", [(64, 8, 16, 128),   # 128 rows: the M = 128 tiles
                                              (64, 8, 8, 128),    # 64 rows
                                              (40, 8, 25, 128),   # 125 rows, group 5
                                              (28, 4, 9, 128),    # 63 rows, group 7
                                              (8, 2, 32, 64),     # 32 nodes, d = 64
                                              (4, 4, 3, 64),      # 3 rows: below the decode kernel's limit
                                              (64, 8, 26, 128),   # 208 rows: two parts of 13 nodes
                                              (32, 2, 32, 128),   # 512 rows, group 16: four parts of 8 nodes
                                              (24, 4, 30, 64),    # 180 rows, group 6, d = 64: 15 + 15 nodes
                                              (40, 8, 51, 128),   # group 5 x 51 nodes = 255 rows: 25 tokens fill a part, so three parts of 17
                                              (30, 2, 17, 64),    # group 15 x 17 nodes = 255 rows: three parts of 6, 6 and 5 tokens
                                              (64, 8, 60, 128),   # 60 nodes (a dynamic draft tree's size): 480 rows, four parts of 15
                                              (28, 4, 64, 128),   # 64 nodes, the mask's width, group 7: 448 rows, four parts of 16
                                              (8, 8, 41, 64)])    # 41 rows of one head each: bits above 32 in a single 64-row part
def test_tree_attention(Hq, Hkv, n_nodes, D, paged):
    _tree_case(2, Hq, Hkv, D, [300 + n_nodes, 128 + 3, n_nodes, 64 + n_nodes // 2], n_nodes, paged=paged, seed=60)


def test_tree_with_chain_parents_equals_verify_attn():
    out, cache, q = _tree_case(1, 16, 4, 128, [200, 77], 6, paged=True, seed=61, chain=True)
    ref = specvlm.verify_attn(cache, q, 5, 1.0 / math.sqrt(128))
    torch.cuda.synchronize()
    assert torch.equal(out, ref)


def test_tree_bad_parents_are_reported():
    cache, _, _ = make_cache(1, 2, 64, [40], paged=False, seed=62)
    q = synth.randn_bf16((1, 1, 4, 4, 64), "cuda", 62, "Qt")
    par = torch.tensor([[-1, 2, 0, 1]], dtype=torch.int32, device="cuda")      # node 1's parent comes later
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    specvlm.verify_tree_attn(cache, q, par, 0.125, d_status=status)
    torch.cuda.synchronize()
    assert int(status.item()) == specvlm.ERR_INVALID_ARG


@pytest.mark.parametrize("batch,n_nodes,vocab", [(1, 26, 152064), (5, 9, 4099), (16, 32, 1000), (3, 64, 4099), (2, 47, 152064)])
def test_tree_accept_bit_exact(batch, n_nodes, vocab):
    rng = np.random.default_rng(63)
    logits = torch.randn((batch, n_nodes, vocab), generator=torch.Generator().manual_seed(63)).cuda()
    lg = logits.cpu().numpy()
    am = lg.argmax(2)
    parents, tokens = [], []
    for b in range(batch):
        par = _random_tree(rng, n_nodes)
        # each node's token: its parent's target arg-max with probability 0.6, else random
        tok = [0] + [int(am[b, par[t]]) if rng.random() < 0.6 else int(rng.integers(0, vocab)) for t in range(1, n_nodes)]
        parents.append(par)
        tokens.append(tok)
    par_d = torch.tensor(parents, dtype=torch.int32, device="cuda")
    tok_d = torch.tensor(tokens, dtype=torch.int32, device="cuda")
    n, nxt, path, g = specvlm.accept_tree(logits, tok_d, par_d, want_argmax=True)
    torch.cuda.synchronize()
    lens = set()
    for b in range(batch):
        rn, rnext, rpath = oracle.accept_tree(lg[b], tokens[b], parents[b])
        assert (int(n[b]), int(nxt[b])) == (rn, rnext)
        assert path[b].cpu().tolist() == rpath + [-1] * (n_nodes - rn)
        assert np.array_equal(g[b].cpu().numpy(), am[b])
        lens.add(rn)
    if batch >= 5:
        assert len(lens) > 1          # the cases really differ


@pytest.mark.parametrize("n_nodes", [12, 60])
@pytest.mark.parametrize("paged", [False, True])
def test_tree_step_chain_verify_accept_compact(paged, n_nodes):
    L, Hq, Hkv, D, vocab = 2, 16, 2, 128, 997
    rng = np.random.default_rng(64)
    lens = [150 + n_nodes, 64 + n_nodes, n_nodes]
    cache, k_host, v_host = make_cache(L, Hkv, D, lens, paged=paged, seed=64)
    parents = [_random_tree(rng, n_nodes) for _ in lens]
    logits = torch.randn((3, n_nodes, vocab), generator=torch.Generator().manual_seed(64)).cuda()
    am = logits.cpu().numpy().argmax(2)
    tokens = [[0] + [int(am[b, parents[b][t]]) if rng.random() < 0.7 else 1 for t in range(1, n_nodes)]
              for b in range(3)]
    par_d = torch.tensor(parents, dtype=torch.int32, device="cuda")
    tok_d = torch.tensor(tokens, dtype=torch.int32, device="cuda")
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    n, nxt, path, _ = specvlm.accept_tree(logits, tok_d, par_d)
    specvlm.compact_tree_kv(cache, path, n, d_status=status)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    new_lens = cache.seq_lens.cpu().tolist()
    gk = host_view(cache.k, cache.block_table, new_lens)
    gv = host_view(cache.v, cache.block_table, new_lens)
    for b in range(3):
        rn, _, rpath = oracle.accept_tree(logits[b].cpu().numpy(), tokens[b], parents[b])
        rk, nl = oracle.compact_tree_kv(k_host[b], lens[b], n_nodes, rpath)
        rv, _ = oracle.compact_tree_kv(v_host[b], lens[b], n_nodes, rpath)
        assert new_lens[b] == nl == lens[b] - n_nodes + 1 + rn
        assert np.array_equal(gk[b], rk[:, :, :nl]) and np.array_equal(gv[b], rv[:, :, :nl])


def test_tree_attention_with_maxima_rising_along_the_sequence():
    """The 128-row tree variant on logits that rise by about 12 log2 units per 128 tokens for some
    rows and fall for others: the reference maximum of a row has to be raised tile after tile."""
    L, Hq, Hkv, D, n_nodes = 2, 64, 8, 128, 16
    lens = [1400 + n_nodes, 300]
    rng = np.random.default_rng(95)
    cache, _, _ = make_cache(L, Hkv, D, lens, paged=False, seed=95)
    g = torch.Generator(device="cuda").manual_seed(96)
    u = torch.randn(D, generator=g, device="cuda")
    u = u / u.norm()
    scale = 1.0 / math.sqrt(D)
    a = 10.0
    b = 12.0 / (scale * a * math.log2(math.e))
    pos = torch.arange(cache.k.shape[3], device="cuda", dtype=torch.float32)
    cache.k.copy_((cache.k.float() + (b * pos / 128.0)[None, None, None, :, None] * u).to(torch.bfloat16))
    k_host = host_view(cache.k, None, lens)
    v_host = host_view(cache.v, None, lens)
    parents = [_random_tree(rng, n_nodes) for _ in lens]
    par = torch.tensor(parents, dtype=torch.int32, device="cuda")
    q = synth.randn_bf16((L, 2, n_nodes, Hq, D), "cuda", 97, "Qt").float()
    slope = torch.tensor([1.0, -1.0, 0.5, 0.0], device="cuda")[torch.arange(Hq, device="cuda") % 4]
    q = (q + a * slope[None, None, None, :, None] * u).to(torch.bfloat16)
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    out = specvlm.verify_tree_attn(cache, q, par, scale, d_status=status)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    got, qh = f64(out), bits(q)
    assert np.isfinite(got).all()
    worst = 0.0
    for l in range(L):
        for bb in range(2):
            ref, _ = oracle.attention_tree(qh[l, bb], k_host[bb][l], v_host[bb][l], lens[bb], parents[bb], scale)
            worst = max(worst, row_rel_err(got[l, bb], ref))
    assert worst <= 1e-2, f"row rel err {worst}"
