"""Cache maintenance (append the new tokens' K/V, drop rejected drafts) against the oracle, bit for
bit, on contiguous and paged caches; and one full speculative step chained on the device: append
-> verify -> accept -> rollback, with the attention read from the appended cache."""
import math

import numpy as np
import pytest
import torch

import oracle
from gpu_util import host_view, make_cache
from helpers import bits, f64, row_rel_err
from paper_2508_16201_b200 import specvlm, synth

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("paged", [False, True])
def test_append_bit_exact_and_lengths(paged):
    L, H, D, n_new = 3, 4, 128, 6
    lens = [130, 64, 1]
    cache, k_host, v_host = make_cache(L, H, D, [n + n_new for n in lens], paged=paged, seed=50)
    cap = [n + n_new for n in lens]
    cache.seq_lens.copy_(torch.tensor(lens, dtype=torch.int32))
    new_k = synth.randn_bf16((L, 3, n_new, H, D), "cuda", 51, "nk")
    new_v = synth.randn_bf16((L, 3, n_new, H, D), "cuda", 51, "nv")
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    specvlm.append_kv(cache, new_k, new_v, d_status=status)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    assert cache.seq_lens.cpu().tolist() == cap
    gk = host_view(cache.k, cache.block_table, cap)
    gv = host_view(cache.v, cache.block_table, cap)
    for b in range(3):
        rk, n = oracle.append_kv(k_host[b], bits(new_k[:, b]), lens[b])
        rv, _ = oracle.append_kv(v_host[b], bits(new_v[:, b]), lens[b])
        assert n == cap[b] and np.array_equal(gk[b], rk) and np.array_equal(gv[b], rv)


def test_append_without_room_is_reported_and_changes_nothing():
    L, H, D = 1, 2, 64
    cache, k_host, _ = make_cache(L, H, D, [20, 20], paged=False, seed=52)
    cache.seq_lens.copy_(torch.tensor([20, 10], dtype=torch.int32))      # sequence 0 is full
    new = synth.randn_bf16((L, 2, 4, H, D), "cuda", 53, "n")
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    specvlm.append_kv(cache, new, new, d_status=status)
    torch.cuda.synchronize()
    assert int(status.item()) == specvlm.ERR_INVALID_ARG
    assert cache.seq_lens.cpu().tolist() == [20, 14]
    assert np.array_equal(host_view(cache.k, None, [20, 20])[0], k_host[0])


def test_rollback_lengths():
    lens = torch.tensor([100, 57, 9], dtype=torch.int32, device="cuda")
    acc = torch.tensor([5, 0, 3], dtype=torch.int32, device="cuda")
    specvlm.rollback_kv(lens, acc, 5)
    torch.cuda.synchronize()
    assert lens.cpu().tolist() == [oracle.rollback_len(100, 5, 5), oracle.rollback_len(57, 5, 0),
                                   oracle.rollback_len(9, 5, 3)]


def test_step_chain_append_verify_accept_rollback():
    L, Hq, Hkv, D, gamma, vocab = 2, 16, 2, 128, 4, 4099
    old = [300, 77]
    cap = [n + gamma + 1 for n in old]
    cache, k_host, v_host = make_cache(L, Hkv, D, cap, paged=True, seed=54)
    cache.seq_lens.copy_(torch.tensor(old, dtype=torch.int32))
    new_k = synth.randn_bf16((L, 2, gamma + 1, Hkv, D), "cuda", 55, "nk")
    new_v = synth.randn_bf16((L, 2, gamma + 1, Hkv, D), "cuda", 55, "nv")
    q = synth.randn_bf16((L, 2, gamma + 1, Hq, D), "cuda", 55, "q")
    logits, drafts = synth.logits_and_drafts(2, gamma, vocab, "cuda", 56)
    scale = 1.0 / math.sqrt(D)
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    specvlm.append_kv(cache, new_k, new_v, d_status=status)
    out = specvlm.verify_attn(cache, q, gamma, scale, d_status=status)
    n_acc, nxt, _ = specvlm.accept(logits, drafts)
    specvlm.rollback_kv(cache.seq_lens, n_acc, gamma, d_status=status)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    got = f64(out)
    for b in range(2):
        rk, n = oracle.append_kv(k_host[b], bits(new_k[:, b]), old[b])
        rv, _ = oracle.append_kv(v_host[b], bits(new_v[:, b]), old[b])
        for l in range(L):
            ref, _ = oracle.attention(bits(q[l, b]), rk[l], rv[l], n, scale)
            assert row_rel_err(got[l, b], ref) <= 1e-2
        a, nx, _ = oracle.accept(logits[b].cpu().numpy(), drafts[b].cpu().numpy())
        assert (int(n_acc[b]), int(nxt[b])) == (a, nx)
        assert int(cache.seq_lens[b]) == oracle.rollback_len(n, gamma, a)
