"""Device-side guards: what the kernels do with data they cannot trust.

The copy kernels turn device-resident integers (kept indices, block-table entries, tree-path
nodes, sequence lengths) into addresses.  Each guard is fed one value that is outside the range
the call's arguments declare but still inside the tensor the test allocated, so that no access
could leave the allocation even if a guard were missing.  Expected: the offending row is skipped
(its destination keeps the sentinel it held), every other row equals the oracle, and
SPECVLM_ERR_INVALID_ARG arrives in d_status.  The last test makes a bounded barrier wait run out
on a barrier nothing arrives at and reads SPECVLM_ERR_TIMEOUT back; the kernel returns normally."""
import numpy as np
import pytest
import torch

import oracle
from gpu_util import host_view, make_cache
from helpers import bits
from paper_2508_16201_b200 import specvlm, synth

pytestmark = pytest.mark.gpu


def _status():
    return torch.zeros(1, dtype=torch.int32, device="cuda")


def _shrunk(cache, n_blocks):
    """The same memory described as a cache of only n_blocks physical blocks."""
    return specvlm.KvCache(cache.k[:, :n_blocks], cache.v[:, :n_blocks], cache.seq_lens, cache.max_seq_len,
                           cache.block_table)


@pytest.mark.parametrize("bad", [-1, "video_len+2"])
def test_gather_skips_kept_index_outside_the_video(bad):
    L, H, D = 2, 2, 128
    vs, nv, nt = 4, 392, 40                       # 4 prefix tokens, so index -1 is still inside the tensor
    src_len = vs + nv + nt
    rng = np.random.default_rng(1)
    kept = np.sort(rng.choice(nv, 39, replace=False)).astype(np.int32)
    src, sk, sv = make_cache(L, H, D, [src_len], paged=False, seed=70)
    dst_len = src_len - nv + len(kept)
    dst, _, _ = make_cache(L, H, D, [dst_len], paged=False, seed=71)
    before = host_view(dst.k, None, [dst_len])[0].copy()
    corrupt = kept.copy()
    corrupt[17] = -1 if bad == -1 else nv + 2
    st = _status()
    specvlm.gather_kv(src, torch.from_numpy(corrupt).cuda(), [0, len(kept)], [vs], [nv], [src_len], dst, d_status=st)
    torch.cuda.synchronize()
    assert int(st.item()) == specvlm.ERR_INVALID_ARG
    ref = oracle.gather_kv(sk[0], kept, vs, nv, src_len)
    got = host_view(dst.k, None, [dst_len])[0]
    j = vs + 17                                   # destination position of the corrupted entry
    keep = np.ones(dst_len, dtype=bool)
    keep[j] = False
    assert np.array_equal(got[:, :, keep], ref[:, :, keep])
    assert np.array_equal(got[:, :, j], before[:, :, j])          # skipped: nothing written there


@pytest.mark.parametrize("side", ["src", "dst"])
def test_gather_skips_block_outside_the_declared_pool(side):
    L, H, D = 1, 2, 64
    nv, nt = 196, 60
    src_len = nv + nt
    kept = np.arange(0, nv, 10, dtype=np.int32)
    dst_len = nt + len(kept)
    src, sk, _ = make_cache(L, H, D, [src_len], paged=True, seed=72)
    dst, _, _ = make_cache(L, H, D, [dst_len], paged=True, seed=73)
    st = _status()
    c = src if side == "src" else dst
    top = int(c.block_table.max())                # the highest physical block in use ...
    small = _shrunk(c, top)                       # ... is outside a pool declared one block shorter
    before = host_view(dst.k, dst.block_table, [dst_len])[0].copy()
    specvlm.gather_kv(small if side == "src" else src, torch.from_numpy(kept).cuda(), [0, len(kept)], [0], [nv],
                      [src_len], small if side == "dst" else dst, d_status=st)
    torch.cuda.synchronize()
    assert int(st.item()) == specvlm.ERR_INVALID_ARG
    ref = oracle.gather_kv(sk[0], kept, 0, nv, src_len)
    got = host_view(dst.k, dst.block_table, [dst_len])[0]
    table = c.block_table.cpu().numpy()[0]
    lb = int(np.where(table == top)[0][0])        # logical block that maps to the refused one
    if side == "dst":
        bad_rows = np.arange(dst_len) // 64 == lb
    else:
        src_pos = np.concatenate([kept, np.arange(nv, src_len)])
        bad_rows = src_pos // 64 == lb
    assert bad_rows.any() and not bad_rows.all()
    assert np.array_equal(got[:, :, ~bad_rows], ref[:, :, ~bad_rows])
    assert np.array_equal(got[:, :, bad_rows], before[:, :, bad_rows])


def test_append_overflowing_sequence_writes_no_row_at_all():
    L, H, D, n_new = 2, 2, 64, 4
    cache, k_host, v_host = make_cache(L, H, D, [20, 20], paged=False, seed=74, extra_capacity=8)
    cache.seq_lens.copy_(torch.tensor([18, 10], dtype=torch.int32))     # 18 + 4 > 20: two rows would still fit
    new = synth.randn_bf16((L, 2, n_new, H, D), "cuda", 75, "n")
    st = _status()
    specvlm.append_kv(cache, new, new, d_status=st)
    torch.cuda.synchronize()
    assert int(st.item()) == specvlm.ERR_INVALID_ARG
    assert cache.seq_lens.cpu().tolist() == [18, 14]
    got = host_view(cache.k, None, [20, 20])
    assert np.array_equal(got[0], k_host[0])                              # rows 18, 19 included
    rk, n = oracle.append_kv(k_host[1][:, :, :14].copy(), bits(new[:, 1]), 10)
    assert n == 14 and np.array_equal(got[1][:, :, :14], rk[:, :, :14])


def test_append_skips_block_outside_the_declared_pool():
    L, H, D, n_new = 1, 2, 64, 3
    lens = [62]                                   # the new rows 62, 63 | 64 straddle two pages
    cache, k_host, _ = make_cache(L, H, D, [lens[0] + n_new], paged=True, seed=76)
    cache.seq_lens.copy_(torch.tensor(lens, dtype=torch.int32))
    table = cache.block_table.cpu().numpy()[0]
    second = int(table[1])
    if second < int(table[0]):                    # make the second page the one outside the pool
        pytest.skip("page order of this seed puts the first page last")
    small = _shrunk(cache, second)
    new = synth.randn_bf16((L, 1, n_new, H, D), "cuda", 77, "n")
    st = _status()
    specvlm.append_kv(small, new, new, d_status=st)
    torch.cuda.synchronize()
    assert int(st.item()) == specvlm.ERR_INVALID_ARG
    got = host_view(cache.k, cache.block_table, [lens[0] + n_new])[0]
    nb = bits(new[:, 0])                          # [L][n_new][H][D]
    assert np.array_equal(got[:, :, 62], nb[:, 0]) and np.array_equal(got[:, :, 63], nb[:, 1])
    assert np.array_equal(got[:, :, 64], k_host[0][:, :, 64])             # the refused page is untouched


@pytest.mark.parametrize("bad_node", [0, "n_nodes"])
def test_compact_tree_skips_path_node_outside_the_window(bad_node):
    L, H, D, n_nodes = 2, 2, 128, 8
    old = 100
    cache, k_host, _ = make_cache(L, H, D, [old + n_nodes], paged=False, seed=78, extra_capacity=16)
    path_ok = [2, 5, 7] + [-1] * (n_nodes - 3)
    path = list(path_ok)
    path[1] = 0 if bad_node == 0 else n_nodes     # position old + n_nodes is inside the spare capacity
    st = _status()
    acc = torch.tensor([3], dtype=torch.int32, device="cuda")
    specvlm.compact_tree_kv(cache, torch.tensor([path], dtype=torch.int32, device="cuda"), acc, d_status=st)
    torch.cuda.synchronize()
    assert int(st.item()) == specvlm.ERR_INVALID_ARG
    ref, n = oracle.compact_tree_kv(k_host[0].copy(), old + n_nodes, n_nodes, path_ok[:3])
    assert int(cache.seq_lens[0]) == n
    got = host_view(cache.k, None, [old + n_nodes])[0]
    rows = np.ones(old + n_nodes, dtype=bool)
    rows[old + 2] = False                         # the destination of the refused move
    rows[n:] = False                              # past the new end nothing is specified
    assert np.array_equal(got[:, :, rows], ref[:, :, rows])
    assert np.array_equal(got[:, :, old + 2], k_host[0][:, :, old + 2])


def test_bounded_wait_runs_out_and_reports_timeout():
    st = _status()
    flag = torch.zeros(1, dtype=torch.int32, device="cuda")
    t0, t1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    t0.record()
    specvlm.debug_wait_timeout(5, st, flag)
    t1.record()
    torch.cuda.synchronize()                      # returns: the kernel gave up by itself
    assert int(st.item()) == specvlm.ERR_TIMEOUT and int(flag.item()) == 1
    assert "timed out" in specvlm.status_string(int(st.item()))
    ms = t0.elapsed_time(t1)
    assert 4.0 <= ms <= 500.0, ms
    # the context is intact: an ordinary call still works afterwards
    logits, drafts = synth.logits_and_drafts(1, 2, 1024, "cuda", 9)
    n, nxt, _ = specvlm.accept(logits, drafts)
    a, nx, _ = oracle.accept(logits[0].cpu().numpy(), drafts[0].cpu().numpy())
    assert (int(n[0]), int(nxt[0])) == (a, nx)
