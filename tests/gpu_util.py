"""Builders used by the GPU parity tests: synthetic caches in the library's layout and their
de-paged host copies for the oracle."""
import numpy as np
import torch

from paper_2508_16201_b200 import specvlm, synth
from helpers import bits


def make_cache(n_layers, n_kv_heads, head_dim, seq_lens, *, paged, seed, device="cuda", page=64,
               poison_tail=False, extra_capacity=0):
    """Random bf16 N(0,1) cache holding len(seq_lens) sequences.

    Returns (KvCache, k_host, v_host) where k_host[b] is the uint16 array
    [n_layers][n_kv_heads][seq_lens[b]][head_dim] of sequence b for the oracle.
    poison_tail fills every slot past a sequence's end with NaN to check that stale memory
    never reaches an output.
    """
    B = len(seq_lens)
    max_len = max(seq_lens)
    if paged:
        need = [(n + page - 1) // page for n in seq_lens]
        pool = sum(need) + 3
        max_blocks = max(need) + 1
        table = synth.page_table(B, max_blocks, pool, need, seed, device)
        shape = (n_layers, pool, n_kv_heads, page, head_dim)
    else:
        cap = max_len + extra_capacity
        table = None
        shape = (n_layers, B, n_kv_heads, cap, head_dim)
    k = synth.randn_bf16(shape, device, seed, "K")
    v = synth.randn_bf16(shape, device, seed, "V")
    lens = torch.tensor(seq_lens, dtype=torch.int32, device=device)
    if poison_tail:
        bt = shape[3]
        for b, n in enumerate(seq_lens):
            if paged:
                for lb in range(max_blocks):
                    blk = int(table[b, lb])
                    if blk < 0:
                        continue
                    lo = max(0, n - lb * page)
                    if lo < page:
                        k[:, blk, :, lo:, :] = float("nan")
                        v[:, blk, :, lo:, :] = float("nan")
            else:
                k[:, b, :, n:, :] = float("nan")
                v[:, b, :, n:, :] = float("nan")
        if paged:   # unused pool blocks too
            used = set(int(x) for x in table.flatten().tolist() if x >= 0)
            for blk in range(pool):
                if blk not in used:
                    k[:, blk] = float("nan")
                    v[:, blk] = float("nan")
    cache = specvlm.KvCache(k, v, lens, max_len, table)
    return cache, host_view(k, table, seq_lens), host_view(v, table, seq_lens)


def host_view(t, table, seq_lens):
    """De-page: list over sequences of uint16 [L][H][len][D]."""
    out = []
    L, NB, H, BT, D = t.shape
    tc = t.cpu()
    tab = table.cpu() if table is not None else None
    for b, n in enumerate(seq_lens):
        if tab is None:
            seq = tc[:, b, :, :n, :]
        else:
            nb = (n + BT - 1) // BT
            blocks = tab[b, :nb].long()
            seq = tc[:, blocks].permute(0, 2, 1, 3, 4).reshape(L, H, nb * BT, D)[:, :, :n, :]
        out.append(bits(seq.contiguous()))
    return out
