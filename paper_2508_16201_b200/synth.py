"""Seeded synthetic inputs for the five workload shapes.

This module holds NONE of the method's arithmetic: it only draws tensors (bf16 N(0,1)
caches and queries, planted salient keys, logits, draft tokens, page tables).  Both the
tests' oracle side and the CUDA side are fed the same tensors produced here.

All draws come from ``torch.Generator`` objects seeded from (seed, tensor tag, layer), so a
single layer can be regenerated on demand.  The bits depend on the device type; a test
always hands the very same tensor (copied to the host) to both sides.
"""
from __future__ import annotations

import dataclasses
import zlib

import torch


@dataclasses.dataclass(frozen=True)
class Workload:
    name: str
    # verifier (target) and draft attention shapes
    t_layers: int
    t_q_heads: int
    t_kv_heads: int
    d_layers: int
    d_q_heads: int
    d_kv_heads: int
    head_dim: int
    # video / text structure, one entry per sequence
    n_frames: tuple
    tokens_per_frame: int
    n_text: tuple
    retention_permille: int
    gamma: int
    vocab: int
    planted_permille: int
    paged: bool = False
    page_tokens: int = 64

    @property
    def batch(self) -> int:
        return len(self.n_frames)

    def n_video(self, b: int = 0) -> int:
        return self.n_frames[b] * self.tokens_per_frame

    def seq_len(self, b: int = 0) -> int:
        return self.n_video(b) + self.n_text[b]

    def k_total(self, b: int = 0) -> int:
        return (self.n_video(b) * self.retention_permille) // 1000

    def k_stage1(self, b: int = 0) -> int:
        return self.k_total(b) // 2


def _seed(seed: int, *tags) -> int:
    s = ("%d|" % seed) + "|".join(str(t) for t in tags)
    return (zlib.crc32(s.encode()) << 20) ^ seed ^ 0x5DEECE66D


def _gen(device, seed: int, *tags) -> torch.Generator:
    g = torch.Generator(device=device)
    g.manual_seed(_seed(seed, *tags) & ((1 << 62) - 1))
    return g


def workload(i: int, *, retention_permille: int | None = None, gamma: int | None = None,
             seed: int = 0) -> Workload:
    """The five workload shapes (1-based, as listed in the benchmark description)."""
    if i == 1:
        w = Workload("cfg1-tiny", 1, 8, 2, 1, 4, 1, 64, (4,), 196, (64,), 100, 4, 1024, 50)
    elif i == 2:
        w = Workload("cfg2-llava-ov-72b-7b", 80, 64, 8, 28, 28, 4, 128, (32,), 196, (128,), 100, 5,
                     152064, 50)
    elif i == 3:
        w = Workload("cfg3-qwen25vl-32b-7b", 64, 40, 8, 28, 28, 4, 128, (32,), 720, (256,), 100, 5,
                     152064, 50)
    elif i == 4:
        w = Workload("cfg4-long-video", 80, 64, 8, 28, 28, 4, 128, (256,), 196, (128,), 100, 6,
                     152064, 30)
    elif i == 5:
        g = _gen("cpu", seed, "cfg5-shapes")
        frames = (torch.randint(1, 5, (16,), generator=g) * 32).tolist()
        text = torch.randint(64, 257, (16,), generator=g).tolist()
        w = Workload("cfg5-batched-paged", 80, 64, 8, 28, 28, 4, 128, tuple(frames), 196,
                     tuple(text), 100, 5, 152064, 50, paged=True)
    else:
        raise ValueError("workload index must be 1..5")
    if retention_permille is not None:
        w = dataclasses.replace(w, retention_permille=retention_permille)
    if gamma is not None:
        w = dataclasses.replace(w, gamma=gamma)
    return w


def randn_bf16(shape, device, seed: int, *tags) -> torch.Tensor:
    g = _gen(device, seed, *tags)
    return torch.randn(shape, generator=g, device=device, dtype=torch.float32).to(torch.bfloat16)


def salient_set(n_video: int, planted_permille: int, seed: int, b: int = 0) -> torch.Tensor:
    """Indices (sorted, int64, CPU) of the planted salient video tokens of sequence b."""
    g = _gen("cpu", seed, "salient", b)
    n = (n_video * planted_permille) // 1000
    return torch.randperm(n_video, generator=g)[:n].sort().values


def plant_salient_(k_video: torch.Tensor, q_text: torch.Tensor, salient: torch.Tensor,
                   strength: float = 2.0) -> None:
    """In place: K[l, g, j, :] += strength * u[l, g] for j in the salient set, where u is the
    unit-normalised mean of the text queries of the heads in KV group g.

    k_video: bf16 [L][Hkv][n_video][d] (a view of the cache's video rows)
    q_text:  bf16 [L][n_text][Hq][d]
    """
    L, n_text, Hq, d = q_text.shape
    Hkv = k_video.shape[1]
    u = q_text.float().view(L, n_text, Hkv, Hq // Hkv, d).mean(dim=(1, 3))      # [L][Hkv][d]
    u = u / u.norm(dim=-1, keepdim=True).clamp_min(1e-20)
    idx = salient.to(k_video.device)
    rows = k_video[:, :, idx, :].float() + strength * u[:, :, None, :]
    k_video[:, :, idx, :] = rows.to(torch.bfloat16)


def plant_salient_paged_(k_pool: torch.Tensor, block_table_row: torch.Tensor, video_start: int, n_video: int,
                         q_text: torch.Tensor, salient: torch.Tensor, strength: float = 2.0) -> None:
    """plant_salient_ for one sequence of a paged cache: k_pool bf16 [L][n_blocks][Hkv][page][d],
    block_table_row int32 [max_blocks] of that sequence; the video occupies positions
    video_start .. video_start + n_video - 1."""
    page = k_pool.shape[3]
    pos = torch.arange(video_start, video_start + n_video, device=k_pool.device)
    blk = block_table_row.to(k_pool.device)[pos // page].long()
    off = pos % page
    rows = k_pool[:, blk, :, off, :].permute(1, 2, 0, 3).contiguous()          # [L][Hkv][n_video][d]
    plant_salient_(rows, q_text, salient, strength)
    k_pool[:, blk, :, off, :] = rows.permute(2, 0, 1, 3)


def page_table(batch: int, max_blocks: int, n_pool_blocks: int, blocks_needed, seed: int,
               device) -> torch.Tensor:
    """Scattered block table [batch][max_blocks] (int32): a seeded permutation of the pool;
    unused entries are -1."""
    g = _gen("cpu", seed, "pages")
    perm = torch.randperm(n_pool_blocks, generator=g).to(torch.int32)
    table = torch.full((batch, max_blocks), -1, dtype=torch.int32)
    pos = 0
    for b in range(batch):
        nb = int(blocks_needed[b])
        table[b, :nb] = perm[pos:pos + nb]
        pos += nb
    assert pos <= n_pool_blocks
    return table.to(device)


def logits_and_drafts(batch: int, gamma: int, vocab: int, device, seed: int):
    """fp32 N(0,1) target logits [B][gamma+1][vocab]; draft tokens [B][gamma] equal to the
    row maximum's index with probability 1/2, else uniform random."""
    g = _gen(device, seed, "logits")
    logits = torch.randn((batch, gamma + 1, vocab), generator=g, device=device, dtype=torch.float32)
    gc = _gen("cpu", seed, "drafts")
    # torch.argmax returns SOME maximal index; exact ties have probability ~0 in N(0,1) draws
    # and the drafts are only inputs, so this does not pre-empt the method's tie rule.
    top = logits[:, :gamma, :].argmax(dim=-1).cpu()
    coin = torch.rand((batch, gamma), generator=gc) < 0.5
    rnd = torch.randint(0, vocab, (batch, gamma), generator=gc)
    drafts = torch.where(coin, top, rnd).to(torch.int32)
    return logits, drafts.to(device)
