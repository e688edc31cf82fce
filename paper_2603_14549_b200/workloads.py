"""Seeded synthetic inputs for the ASAP prune step.

This module only *draws inputs*: packed token spans, post-RoPE Q/K, hidden states
and position ids with the shapes of LLaVA-1.5 / LLaVA-NeXT prefill at the pruning
layer.  It contains none of the method's arithmetic (no attention mass, salience,
mask, softmax, top-k, similarity or merge), so both the CUDA path and the CPU
oracle may consume what it produces.

Layout of one batch (all tensors on the CPU, the caller moves them):

    packed rows   sample b owns rows cu_seqlens[b] .. cu_seqlens[b+1]
    one sample    [ system (S rows) | visual (N_v rows) | text (T_b rows) ]
    q, k          bf16 [total, H, head_dim]   rotary embedding already applied
    hidden        bf16 [total, D]             D = H * head_dim
    pos_ids       int32 [total]               0 .. N_b-1 inside each sample

Recipe (stated so the batch can be re-created anywhere from the seed alone):
Q/K entries are iid N(0,1) drawn in fp32, rotated in fp64 with the half-split
pairing (x_i, x_{i+d/2}), theta_i = 10000^(-2i/d), at the token's position id,
then rounded to bf16.  System/text hidden rows are iid N(0,1).  Visual hidden
rows are a cluster centre c ~ N(0, I_D), chosen uniformly per token, plus
N(0, 0.3^2) noise; optionally the centres are local to 576-token tiles and a
fraction of tokens is scaled to 10x norm.  Every sample has its own generator
seeded by (seed, sample index) so samples can be drawn independently.
"""
from __future__ import annotations

import dataclasses
import math
from typing import List, Optional, Sequence

import torch

SYSTEM_LEN = 35
BASE_SEED = 20260314


@dataclasses.dataclass
class Batch:
    name: str
    B: int
    H: int
    head_dim: int
    D: int
    keep_k: int
    cu_seqlens: torch.Tensor   # int32 [B+1]
    vis_start: torch.Tensor    # int32 [B] sequence-relative
    vis_len: torch.Tensor      # int32 [B]
    text_start: torch.Tensor   # int32 [B]
    text_len: torch.Tensor     # int32 [B]
    q: torch.Tensor            # bf16 [total, H, head_dim]
    k: torch.Tensor            # bf16 [total, H, head_dim]
    hidden: torch.Tensor       # bf16 [total, D]
    pos_ids: torch.Tensor      # int32 [total]
    seed: int = 0

    @property
    def total(self) -> int:
        return int(self.cu_seqlens[-1])

    def sample_rows(self, b: int) -> slice:
        return slice(int(self.cu_seqlens[b]), int(self.cu_seqlens[b + 1]))


def _sample_generator(seed: int, b: int, stream: int = 0) -> torch.Generator:
    g = torch.Generator(device="cpu")
    g.manual_seed((seed * 1000003 + b * 7919 + stream * 104729) % (2 ** 63 - 1))
    return g


def rope_rotate(x: torch.Tensor, pos: torch.Tensor, theta: float = 10000.0) -> torch.Tensor:
    """Rotary embedding, half-split pairing, in fp64.  x: [n, H, d] fp64, pos: [n] integer."""
    n, H, d = x.shape
    half = d // 2
    inv_freq = theta ** (-torch.arange(0, half, dtype=torch.float64) * 2.0 / d)   # [d/2]
    ang = pos.to(torch.float64)[:, None] * inv_freq[None, :]                      # [n, d/2]
    cos = torch.cos(ang)[:, None, :]
    sin = torch.sin(ang)[:, None, :]
    x1, x2 = x[..., :half], x[..., half:]
    return torch.cat([x1 * cos - x2 * sin, x2 * cos + x1 * sin], dim=-1)


def draw_qk(pos: torch.Tensor, H: int, head_dim: int, gen: torch.Generator):
    """N(0,1) Q and K of shape [len(pos), H, head_dim], rotated at `pos`, rounded to bf16."""
    n = pos.numel()
    out = []
    for _ in range(2):
        raw = torch.randn(n, H, head_dim, generator=gen, dtype=torch.float32).to(torch.float64)
        out.append(rope_rotate(raw, pos).to(torch.bfloat16))
    return out[0], out[1]


def draw_visual_hidden(n_vis: int, D: int, gen: torch.Generator, n_centres: int,
                       sigma: float = 0.3, tile: Optional[int] = None,
                       outlier_frac: float = 0.0, outlier_scale: float = 10.0) -> torch.Tensor:
    """Clustered visual hidden states [n_vis, D] in bf16.

    tile=None: one pool of `n_centres` centres for the whole span.
    tile=T:    every block of T consecutive tokens has its own `n_centres` centres.
    """
    rows = torch.empty(n_vis, D, dtype=torch.float32)
    step = n_vis if tile is None else tile
    for lo in range(0, n_vis, step):
        hi = min(lo + step, n_vis)
        centres = torch.randn(n_centres, D, generator=gen, dtype=torch.float32)
        pick = torch.randint(0, n_centres, (hi - lo,), generator=gen)
        noise = torch.randn(hi - lo, D, generator=gen, dtype=torch.float32) * sigma
        rows[lo:hi] = centres[pick] + noise
    if outlier_frac > 0.0:
        n_out = max(1, int(round(outlier_frac * n_vis)))
        who = torch.randperm(n_vis, generator=gen)[:n_out]
        rows[who] *= outlier_scale
    return rows.to(torch.bfloat16)


def make_batch(name: str, B: int, n_vis: int, text_lens: Sequence[int], H: int, head_dim: int,
               keep_k: int, seed: int, centres: Sequence[int], sigma: float = 0.3,
               tile: Optional[int] = None, outlier_frac: float = 0.0,
               system_len: int = SYSTEM_LEN) -> Batch:
    D = H * head_dim
    assert len(text_lens) == B and len(centres) == B
    seq_lens = [system_len + n_vis + int(t) for t in text_lens]
    cu = torch.zeros(B + 1, dtype=torch.int32)
    cu[1:] = torch.cumsum(torch.tensor(seq_lens, dtype=torch.int64), 0).to(torch.int32)
    total = int(cu[-1])
    q = torch.empty(total, H, head_dim, dtype=torch.bfloat16)
    k = torch.empty(total, H, head_dim, dtype=torch.bfloat16)
    hidden = torch.empty(total, D, dtype=torch.bfloat16)
    pos_ids = torch.empty(total, dtype=torch.int32)
    for b in range(B):
        g = _sample_generator(seed, b)
        lo, n = int(cu[b]), seq_lens[b]
        pos = torch.arange(n, dtype=torch.int64)
        pos_ids[lo:lo + n] = pos.to(torch.int32)
        qb, kb = draw_qk(pos, H, head_dim, g)
        q[lo:lo + n], k[lo:lo + n] = qb, kb
        hb = torch.randn(n, D, generator=g, dtype=torch.float32).to(torch.bfloat16)
        hb[system_len:system_len + n_vis] = draw_visual_hidden(
            n_vis, D, g, int(centres[b]), sigma, tile, outlier_frac)
        hidden[lo:lo + n] = hb
    i32 = lambda v: torch.tensor(v, dtype=torch.int32)
    return Batch(name=name, B=B, H=H, head_dim=head_dim, D=D, keep_k=keep_k, cu_seqlens=cu,
                 vis_start=i32([system_len] * B), vis_len=i32([n_vis] * B),
                 text_start=i32([system_len + n_vis] * B), text_len=i32([int(t) for t in text_lens]),
                 q=q, k=k, hidden=hidden, pos_ids=pos_ids, seed=seed)


def _ragged(B: int, lo: int, hi: int, seed: int) -> List[int]:
    g = _sample_generator(seed, 0, stream=1)
    return [int(v) for v in torch.randint(lo, hi + 1, (B,), generator=g)]


def config(name: str, B: Optional[int] = None, seed: Optional[int] = None,
           keep_k: Optional[int] = None) -> Batch:
    """The benchmark shapes (c1-c5: LLaVA-1.5 / LLaVA-NeXT; c6: InternVL-2.5-shaped).  `B` may be lowered (never raised) to draw a prefix
    of the batch: sample b is identical whatever B is, because each sample has its own
    generator and the ragged text lengths are drawn for the full batch first."""
    name = name.lower()
    idx = {"c1": 0, "c2": 1, "c3": 2, "c4": 3, "c5": 4, "c6": 5}[name]
    seed = BASE_SEED + idx if seed is None else seed
    if name == "c1":      # LLaVA-1.5-7B single step
        fullB, nv, H, k = 1, 576, 32, 192
        texts, cents, tile, out = [32], [64], None, 0.0
    elif name == "c2":    # LLaVA-1.5-7B batched, ragged text
        fullB, nv, H, k = 16, 576, 32, 64
        texts = _ragged(fullB, 16, 128, seed)
        g = _sample_generator(seed, 0, stream=2)
        cents = [int(v) for v in torch.randint(32, 129, (fullB,), generator=g)]
        tile, out = None, 0.0
    elif name == "c3":    # LLaVA-NeXT-7B, 4 tiles
        fullB, nv, H, k = 8, 2304, 32, 320
        texts, cents, tile, out = [64] * fullB, [48] * fullB, 576, 0.02
    elif name == "c4":    # LLaVA-NeXT AnyRes max resolution, 5 tiles
        fullB, nv, H, k = 64, 2880, 32, 576
        texts, cents, tile, out = _ragged(fullB, 32, 256, seed), [64] * fullB, None, 0.0
    elif name == "c6":    # InternVL-2.5-8B-shaped: six 448 x 448 tiles of 256 tokens, budget ~510 (Sec. 5.4)
        fullB, nv, H, k = 8, 1536, 32, 510
        texts, cents, tile, out = [64] * fullB, [32] * fullB, 256, 0.0
    else:                 # c5: 13B-shaped, progressive
        fullB, nv, H, k = 32, 2304, 40, 1152
        texts, cents, tile, out = [128] * fullB, [48] * fullB, 576, 0.0
    useB = fullB if B is None else min(B, fullB)
    return make_batch(name, useB, nv, texts[:useB], H, 128, k if keep_k is None else keep_k,
                      seed, cents[:useB], 0.3, tile, out)


def draw_values(batch: "Batch", seed: int) -> torch.Tensor:
    """Value projections for the layer's attention: iid N(0, 1), bf16 [total, H, head_dim], one seeded
    stream per sequence (sequence b is the same whatever the batch prefix)."""
    v = torch.empty(batch.total, batch.H, batch.head_dim, dtype=torch.bfloat16)
    for b in range(batch.B):
        rows = batch.sample_rows(b)
        g = _sample_generator(seed, b, stream=30)
        v[rows] = torch.randn(rows.stop - rows.start, batch.H, batch.head_dim, generator=g).to(torch.bfloat16)
    return v


def random_stage1(batch: "Batch", b: int, keep_k: int, seed: int):
    """Stand-in for stage 1's results of sequence b, for exercising stage 2 alone at sizes where the
    CPU oracle cannot afford stage 1: attention mass (positive, long-tailed), salience (uniform in
    [0, 1], one exact 0 and one exact 1), a random kept subset and its complement, all seeded.
    Returns (mass f32 [nv], salience f32 [nv], keep int32 [k] ascending, drop int32 [nv-k] ascending)."""
    g = _sample_generator(seed, b, stream=20)
    nv = int(batch.vis_len[b])
    mass = torch.exp(torch.randn(nv, generator=g)).float()
    sal = torch.rand(nv, generator=g).float()
    sal[int(torch.randint(0, nv, (1,), generator=g))] = 0.0
    sal[int(torch.randint(0, nv, (1,), generator=g))] = 1.0
    perm = torch.randperm(nv, generator=g)
    keep = torch.sort(perm[:keep_k]).values.to(torch.int32)
    drop = torch.sort(perm[keep_k:]).values.to(torch.int32)
    return mass.numpy(), sal.numpy(), keep.numpy(), drop.numpy()


C5_SCHEDULE = (1152, 576, 288)


def redraw_qk(batch_pos_ids: torch.Tensor, cu_seqlens: torch.Tensor, H: int, head_dim: int,
              seed: int, step: int):
    """Fresh N(0,1) Q/K for a later prune step of the progressive schedule, rotated at the
    surviving tokens' (gathered) position ids."""
    total = int(cu_seqlens[-1])
    q = torch.empty(total, H, head_dim, dtype=torch.bfloat16)
    k = torch.empty(total, H, head_dim, dtype=torch.bfloat16)
    for b in range(cu_seqlens.numel() - 1):
        lo, hi = int(cu_seqlens[b]), int(cu_seqlens[b + 1])
        g = _sample_generator(seed, b, stream=10 + step)
        q[lo:hi], k[lo:hi] = draw_qk(batch_pos_ids[lo:hi].to(torch.int64), H, head_dim, g)
    return q, k


def tiny(B: int, n_vis: Sequence[int], text_lens: Sequence[int], H: int, keep_k: int, seed: int,
         system_len: int = 3, centres: int = 4, head_dim: int = 128) -> Batch:
    """Small ragged batches (per-sample visual lengths) for edge-case tests."""
    assert len(n_vis) == B and len(text_lens) == B
    parts = [make_batch("tiny", 1, int(n_vis[b]), [int(text_lens[b])], H, head_dim, keep_k,
                        seed + 31 * b, [centres], system_len=system_len) for b in range(B)]
    cu = torch.zeros(B + 1, dtype=torch.int32)
    cu[1:] = torch.cumsum(torch.tensor([p.total for p in parts]), 0).to(torch.int32)
    cat = lambda f: torch.cat([getattr(p, f) for p in parts], 0)
    return Batch(name="tiny", B=B, H=H, head_dim=head_dim, D=H * head_dim, keep_k=keep_k,
                 cu_seqlens=cu, vis_start=cat("vis_start"), vis_len=cat("vis_len"),
                 text_start=cat("text_start"), text_len=cat("text_len"), q=cat("q"), k=cat("k"),
                 hidden=cat("hidden"), pos_ids=cat("pos_ids"), seed=seed)
