"""Sharding the Prox FFN along d_ff across ranks (one process per GPU): host logic.

The paper's method is single-GPU (Sec. 4.3); this is the natural split of it.  Rank p holds the
channels F_p = [p * F / P, (p + 1) * F / P) of both proxies, of W_gate / W_up, and the matching
columns of W_down.  Proxy quantization is per channel, so a shard's proxy scores are the full
layer's scores of its channels.  Per call (batch 1):

  1. Stage 1 locally: the shard's proxy scores |u~ SiLU(g~)| (Sec. 4.1 Stage 1).
  2. The channel mask is the GLOBAL top-k2 (a per-rank top-(k2 / P) would be another method):
     every rank bins its scores by the top 11 bits of the fp32 pattern (2048 bins), the bins are
     summed over the ranks (one small all-reduce), every rank finds the bin that holds the k2-th
     score, the candidates of that bin (score bits, global channel) are all-gathered and ranked
     (larger score first, equal scores by lower global channel), which gives the exact cut; each
     rank keeps its channels above the cut.
  3. Stage 2 locally on the kept channels of the shard (Sec. 4.1 Stage 2), partial y.
  4. all-reduce(sum) of y (d_model fp32 values).

The collectives are torch.distributed calls on the caller's process group (NCCL on GPUs, gloo
on CPU ranks); no rank reads another rank's memory.  The shard-local work is behind two
callables so that the same exchange runs over the CUDA library (ShardedProxFFN) and, in the
CPU tests, over any other implementation of the two stages."""
from __future__ import annotations

from typing import Callable, Optional, Tuple

import torch
import torch.distributed as dist

BINS_SHIFT = 20          # fp32 pattern >> 20: sign (0 for scores) + exponent + 3 mantissa bits = 2048 bins
N_BINS = 2048


def shard_range(d_ff: int, world: int, rank: int) -> Tuple[int, int]:
    """Channels [lo, hi) of rank `rank`; d_ff must divide evenly."""
    if d_ff % world:
        raise ValueError("d_ff must be a multiple of the number of ranks")
    per = d_ff // world
    return rank * per, (rank + 1) * per


def global_topk_mask(local_scores: torch.Tensor, k2: int, lo: int, group=None) -> torch.Tensor:
    """Local channel ids (ascending, int64) of this shard that belong to the global top-k2 of the scores of all
    shards; equal scores are taken in order of increasing GLOBAL channel id.  local_scores: fp32 [F_p], >= 0."""
    world = dist.get_world_size(group) if dist.is_initialized() else 1
    keys = local_scores.contiguous().view(torch.int32).to(torch.int64)        # monotone for non-negative floats
    bins = keys >> BINS_SHIFT
    hist = torch.bincount(bins, minlength=N_BINS)
    if world > 1:
        dist.all_reduce(hist, op=dist.ReduceOp.SUM, group=group)
    total = int(hist.sum())
    if not 1 <= k2 <= total:
        raise ValueError("k2 out of range")
    # from the top: the bin where the running count reaches k2
    from_top = torch.flip(torch.cumsum(torch.flip(hist, [0]), 0), [0])        # from_top[b] = scores in bins >= b
    b_star = int(torch.nonzero(from_top >= k2).max())
    above = int(from_top[b_star + 1]) if b_star + 1 < N_BINS else 0
    need = k2 - above                                                         # how many of bin b_star are kept
    cand = torch.nonzero(bins == b_star).flatten()
    pairs = torch.stack([keys[cand], cand + lo], dim=1)                       # (score bits, global channel)
    if world > 1:
        n_local = torch.tensor([pairs.shape[0]], dtype=torch.int64, device=pairs.device)
        counts = [torch.zeros_like(n_local) for _ in range(world)]
        dist.all_gather(counts, n_local, group=group)
        n_max = int(max(int(c) for c in counts))
        padded = torch.full((n_max, 2), -1, dtype=torch.int64, device=pairs.device)
        padded[:pairs.shape[0]] = pairs
        gathered = [torch.empty_like(padded) for _ in range(world)]
        dist.all_gather(gathered, padded, group=group)
        allp = torch.cat([g[:int(c)] for g, c in zip(gathered, counts)], dim=0)
    else:
        allp = pairs
    # rank the bin's candidates: score descending, then global channel ascending
    order = torch.argsort(allp[:, 1], stable=True)
    allp = allp[order]
    order = torch.argsort(allp[:, 0], descending=True, stable=True)
    allp = allp[order]
    cut_key, cut_ch = int(allp[need - 1, 0]), int(allp[need - 1, 1])
    gch = torch.arange(keys.shape[0], device=keys.device, dtype=torch.int64) + lo
    keep = (bins > b_star) | ((bins == b_star) & ((keys > cut_key) | ((keys == cut_key) & (gch <= cut_ch))))
    return torch.nonzero(keep).flatten()


def sharded_forward(stage1_scores: Callable[[torch.Tensor], torch.Tensor],
                    stage2_partial: Callable[[torch.Tensor, torch.Tensor], torch.Tensor],
                    x: torch.Tensor, k2: int, lo: int, group=None):
    """One call of the sharded FFN on this rank.  stage1_scores(x) -> fp32 [F_p] scores of the shard;
    stage2_partial(x, local_sel) -> fp32 [d_model] partial output over the shard's kept channels (zeros if none).
    Returns (local_sel, y) with y the full output (identical on every rank)."""
    scores = stage1_scores(x)
    sel = global_topk_mask(scores, k2, lo, group)
    y = stage2_partial(x, sel).to(torch.float32).contiguous()
    if dist.is_initialized() and dist.get_world_size(group) > 1:
        dist.all_reduce(y, op=dist.ReduceOp.SUM, group=group)
    return sel, y


class ShardedProxFFN:
    """The shard of one layer on this rank's GPU, over the CUDA library: a library handle on the shard's slices
    of the weights (d_ff / world channels).  w_gate, w_up: dev bf16 [F, D] or already the shard's rows;
    w_down: dev bf16 [D, F] or the shard's columns."""

    def __init__(self, d_model: int, d_ff: int, w_gate, w_up, w_down, bits: int = 4, group_size: int = 128,
                 group=None):
        from . import binding as pb                     # fails loudly without the CUDA library
        self.pb, self.group = pb, group
        self.rank = dist.get_rank(group) if dist.is_initialized() else 0
        self.world = dist.get_world_size(group) if dist.is_initialized() else 1
        self.lo, self.hi = shard_range(d_ff, self.world, self.rank)
        self.D, self.Fp = d_model, self.hi - self.lo
        if w_gate.shape[0] == d_ff and self.world > 1:
            w_gate, w_up, w_down = w_gate[self.lo:self.hi], w_up[self.lo:self.hi], w_down[:, self.lo:self.hi]
        self.w = (w_gate.contiguous(), w_up.contiguous(), w_down.contiguous())     # the handle reads these buffers
        self.h = pb.prox_ffn_create(d_model, self.Fp, 1, 1, *self.w)               # fp32 partial outputs
        pb.prox_quantize_proxy(self.h, bits, group_size)
        dev = self.w[0].device
        self.scores = torch.empty(self.Fp, dtype=torch.float32, device=dev)
        self.sel1 = torch.empty(1, 1, dtype=torch.int32, device=dev)
        self.y = torch.empty(d_model, dtype=torch.float32, device=dev)

    def forward(self, x, k1: int, k2: int, stream=None):
        pb = self.pb

        def s1(xv):
            pb.prox_stage1_mask(self.h, xv, 1, k1, 1, self.sel1, self.scores, stream)
            return self.scores

        def s2(xv, sel):
            if sel.numel() == 0:
                return torch.zeros_like(self.y)
            sel32 = sel.to(torch.int32).contiguous()
            pb.prox_stage2_ffn(self.h, xv, 1, sel32, int(sel32.numel()), self.y, stream)
            return self.y

        return sharded_forward(s1, s2, x, k2, self.lo, self.group)

    def close(self):
        if self.h:
            self.pb.prox_ffn_destroy(self.h)
            self.h = None
